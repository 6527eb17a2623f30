// az_tower_static: encoder + convolution tower for callers that must not trigger any device
// allocation.  The only scratch this step needs besides the network's weights is the encoded
// plane tensor between the encoder kernel and the tower kernel; here it lives in a fixed
// device-resident array instead of a buffer obtained from the allocator.
#include "common.cuh"

#include <mutex>

namespace az {
namespace {

constexpr int kStaticMaxBatch = 256;
constexpr size_t kStaticPlaneBytes = (size_t)kStaticMaxBatch * 64 * 32 * sizeof(__nv_bfloat16);   // 1 MiB

// Held by every GPU that loads the library, from load until the process exits.
static __device__ __align__(256) unsigned char g_static_planes[kStaticPlaneBytes];

// In host code the array's name is only a handle for the runtime, not a device address; the
// address a kernel may use comes from cudaGetSymbolAddress, looked up once per device (under a lock:
// the entry point may be called from any thread).
void *g_static_planes_addr[64] = {};
std::mutex g_static_planes_lock;

// `dev` must be the current device: cudaGetSymbolAddress answers for the device that is current.
int static_planes(int dev, void **out) {
    if (dev < 0 || dev >= 64) return AZ_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> hold(g_static_planes_lock);
    if (!g_static_planes_addr[dev]) {
        void *ptr = nullptr;
        AZ_CUDA(cudaGetSymbolAddress(&ptr, g_static_planes));
        g_static_planes_addr[dev] = ptr;
    }
    *out = g_static_planes_addr[dev];
    return AZ_OK;
}

}  // namespace
}  // namespace az

extern "C" int az_tower_static(az_net *net, const void *positions_dev, int batch, void *tower_dev, void *cuda_stream) {
    az::Net *n = reinterpret_cast<az::Net *>(net);
    if (!n || batch < 0 || (batch > 0 && (!positions_dev || !tower_dev))) return AZ_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(positions_dev) & 7) || (reinterpret_cast<uintptr_t>(tower_dev) & 15)) return AZ_ERR_BAD_ARG;
    // bf16 networks with the tensor-core tower only: an 8-bit network would need az_tower's calibration checks
    if (!n->tc_ready || n->fp8 || n->pnet || n->in_pad != 32 || n->arch.channels != 128) return AZ_ERR_UNSUPPORTED;
    if (batch > az::kStaticMaxBatch || (uint32_t)batch > n->arch.max_batch) return AZ_ERR_BATCH_TOO_LARGE;
    // the array of the network's own device is the one its kernels can use: a caller that has switched to another
    // device since az_load_net would be handed that other device's array
    int dev = -1;
    AZ_CUDA(cudaGetDevice(&dev));
    if (dev != n->device) return AZ_ERR_BAD_ARG;
    if (batch == 0) return AZ_OK;
    void *planes = nullptr;
    int rc = az::static_planes(dev, &planes);
    if (rc != AZ_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    // The encoder writes every channel of every square of the `batch` positions it is given, padding
    // included, so nothing in the shared array has to start at zero.
    rc = az::launch_encode(positions_dev, az_position_bytes(&n->arch), batch, (int)n->arch.in_planes, n->in_pad,
                           true, planes, n->status_dev, s);
    if (rc != AZ_OK) return rc;
    return az::launch_tower_tc(*n, planes, nullptr, batch, tower_dev, false, nullptr, s);
}
