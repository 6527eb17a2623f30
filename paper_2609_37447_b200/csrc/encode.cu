// Bitboards -> input planes (App. D.1, Table D.1 conventions: side-to-move canonical, ranks
// reflected and colours exchanged for Black to move, files keep their order, flags and scalars
// fill all 64 squares, halfmove clock capped at 100, missing history zero-filled).
//
// Output layout: [position][square][channel], channel count padded to a multiple of 32 with
// zeros, so that one thread writes one square's channels as consecutive 16-byte stores and a warp
// writes one contiguous run.  One thread per (position, square); the bitboards of a position are
// read by all 64 threads of that position from the same words (broadcast through L1).
// HBM-bound: per position 104 B (784 B with history) in, 64 * channels * sizeof(T) out.
#include "common.cuh"
#include "planes.cuh"

namespace az {
namespace {

template <typename T, int IN_PLANES, int PAD>
__global__ void __launch_bounds__(256)
encode_planes_kernel(const unsigned char *__restrict__ positions, size_t stride, int batch,
                     T *__restrict__ planes, uint32_t *__restrict__ status) {
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int pos = (int)(gid >> 6), c = (int)(gid & 63);
    if (pos >= batch) return;
    const PosCur *r = reinterpret_cast<const PosCur *>(positions + (size_t)pos * stride);
    const int s = r->stm ? (c ^ 56) : c;                    // reflect ranks for Black
    const int hmc = r->halfmove > 100 ? 100 : r->halfmove;
    const float hm = __fdiv_rn((float)hmc, 100.0f);         // single-precision IEEE division
    if (c == 0 && (__popcll(r->pieces[5]) != 1 || __popcll(r->pieces[11]) != 1))
        atomicOr(status, kStatusBadRecord);
    constexpr int PER = 16 / sizeof(T);                     // channels per 16-byte store
    T *out = planes + ((size_t)pos * 64 + c) * PAD;
#pragma unroll 1
    for (int c0 = 0; c0 < PAD; c0 += PER) {
        alignas(16) T v[PER];
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const int ch = c0 + j;
            float f = 0.0f;
            if (ch < IN_PLANES)
                f = IN_PLANES == 19 ? plane19(r, ch, s, hm)
                                    : plane112(reinterpret_cast<const PosH8 *>(r), ch, s, hm);
            v[j] = to_act<T>(f);
        }
        *reinterpret_cast<uint4 *>(out + c0) = *reinterpret_cast<const uint4 *>(v);
    }
}

}  // namespace

int launch_encode(const void *positions, size_t stride, int batch, int in_planes, int in_pad,
                  bool bf16, void *planes, uint32_t *status, cudaStream_t s) {
    if (batch == 0) return AZ_OK;
    const long long threads = (long long)batch * 64;
    const int block = 256;
    const unsigned grid = (unsigned)((threads + block - 1) / block);
    const unsigned char *p = static_cast<const unsigned char *>(positions);
    if (in_planes == 19 && in_pad == 32) {
        if (bf16) encode_planes_kernel<__nv_bfloat16, 19, 32><<<grid, block, 0, s>>>(p, stride, batch, (__nv_bfloat16 *)planes, status);
        else encode_planes_kernel<float, 19, 32><<<grid, block, 0, s>>>(p, stride, batch, (float *)planes, status);
    } else if (in_planes == 112 && in_pad == 128) {
        if (bf16) encode_planes_kernel<__nv_bfloat16, 112, 128><<<grid, block, 0, s>>>(p, stride, batch, (__nv_bfloat16 *)planes, status);
        else encode_planes_kernel<float, 112, 128><<<grid, block, 0, s>>>(p, stride, batch, (float *)planes, status);
    } else {
        return AZ_ERR_BAD_ARCH;
    }
    AZ_LAUNCH_CHECK();
    return AZ_OK;
}

}  // namespace az
