// Shared declarations of the az_eval library: the network object, error plumbing and the
// launch functions each .cu file exports to api.cu.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include <vector>

#include "az_eval.h"

namespace az {

constexpr int kHeadChannels = 32;     // width of the 1x1 projections of the flat policy head and the value head
constexpr int kValueHidden = 128;
constexpr int kFlatMoves = 1858;
constexpr int kPlanes73 = 73;
constexpr int kMaxLegal = AZ_MAX_LEGAL;       // row stride of the legal-moves-only policy output

// Device-side status bits (OR-ed into az_net::status_dev by kernels).
enum : uint32_t {
    kStatusEmptyMask = 1u << 0,       // a position had no legal move: all-zero policy row
    kStatusWaitTimeout = 1u << 1,     // a bounded mbarrier wait ran out
    kStatusBadRecord = 1u << 2,       // a position record without exactly one king per side
};

struct ConvLayerF32 {                 // fp32 path: weights [tap][cin][cout], folded scale / bias
    float *w = nullptr, *scale = nullptr, *bias = nullptr;
    int cin = 0, cout = 0;
};

struct F32Layer {                    // one convolution of the fused fp32 tower: device pointers
    const float *w;                   // [tap][cin][cout]
    const float *scale, *bias;        // folded batch-norm
};

struct Net {
    az_arch arch{};
    int device = 0;
    int in_pad = 0;                   // channels of the encoded plane tensor (32 or 128)
    int n_conv = 0;                   // 1 + 2*blocks
    bool bf16 = false;                // activations stored as bf16 (true for BF16 and FP8 nets)

    // ---- generic (SIMT) path: every conv as [tap][cin_pad][cout] in the activation type ----
    void *conv_w[1 + 2 * 64] = {};    // element type = activation type
    float *conv_scale[1 + 2 * 64] = {};
    float *conv_bias[1 + 2 * 64] = {};

    F32Layer *f32_layers = nullptr;   // device table [n_conv] for the fused fp32 tower (64 channels, 19 planes); null otherwise

    // ---- tensor-core tower (bf16, channels == 128) ----
    void *tc_weights = nullptr;       // packed UMMA B-operand tiles, all layers
    void *tc_weights_split = nullptr; // 256 channels: the same tiles packed in halves of N for the small-batch kernel (two CTAs per group)
    void *tc_weights_split4 = nullptr;// and in quarters (four CTAs per group)
    float *tc_bias = nullptr;         // [n_conv][C] folded bias (scales are folded into the weights)
    bool tc_ready = false;
    bool want_pair = true;            // the CTA-pair form of the tower where the shape has one (az_load_net_ex can turn it off)
    bool tc_pair = false;             // the bf16 128-channel tower runs on CTA pairs (tcgen05 .cta_group::2)
    bool tc_pair8 = false;            // the 8-bit tower of a 128-channel residual network runs on CTA pairs (its bf16 passes, calibration, do not)
    // FP8-e4m3 tower (weights and per-layer constants exist once az_calibrate has run)
    bool fp8 = false, fp8_ready = false;   // 8-bit tower (FP8-e4m3 or int8) and whether it has been calibrated
    bool int8 = false;                      // the 8-bit tower's operands are u8 activations x s8 weights
    bool split_a = false, split_w = false;   // e4m3 tower whose activations (and weights) travel as pairs of e4m3 numbers
    bool calib_broken = false;              // az_calibrate failed half-way through its bias correction
    void *tc8_weights = nullptr;
    float *tc8_lconst = nullptr;      // [n_conv][3][C]
    void *host_master = nullptr;      // fp32 tower weights kept on the host until calibration (FP8 nets)
    double *calib_presum = nullptr;    // set only inside az_calibrate: where the tower kernels add up their pre-activations
    void *tc_head_w = nullptr;        // packed 1x1 head projections (policy | value), fused into the tower kernel
    void *tc_head_w_plain = nullptr;  // 256 channels on CTA pairs: the same in plain slice order for the small-batch cluster kernels
    float *tc_head_bias = nullptr;
    int tc_head_n = 0;                // 64 (flat policy head) or 112 (73-plane policy head)
    void *fc_policy_w = nullptr;      // flat policy FC as GEMM B tiles (K permuted to square*32 + channel)
    void *fc_value_w = nullptr;       // value FC1 as GEMM B tiles
    void *u_policy = nullptr;         // head projections as GEMM A tiles [ceil(B/128)][256][16][8][8] bf16
    void *u_value = nullptr;

    // ---- heads ----
    void *p_w = nullptr;              // planes73: [73][C]; flat: 1x1 conv [32][C]      (activation type)
    float *p_scale = nullptr, *p_bias = nullptr;
    void *p_fw = nullptr;             // flat: [1858][2048] (activation type)
    float *p_fbias = nullptr;
    void *v_cw = nullptr;             // [32][C]
    float *v_cscale = nullptr, *v_cbias = nullptr;
    void *v_w1 = nullptr;             // [128][2048]
    float *v_b1 = nullptr;
    float *v_w2 = nullptr, *v_b2 = nullptr;   // [V][128], [V] fp32

    // ---- workspace (sized for max_batch) ----
    void *planes = nullptr;           // [B][64][in_pad]
    void *act[3] = {};                // [B][64][C] x3 (SIMT tower ping-pong; act[0] doubles as tower output)
    float *logits = nullptr;          // [B][policy_size]
    void *head_p = nullptr;           // [B][2048] flat-policy projection (activation type)
    void *head_v = nullptr;           // [B][2048] value projection
    float *hidden = nullptr;          // [B][128]
    uint32_t *status_dev = nullptr;

    // ---- device staging for host-buffer calls (allocated on first use) ----
    void *stage_pos = nullptr;
    uint64_t *stage_masks = nullptr;
    float *stage_policy = nullptr, *stage_value = nullptr;
    float *stage_compact = nullptr;   // [max_batch][AZ_MAX_LEGAL]
    int *stage_counts = nullptr;

    // ---- pipelined host entry: per-slot staging, the az_net's own streams and events ----
    struct HostSlot {
        void *pos = nullptr;
        uint64_t *masks = nullptr;
        float *policy = nullptr, *value = nullptr, *compact = nullptr;
        int *counts = nullptr;
        cudaEvent_t in_ready = nullptr, computed = nullptr, out_ready = nullptr;
        bool busy = false;
    };
    HostSlot slots[AZ_HOST_SLOTS];
    cudaStream_t s_in = nullptr, s_compute[AZ_HOST_SLOTS] = {}, s_out = nullptr;
    int next_slot = 0;
    // second copy of what the tensor-core path keeps between its three kernels, so that the second
    // slot's evaluation can run beside the first's: the tail of one tower launch (the last, partly
    // filled round of board groups) overlaps the head of the next
    void *alt_u_policy = nullptr, *alt_u_value = nullptr;
    float *alt_logits = nullptr;
    void *alt_act0 = nullptr, *alt_pnet_qk = nullptr;   // the paper's network: backbone output, queries and keys

    // ---- the paper's own network (52 planes, pooled context, query-key policy head) ----
    bool pnet = false;
    float *pnet_gw = nullptr;         // [pooled block][C/2][3C/4] (transposed)
    void *pnet_qk = nullptr;          // [max_batch][64][256] fp32: queries | keys
    float *pnet_small = nullptr;      // the finishing kernel's fp32 parameters, see pnet.cu
    unsigned char *pnet_actions = nullptr;   // [1880][4]: origin, destination, promotion piece + 1 (0 none), pad
    void *pnet_master = nullptr;      // int8 form: the fp32 tower parameters, kept until az_calibrate has quantised them

    // ---- optional event timing of the tower ----
    int profile = 0;                  // 0: off; k: every k-th tower pass is bracketed with events
    unsigned profile_count = 0;
    int n_events = 0;                 // pairs recorded since the last read
    cudaEvent_t *ev_begin = nullptr, *ev_end = nullptr;
};
constexpr int kMaxProfiledPasses = 4096;

// ---- error plumbing ------------------------------------------------------------------------
void set_cuda_error(cudaError_t e, const char *what);
#define AZ_CUDA(call)                                                     \
    do {                                                                  \
        cudaError_t e__ = (call);                                         \
        if (e__ != cudaSuccess) { az::set_cuda_error(e__, #call); return AZ_ERR_CUDA; } \
    } while (0)
#define AZ_LAUNCH_CHECK()                                                 \
    do {                                                                  \
        cudaError_t e__ = cudaGetLastError();                             \
        if (e__ != cudaSuccess) { az::set_cuda_error(e__, "kernel launch"); return AZ_ERR_CUDA; } \
    } while (0)

// Launch `kernel` so that it may begin (prologue only) before the previous kernel in the stream has
// finished; the kernel itself must call ptx::grid_dependency_wait() before reading that kernel's output.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// second evaluation workspace (api.cu)
int ensure_second_workspace(Net &n, bool *available);
void swap_workspace(Net &n);

// ---- kernels' launch functions (each returns AZ_OK or AZ_ERR_CUDA) ---------------------------
int launch_encode52(const void *positions, int batch, bool bf16, void *planes, cudaStream_t s);
int build_pnet(Net &n, const unsigned char *blob, size_t nbytes);
// int8 form, after the calibration pass ([n_conv][C] output maxima); hands back the per-layer constants it uploaded
// ([n_conv][4][C]) and, per layer, how many of its output channels the next layer reads as 8-bit activations
int quantise_pnet(Net &n, const float *absmax, std::vector<float> *lconst_out, std::vector<int> *next_cin_out);
void free_pnet_master(void *master);
int launch_pnet_finish(const Net &n, const uint64_t *masks, int batch, float *policy, float *legal, int *counts,
                       float *value, cudaStream_t s);
size_t tc_packed_layers_bytes(const int *cin_pad, int channels, int n_conv);
void tc_pack_layers(const float *const *w, const float *const *scale, const int *cin, const int *cin_pad,
                    int channels, int n_conv, __nv_bfloat16 *packed);
void tc_pack_qk(const float *wq, const float *wk, int channels, __nv_bfloat16 *packed);
int launch_encode(const void *positions, size_t stride, int batch, int in_planes, int in_pad,
                  bool bf16, void *planes, uint32_t *status, cudaStream_t s);
int launch_legal_masks(const void *positions, size_t stride, int batch, int head, uint64_t *masks,
                       cudaStream_t s);
int launch_conv3x3_simt(const void *in, const void *w, const float *scale, const float *bias,
                        const void *residual, void *out, int batch, int cin, int cout, bool bf16,
                        cudaStream_t s);
int launch_conv1x1(const void *in, const void *w, const float *scale, const float *bias, int batch,
                   int cin, int cout, bool relu, bool bf16_in, void *out, bool out_f32, cudaStream_t s);
int launch_fc(const void *a, const void *w, const float *bias, int m, int n, int k, bool relu,
              bool bf16_in, void *out, bool out_f32, cudaStream_t s);
int launch_value_tail(const float *hidden, const float *w2, const float *b2, int batch, int wdl,
                      float *value, cudaStream_t s);
// pdl: the logits come from the kernel launched just before on the same stream, and this launch may overlap its tail
int launch_masked_softmax_compact(const float *logits, const uint64_t *masks, int batch, int n, int words,
                                  float *out, int *counts, uint32_t *status, bool pdl, cudaStream_t s);
int launch_masked_softmax(const float *logits, const uint64_t *masks, int batch, int n, int words,
                          float *policy, uint32_t *status, bool pdl, cudaStream_t s);

// fused fp32 tower (tower_f32.cu): encoder + all convolutions of a 64-channel, 19-plane fp32 network in one launch
bool tower_f32_shape(const az_arch &a);
int launch_tower_f32(const Net &net, const void *positions, int batch, float *out, cudaStream_t s);
// policy (dense, or legal moves only with counts) and value of those networks with the 73-plane head, one launch
int launch_heads_f32(const Net &n, const void *tower, const uint64_t *masks, int batch, float *policy, float *legal,
                     int *counts, float *value, cudaStream_t s);

// tensor-core tower (tower_tc.cu)
size_t tc_packed_weight_bytes(int in_pad, int channels, int n_conv);
void tc_pack_weights(const float *const *w, const float *const *scale, int in_planes, int in_pad,
                     int channels, int n_conv, int halves, int stage_taps, bool rotate, __nv_bfloat16 *packed_host);
bool tc_pair_shape(int channels, int precision, bool pnet);     // the tower runs on CTA pairs (weights packed in halves)
int tc_head_stage_slices(int channels, int head_n);
// exactly one of `planes` (encoded plane tensor) and `positions` (records to encode in the kernel) is non-null
int launch_tower_tc(const Net &net, const void *planes, const void *positions, int batch, void *tower_out,
                    bool with_heads, unsigned int *absmax, cudaStream_t s);
size_t tc8_packed_weight_bytes(int in_pad, int channels, int n_conv, bool split_w);
void tc8_pack(const float *const *w, const float *const *scale, const float *const *bias, const float *absmax,
              int in_planes, int in_pad, int channels, int n_conv, bool int8, bool split_w, int halves, unsigned char *packed, float *lconst);
int tower_tc_launch_count();
size_t tc_head_weight_bytes(int head_n, int channels);
void tc_pack_head(const float *wp, const float *sp, int n_policy, int n_policy_pad, const float *wv, const float *sv,
                  int channels, int halves, int stage_slices, __nv_bfloat16 *packed);

// tensor-core fully-connected layers of the heads (fc_tc.cu)
size_t fc_tc_weight_bytes(int n, bool policy);
void fc_tc_pack_weights(const float *w, int n, bool policy, __nv_bfloat16 *packed);     // w[n][32*64], K permuted to square*32 + channel; policy: the tile height of the head GEMM's CTA pairs
int launch_fc_tc(const Net &net, int batch, float *value_out, cudaStream_t s);

}  // namespace az
