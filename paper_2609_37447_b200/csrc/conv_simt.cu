// 3x3 convolution + folded batch-norm + optional residual + ReLU on plain FP32 ALUs.
//
// out[b][sq][co] = relu( scale[co] * sum_{tap,ci} W[tap][ci][co] * in[b][sq+tap][ci] + bias[co] (+ res) )
// (block order convolution, normalisation, activation, convolution, normalisation, residual
// addition, activation: Sec. 4.3.6).  This is the exact-arithmetic path: the FP32 network must
// match the reference to 1e-4, which rules out TF32 tensor cores (10-bit mantissa), and it is
// the fallback for shapes the tensor-core tower does not cover.
//
// One CTA per (board, 64 output channels).  The board's input is staged in shared memory as a
// zero-bordered 10x10 frame in 32-channel chunks; a thread owns one output channel and 16
// squares, reads its weights coalesced across the CTA ([tap][ci][co] layout) and the inputs as
// shared-memory broadcasts.  Bound: FP32 FMA issue.
#include "common.cuh"

namespace az {
namespace {

template <typename T> __device__ __forceinline__ float ld_act(const T *p);
template <> __device__ __forceinline__ float ld_act<float>(const float *p) { return *p; }
template <> __device__ __forceinline__ float ld_act<__nv_bfloat16>(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ T st_act(float v);
template <> __device__ __forceinline__ float st_act<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 st_act<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

constexpr int kChunk = 32;       // input channels staged per pass
constexpr int kCoutTile = 64;

template <typename T>
__global__ void __launch_bounds__(256)
conv3x3_simt_kernel(const T *__restrict__ in, const T *__restrict__ w, const float *__restrict__ scale,
                    const float *__restrict__ bias, const T *__restrict__ residual, T *__restrict__ out,
                    int cin, int cout) {
    __shared__ __align__(16) float frame[100][kChunk];       // zero-bordered 10x10 board, 32 channels
    const int b = blockIdx.x;
    const int lane_co = threadIdx.x & 63, sg = threadIdx.x >> 6;   // 4 square groups of 2 rows each
    const int co = blockIdx.y * kCoutTile + lane_co;
    const bool active = co < cout;
    float acc[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = 0.0f;

    for (int c0 = 0; c0 < cin; c0 += kChunk) {
        __syncthreads();
        for (int i = threadIdx.x; i < 100 * kChunk; i += 256) {
            const int p = i / kChunk, ci = i % kChunk;
            const int y = p / 10 - 1, x = p % 10 - 1;
            float v = 0.0f;
            if (y >= 0 && y < 8 && x >= 0 && x < 8 && c0 + ci < cin)
                v = ld_act<T>(in + ((size_t)b * 64 + y * 8 + x) * cin + c0 + ci);
            frame[p][ci] = v;
        }
        __syncthreads();
        if (!active) continue;
        const int nci = min(kChunk, cin - c0);
#pragma unroll 1
        for (int tap = 0; tap < 9; ++tap) {
            const int dy = tap / 3, dx = tap % 3;              // frame offsets 0..2
            const T *wt = w + ((size_t)tap * cin + c0) * cout + co;
#pragma unroll 1
            for (int ci = 0; ci < nci; ci += 4) {
                float wv[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) wv[j] = ci + j < nci ? ld_act<T>(wt + (size_t)(ci + j) * cout) : 0.0f;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int y = sg * 2 + (i >> 3), x = i & 7;
                    const float4 v = *reinterpret_cast<const float4 *>(&frame[(y + dy) * 10 + x + dx][ci]);
                    acc[i] = fmaf(wv[0], v.x, acc[i]);
                    acc[i] = fmaf(wv[1], v.y, acc[i]);
                    acc[i] = fmaf(wv[2], v.z, acc[i]);
                    acc[i] = fmaf(wv[3], v.w, acc[i]);
                }
            }
        }
    }
    if (!active) return;
    const float s = scale[co], bi = bias[co];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const int sq = sg * 16 + i;
        const size_t o = ((size_t)b * 64 + sq) * cout + co;
        float v = fmaf(s, acc[i], bi);
        if (residual) v += ld_act<T>(residual + o);
        out[o] = st_act<T>(fmaxf(v, 0.0f));
    }
}

}  // namespace

int launch_conv3x3_simt(const void *in, const void *w, const float *scale, const float *bias,
                        const void *residual, void *out, int batch, int cin, int cout, bool bf16,
                        cudaStream_t s) {
    if (batch == 0) return AZ_OK;
    dim3 grid((unsigned)batch, (unsigned)((cout + kCoutTile - 1) / kCoutTile));
    if (bf16)
        conv3x3_simt_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(
            (const __nv_bfloat16 *)in, (const __nv_bfloat16 *)w, scale, bias, (const __nv_bfloat16 *)residual,
            (__nv_bfloat16 *)out, cin, cout);
    else
        conv3x3_simt_kernel<float><<<grid, 256, 0, s>>>((const float *)in, (const float *)w, scale, bias,
                                                         (const float *)residual, (float *)out, cin, cout);
    AZ_LAUNCH_CHECK();
    return AZ_OK;
}

}  // namespace az
