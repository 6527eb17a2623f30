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
// shared-memory broadcasts.  Bound: FP32 FMA issue.  This general form serves odd shapes and the
// bf16 nets the tensor-core tower does not cover; fp32 nets with channel counts in multiples of
// 32 / 64 (the fp32 config) take the tiled kernel further down.
#include "common.cuh"

#include <mutex>

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

// The same convolution for fp32 networks whose channel counts are multiples of 32 (in) and 64 (out), tiled
// for the FMA pipes: one CTA per (half board, 64 output channels), 128 threads, a thread owns 4 output
// channels x 4 neighbouring squares of one rank.  Per 32-channel chunk the half board's zero-bordered frame
// (6 x 10 squares) and ALL the chunk's weights (9 taps x 32 x 64, 72 KB) are staged in shared memory, so the
// inner loop is eight 16-byte shared-memory loads (four of weights, conflict-free across the 16 channel
// groups of a warp; four of inputs, broadcasts) per 64 FMAs and touches no global memory.
// 16-byte asynchronous copy global -> shared (all of a thread's copies are in flight together)
__device__ __forceinline__ void cp_async16(float *smem_dst, const void *gmem_src) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

constexpr int kTileThreads = 128;
constexpr int kTileFrame = 60 * kChunk;                   // floats
constexpr int kTileWeights = 9 * kChunk * kCoutTile;      // floats
constexpr int kTileSmem = (kTileFrame + kTileWeights) * 4;

__global__ void __launch_bounds__(kTileThreads)
conv3x3_f32_tiled_kernel(const float *__restrict__ in, const float *__restrict__ w, const float *__restrict__ scale,
                         const float *__restrict__ bias, const float *__restrict__ residual, float *__restrict__ out,
                         int cin, int cout) {
    extern __shared__ __align__(16) float tile_smem[];
    float *frame = tile_smem;                              // [6 ranks][10 files][32 channels]
    float *wt = tile_smem + kTileFrame;                    // [9 taps][32 channels][64 outputs]
    const int b = blockIdx.x, half = blockIdx.y, co0 = blockIdx.z * kCoutTile;
    const int cog = threadIdx.x & 15, sqg = threadIdx.x >> 4;        // 16 groups of 4 outputs, 8 groups of 4 squares
    const int ry = sqg >> 1, x0 = (sqg & 1) * 4;                      // rank within the half board, first file
    float acc[4][4];                                                  // [square][output]
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;

    for (int c0 = 0; c0 < cin; c0 += kChunk) {
        __syncthreads();
        for (int i = threadIdx.x; i < 60 * (kChunk / 4); i += kTileThreads) {
            const int p = i / (kChunk / 4), c4 = i % (kChunk / 4);
            const int y = half * 4 + p / 10 - 1, x = p % 10 - 1;
            if (y >= 0 && y < 8 && x >= 0 && x < 8)
                cp_async16(frame + i * 4, reinterpret_cast<const float4 *>(in + ((size_t)b * 64 + y * 8 + x) * cin + c0) + c4);
            else
                reinterpret_cast<float4 *>(frame)[i] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        }
        for (int i = threadIdx.x; i < 9 * kChunk * (kCoutTile / 4); i += kTileThreads) {
            const int row = i / (kCoutTile / 4), c4 = i % (kCoutTile / 4);   // row = tap * 32 + channel of the chunk
            const int tap = row / kChunk, ci = row % kChunk;
            cp_async16(wt + i * 4, reinterpret_cast<const float4 *>(w + ((size_t)tap * cin + c0 + ci) * cout + co0) + c4);
        }
        cp_async_wait_all();                               // every copy of this thread has landed; the barrier publishes them
        __syncthreads();
#pragma unroll 1
        for (int tap = 0; tap < 9; ++tap) {
            const float *fr = frame + ((ry + tap / 3) * 10 + x0 + tap % 3) * kChunk;
            const float *wr = wt + tap * kChunk * kCoutTile + cog * 4;
#pragma unroll 2
            for (int ci = 0; ci < kChunk; ci += 4) {
                float4 wv[4], iv[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) wv[k] = *reinterpret_cast<const float4 *>(wr + (ci + k) * kCoutTile);
#pragma unroll
                for (int i = 0; i < 4; ++i) iv[i] = *reinterpret_cast<const float4 *>(fr + i * kChunk + ci);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float a[4] = {iv[i].x, iv[i].y, iv[i].z, iv[i].w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        acc[i][0] = fmaf(a[k], wv[k].x, acc[i][0]);
                        acc[i][1] = fmaf(a[k], wv[k].y, acc[i][1]);
                        acc[i][2] = fmaf(a[k], wv[k].z, acc[i][2]);
                        acc[i][3] = fmaf(a[k], wv[k].w, acc[i][3]);
                    }
                }
            }
        }
    }
    const float4 s4 = *reinterpret_cast<const float4 *>(scale + co0 + cog * 4);
    const float4 b4 = *reinterpret_cast<const float4 *>(bias + co0 + cog * 4);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int sq = (half * 4 + ry) * 8 + x0 + i;
        const size_t o = ((size_t)b * 64 + sq) * cout + co0 + cog * 4;
        float4 v = make_float4(fmaf(s4.x, acc[i][0], b4.x), fmaf(s4.y, acc[i][1], b4.y), fmaf(s4.z, acc[i][2], b4.z), fmaf(s4.w, acc[i][3], b4.w));
        if (residual) {
            const float4 r = *reinterpret_cast<const float4 *>(residual + o);
            v.x += r.x; v.y += r.y; v.z += r.z; v.w += r.w;
        }
        *reinterpret_cast<float4 *>(out + o) = make_float4(fmaxf(v.x, 0.0f), fmaxf(v.y, 0.0f), fmaxf(v.z, 0.0f), fmaxf(v.w, 0.0f));
    }
}

}  // namespace

int launch_conv3x3_simt(const void *in, const void *w, const float *scale, const float *bias,
                        const void *residual, void *out, int batch, int cin, int cout, bool bf16,
                        cudaStream_t s) {
    if (batch == 0) return AZ_OK;
    if (!bf16 && cin % kChunk == 0 && cout % kCoutTile == 0) {
        static bool configured[64] = {};
        static std::mutex configured_lock;                  // any thread may make a device's first launch
        int dev = 0;
        AZ_CUDA(cudaGetDevice(&dev));
        {
            std::lock_guard<std::mutex> hold(configured_lock);
            if (dev >= 0 && dev < 64 && !configured[dev]) {
                AZ_CUDA(cudaFuncSetAttribute(conv3x3_f32_tiled_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTileSmem));
                configured[dev] = true;
            }
        }
        conv3x3_f32_tiled_kernel<<<dim3((unsigned)batch, 2, (unsigned)(cout / kCoutTile)), kTileThreads, kTileSmem, s>>>(
            (const float *)in, (const float *)w, scale, bias, (const float *)residual, (float *)out, cin, cout);
        AZ_LAUNCH_CHECK();
        return AZ_OK;
    }
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
