// Policy and value heads and the legal-move-masked softmax (Sec. 3.5, Sec. 4.3.1, Sec. 4.3.4,
// App. D.1).  Generic FP32-ALU kernels; inputs may be float32 or bfloat16, accumulation is fp32.
//
//   conv1x1        out[b][co*64+sq] = act( scale[co] * sum_ci W[co][ci]*h[b][sq][ci] + bias[co] )
//                  (the 73-plane policy logits, and the 32-channel projections of the flat policy
//                  head and of the value head; the output is already the channel-major flattening
//                  the fully-connected layers consume)
//   fc             out[m][n] = act( sum_k A[m][k]*W[n][k] + bias[n] )
//   value_tail     128 -> 1 tanh, or 128 -> 3 softmax giving (win, draw, loss) for the mover
//   masked_softmax p_i = exp(l_i - max_legal) / sum_legal exp(l_j - max_legal) on legal entries,
//                  exactly 0 elsewhere ("illegal actions are masked before softmax over the legal
//                  moves"); one CTA per position, logits held in registers, warp-shuffle reductions.
#include "common.cuh"

namespace az {
namespace {

template <typename T> __device__ __forceinline__ float ld_act(const T *p);
template <> __device__ __forceinline__ float ld_act<float>(const float *p) { return *p; }
template <> __device__ __forceinline__ float ld_act<__nv_bfloat16>(const __nv_bfloat16 *p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ T st_act(float v);
template <> __device__ __forceinline__ float st_act<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 st_act<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// ---- 1x1 convolution over one board per CTA --------------------------------------------------
constexpr int kMaxCoutPerThread = 20;      // cout <= 80 with 4 channel groups

template <typename TIN, typename TOUT>
__global__ void __launch_bounds__(256)
conv1x1_kernel(const TIN *__restrict__ h, const TIN *__restrict__ w, const float *__restrict__ scale,
               const float *__restrict__ bias, int cin, int cout, int relu, TOUT *__restrict__ out) {
    __shared__ float hs[64][65];                 // [ci within chunk][square], padded against bank conflicts
    const int b = blockIdx.x, sq = threadIdx.x & 63, cg = threadIdx.x >> 6;
    float acc[kMaxCoutPerThread];
#pragma unroll
    for (int j = 0; j < kMaxCoutPerThread; ++j) acc[j] = 0.0f;
    for (int c0 = 0; c0 < cin; c0 += 64) {
        __syncthreads();
        for (int i = threadIdx.x; i < 64 * 64; i += 256) {
            const int s = i >> 6, ci = i & 63;
            hs[ci][s] = c0 + ci < cin ? ld_act<TIN>(h + ((size_t)b * 64 + s) * cin + c0 + ci) : 0.0f;
        }
        __syncthreads();
        const int nci = min(64, cin - c0);
#pragma unroll
        for (int j = 0; j < kMaxCoutPerThread; ++j) {
            const int co = cg + 4 * j;
            if (co < cout) {
                const TIN *wr = w + (size_t)co * cin + c0;
                float a = acc[j];
                for (int ci = 0; ci < nci; ++ci) a = fmaf(ld_act<TIN>(wr + ci), hs[ci][sq], a);
                acc[j] = a;
            }
        }
    }
#pragma unroll
    for (int j = 0; j < kMaxCoutPerThread; ++j) {
        const int co = cg + 4 * j;
        if (co < cout) {
            float v = fmaf(scale ? scale[co] : 1.0f, acc[j], bias[co]);
            if (relu) v = fmaxf(v, 0.0f);
            out[(size_t)b * cout * 64 + co * 64 + sq] = st_act<TOUT>(v);
        }
    }
}

// ---- fully-connected layer: 64x64 output tile per CTA, 4x4 per thread -------------------------
template <typename TIN, typename TOUT>
__global__ void __launch_bounds__(256)
fc_kernel(const TIN *__restrict__ a, const TIN *__restrict__ w, const float *__restrict__ bias,
          int m, int n, int k, int relu, TOUT *__restrict__ out) {
    __shared__ float as[16][65], ws[16][65];
    const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < k; k0 += 16) {
        __syncthreads();
        for (int i = threadIdx.x; i < 64 * 16; i += 256) {
            const int r = i >> 4, kk = i & 15;
            as[kk][r] = (m0 + r < m && k0 + kk < k) ? ld_act<TIN>(a + (size_t)(m0 + r) * k + k0 + kk) : 0.0f;
            ws[kk][r] = (n0 + r < n && k0 + kk < k) ? ld_act<TIN>(w + (size_t)(n0 + r) * k + k0 + kk) : 0.0f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            float av[4], wv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { av[i] = as[kk][ty * 4 + i]; wv[i] = ws[kk][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], wv[j], acc[i][j]);
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int mm = m0 + ty * 4 + i, nn = n0 + tx * 4 + j;
            if (mm < m && nn < n) {
                float v = acc[i][j] + bias[nn];
                if (relu) v = fmaxf(v, 0.0f);
                out[(size_t)mm * n + nn] = st_act<TOUT>(v);
            }
        }
}

// ---- fully-connected layer for few rows (the fp32 network's value head: 64 x 2048 -> 128): the tiled kernel above
// would run on two CTAs.  Here a warp owns one output column and sixteen rows: its column of weights stays in
// registers (K / 32 values per lane, K <= 2048), every row is one coalesced pass over K and a shuffle reduction.
constexpr int kFcRows = 16;
__global__ void __launch_bounds__(256)
fc_fewrows_kernel(const float *__restrict__ a, const float *__restrict__ w, const float *__restrict__ bias,
                  int m, int n, int k, int relu, float *__restrict__ out) {
    const int lane = threadIdx.x & 31, col = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (col >= n) return;                                    // whole warps leave together
    const int m0 = blockIdx.y * kFcRows;
    const int k4 = k / 128;                                  // float4 per lane
    float4 wv[16];
    const float4 *wp = reinterpret_cast<const float4 *>(w + (size_t)col * k);
#pragma unroll
    for (int j = 0; j < 16; ++j) wv[j] = j < k4 ? __ldg(wp + j * 32 + lane) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    const float bv = bias[col];
    for (int r = m0; r < m0 + kFcRows && r < m; ++r) {
        const float4 *ap = reinterpret_cast<const float4 *>(a + (size_t)r * k);
        float acc0 = 0.0f, acc1 = 0.0f;
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            if (j < k4) {
                const float4 av = __ldg(ap + j * 32 + lane);
                acc0 = fmaf(av.x, wv[j].x, acc0); acc1 = fmaf(av.y, wv[j].y, acc1);
                acc0 = fmaf(av.z, wv[j].z, acc0); acc1 = fmaf(av.w, wv[j].w, acc1);
            }
        }
        float v = acc0 + acc1;
#pragma unroll
        for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) {
            v += bv;
            out[(size_t)r * n + col] = relu ? fmaxf(v, 0.0f) : v;
        }
    }
}

// ---- value tail: one warp per position ---------------------------------------------------------
__global__ void __launch_bounds__(128)
value_tail_kernel(const float *__restrict__ hidden, const float *__restrict__ w2, const float *__restrict__ b2,
                  int batch, int wdl, float *__restrict__ value) {
    const int pos = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (pos >= batch) return;
    const int V = wdl ? 3 : 1;
    float z[3] = {0.0f, 0.0f, 0.0f};
    for (int v = 0; v < V; ++v) {
        float a = 0.0f;
        for (int i = lane; i < kValueHidden; i += 32) a = fmaf(w2[v * kValueHidden + i], hidden[(size_t)pos * kValueHidden + i], a);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        z[v] = a + b2[v];
    }
    if (lane == 0) {
        if (!wdl) value[pos] = tanhf(z[0]);
        else {
            const float mx = fmaxf(z[0], fmaxf(z[1], z[2]));
            const float e0 = expf(z[0] - mx), e1 = expf(z[1] - mx), e2 = expf(z[2] - mx);
            const float inv = 1.0f / (e0 + e1 + e2);
            value[(size_t)pos * 3 + 0] = e0 * inv;
            value[(size_t)pos * 3 + 1] = e1 * inv;
            value[(size_t)pos * 3 + 2] = e2 * inv;
        }
    }
}

__device__ __forceinline__ void grid_dependency_wait_if(int pdl) {
    if (pdl) asm volatile("griddepcontrol.wait;" ::: "memory");
}

// ---- masked softmax: one CTA (128 threads) per position ----------------------------------------
template <int ITEMS>       // elements per thread: ceil(n / 128)
__global__ void __launch_bounds__(128)
masked_softmax_kernel(const float *__restrict__ logits, const unsigned long long *__restrict__ masks,
                      int n, int words, float *__restrict__ policy, uint32_t *__restrict__ status, int pdl) {
    __shared__ float red[4];
    __shared__ unsigned long long mw[80];
    const int pos = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    if (tid < words) mw[tid] = masks[(size_t)pos * words + tid];
    __syncthreads();
    grid_dependency_wait_if(pdl);                   // the logits come from the previous kernel in the stream
    const float *row = logits + (size_t)pos * n;
    float v[ITEMS];
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
        const int i = tid + 128 * j;
        const bool legal = i < n && ((mw[i >> 6] >> (i & 63)) & 1ull);
        v[j] = legal ? __ldcg(row + i) : -INFINITY;      // (written by the kernel before: not through the read-only path)
        mx = fmaxf(mx, v[j]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (lane == 0) red[wid] = mx;
    __syncthreads();
    mx = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
    __syncthreads();
    const bool any = mx > -INFINITY;
    float sum = 0.0f;
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
        v[j] = (any && v[j] > -INFINITY) ? expf(v[j] - mx) : 0.0f;
        sum += v[j];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if (lane == 0) red[wid] = sum;
    __syncthreads();
    sum = (red[0] + red[1]) + (red[2] + red[3]);
    const float inv = any ? 1.0f / sum : 0.0f;
    float *dst = policy + (size_t)pos * n;
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
        const int i = tid + 128 * j;
        if (i < n) dst[i] = v[j] * inv;
    }
    if (!any && tid == 0) atomicOr(status, kStatusEmptyMask);
}

// ---- masked softmax, legal moves only: one warp per position -------------------------------------
// out[pos][j] = probability of the j-th legal move in ascending policy-index order (the order in which
// a consumer walks the mask's set bits), j < counts[pos] <= kMaxLegal; entries beyond are not written.
__global__ void __launch_bounds__(128)
masked_softmax_compact_kernel(const float *__restrict__ logits, const unsigned long long *__restrict__ masks,
                              int batch, int n, int words, float *__restrict__ out, int *__restrict__ counts,
                              uint32_t *__restrict__ status, int pdl) {
    __shared__ float vals[4][kMaxLegal];
    const int wid = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int pos = blockIdx.x * 4 + wid;
    grid_dependency_wait_if(pdl);                   // the logits come from the previous kernel in the stream
    if (pos >= batch) return;
    const float *row = logits + (size_t)pos * n;
    float *v = vals[wid];
    // lane w owns mask words w, w+32, w+64; ranks of its bits come from a warp prefix sum of popcounts
    unsigned long long mw[3];
    int cnt = 0;
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        const int w = lane + 32 * k;
        mw[k] = w < words ? masks[(size_t)pos * words + w] : 0ull;
        // bits beyond the last policy index are ignored
        if (w < words && (w + 1) * 64 > n) mw[k] &= (n - w * 64 >= 64) ? ~0ull : ((1ull << (n - w * 64)) - 1ull);
    }
    int base[3];
    int total = 0;
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        cnt = __popcll(mw[k]);
        int incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        base[k] = total + incl - cnt;
        total += __shfl_sync(0xffffffffu, incl, 31);
    }
    const int n_legal = total < kMaxLegal ? total : kMaxLegal;
    float mx = -INFINITY;
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        unsigned long long bits = mw[k];
        int j = base[k];
        while (bits) {
            const int bit = __ffsll((long long)bits) - 1;
            bits &= bits - 1;
            if (j < kMaxLegal) {
                const float l = __ldcg(row + (lane + 32 * k) * 64 + bit);
                v[j] = l;
                mx = fmaxf(mx, l);
            }
            ++j;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    __syncwarp();
    float sum = 0.0f;
    for (int j = lane; j < n_legal; j += 32) { const float e = expf(v[j] - mx); v[j] = e; sum += e; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    const float inv = n_legal > 0 ? 1.0f / sum : 0.0f;
    float *dst = out + (size_t)pos * kMaxLegal;
    for (int j = lane; j < n_legal; j += 32) dst[j] = v[j] * inv;
    if (lane == 0) {
        counts[pos] = n_legal;
        if (n_legal == 0) atomicOr(status, kStatusEmptyMask);
    }
}

}  // namespace

int launch_masked_softmax_compact(const float *logits, const uint64_t *masks, int batch, int n, int words,
                                  float *out, int *counts, uint32_t *status, bool pdl, cudaStream_t s) {
    if (batch == 0) return AZ_OK;
    if (words > 96) return AZ_ERR_BAD_ARCH;
    if (pdl)
        AZ_CUDA(launch_dependent(masked_softmax_compact_kernel, dim3((batch + 3) / 4), dim3(128), 0, s, logits,
                                 reinterpret_cast<const unsigned long long *>(masks), batch, n, words, out, counts, status, 1));
    else {
        masked_softmax_compact_kernel<<<(batch + 3) / 4, 128, 0, s>>>(
            logits, reinterpret_cast<const unsigned long long *>(masks), batch, n, words, out, counts, status, 0);
        AZ_LAUNCH_CHECK();
    }
    return AZ_OK;
}

int launch_conv1x1(const void *in, const void *w, const float *scale, const float *bias, int batch,
                   int cin, int cout, bool relu, bool bf16_in, void *out, bool out_f32, cudaStream_t s) {
    if (batch == 0) return AZ_OK;
    if (cout > 4 * kMaxCoutPerThread) return AZ_ERR_BAD_ARCH;
    typedef __nv_bfloat16 bf;
    if (bf16_in && out_f32) conv1x1_kernel<bf, float><<<batch, 256, 0, s>>>((const bf *)in, (const bf *)w, scale, bias, cin, cout, relu, (float *)out);
    else if (bf16_in) conv1x1_kernel<bf, bf><<<batch, 256, 0, s>>>((const bf *)in, (const bf *)w, scale, bias, cin, cout, relu, (bf *)out);
    else conv1x1_kernel<float, float><<<batch, 256, 0, s>>>((const float *)in, (const float *)w, scale, bias, cin, cout, relu, (float *)out);
    AZ_LAUNCH_CHECK();
    return AZ_OK;
}

int launch_fc(const void *a, const void *w, const float *bias, int m, int n, int k, bool relu,
              bool bf16_in, void *out, bool out_f32, cudaStream_t s) {
    if (m == 0) return AZ_OK;
    typedef __nv_bfloat16 bf;
    if (!bf16_in && out_f32 && m <= 256 && k % 128 == 0 && k <= 2048) {
        fc_fewrows_kernel<<<dim3((unsigned)((n + 7) / 8), (unsigned)((m + kFcRows - 1) / kFcRows)), 256, 0, s>>>(
            (const float *)a, (const float *)w, bias, m, n, k, relu, (float *)out);
        AZ_LAUNCH_CHECK();
        return AZ_OK;
    }
    dim3 grid((unsigned)((n + 63) / 64), (unsigned)((m + 63) / 64));
    if (bf16_in && out_f32) fc_kernel<bf, float><<<grid, 256, 0, s>>>((const bf *)a, (const bf *)w, bias, m, n, k, relu, (float *)out);
    else if (bf16_in) fc_kernel<bf, bf><<<grid, 256, 0, s>>>((const bf *)a, (const bf *)w, bias, m, n, k, relu, (bf *)out);
    else fc_kernel<float, float><<<grid, 256, 0, s>>>((const float *)a, (const float *)w, bias, m, n, k, relu, (float *)out);
    AZ_LAUNCH_CHECK();
    return AZ_OK;
}

int launch_value_tail(const float *hidden, const float *w2, const float *b2, int batch, int wdl,
                      float *value, cudaStream_t s) {
    if (batch == 0) return AZ_OK;
    value_tail_kernel<<<(batch + 3) / 4, 128, 0, s>>>(hidden, w2, b2, batch, wdl, value);
    AZ_LAUNCH_CHECK();
    return AZ_OK;
}

int launch_masked_softmax(const float *logits, const uint64_t *masks, int batch, int n, int words,
                          float *policy, uint32_t *status, bool pdl, cudaStream_t s) {
    if (batch == 0) return AZ_OK;
    const unsigned long long *m = reinterpret_cast<const unsigned long long *>(masks);
    if (n > 128 * 37) return AZ_ERR_BAD_ARCH;
    if (pdl) {
        if (n <= 128 * 15) AZ_CUDA(launch_dependent(masked_softmax_kernel<15>, dim3(batch), dim3(128), 0, s, logits, m, n, words, policy, status, 1));
        else AZ_CUDA(launch_dependent(masked_softmax_kernel<37>, dim3(batch), dim3(128), 0, s, logits, m, n, words, policy, status, 1));
        return AZ_OK;
    }
    if (n <= 128 * 15) masked_softmax_kernel<15><<<batch, 128, 0, s>>>(logits, m, n, words, policy, status, 0);
    else masked_softmax_kernel<37><<<batch, 128, 0, s>>>(logits, m, n, words, policy, status, 0);
    AZ_LAUNCH_CHECK();
    return AZ_OK;
}

}  // namespace az
