// The residual convolution tower of fp32 networks as ONE kernel on the FP32 FMA pipes (block order
// convolution, normalisation, activation, convolution, normalisation, residual addition, activation:
// Sec. 4.3.6; batch-norm folded into per-channel scale and bias, App. D.3).  The fp32 network must match
// the reference to 1e-4, which rules out TF32 tensor cores (10-bit mantissa): bound = FP32 FMA issue.
//
// A board is carried through every layer by a cluster of two CTAs, each owning four ranks of it (boards are few
// in the fp32 workload, 64: one CTA per board would leave most of the 148 SMs idle).  Activations never leave
// shared memory: a CTA keeps its four ranks plus one halo rank above and below as a zero-bordered frame
// [channel][6 ranks][12 files] (files 1..8 hold the board, 0 and 9 are the zero border, 10 and 11 padding),
// ping-ponged between two buffers from layer to layer.  After every layer the rank next to the other CTA's
// ranks is sent into that CTA's frame as asynchronous stores through distributed shared memory, which count
// as transaction bytes on the receiver's mbarrier: the sender neither fences nor waits.  Input planes are
// encoded from the position record straight into the frame.
//
// Work split inside a CTA (256 threads): a thread owns one output channel and the sixteen squares of two ranks; a
// warp 32 output channels of one pair of ranks; the eight warps are two sets of four that take the even and the
// odd input channels and add their partial sums through shared memory at the end of a layer.  Per input channel a
// thread reads the four ranks it needs as ten-float rows (broadcast loads, the same for all lanes) and its nine
// weights (one float per lane, consecutive across the warp): 21 shared-memory loads per 144 FMAs.  Weights stream
// global -> shared in chunks of sixteen input channels (9 taps x 16 x 64 outputs, 36 KB) with cp.async,
// double-buffered across layer boundaries; the layers' pointers are copied into shared memory once and a layer's
// scale and bias are fetched at its start, so that no dependent global load sits in the loop.  The residual
// stream of a thread's own outputs stays in its registers.
#include "common.cuh"
#include "planes.cuh"
#include "ptx.cuh"

#include <mutex>

namespace az {
namespace {

constexpr int kC = 64;                         // channels of the tower
constexpr int kInPad = 32;                     // input channels of the first layer (19 planes + zero padding)
constexpr int kSets = 2;                         // sets of four warps that share a layer's input channels (four sets: measured slower)
constexpr int kThreads = 128 * kSets;
constexpr int kRows = 6, kCols = 12;           // frame geometry per channel
constexpr int kFrameFloats = kC * kRows * kCols;               // 4608 floats = 18 KB per buffer
#ifndef AZ_F32_CHUNK
#define AZ_F32_CHUNK 16
#endif
constexpr int kChunkCi = AZ_F32_CHUNK;
constexpr int kChunkFloats = 9 * kChunkCi * kC;                // 9216 floats = 36 KB per buffer
constexpr int kHaloBytes = kC * 8 * 4;                          // one rank of all channels
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr int kPartialFloats = (kSets - 1) * 16 * 128;          // the other sets' partial sums, [set - 1][16][128 threads]
constexpr int kMaxConv = 1 + 2 * 64;
constexpr int kSmemBytes = (2 * kFrameFloats + 2 * kChunkFloats + kPartialFloats) * 4 + 64 + kMaxConv * (int)sizeof(F32Layer);

struct F32Args {
    const unsigned char *positions;
    size_t position_stride;
    const F32Layer *layers;          // [n_conv] device table: weights [tap][cin][64], scale[64], bias[64]
    float *out;                      // [batch][64][64]
    uint32_t *status;
    int batch, n_conv;
};

__device__ __forceinline__ void cp_async16(float *smem_dst, const void *gmem_src) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
#ifndef AZ_F32_UNROLL
#define AZ_F32_UNROLL 8
#endif
constexpr int kCiUnroll = AZ_F32_UNROLL;      // input channels of a chunk unrolled together in the inner loop

__device__ __forceinline__ void st_async_cluster_f32(uint32_t cluster_addr, float v, uint32_t cluster_bar) {
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];"
                 ::"r"(cluster_addr), "r"(__float_as_uint(v)), "r"(cluster_bar) : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
tower_f32_kernel(const F32Args args) {
    extern __shared__ __align__(16) float smem_f[];
    float *frame = smem_f;                                      // [2][64][6][12]
    float *wbuf = smem_f + 2 * kFrameFloats;                    // [2][9 taps][16 ci][64 co]
    float *partial = wbuf + 2 * kChunkFloats;                   // [16][128]
    unsigned long long *bars = reinterpret_cast<unsigned long long *>(partial + kPartialFloats);   // halo[2]
    F32Layer *tbl = reinterpret_cast<F32Layer *>(bars + 8);     // the layers' pointers, copied once: no dependent global load per chunk
    __shared__ int abort_flag;
    const uint32_t rank = ptx::cluster_ctarank();
    const int board = blockIdx.x >> 1;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int ci_set = warp >> 2;                               // this set takes the input channels ci % kSets == ci_set
    const int row_pair = (warp >> 1) & 1;                       // ranks 4*rank + 2*row_pair, + 1
    const int co = (warp & 1) * 32 + lane;
    const int t128 = tid & 127;                                 // this thread among its set's 128
    const uint32_t halo_bar[2] = {ptx::smem_addr(&bars[0]), ptx::smem_addr(&bars[1])};

    for (int i = tid; i < 2 * kFrameFloats / 4; i += kThreads) reinterpret_cast<float4 *>(frame)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int i = tid; i < args.n_conv; i += kThreads) tbl[i] = args.layers[i];
    if (tid == 0) {
        ptx::mbar_init(halo_bar[0], 1);
        ptx::mbar_init(halo_bar[1], 1);
        abort_flag = 0;
        ptx::fence_barrier_init();
    }
    __syncthreads();
    // ---- input planes of this CTA's six ranks -> frame buffer 0 (channels 19..31 stay zero)
    {
        const PosCur *rec = reinterpret_cast<const PosCur *>(args.positions + (size_t)board * args.position_stride);
        const float hm = halfmove_plane(rec);
        if (tid == 0 && rank == 0 && (__popcll(rec->pieces[5]) != 1 || __popcll(rec->pieces[11]) != 1))
            atomicOr(args.status, kStatusBadRecord);
        for (int i = tid; i < 19 * kRows * 8; i += kThreads) {
            const int ch = i / (kRows * 8), r = (i / 8) % kRows, x = i % 8;
            const int y = 4 * (int)rank - 1 + r;
            if (y >= 0 && y < 8) {
                const int sq = y * 8 + x, s_abs = rec->stm ? (sq ^ 56) : sq;
                frame[(ch * kRows + r) * kCols + 1 + x] = plane19(rec, ch, s_abs, hm);
            }
        }
    }
    // nothing may reach into the other CTA before its barriers and frames are initialised
    ptx::cluster_arrive();
    ptx::cluster_wait();
    ptx::launch_dependents();        // the heads kernel may start its set-up; it waits for this grid before reading its output

    const int n_conv = args.n_conv;
    auto chunks_of = [&](int l) { return (l == 0 ? kInPad : kC) / kChunkCi; };
    int total_chunks = 0;
    for (int l = 0; l < n_conv; ++l) total_chunks += chunks_of(l);
    // chunk `idx` of the whole sequence -> (layer, chunk within the layer)
    auto issue = [&](int l, int k, int buf) {
        const float *w = tbl[l].w;
        const int cin = l == 0 ? kInPad : kC;
        float *dst = wbuf + buf * kChunkFloats;
        for (int i = tid; i < kChunkFloats / 4; i += kThreads) {
            const int row = i / (kC / 4), c4 = i % (kC / 4);                  // row = tap * 8 + ci within the chunk
            const int tap = row / kChunkCi, ci = row % kChunkCi;
            cp_async16(dst + i * 4, reinterpret_cast<const float4 *>(w + ((size_t)tap * cin + k * kChunkCi + ci) * kC) + c4);
        }
    };

    float acc[2][8], h_reg[2][8];
#pragma unroll
    for (int x = 0; x < 8; ++x) { acc[0][x] = acc[1][x] = 0.0f; h_reg[0][x] = h_reg[1][x] = 0.0f; }
    int l = 0, k = 0;                          // the chunk being computed
    int nl = 0, nk = 0;                        // the chunk being fetched
    uint32_t halo_phase[2] = {0, 0};
    bool ok = true;
    float ch_scale = 0.0f, ch_bias = 0.0f;      // this layer's folded normalisation of this thread's channel, fetched at the layer's start
    issue(0, 0, 0);
    nk = 1;
    if (nk == chunks_of(0)) { nl = 1; nk = 0; }
    for (int idx = 0; idx < total_chunks; ++idx) {
        cp_async_wait_all();
        __syncthreads();                       // chunk idx has landed for everyone; everyone is done with chunk idx - 1 and,
                                               // at a layer's first chunk, with writing the previous layer's outputs
        const int cur = l & 1;                 // frame buffer this layer reads
        if (k == 0 && l > 0) {
            // the other CTA's rank next to ours, sent while it finished layer l - 1
            bool done = false;
            for (uint32_t i = 0; i < kSpinLimit; ++i) {
                if (ptx::mbar_try_wait_cluster(halo_bar[cur], halo_phase[cur])) { done = true; break; }
                if ((i & 63u) == 63u && *(volatile int *)&abort_flag) break;
            }
            halo_phase[cur] ^= 1u;
            if (!done) {
                if (!*(volatile int *)&abort_flag) { abort_flag = 1; atomicOr(args.status, kStatusWaitTimeout); }
                ok = false;
            }
        }
        if (idx + 1 < total_chunks) {
            issue(nl, nk, (idx + 1) & 1);
            if (++nk == chunks_of(nl)) { ++nl; nk = 0; }
        }
        if (k == 0 && tid == 0 && l + 1 < n_conv)
            ptx::mbar_arrive_expect_tx(halo_bar[(l + 1) & 1], kHaloBytes);   // what the other CTA will send after this layer
        if (k == 0 && ci_set == 0) { ch_scale = __ldg(tbl[l].scale + co); ch_bias = __ldg(tbl[l].bias + co); }
        // ---- this set's four of the chunk's eight input channels
        {
            const float *wb = wbuf + (idx & 1) * kChunkFloats + co;
            const float *fb = frame + cur * kFrameFloats + ((k * kChunkCi) * kRows + 2 * row_pair) * kCols;
#pragma unroll kCiUnroll
            for (int c2 = 0; c2 < kChunkCi / kSets; ++c2) {
                const int ci = kSets * c2 + ci_set;
                float a[4][10];
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const float *rp = fb + (ci * kRows + r) * kCols;
                    const float4 v0 = *reinterpret_cast<const float4 *>(rp), v1 = *reinterpret_cast<const float4 *>(rp + 4);
                    const float2 v2 = *reinterpret_cast<const float2 *>(rp + 8);
                    a[r][0] = v0.x; a[r][1] = v0.y; a[r][2] = v0.z; a[r][3] = v0.w;
                    a[r][4] = v1.x; a[r][5] = v1.y; a[r][6] = v1.z; a[r][7] = v1.w;
                    a[r][8] = v2.x; a[r][9] = v2.y;
                }
                float w[9];
#pragma unroll
                for (int t = 0; t < 9; ++t) w[t] = wb[(t * kChunkCi + ci) * kC];
#pragma unroll
                for (int r = 0; r < 2; ++r)
#pragma unroll
                    for (int dy = 0; dy < 3; ++dy)
#pragma unroll
                        for (int dx = 0; dx < 3; ++dx)
#pragma unroll
                            for (int x = 0; x < 8; ++x) acc[r][x] = fmaf(w[dy * 3 + dx], a[r + dy][x + dx], acc[r][x]);
            }
        }
        // ---- layer finished: the two sets' partial sums, folded normalisation, residual, activation; outputs to the
        // other buffer / to global
        if (++k == chunks_of(l)) {
            if (ci_set > 0) {
#pragma unroll
                for (int r = 0; r < 2; ++r)
#pragma unroll
                    for (int x = 0; x < 8; ++x) { partial[((ci_set - 1) * 16 + r * 8 + x) * 128 + t128] = acc[r][x]; acc[r][x] = 0.0f; }
            }
            __syncthreads();
            if (ci_set == 0) {
                const float s = ch_scale, bi = ch_bias;
                const bool conv2 = l >= 2 && (l & 1) == 0;          // second convolution of a block: the residual comes in
                const bool last = l == n_conv - 1;
                const int nxt = (l + 1) & 1;
#pragma unroll
                for (int r = 0; r < 2; ++r) {
                    const int row_local = 2 * row_pair + r;          // 0..3: board rank 4*rank + row_local
                    float v[8];
#pragma unroll
                    for (int x = 0; x < 8; ++x) {
                        float sum = acc[r][x];
#pragma unroll
                        for (int ps = 0; ps < kSets - 1; ++ps) sum += partial[(ps * 16 + r * 8 + x) * 128 + t128];
                        float t = fmaf(s, sum, bi);
                        if (conv2) t += h_reg[r][x];
                        v[x] = fmaxf(t, 0.0f);
                        acc[r][x] = 0.0f;
                        if ((l & 1) == 0) h_reg[r][x] = v[x];        // input layer and second convolutions: the residual stream
                    }
                    const int y = 4 * (int)rank + row_local;
                    if (last) {
                        float *dst = args.out + ((size_t)board * 64 + y * 8) * kC + co;
#pragma unroll
                        for (int x = 0; x < 8; ++x) dst[(size_t)x * kC] = v[x];
                    } else {
                        float *dst = frame + nxt * kFrameFloats + (co * kRows + row_local + 1) * kCols + 1;
#pragma unroll
                        for (int x = 0; x < 8; ++x) dst[x] = v[x];
                        // the rank next to the other CTA's ranks also goes into its frame: our rank 3 is its halo rank 0
                        // (CTA 0 -> CTA 1), our rank 0 its halo rank 5 (CTA 1 -> CTA 0)
                        if (ok && row_local == (rank == 0 ? 3 : 0)) {
                            const int peer_row = rank == 0 ? 0 : 5;
                            const uint32_t local = ptx::smem_addr(frame + nxt * kFrameFloats + (co * kRows + peer_row) * kCols + 1);
                            const uint32_t remote = ptx::map_to_cta(local, rank ^ 1u);
                            const uint32_t rbar = ptx::map_to_cta(halo_bar[nxt], rank ^ 1u);
#pragma unroll
                            for (int x = 0; x < 8; ++x) st_async_cluster_f32(remote + 4u * x, v[x], rbar);
                        }
                    }
                }
            }
            ++l;
            k = 0;
        }
    }
    // neither CTA may leave while the other's stores and barrier updates may still be on their way to it
    ptx::cluster_arrive();
    ptx::cluster_wait();
}

std::mutex g_config_lock;
bool g_configured[64] = {};

}  // namespace

bool tower_f32_shape(const az_arch &a) { return a.precision == AZ_PREC_FP32 && a.channels == kC && a.in_planes == 19; }

int launch_tower_f32(const Net &net, const void *positions, int batch, float *out, cudaStream_t s) {
    if (batch == 0) return AZ_OK;
    int dev = 0;
    AZ_CUDA(cudaGetDevice(&dev));
    {
        std::lock_guard<std::mutex> hold(g_config_lock);
        if (dev >= 0 && dev < 64 && !g_configured[dev]) {
            AZ_CUDA(cudaFuncSetAttribute(tower_f32_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
            g_configured[dev] = true;
        }
    }
    F32Args a;
    a.positions = static_cast<const unsigned char *>(positions);
    a.position_stride = az_position_bytes(&net.arch);
    a.layers = net.f32_layers;
    a.out = out;
    a.status = net.status_dev;
    a.batch = batch;
    a.n_conv = net.n_conv;
    tower_f32_kernel<<<dim3(2u * (unsigned)batch), kThreads, kSmemBytes, s>>>(a);
    AZ_LAUNCH_CHECK();
    return AZ_OK;
}

}  // namespace az

// ---- heads of the same networks in one launch ------------------------------------------------------------------------
// 73-plane policy head (a bare 1x1 convolution with bias: logit[p*64 + sq] = sum_c Wp[p][c] h[sq][c] + bp[p]), the
// legal-move-masked softmax over its 4,672 logits ("illegal actions are masked before softmax over the legal moves",
// App. D.1) and the value head (1x1 convolution to 32 channels, folded normalisation, ReLU, channel-major flattening,
// 128 hidden units with ReLU, then one tanh scalar or three logits and a softmax giving win, draw, loss; Sec. 4.3.4,
// App. D.1), all in fp32.  One CTA of 256 threads per position: a thread keeps its square's 64 features in
// registers, computes the logits of 18-19 planes and 8 value channels for that square (weights are warp-uniform
// loads), holds its logits through the softmax's two block reductions, and the warps then share the hidden layer's
// 128 rows (1 MB of weights per position, streamed from L2, coalesced).
namespace az {
namespace {

constexpr int kHeadThreads = 256;
constexpr int kPolicyPerThread = (kPlanes73 + 3) / 4;          // 19

__device__ __forceinline__ float block_reduce(float v, bool is_max, float *red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float t = __shfl_xor_sync(0xffffffffu, v, o);
        v = is_max ? fmaxf(v, t) : v + t;
    }
    __syncthreads();                                            // red[] may still be read from the previous use
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = red[0];
#pragma unroll
    for (int w = 1; w < kHeadThreads / 32; ++w) r = is_max ? fmaxf(r, red[w]) : r + red[w];
    return r;
}

struct HeadsF32Args {
    const float *h;                  // [batch][64][64] tower output
    const float *p_w, *p_b;          // [73][64], [73]
    const float *v_cw, *v_cs, *v_cb; // [32][64], [32], [32]
    const float *v_w1, *v_b1;        // [128][2048], [128]
    const float *v_w2, *v_b2;        // [V][128], [V]
    const unsigned long long *masks; // [batch][73]
    float *policy;                   // [batch][4672], or null with legal / counts set
    float *legal;                    // [batch][AZ_MAX_LEGAL]
    int *counts;
    float *value;                    // [batch][V]
    uint32_t *status;
    int wdl;
};

__global__ void __launch_bounds__(kHeadThreads)
heads_f32_kernel(const HeadsF32Args a) {
    __shared__ __align__(16) float u[kHeadChannels * 64];      // value projection, channel-major
    __shared__ float hidden[kValueHidden];
    __shared__ float part[kValueHidden * 8];                     // the hidden layer's per-warp partial sums
    __shared__ float red[kHeadThreads / 32];
    __shared__ int rank_base[kPlanes73 + 1];
    // two CTAs per position, on two SMs: the even one computes the policy, the odd one the value (both need nothing but
    // the position's tower output, and one after the other they were a chain of load latencies on one SM)
    const int pos = blockIdx.x >> 1, tid = threadIdx.x, sq = tid & 63, pg = tid >> 6, lane = tid & 31, warp = tid >> 5;
    const bool policy_cta = (blockIdx.x & 1) == 0;
    // before the tower's output exists: ask L2 for this CTA's share of the weights (the hidden layer's megabyte is split
    // over the value CTAs, the policy map over the policy CTAs)
    {
        const char *wb = reinterpret_cast<const char *>(policy_cta ? a.p_w : a.v_w1);
        const size_t bytes = policy_cta ? sizeof(float) * kPlanes73 * kC : sizeof(float) * (size_t)kValueHidden * kHeadChannels * 64;
        const size_t n_cta = gridDim.x >> 1, share = (bytes / n_cta + 127) & ~(size_t)127;
        const size_t off = (size_t)pos * share + (size_t)tid * 128;
        if ((size_t)tid * 128 < share && off < bytes) asm volatile("prefetch.global.L2 [%0];" ::"l"(wb + off));
    }
    ptx::grid_dependency_wait();
    float hr[kC];
    {
        const float4 *src = reinterpret_cast<const float4 *>(a.h + ((size_t)pos * 64 + sq) * kC);
#pragma unroll
        // (not through the read-only path: this kernel may have started before the tower kernel wrote these lines)
        for (int i = 0; i < kC / 4; ++i) { const float4 v = __ldcg(src + i); hr[4 * i] = v.x; hr[4 * i + 1] = v.y; hr[4 * i + 2] = v.z; hr[4 * i + 3] = v.w; }
    }
    if (policy_cta) {
    // ---- policy logits of this square: planes pg, pg + 4, ...
    float lg[kPolicyPerThread];
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < kPolicyPerThread; ++j) {
        const int p = pg + 4 * j;
        lg[j] = -INFINITY;
        if (p < kPlanes73) {
            const float4 *wr = reinterpret_cast<const float4 *>(a.p_w + (size_t)p * kC);
            float acc0 = 0.0f, acc1 = 0.0f;
#pragma unroll
            for (int i = 0; i < kC / 4; ++i) {
                const float4 w = __ldg(wr + i);
                acc0 = fmaf(w.x, hr[4 * i], acc0); acc1 = fmaf(w.y, hr[4 * i + 1], acc1);
                acc0 = fmaf(w.z, hr[4 * i + 2], acc0); acc1 = fmaf(w.w, hr[4 * i + 3], acc1);
            }
            const bool legal = (a.masks[(size_t)pos * kPlanes73 + p] >> sq) & 1ull;
            if (legal) lg[j] = acc0 + acc1 + __ldg(a.p_b + p);
        }
        mx = fmaxf(mx, lg[j]);
    }
    // ---- masked softmax over the position's legal logits
    mx = block_reduce(mx, true, red);
    const bool any = mx > -INFINITY;
    float sum = 0.0f;
#pragma unroll
    for (int j = 0; j < kPolicyPerThread; ++j) {
        lg[j] = (any && lg[j] > -INFINITY) ? expf(lg[j] - mx) : 0.0f;
        sum += lg[j];
    }
    sum = block_reduce(sum, false, red);
    const float inv = any ? 1.0f / sum : 0.0f;
    if (a.policy != nullptr) {
        float *dst = a.policy + (size_t)pos * (kPlanes73 * 64);
#pragma unroll
        for (int j = 0; j < kPolicyPerThread; ++j) {
            const int p = pg + 4 * j;
            if (p < kPlanes73) dst[p * 64 + sq] = lg[j] * inv;
        }
    } else {
        // legal moves only, in ascending policy index (plane-major): the rank of a move is the number of legal moves
        // in the planes before its plane plus the number of set bits below its square in its plane's word
        if (tid == 0) {
            int run = 0;
            for (int p = 0; p < kPlanes73; ++p) { rank_base[p] = run; run += __popcll(a.masks[(size_t)pos * kPlanes73 + p]); }
            rank_base[kPlanes73] = run;
        }
        __syncthreads();
        float *dst = a.legal + (size_t)pos * kMaxLegal;
#pragma unroll
        for (int j = 0; j < kPolicyPerThread; ++j) {
            const int p = pg + 4 * j;
            if (p < kPlanes73) {
                const unsigned long long word = a.masks[(size_t)pos * kPlanes73 + p];
                if ((word >> sq) & 1ull) {
                    const int rk = rank_base[p] + __popcll(word & ((1ull << sq) - 1ull));
                    if (rk < kMaxLegal) dst[rk] = lg[j] * inv;
                }
            }
        }
        if (tid == 0) a.counts[pos] = rank_base[kPlanes73] < kMaxLegal ? rank_base[kPlanes73] : kMaxLegal;
    }
    if (!any && tid == 0) atomicOr(a.status, kStatusEmptyMask);
    return;
    }
    // ---- value projection of this square: channels pg, pg + 4, ...
#pragma unroll
    for (int j = 0; j < kHeadChannels / 4; ++j) {
        const int c = pg + 4 * j;
        const float4 *wr = reinterpret_cast<const float4 *>(a.v_cw + (size_t)c * kC);
        float acc0 = 0.0f, acc1 = 0.0f;
#pragma unroll
        for (int i = 0; i < kC / 4; ++i) {
            const float4 w = __ldg(wr + i);
            acc0 = fmaf(w.x, hr[4 * i], acc0); acc1 = fmaf(w.y, hr[4 * i + 1], acc1);
            acc0 = fmaf(w.z, hr[4 * i + 2], acc0); acc1 = fmaf(w.w, hr[4 * i + 3], acc1);
        }
        u[c * 64 + sq] = fmaxf(fmaf(__ldg(a.v_cs + c), acc0 + acc1, __ldg(a.v_cb + c)), 0.0f);
    }
    __syncthreads();
    // ---- hidden layer: all eight warps share every row (a thread holds eight of the 2,048 inputs in registers and
    // reads the matching eight weights of sixteen rows at a time, 32 independent 16-byte loads in flight), the warps'
    // partial sums meet in shared memory
    {
        const float4 x0 = reinterpret_cast<const float4 *>(u)[2 * tid], x1 = reinterpret_cast<const float4 *>(u)[2 * tid + 1];
        for (int j0 = 0; j0 < kValueHidden; j0 += 16) {
            float4 w0[16], w1[16];
#pragma unroll
            for (int r = 0; r < 16; ++r) {
                const float4 *wr = reinterpret_cast<const float4 *>(a.v_w1 + (size_t)(j0 + r) * (kHeadChannels * 64)) + 2 * tid;
                w0[r] = __ldg(wr);
                w1[r] = __ldg(wr + 1);
            }
#pragma unroll
            for (int r = 0; r < 16; ++r) {
                float v = fmaf(w0[r].x, x0.x, fmaf(w0[r].y, x0.y, fmaf(w0[r].z, x0.z, w0[r].w * x0.w))) +
                          fmaf(w1[r].x, x1.x, fmaf(w1[r].y, x1.y, fmaf(w1[r].z, x1.z, w1[r].w * x1.w)));
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                if (lane == 0) part[(j0 + r) * 8 + warp] = v;
            }
        }
        __syncthreads();
        if (tid < kValueHidden) {
            float v = 0.0f;
#pragma unroll
            for (int w = 0; w < 8; ++w) v += part[tid * 8 + w];
            hidden[tid] = fmaxf(v + __ldg(a.v_b1 + tid), 0.0f);
        }
    }
    __syncthreads();
    // ---- value tail: 128 -> 1 tanh, or 128 -> 3 softmax (win, draw, loss for the player to move)
    if (warp == 0) {
        const int V = a.wdl ? 3 : 1;
        float z[3] = {0.0f, 0.0f, 0.0f};
        for (int v = 0; v < V; ++v) {
            float acc = 0.0f;
            for (int i = lane; i < kValueHidden; i += 32) acc = fmaf(__ldg(a.v_w2 + v * kValueHidden + i), hidden[i], acc);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            z[v] = acc + __ldg(a.v_b2 + v);
        }
        if (lane == 0) {
            if (!a.wdl) a.value[pos] = tanhf(z[0]);
            else {
                const float m = fmaxf(z[0], fmaxf(z[1], z[2]));
                const float e0 = expf(z[0] - m), e1 = expf(z[1] - m), e2 = expf(z[2] - m);
                const float iv = 1.0f / (e0 + e1 + e2);
                a.value[(size_t)pos * 3 + 0] = e0 * iv;
                a.value[(size_t)pos * 3 + 1] = e1 * iv;
                a.value[(size_t)pos * 3 + 2] = e2 * iv;
            }
        }
    }
}

}  // namespace

int launch_heads_f32(const Net &n, const void *tower, const uint64_t *masks, int batch, float *policy, float *legal,
                     int *counts, float *value, cudaStream_t s) {
    if (batch == 0) return AZ_OK;
    HeadsF32Args a;
    a.h = static_cast<const float *>(tower);
    a.p_w = static_cast<const float *>(n.p_w); a.p_b = n.p_bias;
    a.v_cw = static_cast<const float *>(n.v_cw); a.v_cs = n.v_cscale; a.v_cb = n.v_cbias;
    a.v_w1 = static_cast<const float *>(n.v_w1); a.v_b1 = n.v_b1;
    a.v_w2 = n.v_w2; a.v_b2 = n.v_b2;
    a.masks = reinterpret_cast<const unsigned long long *>(masks);
    a.policy = policy; a.legal = legal; a.counts = counts; a.value = value;
    a.status = n.status_dev;
    a.wdl = n.arch.value_head == AZ_VALUE_WDL;
    AZ_CUDA(launch_dependent(heads_f32_kernel, dim3(2 * batch), dim3(kHeadThreads), 0, s, a));
    return AZ_OK;
}

}  // namespace az
