// Fully-connected layers of the heads on tcgen05 tensor cores (Sec. 4.3.1 dense policy head: a
// small spatial projection flattened into the move logits; Sec. 4.3.4 / App. D.1 value head:
// flatten, hidden layer, three logits, softmax giving win/draw/loss, or one tanh scalar).
//
//   policy  logits[b][n] = sum_k U_p[b][k] * Wp[n][k] + bp[n]          n < 1858, k < 2048
//   value   hidden[b][j] = relu(sum_k U_v[b][k] * W1[j][k] + b1[j])    j < 128, then the 128 -> 1|3
//           tail and tanh / softmax, all inside the epilogue of the value tile.
//
// Both operands are bf16 and already sit in global memory as ready-made no-swizzle K-major core-matrix
// tiles of 128 rows (the tower kernel writes U that way, the weights are packed at load), so a pipeline
// stage of 64 k is two contiguous 16 KB bulk copies.  K runs over square*32 + channel; the weights are
// permuted to match at load time.
//
// The kernel is bound by operand traffic from L2, so the policy's tiles are as large as two SMs can make
// them: a cluster of two CTAs computes 256 positions x 256 logits with tcgen05 .cta_group::2 products
// (M = 256: 128 rows from each CTA's own shared memory; N = 256: each CTA holds the weight rows of HALF of
// the columns).  Each CTA streams 1 MB for 128 x 256 outputs, half of what 128 x 128 tiles need, and
// the whole launch reads 64 MB from L2 instead of 128 (batch 1024).  The first CTA issues the products of
// the pair; the second tells it when its own copies have landed.  The value head's single 128-column tile
// runs on the same grid as one more column of CTAs, each on its own (.cta_group::1).
// blockIdx.y: the policy's 256-column tiles, then the value column; blockIdx.x: tiles of 128 positions
// (an even number of them: the cluster is two CTAs along x, as products shared by a CTA pair require; a tile
// beyond the batch computes on the first tile's rows and writes nothing).
#include "common.cuh"
#include "ptx.cuh"

#include <mutex>

namespace az {
namespace {

constexpr int kK = kHeadChannels * 64;         // 2048
constexpr int kStageK = 64;
constexpr int kNumKStages = kK / kStageK;      // 32
constexpr int kOperandStageBytes = 128 * kStageK * 2;   // 16384
constexpr int kStages = 5;
constexpr int kThreads = 32 * 6;               // producer, issuer, 4 epilogue warps
#ifndef AZ_FC_PAIR_COLS
#define AZ_FC_PAIR_COLS 256
#endif
constexpr int kPairCols = AZ_FC_PAIR_COLS;       // columns of a pair's output tile (256 or 128)
constexpr int kPairRows = kPairCols / 2;        // weight rows a CTA of a pair holds per stage
constexpr int kPairBStageBytes = kPairRows * kStageK * 2;
constexpr uint32_t kTmemCols = 256;
constexpr uint32_t kSpinLimit = 1u << 24;
constexpr int kLogitPitch = kPairCols + 1;       // floats per row of the logits tile staged in shared memory

static_assert(128 * kLogitPitch * 4 <= 2 * kStages * kOperandStageBytes, "the logits tile is staged in the operand stages");
constexpr int kOffA = 0;
constexpr int kOffB = kStages * kOperandStageBytes;
constexpr int kOffBars = 2 * kStages * kOperandStageBytes;      // full[5], empty[5], peer[5], acc
constexpr int kOffTmemPtr = kOffBars + (3 * kStages + 1) * 8;
constexpr int kOffAbort = kOffTmemPtr + 4;
constexpr int kOffTail = (kOffAbort + 4 + 15) & ~15;           // value tail weights: w2[3][128], b2[3]
constexpr int kSmemBytes = kOffTail + (3 * kValueHidden + 4) * 4;

struct FcArgs {
    const __nv_bfloat16 *u_policy, *u_value;    // A tiles [m_tile][256][16][8][8]
    const __nv_bfloat16 *w_policy, *w_value;    // B tiles [n_tile][256][16][8][8] (the policy's: an even number of tiles)
    const float *b_policy, *b_value;            // [1858], [128]
    const float *w2, *b2;                       // value tail [V][128], [V]
    float *logits;                              // [batch][1858]
    float *value;                               // [batch][V]
    uint32_t *status;
    int batch, n_policy, n_policy_tiles, wdl;   // n_policy_tiles: tiles of kPairCols columns
};

__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint32_t *status) {
    return bounded_wait(bar, parity, abort_flag, status, kStatusWaitTimeout, kSpinLimit);
}
__device__ __forceinline__ bool wait_bar_cluster(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint32_t *status) {
    return bounded_wait<true>(bar, parity, abort_flag, status, kStatusWaitTimeout, kSpinLimit);
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
fc_tc_kernel(const FcArgs args) {
    extern __shared__ __align__(128) unsigned char smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = ptx::smem_addr(smem);
    // start-address field of a matrix descriptor: an offset within THIS CTA's shared memory (inside a cluster a
    // CTA's shared addresses carry its rank in high bits)
    const uint32_t desc_base = (smem_base >> 4) & 0x3FFFu;
    const uint32_t bars = smem_base + kOffBars;
    auto bar_full = [&](int s) { return bars + 8u * s; };
    auto bar_empty = [&](int s) { return bars + 8u * (kStages + s); };
    auto bar_peer = [&](int s) { return bars + 8u * (2 * kStages + s); };     // first CTA's: the second CTA's copies of stage s have landed
    const uint32_t bar_acc = bars + 8u * (3 * kStages);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + kOffAbort);
    uint32_t *tmem_ptr_smem = reinterpret_cast<uint32_t *>(smem + kOffTmemPtr);
    float *tail = reinterpret_cast<float *>(smem + kOffTail);

    const bool is_value = (int)blockIdx.y == args.n_policy_tiles;
    const bool pair = !is_value;                       // the same for both CTAs of a cluster
    const uint32_t rank = ptx::cluster_ctarank();      // along x
    const bool leader = rank == 0;
    const int m_tile = blockIdx.x;
    const bool tile_live = m_tile * 128 < args.batch;
    const int V = args.wdl ? 3 : 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { ptx::mbar_init(bar_full(s), 1); ptx::mbar_init(bar_empty(s), 1); ptx::mbar_init(bar_peer(s), 1); }
        ptx::mbar_init(bar_acc, 1);
        *abort_flag = 0;
        ptx::fence_barrier_init();
    }
    if (is_value)
        for (int i = threadIdx.x; i < V * kValueHidden + V; i += kThreads)
            tail[i] = i < V * kValueHidden ? args.w2[i] : args.b2[i - V * kValueHidden];
    if (warp == 0) {
        if (pair) { ptx::tmem_alloc_pair(ptx::smem_addr(tmem_ptr_smem), kTmemCols); ptx::tmem_relinquish_pair(); }
        else { ptx::tmem_alloc(ptx::smem_addr(tmem_ptr_smem), kTmemCols); ptx::tmem_relinquish(); }
    }
    ptx::tc_fence_before();
    __syncthreads();
    // nothing may reach into the other CTA (arrivals, commits, products that read its shared memory) before its
    // barriers exist
    ptx::cluster_arrive();
    ptx::cluster_wait();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_ptr_smem;
    // everything above overlaps the tower kernel's tail; its output (U tiles, for 73-plane heads the logits)
    // is read only below
    ptx::grid_dependency_wait();
    ptx::launch_dependents();

    if (warp == 0) {
        // ---- producer: two 16 KB bulk copies per stage: this CTA's 128 rows of A, and 128 rows of B (pair: the weight
        // rows of this CTA's half of the 256 columns)
        const int a_tile = tile_live ? m_tile : 0;
        const int b_tile = is_value ? 0 : 2 * (int)blockIdx.y + (int)rank;      // (the policy's tiles: kPairRows rows each)
        const uint32_t b_bytes = is_value ? (uint32_t)kOperandStageBytes : (uint32_t)kPairBStageBytes;
        const unsigned char *a_src = reinterpret_cast<const unsigned char *>(is_value ? args.u_value : args.u_policy) +
                                     (size_t)a_tile * (kK * 128 * 2);
        const unsigned char *b_src = reinterpret_cast<const unsigned char *>(is_value ? args.w_value : args.w_policy) +
                                     (size_t)b_tile * ((size_t)kK * (is_value ? 128 : kPairRows) * 2);
        bool ok = true;
        int issued = 0;
        for (int ks = 0; ks < kNumKStages; ++ks) {
            const int s = ks % kStages;
            ok = wait_bar(bar_empty(s), ((ks / kStages) & 1) ^ 1u, abort_flag, args.status);
            if (!ok) break;
            if (lane == 0) {
                ptx::mbar_arrive_expect_tx(bar_full(s), (uint32_t)kOperandStageBytes + b_bytes);
                ptx::bulk_copy_g2s(smem_base + kOffA + s * kOperandStageBytes, a_src + (size_t)ks * kOperandStageBytes, kOperandStageBytes, bar_full(s));
                ptx::bulk_copy_g2s(smem_base + kOffB + s * kOperandStageBytes, b_src + (size_t)ks * b_bytes, b_bytes, bar_full(s));
            }
            issued = ks + 1;
            __syncwarp();
        }
        if (!ok)   // let copies in flight land before the shared memory is released
            for (int ks = issued > kStages ? issued - kStages : 0; ks < issued; ++ks)
                for (uint32_t i = 0; i < (1u << 20); ++i)
                    if (ptx::mbar_try_wait(bar_full(ks % kStages), (ks / kStages) & 1)) break;
    } else if (warp == 1 && pair && !leader) {
        // ---- pair, second CTA: no products are issued here; tell the first CTA when a stage's copies have landed
        // (they signal a barrier of this CTA, and a barrier can be waited on only by its own CTA)
        bool ok = true;
        for (int ks = 0; ks < kNumKStages && ok; ++ks) {
            const int s = ks % kStages;
            ok = wait_bar(bar_full(s), (ks / kStages) & 1, abort_flag, args.status);
            if (!ok) break;
            // (relaxed: this thread publishes no writes of its own; the copies were written by the bulk-copy engine and
            // are read by this CTA's own tensor core, and a releasing cluster-scope arrival costs about a thousand cycles)
            if (lane == 0) ptx::mbar_arrive_cluster_relaxed(ptx::map_to_cta(bar_peer(s), 0));
            __syncwarp();
        }
    } else if (warp == 1) {
        // ---- MMA issuer: four K=16 steps per stage
        constexpr uint32_t idesc_solo = ptx::idesc_bf16_f32(128, 128), idesc_pair = ptx::idesc_bf16_f32(256, kPairCols);
        constexpr uint32_t lbo_pair = (uint32_t)(kPairRows * 16 >> 4) << 16;   // the pair's B: K core matrices kPairRows x 16 bytes apart
        constexpr uint32_t desc_hi = (uint32_t)(128 >> 4) | (1u << 14);        // 8-row groups 128 B apart
        constexpr uint32_t lbo = (uint32_t)(2048 >> 4) << 16;                  // K core matrices 2048 B apart
        const uint32_t elected = ptx::elect_one();
        bool ok = true;
        for (int ks = 0; ks < kNumKStages && ok; ++ks) {
            const int s = ks % kStages;
            ok = wait_bar(bar_full(s), (ks / kStages) & 1, abort_flag, args.status);
            if (ok && pair) ok = wait_bar_cluster(bar_peer(s), (ks / kStages) & 1, abort_flag, args.status);
            if (!ok) break;
            ptx::tc_fence_after();
            const uint32_t a_lo = (desc_base + (uint32_t)((kOffA + s * kOperandStageBytes) >> 4)) | lbo;
            const uint32_t b_lo = (desc_base + (uint32_t)((kOffB + s * kOperandStageBytes) >> 4)) | (pair ? lbo_pair : lbo);
            if (pair) {
#pragma unroll
                for (int j = 0; j < kStageK / 16; ++j)
                    ptx::mma_bf16_elect_pair(tmem_base, a_lo + (uint32_t)(j * 256), desc_hi, b_lo + (uint32_t)(j * 2 * kPairRows), desc_hi, idesc_pair,
                                             (ks > 0 || j > 0) ? 1u : 0u, elected);
            } else {
#pragma unroll
                for (int j = 0; j < kStageK / 16; ++j)
                    ptx::mma_bf16_elect(tmem_base, a_lo + (uint32_t)(j * 256), desc_hi, b_lo + (uint32_t)(j * 256), desc_hi, idesc_solo,
                                        (ks > 0 || j > 0) ? 1u : 0u, elected);
            }
            if (elected) {
                if (pair) { ptx::mma_commit_pair(bar_empty(s)); if (ks == kNumKStages - 1) ptx::mma_commit_pair(bar_acc); }
                else { ptx::mma_commit(bar_empty(s)); if (ks == kNumKStages - 1) ptx::mma_commit(bar_acc); }
            }
            __syncwarp();
        }
        if (!ok && elected) { if (pair) ptx::mma_commit_pair(bar_acc); else ptx::mma_commit(bar_acc); }   // lets the epilogues' bounded waits end early
        __syncwarp();
    } else {
        // ---- epilogue: this CTA's 128 rows; pair: 256 columns, value: 128
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const int m = m_tile * 128 + row;
        const bool live = tile_live && m < args.batch;
        const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
        bool ok = wait_bar(bar_acc, 0, abort_flag, args.status);
        ptx::tc_fence_after();
        float z[3] = {0.0f, 0.0f, 0.0f};
        if (ok) {
            const int n_chunks = is_value ? 8 : kPairCols / 16;
#pragma unroll 1
            for (int j = 0; j < n_chunks; ++j) {
                uint32_t r[16];
                ptx::tmem_ld16(t_lane + (uint32_t)(j * 16), r);
                ptx::tmem_ld_wait();
                if (is_value) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int n = j * 16 + i;
                        const float h = fmaxf(__uint_as_float(r[i]) + __ldg(args.b_value + n), 0.0f);
                        z[0] = fmaf(tail[n], h, z[0]);
                        if (V == 3) { z[1] = fmaf(tail[kValueHidden + n], h, z[1]); z[2] = fmaf(tail[2 * kValueHidden + n], h, z[2]); }
                    }
                } else {
                    // logits: through shared memory, so that they leave as whole rows.  (A thread holds one ROW of the
                    // tile; stored from here, every store instruction of a warp would touch 32 rows, 32 transactions:
                    // measured 33,000 cycles for the tile, more than the products take.)  The operand stages are free: all
                    // products have completed.  Pitch 257: lanes of a warp, one row each, fall into different banks.
                    float *stage = reinterpret_cast<float *>(smem);
#pragma unroll
                    for (int i = 0; i < 16; ++i) stage[row * kLogitPitch + j * 16 + i] = __uint_as_float(r[i]);
                }
            }
        }
        // (every epilogue warp comes here, whatever its wait returned: the four meet at a hardware barrier)
        if (!is_value) asm volatile("bar.sync 1, 128;" ::: "memory");
        if (ok) {
            if (!is_value) {
                const float *stage = reinterpret_cast<const float *>(smem);
                const int n0 = (int)blockIdx.y * kPairCols + lane;
                float bias[kPairCols / 32];
#pragma unroll
                for (int k = 0; k < kPairCols / 32; ++k) bias[k] = n0 + 32 * k < args.n_policy ? __ldg(args.b_policy + n0 + 32 * k) : 0.0f;
                // warp q writes rows q, q + 4, ...: a store instruction covers 32 consecutive logits of one row
                for (int rr = q; rr < 128; rr += 4) {
                    const int mm = m_tile * 128 + rr;
                    if (!tile_live || mm >= args.batch) break;
                    float *dst = args.logits + (size_t)mm * args.n_policy;
#pragma unroll
                    for (int k = 0; k < kPairCols / 32; ++k)
                        if (n0 + 32 * k < args.n_policy) dst[n0 + 32 * k] = stage[rr * kLogitPitch + lane + 32 * k] + bias[k];
                }
            }
            if (is_value && live) {
                const float *b2 = tail + V * kValueHidden;
                if (V == 1) args.value[m] = tanhf(z[0] + b2[0]);
                else {
                    const float a = z[0] + b2[0], b = z[1] + b2[1], c = z[2] + b2[2];
                    const float mx = fmaxf(a, fmaxf(b, c));
                    const float e0 = expf(a - mx), e1 = expf(b - mx), e2 = expf(c - mx);
                    const float inv = 1.0f / (e0 + e1 + e2);
                    args.value[(size_t)m * 3 + 0] = e0 * inv;
                    args.value[(size_t)m * 3 + 1] = e1 * inv;
                    args.value[(size_t)m * 3 + 2] = e2 * inv;
                }
            }
        }
    }
    ptx::tc_fence_before();
    __syncthreads();
    // neither CTA may leave (and release shared memory and TMEM that the pair's products and commits address) before
    // both are through
    ptx::cluster_arrive();
    ptx::cluster_wait();
    if (warp == 0) {
        ptx::tc_fence_after();
        if (pair) ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
        else ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace

// bytes of the packed weight tiles of an n-row matrix.  The value head's hidden layer is one tile of 128 rows; the
// policy's tiles have kPairRows rows (what one CTA of a pair holds of a kPairCols-column tile), an even number of them
size_t fc_tc_weight_bytes(int n, bool policy) {
    if (!policy) return (size_t)((n + 127) / 128) * kK * 128 * 2;
    return (size_t)(2 * ((n + kPairCols - 1) / kPairCols)) * kK * kPairRows * 2;
}

// w[n][2048] with the input flattened channel-major (channel*64 + square)  ->  tiles of `rows` rows
// [tile][8-wide K chunk (256)][row group (rows/8)][row (8)][k (8)] with K = square*32 + channel.
void fc_tc_pack_weights(const float *w, int n, bool policy, __nv_bfloat16 *packed) {
    const int rows = policy ? kPairRows : 128;
    const int tiles = (int)(fc_tc_weight_bytes(n, policy) / ((size_t)kK * rows * 2));
    __nv_bfloat16 *dst = packed;
    for (int t = 0; t < tiles; ++t)
        for (int kc8 = 0; kc8 < kK / 8; ++kc8)
            for (int ng = 0; ng < rows / 8; ++ng)
                for (int r = 0; r < 8; ++r)
                    for (int e = 0; e < 8; ++e) {
                        const int row = t * rows + ng * 8 + r, k = kc8 * 8 + e;
                        const int sq = k / kHeadChannels, c = k % kHeadChannels;
                        *dst++ = __float2bfloat16_rn(row < n ? w[(size_t)row * kK + c * 64 + sq] : 0.0f);
                    }
}

int launch_fc_tc(const Net &net, int batch, float *value_out, cudaStream_t s) {
    if (batch == 0) return AZ_OK;
    static bool configured[64] = {};
    static std::mutex configured_lock;                  // any thread may make a device's first launch
    int dev = 0;
    AZ_CUDA(cudaGetDevice(&dev));
    {
        std::lock_guard<std::mutex> hold(configured_lock);
        if (dev >= 0 && dev < 64 && !configured[dev]) {
            AZ_CUDA(cudaFuncSetAttribute(fc_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
            configured[dev] = true;
        }
    }
    const bool flat = net.arch.policy_head == AZ_POLICY_FLAT1858;
    FcArgs a;
    a.u_policy = static_cast<const __nv_bfloat16 *>(net.u_policy);
    a.u_value = static_cast<const __nv_bfloat16 *>(net.u_value);
    a.w_policy = static_cast<const __nv_bfloat16 *>(net.fc_policy_w);
    a.w_value = static_cast<const __nv_bfloat16 *>(net.fc_value_w);
    a.b_policy = net.p_fbias;
    a.b_value = net.v_b1;
    a.w2 = net.v_w2;
    a.b2 = net.v_b2;
    a.logits = net.logits;
    a.value = value_out;
    a.status = net.status_dev;
    a.batch = batch;
    a.n_policy = kFlatMoves;
    a.n_policy_tiles = flat ? (kFlatMoves + kPairCols - 1) / kPairCols : 0;
    a.wdl = net.arch.value_head == AZ_VALUE_WDL;
    const int m_tiles = (batch + 127) / 128;
    // clusters of two CTAs along x (the kernel's own attribute); started as soon as the tower kernel lets its dependents go
    const dim3 grid((unsigned)((m_tiles + 1) & ~1), (unsigned)(a.n_policy_tiles + 1));
    AZ_CUDA(launch_dependent(fc_tc_kernel, grid, dim3(kThreads), kSmemBytes, s, a));
    return AZ_OK;
}

}  // namespace az
