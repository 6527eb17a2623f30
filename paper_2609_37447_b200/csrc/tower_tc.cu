// The residual convolution tower on tcgen05 tensor cores (bf16 operands, fp32 accumulation in
// TMEM), one persistent kernel for the whole tower (Sec. 3.5 shared residual backbone; block order
// convolution, normalisation, activation, convolution, normalisation, residual addition,
// activation, Sec. 4.3.6; batch-norm folded on the deployment copy, App. D.3).
//
// Boards are independent, so a CTA takes four boards and carries them through every layer without
// leaving the SM: there is no grid-wide synchronisation and inter-layer activations never touch
// HBM.  The 3x3 convolution is an implicit GEMM, M = 128 rows (2 boards x 64 squares, a "group"),
// N = 128 output channels, K = 9 taps x input channels.
//
//  * A operand: the group's activations live in shared memory as a zero-bordered frame in the
//    no-swizzle K-major core-matrix layout: for every 8-channel slice a plane of 16-byte slots,
//    slot(y, b, x) = ((y+1)*2 + b)*9 + (x+1); slot 0 of every 9-slot strip and the strips y = -1
//    and y = 8 are never written and stay zero.  Eight consecutive GEMM rows (one board row) are
//    eight consecutive slots, row groups are 9 slots (144 B) apart, and a tap (dy, dx) is nothing
//    but a start-address offset of (dy*18 + dx) slots: the implicit GEMM moves no data.
//  * B operand: weights (batch-norm scale folded in, bf16) pre-packed on the host as ready-made
//    core-matrix tiles, streamed L2 -> shared memory by bulk async copies through a 3-stage ring;
//    one stage = 16 input channels x 9 taps x 128 outputs, shared by both groups of the CTA.
//  * D: per group 128 TMEM columns H (the fp32 residual stream) and 128 columns ACC.  conv1 writes
//    ACC; conv2 accumulates straight onto H, so the residual addition costs nothing and the
//    residual stream is never re-rounded to bf16.
//  * Epilogue (4 warps per group): bias + ReLU, fp32 back to H where needed, bf16 into the SAME
//    shared-memory frame in place (all MMAs that read it have completed), 16 channels at a time, each
//    slice handing the next layer's MMAs a "ready" mbarrier so that the tensor pipe restarts
//    after the first slice instead of after the whole epilogue.
// Warp roles: warp 0 weight producer, warps 1-2 MMA issuers of group 0 / 1, warps 3-6 / 7-10
// epilogue of group 0 / 1.  The tensor pipe does not buffer work across gaps in the issuing
// thread's instruction stream (measured: a stall of the issuer between two MMAs is pipe idle
// time), so each group has its own issuer: while one waits on its barriers the other's MMAs run.
// Every mbarrier wait is bounded; on expiry the CTA raises a status bit, stops issuing work,
// drains, frees its TMEM and exits.
#include "common.cuh"
#include "planes.cuh"
#include "ptx.cuh"

#include <cuda_fp8.h>

#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <mutex>
#include <vector>

namespace az {
namespace {

constexpr int kNB = 2;                         // boards per group (128 GEMM rows)
constexpr int kSlots = 10 * kNB * 9 + 1;       // 181 sixteen-byte slots per 8-channel plane
constexpr int kPlaneBytes = kSlots * 16;       // 2896
constexpr int kRowGroupBytes = 9 * 16;         // stride between 8-row groups (SBO)
constexpr uint32_t kTmemCols = 512;
constexpr int kMaxSmem = 232448;
// high words of the shared-memory matrix descriptors (no swizzle, K-major): stride between 8-row
// groups in bits 0-13, descriptor version 1 in bit 14; the low word carries the stride between the
// two K core matrices in bits 16-29 above the start address.
constexpr uint32_t kADescHi = (uint32_t)(kRowGroupBytes >> 4) | (1u << 14);
constexpr uint32_t kBDescHi = (uint32_t)(128 >> 4) | (1u << 14);
constexpr uint32_t kADescLbo = (uint32_t)(kPlaneBytes >> 4) << 16;
constexpr uint32_t kSpinLimit = 1u << 24;

// Shape-dependent constants.  128 channels: two groups per CTA share every weight stage (16 input
// channels x 9 taps).  256 channels: the frame and the accumulators of ONE group fill shared memory
// and TMEM, and a stage is 16 input channels x 3 taps.  160 channels (the paper's 14 x 160 network):
// one group as well (two would need 640 TMEM columns), stages of 9 taps.
// SETS: how many sets of four epilogue warps share a group's layer (each set takes a contiguous run of
// the 16-channel slices).  Two sets for the FP8 tower, whose MMAs are twice as fast as its epilogue needs.
// PAIR: two CTAs on neighbouring SMs (a cluster of two) share every MMA: M = 256 rows, 128 from each CTA's own
// frame, N = C with each CTA holding HALF of every weight tile in its own shared memory (tcgen05 .cta_group::2).
// The shared-memory pipe that bounds the 128-channel shape then carries 6 KB of operands per MMA instead of 8.
// NSPLIT > 1 (small batches of the 256-channel shape): a cluster of NSPLIT CTAs carries ONE group; each CTA computes
// C / NSPLIT of every layer's output channels from the whole input (its own copy of the frame).  Its epilogue writes the
// slices into its own frame; a warp of its own sends each finished slice on to the other CTAs' frames as one bulk copy
// through distributed shared memory, counted on the receiver's hand-off barrier; another acknowledges the slices
// received.  Each CTA walks a layer's K starting at its own slices, so the exchange overlaps its first MMAs.  A layer
// then takes 1/2 (two CTAs) or 3/8 (four: MMAs of 64 columns are bound by the operand reads, 48 cycles, not 32) of the
// tensor time.
template <int C, int GROUPS, int SETS, bool PAIR = false, int NSPLIT = 1>
struct Shape {
    static constexpr int kC = C, kGroups = GROUPS, kSets = SETS;
    static constexpr bool kPair = PAIR;
    static constexpr int kHalves = PAIR ? 2 : 1;
    static constexpr int kNSplit = NSPLIT;
    static constexpr int kN = C / NSPLIT;                            // output channels this CTA computes (TMEM columns per region)
    static constexpr int kParts = kHalves * kNSplit;                 // CTAs of a cluster that each hold one part of every weight tile
    static_assert(!(PAIR && NSPLIT > 1), "one or the other");
    static constexpr int kSlices = kC / 16;                          // 16-channel slices of a layer's output
    static constexpr int kFrameBytes = kPlaneBytes * (kC / 8);       // 46336 / 92672 per group
    static constexpr int kTileBytes = kC * 32 / kParts;              // one tap: this CTA's rows of the N = C tile x 32 bytes of K
    static constexpr int kStageTaps = (kC == 256 && NSPLIT == 1) ? 3 : 9;
    static constexpr int kStagesPerSlice = 9 / kStageTaps;
    static constexpr int kStageBytes = kStageTaps * kTileBytes;      // 36864 / 24576; pair: 18432
    static constexpr int kStages = NSPLIT == 4 ? 6 : NSPLIT > 1 ? 3 : kC == 256 ? (PAIR ? 10 : 5) : PAIR ? (SETS == 2 ? 6 : 7) : 3;     // (N-split: 108 KB of 18 / 36 KB stages)
    // pair: the second group's issuer runs this many weight stages behind the first's (half a layer), so that each
    // group's layer hand-over falls into the middle of the other's layer; the halved stages make the ring deep enough
#ifndef AZ_PAIR_LAG
#define AZ_PAIR_LAG 4
#endif
    static constexpr int kLag = PAIR ? AZ_PAIR_LAG : 0;
    static constexpr int kEpiWarps = 4 * kGroups * kSets;
    static constexpr int kThreads = 32 * (1 + kGroups + kEpiWarps + (NSPLIT > 1 ? 2 : 0));  // producer, one issuer per group, 4 epilogue warps per group and set; N-split: a warp that sends the finished slices to the other CTAs and one that acknowledges theirs
    static constexpr uint32_t kBDescLbo = (uint32_t)(kC / kParts) << 16;    // K core matrices (rows of this CTA's tile)*16 bytes apart
    static constexpr int kOffFrames = 0;
    static constexpr int kOffWeights = kGroups * kFrameBytes;
    static constexpr int kOffBars = kOffWeights + kStages * kStageBytes;
    // barriers: w_full[S], w_empty[S], acc_full[G], a_ready[G][slices], done, lead[S], pool[G], peer_full[S], peers_done[G], ack[G]
    static constexpr int kNumBars = 2 * kStages + kGroups + kGroups * kSlices + 1 + kStages + kGroups + kStages + 2 * kGroups;
    static constexpr int kOffTmemPtr = kOffBars + kNumBars * 8;
    static constexpr int kOffAbort = kOffTmemPtr + 4;
    static constexpr int kOffConst = (kOffAbort + 4 + 15) & ~15;     // per-warp copies of the current layer's channel constants
    // per epilogue warp: the current layer's channel constants for the channels of its own slices
    // after the constants: head biases (up to 256), then the pooled-context scratch of the paper's network
    // per group: partial sums and maxima [4 warps][2 boards][C/4], pooled vector [2][C/2], context [2][3C/4]
    static constexpr int kCtxStride = (3 * kC / 4 + 15) & ~15;      // context entries per board, padded with zeros to whole slices
    static constexpr int kPoolFloats = kGroups * (2 * 4 * 2 * (kC / 4) + 2 * (kC / 2) + 2 * kCtxStride);
    static constexpr int smem_bytes(bool fp8, bool pnet = false) {
        return kOffConst + kEpiWarps * (fp8 ? (pnet ? 4 : 3) : 1) * (kC / kSets) * 4 + 256 * 4 + (pnet ? kPoolFloats * 4 : 0);
    }
    // (four constant vectors per channel in the 8-bit forms, one in bf16; the 176-channel shape exists in bf16 only)
    static_assert(kOffConst + kEpiWarps * ((kC == 176 || (PAIR && SETS == 1)) ? 1 : 4) * (kC / kSets) * 4 + 1024 + (PAIR ? 0 : kPoolFloats * 4) <= kMaxSmem || kC == 256, "shared memory budget");
    static_assert(kGroups * 2 * kN <= (int)kTmemCols, "TMEM: per group N columns of residual stream and N of accumulator");
};

struct TowerArgs {
    const __nv_bfloat16 *planes;     // [batch][64][in_pad] already encoded planes, or null:
    const unsigned char *positions;  // then the boards are encoded here from their position records
    size_t position_stride;
    int in_planes;                   // 19 or 112
    const void *weights;             // packed stages
    const float *bias;               // [n_conv][C]
    __nv_bfloat16 *out;              // [batch][64][C] or null
    uint32_t *status;
    int batch;
    int n_conv;                      // 1 + 2*blocks
    int in_pad;                      // channels of the plane tensor (32 or 128)
#ifdef AZ_TRACE
    int trace;                       // diagnostic builds only: CTA 0 prints how long each role waited
#endif
    // fused 1x1 head projections (one extra MMA layer on the final activations); head_n == 0: none
    int head_n;                      // 64: flat policy proj (32) | value proj (32); 112: 73 policy planes (+7 pad) | value proj (32)
    const __nv_bfloat16 *head_w;     // packed [slice][k8 2][n-group head_n/8][8][8]
    const float *head_bias;          // [head_n]
    __nv_bfloat16 *u_policy;         // flat head: projection as GEMM A tiles, K index = square*32 + channel
    __nv_bfloat16 *u_value;          // value projection, same layout
    float *logits;                   // 73-plane head: [batch][73*64] fp32 logits, index = plane*64 + square
    // FP8 tower: per-layer channel constants [n_conv][4][C]: output scale, bias, 1/next activation
    // scale, 1/(next conv2 weight scale) for the residual stream kept in TMEM
    const float *lconst;
    // calibration run (bf16 kernel): per-layer, per-channel maximum of the layer outputs, as float bits
    unsigned int *absmax;            // [n_conv][C]
    // calibration runs (either kernel): per-layer, per-channel SUM of the pre-activation values over all squares of
    // all boards, in the kernel's own output units (real values in bf16, real x the next layer's activation scale in
    // the 8-bit forms); the host compares the two networks' means and corrects the 8-bit biases (see az_calibrate)
    double *presum;                  // [n_conv][C] or null (double: the host subtracts two nearly equal means)
    // the paper's own network (kPnet instantiation; Sec. 3.2, 4.3.3, 4.3.6, App. D.1): activations capped
    // at six, pooled context in blocks 1, 3, 5, ..., query / key projections as the fused head layer
    int split_w;                     // e4m3 tower with split operands: the weights are pairs as well (two stages per slice)
    const float *gw;                 // [pooled block][C/2][3C/4] fp32, transposed: pooled vector -> context
    float *qk_out;                   // [batch][64][256] fp32: queries (128) then keys (128) per square
};

// One round of a CTA's work: which two-board groups sit in its slots (-1 = the slot idles).
struct Round {
    int group[2];
    bool valid;
};

// Static schedule, computed identically by every warp.  G groups on P CTAs.  Full rounds give every CTA two
// groups.  What is left for the last round is spread one group per CTA if there are CTAs enough (a CTA alone
// with one group needs about 0.8 of a two-group round, measured), else paired onto as few CTAs as possible
// (measured faster than mixing one- and two-group CTAs: the round lasts as long either way and fewer busy
// SMs run at higher clocks under the power cap).
template <class S>
__device__ __forceinline__ Round get_round(int r, int cta, int P, int G) {
    Round rd;
    rd.group[0] = rd.group[1] = -1; rd.valid = false;
    if (S::kGroups == 1) {
        const int g = r * P + cta;
        if (g < G) { rd.group[0] = g; rd.valid = true; }
        return rd;
    }
    const int full = G / (2 * P), left = G - full * 2 * P, base = full * 2 * P;
    if (r < full) { rd.group[0] = r * 2 * P + 2 * cta; rd.group[1] = rd.group[0] + 1; rd.valid = true; return rd; }
    if (r > full || left == 0) return rd;
    if (left <= P) {
        if (cta < left) { rd.group[0] = base + cta; rd.valid = true; }
    } else if (2 * cta < left) {
        rd.group[0] = base + 2 * cta; rd.valid = true;
        if (2 * cta + 1 < left) rd.group[1] = base + 2 * cta + 1;
    }
    return rd;
}

// N-split: the order in which the CTA of rank `rank` walks the K slices of a layer after the input layer: first the
// out_slices slices it produced itself (they are in its frame first), then the other CTAs', their first slices, then their
// second ones, and so on, which is the order in which they arrive.  The weights are packed in the same order.
__host__ __device__ inline int nsplit_k_slice(int nsplit, int out_slices, int rank, int ki) {
    if (ki < out_slices) return rank * out_slices + ki;
    const int j = ki - out_slices, i = j / (nsplit - 1), p = (rank + 1 + j % (nsplit - 1)) % nsplit;
    return p * out_slices + i;
}

__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint32_t *status,
                                         long long *waited = nullptr) {
    return bounded_wait(bar, parity, abort_flag, status, kStatusWaitTimeout, kSpinLimit, waited);
}
// the same for a barrier that threads of the pair's other CTA arrive on (acquire at cluster scope)
__device__ __forceinline__ bool wait_bar_cluster(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint32_t *status,
                                                 long long *waited = nullptr) {
    return bounded_wait<true>(bar, parity, abort_flag, status, kStatusWaitTimeout, kSpinLimit, waited);
}

// slices of the head projection's K that travel in one weight stage (the last stage may carry fewer: eleven
// slices of the 176-channel shape go as six and five)
template <class S> __device__ __host__ constexpr int head_slices_per_stage(int head_n) {
    return S::kC == 128 ? (head_n == 256 ? 4 : S::kSlices) : S::kC == 160 ? 5 : S::kC == 176 ? 6 : (S::kNSplit == 4 ? (head_n == 64 ? 8 : 4) : S::kNSplit > 1 ? (head_n == 64 ? 16 : 8) : head_n == 64 ? 8 : 4);    // (split: stages of 18 / 36 KB)
}
template <class S> __device__ __host__ constexpr int head_stages(int head_n) {
    return head_n ? (S::kSlices + head_slices_per_stage<S>(head_n) - 1) / head_slices_per_stage<S>(head_n) : 0;
}

// kFp8: the 8-bit tower (layers after the input layer read 8-bit operands, 32 channels per MMA); with
// kInt8 those operands are unsigned 8-bit activations and signed 8-bit weights (kind::i8, int32
// accumulators, the residual stream kept as int32 in the same units), else e4m3 (kind::f8f6f4).
// kSplitA (e4m3 only): every activation travels as TWO e4m3 numbers, the rounded value and the rounded
// remainder (planes C/16 .. C/8 - 1 of the frame, which the 8-bit forms otherwise leave unused), and every weight
// stage is multiplied with both; with args.split_w the weights are pairs too (a second stage per slice holds the
// remainders, multiplied with the activations' first parts).  Three products per layer instead of one: the
// operands are still e4m3, the result carries about seven mantissa bits per operand instead of three.
template <bool kFp8, class S, bool kPnet = false, bool kInt8 = false, bool kSplitA = false>
__global__ void __launch_bounds__(S::kThreads, 1)
tower_tc_kernel(const TowerArgs args) {
    static_assert(!kInt8 || kFp8, "the int8 tower is a form of the 8-bit tower");
    static_assert(!kSplitA || (kFp8 && !kInt8 && !kPnet && S::kC == 128), "split operands exist for the e4m3 tower of the 128-channel residual networks");
    static_assert(!kPnet || S::kC == 128 || S::kC == 160 || S::kC == 176, "the paper's network runs on the 128-, 160- and 176-channel shapes");
    static_assert(S::kC != 176 || S::kSets == 1, "eleven slices do not split over two sets");
    static_assert(!(kPnet && kFp8) || kInt8, "of the 8-bit towers the int8 one carries the paper's network");
    constexpr int kC = S::kC, kGroups = S::kGroups, kStages = S::kStages, kSlices = S::kSlices;
    constexpr int kFrameBytes = S::kFrameBytes, kStageBytes = S::kStageBytes, kThreads = S::kThreads;
    static_assert(!kFp8 || kC == 128 || (kPnet && kC == 160), "the 8-bit towers exist for 128 channels and, for the paper's network, 160");
    extern __shared__ __align__(128) unsigned char smem[];
    // the warp index through a shuffle: the compiler then knows it is the same in all lanes, and role-
    // dependent address arithmetic can stay on the uniform datapath
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const uint32_t smem_base = ptx::smem_addr(smem);
    // start-address field of a shared-memory matrix descriptor: 14 bits, in 16-byte units, an offset within THIS CTA's
    // shared memory.  (Inside a cluster a CTA's shared addresses carry its rank above bit 23; left in, those bits
    // would run into the descriptor's stride field.)
    const uint32_t desc_base = (smem_base >> 4) & 0x3FFFu;
    const uint32_t bars = smem_base + S::kOffBars;
    auto bar_w_full = [&](int s) { return bars + 8u * s; };
    auto bar_w_empty = [&](int s) { return bars + 8u * (kStages + s); };
    auto bar_acc_full = [&](int g) { return bars + 8u * (2 * kStages + g); };
    auto bar_a_ready = [&](int g, int kc) { return bars + 8u * (2 * kStages + kGroups + g * kSlices + kc); };
    const uint32_t bar_done = bars + 8u * (2 * kStages + kGroups + kGroups * kSlices);
    auto bar_lead = [&](int s) { return bar_done + 8u * (1 + s); };   // group 0 has issued its MMAs on stage s
    auto bar_pool = [&](int g) { return bar_done + 8u * (1 + kStages + g); };   // the four epilogue warps of group g meet here
    auto bar_peer = [&](int s) { return bar_done + 8u * (1 + kStages + kGroups + s); };   // pair: the other CTA's half of stage s has landed
    // CTA pair: rank 0 issues every MMA of the pair; rank 1 supplies its rows, its half of the weights, its epilogue
    auto bar_pdone = [&](int g) { return bar_done + 8u * (1 + kStages + kGroups + kStages + g); };   // N-split: the other CTAs' MMAs of this layer are complete
    auto bar_ack = [&](int g) { return bar_done + 8u * (1 + kStages + kGroups + kStages + kGroups + g); };   // N-split: the other CTAs hold this CTA's slices of the layer
    constexpr bool kPair = S::kPair;
    static_assert(!kPair || !kPnet, "CTA pairs exist for the residual networks");
    constexpr int kNSplit = S::kNSplit, kN = S::kN;
    constexpr bool kCluster = kPair || kNSplit > 1;
    static_assert(kNSplit == 1 || (!kFp8 && !kPnet && kGroups == 1 && S::kSets == 1), "the N-split exists for the one-group bf16 shape of the residual networks");
    const uint32_t cta_rank = kCluster ? ptx::cluster_ctarank() : 0u;
    const bool leader = cta_rank == 0;
    constexpr int kOutSlices = kN / 16;                          // 16-channel slices of a layer's output that this CTA produces
    const int out0 = kNSplit > 1 ? (int)cta_rank * kOutSlices : 0;   // the first of them
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + S::kOffAbort);
    uint32_t *tmem_ptr_smem = reinterpret_cast<uint32_t *>(smem + S::kOffTmemPtr);
    constexpr int kVecs = kFp8 ? (kPnet ? 4 : 3) : 1;           // per layer: (scale, bias, h ratio[, cap]) or bias
    constexpr int kConstFloats = kVecs * kC;
    constexpr int kMyC = kN / S::kSets;                         // channels an epilogue warp is responsible for
    constexpr int kMyConstFloats = kVecs * kMyC;
    float *head_bias_smem = reinterpret_cast<float *>(smem + S::kOffConst) + S::kEpiWarps * kMyConstFloats;

    // ---- set-up: zero the frames (their borders stay zero for the kernel's lifetime), barriers, TMEM
    for (int i = threadIdx.x; i < kGroups * kFrameBytes / 16; i += kThreads)
        reinterpret_cast<uint4 *>(smem + S::kOffFrames)[i] = make_uint4(0, 0, 0, 0);
    for (int i = threadIdx.x; i < args.head_n; i += kThreads) head_bias_smem[i] = args.head_bias[i];
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(bar_w_full(s), 1);
            ptx::mbar_init(bar_w_empty(s), kGroups);
            ptx::mbar_init(bar_lead(s), 1);
            ptx::mbar_init(bar_peer(s), 1);
        }
        for (int g = 0; g < kGroups; ++g) {
            ptx::mbar_init(bar_acc_full(g), 1);
            ptx::mbar_init(bar_pdone(g), kNSplit > 1 ? kNSplit - 1 : 1);
            ptx::mbar_init(bar_ack(g), kNSplit > 1 ? kNSplit - 1 : 1);
            ptx::mbar_init(bar_pool(g), 4 * S::kSets);
            // (pair: the first CTA's barriers also count the other CTA's epilogue warps)
            for (int kc = 0; kc < kSlices; ++kc) ptx::mbar_init(bar_a_ready(g, kc), 4 * S::kSets * S::kHalves);
        }
        ptx::mbar_init(bar_done, kGroups);
        *abort_flag = 0;
        ptx::fence_barrier_init();
    }
    ptx::fence_proxy_async_smem();
    if (warp == 0) {
        if (kPair) { ptx::tmem_alloc_pair(ptx::smem_addr(tmem_ptr_smem), kTmemCols); ptx::tmem_relinquish_pair(); }
        else { ptx::tmem_alloc(ptx::smem_addr(tmem_ptr_smem), kTmemCols); ptx::tmem_relinquish(); }
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (kCluster) {
        // nothing may reach into the other CTA (remote arrivals, commits, stores, MMAs reading its shared memory) before
        // its barriers and frames are initialised
        ptx::cluster_arrive();
        ptx::cluster_wait();
    }
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_ptr_smem;
    // the head kernel that follows may set itself up on idle SMs; it waits for this grid before reading
    ptx::launch_dependents();

    // pair: the schedule deals out PAIRS of groups (four boards) to pairs of CTAs; the CTA of rank r takes the r-th
    // group of each (a group beyond the batch runs on dead boards and writes nothing)
    const int n_groups = kPair ? ((args.batch + kNB - 1) / kNB + 1) / 2 : (args.batch + kNB - 1) / kNB;
    const int n_conv = args.n_conv;
    const int head_n = args.head_n;
    const int in_slices = args.in_pad / 16;
    const int hsps = head_slices_per_stage<S>(head_n);
    // the paper's network: the first convolution of blocks 1, 3, 5, ... (layers 3, 7, 11, ...) feeds the pooled
    // context, and the second convolution of those blocks (layers 4, 8, 12, ...) reads 3C/4 channels only
    auto pool_layer = [&](int l) { return kPnet && (l & 3) == 3; };
    auto short_layer = [&](int l) { return kPnet && l >= 4 && (l & 3) == 0; };
    constexpr int kShortSlices = (3 * kC / 4 + 15) / 16;      // slices that hold the 3C/4 channels a pooled block hands on
    auto round_of = [&](int r) { return get_round<S>(r, (int)blockIdx.x / S::kParts, (int)gridDim.x / S::kParts, n_groups); };
    auto my_group = [&](const Round &rd, int g) { return kPair ? 2 * rd.group[g] + (int)cta_rank : rd.group[g]; };   // valid when rd.group[g] >= 0
    auto slices_of = [&](int l) {                                                               // K per MMA: 16 bf16 or 32 e4m3
        return l == 0 ? in_slices : short_layer(l) ? (kFp8 ? kShortSlices / 2 : kShortSlices) : (kFp8 ? kC / 32 : kC / 16);
    };
    // weight stages of layer l: per slice three 3-tap stages in the 256-channel shape, else one; twice that where
    // the weights of an e4m3 layer come as pairs
    auto stages_of = [&](int l) { return slices_of(l) * S::kStagesPerSlice * ((kSplitA && l > 0 && args.split_w) ? 2 : 1); };
    // role tracing (clocks spent waiting, printed by CTA 0) exists in diagnostic builds only (-DAZ_TRACE)
#ifdef AZ_TRACE
    const bool tr = args.trace && blockIdx.x == 0;
#else
    constexpr bool tr = false;
#endif
    long long t_wait[3] = {0, 0, 0};
    long long t_issue = 0;
    const long long t_begin = tr ? clock64() : 0;

    if (warp == 0) {
        // ================= weight producer =================
        int stage = 0;
        uint32_t phase = 0;
        uint32_t last_parity[kStages] = {};
        bool issued[kStages] = {};
        bool ok = true;
        for (int r = 0; ok; ++r) {
            const Round rd = round_of(r);
            if (!rd.valid) break;
            int n_stages = 0;
            for (int l = 0; l < n_conv; ++l) n_stages += stages_of(l);
            const int n_head_stages = head_stages<S>(head_n);
            // N-split (few CTAs, each waiting on its own stream of weights): ask L2 for every stage one layer before it
            // is copied, so that the copy's latency is L2's, not DRAM's
            constexpr int kAhead = kSlices * S::kStagesPerSlice;
            auto stage_src = [&](int st_) { return reinterpret_cast<const unsigned char *>(args.weights) + ((size_t)st_ * S::kParts + cta_rank) * kStageBytes; };
            if (kNSplit > 1 && lane == 0)
                for (int st = 0; st < kAhead && st < n_stages; ++st) ptx::bulk_prefetch_l2(stage_src(st), (uint32_t)kStageBytes);
            for (int st = 0; st < n_stages + n_head_stages && ok; ++st) {
                if (kNSplit > 1 && lane == 0 && st + kAhead < n_stages) ptx::bulk_prefetch_l2(stage_src(st + kAhead), (uint32_t)kStageBytes);
                // tower stages are contiguous and equally sized; the head projections follow as small stages of their own
                const bool head = st >= n_stages;
                // (pair: every stage is stored as this CTA's half, then the other's)
                const int head_left = kSlices - (st - n_stages) * hsps;         // slices the head still has to fetch
                const uint32_t bytes = head ? (uint32_t)((head_left < hsps ? head_left : hsps) * head_n * 32 / S::kHalves) : (uint32_t)kStageBytes;
                const unsigned char *src = head ? reinterpret_cast<const unsigned char *>(args.head_w) + (size_t)(st - n_stages) * hsps * head_n * 32 + (S::kHalves > 1 ? (size_t)cta_rank * bytes : (size_t)0)
                                                : reinterpret_cast<const unsigned char *>(args.weights) + ((size_t)st * S::kParts + cta_rank) * kStageBytes;
                ok = wait_bar(bar_w_empty(stage), phase ^ 1u, abort_flag, args.status, tr ? &t_wait[0] : nullptr);
                if (!ok) break;
                if (lane == 0) {
                    ptx::mbar_arrive_expect_tx(bar_w_full(stage), bytes);
                    ptx::bulk_copy_g2s(smem_base + S::kOffWeights + stage * kStageBytes, src, bytes, bar_w_full(stage));
                }
                issued[stage] = true; last_parity[stage] = phase;
                if (++stage == kStages) { stage = 0; phase ^= 1u; }
                __syncwarp();
            }
        }
        if (!ok) {
            // copies already in flight must land before the CTA's shared memory is released
            for (int s = 0; s < kStages; ++s)
                if (issued[s])
                    for (uint32_t i = 0; i < (1u << 20); ++i)
                        if (ptx::mbar_try_wait(bar_w_full(s), last_parity[s])) break;
        }
    } else if (warp <= kGroups) {
        if (kPair && !leader) {
            // ================= pair, second CTA: no MMAs are issued here =================
            // Warp 1 tells the first CTA's issuers when this CTA's half of a weight stage has landed (its bulk copies
            // signal a barrier of this CTA; a barrier can only be waited on by its own CTA).  Then it waits for the
            // pair's last MMAs, which also write this CTA's TMEM.
            if (warp == 1) {
                int stage = 0;
                uint32_t phase = 0;
                bool ok = true;
                for (int r = 0; ok; ++r) {
                    const Round rd = round_of(r);
                    if (!rd.valid) break;
                    int n_stages = head_stages<S>(head_n);
                    for (int l = 0; l < n_conv; ++l) n_stages += stages_of(l);
                    for (int st = 0; st < n_stages && ok; ++st) {
                        ok = wait_bar(bar_w_full(stage), phase, abort_flag, args.status);
                        if (!ok) break;
                        if (lane == 0) ptx::mbar_arrive_cluster_relaxed(ptx::map_to_cta(bar_peer(stage), 0));   // (the copies were written by the bulk-copy engine; this thread publishes nothing of its own)
                        __syncwarp();
                        if (++stage == kStages) { stage = 0; phase ^= 1u; }
                    }
                }
                for (uint32_t i = 0; i < (1u << 22); ++i)
                    if (ptx::mbar_try_wait_cluster(bar_done, 0)) break;
            }
        } else {
        // ================= MMA issuer of group g =================
        const int g = warp - 1;
        constexpr uint32_t idesc = ptx::idesc_bf16_f32(128 * S::kHalves, kN);
        // a weight stage is ready when this CTA's copy has landed and, in a pair, the other CTA's half as well
        auto wait_stage = [&](int st_, uint32_t ph_, long long *w_) -> bool {
            bool k_ = wait_bar(bar_w_full(st_), ph_, abort_flag, args.status, w_);
            if (kPair && k_) k_ = wait_bar_cluster(bar_peer(st_), ph_, abort_flag, args.status, w_);
            return k_;
        };
        // barrier(s) that arrive when the MMAs issued so far have completed: this CTA's, in a pair both CTAs'
        auto commit = [&](uint32_t bar_) { if (kPair) ptx::mma_commit_pair(bar_); else ptx::mma_commit(bar_); };
        constexpr uint32_t idesc8 = kInt8 ? ptx::idesc_u8s8_s32(128 * S::kHalves, kN) : ptx::idesc_e4m3_f32(128 * S::kHalves, kN);
        int stage = 0;
        uint32_t phase = 0;
        uint32_t a_phase = 0;
        bool ok = true;
        const uint32_t d_h = tmem_base + (uint32_t)(g * 2 * kN);
        const uint32_t frame_lo = (desc_base + (uint32_t)((S::kOffFrames + g * kFrameBytes) >> 4) + (uint32_t)(kNB * 9 + 1)) | kADescLbo;
        // The two issuers take strict turns on every weight stage: group 1 issues its MMAs on a stage
        // only after group 0 has issued its own (bar_lead).  While one issuer sits in its barrier round
        // trips the other's MMAs keep the tensor pipe busy, and the groups reach their layer boundaries
        // one stage apart instead of together.
        const bool follow = kGroups == 2 && g == 1;
        const bool lead = kGroups == 2 && g == 0;
        const uint32_t elected = ptx::elect_one();              // the lane that issues; the warp stays converged
        // group 1 issues on stage number i (counted over the whole launch) once group 0 has issued on stage
        // min(i + kLag, last stage of i's layer): it trails by kLag stages through the first part of a layer and catches
        // up to the layer's end while group 0 sits in its layer hand-over, so that each group's hand-over is covered by
        // the other's MMAs (kLag == 0: strict turns on every stage)
        int gi = 0, layer_last = 0;
        auto wait_lead = [&](long long *w_) -> bool {
            const int j = gi + S::kLag < layer_last ? gi + S::kLag : (gi > layer_last ? gi : layer_last);
            return wait_bar(bar_lead(j % kStages), (uint32_t)(j / kStages) & 1u, abort_flag, args.status, w_);
        };
        for (int r = 0; ok; ++r) {
            const Round rd = round_of(r);
            if (!rd.valid) break;
            if ((g == 0 ? rd.group[0] : rd.group[1]) < 0) {
                // a slot without a group this round still takes part in the ring protocol: it waits for
                // every stage of the round and releases it without issuing anything
                int n_stages = head_stages<S>(head_n);
                for (int l = 0; l < n_conv; ++l) n_stages += stages_of(l);
                for (int st = 0; st < n_stages && ok; ++st) {
                    layer_last = gi;
                    ok = wait_stage(stage, phase, nullptr);
                    if (ok && follow) ok = wait_lead(nullptr);
                    if (!ok) break;
                    if (lane == 0) {
                        if (kPair) {      // (relaxed: nothing is published, the slot merely does not need the stage)
                            ptx::mbar_arrive_cluster_relaxed(ptx::map_to_cta(bar_w_empty(stage), 0));
                            ptx::mbar_arrive_cluster_relaxed(ptx::map_to_cta(bar_w_empty(stage), 1));
                        } else ptx::mbar_arrive(bar_w_empty(stage));
                        if (lead) ptx::mbar_arrive(bar_lead(stage));
                    }
                    __syncwarp();
                    ++gi;
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
                continue;
            }
            for (int l = 0; l < n_conv && ok; ++l) {
                const int nkc = slices_of(l);
                const bool e4m3 = kFp8 && l > 0;                       // the input layer stays bf16
                const bool conv2 = l >= 2 && (l & 1) == 0;             // accumulates onto the residual stream
                const uint32_t d = d_h + (((l & 1) == 1) ? (uint32_t)kN : 0u);   // conv1 writes the ACC columns
                layer_last = gi + stages_of(l) - 1;
                for (int ki = 0; ki < nkc && ok; ++ki) {
                    // N-split: a CTA walks a layer's K starting at the slices it produced itself (the other CTAs' arrive
                    // while these are being multiplied); its weights are packed in that order
                    const int kc = (kNSplit > 1 && l > 0) ? nsplit_k_slice(kNSplit, kOutSlices, (int)cta_rank, ki) : ki;
                    // one group per CTA: the slice's first weight stage is normally there long before its activations;
                    // looking at it first leaves nothing between the activations' arrival and the first MMA
                    if (kGroups == 1) {
                        ok = wait_stage(stage, phase, tr ? &t_wait[0] : nullptr);
                        if (!ok) break;
                    }
                    ok = kPair ? wait_bar_cluster(bar_a_ready(g, kc), (a_phase >> kc) & 1u, abort_flag, args.status, tr ? &t_wait[1] : nullptr)
                                  : wait_bar(bar_a_ready(g, kc), (a_phase >> kc) & 1u, abort_flag, args.status, tr ? &t_wait[1] : nullptr);
                    if (!ok) break;
                    a_phase ^= 1u << kc;
                    // low descriptor word in 16-byte units; row m = 0 sits at slot 2*9 + 1 = 19
                    const uint32_t a_lo = frame_lo + (uint32_t)(2 * kc * kSlots);
                    const int n_parts = (kSplitA && e4m3 && args.split_w) ? 2 : 1;      // weight pairs: first parts, then remainders
#pragma unroll 1
                    for (int part = 0; part < n_parts && ok; ++part) {
#pragma unroll
                    for (int st = 0; st < S::kStagesPerSlice; ++st) {
                        if (kGroups > 1 || st > 0 || part > 0) {
                            ok = wait_stage(stage, phase, tr ? &t_wait[0] : nullptr);
                            if (!ok) break;
                            if (follow) {
                                ok = wait_lead(tr ? &t_wait[2] : nullptr);
                                if (!ok) break;
                            }
                        }
                        ptx::tc_fence_after();
                        const long long ti0 = tr ? clock64() : 0;
                        {
                            const uint32_t b_lo = (desc_base + (uint32_t)((S::kOffWeights + stage * kStageBytes) >> 4)) | S::kBDescLbo;
                            // the operand type is chosen once per stage: a branch between consecutive MMAs
                            // costs more than the MMA itself takes on the tensor pipe
                            if (e4m3) {
#pragma unroll
                                for (int t = 0; t < S::kStageTaps; ++t) {
                                    const int tap = st * S::kStageTaps + t;
                                    const int dy = tap / 3 - 1, dx = tap % 3 - 1;
                                    const uint32_t first = (tap == 0 && !conv2 && ki == 0 && part == 0) ? 0u : 1u;
                                    const uint32_t a_t = a_lo + (uint32_t)(dy * kNB * 9 + dx), b_t = b_lo + (uint32_t)(t * (S::kTileBytes / 16));
                                    if (kInt8) {
                                        if (kPair) ptx::mma_i8_elect_pair(d, a_t, kADescHi, b_t, kBDescHi, idesc8, first, elected);
                                        else ptx::mma_i8_elect(d, a_t, kADescHi, b_t, kBDescHi, idesc8, first, elected);
                                    } else {
                                        if (kPair) ptx::mma_e4m3_elect_pair(d, a_t, kADescHi, b_t, kBDescHi, idesc8, first, elected);
                                        else ptx::mma_e4m3_elect(d, a_t, kADescHi, b_t, kBDescHi, idesc8, first, elected);
                                    }
                                    // the activations' remainders against the same weights (first parts of the weights only:
                                    // remainder times remainder is below what fp32 accumulation keeps anyway)
                                    if (kSplitA && part == 0) {
                                        if (kPair) ptx::mma_e4m3_elect_pair(d, a_t + (uint32_t)((kC / 16) * kSlots), kADescHi, b_t, kBDescHi, idesc8, 1u, elected);
                                        else ptx::mma_e4m3_elect(d, a_t + (uint32_t)((kC / 16) * kSlots), kADescHi, b_t, kBDescHi, idesc8, 1u, elected);
                                    }
                                }
                            } else {
#pragma unroll
                                for (int t = 0; t < S::kStageTaps; ++t) {
                                    const int tap = st * S::kStageTaps + t;
                                    const int dy = tap / 3 - 1, dx = tap % 3 - 1;
                                    if (kPair)
                                        ptx::mma_bf16_elect_pair(d, a_lo + (uint32_t)(dy * kNB * 9 + dx), kADescHi,
                                                                 b_lo + (uint32_t)(t * (S::kTileBytes / 16)), kBDescHi, idesc,
                                                                 (tap == 0 && !conv2 && ki == 0) ? 0u : 1u, elected);
                                    else
                                        ptx::mma_bf16_elect(d, a_lo + (uint32_t)(dy * kNB * 9 + dx), kADescHi,
                                                            b_lo + (uint32_t)(t * (S::kTileBytes / 16)), kBDescHi, idesc,
                                                            (tap == 0 && !conv2 && ki == 0) ? 0u : 1u, elected);
                                }
                            }
                            if (elected) {
                                if (ki == nkc - 1 && st == S::kStagesPerSlice - 1 && part == n_parts - 1) commit(bar_acc_full(g));
                                commit(bar_w_empty(stage));
                                if (lead) ptx::mbar_arrive(bar_lead(stage));
                            }
                        }
                        __syncwarp();
                        if (tr) t_issue += clock64() - ti0;
                        ++gi;
                        if (++stage == kStages) { stage = 0; phase ^= 1u; }
                    }
                    }
                }
            }
            if (head_n && ok) {
                // head projections: a 1x1 convolution = the centre tap only, N = head_n, into the ACC columns
                const uint32_t idesc_h = ptx::idesc_bf16_f32(128 * S::kHalves, head_n);
                layer_last = gi + head_stages<S>(head_n) - 1;
                if (kPnet) {
                    // 256 output columns = the residual stream's columns and the accumulator's: the last
                    // layer's epilogue must have read all of them before the first MMA overwrites any
                    for (int kc = 0; kc < kSlices && ok; ++kc) {
                        ok = wait_bar(bar_a_ready(g, kc), (a_phase >> kc) & 1u, abort_flag, args.status, tr ? &t_wait[1] : nullptr);
                        a_phase ^= 1u << kc;
                    }
                    if (!ok) break;
                }
                for (int kc = 0; kc < kSlices && ok; ++kc) {
                    if (kc % hsps == 0) {
                        ok = wait_stage(stage, phase, tr ? &t_wait[0] : nullptr);
                        if (!ok) break;
                        if (follow) {
                            ok = wait_lead(tr ? &t_wait[2] : nullptr);
                            if (!ok) break;
                        }
                    }
                    if (!kPnet) {
                        ok = kPair ? wait_bar_cluster(bar_a_ready(g, kc), (a_phase >> kc) & 1u, abort_flag, args.status, tr ? &t_wait[1] : nullptr)
                                      : wait_bar(bar_a_ready(g, kc), (a_phase >> kc) & 1u, abort_flag, args.status, tr ? &t_wait[1] : nullptr);
                        if (!ok) break;
                        a_phase ^= 1u << kc;
                    }
                    ptx::tc_fence_after();
                    const bool stage_done = (kc % hsps) == hsps - 1 || kc == kSlices - 1;
                    {
                        const uint32_t a_lo = frame_lo + (uint32_t)(2 * kc * kSlots);
                        // (pair: this CTA's half of the head tile, head_n / 2 rows)
                        const uint32_t b_lo = (desc_base + (uint32_t)((S::kOffWeights + stage * kStageBytes) >> 4) + (uint32_t)((kc % hsps) * head_n * 2 / S::kHalves)) |
                                              ((uint32_t)(head_n / S::kHalves) << 16);          // K core matrices rows*16 bytes apart
                        if (kPair) ptx::mma_bf16_elect_pair(d_h + (uint32_t)kC, a_lo, kADescHi, b_lo, kBDescHi, idesc_h, kc > 0 ? 1u : 0u, elected);
                        else ptx::mma_bf16_elect(d_h + (kPnet ? 0u : (uint32_t)kN), a_lo, kADescHi, b_lo, kBDescHi, idesc_h, kc > 0 ? 1u : 0u, elected);
                    }
                    if (elected) {
                        if (kc == kSlices - 1) commit(bar_acc_full(g));
                        if (stage_done) {
                            commit(bar_w_empty(stage));
                            if (lead) ptx::mbar_arrive(bar_lead(stage));
                        }
                    }
                    __syncwarp();
                    if (stage_done) {
                        ++gi;
                        if (++stage == kStages) { stage = 0; phase ^= 1u; }
                    }
                }
            }
        }
        // all issued MMAs must have completed before TMEM is freed
        if (elected) commit(bar_done);
        __syncwarp();
        for (uint32_t i = 0; i < (1u << 22); ++i)
            if (ptx::mbar_try_wait(bar_done, 0)) break;
        }
    } else if (kNSplit > 1 && warp == 1 + kGroups + S::kEpiWarps) {
        // ================= N-split: the finished slices of this CTA -> the other CTAs' frames =================
        // A slice (two planes of the frame, 5792 contiguous bytes, borders included: they are zero everywhere) goes out as
        // one bulk copy per receiving CTA once the four epilogue warps have handed it off here; its bytes count on the
        // RECEIVER's hand-off barrier of the slice, on which four lanes arrive for the four warps that barrier expects.
        // A layer's slices go out only after every receiver's MMAs of that layer, which read the frames the copies land
        // in, are complete (bar_pdone: each CTA's epilogue announces its own completion to the others).
        constexpr uint32_t kSliceBytes = 2 * kPlaneBytes;
        const uint32_t frame_addr = smem_base + S::kOffFrames;
        uint32_t s_phase = 0, pdone_phase = 0, acc_phase = 0;
        bool ok = true;
        for (int r = 0; ok; ++r) {
            const Round rd = round_of(r);
            if (!rd.valid) break;
            // hand-offs of a round: the input planes (not sent: every CTA encodes its own copy), then every layer
            for (int h = 0; h <= n_conv && ok; ++h) {
                if (h > 0) {
                    // this CTA's MMAs of the layer are complete: the other CTAs may send their slices into its frame.  (Said
                    // from here, not from the epilogue, whose warps are on the layer's critical path.)
                    ok = wait_bar(bar_acc_full(0), acc_phase, abort_flag, args.status);
                    acc_phase ^= 1u;
                    if (!ok) break;
                    if (lane == 0) {
#pragma unroll
                        for (int p = 0; p < kNSplit; ++p)
                            if (p != (int)cta_rank) ptx::mbar_arrive_cluster_relaxed(ptx::map_to_cta(bar_pdone(0), (uint32_t)p));
                    }
                    __syncwarp();
                    ok = wait_bar_cluster(bar_pdone(0), pdone_phase, abort_flag, args.status);
                    pdone_phase ^= 1u;
                    if (!ok || (h == n_conv && head_n == 0)) break;         // the last layer's output is read again only by the heads
                }
                for (int kl = 0; kl < kOutSlices && ok; ++kl) {
                    const int kc = out0 + kl;
                    if (h == 0 && kc >= in_slices) continue;                // the input planes fill the first in_slices slices only
                    ok = wait_bar(bar_a_ready(0, kc), (s_phase >> kl) & 1u, abort_flag, args.status);
                    if (!ok) break;
                    s_phase ^= 1u << kl;
                    if (h == 0) continue;
#pragma unroll
                    for (int p = 0; p < kNSplit; ++p)
                        if (p != (int)cta_rank) {
                            const uint32_t rbar = ptx::map_to_cta(bar_a_ready(0, kc), (uint32_t)p);
                            if (lane < 4) ptx::mbar_arrive_expect_tx_cluster(rbar, kSliceBytes / 4);
                            if (lane == 0)
                                ptx::bulk_copy_s2s(ptx::map_to_cta(frame_addr + (uint32_t)(2 * kc) * kPlaneBytes, (uint32_t)p),
                                                   frame_addr + (uint32_t)(2 * kc) * kPlaneBytes, kSliceBytes, rbar);
                        }
                    __syncwarp();
                }
            }
            if (ok && head_n != 0) {                                        // (the head projections complete a phase of their own)
                ok = wait_bar(bar_acc_full(0), acc_phase, abort_flag, args.status);
                acc_phase ^= 1u;
            }
        }
    } else if (kNSplit > 1 && warp == 2 + kGroups + S::kEpiWarps) {
        // ================= N-split: acknowledge the other CTAs' slices =================
        // The copies that bring a slice here read the SENDER's frame asynchronously; the sender may overwrite those planes
        // (its epilogue of the next layer) only when the copies are done.  Their completion is visible here, on the slice's
        // hand-off barrier: once all slices of a sender's layer have landed, tell the sender (bar_ack there).
        uint32_t k_phase = 0;
        bool ok = true;
        for (int r = 0; ok; ++r) {
            const Round rd = round_of(r);
            if (!rd.valid) break;
            const int n_sent = head_n != 0 ? n_conv : n_conv - 1;
            for (int h = 0; h <= n_sent && ok; ++h)
                for (int pi = 1; pi < kNSplit && ok; ++pi) {
                    const int p = ((int)cta_rank + pi) % kNSplit;
                    for (int kl = 0; kl < kOutSlices && ok; ++kl) {
                        const int kc = p * kOutSlices + kl;
                        if (h == 0 && kc >= in_slices) continue;
                        ok = wait_bar(bar_a_ready(0, kc), (k_phase >> kc) & 1u, abort_flag, args.status);
                        k_phase ^= 1u << kc;
                    }
                    if (ok && h > 0 && lane == 0) ptx::mbar_arrive_cluster_relaxed(ptx::map_to_cta(bar_ack(0), (uint32_t)p));
                    __syncwarp();
                }
        }
    } else {
        // ================= epilogue: 4 warps per group and set =================
        // A set's last hand-off of a layer comes after its TMEM loads and stores of that layer have
        // completed, and every later writer of those columns (an MMA two layers on) is gated, through the
        // accumulator barrier of the layer between, by the hand-offs of ALL sets.
        const int ew = warp - 1 - kGroups;                    // 0 .. 4*groups*sets-1
        const int g = ew / (4 * S::kSets);
        // this warp's share of every layer: the slices kc = ks * sets + set.  Interleaved, so that with two
        // sets the two slices of the next layer's first 32-channel e4m3 step are produced side by side.
        const int set = (ew >> 2) % S::kSets;
        constexpr int kMySlices = kOutSlices / S::kSets;
        const int q = warp & 3;                               // TMEM lane quarter this warp may access
        const int m = q * 32 + lane;                          // GEMM row = TMEM lane
        const int g8 = m >> 3, y = g8 >> 1, b = g8 & 1, x = m & 7;
        const int slot = (g8 + kNB) * 9 + x + 1;
        unsigned char *frame = smem + S::kOffFrames + g * kFrameBytes;
        const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(g * 2 * kN);
        float *lc = reinterpret_cast<float *>(smem + S::kOffConst) + ew * kMyConstFloats;   // this warp's copy of the layer constants
        // pooled-context scratch of this group (paper's network only)
        constexpr int kPoolC = kC / 4, kRegC = kC - kC / 4;
        float *pool_part = head_bias_smem + 256 + g * (S::kPoolFloats / kGroups);   // [sum|max][warp q][board][kPoolC]
        float *pool_vec = pool_part + 2 * 4 * 2 * kPoolC;                          // [board][2 * kPoolC]: means, then maxima
        float *pool_ctx = pool_vec + 2 * 2 * kPoolC;                               // [board][kCtxStride], zero beyond kRegC
        constexpr int kCtxStride = S::kCtxStride;
        uint32_t pool_phase = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        // hand-off of a slice to the issuer: a barrier of this CTA; in a pair the first CTA's (which counts both CTAs'
        // warps).  With the N-split this hands off the CTA's OWN copy of the slice, to its issuer and to the warp that
        // sends it on to the other CTAs.
        auto ready = [&](int kc_) {
            // (pair, second CTA: a relaxed arrival.  Its slice sits in its OWN shared memory, made visible to the async
            // proxy by the fence before this call, and is read by its own tensor core when the first CTA's product
            // arrives; a releasing cluster-scope arrival costs the warp about a thousand cycles, eight times a layer.)
            if (kPair && !leader) ptx::mbar_arrive_cluster_relaxed(ptx::map_to_cta(bar_a_ready(g, kc_), 0));
            else ptx::mbar_arrive(bar_a_ready(g, kc_));
        };
        uint32_t ack_phase = 0;
        if (kPnet) {
            // the pooled-context maps are read in the middle of a layer's hand-over, where a miss to DRAM would
            // sit on the critical path: ask for all of them now (148 CTAs ask for the same lines; L2 merges them)
            const int n_pooled = (n_conv - 1) / 4;
            const char *gwb = reinterpret_cast<const char *>(args.gw);
            const size_t bytes = (size_t)n_pooled * kRegC * 2 * kPoolC * sizeof(float);
            for (size_t off = (size_t)(ew * 32 + lane) * 128; off < bytes; off += (size_t)S::kEpiWarps * 32 * 128)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(gwb + off));
        }
        for (int r = 0; ok; ++r) {
            const Round rd = round_of(r);
            if (!rd.valid) break;
            if ((g == 0 ? rd.group[0] : rd.group[1]) < 0) continue;                     // this slot sits the round out
            const int board = my_group(rd, g) * kNB + b;
            const bool live = board < args.batch;
            const int sq = y * 8 + x;
            // ---- the group's input planes -> the first in_pad/8 planes of the frame, either copied from an
            // encoded plane tensor or encoded on the spot from the position record (App. D.1 conventions)
            {
                if (args.planes != nullptr) {
                    const uint4 *src = reinterpret_cast<const uint4 *>(args.planes + ((size_t)board * 64 + sq) * args.in_pad);
                    for (int j = set; j < args.in_pad / 8; j += S::kSets) {
                        const uint4 v = live ? __ldg(src + j) : make_uint4(0, 0, 0, 0);
                        *reinterpret_cast<uint4 *>(frame + j * kPlaneBytes + slot * 16) = v;
                    }
                } else if (kPnet) {
                    // the paper's 52 planes (64 channels = 8 planes of the frame) from the 128-byte record
                    const PosM8 *rec = reinterpret_cast<const PosM8 *>(args.positions + (size_t)(live ? board : 0) * args.position_stride);
                    if (live && sq == 0 && (__popcll(rec->pieces[5]) != 1 || __popcll(rec->pieces[11]) != 1))
                        atomicOr(args.status, kStatusBadRecord);
                    float pv[64];
                    planes52_square(rec, sq, pv);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        uint32_t w[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const __nv_bfloat162 h2 = __floats2bfloat162_rn(pv[8 * j + 2 * i], pv[8 * j + 2 * i + 1]);
                            w[i] = *reinterpret_cast<const uint32_t *>(&h2);
                        }
                        if (S::kSets == 1 || (j % S::kSets) == set)
                            *reinterpret_cast<uint4 *>(frame + j * kPlaneBytes + slot * 16) =
                                live ? make_uint4(w[0], w[1], w[2], w[3]) : make_uint4(0, 0, 0, 0);
                    }
                } else {
                    const PosCur *rec = reinterpret_cast<const PosCur *>(args.positions + (size_t)(live ? board : 0) * args.position_stride);
                    const int s_abs = rec->stm ? (sq ^ 56) : sq;            // reflect ranks for Black
                    const float hm = halfmove_plane(rec);
                    if (live && sq == 0 && (__popcll(rec->pieces[5]) != 1 || __popcll(rec->pieces[11]) != 1))
                        atomicOr(args.status, kStatusBadRecord);
                    if (args.in_planes == 19 && args.in_pad == 32) {
                        uint4 v[4];
                        planes19_bf16(rec, sq, v);
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            if (S::kSets == 1 || (j % S::kSets) == set)
                                *reinterpret_cast<uint4 *>(frame + j * kPlaneBytes + slot * 16) = live ? v[j] : make_uint4(0, 0, 0, 0);
                    } else {
                        for (int j = set; j < args.in_pad / 8; j += S::kSets) {
                            const uint4 v = live ? planes_chunk8_bf16(rec, args.in_planes, j * 8, s_abs, hm) : make_uint4(0, 0, 0, 0);
                            *reinterpret_cast<uint4 *>(frame + j * kPlaneBytes + slot * 16) = v;
                        }
                    }
                }
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0)
                    for (int kc = 0; kc < in_slices; ++kc) ready(kc);      // (N-split: every CTA encodes its own copy of the input)
            }
            for (int l = 0; l < n_conv && ok; ++l) {
                const bool from_acc = (l & 1) == 1;
                const bool last = l == n_conv - 1 && head_n == 0;        // nothing follows: results go to global only
                const bool to_global = l == n_conv - 1 && args.out != nullptr;
                const bool next_e4m3 = kFp8 && l + 1 < n_conv;           // the next layer reads e4m3 operands
                {
                    // this layer's channel constants -> this warp's own copy in shared memory (every thread
                    // needs all channels; a private copy needs no cross-warp barrier, which could not be
                    // bounded the way the mbarrier waits are).  Issued before the wait below hides its latency.
                    const float *src = kFp8 ? args.lconst + (size_t)l * kConstFloats : args.bias + (size_t)l * kC;
                    __syncwarp();
#pragma unroll
                    for (int idx = lane; idx < kMyConstFloats / 4; idx += 32) {
                        // own copy: [vector][own slice ks][16 channels]
                        const int vec = idx / (kMyC / 4), within = idx % (kMyC / 4);
                        const int kc = out0 + (within >> 2) * S::kSets + set;
                        reinterpret_cast<float4 *>(lc)[idx] = __ldg(reinterpret_cast<const float4 *>(src) + vec * (kC / 4) + kc * 4 + (within & 3));
                    }
                    __syncwarp();
                }
                ok = wait_bar(bar_acc_full(g), acc_phase, abort_flag, args.status, tr ? &t_wait[0] : nullptr);
                if (!ok) break;
                acc_phase ^= 1u;
                ptx::tc_fence_after();
                if (kNSplit > 1 && l > 0) {
                    // before this layer's slices overwrite the last layer's in this frame, the copies that carry those to the
                    // other CTAs must be done reading them: the receivers have said so (bar_ack; long ago, as a rule)
                    ok = wait_bar_cluster(bar_ack(g), ack_phase, abort_flag, args.status, tr ? &t_wait[1] : nullptr);
                    ack_phase ^= 1u;
                    if (!ok) break;
                }
                const float *bias = kFp8 ? lc + kMyC : lc;
                __nv_bfloat16 *dst = args.out + ((size_t)board * 64 + sq) * kC;
                const uint32_t t_src = t_lane + (uint32_t)(from_acc ? kN : 0);
                const bool keep_h = !from_acc && l != n_conv - 1;   // the residual stream stays in TMEM as fp32
                uint32_t r[2][16];
                const bool pooled = pool_layer(l);
                if (kPnet && pooled) {
                    // ---- pooled context (Sec. 3.2, 4.3.3): the last C/4 channels of this first convolution are
                    // activated, averaged and maximised over each board's 64 squares, mapped to 3C/4 values and
                    // added to the other channels before THEIR activation.
                    // (1) this warp's 32 rows: 16 of board 0 (lanes with bit 3 clear) and 16 of board 1.  Eight
                    // channels at a time are reduced over eight lanes by a halving butterfly (a lane passes on the
                    // half of its values that its partner keeps): 4 + 2 + 1 exchanges, after which every lane of
                    // the eight holds one channel; one more exchange joins the board's two row groups.  Sums and
                    // maxima travel together.
                    // With two sets the eight-channel chunks go to the set that owns their 16-channel slice (whose
                    // constants that set's warps hold).
#pragma unroll
                    for (int pc = 0; pc < (kPoolC + 7) / 8; ++pc) {             // (176 channels: the last chunk is half a chunk)
                        const int pslice = (kRegC + pc * 8) / 16;                 // the slice this chunk lies in
                        if (S::kSets > 1 && (pslice % S::kSets) != set) continue;
                        const int cidx = (pslice / S::kSets) * 16 + (kRegC + pc * 8) % 16;   // in this warp's copy of the constants
                        uint32_t r8[8];
                        ptx::tmem_ld8(t_src + (uint32_t)(kRegC + pc * 8), r8);
                        ptx::tmem_ld_wait();
                        float sm[8], mx[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            // (8-bit tower: int32 accumulator times the weight scale; these channels are not handed on,
                            // so their constants carry no activation scale and the value is in real units)
                            const float pre = kFp8 ? fmaf(__int2float_rn((int)r8[i]), lc[cidx + i], bias[cidx + i])
                                                   : __uint_as_float(r8[i]) + bias[cidx + i];
                            sm[i] = (live && pc * 8 + i < kPoolC) ? fminf(fmaxf(pre, 0.0f), 6.0f) : 0.0f;
                            mx[i] = sm[i];
                        }
#pragma unroll
                        for (int step = 0; step < 3; ++step) {
                            const int half = 4 >> step;                    // values kept after this step
                            const bool upper = (lane >> step) & 1;         // this lane keeps the upper half
#pragma unroll
                            for (int i = 0; i < half; ++i) {
                                const float give_s = upper ? sm[i] : sm[half + i], keep_s = upper ? sm[half + i] : sm[i];
                                const float give_m = upper ? mx[i] : mx[half + i], keep_m = upper ? mx[half + i] : mx[i];
                                sm[i] = keep_s + __shfl_xor_sync(0xffffffffu, give_s, 1 << step);
                                mx[i] = fmaxf(keep_m, __shfl_xor_sync(0xffffffffu, give_m, 1 << step));
                            }
                        }
                        sm[0] += __shfl_xor_sync(0xffffffffu, sm[0], 16);
                        mx[0] = fmaxf(mx[0], __shfl_xor_sync(0xffffffffu, mx[0], 16));
                        if (lane < 16) {                                   // lanes 0-7 board 0, lanes 8-15 board 1
                            const int c0 = pc * 8 + 4 * (lane & 1) + 2 * ((lane >> 1) & 1) + ((lane >> 2) & 1);
                            if (c0 < kPoolC) {
                                pool_part[(q * 2 + b) * kPoolC + c0] = sm[0];
                                pool_part[4 * 2 * kPoolC + (q * 2 + b) * kPoolC + c0] = mx[0];
                            }
                        }
                    }
                    constexpr int kGroupThreads = 128 * S::kSets;
                    const int gt = (ew % (4 * S::kSets)) * 32 + lane;          // this thread among the group's epilogue threads
                    auto meet = [&]() -> bool {                                // the group's epilogue warps, bounded
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(bar_pool(g));
                        const bool met = wait_bar(bar_pool(g), pool_phase, abort_flag, args.status);
                        pool_phase ^= 1u;
                        return met;
                    };
                    ok = meet();
                    if (!ok) break;
                    // (2) the four warps' partial results -> the pooled vector: one entry per thread
                    for (int e = gt; e < 2 * 2 * kPoolC; e += kGroupThreads) {   // e = board * 2 * kPoolC + entry
                        const int pb = e / (2 * kPoolC), j = e % (2 * kPoolC), c = j % kPoolC;
                        const float *src = pool_part + (j >= kPoolC ? 4 * 2 * kPoolC : 0);
                        float acc = src[(0 * 2 + pb) * kPoolC + c];
#pragma unroll
                        for (int w4 = 1; w4 < 4; ++w4) {
                            const float t = src[(w4 * 2 + pb) * kPoolC + c];
                            acc = j >= kPoolC ? fmaxf(acc, t) : acc + t;
                        }
                        pool_vec[pb * 2 * kPoolC + j] = j >= kPoolC ? acc : acc * (1.0f / 64.0f);
                    }
                    constexpr int kCtxPad = kCtxStride > kRegC ? kCtxStride - kRegC : 1;
                    if (kCtxStride > kRegC)                                    // the padding of the context stays zero
                        for (int z = gt; z < 2 * kCtxPad; z += kGroupThreads)
                            pool_ctx[(z / kCtxPad) * kCtxStride + kRegC + z % kCtxPad] = 0.0f;
                    ok = meet();
                    if (!ok) break;
                    // (3) context = gw . pooled vector: 2 boards x 3C/4 outputs over the group's 128 threads.  The map
                    // is stored transposed, [entry of the pooled vector][output], so that neighbouring threads read
                    // neighbouring words.
                    {
                        const float *gwt = args.gw + (size_t)((l - 3) >> 2) * kRegC * 2 * kPoolC;
                        for (int e = gt; e < 2 * kRegC; e += kGroupThreads) {
                            const int pb = e / kRegC, rr0 = e % kRegC;
                            const float *vec = pool_vec + pb * 2 * kPoolC;
                            float acc0 = 0.0f, acc1 = 0.0f;
#pragma unroll 16
                            for (int j = 0; j < 2 * kPoolC; j += 2) {
                                acc0 = fmaf(__ldg(gwt + (size_t)j * kRegC + rr0), vec[j], acc0);
                                acc1 = fmaf(__ldg(gwt + (size_t)(j + 1) * kRegC + rr0), vec[j + 1], acc1);
                            }
                            pool_ctx[pb * kCtxStride + rr0] = acc0 + acc1;
                        }
                    }
                    ok = meet();
                    if (!ok) break;
                }
                auto write_back_h = [&](int ks, int kl_, const float (&v)[16]) {
                    // fp32 copy back to H (FP8: pre-divided by the next conv2's weight scale, so that
                    // conv2 can accumulate its raw products straight onto it).  With one group per CTA this
                    // comes AFTER the slice's hand-off (the next layer's MMAs wait for the frame, not for H, and
                    // nothing else covers the layer boundary); with two groups, whose boundaries cover each
                    // other, before it (measured).  Its completion is awaited once, after the loop: the next
                    // reader of H is the conv2 two layers on, whose MMAs are gated by barriers these same
                    // threads arrive on only after that wait.
                    uint32_t w[16];
#pragma unroll
                    for (int i = 0; i < 16; i += 4) {
                        float4 hs = make_float4(1.0f, 1.0f, 1.0f, 1.0f);
                        if (kFp8) hs = *reinterpret_cast<const float4 *>(lc + 2 * kMyC + ks * 16 + i);
                        if (kInt8) {    // the stream in the next second convolution's integer units, rounded
                            w[i + 0] = (uint32_t)__float2int_rn(v[i + 0] * hs.x);
                            w[i + 1] = (uint32_t)__float2int_rn(v[i + 1] * hs.y);
                            w[i + 2] = (uint32_t)__float2int_rn(v[i + 2] * hs.z);
                            w[i + 3] = (uint32_t)__float2int_rn(v[i + 3] * hs.w);
                        } else {
                            w[i + 0] = __float_as_uint(kFp8 ? v[i + 0] * hs.x : v[i + 0]);
                            w[i + 1] = __float_as_uint(kFp8 ? v[i + 1] * hs.y : v[i + 1]);
                            w[i + 2] = __float_as_uint(kFp8 ? v[i + 2] * hs.z : v[i + 2]);
                            w[i + 3] = __float_as_uint(kFp8 ? v[i + 3] * hs.w : v[i + 3]);
                        }
                    }
                    ptx::tmem_st16(t_lane + (uint32_t)(kl_ * 16), w);
                };
                const float *ctx = pool_ctx + b * kCtxStride;                  // this row's board
                const int n_kc = (kPnet && pooled) ? kShortSlices : kOutSlices;   // the pooled channels are not handed on
                ptx::tmem_ld16(t_src + (uint32_t)(set * 16), r[0]);
#pragma unroll
                for (int ks = 0; ks < kMySlices; ++ks) {
                    const int kl = ks * S::kSets + set;             // the slice among this CTA's output slices (its TMEM columns); ks indexes this warp's constants
                    const int kc = out0 + kl;                       // the slice among the layer's output channels (frame planes, global memory)
                    if (kPnet && kl >= n_kc) break;
                    ptx::tmem_ld_wait();
                    if (kl + S::kSets < n_kc) ptx::tmem_ld16(t_src + (uint32_t)((kl + S::kSets) * 16), r[(ks + 1) & 1]);
                    uint32_t(&rr)[16] = r[ks & 1];
                    float v[16];
#pragma unroll
                    for (int i = 0; i < 16; i += 4) {
                        const float4 bv = *reinterpret_cast<const float4 *>(bias + ks * 16 + i);
                        if (kFp8) {
                            const float4 os = *reinterpret_cast<const float4 *>(lc + ks * 16 + i);
                            // int8 tower: layers after the input layer accumulate in int32 (the input layer's MMAs are bf16 -> fp32)
                            const bool ints = kInt8 && l > 0;
                            const float a0 = ints ? __int2float_rn((int)rr[i + 0]) : __uint_as_float(rr[i + 0]);
                            const float a1 = ints ? __int2float_rn((int)rr[i + 1]) : __uint_as_float(rr[i + 1]);
                            const float a2 = ints ? __int2float_rn((int)rr[i + 2]) : __uint_as_float(rr[i + 2]);
                            const float a3 = ints ? __int2float_rn((int)rr[i + 3]) : __uint_as_float(rr[i + 3]);
                            v[i + 0] = fmaf(a0, os.x, bv.x);
                            v[i + 1] = fmaf(a1, os.y, bv.y);
                            v[i + 2] = fmaf(a2, os.z, bv.z);
                            v[i + 3] = fmaf(a3, os.w, bv.w);
                        } else {
                            v[i + 0] = __uint_as_float(rr[i + 0]) + bv.x;
                            v[i + 1] = __uint_as_float(rr[i + 1]) + bv.y;
                            v[i + 2] = __uint_as_float(rr[i + 2]) + bv.z;
                            v[i + 3] = __uint_as_float(rr[i + 3]) + bv.w;
                        }
                    }
                    if (kPnet && pooled) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[i] += ctx[kc * 16 + i];
                    }
                    if (args.presum != nullptr) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            float sm = live ? v[i] : 0.0f;
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) sm += __shfl_xor_sync(0xffffffffu, sm, o);
                            if (lane == i) atomicAdd(args.presum + l * kC + kc * 16 + i, (double)sm);
                        }
                    }
                    // ReLU: a first convolution's output is only ever read as packed operands, and the
                    // conversion clamps; elsewhere the fp32 value itself goes on (residual stream, output)
                    if (!from_acc || (!kFp8 && args.absmax != nullptr)) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[i] = fmaxf(v[i], 0.0f);
                    }
                    // activations capped at six (Sec. 4.3.6).  A first convolution's output in the int8 form goes nowhere
                    // but into the saturating conversion to unsigned 8-bit, whose 255 stands for the channel's calibrated
                    // maximum, itself at most six: the cap is implied there.
                    if (kPnet && !(kInt8 && from_acc)) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[i] = fminf(v[i], kFp8 ? lc[3 * kMyC + ks * 16 + i] : 6.0f);   // six, in the layer's output units
                    }
                    if (!kFp8 && args.absmax != nullptr) {
                        // calibration: largest output of this layer per channel over all rows of the warp
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            float mx = live ? v[i] : 0.0f;
#pragma unroll
                            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                            if (lane == i) atomicMax(args.absmax + l * kC + kc * 16 + i, __float_as_uint(mx));
                        }
                    }
                    if (to_global && live) {
                        uint32_t pk[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) pk[i] = ptx::pack_bf16x2_relu(v[2 * i], v[2 * i + 1]);
                        reinterpret_cast<uint4 *>(dst + kc * 16)[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        reinterpret_cast<uint4 *>(dst + kc * 16)[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                    }

                    if (!last) {
                        if (next_e4m3) {
                            // 16 channels -> 16 e4m3 bytes (saturating, round to nearest even) = one slot of plane kc
                            uint32_t pk[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                if (kInt8)      // unsigned 8-bit, saturating: clamps at zero (ReLU) and at 255
                                    pk[i] = ptx::cvt_u8_sat(v[4 * i]) | (ptx::cvt_u8_sat(v[4 * i + 1]) << 8) |
                                            (ptx::cvt_u8_sat(v[4 * i + 2]) << 16) | (ptx::cvt_u8_sat(v[4 * i + 3]) << 24);
                                else
                                    pk[i] = ptx::pack_e4m3x2_relu(v[4 * i], v[4 * i + 1]) | (ptx::pack_e4m3x2_relu(v[4 * i + 2], v[4 * i + 3]) << 16);
                            }
                            *reinterpret_cast<uint4 *>(frame + kc * kPlaneBytes + slot * 16) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                            if (kSplitA) {
                                // the remainder of every activation after its own rounding, rounded in turn, into the
                                // second half of the frame (a value beyond the calibrated range saturates the first
                                // part and spills into the second)
                                uint32_t pl[4];
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    float h0, h1, h2, h3;
                                    ptx::unpack_e4m3x2(pk[i] & 0xFFFFu, h0, h1);
                                    ptx::unpack_e4m3x2(pk[i] >> 16, h2, h3);
                                    pl[i] = ptx::pack_e4m3x2(fmaxf(v[4 * i], 0.0f) - h0, fmaxf(v[4 * i + 1], 0.0f) - h1) |
                                            (ptx::pack_e4m3x2(fmaxf(v[4 * i + 2], 0.0f) - h2, fmaxf(v[4 * i + 3], 0.0f) - h3) << 16);
                                }
                                *reinterpret_cast<uint4 *>(frame + (kC / 16 + kc) * kPlaneBytes + slot * 16) = make_uint4(pl[0], pl[1], pl[2], pl[3]);
                            }
                        } else {
                            uint32_t pk[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) pk[i] = ptx::pack_bf16x2_relu(v[2 * i], v[2 * i + 1]);
                            *reinterpret_cast<uint4 *>(frame + (2 * kc) * kPlaneBytes + slot * 16) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                            *reinterpret_cast<uint4 *>(frame + (2 * kc + 1) * kPlaneBytes + slot * 16) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                        }
                        if (kGroups > 1 && keep_h) write_back_h(ks, kl, v);
                        // e4m3 layers consume 32 channels per MMA: one hand-off per two slices.  With two sets
                        // every barrier counts both sets' warps: a pair of slices is handed off by the four
                        // warps of each set, and where the next layer reads 16-channel slices (the bf16 head)
                        // each set also signs for its neighbour's slice once its own is written.
                        if (S::kSets == 2 || !next_e4m3 || (kc & 1)) {
                            ptx::fence_proxy_async_smem();
                            ptx::tc_fence_before();
                            __syncwarp();
                            if (lane == 0) {
                                ready(next_e4m3 ? (kc >> 1) : kc);
                                if (S::kSets == 2 && !next_e4m3) ready(kc ^ 1);
                            }
                        }
                        if (kGroups == 1 && keep_h) write_back_h(ks, kl, v);
                    }
                }
                if (keep_h) ptx::tmem_st_wait();
            }
            if (head_n && ok) {
                // ---- head projections out of the ACC columns
                ok = wait_bar(bar_acc_full(g), acc_phase, abort_flag, args.status, tr ? &t_wait[0] : nullptr);
                if (!ok) break;
                acc_phase ^= 1u;
                if (kNSplit > 1) {                                 // (the last layer's slices were sent as well)
                    ok = wait_bar_cluster(bar_ack(g), ack_phase, abort_flag, args.status);
                    ack_phase ^= 1u;
                    if (!ok) break;
                }
                // the residual towers' head rows are few: set 0 writes them all; the paper network's sixteen slices of
                // queries and keys are dealt out over the sets
                if (!kPnet && set != 0) continue;
                ptx::tc_fence_after();
                const float *hb = head_bias_smem;
                // this row's place in the GEMM A tiles: [tile of 128 boards][8-wide K chunk][board/8][board%8][8 k]
                const size_t u_row = ((size_t)(board >> 7) * 256 * 16 + (size_t)((board & 127) >> 3)) * 128 + (size_t)(board & 7) * 16;
                const int n_slices = head_n / 16;
                const int value_slice0 = n_slices - 2;               // the value projection is the last 32 columns
#pragma unroll 1
                for (int j = kPnet ? set : 0; j < n_slices; j += kPnet ? S::kSets : 1) {
                    uint32_t rr[16];
                    ptx::tmem_ld16(t_lane + (kPnet ? 0u : (uint32_t)kN) + (uint32_t)(j * 16), rr);
                    ptx::tmem_ld_wait();
                    float v[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(rr[i]) + hb[j * 16 + i];
                    if (!live || (kNSplit > 1 && cta_rank != 0)) {
                        // rows past the end of the batch produce nothing; with the N-split every CTA computes the (small)
                        // head projections from its own copy of the frame and the first one writes them
                    } else if (kPnet) {
                        // queries (columns 0..127) and keys (128..255) of this square, fp32 as accumulated, row-major
                        float4 *qk = reinterpret_cast<float4 *>(args.qk_out + ((size_t)board * 64 + sq) * 256 + j * 16);
#pragma unroll
                        for (int i = 0; i < 4; ++i) qk[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                    } else if (head_n == 112 && j < value_slice0) {
                        // 73 policy planes: raw logits, index = plane*64 + square
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const int plane = j * 16 + i;
                            if (plane < kPlanes73) args.logits[(size_t)board * (kPlanes73 * 64) + plane * 64 + sq] = v[i];
                        }
                    } else {
                        uint32_t pk[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const __nv_bfloat162 h2 = __floats2bfloat162_rn(fmaxf(v[2 * i], 0.0f), fmaxf(v[2 * i + 1], 0.0f));
                            pk[i] = *reinterpret_cast<const uint32_t *>(&h2);
                        }
                        const bool is_value = j >= value_slice0;
                        const int c8 = 2 * (is_value ? j - value_slice0 : j);       // 8-channel chunk within the 32
                        unsigned char *u = reinterpret_cast<unsigned char *>(is_value ? args.u_value : args.u_policy) + u_row;
                        *reinterpret_cast<uint4 *>(u + (size_t)(sq * 4 + c8) * 2048) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                        *reinterpret_cast<uint4 *>(u + (size_t)(sq * 4 + c8 + 1) * 2048) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                    }
                }
            }
        }
    }

    if (tr && lane == 0 && (warp <= kGroups + 1))
        printf("tower trace: warp %d total %lld clk, waited %lld / %lld / %lld clk, issue %lld clk\n", warp, clock64() - t_begin,
               t_wait[0], t_wait[1], t_wait[2], t_issue);
    // ---- teardown
    ptx::tc_fence_before();
    __syncthreads();
    if (kCluster) {
        // neither CTA may leave (and release shared memory and TMEM that the other's arrivals, commits, stores and MMAs
        // address) before both are through
        ptx::cluster_arrive();
        ptx::cluster_wait();
    }
    if (warp == 0) {
        ptx::tc_fence_after();
        if (kPair) ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
        else ptx::tmem_dealloc(tmem_base, kTmemCols);
    }
}

#ifndef AZ_NSPLIT_MAX
#define AZ_NSPLIT_MAX 4                  // the widest split of a group over CTAs that the launches use
#endif
#ifndef AZ_C128_SETS
#define AZ_C128_SETS 1
#endif
typedef Shape<128, 2, AZ_C128_SETS> Shape128;
typedef Shape<128, 2, AZ_C128_SETS, true> Shape128Pair;    // the bf16 residual networks: CTA pairs on 256-row tiles
#ifndef AZ_FP8_EPI_SETS
#define AZ_FP8_EPI_SETS 2
#endif
typedef Shape<128, 2, AZ_FP8_EPI_SETS> Shape128F8;
typedef Shape<128, 2, AZ_FP8_EPI_SETS, true> Shape128F8Pair;   // the 8-bit towers on CTA pairs
typedef Shape<256, 1, 1> Shape256;
typedef Shape<256, 1, 1, true> Shape256Pair;              // CTA pairs: each CTA its own group and half of every weight tile
typedef Shape<256, 1, 1, false, 2> Shape256Split2;      // small batches: two CTAs per group, 128 output channels each
typedef Shape<256, 1, 1, false, 4> Shape256Split4;      // smaller still: four CTAs per group, 64 output channels each
// the paper's 160-channel network: one group, whose epilogue (not its MMAs) sets the pace with four warps;
// two sets of four share each layer
#ifndef AZ_P160_SETS
#define AZ_P160_SETS 2
#endif
typedef Shape<160, 1, AZ_P160_SETS> Shape160;
#ifndef AZ_P128_SETS
#define AZ_P128_SETS 2
#endif
typedef Shape<128, 2, AZ_P128_SETS> Shape128P;           // the paper's 128-channel network
typedef Shape<176, 1, 1> Shape176;                       // the ladder's largest size, 19 x 176 (eleven slices: one set)
constexpr int kStageBytes = Shape128::kStageBytes;       // host-side packing of the 128-channel stages

}  // namespace

// Packed layout: for layer l, 16-channel slice kc, tap, the N=128 x K=16 tile as core matrices
// [k8 (2)][n-group (16)][n in group (8)][k in slice (8)] bf16, scale folded into the weights.
size_t tc_packed_weight_bytes(int in_pad, int channels, int n_conv) {
    const size_t slices = (size_t)in_pad / 16 + (size_t)(n_conv - 1) * (channels / 16);
    return slices * 9 * (size_t)channels * 32;             // per slice and tap: N = channels rows x 32 bytes of K
}

// halves > 1 (CTA pairs, or 2 / 4 CTAs splitting the output channels): every weight stage (layer, slice, stage_taps
// taps: nine, or three in the 256-channel shape) is stored as `halves` parts of N, rows [0, C/halves) of the stage's
// taps for the cluster's first CTA, then the next CTA's rows, and so on.  rotate (the N-split): after the input
// layer, part h walks K in the order nsplit_k_slice gives, its own output slices of the layer before first.
void tc_pack_weights(const float *const *w, const float *const *scale, int in_planes, int in_pad,
                     int channels, int n_conv, int halves, int stage_taps, bool rotate, __nv_bfloat16 *packed) {
    __nv_bfloat16 *dst = packed;
    const int groups_per_half = channels / 8 / halves;
    for (int l = 0; l < n_conv; ++l) {
        const int cin = l == 0 ? in_planes : channels;
        const int nkc = (l == 0 ? in_pad : channels) / 16;
        for (int kp = 0; kp < nkc; ++kp)
            for (int st = 0; st < 9 / stage_taps; ++st)
                for (int h = 0; h < halves; ++h)
                    for (int t = 0; t < stage_taps; ++t)
                        for (int k8 = 0; k8 < 2; ++k8)
                            for (int ng = h * groups_per_half; ng < (h + 1) * groups_per_half; ++ng)
                                for (int r = 0; r < 8; ++r)
                                    for (int e = 0; e < 8; ++e) {
                                        const int kc = (rotate && l > 0) ? nsplit_k_slice(halves, nkc / halves, h, kp) : kp;
                                        const int tap = st * stage_taps + t;
                                        const int n = ng * 8 + r, ci = kc * 16 + k8 * 8 + e;
                                        float v = 0.0f;
                                        if (ci < cin) v = scale[l][n] * w[l][((size_t)n * cin + ci) * 9 + tap];
                                        *dst++ = __float2bfloat16_rn(v);
                                    }
    }
}
bool tc_pair_shape(int channels, int precision, bool pnet) {
    return !pnet && ((channels == 128 && precision != AZ_PREC_FP32) || (channels == 256 && precision == AZ_PREC_BF16));
}
// 16-channel slices of the head projection's K that travel in one weight stage of the network's main tower kernel
int tc_head_stage_slices(int channels, int head_n) {
    return channels == 256 ? head_slices_per_stage<Shape256>(head_n) : head_slices_per_stage<Shape128>(head_n);
}

// The same tiles for a tower whose layers read different numbers of input channels (the paper's
// network: 52 planes padded to 64 into the input layer, 3C/4 channels into the second convolution
// of every pooled block).  cin[l] real input channels, cin_pad[l] a multiple of 16.
size_t tc_packed_layers_bytes(const int *cin_pad, int channels, int n_conv) {
    size_t slices = 0;
    for (int l = 0; l < n_conv; ++l) slices += (size_t)cin_pad[l] / 16;
    return slices * 9 * (size_t)channels * 32;
}

void tc_pack_layers(const float *const *w, const float *const *scale, const int *cin, const int *cin_pad,
                    int channels, int n_conv, __nv_bfloat16 *packed) {
    __nv_bfloat16 *dst = packed;
    for (int l = 0; l < n_conv; ++l)
        for (int kc = 0; kc < cin_pad[l] / 16; ++kc)
            for (int tap = 0; tap < 9; ++tap)
                for (int k8 = 0; k8 < 2; ++k8)
                    for (int ng = 0; ng < channels / 8; ++ng)
                        for (int r = 0; r < 8; ++r)
                            for (int e = 0; e < 8; ++e) {
                                const int n = ng * 8 + r, ci = kc * 16 + k8 * 8 + e;
                                float v = 0.0f;
                                if (ci < cin[l]) v = scale[l][n] * w[l][((size_t)n * cin[l] + ci) * 9 + tap];
                                *dst++ = __float2bfloat16_rn(v);
                            }
}

// Head layer of the paper's network: one N = 256 tile per 16-channel slice, rows 0..127 the query
// map, rows 128..255 the key map (both already composed with the token projection).
void tc_pack_qk(const float *wq, const float *wk, int channels, __nv_bfloat16 *packed) {
    __nv_bfloat16 *dst = packed;
    for (int kc = 0; kc < channels / 16; ++kc)
        for (int k8 = 0; k8 < 2; ++k8)
            for (int ng = 0; ng < 256 / 8; ++ng)
                for (int r = 0; r < 8; ++r)
                    for (int e = 0; e < 8; ++e) {
                        const int n = ng * 8 + r, ci = kc * 16 + k8 * 8 + e;
                        const float v = n < 128 ? wq[(size_t)n * channels + ci] : wk[(size_t)(n - 128) * channels + ci];
                        *dst++ = __float2bfloat16_rn(v);
                    }
}

int tower_tc_launch_count() { return 1; }

// ---- FP8-e4m3 tower (Sec. 4.3.6: trunk convolutions quantised, start block and heads at higher
// precision, ranges fixed on calibration positions).  Layer 0 keeps bf16 operands.  For a layer
// l >= 1 with input activation scale sa[ci] (calibration maximum / 448) the folded weight
//     W'[co][ci][tap] = bn_scale[co] * W[co][ci][tap] * sa[ci]
// is stored as e4m3 with one fp32 scale per output channel, ws[co] = max|W'[co]| / 448, so that
//     conv = ws[co] * sum_k q_a[k] * q_w[co][k],   q_a = e4m3(a / sa), q_w = e4m3(W' / ws).
// With qs = 1/sa of the next layer (1 after the last), lconst[l] = { ws * qs (ws = 1 for layer 0),
// bias * qs, 1 / (qs * ws of the next conv2) }: the epilogue forms v' = acc * lconst0 + lconst1, which is
// the layer's output already divided by the next layer's activation scale, converts it to e4m3 (the
// conversion clamps at zero: ReLU commutes with the positive scale), and on the residual stream writes
// relu(v') * lconst2 back to TMEM, the stream pre-divided by the next conv2's weight scale.
size_t tc8_packed_weight_bytes(int in_pad, int channels, int n_conv, bool split_w) {
    return ((size_t)in_pad / 16 + (size_t)(n_conv - 1) * (channels / 32) * (split_w ? 2 : 1)) * kStageBytes;
}

// int8 form (the paper's deployed precision, Sec. 4.3.6): activations unsigned 8-bit with sa =
// calibration maximum / 255 (they are never negative), weights signed 8-bit with ws = max|W'| / 127,
// round to nearest; same constants, same layout.
// split_w (e4m3 only): every weight as a pair, q_w = e4m3(W' / ws) and e4m3(W' / ws - q_w); per 32-channel slice
// the stage of first parts is followed by a stage of remainders.
// halves == 2 (CTA pairs): every stage as rows [0, C/2) of its nine taps, then rows [C/2, C), as in tc_pack_weights.
void tc8_pack(const float *const *w, const float *const *scale, const float *const *bias, const float *absmax,
              int in_planes, int in_pad, int channels, int n_conv, bool int8, bool split_w, int halves, unsigned char *packed, float *lconst) {
    const int C = channels;
    const float kMax = int8 ? 255.0f : 448.0f, kMaxW = int8 ? 127.0f : 448.0f, kTiny = 1e-30f;
    std::vector<float> sa((size_t)n_conv * C, 1.0f), ws((size_t)n_conv * C, 1.0f);
    for (int l = 1; l < n_conv; ++l)
        for (int c = 0; c < C; ++c) sa[(size_t)l * C + c] = fmaxf(absmax[(size_t)(l - 1) * C + c], kTiny) / kMax;
    // layer 0: bf16 tiles exactly as in the bf16 tower
    tc_pack_weights(w, scale, in_planes, in_pad, C, 1, halves, 9, false, reinterpret_cast<__nv_bfloat16 *>(packed));
    unsigned char *dst = packed + (size_t)(in_pad / 16) * kStageBytes;
    std::vector<float> wf((size_t)C * C * 9);
    for (int l = 1; l < n_conv; ++l) {
        for (int co = 0; co < C; ++co) {
            float mx = 0.0f;
            for (int ci = 0; ci < C; ++ci)
                for (int tap = 0; tap < 9; ++tap) {
                    const float v = scale[l][co] * w[l][((size_t)co * C + ci) * 9 + tap] * sa[(size_t)l * C + ci];
                    wf[((size_t)co * C + ci) * 9 + tap] = v;
                    mx = fmaxf(mx, fabsf(v));
                }
            ws[(size_t)l * C + co] = fmaxf(mx, kTiny) / kMaxW;
        }
        for (int kc = 0; kc < C / 32; ++kc)
            for (int part = 0; part < (split_w ? 2 : 1); ++part)
              for (int h = 0; h < halves; ++h)
                for (int tap = 0; tap < 9; ++tap)
                    for (int k16 = 0; k16 < 2; ++k16)
                        for (int ng = h * (C / 8 / halves); ng < (h + 1) * (C / 8 / halves); ++ng)
                            for (int r = 0; r < 8; ++r)
                                for (int e = 0; e < 16; ++e) {
                                    const int n = ng * 8 + r, ci = kc * 32 + k16 * 16 + e;
                                    const float v = wf[((size_t)n * C + ci) * 9 + tap] / ws[(size_t)l * C + n];
                                    if (int8) {
                                        const float q = fminf(fmaxf(nearbyintf(v), -127.0f), 127.0f);
                                        *dst++ = (unsigned char)(signed char)q;
                                    } else {
                                        const __nv_fp8_storage_t q = __nv_cvt_float_to_fp8(v, __NV_SATFINITE, __NV_E4M3);
                                        if (part == 0) *dst++ = (unsigned char)q;
                                        else {
                                            const float first = __half2float(__half(__nv_cvt_fp8_to_halfraw(q, __NV_E4M3)));
                                            *dst++ = (unsigned char)__nv_cvt_float_to_fp8(v - first, __NV_SATFINITE, __NV_E4M3);
                                        }
                                    }
                                }
    }
    for (int l = 0; l < n_conv; ++l) {
        float *lc = lconst + (size_t)l * 3 * C;
        for (int c = 0; c < C; ++c) {
            const float qs = l + 1 < n_conv ? 1.0f / sa[(size_t)(l + 1) * C + c] : 1.0f;
            const float hs = ((l & 1) == 0 && l + 2 < n_conv) ? 1.0f / ws[(size_t)(l + 2) * C + c] : 1.0f;
            lc[c] = (l == 0 ? 1.0f : ws[(size_t)l * C + c]) * qs;
            lc[C + c] = bias[l][c] * qs;
            lc[2 * C + c] = hs / qs;
        }
    }
}

// Head projections as one N = head_n tile per 16-channel slice: rows [0, n_policy) the policy
// projection (scaled where it has a folded batch-norm), zero rows up to n_policy_pad, then the 32
// rows of the value projection.  Same core-matrix order as the tower's weight tiles.
size_t tc_head_weight_bytes(int head_n, int channels) { return (size_t)head_n * channels * 2; }

// halves == 2 (CTA pairs): per weight stage of `stage_slices` slices, rows [0, head_n/2) of the stage's slices, then rows
// [head_n/2, head_n) (128 channels: all eight slices are one stage).  halves == 1: plain slice order.
void tc_pack_head(const float *wp, const float *sp, int n_policy, int n_policy_pad, const float *wv, const float *sv,
                  int channels, int halves, int stage_slices, __nv_bfloat16 *packed) {
    const int head_n = n_policy_pad + kHeadChannels;
    const int groups_per_half = head_n / 8 / halves;
    const int n_slices = channels / 16;
    __nv_bfloat16 *dst = packed;
    for (int s0 = 0; s0 < n_slices; s0 += stage_slices)
        for (int h = 0; h < halves; ++h)
            for (int kc = s0; kc < s0 + stage_slices && kc < n_slices; ++kc)
                for (int k8 = 0; k8 < 2; ++k8)
                    for (int ng = h * groups_per_half; ng < (h + 1) * groups_per_half; ++ng)
                        for (int r = 0; r < 8; ++r)
                            for (int e = 0; e < 8; ++e) {
                                const int n = ng * 8 + r, ci = kc * 16 + k8 * 8 + e;
                                float v = 0.0f;
                                if (n < n_policy) v = (sp ? sp[n] : 1.0f) * wp[(size_t)n * channels + ci];
                                else if (n >= n_policy_pad) v = sv[n - n_policy_pad] * wv[(size_t)(n - n_policy_pad) * channels + ci];
                                *dst++ = __float2bfloat16_rn(v);
                            }
}

int launch_tower_tc(const Net &net, const void *planes, const void *positions, int batch, void *tower_out,
                    bool with_heads, unsigned int *absmax, cudaStream_t s) {
    if (batch == 0) return AZ_OK;
    static int sm_count[64] = {};
    static std::mutex sm_count_lock;                    // any thread may make a device's first launch
    int dev = 0;
    AZ_CUDA(cudaGetDevice(&dev));
    std::unique_lock<std::mutex> hold(sm_count_lock);
    if (dev >= 0 && dev < 64 && sm_count[dev] == 0) {
        int n = 0;
        AZ_CUDA(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev));
        AZ_CUDA(cudaFuncSetAttribute(tower_tc_kernel<false, Shape128>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
        AZ_CUDA(cudaFuncSetAttribute(tower_tc_kernel<false, Shape128Pair>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
        AZ_CUDA(cudaFuncSetAttribute(tower_tc_kernel<true, Shape128F8>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
        AZ_CUDA(cudaFuncSetAttribute(tower_tc_kernel<true, Shape128F8, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
        AZ_CUDA(cudaFuncSetAttribute(tower_tc_kernel<true, Shape128F8, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
        AZ_CUDA(cudaFuncSetAttribute(tower_tc_kernel<true, Shape128F8Pair>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
        AZ_CUDA(cudaFuncSetAttribute(tower_tc_kernel<true, Shape128F8Pair, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
        AZ_CUDA(cudaFuncSetAttribute(tower_tc_kernel<true, Shape128F8Pair, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
        AZ_CUDA(cudaFuncSetAttribute(tower_tc_kernel<false, Shape256>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
        AZ_CUDA(cudaFuncSetAttribute(tower_tc_kernel<false, Shape256Pair>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
        AZ_CUDA(cudaFuncSetAttribute(tower_tc_kernel<false, Shape256Split2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
        AZ_CUDA(cudaFuncSetAttribute(tower_tc_kernel<false, Shape256Split4>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
        AZ_CUDA(cudaFuncSetAttribute(tower_tc_kernel<false, Shape128P, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
        AZ_CUDA(cudaFuncSetAttribute(tower_tc_kernel<false, Shape160, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
        AZ_CUDA(cudaFuncSetAttribute(tower_tc_kernel<true, Shape128P, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
        AZ_CUDA(cudaFuncSetAttribute(tower_tc_kernel<true, Shape160, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
        AZ_CUDA(cudaFuncSetAttribute(tower_tc_kernel<false, Shape176, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem));
        sm_count[dev] = n;
    }
    const int sms = (dev >= 0 && dev < 64) ? sm_count[dev] : 148;
    hold.unlock();
    const bool fp8 = net.fp8_ready && absmax == nullptr;      // the calibration pass itself runs in bf16
    const bool wide = net.arch.channels == 256;
    TowerArgs a;
    a.planes = static_cast<const __nv_bfloat16 *>(planes);
    a.positions = static_cast<const unsigned char *>(positions);
    a.position_stride = az_position_bytes(&net.arch);
    a.in_planes = (int)net.arch.in_planes;
    a.weights = fp8 ? net.tc8_weights : net.tc_weights;
    a.bias = net.tc_bias;
    a.out = static_cast<__nv_bfloat16 *>(tower_out);
    a.status = net.status_dev;
    a.batch = batch;
    a.n_conv = net.n_conv;
    a.in_pad = net.in_pad;
    a.head_n = with_heads ? net.tc_head_n : 0;
    a.head_w = static_cast<const __nv_bfloat16 *>(net.tc_head_w);
    a.head_bias = net.tc_head_bias;
    a.u_policy = static_cast<__nv_bfloat16 *>(net.u_policy);
    a.u_value = static_cast<__nv_bfloat16 *>(net.u_value);
    a.logits = net.logits;
    a.lconst = net.tc8_lconst;
    a.absmax = absmax;
    a.presum = net.calib_presum;
    a.split_w = net.split_w ? 1 : 0;
    a.gw = net.pnet_gw;
    a.qk_out = static_cast<float *>(net.pnet_qk);
#ifdef AZ_TRACE
    static const bool trace = getenv("AZ_TOWER_TRACE") != nullptr;
    a.trace = trace ? atoi(getenv("AZ_TOWER_TRACE")) : 0;
#endif
    // one CTA per SM, or one per two-board group when there are fewer groups than SMs
    const int n_groups = (batch + kNB - 1) / kNB;
    const int grid = n_groups < sms ? n_groups : sms;
    if (net.pnet && net.arch.channels == 176) tower_tc_kernel<false, Shape176, true><<<grid, Shape176::kThreads, Shape176::smem_bytes(false, true), s>>>(a);
    else if (net.pnet && net.arch.channels == 160 && fp8) tower_tc_kernel<true, Shape160, true, true><<<grid, Shape160::kThreads, Shape160::smem_bytes(true, true), s>>>(a);
    else if (net.pnet && net.arch.channels == 160) tower_tc_kernel<false, Shape160, true><<<grid, Shape160::kThreads, Shape160::smem_bytes(false, true), s>>>(a);
    else if (net.pnet && fp8) tower_tc_kernel<true, Shape128P, true, true><<<grid, Shape128P::kThreads, Shape128P::smem_bytes(true, true), s>>>(a);
    else if (net.pnet) tower_tc_kernel<false, Shape128P, true><<<grid, Shape128P::kThreads, Shape128P::smem_bytes(false, true), s>>>(a);
    else if (wide && n_groups * 2 <= sms) {
        // few boards: a cluster of four or two CTAs per group, each computing a quarter or half of every layer's output
        // channels from a copy of the weights packed for that split
        const int split = (net.tc_weights_split4 != nullptr && n_groups * 4 <= sms && AZ_NSPLIT_MAX >= 4) ? 4 : 2;
        a.weights = split == 4 ? net.tc_weights_split4 : net.tc_weights_split;
        a.head_w = static_cast<const __nv_bfloat16 *>(net.tc_head_w_plain ? net.tc_head_w_plain : net.tc_head_w);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(split * n_groups); cfg.blockDim = dim3(Shape256Split2::kThreads);
        cfg.dynamicSmemBytes = split == 4 ? Shape256Split4::smem_bytes(false) : Shape256Split2::smem_bytes(false); cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = split; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        if (split == 4) AZ_CUDA(cudaLaunchKernelEx(&cfg, tower_tc_kernel<false, Shape256Split4>, a));
        else AZ_CUDA(cudaLaunchKernelEx(&cfg, tower_tc_kernel<false, Shape256Split2>, a));
        return AZ_OK;
    }
    else if (wide && net.tc_pair) {
        // clusters of two CTAs, one group each
        const int n_super = (n_groups + 1) / 2, pairs = n_super < sms / 2 ? n_super : sms / 2;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * pairs); cfg.blockDim = dim3(Shape256Pair::kThreads);
        cfg.dynamicSmemBytes = Shape256Pair::smem_bytes(false); cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        AZ_CUDA(cudaLaunchKernelEx(&cfg, tower_tc_kernel<false, Shape256Pair>, a));
        return AZ_OK;
    }
    else if (wide) tower_tc_kernel<false, Shape256><<<grid, Shape256::kThreads, Shape256::smem_bytes(false), s>>>(a);
    else if (fp8 && net.tc_pair8) {
        // the 8-bit towers on clusters of two CTAs; a pair takes pairs of groups
        const int n_super = (n_groups + 1) / 2, pairs = n_super < sms / 2 ? n_super : sms / 2;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * pairs); cfg.blockDim = dim3(Shape128F8Pair::kThreads);
        cfg.dynamicSmemBytes = Shape128F8Pair::smem_bytes(true); cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        if (net.int8) AZ_CUDA(cudaLaunchKernelEx(&cfg, tower_tc_kernel<true, Shape128F8Pair, false, true>, a));
        else if (net.split_a) AZ_CUDA(cudaLaunchKernelEx(&cfg, tower_tc_kernel<true, Shape128F8Pair, false, false, true>, a));
        else AZ_CUDA(cudaLaunchKernelEx(&cfg, tower_tc_kernel<true, Shape128F8Pair>, a));
        return AZ_OK;
    }
    else if (fp8 && net.int8) tower_tc_kernel<true, Shape128F8, false, true><<<grid, Shape128F8::kThreads, Shape128F8::smem_bytes(true), s>>>(a);
    else if (fp8 && net.split_a) tower_tc_kernel<true, Shape128F8, false, false, true><<<grid, Shape128F8::kThreads, Shape128F8::smem_bytes(true), s>>>(a);
    else if (fp8) tower_tc_kernel<true, Shape128F8><<<grid, Shape128F8::kThreads, Shape128F8::smem_bytes(true), s>>>(a);
    else if (net.tc_pair) {
        // clusters of two CTAs; a pair takes pairs of groups
        const int n_super = (n_groups + 1) / 2, pairs = n_super < sms / 2 ? n_super : sms / 2;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * pairs); cfg.blockDim = dim3(Shape128Pair::kThreads);
        cfg.dynamicSmemBytes = Shape128Pair::smem_bytes(false); cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        AZ_CUDA(cudaLaunchKernelEx(&cfg, tower_tc_kernel<false, Shape128Pair>, a));
        return AZ_OK;
    }
    else tower_tc_kernel<false, Shape128><<<grid, Shape128::kThreads, Shape128::smem_bytes(false), s>>>(a);
    AZ_LAUNCH_CHECK();
    return AZ_OK;
}

}  // namespace az
