// Batched tree search on the GPU (Sec. 3.4, Eq. 1; Sec. 4.1 parallel leaves; Sec. 5.1: many games
// interleaved, two batches outstanding; App. D.2 constants).  The trees of all games live in device
// memory; one step of a group of games is: select (one warp per game walks Eq. 1 from the root to an
// edge without a child, reserving its path, and builds the successor position), the legal-move masks
// of the new positions, their evaluation, expand-and-backup (one warp per game).  Nothing returns
// to the host between steps.
//
// Every decision is float32 arithmetic with one rounding per operation (__fmul_rn and friends keep
// the compiler from contracting them), so that a sequential host implementation of the same rules
// reproduces the trees bit for bit.
#include "common.cuh"
#include "chess.cuh"
#include "az_search.h"

#include <mutex>
#include <new>
#include <utility>
#include <vector>

namespace az {
namespace {

constexpr int kWarps = 4;                        // warps (games, positions) per block
constexpr int kMaxDepth = AZ_SEARCH_MAX_DEPTH;

enum : int { kSlotNone = 0, kSlotEval = 1, kSlotTerminal = 2 };

struct alignas(16) Edge {                        // 32 bytes
    int action, child, n, m;
    float prior, w;
    int cbegin, ccnt;                            // the child's edge range once it has been expanded (a copy of its node's
};                                               // fields): a descent fetches the child's node and edges side by side
struct alignas(16) Node {                        // 32 bytes
    int edge_begin, n_edges;                     // n_edges < 0: waiting for its evaluation
    int terminal; float tvalue;
    int nvis; float wsum;                        // values backed up through the node, its own first
    int nsum;                                    // sum over the edges of N + m
    int pad;
};
struct GameState { int n_nodes, n_edges, flags, idle, root_submitted, hist_n, pad[2]; };
constexpr int kMaxHistory = 128;                 // earlier positions of a game kept for the repetition test
constexpr int kRepByte = 100;                    // offset of `repetitions` in a position record

// inverse of the from-to numbering: pair number -> origin | destination << 6 (mover's orientation);
// promotion combination -> origin file | destination file << 3
__device__ unsigned short g_inv_pair[1792];
__device__ unsigned char g_inv_promo[22];

struct Move { int from, to, promo; };

// policy index -> move in the mover's orientation (promo 0 none, 1 N, 2 B, 3 R, 4 Q)
__device__ Move decode_action(int head, int action) {
    Move mv{0, 0, 0};
    if (head == AZ_POLICY_PLANES73) {
        const int plane = action >> 6;
        mv.from = action & 63;
        int df, dr;
        if (plane < 56) {
            const int d = plane / 7, dist = plane % 7 + 1;         // N NE E SE S SW W NW
            df = (d == 1 || d == 2 || d == 3) ? dist : (d == 5 || d == 6 || d == 7) ? -dist : 0;
            dr = (d == 0 || d == 1 || d == 7) ? dist : (d == 3 || d == 4 || d == 5) ? -dist : 0;
        } else if (plane < 64) {
            const int k = plane - 56;                              // (1,2) (2,1) (2,-1) (1,-2) (-1,-2) (-2,-1) (-2,1) (-1,2)
            const int adf = (k == 0 || k == 3 || k == 4 || k == 7) ? 1 : 2;
            df = k < 4 ? adf : -adf;
            dr = (k == 0 || k == 1 || k == 6 || k == 7) ? 3 - adf : adf - 3;
        } else {
            mv.promo = (plane - 64) / 3 + 1;
            df = (plane - 64) % 3 - 1;
            dr = 1;
        }
        mv.to = mv.from + df + 8 * dr;
    } else if (action < 1792) {
        const unsigned e = g_inv_pair[action];
        mv.from = e & 63; mv.to = e >> 6;
    } else {
        const int per = head == AZ_POLICY_FLAT1858 ? 3 : 4;
        const int k = (action - 1792) / per, j = (action - 1792) % per;
        const unsigned e = g_inv_promo[k < 22 ? k : 0];
        mv.from = 48 + (e & 7); mv.to = 56 + (e >> 3);
        mv.promo = head == AZ_POLICY_FLAT1858 ? j + 1 : 4 - j;     // 1,858: N B R; 1,880: Q R B N
    }
    return mv;
}

// The warp writes the successor of record `in` under `action` to `out` (global memory, distinct from in).
// Returns false (all lanes) if the action's origin holds no piece of the mover; out is then a copy.
__device__ bool apply_action_warp(const unsigned char *in, unsigned char *out, int stride, int head, int action, int lane) {
    const u64 *iw = reinterpret_cast<const u64 *>(in);
    u64 *ow = reinterpret_cast<u64 *>(out);
    // ---- the new current position, computed by every lane alike
    const u64 tail = iw[12];
    const int stm = (int)(tail & 1), castling = (int)((tail >> 8) & 0xff), halfmove = (int)((tail >> 24) & 0xff);
    const int reps = (int)((tail >> 32) & 0xff);
    u64 own[6], opp[6];
#pragma unroll
    for (int j = 0; j < 6; ++j) { const u64 wh = iw[j], bl = iw[6 + j]; own[j] = stm ? bl : wh; opp[j] = stm ? wh : bl; }
    Move mv = decode_action(head, action);
    int from = mv.from & 63, to = mv.to & 63;
    if (stm) { from ^= 56; to ^= 56; }
    const u64 fb = 1ull << from, tb = 1ull << to;
    int k = -1;
#pragma unroll
    for (int j = 0; j < 6; ++j) if (own[j] & fb) k = j;
    const bool ok = k >= 0;
    int moved_to = to;                                             // the king's destination when castling
    bool capture = false;
    if (ok) {
        if (k == 5 && (own[3] & tb)) {                             // the king "takes" its own rook: castling
            const int r0 = stm ? 56 : 0;
            const bool king_side = to > from;
            moved_to = r0 + (king_side ? 6 : 2);
            own[5] = 1ull << moved_to;
            own[3] = (own[3] & ~tb) | (1ull << (r0 + (king_side ? 5 : 3)));
        } else {
#pragma unroll
            for (int j = 0; j < 6; ++j) { if (opp[j] & tb) capture = true; opp[j] &= ~tb; }
            if (k == 0 && ((from ^ to) & 7) != 0 && !capture) {    // en passant: the pawn taken stands beside the origin
                opp[0] &= ~(1ull << ((to & 7) + 8 * (from >> 3)));
                capture = true;
            }
            const bool promotes = k == 0 && (to >> 3) == (stm ? 0 : 7);
            const int dest = promotes ? (mv.promo ? mv.promo : 4) : k;
#pragma unroll
            for (int j = 0; j < 6; ++j) { if (j == k) own[j] &= ~fb; if (j == dest) own[j] |= tb; }
        }
    }
    int rights = castling;
    if (ok) {
        const int a = from, b = to;
        const int lose = (a == 4 || b == 4 ? 3 : 0) | (a == 7 || b == 7 ? 1 : 0) | (a == 0 || b == 0 ? 2 : 0) |
                         (a == 60 || b == 60 ? 12 : 0) | (a == 63 || b == 63 ? 4 : 0) | (a == 56 || b == 56 ? 8 : 0);
        rights &= ~lose;
    }
    const int dist = to > from ? to - from : from - to;
    const int ep = ok && k == 0 && dist == 16 ? (from + to) >> 1 : 64;
    const int hm = (k == 0 || capture) ? 0 : (halfmove < 255 ? halfmove + 1 : 255);
    u64 new_tail = tail;
    if (ok) new_tail = (tail & 0xffffff0000000000ull) | (u64)(stm ^ 1) | ((u64)rights << 8) | ((u64)ep << 16) | ((u64)hm << 24);
    // ---- write: the current position by lanes 0..12, then what the record carries besides it
    {
        u64 val = new_tail;
        const int own_base = stm * 6, opp_base = 6 - own_base;
#pragma unroll
        for (int j = 0; j < 6; ++j) { if (lane == own_base + j) val = own[j]; if (lane == opp_base + j) val = opp[j]; }
        if (lane < 13) ow[lane] = val;
    }
    if (stride == 784) {
        // seven earlier boards: the old current position enters at the front, the oldest leaves
        for (int i = lane; i < 84; i += 32) ow[13 + i] = !ok ? iw[13 + i] : i < 12 ? iw[i] : iw[13 + i - 12];
        if (lane == 13) {
            const u64 old = iw[97];                                // hist_rep[7] | n_hist << 56
            const u64 n_hist = old >> 56;
            ow[97] = !ok ? old : (((old << 8) | (u64)reps) & 0x00ffffffffffffffull) | ((n_hist < 7 ? n_hist + 1 : 7) << 56);
        }
    } else if (stride == 128) {
        if (lane == 13) ow[13] = !ok ? iw[13] : (iw[13] << 8) | (u64)from;
        if (lane == 14) ow[14] = !ok ? iw[14] : (iw[14] << 8) | (u64)moved_to;
        if (lane == 15) {
            const u64 old = iw[15];
            const u64 n = old & 0xff;
            ow[15] = !ok ? old : (old & ~0xffull) | (n < 8 ? n + 1 : 8);
        }
    }
    return ok;
}

__global__ void __launch_bounds__(32 * kWarps)
apply_moves_kernel(const unsigned char *__restrict__ positions, int stride, int batch, int head,
                   const int *__restrict__ actions, unsigned char *__restrict__ out, uint32_t *status) {
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i = blockIdx.x * kWarps + w;
    if (i >= batch) return;
    const bool ok = apply_action_warp(positions + (size_t)i * stride, out + (size_t)i * stride, stride, head, actions[i], lane);
    if (!ok && lane == 0 && status) atomicOr(status, AZ_SEARCH_FLAG_BAD_ACTION);
}

// ---- the stand-in evaluator ---------------------------------------------------------------------
__device__ __forceinline__ u64 mix64(u64 x) {
    x ^= x >> 30; x *= 0xbf58476d1ce4e5b9ull;
    x ^= x >> 27; x *= 0x94d049bb133111ebull;
    x ^= x >> 31;
    return x;
}
__device__ u64 position_key(const u64 *rec, u64 seed) {
    u64 h = mix64(seed);
#pragma unroll
    for (int i = 0; i < 12; ++i) h = mix64(h ^ rec[i]);
    const u64 tail = rec[12];
    return mix64(h ^ (tail & 0xffffffull));                        // side to move | castling << 8 | en-passant square << 16
}

// Positions are compared through this hash (pieces, side to move, castling rights, en-passant square).
constexpr u64 kRepSeed = 0x243f6a8885a308d3ull;

// Repetition count of a position with hash h and halfmove clock `halfmove` that is reached from the path
// pn[0 .. depth-1] (root first): one more than the count of its most recent earlier occurrence within the last
// `halfmove` plies, ancestors first, then the game's positions before the root; 0 without one.  All lanes call
// and get the same answer.
__device__ int repetition_count_warp(const u64 *__restrict__ node_hash, const unsigned char *__restrict__ npos, int stride,
                                     const int *pn, int depth, const u64 *__restrict__ hist_hash,
                                     const unsigned char *__restrict__ hist_rep, int hist_n, u64 h, int halfmove, int lane) {
    const int reach = min(halfmove, depth + hist_n);
    int best_k = 0x7fffffff;
    for (int k = lane + 1; k <= reach; k += 32) {
        const u64 c = k <= depth ? node_hash[pn[depth - k]] : hist_hash[hist_n - (k - depth)];
        if (c == h) { best_k = k; break; }
    }
#pragma unroll
    for (int d = 16; d; d >>= 1) best_k = min(best_k, __shfl_xor_sync(0xffffffffu, best_k, d));
    if (best_k == 0x7fffffff) return 0;
    const int before = best_k <= depth ? npos[(size_t)pn[depth - best_k] * stride + kRepByte] : hist_rep[hist_n - (best_k - depth)];
    return before < 255 ? before + 1 : 255;
}

// The set bits of a mask row in ascending order, dealt over the warp: lane L owns words L, L + 32, L + 64.
// Calls f(action, rank) for every set bit, rank = the number of set bits before it; returns the total.
template <typename F>
__device__ __forceinline__ int for_each_legal(const u64 *__restrict__ row, int words, int lane, F f) {
    int base = 0;
    for (int r = 0; r * 32 < words; ++r) {
        const int wi = r * 32 + lane;
        u64 bits = wi < words ? row[wi] : 0ull;
        const int c = __popcll(bits);
        int incl = c;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) { const int t = __shfl_up_sync(0xffffffffu, incl, d); if (lane >= d) incl += t; }
        int rank = base + incl - c;
        while (bits) {
            const int b = __ffsll((long long)bits) - 1;
            bits &= bits - 1;
            f(wi * 64 + b, rank++);
        }
        base += __shfl_sync(0xffffffffu, incl, 31);
    }
    return base;
}

__global__ void __launch_bounds__(32 * kWarps)
standin_eval_kernel(const unsigned char *__restrict__ positions, int stride, const u64 *__restrict__ masks, int words,
                    int batch, u64 seed, float *__restrict__ legal, int *__restrict__ counts, float *__restrict__ value, int vs) {
    __shared__ int s_w[kWarps][AZ_MAX_LEGAL];
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i = blockIdx.x * kWarps + w;
    if (i >= batch) return;
    const u64 key = position_key(reinterpret_cast<const u64 *>(positions + (size_t)i * stride), seed);
    int sum = 0;
    int *wt = s_w[w];
    const int n = for_each_legal(masks + (size_t)i * words, words, lane, [&](int action, int rank) {
        const int r = (int)(mix64(key + (u64)(action + 1) * 0x9e3779b97f4a7c15ull) >> 54);
        const int weight = 1 + r * r / 64;
        if (rank < AZ_MAX_LEGAL) wt[rank] = weight;
        sum += weight;
    });
#pragma unroll
    for (int d = 16; d; d >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
    __syncwarp();
    const int cnt = n < AZ_MAX_LEGAL ? n : AZ_MAX_LEGAL;
    for (int j = lane; j < cnt; j += 32) legal[(size_t)i * AZ_MAX_LEGAL + j] = __fdiv_rn((float)wt[j], (float)sum);
    if (lane == 0) {
        counts[i] = cnt;
        const int t = (int)(mix64(key ^ 0x5851f42d4c957f2dull) >> 40);
        const float u = __fsub_rn(__fmul_rn((float)t, 0x1p-23f), 1.0f);
        value[(size_t)i * vs] = __fmul_rn(u, 0.75f);
    }
}

// ---- the trees ------------------------------------------------------------------------------------
struct Trees {
    Node *nodes; Edge *edges; unsigned char *node_pos; GameState *games;
    u64 *node_hash;                              // [games][node_cap]: position hash of every node (repetition test)
    u64 *hist_hash; unsigned char *hist_rep;     // [games][kMaxHistory]: the game's positions before the root, oldest first
    int node_cap, edge_cap, stride, head, leaves;
    float c_puct, fpu_reduction, discount;
};
struct Batch {                                   // one group's step
    unsigned char *pos;                          // [rows][stride]
    int *kind, *leaf, *depth;                    // [rows]
    int *path_e, *path_n;                        // [rows][kMaxDepth]
};

// Removes the reservations of the first `depth` levels of a path (all lanes call).
__device__ __forceinline__ void undo_path(const Trees &t, Edge *edges, Node *nodes, const int *pe, const int *pn, int depth, int lane) {
    for (int d = lane; d < depth; d += 32) { edges[pe[d]].m -= 1; nodes[pn[d]].nsum -= 1; }
}

// select: one warp per game, `leaves` traversals one after the other
__global__ void __launch_bounds__(32 * kWarps)
search_select_kernel(Trees t, Batch b, int game0, int n_games, int root_step) {
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gl = blockIdx.x * kWarps + w;
    if (gl >= n_games) return;
    const int g = game0 + gl;
    Node *nodes = t.nodes + (size_t)g * t.node_cap;
    Edge *edges = t.edges + (size_t)g * t.edge_cap;
    unsigned char *npos = t.node_pos + (size_t)g * t.node_cap * t.stride;
    GameState *gs = t.games + g;
    for (int j = 0; j < t.leaves; ++j) {
        const int row = gl * t.leaves + j;
        int *pe = b.path_e + (size_t)row * kMaxDepth, *pn = b.path_n + (size_t)row * kMaxDepth;
        int kind = kSlotNone, leaf = -1, depth = 0;
        if (root_step && gs->root_submitted && j == 0) {
            // a step that exists only for the trees whose root still waits for its evaluation: this tree sits it out
            for (int jj = lane; jj < t.leaves; jj += 32) b.kind[gl * t.leaves + jj] = kSlotNone;
            __syncwarp();
            break;
        }
        if (!gs->root_submitted) {
            // the root's own evaluation, once; the step's other rows idle
            __syncwarp();
            if (lane == 0) gs->root_submitted = 1;
            __syncwarp();
            kind = kSlotEval; leaf = 0;
            const u64 *src = reinterpret_cast<const u64 *>(npos);
            u64 *dst = reinterpret_cast<u64 *>(b.pos + (size_t)row * t.stride);
            for (int i = lane; i < t.stride / 8; i += 32) dst[i] = src[i];
        } else {
            int node = 0;
            bool given_up = false;
            // where the current node's edges lie, known before its node record arrives (from the edge that led here)
            int ebegin = 0, ecnt = 0;
            { const Node r0 = nodes[0]; ebegin = r0.edge_begin; ecnt = r0.n_edges; }
            for (;;) {
                const Node nd = nodes[node];
                Edge first{};                                           // this lane's first edge, fetched beside the node
                if (lane < ecnt) first = edges[ebegin + lane];
                if (nd.terminal) { kind = kSlotTerminal; leaf = node; break; }
                if (nd.n_edges < 0) { given_up = true; break; }
                if (depth == kMaxDepth) { if (lane == 0) gs->flags |= AZ_SEARCH_FLAG_DEPTH; given_up = true; break; }
                const float sqrt_n = __fsqrt_rn((float)(nd.nsum > 1 ? nd.nsum : 1));
                const float fpu = __fsub_rn(__fdiv_rn(nd.wsum, (float)nd.nvis), t.fpu_reduction);
                float best_score = 0.0f; int best = -1;
                Edge mine{};                                            // the edge behind this lane's best score
                for (int i = lane; i < nd.n_edges; i += 32) {
                    const Edge e = i == lane ? first : edges[nd.edge_begin + i];
                    const int n = e.n + e.m;
                    const float q = n > 0 ? __fdiv_rn(__fsub_rn(e.w, (float)e.m), (float)n) : fpu;
                    float u = __fmul_rn(t.c_puct, e.prior);
                    u = __fmul_rn(u, sqrt_n);
                    u = __fdiv_rn(u, (float)(1 + n));
                    const float score = __fadd_rn(q, u);
                    if (best < 0 || score > best_score) { best = i; best_score = score; mine = e; }
                }
#pragma unroll
                for (int d = 16; d; d >>= 1) {
                    const float os = __shfl_xor_sync(0xffffffffu, best_score, d);
                    const int ob = __shfl_xor_sync(0xffffffffu, best, d);
                    // the larger score wins, of equal scores the lower index; a lane without edges never wins
                    if (ob >= 0 && (best < 0 || os > best_score || (os == best_score && ob < best))) { best = ob; best_score = os; }
                }
                const int ei = nd.edge_begin + best;
                Edge chosen;                                            // from the lane that scored it (edge i sits in lane i % 32)
                chosen.action = __shfl_sync(0xffffffffu, mine.action, best & 31);
                chosen.child = __shfl_sync(0xffffffffu, mine.child, best & 31);
                chosen.m = __shfl_sync(0xffffffffu, mine.m, best & 31);
                chosen.cbegin = __shfl_sync(0xffffffffu, mine.cbegin, best & 31);
                chosen.ccnt = __shfl_sync(0xffffffffu, mine.ccnt, best & 31);
                __syncwarp();
                if (lane == 0) {
                    edges[ei].m = chosen.m + 1;
                    nodes[node].nsum = nd.nsum + 1;
                    pe[depth] = ei; pn[depth] = node;
                }
                ++depth;
                __syncwarp();
                if (chosen.child < 0) {
                    const int child = gs->n_nodes;
                    if (child >= t.node_cap) { if (lane == 0) gs->flags |= AZ_SEARCH_FLAG_NODES_FULL; given_up = true; break; }
                    __syncwarp();
                    if (lane == 0) {
                        gs->n_nodes = child + 1;
                        edges[ei].child = child;
                        Node c{};
                        c.n_edges = -1;
                        nodes[child] = c;
                    }
                    unsigned char *cpos = npos + (size_t)child * t.stride;
                    apply_action_warp(npos + (size_t)node * t.stride, cpos, t.stride, t.head, chosen.action, lane);
                    __syncwarp();
                    {
                        // the new position's repetition count (the input planes show it; twice before = a draw)
                        const u64 *cw = reinterpret_cast<const u64 *>(cpos);
                        const u64 h = position_key(cw, kRepSeed);
                        const int halfmove = (int)((cw[12] >> 24) & 0xff);
                        u64 *hashes = t.node_hash + (size_t)g * t.node_cap;
                        const int reps = repetition_count_warp(hashes, npos, t.stride, pn, depth, t.hist_hash + (size_t)g * kMaxHistory,
                                                               t.hist_rep + (size_t)g * kMaxHistory, gs->hist_n, h, halfmove, lane);
                        if (lane == 0) { hashes[child] = h; cpos[kRepByte] = (unsigned char)reps; }
                        __syncwarp();
                    }
                    const u64 *src = reinterpret_cast<const u64 *>(cpos);
                    u64 *dst = reinterpret_cast<u64 *>(b.pos + (size_t)row * t.stride);
                    for (int i = lane; i < t.stride / 8; i += 32) dst[i] = src[i];
                    kind = kSlotEval; leaf = child;
                    break;
                }
                node = chosen.child;
                ebegin = chosen.cbegin; ecnt = chosen.ccnt;
            }
            if (given_up) {
                __syncwarp();
                undo_path(t, edges, nodes, pe, pn, depth, lane);
                if (lane == 0) gs->idle += 1;
                kind = kSlotNone;
            }
        }
        __syncwarp();
        if (lane == 0) { b.kind[row] = kind; b.leaf[row] = leaf; b.depth[row] = depth; }
        __syncwarp();
    }
}

// expand and back up: one warp per game, the step's rows in order
__global__ void __launch_bounds__(32 * kWarps)
search_finish_kernel(Trees t, Batch b, int game0, int n_games, const u64 *__restrict__ masks, int words,
                     const float *__restrict__ legal, const int *__restrict__ counts, const float *__restrict__ value, int vs) {
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int gl = blockIdx.x * kWarps + w;
    if (gl >= n_games) return;
    const int g = game0 + gl;
    Node *nodes = t.nodes + (size_t)g * t.node_cap;
    Edge *edges = t.edges + (size_t)g * t.edge_cap;
    GameState *gs = t.games + g;
    for (int j = 0; j < t.leaves; ++j) {
        const int row = gl * t.leaves + j;
        const int kind = b.kind[row];
        if (kind == kSlotNone) continue;
        const int leaf = b.leaf[row], depth = b.depth[row];
        float v;
        if (kind == kSlotEval) {
            const int cnt = counts[row];
            const float net_v = vs == 3 ? __fsub_rn(value[(size_t)row * 3], value[(size_t)row * 3 + 2]) : value[row];
            const u64 *rec = reinterpret_cast<const u64 *>(b.pos + (size_t)row * t.stride);
            const int halfmove = (int)((rec[12] >> 24) & 0xff), reps = (int)((rec[12] >> 32) & 0xff);
            Node nd = nodes[leaf];
            nd.nsum = 0; nd.n_edges = 0;
            if (cnt == 0) {
                // no legal move: mated if the mover's king is attacked, else stalemate
                const int stm = (int)(rec[12] & 1);
                u64 opp[6], occ = 0;
#pragma unroll
                for (int k = 0; k < 6; ++k) { opp[k] = rec[(stm ^ 1) * 6 + k]; occ |= opp[k] | rec[stm * 6 + k]; }
                const u64 king = rec[stm * 6 + 5];
                const bool check = king && attacked(__ffsll((long long)king) - 1, stm ^ 1, opp, occ);
                nd.terminal = 1; nd.tvalue = check ? -1.0f : 0.0f;
            } else if (halfmove >= 100 || reps >= 2) {
                nd.terminal = 1; nd.tvalue = 0.0f;
            } else if (gs->n_edges + cnt > t.edge_cap) {
                if (lane == 0) gs->flags |= AZ_SEARCH_FLAG_EDGES_FULL;
                nd.terminal = 1; nd.tvalue = net_v;
            } else {
                const int begin = gs->n_edges;
                nd.edge_begin = begin; nd.n_edges = cnt;
                const float *pr = legal + (size_t)row * AZ_MAX_LEGAL;
                for_each_legal(masks + (size_t)row * words, words, lane, [&](int action, int rank) {
                    if (rank < cnt) {
                        Edge e;
                        e.action = action; e.child = -1; e.n = 0; e.m = 0; e.prior = pr[rank]; e.w = 0.0f;
                        e.cbegin = 0; e.ccnt = 0;
                        edges[begin + rank] = e;
                    }
                });
                __syncwarp();
                if (lane == 0) {
                    gs->n_edges = begin + cnt;
                    if (depth > 0) {                                    // the edge that leads here learns where the new edges lie
                        Edge *up = edges + b.path_e[(size_t)row * kMaxDepth + depth - 1];
                        up->cbegin = begin; up->ccnt = cnt;
                    }
                }
            }
            v = nd.terminal ? nd.tvalue : net_v;
            nd.nvis = 1; nd.wsum = v;
            __syncwarp();
            if (lane == 0) nodes[leaf] = nd;
        } else {
            const Node nd = nodes[leaf];
            v = nd.tvalue;
            __syncwarp();
            if (lane == 0) { nodes[leaf].nvis = nd.nvis + 1; nodes[leaf].wsum = __fadd_rn(nd.wsum, v); }
        }
        __syncwarp();
        // up the path: level d takes the value after depth - d sign changes and discounts; the levels touch
        // different edges and nodes, so the lanes update them side by side
        const int *pe = b.path_e + (size_t)row * kMaxDepth, *pn = b.path_n + (size_t)row * kMaxDepth;
        for (int base = 0; base < depth; base += 32) {
            const int up = base + lane;                            // 0: the edge into the leaf
            float x = v;
            for (int s = 0; s <= up && s < depth; ++s) x = __fmul_rn(-x, t.discount);
            if (up < depth) {
                const int d = depth - 1 - up;
                Edge *e = edges + pe[d];
                e->n += 1; e->w = __fadd_rn(e->w, x); e->m -= 1;
                Node *p = nodes + pn[d];
                p->nvis += 1; p->wsum = __fadd_rn(p->wsum, x);
            }
        }
        __syncwarp();
    }
}

std::mutex g_inv_mutex;
bool g_inv_ready[64] = {};

int ensure_inverse_tables() {
    int dev = 0;
    AZ_CUDA(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lock(g_inv_mutex);
    if (dev < 64 && g_inv_ready[dev]) return AZ_OK;
    static short pair[64 * 64];
    static short promo[8 * 3];
    static unsigned short inv_pair[1792];
    static unsigned char inv_promo[22];
    if (build_flat_tables(pair, promo) != kFlatMoves) return AZ_ERR_BAD_ARCH;
    for (int from = 0; from < 64; ++from)
        for (int to = 0; to < 64; ++to)
            if (pair[from * 64 + to] >= 0) {
                if (pair[from * 64 + to] >= 1792) return AZ_ERR_BAD_ARCH;
                inv_pair[pair[from * 64 + to]] = (unsigned short)(from | to << 6);
            }
    for (int file = 0; file < 8; ++file)
        for (int step = 0; step < 3; ++step)
            if (promo[file * 3 + step] >= 0) {
                const int k = (promo[file * 3 + step] - 1792) / 3;
                if (k < 0 || k >= 22) return AZ_ERR_BAD_ARCH;
                inv_promo[k] = (unsigned char)(file | (file + step - 1) << 3);
            }
    AZ_CUDA(cudaMemcpyToSymbol(g_inv_pair, inv_pair, sizeof inv_pair));
    AZ_CUDA(cudaMemcpyToSymbol(g_inv_promo, inv_promo, sizeof inv_promo));
    if (dev < 64) g_inv_ready[dev] = true;
    return AZ_OK;
}

struct Group {
    cudaStream_t owned = nullptr;                // null: the group takes turns with group 0 on that group's stream
    cudaStream_t stream = nullptr;               // the stream its steps are queued on
    int game0 = 0, n_games = 0, rows = 0;
    Batch batch{};
    uint64_t *masks = nullptr;
    float *legal = nullptr, *value = nullptr;
    int *counts = nullptr;
    cudaEvent_t done = nullptr;
};

struct Search {
    az_search_config cfg{};
    Net *net = nullptr;
    int device = 0;
    int words = 0, vs = 1;
    Trees trees{};
    Group groups[2];
    int n_groups = 1;
    bool second_workspace = false;
    cudaEvent_t ev_begin = nullptr, ev_end = nullptr;
    unsigned char *roots_stage = nullptr;        // device copy of the root records
    int *out_actions = nullptr, *out_visits = nullptr, *out_counts = nullptr;   // read-out of all roots
    bool need_root_step = true;                  // some tree's root still waits for its evaluation
    bool pending = false;                        // az_search_run_async has queued steps that az_search_wait has not collected
    // played moves: the kept subtrees are written to a second set of pools, which then becomes the first
    Node *alt_nodes = nullptr; Edge *alt_edges = nullptr; unsigned char *alt_node_pos = nullptr; u64 *alt_node_hash = nullptr;
    int *remap = nullptr;                        // [games][2][max_nodes]: old index of every kept node, edge that leads to it
    int *adv_actions = nullptr, *adv_played = nullptr, *adv_fresh = nullptr;
};

void free_search(Search *s) {
    if (!s) return;
    if (s->pending && s->ev_end) cudaEventSynchronize(s->ev_end);       // queued steps still use what is freed below
    cudaFree(s->trees.nodes); cudaFree(s->trees.edges); cudaFree(s->trees.node_pos); cudaFree(s->trees.games);
    cudaFree(s->trees.node_hash); cudaFree(s->trees.hist_hash); cudaFree(s->trees.hist_rep); cudaFree(s->alt_node_hash);
    cudaFree(s->roots_stage);
    cudaFree(s->out_actions); cudaFree(s->out_visits); cudaFree(s->out_counts);
    cudaFree(s->alt_nodes); cudaFree(s->alt_edges); cudaFree(s->alt_node_pos); cudaFree(s->remap);
    cudaFree(s->adv_actions); cudaFree(s->adv_played); cudaFree(s->adv_fresh);
    for (Group &g : s->groups) {
        cudaFree(g.batch.pos); cudaFree(g.batch.kind); cudaFree(g.batch.leaf); cudaFree(g.batch.depth);
        cudaFree(g.batch.path_e); cudaFree(g.batch.path_n);
        cudaFree(g.masks); cudaFree(g.legal); cudaFree(g.value); cudaFree(g.counts);
        if (g.done) cudaEventDestroy(g.done);
        if (g.owned) cudaStreamDestroy(g.owned);
    }
    if (s->ev_begin) cudaEventDestroy(s->ev_begin);
    if (s->ev_end) cudaEventDestroy(s->ev_end);
    delete s;
}

// New trees: block b empties game index[b] (game b without an index) and gives it root record b.
__global__ void reset_trees_kernel(Trees t, const unsigned char *__restrict__ roots, int count, const int *__restrict__ index) {
    if ((int)blockIdx.x >= count) return;
    const int g = index ? index[blockIdx.x] : (int)blockIdx.x;
    if (threadIdx.x == 0) {
        GameState gs{};
        gs.n_nodes = 1;
        t.games[g] = gs;
        Node root{};
        root.n_edges = -1;
        t.nodes[(size_t)g * t.node_cap] = root;
    }
    const u64 *src = reinterpret_cast<const u64 *>(roots + (size_t)blockIdx.x * t.stride);
    u64 *dst = reinterpret_cast<u64 *>(t.node_pos + (size_t)g * t.node_cap * t.stride);
    for (int i = threadIdx.x; i < t.stride / 8; i += blockDim.x) dst[i] = src[i];
    if (threadIdx.x == 0) t.node_hash[(size_t)g * t.node_cap] = position_key(src, kRepSeed);
}

// A move is played in every game (Sec. 3.3: the relevant subtree becomes the next root).  One warp per game:
// the root's edge of the action (given, or the most visited one, ties to the lower action) is looked up; the
// subtree under it is copied to the other pools breadth-first, a node's children in the order of its edges;
// without a child the new tree is the bare successor position.  actions[g] == -1, a root without edges or an
// action the root does not have leave the game's tree as it is (copied whole); played[g] tells which it was.
__global__ void __launch_bounds__(32 * kWarps)
search_advance_kernel(Trees t, Node *new_nodes, Edge *new_edges, unsigned char *new_pos, u64 *new_hash, int games,
                      const int *__restrict__ actions, int *__restrict__ played, int *__restrict__ remap_all, int *any_fresh) {
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = blockIdx.x * kWarps + w;
    if (g >= games) return;
    const Node *nodes = t.nodes + (size_t)g * t.node_cap;
    const Edge *edges = t.edges + (size_t)g * t.edge_cap;
    const unsigned char *npos = t.node_pos + (size_t)g * t.node_cap * t.stride;
    Node *nn = new_nodes + (size_t)g * t.node_cap;
    Edge *ne = new_edges + (size_t)g * t.edge_cap;
    unsigned char *np = new_pos + (size_t)g * t.node_cap * t.stride;
    int *remap = remap_all + (size_t)g * 2 * t.node_cap;            // [old index of kept node | index of the edge that leads to it]
    int *up_edge = remap + t.node_cap;
    GameState *gs = t.games + g;
    const u64 *hashes = t.node_hash + (size_t)g * t.node_cap;
    u64 *nh = new_hash + (size_t)g * t.node_cap;
    u64 *hist_hash = t.hist_hash + (size_t)g * kMaxHistory;
    unsigned char *hist_rep = t.hist_rep + (size_t)g * kMaxHistory;
    const Node root = nodes[0];
    const int want = actions ? actions[g] : -2;
    // ---- the root's edge
    int best = -1, best_n = -1;
    for (int i = lane; i < root.n_edges; i += 32) {
        const Edge e = edges[root.edge_begin + i];
        if (want == -2 ? e.n > best_n : e.action == want) { best = i; best_n = e.n; }
    }
#pragma unroll
    for (int d = 16; d; d >>= 1) {
        const int on = __shfl_xor_sync(0xffffffffu, best_n, d), ob = __shfl_xor_sync(0xffffffffu, best, d);
        if (ob >= 0 && (best < 0 || on > best_n || (on == best_n && ob < best))) { best = ob; best_n = on; }
    }
    const int words = t.stride / 8;
    if (best < 0 || want == -1) {
        // nothing is played: the tree moves to the other pools as it is
        if (lane == 0) {
            played[g] = -1;
            if (want >= 0) gs->flags |= AZ_SEARCH_FLAG_BAD_ACTION;
        }
        const int n_nodes = gs->n_nodes, n_edges = gs->n_edges;
        for (int i = lane; i < n_nodes; i += 32) { nn[i] = nodes[i]; nh[i] = hashes[i]; }
        for (int i = lane; i < n_edges; i += 32) ne[i] = edges[i];
        const u64 *src = reinterpret_cast<const u64 *>(npos);
        u64 *dst = reinterpret_cast<u64 *>(np);
        for (size_t i = lane; i < (size_t)n_nodes * words; i += 32) dst[i] = src[i];
        return;
    }
    const Edge e0 = edges[root.edge_begin + best];
    if (lane == 0) played[g] = e0.action;
    const int hist_n = gs->hist_n;
    const u64 old_root_hash = hashes[0];
    const int old_root_reps = npos[kRepByte];
    // the old root joins the game's earlier positions, unless the move is irreversible (then nothing before it can
    // recur); called once the new root's record is in place
    auto push_history = [&]() {
        __syncwarp();
        const int halfmove = (int)((reinterpret_cast<const u64 *>(np)[12] >> 24) & 0xff);
        if (halfmove == 0) { if (lane == 0) gs->hist_n = 0; return; }
        int n = hist_n;
        if (n == kMaxHistory) {                                        // the oldest entry leaves
            u64 hv[kMaxHistory / 32]; unsigned char rv[kMaxHistory / 32];
#pragma unroll
            for (int r = 0; r < kMaxHistory / 32; ++r) {
                const int i = r * 32 + lane;
                hv[r] = i + 1 < kMaxHistory ? hist_hash[i + 1] : 0ull;
                rv[r] = i + 1 < kMaxHistory ? hist_rep[i + 1] : (unsigned char)0;
            }
            __syncwarp();
#pragma unroll
            for (int r = 0; r < kMaxHistory / 32; ++r) { hist_hash[r * 32 + lane] = hv[r]; hist_rep[r * 32 + lane] = rv[r]; }
            __syncwarp();
            n -= 1;
        }
        if (lane == 0) { hist_hash[n] = old_root_hash; hist_rep[n] = (unsigned char)old_root_reps; gs->hist_n = n + 1; }
    };
    if (e0.child < 0) {
        apply_action_warp(npos, np, t.stride, t.head, e0.action, lane);
        if (lane == 0) remap[0] = 0;                                   // the path to the new position: the old root alone
        __syncwarp();
        const u64 *cw = reinterpret_cast<const u64 *>(np);
        const u64 h = position_key(cw, kRepSeed);
        const int reps = repetition_count_warp(hashes, npos, t.stride, remap, 1, hist_hash, hist_rep, hist_n, h,
                                               (int)((cw[12] >> 24) & 0xff), lane);
        if (lane == 0) {
            np[kRepByte] = (unsigned char)reps;
            nh[0] = h;
            Node fresh{};
            fresh.n_edges = -1;
            nn[0] = fresh;
            gs->n_nodes = 1; gs->n_edges = 0; gs->root_submitted = 0;
            atomicOr(any_fresh, 1);
        }
        push_history();
        return;
    }
    // ---- breadth-first copy: new node i was old node remap[i]
    if (lane == 0) remap[0] = e0.child;
    __syncwarp();
    int n_new = 1, e_new = 0;
    for (int i = 0; i < n_new; ++i) {
        const int o = remap[i];
        Node nd = nodes[o];
        const u64 *src = reinterpret_cast<const u64 *>(npos + (size_t)o * t.stride);
        u64 *dst = reinterpret_cast<u64 *>(np + (size_t)i * t.stride);
        for (int k = lane; k < words; k += 32) dst[k] = src[k];
        const int begin = nd.edge_begin, cnt = nd.n_edges > 0 ? nd.n_edges : 0;
        for (int base = 0; base < cnt; base += 32) {
            const int j = base + lane;
            Edge e{};
            bool has = false;
            if (j < cnt) { e = edges[begin + j]; has = e.child >= 0; }
            const unsigned m = __ballot_sync(0xffffffffu, has);
            if (has) {
                const int id = n_new + __popc(m & ((1u << lane) - 1u));
                remap[id] = e.child;
                up_edge[id] = e_new + j;                               // the kept node's edge range is filled in when its turn comes
                e.child = id;
            }
            if (j < cnt) ne[e_new + j] = e;
            n_new += __popc(m);
        }
        if (lane == 0) {
            if (i > 0) { ne[up_edge[i]].cbegin = e_new; ne[up_edge[i]].ccnt = cnt; }
            nd.edge_begin = e_new; nn[i] = nd; nh[i] = hashes[o];
        }
        e_new += cnt;
        __syncwarp();
    }
    if (lane == 0) { gs->n_nodes = n_new; gs->n_edges = e_new; }
    push_history();
}

// Root noise (Sec. 3.4; App. D.2): P <- (1 - epsilon) P + epsilon * noise on the edges of every game's current
// root, noise[g][i] belonging to the root's i-th edge; one rounding per operation.  Roots that have not been
// evaluated yet, or have no moves, are left alone; changed[g] tells how many edges were touched.
__global__ void root_noise_kernel(Trees t, int games, const float *__restrict__ noise, float epsilon, int *__restrict__ changed) {
    const int g = blockIdx.x;
    if (g >= games) return;
    const Node root = t.nodes[(size_t)g * t.node_cap];
    const int k = root.n_edges > 0 ? (root.n_edges < AZ_MAX_LEGAL ? root.n_edges : AZ_MAX_LEGAL) : 0;
    Edge *e = t.edges + (size_t)g * t.edge_cap + root.edge_begin;
    const float keep = __fsub_rn(1.0f, epsilon);
    for (int i = threadIdx.x; i < k; i += blockDim.x)
        e[i].prior = __fadd_rn(__fmul_rn(keep, e[i].prior), __fmul_rn(epsilon, noise[(size_t)g * AZ_MAX_LEGAL + i]));
    if (threadIdx.x == 0) changed[g] = k;
}

// root actions and visit counts of every game, in rows of AZ_MAX_LEGAL
__global__ void gather_roots_kernel(Trees t, int games, int *__restrict__ actions, int *__restrict__ visits, int *__restrict__ counts) {
    const int g = blockIdx.x;
    if (g >= games) return;
    const Node root = t.nodes[(size_t)g * t.node_cap];
    const int k = root.n_edges > 0 ? (root.n_edges < AZ_MAX_LEGAL ? root.n_edges : AZ_MAX_LEGAL) : 0;
    const Edge *e = t.edges + (size_t)g * t.edge_cap + root.edge_begin;
    for (int i = threadIdx.x; i < k; i += blockDim.x) {
        actions[(size_t)g * AZ_MAX_LEGAL + i] = e[i].action;
        visits[(size_t)g * AZ_MAX_LEGAL + i] = e[i].n;
    }
    if (threadIdx.x == 0) counts[g] = k;
}

// one step of one group: four launches (five with the paper's network or a tensor-core net: their
// evaluation is two or three kernels)
int queue_step(Search &s, int gi, bool root_step) {
    Group &g = s.groups[gi];
    const unsigned blocks = (unsigned)((g.n_games + kWarps - 1) / kWarps);
    search_select_kernel<<<blocks, 32 * kWarps, 0, g.stream>>>(s.trees, g.batch, g.game0, g.n_games, root_step ? 1 : 0);
    AZ_LAUNCH_CHECK();
    int rc = launch_legal_masks(g.batch.pos, (size_t)s.trees.stride, g.rows, s.trees.head, g.masks, g.stream);
    if (rc != AZ_OK) return rc;
    if (s.cfg.evaluator == AZ_SEARCH_EVAL_STANDIN) {
        standin_eval_kernel<<<(unsigned)((g.rows + kWarps - 1) / kWarps), 32 * kWarps, 0, g.stream>>>(
            g.batch.pos, s.trees.stride, (const u64 *)g.masks, s.words, g.rows, s.cfg.seed, g.legal, g.counts, g.value, s.vs);
        AZ_LAUNCH_CHECK();
    } else {
        const bool alt = s.second_workspace && gi == 1;
        if (alt) swap_workspace(*s.net);
        rc = az_evaluate_legal(reinterpret_cast<az_net *>(s.net), g.batch.pos, g.masks, g.rows, g.legal, g.counts, g.value, g.stream);
        if (alt) swap_workspace(*s.net);
        if (rc != AZ_OK) return rc;
    }
    search_finish_kernel<<<blocks, 32 * kWarps, 0, g.stream>>>(s.trees, g.batch, g.game0, g.n_games, (const u64 *)g.masks, s.words,
                                                               g.legal, g.counts, g.value, s.vs);
    AZ_LAUNCH_CHECK();
    return AZ_OK;
}

}  // namespace
}  // namespace az

using az::Search;

extern "C" {

int az_apply_moves(const void *positions_dev, size_t position_stride, int batch, int policy_head,
                   const int32_t *actions_dev, void *out_positions_dev, uint32_t *status_dev, void *cuda_stream) {
    if (batch < 0 || policy_head < 0 || policy_head > AZ_POLICY_FROMTO1880) return AZ_ERR_BAD_ARG;
    if (position_stride != 104 && position_stride != 784 && position_stride != 128) return AZ_ERR_BAD_ARG;
    if (batch == 0) return AZ_OK;
    if (!positions_dev || !actions_dev || !out_positions_dev || positions_dev == out_positions_dev) return AZ_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(positions_dev) & 7) || (reinterpret_cast<uintptr_t>(out_positions_dev) & 7) ||
        (reinterpret_cast<uintptr_t>(actions_dev) & 3) || (reinterpret_cast<uintptr_t>(status_dev) & 3))
        return AZ_ERR_BAD_ARG;
    int rc = az::ensure_inverse_tables();
    if (rc != AZ_OK) return rc;
    az::apply_moves_kernel<<<(unsigned)((batch + az::kWarps - 1) / az::kWarps), 32 * az::kWarps, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        static_cast<const unsigned char *>(positions_dev), (int)position_stride, batch, policy_head, actions_dev,
        static_cast<unsigned char *>(out_positions_dev), status_dev);
    AZ_LAUNCH_CHECK();
    return AZ_OK;
}

int az_standin_evaluate(const void *positions_dev, size_t position_stride, const uint64_t *legal_masks_dev, int batch,
                        int policy_head, uint64_t seed, float *legal_policy_dev, int32_t *legal_counts_dev,
                        float *value_dev, void *cuda_stream) {
    if (batch < 0 || policy_head < 0 || policy_head > AZ_POLICY_FROMTO1880 || position_stride < 104 || (position_stride & 7)) return AZ_ERR_BAD_ARG;
    if (batch == 0) return AZ_OK;
    if (!positions_dev || !legal_masks_dev || !legal_policy_dev || !legal_counts_dev || !value_dev) return AZ_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(positions_dev) & 7) || (reinterpret_cast<uintptr_t>(legal_masks_dev) & 7)) return AZ_ERR_BAD_ARG;
    const int words = policy_head == AZ_POLICY_PLANES73 ? 73 : 30;
    az::standin_eval_kernel<<<(unsigned)((batch + az::kWarps - 1) / az::kWarps), 32 * az::kWarps, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        static_cast<const unsigned char *>(positions_dev), (int)position_stride, (const az::u64 *)legal_masks_dev, words, batch,
        seed, legal_policy_dev, legal_counts_dev, value_dev, 1);
    AZ_LAUNCH_CHECK();
    return AZ_OK;
}

int az_search_create(az_net *net, const az_search_config *c, az_search **out) {
    if (!c || !out) return AZ_ERR_BAD_ARG;
    *out = nullptr;
    if (c->games < 1 || c->leaves < 1 || c->leaves > AZ_SEARCH_MAX_LEAVES || c->groups < 1 || c->groups > 2 ||
        c->max_nodes < 2 || c->max_edges < 1 || c->evaluator > AZ_SEARCH_EVAL_STANDIN || c->policy_head > AZ_POLICY_FROMTO1880)
        return AZ_ERR_BAD_ARG;
    if (c->position_bytes != 104 && c->position_bytes != 784 && c->position_bytes != 128) return AZ_ERR_BAD_ARG;
    if (!(c->c_puct >= 0.0f) || !(c->discount > 0.0f && c->discount <= 1.0f) || !(c->fpu_reduction >= 0.0f)) return AZ_ERR_BAD_ARG;
    az::Net *n = reinterpret_cast<az::Net *>(net);
    if (c->evaluator == AZ_SEARCH_EVAL_NET) {
        if (!n) return AZ_ERR_BAD_ARG;
        if (n->arch.policy_head != c->policy_head || az_position_bytes(&n->arch) != c->position_bytes) return AZ_ERR_BAD_ARCH;
        if (n->fp8 && !n->fp8_ready) return AZ_ERR_NOT_CALIBRATED;
    }
    const int n_groups = c->games >= 2 ? (int)c->groups : 1;
    const int per_group = (int)((c->games + n_groups - 1) / n_groups);
    if (c->evaluator == AZ_SEARCH_EVAL_NET && (uint64_t)per_group * c->leaves > n->arch.max_batch) return AZ_ERR_BATCH_TOO_LARGE;
    // everything below is allocated on the network's device; the caller's current device is put back on return
    struct DeviceGuard {
        int prev = -1;
        ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
    } device_guard;
    if (n) {
        int cur = 0;
        AZ_CUDA(cudaGetDevice(&cur));
        if (cur != n->device) { AZ_CUDA(cudaSetDevice(n->device)); device_guard.prev = cur; }
    }
    int rc = az::ensure_inverse_tables();
    if (rc != AZ_OK) return rc;
    Search *s = new (std::nothrow) Search();
    if (!s) return AZ_ERR_BAD_ARG;
    s->cfg = *c;
    s->net = c->evaluator == AZ_SEARCH_EVAL_NET ? n : nullptr;
    s->n_groups = n_groups;
    s->words = c->policy_head == AZ_POLICY_PLANES73 ? 73 : 30;
    s->vs = s->net ? (int)az_value_size(&s->net->arch) : 1;
    az::Trees &t = s->trees;
    t.node_cap = (int)c->max_nodes; t.edge_cap = (int)c->max_edges; t.stride = (int)c->position_bytes;
    t.head = (int)c->policy_head; t.leaves = (int)c->leaves;
    t.c_puct = c->c_puct; t.fpu_reduction = c->fpu_reduction; t.discount = c->discount;
    const size_t G = c->games;
#define AZ_SEARCH_ALLOC(ptr, bytes)                                                          \
    do {                                                                                     \
        cudaError_t e__ = cudaMalloc((void **)&(ptr), (bytes));                              \
        if (e__ != cudaSuccess) { az::set_cuda_error(e__, "cudaMalloc (search)"); az::free_search(s); return AZ_ERR_CUDA; } \
    } while (0)
    AZ_SEARCH_ALLOC(t.nodes, G * t.node_cap * sizeof(az::Node));
    AZ_SEARCH_ALLOC(t.edges, G * t.edge_cap * sizeof(az::Edge));
    AZ_SEARCH_ALLOC(t.node_pos, G * t.node_cap * (size_t)t.stride);
    AZ_SEARCH_ALLOC(t.games, G * sizeof(az::GameState));
    AZ_SEARCH_ALLOC(t.node_hash, G * t.node_cap * sizeof(az::u64));
    AZ_SEARCH_ALLOC(t.hist_hash, G * az::kMaxHistory * sizeof(az::u64));
    AZ_SEARCH_ALLOC(t.hist_rep, G * az::kMaxHistory);
    AZ_SEARCH_ALLOC(s->roots_stage, G * (size_t)t.stride);
    AZ_SEARCH_ALLOC(s->out_actions, G * AZ_MAX_LEGAL * sizeof(int));
    AZ_SEARCH_ALLOC(s->out_visits, G * AZ_MAX_LEGAL * sizeof(int));
    AZ_SEARCH_ALLOC(s->out_counts, G * sizeof(int));
    cudaMemset(s->out_actions, 0, G * AZ_MAX_LEGAL * sizeof(int));
    cudaMemset(s->out_visits, 0, G * AZ_MAX_LEGAL * sizeof(int));
    if (s->net && n_groups == 2) {
        rc = az::ensure_second_workspace(*s->net, &s->second_workspace);
        if (rc != AZ_OK) { az::free_search(s); return rc; }
    }
    for (int gi = 0; gi < n_groups; ++gi) {
        az::Group &g = s->groups[gi];
        g.game0 = gi * per_group;
        g.n_games = (int)G - g.game0 < per_group ? (int)G - g.game0 : per_group;
        g.rows = g.n_games * (int)c->leaves;
        // without a second evaluation workspace both groups take turns on one stream
        if (gi == 1 && s->net && !s->second_workspace) g.stream = s->groups[0].stream;
        else {
            if (cudaStreamCreateWithFlags(&g.owned, cudaStreamNonBlocking) != cudaSuccess) { az::free_search(s); return AZ_ERR_CUDA; }
            g.stream = g.owned;
        }
        if (cudaEventCreateWithFlags(&g.done, cudaEventDisableTiming) != cudaSuccess) { az::free_search(s); return AZ_ERR_CUDA; }
        const size_t R = (size_t)g.rows;
        AZ_SEARCH_ALLOC(g.batch.pos, R * t.stride);
        AZ_SEARCH_ALLOC(g.batch.kind, R * sizeof(int));
        AZ_SEARCH_ALLOC(g.batch.leaf, R * sizeof(int));
        AZ_SEARCH_ALLOC(g.batch.depth, R * sizeof(int));
        AZ_SEARCH_ALLOC(g.batch.path_e, R * az::kMaxDepth * sizeof(int));
        AZ_SEARCH_ALLOC(g.batch.path_n, R * az::kMaxDepth * sizeof(int));
        AZ_SEARCH_ALLOC(g.masks, R * s->words * sizeof(uint64_t));
        AZ_SEARCH_ALLOC(g.legal, R * AZ_MAX_LEGAL * sizeof(float));
        AZ_SEARCH_ALLOC(g.value, R * s->vs * sizeof(float));
        AZ_SEARCH_ALLOC(g.counts, R * sizeof(int));
    }
#undef AZ_SEARCH_ALLOC
    if (cudaEventCreate(&s->ev_begin) != cudaSuccess || cudaEventCreate(&s->ev_end) != cudaSuccess) { az::free_search(s); return AZ_ERR_CUDA; }
    *out = reinterpret_cast<az_search *>(s);
    return AZ_OK;
}

void az_search_destroy(az_search *search) { az::free_search(reinterpret_cast<Search *>(search)); }

int az_search_set_roots(az_search *search, const void *positions_host) {
    Search *s = reinterpret_cast<Search *>(search);
    if (!s || !positions_host) return AZ_ERR_BAD_ARG;
    if (s->pending) return AZ_ERR_BUSY;
    const az::Trees &t = s->trees;
    cudaStream_t st = s->groups[0].stream;
    AZ_CUDA(cudaMemcpyAsync(s->roots_stage, positions_host, (size_t)s->cfg.games * t.stride, cudaMemcpyHostToDevice, st));
    az::reset_trees_kernel<<<s->cfg.games, 32, 0, st>>>(t, s->roots_stage, (int)s->cfg.games, nullptr);
    AZ_LAUNCH_CHECK();
    // the rows of every group's batch must hold valid records from the first step on (rows that idle are still evaluated)
    for (int gi = 0; gi < s->n_groups; ++gi) {
        az::Group &g = s->groups[gi];
        for (uint32_t j = 0; j < s->cfg.leaves; ++j)
            AZ_CUDA(cudaMemcpy2DAsync(g.batch.pos + (size_t)j * t.stride, (size_t)t.stride * s->cfg.leaves,
                                      s->roots_stage + (size_t)g.game0 * t.stride, (size_t)t.stride, (size_t)t.stride,
                                      (size_t)g.n_games, cudaMemcpyDeviceToDevice, st));
    }
    AZ_CUDA(cudaStreamSynchronize(st));
    s->need_root_step = true;
    return AZ_OK;
}

int az_search_replace_roots(az_search *search, const int32_t *games_host, int count, const void *positions_host) {
    Search *s = reinterpret_cast<Search *>(search);
    if (!s || count < 0 || (uint32_t)count > s->cfg.games) return AZ_ERR_BAD_ARG;
    if (count == 0) return AZ_OK;
    if (!games_host || !positions_host) return AZ_ERR_BAD_ARG;
    if (s->pending) return AZ_ERR_BUSY;
    {
        std::vector<bool> seen(s->cfg.games, false);
        for (int i = 0; i < count; ++i) {
            if (games_host[i] < 0 || (uint32_t)games_host[i] >= s->cfg.games || seen[games_host[i]]) return AZ_ERR_BAD_ARG;
            seen[games_host[i]] = true;
        }
    }
    const az::Trees &t = s->trees;
    cudaStream_t st = s->groups[0].stream;
    AZ_CUDA(cudaMemcpyAsync(s->roots_stage, positions_host, (size_t)count * t.stride, cudaMemcpyHostToDevice, st));
    AZ_CUDA(cudaMemcpyAsync(s->out_counts, games_host, (size_t)count * sizeof(int), cudaMemcpyHostToDevice, st));   // borrowed as the index list
    az::reset_trees_kernel<<<(unsigned)count, 32, 0, st>>>(t, s->roots_stage, count, s->out_counts);
    AZ_LAUNCH_CHECK();
    AZ_CUDA(cudaStreamSynchronize(st));
    s->need_root_step = true;
    return AZ_OK;
}

int az_search_run_async(az_search *search, int simulations) {
    Search *s = reinterpret_cast<Search *>(search);
    if (!s || simulations < 0) return AZ_ERR_BAD_ARG;
    if (s->pending) return AZ_ERR_BUSY;
    cudaStream_t s0 = s->groups[0].stream;
    cudaStream_t s1 = s->n_groups == 2 ? s->groups[1].stream : s0;
    AZ_CUDA(cudaEventRecord(s->ev_begin, s0));
    if (s1 != s0) AZ_CUDA(cudaStreamWaitEvent(s1, s->ev_begin, 0));
    // a tree whose root has not been evaluated spends a step on that; the other trees sit that step out
    const int steps = simulations + (s->need_root_step ? 1 : 0);
    for (int step = 0; step < steps; ++step)
        for (int gi = 0; gi < s->n_groups; ++gi) {
            const int rc = az::queue_step(*s, gi, s->need_root_step && step == 0);
            if (rc != AZ_OK) {
                // kernels of earlier steps may already be queued on both streams and still use the trees: let them
                // finish before the caller gets the error (and may destroy the search or set new roots)
                cudaStreamSynchronize(s0);
                if (s1 != s0) cudaStreamSynchronize(s1);
                return rc;
            }
        }
    if (s1 != s0) {
        AZ_CUDA(cudaEventRecord(s->groups[1].done, s1));
        AZ_CUDA(cudaStreamWaitEvent(s0, s->groups[1].done, 0));
    }
    AZ_CUDA(cudaEventRecord(s->ev_end, s0));
    s->need_root_step = false;
    s->pending = true;
    return AZ_OK;
}

int az_search_wait(az_search *search, float *elapsed_ms_out) {
    Search *s = reinterpret_cast<Search *>(search);
    if (!s || !s->pending) return AZ_ERR_BAD_ARG;
    s->pending = false;
    AZ_CUDA(cudaEventSynchronize(s->ev_end));
    if (elapsed_ms_out) AZ_CUDA(cudaEventElapsedTime(elapsed_ms_out, s->ev_begin, s->ev_end));
    if (s->net) {
        uint32_t status = 0;
        AZ_CUDA(cudaMemcpy(&status, s->net->status_dev, sizeof status, cudaMemcpyDeviceToHost));
        if (status & az::kStatusWaitTimeout) return AZ_ERR_DEVICE_TIMEOUT;
    }
    return AZ_OK;
}

int az_search_run(az_search *search, int simulations, float *elapsed_ms_out) {
    const int rc = az_search_run_async(search, simulations);
    return rc != AZ_OK ? rc : az_search_wait(search, elapsed_ms_out);
}

int az_search_root(az_search *search, int game, int32_t *actions_host, int32_t *visits_host, float *w_host,
                   float *prior_host, int32_t *count_out) {
    Search *s = reinterpret_cast<Search *>(search);
    if (!s || game < 0 || (uint32_t)game >= s->cfg.games || !actions_host || !visits_host || !w_host || !prior_host || !count_out)
        return AZ_ERR_BAD_ARG;
    if (s->pending) return AZ_ERR_BUSY;
    az::Node root;
    AZ_CUDA(cudaMemcpy(&root, s->trees.nodes + (size_t)game * s->trees.node_cap, sizeof root, cudaMemcpyDeviceToHost));
    const int k = root.n_edges > 0 ? (root.n_edges < AZ_MAX_LEGAL ? root.n_edges : AZ_MAX_LEGAL) : 0;
    *count_out = k;
    if (k == 0) return AZ_OK;
    az::Edge e[AZ_MAX_LEGAL];
    AZ_CUDA(cudaMemcpy(e, s->trees.edges + (size_t)game * s->trees.edge_cap + root.edge_begin, (size_t)k * sizeof(az::Edge), cudaMemcpyDeviceToHost));
    for (int i = 0; i < k; ++i) { actions_host[i] = e[i].action; visits_host[i] = e[i].n; w_host[i] = e[i].w; prior_host[i] = e[i].prior; }
    return AZ_OK;
}

int az_search_root_visits(az_search *search, int32_t *actions_host, int32_t *visits_host, int32_t *counts_host) {
    Search *s = reinterpret_cast<Search *>(search);
    if (!s || !actions_host || !visits_host || !counts_host) return AZ_ERR_BAD_ARG;
    if (s->pending) return AZ_ERR_BUSY;
    cudaStream_t st = s->groups[0].stream;
    const size_t G = s->cfg.games;
    az::gather_roots_kernel<<<(unsigned)G, 64, 0, st>>>(s->trees, (int)G, s->out_actions, s->out_visits, s->out_counts);
    AZ_LAUNCH_CHECK();
    AZ_CUDA(cudaMemcpyAsync(counts_host, s->out_counts, G * sizeof(int), cudaMemcpyDeviceToHost, st));
    AZ_CUDA(cudaMemcpyAsync(actions_host, s->out_actions, G * AZ_MAX_LEGAL * sizeof(int), cudaMemcpyDeviceToHost, st));
    AZ_CUDA(cudaMemcpyAsync(visits_host, s->out_visits, G * AZ_MAX_LEGAL * sizeof(int), cudaMemcpyDeviceToHost, st));
    AZ_CUDA(cudaStreamSynchronize(st));
    return AZ_OK;
}

int az_search_advance(az_search *search, const int32_t *actions_host, int32_t *played_host) {
    Search *s = reinterpret_cast<Search *>(search);
    if (!s) return AZ_ERR_BAD_ARG;
    if (s->pending) return AZ_ERR_BUSY;
    az::Trees &t = s->trees;
    const size_t G = s->cfg.games;
    cudaStream_t st = s->groups[0].stream;
    if (!s->alt_nodes) {
        AZ_CUDA(cudaMalloc((void **)&s->alt_nodes, G * t.node_cap * sizeof(az::Node)));
        AZ_CUDA(cudaMalloc((void **)&s->alt_edges, G * t.edge_cap * sizeof(az::Edge)));
        AZ_CUDA(cudaMalloc((void **)&s->alt_node_pos, G * t.node_cap * (size_t)t.stride));
        AZ_CUDA(cudaMalloc((void **)&s->alt_node_hash, G * t.node_cap * sizeof(az::u64)));
        AZ_CUDA(cudaMalloc((void **)&s->remap, G * 2 * t.node_cap * sizeof(int)));
        AZ_CUDA(cudaMalloc((void **)&s->adv_actions, G * sizeof(int)));
        AZ_CUDA(cudaMalloc((void **)&s->adv_played, G * sizeof(int)));
        AZ_CUDA(cudaMalloc((void **)&s->adv_fresh, sizeof(int)));
    }
    if (actions_host) AZ_CUDA(cudaMemcpyAsync(s->adv_actions, actions_host, G * sizeof(int), cudaMemcpyHostToDevice, st));
    AZ_CUDA(cudaMemsetAsync(s->adv_fresh, 0, sizeof(int), st));
    az::search_advance_kernel<<<(unsigned)((G + az::kWarps - 1) / az::kWarps), 32 * az::kWarps, 0, st>>>(
        t, s->alt_nodes, s->alt_edges, s->alt_node_pos, s->alt_node_hash, (int)G, actions_host ? s->adv_actions : nullptr, s->adv_played, s->remap, s->adv_fresh);
    AZ_LAUNCH_CHECK();
    int fresh = 0;
    if (played_host) AZ_CUDA(cudaMemcpyAsync(played_host, s->adv_played, G * sizeof(int), cudaMemcpyDeviceToHost, st));
    AZ_CUDA(cudaMemcpyAsync(&fresh, s->adv_fresh, sizeof(int), cudaMemcpyDeviceToHost, st));
    AZ_CUDA(cudaStreamSynchronize(st));
    std::swap(t.nodes, s->alt_nodes);
    std::swap(t.edges, s->alt_edges);
    std::swap(t.node_pos, s->alt_node_pos);
    std::swap(t.node_hash, s->alt_node_hash);
    if (fresh) s->need_root_step = true;
    return AZ_OK;
}

int az_search_root_noise(az_search *search, const float *noise_host, float epsilon, int32_t *changed_host) {
    Search *s = reinterpret_cast<Search *>(search);
    if (!s || !noise_host || !(epsilon >= 0.0f && epsilon <= 1.0f)) return AZ_ERR_BAD_ARG;
    if (s->pending) return AZ_ERR_BUSY;
    const size_t G = s->cfg.games;
    cudaStream_t st = s->groups[0].stream;
    // the read-out buffers double as staging: visits (int32 [games][AZ_MAX_LEGAL]) holds the noise, counts the answer
    float *noise_dev = reinterpret_cast<float *>(s->out_visits);
    AZ_CUDA(cudaMemcpyAsync(noise_dev, noise_host, G * AZ_MAX_LEGAL * sizeof(float), cudaMemcpyHostToDevice, st));
    az::root_noise_kernel<<<(unsigned)G, 64, 0, st>>>(s->trees, (int)G, noise_dev, epsilon, s->out_counts);
    AZ_LAUNCH_CHECK();
    if (changed_host) AZ_CUDA(cudaMemcpyAsync(changed_host, s->out_counts, G * sizeof(int), cudaMemcpyDeviceToHost, st));
    AZ_CUDA(cudaStreamSynchronize(st));
    return AZ_OK;
}

int az_search_root_positions(az_search *search, void *positions_host) {
    Search *s = reinterpret_cast<Search *>(search);
    if (!s || !positions_host) return AZ_ERR_BAD_ARG;
    if (s->pending) return AZ_ERR_BUSY;
    const az::Trees &t = s->trees;
    AZ_CUDA(cudaMemcpy2D(positions_host, (size_t)t.stride, t.node_pos, (size_t)t.node_cap * t.stride, (size_t)t.stride,
                         (size_t)s->cfg.games, cudaMemcpyDeviceToHost));
    return AZ_OK;
}

int az_search_tree(az_search *search, int game, int32_t *counts_out, int32_t *node_visits_host, float *node_value_sum_host) {
    Search *s = reinterpret_cast<Search *>(search);
    if (!s || game < 0 || (uint32_t)game >= s->cfg.games || !counts_out) return AZ_ERR_BAD_ARG;
    if (s->pending) return AZ_ERR_BUSY;
    az::GameState gs;
    AZ_CUDA(cudaMemcpy(&gs, s->trees.games + game, sizeof gs, cudaMemcpyDeviceToHost));
    counts_out[0] = gs.n_nodes; counts_out[1] = gs.n_edges; counts_out[2] = gs.flags; counts_out[3] = gs.idle;
    if (node_visits_host || node_value_sum_host) {
        az::Node *host = new (std::nothrow) az::Node[(size_t)gs.n_nodes];
        if (!host) return AZ_ERR_BAD_ARG;
        cudaError_t e = cudaMemcpy(host, s->trees.nodes + (size_t)game * s->trees.node_cap, (size_t)gs.n_nodes * sizeof(az::Node), cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) { delete[] host; az::set_cuda_error(e, "cudaMemcpy (tree)"); return AZ_ERR_CUDA; }
        for (int i = 0; i < gs.n_nodes; ++i) {
            if (node_visits_host) node_visits_host[i] = host[i].nvis;
            if (node_value_sum_host) node_value_sum_host[i] = host[i].wsum;
        }
        delete[] host;
    }
    return AZ_OK;
}

int az_search_launches_per_step(const az_search *search) {
    const Search *s = reinterpret_cast<const Search *>(search);
    if (!s) return 0;
    const int eval = s->net ? az_launches_per_evaluate(reinterpret_cast<const az_net *>(s->net), s->groups[0].rows) : 1;
    return 3 + eval;
}

}  // extern "C"
