// Legal-move masks on the GPU (App. D.1: illegal actions are masked before the softmax; castling
// is the king-to-own-rook pair, en passant the pawn's ordinary origin-destination pair).
//
// Bitboard move generation, one warp per position: pseudo-legal target sets per piece from
// shift/ray arithmetic (one lane per square pair), then every listed move tried on a copy of the
// bitboards (moves dealt out over the lanes) and kept if the mover's king is not attacked
// afterwards.  The mask row is built in shared memory and written once.  The work per position is
// a few thousand integer operations; masks are an input of az_evaluate, so the kernel runs off
// that call's timed path.
#include "common.cuh"
#include "chess.cuh"

#include <mutex>

namespace az {
namespace {

// flat-1858 index tables, built on the host once per device
__device__ short g_flat_pair[64 * 64];
__device__ short g_flat_promo[8 * 3];

template <int HEAD>
__device__ __forceinline__ void set_move(u64 *row, int stm, int from, int to, int promo) {
    // mover-oriented coordinates: reflect ranks for Black
    if (stm) { from ^= 56; to ^= 56; }
    int idx;
    if (HEAD == AZ_POLICY_PLANES73) {
        const int df = (to & 7) - (from & 7), dr = (to >> 3) - (from >> 3);
        int plane;
        if (promo) {                                     // under-promotion: 1 N, 2 B, 3 R
            plane = 64 + 3 * (promo - 1) + (df + 1);
        } else {
            const int adf = df < 0 ? -df : df, adr = dr < 0 ? -dr : dr;
            if (adf != adr && adf != 0 && adr != 0) {     // knight jump
                // (1,2)=0 (2,1)=1 (2,-1)=2 (1,-2)=3 (-1,-2)=4 (-2,-1)=5 (-2,1)=6 (-1,2)=7
                const int k = df > 0 ? (dr > 0 ? (adf == 1 ? 0 : 1) : (adf == 2 ? 2 : 3))
                                     : (dr < 0 ? (adf == 1 ? 4 : 5) : (adf == 2 ? 6 : 7));
                plane = 56 + k;
            } else {
                // N=0 NE=1 E=2 SE=3 S=4 SW=5 W=6 NW=7
                const int d = df == 0 ? (dr > 0 ? 0 : 4)
                            : df > 0 ? (dr > 0 ? 1 : dr == 0 ? 2 : 3)
                                     : (dr < 0 ? 5 : dr == 0 ? 6 : 7);
                plane = 7 * d + (adf > adr ? adf : adr) - 1;
            }
        }
        idx = plane * 64 + from;
    } else if (HEAD == AZ_POLICY_FLAT1858) {
        idx = promo ? g_flat_promo[(from & 7) * 3 + ((to & 7) - (from & 7) + 1)] + (promo - 1)
                    : g_flat_pair[from * 64 + to];
    } else {
        // the paper's 1,880 actions: the same pairs, then four promotion pieces per (file, direction) in the
        // order queen, rook, bishop, knight (promo 4, 3, 2, 1); the 1,858 table numbers three per combination
        idx = promo ? 1792 + 4 * ((g_flat_promo[(from & 7) * 3 + ((to & 7) - (from & 7) + 1)] - 1792) / 3) + (4 - promo)
                    : g_flat_pair[from * 64 + to];
    }
    atomicOr(row + (idx >> 6), 1ull << (idx & 63));          // the row sits in shared memory, lanes share it
}

// One warp per position.  Step 1: lane L looks at squares L and L + 32; if one of the mover's pieces
// stands there it lists that piece's pseudo-legal moves in shared memory.  Step 2: the listed moves
// are dealt out over the 32 lanes; each is tried on a copy of the bitboards and, if the mover's king
// is not attacked afterwards, its bit (four bits for a promotion) is set in the shared mask row.
constexpr int kWarpsPerBlock = 4;
constexpr int kMaxListed = 384;            // pseudo-legal moves of one position (218 legal at most in chess)

template <int HEAD>
__global__ void __launch_bounds__(32 * kWarpsPerBlock)
legal_masks_kernel(const unsigned char *__restrict__ positions, size_t stride, int batch,
                   u64 *__restrict__ masks) {
    constexpr int WORDS = HEAD == AZ_POLICY_PLANES73 ? 73 : 30;
    __shared__ u64 s_row[kWarpsPerBlock][WORDS];
    __shared__ unsigned s_list[kWarpsPerBlock][kMaxListed];
    __shared__ int s_count[kWarpsPerBlock];
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int pos = blockIdx.x * kWarpsPerBlock + w;
    if (pos >= batch) return;                                // whole warps leave together
    const PosCur *r = reinterpret_cast<const PosCur *>(positions + (size_t)pos * stride);
    u64 own[6], opp[6];
    const int stm = r->stm & 1;
#pragma unroll
    for (int k = 0; k < 6; ++k) { own[k] = r->pieces[stm * 6 + k]; opp[k] = r->pieces[(stm ^ 1) * 6 + k]; }
    u64 own_occ = 0, opp_occ = 0;
#pragma unroll
    for (int k = 0; k < 6; ++k) { own_occ |= own[k]; opp_occ |= opp[k]; }
    const u64 occ = own_occ | opp_occ;
    const int them = stm ^ 1;
    const int king_sq = own[5] ? __ffsll((long long)own[5]) - 1 : 0;
    const int ep = r->ep_square;
    u64 *row = s_row[w];
    unsigned *list = s_list[w];
    for (int i = lane; i < WORDS; i += 32) row[i] = 0;
    if (lane == 0) s_count[w] = 0;
    __syncwarp();

    // ---- step 1: pseudo-legal moves, entry = kind | from << 3 | to << 9
#pragma unroll 1
    for (int half = 0; half < 2; ++half) {
        const int from = lane + 32 * half;
        const u64 fb = 1ull << from;
        if (!(own_occ & fb)) continue;
        int k = 0;
#pragma unroll
        for (int j = 1; j < 6; ++j) if (own[j] & fb) k = j;
        u64 targets;
        if (k == 0) {
            u64 push, cap;
            if (stm == 0) {
                push = (fb << 8) & ~occ;
                if (push && (from >> 3) == 1) push |= (fb << 16) & ~occ;
                cap = (((fb << 9) & ~FILE_A) | ((fb << 7) & ~FILE_H));
            } else {
                push = (fb >> 8) & ~occ;
                if (push && (from >> 3) == 6) push |= (fb >> 16) & ~occ;
                cap = (((fb >> 9) & ~FILE_H) | ((fb >> 7) & ~FILE_A));
            }
            const u64 ep_bit = ep < 64 ? (1ull << ep) : 0ull;
            targets = push | (cap & (opp_occ | (ep_bit & ~occ)));
        } else if (k == 1) targets = knight_set(fb) & ~own_occ;
        else if (k == 5) targets = king_set(fb) & ~own_occ;
        else {
            targets = 0;
            if (k != 3) targets |= ray_set(from, occ, true);
            if (k != 2) targets |= ray_set(from, occ, false);
            targets &= ~own_occ;
        }
        int at = atomicAdd(&s_count[w], __popcll(targets));
        while (targets) {
            const int to = __ffsll((long long)targets) - 1;
            targets &= targets - 1;
            if (at < kMaxListed) list[at] = (unsigned)k | ((unsigned)from << 3) | ((unsigned)to << 9);
            ++at;
        }
    }
    __syncwarp();
    const int listed = min(s_count[w], kMaxListed);

    // ---- step 2: keep the moves that do not leave the mover's king attacked
    for (int i = lane; i < listed; i += 32) {
        const unsigned e = list[i];
        const int k = e & 7, from = (e >> 3) & 63, to = (e >> 9) & 63;
        const u64 fb = 1ull << from, tb = 1ull << to;
        u64 o[6];
#pragma unroll
        for (int j = 0; j < 6; ++j) o[j] = opp[j] & ~tb;
        u64 n_occ = (occ & ~fb) | tb;
        if (k == 0 && to == ep && ((from ^ to) & 7) != 0 && !((opp_occ >> to) & 1ull)) {
            const int ep_cap = (to & 7) + 8 * (from >> 3);   // the pawn taken en passant leaves the board too
            o[0] &= ~(1ull << ep_cap);
            n_occ &= ~(1ull << ep_cap);
        }
        if (attacked(k == 5 ? to : king_sq, them, o, n_occ)) continue;
        const bool promotes = k == 0 && ((to >> 3) == (stm ? 0 : 7));
        if (HEAD == AZ_POLICY_FROMTO1880 && promotes) {
            // a promoting move has only its four promotion actions
            set_move<HEAD>(row, stm, from, to, 1);
            set_move<HEAD>(row, stm, from, to, 2);
            set_move<HEAD>(row, stm, from, to, 3);
            set_move<HEAD>(row, stm, from, to, 4);
            continue;
        }
        set_move<HEAD>(row, stm, from, to, 0);               // plain pair (= queen promotion)
        if (promotes) {
            set_move<HEAD>(row, stm, from, to, 1);
            set_move<HEAD>(row, stm, from, to, 2);
            set_move<HEAD>(row, stm, from, to, 3);
        }
    }
    // castling: rights, king and rook at home, squares between empty, king's path not attacked
    // (lane 0 the king side, lane 1 the queen side)
    if (lane < 2) {
        const int r0 = stm ? 56 : 0;
        const int kbit = stm ? 4 : 1, qbit = stm ? 8 : 2;
        const int c = r->castling;
        if ((c & (kbit | qbit)) && king_sq == r0 + 4 && !attacked(r0 + 4, them, opp, occ)) {
            if (lane == 0 && (c & kbit) && ((own[3] >> (r0 + 7)) & 1ull) && !(occ & (3ull << (r0 + 5))) &&
                !attacked(r0 + 5, them, opp, occ) && !attacked(r0 + 6, them, opp, occ))
                set_move<HEAD>(row, stm, r0 + 4, r0 + 7, 0);
            if (lane == 1 && (c & qbit) && ((own[3] >> r0) & 1ull) && !(occ & (7ull << (r0 + 1))) &&
                !attacked(r0 + 3, them, opp, occ) && !attacked(r0 + 2, them, opp, occ))
                set_move<HEAD>(row, stm, r0 + 4, r0, 0);
        }
    }
    __syncwarp();
    u64 *dst = masks + (size_t)pos * WORDS;
    for (int i = lane; i < WORDS; i += 32) dst[i] = row[i];
}

// ---- host: flat-1858 tables -------------------------------------------------------------------
std::mutex g_table_mutex;
bool g_table_ready[64] = {};

int ensure_tables() {
    int dev = 0;
    AZ_CUDA(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lock(g_table_mutex);
    if (dev < 64 && g_table_ready[dev]) return AZ_OK;
    static short pair[64 * 64];
    static short promo[8 * 3];
    const int next = build_flat_tables(pair, promo);
    AZ_CUDA(cudaMemcpyToSymbol(g_flat_pair, pair, sizeof pair));
    AZ_CUDA(cudaMemcpyToSymbol(g_flat_promo, promo, sizeof promo));
    if (dev < 64) g_table_ready[dev] = true;
    return next == kFlatMoves ? AZ_OK : AZ_ERR_BAD_ARCH;
}

}  // namespace

int launch_legal_masks(const void *positions, size_t stride, int batch, int head, uint64_t *masks,
                       cudaStream_t s) {
    if (batch == 0) return AZ_OK;
    const unsigned char *p = static_cast<const unsigned char *>(positions);
    const int block = 32 * kWarpsPerBlock;
    const unsigned grid = (unsigned)((batch + kWarpsPerBlock - 1) / kWarpsPerBlock);
    if (head == AZ_POLICY_PLANES73) {
        legal_masks_kernel<AZ_POLICY_PLANES73><<<grid, block, 0, s>>>(p, stride, batch, (u64 *)masks);
    } else {
        int rc = ensure_tables();
        if (rc != AZ_OK) return rc;
        if (head == AZ_POLICY_FLAT1858) legal_masks_kernel<AZ_POLICY_FLAT1858><<<grid, block, 0, s>>>(p, stride, batch, (u64 *)masks);
        else legal_masks_kernel<AZ_POLICY_FROMTO1880><<<grid, block, 0, s>>>(p, stride, batch, (u64 *)masks);
    }
    AZ_LAUNCH_CHECK();
    return AZ_OK;
}

}  // namespace az
