// Bitboard helpers shared by the legal-move kernel and the search kernels: attack sets, the
// attacked-square test, and the host-side numbering of the from-to action lists (App. D.1).
#pragma once

namespace az {
namespace {

typedef unsigned long long u64;

constexpr u64 FILE_A = 0x0101010101010101ull;
constexpr u64 FILE_B = FILE_A << 1;
constexpr u64 FILE_G = FILE_A << 6;
constexpr u64 FILE_H = FILE_A << 7;

struct alignas(8) PosCur {
    u64 pieces[12];
    unsigned char stm, castling, ep_square, halfmove, repetitions, pad[3];
};

__device__ __forceinline__ u64 knight_set(u64 b) {
    return ((b << 17) & ~FILE_A) | ((b << 15) & ~FILE_H) | ((b << 10) & ~(FILE_A | FILE_B)) |
           ((b << 6) & ~(FILE_G | FILE_H)) | ((b >> 17) & ~FILE_H) | ((b >> 15) & ~FILE_A) |
           ((b >> 10) & ~(FILE_G | FILE_H)) | ((b >> 6) & ~(FILE_A | FILE_B));
}
__device__ __forceinline__ u64 king_set(u64 b) {
    return ((b << 1) & ~FILE_A) | ((b >> 1) & ~FILE_H) | (b << 8) | (b >> 8) | ((b << 9) & ~FILE_A) |
           ((b << 7) & ~FILE_H) | ((b >> 7) & ~FILE_A) | ((b >> 9) & ~FILE_H);
}
// squares seen from sq along the four diagonal (diag) or four straight lines, stopping at (and
// including) the first occupied square
__device__ inline u64 ray_set(int sq, u64 occ, bool diag) {
    u64 att = 0;
#pragma unroll
    for (int d = 0; d < 4; ++d) {
        const int df = diag ? ((d & 1) ? -1 : 1) : (d == 0 ? 1 : d == 1 ? -1 : 0);
        const int dr = diag ? ((d & 2) ? -1 : 1) : (d == 2 ? 1 : d == 3 ? -1 : 0);
        int f = (sq & 7) + df, r = (sq >> 3) + dr;
        while (f >= 0 && f < 8 && r >= 0 && r < 8) {
            const u64 b = 1ull << (r * 8 + f);
            att |= b;
            if (occ & b) break;
            f += df; r += dr;
        }
    }
    return att;
}
// is `sq` attacked by side `by` (0 white, 1 black), given that side's bitboards bb[6] and the occupancy
__device__ inline bool attacked(int sq, int by, const u64 *bb, u64 occ) {
    const u64 b = 1ull << sq;
    const u64 pawn_src = by == 0 ? (((b >> 9) & ~FILE_H) | ((b >> 7) & ~FILE_A))
                                 : (((b << 9) & ~FILE_A) | ((b << 7) & ~FILE_H));
    if (pawn_src & bb[0]) return true;
    if (knight_set(b) & bb[1]) return true;
    if (king_set(b) & bb[5]) return true;
    if (ray_set(sq, occ, true) & (bb[2] | bb[4])) return true;
    if (ray_set(sq, occ, false) & (bb[3] | bb[4])) return true;
    return false;
}

// Numbering of the from-to list.  An origin reaches a destination if they share a line or are a
// knight jump apart; entries are numbered by walking origins and destinations upward (1,792 pairs);
// the promotion entries follow, one run per (origin file, destination file) combination: pair[] gets
// each pair's number or -1, promo[file * 3 + step] the first number of the combination's run in the
// 1,858 list (three under-promotions each).  Returns the list's size, 1,858.
inline int build_flat_tables(short *pair, short *promo) {
    short next = 0;
    for (int from = 0; from < 64; ++from) {
        const int ff = from % 8, fr = from / 8;
        for (int to = 0; to < 64; ++to) {
            const int tf = to % 8, tr = to / 8;
            const int a = ff > tf ? ff - tf : tf - ff, b = fr > tr ? fr - tr : tr - fr;
            const bool line = (a == 0) != (b == 0) || (a == b && a != 0);
            const bool jump = a * b == 2;
            pair[from * 64 + to] = (line || jump) ? next++ : (short)-1;
        }
    }
    for (int file = 0; file < 8; ++file)
        for (int step = 0; step < 3; ++step) {
            const int tf = file + step - 1;
            if (tf < 0 || tf > 7) { promo[file * 3 + step] = -1; continue; }
            promo[file * 3 + step] = next;
            next += 3;
        }
    return next;
}

}  // namespace
}  // namespace az
