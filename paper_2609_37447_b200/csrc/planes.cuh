// Position records and the value of every input plane (App. D.1, Table D.1 conventions), shared by
// the stand-alone encoder kernel and by the tower kernel, which encodes its boards directly into
// its shared-memory frame.
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace az {
namespace {

struct alignas(8) PosCur {
    unsigned long long pieces[12];
    unsigned char stm, castling, ep_square, halfmove, repetitions, pad[3];
};
struct alignas(8) PosH8 {
    PosCur cur;
    unsigned long long hist_pieces[7][12];
    unsigned char hist_rep[7];
    unsigned char n_hist;
};

template <typename T> __device__ __forceinline__ T to_act(float v);
template <> __device__ __forceinline__ float to_act<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 to_act<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// value of one channel of the 19-plane layout at absolute square s
__device__ __forceinline__ float plane19(const PosCur *r, int ch, int s, float hm) {
    const int stm = r->stm;
    if (ch < 12) {
        const int own = ch < 6;
        const int idx = ((stm != 0) == (own != 0) ? 6 : 0) + (ch % 6);   // own pieces of Black sit at 6..11
        return (float)((r->pieces[idx] >> s) & 1ull);
    }
    const int c = r->castling;
    switch (ch) {
        case 12: return (float)stm;
        case 13: return (float)((c >> (stm ? 2 : 0)) & 1);
        case 14: return (float)((c >> (stm ? 3 : 1)) & 1);
        case 15: return (float)((c >> (stm ? 0 : 2)) & 1);
        case 16: return (float)((c >> (stm ? 1 : 3)) & 1);
        case 17: return hm;
        case 18: return r->repetitions >= 1 ? 1.0f : 0.0f;
        default: return 0.0f;
    }
}

__device__ __forceinline__ float plane112(const PosH8 *h, int ch, int s, float hm) {
    const PosCur *r = &h->cur;
    const int stm = r->stm;
    if (ch < 104) {
        const int t = ch / 13, k = ch % 13;
        if (t > h->n_hist) return 0.0f;
        if (k == 12) return (t == 0 ? r->repetitions : h->hist_rep[t - 1]) >= 1 ? 1.0f : 0.0f;
        const int own = k < 6;
        const int idx = ((stm != 0) == (own != 0) ? 6 : 0) + (k % 6);
        const unsigned long long bb = t == 0 ? r->pieces[idx] : h->hist_pieces[t - 1][idx];
        return (float)((bb >> s) & 1ull);
    }
    const int c = r->castling;
    switch (ch) {
        case 104: return (float)((c >> (stm ? 2 : 0)) & 1);
        case 105: return (float)((c >> (stm ? 3 : 1)) & 1);
        case 106: return (float)((c >> (stm ? 0 : 2)) & 1);
        case 107: return (float)((c >> (stm ? 1 : 3)) & 1);
        case 108: return (float)stm;
        case 109: return hm;
        case 111: return 1.0f;
        default: return 0.0f;
    }
}


// halfmove plane: the clock capped at 100, divided by 100 in IEEE single precision
__device__ __forceinline__ float halfmove_plane(const PosCur *r) {
    const int hmc = r->halfmove > 100 ? 100 : r->halfmove;
    return __fdiv_rn((float)hmc, 100.0f);
}

// eight consecutive channels [c0, c0+8) of one square as bf16 (channels >= in_planes are zero);
// `s` is the absolute square of the mover-oriented square being encoded
__device__ __forceinline__ uint4 planes_chunk8_bf16(const PosCur *r, int in_planes, int c0, int s, float hm) {
    uint32_t pk[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        float f[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int ch = c0 + 2 * j + e;
            f[e] = ch >= in_planes ? 0.0f
                 : in_planes == 19 ? plane19(r, ch, s, hm)
                                   : plane112(reinterpret_cast<const PosH8 *>(r), ch, s, hm);
        }
        const __nv_bfloat162 h2 = __floats2bfloat162_rn(f[0], f[1]);
        pk[j] = *reinterpret_cast<const uint32_t *>(&h2);
    }
    return make_uint4(pk[0], pk[1], pk[2], pk[3]);
}

// All 32 (19 + padding) channels of one square of the 19-plane layout as four 16-byte bf16 chunks,
// for a caller on a latency-critical path: the record's thirteen words are fetched with independent
// loads (one memory round trip) and every channel is then a bit test in registers.  `c` is the
// mover-oriented square.  Bit-identical to planes_chunk8_bf16 / plane19.
__device__ __forceinline__ void planes19_bf16(const PosCur *r, int c, uint4 (&out)[4]) {
    unsigned long long w[13];
    const unsigned long long *src = reinterpret_cast<const unsigned long long *>(r);
#pragma unroll
    for (int i = 0; i < 13; ++i) w[i] = __ldg(src + i);
    const unsigned int tail = (unsigned int)w[12];          // stm, castling, ep_square, halfmove
    const unsigned int tail_hi = (unsigned int)(w[12] >> 32);   // repetitions, padding
    const int stm = tail & 0xff, castling = (tail >> 8) & 0xff, halfmove = (tail >> 24) & 0xff;
    const int repetitions = tail_hi & 0xff;
    const int s = stm ? (c ^ 56) : c;
    const unsigned int one = 0x3F80u;                       // bf16 1.0
    unsigned int v[32];
#pragma unroll
    for (int k = 0; k < 6; ++k) {
        const unsigned long long own = stm ? w[6 + k] : w[k], opp = stm ? w[k] : w[6 + k];
        v[k] = ((own >> s) & 1ull) ? one : 0u;
        v[6 + k] = ((opp >> s) & 1ull) ? one : 0u;
    }
    v[12] = stm ? one : 0u;
    v[13] = ((castling >> (stm ? 2 : 0)) & 1) ? one : 0u;
    v[14] = ((castling >> (stm ? 3 : 1)) & 1) ? one : 0u;
    v[15] = ((castling >> (stm ? 0 : 2)) & 1) ? one : 0u;
    v[16] = ((castling >> (stm ? 1 : 3)) & 1) ? one : 0u;
    const __nv_bfloat16 hm = __float2bfloat16_rn(__fdiv_rn((float)(halfmove > 100 ? 100 : halfmove), 100.0f));
    v[17] = (unsigned int)*reinterpret_cast<const unsigned short *>(&hm);
    v[18] = repetitions >= 1 ? one : 0u;
#pragma unroll
    for (int k = 19; k < 32; ++k) v[k] = 0u;
#pragma unroll
    for (int j = 0; j < 4; ++j)
        out[j] = make_uint4(v[8 * j] | (v[8 * j + 1] << 16), v[8 * j + 2] | (v[8 * j + 3] << 16),
                            v[8 * j + 4] | (v[8 * j + 5] << 16), v[8 * j + 6] | (v[8 * j + 7] << 16));
}


// ---- the 52 planes of the paper's own network (App. D.1, Table D.1), one square at a time ----
typedef unsigned long long u64;

struct alignas(8) PosM8 {
    u64 pieces[12];
    unsigned char stm, castling, ep_square, halfmove, repetitions, pad[3];
    unsigned char move_from[8], move_to[8];
    unsigned char n_moves, pad2[7];
};
static_assert(sizeof(PosM8) == 128, "record with the last eight moves");

constexpr u64 kFileA = 0x0101010101010101ull, kFileH = kFileA << 7;
constexpr u64 kFileAB = kFileA | (kFileA << 1), kFileGH = kFileH | (kFileH >> 1);

__device__ __forceinline__ u64 knight_reach(u64 b) {
    return ((b << 17) & ~kFileA) | ((b << 15) & ~kFileH) | ((b << 10) & ~kFileAB) | ((b << 6) & ~kFileGH) |
           ((b >> 17) & ~kFileH) | ((b >> 15) & ~kFileA) | ((b >> 10) & ~kFileGH) | ((b >> 6) & ~kFileAB);
}
// first occupied square met from sq in direction (df, dr), as a bit (0 if the edge comes first)
__device__ __forceinline__ u64 first_hit(int sq, int df, int dr, u64 occ) {
    int f = (sq & 7) + df, r = (sq >> 3) + dr;
    while (f >= 0 && f < 8 && r >= 0 && r < 8) {
        const u64 b = 1ull << (r * 8 + f);
        if (occ & b) return b;
        f += df; r += dr;
    }
    return 0;
}


// all 64 channel values (52 used) of tensor square c (row * 8 + column in the mover's orientation)
__device__ __forceinline__ void planes52_square(const PosM8 *r, int c, float (&v)[64]) {
    const int stm = r->stm & 1;
    const int flip = stm ? 56 : 0;
    const int s = c ^ flip;                                   // absolute square of this tensor square
    const u64 sb = 1ull << s;
    u64 own[6], opp[6];
#pragma unroll
    for (int k = 0; k < 6; ++k) { own[k] = r->pieces[stm * 6 + k]; opp[k] = r->pieces[(stm ^ 1) * 6 + k]; }
    u64 own_occ = 0, opp_occ = 0;
#pragma unroll
    for (int k = 0; k < 6; ++k) { own_occ |= own[k]; opp_occ |= opp[k]; }
    const u64 occ = own_occ | opp_occ;

    // the opponent pieces that give check
    u64 checkers = 0;
    if (own[5]) {
        const u64 kb = own[5] & (~own[5] + 1);
        const int ks = __ffsll((long long)kb) - 1;
        const u64 pawn_from = stm == 0 ? (((kb << 7) & ~kFileH) | ((kb << 9) & ~kFileA))
                                       : (((kb >> 7) & ~kFileA) | ((kb >> 9) & ~kFileH));
        checkers = (pawn_from & opp[0]) | (knight_reach(kb) & opp[1]);
        const u64 diag = first_hit(ks, 1, 1, occ) | first_hit(ks, 1, -1, occ) | first_hit(ks, -1, 1, occ) | first_hit(ks, -1, -1, occ);
        const u64 line = first_hit(ks, 1, 0, occ) | first_hit(ks, -1, 0, occ) | first_hit(ks, 0, 1, occ) | first_hit(ks, 0, -1, occ);
        checkers |= (diag & (opp[2] | opp[4])) | (line & (opp[3] | opp[4]));
    }

#pragma unroll
    for (int k = 0; k < 6; ++k) {
        v[k] = (own[k] & sb) ? 1.0f : 0.0f;
        v[6 + k] = (opp[k] & sb) ? 1.0f : 0.0f;
    }
    const int cr = r->castling;
    v[12] = (float)((cr >> (stm ? 2 : 0)) & 1);
    v[13] = (float)((cr >> (stm ? 3 : 1)) & 1);
    v[14] = (float)((cr >> (stm ? 0 : 2)) & 1);
    v[15] = (float)((cr >> (stm ? 1 : 3)) & 1);
    v[16] = (own_occ & sb) ? 1.0f : 0.0f;
    v[17] = (opp_occ & sb) ? 1.0f : 0.0f;
    v[18] = (checkers & sb) ? 1.0f : 0.0f;
    v[19] = (r->ep_square < 64 && r->ep_square == s) ? 1.0f : 0.0f;
    v[20] = r->repetitions >= 1 ? 1.0f : 0.0f;
    v[21] = r->repetitions >= 2 ? 1.0f : 0.0f;
    const int nm = r->n_moves > 8 ? 8 : r->n_moves;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
        v[22 + 2 * t] = (t < nm && r->move_from[t] == s) ? 1.0f : 0.0f;
        v[23 + 2 * t] = (t < nm && r->move_to[t] == s) ? 1.0f : 0.0f;
    }
    v[38] = (((c >> 3) + (c & 7)) & 1) == 0 ? 1.0f : 0.0f;    // fixed in tensor coordinates, corner (0, 0) set
    {
        // exactly one bishop each, on squares of different colour
        const bool one_each = __popcll(own[2]) == 1 && __popcll(opp[2]) == 1;
        const int a = __ffsll((long long)own[2]) - 1, b = __ffsll((long long)opp[2]) - 1;
        v[39] = (one_each && ((((a & 7) + (a >> 3)) ^ ((b & 7) + (b >> 3))) & 1)) ? 1.0f : 0.0f;
    }
#pragma unroll
    for (int k = 0; k < 6; ++k) v[40 + k] = (float)(__popcll(own[k]) - __popcll(opp[k]));
    v[46] = (float)(r->halfmove > 100 ? 100 : r->halfmove);
#pragma unroll
    for (int k = 0; k < 5; ++k) v[47 + k] = (float)__popcll(own[k]);
#pragma unroll
    for (int k = 52; k < 64; ++k) v[k] = 0.0f;

}

}  // namespace
}  // namespace az
