// Bitboards and the last eight moves -> the 52 input planes of the paper's network (App. D.1,
// Table D.1): pieces, castling rights, occupancies, checkers, en-passant target, repetition
// flags, recent moves as origin / destination squares, fixed checkerboard, opposite-bishops flag,
// material balances, halfmove clock and piece counts, all from the mover's side (Black to move:
// ranks reflected, colours exchanged, files kept).
//
// Output layout: [position][square][64 channels] (52 used, the rest zero), square = row * 8 + column
// in mover orientation, float32 or bfloat16; every value is a small integer, exact in both.
// One thread per (position, square); the 64 threads of a position read the same 128-byte record
// (broadcast through L1) and each writes its square's channels as consecutive 16-byte stores.
// HBM-bound: 128 B in, 64 * 64 * sizeof(T) out per position.
#include "common.cuh"

namespace az {
namespace {

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

template <typename T> struct Pack;
template <> struct Pack<float> {
    static constexpr int kPer = 4;
    static __device__ __forceinline__ uint4 make(const float *v) {
        return make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
    }
};
template <> struct Pack<__nv_bfloat16> {
    static constexpr int kPer = 8;
    static __device__ __forceinline__ uint4 make(const float *v) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
            w[i] = *reinterpret_cast<const uint32_t *>(&h);
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
};

template <typename T>
__global__ void __launch_bounds__(256)
encode52_kernel(const unsigned char *__restrict__ positions, int batch, T *__restrict__ planes) {
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int pos = (int)(gid >> 6), c = (int)(gid & 63);
    if (pos >= batch) return;
    const PosM8 *r = reinterpret_cast<const PosM8 *>(positions + (size_t)pos * sizeof(PosM8));
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

    float v[64];
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

    T *out = planes + ((size_t)pos * 64 + c) * 64;
#pragma unroll
    for (int c0 = 0; c0 < 64; c0 += Pack<T>::kPer)
        *reinterpret_cast<uint4 *>(out + c0) = Pack<T>::make(v + c0);
}

}  // namespace

int launch_encode52(const void *positions, int batch, bool bf16, void *planes, cudaStream_t s) {
    if (batch == 0) return AZ_OK;
    const long long threads = (long long)batch * 64;
    const int block = 256;
    const unsigned grid = (unsigned)((threads + block - 1) / block);
    const unsigned char *p = static_cast<const unsigned char *>(positions);
    if (bf16) encode52_kernel<__nv_bfloat16><<<grid, block, 0, s>>>(p, batch, static_cast<__nv_bfloat16 *>(planes));
    else encode52_kernel<float><<<grid, block, 0, s>>>(p, batch, static_cast<float *>(planes));
    AZ_LAUNCH_CHECK();
    return AZ_OK;
}

}  // namespace az
