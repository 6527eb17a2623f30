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

}  // namespace
}  // namespace az
