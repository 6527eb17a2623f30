// Bitboards -> input planes (App. D.1, Table D.1 conventions: side-to-move canonical, ranks
// reflected and colours exchanged for Black to move, files keep their order, flags and scalars
// fill all 64 squares, halfmove clock capped at 100, missing history zero-filled).
//
// Output layout: [position][square][channel], channel count padded to a multiple of 32 with
// zeros, so that one thread writes one square's channels as consecutive 16-byte stores and a warp
// writes one contiguous run.  One thread per (position, square); the bitboards of a position are
// read by all 64 threads of that position from the same words (broadcast through L1).
// HBM-bound: per position 104 B (784 B with history) in, 64 * channels * sizeof(T) out.
#include "common.cuh"

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

template <typename T, int IN_PLANES, int PAD>
__global__ void __launch_bounds__(256)
encode_planes_kernel(const unsigned char *__restrict__ positions, size_t stride, int batch,
                     T *__restrict__ planes, uint32_t *__restrict__ status) {
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int pos = (int)(gid >> 6), c = (int)(gid & 63);
    if (pos >= batch) return;
    const PosCur *r = reinterpret_cast<const PosCur *>(positions + (size_t)pos * stride);
    const int s = r->stm ? (c ^ 56) : c;                    // reflect ranks for Black
    const int hmc = r->halfmove > 100 ? 100 : r->halfmove;
    const float hm = __fdiv_rn((float)hmc, 100.0f);         // single-precision IEEE division
    if (c == 0 && (__popcll(r->pieces[5]) != 1 || __popcll(r->pieces[11]) != 1))
        atomicOr(status, kStatusBadRecord);
    constexpr int PER = 16 / sizeof(T);                     // channels per 16-byte store
    T *out = planes + ((size_t)pos * 64 + c) * PAD;
#pragma unroll 1
    for (int c0 = 0; c0 < PAD; c0 += PER) {
        alignas(16) T v[PER];
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const int ch = c0 + j;
            float f = 0.0f;
            if (ch < IN_PLANES)
                f = IN_PLANES == 19 ? plane19(r, ch, s, hm)
                                    : plane112(reinterpret_cast<const PosH8 *>(r), ch, s, hm);
            v[j] = to_act<T>(f);
        }
        *reinterpret_cast<uint4 *>(out + c0) = *reinterpret_cast<const uint4 *>(v);
    }
}

}  // namespace

int launch_encode(const void *positions, size_t stride, int batch, int in_planes, int in_pad,
                  bool bf16, void *planes, uint32_t *status, cudaStream_t s) {
    if (batch == 0) return AZ_OK;
    const long long threads = (long long)batch * 64;
    const int block = 256;
    const unsigned grid = (unsigned)((threads + block - 1) / block);
    const unsigned char *p = static_cast<const unsigned char *>(positions);
    if (in_planes == 19 && in_pad == 32) {
        if (bf16) encode_planes_kernel<__nv_bfloat16, 19, 32><<<grid, block, 0, s>>>(p, stride, batch, (__nv_bfloat16 *)planes, status);
        else encode_planes_kernel<float, 19, 32><<<grid, block, 0, s>>>(p, stride, batch, (float *)planes, status);
    } else if (in_planes == 112 && in_pad == 128) {
        if (bf16) encode_planes_kernel<__nv_bfloat16, 112, 128><<<grid, block, 0, s>>>(p, stride, batch, (__nv_bfloat16 *)planes, status);
        else encode_planes_kernel<float, 112, 128><<<grid, block, 0, s>>>(p, stride, batch, (float *)planes, status);
    } else {
        return AZ_ERR_BAD_ARCH;
    }
    AZ_LAUNCH_CHECK();
    return AZ_OK;
}

}  // namespace az
