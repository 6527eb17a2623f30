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
#include "planes.cuh"

namespace az {
namespace {

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
    float v[64];
    planes52_square(r, c, v);

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
