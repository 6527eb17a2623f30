// The paper's own inference network (Sec. 3.2, 4.3, App. D.1) on top of the tensor-core tower:
// loading (blob -> packed tiles), and the finishing kernel that turns the tower's outputs into the
// policy over the 1,880 actions and the win/draw/loss value.
//
// What runs where.  az_encode52's kernel writes the 52 planes (bf16, 64 channels per square); the
// tower kernel's paper-network instantiation runs the input convolution, the scaled post-activation
// blocks (activations capped at six, pooled context in blocks 1, 3, 5, ...) and, as its fused head
// layer, the query and key maps of every square.  The token projection has no activation, so query,
// key and promotion-offset maps are linear in the backbone's features and are composed with it at
// load (W_q' = W_q W_t / sqrt(K), b_q' = (W_q b_t + b_q) / sqrt(K), and likewise for keys and
// offsets, without the 1/sqrt(K)).  The finishing kernel, one CTA per position, computes
//   - the value head: 2-channel 1x1 convolution + folded normalisation + ReLU, 48 hidden units with
//     ReLU, three logits, softmax (fp32 ALU: 22 k multiply-adds per position);
//   - the logits of the LEGAL actions only, q_origin . k_destination (+ the promotion piece's offset,
//     a 128-long dot product with the origin square's features), and the softmax over them; illegal
//     actions get exactly zero.
// Shares nothing with oracle/.
#include "common.cuh"
#include "ptx.cuh"

#include <cmath>
#include <cstring>
#include <new>
#include <vector>

namespace az {
namespace {

constexpr int kPlanes52 = 52, kActions = 1880, kKey = 128, kVC = 2, kVH = 48;

// offsets (in floats) into Net::pnet_small for a backbone of C channels
struct Small {
    int o_w, o_b, v_cw, v_cs, v_cb, v_w1, v_b1, v_w2, v_b2, total;
    __host__ __device__ explicit Small(int C) {
        o_w = 0;                        // [4][C]
        o_b = o_w + 4 * C;              // [4]
        v_cw = o_b + 4;                 // [2][C]
        v_cs = v_cw + kVC * C;          // [2]
        v_cb = v_cs + kVC;              // [2]
        v_w1 = v_cb + kVC;              // [128][48] (input-major)
        v_b1 = v_w1 + kVH * kVC * 64;   // [48]
        v_w2 = v_b1 + kVH;              // [3][48]
        v_b2 = v_w2 + 3 * kVH;          // [3]
        total = v_b2 + 3;
    }
};

// (Both operands of these two products come from the tower kernel, which may still be running when this kernel starts
// (programmatic dependent launch).  They are read through the read-only path, whose hit rate these products need (a
// row is read once per legal move), but such loads the compiler may move ahead of the dependency wait: the kernel
// therefore takes their base pointers through an opaque assembly statement placed AFTER the wait.)
__device__ __forceinline__ float dot128_f32(const float *a, const float *b) {
    const float4 *pa = reinterpret_cast<const float4 *>(a), *pb = reinterpret_cast<const float4 *>(b);
    float acc = 0.0f;
#pragma unroll 8
    for (int i = 0; i < 32; ++i) {
        const float4 x = __ldg(pa + i), y = __ldg(pb + i);
        acc = fmaf(x.x, y.x, acc); acc = fmaf(x.y, y.y, acc);
        acc = fmaf(x.z, y.z, acc); acc = fmaf(x.w, y.w, acc);
    }
    return acc;
}
// fp32 weights . bf16 features, n a multiple of 8
__device__ __forceinline__ float dot_f32_bf16(const float *w, const __nv_bfloat16 *h, int n) {
    const uint4 *ph = reinterpret_cast<const uint4 *>(h);
    float acc = 0.0f;
#pragma unroll 4
    for (int i = 0; i < n / 8; ++i) {
        const uint4 y = __ldg(ph + i);
        const uint32_t ys[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 fy = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&ys[j]));
            acc = fmaf(w[i * 8 + 2 * j], fy.x, acc);
            acc = fmaf(w[i * 8 + 2 * j + 1], fy.y, acc);
        }
    }
    return acc;
}

constexpr int kFinishThreads = 128;

__device__ __forceinline__ float block_reduce(float v, bool is_max, float *scratch) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float t = __shfl_xor_sync(0xffffffffu, v, o);
        v = is_max ? fmaxf(v, t) : v + t;
    }
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = scratch[0];
#pragma unroll
    for (int w = 1; w < kFinishThreads / 32; ++w) r = is_max ? fmaxf(r, scratch[w]) : r + scratch[w];
    return r;
}

// One CTA per position.  The legal actions are first listed (ascending action index, which is also
// the order of the legal-moves-only output), then each gets a thread for its 128-long dot product.
__global__ void __launch_bounds__(kFinishThreads)
pnet_finish_kernel(const __nv_bfloat16 *__restrict__ h, const float *__restrict__ qk,
                   const uint64_t *__restrict__ masks, const float *__restrict__ small,
                   const uchar4 *__restrict__ actions, int batch, int C, float *__restrict__ policy,
                   float *__restrict__ legal, int *__restrict__ counts,
                   float *__restrict__ value, uint32_t *__restrict__ status) {
    const int pos = blockIdx.x, tid = threadIdx.x;
    const Small S(C);
    __shared__ float v_s[kVC * 64], hid_s[kVH], red[kFinishThreads / 32], lg_s[AZ_MAX_LEGAL];
    __shared__ unsigned short list_s[AZ_MAX_LEGAL];
    __shared__ int first_s[31];
    // ---- the legal actions, from the mask alone (before the tower's results are needed)
    const uint64_t *row = masks + (size_t)pos * 30;
    if (tid < 30) first_s[tid + 1] = __popcll(row[tid]);
    __syncthreads();
    if (tid == 0) {
        first_s[0] = 0;
        for (int w = 1; w <= 30; ++w) first_s[w] += first_s[w - 1];
    }
    __syncthreads();
    const int n_legal = min(first_s[30], AZ_MAX_LEGAL);
    if (tid < 30) {
        uint64_t bits = row[tid];
        int at = first_s[tid];
        while (bits && at < AZ_MAX_LEGAL) {
            list_s[at++] = (unsigned short)(tid * 64 + __ffsll((long long)bits) - 1);
            bits &= bits - 1;
        }
    }
    ptx::grid_dependency_wait();                     // from here on the tower's outputs are read
    const __nv_bfloat16 *hp = h + (size_t)pos * 64 * C;
    const float *qkp = qk + (size_t)pos * 64 * 256;
    asm volatile("" : "+l"(hp), "+l"(qkp) : : "memory");   // no load through these pointers can be scheduled above the wait

    // ---- value head
    {
        const int c = tid >> 6, sq = tid & 63;
        const float d = dot_f32_bf16(small + S.v_cw + c * C, hp + sq * C, C);
        v_s[c * 64 + sq] = fmaxf(fmaf(small[S.v_cs + c], d, small[S.v_cb + c]), 0.0f);
    }
    __syncthreads();
    if (tid < kVH) {
        const float *w = small + S.v_w1 + tid;       // stored [input][hidden unit]: neighbouring threads, neighbouring words
        float acc0 = small[S.v_b1 + tid], acc1 = 0.0f;
#pragma unroll 16
        for (int i = 0; i < kVC * 64; i += 2) {
            acc0 = fmaf(__ldg(w + i * kVH), v_s[i], acc0);
            acc1 = fmaf(__ldg(w + (i + 1) * kVH), v_s[i + 1], acc1);
        }
        hid_s[tid] = fmaxf(acc0 + acc1, 0.0f);
    }
    // ---- policy: one thread per legal action
    float mx = -INFINITY;
    for (int t = tid; t < n_legal; t += kFinishThreads) {
        const uchar4 a = actions[list_s[t]];                                   // origin, destination, piece + 1
        float s = dot128_f32(qkp + a.x * 256, qkp + a.y * 256 + 128);
        if (a.z) s += dot_f32_bf16(small + S.o_w + (a.z - 1) * C, hp + a.x * C, C) + small[S.o_b + a.z - 1];
        lg_s[t] = s;
        mx = fmaxf(mx, s);
    }
    mx = block_reduce(mx, true, red);                                      // (its barriers also publish hid_s and lg_s)
    if (tid == 0) {
        float z[3], m = -INFINITY, sum = 0.0f;
#pragma unroll
        for (int c = 0; c < 3; ++c) {
            float acc = small[S.v_b2 + c];
            for (int j = 0; j < kVH; ++j) acc = fmaf(small[S.v_w2 + c * kVH + j], hid_s[j], acc);
            z[c] = acc;
            m = fmaxf(m, acc);
        }
#pragma unroll
        for (int c = 0; c < 3; ++c) { z[c] = __expf(z[c] - m); sum += z[c]; }
#pragma unroll
        for (int c = 0; c < 3; ++c) value[(size_t)pos * 3 + c] = z[c] / sum;
    }
    float sum = 0.0f;
    for (int t = tid; t < n_legal; t += kFinishThreads) {
        const float e = __expf(lg_s[t] - mx);
        lg_s[t] = e;
        sum += e;
    }
    sum = block_reduce(sum, false, red);
    if (n_legal == 0) {                                                    // no legal action: an all-zero row and a status bit
        if (tid == 0) atomicOr(status, kStatusEmptyMask);
        sum = 1.0f;
    }
    const float inv = 1.0f / sum;
    if (policy != nullptr) {
        float *out = policy + (size_t)pos * kActions;
        for (int i = tid; i < kActions / 4; i += kFinishThreads) reinterpret_cast<float4 *>(out)[i] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        __syncthreads();
        for (int t = tid; t < n_legal; t += kFinishThreads) out[list_s[t]] = lg_s[t] * inv;
    } else {
        for (int t = tid; t < n_legal; t += kFinishThreads) legal[(size_t)pos * AZ_MAX_LEGAL + t] = lg_s[t] * inv;
        if (tid == 0) counts[pos] = n_legal;
    }
}

struct PBlob {
    int L, C;
    const float *in_w, *in_s, *in_b;
    std::vector<const float *> w1, s1, b1, gw, w2, s2, b2;
    const float *t_w, *t_b, *q_w, *q_b, *k_w, *k_b, *o_w, *o_b;
    const float *v_cw, *v_cs, *v_cb, *v_w1, *v_b1, *v_w2, *v_b2;
};

int parse_pnet(const az_arch &a, const unsigned char *blob, size_t nbytes, PBlob &v) {
    if (nbytes < 64 || memcmp(blob, "AZPNET1", 8) != 0) return AZ_ERR_BAD_WEIGHTS;
    uint32_t h[7];
    memcpy(h, blob + 8, sizeof h);
    if (h[0] != 1 || h[1] != a.blocks || h[2] != a.channels || h[3] != (uint32_t)kKey || h[4] != (uint32_t)kVC ||
        h[5] != (uint32_t)kVH)
        return AZ_ERR_BAD_WEIGHTS;
    const size_t C = a.channels, L = a.blocks, P = C / 4, R = C - P;
    size_t need = C * kPlanes52 * 9 + 2 * C;
    for (size_t b = 0; b < L; ++b) need += C * C * 9 + 2 * C + ((b & 1) ? R * 2 * P + C * R * 9 : C * C * 9) + 2 * C;
    need += (size_t)kKey * C + kKey + 2 * ((size_t)kKey * kKey + kKey) + 4 * kKey + 4;
    need += (size_t)kVC * C + 2 * kVC + (size_t)kVH * kVC * 64 + kVH + 3 * kVH + 3;
    if (nbytes != 64 + 4 * need) return AZ_ERR_BAD_WEIGHTS;
    const float *p = reinterpret_cast<const float *>(blob + 64);
    for (size_t i = 0; i < need; ++i)
        if (!std::isfinite(p[i])) return AZ_ERR_BAD_WEIGHTS;
    auto take = [&p](size_t n) { const float *q = p; p += n; return q; };
    v.L = (int)L; v.C = (int)C;
    v.in_w = take(C * kPlanes52 * 9); v.in_s = take(C); v.in_b = take(C);
    for (size_t b = 0; b < L; ++b) {
        v.w1.push_back(take(C * C * 9)); v.s1.push_back(take(C)); v.b1.push_back(take(C));
        v.gw.push_back((b & 1) ? take(R * 2 * P) : nullptr);
        v.w2.push_back(take(C * ((b & 1) ? R : C) * 9)); v.s2.push_back(take(C)); v.b2.push_back(take(C));
    }
    v.t_w = take((size_t)kKey * C); v.t_b = take(kKey);
    v.q_w = take((size_t)kKey * kKey); v.q_b = take(kKey);
    v.k_w = take((size_t)kKey * kKey); v.k_b = take(kKey);
    v.o_w = take(4 * kKey); v.o_b = take(4);
    v.v_cw = take((size_t)kVC * C); v.v_cs = take(kVC); v.v_cb = take(kVC);
    v.v_w1 = take((size_t)kVH * kVC * 64); v.v_b1 = take(kVH);
    v.v_w2 = take(3 * kVH); v.v_b2 = take(3);
    return AZ_OK;
}

// out[rows][C] = m[rows][K] * t_w[K][C] * f,  out_b[rows] = (m * t_b + b) * f   (double accumulation)
void compose(const float *m, const float *b, int rows, const float *t_w, const float *t_b, int C, double f,
             std::vector<float> &out, std::vector<float> &out_b) {
    out.assign((size_t)rows * C, 0.0f);
    out_b.assign(rows, 0.0f);
    for (int r = 0; r < rows; ++r) {
        for (int c = 0; c < C; ++c) {
            double acc = 0.0;
            for (int k = 0; k < kKey; ++k) acc += (double)m[(size_t)r * kKey + k] * (double)t_w[(size_t)k * C + c];
            out[(size_t)r * C + c] = (float)(acc * f);
        }
        double acc = b[r];
        for (int k = 0; k < kKey; ++k) acc += (double)m[(size_t)r * kKey + k] * (double)t_b[k];
        out_b[r] = (float)(acc * f);
    }
}

// fp32 master copy of the tower for the int8 form (quantised once the calibration ranges are known)
struct PnetMaster {
    std::vector<std::vector<float>> w, scale, bias;   // per convolution layer
    std::vector<int> cin;                             // input channels of each layer
    std::vector<std::vector<float>> gw;               // per pooled block: [3C/4][C/2]
};

}  // namespace

void free_pnet_master(void *master) { delete static_cast<PnetMaster *>(master); }

// int8 form of the paper's tower (Sec. 4.3.6: the trunk's convolutions in INT8, the pooled context and
// the heads in floating point).  As in the plain int8 tower: layer l >= 1 reads unsigned 8-bit
// activations with a per-input-channel scale sa (calibration maximum / 255, folded into the weight
// rows) and signed 8-bit weights with a per-output-channel scale ws (max / 127).  Per layer four
// constant vectors: os * qs, bias * qs, hs / qs, 6 * qs, where os = ws (1 for the input layer), qs =
// 1 / sa of the next layer for the channels that are handed on and 1 for the pooled ones (so that
// their values stay in real units), hs = 1 / ws of the next second convolution on the residual
// stream.  The context map's rows are multiplied by the same qs, since the context is added to
// values that are already in those units.
int quantise_pnet(Net &n, const float *absmax, std::vector<float> *lconst_out, std::vector<int> *next_cin_out) {
    const PnetMaster *m = static_cast<const PnetMaster *>(n.pnet_master);
    if (!m) return AZ_ERR_UNSUPPORTED;
    const int C = (int)n.arch.channels, L = n.n_conv, P = C / 4, R = C - P;
    const float kTiny = 1e-30f;
    const size_t kStage = (size_t)9 * C * 32;         // bytes of one weight stage: 9 taps x C outputs x 32 bytes of K
    std::vector<float> sa((size_t)L * C, 1.0f), ws((size_t)L * C, 1.0f);
    for (int l = 1; l < L; ++l)
        for (int c = 0; c < m->cin[l]; ++c) sa[(size_t)l * C + c] = fmaxf(absmax[(size_t)(l - 1) * C + c], kTiny) / 255.0f;
    size_t bytes = (size_t)(n.in_pad / 16) * kStage;
    for (int l = 1; l < L; ++l) bytes += (size_t)((m->cin[l] + 31) / 32) * kStage;
    std::vector<unsigned char> packed(bytes, 0);
    // input layer: bf16 tiles as in the bf16 tower
    {
        const float *w0 = m->w[0].data(), *s0 = m->scale[0].data();
        const int cin0 = m->cin[0], pad0 = n.in_pad;
        tc_pack_layers(&w0, &s0, &cin0, &pad0, C, 1, reinterpret_cast<__nv_bfloat16 *>(packed.data()));
    }
    unsigned char *dst = packed.data() + (size_t)(n.in_pad / 16) * kStage;
    for (int l = 1; l < L; ++l) {
        const int cin = m->cin[l];
        std::vector<float> wf((size_t)C * cin * 9);
        for (int co = 0; co < C; ++co) {
            float mx = 0.0f;
            for (int ci = 0; ci < cin; ++ci)
                for (int tap = 0; tap < 9; ++tap) {
                    const float v = m->scale[l][co] * m->w[l][((size_t)co * cin + ci) * 9 + tap] * sa[(size_t)l * C + ci];
                    wf[((size_t)co * cin + ci) * 9 + tap] = v;
                    mx = fmaxf(mx, fabsf(v));
                }
            ws[(size_t)l * C + co] = fmaxf(mx, kTiny) / 127.0f;
        }
        for (int kc = 0; kc < (cin + 31) / 32; ++kc)
            for (int tap = 0; tap < 9; ++tap)
                for (int k16 = 0; k16 < 2; ++k16)
                    for (int ng = 0; ng < C / 8; ++ng)
                        for (int r = 0; r < 8; ++r)
                            for (int e = 0; e < 16; ++e) {
                                const int co = ng * 8 + r, ci = kc * 32 + k16 * 16 + e;
                                float q = 0.0f;
                                if (ci < cin) q = fminf(fmaxf(nearbyintf(wf[((size_t)co * cin + ci) * 9 + tap] / ws[(size_t)l * C + co]), -127.0f), 127.0f);
                                *dst++ = (unsigned char)(signed char)q;
                            }
    }
    std::vector<float> lconst((size_t)L * 4 * C), gwt;
    for (int l = 0; l < L; ++l) {
        float *lc = lconst.data() + (size_t)l * 4 * C;
        const int next_cin = l + 1 < L ? m->cin[l + 1] : 0;       // channels of this layer's output that are handed on as 8-bit
        for (int c = 0; c < C; ++c) {
            const float qs = c < next_cin ? 1.0f / sa[(size_t)(l + 1) * C + c] : 1.0f;
            const float hs = ((l & 1) == 0 && l + 2 < L) ? 1.0f / ws[(size_t)(l + 2) * C + c] : 1.0f;
            lc[c] = (l == 0 ? 1.0f : ws[(size_t)l * C + c]) * qs;
            lc[C + c] = m->bias[l][c] * qs;
            lc[2 * C + c] = hs / qs;
            lc[3 * C + c] = 6.0f * qs;
        }
        if ((l & 3) == 3) {                                          // first convolution of a pooled block: its context map
            const std::vector<float> &g = m->gw[(l - 3) / 4];
            for (int j = 0; j < 2 * P; ++j)
                for (int r = 0; r < R; ++r) gwt.push_back(g[(size_t)r * 2 * P + j] / sa[(size_t)(l + 1) * C + r]);
        }
    }
    if (gwt.empty()) gwt.push_back(0.0f);
    if (!n.tc8_weights) AZ_CUDA(cudaMalloc(&n.tc8_weights, bytes));
    if (!n.tc8_lconst) AZ_CUDA(cudaMalloc((void **)&n.tc8_lconst, lconst.size() * sizeof(float)));
    AZ_CUDA(cudaMemcpy(n.tc8_weights, packed.data(), bytes, cudaMemcpyHostToDevice));
    AZ_CUDA(cudaMemcpy(n.tc8_lconst, lconst.data(), lconst.size() * sizeof(float), cudaMemcpyHostToDevice));
    // the scaled context maps replace the plain ones (the calibration pass, which needed those, is over)
    AZ_CUDA(cudaMemcpy(n.pnet_gw, gwt.data(), gwt.size() * sizeof(float), cudaMemcpyHostToDevice));
    n.fp8_ready = true;
    if (next_cin_out) {
        next_cin_out->assign(L, 0);
        for (int l = 0; l + 1 < L; ++l) (*next_cin_out)[l] = m->cin[l + 1];
    }
    if (lconst_out) *lconst_out = std::move(lconst);
    return AZ_OK;
}

// Builds the device side of a paper-network az_net: 128 or 160 channels, bf16 (the caller refuses
// other sizes).
int build_pnet(Net &n, const unsigned char *blob, size_t nbytes) {
    const az_arch &a = n.arch;
    PBlob v;
    int rc = parse_pnet(a, blob, nbytes, v);
    if (rc != AZ_OK) return rc;
    const int C = v.C, L = v.L, P = C / 4, R = C - P;
    n.bf16 = true;
    n.pnet = true;
    n.int8 = a.precision == AZ_PREC_INT8;
    n.fp8 = n.int8;                                      // the 8-bit tower; usable after az_calibrate
    n.in_pad = 64;
    n.n_conv = 1 + 2 * L;
    // tower tiles
    std::vector<const float *> w, s;
    std::vector<int> cin, cin_pad;
    std::vector<float> bias((size_t)n.n_conv * C);
    w.push_back(v.in_w); s.push_back(v.in_s); cin.push_back(kPlanes52); cin_pad.push_back(64);
    memcpy(&bias[0], v.in_b, sizeof(float) * C);
    for (int b = 0; b < L; ++b) {
        w.push_back(v.w1[b]); s.push_back(v.s1[b]); cin.push_back(C); cin_pad.push_back(C);
        memcpy(&bias[(size_t)(1 + 2 * b) * C], v.b1[b], sizeof(float) * C);
        w.push_back(v.w2[b]); s.push_back(v.s2[b]); cin.push_back((b & 1) ? R : C); cin_pad.push_back((b & 1) ? ((R + 15) & ~15) : C);
        memcpy(&bias[(size_t)(2 + 2 * b) * C], v.b2[b], sizeof(float) * C);
    }
    if (n.int8) {
        PnetMaster *m = new (std::nothrow) PnetMaster();
        if (!m) return AZ_ERR_BAD_ARG;
        n.pnet_master = m;
        for (int l = 0; l < n.n_conv; ++l) {
            m->w.emplace_back(w[l], w[l] + (size_t)C * cin[l] * 9);
            m->scale.emplace_back(s[l], s[l] + C);
            m->bias.emplace_back(&bias[(size_t)l * C], &bias[(size_t)l * C] + C);
            m->cin.push_back(cin[l]);
        }
        for (int b = 1; b < L; b += 2) m->gw.emplace_back(v.gw[b], v.gw[b] + (size_t)R * 2 * P);
    }
    const size_t bytes = tc_packed_layers_bytes(cin_pad.data(), C, n.n_conv);
    std::vector<__nv_bfloat16> packed(bytes / sizeof(__nv_bfloat16));
    tc_pack_layers(w.data(), s.data(), cin.data(), cin_pad.data(), C, n.n_conv, packed.data());
    AZ_CUDA(cudaMalloc(&n.tc_weights, bytes));
    AZ_CUDA(cudaMemcpy(n.tc_weights, packed.data(), bytes, cudaMemcpyHostToDevice));
    AZ_CUDA(cudaMalloc((void **)&n.tc_bias, bias.size() * sizeof(float)));
    AZ_CUDA(cudaMemcpy(n.tc_bias, bias.data(), bias.size() * sizeof(float), cudaMemcpyHostToDevice));
    // pooled-context maps of blocks 1, 3, 5, ...
    {
        std::vector<float> gw;
        for (int b = 1; b < L; b += 2)                       // stored transposed: [entry of the pooled vector][output]
            for (int j = 0; j < 2 * P; ++j)
                for (int r = 0; r < R; ++r) gw.push_back(v.gw[b][(size_t)r * 2 * P + j]);
        if (gw.empty()) gw.push_back(0.0f);
        AZ_CUDA(cudaMalloc((void **)&n.pnet_gw, gw.size() * sizeof(float)));
        AZ_CUDA(cudaMemcpy(n.pnet_gw, gw.data(), gw.size() * sizeof(float), cudaMemcpyHostToDevice));
    }
    // head layer: queries and keys composed with the token projection, 1/sqrt(K) folded into the queries
    std::vector<float> wq, bq, wk, bk, wo, bo;
    compose(v.q_w, v.q_b, kKey, v.t_w, v.t_b, C, 1.0 / std::sqrt((double)kKey), wq, bq);
    compose(v.k_w, v.k_b, kKey, v.t_w, v.t_b, C, 1.0, wk, bk);
    compose(v.o_w, v.o_b, 4, v.t_w, v.t_b, C, 1.0, wo, bo);
    n.tc_head_n = 256;
    std::vector<__nv_bfloat16> hw((size_t)256 * C);
    tc_pack_qk(wq.data(), wk.data(), C, hw.data());
    AZ_CUDA(cudaMalloc(&n.tc_head_w, hw.size() * sizeof(__nv_bfloat16)));
    AZ_CUDA(cudaMemcpy(n.tc_head_w, hw.data(), hw.size() * sizeof(__nv_bfloat16), cudaMemcpyHostToDevice));
    std::vector<float> hb(256);
    for (int i = 0; i < 128; ++i) { hb[i] = bq[i]; hb[128 + i] = bk[i]; }
    AZ_CUDA(cudaMalloc((void **)&n.tc_head_bias, hb.size() * sizeof(float)));
    AZ_CUDA(cudaMemcpy(n.tc_head_bias, hb.data(), hb.size() * sizeof(float), cudaMemcpyHostToDevice));
    // the finishing kernel's parameters
    const Small S(C);
    std::vector<float> small(S.total);
    memcpy(&small[S.o_w], wo.data(), sizeof(float) * 4 * C);
    memcpy(&small[S.o_b], bo.data(), sizeof(float) * 4);
    memcpy(&small[S.v_cw], v.v_cw, sizeof(float) * kVC * C);
    memcpy(&small[S.v_cs], v.v_cs, sizeof(float) * kVC);
    memcpy(&small[S.v_cb], v.v_cb, sizeof(float) * kVC);
    for (int j = 0; j < kVH; ++j)                        // stored [input][hidden unit]
        for (int i = 0; i < kVC * 64; ++i) small[S.v_w1 + (size_t)i * kVH + j] = v.v_w1[(size_t)j * kVC * 64 + i];
    memcpy(&small[S.v_b1], v.v_b1, sizeof(float) * kVH);
    memcpy(&small[S.v_w2], v.v_w2, sizeof(float) * 3 * kVH);
    memcpy(&small[S.v_b2], v.v_b2, sizeof(float) * 3);
    AZ_CUDA(cudaMalloc((void **)&n.pnet_small, small.size() * sizeof(float)));
    AZ_CUDA(cudaMemcpy(n.pnet_small, small.data(), small.size() * sizeof(float), cudaMemcpyHostToDevice));
    // the action list (Sec. 3.2, App. D.1), generated: 1,792 origin-destination pairs a queen ray or a knight
    // jump apart, origins then destinations ascending; then, for origins on the seventh rank ascending and the
    // destinations origin+7, +8, +9 that stay on the board, the pieces queen, rook, bishop, knight
    {
        std::vector<unsigned char> act((size_t)kActions * 4, 0);
        int next = 0;
        for (int from = 0; from < 64; ++from)
            for (int to = 0; to < 64; ++to) {
                const int df = abs((to & 7) - (from & 7)), dr = abs((to >> 3) - (from >> 3));
                if (from == to) continue;
                if (df == 0 || dr == 0 || df == dr || df * dr == 2) {
                    act[4 * next] = (unsigned char)from; act[4 * next + 1] = (unsigned char)to; ++next;
                }
            }
        for (int from = 48; from < 56; ++from)
            for (int to = from + 7; to <= from + 9; ++to) {
                if (to > 63 || abs((to & 7) - (from & 7)) > 1) continue;
                for (int piece = 0; piece < 4; ++piece) {
                    act[4 * next] = (unsigned char)from; act[4 * next + 1] = (unsigned char)to;
                    act[4 * next + 2] = (unsigned char)(piece + 1); ++next;
                }
            }
        if (next != kActions) return AZ_ERR_BAD_ARCH;
        AZ_CUDA(cudaMalloc((void **)&n.pnet_actions, act.size()));
        AZ_CUDA(cudaMemcpy(n.pnet_actions, act.data(), act.size(), cudaMemcpyHostToDevice));
    }
    // workspace: planes, tower output, queries and keys, status
    const size_t B = a.max_batch;
    AZ_CUDA(cudaMalloc(&n.planes, B * 64 * 64 * sizeof(__nv_bfloat16)));
    AZ_CUDA(cudaMalloc(&n.act[0], B * 64 * C * sizeof(__nv_bfloat16)));
    AZ_CUDA(cudaMalloc(&n.pnet_qk, B * 64 * 256 * sizeof(float)));
    AZ_CUDA(cudaMalloc((void **)&n.status_dev, sizeof(uint32_t)));
    AZ_CUDA(cudaMemset(n.status_dev, 0, sizeof(uint32_t)));
    n.tc_ready = true;
    return AZ_OK;
}

int launch_pnet_finish(const Net &n, const uint64_t *masks, int batch, float *policy, float *legal, int *counts,
                       float *value, cudaStream_t s) {
    if (batch == 0) return AZ_OK;
    // A dependent launch: its CTAs become resident while the tower's last round still runs and start the moment the
    // tower has finished.  One stream alone would do 2 % better with an ordinary launch at batch 1024 (started early,
    // the many small CTAs pile onto the SMs that the last round leaves idle first), but with two batches in flight on
    // two streams an ordinary launch queues behind the OTHER batch's tower kernel, which takes the SMs as they become
    // free and holds them for its whole run: 8 to 18 % less end-to-end throughput, measured.
    AZ_CUDA(launch_dependent(pnet_finish_kernel, dim3((unsigned)batch), dim3(kFinishThreads), 0, s,
                             static_cast<const __nv_bfloat16 *>(n.act[0]), static_cast<const float *>(n.pnet_qk), masks,
                             static_cast<const float *>(n.pnet_small), reinterpret_cast<const uchar4 *>(n.pnet_actions), batch,
                             (int)n.arch.channels, policy, legal, counts, value, n.status_dev));
    return AZ_OK;
}

}  // namespace az
