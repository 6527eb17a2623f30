// The C ABI of az_eval: argument checks, weight-blob parsing and repacking, workspace ownership,
// and the sequence of kernel launches that makes up one evaluation.
#include "common.cuh"

#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <utility>
#include <vector>

namespace az {

static thread_local std::string g_cuda_error;

void set_cuda_error(cudaError_t e, const char *what) {
    g_cuda_error = std::string(what) + ": " + cudaGetErrorString(e);
}

namespace {

constexpr size_t kHeaderBytes = 64;

struct BlobView {                       // float32 tensors of the blob, in file order
    const float *in_w, *in_s, *in_b;
    std::vector<const float *> w1, s1, b1, w2, s2, b2;
    const float *p_w, *p_s, *p_b, *p_fw, *p_fb;
    const float *v_cw, *v_cs, *v_cb, *v_w1, *v_b1, *v_w2, *v_b2;
};

struct HostMaster {                     // fp32 tower parameters of an FP8 net, kept until az_calibrate has quantised them
    std::vector<std::vector<float>> w, scale, bias;
};

bool arch_ok(const az_arch &a) {
    if (a.abi_version != AZ_ABI_VERSION) return false;
    if (a.in_planes != 19 && a.in_planes != 112 && a.in_planes != 52) return false;
    if (a.blocks > 64 || a.channels < 8 || a.channels > 512 || a.channels % 8) return false;
    if (a.policy_head > 2 || a.value_head > 1 || a.precision > AZ_PREC_FP8_E4M3_X2A) return false;
    // the paper's own network: 52 planes go with the 1,880-action head and the win/draw/loss value, and only with them
    if ((a.in_planes == 52) != (a.policy_head == AZ_POLICY_FROMTO1880)) return false;
    if (a.in_planes == 52 && a.value_head != AZ_VALUE_WDL) return false;
    if (a.max_batch == 0 || a.max_batch > (1u << 20)) return false;
    return true;
}

int parse_blob(const az_arch &a, const unsigned char *blob, size_t nbytes, BlobView &v) {
    if (nbytes < kHeaderBytes || memcmp(blob, "AZNETv1", 8) != 0) return AZ_ERR_BAD_WEIGHTS;
    uint32_t h[7];
    memcpy(h, blob + 8, sizeof h);
    if (h[0] != 1 || h[1] != a.in_planes || h[2] != a.blocks || h[3] != a.channels ||
        h[4] != a.policy_head || h[5] != a.value_head)
        return AZ_ERR_BAD_WEIGHTS;
    const size_t C = a.channels, P = a.in_planes, L = a.blocks;
    const size_t V = a.value_head == AZ_VALUE_WDL ? 3 : 1;
    size_t need = C * P * 9 + 2 * C + L * (2 * C * C * 9 + 4 * C);
    need += a.policy_head == AZ_POLICY_PLANES73 ? (size_t)kPlanes73 * C + kPlanes73
                                                : (size_t)kHeadChannels * C + 2 * kHeadChannels +
                                                      (size_t)kFlatMoves * kHeadChannels * 64 + kFlatMoves;
    need += (size_t)kHeadChannels * C + 2 * kHeadChannels + (size_t)kValueHidden * kHeadChannels * 64 +
            kValueHidden + V * kValueHidden + V;
    if (nbytes != kHeaderBytes + 4 * need) return AZ_ERR_BAD_WEIGHTS;
    const float *p = reinterpret_cast<const float *>(blob + kHeaderBytes);
    for (size_t i = 0; i < need; ++i)
        if (!std::isfinite(p[i])) return AZ_ERR_BAD_WEIGHTS;
    auto take = [&p](size_t n) { const float *q = p; p += n; return q; };
    v.in_w = take(C * P * 9); v.in_s = take(C); v.in_b = take(C);
    for (size_t b = 0; b < L; ++b) {
        v.w1.push_back(take(C * C * 9)); v.s1.push_back(take(C)); v.b1.push_back(take(C));
        v.w2.push_back(take(C * C * 9)); v.s2.push_back(take(C)); v.b2.push_back(take(C));
    }
    v.p_s = v.p_fw = v.p_fb = nullptr;
    if (a.policy_head == AZ_POLICY_PLANES73) { v.p_w = take((size_t)kPlanes73 * C); v.p_b = take(kPlanes73); }
    else {
        v.p_w = take((size_t)kHeadChannels * C); v.p_s = take(kHeadChannels); v.p_b = take(kHeadChannels);
        v.p_fw = take((size_t)kFlatMoves * kHeadChannels * 64); v.p_fb = take(kFlatMoves);
    }
    v.v_cw = take((size_t)kHeadChannels * C); v.v_cs = take(kHeadChannels); v.v_cb = take(kHeadChannels);
    v.v_w1 = take((size_t)kValueHidden * kHeadChannels * 64); v.v_b1 = take(kValueHidden);
    v.v_w2 = take(V * kValueHidden); v.v_b2 = take(V);
    return AZ_OK;
}

// host float32 -> device buffer of the activation type (float32 or bfloat16, round to nearest even)
int upload_act(const float *src, size_t n, bool bf16, void **dst) {
    if (bf16) {
        std::vector<__nv_bfloat16> tmp(n);
        for (size_t i = 0; i < n; ++i) tmp[i] = __float2bfloat16_rn(src[i]);
        AZ_CUDA(cudaMalloc(dst, n * sizeof(__nv_bfloat16)));
        AZ_CUDA(cudaMemcpy(*dst, tmp.data(), n * sizeof(__nv_bfloat16), cudaMemcpyHostToDevice));
    } else {
        AZ_CUDA(cudaMalloc(dst, n * sizeof(float)));
        AZ_CUDA(cudaMemcpy(*dst, src, n * sizeof(float), cudaMemcpyHostToDevice));
    }
    return AZ_OK;
}
int upload_f32(const float *src, size_t n, float **dst) {
    AZ_CUDA(cudaMalloc((void **)dst, n * sizeof(float)));
    AZ_CUDA(cudaMemcpy(*dst, src, n * sizeof(float), cudaMemcpyHostToDevice));
    return AZ_OK;
}

// [cout][cin][3][3] -> [tap][cin_pad][cout], zero rows for padded input channels
int upload_conv_simt(const float *w, int cin, int cin_pad, int cout, bool bf16, void **dst) {
    std::vector<float> t((size_t)9 * cin_pad * cout, 0.0f);
    for (int co = 0; co < cout; ++co)
        for (int ci = 0; ci < cin; ++ci)
            for (int tap = 0; tap < 9; ++tap)
                t[((size_t)tap * cin_pad + ci) * cout + co] = w[((size_t)co * cin + ci) * 9 + tap];
    return upload_act(t.data(), t.size(), bf16, dst);
}

size_t act_bytes(const Net &n) { return n.bf16 ? 2 : 4; }

int alloc_simt_buffers(Net &n) {
    const size_t bytes = (size_t)n.arch.max_batch * 64 * n.arch.channels * act_bytes(n);
    for (int i = 1; i < 3; ++i)
        if (!n.act[i]) AZ_CUDA(cudaMalloc(&n.act[i], bytes));
    return AZ_OK;
}

int build_net(Net &n, const BlobView &v) {
    const az_arch &a = n.arch;
    const int C = (int)a.channels, L = (int)a.blocks;
    n.bf16 = a.precision != AZ_PREC_FP32;
    n.in_pad = a.in_planes == 19 ? 32 : 128;
    n.n_conv = 1 + 2 * L;
    int rc;

    // tensor-core tower: bf16, 128 channels, 19-plane input
    n.fp8 = a.precision >= AZ_PREC_FP8_E4M3;          // every 8-bit form
    n.int8 = a.precision == AZ_PREC_INT8;
    n.split_a = a.precision == AZ_PREC_FP8_E4M3_X2 || a.precision == AZ_PREC_FP8_E4M3_X2A;
    n.split_w = a.precision == AZ_PREC_FP8_E4M3_X2;
    // tensor-core tower: bf16 with 128 or 256 channels; the FP8 tower exists for 128 channels
    const bool tc_shape = a.precision != AZ_PREC_FP32 && (C == 128 || (C == 256 && !n.fp8));
    if (n.fp8 && !tc_shape) return AZ_ERR_UNSUPPORTED;
    if (tc_shape) {
        std::vector<const float *> w, s, b;
        w.push_back(v.in_w); s.push_back(v.in_s); b.push_back(v.in_b);
        for (int i = 0; i < L; ++i) {
            w.push_back(v.w1[i]); s.push_back(v.s1[i]); b.push_back(v.b1[i]);
            w.push_back(v.w2[i]); s.push_back(v.s2[i]); b.push_back(v.b2[i]);
        }
        const size_t bytes = tc_packed_weight_bytes(n.in_pad, C, n.n_conv);
        std::vector<__nv_bfloat16> packed(bytes / sizeof(__nv_bfloat16));
        // CTA pairs: the bf16 tower of a bf16 network, or the 8-bit tower of an 8-bit one (whose bf16 passes, the
        // calibration's, stay on single CTAs: their weights are packed whole)
        const bool pair_shape = n.want_pair && tc_pair_shape(C, (int)a.precision, false);
        n.tc_pair = pair_shape && a.precision == AZ_PREC_BF16;
        n.tc_pair8 = pair_shape && a.precision != AZ_PREC_BF16;
        const int halves = n.tc_pair ? 2 : 1;
        tc_pack_weights(w.data(), s.data(), (int)a.in_planes, n.in_pad, C, n.n_conv, halves, C == 256 ? 3 : 9, false, packed.data());
        AZ_CUDA(cudaMalloc(&n.tc_weights, bytes));
        AZ_CUDA(cudaMemcpy(n.tc_weights, packed.data(), bytes, cudaMemcpyHostToDevice));
        if (C == 256) {
            // small batches run two CTAs per group, each on half of the output channels: the same tiles, packed per half
            tc_pack_weights(w.data(), s.data(), (int)a.in_planes, n.in_pad, C, n.n_conv, 2, 9, true, packed.data());
            AZ_CUDA(cudaMalloc(&n.tc_weights_split, bytes));
            AZ_CUDA(cudaMemcpy(n.tc_weights_split, packed.data(), bytes, cudaMemcpyHostToDevice));
            tc_pack_weights(w.data(), s.data(), (int)a.in_planes, n.in_pad, C, n.n_conv, 4, 9, true, packed.data());
            AZ_CUDA(cudaMalloc(&n.tc_weights_split4, bytes));
            AZ_CUDA(cudaMemcpy(n.tc_weights_split4, packed.data(), bytes, cudaMemcpyHostToDevice));
        }
        std::vector<float> bias((size_t)n.n_conv * C);
        for (int l = 0; l < n.n_conv; ++l) memcpy(&bias[(size_t)l * C], b[l], sizeof(float) * C);
        if ((rc = upload_f32(bias.data(), bias.size(), &n.tc_bias)) != AZ_OK) return rc;
        if (n.fp8) {
            HostMaster *hm = new (std::nothrow) HostMaster();
            if (!hm) return AZ_ERR_BAD_ARG;
            n.host_master = hm;
            for (int l = 0; l < n.n_conv; ++l) {
                const size_t cin = l == 0 ? a.in_planes : C;
                hm->w.emplace_back(w[l], w[l] + (size_t)C * cin * 9);
                hm->scale.emplace_back(s[l], s[l] + C);
                hm->bias.emplace_back(b[l], b[l] + C);
            }
        }
        // fused head projections and tensor-core fully-connected layers
        const bool flat = a.policy_head == AZ_POLICY_FLAT1858;
        const int n_policy = flat ? kHeadChannels : kPlanes73, n_policy_pad = flat ? kHeadChannels : 80;
        n.tc_head_n = n_policy_pad + kHeadChannels;
        std::vector<__nv_bfloat16> hw(tc_head_weight_bytes(n.tc_head_n, C) / sizeof(__nv_bfloat16));
        const int head_halves = (n.tc_pair || n.tc_pair8) ? 2 : 1;
        tc_pack_head(v.p_w, flat ? v.p_s : nullptr, n_policy, n_policy_pad, v.v_cw, v.v_cs, C, head_halves,
                     tc_head_stage_slices(C, n.tc_head_n), hw.data());
        AZ_CUDA(cudaMalloc(&n.tc_head_w, hw.size() * sizeof(__nv_bfloat16)));
        AZ_CUDA(cudaMemcpy(n.tc_head_w, hw.data(), hw.size() * sizeof(__nv_bfloat16), cudaMemcpyHostToDevice));
        if (C == 256 && head_halves == 2) {
            // the small-batch cluster kernels read the head projections whole, in plain slice order
            tc_pack_head(v.p_w, flat ? v.p_s : nullptr, n_policy, n_policy_pad, v.v_cw, v.v_cs, C, 1, C / 16, hw.data());
            AZ_CUDA(cudaMalloc(&n.tc_head_w_plain, hw.size() * sizeof(__nv_bfloat16)));
            AZ_CUDA(cudaMemcpy(n.tc_head_w_plain, hw.data(), hw.size() * sizeof(__nv_bfloat16), cudaMemcpyHostToDevice));
        }
        std::vector<float> hb(n.tc_head_n, 0.0f);
        for (int i = 0; i < n_policy; ++i) hb[i] = v.p_b[i];
        for (int i = 0; i < kHeadChannels; ++i) hb[n_policy_pad + i] = v.v_cb[i];
        if ((rc = upload_f32(hb.data(), hb.size(), &n.tc_head_bias)) != AZ_OK) return rc;
        {
            std::vector<__nv_bfloat16> fw(fc_tc_weight_bytes(kValueHidden, false) / sizeof(__nv_bfloat16));
            fc_tc_pack_weights(v.v_w1, kValueHidden, false, fw.data());
            AZ_CUDA(cudaMalloc(&n.fc_value_w, fw.size() * sizeof(__nv_bfloat16)));
            AZ_CUDA(cudaMemcpy(n.fc_value_w, fw.data(), fw.size() * sizeof(__nv_bfloat16), cudaMemcpyHostToDevice));
        }
        if (flat) {
            std::vector<__nv_bfloat16> fw(fc_tc_weight_bytes(kFlatMoves, true) / sizeof(__nv_bfloat16));
            fc_tc_pack_weights(v.p_fw, kFlatMoves, true, fw.data());
            AZ_CUDA(cudaMalloc(&n.fc_policy_w, fw.size() * sizeof(__nv_bfloat16)));
            AZ_CUDA(cudaMemcpy(n.fc_policy_w, fw.data(), fw.size() * sizeof(__nv_bfloat16), cudaMemcpyHostToDevice));
        }
        const size_t u_bytes = (size_t)((a.max_batch + 127) / 128) * kHeadChannels * 64 * 128 * sizeof(__nv_bfloat16);
        AZ_CUDA(cudaMalloc(&n.u_value, u_bytes));
        AZ_CUDA(cudaMemset(n.u_value, 0, u_bytes));
        if (flat) { AZ_CUDA(cudaMalloc(&n.u_policy, u_bytes)); AZ_CUDA(cudaMemset(n.u_policy, 0, u_bytes)); }
        n.tc_ready = true;
    } else {
        if ((rc = upload_conv_simt(v.in_w, (int)a.in_planes, n.in_pad, C, n.bf16, &n.conv_w[0])) != AZ_OK) return rc;
        if ((rc = upload_f32(v.in_s, C, &n.conv_scale[0])) != AZ_OK) return rc;
        if ((rc = upload_f32(v.in_b, C, &n.conv_bias[0])) != AZ_OK) return rc;
        for (int i = 0; i < L; ++i) {
            const int l1 = 1 + 2 * i, l2 = 2 + 2 * i;
            if ((rc = upload_conv_simt(v.w1[i], C, C, C, n.bf16, &n.conv_w[l1])) != AZ_OK) return rc;
            if ((rc = upload_f32(v.s1[i], C, &n.conv_scale[l1])) != AZ_OK) return rc;
            if ((rc = upload_f32(v.b1[i], C, &n.conv_bias[l1])) != AZ_OK) return rc;
            if ((rc = upload_conv_simt(v.w2[i], C, C, C, n.bf16, &n.conv_w[l2])) != AZ_OK) return rc;
            if ((rc = upload_f32(v.s2[i], C, &n.conv_scale[l2])) != AZ_OK) return rc;
            if ((rc = upload_f32(v.b2[i], C, &n.conv_bias[l2])) != AZ_OK) return rc;
        }
        if ((rc = alloc_simt_buffers(n)) != AZ_OK) return rc;
        if (tower_f32_shape(a)) {
            std::vector<F32Layer> table(n.n_conv);
            for (int l = 0; l < n.n_conv; ++l)
                table[l] = F32Layer{static_cast<const float *>(n.conv_w[l]), n.conv_scale[l], n.conv_bias[l]};
            AZ_CUDA(cudaMalloc((void **)&n.f32_layers, table.size() * sizeof(F32Layer)));
            AZ_CUDA(cudaMemcpy(n.f32_layers, table.data(), table.size() * sizeof(F32Layer), cudaMemcpyHostToDevice));
        }
    }

    // heads
    const int V = a.value_head == AZ_VALUE_WDL ? 3 : 1;
    const bool simt_heads = !n.tc_ready;      // the tensor-core path carries its own packed head weights
    if (a.policy_head == AZ_POLICY_PLANES73) {
        if (simt_heads && (rc = upload_act(v.p_w, (size_t)kPlanes73 * C, n.bf16, &n.p_w)) != AZ_OK) return rc;
        if ((rc = upload_f32(v.p_b, kPlanes73, &n.p_bias)) != AZ_OK) return rc;
    } else {
        if (simt_heads && (rc = upload_act(v.p_w, (size_t)kHeadChannels * C, n.bf16, &n.p_w)) != AZ_OK) return rc;
        if ((rc = upload_f32(v.p_s, kHeadChannels, &n.p_scale)) != AZ_OK) return rc;
        if ((rc = upload_f32(v.p_b, kHeadChannels, &n.p_bias)) != AZ_OK) return rc;
        if (simt_heads && (rc = upload_act(v.p_fw, (size_t)kFlatMoves * kHeadChannels * 64, n.bf16, &n.p_fw)) != AZ_OK) return rc;
        if ((rc = upload_f32(v.p_fb, kFlatMoves, &n.p_fbias)) != AZ_OK) return rc;
    }
    if (simt_heads && (rc = upload_act(v.v_cw, (size_t)kHeadChannels * C, n.bf16, &n.v_cw)) != AZ_OK) return rc;
    if ((rc = upload_f32(v.v_cs, kHeadChannels, &n.v_cscale)) != AZ_OK) return rc;
    if ((rc = upload_f32(v.v_cb, kHeadChannels, &n.v_cbias)) != AZ_OK) return rc;
    if (simt_heads && (rc = upload_act(v.v_w1, (size_t)kValueHidden * kHeadChannels * 64, n.bf16, &n.v_w1)) != AZ_OK) return rc;
    if ((rc = upload_f32(v.v_b1, kValueHidden, &n.v_b1)) != AZ_OK) return rc;
    if ((rc = upload_f32(v.v_w2, (size_t)V * kValueHidden, &n.v_w2)) != AZ_OK) return rc;
    if ((rc = upload_f32(v.v_b2, V, &n.v_b2)) != AZ_OK) return rc;

    // workspace
    const size_t B = a.max_batch;
    AZ_CUDA(cudaMalloc(&n.planes, B * 64 * n.in_pad * act_bytes(n)));
    AZ_CUDA(cudaMalloc(&n.act[0], B * 64 * C * act_bytes(n)));
    AZ_CUDA(cudaMalloc((void **)&n.logits, B * az_policy_size(&a) * sizeof(float)));
    AZ_CUDA(cudaMalloc(&n.head_p, B * kHeadChannels * 64 * act_bytes(n)));
    AZ_CUDA(cudaMalloc(&n.head_v, B * kHeadChannels * 64 * act_bytes(n)));
    AZ_CUDA(cudaMalloc((void **)&n.hidden, B * kValueHidden * sizeof(float)));
    AZ_CUDA(cudaMalloc((void **)&n.status_dev, sizeof(uint32_t)));
    AZ_CUDA(cudaMemset(n.status_dev, 0, sizeof(uint32_t)));
    return AZ_OK;
}

void free_net(Net *n) {
    if (!n) return;
    for (int i = 0; i < 1 + 2 * 64; ++i) { cudaFree(n->conv_w[i]); cudaFree(n->conv_scale[i]); cudaFree(n->conv_bias[i]); }
    cudaFree(n->f32_layers);
    cudaFree(n->tc_weights); cudaFree(n->tc_weights_split); cudaFree(n->tc_weights_split4); cudaFree(n->tc_bias); cudaFree(n->tc_head_w); cudaFree(n->tc_head_w_plain); cudaFree(n->tc_head_bias);
    cudaFree(n->tc8_weights); cudaFree(n->tc8_lconst);
    delete static_cast<HostMaster *>(n->host_master);
    cudaFree(n->fc_policy_w); cudaFree(n->fc_value_w); cudaFree(n->u_policy); cudaFree(n->u_value);
    cudaFree(n->p_w); cudaFree(n->p_scale); cudaFree(n->p_bias); cudaFree(n->p_fw); cudaFree(n->p_fbias);
    cudaFree(n->v_cw); cudaFree(n->v_cscale); cudaFree(n->v_cbias); cudaFree(n->v_w1); cudaFree(n->v_b1);
    cudaFree(n->v_w2); cudaFree(n->v_b2);
    cudaFree(n->planes);
    for (int i = 0; i < 3; ++i) cudaFree(n->act[i]);
    cudaFree(n->stage_pos); cudaFree(n->stage_masks); cudaFree(n->stage_policy); cudaFree(n->stage_value);
    cudaFree(n->stage_compact); cudaFree(n->stage_counts);
    for (Net::HostSlot &sl : n->slots) {
        cudaFree(sl.pos); cudaFree(sl.masks); cudaFree(sl.policy); cudaFree(sl.value); cudaFree(sl.compact); cudaFree(sl.counts);
        if (sl.in_ready) cudaEventDestroy(sl.in_ready);
        if (sl.computed) cudaEventDestroy(sl.computed);
        if (sl.out_ready) cudaEventDestroy(sl.out_ready);
    }
    if (n->s_in) cudaStreamDestroy(n->s_in);
    for (cudaStream_t s : n->s_compute) if (s) cudaStreamDestroy(s);
    if (n->s_out) cudaStreamDestroy(n->s_out);
    cudaFree(n->alt_u_policy); cudaFree(n->alt_u_value); cudaFree(n->alt_logits);
    cudaFree(n->alt_act0); cudaFree(n->alt_pnet_qk);
    cudaFree(n->pnet_gw); cudaFree(n->pnet_qk); cudaFree(n->pnet_small); cudaFree(n->pnet_actions);
    free_pnet_master(n->pnet_master);
    if (n->ev_begin) for (int i = 0; i < kMaxProfiledPasses; ++i) { cudaEventDestroy(n->ev_begin[i]); cudaEventDestroy(n->ev_end[i]); }
    delete[] n->ev_begin; delete[] n->ev_end;
    cudaFree(n->logits); cudaFree(n->head_p); cudaFree(n->head_v); cudaFree(n->hidden); cudaFree(n->status_dev);
    delete n;
}

// encoder + tower; *tower_out receives the buffer holding [batch][64][C].  With `fused_heads` (tensor-core
// path only) the tower kernel also runs the 1x1 head projections and leaves the activations on chip.
int run_tower(Net &n, const void *positions, int batch, void **tower_out, bool fused_heads, cudaStream_t s) {
    int rc = AZ_OK;
    const int C = (int)n.arch.channels;
    const bool timed = n.profile > 0 && n.n_events < kMaxProfiledPasses && (++n.profile_count % (unsigned)n.profile) == 0;
    if (n.pnet) {
        // the paper's network: the tower encodes the 52 planes itself, as the other tensor-core towers do
        if (timed) AZ_CUDA(cudaEventRecord(n.ev_begin[n.n_events], s));
        *tower_out = n.act[0];
        rc = launch_tower_tc(n, nullptr, positions, batch, n.act[0], fused_heads, nullptr, s);
        if (rc == AZ_OK && timed) AZ_CUDA(cudaEventRecord(n.ev_end[n.n_events++], s));
        return rc;
    }
    if (n.tc_ready) {
        // the tensor-core tower encodes its boards itself, straight into shared memory
        if (timed) AZ_CUDA(cudaEventRecord(n.ev_begin[n.n_events], s));
        *tower_out = fused_heads ? nullptr : n.act[0];
        rc = launch_tower_tc(n, nullptr, positions, batch, *tower_out, fused_heads, nullptr, s);
        if (rc == AZ_OK && timed) AZ_CUDA(cudaEventRecord(n.ev_end[n.n_events++], s));
        return rc;
    }
    if (n.f32_layers) {
        // 64-channel fp32 networks: encoder and every convolution in one launch, activations resident in shared memory
        if (timed) AZ_CUDA(cudaEventRecord(n.ev_begin[n.n_events], s));
        *tower_out = n.act[0];
        rc = launch_tower_f32(n, positions, batch, static_cast<float *>(n.act[0]), s);
        if (rc == AZ_OK && timed) AZ_CUDA(cudaEventRecord(n.ev_end[n.n_events++], s));
        return rc;
    }
    rc = launch_encode(positions, az_position_bytes(&n.arch), batch, (int)n.arch.in_planes, n.in_pad,
                       n.bf16, n.planes, n.status_dev, s);
    if (rc != AZ_OK) return rc;
    if (timed) AZ_CUDA(cudaEventRecord(n.ev_begin[n.n_events], s));
    void *x = n.act[0], *t = n.act[1], *y = n.act[2];
    rc = launch_conv3x3_simt(n.planes, n.conv_w[0], n.conv_scale[0], n.conv_bias[0], nullptr, x, batch,
                             n.in_pad, C, n.bf16, s);
    if (rc != AZ_OK) return rc;
    for (int b = 0; b < (int)n.arch.blocks; ++b) {
        const int l1 = 1 + 2 * b, l2 = 2 + 2 * b;
        rc = launch_conv3x3_simt(x, n.conv_w[l1], n.conv_scale[l1], n.conv_bias[l1], nullptr, t, batch, C, C, n.bf16, s);
        if (rc != AZ_OK) return rc;
        rc = launch_conv3x3_simt(t, n.conv_w[l2], n.conv_scale[l2], n.conv_bias[l2], x, y, batch, C, C, n.bf16, s);
        if (rc != AZ_OK) return rc;
        void *tmp = x; x = y; y = tmp;
    }
    *tower_out = x;
    if (timed) AZ_CUDA(cudaEventRecord(n.ev_end[n.n_events++], s));
    return AZ_OK;
}

}  // namespace

// Second copy of what an evaluation keeps between its kernels, so that two evaluations of one az_net can
// run side by side on two streams.  The tensor-core path keeps the head GEMM's operands and the logits,
// the paper's network its backbone output and the queries/keys; the other paths have one workspace only.
int ensure_second_workspace(Net &n, bool *available) {
    const az_arch &a = n.arch;
    const size_t B = a.max_batch;
    *available = false;
    if (n.pnet) {
        if (!n.alt_act0) {
            AZ_CUDA(cudaMalloc(&n.alt_act0, B * 64 * a.channels * sizeof(__nv_bfloat16)));
            AZ_CUDA(cudaMalloc(&n.alt_pnet_qk, B * 64 * 256 * sizeof(float)));
        }
        *available = true;
    } else if (n.tc_ready) {
        if (!n.alt_u_value) {
            const size_t u_bytes = (size_t)((a.max_batch + 127) / 128) * kHeadChannels * 64 * 128 * sizeof(__nv_bfloat16);
            AZ_CUDA(cudaMalloc(&n.alt_u_value, u_bytes));
            AZ_CUDA(cudaMemset(n.alt_u_value, 0, u_bytes));
            if (n.u_policy) { AZ_CUDA(cudaMalloc(&n.alt_u_policy, u_bytes)); AZ_CUDA(cudaMemset(n.alt_u_policy, 0, u_bytes)); }
            AZ_CUDA(cudaMalloc((void **)&n.alt_logits, B * az_policy_size(&a) * sizeof(float)));
        }
        *available = true;
    }
    return AZ_OK;
}
// Kernel arguments are captured when a kernel is launched: pointing the net at the other copy for the
// duration of the (asynchronous) launches is all it takes.
void swap_workspace(Net &n) {
    if (n.pnet) { std::swap(n.act[0], n.alt_act0); std::swap(n.pnet_qk, n.alt_pnet_qk); }
    else { std::swap(n.u_policy, n.alt_u_policy); std::swap(n.u_value, n.alt_u_value); std::swap(n.logits, n.alt_logits); }
}

}  // namespace az

using az::Net;

extern "C" {

size_t az_position_bytes(const az_arch *a) {
    return a && a->in_planes == 112 ? sizeof(az_position_h8) : a && a->in_planes == 52 ? sizeof(az_position_m8) : sizeof(az_position);
}
size_t az_policy_size(const az_arch *a) {
    return a && a->policy_head == AZ_POLICY_FLAT1858 ? az::kFlatMoves : a && a->policy_head == AZ_POLICY_FROMTO1880 ? 1880 : az::kPlanes73 * 64;
}
size_t az_mask_words(const az_arch *a) { return a && a->policy_head != AZ_POLICY_PLANES73 ? 30 : 73; }
size_t az_value_size(const az_arch *a) { return a && a->value_head == AZ_VALUE_WDL ? 3 : 1; }
size_t az_plane_channels(const az_arch *a) { return a && a->in_planes == 112 ? 128 : a && a->in_planes == 52 ? 64 : 32; }

int az_load_net(const az_arch *arch, const void *weights_host, size_t nbytes, az_net **out) {
    return az_load_net_ex(arch, weights_host, nbytes, 0u, out);
}

int az_load_net_ex(const az_arch *arch, const void *weights_host, size_t nbytes, uint32_t flags, az_net **out) {
    static_assert(sizeof(az_position) == 104 && sizeof(az_position_h8) == 784 && sizeof(az_position_m8) == 128, "record layout");
    if (!arch || !weights_host || !out) return AZ_ERR_BAD_ARG;
    *out = nullptr;
    if (flags & ~(uint32_t)(AZ_LOAD_TOWER_CTA_PAIRS | AZ_LOAD_TOWER_SINGLE_CTAS)) return AZ_ERR_BAD_ARG;
    if ((flags & AZ_LOAD_TOWER_CTA_PAIRS) && (flags & AZ_LOAD_TOWER_SINGLE_CTAS)) return AZ_ERR_BAD_ARG;
    if (!az::arch_ok(*arch)) return AZ_ERR_BAD_ARCH;
    const bool pnet = arch->in_planes == 52;
    if ((flags & AZ_LOAD_TOWER_CTA_PAIRS) && !az::tc_pair_shape((int)arch->channels, (int)arch->precision, pnet)) return AZ_ERR_UNSUPPORTED;
    // the paper's network ladder: 128, 160 and 176 channels in bf16; 128 and 160 also in int8 (its MMAs take 32
    // channels at a time, which 176 is not a multiple of)
    if (pnet && !((arch->precision == AZ_PREC_BF16 && (arch->channels == 128 || arch->channels == 160 || arch->channels == 176)) ||
                  (arch->precision == AZ_PREC_INT8 && (arch->channels == 128 || arch->channels == 160))))
        return AZ_ERR_UNSUPPORTED;
    az::BlobView view;
    int rc = AZ_OK;
    if (!pnet) rc = az::parse_blob(*arch, static_cast<const unsigned char *>(weights_host), nbytes, view);
    if (rc != AZ_OK) return rc;
    Net *n = new (std::nothrow) Net();
    if (!n) return AZ_ERR_BAD_ARG;
    n->arch = *arch;
    n->want_pair = (flags & AZ_LOAD_TOWER_SINGLE_CTAS) == 0;
    cudaError_t e = cudaGetDevice(&n->device);
    if (e != cudaSuccess) { az::set_cuda_error(e, "cudaGetDevice"); delete n; return AZ_ERR_CUDA; }
    rc = pnet ? az::build_pnet(*n, static_cast<const unsigned char *>(weights_host), nbytes) : az::build_net(*n, view);
    if (rc != AZ_OK) { az::free_net(n); return rc; }
    *out = reinterpret_cast<az_net *>(n);
    return AZ_OK;
}

void az_free_net(az_net *net) { az::free_net(reinterpret_cast<Net *>(net)); }

int az_encode(az_net *net, const void *positions_dev, int batch, void *planes_dev, void *cuda_stream) {
    Net *n = reinterpret_cast<Net *>(net);
    if (!n || batch < 0 || (batch > 0 && (!positions_dev || !planes_dev))) return AZ_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(positions_dev) & 7) || (reinterpret_cast<uintptr_t>(planes_dev) & 15)) return AZ_ERR_BAD_ARG;
    if ((uint32_t)batch > n->arch.max_batch) return AZ_ERR_BATCH_TOO_LARGE;
    if (n->pnet) return az::launch_encode52(positions_dev, batch, true, planes_dev, static_cast<cudaStream_t>(cuda_stream));
    return az::launch_encode(positions_dev, az_position_bytes(&n->arch), batch, (int)n->arch.in_planes,
                             n->in_pad, n->bf16, planes_dev, n->status_dev, static_cast<cudaStream_t>(cuda_stream));
}

int az_encode52(const void *positions_dev, int batch, int bf16, void *planes_dev, void *cuda_stream) {
    if (batch < 0 || (batch > 0 && (!positions_dev || !planes_dev))) return AZ_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(positions_dev) & 7) || (reinterpret_cast<uintptr_t>(planes_dev) & 15)) return AZ_ERR_BAD_ARG;
    return az::launch_encode52(positions_dev, batch, bf16 != 0, planes_dev, static_cast<cudaStream_t>(cuda_stream));
}

int az_tower(az_net *net, const void *positions_dev, int batch, void *tower_dev, void *cuda_stream) {
    Net *n = reinterpret_cast<Net *>(net);
    if (!n || batch < 0 || (batch > 0 && (!positions_dev || !tower_dev))) return AZ_ERR_BAD_ARG;
    if (reinterpret_cast<uintptr_t>(positions_dev) & 7) return AZ_ERR_BAD_ARG;
    if ((uint32_t)batch > n->arch.max_batch) return AZ_ERR_BATCH_TOO_LARGE;
    if (batch == 0) return AZ_OK;
    if (n->fp8 && !n->fp8_ready) return AZ_ERR_NOT_CALIBRATED;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    void *x = nullptr;
    int rc = az::run_tower(*n, positions_dev, batch, &x, false, s);
    if (rc != AZ_OK) return rc;
    AZ_CUDA(cudaMemcpyAsync(tower_dev, x, (size_t)batch * 64 * n->arch.channels * az::act_bytes(*n),
                            cudaMemcpyDeviceToDevice, s));
    return AZ_OK;
}

// policy_dev (dense rows) or legal_dev + counts_dev (legal moves only): exactly one form is requested
static int evaluate_impl(az_net *net, const void *positions_dev, const uint64_t *legal_masks_dev, int batch,
                         float *policy_dev, float *legal_dev, int32_t *counts_dev, float *value_dev, void *cuda_stream) {
    Net *n = reinterpret_cast<Net *>(net);
    if (!n || batch < 0) return AZ_ERR_BAD_ARG;
    if (batch == 0) return AZ_OK;
    const bool dense = policy_dev != nullptr;
    if (!positions_dev || !legal_masks_dev || !value_dev || (!dense && (!legal_dev || !counts_dev))) return AZ_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(positions_dev) & 7) || (reinterpret_cast<uintptr_t>(legal_masks_dev) & 7) ||
        (reinterpret_cast<uintptr_t>(dense ? (void *)policy_dev : (void *)legal_dev) & 3) ||
        (reinterpret_cast<uintptr_t>(counts_dev) & 3) || (reinterpret_cast<uintptr_t>(value_dev) & 3))
        return AZ_ERR_BAD_ARG;
    if ((uint32_t)batch > n->arch.max_batch) return AZ_ERR_BATCH_TOO_LARGE;
    if (n->fp8 && !n->fp8_ready) return AZ_ERR_NOT_CALIBRATED;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const az_arch &a = n->arch;
    const int C = (int)a.channels;
    void *h = nullptr;
    int rc = az::run_tower(*n, positions_dev, batch, &h, n->tc_ready, s);
    if (rc != AZ_OK) return rc;
    if (n->pnet) return az::launch_pnet_finish(*n, legal_masks_dev, batch, policy_dev, legal_dev, counts_dev, value_dev, s);
    if (n->tc_ready) {
        // the tower kernel has produced the 73-plane logits or the flat head's projection, and the value
        // projection; one GEMM launch finishes both heads, the softmax follows
        rc = az::launch_fc_tc(*n, batch, value_dev, s);
        if (rc != AZ_OK) return rc;
        if (!dense)
            return az::launch_masked_softmax_compact(n->logits, legal_masks_dev, batch, (int)az_policy_size(&a),
                                                     (int)az_mask_words(&a), legal_dev, counts_dev, n->status_dev, true, s);
        return az::launch_masked_softmax(n->logits, legal_masks_dev, batch, (int)az_policy_size(&a), (int)az_mask_words(&a),
                                         policy_dev, n->status_dev, true, s);
    }
    if (n->f32_layers && a.policy_head == AZ_POLICY_PLANES73)      // 64-channel fp32 networks: both heads and the softmax in one launch
        return az::launch_heads_f32(*n, h, legal_masks_dev, batch, policy_dev, legal_dev, counts_dev, value_dev, s);
    if (a.policy_head == AZ_POLICY_PLANES73) {
        rc = az::launch_conv1x1(h, n->p_w, nullptr, n->p_bias, batch, C, az::kPlanes73, false, n->bf16, n->logits, true, s);
        if (rc != AZ_OK) return rc;
    } else {
        rc = az::launch_conv1x1(h, n->p_w, n->p_scale, n->p_bias, batch, C, az::kHeadChannels, true, n->bf16, n->head_p, !n->bf16, s);
        if (rc != AZ_OK) return rc;
        rc = az::launch_fc(n->head_p, n->p_fw, n->p_fbias, batch, az::kFlatMoves, az::kHeadChannels * 64, false, n->bf16, n->logits, true, s);
        if (rc != AZ_OK) return rc;
    }
    rc = az::launch_conv1x1(h, n->v_cw, n->v_cscale, n->v_cbias, batch, C, az::kHeadChannels, true, n->bf16, n->head_v, !n->bf16, s);
    if (rc != AZ_OK) return rc;
    rc = az::launch_fc(n->head_v, n->v_w1, n->v_b1, batch, az::kValueHidden, az::kHeadChannels * 64, true, n->bf16, n->hidden, true, s);
    if (rc != AZ_OK) return rc;
    rc = az::launch_value_tail(n->hidden, n->v_w2, n->v_b2, batch, a.value_head == AZ_VALUE_WDL, value_dev, s);
    if (rc != AZ_OK) return rc;
    if (!dense)
        return az::launch_masked_softmax_compact(n->logits, legal_masks_dev, batch, (int)az_policy_size(&a),
                                                 (int)az_mask_words(&a), legal_dev, counts_dev, n->status_dev, false, s);
    return az::launch_masked_softmax(n->logits, legal_masks_dev, batch, (int)az_policy_size(&a), (int)az_mask_words(&a),
                                     policy_dev, n->status_dev, false, s);
}

int az_evaluate(az_net *net, const void *positions_dev, const uint64_t *legal_masks_dev, int batch,
                float *policy_dev, float *value_dev, void *cuda_stream) {
    if (!policy_dev && batch > 0) return AZ_ERR_BAD_ARG;
    return evaluate_impl(net, positions_dev, legal_masks_dev, batch, policy_dev, nullptr, nullptr, value_dev, cuda_stream);
}

int az_evaluate_legal(az_net *net, const void *positions_dev, const uint64_t *legal_masks_dev, int batch,
                      float *legal_policy_dev, int32_t *legal_counts_dev, float *value_dev, void *cuda_stream) {
    if ((!legal_policy_dev || !legal_counts_dev) && batch > 0) return AZ_ERR_BAD_ARG;
    return evaluate_impl(net, positions_dev, legal_masks_dev, batch, nullptr, legal_policy_dev, legal_counts_dev, value_dev, cuda_stream);
}

int az_evaluate_legal_host(az_net *net, const void *positions_host, const uint64_t *legal_masks_host, int batch,
                           float *legal_policy_host, int32_t *legal_counts_host, float *value_host, void *cuda_stream) {
    Net *n = reinterpret_cast<Net *>(net);
    if (!n || batch < 0) return AZ_ERR_BAD_ARG;
    if (batch == 0) return AZ_OK;
    if (!positions_host || !legal_masks_host || !legal_policy_host || !legal_counts_host || !value_host) return AZ_ERR_BAD_ARG;
    if ((uint32_t)batch > n->arch.max_batch) return AZ_ERR_BATCH_TOO_LARGE;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const az_arch &a = n->arch;
    const size_t B = a.max_batch, pb = az_position_bytes(&a), mw = az_mask_words(&a), vs = az_value_size(&a);
    if (!n->stage_pos) {
        AZ_CUDA(cudaMalloc(&n->stage_pos, B * pb));
        AZ_CUDA(cudaMalloc((void **)&n->stage_masks, B * mw * sizeof(uint64_t)));
        AZ_CUDA(cudaMalloc((void **)&n->stage_policy, B * az_policy_size(&a) * sizeof(float)));
        AZ_CUDA(cudaMalloc((void **)&n->stage_value, B * vs * sizeof(float)));
    }
    if (!n->stage_compact) {
        AZ_CUDA(cudaMalloc((void **)&n->stage_compact, B * AZ_MAX_LEGAL * sizeof(float)));
        AZ_CUDA(cudaMalloc((void **)&n->stage_counts, B * sizeof(int)));
    }
    AZ_CUDA(cudaMemcpyAsync(n->stage_pos, positions_host, (size_t)batch * pb, cudaMemcpyHostToDevice, s));
    AZ_CUDA(cudaMemcpyAsync(n->stage_masks, legal_masks_host, (size_t)batch * mw * sizeof(uint64_t), cudaMemcpyHostToDevice, s));
    int rc = az_evaluate_legal(net, n->stage_pos, n->stage_masks, batch, n->stage_compact, n->stage_counts, n->stage_value, cuda_stream);
    if (rc != AZ_OK) return rc;
    AZ_CUDA(cudaMemcpyAsync(legal_policy_host, n->stage_compact, (size_t)batch * AZ_MAX_LEGAL * sizeof(float), cudaMemcpyDeviceToHost, s));
    AZ_CUDA(cudaMemcpyAsync(legal_counts_host, n->stage_counts, (size_t)batch * sizeof(int), cudaMemcpyDeviceToHost, s));
    AZ_CUDA(cudaMemcpyAsync(value_host, n->stage_value, (size_t)batch * vs * sizeof(float), cudaMemcpyDeviceToHost, s));
    AZ_CUDA(cudaStreamSynchronize(s));
    return AZ_OK;
}

int az_evaluate_host(az_net *net, const void *positions_host, const uint64_t *legal_masks_host, int batch,
                     float *policy_host, float *value_host, void *cuda_stream) {
    Net *n = reinterpret_cast<Net *>(net);
    if (!n || batch < 0) return AZ_ERR_BAD_ARG;
    if (batch == 0) return AZ_OK;
    if (!positions_host || !legal_masks_host || !policy_host || !value_host) return AZ_ERR_BAD_ARG;
    if ((uint32_t)batch > n->arch.max_batch) return AZ_ERR_BATCH_TOO_LARGE;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const az_arch &a = n->arch;
    const size_t B = a.max_batch, pb = az_position_bytes(&a), mw = az_mask_words(&a), ps = az_policy_size(&a), vs = az_value_size(&a);
    if (!n->stage_pos) {
        AZ_CUDA(cudaMalloc(&n->stage_pos, B * pb));
        AZ_CUDA(cudaMalloc((void **)&n->stage_masks, B * mw * sizeof(uint64_t)));
        AZ_CUDA(cudaMalloc((void **)&n->stage_policy, B * ps * sizeof(float)));
        AZ_CUDA(cudaMalloc((void **)&n->stage_value, B * vs * sizeof(float)));
    }
    AZ_CUDA(cudaMemcpyAsync(n->stage_pos, positions_host, (size_t)batch * pb, cudaMemcpyHostToDevice, s));
    AZ_CUDA(cudaMemcpyAsync(n->stage_masks, legal_masks_host, (size_t)batch * mw * sizeof(uint64_t), cudaMemcpyHostToDevice, s));
    int rc = az_evaluate(net, n->stage_pos, n->stage_masks, batch, n->stage_policy, n->stage_value, cuda_stream);
    if (rc != AZ_OK) return rc;
    AZ_CUDA(cudaMemcpyAsync(policy_host, n->stage_policy, (size_t)batch * ps * sizeof(float), cudaMemcpyDeviceToHost, s));
    AZ_CUDA(cudaMemcpyAsync(value_host, n->stage_value, (size_t)batch * vs * sizeof(float), cudaMemcpyDeviceToHost, s));
    AZ_CUDA(cudaStreamSynchronize(s));
    return AZ_OK;
}

int az_submit_host(az_net *net, const void *positions_host, const uint64_t *legal_masks_host, int batch,
                   float *policy_host, float *legal_policy_host, int32_t *legal_counts_host,
                   float *value_host, int *ticket) {
    Net *n = reinterpret_cast<Net *>(net);
    if (!n || batch <= 0 || !ticket || !positions_host || !legal_masks_host || !value_host) return AZ_ERR_BAD_ARG;
    const bool dense = policy_host != nullptr;
    if (!dense && (!legal_policy_host || !legal_counts_host)) return AZ_ERR_BAD_ARG;
    if ((uint32_t)batch > n->arch.max_batch) return AZ_ERR_BATCH_TOO_LARGE;
    if (n->fp8 && !n->fp8_ready) return AZ_ERR_NOT_CALIBRATED;
    const az_arch &a = n->arch;
    const size_t B = a.max_batch, pb = az_position_bytes(&a), mw = az_mask_words(&a), ps = az_policy_size(&a), vs = az_value_size(&a);
    if (!n->s_in) {
        AZ_CUDA(cudaStreamCreateWithFlags(&n->s_in, cudaStreamNonBlocking));
        AZ_CUDA(cudaStreamCreateWithFlags(&n->s_out, cudaStreamNonBlocking));
        AZ_CUDA(cudaStreamCreateWithFlags(&n->s_compute[0], cudaStreamNonBlocking));
        // with a second copy of the workspace odd slots run on a stream of their own; the paths that share
        // one workspace take turns on one stream
        bool second = false;
        const int rc2 = az::ensure_second_workspace(*n, &second);
        if (rc2 != AZ_OK) return rc2;
        if (second) AZ_CUDA(cudaStreamCreateWithFlags(&n->s_compute[1], cudaStreamNonBlocking));
    }
    Net::HostSlot &sl = n->slots[n->next_slot];
    if (sl.busy) return AZ_ERR_BUSY;
    const bool alt = n->s_compute[1] != nullptr && (n->next_slot & 1);
    cudaStream_t sc = alt ? n->s_compute[1] : n->s_compute[0];
    if (!sl.pos) {
        AZ_CUDA(cudaMalloc(&sl.pos, B * pb));
        AZ_CUDA(cudaMalloc((void **)&sl.masks, B * mw * sizeof(uint64_t)));
        AZ_CUDA(cudaMalloc((void **)&sl.value, B * vs * sizeof(float)));
        AZ_CUDA(cudaEventCreateWithFlags(&sl.in_ready, cudaEventDisableTiming));
        AZ_CUDA(cudaEventCreateWithFlags(&sl.computed, cudaEventDisableTiming));
        AZ_CUDA(cudaEventCreateWithFlags(&sl.out_ready, cudaEventDisableTiming));
    }
    if (dense && !sl.policy) AZ_CUDA(cudaMalloc((void **)&sl.policy, B * ps * sizeof(float)));
    if (!dense && !sl.compact) {
        AZ_CUDA(cudaMalloc((void **)&sl.compact, B * AZ_MAX_LEGAL * sizeof(float)));
        AZ_CUDA(cudaMalloc((void **)&sl.counts, B * sizeof(int)));
    }
    // A slot is handed out again only after az_wait_host saw its result copy finish, and that copy was
    // ordered after the slot's kernels: neither the staging inputs nor the outputs are still in use.
    AZ_CUDA(cudaMemcpyAsync(sl.pos, positions_host, (size_t)batch * pb, cudaMemcpyHostToDevice, n->s_in));
    AZ_CUDA(cudaMemcpyAsync(sl.masks, legal_masks_host, (size_t)batch * mw * sizeof(uint64_t), cudaMemcpyHostToDevice, n->s_in));
    AZ_CUDA(cudaEventRecord(sl.in_ready, n->s_in));
    AZ_CUDA(cudaStreamWaitEvent(sc, sl.in_ready, 0));
    // kernel arguments are captured when a kernel is launched: pointing the net at the other copy for
    // the duration of the (asynchronous) launches is all it takes
    if (alt) az::swap_workspace(*n);
    const int rc = dense ? az_evaluate(net, sl.pos, sl.masks, batch, sl.policy, sl.value, sc)
                         : az_evaluate_legal(net, sl.pos, sl.masks, batch, sl.compact, sl.counts, sl.value, sc);
    if (alt) az::swap_workspace(*n);
    if (rc != AZ_OK) return rc;
    AZ_CUDA(cudaEventRecord(sl.computed, sc));
    AZ_CUDA(cudaStreamWaitEvent(n->s_out, sl.computed, 0));
    if (dense) {
        AZ_CUDA(cudaMemcpyAsync(policy_host, sl.policy, (size_t)batch * ps * sizeof(float), cudaMemcpyDeviceToHost, n->s_out));
    } else {
        AZ_CUDA(cudaMemcpyAsync(legal_policy_host, sl.compact, (size_t)batch * AZ_MAX_LEGAL * sizeof(float), cudaMemcpyDeviceToHost, n->s_out));
        AZ_CUDA(cudaMemcpyAsync(legal_counts_host, sl.counts, (size_t)batch * sizeof(int), cudaMemcpyDeviceToHost, n->s_out));
    }
    AZ_CUDA(cudaMemcpyAsync(value_host, sl.value, (size_t)batch * vs * sizeof(float), cudaMemcpyDeviceToHost, n->s_out));
    AZ_CUDA(cudaEventRecord(sl.out_ready, n->s_out));
    sl.busy = true;
    *ticket = n->next_slot;
    n->next_slot = (n->next_slot + 1) % AZ_HOST_SLOTS;
    return AZ_OK;
}

int az_wait_host(az_net *net, int ticket) {
    Net *n = reinterpret_cast<Net *>(net);
    if (!n || ticket < 0 || ticket >= AZ_HOST_SLOTS || !n->slots[ticket].busy) return AZ_ERR_BAD_ARG;
    Net::HostSlot &sl = n->slots[ticket];
    sl.busy = false;
    AZ_CUDA(cudaEventSynchronize(sl.out_ready));
    return AZ_OK;
}

int az_profile_tower(az_net *net, int enable) {
    Net *n = reinterpret_cast<Net *>(net);
    if (!n) return AZ_ERR_BAD_ARG;
    if (enable && !n->ev_begin) {
        n->ev_begin = new (std::nothrow) cudaEvent_t[az::kMaxProfiledPasses];
        n->ev_end = new (std::nothrow) cudaEvent_t[az::kMaxProfiledPasses];
        if (!n->ev_begin || !n->ev_end) return AZ_ERR_BAD_ARG;
        for (int i = 0; i < az::kMaxProfiledPasses; ++i) {
            AZ_CUDA(cudaEventCreate(&n->ev_begin[i]));
            AZ_CUDA(cudaEventCreate(&n->ev_end[i]));
        }
    }
    if (enable < 0) return AZ_ERR_BAD_ARG;
    n->profile = enable;
    n->profile_count = 0;
    return AZ_OK;
}

int az_tower_time(az_net *net, float *total_ms_out, int *passes_out) {
    Net *n = reinterpret_cast<Net *>(net);
    if (!n || !total_ms_out || !passes_out) return AZ_ERR_BAD_ARG;
    float total = 0.0f;
    for (int i = 0; i < n->n_events; ++i) {
        float ms = 0.0f;
        AZ_CUDA(cudaEventSynchronize(n->ev_end[i]));
        AZ_CUDA(cudaEventElapsedTime(&ms, n->ev_begin[i], n->ev_end[i]));
        total += ms;
    }
    *total_ms_out = total;
    *passes_out = n->n_events;
    n->n_events = 0;
    return AZ_OK;
}

int az_legal_masks(const void *positions_dev, size_t position_stride, int batch, int policy_head,
                   uint64_t *masks_dev, void *cuda_stream) {
    if (batch < 0 || policy_head < AZ_POLICY_PLANES73 || policy_head > AZ_POLICY_FROMTO1880) return AZ_ERR_BAD_ARG;
    if (batch == 0) return AZ_OK;
    if (!positions_dev || !masks_dev || position_stride < sizeof(az_position) || (position_stride & 7)) return AZ_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(positions_dev) & 7) || (reinterpret_cast<uintptr_t>(masks_dev) & 7)) return AZ_ERR_BAD_ARG;
    return az::launch_legal_masks(positions_dev, position_stride, batch, policy_head, masks_dev,
                                  static_cast<cudaStream_t>(cuda_stream));
}

int az_calibrate(az_net *net, const void *positions_dev, int count, void *cuda_stream) {
    return az_calibrate_ex(net, positions_dev, count, 0u, cuda_stream);
}

int az_calibrate_ex(az_net *net, const void *positions_dev, int count, uint32_t flags, void *cuda_stream) {
    Net *n = reinterpret_cast<Net *>(net);
    if (!n || count <= 0 || !positions_dev || (reinterpret_cast<uintptr_t>(positions_dev) & 7)) return AZ_ERR_BAD_ARG;
    if (flags & ~(uint32_t)AZ_CALIBRATE_NO_BIAS_CORRECTION) return AZ_ERR_BAD_ARG;
    if (!n->fp8 || (!n->host_master && !n->pnet_master)) return AZ_ERR_UNSUPPORTED;
    // the paper network's context maps are rescaled by its first calibration, finished or not
    if (n->pnet && (n->fp8_ready || n->calib_broken)) return AZ_ERR_UNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const int C = (int)n->arch.channels, L = n->n_conv;
    const size_t pb = az_position_bytes(&n->arch);
    // 1. bf16 tower over the calibration positions, recording every layer's per-channel output maximum and the sum
    //    of its pre-activation values (for the bias correction of step 3)
    unsigned int *absmax_dev = nullptr;
    double *presum_dev = nullptr;
    AZ_CUDA(cudaMalloc((void **)&absmax_dev, (size_t)L * C * sizeof(unsigned int)));
    if (cudaMalloc((void **)&presum_dev, (size_t)L * C * sizeof(double)) != cudaSuccess) { cudaFree(absmax_dev); return AZ_ERR_CUDA; }
    cudaError_t e = cudaMemsetAsync(absmax_dev, 0, (size_t)L * C * sizeof(unsigned int), s);
    if (e == cudaSuccess) e = cudaMemsetAsync(presum_dev, 0, (size_t)L * C * sizeof(double), s);
    int rc = AZ_OK;
    // one pass of the tower (whichever form is ready) over all calibration positions
    auto tower_pass = [&](unsigned int *absmax_hook) {
        for (int first = 0; first < count && rc == AZ_OK && e == cudaSuccess; first += (int)n->arch.max_batch) {
            const int chunk = count - first < (int)n->arch.max_batch ? count - first : (int)n->arch.max_batch;
            const unsigned char *p = static_cast<const unsigned char *>(positions_dev) + (size_t)first * pb;
            rc = az::launch_tower_tc(*n, nullptr, p, chunk, nullptr, false, absmax_hook, s);
        }
    };
    n->calib_presum = presum_dev;
    tower_pass(absmax_dev);
    n->calib_presum = nullptr;
    std::vector<float> absmax((size_t)L * C);
    std::vector<double> mean_exact((size_t)L * C);
    if (rc == AZ_OK && e == cudaSuccess) e = cudaMemcpyAsync(absmax.data(), absmax_dev, absmax.size() * sizeof(float), cudaMemcpyDeviceToHost, s);
    if (rc == AZ_OK && e == cudaSuccess) e = cudaMemcpyAsync(mean_exact.data(), presum_dev, mean_exact.size() * sizeof(double), cudaMemcpyDeviceToHost, s);
    if (rc == AZ_OK && e == cudaSuccess) e = cudaStreamSynchronize(s);
    cudaFree(absmax_dev);
    if (rc != AZ_OK || e != cudaSuccess) cudaFree(presum_dev);
    if (rc != AZ_OK) return rc;
    if (e != cudaSuccess) { az::set_cuda_error(e, "az_calibrate"); return AZ_ERR_CUDA; }
    // from here on presum_dev is freed on every path through free_presum
    struct Guard { double *p; ~Guard() { cudaFree(p); } } free_presum{presum_dev};
    // 2. quantise the tower with those ranges
    std::vector<float> lconst;
    std::vector<int> next_cin(L, C);                  // output channels of layer l that the next layer reads as 8-bit activations
    next_cin[L - 1] = 0;
    int vecs = 3;                                     // constant vectors per layer: scale, bias, residual ratio (+ cap)
    if (n->pnet) {
        rc = az::quantise_pnet(*n, absmax.data(), &lconst, &next_cin);
        if (rc != AZ_OK) return rc;
        vecs = 4;
    } else {
        az::HostMaster *hm = static_cast<az::HostMaster *>(n->host_master);
        std::vector<const float *> w, sc, bi;
        for (int l = 0; l < L; ++l) { w.push_back(hm->w[l].data()); sc.push_back(hm->scale[l].data()); bi.push_back(hm->bias[l].data()); }
        const size_t bytes = az::tc8_packed_weight_bytes(n->in_pad, C, L, n->split_w);
        std::vector<unsigned char> packed(bytes);
        lconst.resize((size_t)L * 3 * C);
        az::tc8_pack(w.data(), sc.data(), bi.data(), absmax.data(), (int)n->arch.in_planes, n->in_pad, C, L, n->int8, n->split_w, n->tc_pair8 ? 2 : 1, packed.data(), lconst.data());
        if (!n->tc8_weights) AZ_CUDA(cudaMalloc(&n->tc8_weights, bytes));
        if (!n->tc8_lconst) AZ_CUDA(cudaMalloc((void **)&n->tc8_lconst, lconst.size() * sizeof(float)));
        AZ_CUDA(cudaMemcpy(n->tc8_weights, packed.data(), bytes, cudaMemcpyHostToDevice));
        AZ_CUDA(cudaMemcpy(n->tc8_lconst, lconst.data(), lconst.size() * sizeof(float), cudaMemcpyHostToDevice));
        n->fp8_ready = true;
        n->calib_broken = false;
    }
    // 3. bias correction (the usual post-training remedy for the systematic part of the rounding error: weights
    //    rounded to 8 bits meet activations that are not zero-mean, which shifts every output channel's mean).
    //    Layer by layer, in order, the 8-bit tower runs over the calibration positions and the layer's biases are
    //    moved so that its mean pre-activation per channel equals the bf16 tower's.  Layer 0 is bf16 in both.  In
    //    the paper's network the pooled quarter of a pooled block's first convolution stays as it is (those
    //    channels are not handed on as 8-bit activations and take another path through the kernel).
    if (flags & AZ_CALIBRATE_NO_BIAS_CORRECTION) return AZ_OK;
    // a failure from here on leaves the biases partly corrected: the net then counts as not calibrated
    struct Unready { Net *n; bool armed; ~Unready() { if (armed) { n->fp8_ready = false; n->calib_broken = true; } } } unready{n, true};
    const float kMax = n->int8 ? 255.0f : 448.0f;
    const double cells = (double)count * 64.0;
    std::vector<double> sum_q(C);
    for (int l = 1; l < L; ++l) {
        AZ_CUDA(cudaMemsetAsync(presum_dev, 0, (size_t)L * C * sizeof(double), s));
        n->calib_presum = presum_dev;
        tower_pass(nullptr);
        n->calib_presum = nullptr;
        if (rc != AZ_OK) return rc;
        if (e != cudaSuccess) { az::set_cuda_error(e, "az_calibrate"); return AZ_ERR_CUDA; }
        AZ_CUDA(cudaMemcpyAsync(sum_q.data(), presum_dev + (size_t)l * C, (size_t)C * sizeof(double), cudaMemcpyDeviceToHost, s));
        AZ_CUDA(cudaStreamSynchronize(s));
        float *bias_q = lconst.data() + ((size_t)l * vecs + 1) * C;    // bias x the layer's output scale
        const bool pooled_layer = n->pnet && (l & 3) == 3;
        const int correct = pooled_layer ? C - C / 4 : C;
        for (int c = 0; c < correct; ++c) {
            const float top = absmax[(size_t)l * C + c];                              // the channel's largest output
            if (!(top > 1e-20f)) continue;                                            // a dead channel has nothing to correct
            const float qs = c < next_cin[l] ? kMax / top : 1.0f;
            const double want = mean_exact[(size_t)l * C + c] / cells;                // real units
            const double have = sum_q[c] / cells / qs;
            double corr = want - have;
            if (!std::isfinite(corr)) continue;
            // a shift of the mean is a fraction of the channel's range; anything larger is not rounding error
            if (corr > 0.25 * top) corr = 0.25 * top;
            if (corr < -0.25 * top) corr = -0.25 * top;
            bias_q[c] += (float)(corr * qs);
        }
        AZ_CUDA(cudaMemcpyAsync(n->tc8_lconst + ((size_t)l * vecs + 1) * C, bias_q, (size_t)C * sizeof(float), cudaMemcpyHostToDevice, s));
    }
    AZ_CUDA(cudaStreamSynchronize(s));
    unready.armed = false;
    return AZ_OK;
}

int az_device_status(az_net *net, void *cuda_stream, uint32_t *status_out) {
    Net *n = reinterpret_cast<Net *>(net);
    if (!n || !status_out) return AZ_ERR_BAD_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    AZ_CUDA(cudaMemcpyAsync(status_out, n->status_dev, sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
    AZ_CUDA(cudaMemsetAsync(n->status_dev, 0, sizeof(uint32_t), s));
    AZ_CUDA(cudaStreamSynchronize(s));
    return (*status_out & az::kStatusWaitTimeout) ? AZ_ERR_DEVICE_TIMEOUT : AZ_OK;
}

int az_launches_per_evaluate(const az_net *net, int batch) {
    const Net *n = reinterpret_cast<const Net *>(net);
    if (!n || batch <= 0) return 0;
    if (n->pnet) return az::tower_tc_launch_count() /*encoder + tower + query/key maps*/ + 1 /*scores, softmax, value head*/;
    if (n->tc_ready) return az::tower_tc_launch_count() /*encoder + tower + head projections*/ + 1 /*head GEMMs*/ + 1 /*softmax*/;
    const int policy = n->arch.policy_head == AZ_POLICY_PLANES73 ? 1 : 2;
    if (n->f32_layers && n->arch.policy_head == AZ_POLICY_PLANES73) return 1 /*encoder + tower*/ + 1 /*heads + softmax*/;
    if (n->f32_layers) return 1 /*encoder + tower*/ + policy + 3 /*value*/ + 1 /*softmax*/;
    return 1 /*encode*/ + n->n_conv + policy + 3 /*value*/ + 1 /*softmax*/;
}

const char *az_strerror(int code) {
    switch (code) {
        case AZ_OK: return "ok";
        case AZ_ERR_BAD_ARG: return "bad argument";
        case AZ_ERR_BAD_ARCH: return "unsupported network shape";
        case AZ_ERR_BAD_WEIGHTS: return "malformed weight blob";
        case AZ_ERR_BATCH_TOO_LARGE: return "batch exceeds max_batch";
        case AZ_ERR_CUDA: return "CUDA runtime error";
        case AZ_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait ran out";
        case AZ_ERR_NOT_CALIBRATED: return "FP8 network not calibrated";
        case AZ_ERR_UNSUPPORTED: return "not supported by this build";
        case AZ_ERR_BUSY: return "all in-flight slots are taken";
        default: return "unknown error";
    }
}

const char *az_last_cuda_error(void) { return az::g_cuda_error.c_str(); }

}  // extern "C"
