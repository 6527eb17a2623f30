/*
 * ORACLE (test infrastructure, not the product): the paper's own inference network in double
 * precision, step by step as Sec. 3.2, Sec. 4.3 and App. D.1 describe it.
 *
 *  - Input: 52 planes (orc_encode52), 3x3 input convolution, folded normalisation, capped activation.
 *  - Backbone: L scaled post-activation residual blocks (Sec. 4.3.6): convolution, normalisation,
 *    capped activation, convolution, normalisation, scaled residual addition, capped activation;
 *    activations capped at six, act(z) = min(max(z, 0), 6); the branch scale 1/sqrt(L) is folded
 *    into the second convolution's scale and bias by whoever writes the weights ("at export").
 *  - Global context in every second block (blocks 1, 3, 5, ... counting from 0; Sec. 3.2, 4.3.3):
 *    board-wide means and maxima of one quarter of the channels are projected back as biases on
 *    the local features.  Reading adopted where the text is silent, chosen so that the parameter
 *    count of the 14 x 160 network comes out at the paper's 6.3 million: in such a block the LAST
 *    C/4 output channels of the first convolution are the pooled ones; after normalisation and
 *    activation their mean and their maximum over the 64 squares (means first, then maxima) go
 *    through one bias-free linear map to 3C/4 values, which are added to the other 3C/4 channels
 *    before their activation; the second convolution reads those 3C/4 channels only.
 *  - Policy head (App. D.1): every square's features are projected to a K = 128 dimensional token
 *    (1x1 convolution with bias, no activation), query and key vectors are linear maps of the
 *    token, the score of (origin, destination) is q_origin . k_destination / sqrt(K); the 1,792
 *    pair actions take their score, the 88 promotion actions add an offset per promotion piece
 *    (queen, rook, bishop, knight), a linear map of the origin's token (reading: the text says
 *    only that offsets distinguish the pieces).  Squares are in the mover's orientation.
 *  - Value head (App. D.1): 1x1 convolution to two channels, normalisation, ReLU, flattening
 *    (channel-major), a 48-unit hidden layer with ReLU, three logits, softmax = win, draw, loss
 *    for the player to move.
 *  - Illegal actions are masked before the softmax over the legal moves.
 *
 * Weight blob: 64-byte header ("AZPNET1\0", uint32 version = 1, blocks, channels, key size, value
 * channels, value hidden units, tensor count, zero padding), then float32 tensors:
 *   in.w[C][52][3][3] in.scale[C] in.bias[C]
 *   per block: w1[C][C][3][3] scale1[C] bias1[C]; pooled blocks: gw[3C/4][C/2];
 *              w2[C][C or 3C/4][3][3] scale2[C] bias2[C]
 *   t.w[K][C] t.b[K]  q.w[K][K] q.b[K]  k.w[K][K] k.b[K]  o.w[4][K] o.b[4]
 *   v.cw[VC][C] v.cscale[VC] v.cbias[VC]  v.w1[VH][VC*64] v.b1[VH]  v.w2[3][VH] v.b2[3]
 *
 * Pins (tests, CPU only): the whole network against a float64 library composition; the pooled
 * block against its plain definition on tiny sizes; closed forms of the score (identity maps give
 * a symmetric Gram matrix), of the cap and of the promotion offsets.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

void orc_conv3x3(const float *W, const double *in, int cin, int cout, double *out);
void orc_masked_softmax(const double *logits, const uint64_t *mask, int n, double *probs);
int orc_policy_index(int head, int stm, int from, int to, int promo, int castle);

typedef struct {
    int L, C, K, VC, VH;
    const float *in_w, *in_s, *in_b;
    const float **w1, **s1, **b1, **gw, **w2, **s2, **b2;
    const float *t_w, *t_b, *q_w, *q_b, *k_w, *k_b, *o_w, *o_b;
    const float *v_cw, *v_cs, *v_cb, *v_w1, *v_b1, *v_w2, *v_b2;
} PNet;

enum { P_PLANES = 52, P_ACTIONS = 1880, P_PAIRS = 1792 };

static int pooled_block(int b) { return (b & 1) == 1; }

static int parse(const uint8_t *blob, size_t nbytes, PNet *net) {
    if (nbytes < 64 || memcmp(blob, "AZPNET1", 8) != 0) return -1;
    uint32_t h[7];
    memcpy(h, blob + 8, sizeof h);
    if (h[0] != 1) return -1;
    net->L = (int)h[1]; net->C = (int)h[2]; net->K = (int)h[3]; net->VC = (int)h[4]; net->VH = (int)h[5];
    const int L = net->L, C = net->C, K = net->K, P = C / 4, R = C - P;
    if (C % 4 || L < 0 || K <= 0) return -1;
    const float *p = (const float *)(blob + 64);
    const float *end = (const float *)(blob + (nbytes & ~(size_t)3));
#define TAKE(dst, count) do { dst = p; p += (size_t)(count); if (p > end) return -1; } while (0)
    TAKE(net->in_w, (size_t)C * P_PLANES * 9); TAKE(net->in_s, C); TAKE(net->in_b, C);
    net->w1 = malloc(sizeof(float *) * 7 * (size_t)(L > 0 ? L : 1));
    net->s1 = net->w1 + L; net->b1 = net->s1 + L; net->gw = net->b1 + L; net->w2 = net->gw + L;
    net->s2 = net->w2 + L; net->b2 = net->s2 + L;
    for (int b = 0; b < L; ++b) {
        TAKE(net->w1[b], (size_t)C * C * 9); TAKE(net->s1[b], C); TAKE(net->b1[b], C);
        net->gw[b] = NULL;
        if (pooled_block(b)) TAKE(net->gw[b], (size_t)R * 2 * P);
        TAKE(net->w2[b], (size_t)C * (pooled_block(b) ? R : C) * 9); TAKE(net->s2[b], C); TAKE(net->b2[b], C);
    }
    TAKE(net->t_w, (size_t)K * C); TAKE(net->t_b, K);
    TAKE(net->q_w, (size_t)K * K); TAKE(net->q_b, K);
    TAKE(net->k_w, (size_t)K * K); TAKE(net->k_b, K);
    TAKE(net->o_w, (size_t)4 * K); TAKE(net->o_b, 4);
    TAKE(net->v_cw, (size_t)net->VC * C); TAKE(net->v_cs, net->VC); TAKE(net->v_cb, net->VC);
    TAKE(net->v_w1, (size_t)net->VH * net->VC * 64); TAKE(net->v_b1, net->VH);
    TAKE(net->v_w2, (size_t)3 * net->VH); TAKE(net->v_b2, 3);
#undef TAKE
    return 0;
}

static double cap6(double z) { return z < 0.0 ? 0.0 : (z > 6.0 ? 6.0 : z); }

/* t[c][sq] = s[c] * t[c][sq] + b[c] */
static void scale_bias(double *t, const float *s, const float *b, int c) {
    for (int i = 0; i < c; ++i)
        for (int q = 0; q < 64; ++q) t[i * 64 + q] = (double)s[i] * t[i * 64 + q] + (double)b[i];
}

/* out[o][sq] = sum_c W[o][c] * in[c][sq] (+ bias[o]) */
static void pointwise(const float *W, const float *bias, const double *in, int cin, int cout, double *out) {
    for (int o = 0; o < cout; ++o)
        for (int q = 0; q < 64; ++q) {
            double acc = bias ? (double)bias[o] : 0.0;
            for (int c = 0; c < cin; ++c) acc += (double)W[(size_t)o * cin + c] * in[c * 64 + q];
            out[o * 64 + q] = acc;
        }
}

/* the action list: (origin, destination, piece) of every index, built once from the index map */
static int16_t act_from[P_ACTIONS], act_to[P_ACTIONS], act_piece[P_ACTIONS];
static int act_ready = 0;
static int build_actions(void) {
    for (int i = 0; i < P_ACTIONS; ++i) act_from[i] = -1;
    for (int f = 0; f < 64; ++f)
        for (int t = 0; t < 64; ++t) {
            int i = orc_policy_index(2, 0, f, t, 0, 0);
            if (i >= 0) { act_from[i] = (int16_t)f; act_to[i] = (int16_t)t; act_piece[i] = -1; }
            for (int promo = 1; promo <= 4; ++promo) {
                int j = orc_policy_index(2, 0, f, t, promo, 0);
                if (j >= 0) { act_from[j] = (int16_t)f; act_to[j] = (int16_t)t; act_piece[j] = (int16_t)(4 - promo); }
            }
        }
    for (int i = 0; i < P_ACTIONS; ++i) if (act_from[i] < 0) return -1;
    act_ready = 1;
    return 0;
}

static void forward_one(const PNet *net, const double *planes, const uint64_t *mask, double *policy, double *value,
                        double *raw_logits, double *tower_out) {
    const int L = net->L, C = net->C, K = net->K, P = C / 4, R = C - P;
    double *h = malloc(sizeof(double) * (size_t)C * 64), *t = malloc(sizeof(double) * (size_t)C * 64);
    double *y = malloc(sizeof(double) * (size_t)C * 64);
    orc_conv3x3(net->in_w, planes, P_PLANES, C, h);
    scale_bias(h, net->in_s, net->in_b, C);
    for (int i = 0; i < C * 64; ++i) h[i] = cap6(h[i]);
    for (int b = 0; b < L; ++b) {
        orc_conv3x3(net->w1[b], h, C, C, t);
        scale_bias(t, net->s1[b], net->b1[b], C);
        int cin2 = C;
        if (pooled_block(b)) {
            double *g_in = malloc(sizeof(double) * 2 * (size_t)P);
            for (int c = 0; c < P; ++c) {
                double sum = 0.0, mx = 0.0;
                for (int q = 0; q < 64; ++q) {
                    double a = cap6(t[(R + c) * 64 + q]);
                    sum += a;
                    if (q == 0 || a > mx) mx = a;
                }
                g_in[c] = sum / 64.0;
                g_in[P + c] = mx;
            }
            for (int r = 0; r < R; ++r) {
                double g = 0.0;
                for (int j = 0; j < 2 * P; ++j) g += (double)net->gw[b][(size_t)r * 2 * P + j] * g_in[j];
                for (int q = 0; q < 64; ++q) t[r * 64 + q] += g;
            }
            free(g_in);
            cin2 = R;
        }
        for (int i = 0; i < cin2 * 64; ++i) t[i] = cap6(t[i]);
        orc_conv3x3(net->w2[b], t, cin2, C, y);
        scale_bias(y, net->s2[b], net->b2[b], C);
        for (int i = 0; i < C * 64; ++i) h[i] = cap6(h[i] + y[i]);
    }
    if (tower_out) memcpy(tower_out, h, sizeof(double) * (size_t)C * 64);

    /* policy: tokens, queries, keys, scores, gather */
    double *u = malloc(sizeof(double) * (size_t)K * 64), *q = malloc(sizeof(double) * (size_t)K * 64);
    double *k = malloc(sizeof(double) * (size_t)K * 64), *o = malloc(sizeof(double) * 4 * 64);
    pointwise(net->t_w, net->t_b, h, C, K, u);
    pointwise(net->q_w, net->q_b, u, K, K, q);
    pointwise(net->k_w, net->k_b, u, K, K, k);
    pointwise(net->o_w, net->o_b, u, K, 4, o);
    double *logits = malloc(sizeof(double) * P_ACTIONS);
    const double inv = 1.0 / sqrt((double)K);
    for (int i = 0; i < P_ACTIONS; ++i) {
        const int f = act_from[i], to = act_to[i];
        double s = 0.0;
        for (int d = 0; d < K; ++d) s += q[d * 64 + f] * k[d * 64 + to];
        s *= inv;
        if (act_piece[i] >= 0) s += o[act_piece[i] * 64 + f];
        logits[i] = s;
    }
    if (raw_logits) memcpy(raw_logits, logits, sizeof(double) * P_ACTIONS);
    orc_masked_softmax(logits, mask, P_ACTIONS, policy);

    /* value */
    const int VC = net->VC, VH = net->VH;
    double *v = malloc(sizeof(double) * (size_t)VC * 64), *hid = malloc(sizeof(double) * (size_t)VH);
    pointwise(net->v_cw, NULL, h, C, VC, v);
    scale_bias(v, net->v_cs, net->v_cb, VC);
    for (int i = 0; i < VC * 64; ++i) if (v[i] < 0.0) v[i] = 0.0;
    for (int j = 0; j < VH; ++j) {
        double acc = (double)net->v_b1[j];
        for (int i = 0; i < VC * 64; ++i) acc += (double)net->v_w1[(size_t)j * VC * 64 + i] * v[i];
        hid[j] = acc < 0.0 ? 0.0 : acc;
    }
    double z[3], m = -INFINITY, sum = 0.0;
    for (int c = 0; c < 3; ++c) {
        double acc = (double)net->v_b2[c];
        for (int j = 0; j < VH; ++j) acc += (double)net->v_w2[(size_t)c * VH + j] * hid[j];
        z[c] = acc;
        if (acc > m) m = acc;
    }
    for (int c = 0; c < 3; ++c) { z[c] = exp(z[c] - m); sum += z[c]; }
    for (int c = 0; c < 3; ++c) value[c] = z[c] / sum;
    free(h); free(t); free(y); free(u); free(q); free(k); free(o); free(logits); free(v); free(hid);
}

/* planes [n][52][64] doubles, masks [n][30] words, policy [n][1880], value [n][3]; raw_logits
 * (optional) [n][1880], tower_out (optional) [n][C][64].  Returns 0, -1 on a malformed blob. */
int orc_pnet_forward(const uint8_t *blob, size_t nbytes, const double *planes, const uint64_t *masks, int n,
                     double *policy, double *value, double *raw_logits, double *tower_out) {
    PNet net;
    if (parse(blob, nbytes, &net) != 0) return -1;
    if (!act_ready && build_actions() != 0) { free(net.w1); return -1; }
#pragma omp parallel for schedule(dynamic, 1)
    for (int i = 0; i < n; ++i)
        forward_one(&net, planes + (size_t)i * P_PLANES * 64, masks + (size_t)i * 30, policy + (size_t)i * P_ACTIONS,
                    value + (size_t)i * 3, raw_logits ? raw_logits + (size_t)i * P_ACTIONS : NULL,
                    tower_out ? tower_out + (size_t)i * net.C * 64 : NULL);
    free(net.w1);
    return 0;
}
