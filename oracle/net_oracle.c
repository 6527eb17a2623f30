/*
 * ORACLE (test infrastructure, not the product): the policy/value network and the
 * legal-move-masked softmax in double precision, straight from their definitions.
 *
 * Shares nothing with the CUDA library.  Reads the float32 master weights of the
 * weight blob and evaluates everything in fp64:
 *  - 3x3 convolution = direct summation with zero padding,
 *        out[co][y][x] = sum_ci sum_{dy,dx in -1..1} W[co][ci][dy+1][dx+1] * in[ci][y+dy][x+dx];
 *  - residual block in the conventional order convolution, normalisation, activation,
 *    convolution, normalisation, residual addition, activation (Sec. 4.3.6), with the
 *    batch-norm folded into a per-channel scale and bias on a deployment copy (Sec. 4.3.6,
 *    App. D.3) and a plain ReLU as the activation (the workload definitions' block);
 *  - heads: a 1x1 projection, then either per-square move planes or a flattened
 *    fully-connected layer (Sec. 4.3.1); value = 1x1 conv, norm, ReLU, flatten, hidden
 *    layer, then three logits with a softmax giving win/draw/loss for the player to
 *    move, or one tanh scalar (Sec. 4.3.4, App. D.1);
 *  - illegal actions are masked before the softmax over the legal moves (App. D.1):
 *    p_i = exp(l_i - max_legal) / sum_legal exp(l_j - max_legal), exactly 0 elsewhere.
 * Flattening is channel-major (index = channel*64 + square).
 *
 * Pins (tests, CPU only): convolution against a brute-force im2col matrix product and
 * against a library float64 convolution, closed forms (identity kernel, all-ones kernel
 * giving 9/6/4 neighbours), whole network against a float64 library composition,
 * softmax invariants (sums to 1, zeros off the mask, uniform logits, shift invariance).
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int in_planes, blocks, channels, policy_head, value_head;
    const float *in_w, *in_s, *in_b;
    const float **w1, **s1, **b1, **w2, **s2, **b2;
    const float *p_w, *p_bias;                              /* 73-plane head */
    const float *p_cw, *p_cs, *p_cb, *p_fw, *p_fb;          /* flat head */
    const float *v_cw, *v_cs, *v_cb, *v_w1, *v_b1, *v_w2, *v_b2;
} Net;

enum { HEAD_CH = 32, V_HIDDEN = 128, FLAT_MOVES = 1858 };

static int parse_blob(const uint8_t *blob, size_t nbytes, Net *net) {
    if (nbytes < 64 || memcmp(blob, "AZNETv1", 8) != 0) return -1;
    uint32_t h[7];
    memcpy(h, blob + 8, sizeof h);
    if (h[0] != 1) return -1;
    net->in_planes = (int)h[1]; net->blocks = (int)h[2]; net->channels = (int)h[3];
    net->policy_head = (int)h[4]; net->value_head = (int)h[5];
    int C = net->channels, P = net->in_planes, L = net->blocks;
    const float *p = (const float *)(blob + 64);
    const float *end = (const float *)(blob + (nbytes & ~(size_t)3));
#define TAKE(dst, count) do { dst = p; p += (size_t)(count); if (p > end) return -1; } while (0)
    TAKE(net->in_w, (size_t)C * P * 9); TAKE(net->in_s, C); TAKE(net->in_b, C);
    net->w1 = malloc(sizeof(float *) * 6 * (size_t)(L > 0 ? L : 1));
    net->s1 = net->w1 + L; net->b1 = net->s1 + L; net->w2 = net->b1 + L; net->s2 = net->w2 + L; net->b2 = net->s2 + L;
    for (int b = 0; b < L; ++b) {
        TAKE(net->w1[b], (size_t)C * C * 9); TAKE(net->s1[b], C); TAKE(net->b1[b], C);
        TAKE(net->w2[b], (size_t)C * C * 9); TAKE(net->s2[b], C); TAKE(net->b2[b], C);
    }
    if (net->policy_head == 0) { TAKE(net->p_w, (size_t)73 * C); TAKE(net->p_bias, 73); }
    else {
        TAKE(net->p_cw, (size_t)HEAD_CH * C); TAKE(net->p_cs, HEAD_CH); TAKE(net->p_cb, HEAD_CH);
        TAKE(net->p_fw, (size_t)FLAT_MOVES * HEAD_CH * 64); TAKE(net->p_fb, FLAT_MOVES);
    }
    TAKE(net->v_cw, (size_t)HEAD_CH * C); TAKE(net->v_cs, HEAD_CH); TAKE(net->v_cb, HEAD_CH);
    TAKE(net->v_w1, (size_t)V_HIDDEN * HEAD_CH * 64); TAKE(net->v_b1, V_HIDDEN);
    int V = net->value_head ? 3 : 1;
    TAKE(net->v_w2, (size_t)V * V_HIDDEN); TAKE(net->v_b2, V);
#undef TAKE
    return 0;
}

/* out[co][y][x] = sum over ci and the 3x3 window of W[co][ci][ky][kx] * in[ci][y+ky-1][x+kx-1],
 * terms outside the 8x8 board contributing zero.  The input is first copied into a 10x10 frame
 * with a zero border so that the sum can be written without case distinctions. */
static void conv3x3(const float *W, const double *in, int cin, int cout, double *out) {
    double *frame = calloc((size_t)cin * 100, sizeof(double));
    for (int ci = 0; ci < cin; ++ci)
        for (int y = 0; y < 8; ++y)
            for (int x = 0; x < 8; ++x)
                frame[ci * 100 + (y + 1) * 10 + (x + 1)] = in[ci * 64 + y * 8 + x];
    for (int co = 0; co < cout; ++co) {
        double acc[8][8];
        memset(acc, 0, sizeof acc);
        for (int ci = 0; ci < cin; ++ci) {
            const float *w = W + ((size_t)co * cin + ci) * 9;
            const double *f = frame + ci * 100;
            for (int ky = 0; ky < 3; ++ky)
                for (int kx = 0; kx < 3; ++kx) {
                    double wv = (double)w[ky * 3 + kx];
                    for (int y = 0; y < 8; ++y)
                        for (int x = 0; x < 8; ++x)
                            acc[y][x] += wv * f[(y + ky) * 10 + (x + kx)];
                }
        }
        memcpy(out + (size_t)co * 64, acc, sizeof acc);
    }
    free(frame);
}

/* Standalone entry for the convolution pins: W[cout][cin][3][3] float32, in[cin][64], out[cout][64]. */
void orc_conv3x3(const float *W, const double *in, int cin, int cout, double *out) {
    conv3x3(W, in, cin, cout, out);
}

static void scale_bias(double *t, const float *s, const float *b, int c) {
    for (int co = 0; co < c; ++co)
        for (int i = 0; i < 64; ++i) t[co * 64 + i] = (double)s[co] * t[co * 64 + i] + (double)b[co];
}
static void relu(double *t, size_t n) { for (size_t i = 0; i < n; ++i) if (t[i] < 0.0) t[i] = 0.0; }

/* 1x1 convolution: out[co][sq] = sum_ci W[co][ci] * in[ci][sq] */
static void conv1x1(const float *W, const double *in, int cin, int cout, double *out) {
    for (int co = 0; co < cout; ++co)
        for (int i = 0; i < 64; ++i) {
            double a = 0.0;
            for (int ci = 0; ci < cin; ++ci) a += (double)W[(size_t)co * cin + ci] * in[ci * 64 + i];
            out[co * 64 + i] = a;
        }
}
static void dense(const float *W, const float *b, const double *in, int nin, int nout, double *out) {
    for (int o = 0; o < nout; ++o) {
        double a = (double)b[o];
        for (int i = 0; i < nin; ++i) a += (double)W[(size_t)o * nin + i] * in[i];
        out[o] = a;
    }
}

static void masked_softmax(const double *logits, const uint64_t *mask, int n, double *probs) {
    double mx = 0.0; int any = 0;
    for (int i = 0; i < n; ++i)
        if ((mask[i >> 6] >> (i & 63)) & 1ULL) { if (!any || logits[i] > mx) mx = logits[i]; any = 1; }
    double sum = 0.0;
    for (int i = 0; i < n; ++i) {
        probs[i] = 0.0;
        if ((mask[i >> 6] >> (i & 63)) & 1ULL) { probs[i] = exp(logits[i] - mx); sum += probs[i]; }
    }
    if (any) for (int i = 0; i < n; ++i) probs[i] /= sum;
}

/* Standalone entry for the softmax pins. */
void orc_masked_softmax(const double *logits, const uint64_t *mask, int n, double *probs) {
    masked_softmax(logits, mask, n, probs);
}

static void forward_one(const Net *net, const double *planes, const uint64_t *mask,
                        double *policy, double *value, double *raw_logits, double *raw_value,
                        double *tower_out) {
    int C = net->channels;
    size_t act = (size_t)C * 64;
    double *h = malloc(sizeof(double) * act), *t = malloc(sizeof(double) * act), *u = malloc(sizeof(double) * act);
    conv3x3(net->in_w, planes, net->in_planes, C, h);
    scale_bias(h, net->in_s, net->in_b, C); relu(h, act);
    for (int b = 0; b < net->blocks; ++b) {
        conv3x3(net->w1[b], h, C, C, t);
        scale_bias(t, net->s1[b], net->b1[b], C); relu(t, act);
        conv3x3(net->w2[b], t, C, C, u);
        scale_bias(u, net->s2[b], net->b2[b], C);
        for (size_t i = 0; i < act; ++i) h[i] += u[i];
        relu(h, act);
    }
    if (tower_out) memcpy(tower_out, h, sizeof(double) * act);

    int npol = net->policy_head == 0 ? 73 * 64 : FLAT_MOVES;
    double *logits = malloc(sizeof(double) * (size_t)npol);
    if (net->policy_head == 0) {
        conv1x1(net->p_w, h, C, 73, logits);
        for (int p = 0; p < 73; ++p) for (int i = 0; i < 64; ++i) logits[p * 64 + i] += (double)net->p_bias[p];
    } else {
        double pc[HEAD_CH * 64];
        conv1x1(net->p_cw, h, C, HEAD_CH, pc);
        scale_bias(pc, net->p_cs, net->p_cb, HEAD_CH); relu(pc, HEAD_CH * 64);
        dense(net->p_fw, net->p_fb, pc, HEAD_CH * 64, FLAT_MOVES, logits);
    }
    if (raw_logits) memcpy(raw_logits, logits, sizeof(double) * (size_t)npol);
    masked_softmax(logits, mask, npol, policy);

    double vc[HEAD_CH * 64], hid[V_HIDDEN], z[3];
    conv1x1(net->v_cw, h, C, HEAD_CH, vc);
    scale_bias(vc, net->v_cs, net->v_cb, HEAD_CH); relu(vc, HEAD_CH * 64);
    dense(net->v_w1, net->v_b1, vc, HEAD_CH * 64, V_HIDDEN, hid);
    relu(hid, V_HIDDEN);
    int V = net->value_head ? 3 : 1;
    dense(net->v_w2, net->v_b2, hid, V_HIDDEN, V, z);
    if (raw_value) memcpy(raw_value, z, sizeof(double) * (size_t)V);
    if (V == 1) value[0] = tanh(z[0]);
    else {
        double mx = z[0] > z[1] ? z[0] : z[1]; if (z[2] > mx) mx = z[2];
        double e0 = exp(z[0] - mx), e1 = exp(z[1] - mx), e2 = exp(z[2] - mx), s = e0 + e1 + e2;
        value[0] = e0 / s; value[1] = e1 / s; value[2] = e2 / s;   /* win, draw, loss */
    }
    free(logits); free(h); free(t); free(u);
}

/*
 * planes [n][in_planes][64] doubles; masks [n][73 or 30] words; policy [n][4672 or 1858];
 * value [n][1 or 3].  Optional outputs (may be NULL): raw_logits like policy, raw_value like
 * value (before tanh / softmax), tower_out [n][C][64] (the tower's final activations).
 * Positions are independent and are spread over the host's threads.  Returns 0 or -1 (bad blob).
 */
int orc_forward(const uint8_t *blob, size_t nbytes, const double *planes, const uint64_t *masks,
                int n, double *policy, double *value, double *raw_logits, double *raw_value,
                double *tower_out) {
    Net net; memset(&net, 0, sizeof net);
    if (parse_blob(blob, nbytes, &net) != 0) { free((void *)net.w1); return -1; }
    int npol = net.policy_head == 0 ? 73 * 64 : FLAT_MOVES;
    int words = net.policy_head == 0 ? 73 : 30;
    int V = net.value_head ? 3 : 1;
    size_t pin = (size_t)net.in_planes * 64, act = (size_t)net.channels * 64;
#pragma omp parallel for schedule(dynamic, 1)
    for (int i = 0; i < n; ++i)
        forward_one(&net, planes + (size_t)i * pin, masks + (size_t)i * words,
                    policy + (size_t)i * npol, value + (size_t)i * V,
                    raw_logits ? raw_logits + (size_t)i * npol : NULL,
                    raw_value ? raw_value + (size_t)i * V : NULL,
                    tower_out ? tower_out + (size_t)i * act : NULL);
    free((void *)net.w1);
    return 0;
}

int orc_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
