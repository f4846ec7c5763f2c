/*
 * ppo_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, CPU-only restatement of one PPO learner step over a rollout
 * buffer D (Algorithm 2: D <- D U {(obs, actions, rew, done)}; TrainPPO(pi, D)).
 * It exists so that the CUDA library can be checked against something that can
 * be read by eye.  It shares no code, header, table or constant generator with
 * the CUDA path, and nothing in the product may call it.
 *
 * Arithmetic is fp64 throughout.  The only places where a narrower precision is
 * part of the definition are: the operands of every layer's contraction are bf16
 * values (weight matrices are rounded to bf16, round to nearest even, and with
 * act_bf16 != 0 every layer's output is rounded to bf16 before the next layer
 * reads it), while sums are kept in fp64; depth pixels arrive as fp16 values
 * (exactly representable in fp64); the outputs of Adam are rounded to fp32.
 * Rounding the activations matters for more than accuracy: the ReLU gate
 * (output > 0) is a discrete decision, and it has to be taken on the same values
 * on both sides of a comparison.  The backward pass treats every rounding as the
 * identity (straight through) and rounds nothing itself.
 *
 * Every function states the passage it follows.  The paper itself gives
 * TrainPPO only by name (Algorithm 2; Section III-C: "PPO", "CNN ... ReLU");
 * the formulas are the textbook definitions of GAE(gamma, lambda), PPO-clip,
 * the diagonal Gaussian policy and Adam that it cites.
 *
 * Pinned by tests/test_oracle_*.py (worked 2-env x 3-step example, closed
 * forms, finite differences, brute force permutation checks, textbook special
 * cases).  No function here is "parity unpinned".
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC (see oracle/build.py).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_MAX_CONV 8
#define ORC_MAX_FC 4

/* Network shape.  Section III-C: a CNN with ReLU on the depth image, combined
 * with proprioception, then fully connected layers.  Every conv has stride 2
 * and zero padding k/2; widths come from the workload description. */
typedef struct {
    int32_t H, W;                 /* depth image */
    int32_t n_conv;
    int32_t conv_c[ORC_MAX_CONV]; /* output channels */
    int32_t conv_k[ORC_MAX_CONV]; /* square kernel size (odd) */
    int32_t n_fc;
    int32_t fc[ORC_MAX_FC];       /* hidden widths */
    int32_t P, A;                 /* proprio width, action width */
    /* The depth CNN as Section III-C words it ("layer normalization, and ReLU", "a fully connected layer which
     * outputs a 32 dimensional embedding"); both 0 for the networks the workloads describe.
     *   norm != 0 : every conv output is layer-normalised over its channels at each pixel (learned scale gamma and
     *               shift beta per channel, variance over the channels, eps 1e-5) before the ReLU;
     *   embed > 0 : the last conv output is flattened (pixel-major, channel innermost) and mapped by a fully
     *               connected layer with ReLU to `embed` values, which take the place of the pooled vector. */
    int32_t norm, embed;
    /* The recurrent trunk of Section III-C ("fed into two LSTM layers with 1024 units, the output of which is fed
     * into a 3 layer fully-connected network"): n_lstm stacked LSTM layers of lstm_h units between h_0 (the depth
     * feature joined with proprioception) and the fully connected layers; 0 layers for the feed-forward networks. */
    int32_t n_lstm, lstm_h;
} orc_model;

#define ORC_MAX_LSTM 4
#define ORC_MAX_TENSORS (4 * ORC_MAX_CONV + 2 * ORC_MAX_FC + 3 * ORC_MAX_LSTM + 5)
#define ORC_LN_EPS 1e-5

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---------------------------------------------------------------- buffer -- */

/* Section III-B: the buffer holds, per env and per step of the horizon, one
 * depth frame; its size is N*T*H*W*elem bytes (the text's example: 512 envs,
 * 320x240, 16 steps, fp32 = "2.5GB"). */
uint64_t orc_depth_bytes(uint64_t N, uint64_t T, uint64_t H, uint64_t W, uint64_t elem) {
    return N * T * H * W * elem;
}

/* ------------------------------------------------------------------- GAE -- */

/* GAE(gamma, lambda) for TrainPPO (Algorithm 2).  Time-major arrays [T][N].
 * done[t][n] was returned by the same Env.Step as reward[t][n], so it cuts
 * the bootstrap from step t to step t+1.
 *   delta_t = r_t + gamma * V_{t+1} * (1 - d_t) - V_t
 *   A_t     = delta_t + gamma * lambda * (1 - d_t) * A_{t+1}
 *   R_t     = A_t + V_t,      V_T = last_value, A_T = 0 */
void orc_gae(int T, int N, const float *reward, const float *value, const uint8_t *done,
             const float *last_value, double gamma, double lambda, double *adv, double *ret) {
    for (int n = 0; n < N; ++n) {
        double v_next = (double)last_value[n];
        double a_next = 0.0;
        for (int t = T - 1; t >= 0; --t) {
            size_t i = (size_t)t * N + n;
            double not_done = done[i] ? 0.0 : 1.0;
            double v = (double)value[i];
            double delta = (double)reward[i] + gamma * v_next * not_done - v;
            double a = delta + gamma * lambda * not_done * a_next;
            adv[i] = a;
            ret[i] = a + v;
            v_next = v;
            a_next = a;
        }
    }
}

/* Advantage normalisation over the whole buffer, once, before minibatching:
 * mu = mean, sigma = unbiased (M-1) standard deviation, a <- (a-mu)/(sigma+1e-8). */
void orc_adv_normalize(size_t M, double *adv, double *mean_out, double *std_out) {
    double s = 0.0;
    for (size_t i = 0; i < M; ++i) s += adv[i];
    double mu = s / (double)M;
    double q = 0.0;
    for (size_t i = 0; i < M; ++i) q += (adv[i] - mu) * (adv[i] - mu);
    double sigma = (M > 1) ? sqrt(q / (double)(M - 1)) : 0.0;
    for (size_t i = 0; i < M; ++i) adv[i] = (adv[i] - mu) / (sigma + 1e-8);
    if (mean_out) *mean_out = mu;
    if (std_out) *std_out = sigma;
}

/* ----------------------------------------------------------- permutation -- */

/* Seeded bijection on [0, M): a 6-round balanced Feistel network on 2h bits
 * (2^(2h) >= M) with cycle walking.  All arithmetic is uint32 with wrap-around. */
uint32_t orc_mix32(uint32_t x) {
    x ^= x >> 16;
    x *= 0x9E3779B9u;
    x ^= x >> 15;
    x *= 0x6A09E667u;
    x ^= x >> 16;
    return x;
}

void orc_perm_keys(uint64_t seed, uint32_t epoch, uint32_t key[6]) {
    uint32_t lo = (uint32_t)(seed & 0xFFFFFFFFu), hi = (uint32_t)(seed >> 32);
    for (uint32_t j = 0; j < 6; ++j) {
        uint32_t a = orc_mix32(hi + 0x9E3779B9u * (j + 1));
        uint32_t b = orc_mix32(epoch + 0xBB67AE85u * (j + 1));
        key[j] = orc_mix32(lo ^ a ^ b);
    }
}

int orc_perm_half_bits(uint32_t M) {
    int bits = 0; /* smallest bits with 2^bits >= M */
    while (((uint64_t)1 << bits) < (uint64_t)M) ++bits;
    int h = (bits + 1) / 2;
    return h < 1 ? 1 : h;
}

uint32_t orc_perm(uint64_t seed, uint32_t epoch, uint32_t M, uint32_t i) {
    uint32_t key[6];
    orc_perm_keys(seed, epoch, key);
    int h = orc_perm_half_bits(M);
    uint32_t mask = ((uint32_t)1 << h) - 1u;
    uint32_t x = i;
    do {
        uint32_t L = x >> h, R = x & mask;
        for (int j = 0; j < 6; ++j) {
            uint32_t newR = L ^ (orc_mix32(R ^ key[j]) & mask);
            L = R;
            R = newR;
        }
        x = (L << h) | R;
    } while (x >= M);
    return x;
}

/* Minibatch k of K (B = M/K rows): row j holds sample orc_perm(k*B + j). */
void orc_perm_fill(uint64_t seed, uint32_t epoch, uint32_t M, uint32_t start, uint32_t count, uint32_t *out) {
    for (uint32_t j = 0; j < count; ++j) out[j] = orc_perm(seed, epoch, M, start + j);
}

/* ---------------------------------------------------------------- layout -- */

double orc_round_bf16(double x) {
    float f = (float)x;
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7F800000u) == 0x7F800000u) return (double)f; /* inf / nan unchanged */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb; /* round to nearest, ties to even */
    u &= 0xFFFF0000u;
    memcpy(&f, &u, 4);
    return (double)f;
}

static int conv_out(int in, int k) { return (in + 2 * (k / 2) - k) / 2 + 1; }

void orc_conv_shapes(const orc_model *m, int32_t *Ho, int32_t *Wo) {
    int h = m->H, w = m->W;
    for (int l = 0; l < m->n_conv; ++l) {
        h = conv_out(h, m->conv_k[l]);
        w = conv_out(w, m->conv_k[l]);
        Ho[l] = h;
        Wo[l] = w;
    }
}

/* Parameter vector layout (an interface shared with the caller, restated here):
 * tensors in the order conv W_l [Cout][k][k][Cin], conv b_l, ..., fc W [out][in],
 * fc b, ..., head W [A+1][hid] (rows 0..A-1 mean, row A value), head b [A+1],
 * log-sigma [A]; each tensor starts at a multiple of 64 elements.  With norm != 0 every conv b_l is followed by
 * gamma_l [Cout] and beta_l [Cout]; with embed > 0 the conv tensors are followed by embed W [E][Ho*Wo*C_L] and
 * embed b [E], and the first fc layer reads E + P values.
 * offsets/sizes must have room for ORC_MAX_TENSORS entries.
 * Returns the total length of the vector; *n_tensors gets the tensor count. */
int64_t orc_param_layout(const orc_model *m, int64_t *offsets, int64_t *sizes, int32_t *is_matrix, int32_t *n_tensors) {
    int64_t off = 0;
    int n = 0;
    int cin = 1;
#define PUSH(sz, mat)                        \
    do {                                     \
        offsets[n] = off;                    \
        sizes[n] = (sz);                     \
        is_matrix[n] = (mat);                \
        off += ((int64_t)(sz) + 63) / 64 * 64; \
        ++n;                                 \
    } while (0)
    for (int l = 0; l < m->n_conv; ++l) {
        PUSH((int64_t)m->conv_c[l] * m->conv_k[l] * m->conv_k[l] * cin, 1);
        PUSH(m->conv_c[l], 0);
        if (m->norm) {
            PUSH(m->conv_c[l], 0);
            PUSH(m->conv_c[l], 0);
        }
        cin = m->conv_c[l];
    }
    int in = cin + m->P;
    if (m->embed > 0) {
        int32_t Ho[ORC_MAX_CONV], Wo[ORC_MAX_CONV];
        orc_conv_shapes(m, Ho, Wo);
        PUSH((int64_t)m->embed * Ho[m->n_conv - 1] * Wo[m->n_conv - 1] * cin, 1);
        PUSH(m->embed, 0);
        in = m->embed + m->P;
    }
    /* LSTM layer: W_x [4H][in], W_h [4H][H] (gate blocks in the order input, forget, cell, output), b [4H] */
    for (int l = 0; l < m->n_lstm; ++l) {
        PUSH((int64_t)4 * m->lstm_h * in, 1);
        PUSH((int64_t)4 * m->lstm_h * m->lstm_h, 1);
        PUSH((int64_t)4 * m->lstm_h, 0);
        in = m->lstm_h;
    }
    for (int l = 0; l < m->n_fc; ++l) {
        PUSH((int64_t)m->fc[l] * in, 1);
        PUSH(m->fc[l], 0);
        in = m->fc[l];
    }
    PUSH((int64_t)(m->A + 1) * in, 1);
    PUSH(m->A + 1, 0);
    PUSH(m->A, 0);
#undef PUSH
    *n_tensors = n;
    return off;
}

/* Weight matrices are used as bf16-rounded copies of the fp32 master; biases
 * and log-sigma are used as they are. */
void orc_round_weights(const orc_model *m, const double *theta, double *theta_used) {
    int64_t offs[ORC_MAX_TENSORS], szs[ORC_MAX_TENSORS];
    int32_t mat[ORC_MAX_TENSORS], n;
    int64_t total = orc_param_layout(m, offs, szs, mat, &n);
    for (int64_t i = 0; i < total; ++i) theta_used[i] = theta[i];
    for (int t = 0; t < n; ++t)
        if (mat[t])
            for (int64_t i = 0; i < szs[t]; ++i) theta_used[offs[t] + i] = orc_round_bf16(theta[offs[t] + i]);
}

/* Per-sample activation record: [image H*W | a_1 | ... | a_L | h_0 = pooled (or embedding) ++ proprio | h_1 | ... |
 * h_F], followed with norm != 0 by what the backward pass of the normalisation needs, layer by layer: the
 * normalised values xhat_l [Ho*Wo*C] and the reciprocal standard deviations rstd_l [Ho*Wo]. */
static int64_t act_main_len(const orc_model *m) {
    int32_t Ho[ORC_MAX_CONV], Wo[ORC_MAX_CONV];
    orc_conv_shapes(m, Ho, Wo);
    int64_t s = (int64_t)m->H * m->W;
    for (int l = 0; l < m->n_conv; ++l) s += (int64_t)Ho[l] * Wo[l] * m->conv_c[l];
    s += (m->embed > 0 ? m->embed : m->conv_c[m->n_conv - 1]) + m->P;
    for (int l = 0; l < m->n_fc; ++l) s += m->fc[l];
    return s;
}

int64_t orc_act_stride(const orc_model *m) {
    int32_t Ho[ORC_MAX_CONV], Wo[ORC_MAX_CONV];
    orc_conv_shapes(m, Ho, Wo);
    int64_t s = act_main_len(m);
    if (m->norm)
        for (int l = 0; l < m->n_conv; ++l) s += (int64_t)Ho[l] * Wo[l] * (m->conv_c[l] + 1);
    return s;
}

/* --------------------------------------------------------------- encoder -- */

/* Forward of one sample (Section III-C: CNN + ReLU on depth, concatenated with
 * proprioception, fully connected layers; heads give the Gaussian mean and the value).
 *   conv: y[oh][ow][co] = ReLU(b[co] + sum_{kh,kw,ci} W[co][kh][kw][ci] * x[2*oh+kh-p][2*ow+kw-p][ci])
 *         (cross-correlation, zero outside the image, p = k/2)
 *   g = mean of the last conv output over its pixels; h_0 = [g, proprio]
 *   h_l = ReLU(W_l h_{l-1} + b_l);  out = W_head h_F + b_head; mu = out[0..A), V = out[A].
 * With act_bf16 != 0 every conv output, h_0 and every hidden h_l is rounded to bf16 where it
 * is stored (the next layer's operand); the head output is not rounded. */
/* phase 0: the whole feed-forward network.  With a recurrent trunk the sample is processed in two phases around
 * it: phase 1 stops after h_0; phase 2 runs the fully connected layers and the head on `trunk_out` (the top LSTM
 * layer's output for this sample, lstm_h values) and stores h_1.. behind h_0 as usual. */
static void fwd_one(const orc_model *m, const double *th, const int64_t *offs, const double *depth,
                    const double *proprio, double *act, double *mu, double *V, int act_bf16, int phase,
                    const double *trunk_out) {
    int32_t Ho[ORC_MAX_CONV], Wo[ORC_MAX_CONV];
    orc_conv_shapes(m, Ho, Wo);
    if (phase == 2) {
        int ti = 2 * m->n_conv + (m->norm ? 2 * m->n_conv : 0) + (m->embed > 0 ? 2 : 0) + 3 * m->n_lstm;
        int h0w = (m->embed > 0 ? m->embed : m->conv_c[m->n_conv - 1]) + m->P;
        double *y = act + act_main_len(m);
        for (int l = 0; l < m->n_fc; ++l) y -= m->fc[l]; /* h_1 sits right behind h_0 */
        (void)h0w;
        const double *h = trunk_out;
        int in = m->lstm_h;
        for (int l = 0; l < m->n_fc; ++l) {
            const double *Wt = th + offs[ti], *b = th + offs[ti + 1];
            ti += 2;
            for (int o = 0; o < m->fc[l]; ++o) {
                double acc = b[o];
                for (int i = 0; i < in; ++i) acc += Wt[(int64_t)o * in + i] * h[i];
                acc = acc > 0.0 ? acc : 0.0;
                y[o] = act_bf16 ? orc_round_bf16(acc) : acc;
            }
            h = y;
            in = m->fc[l];
            y += m->fc[l];
        }
        const double *Wh = th + offs[ti], *bh = th + offs[ti + 1];
        for (int o = 0; o <= m->A; ++o) {
            double acc = bh[o];
            for (int i = 0; i < in; ++i) acc += Wh[(int64_t)o * in + i] * h[i];
            if (o < m->A) mu[o] = acc; else *V = acc;
        }
        return;
    }
    double *x = act;
    double *extra = act + act_main_len(m); /* xhat_l, rstd_l of the normalised layers */
    for (int64_t i = 0; i < (int64_t)m->H * m->W; ++i) x[i] = depth[i];
    int hin = m->H, win = m->W, cin = 1;
    int ti = 0;
    for (int l = 0; l < m->n_conv; ++l) {
        int k = m->conv_k[l], p = k / 2, co_n = m->conv_c[l];
        const double *Wt = th + offs[ti], *b = th + offs[ti + 1];
        ti += 2;
        const double *gam = NULL, *bet = NULL;
        if (m->norm) {
            gam = th + offs[ti];
            bet = th + offs[ti + 1];
            ti += 2;
        }
        double *y = x + (int64_t)hin * win * cin;
        for (int oh = 0; oh < Ho[l]; ++oh)
            for (int ow = 0; ow < Wo[l]; ++ow) {
                int64_t px = (int64_t)oh * Wo[l] + ow;
                double *z = y + px * co_n; /* pre-activations of this pixel, then its outputs */
                for (int co = 0; co < co_n; ++co) {
                    double acc = b[co];
                    for (int kh = 0; kh < k; ++kh) {
                        int ih = 2 * oh + kh - p;
                        if (ih < 0 || ih >= hin) continue;
                        for (int kw = 0; kw < k; ++kw) {
                            int iw = 2 * ow + kw - p;
                            if (iw < 0 || iw >= win) continue;
                            const double *wp = Wt + (((int64_t)co * k + kh) * k + kw) * cin;
                            const double *xp = x + ((int64_t)ih * win + iw) * cin;
                            for (int ci = 0; ci < cin; ++ci) acc += wp[ci] * xp[ci];
                        }
                    }
                    z[co] = acc;
                }
                if (m->norm) {
                    /* layer normalisation over the channels of this pixel:
                     * mean = sum z / C, var = sum (z - mean)^2 / C, xhat = (z - mean) / sqrt(var + eps),
                     * z <- gamma * xhat + beta */
                    double mean = 0.0, var = 0.0;
                    for (int co = 0; co < co_n; ++co) mean += z[co];
                    mean /= (double)co_n;
                    for (int co = 0; co < co_n; ++co) var += (z[co] - mean) * (z[co] - mean);
                    var /= (double)co_n;
                    double rstd = 1.0 / sqrt(var + ORC_LN_EPS);
                    double *xh = extra + px * co_n;
                    extra[(int64_t)Ho[l] * Wo[l] * co_n + px] = rstd;
                    for (int co = 0; co < co_n; ++co) {
                        double v = (z[co] - mean) * rstd;
                        z[co] = gam[co] * v + bet[co];
                        xh[co] = act_bf16 ? orc_round_bf16(v) : v;
                    }
                }
                for (int co = 0; co < co_n; ++co) {
                    double acc = z[co] > 0.0 ? z[co] : 0.0;
                    z[co] = act_bf16 ? orc_round_bf16(acc) : acc;
                }
            }
        if (m->norm) extra += (int64_t)Ho[l] * Wo[l] * (co_n + 1);
        x = y;
        hin = Ho[l];
        win = Wo[l];
        cin = co_n;
    }
    /* global average pool (or, with embed > 0, flatten -> fully connected -> ReLU), then concatenate proprio */
    double *h = x + (int64_t)hin * win * cin;
    int feat = cin;
    if (m->embed > 0) {
        const double *We = th + offs[ti], *be = th + offs[ti + 1];
        ti += 2;
        int64_t flat = (int64_t)hin * win * cin;
        feat = m->embed;
        for (int e = 0; e < feat; ++e) {
            double acc = be[e];
            for (int64_t i = 0; i < flat; ++i) acc += We[(int64_t)e * flat + i] * x[i];
            acc = acc > 0.0 ? acc : 0.0;
            h[e] = act_bf16 ? orc_round_bf16(acc) : acc;
        }
    } else {
        for (int c = 0; c < cin; ++c) {
            double s = 0.0;
            for (int px = 0; px < hin * win; ++px) s += x[(int64_t)px * cin + c];
            h[c] = s / (double)(hin * win);
            if (act_bf16) h[c] = orc_round_bf16(h[c]);
        }
    }
    for (int j = 0; j < m->P; ++j) h[feat + j] = act_bf16 ? orc_round_bf16(proprio[j]) : proprio[j];
    if (phase == 1) return;
    int in = feat + m->P;
    for (int l = 0; l < m->n_fc; ++l) {
        const double *Wt = th + offs[ti], *b = th + offs[ti + 1];
        ti += 2;
        double *y = h + in;
        for (int o = 0; o < m->fc[l]; ++o) {
            double acc = b[o];
            for (int i = 0; i < in; ++i) acc += Wt[(int64_t)o * in + i] * h[i];
            acc = acc > 0.0 ? acc : 0.0;
            y[o] = act_bf16 ? orc_round_bf16(acc) : acc;
        }
        h = y;
        in = m->fc[l];
    }
    const double *Wh = th + offs[ti], *bh = th + offs[ti + 1];
    for (int o = 0; o <= m->A; ++o) {
        double acc = bh[o];
        for (int i = 0; i < in; ++i) acc += Wh[(int64_t)o * in + i] * h[i];
        if (o < m->A) mu[o] = acc; else *V = acc;
    }
}

/* Chain rule through fwd_one for one sample; adds this sample's gradient into g
 * (same layout as the parameter vector).  ReLU' = 1 where the stored output is
 * > 0 (equivalently the pre-activation is > 0), else 0.  The log-sigma slot of g
 * is not touched here (it has no path through the network). */
/* phase 0: the whole feed-forward network.  Around a recurrent trunk: phase 2 goes from the head down through the
 * fully connected layers, whose first input was `trunk_out`, and leaves dL/d(trunk_out) in d_trunk [lstm_h];
 * phase 1 starts from d_trunk = dL/dh_0 [width of h_0] and goes down through the pooling or embedding and the
 * convolutions. */
static void bwd_one(const orc_model *m, const double *th, const int64_t *offs, int n_tensors, const double *act,
                    const double *dmu, double dV, double *g, double *scratch, int phase, const double *trunk_out,
                    double *d_trunk) {
    int32_t Ho[ORC_MAX_CONV], Wo[ORC_MAX_CONV];
    orc_conv_shapes(m, Ho, Wo);
    /* locate activations */
    const double *a[ORC_MAX_CONV + 1];
    int hs[ORC_MAX_CONV + 1], ws[ORC_MAX_CONV + 1], cs[ORC_MAX_CONV + 1];
    a[0] = act; hs[0] = m->H; ws[0] = m->W; cs[0] = 1;
    for (int l = 0; l < m->n_conv; ++l) {
        a[l + 1] = a[l] + (int64_t)hs[l] * ws[l] * cs[l];
        hs[l + 1] = Ho[l]; ws[l + 1] = Wo[l]; cs[l + 1] = m->conv_c[l];
    }
    int L = m->n_conv, F = m->n_fc;
    const double *hv[ORC_MAX_FC + 1];
    int hn[ORC_MAX_FC + 1];
    hv[0] = a[L] + (int64_t)hs[L] * ws[L] * cs[L];
    hn[0] = (m->embed > 0 ? m->embed : cs[L]) + m->P;
    /* xhat_l and rstd_l of the normalised layers sit behind the main record */
    const double *xh[ORC_MAX_CONV + 1], *rs[ORC_MAX_CONV + 1];
    {
        const double *e = act + act_main_len(m);
        for (int l = 1; l <= L; ++l) {
            xh[l] = e;
            rs[l] = e + (int64_t)hs[l] * ws[l] * cs[l];
            e += (int64_t)hs[l] * ws[l] * (cs[l] + 1);
        }
    }
    for (int l = 0; l < F; ++l) { hv[l + 1] = hv[l] + hn[l]; hn[l + 1] = m->fc[l]; }
    const int h0w = hn[0];
    if (phase == 2) { /* the fully connected layers read the trunk's output, not h_0 */
        hv[0] = trunk_out;
        hn[0] = m->lstm_h;
    }

    /* scratch: two ping-pong gradient buffers large enough for any activation */
    int64_t big = (int64_t)m->H * m->W;
    for (int l = 1; l <= L; ++l) { int64_t s = (int64_t)hs[l] * ws[l] * cs[l]; if (s > big) big = s; }
    for (int l = 0; l <= F; ++l) if (hn[l] > big) big = hn[l];
    if (h0w > big) big = h0w;
    double *d_cur = scratch, *d_prev = scratch + big;

    /* head */
    int ti = n_tensors - 3; /* head W, head b, log-sigma */
    if (phase == 1) {
        for (int i = 0; i < h0w; ++i) d_cur[i] = d_trunk[i];
        ti -= 2 * F + 3 * m->n_lstm; /* past the fully connected and the LSTM tensors */
    }
    if (phase != 1) {
        const double *Wh = th + offs[ti];
        double *gW = g + offs[ti], *gb = g + offs[ti + 1];
        int in = hn[F];
        for (int i = 0; i < in; ++i) d_cur[i] = 0.0;
        for (int o = 0; o <= m->A; ++o) {
            double d = (o < m->A) ? dmu[o] : dV;
            gb[o] += d;
            for (int i = 0; i < in; ++i) {
                gW[(int64_t)o * in + i] += d * hv[F][i];
                d_cur[i] += Wh[(int64_t)o * in + i] * d;
            }
        }
    }
    /* hidden fc layers, last to first; d_cur holds dL/dh_l (post-ReLU) */
    for (int l = F; l >= 1 && phase != 1; --l) {
        ti -= 2;
        const double *Wt = th + offs[ti];
        double *gW = g + offs[ti], *gb = g + offs[ti + 1];
        int in = hn[l - 1], out = hn[l];
        for (int i = 0; i < in; ++i) d_prev[i] = 0.0;
        for (int o = 0; o < out; ++o) {
            double dz = hv[l][o] > 0.0 ? d_cur[o] : 0.0;
            gb[o] += dz;
            for (int i = 0; i < in; ++i) {
                gW[(int64_t)o * in + i] += dz * hv[l - 1][i];
                d_prev[i] += Wt[(int64_t)o * in + i] * dz;
            }
        }
        double *tmp = d_cur; d_cur = d_prev; d_prev = tmp;
    }
    if (phase == 2) {
        for (int i = 0; i < m->lstm_h; ++i) d_trunk[i] = d_cur[i];
        return;
    }
    /* un-pool: every pixel of the last conv output gets dg[c] / (Ho*Wo); the proprio part ends here.
     * With embed > 0: back through ReLU and the fully connected embedding into the flattened conv output. */
    if (m->embed > 0) {
        ti -= 2;
        const double *We = th + offs[ti];
        double *gW = g + offs[ti], *gb = g + offs[ti + 1];
        int64_t flat = (int64_t)hs[L] * ws[L] * cs[L];
        for (int64_t i = 0; i < flat; ++i) d_prev[i] = 0.0;
        for (int e = 0; e < m->embed; ++e) {
            double dz = hv[0][e] > 0.0 ? d_cur[e] : 0.0;
            gb[e] += dz;
            for (int64_t i = 0; i < flat; ++i) {
                gW[(int64_t)e * flat + i] += dz * a[L][i];
                d_prev[i] += We[(int64_t)e * flat + i] * dz;
            }
        }
        double *tmp = d_cur; d_cur = d_prev; d_prev = tmp;
    } else {
        int npx = hs[L] * ws[L], c_n = cs[L];
        for (int px = 0; px < npx; ++px)
            for (int c = 0; c < c_n; ++c) d_prev[(int64_t)px * c_n + c] = d_cur[c] / (double)npx;
        double *tmp = d_cur; d_cur = d_prev; d_prev = tmp;
    }
    /* conv layers, last to first; d_cur holds dL/da_l (post-ReLU) */
    for (int l = L; l >= 1; --l) {
        const double *gam = NULL;
        double *ggam = NULL, *gbet = NULL;
        if (m->norm) {
            ti -= 2;
            gam = th + offs[ti];
            ggam = g + offs[ti];
            gbet = g + offs[ti + 1];
        }
        ti -= 2;
        int k = m->conv_k[l - 1], p = k / 2, co_n = cs[l], cin = cs[l - 1];
        int hin = hs[l - 1], win = ws[l - 1];
        const double *Wt = th + offs[ti];
        double *gW = g + offs[ti], *gb = g + offs[ti + 1];
        const double *x = a[l - 1], *y = a[l];
        if (l > 1) for (int64_t i = 0; i < (int64_t)hin * win * cin; ++i) d_prev[i] = 0.0;
        for (int oh = 0; oh < hs[l]; ++oh)
            for (int ow = 0; ow < ws[l]; ++ow) {
                int64_t px = (int64_t)oh * ws[l] + ow;
                if (m->norm) {
                    /* through ReLU and the normalisation of this pixel, in place in d_cur:
                     * dy = ReLU'(.) d;  dgamma += dy xhat;  dbeta += dy;  t = gamma dy;
                     * dz = rstd (t - mean(t) - xhat mean(t xhat)) */
                    double *d = d_cur + px * co_n;
                    const double *v = xh[l] + px * co_n;
                    double m1 = 0.0, m2 = 0.0;
                    for (int co = 0; co < co_n; ++co) {
                        double dy = y[px * co_n + co] > 0.0 ? d[co] : 0.0;
                        ggam[co] += dy * v[co];
                        gbet[co] += dy;
                        d[co] = gam[co] * dy;
                        m1 += d[co];
                        m2 += d[co] * v[co];
                    }
                    m1 /= (double)co_n;
                    m2 /= (double)co_n;
                    for (int co = 0; co < co_n; ++co) d[co] = rs[l][px] * (d[co] - m1 - v[co] * m2);
                }
                for (int co = 0; co < co_n; ++co) {
                    int64_t oi = px * co_n + co;
                    double dz = m->norm ? d_cur[oi] : (y[oi] > 0.0 ? d_cur[oi] : 0.0);
                    if (dz == 0.0) continue;
                    gb[co] += dz;
                    for (int kh = 0; kh < k; ++kh) {
                        int ih = 2 * oh + kh - p;
                        if (ih < 0 || ih >= hin) continue;
                        for (int kw = 0; kw < k; ++kw) {
                            int iw = 2 * ow + kw - p;
                            if (iw < 0 || iw >= win) continue;
                            int64_t wi = (((int64_t)co * k + kh) * k + kw) * cin;
                            int64_t xi = ((int64_t)ih * win + iw) * cin;
                            for (int ci = 0; ci < cin; ++ci) {
                                gW[wi + ci] += dz * x[xi + ci];
                                if (l > 1) d_prev[xi + ci] += Wt[wi + ci] * dz;
                            }
                        }
                    }
                }
            }
        double *tmp = d_cur; d_cur = d_prev; d_prev = tmp;
    }
}

int64_t orc_bwd_scratch_len(const orc_model *m) {
    int32_t Ho[ORC_MAX_CONV], Wo[ORC_MAX_CONV];
    orc_conv_shapes(m, Ho, Wo);
    int64_t big = (int64_t)m->H * m->W;
    for (int l = 0; l < m->n_conv; ++l) { int64_t s = (int64_t)Ho[l] * Wo[l] * m->conv_c[l]; if (s > big) big = s; }
    int64_t h0 = (m->embed > 0 ? m->embed : m->conv_c[m->n_conv - 1]) + m->P;
    if (h0 > big) big = h0;
    if (m->n_lstm > 0 && m->lstm_h > big) big = m->lstm_h;
    for (int l = 0; l < m->n_fc; ++l) if (m->fc[l] > big) big = m->fc[l];
    return 2 * big;
}

/* Forward of B samples.  theta_used: parameter vector with weight matrices already
 * bf16-rounded (orc_round_weights).  acts: B * orc_act_stride doubles (kept for backward). */
void orc_encoder_fwd(const orc_model *m, const double *theta_used, int B, const double *depth, const double *proprio,
                     double *acts, double *mu, double *V, int act_bf16) {
    int64_t offs[ORC_MAX_TENSORS], szs[ORC_MAX_TENSORS];
    int32_t mat[ORC_MAX_TENSORS], n;
    orc_param_layout(m, offs, szs, mat, &n);
    int64_t stride = orc_act_stride(m);
#pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < B; ++b)
        fwd_one(m, theta_used, offs, depth + (int64_t)b * m->H * m->W, proprio + (int64_t)b * m->P,
                acts + b * stride, mu + (int64_t)b * m->A, V + b, act_bf16, 0, NULL);
}

/* Backward of B samples: grad (length = parameter vector) += sum over samples of the
 * per-sample gradient, given dL/dmu [B][A] and dL/dV [B]. */
void orc_encoder_bwd(const orc_model *m, const double *theta_used, int B, const double *acts, const double *dmu,
                     const double *dV, double *grad) {
    int64_t offs[ORC_MAX_TENSORS], szs[ORC_MAX_TENSORS];
    int32_t mat[ORC_MAX_TENSORS], n;
    int64_t total = orc_param_layout(m, offs, szs, mat, &n);
    int64_t stride = orc_act_stride(m);
    int64_t slen = orc_bwd_scratch_len(m);
#pragma omp parallel
    {
        double *g_local = (double *)calloc((size_t)total, sizeof(double));
        double *scratch = (double *)malloc((size_t)slen * sizeof(double));
#pragma omp for schedule(dynamic)
        for (int b = 0; b < B; ++b)
            bwd_one(m, theta_used, offs, n, acts + b * stride, dmu + (int64_t)b * m->A, dV[b], g_local, scratch, 0, NULL,
                    NULL);
#pragma omp critical
        for (int64_t i = 0; i < total; ++i) grad[i] += g_local[i];
        free(g_local);
        free(scratch);
    }
}

/* ------------------------------------------------------------------ loss -- */

/* PPO-clip loss with a diagonal Gaussian policy (state-independent log-sigma), an
 * unclipped squared-error value loss and an entropy bonus, and its gradient with
 * respect to mu, V and log-sigma.  Rows i < B, means over B_total rows.
 *   z = (a - mu)/sigma, sigma = exp(logsigma)
 *   logp = sum_j [ -z_j^2/2 - logsigma_j - ln(2 pi)/2 ]
 *   r = exp(logp - logp_old);  s = min(r*Adv, clamp(r, 1-eps, 1+eps)*Adv)
 *   L_pi = -mean(s);  L_V = mean((V - R)^2);  H = sum_j logsigma_j + (A/2)(1 + ln(2 pi))
 *   L = L_pi + c_v L_V - c_e H
 * out[0..4] += {L_pi, L_V, H * B/B_total, mean(logp_old - logp), mean(|r-1| > eps)} contributions
 * of these B rows (so that micro-batches sum to the minibatch value; H is a constant of the
 * parameters and is reported weighted by the share of rows).
 * dlogsigma[j] += sum_i dL/dlogp_i * (z_ij^2 - 1) - c_e * B/B_total. */
void orc_loss(int B, int B_total, int A, const double *mu, const double *V, const double *logsigma,
              const double *action, const double *logp_old, const double *adv, const double *ret, double clip,
              double c_v, double c_e, double *out, double *dmu, double *dV, double *dlogsigma) {
    const double half_log_2pi = 0.5 * log(2.0 * M_PI);
    double Bt = (double)B_total;
    double H = 0.0;
    for (int j = 0; j < A; ++j) H += logsigma[j];
    H += 0.5 * A * (1.0 + 2.0 * half_log_2pi);
    for (int i = 0; i < B; ++i) {
        double logp = 0.0;
        for (int j = 0; j < A; ++j) {
            double sg = exp(logsigma[j]);
            double z = (action[(int64_t)i * A + j] - mu[(int64_t)i * A + j]) / sg;
            logp += -0.5 * z * z - logsigma[j] - half_log_2pi;
        }
        double r = exp(logp - logp_old[i]);
        double rc = r < 1.0 - clip ? 1.0 - clip : (r > 1.0 + clip ? 1.0 + clip : r);
        double s_un = r * adv[i], s_cl = rc * adv[i];
        double s, gs;
        if (s_un <= s_cl) { s = s_un; gs = adv[i]; } else { s = s_cl; gs = 0.0; }
        out[0] += -s / Bt;
        double verr = V[i] - ret[i];
        out[1] += verr * verr / Bt;
        out[3] += (logp_old[i] - logp) / Bt;
        out[4] += (fabs(r - 1.0) > clip ? 1.0 : 0.0) / Bt;
        double dlogp = -gs * r / Bt;
        for (int j = 0; j < A; ++j) {
            double sg = exp(logsigma[j]);
            double z = (action[(int64_t)i * A + j] - mu[(int64_t)i * A + j]) / sg;
            dmu[(int64_t)i * A + j] = dlogp * z / sg;
            dlogsigma[j] += dlogp * (z * z - 1.0);
        }
        dV[i] = 2.0 * c_v * verr / Bt;
    }
    out[2] += H * (double)B / Bt;
    for (int j = 0; j < A; ++j) dlogsigma[j] += -c_e * (double)B / Bt;
}

/* Rollout-time action of the policy (Algorithm 2, actions <- pi(obs)):
 * a = mu + sigma * eps with eps ~ N(0, I) supplied by the caller, and its log-probability. */
void orc_sample_action(int B, int A, const double *mu, const double *logsigma, const double *eps, double *action,
                       double *logp) {
    const double half_log_2pi = 0.5 * log(2.0 * M_PI);
    for (int i = 0; i < B; ++i) {
        double lp = 0.0;
        for (int j = 0; j < A; ++j) {
            double e = eps[(int64_t)i * A + j];
            action[(int64_t)i * A + j] = mu[(int64_t)i * A + j] + exp(logsigma[j]) * e;
            lp += -0.5 * e * e - logsigma[j] - half_log_2pi;
        }
        logp[i] = lp;
    }
}

/* ------------------------------------------------------------------ Adam -- */

/* Adam with bias correction, epsilon outside the square root and after the
 * correction, no weight decay; step is 1-based.  theta is rounded to fp32 on output
 * (the master copy is fp32); m and v are kept in fp64 here. */
void orc_adam(int64_t n, double *theta, double *m, double *v, const double *g, double lr, double beta1, double beta2,
              double eps, int64_t step) {
    double c1 = 1.0 - pow(beta1, (double)step), c2 = 1.0 - pow(beta2, (double)step);
    for (int64_t i = 0; i < n; ++i) {
        m[i] = beta1 * m[i] + (1.0 - beta1) * g[i];
        v[i] = beta2 * v[i] + (1.0 - beta2) * g[i] * g[i];
        double mhat = m[i] / c1, vhat = v[i] / c2;
        theta[i] = (double)(float)(theta[i] - lr * mhat / (sqrt(vhat) + eps));
    }
}

/* ------------------------------------------------------------ depth producer -- */

/* A stand-in for the simulator's tiled depth rendering (Section III-C renders a depth image per environment; the
 * paper gives no formulas, so the camera and the scene are a reading): one pinhole camera per env at the origin,
 * looking along +z, pixel (v, u) of an H x W image sees the ray through ((u + 0.5 - W/2) / f, (v + 0.5 - H/2) / f, 1)
 * with f = (W/2) / tan(hfov/2).  The scene of an env is the plane n . p = d (unit n in params[0..2], d in params[3]) and
 * n_prims primitives of 8 doubles each: {type, x, y, z, p0, p1, p2, p3}
 *   type 0 sphere : centre (x,y,z), radius p0
 *   type 1 box    : centre (x,y,z), half extents (p0,p1,p2), axis aligned
 *   type 2 capsule: segment from (x,y,z) to (x,y,z) + (p0,p1,p2), radius p3
 * The depth of a pixel is the z coordinate of the nearest intersection in front of the camera; it is kept when it
 * lies in [near, far] and is 0 (no return) otherwise, then rounded to fp16 (nearest even) and returned as a double. */
static double round_fp16(double x) {
    if (x == 0.0) return 0.0;
    int e;
    double m = frexp(fabs(x), &e);          /* |x| = m 2^e, m in [0.5, 1) */
    int emin = -13;                          /* smallest normal 2^-14 = 0.5 * 2^-13 */
    int shift = (e < emin ? emin : e) - 11;  /* 11 significant bits above 2^shift */
    double q = ldexp(fabs(x), -shift);
    double r = nearbyint(q);                 /* ties to even in the default rounding mode */
    (void)m;
    double y = ldexp(r, shift);
    if (y > 65504.0) y = INFINITY;
    return x < 0 ? -y : y;
}

static double hit_sphere(const double o[3], const double d[3], const double c[3], double r) {
    /* |o + t d - c|^2 = r^2, nearest t > 0 */
    double oc[3] = {o[0] - c[0], o[1] - c[1], o[2] - c[2]};
    double a = d[0] * d[0] + d[1] * d[1] + d[2] * d[2];
    double b = oc[0] * d[0] + oc[1] * d[1] + oc[2] * d[2];
    double cc = oc[0] * oc[0] + oc[1] * oc[1] + oc[2] * oc[2] - r * r;
    double disc = b * b - a * cc;
    if (disc < 0.0) return INFINITY;
    double s = sqrt(disc);
    double t = (-b - s) / a;
    if (t > 0.0) return t;
    t = (-b + s) / a;
    return t > 0.0 ? t : INFINITY;
}

static double hit_box(const double d[3], const double c[3], const double h[3]) {
    /* slabs, ray from the origin */
    double t0 = 0.0, t1 = INFINITY;
    for (int i = 0; i < 3; ++i) {
        double lo = c[i] - h[i], hi = c[i] + h[i];
        if (d[i] == 0.0) {
            if (lo > 0.0 || hi < 0.0) return INFINITY;
            continue;
        }
        double a = lo / d[i], b = hi / d[i];
        if (a > b) { double tmp = a; a = b; b = tmp; }
        if (a > t0) t0 = a;
        if (b < t1) t1 = b;
    }
    if (t0 > t1) return INFINITY;
    return t0 > 0.0 ? t0 : (t1 > 0.0 && t1 < INFINITY ? t1 : INFINITY);
}

static double hit_capsule(const double d[3], const double pa[3], const double ab[3], double r) {
    /* cylinder around the segment plus the two end spheres; ray from the origin */
    double best = INFINITY;
    const double o[3] = {0.0, 0.0, 0.0};
    double pb[3] = {pa[0] + ab[0], pa[1] + ab[1], pa[2] + ab[2]};
    double t = hit_sphere(o, d, pa, r);
    if (t < best) best = t;
    t = hit_sphere(o, d, pb, r);
    if (t < best) best = t;
    double l2 = ab[0] * ab[0] + ab[1] * ab[1] + ab[2] * ab[2];
    if (l2 > 0.0) {
        /* components perpendicular to the axis: |(t d - pa)_perp|^2 = r^2 */
        double dd = (d[0] * ab[0] + d[1] * ab[1] + d[2] * ab[2]) / l2;
        double pp = (-(pa[0] * ab[0] + pa[1] * ab[1] + pa[2] * ab[2])) / l2; /* axis coordinate of the origin */
        double dp[3], op[3];
        for (int i = 0; i < 3; ++i) {
            dp[i] = d[i] - dd * ab[i];
            op[i] = -pa[i] - pp * ab[i];
        }
        double a = dp[0] * dp[0] + dp[1] * dp[1] + dp[2] * dp[2];
        double b = op[0] * dp[0] + op[1] * dp[1] + op[2] * dp[2];
        double c = op[0] * op[0] + op[1] * op[1] + op[2] * op[2] - r * r;
        double disc = b * b - a * c;
        if (a > 0.0 && disc >= 0.0) {
            double s = sqrt(disc);
            double ts[2] = {(-b - s) / a, (-b + s) / a};
            for (int k = 0; k < 2; ++k) {
                double u = pp + ts[k] * dd; /* position along the axis in units of its length */
                if (ts[k] > 0.0 && u >= 0.0 && u <= 1.0 && ts[k] < best) best = ts[k];
            }
        }
    }
    return best;
}

void orc_render_depth(int N, int H, int W, double hfov, double near, double far, const double *plane /*[N][4]*/,
                      int n_prims, const double *prims /*[N][n_prims][8]*/, double *depth /*[N][H][W]*/) {
    double f = (0.5 * W) / tan(0.5 * hfov);
#pragma omp parallel for schedule(static)
    for (int n = 0; n < N; ++n) {
        const double *pl = plane + 4 * (int64_t)n;
        for (int v = 0; v < H; ++v)
            for (int u = 0; u < W; ++u) {
                double d[3] = {(u + 0.5 - 0.5 * W) / f, (v + 0.5 - 0.5 * H) / f, 1.0};
                double best = INFINITY;
                double nd = pl[0] * d[0] + pl[1] * d[1] + pl[2] * d[2];
                if (nd != 0.0) {
                    double t = pl[3] / nd;
                    if (t > 0.0) best = t;
                }
                for (int p = 0; p < n_prims; ++p) {
                    const double *q = prims + ((int64_t)n * n_prims + p) * 8;
                    int type = (int)q[0];
                    double t = INFINITY;
                    if (type == 0) {
                        const double o[3] = {0.0, 0.0, 0.0};
                        t = hit_sphere(o, d, q + 1, q[4]);
                    } else if (type == 1) {
                        t = hit_box(d, q + 1, q + 4);
                    } else if (type == 2) {
                        t = hit_capsule(d, q + 1, q + 4, q[7]);
                    }
                    if (t < best) best = t;
                }
                double z = best; /* d has z = 1: the ray parameter is the depth */
                depth[((int64_t)n * H + v) * W + u] = (z >= near && z <= far) ? round_fp16(z) : 0.0;
            }
    }
}

double orc_round_fp16(double x) { return round_fp16(x); }

/* ------------------------------------------------------- recurrent trunk -- */

/* Length of the per-row record of the recurrent trunk: for every LSTM layer the gate activations i, f, g, o
 * (4H), the cell state c (H), the output h (H) and the state the step started from, h_prev (H) and c_prev (H). */
int64_t orc_lstm_rec_len(const orc_model *m) { return (int64_t)m->n_lstm * 8 * m->lstm_h; }

static double sigmoid(double x) { return 1.0 / (1.0 + exp(-x)); }

/* Forward over a minibatch of sequences (Section III-C: CNN embedding joined with proprioception -> LSTM layers ->
 * fully connected layers -> heads).  Rows are time-major: row r = t * Be + e is env e of the minibatch at step t.
 * Per LSTM layer, with x_t the layer's input (h_0 of the row, or the output of the layer below):
 *   (i, f, g, o) = (sigmoid, sigmoid, tanh, sigmoid)(W_x x_t + W_h h_prev + b),   c_t = f c_prev + i g,
 *   h_t = o tanh(c_t),
 * the state a step starts from being the caller's (h_init, c_init) [L][Be][H] at t = 0 and afterwards the previous
 * step's (h, c), zeroed where done[t-1][e] != 0 (the episode ended: Algorithm 2 stores done with the step that
 * returned it).  With act_bf16 the stored h (the operand of the next contractions) is rounded to bf16; c is not.
 * acts [R][orc_act_stride] and lrec [R][orc_lstm_rec_len] are kept for the backward pass. */
void orc_encoder_fwd_seq(const orc_model *m, const double *theta_used, int T, int Be, const double *depth,
                         const double *proprio, const uint8_t *done, const double *h_init, const double *c_init,
                         double *acts, double *lrec, double *mu, double *V, int act_bf16) {
    int64_t offs[ORC_MAX_TENSORS], szs[ORC_MAX_TENSORS];
    int32_t mat[ORC_MAX_TENSORS], n;
    orc_param_layout(m, offs, szs, mat, &n);
    const int64_t stride = orc_act_stride(m), lstride = orc_lstm_rec_len(m);
    const int R = T * Be, H = m->lstm_h, L = m->n_lstm;
    const int h0w = (m->embed > 0 ? m->embed : m->conv_c[m->n_conv - 1]) + m->P;
    int64_t h0_off = act_main_len(m) - h0w;
    for (int l = 0; l < m->n_fc; ++l) h0_off -= m->fc[l];
#pragma omp parallel for schedule(dynamic)
    for (int r = 0; r < R; ++r)
        fwd_one(m, theta_used, offs, depth + (int64_t)r * m->H * m->W, proprio + (int64_t)r * m->P, acts + r * stride,
                NULL, NULL, act_bf16, 1, NULL);
    const int ti0 = 2 * m->n_conv + (m->norm ? 2 * m->n_conv : 0) + (m->embed > 0 ? 2 : 0);
    for (int l = 0; l < L; ++l) {
        const int in = l == 0 ? h0w : H;
        const double *Wx = theta_used + offs[ti0 + 3 * l], *Wh = theta_used + offs[ti0 + 3 * l + 1];
        const double *b = theta_used + offs[ti0 + 3 * l + 2];
        for (int t = 0; t < T; ++t) {
#pragma omp parallel for schedule(static)
            for (int e = 0; e < Be; ++e) {
                const int r = t * Be + e;
                double *rec = lrec + r * lstride + (int64_t)l * 8 * H;
                double *gi = rec, *gf = rec + H, *gg = rec + 2 * H, *go = rec + 3 * H;
                double *c = rec + 4 * H, *h = rec + 5 * H, *hp = rec + 6 * H, *cp = rec + 7 * H;
                const double *x = l == 0 ? acts + r * stride + h0_off : lrec + r * lstride + (int64_t)(l - 1) * 8 * H + 5 * H;
                if (t == 0) {
                    for (int j = 0; j < H; ++j) {
                        hp[j] = h_init[((int64_t)l * Be + e) * H + j];
                        cp[j] = c_init[((int64_t)l * Be + e) * H + j];
                    }
                } else {
                    const double *prev = lrec + (int64_t)(r - Be) * lstride + (int64_t)l * 8 * H;
                    const double keep = done[(t - 1) * Be + e] ? 0.0 : 1.0;
                    for (int j = 0; j < H; ++j) {
                        hp[j] = keep * prev[5 * H + j];
                        cp[j] = keep * prev[4 * H + j];
                    }
                }
                for (int j = 0; j < 4 * H; ++j) {
                    double acc = b[j];
                    for (int k = 0; k < in; ++k) acc += Wx[(int64_t)j * in + k] * x[k];
                    for (int k = 0; k < H; ++k) acc += Wh[(int64_t)j * H + k] * hp[k];
                    rec[j] = (j >= 2 * H && j < 3 * H) ? tanh(acc) : sigmoid(acc);
                }
                for (int j = 0; j < H; ++j) {
                    c[j] = gf[j] * cp[j] + gi[j] * gg[j];
                    const double hv = go[j] * tanh(c[j]);
                    h[j] = act_bf16 ? orc_round_bf16(hv) : hv;
                }
            }
        }
    }
#pragma omp parallel for schedule(dynamic)
    for (int r = 0; r < R; ++r)
        fwd_one(m, theta_used, offs, NULL, NULL, acts + r * stride, mu + (int64_t)r * m->A, V + r, act_bf16, 2,
                lrec + r * lstride + (int64_t)(L - 1) * 8 * H + 5 * H);
}

/* Backward through orc_encoder_fwd_seq (back-propagation through time over the T steps of the minibatch; the
 * initial states are constants).  grad += dL/dtheta. */
void orc_encoder_bwd_seq(const orc_model *m, const double *theta_used, int T, int Be, const uint8_t *done,
                         const double *acts, const double *lrec, const double *dmu, const double *dV, double *grad) {
    int64_t offs[ORC_MAX_TENSORS], szs[ORC_MAX_TENSORS];
    int32_t mat[ORC_MAX_TENSORS], n;
    const int64_t total = orc_param_layout(m, offs, szs, mat, &n);
    const int64_t stride = orc_act_stride(m), lstride = orc_lstm_rec_len(m), slen = orc_bwd_scratch_len(m);
    const int R = T * Be, H = m->lstm_h, L = m->n_lstm;
    const int h0w = (m->embed > 0 ? m->embed : m->conv_c[m->n_conv - 1]) + m->P;
    int64_t h0_off = act_main_len(m) - h0w;
    for (int l = 0; l < m->n_fc; ++l) h0_off -= m->fc[l];
    const int wmax = H > h0w ? H : h0w;
    double *dx = (double *)calloc((size_t)R * wmax, sizeof(double));   /* gradient w.r.t. a layer's output rows */
    double *dxl = (double *)calloc((size_t)R * wmax, sizeof(double));  /* gradient w.r.t. the layer's input rows */
    /* fully connected layers and head, row by row */
#pragma omp parallel
    {
        double *g_local = (double *)calloc((size_t)total, sizeof(double));
        double *scratch = (double *)malloc((size_t)slen * sizeof(double));
#pragma omp for schedule(dynamic)
        for (int r = 0; r < R; ++r)
            bwd_one(m, theta_used, offs, n, acts + r * stride, dmu + (int64_t)r * m->A, dV[r], g_local, scratch, 2,
                    lrec + r * lstride + (int64_t)(L - 1) * 8 * H + 5 * H, dx + (int64_t)r * wmax);
#pragma omp critical
        for (int64_t i = 0; i < total; ++i) grad[i] += g_local[i];
        free(g_local);
        free(scratch);
    }
    const int ti0 = 2 * m->n_conv + (m->norm ? 2 * m->n_conv : 0) + (m->embed > 0 ? 2 : 0);
    double *dh_carry = (double *)malloc((size_t)Be * H * sizeof(double));
    double *dc_carry = (double *)malloc((size_t)Be * H * sizeof(double));
    double *dgate = (double *)malloc((size_t)4 * H * sizeof(double));
    for (int l = L - 1; l >= 0; --l) {
        const int in = l == 0 ? h0w : H;
        const double *Wx = theta_used + offs[ti0 + 3 * l], *Wh = theta_used + offs[ti0 + 3 * l + 1];
        double *gWx = grad + offs[ti0 + 3 * l], *gWh = grad + offs[ti0 + 3 * l + 1], *gb = grad + offs[ti0 + 3 * l + 2];
        for (int64_t i = 0; i < (int64_t)Be * H; ++i) dh_carry[i] = dc_carry[i] = 0.0;
        for (int64_t i = 0; i < (int64_t)R * wmax; ++i) dxl[i] = 0.0;
        for (int t = T - 1; t >= 0; --t)
            for (int e = 0; e < Be; ++e) {
                const int r = t * Be + e;
                const double *rec = lrec + r * lstride + (int64_t)l * 8 * H;
                const double *gi = rec, *gf = rec + H, *gg = rec + 2 * H, *go = rec + 3 * H;
                const double *c = rec + 4 * H, *hp = rec + 6 * H, *cp = rec + 7 * H;
                const double *x = l == 0 ? acts + r * stride + h0_off : lrec + r * lstride + (int64_t)(l - 1) * 8 * H + 5 * H;
                double *dhc = dh_carry + (int64_t)e * H, *dcc = dc_carry + (int64_t)e * H;
                for (int j = 0; j < H; ++j) {
                    const double dh = dx[(int64_t)r * wmax + j] + dhc[j];
                    const double tc = tanh(c[j]);
                    const double dc = dcc[j] + dh * go[j] * (1.0 - tc * tc);
                    dgate[j] = dc * gg[j] * gi[j] * (1.0 - gi[j]);             /* input gate, pre-activation */
                    dgate[H + j] = dc * cp[j] * gf[j] * (1.0 - gf[j]);         /* forget gate */
                    dgate[2 * H + j] = dc * gi[j] * (1.0 - gg[j] * gg[j]);     /* cell candidate */
                    dgate[3 * H + j] = dh * tc * go[j] * (1.0 - go[j]);        /* output gate */
                    dcc[j] = dc * gf[j];                                       /* into c_prev */
                }
                for (int j = 0; j < H; ++j) dhc[j] = 0.0;
                double *dxr = dxl + (int64_t)r * wmax;
                for (int j = 0; j < 4 * H; ++j) {
                    const double d = dgate[j];
                    gb[j] += d;
                    for (int k = 0; k < in; ++k) {
                        gWx[(int64_t)j * in + k] += d * x[k];
                        dxr[k] += Wx[(int64_t)j * in + k] * d;
                    }
                    for (int k = 0; k < H; ++k) {
                        gWh[(int64_t)j * H + k] += d * hp[k];
                        dhc[k] += Wh[(int64_t)j * H + k] * d;
                    }
                }
                /* the state this step started from was the previous step's, zeroed after a done */
                const double keep = (t > 0 && !done[(t - 1) * Be + e]) ? 1.0 : 0.0;
                for (int j = 0; j < H; ++j) {
                    dhc[j] *= keep;
                    dcc[j] *= keep;
                }
            }
        double *tmp = dx; dx = dxl; dxl = tmp;
    }
    /* h_0 and below, row by row */
#pragma omp parallel
    {
        double *g_local = (double *)calloc((size_t)total, sizeof(double));
        double *scratch = (double *)malloc((size_t)slen * sizeof(double));
#pragma omp for schedule(dynamic)
        for (int r = 0; r < R; ++r)
            bwd_one(m, theta_used, offs, n, acts + r * stride, NULL, 0.0, g_local, scratch, 1, NULL, dx + (int64_t)r * wmax);
#pragma omp critical
        for (int64_t i = 0; i < total; ++i) grad[i] += g_local[i];
        free(g_local);
        free(scratch);
    }
    free(dx); free(dxl); free(dh_carry); free(dc_carry); free(dgate);
}
