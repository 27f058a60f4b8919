/*
 * sla_oracle.c — TEST INFRASTRUCTURE, not the product (see sla_oracle.h).
 *
 * Token-by-token recurrent form of Softmax Linear Attention in fp64.
 * One (batch, head) sequence at a time; the only coupling between heads is the
 * softmax over the H gate logits of a token (Eq. 4), computed first.
 *
 * Readings of the paper taken here:
 *  - the read-out at step t uses the state after the write of step t (Eq. 5-6);
 *  - GLA's forget gate acts per key dimension: S <- diag(alpha_t) S  (Eq. 12);
 *  - Gated DeltaNet (Eq. 14-16) is printed without its decay; a scalar decay
 *    alpha_t = exp(g_t) is applied to S_{t-1} before the delta step, so g = 0
 *    gives the printed equations.  The key-side gate multiplies v only; the
 *    erase term uses the ungated key.  beta_t is a scalar per (token, head).
 *  - no normaliser and no feature map inside: q, k arrive already mapped;
 *    `scale` multiplies q.
 */
#include "sla_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int sla_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Eq. 4 — softmax across the head axis. */
void sla_oracle_head_softmax(const double *logits, long n_tok, int H, double *gates) {
    for (long t = 0; t < n_tok; ++t) {
        const double *l = logits + t * H;
        double *g = gates + t * H;
        double m = l[0];
        for (int h = 1; h < H; ++h) if (l[h] > m) m = l[h];
        double z = 0.0;
        for (int h = 0; h < H; ++h) { g[h] = exp(l[h] - m); z += g[h]; }
        for (int h = 0; h < H; ++h) g[h] /= z;
    }
}

/*
 * Eq. 4, the score projections that feed the head softmax.  Reading taken: W_G in R^{d x H} with d the per-head
 * width (the paper's parameter count, about 0.05M for 24 layers of two such matrices at hidden 1024 with 4 heads,
 * only fits d = 256 = 1024 / 4), and the score of head h comes from that head's own vector through column h:
 *     s[b,t,h] = sum_c x[b,t,h,c] * W[c,h]        (x = q with W_GQ, x = k with W_GK)
 * x: [n_tok, H, d], W: [d, H], s: [n_tok, H].
 */
void sla_oracle_gate_scores(long n_tok, int H, int d, const double *x, const double *W, double *s) {
    for (long t = 0; t < n_tok; ++t)
        for (int h = 0; h < H; ++h) {
            double acc = 0.0;
            for (int c = 0; c < d; ++c) acc += x[(t * H + h) * d + c] * W[(long)c * H + h];
            s[t * H + h] = acc;
        }
}

/* Reverse of sla_oracle_gate_scores: dx[b,t,h,c] += ds[b,t,h] W[c,h] (ADDED to what dx holds: x also feeds the
 * recurrence), dW[c,h] = sum_t ds[t,h] x[t,h,c] (overwritten). */
void sla_oracle_gate_scores_backward(long n_tok, int H, int d, const double *x, const double *W,
                                     const double *ds, double *dx, double *dW) {
    for (long i = 0; i < (long)d * H; ++i) dW[i] = 0.0;
    for (long t = 0; t < n_tok; ++t)
        for (int h = 0; h < H; ++h) {
            double g = ds[t * H + h];
            for (int c = 0; c < d; ++c) {
                dx[(t * H + h) * d + c] += g * W[(long)c * H + h];
                dW[(long)c * H + h] += g * x[(t * H + h) * d + c];
            }
        }
}

/*
 * Eq. 7, the output projection: the heads' outputs of a token, concatenated, times W^O:
 *     y[t,n] = sum_c o[t,c] * W[c,n]        (c runs over the H*d_v concatenated features)
 * o: [n_tok, K], W: [K, N], y: [n_tok, N].  Tokens are independent (the loop over them runs in parallel).
 */
void sla_oracle_out_proj(long n_tok, int K, int N, const double *o, const double *W, double *y) {
#pragma omp parallel for schedule(static)
    for (long t = 0; t < n_tok; ++t) {
        double *yt = y + t * N;
        for (int n = 0; n < N; ++n) yt[n] = 0.0;
        for (int c = 0; c < K; ++c) {
            double a = o[t * K + c];
            const double *Wc = W + (long)c * N;
            for (int n = 0; n < N; ++n) yt[n] += a * Wc[n];
        }
    }
}

/* Reverse of sla_oracle_out_proj: d_o[t,c] = sum_n dy[t,n] W[c,n];  dW[c,n] = sum_t o[t,c] dy[t,n] (tokens in order). */
void sla_oracle_out_proj_backward(long n_tok, int K, int N, const double *o, const double *W, const double *dy,
                                  double *d_o, double *dW) {
#pragma omp parallel for schedule(static)
    for (long t = 0; t < n_tok; ++t)
        for (int c = 0; c < K; ++c) {
            double acc = 0.0;
            for (int n = 0; n < N; ++n) acc += dy[t * N + n] * W[(long)c * N + n];
            d_o[t * K + c] = acc;
        }
#pragma omp parallel for schedule(static)
    for (int c = 0; c < K; ++c) {
        double *dWc = dW + (long)c * N;
        for (int n = 0; n < N; ++n) dWc[n] = 0.0;
        for (long t = 0; t < n_tok; ++t) {
            double a = o[t * K + c];
            for (int n = 0; n < N; ++n) dWc[n] += a * dy[t * N + n];
        }
    }
}

/*
 * Feature map of the Gated-DeltaNet instantiation ("short-convolution module" followed by SiLU, Experimental setup),
 * as published for Gated DeltaNet: a depthwise causal convolution of K taps over time, channel by channel, then
 * SiLU, then (for q and k) L2 normalisation over the d features of each head.
 *     y[b,t,c] = sum_{j<K} w[c,j] x[b,t-(K-1)+j,c]      (tokens before the sequence start read as zero)
 *     z = y * sigmoid(y)
 *     out[b,t,h,:] = z[b,t,h,:] / sqrt(sum_d z[b,t,h,d]^2 + eps)      when normalize != 0, else out = z
 * x, out: [B,T,C] with C = H*d channels; w: [C,K].
 */
static double silu(double y) { return y / (1.0 + exp(-y)); }
static double silu_grad(double y) { double s = 1.0 / (1.0 + exp(-y)); return s * (1.0 + y * (1.0 - s)); }

void sla_oracle_shortconv(int B, int T, int H, int d, int K, int normalize, double eps,
                          const double *x, const double *w, double *out) {
    long C = (long)H * d;
    for (int b = 0; b < B; ++b)
        for (int t = 0; t < T; ++t) {
            double *o = out + ((long)b * T + t) * C;
            for (long c = 0; c < C; ++c) {
                double y = 0.0;
                for (int j = 0; j < K; ++j) {
                    int tt = t - (K - 1) + j;
                    if (tt >= 0) y += w[c * K + j] * x[((long)b * T + tt) * C + c];
                }
                o[c] = silu(y);
            }
            if (normalize)
                for (int h = 0; h < H; ++h) {
                    double ss = 0.0;
                    for (int c = 0; c < d; ++c) ss += o[(long)h * d + c] * o[(long)h * d + c];
                    double r = sqrt(ss + eps);
                    for (int c = 0; c < d; ++c) o[(long)h * d + c] /= r;
                }
        }
}

/* Reverse of sla_oracle_shortconv: dx [B,T,C] and dw [C,K], both overwritten. */
void sla_oracle_shortconv_backward(int B, int T, int H, int d, int K, int normalize, double eps,
                                   const double *x, const double *w, const double *dout,
                                   double *dx, double *dw) {
    long C = (long)H * d;
    double *y = (double *)malloc(sizeof(double) * C);
    double *z = (double *)malloc(sizeof(double) * C);
    double *dz = (double *)malloc(sizeof(double) * C);
    for (long i = 0; i < (long)B * T * C; ++i) dx[i] = 0.0;
    for (long i = 0; i < C * K; ++i) dw[i] = 0.0;
    for (int b = 0; b < B; ++b)
        for (int t = 0; t < T; ++t) {
            const double *go = dout + ((long)b * T + t) * C;
            for (long c = 0; c < C; ++c) {
                double acc = 0.0;
                for (int j = 0; j < K; ++j) {
                    int tt = t - (K - 1) + j;
                    if (tt >= 0) acc += w[c * K + j] * x[((long)b * T + tt) * C + c];
                }
                y[c] = acc;
                z[c] = silu(acc);
                dz[c] = go[c];
            }
            if (normalize)
                for (int h = 0; h < H; ++h) {
                    double ss = 0.0, dot = 0.0;
                    for (int c = 0; c < d; ++c) {
                        ss += z[(long)h * d + c] * z[(long)h * d + c];
                        dot += z[(long)h * d + c] * go[(long)h * d + c];
                    }
                    double r = sqrt(ss + eps);
                    /* out = z / r, r = sqrt(|z|^2 + eps):  dz = dout / r - z (z . dout) / r^3 */
                    for (int c = 0; c < d; ++c)
                        dz[(long)h * d + c] = go[(long)h * d + c] / r - z[(long)h * d + c] * dot / (r * r * r);
                }
            for (long c = 0; c < C; ++c) {
                double dy = dz[c] * silu_grad(y[c]);
                for (int j = 0; j < K; ++j) {
                    int tt = t - (K - 1) + j;
                    if (tt >= 0) {
                        dx[((long)b * T + tt) * C + c] += w[c * K + j] * dy;
                        dw[c * K + j] += dy * x[((long)b * T + tt) * C + c];
                    }
                }
            }
        }
    free(y); free(z); free(dz);
}

/* Per-step decay factors a[0..d_k) for sequence (b,h) at token t. */
static void decay_factors(int variant, const double *log_decay, long bt, int H, int h, int d_k,
                          double *a) {
    if (variant == SLA_ORACLE_RETNET) {
        double g = exp(log_decay[h]);
        for (int d = 0; d < d_k; ++d) a[d] = g;
    } else if (variant == SLA_ORACLE_GLA) {
        const double *g = log_decay + (bt * H + h) * (long)d_k;
        for (int d = 0; d < d_k; ++d) a[d] = exp(g[d]);
    } else {
        double g = exp(log_decay[bt * H + h]);
        for (int d = 0; d < d_k; ++d) a[d] = g;
    }
}

/*
 * One state transition on S [d_k, d_v] (row = key dimension).
 *   RETNET / GLA (Eq. 10, 12):  S <- diag(a) S + kw^T vw          kw = Gk k, vw = v
 *   GDN (Eq. 14-15 + decay):    Sbar = a S ; r = vw - kw Sbar ; u = beta r ; S <- Sbar + kw^T u
 *                                                                  kw = k,   vw = Gk v
 * r_out (d_v, GDN only, nullable) receives r.
 */
static void state_step(int variant, int d_k, int d_v, const double *a, double beta,
                       const double *kw, const double *vw, double *S, double *r_out) {
    for (int d = 0; d < d_k; ++d)
        for (int j = 0; j < d_v; ++j) S[d * d_v + j] *= a[d];
    if (variant == SLA_ORACLE_GDN) {
        double *r = (double *)malloc(sizeof(double) * d_v);
        for (int j = 0; j < d_v; ++j) {
            double acc = 0.0;
            for (int d = 0; d < d_k; ++d) acc += kw[d] * S[d * d_v + j];
            r[j] = vw[j] - acc;
        }
        for (int d = 0; d < d_k; ++d)
            for (int j = 0; j < d_v; ++j) S[d * d_v + j] += kw[d] * (beta * r[j]);
        if (r_out) memcpy(r_out, r, sizeof(double) * d_v);
        free(r);
    } else {
        for (int d = 0; d < d_k; ++d)
            for (int j = 0; j < d_v; ++j) S[d * d_v + j] += kw[d] * vw[j];
    }
}

/* Gated operands of one token: qw = scale Gq q ; (kw, vw) as state_step wants them. */
static void gated_operands(int variant, int d_k, int d_v, double scale, double Gq, double Gk,
                           const double *q, const double *k, const double *v,
                           double *qw, double *kw, double *vw) {
    for (int d = 0; d < d_k; ++d) qw[d] = scale * Gq * q[d];
    if (variant == SLA_ORACLE_GDN) {
        for (int d = 0; d < d_k; ++d) kw[d] = k[d];
        for (int j = 0; j < d_v; ++j) vw[j] = Gk * v[j];
    } else {
        for (int d = 0; d < d_k; ++d) kw[d] = Gk * k[d];
        for (int j = 0; j < d_v; ++j) vw[j] = v[j];
    }
}

static int bad_shape(int variant, long B, long T, int H, int d_k, int d_v) {
    return variant < 0 || variant > 2 || B < 0 || T < 0 || H < 1 || d_k < 1 || d_v < 1;
}

int sla_oracle_forward(int variant, int B, int T, int H, int d_k, int d_v, double scale,
                       const double *q, const double *k, const double *v,
                       const double *log_decay, const double *beta,
                       const double *lq, const double *lk, const double *h0,
                       double *o, double *ht) {
    if (bad_shape(variant, B, T, H, d_k, d_v)) return -1;
    if (variant == SLA_ORACLE_GDN && !beta) return -1;
    long n_tok = (long)B * T;
    double *Gq = (double *)malloc(sizeof(double) * (n_tok * H + 1));
    double *Gk = (double *)malloc(sizeof(double) * (n_tok * H + 1));
    sla_oracle_head_softmax(lq, n_tok, H, Gq);
    sla_oracle_head_softmax(lk, n_tok, H, Gk);
    long sdim = (long)d_k * d_v;

#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < H; ++h) {
            double *S = (double *)calloc(sdim, sizeof(double));
            double *a = (double *)malloc(sizeof(double) * d_k);
            double *qw = (double *)malloc(sizeof(double) * d_k);
            double *kw = (double *)malloc(sizeof(double) * d_k);
            double *vw = (double *)malloc(sizeof(double) * d_v);
            if (h0) memcpy(S, h0 + ((long)b * H + h) * sdim, sizeof(double) * sdim);
            for (int t = 0; t < T; ++t) {
                long bt = (long)b * T + t;
                long row = bt * H + h;
                decay_factors(variant, log_decay, bt, H, h, d_k, a);
                gated_operands(variant, d_k, d_v, scale, Gq[row], Gk[row],
                               q + row * d_k, k + row * d_k, v + row * d_v, qw, kw, vw);
                state_step(variant, d_k, d_v, a, beta ? beta[row] : 0.0, kw, vw, S, NULL);
                double *ot = o + row * d_v;                      /* Eq. 6: read after write */
                for (int j = 0; j < d_v; ++j) {
                    double acc = 0.0;
                    for (int d = 0; d < d_k; ++d) acc += qw[d] * S[d * d_v + j];
                    ot[j] = acc;
                }
            }
            if (ht) memcpy(ht + ((long)b * H + h) * sdim, S, sizeof(double) * sdim);
            free(S); free(a); free(qw); free(kw); free(vw);
        }
    }
    free(Gq); free(Gk);
    return 0;
}

int sla_oracle_decode_step(int variant, int Bdec, int H, int d_k, int d_v, double scale,
                           const double *q_t, const double *k_t, const double *v_t,
                           const double *log_decay_t, const double *beta_t,
                           const double *lq_t, const double *lk_t,
                           double *state, double *o_t) {
    /* A decode step is the T = 1 forward on the caller's state. */
    if (!state) return -1;
    return sla_oracle_forward(variant, Bdec, 1, H, d_k, d_v, scale, q_t, k_t, v_t, log_decay_t,
                              beta_t, lq_t, lk_t, state, o_t, state);
}

int sla_oracle_decode_steps(int variant, int Bdec, int n_tok, int H, int d_k, int d_v, double scale,
                            const double *q, const double *k, const double *v,
                            const double *log_decay, const double *beta,
                            const double *lq, const double *lk,
                            double *state, double *o) {
    /* n_tok consecutive steps of every sequence: token t reads the state token t-1 left, i.e. the
     * recurrence of sla_oracle_forward over n_tok tokens started from the caller's state. */
    if (!state) return -1;
    return sla_oracle_forward(variant, Bdec, n_tok, H, d_k, d_v, scale, q, k, v, log_decay, beta,
                              lq, lk, state, o, state);
}

/* Softmax backward over heads: dl_h = G_h (dG_h - sum_h' G_h' dG_h'). */
static void head_softmax_backward(const double *G, const double *dG, long n_tok, int H, double *dl) {
    for (long t = 0; t < n_tok; ++t) {
        double dot = 0.0;
        for (int h = 0; h < H; ++h) dot += G[t * H + h] * dG[t * H + h];
        for (int h = 0; h < H; ++h) dl[t * H + h] = G[t * H + h] * (dG[t * H + h] - dot);
    }
}

#define SEG 64   /* states are re-derived SEG tokens at a time from a checkpoint */

int sla_oracle_backward(int variant, int B, int T, int H, int d_k, int d_v, double scale,
                        const double *q, const double *k, const double *v,
                        const double *log_decay, const double *beta,
                        const double *lq, const double *lk, const double *h0,
                        const double *dO, const double *dht,
                        double *dq, double *dk, double *dv,
                        double *dlog_decay, double *dbeta,
                        double *dlq, double *dlk, double *dh0) {
    if (bad_shape(variant, B, T, H, d_k, d_v)) return -1;
    if (variant == SLA_ORACLE_GDN && !beta) return -1;
    long n_tok = (long)B * T;
    long sdim = (long)d_k * d_v;
    double *Gq = (double *)malloc(sizeof(double) * (n_tok * H + 1));
    double *Gk = (double *)malloc(sizeof(double) * (n_tok * H + 1));
    double *dGq = (double *)calloc(n_tok * H + 1, sizeof(double));
    double *dGk = (double *)calloc(n_tok * H + 1, sizeof(double));
    sla_oracle_head_softmax(lq, n_tok, H, Gq);
    sla_oracle_head_softmax(lk, n_tok, H, Gk);
    /* RETNET's log gamma_h is shared by every (b,t): per-(b,h) partial sums, added up at the end. */
    double *dgamma_part = (double *)calloc((long)B * H + 1, sizeof(double));
    int nseg = (T + SEG - 1) / SEG;

#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < H; ++h) {
            double *ck = (double *)malloc(sizeof(double) * sdim * (nseg + 1)); /* S before each segment */
            double *buf = (double *)malloc(sizeof(double) * sdim * (SEG + 1)); /* S_{t-1}..S_t inside one */
            double *S = (double *)calloc(sdim, sizeof(double));
            double *dS = (double *)calloc(sdim, sizeof(double));
            double *a = (double *)malloc(sizeof(double) * d_k);
            double *qw = (double *)malloc(sizeof(double) * d_k);
            double *kw = (double *)malloc(sizeof(double) * d_k);
            double *vw = (double *)malloc(sizeof(double) * d_v);
            double *rr = (double *)malloc(sizeof(double) * d_v * SEG);       /* GDN residuals r_t */
            double *dqw = (double *)malloc(sizeof(double) * d_k);
            double *dkw = (double *)malloc(sizeof(double) * d_k);
            double *dvw = (double *)malloc(sizeof(double) * d_v);
            double *du = (double *)malloc(sizeof(double) * d_v);
            if (h0) memcpy(S, h0 + ((long)b * H + h) * sdim, sizeof(double) * sdim);

            /* forward sweep: keep the state at every segment boundary */
            for (int t = 0; t < T; ++t) {
                if (t % SEG == 0) memcpy(ck + (long)(t / SEG) * sdim, S, sizeof(double) * sdim);
                long bt = (long)b * T + t, row = bt * H + h;
                decay_factors(variant, log_decay, bt, H, h, d_k, a);
                gated_operands(variant, d_k, d_v, scale, Gq[row], Gk[row],
                               q + row * d_k, k + row * d_k, v + row * d_v, qw, kw, vw);
                state_step(variant, d_k, d_v, a, beta ? beta[row] : 0.0, kw, vw, S, NULL);
            }
            if (dht) memcpy(dS, dht + ((long)b * H + h) * sdim, sizeof(double) * sdim);

            for (int s = nseg - 1; s >= 0; --s) {
                int t0 = s * SEG, t1 = (t0 + SEG < T) ? t0 + SEG : T;
                /* re-derive S_{t0-1} .. S_{t1-1}: buf[i] = state before token t0+i */
                memcpy(buf, ck + (long)s * sdim, sizeof(double) * sdim);
                for (int t = t0; t < t1; ++t) {
                    long bt = (long)b * T + t, row = bt * H + h;
                    double *Sn = buf + (long)(t - t0 + 1) * sdim;
                    memcpy(Sn, buf + (long)(t - t0) * sdim, sizeof(double) * sdim);
                    decay_factors(variant, log_decay, bt, H, h, d_k, a);
                    gated_operands(variant, d_k, d_v, scale, Gq[row], Gk[row],
                                   q + row * d_k, k + row * d_k, v + row * d_v, qw, kw, vw);
                    state_step(variant, d_k, d_v, a, beta ? beta[row] : 0.0, kw, vw, Sn,
                               rr + (long)(t - t0) * d_v);
                }
                for (int t = t1 - 1; t >= t0; --t) {
                    long bt = (long)b * T + t, row = bt * H + h;
                    const double *Sp = buf + (long)(t - t0) * sdim;       /* S_{t-1} */
                    const double *St = buf + (long)(t - t0 + 1) * sdim;   /* S_t     */
                    const double *dOt = dO + row * d_v;
                    const double *qt = q + row * d_k, *kt = k + row * d_k, *vt = v + row * d_v;
                    decay_factors(variant, log_decay, bt, H, h, d_k, a);
                    gated_operands(variant, d_k, d_v, scale, Gq[row], Gk[row], qt, kt, vt, qw, kw, vw);

                    /* o_t = qw S_t */
                    for (int d = 0; d < d_k; ++d) {
                        double acc = 0.0;
                        for (int j = 0; j < d_v; ++j) {
                            acc += dOt[j] * St[d * d_v + j];
                            dS[d * d_v + j] += qw[d] * dOt[j];
                        }
                        dqw[d] = acc;
                    }
                    /* now dS = dL/dS_t in full */
                    double dg_scalar = 0.0;
                    if (variant != SLA_ORACLE_GDN) {
                        /* S_t = diag(a) S_{t-1} + kw^T vw */
                        for (int j = 0; j < d_v; ++j) dvw[j] = 0.0;
                        for (int d = 0; d < d_k; ++d) {
                            double acck = 0.0, acca = 0.0;
                            for (int j = 0; j < d_v; ++j) {
                                double g = dS[d * d_v + j];
                                acck += g * vw[j];
                                dvw[j] += kw[d] * g;
                                acca += g * Sp[d * d_v + j];
                                dS[d * d_v + j] = a[d] * g;               /* -> dL/dS_{t-1} */
                            }
                            dkw[d] = acck;
                            double dg = acca * a[d];                      /* d/d(log a) */
                            if (variant == SLA_ORACLE_GLA) {
                                if (dlog_decay) dlog_decay[row * d_k + d] = dg;
                            } else {
                                dg_scalar += dg;
                            }
                        }
                        if (variant == SLA_ORACLE_RETNET) dgamma_part[(long)b * H + h] += dg_scalar;
                        /* kw = Gk k ; vw = v */
                        double dotk = 0.0;
                        for (int d = 0; d < d_k; ++d) {
                            dotk += kt[d] * dkw[d];
                            if (dk) dk[row * d_k + d] = Gk[row] * dkw[d];
                        }
                        dGk[row] = dotk;
                        if (dv) for (int j = 0; j < d_v; ++j) dv[row * d_v + j] = dvw[j];
                    } else {
                        /* Sbar = a S_{t-1}; r = vw - kw Sbar; u = beta r; S_t = Sbar + kw^T u */
                        const double *r = rr + (long)(t - t0) * d_v;
                        double bta = beta[row], al = a[0];
                        double dbt = 0.0;
                        for (int j = 0; j < d_v; ++j) {
                            double acc = 0.0;
                            for (int d = 0; d < d_k; ++d) acc += kw[d] * dS[d * d_v + j];
                            du[j] = acc;
                            dbt += acc * r[j];
                        }
                        if (dbeta) dbeta[row] = dbt;
                        for (int d = 0; d < d_k; ++d) {
                            double acc = 0.0;
                            for (int j = 0; j < d_v; ++j) {
                                double dr = bta * du[j];
                                /* from kw^T u and from -kw Sbar inside r */
                                acc += dS[d * d_v + j] * (bta * r[j]) - dr * (al * Sp[d * d_v + j]);
                            }
                            dkw[d] = acc;
                        }
                        for (int d = 0; d < d_k; ++d)
                            for (int j = 0; j < d_v; ++j) {
                                double dSbar = dS[d * d_v + j] - kw[d] * (bta * du[j]);
                                dg_scalar += dSbar * Sp[d * d_v + j];
                                dS[d * d_v + j] = al * dSbar;             /* -> dL/dS_{t-1} */
                            }
                        if (dlog_decay) dlog_decay[row] = dg_scalar * al;
                        /* kw = k ; vw = Gk v ; dvw = beta du */
                        double dotv = 0.0;
                        for (int j = 0; j < d_v; ++j) {
                            double dvwj = bta * du[j];
                            dotv += vt[j] * dvwj;
                            if (dv) dv[row * d_v + j] = Gk[row] * dvwj;
                        }
                        dGk[row] = dotv;
                        if (dk) for (int d = 0; d < d_k; ++d) dk[row * d_k + d] = dkw[d];
                    }
                    /* qw = scale Gq q */
                    double dotq = 0.0;
                    for (int d = 0; d < d_k; ++d) {
                        dotq += qt[d] * dqw[d];
                        if (dq) dq[row * d_k + d] = scale * Gq[row] * dqw[d];
                    }
                    dGq[row] = scale * dotq;
                }
            }
            if (dh0) memcpy(dh0 + ((long)b * H + h) * sdim, dS, sizeof(double) * sdim);
            free(ck); free(buf); free(S); free(dS); free(a); free(qw); free(kw); free(vw);
            free(rr); free(dqw); free(dkw); free(dvw); free(du);
        }
    }
    if (variant == SLA_ORACLE_RETNET && dlog_decay) {
        for (int h = 0; h < H; ++h) {
            double acc = 0.0;
            for (int b = 0; b < B; ++b) acc += dgamma_part[(long)b * H + h];
            dlog_decay[h] = acc;
        }
    }
    if (dlq) head_softmax_backward(Gq, dGq, n_tok, H, dlq);
    if (dlk) head_softmax_backward(Gk, dGk, n_tok, H, dlk);
    free(Gq); free(Gk); free(dGq); free(dGk); free(dgamma_part);
    return 0;
}
