/*
 * sla_oracle.h — TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, fp64 CPU statement of what the Softmax-Linear-Attention layer
 * computes, written token by token from the paper's recurrent equations.  Only
 * the tests, the smoke check and the benchmark's CPU-baseline leg may call it;
 * it shares no code with the CUDA library and the CUDA library never calls it.
 *
 * Tensor layouts (all dense, row-major, fp64):
 *   q, k        [B, T, H, d_k]        v, o, dO      [B, T, H, d_v]
 *   lq, lk      [B, T, H]   head-gate logits for the query / key side
 *   log_decay   RETNET: [H]  (log gamma_h)     GLA: [B, T, H, d_k]     GDN: [B, T, H]
 *   beta        GDN: [B, T, H]   (ignored otherwise, may be NULL)
 *   h0, ht      [B, H, d_k, d_v]   initial / final state, NULL = zeros / not wanted
 *
 * Pins (tests/test_oracle_*.py): gates against closed forms and the limits of
 * Thm 3.2 / Thm 3.3; the recurrence against a brute-force quadratic form with
 * an explicit decay mask (Eq. 3, App. A) and against unrolled transition-matrix
 * products for the delta rule; the backward sweep against central finite
 * differences of the forward.  No function here is "parity unpinned".
 */
#ifndef SLA_ORACLE_H
#define SLA_ORACLE_H

#ifdef __cplusplus
extern "C" {
#endif

enum { SLA_ORACLE_RETNET = 0, SLA_ORACLE_GLA = 1, SLA_ORACLE_GDN = 2 };

/* Threads the (b,h) loops will use. */
int sla_oracle_num_threads(void);

/* Eq. 4: softmax over the H heads of one token, for n_tok tokens.
 * logits, gates: [n_tok, H]. */
void sla_oracle_head_softmax(const double *logits, long n_tok, int H, double *gates);

/* Eq. 5-7 with the decay / delta-rule instantiations of Eq. 10-16.
 * Returns 0, or -1 on a bad argument. */
int sla_oracle_forward(int variant, int B, int T, int H, int d_k, int d_v, double scale,
                       const double *q, const double *k, const double *v,
                       const double *log_decay, const double *beta,
                       const double *lq, const double *lk, const double *h0,
                       double *o, double *ht);

/* Reverse sweep of sla_oracle_forward.  dO [B,T,H,d_v]; dht nullable.
 * Outputs (each nullable): dq, dk, dv in the shapes of their primals;
 * dlog_decay in the shape of log_decay (RETNET: [H], summed over b,t);
 * dbeta [B,T,H] (GDN); dlq, dlk [B,T,H]; dh0 [B,H,d_k,d_v]. */
int sla_oracle_backward(int variant, int B, int T, int H, int d_k, int d_v, double scale,
                        const double *q, const double *k, const double *v,
                        const double *log_decay, const double *beta,
                        const double *lq, const double *lk, const double *h0,
                        const double *dO, const double *dht,
                        double *dq, double *dk, double *dv,
                        double *dlog_decay, double *dbeta,
                        double *dlq, double *dlk, double *dh0);

/* One recurrent step for Bdec sequences (the T = 1 case on a caller-held
 * state).  q_t, k_t [Bdec,H,d_k]; v_t, o_t [Bdec,H,d_v]; log_decay_t RETNET [H],
 * GLA [Bdec,H,d_k], GDN [Bdec,H]; beta_t [Bdec,H]; lq_t, lk_t [Bdec,H];
 * state [Bdec,H,d_k,d_v] updated in place. */
int sla_oracle_decode_step(int variant, int Bdec, int H, int d_k, int d_v, double scale,
                           const double *q_t, const double *k_t, const double *v_t,
                           const double *log_decay_t, const double *beta_t,
                           const double *lq_t, const double *lk_t,
                           double *state, double *o_t);

/* Eq. 4, score projections: s[t,h] = sum_c x[t,h,c] W[c,h]; x [n_tok,H,d], W [d,H], s [n_tok,H].
 * Pinned by: an einsum of the same contraction, H = 1 (a plain matrix-vector product), lambda*W sharpening the gates
 * to one-hot (Thm 3.2), finite differences of the whole layer with respect to W and through x. */
void sla_oracle_gate_scores(long n_tok, int H, int d, const double *x, const double *W, double *s);
/* dx += ds W^T per head (accumulated), dW = sum_t ds x (overwritten). */
void sla_oracle_gate_scores_backward(long n_tok, int H, int d, const double *x, const double *W,
                                     const double *ds, double *dx, double *dW);
/* Eq. 7: y = o W^O over the concatenated head outputs; o [n_tok,K], W [K,N], y [n_tok,N]; and its reverse. */
void sla_oracle_out_proj(long n_tok, int K, int N, const double *o, const double *W, double *y);
void sla_oracle_out_proj_backward(long n_tok, int K, int N, const double *o, const double *W, const double *dy,
                                  double *d_o, double *dW);

/* Feature map of the Gated-DeltaNet instantiation: depthwise causal convolution over time (K taps, w [C,K], C = H*d
 * channels), SiLU, and with normalize != 0 L2 normalisation over the d features of each head (eps inside the root).
 * x, out [B,T,C].  Pinned by: a library convolution per channel, K = 1 with unit weight = SiLU itself, unit row norms,
 * causality, finite differences of the reverse sweep. */
void sla_oracle_shortconv(int B, int T, int H, int d, int K, int normalize, double eps,
                          const double *x, const double *w, double *out);
void sla_oracle_shortconv_backward(int B, int T, int H, int d, int K, int normalize, double eps,
                                   const double *x, const double *w, const double *dout,
                                   double *dx, double *dw);

/* n_tok consecutive recurrent steps per sequence on a caller-held state (multi-token decode).
 * q, k [Bdec,n_tok,H,d_k]; v, o [Bdec,n_tok,H,d_v]; log_decay RETNET [H], GLA [Bdec,n_tok,H,d_k],
 * GDN [Bdec,n_tok,H]; beta, lq, lk [Bdec,n_tok,H]; state [Bdec,H,d_k,d_v] updated in place.
 * Pinned by: equals n_tok calls of sla_oracle_decode_step on the token slices. */
int sla_oracle_decode_steps(int variant, int Bdec, int n_tok, int H, int d_k, int d_v, double scale,
                            const double *q, const double *k, const double *v,
                            const double *log_decay, const double *beta,
                            const double *lq, const double *lk,
                            double *state, double *o);

#ifdef __cplusplus
}
#endif
#endif
