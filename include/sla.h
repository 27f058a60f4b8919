/*
 * sla.h — C ABI of the B200 (sm_100a) Softmax-Linear-Attention hot path.
 *
 * The layer (paper Sec. 3.2): per token the H head-gate logits are turned into gates by a
 * softmax over the heads (Eq. 4); every head then runs a gated linear recurrence on a
 * d_k x d_v state (Eq. 5-6) in one of three instantiations (Eq. 10-16); the per-head
 * read-outs are concatenated (Eq. 7, without W^O).  Training-time evaluation is chunkwise
 * ("Chunkwise Parallel Training"): dense products inside a chunk, the state passed between
 * chunks.  The result does not depend on the chunk size.
 *
 * Conventions for every call
 *  - All tensor pointers are DEVICE pointers owned by the caller, dense, row-major, aligned
 *    to 16 bytes.  The library allocates no device memory in sla_forward / sla_backward /
 *    sla_decode_step: scratch comes from the caller's `workspace`
 *    (size from sla_plan_workspace_bytes); the library keeps nothing in it between calls.
 *  - Work is enqueued on `cuda_stream` (a cudaStream_t cast to void*, NULL = default stream)
 *    and the call returns without waiting.
 *  - Every function returns an sla_status; nothing throws or aborts across the boundary.
 *    Shapes the kernels do not cover are refused at sla_plan_create (SLA_ERR_UNSUPPORTED);
 *    a device that is not sm_100 is refused with SLA_ERR_ARCH.  There is no CPU fallback.
 *  - io dtype (q, k, v, o and their gradients): fp32 or bf16.  Log-decay, beta, gate logits,
 *    states and their gradients are always fp32.  Accumulation is fp32.
 *
 * Shapes:  q, k [B,T,H,d_k]   v, o, dO [B,T,H,d_v]   gate logits [B,T,H]
 *          log_decay  RETNET [H] (log gamma_h) | GLA [B,T,H,d_k] | GDN [B,T,H]   (all <= 0)
 *          beta       GDN [B,T,H] in (0,1), else NULL
 *          h0, ht, dht, dh0 [B,H,d_k,d_v]  (row = key dimension)
 *
 * Decay range.  The recurrences of Eq. 10-16 are defined for every log_decay <= 0, but the chunkwise kernels
 * split the decay between two tokens of a chunk as e^{b_i} * e^{-b_j} (b = cumulative log-decay inside the chunk)
 * and keep both factors in fp32 / bf16.  They are exact re-associations as long as the cumulative log-decay over
 * one chunk stays above -SLA_MAX_CHUNK_DECAY (about -1.2 per token at the largest chunk of 64, -4.7 per token at
 * chunk 16).  Every chunk is checked on the device: a chunk beyond the limit raises the plan's status word, the
 * call still completes (its results for that sequence are then not meaningful and may hold inf or NaN), and the next
 * sla_plan_poll returns SLA_ERR_RANGE.  A smaller chunk widens the range; decode steps have no limit.
 */
#ifndef SLA_H
#define SLA_H

#define SLA_MAX_CHUNK_DECAY 76.0f    /* see "Decay range" above */

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sla_plan sla_plan;          /* opaque host object */

typedef enum {
    SLA_OK = 0,
    SLA_ERR_INVALID_ARG = 1,   /* null / misaligned pointer, bad struct_size, bad enum        */
    SLA_ERR_UNSUPPORTED = 2,   /* a shape or option the kernels do not cover                   */
    SLA_ERR_WORKSPACE = 3,     /* workspace NULL or smaller than sla_plan_workspace_bytes      */
    SLA_ERR_ARCH = 4,          /* current device is not compute capability 10.x                */
    SLA_ERR_CUDA = 5,          /* a CUDA runtime call failed (launch, attribute, allocation)   */
    SLA_ERR_TIMEOUT = 6,       /* a bounded device-side wait expired (reported by sla_plan_poll) */
    SLA_ERR_RANGE = 7          /* a chunk's cumulative log-decay left the range the chunkwise kernels can
                                  represent (reported by sla_plan_poll; see "Decay range" below)       */
} sla_status;

typedef enum { SLA_RETNET = 0, SLA_GLA = 1, SLA_GDN = 2 } sla_variant;
typedef enum { SLA_FP32 = 0, SLA_BF16 = 1 } sla_dtype;

/* flags */
#define SLA_FLAG_FORCE_GENERIC 1u  /* use the fp32 CUDA-core chunk kernels even where a tensor-core
                                      kernel exists for the shape (same function, other rounding) */
#define SLA_FLAG_SAVE_FOR_BACKWARD 2u
/* Training plans: sla_forward also leaves in its workspace what the chunkwise backward pass would
 * otherwise recompute first (Softmax-GLA: the state before every chunk; Softmax-GDN: per chunk the
 * state, the corrected values U and the inverse T of the WY form).  sla_plan_workspace_bytes then
 * reports the backward size for the forward too.  A following sla_backward on the same plan that is
 * given the same workspace, the same q, k, v, log_decay, beta, logits and h0 pointers and the same
 * stream as that sla_forward uses what was left and skips its recomputation; any other call
 * recomputes, so results never depend on the flag.  Contract: between the two calls the caller
 * changes neither the workspace nor the contents of those inputs.  Ignored (nothing is left, the
 * backward recomputes) by the fp32 CUDA-core kernels and where the forward cuts long sequences
 * into segments. */

typedef struct {
    uint32_t struct_size;      /* sizeof(sla_desc) */
    int32_t  variant;          /* sla_variant */
    int32_t  io_dtype;         /* sla_dtype   */
    int32_t  B, T, H;          /* batch, tokens, heads (1 <= H <= 32) */
    int32_t  d_k, d_v;         /* per-head key / value width: multiples of 16, <= 128 */
    int32_t  chunk;            /* chunk size C: 16, 32 or 64; T need not be a multiple of it */
    float    scale;            /* multiplies q (the paper's linear forms have none: use 1) */
    uint32_t flags;
} sla_desc;

/* Validates the description against the current CUDA device and builds a plan.
 * The plan is bound to that device; it owns one small device status word and nothing else. */
sla_status sla_plan_create(sla_plan **out, const sla_desc *desc);
sla_status sla_plan_destroy(sla_plan *plan);

/*
 * Packed variable-length batches (training data packed to a fixed token budget; the paper trains at a maximum sequence
 * length of 4096 on such data).  For a plan with B == 1 the T tokens are n_seq sequences laid one after another:
 * sequence s covers tokens cu_seqlens[s] .. cu_seqlens[s+1]-1 (cu_seqlens: HOST array of n_seq + 1 ascending offsets,
 * first 0, last T; no empty sequence).  After this call sla_forward / sla_backward on the plan run the recurrence of
 * Eq. 5-6 per sequence: the state starts from h0[s] (or zero) at each sequence's first token, chunks are cut from each
 * sequence's own start and never straddle a boundary, and h0, ht, dht, dh0 have the shape [n_seq,H,d_k,d_v].
 * sla_plan_workspace_bytes changes with the table: query it again.  n_seq == 0 returns the plan to a regular batch.
 * The plan copies the table (and owns a few small device arrays for it until it is destroyed or the table replaced);
 * this is a set-up call, not to be made between a forward and its backward pass.  Only plans that select the
 * tensor-core kernels (bf16, d_k and d_v 128 or 64, chunk 64) take a table: SLA_ERR_UNSUPPORTED otherwise.  Calls on one
 * plan must be ordered on one stream (the per-sequence tensor maps are uploaded in stream order).
 */
sla_status sla_plan_set_sequences(sla_plan *plan, const int32_t *cu_seqlens, int32_t n_seq);

/* Bytes of caller-provided scratch that sla_forward / sla_backward need for this plan (it depends on the kernels the
 * plan selects; 0 means none is needed and the workspace pointer may then be NULL). */
sla_status sla_plan_workspace_bytes(const sla_plan *plan, size_t *forward_bytes, size_t *backward_bytes);

/* Synchronises with nothing; copies the plan's device status word back (on the legacy default
 * stream, so call it after synchronising the stream that ran the work) and clears it.  SLA_ERR_TIMEOUT if a
 * kernel gave up a bounded wait since the last poll; else SLA_ERR_RANGE if a chunk's cumulative log-decay
 * was beyond SLA_MAX_CHUNK_DECAY; SLA_OK otherwise. */
sla_status sla_plan_poll(sla_plan *plan);

/* Diagnostic of the failure path (the paper has no counterpart): enqueues a one-warp kernel whose bounded wait can
 * never be satisfied (limit 2 ms).  It gives up, raises the plan's status word like a tensor-core kernel whose wait
 * expired, and returns normally: after synchronising the stream, sla_plan_poll reports SLA_ERR_TIMEOUT once and the
 * context stays usable. */
sla_status sla_plan_selftest_timeout(sla_plan *plan, void *cuda_stream);

/* Number of kernel launches the last sla_forward / sla_backward / sla_decode_step on this plan
 * enqueued (for launch accounting in benchmarks). */
int32_t sla_plan_last_launch_count(const sla_plan *plan);

/*
 * Optional per-kernel timing (measurement aid; the paper has no counterpart).  While enabled, every
 * entry point records one CUDA event before its first kernel and one after each kernel on the
 * launch stream.  sla_plan_kernel_timing_collect waits for the last recorded event, folds the
 * elapsed times into per-kernel totals (by kernel name) and returns how many names there are;
 * sla_plan_kernel_timing_get reads one total.  `name` points at a string literal owned by the library.
 * Enabling (or disabling) clears the totals.  Events are created on first use and reused.
 */
sla_status sla_plan_set_kernel_timing(sla_plan *plan, int32_t enable);
sla_status sla_plan_kernel_timing_collect(sla_plan *plan, int32_t *n_kernels);
sla_status sla_plan_kernel_timing_get(const sla_plan *plan, int32_t index, const char **name,
                                      int32_t *launches, float *total_ms);

const char *sla_status_string(sla_status s);

/*
 * Forward (Eq. 4-7 with Eq. 10-16, evaluated chunkwise).
 *   gates   Gq = softmax_H(gq_logits), Gk = softmax_H(gk_logits)              (Eq. 4)
 *   RETNET  S_t = gamma_h S_{t-1} + (Gk k_t)^T v_t                            (Eq. 10)
 *   GLA     S_t = diag(exp(log_decay_t)) S_{t-1} + (Gk k_t)^T v_t             (Eq. 12)
 *   GDN     Sb = exp(log_decay_t) S_{t-1};  u = beta_t (Gk v_t - k_t Sb);  S_t = Sb + k_t^T u   (Eq. 14-15)
 *   o_t     = (scale Gq q_t) S_t, heads concatenated along the last axes      (Eq. 6-7, 11, 13, 16)
 * h0 may be NULL (zero state); ht may be NULL (final state not wanted).
 * gq_logits and gk_logits may alias.  Outputs must not alias inputs.
 * With T == 0 (and B > 0) there is nothing to read: o is not touched and ht, if given, receives h0 (or zeros).
 */
sla_status sla_forward(sla_plan *plan,
                       const void *q, const void *k, const void *v,
                       const float *log_decay, const float *beta,
                       const float *gq_logits, const float *gk_logits,
                       const float *h0,
                       void *o, float *ht,
                       void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Backward of sla_forward (the paper states no gradients; these are the chain rule applied to
 * Eq. 4-7, 10-16, evaluated chunkwise with the chunk states recomputed).
 * Inputs: the primal inputs of sla_forward, dO (io dtype) and optionally dht (gradient
 * flowing into the final state).  Outputs, written in full (not accumulated): dq, dk, dv
 * (io dtype); dlog_decay fp32 in the shape of log_decay (must be NULL for RETNET, whose gamma_h
 * is a constant); dbeta fp32 [B,T,H] (GDN, else NULL); dgq_logits, dgk_logits fp32 [B,T,H];
 * dh0 fp32 or NULL.  dgq_logits and dgk_logits must not alias each other.
 */
sla_status sla_backward(sla_plan *plan,
                        const void *q, const void *k, const void *v,
                        const float *log_decay, const float *beta,
                        const float *gq_logits, const float *gk_logits,
                        const float *h0,
                        const void *dO, const float *dht,
                        void *dq, void *dk, void *dv,
                        float *dlog_decay, float *dbeta,
                        float *dgq_logits, float *dgk_logits, float *dh0,
                        void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * One recurrent step (Eq. 5-6 / 10-16 at a single t) for Bdec sequences on a caller-held
 * state, updated in place.  Uses the plan's variant, dtype, H, d_k, d_v and scale; the plan's
 * B, T and chunk are ignored.  q_t, k_t [Bdec,H,d_k]; v_t, o_t [Bdec,H,d_v];
 * log_decay_t RETNET [H] | GLA [Bdec,H,d_k] | GDN [Bdec,H]; beta_t [Bdec,H] (GDN);
 * logits [Bdec,H]; state [Bdec,H,d_k,d_v] fp32.  Needs no workspace.
 */
sla_status sla_decode_step(sla_plan *plan, int32_t Bdec,
                           const void *q_t, const void *k_t, const void *v_t,
                           const float *log_decay_t, const float *beta_t,
                           const float *gq_logits_t, const float *gk_logits_t,
                           float *state, void *o_t, void *cuda_stream);

/*
 * Gate score projections (Eq. 4: G^Q = softmax(Q W_GQ), G^K = softmax(K W_GK), W in R^{d x H} with d the per-head
 * width).  The paper leaves open what a d-wide projection is applied to in a multi-head layer; its parameter count
 * (about 0.05M for 24 layers at hidden 1024 with 4 heads, i.e. d = 256) fixes d as the per-head width, and the reading
 * taken here is that head h scores itself through column h:
 *     gq_logits[b,t,h] = sum_c q[b,t,h,c] w_gq[c,h]          gk_logits[b,t,h] = sum_c k[b,t,h,c] w_gk[c,h]
 * q, k are the tensors handed to sla_forward (d = d_k); w_gq, w_gk fp32 [d_k,H] row-major; the logits feed sla_forward
 * unchanged.  One streaming pass over q and k; needs no workspace.
 */
sla_status sla_gate_scores_forward(sla_plan *plan, const void *q, const void *k,
                                   const float *w_gq, const float *w_gk,
                                   float *gq_logits, float *gk_logits, void *cuda_stream);
/*
 * Reverse of sla_gate_scores_forward (chain rule of Eq. 4), run AFTER sla_backward on its outputs: dgq_logits,
 * dgk_logits are sla_backward's logit gradients; dq, dk are sla_backward's dq, dk and are updated in place,
 *     dq[b,t,h,:] += dgq_logits[b,t,h] w_gq[:,h]             dk[b,t,h,:] += dgk_logits[b,t,h] w_gk[:,h]
 * (q and k reach the loss on two routes); dw_gq, dw_gk fp32 [d_k,H] are written in full,
 *     dw_gq[c,h] = sum_{b,t} dgq_logits[b,t,h] q[b,t,h,c]    (same for k),
 * summed in a fixed order (identical bits on every run).  Workspace: sla_plan_gate_scores_workspace_bytes.
 */
sla_status sla_plan_gate_scores_workspace_bytes(const sla_plan *plan, size_t *bytes);
sla_status sla_gate_scores_backward(sla_plan *plan, const void *q, const void *k,
                                    const float *w_gq, const float *w_gk,
                                    const float *dgq_logits, const float *dgk_logits,
                                    void *dq, void *dk, float *dw_gq, float *dw_gk,
                                    void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Output projection (Eq. 7: y_t = Concat_h(o_{t,h}) W^O).  o [B,T,H*d_v] is sla_forward's output (the heads of a
 * token are already side by side), w_o [H*d_v, d_model] row-major, y [B,T,d_model]; all bf16 (the plan's io dtype
 * must be SLA_BF16: the products run on the bf16 tensor cores with fp32 accumulation; fp32 plans get
 * SLA_ERR_UNSUPPORTED), d_model and H*d_v multiples of 8.  A dense contraction: one persistent tcgen05 kernel.
 * Needs no workspace.  y may not alias o.
 */
sla_status sla_out_proj_forward(sla_plan *plan, const void *o, const void *w_o, int32_t d_model, void *y,
                                void *cuda_stream);
/*
 * Reverse of sla_out_proj_forward: d_o [B,T,H*d_v] (bf16; it is the dO that sla_backward takes) = dy W^O^T and
 * dw_o fp32 [H*d_v, d_model] = sum over tokens of o_t^T dy_t, both written in full; the token sum of dw_o runs in a
 * fixed order inside one accumulator per element (identical bits on every run).  Two launches, no workspace.
 */
sla_status sla_out_proj_backward(sla_plan *plan, const void *o, const void *w_o, const void *dy, int32_t d_model,
                                 void *d_o, float *dw_o, void *cuda_stream);

/*
 * Feature map of the Gated-DeltaNet instantiation (Experimental setup: GDN uses "the short-convolution module" and SiLU
 * as activation; RetNet and GLA use the identity and need none of this).  The paper names the module and cites Gated
 * DeltaNet for it; what is computed here is that published design: per channel a causal convolution over time,
 * SiLU, and - for q and k - L2 normalisation over the d features of each head:
 *     y[b,t,c] = sum_{j<K} w[c,j] x[b,t-(K-1)+j,c]   (tokens before the sequence start read as zero; no bias)
 *     z = y * sigmoid(y)
 *     out[b,t,h,:] = z[b,t,h,:] / sqrt(sum_d z[b,t,h,d]^2 + SLA_SHORTCONV_EPS)   if normalize != 0, else out = z
 * x, out [B,T,H,d] in the plan's io dtype (d = the per-head width of THIS tensor, a multiple of 16 up to 128: d_k for
 * q and k, d_v for v); w fp32 [H*d, K], 1 <= K <= 4.  One call per tensor: q and k with normalize = 1, v with 0; the
 * outputs are what sla_forward takes.  out may not alias x.  Uses the plan's B, T, H and io dtype.
 */
#define SLA_SHORTCONV_EPS 1e-6f
sla_status sla_shortconv_forward(sla_plan *plan, const void *x, const float *w, int32_t d, int32_t K,
                                 int32_t normalize, void *out, void *cuda_stream);
/*
 * Reverse of sla_shortconv_forward: from dout (gradient with respect to out, e.g. sla_backward's dq) to
 * dx [B,T,H,d] (io dtype) and dw fp32 [H*d, K], both written in full; y is recomputed from x, nothing is kept from
 * the forward call.  dw is summed in a fixed order.  Workspace: sla_plan_shortconv_workspace_bytes(plan, d).
 */
sla_status sla_plan_shortconv_workspace_bytes(const sla_plan *plan, int32_t d, size_t *bytes);
sla_status sla_shortconv_backward(sla_plan *plan, const void *x, const float *w, int32_t d, int32_t K,
                                  int32_t normalize, const void *dout, void *dx, float *dw,
                                  void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Multi-token decode: n_tokens consecutive recurrent steps (Eq. 5-6 / 10-16) per sequence in one call - what a
 * serving loop needs when several tokens of a sequence are known at once (chunked prefill of a short prompt tail,
 * verification of speculated tokens).  Token t of sequence b reads the state token t-1 left; the state travels
 * from and to memory once per call instead of once per token, every token's output is produced.  Same arithmetic,
 * in the same order, as n_tokens calls of sla_decode_step (the results are equal bit for bit).
 * q, k [Bdec,n_tokens,H,d_k]; v, o [Bdec,n_tokens,H,d_v]; log_decay RETNET [H] | GLA [Bdec,n_tokens,H,d_k] |
 * GDN [Bdec,n_tokens,H]; beta [Bdec,n_tokens,H] (GDN); logits [Bdec,n_tokens,H]; state [Bdec,H,d_k,d_v] fp32,
 * updated in place.  n_tokens == 1 is sla_decode_step.  Needs no workspace.
 */
sla_status sla_decode_steps(sla_plan *plan, int32_t Bdec, int32_t n_tokens,
                            const void *q, const void *k, const void *v,
                            const float *log_decay, const float *beta,
                            const float *gq_logits, const float *gk_logits,
                            float *state, void *o, void *cuda_stream);

/*
 * sla_forward with built-in scratch (an addition of this library; the paper has no counterpart).
 *
 * Some callers are not allowed to obtain device memory at the point where they run the layer: a
 * plugin executing inside a host runtime that owns the allocator and forbids allocation in its
 * execute callback, a latency-critical serving loop whose memory budget is frozen after start-up,
 * or a process whose device memory has been reserved in full by another pool, where a fresh
 * allocation would fail.  Such callers cannot provide the `workspace` that sla_forward wants.
 * This entry point computes exactly what sla_forward computes (always with the fp32 CUDA-core chunk
 * kernels) and keeps its scratch in a fixed array of SLA_NOALLOC_SCRATCH_BYTES that is part of the
 * library image: every GPU on which the library is loaded holds that array until the process
 * exits.  The call itself allocates and frees nothing: no cudaMalloc, no cudaFree, no allocating library
 * routine.  Inputs and outputs are still the caller's, with the meanings, layouts and rules of
 * sla_forward.
 *
 *  - Size limit: if the forward workspace of the fp32 CUDA-core kernels for this shape (what
 *    sla_plan_workspace_bytes reports for a plan created with SLA_FLAG_FORCE_GENERIC) exceeds
 *    SLA_NOALLOC_SCRATCH_BYTES the call does nothing and returns SLA_ERR_WORKSPACE.
 *  - First call on a device: looks up the device address of the array (one runtime query, made
 *    with that device current; result cached per device).  Where the CUDA runtime loads modules
 *    lazily, this query is also the moment the driver places the array on that GPU, so free device
 *    memory drops by SLA_NOALLOC_SCRATCH_BYTES once, here, and never again.  Make this first call
 *    at start-up, outside any stream capture.
 *  - The array is shared by every plan and every call in the process and keeps what the last call
 *    left in it.  The kernels write each part of it before reading it, so stale contents are never
 *    used; but two calls whose kernels may overlap on the GPU (different streams without
 *    ordering, or several host threads) race on it.  Serialise them.
 *  - The plan must belong to the current device (SLA_ERR_INVALID_ARG otherwise).
 */
#define SLA_NOALLOC_SCRATCH_BYTES (32u << 20)
sla_status sla_forward_noalloc(sla_plan *plan,
                               const void *q, const void *k, const void *v,
                               const float *log_decay, const float *beta,
                               const float *gq_logits, const float *gk_logits,
                               const float *h0,
                               void *o, float *ht, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SLA_H */
