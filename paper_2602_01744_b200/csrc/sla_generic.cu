// Chunkwise Softmax-Linear-Attention on CUDA cores, fp32 arithmetic, for every variant and
// both I/O dtypes.  This is the precision path (fp32 I/O needs more than bf16 tensor-core
// operands give) and the path for shapes the tensor-core kernels do not cover.
//
// Per (batch, head) sequence and chunk of C tokens (local index i), with
//   b_i   inclusive cumulative log-decay inside the chunk (per key dimension for GLA),
//   qh_i = scale*Gq_i*q_i*exp(b_i),   kh_j = Gk_j*k_j*exp(-b_j)   (GDN: kh_j = k_j*exp(-b_j)),
//   S     state at the chunk start,
// the chunk computes  A = tril(qh kh^T),  O = A V + qh S,  S' = diag(exp(b_last)) S + kbar^T V
// with kbar_j = kh_j*exp(b_last)  (GDN: V is replaced by U = U0 - W S from the WY solve).
// All of these are exact re-associations of the recurrence (Eq. 5-6, 10-16).
#include "sla_generic.cuh"

namespace sla {
namespace {

using namespace detail;

// ------------------------------------------------------------------------------------------
// a1: head-softmax gates, HP lanes per token (HP = power of two >= H), max and sum by shuffles.
template <int HP>
__global__ void k_gate_fwd(const float *__restrict__ lq, const float *__restrict__ lk,
                           float *__restrict__ Gq, float *__restrict__ Gk, long n_tok, int H) {
    const float *l = blockIdx.y ? lk : lq;
    float *G = blockIdx.y ? Gk : Gq;
    long gt = (long)blockIdx.x * blockDim.x + threadIdx.x;
    long tok = gt / HP;
    int h = (int)(gt % HP);
    bool valid = tok < n_tok && h < H;
    float x = valid ? l[tok * H + h] : -INFINITY;
    float m = x;
#pragma unroll
    for (int o = HP / 2; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(FULL, m, o));
    float e = valid ? expf(x - m) : 0.f;
    float s = e;
#pragma unroll
    for (int o = HP / 2; o > 0; o >>= 1) s += __shfl_xor_sync(FULL, s, o);
    if (valid) G[tok * H + h] = e / s;
}

// gate backward: dl_h = G_h (dG_h - sum_h' G_h' dG_h')
template <int HP>
__global__ void k_gate_bwd(const float *__restrict__ Gq, const float *__restrict__ Gk,
                           const float *__restrict__ dGq, const float *__restrict__ dGk,
                           float *__restrict__ dlq, float *__restrict__ dlk, long n_tok, int H) {
    const float *G = blockIdx.y ? Gk : Gq;
    const float *dG = blockIdx.y ? dGk : dGq;
    float *dl = blockIdx.y ? dlk : dlq;
    long gt = (long)blockIdx.x * blockDim.x + threadIdx.x;
    long tok = gt / HP;
    int h = (int)(gt % HP);
    bool valid = tok < n_tok && h < H;
    float g = valid ? G[tok * H + h] : 0.f;
    float dg = valid ? dG[tok * H + h] : 0.f;
    float s = g * dg;
#pragma unroll
    for (int o = HP / 2; o > 0; o >>= 1) s += __shfl_xor_sync(FULL, s, o);
    if (valid) dl[tok * H + h] = g * (dg - s);
}

// ------------------------------------------------------------------------------------------
// a2: chunk-local inclusive cumulative log-decay.  grid (NT, B*H).
// A chunk whose cumulative log-decay is beyond the range of the e^{b}, e^{-b} factors raises STATUS_RANGE.
__global__ void k_cumdecay(Dims d, const float *__restrict__ log_decay, float *__restrict__ bcum, int *status) {
    int n = blockIdx.x, bh = blockIdx.y, b = bh / d.H, h = bh % d.H;
    int t0 = n * d.C, cn = min(d.C, d.T - t0);
    if (d.variant == SLA_GLA) {
        for (int dd = threadIdx.x; dd < d.dk; dd += blockDim.x) {
            float acc = 0.f;
            for (int i = 0; i < cn; ++i) {
                size_t idx = tok_row(d, b, t0 + i, h) * d.dk + dd;
                acc += log_decay[idx];
                bcum[idx] = acc;
            }
            if (acc < -SLA_MAX_CHUNK_DECAY) atomicOr(status, STATUS_RANGE);
        }
    } else if (threadIdx.x == 0) {
        float acc = 0.f;
        for (int i = 0; i < cn; ++i) {
            size_t row = tok_row(d, b, t0 + i, h);
            acc += (d.variant == SLA_RETNET) ? log_decay[h] : log_decay[row];
            bcum[row] = acc;
        }
        if (acc < -SLA_MAX_CHUNK_DECAY) atomicOr(status, STATUS_RANGE);
    }
}

// ------------------------------------------------------------------------------------------
// GDN WY preparation (per tile): L_ij = beta_i exp(b_i-b_j) (k_i.k_j), j<i; forward substitution
// (I+L)[W|U0] = [diag(beta exp(b)) K | diag(beta Gk) V].  One thread per right-hand-side column.
template <typename TIO>
__global__ void __launch_bounds__(256)
k_gdn_prepare(Dims d, const TIO *__restrict__ k, const TIO *__restrict__ v,
              const float *__restrict__ beta, const float *__restrict__ Gk,
              const float *__restrict__ bcum, float *__restrict__ Wout, float *__restrict__ U0out) {
    extern __shared__ float sm[];
    int n = blockIdx.x, bh = blockIdx.y, b = bh / d.H, h = bh % d.H;
    int t0 = n * d.C, cn = min(d.C, d.T - t0);
    int ldk = d.dk + 1, ldl = CMAX + 1, ldx = d.dk + d.dv;
    float *Ks = sm;                       // [CMAX][ldk]   raw keys
    float *Ls = Ks + CMAX * ldk;          // [CMAX][ldl]
    float *Xs = Ls + CMAX * ldl;          // [CMAX][ldx]
    float *bs = Xs + CMAX * ldx;          // [CMAX] cumulative log-decay
    float *bt = bs + CMAX;                // [CMAX] beta
    for (int i = threadIdx.x; i < CMAX; i += blockDim.x) {
        bool ok = i < cn;
        size_t row = ok ? tok_row(d, b, t0 + i, h) : 0;
        bs[i] = ok ? bcum[row] : 0.f;
        bt[i] = ok ? beta[row] : 0.f;
    }
    for (int idx = threadIdx.x; idx < CMAX * d.dk; idx += blockDim.x) {
        int i = idx / d.dk, dd = idx % d.dk;
        Ks[i * ldk + dd] = i < cn ? ldf(k, tok_row(d, b, t0 + i, h) * d.dk + dd) : 0.f;
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < CMAX * d.dk; idx += blockDim.x) {
        int i = idx / d.dk, dd = idx % d.dk;
        Xs[i * ldx + dd] = bt[i] * expf(bs[i]) * Ks[i * ldk + dd];
    }
    for (int idx = threadIdx.x; idx < CMAX * d.dv; idx += blockDim.x) {
        int i = idx / d.dv, j = idx % d.dv;
        float val = 0.f;
        if (i < cn) {
            size_t row = tok_row(d, b, t0 + i, h);
            val = bt[i] * Gk[row] * ldf(v, row * d.dv + j);
        }
        Xs[i * ldx + d.dk + j] = val;
    }
    for (int idx = threadIdx.x; idx < CMAX * CMAX; idx += blockDim.x) {
        int i = idx % CMAX, j = idx / CMAX;
        float acc = 0.f;
        if (j < i) {
            for (int dd = 0; dd < d.dk; ++dd) acc = fmaf(Ks[i * ldk + dd], Ks[j * ldk + dd], acc);
            acc *= bt[i] * expf(bs[i] - bs[j]);
        }
        Ls[i * ldl + j] = acc;
    }
    __syncthreads();
    for (int col = threadIdx.x; col < ldx; col += blockDim.x) {
        for (int i = 1; i < cn; ++i) {
            float acc = Xs[i * ldx + col];
            for (int j = 0; j < i; ++j) acc = fmaf(-Ls[i * ldl + j], Xs[j * ldx + col], acc);
            Xs[i * ldx + col] = acc;
        }
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < cn * d.dk; idx += blockDim.x) {
        int i = idx / d.dk, dd = idx % d.dk;
        Wout[tok_row(d, b, t0 + i, h) * d.dk + dd] = Xs[i * ldx + dd];
    }
    for (int idx = threadIdx.x; idx < cn * d.dv; idx += blockDim.x) {
        int i = idx / d.dv, j = idx % d.dv;
        U0out[tok_row(d, b, t0 + i, h) * d.dv + j] = Xs[i * ldx + d.dk + j];
    }
}

// ------------------------------------------------------------------------------------------
// a4: inter-chunk state pass.  grid (dv/VS, B*H); thread dd owns row dd of a [dk x VS] slice of S.
// Stores the state before every chunk (slot n) and the final state (slot NT, and ht).
// GDN: also turns U0 into U = U0 - W S in place.
template <typename TIO>
__global__ void __launch_bounds__(128)
k_state_scan(Dims d, const TIO *__restrict__ k, const TIO *__restrict__ v,
             const float *__restrict__ Gk, const float *__restrict__ bcum,
             const float *__restrict__ h0, float *__restrict__ states, float *__restrict__ ht,
             const float *__restrict__ Wws, const float *__restrict__ U0ws, float *__restrict__ Uws) {
    extern __shared__ float sm[];
    int vs0 = blockIdx.x * VS, bh = blockIdx.y, b = bh / d.H, h = bh % d.H;
    int ldk = d.dk + 1, lds = VS + 1;
    float *Kb = sm;                         // [CMAX][ldk]  k~ * exp(b_last - b)
    float *Vs = Kb + CMAX * ldk;            // [CMAX][VS]   V (or U) slice
    float *Ws = Vs + CMAX * VS;             // [CMAX][ldk]  GDN only
    float *Ss = Ws + CMAX * ldk;            // [dk][lds]    GDN only
    const int dd = threadIdx.x;
    const bool own = dd < d.dk;
    const bool gdn = d.variant == SLA_GDN;
    float S[VS];
#pragma unroll
    for (int j = 0; j < VS; ++j)
        S[j] = (own && h0) ? h0[((size_t)bh * d.dk + dd) * d.dv + vs0 + j] : 0.f;

    for (int n = 0; n < d.NT; ++n) {
        int t0 = n * d.C, cn = min(d.C, d.T - t0);
        if (own) {
            float *dst = states + state_off(d, bh, n, d.NT + 1) + (size_t)dd * d.dv + vs0;
#pragma unroll
            for (int j = 0; j < VS; ++j) dst[j] = S[j];
            if (gdn)
#pragma unroll
                for (int j = 0; j < VS; ++j) Ss[dd * lds + j] = S[j];
        }
        size_t row_last = tok_row(d, b, t0 + cn - 1, h);
        for (int idx = threadIdx.x; idx < cn * d.dk; idx += blockDim.x) {
            int i = idx / d.dk, c = idx % d.dk;
            size_t row = tok_row(d, b, t0 + i, h);
            float e = expf(bcum_at(d, bcum, row_last, c) - bcum_at(d, bcum, row, c));
            float gk = gdn ? 1.f : Gk[row];
            Kb[i * ldk + c] = gk * ldf(k, row * d.dk + c) * e;
            if (gdn) Ws[i * ldk + c] = Wws[row * d.dk + c];
        }
        for (int idx = threadIdx.x; idx < cn * VS; idx += blockDim.x) {
            int i = idx / VS, j = idx % VS;
            size_t row = tok_row(d, b, t0 + i, h);
            Vs[idx] = gdn ? U0ws[row * d.dv + vs0 + j] : ldf(v, row * d.dv + vs0 + j);
        }
        __syncthreads();
        if (gdn) {
            for (int idx = threadIdx.x; idx < cn * VS; idx += blockDim.x) {
                int i = idx % cn, j = idx / cn;
                float acc = Vs[i * VS + j];
                for (int c = 0; c < d.dk; ++c) acc = fmaf(-Ws[i * ldk + c], Ss[c * lds + j], acc);
                Vs[i * VS + j] = acc;
                Uws[tok_row(d, b, t0 + i, h) * d.dv + vs0 + j] = acc;
            }
            __syncthreads();
        }
        if (own) {
            float dec = expf(bcum_at(d, bcum, row_last, dd));
#pragma unroll
            for (int j = 0; j < VS; ++j) S[j] *= dec;
            for (int i = 0; i < cn; ++i) {
                float kb = Kb[i * ldk + dd];
#pragma unroll
                for (int j = 0; j < VS; ++j) S[j] = fmaf(kb, Vs[i * VS + j], S[j]);
            }
        }
        __syncthreads();
    }
    if (own) {
        float *dst = states + state_off(d, bh, d.NT, d.NT + 1) + (size_t)dd * d.dv + vs0;
#pragma unroll
        for (int j = 0; j < VS; ++j) dst[j] = S[j];
        if (ht) {
            float *hdst = ht + ((size_t)bh * d.dk + dd) * d.dv + vs0;
#pragma unroll
            for (int j = 0; j < VS; ++j) hdst[j] = S[j];
        }
    }
}

// ------------------------------------------------------------------------------------------
// a3 + a5: per tile, A = tril(qh kh^T) ; O = A V + qh S ; store in the I/O dtype (heads concatenated).
template <typename TIO>
__global__ void __launch_bounds__(256)
k_output(Dims d, const TIO *__restrict__ q, const TIO *__restrict__ k, const TIO *__restrict__ v,
         const float *__restrict__ Gq, const float *__restrict__ Gk, const float *__restrict__ bcum,
         const float *__restrict__ states, const float *__restrict__ Uws, TIO *__restrict__ o) {
    extern __shared__ float sm[];
    int n = blockIdx.x, bh = blockIdx.y, b = bh / d.H, h = bh % d.H;
    int t0 = n * d.C, cn = min(d.C, d.T - t0);
    int ldk = d.dk + 1, ldv = d.dv + 1, lda = CMAX + 1;
    float *Qs = sm;
    float *Ks = Qs + CMAX * ldk;
    float *Vs = Ks + CMAX * ldk;
    float *As = Vs + CMAX * ldv;
    float *Ss = As + CMAX * lda;             // [dk][ldv]
    const int ty = threadIdx.x >> 5, tx = threadIdx.x & 31;
    const bool gdn = d.variant == SLA_GDN;

    load_qk_hat(d, q, k, Gq, Gk, bcum, b, h, t0, cn, Qs, Ks, ldk);
    for (int idx = threadIdx.x; idx < CMAX * d.dv; idx += blockDim.x) {
        int i = idx / d.dv, j = idx % d.dv;
        float val = 0.f;
        if (i < cn) {
            size_t row = tok_row(d, b, t0 + i, h);
            val = gdn ? Uws[row * d.dv + j] : ldf(v, row * d.dv + j);
        }
        Vs[i * ldv + j] = val;
    }
    const float *Sg = states + state_off(d, bh, n, d.NT + 1);
    for (int idx = threadIdx.x; idx < d.dk * d.dv; idx += blockDim.x)
        Ss[(idx / d.dv) * ldv + idx % d.dv] = Sg[idx];
    __syncthreads();

    {
        float acc[8][2];
        zero_acc(acc);
        tile_gemm<2>(acc, Qs, ldk, 1, Ks, 1, ldk, d.dk, CMAX, ty, tx);
#pragma unroll
        for (int r = 0; r < 8; ++r)
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) {
                int i = ty + 8 * r, j = tx + 32 * cb;
                As[i * lda + j] = (j <= i) ? acc[r][cb] : 0.f;
            }
    }
    __syncthreads();
    float acc[8][4];
    zero_acc(acc);
    tile_gemm<4>(acc, As, lda, 1, Vs, ldv, 1, cn, d.dv, ty, tx);
    tile_gemm<4>(acc, Qs, ldk, 1, Ss, ldv, 1, d.dk, d.dv, ty, tx);
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        int i = ty + 8 * r;
        if (i >= cn) continue;
        size_t row = tok_row(d, b, t0 + i, h);
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
            int j = tx + 32 * cb;
            if (j < d.dv) stf(o, row * d.dv + j, acc[r][cb]);
        }
    }
}

// ------------------------------------------------------------------------------------------
// backward, state-gradient pass (reverse chunk order).  grid (dv/VS, B*H); thread dd owns row dd of
// a [dk x VS] slice of dS.  Stores dS entering each chunk from the right (slot n = gradient w.r.t.
// the state after chunk n).  RETNET/GLA: dS' = diag(exp(b_last)) dS + qh^T dO.
// GDN: dU = Pq^T dO + diag(E) K dS ;  dS' = exp(b_last) dS + qh^T dO - W^T dU   (dU stored).
template <typename TIO>
__global__ void __launch_bounds__(128)
k_dstate_scan(Dims d, const TIO *__restrict__ q, const TIO *__restrict__ k, const TIO *__restrict__ dO,
              const float *__restrict__ Gq, const float *__restrict__ bcum,
              const float *__restrict__ dht, float *__restrict__ dstates, float *__restrict__ dh0,
              const float *__restrict__ Wws, float *__restrict__ dUws) {
    extern __shared__ float sm[];
    int vs0 = blockIdx.x * VS, bh = blockIdx.y, b = bh / d.H, h = bh % d.H;
    int ldk = d.dk + 1, lds = VS + 1, lda = CMAX + 1;
    float *Qs = sm;                          // [CMAX][ldk]  qh
    float *dOs = Qs + CMAX * ldk;            // [CMAX][VS]
    float *Ks = dOs + CMAX * VS;             // GDN: [CMAX][ldk]  k*exp(-b)
    float *Ws = Ks + CMAX * ldk;             // GDN: [CMAX][ldk]
    float *Ps = Ws + CMAX * ldk;             // GDN: [CMAX][lda]  Pq
    float *dSs = Ps + CMAX * lda;            // GDN: [dk][lds]
    float *dUs = dSs + d.dk * lds;           // GDN: [CMAX][VS]
    const int dd = threadIdx.x;
    const bool own = dd < d.dk;
    const bool gdn = d.variant == SLA_GDN;
    float dS[VS];
#pragma unroll
    for (int j = 0; j < VS; ++j)
        dS[j] = (own && dht) ? dht[((size_t)bh * d.dk + dd) * d.dv + vs0 + j] : 0.f;

    for (int n = d.NT - 1; n >= 0; --n) {
        int t0 = n * d.C, cn = min(d.C, d.T - t0);
        if (own) {
            float *dst = dstates + state_off(d, bh, n, d.NT) + (size_t)dd * d.dv + vs0;
#pragma unroll
            for (int j = 0; j < VS; ++j) dst[j] = dS[j];
            if (gdn)
#pragma unroll
                for (int j = 0; j < VS; ++j) dSs[dd * lds + j] = dS[j];
        }
        size_t row_last = tok_row(d, b, t0 + cn - 1, h);
        for (int idx = threadIdx.x; idx < CMAX * d.dk; idx += blockDim.x) {
            int i = idx / d.dk, c = idx % d.dk;
            float qv = 0.f, kv = 0.f, wv = 0.f;
            if (i < cn) {
                size_t row = tok_row(d, b, t0 + i, h);
                float bb = bcum_at(d, bcum, row, c);
                qv = d.scale * Gq[row] * ldf(q, row * d.dk + c) * expf(bb);
                if (gdn) {
                    kv = ldf(k, row * d.dk + c) * expf(-bb);
                    wv = Wws[row * d.dk + c];
                }
            }
            Qs[i * ldk + c] = qv;
            if (gdn) { Ks[i * ldk + c] = kv; Ws[i * ldk + c] = wv; }
        }
        for (int idx = threadIdx.x; idx < CMAX * VS; idx += blockDim.x) {
            int i = idx / VS, j = idx % VS;
            dOs[idx] = i < cn ? ldf(dO, tok_row(d, b, t0 + i, h) * d.dv + vs0 + j) : 0.f;
        }
        __syncthreads();
        float dec = own ? expf(bcum_at(d, bcum, row_last, dd)) : 0.f;
        if (gdn) {
            float elast = expf(bcum[row_last]);
            for (int idx = threadIdx.x; idx < CMAX * CMAX; idx += blockDim.x) {
                int i = idx % CMAX, j = idx / CMAX;
                float acc = 0.f;
                if (j <= i && i < cn)
                    for (int c = 0; c < d.dk; ++c) acc = fmaf(Qs[i * ldk + c], Ks[j * ldk + c], acc);
                Ps[i * lda + j] = acc;
            }
            __syncthreads();
            for (int idx = threadIdx.x; idx < cn * VS; idx += blockDim.x) {
                int i = idx % cn, j = idx / cn;
                float acc = 0.f;
                for (int i2 = i; i2 < cn; ++i2) acc = fmaf(Ps[i2 * lda + i], dOs[i2 * VS + j], acc);
                float acc2 = 0.f;
                for (int c = 0; c < d.dk; ++c) acc2 = fmaf(Ks[i * ldk + c], dSs[c * lds + j], acc2);
                acc = fmaf(elast, acc2, acc);
                dUs[i * VS + j] = acc;
                dUws[tok_row(d, b, t0 + i, h) * d.dv + vs0 + j] = acc;
            }
            __syncthreads();
        }
        if (own) {
#pragma unroll
            for (int j = 0; j < VS; ++j) dS[j] *= dec;
            for (int i = 0; i < cn; ++i) {
                float qv = Qs[i * ldk + dd];
#pragma unroll
                for (int j = 0; j < VS; ++j) dS[j] = fmaf(qv, dOs[i * VS + j], dS[j]);
            }
            if (gdn)
                for (int i = 0; i < cn; ++i) {
                    float wv = Ws[i * ldk + dd];
#pragma unroll
                    for (int j = 0; j < VS; ++j) dS[j] = fmaf(-wv, dUs[i * VS + j], dS[j]);
                }
        }
        __syncthreads();
    }
    if (own && dh0) {
        float *dst = dh0 + ((size_t)bh * d.dk + dd) * d.dv + vs0;
#pragma unroll
        for (int j = 0; j < VS; ++j) dst[j] = dS[j];
    }
}

// ------------------------------------------------------------------------------------------
// backward, per-tile gradients for RETNET / GLA.
//   dA = tril(dO V^T) ; dZ = diag(exp(b_last)) dS_next
//   dqh = dA kh + dO S^T ; dkh = dA^T qh + V dZ^T ; dV = A^T dO + kh dZ
//   db = qh*dqh - kh*dkh (+ rowsum(dS_next*S_next) on the last row) ; dlog_decay = suffix sum of db
template <typename TIO>
__global__ void __launch_bounds__(256)
k_grads_lin(Dims d, const TIO *__restrict__ q, const TIO *__restrict__ k, const TIO *__restrict__ v,
            const TIO *__restrict__ dO, const float *__restrict__ Gq, const float *__restrict__ Gk,
            const float *__restrict__ bcum, const float *__restrict__ states,
            const float *__restrict__ dstates, TIO *__restrict__ dq, TIO *__restrict__ dk,
            TIO *__restrict__ dv, float *__restrict__ dlog_decay, float *__restrict__ dGq,
            float *__restrict__ dGk) {
    extern __shared__ float sm[];
    int n = blockIdx.x, bh = blockIdx.y, b = bh / d.H, h = bh % d.H;
    int t0 = n * d.C, cn = min(d.C, d.T - t0);
    int ldk = d.dk + 1, ldv = d.dv + 1, lda = CMAX + 1;
    float *Qs = sm;
    float *Ks = Qs + CMAX * ldk;
    float *Vs = Ks + CMAX * ldk;
    float *dOs = Vs + CMAX * ldv;
    float *As = dOs + CMAX * ldv;
    float *dAs = As + CMAX * lda;
    float *Ss = dAs + CMAX * lda;             // [dk][ldv]: S, then dZ
    float *Rs = Ss + d.dk * ldv;              // [dk]
    const int ty = threadIdx.x >> 5, tx = threadIdx.x & 31;
    size_t row_last = tok_row(d, b, t0 + cn - 1, h);

    load_qk_hat(d, q, k, Gq, Gk, bcum, b, h, t0, cn, Qs, Ks, ldk);
    for (int idx = threadIdx.x; idx < CMAX * d.dv; idx += blockDim.x) {
        int i = idx / d.dv, j = idx % d.dv;
        float vv = 0.f, gg = 0.f;
        if (i < cn) {
            size_t row = tok_row(d, b, t0 + i, h);
            vv = ldf(v, row * d.dv + j);
            gg = ldf(dO, row * d.dv + j);
        }
        Vs[i * ldv + j] = vv;
        dOs[i * ldv + j] = gg;
    }
    const float *Sg = states + state_off(d, bh, n, d.NT + 1);
    for (int idx = threadIdx.x; idx < d.dk * d.dv; idx += blockDim.x)
        Ss[(idx / d.dv) * ldv + idx % d.dv] = Sg[idx];
    __syncthreads();
    {
        float a1[8][2], a2[8][2];
        zero_acc(a1);
        zero_acc(a2);
        tile_gemm<2>(a1, Qs, ldk, 1, Ks, 1, ldk, d.dk, CMAX, ty, tx);
        tile_gemm<2>(a2, dOs, ldv, 1, Vs, 1, ldv, d.dv, CMAX, ty, tx);
#pragma unroll
        for (int r = 0; r < 8; ++r)
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) {
                int i = ty + 8 * r, j = tx + 32 * cb;
                As[i * lda + j] = (j <= i) ? a1[r][cb] : 0.f;
                dAs[i * lda + j] = (j <= i) ? a2[r][cb] : 0.f;
            }
    }
    __syncthreads();
    float db[8][4];
    {   // dqh and the query-side outputs
        float acc[8][4];
        zero_acc(acc);
        tile_gemm<4>(acc, dAs, lda, 1, Ks, ldk, 1, cn, d.dk, ty, tx);
        tile_gemm<4>(acc, dOs, ldv, 1, Ss, 1, ldv, d.dv, d.dk, ty, tx);
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            int i = ty + 8 * r;
            float gsum = 0.f;
            size_t row = i < cn ? tok_row(d, b, t0 + i, h) : 0;
            float gq = i < cn ? Gq[row] : 0.f;
#pragma unroll
            for (int cb = 0; cb < 4; ++cb) {
                int c = tx + 32 * cb;
                db[r][cb] = 0.f;
                if (i < cn && c < d.dk) {
                    db[r][cb] = Qs[i * ldk + c] * acc[r][cb];
                    float dqt = acc[r][cb] * expf(bcum_at(d, bcum, row, c));
                    gsum = fmaf(d.scale * ldf(q, row * d.dk + c), dqt, gsum);
                    stf(dq, row * d.dk + c, d.scale * gq * dqt);
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) gsum += __shfl_xor_sync(FULL, gsum, o);
            if (tx == 0 && i < cn) dGq[row] = gsum;
        }
    }
    __syncthreads();
    {   // Ss <- dZ = diag(exp(b_last)) dS_next ; Rs <- rowsum(dS_next * S_next)
        const float *dSg = dstates + state_off(d, bh, n, d.NT);
        const float *Sn = states + state_off(d, bh, n + 1, d.NT + 1);
        for (int r0 = ty; r0 < d.dk; r0 += 8) {
            float e = expf(bcum_at(d, bcum, row_last, r0));
            float part = 0.f;
            for (int j = tx; j < d.dv; j += 32) {
                float g = dSg[(size_t)r0 * d.dv + j];
                part = fmaf(g, Sn[(size_t)r0 * d.dv + j], part);
                Ss[r0 * ldv + j] = e * g;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(FULL, part, o);
            if (tx == 0) Rs[r0] = part;
        }
    }
    __syncthreads();
    {   // dkh and the key-side outputs
        float acc[8][4];
        zero_acc(acc);
        tile_gemm<4>(acc, dAs, 1, lda, Qs, ldk, 1, cn, d.dk, ty, tx);
        tile_gemm<4>(acc, Vs, ldv, 1, Ss, 1, ldv, d.dv, d.dk, ty, tx);
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            int i = ty + 8 * r;
            float gsum = 0.f;
            size_t row = i < cn ? tok_row(d, b, t0 + i, h) : 0;
            float gk = i < cn ? Gk[row] : 0.f;
#pragma unroll
            for (int cb = 0; cb < 4; ++cb) {
                int c = tx + 32 * cb;
                if (i < cn && c < d.dk) {
                    db[r][cb] -= Ks[i * ldk + c] * acc[r][cb];
                    float dkt = acc[r][cb] * expf(-bcum_at(d, bcum, row, c));
                    gsum = fmaf(ldf(k, row * d.dk + c), dkt, gsum);
                    stf(dk, row * d.dk + c, gk * dkt);
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) gsum += __shfl_xor_sync(FULL, gsum, o);
            if (tx == 0 && i < cn) dGk[row] = gsum;
        }
    }
    {   // dV = A^T dO + kh dZ
        float acc[8][4];
        zero_acc(acc);
        tile_gemm<4>(acc, As, 1, lda, dOs, ldv, 1, cn, d.dv, ty, tx);
        tile_gemm<4>(acc, Ks, ldk, 1, Ss, ldv, 1, d.dk, d.dv, ty, tx);
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            int i = ty + 8 * r;
            if (i >= cn) continue;
            size_t row = tok_row(d, b, t0 + i, h);
#pragma unroll
            for (int cb = 0; cb < 4; ++cb) {
                int j = tx + 32 * cb;
                if (j < d.dv) stf(dv, row * d.dv + j, acc[r][cb]);
            }
        }
    }
    if (d.variant != SLA_GLA || !dlog_decay) return;
    __syncthreads();            // every thread is done with Vs
    float *dbs = Vs;            // reuse as [CMAX][ldk] (ldk <= ldv is not needed: Vs..dOs are contiguous)
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
            int i = ty + 8 * r, c = tx + 32 * cb;
            if (c < d.dk) dbs[i * ldk + c] = db[r][cb];
        }
    __syncthreads();
    for (int c = threadIdx.x; c < d.dk; c += blockDim.x) {
        float run = Rs[c];
        for (int i = cn - 1; i >= 0; --i) {
            run += dbs[i * ldk + c];
            dlog_decay[tok_row(d, b, t0 + i, h) * d.dk + c] = run;
        }
    }
}

// ------------------------------------------------------------------------------------------
// host side
size_t smem_prepare(const Dims &d) {
    return sizeof(float) * (CMAX * (d.dk + 1) + CMAX * (CMAX + 1) + CMAX * (d.dk + d.dv) + 2 * CMAX);
}
size_t smem_scan(const Dims &d) {
    return sizeof(float) * (2 * CMAX * (d.dk + 1) + CMAX * VS + d.dk * (VS + 1));
}
size_t smem_output(const Dims &d) {
    return sizeof(float) * (2 * CMAX * (d.dk + 1) + CMAX * (d.dv + 1) + CMAX * (CMAX + 1) + d.dk * (d.dv + 1));
}
size_t smem_dscan(const Dims &d) {
    return sizeof(float) * (3 * CMAX * (d.dk + 1) + 2 * CMAX * VS + CMAX * (CMAX + 1) + d.dk * (VS + 1));
}
size_t smem_grads_lin(const Dims &d) {
    return sizeof(float) * (2 * CMAX * (d.dk + 1) + 2 * CMAX * (d.dv + 1) + 2 * CMAX * (CMAX + 1) +
                            d.dk * (d.dv + 1) + d.dk);
}

template <int HP>
void launch_gate_fwd(const float *lq, const float *lk, float *Gq, float *Gk, long n_tok, int H,
                     cudaStream_t st) {
    long threads = n_tok * HP;
    dim3 grid((unsigned)((threads + 255) / 256), 2);
    k_gate_fwd<HP><<<grid, 256, 0, st>>>(lq, lk, Gq, Gk, n_tok, H);
}
template <int HP>
void launch_gate_bwd(const float *Gq, const float *Gk, const float *dGq, const float *dGk, float *dlq,
                     float *dlk, long n_tok, int H, cudaStream_t st) {
    long threads = n_tok * HP;
    dim3 grid((unsigned)((threads + 255) / 256), 2);
    k_gate_bwd<HP><<<grid, 256, 0, st>>>(Gq, Gk, dGq, dGk, dlq, dlk, n_tok, H);
}

template <typename TIO>
int forward_t(const Dims &d, const Workspace &w, const FwdArgs &a, bool write_o, cudaStream_t st, Tracer &tr) {
    float *ws = a.ws;
    float *Gq = ws + w.Gq, *Gk = ws + w.Gk, *bcum = ws + w.bcum, *states = ws + w.states;
    float *Wws = ws + w.W, *U0ws = ws + w.U0, *Uws = ws + w.U;
    long n_tok = (long)d.B * d.T;
    int launches = 0;
    int hp = 1;
    while (hp < d.H) hp <<= 1;
    switch (hp) {
        case 1: launch_gate_fwd<1>(a.lq, a.lk, Gq, Gk, n_tok, d.H, st); break;
        case 2: launch_gate_fwd<2>(a.lq, a.lk, Gq, Gk, n_tok, d.H, st); break;
        case 4: launch_gate_fwd<4>(a.lq, a.lk, Gq, Gk, n_tok, d.H, st); break;
        case 8: launch_gate_fwd<8>(a.lq, a.lk, Gq, Gk, n_tok, d.H, st); break;
        case 16: launch_gate_fwd<16>(a.lq, a.lk, Gq, Gk, n_tok, d.H, st); break;
        default: launch_gate_fwd<32>(a.lq, a.lk, Gq, Gk, n_tok, d.H, st); break;
    }
    tr.mark("gate_fwd");
    ++launches;
    dim3 tiles(d.NT, d.B * d.H);
    k_cumdecay<<<tiles, d.variant == SLA_GLA ? 128 : 32, 0, st>>>(d, a.log_decay, bcum, a.status);
    tr.mark("cumdecay");
    ++launches;
    const TIO *q = (const TIO *)a.q, *k = (const TIO *)a.k, *v = (const TIO *)a.v;
    if (d.variant == SLA_GDN) {
        k_gdn_prepare<TIO><<<tiles, 256, smem_prepare(d), st>>>(d, k, v, a.beta, Gk, bcum, Wws, U0ws);
        tr.mark("gdn_prepare");
        ++launches;
    }
    dim3 slices(d.dv / VS, d.B * d.H);
    k_state_scan<TIO><<<slices, 128, smem_scan(d), st>>>(d, k, v, Gk, bcum, a.h0, states, a.ht, Wws, U0ws, Uws);
    tr.mark("state_scan");
    ++launches;
    if (write_o) {
        k_output<TIO><<<tiles, 256, smem_output(d), st>>>(d, q, k, v, Gq, Gk, bcum, states, Uws, (TIO *)a.o);
        tr.mark("output");
        ++launches;
    }
    return cudaGetLastError() == cudaSuccess ? launches : -1;
}

template <typename TIO>
int backward_lin_t(const Dims &d, const Workspace &w, const BwdArgs &a, cudaStream_t st, Tracer &tr) {
    float *ws = a.ws;
    float *Gq = ws + w.Gq, *Gk = ws + w.Gk, *bcum = ws + w.bcum, *states = ws + w.states;
    float *dstates = ws + w.dstates, *dGq = ws + w.dGq, *dGk = ws + w.dGk;
    int launches = 0;
    const TIO *q = (const TIO *)a.q, *k = (const TIO *)a.k, *v = (const TIO *)a.v, *dO = (const TIO *)a.dO;
    dim3 tiles(d.NT, d.B * d.H), slices(d.dv / VS, d.B * d.H);
    k_dstate_scan<TIO><<<slices, 128, smem_dscan(d), st>>>(d, q, k, dO, Gq, bcum, a.dht, dstates, a.dh0,
                                                           nullptr, nullptr);
    tr.mark("dstate_scan");
    ++launches;
    k_grads_lin<TIO><<<tiles, 256, smem_grads_lin(d), st>>>(d, q, k, v, dO, Gq, Gk, bcum, states, dstates,
                                                            (TIO *)a.dq, (TIO *)a.dk, (TIO *)a.dv,
                                                            a.dlog_decay, dGq, dGk);
    tr.mark("grads_lin");
    ++launches;
    return cudaGetLastError() == cudaSuccess ? launches : -1;
}

template <typename TIO> bool configure_t() {
    Dims d{};
    d.dk = d.dv = 128;
    bool ok = true;
    ok &= set_smem(k_gdn_prepare<TIO>, smem_prepare(d));
    ok &= set_smem(k_state_scan<TIO>, smem_scan(d));
    ok &= set_smem(k_output<TIO>, smem_output(d));
    ok &= set_smem(k_dstate_scan<TIO>, smem_dscan(d));
    ok &= set_smem(k_grads_lin<TIO>, smem_grads_lin(d));
    return ok;
}

}  // namespace

int generic_configure() {
    bool ok = configure_t<float>() && configure_t<__nv_bfloat16>();
    return ok ? 0 : -1;
}

int generic_forward(const Dims &d, const Workspace &w, const FwdArgs &a, bool write_o, cudaStream_t st, Tracer &tr) {
    return d.io_bf16 ? forward_t<__nv_bfloat16>(d, w, a, write_o, st, tr) : forward_t<float>(d, w, a, write_o, st, tr);
}

int generic_backward(const Dims &d, const Workspace &w, const BwdArgs &a, cudaStream_t st, Tracer &tr) {
    // recompute gates, cumulative decays and the per-chunk states (no output store)
    FwdArgs f{a.q, a.k, a.v, a.log_decay, a.beta, a.lq, a.lk, a.h0, nullptr, nullptr, a.ws, a.status};
    int n1 = generic_forward(d, w, f, false, st, tr);
    if (n1 < 0) return -1;
    int n2;
    if (d.variant == SLA_GDN) {
        float *ws = a.ws;
        dim3 slices(d.dv / VS, d.B * d.H);
        if (d.io_bf16)
            k_dstate_scan<__nv_bfloat16><<<slices, 128, smem_dscan(d), st>>>(
                d, (const __nv_bfloat16 *)a.q, (const __nv_bfloat16 *)a.k, (const __nv_bfloat16 *)a.dO, ws + w.Gq,
                ws + w.bcum, a.dht, ws + w.dstates, a.dh0, ws + w.W, ws + w.dU);
        else
            k_dstate_scan<float><<<slices, 128, smem_dscan(d), st>>>(
                d, (const float *)a.q, (const float *)a.k, (const float *)a.dO, ws + w.Gq, ws + w.bcum, a.dht,
                ws + w.dstates, a.dh0, ws + w.W, ws + w.dU);
        tr.mark("dstate_scan");
        if (cudaGetLastError() != cudaSuccess) return -1;
        n2 = gdn_backward_tiles(d, w, a, st, tr);
        if (n2 > 0) n2 += 1;
    } else {
        n2 = d.io_bf16 ? backward_lin_t<__nv_bfloat16>(d, w, a, st, tr) : backward_lin_t<float>(d, w, a, st, tr);
    }
    if (n2 < 0) return -1;
    float *ws = a.ws;
    long n_tok = (long)d.B * d.T;
    int hp = 1;
    while (hp < d.H) hp <<= 1;
    const float *Gq = ws + w.Gq, *Gk = ws + w.Gk, *dGq = ws + w.dGq, *dGk = ws + w.dGk;
    switch (hp) {
        case 1: launch_gate_bwd<1>(Gq, Gk, dGq, dGk, a.dlq, a.dlk, n_tok, d.H, st); break;
        case 2: launch_gate_bwd<2>(Gq, Gk, dGq, dGk, a.dlq, a.dlk, n_tok, d.H, st); break;
        case 4: launch_gate_bwd<4>(Gq, Gk, dGq, dGk, a.dlq, a.dlk, n_tok, d.H, st); break;
        case 8: launch_gate_bwd<8>(Gq, Gk, dGq, dGk, a.dlq, a.dlk, n_tok, d.H, st); break;
        case 16: launch_gate_bwd<16>(Gq, Gk, dGq, dGk, a.dlq, a.dlk, n_tok, d.H, st); break;
        default: launch_gate_bwd<32>(Gq, Gk, dGq, dGk, a.dlq, a.dlk, n_tok, d.H, st); break;
    }
    tr.mark("gate_bwd");
    if (cudaGetLastError() != cudaSuccess) return -1;
    return n1 + n2 + 1;
}

}  // namespace sla
