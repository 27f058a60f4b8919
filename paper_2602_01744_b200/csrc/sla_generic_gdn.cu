// Backward of the gated delta rule (Eq. 14-16) in chunkwise WY form, fp32 on CUDA cores.
//
// Per chunk, with T = (I+L)^{-1}, W = T diag(beta e^b) K, U0 = T diag(beta) V', U = U0 - W S:
//   dW = -dU S^T ;  dKbg = T^T dW ;  dVb = T^T dU      (back-substitution, never forming T)
//   dL = -strict_tril(dKbg W^T + dVb U0^T) ;  dM = dL (.) D          D_ij = exp(b_i - b_j)
//   dPq = tril(dO U^T) ;  dQK = dPq (.) D
//   dq~ = e^b (dO S^T) + dQK K
//   dk  = dQK^T q~ + E (U dS^T) + diag(beta) dM K + (diag(beta) dM)^T K + beta e^b dKbg ,  E_i = exp(b_last - b_i)
//   dv' = beta dVb ;  dbeta = rowsum(dM (.) K K^T) + e^b (dKbg . k) + dVb . v'
//   db  = e^b (dO S^T . q~) + beta e^b (dKbg . k) + rowsum(X) - colsum(X) - e  (+ sum(e) + e^{b_last} <dS,S> on
//         the last row),  X = dPq (.) Pq + dL (.) L,  e_i = E_i (k_i . (U dS^T)_i) ;  dlog_decay = suffix sum of db.
#include "sla_generic.cuh"

namespace sla {
namespace {

using namespace detail;

// G1: triangular back-substitution and everything that only needs dKbg / dVb row by row.
template <typename TIO>
__global__ void __launch_bounds__(256)
k_gdn_bwd_solve(Dims d, const TIO *__restrict__ k, const TIO *__restrict__ v,
                const float *__restrict__ beta, const float *__restrict__ Gk,
                const float *__restrict__ bcum, const float *__restrict__ states,
                const float *__restrict__ dUws, float *__restrict__ dKbg_ws, float *__restrict__ dVb_ws,
                float *__restrict__ dbpart, TIO *__restrict__ dv, float *__restrict__ dGk,
                float *__restrict__ dbeta) {
    extern __shared__ float sm[];
    int n = blockIdx.x, bh = blockIdx.y, b = bh / d.H, h = bh % d.H;
    int t0 = n * d.C, cn = min(d.C, d.T - t0);
    int ldk = d.dk + 1, ldl = CMAX + 1, ldv = d.dv + 1, ldx = d.dk + d.dv;
    float *Ks = sm;                       // [CMAX][ldk]
    float *Ls = Ks + CMAX * ldk;          // [CMAX][ldl]
    float *dUs = Ls + CMAX * ldl;         // [CMAX][ldv]
    float *Ss = dUs + CMAX * ldv;         // [dk][ldv]
    float *Xs = Ss + d.dk * ldv;          // [CMAX][ldx]
    float *bs = Xs + CMAX * ldx;          // [CMAX]
    float *bt = bs + CMAX;                // [CMAX]
    const int ty = threadIdx.x >> 5, tx = threadIdx.x & 31;
    for (int i = threadIdx.x; i < CMAX; i += blockDim.x) {
        size_t row = tok_row(d, b, t0 + min(i, cn - 1), h);
        bs[i] = bcum[row];
        bt[i] = i < cn ? beta[row] : 0.f;
    }
    for (int idx = threadIdx.x; idx < CMAX * d.dk; idx += blockDim.x) {
        int i = idx / d.dk, c = idx % d.dk;
        Ks[i * ldk + c] = i < cn ? ldf(k, tok_row(d, b, t0 + i, h) * d.dk + c) : 0.f;
    }
    for (int idx = threadIdx.x; idx < CMAX * d.dv; idx += blockDim.x) {
        int i = idx / d.dv, j = idx % d.dv;
        dUs[i * ldv + j] = i < cn ? dUws[tok_row(d, b, t0 + i, h) * d.dv + j] : 0.f;
    }
    const float *Sg = states + state_off(d, bh, n, d.NT + 1);
    for (int idx = threadIdx.x; idx < d.dk * d.dv; idx += blockDim.x)
        Ss[(idx / d.dv) * ldv + idx % d.dv] = Sg[idx];
    __syncthreads();
    for (int idx = threadIdx.x; idx < CMAX * CMAX; idx += blockDim.x) {
        int i = idx % CMAX, j = idx / CMAX;
        float acc = 0.f;
        if (j < i) {
            for (int c = 0; c < d.dk; ++c) acc = fmaf(Ks[i * ldk + c], Ks[j * ldk + c], acc);
            acc *= bt[i] * expf(bs[i] - bs[j]);
        }
        Ls[i * ldl + j] = acc;
    }
    {
        float acc[8][4];
        zero_acc(acc);
        tile_gemm<4>(acc, dUs, ldv, 1, Ss, 1, ldv, d.dv, d.dk, ty, tx);
#pragma unroll
        for (int r = 0; r < 8; ++r)
#pragma unroll
            for (int cb = 0; cb < 4; ++cb) {
                int i = ty + 8 * r, c = tx + 32 * cb;
                if (c < d.dk) Xs[i * ldx + c] = -acc[r][cb];
            }
    }
    for (int idx = threadIdx.x; idx < CMAX * d.dv; idx += blockDim.x) {
        int i = idx / d.dv, j = idx % d.dv;
        Xs[i * ldx + d.dk + j] = dUs[i * ldv + j];
    }
    __syncthreads();
    for (int col = threadIdx.x; col < ldx; col += blockDim.x) {
        for (int i = cn - 2; i >= 0; --i) {
            float acc = Xs[i * ldx + col];
            for (int j = i + 1; j < cn; ++j) acc = fmaf(-Ls[j * ldl + i], Xs[j * ldx + col], acc);
            Xs[i * ldx + col] = acc;
        }
    }
    __syncthreads();
    for (int i = ty; i < cn; i += 8) {
        size_t row = tok_row(d, b, t0 + i, h);
        float gk = Gk[row], bi = bt[i], gam = expf(bs[i]);
        float t2 = 0.f, sv = 0.f;
        for (int c = tx; c < d.dk; c += 32) {
            float x = Xs[i * ldx + c];
            dKbg_ws[row * d.dk + c] = x;
            t2 = fmaf(x, Ks[i * ldk + c], t2);
        }
        for (int j = tx; j < d.dv; j += 32) {
            float x = Xs[i * ldx + d.dk + j];
            dVb_ws[row * d.dv + j] = x;
            sv = fmaf(ldf(v, row * d.dv + j), x, sv);
            stf(dv, row * d.dv + j, gk * bi * x);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            t2 += __shfl_xor_sync(FULL, t2, o);
            sv += __shfl_xor_sync(FULL, sv, o);
        }
        if (tx == 0) {
            dbeta[row] = gam * t2 + gk * sv;      // k_gdn_grads adds rowsum(dM (.) K K^T)
            dbpart[row] = bi * gam * t2;
            dGk[row] = bi * sv;
        }
    }
}

// G2: the remaining gradients of one tile.
template <typename TIO>
__global__ void __launch_bounds__(256)
k_gdn_grads(Dims d, const TIO *__restrict__ q, const TIO *__restrict__ k, const TIO *__restrict__ dO,
            const float *__restrict__ beta, const float *__restrict__ Gq, const float *__restrict__ bcum,
            const float *__restrict__ states, const float *__restrict__ dstates,
            const float *__restrict__ Wws, const float *__restrict__ U0ws, const float *__restrict__ Uws,
            const float *__restrict__ dKbg_ws, const float *__restrict__ dVb_ws,
            const float *__restrict__ dbpart, TIO *__restrict__ dq, TIO *__restrict__ dk,
            float *__restrict__ dlog_decay, float *__restrict__ dbeta, float *__restrict__ dGq) {
    extern __shared__ float sm[];
    int n = blockIdx.x, bh = blockIdx.y, b = bh / d.H, h = bh % d.H;
    int t0 = n * d.C, cn = min(d.C, d.T - t0);
    int ldt = max(d.dk, d.dv) + 1, lda = CMAX + 1;
    float *T0 = sm, *T1 = T0 + CMAX * ldt, *T2 = T1 + CMAX * ldt, *T3 = T2 + CMAX * ldt;
    float *M0 = T3 + CMAX * ldt, *M1 = M0 + CMAX * lda, *M2 = M1 + CMAX * lda;
    float *bs = M2 + CMAX * lda;          // [CMAX] cumulative log-decay
    float *bt = bs + CMAX;                // [CMAX] beta
    float *rowX = bt + CMAX;              // [CMAX]
    float *db1 = rowX + CMAX;             // [CMAX] rowsum(dM (.) KK)
    float *dbv = db1 + CMAX;              // [CMAX] db
    float *ev = dbv + CMAX;               // [CMAX] e_i
    float *colpart = ev + CMAX;           // [8][CMAX]
    float *red = colpart + 8 * CMAX;      // [8]
    const int ty = threadIdx.x >> 5, tx = threadIdx.x & 31;

    auto load_tile = [&](float *dst, const float *src, int width) {
        for (int idx = threadIdx.x; idx < CMAX * width; idx += blockDim.x) {
            int i = idx / width, c = idx % width;
            dst[i * ldt + c] = i < cn ? src[tok_row(d, b, t0 + i, h) * width + c] : 0.f;
        }
    };
    for (int i = threadIdx.x; i < CMAX; i += blockDim.x) {
        size_t row = tok_row(d, b, t0 + min(i, cn - 1), h);
        bs[i] = bcum[row];
        bt[i] = i < cn ? beta[row] : 0.f;
    }
    // phase A: dL = -strict_tril(dKbg W^T + dVb U0^T)
    load_tile(T0, dKbg_ws, d.dk);
    load_tile(T1, Wws, d.dk);
    load_tile(T2, dVb_ws, d.dv);
    load_tile(T3, U0ws, d.dv);
    __syncthreads();
    {
        float a[8][2];
        zero_acc(a);
        tile_gemm<2>(a, T0, ldt, 1, T1, 1, ldt, d.dk, CMAX, ty, tx);
        tile_gemm<2>(a, T2, ldt, 1, T3, 1, ldt, d.dv, CMAX, ty, tx);
#pragma unroll
        for (int r = 0; r < 8; ++r)
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) {
                int i = ty + 8 * r, j = tx + 32 * cb;
                M0[i * lda + j] = (j < i) ? -a[r][cb] : 0.f;
            }
    }
    __syncthreads();
    // phase B operands: T0 = q~ (gated, scaled, no decay), T1 = K, T2 = dO, T3 = U
    for (int idx = threadIdx.x; idx < CMAX * d.dk; idx += blockDim.x) {
        int i = idx / d.dk, c = idx % d.dk;
        float qv = 0.f, kv = 0.f;
        if (i < cn) {
            size_t row = tok_row(d, b, t0 + i, h);
            qv = d.scale * Gq[row] * ldf(q, row * d.dk + c);
            kv = ldf(k, row * d.dk + c);
        }
        T0[i * ldt + c] = qv;
        T1[i * ldt + c] = kv;
    }
    for (int idx = threadIdx.x; idx < CMAX * d.dv; idx += blockDim.x) {
        int i = idx / d.dv, j = idx % d.dv;
        T2[i * ldt + j] = i < cn ? ldf(dO, tok_row(d, b, t0 + i, h) * d.dv + j) : 0.f;
    }
    load_tile(T3, Uws, d.dv);
    __syncthreads();
    {
        float a1[8][2], a2[8][2], a3[8][2];
        zero_acc(a1);
        zero_acc(a2);
        zero_acc(a3);
        tile_gemm<2>(a1, T0, ldt, 1, T1, 1, ldt, d.dk, CMAX, ty, tx);
        tile_gemm<2>(a2, T2, ldt, 1, T3, 1, ldt, d.dv, CMAX, ty, tx);
        tile_gemm<2>(a3, T1, ldt, 1, T1, 1, ldt, d.dk, CMAX, ty, tx);
        float colacc[2] = {0.f, 0.f};
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            int i = ty + 8 * r;
            float rx = 0.f, r1 = 0.f;
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) {
                int j = tx + 32 * cb;
                float D = (j <= i) ? expf(bs[i] - bs[j]) : 0.f;
                float Pq = a1[r][cb] * D;
                float dPq = (j <= i) ? a2[r][cb] : 0.f;
                float Lij = (j < i) ? bt[i] * a3[r][cb] * D : 0.f;
                float dL = M0[i * lda + j];
                float dM = dL * D;
                M1[i * lda + j] = dPq * D;
                M2[i * lda + j] = bt[i] * dM;
                float x = dPq * Pq + dL * Lij;
                rx += x;
                colacc[cb] += x;
                r1 = fmaf(dM, a3[r][cb], r1);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                rx += __shfl_xor_sync(FULL, rx, o);
                r1 += __shfl_xor_sync(FULL, r1, o);
            }
            if (tx == 0) { rowX[i] = rx; db1[i] = r1; }
        }
        colpart[ty * CMAX + tx] = colacc[0];
        colpart[ty * CMAX + tx + 32] = colacc[1];
    }
    __syncthreads();
    const float *Sg = states + state_off(d, bh, n, d.NT + 1);
    const float *dSg = dstates + state_off(d, bh, n, d.NT);
    {   // query side
        float acc[8][4];
        zero_acc(acc);
        tile_gemm<4>(acc, T2, ldt, 1, Sg, 1, d.dv, d.dv, d.dk, ty, tx);
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            int i = ty + 8 * r;
            float gam = expf(bs[i]), s = 0.f;
#pragma unroll
            for (int cb = 0; cb < 4; ++cb) {
                int c = tx + 32 * cb;
                if (c < d.dk) s = fmaf(acc[r][cb], T0[i * ldt + c], s);
                acc[r][cb] *= gam;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(FULL, s, o);
            if (tx == 0) dbv[i] = gam * s;
        }
        tile_gemm<4>(acc, M1, lda, 1, T1, ldt, 1, cn, d.dk, ty, tx);
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            int i = ty + 8 * r;
            float gsum = 0.f;
            size_t row = i < cn ? tok_row(d, b, t0 + i, h) : 0;
            float gq = i < cn ? Gq[row] : 0.f;
#pragma unroll
            for (int cb = 0; cb < 4; ++cb) {
                int c = tx + 32 * cb;
                if (i < cn && c < d.dk) {
                    gsum = fmaf(d.scale * ldf(q, row * d.dk + c), acc[r][cb], gsum);
                    stf(dq, row * d.dk + c, d.scale * gq * acc[r][cb]);
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) gsum += __shfl_xor_sync(FULL, gsum, o);
            if (tx == 0 && i < cn) dGq[row] = gsum;
        }
    }
    {   // key side
        float acc[8][4];
        zero_acc(acc);
        tile_gemm<4>(acc, T3, ldt, 1, dSg, 1, d.dv, d.dv, d.dk, ty, tx);
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            int i = ty + 8 * r;
            float E = expf(bs[cn - 1] - bs[i]), s = 0.f;
#pragma unroll
            for (int cb = 0; cb < 4; ++cb) {
                int c = tx + 32 * cb;
                if (c < d.dk) s = fmaf(acc[r][cb], T1[i * ldt + c], s);
                acc[r][cb] *= E;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(FULL, s, o);
            if (tx == 0) ev[i] = i < cn ? E * s : 0.f;
        }
        tile_gemm<4>(acc, M1, 1, lda, T0, ldt, 1, cn, d.dk, ty, tx);
        tile_gemm<4>(acc, M2, lda, 1, T1, ldt, 1, cn, d.dk, ty, tx);
        tile_gemm<4>(acc, M2, 1, lda, T1, ldt, 1, cn, d.dk, ty, tx);
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            int i = ty + 8 * r;
            if (i >= cn) continue;
            size_t row = tok_row(d, b, t0 + i, h);
            float bg = bt[i] * expf(bs[i]);
#pragma unroll
            for (int cb = 0; cb < 4; ++cb) {
                int c = tx + 32 * cb;
                if (c < d.dk) stf(dk, row * d.dk + c, fmaf(bg, dKbg_ws[row * d.dk + c], acc[r][cb]));
            }
        }
    }
    {   // <dS, S>
        float part = 0.f;
        for (int idx = threadIdx.x; idx < d.dk * d.dv; idx += blockDim.x) part = fmaf(dSg[idx], Sg[idx], part);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(FULL, part, o);
        if (tx == 0) red[ty] = part;
    }
    __syncthreads();
    if (threadIdx.x < CMAX) {
        int i = threadIdx.x;
        float cs = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) cs += colpart[w * CMAX + i];
        float val = 0.f;
        if (i < cn) {
            size_t row = tok_row(d, b, t0 + i, h);
            val = dbv[i] + dbpart[row] + rowX[i] - cs - ev[i];
            dbeta[row] += db1[i];
        }
        dbv[i] = val;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float dot = 0.f, esum = 0.f;
        for (int w = 0; w < 8; ++w) dot += red[w];
        for (int i = 0; i < cn; ++i) esum += ev[i];
        float run = esum + expf(bs[cn - 1]) * dot;
        for (int i = cn - 1; i >= 0; --i) {
            run += dbv[i];
            dlog_decay[tok_row(d, b, t0 + i, h)] = run;
        }
    }
}

size_t smem_solve(const Dims &d) {
    return sizeof(float) * (CMAX * (d.dk + 1) + CMAX * (CMAX + 1) + CMAX * (d.dv + 1) + d.dk * (d.dv + 1) +
                            CMAX * (d.dk + d.dv) + 2 * CMAX);
}
size_t smem_grads(const Dims &d) {
    int ldt = (d.dk > d.dv ? d.dk : d.dv) + 1;
    return sizeof(float) * (4 * CMAX * ldt + 3 * CMAX * (CMAX + 1) + 6 * CMAX + 8 * CMAX + 8);
}

template <typename TIO>
int backward_gdn_t(const Dims &d, const Workspace &w, const BwdArgs &a, cudaStream_t st, Tracer &tr) {
    float *ws = a.ws;
    const float *Gq = ws + w.Gq, *Gk = ws + w.Gk, *bcum = ws + w.bcum, *states = ws + w.states;
    const float *dstates = ws + w.dstates;
    const TIO *q = (const TIO *)a.q, *k = (const TIO *)a.k, *v = (const TIO *)a.v, *dO = (const TIO *)a.dO;
    dim3 tiles(d.NT, d.B * d.H);
    k_gdn_bwd_solve<TIO><<<tiles, 256, smem_solve(d), st>>>(d, k, v, a.beta, Gk, bcum, states, ws + w.dU,
                                                            ws + w.dKbg, ws + w.dVb, ws + w.dbpart,
                                                            (TIO *)a.dv, ws + w.dGk, a.dbeta);
    tr.mark("gdn_bwd_solve");
    k_gdn_grads<TIO><<<tiles, 256, smem_grads(d), st>>>(d, q, k, dO, a.beta, Gq, bcum, states, dstates,
                                                        ws + w.W, ws + w.U0, ws + w.U, ws + w.dKbg, ws + w.dVb,
                                                        ws + w.dbpart, (TIO *)a.dq, (TIO *)a.dk, a.dlog_decay,
                                                        a.dbeta, ws + w.dGq);
    tr.mark("gdn_grads");
    return cudaGetLastError() == cudaSuccess ? 2 : -1;
}

}  // namespace

int gdn_configure() {
    Dims d{};
    d.dk = d.dv = 128;
    bool ok = set_smem(k_gdn_bwd_solve<float>, smem_solve(d)) && set_smem(k_gdn_bwd_solve<__nv_bfloat16>, smem_solve(d)) &&
              set_smem(k_gdn_grads<float>, smem_grads(d)) && set_smem(k_gdn_grads<__nv_bfloat16>, smem_grads(d));
    return ok ? 0 : -1;
}

int gdn_backward_tiles(const Dims &d, const Workspace &w, const BwdArgs &a, cudaStream_t st, Tracer &tr) {
    return d.io_bf16 ? backward_gdn_t<__nv_bfloat16>(d, w, a, st, tr) : backward_gdn_t<float>(d, w, a, st, tr);
}

}  // namespace sla
