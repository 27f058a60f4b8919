// Gate score projections of Eq. 4: the logits the head softmax runs on,
//     lq[b,t,h] = sum_c q[b,t,h,c] W_GQ[c,h]        lk[b,t,h] = sum_c k[b,t,h,c] W_GK[c,h]
// (W in R^{d x H}, d the per-head width: every head scores itself through its own column), and their reverse:
//     dq[b,t,h,:] += dlq[b,t,h] W_GQ[:,h]           dW_GQ[c,h] = sum_{b,t} dlq[b,t,h] q[b,t,h,c]      (same for k).
// Both are streaming passes over q and k (HBM-bound; the arithmetic is one multiply-add per element).  A thread owns
// one 16-byte vector of the token row [H*d] for the whole launch - its slice of W sits in registers - and walks the
// tokens of its CTA, so every access of a warp is one contiguous run of 512 bytes.  The weight gradient is summed per
// thread in registers, written per CTA, and reduced over the CTAs in a fixed order (same bits on every run).
#include "sla_internal.h"

#include <algorithm>

namespace sla {
namespace {

template <typename TIO> struct Vec;
template <> struct Vec<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ void widen(const uint4 v, float (&x)[4]) {
        x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y); x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
    }
    static __device__ __forceinline__ void load(const float *p, float (&x)[4]) {
        const float4 v = __ldg(reinterpret_cast<const float4 *>(p));
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    }
    static __device__ __forceinline__ void load_rw(const float *p, float (&x)[4]) {     // memory this kernel also writes
        const float4 v = *reinterpret_cast<const float4 *>(p);
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    }
    static __device__ __forceinline__ void store(float *p, const float (&x)[4]) {
        *reinterpret_cast<float4 *>(p) = make_float4(x[0], x[1], x[2], x[3]);
    }
};
template <> struct Vec<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ void widen(const uint4 v, float (&x)[8]) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&w[e]));
            x[2 * e] = f.x; x[2 * e + 1] = f.y;
        }
    }
    static __device__ __forceinline__ void load(const __nv_bfloat16 *p, float (&x)[8]) {
        widen(__ldg(reinterpret_cast<const uint4 *>(p)), x);
    }
    static __device__ __forceinline__ void load_rw(const __nv_bfloat16 *p, float (&x)[8]) {
        widen(*reinterpret_cast<const uint4 *>(p), x);
    }
    static __device__ __forceinline__ void store(__nv_bfloat16 *p, const float (&x)[8]) {
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            __nv_bfloat162 v = __floats2bfloat162_rn(x[2 * e], x[2 * e + 1]);
            w[e] = *reinterpret_cast<uint32_t *>(&v);
        }
        *reinterpret_cast<uint4 *>(p) = make_uint4(w[0], w[1], w[2], w[3]);
    }
};

constexpr int TOKS = 8;          // tokens per block of loads of the forward pass (kept packed, 16 bytes each, until used)

// Forward.  grid (CTAs, 2 sides); blockDim = H*d/N threads rounded up to whole warps.  A head's d/N partial dots sit in
// d/N consecutive threads: when that is a power of two (<= 32) they are folded with shuffles and every warp streams on
// its own, SHFL tokens in flight; otherwise they meet in shared memory, TOKS tokens per barrier pair.
template <typename TIO, bool SHFL>
__global__ void __launch_bounds__(256, 4)
k_gate_scores_fwd(long n_tok, int H, int d, int hpc, const TIO *__restrict__ q, const TIO *__restrict__ k,
                                  const float *__restrict__ Wq, const float *__restrict__ Wk,
                                  float *__restrict__ lq, float *__restrict__ lk) {
    constexpr int N = Vec<TIO>::N;
    constexpr int NT = TOKS;                         // tokens per block of loads
    extern __shared__ float part[];                  // [TOKS][blockDim.x] partial dots (not used with SHFL)
    const TIO *x = blockIdx.y ? k : q;
    const float *W = blockIdx.y ? Wk : Wq;
    float *out = blockIdx.y ? lk : lq;
    const int vpr = d / N;                           // vectors per head row
    const int hb = blockIdx.z * hpc, nh = min(hpc, H - hb);      // this CTA's heads: hb .. hb + nh - 1
    const int tid = threadIdx.x, gv = hb * vpr + tid;            // gv: vector index inside the token row
    const bool live = tid < nh * vpr;
    const int h = live ? gv / vpr : 0, c0 = live ? (gv % vpr) * N : 0;
    float w[N];
#pragma unroll
    for (int e = 0; e < N; ++e) w[e] = live ? __ldg(W + (size_t)(c0 + e) * H + h) : 0.f;
    // blocks of NT tokens are dealt round robin to the CTAs: at any moment the whole grid reads one contiguous stretch
    // of memory (DRAM pages stay open), not one far-apart stream per CTA
    const long t1 = n_tok;
    for (long t = (long)blockIdx.x * NT; t < t1; t += (long)gridDim.x * NT) {
        uint4 raw[NT];
#pragma unroll
        for (int s = 0; s < NT; ++s)                 // all loads of the block in flight at once
            raw[s] = (live && t + s < t1) ? __ldg(reinterpret_cast<const uint4 *>(x + ((size_t)(t + s) * H) * d + (size_t)gv * N))
                                          : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int s = 0; s < NT; ++s) {
            float acc = 0.f, xv[N];
            Vec<TIO>::widen(raw[s], xv);
#pragma unroll
            for (int e = 0; e < N; ++e) acc = fmaf(xv[e], w[e], acc);
            if (SHFL) {
                for (int o = vpr >> 1; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
                if (live && t + s < t1 && tid % vpr == 0) out[(t + s) * H + h] = acc;
            } else {
                part[s * blockDim.x + tid] = acc;
            }
        }
        if (!SHFL) {
            __syncthreads();
            for (int i = tid; i < NT * nh; i += blockDim.x) {    // (token slot, head): the head's vpr partial dots
                const int s = i / nh, hh = i % nh;
                if (t + s < t1) {
                    float acc = 0.f;
                    for (int j = 0; j < vpr; ++j) acc += part[s * blockDim.x + hh * vpr + j];
                    out[(t + s) * H + hb + hh] = acc;
                }
            }
            __syncthreads();
        }
    }
}

// Backward.  dx += dl W^T in place; per-CTA partial sums of dW into `partial` [2 sides][CTAs][H*d].
template <typename TIO>
__global__ void __launch_bounds__(256, 2)
k_gate_scores_bwd(long n_tok, int H, int d, int hpc, const TIO *__restrict__ q, const TIO *__restrict__ k,
                                  const float *__restrict__ Wq, const float *__restrict__ Wk,
                                  const float *__restrict__ dlq, const float *__restrict__ dlk,
                                  TIO *__restrict__ dq, TIO *__restrict__ dk, float *__restrict__ partial) {
    constexpr int N = Vec<TIO>::N;
    const TIO *x = blockIdx.y ? k : q;
    const float *W = blockIdx.y ? Wk : Wq;
    const float *dl = blockIdx.y ? dlk : dlq;
    TIO *dx = blockIdx.y ? dk : dq;
    const int vpr = d / N, nvec = H * vpr;
    const int hb = blockIdx.z * hpc, nh = min(hpc, H - hb);
    const int tid = threadIdx.x, gv = hb * vpr + tid;
    if (tid >= nh * vpr) return;
    const int h = gv / vpr, c0 = (gv % vpr) * N;
    float w[N], acc[N];
#pragma unroll
    for (int e = 0; e < N; ++e) {
        w[e] = __ldg(W + (size_t)(c0 + e) * H + h);
        acc[e] = 0.f;
    }
    constexpr int UNR = 8;       // tokens whose loads (kept packed, 16 bytes each) are all in flight before the first
                                 // store: the compiler may not move a load of dx above a store to dx on its own
    // blocks of UNR tokens are dealt round robin to the CTAs (the grid sweeps memory as one front)
    const long t1 = n_tok;
    for (long t = (long)blockIdx.x * UNR; t < t1; t += (long)gridDim.x * UNR) {
        uint4 rx[UNR], rg[UNR];
        float g[UNR];
#pragma unroll
        for (int s = 0; s < UNR; ++s) {
            const bool ok = t + s < t1;
            const size_t off = ((size_t)(ok ? t + s : t) * H) * d + (size_t)gv * N;
            rx[s] = __ldg(reinterpret_cast<const uint4 *>(x + off));
            rg[s] = *reinterpret_cast<const uint4 *>(dx + off);
            g[s] = ok ? __ldg(dl + (t + s) * H + h) : 0.f;
        }
#pragma unroll
        for (int s = 0; s < UNR; ++s)
            if (t + s < t1) {
                float xv[N], gvec[N];
                Vec<TIO>::widen(rx[s], xv);
                Vec<TIO>::widen(rg[s], gvec);
#pragma unroll
                for (int e = 0; e < N; ++e) {
                    acc[e] = fmaf(g[s], xv[e], acc[e]);
                    gvec[e] = fmaf(g[s], w[e], gvec[e]);
                }
                Vec<TIO>::store(dx + ((size_t)(t + s) * H) * d + (size_t)gv * N, gvec);
            }
    }
    float *dst = partial + ((size_t)blockIdx.y * gridDim.x + blockIdx.x) * nvec * N + (size_t)gv * N;
#pragma unroll
    for (int e = 0; e < N; ++e) dst[e] = acc[e];
}

// dW[c,h] = sum over the CTAs' partial sums (stored [h][c]): one warp per element, lane l adds the partials of CTAs
// l, l+32, .. in order, then the lanes are folded in a fixed tree - the same bits on every run.  grid (H*d/8, 2 sides).
__global__ void k_gate_scores_dw(int n_cta, int H, int d, const float *__restrict__ partial, float *__restrict__ dWq,
                                 float *__restrict__ dWk) {
    const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31, n = H * d;
    if (i >= n) return;
    const float *src = partial + (size_t)blockIdx.y * n_cta * n + i;
    float acc = 0.f;
    for (int c = lane; c < n_cta; c += 32) acc += src[(size_t)c * n];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) (blockIdx.y ? dWk : dWq)[(size_t)(i % d) * H + i / d] = acc;
}

int score_ctas(long n_tok) {
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long want = 4L * sms;
    return (int)(n_tok < want ? (n_tok > 0 ? n_tok : 1) : want);
}

}  // namespace

size_t gate_scores_workspace_bytes(const Dims &d) {
    return (size_t)2 * score_ctas((long)d.B * d.T) * d.H * d.dk * sizeof(float);
}

int gate_scores_forward(const Dims &d, const void *q, const void *k, const float *Wq, const float *Wk, float *lq,
                        float *lk, cudaStream_t st, Tracer &tr) {
    const long n_tok = (long)d.B * d.T;
    const int N = d.io_bf16 ? 8 : 4, vpr = d.dk / N;
    const int hpc = std::max(1, std::min(d.H, 256 / vpr)), threads = (hpc * vpr + 31) / 32 * 32;   // heads per CTA
    dim3 grid(score_ctas(n_tok), 2, (d.H + hpc - 1) / hpc);
    const size_t smem = (size_t)TOKS * threads * sizeof(float);
    const bool shfl = vpr <= 32 && (vpr & (vpr - 1)) == 0;
#define SLA_SCORES_FWD(TIO, SH) \
    k_gate_scores_fwd<TIO, SH><<<grid, threads, SH ? 0 : smem, st>>>(n_tok, d.H, d.dk, hpc, (const TIO *)q, (const TIO *)k, Wq, Wk, lq, lk)
    if (d.io_bf16) { if (shfl) SLA_SCORES_FWD(__nv_bfloat16, true); else SLA_SCORES_FWD(__nv_bfloat16, false); }
    else { if (shfl) SLA_SCORES_FWD(float, true); else SLA_SCORES_FWD(float, false); }
#undef SLA_SCORES_FWD
    tr.mark("gate_scores_fwd");
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int gate_scores_backward(const Dims &d, const void *q, const void *k, const float *Wq, const float *Wk, const float *dlq,
                         const float *dlk, void *dq, void *dk, float *dWq, float *dWk, float *ws, cudaStream_t st,
                         Tracer &tr) {
    const long n_tok = (long)d.B * d.T;
    const int N = d.io_bf16 ? 8 : 4, vpr = d.dk / N;
    const int hpc = std::max(1, std::min(d.H, 256 / vpr)), threads = (hpc * vpr + 31) / 32 * 32;
    const int ctas = score_ctas(n_tok);
    dim3 grid(ctas, 2, (d.H + hpc - 1) / hpc);
    if (d.io_bf16)
        k_gate_scores_bwd<__nv_bfloat16><<<grid, threads, 0, st>>>(n_tok, d.H, d.dk, hpc, (const __nv_bfloat16 *)q,
                                                                   (const __nv_bfloat16 *)k, Wq, Wk, dlq, dlk,
                                                                   (__nv_bfloat16 *)dq, (__nv_bfloat16 *)dk, ws);
    else
        k_gate_scores_bwd<float><<<grid, threads, 0, st>>>(n_tok, d.H, d.dk, hpc, (const float *)q, (const float *)k, Wq, Wk, dlq,
                                                           dlk, (float *)dq, (float *)dk, ws);
    tr.mark("gate_scores_bwd");
    dim3 g2((d.H * d.dk + 7) / 8, 2);
    k_gate_scores_dw<<<g2, 256, 0, st>>>(ctas, d.H, d.dk, ws, dWq, dWk);
    tr.mark("gate_scores_dw");
    return cudaGetLastError() == cudaSuccess ? 2 : -1;
}

}  // namespace sla
