// Feature map of the Gated-DeltaNet instantiation (Experimental setup: "short-convolution module" and SiLU), inside the
// boundary so that its gradient is too: per channel a causal convolution of K <= 4 taps over time, SiLU, and for q and k
// L2 normalisation over the d features of each head,
//     y[b,t,c] = sum_j w[c,j] x[b,t-(K-1)+j,c]      z = y sigmoid(y)      out = z / sqrt(sum_d z^2 + eps)  (or out = z).
// Streaming kernels (HBM-bound): a thread owns one 16-byte vector of the token row [H*d] for the whole launch, its taps
// in registers, and walks the tokens of its CTA's slice of one sequence with a sliding window over time.  The per-head
// sums of the normalisation go through shared memory, a few tokens per barrier.  The reverse pass walks the slice
// backwards (dx of a token needs dy of the next K-1 tokens: a sliding window again, warmed up on the tokens after the
// slice) and recomputes y instead of storing it; weight gradients are summed per thread, written per CTA and reduced
// over the CTAs in a fixed order.
#include "sla_internal.h"

#include <algorithm>

namespace sla {
namespace {

constexpr int KMAX = 4;
constexpr int TOKS = 4;          // tokens between two barriers, forward
constexpr int TOKB = 2;          // ... and backward (more live values per token)

template <typename TIO> struct V;
template <> struct V<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ void widen(const uint4 v, float (&x)[4]) {
        x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y); x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
    }
    static __device__ __forceinline__ void load(const float *p, float (&x)[4]) {
        const float4 v = *reinterpret_cast<const float4 *>(p);
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    }
    static __device__ __forceinline__ void store(float *p, const float (&x)[4]) {
        *reinterpret_cast<float4 *>(p) = make_float4(x[0], x[1], x[2], x[3]);
    }
};
template <> struct V<__nv_bfloat16> {
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

struct ConvDims { int T, H, d, K, per, hpc; float eps; };   // per: tokens of one sequence per CTA; hpc: heads per CTA (grid.z covers H)

// taps of this thread's channels, padded at the front to KMAX: y_t = sum_j wt[j] x[t-3+j]
template <int N>
__device__ __forceinline__ void load_taps(const float *w, int c0, int K, bool live, float (&wt)[KMAX][N]) {
#pragma unroll
    for (int j = 0; j < KMAX; ++j)
#pragma unroll
        for (int e = 0; e < N; ++e) wt[j][e] = (live && j >= KMAX - K) ? __ldg(w + (size_t)(c0 + e) * K + j - (KMAX - K)) : 0.f;
}
// x[b, t, this thread's vector], zero before the sequence start
template <typename TIO, int N>
__device__ __forceinline__ void load_x(const TIO *row0, int t, size_t stride, bool live, float (&x)[N]) {
    if (live && t >= 0) {
        V<TIO>::load(row0 + (size_t)t * stride, x);
    } else {
#pragma unroll
        for (int e = 0; e < N; ++e) x[e] = 0.f;
    }
}

// SHFL: a head's d/N vectors sit in d/N consecutive lanes of one warp (a power of two <= 32), so the per-head sums of
// the normalisation are folded with shuffles and the warps run free of each other; otherwise through shared memory.
template <typename TIO, bool NORM, bool SHFL>
__global__ void __launch_bounds__(256, 2)
k_shortconv_fwd(ConvDims cd, const TIO *__restrict__ x, const float *__restrict__ w, TIO *__restrict__ out) {
    constexpr int N = V<TIO>::N;
    extern __shared__ float sm[];                       // part [TOKS][threads], rinv [TOKS][H]
    float *part = sm, *rinv = sm + TOKS * blockDim.x;
    const int C = cd.H * cd.d, vpr = cd.d / N, tid = threadIdx.x;
    const int hb = blockIdx.z * cd.hpc, nh = min(cd.hpc, cd.H - hb);       // this CTA's heads: hb .. hb + nh - 1
    const bool live = tid < nh * vpr;
    const int h = live ? tid / vpr : 0;                                     // (local head)
    const int gv = hb * vpr + tid;                                          // vector index inside the token row
    float wt[KMAX][N];
    load_taps<N>(w, gv * N, cd.K, live, wt);
    const int b = blockIdx.y, t0 = blockIdx.x * cd.per, t1 = min(cd.T, t0 + cd.per);
    const TIO *xr = x + ((size_t)b * cd.T) * C + (size_t)gv * N;
    TIO *orow = out + ((size_t)b * cd.T) * C + (size_t)gv * N;
    float xm3[N], xm2[N], xm1[N];
    load_x<TIO, N>(xr, t0 - 3, C, live, xm3);
    load_x<TIO, N>(xr, t0 - 2, C, live, xm2);
    load_x<TIO, N>(xr, t0 - 1, C, live, xm1);
    for (int t = t0; t < t1; t += TOKS) {
        float z[TOKS][N];
#pragma unroll
        for (int s = 0; s < TOKS; ++s)                  // all loads of the block in flight at once
            if (t + s < t1) load_x<TIO, N>(xr, t + s, C, live, z[s]);
#pragma unroll
        for (int s = 0; s < TOKS; ++s) {
            float ss = 0.f;
            if (t + s < t1) {
#pragma unroll
                for (int e = 0; e < N; ++e) {
                    const float xc = z[s][e];
                    const float y = fmaf(wt[0][e], xm3[e], fmaf(wt[1][e], xm2[e], fmaf(wt[2][e], xm1[e], wt[3][e] * xc)));
                    z[s][e] = __fdividef(y, 1.f + __expf(-y));
                    ss = fmaf(z[s][e], z[s][e], ss);
                    xm3[e] = xm2[e]; xm2[e] = xm1[e]; xm1[e] = xc;
                }
                if (!NORM && live) V<TIO>::store(orow + (size_t)(t + s) * C, z[s]);
            }
            if (NORM && SHFL) {
                for (int o = vpr >> 1; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
                if (live && t + s < t1) {
                    const float r = 1.f / sqrtf(ss + cd.eps);
#pragma unroll
                    for (int e = 0; e < N; ++e) z[s][e] *= r;
                    V<TIO>::store(orow + (size_t)(t + s) * C, z[s]);
                }
            } else if (NORM) {
                part[s * blockDim.x + tid] = ss;
            }
        }
        if (NORM && !SHFL) {
            __syncthreads();
            if (tid < TOKS * nh) {                      // one thread per (token slot, head)
                const int s = tid / nh, hh = tid % nh;
                float acc = 0.f;
                for (int j = 0; j < vpr; ++j) acc += part[s * blockDim.x + hh * vpr + j];
                rinv[s * cd.hpc + hh] = 1.f / sqrtf(acc + cd.eps);
            }
            __syncthreads();
#pragma unroll
            for (int s = 0; s < TOKS; ++s)
                if (live && t + s < t1) {
                    const float r = rinv[s * cd.hpc + h];
#pragma unroll
                    for (int e = 0; e < N; ++e) z[s][e] *= r;
                    V<TIO>::store(orow + (size_t)(t + s) * C, z[s]);
                }
        }
    }
}

// Forward without state carried from token to token, for heads that are a power-of-two run of lanes: blocks of TB
// tokens of a sequence are dealt round robin to the CTAs; a thread fetches its vector of the block's TB + 3 token rows as
// packed 16-byte values, all in flight together (the three rows before the block come from L2, its neighbour has just
// read them), and widens them one by one as the window moves.  Head sums by shuffles, no shared memory, no barrier.
template <typename TIO, bool NORM>
__global__ void __launch_bounds__(256, 2)
k_shortconv_fwd_blocks(ConvDims cd, int B, const TIO *__restrict__ x, const float *__restrict__ w, TIO *__restrict__ out) {
    constexpr int N = V<TIO>::N;
    constexpr int TB = 8;
    const int C = cd.H * cd.d, vpr = cd.d / N, tid = threadIdx.x;
    const int hb = blockIdx.z * cd.hpc, nh = min(cd.hpc, cd.H - hb);
    const bool live = tid < nh * vpr;
    const int gv = hb * vpr + tid;
    float wt[KMAX][N];
    load_taps<N>(w, gv * N, cd.K, live, wt);
    const int nblk = (cd.T + TB - 1) / TB;
    for (long item = blockIdx.x; item < (long)B * nblk; item += gridDim.x) {
        const int b = (int)(item / nblk), t = (int)(item % nblk) * TB;
        const TIO *xr = x + ((size_t)b * cd.T) * C + (size_t)gv * N;
        TIO *orow = out + ((size_t)b * cd.T) * C + (size_t)gv * N;
        uint4 raw[TB + 3];
#pragma unroll
        for (int s = 0; s < TB + 3; ++s) {
            const int tt = t - 3 + s;
            raw[s] = (live && tt >= 0 && tt < cd.T) ? __ldg(reinterpret_cast<const uint4 *>(xr + (size_t)tt * C)) : make_uint4(0u, 0u, 0u, 0u);
        }
        float xm3[N], xm2[N], xm1[N];
        V<TIO>::widen(raw[0], xm3);
        V<TIO>::widen(raw[1], xm2);
        V<TIO>::widen(raw[2], xm1);
#pragma unroll
        for (int s = 0; s < TB; ++s) {
            float xc[N], z[N], ss = 0.f;
            V<TIO>::widen(raw[s + 3], xc);
#pragma unroll
            for (int e = 0; e < N; ++e) {
                const float y = fmaf(wt[0][e], xm3[e], fmaf(wt[1][e], xm2[e], fmaf(wt[2][e], xm1[e], wt[3][e] * xc[e])));
                z[e] = __fdividef(y, 1.f + __expf(-y));
                ss = fmaf(z[e], z[e], ss);
                xm3[e] = xm2[e]; xm2[e] = xm1[e]; xm1[e] = xc[e];
            }
            if (NORM) {
                for (int o = vpr >> 1; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
                const float r = 1.f / sqrtf(ss + cd.eps);
#pragma unroll
                for (int e = 0; e < N; ++e) z[e] *= r;
            }
            if (live && t + s < cd.T) V<TIO>::store(orow + (size_t)(t + s) * C, z);
        }
    }
}

// Reverse pass.  partial: [CTAs][H*d][KMAX] per-CTA sums of the tap gradients.
template <typename TIO, bool NORM, bool SHFL>
__global__ void __launch_bounds__(256, 2)
k_shortconv_bwd(ConvDims cd, const TIO *__restrict__ x, const float *__restrict__ w, const TIO *__restrict__ dout,
                TIO *__restrict__ dx, float *__restrict__ partial) {
    constexpr int N = V<TIO>::N;
    extern __shared__ float sm[];                       // pss, pdot [TOKB][threads]; ca, cb [TOKB][H]
    float *pss = sm, *pdot = sm + TOKB * blockDim.x, *ca = sm + 2 * TOKB * blockDim.x, *cb = ca + TOKB * cd.hpc;
    const int C = cd.H * cd.d, vpr = cd.d / N, tid = threadIdx.x;
    const int hb = blockIdx.z * cd.hpc, nh = min(cd.hpc, cd.H - hb);
    const bool live = tid < nh * vpr;
    const int h = live ? tid / vpr : 0;
    const int gv = hb * vpr + tid;
    float wt[KMAX][N];
    load_taps<N>(w, gv * N, cd.K, live, wt);
    const int b = blockIdx.y, t0 = blockIdx.x * cd.per, t1 = min(cd.T, t0 + cd.per);
    const int ue = min(cd.T, t1 + KMAX - 1) - 1;        // last token whose dy this CTA needs
    const size_t rowoff = ((size_t)b * cd.T) * C + (size_t)gv * N;
    const TIO *xr = x + rowoff, *gr = dout + rowoff;
    TIO *dxr = dx + rowoff;
    float dy1[N], dy2[N], dy3[N], acc[KMAX][N];         // dy of tokens u+1, u+2, u+3
#pragma unroll
    for (int e = 0; e < N; ++e) {
        dy1[e] = dy2[e] = dy3[e] = 0.f;
#pragma unroll
        for (int j = 0; j < KMAX; ++j) acc[j][e] = 0.f;
    }
    for (int top = ue; top >= t0; top -= TOKB) {
        float zs[TOKB][N], gs[TOKB][N], dz[TOKB][N], fa_r[TOKB], fb_r[TOKB];
#pragma unroll
        for (int s = 0; s < TOKB; ++s) {
            const int u = top - s;
            float ss = 0.f, dot = 0.f;
            fa_r[s] = 1.f;
            fb_r[s] = 0.f;
            if (u >= t0) {
                float x0[N], x1[N], x2[N], x3[N];
                load_x<TIO, N>(xr, u - 3, C, live, x0);
                load_x<TIO, N>(xr, u - 2, C, live, x1);
                load_x<TIO, N>(xr, u - 1, C, live, x2);
                load_x<TIO, N>(xr, u, C, live, x3);
                load_x<TIO, N>(gr, u, C, live, dz[s]);
#pragma unroll
                for (int e = 0; e < N; ++e) {
                    const float y = fmaf(wt[0][e], x0[e], fmaf(wt[1][e], x1[e], fmaf(wt[2][e], x2[e], wt[3][e] * x3[e])));
                    const float sg = __fdividef(1.f, 1.f + __expf(-y));
                    zs[s][e] = y * sg;
                    gs[s][e] = sg * (1.f + y * (1.f - sg));         // d silu / dy
                    ss = fmaf(zs[s][e], zs[s][e], ss);
                    dot = fmaf(zs[s][e], dz[s][e], dot);
                }
            }
            if (NORM && SHFL) {         // out = z / r:  dz = dout / r - z (z . dout) / r^3, the head sums by shuffles
                for (int o = vpr >> 1; o > 0; o >>= 1) {
                    ss += __shfl_xor_sync(0xffffffffu, ss, o);
                    dot += __shfl_xor_sync(0xffffffffu, dot, o);
                }
                const float r = sqrtf(ss + cd.eps);
                fa_r[s] = 1.f / r;
                fb_r[s] = dot / (r * r * r);
            } else if (NORM) {
                pss[s * blockDim.x + tid] = ss;
                pdot[s * blockDim.x + tid] = dot;
            }
        }
        if (NORM && !SHFL) {
            __syncthreads();
            if (tid < TOKB * nh) {
                const int s = tid / nh, hh = tid % nh;
                float a = 0.f, d2 = 0.f;
                for (int j = 0; j < vpr; ++j) {
                    a += pss[s * blockDim.x + hh * vpr + j];
                    d2 += pdot[s * blockDim.x + hh * vpr + j];
                }
                const float r = sqrtf(a + cd.eps);
                ca[s * cd.hpc + hh] = 1.f / r;                      // out = z / r:  dz = dout / r - z (z . dout) / r^3
                cb[s * cd.hpc + hh] = d2 / (r * r * r);
            }
            __syncthreads();
        }
#pragma unroll
        for (int s = 0; s < TOKB; ++s) {
            const int u = top - s;
            if (u < t0) continue;
            float dy[N], dxu[N];
            const float fa = !NORM ? 1.f : SHFL ? fa_r[s] : ca[s * cd.hpc + h], fb = !NORM ? 0.f : SHFL ? fb_r[s] : cb[s * cd.hpc + h];
#pragma unroll
            for (int e = 0; e < N; ++e) {
                dy[e] = (dz[s][e] * fa - zs[s][e] * fb) * gs[s][e];
                dxu[e] = fmaf(wt[3][e], dy[e], fmaf(wt[2][e], dy1[e], fmaf(wt[1][e], dy2[e], wt[0][e] * dy3[e])));
            }
            if (u < t1 && live) {                                   // this CTA's own tokens: dx out, tap gradients in
                V<TIO>::store(dxr + (size_t)u * C, dxu);
#pragma unroll
                for (int j = 0; j < KMAX; ++j) {
                    float xv[N];
                    load_x<TIO, N>(xr, u - (KMAX - 1) + j, C, true, xv);
#pragma unroll
                    for (int e = 0; e < N; ++e) acc[j][e] = fmaf(dy[e], xv[e], acc[j][e]);
                }
            }
#pragma unroll
            for (int e = 0; e < N; ++e) { dy3[e] = dy2[e]; dy2[e] = dy1[e]; dy1[e] = dy[e]; }
        }
    }
    if (live) {
        float *dst = partial + (((size_t)blockIdx.y * gridDim.x + blockIdx.x) * C + (size_t)gv * N) * KMAX;
#pragma unroll
        for (int e = 0; e < N; ++e)
#pragma unroll
            for (int j = 0; j < KMAX; ++j) dst[e * KMAX + j] = acc[j][e];
    }
}

// Reverse pass without state carried from block to block (bf16, heads that are a power-of-two run of lanes): blocks of
// TB tokens are dealt round robin to the CTAs; a thread owns FOUR channels and fetches, packed and all in flight together,
// the TB + 6 rows of x and the TB + 3 rows of dout its block needs (dx of a token needs dy of the three tokens after it,
// each of which needs the three rows of x before it; the overlap with the neighbouring blocks comes from L2).  It then
// walks the block backwards with the window in registers: every row is widened once and serves y, dx and the tap
// gradients.  Head sums by shuffles, no shared memory, no barrier.  Tap gradients are summed per thread over its blocks
// and written per CTA.
template <bool NORM>
__global__ void __launch_bounds__(256, 2)
k_shortconv_bwd_blocks(ConvDims cd, int B, const __nv_bfloat16 *__restrict__ x, const float *__restrict__ w,
                       const __nv_bfloat16 *__restrict__ dout, __nv_bfloat16 *__restrict__ dx, float *__restrict__ partial) {
    constexpr int N = 4, TB = 8;
    const int C = cd.H * cd.d, vpr = cd.d / N, tid = threadIdx.x;
    const int hb = blockIdx.z * cd.hpc, nh = min(cd.hpc, cd.H - hb);
    const bool live = tid < nh * vpr;
    const int gv = hb * vpr + tid;
    float wt[KMAX][N], acc[KMAX][N];
    load_taps<N>(w, gv * N, cd.K, live, wt);
#pragma unroll
    for (int j = 0; j < KMAX; ++j)
#pragma unroll
        for (int e = 0; e < N; ++e) acc[j][e] = 0.f;
    auto widen = [](const uint2 v, float (&f)[N]) {
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&v.x));
        const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&v.y));
        f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y;
    };
    const int nblk = (cd.T + TB - 1) / TB;
    for (long item = blockIdx.x; item < (long)B * nblk; item += gridDim.x) {
        const int b = (int)(item / nblk), t = (int)(item % nblk) * TB;
        const size_t rowoff = ((size_t)b * cd.T) * C + (size_t)gv * N;
        const __nv_bfloat16 *xr = x + rowoff, *gr = dout + rowoff;
        uint2 rx[TB + 6], rg[TB + 3];                   // x rows t-3 .. t+TB+2, dout rows t .. t+TB+2 (zero outside the sequence)
#pragma unroll
        for (int s = 0; s < TB + 6; ++s) {
            const int tt = t - 3 + s;
            rx[s] = (live && tt >= 0 && tt < cd.T) ? __ldg(reinterpret_cast<const uint2 *>(xr + (size_t)tt * C)) : make_uint2(0u, 0u);
        }
#pragma unroll
        for (int s = 0; s < TB + 3; ++s) {
            const int tt = t + s;
            rg[s] = (live && tt < cd.T) ? __ldg(reinterpret_cast<const uint2 *>(gr + (size_t)tt * C)) : make_uint2(0u, 0u);
        }
        float x1[N], x2[N], x3[N], dy1[N], dy2[N], dy3[N];      // x of tokens u-2, u-1, u; dy of tokens u+1, u+2, u+3
        widen(rx[TB + 3], x1);
        widen(rx[TB + 4], x2);
        widen(rx[TB + 5], x3);
#pragma unroll
        for (int e = 0; e < N; ++e) dy1[e] = dy2[e] = dy3[e] = 0.f;
#pragma unroll
        for (int s = TB + 2; s >= 0; --s) {             // token u = t + s; past the sequence end dout = 0 makes dy = 0
            float x0[N], g[N], z[N], gs[N], dy[N], ss = 0.f, dot = 0.f;
            widen(rx[s], x0);                           // x of token u-3
            widen(rg[s], g);
#pragma unroll
            for (int e = 0; e < N; ++e) {
                const float y = fmaf(wt[0][e], x0[e], fmaf(wt[1][e], x1[e], fmaf(wt[2][e], x2[e], wt[3][e] * x3[e])));
                const float sg = __fdividef(1.f, 1.f + __expf(-y));
                z[e] = y * sg;
                gs[e] = sg * (1.f + y * (1.f - sg));            // d silu / dy
                ss = fmaf(z[e], z[e], ss);
                dot = fmaf(z[e], g[e], dot);
            }
            float fa = 1.f, fb = 0.f;
            if (NORM) {                                 // out = z / r:  dz = dout / r - z (z . dout) / r^3
                for (int o = vpr >> 1; o > 0; o >>= 1) {
                    ss += __shfl_xor_sync(0xffffffffu, ss, o);
                    dot += __shfl_xor_sync(0xffffffffu, dot, o);
                }
                const float ri = rsqrtf(ss + cd.eps);
                fa = ri;
                fb = dot * ri * ri * ri;
            }
#pragma unroll
            for (int e = 0; e < N; ++e) dy[e] = (g[e] * fa - z[e] * fb) * gs[e];
            if (s < TB) {                               // this block's own tokens: dx out, tap gradients in
                __nv_bfloat162 lo = __floats2bfloat162_rn(
                    fmaf(wt[3][0], dy[0], fmaf(wt[2][0], dy1[0], fmaf(wt[1][0], dy2[0], wt[0][0] * dy3[0]))),
                    fmaf(wt[3][1], dy[1], fmaf(wt[2][1], dy1[1], fmaf(wt[1][1], dy2[1], wt[0][1] * dy3[1]))));
                __nv_bfloat162 hi = __floats2bfloat162_rn(
                    fmaf(wt[3][2], dy[2], fmaf(wt[2][2], dy1[2], fmaf(wt[1][2], dy2[2], wt[0][2] * dy3[2]))),
                    fmaf(wt[3][3], dy[3], fmaf(wt[2][3], dy1[3], fmaf(wt[1][3], dy2[3], wt[0][3] * dy3[3]))));
                if (live && t + s < cd.T)
                    *reinterpret_cast<uint2 *>(dx + rowoff + (size_t)(t + s) * C) =
                        make_uint2(*reinterpret_cast<uint32_t *>(&lo), *reinterpret_cast<uint32_t *>(&hi));
#pragma unroll
                for (int e = 0; e < N; ++e) {
                    acc[0][e] = fmaf(dy[e], x0[e], acc[0][e]);
                    acc[1][e] = fmaf(dy[e], x1[e], acc[1][e]);
                    acc[2][e] = fmaf(dy[e], x2[e], acc[2][e]);
                    acc[3][e] = fmaf(dy[e], x3[e], acc[3][e]);
                }
            }
#pragma unroll
            for (int e = 0; e < N; ++e) {
                dy3[e] = dy2[e]; dy2[e] = dy1[e]; dy1[e] = dy[e];
                x3[e] = x2[e]; x2[e] = x1[e]; x1[e] = x0[e];
            }
        }
    }
    if (live) {
        float *dst = partial + ((size_t)blockIdx.x * C + (size_t)gv * N) * KMAX;
#pragma unroll
        for (int e = 0; e < N; ++e)
            *reinterpret_cast<float4 *>(dst + e * KMAX) = make_float4(acc[0][e], acc[1][e], acc[2][e], acc[3][e]);
    }
}

// dw[c, j] = sum over the CTAs' partial sums: one warp per element, lane l adds the partials of CTAs l, l+32, .. in
// order, then the lanes are folded in a fixed tree (same bits on every run)
__global__ void k_shortconv_dw(int n_cta, int C, int K, const float *__restrict__ partial, float *__restrict__ dw) {
    const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (i >= C * K) return;
    const int c = i / K, j = i % K + (KMAX - K);
    float acc = 0.f;
    for (int n = lane; n < n_cta; n += 32) acc += partial[((size_t)n * C + c) * KMAX + j];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) dw[i] = acc;
}

int tokens_per_cta(const Dims &d) {       // about four CTAs per SM, slices of at least 32 tokens
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long total = (long)d.B * d.T, want = 4L * sms;
    long per = (total + want - 1) / want;
    if (per < 32) per = 32;           // (the reverse pass recomputes three tokens beyond its slice)
    return (int)per;
}

}  // namespace

size_t shortconv_workspace_bytes(const Dims &d, int width) {
    const int per = tokens_per_cta(d);
    const size_t ctas = (size_t)((d.T + per - 1) / per) * d.B;
    return ctas * d.H * width * KMAX * sizeof(float);
}

int shortconv_forward(const Dims &d, int width, int K, bool normalize, float eps, const void *x, const float *w, void *out,
                      cudaStream_t st, Tracer &tr) {
    const int N = d.io_bf16 ? 8 : 4, vpr = width / N;
    const int hpc = std::max(1, std::min(d.H, 256 / vpr)), threads = (hpc * vpr + 31) / 32 * 32;
    ConvDims cd{d.T, d.H, width, K, tokens_per_cta(d), hpc, eps};
    dim3 grid((d.T + cd.per - 1) / cd.per, d.B, (d.H + hpc - 1) / hpc);
    const size_t smem = (size_t)(TOKS * threads + TOKS * hpc) * sizeof(float);
    const bool shfl = vpr <= 32 && (vpr & (vpr - 1)) == 0;
    if (shfl || !normalize) {
        int dev = 0, sms = 148;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const long items = (long)d.B * ((d.T + 7) / 8);
        dim3 g((unsigned)std::min<long>(items, 2L * sms), 1, (d.H + hpc - 1) / hpc);
        if (d.io_bf16) {
            if (normalize) k_shortconv_fwd_blocks<__nv_bfloat16, true><<<g, threads, 0, st>>>(cd, d.B, (const __nv_bfloat16 *)x, w, (__nv_bfloat16 *)out);
            else k_shortconv_fwd_blocks<__nv_bfloat16, false><<<g, threads, 0, st>>>(cd, d.B, (const __nv_bfloat16 *)x, w, (__nv_bfloat16 *)out);
        } else {
            if (normalize) k_shortconv_fwd_blocks<float, true><<<g, threads, 0, st>>>(cd, d.B, (const float *)x, w, (float *)out);
            else k_shortconv_fwd_blocks<float, false><<<g, threads, 0, st>>>(cd, d.B, (const float *)x, w, (float *)out);
        }
        tr.mark("shortconv_fwd");
        return cudaGetLastError() == cudaSuccess ? 1 : -1;
    }
#define SLA_LAUNCH_FWD(TIO, NORM, SH) \
    k_shortconv_fwd<TIO, NORM, SH><<<grid, threads, smem, st>>>(cd, (const TIO *)x, w, (TIO *)out)
    if (d.io_bf16) {
        if (!normalize) SLA_LAUNCH_FWD(__nv_bfloat16, false, true);
        else if (shfl) SLA_LAUNCH_FWD(__nv_bfloat16, true, true);
        else SLA_LAUNCH_FWD(__nv_bfloat16, true, false);
    } else {
        if (!normalize) SLA_LAUNCH_FWD(float, false, true);
        else if (shfl) SLA_LAUNCH_FWD(float, true, true);
        else SLA_LAUNCH_FWD(float, true, false);
    }
#undef SLA_LAUNCH_FWD
    tr.mark("shortconv_fwd");
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int shortconv_backward(const Dims &d, int width, int K, bool normalize, float eps, const void *x, const float *w,
                       const void *dout, void *dx, float *dw, float *ws, cudaStream_t st, Tracer &tr) {
    const int N = d.io_bf16 ? 8 : 4, vpr = width / N;
    const int hpc = std::max(1, std::min(d.H, 256 / vpr)), threads = (hpc * vpr + 31) / 32 * 32;
    ConvDims cd{d.T, d.H, width, K, tokens_per_cta(d), hpc, eps};
    dim3 grid((d.T + cd.per - 1) / cd.per, d.B, (d.H + hpc - 1) / hpc);
    const size_t smem = (size_t)(2 * TOKB * threads + 2 * TOKB * hpc) * sizeof(float);
    const bool shfl = vpr <= 32 && (vpr & (vpr - 1)) == 0;
    const int C = d.H * width;
    const int vpr4 = width / 4;
    if (d.io_bf16 && vpr4 <= 32 && (vpr4 & (vpr4 - 1)) == 0) {
        int dev = 0, sms = 148;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const int hpc4 = std::max(1, std::min(d.H, 256 / vpr4)), threads4 = (hpc4 * vpr4 + 31) / 32 * 32;
        ConvDims cd4{d.T, d.H, width, K, cd.per, hpc4, eps};
        // (no more CTAs than the workspace has partial-sum slots for)
        const long slots = (long)grid.x * grid.y;
        dim3 g((unsigned)std::min<long>(slots, 2L * sms), 1, (d.H + hpc4 - 1) / hpc4);
        if (normalize) k_shortconv_bwd_blocks<true><<<g, threads4, 0, st>>>(cd4, d.B, (const __nv_bfloat16 *)x, w, (const __nv_bfloat16 *)dout, (__nv_bfloat16 *)dx, ws);
        else k_shortconv_bwd_blocks<false><<<g, threads4, 0, st>>>(cd4, d.B, (const __nv_bfloat16 *)x, w, (const __nv_bfloat16 *)dout, (__nv_bfloat16 *)dx, ws);
        tr.mark("shortconv_bwd");
        k_shortconv_dw<<<(C * K + 7) / 8, 256, 0, st>>>((int)g.x, C, K, ws, dw);
        tr.mark("shortconv_dw");
        return cudaGetLastError() == cudaSuccess ? 2 : -1;
    }
#define SLA_LAUNCH_BWD(TIO, NORM, SH) \
    k_shortconv_bwd<TIO, NORM, SH><<<grid, threads, smem, st>>>(cd, (const TIO *)x, w, (const TIO *)dout, (TIO *)dx, ws)
    if (d.io_bf16) {
        if (!normalize) SLA_LAUNCH_BWD(__nv_bfloat16, false, true);
        else if (shfl) SLA_LAUNCH_BWD(__nv_bfloat16, true, true);
        else SLA_LAUNCH_BWD(__nv_bfloat16, true, false);
    } else {
        if (!normalize) SLA_LAUNCH_BWD(float, false, true);
        else if (shfl) SLA_LAUNCH_BWD(float, true, true);
        else SLA_LAUNCH_BWD(float, true, false);
    }
#undef SLA_LAUNCH_BWD
    tr.mark("shortconv_bwd");
    k_shortconv_dw<<<(C * K + 7) / 8, 256, 0, st>>>((int)(grid.x * grid.y), C, K, ws, dw);
    tr.mark("shortconv_dw");
    return cudaGetLastError() == cudaSuccess ? 2 : -1;
}

}  // namespace sla
