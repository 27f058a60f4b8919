// Device helpers shared by the fp32 CUDA-core chunk kernels.
#pragma once
#include "sla_internal.h"

#include <math.h>

namespace sla {
namespace detail {

constexpr int CMAX = 64;       // largest chunk
constexpr int VS = 16;         // state columns owned by one CTA of the scan kernels
constexpr unsigned FULL = 0xffffffffu;

template <typename T> __device__ __forceinline__ float ldf(const T *p, size_t i);
template <> __device__ __forceinline__ float ldf<float>(const float *p, size_t i) { return p[i]; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16 *p, size_t i) {
    return __bfloat162float(p[i]);
}
template <typename T> __device__ __forceinline__ void stf(T *p, size_t i, float v);
template <> __device__ __forceinline__ void stf<float>(float *p, size_t i, float v) { p[i] = v; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16 *p, size_t i, float v) {
    p[i] = __float2bfloat16_rn(v);
}

__device__ __forceinline__ size_t tok_row(const Dims &d, int b, int t, int h) {
    return ((size_t)b * d.T + t) * d.H + h;
}
// chunk-local cumulative log-decay of token row `row`, key dimension dd
__device__ __forceinline__ float bcum_at(const Dims &d, const float *bcum, size_t row, int dd) {
    return d.variant == SLA_GLA ? bcum[row * d.dk + dd] : bcum[row];
}
__device__ __forceinline__ size_t state_off(const Dims &d, int bh, int n, int slots) {
    return ((size_t)bh * slots + n) * d.dk * d.dv;
}

// ------------------------------------------------------------------------------------------
// Shared-memory tile product used by the per-tile kernels.  256 threads: ty = warp (0..7),
// tx = lane.  Thread (ty,tx) owns rows ty+8r (r<8) and columns tx+32cb (cb<NB) of a 64 x N tile:
//   acc[r][cb] += sum_k A[(ty+8r)*sa_i + k*sa_k] * Bm[k*sb_k + (tx+32cb)*sb_j]
// A reads are warp-wide broadcasts; Bm reads are conflict-free when the stride that multiplies
// the lane index is odd (all tiles are stored with an odd leading dimension).
template <int NB>
__device__ __forceinline__ void tile_gemm(float (&acc)[8][NB], const float *A, int sa_i, int sa_k,
                                          const float *Bm, int sb_k, int sb_j, int K, int N, int ty,
                                          int tx) {
    for (int k = 0; k < K; ++k) {
        float a[8];
#pragma unroll
        for (int r = 0; r < 8; ++r) a[r] = A[(ty + 8 * r) * sa_i + k * sa_k];
#pragma unroll
        for (int cb = 0; cb < NB; ++cb) {
            int j = tx + 32 * cb;
            float bv = (j < N) ? Bm[k * sb_k + j * sb_j] : 0.f;
#pragma unroll
            for (int r = 0; r < 8; ++r) acc[r][cb] = fmaf(a[r], bv, acc[r][cb]);
        }
    }
}

template <int NB> __device__ __forceinline__ void zero_acc(float (&acc)[8][NB]) {
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
        for (int cb = 0; cb < NB; ++cb) acc[r][cb] = 0.f;
}

// Load the decayed, gated operands of one chunk into shared memory (rows >= cn zero-filled).
//   Qs[i][dd] = scale*Gq_i*q*exp(b)   Ks[i][dd] = gk_i*k*exp(-b)   (gk_i = Gk_i, or 1 for GDN)
template <typename TIO>
__device__ __forceinline__ void load_qk_hat(const Dims &d, const TIO *q, const TIO *k,
                                            const float *Gq, const float *Gk, const float *bcum, int b,
                                            int h, int t0, int cn, float *Qs, float *Ks, int ld) {
    for (int idx = threadIdx.x; idx < CMAX * d.dk; idx += blockDim.x) {
        int i = idx / d.dk, dd = idx % d.dk;
        float qv = 0.f, kv = 0.f;
        if (i < cn) {
            size_t row = tok_row(d, b, t0 + i, h);
            float bb = bcum_at(d, bcum, row, dd);
            float gk = d.variant == SLA_GDN ? 1.f : Gk[row];
            if (Qs) qv = d.scale * Gq[row] * ldf(q, row * d.dk + dd) * expf(bb);
            if (Ks) kv = gk * ldf(k, row * d.dk + dd) * expf(-bb);
        }
        if (Qs) Qs[i * ld + dd] = qv;
        if (Ks) Ks[i * ld + dd] = kv;
    }
}


template <typename F> inline bool set_smem(F *fn, size_t bytes) {
    return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) == cudaSuccess;
}

}  // namespace detail
}  // namespace sla
