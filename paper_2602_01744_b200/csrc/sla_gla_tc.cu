// Softmax-GLA forward on the 5th-generation tensor cores (bf16 I/O, d_k = d_v = 128, chunk 64).
//
// One CTA owns one (batch, head) sequence and walks its chunks in order, so q, k, v, log-decay are
// read from HBM exactly once and o is written once; nothing else touches HBM.
// Per chunk (local token i, cumulative log-decay b_i, gates folded in):
//   TMA      q, k, v (bf16, 128B-swizzled tiles) and log-decay (fp32) of the NEXT chunk -> shared memory
//   CUDA     gates = softmax over heads (Eq. 4); b = cumsum(log-decay); qh = scale*Gq*q*e^b, kh = Gk*k*e^-b
//            written back in place (the swizzled tiles are the MMA operands)
//   tcgen05  A = qh kh^T (M64 N64 K128) ; O = qh S (M64 N128 K128) ; S += kh^T V (M128 N128 K64)  -> TMEM
//   CUDA     A -> causal mask -> bf16 -> shared memory
//   tcgen05  O += A V (M64 N128 K64)
//   CUDA     S <- diag(e^{b_last}) S (TMEM, fp32) and its bf16 copy in shared memory for the next chunk;
//            O -> bf16 -> HBM
// The state never leaves the SM: fp32 in TMEM (Eq. 12's S), bf16 copy in shared memory as MMA operand.
#include "sla_gla_tc.cuh"

namespace sla {
namespace {

using namespace ptx;
using namespace tc;

constexpr uint32_t STAGE = 3 * TILE_BF16 + TILE_G;  // 80 KiB
constexpr uint32_t OFF_Q = 0, OFF_K = TILE_BF16, OFF_V = 2 * TILE_BF16, OFF_G = 3 * TILE_BF16;
constexpr uint32_t OFF_S = 2 * STAGE;               // bf16 state operand: two halves of [128 rows][128 B]
constexpr uint32_t OFF_A = OFF_S + 2 * D * 128;     // masked A, [64 rows][128 B]
constexpr uint32_t OFF_TOT = OFF_A + C * 128;       // [16][128] fp32 partial column sums
constexpr uint32_t OFF_EB = OFF_TOT + 16 * D * 4;   // [128] exp(b_last)
constexpr uint32_t OFF_GQ = OFF_EB + D * 4;         // [64] scale*Gq
constexpr uint32_t OFF_GK = OFF_GQ + C * 4;         // [64] Gk
constexpr uint32_t OFF_BAR = OFF_GK + C * 4;        // mbarriers: full[2], a, z, o
constexpr uint32_t OFF_TMEM = OFF_BAR + 5 * 8;
constexpr uint32_t SMEM_BYTES = OFF_TMEM + 16 + 1024;   // + slack to align the base to 1024 B

constexpr uint32_t COL_A = 0, COL_O = 64, COL_S = 192, TMEM_COLS = 512;

struct FwdParams {
    const float *lq, *lk, *h0;
    __nv_bfloat16 *o;
    float *ht;
    int *status;
    int T, H, NT;
    float scale;
    unsigned long long *phase_ts;   // optional: block 0 / thread 0 writes a timestamp at each phase of chunk 8
};
#define SLA_TS(k) do { if (p.phase_ts && bh == 0 && tid == 0 && n == 8) p.phase_ts[k] = globaltimer_ns(); } while (0)

__global__ void __launch_bounds__(256, 1)
k_gla_fwd_tc(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
             const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_g, FwdParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *sm = smem_raw + (base - raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.x, b = bh / p.H, h = bh % p.H;
    const uint32_t bar_full0 = base + OFF_BAR, bar_a = bar_full0 + 16, bar_z = bar_full0 + 24, bar_o = bar_full0 + 32;
    float *tot = reinterpret_cast<float *>(sm + OFF_TOT);
    float *eblast = reinterpret_cast<float *>(sm + OFF_EB);
    float *gq_s = reinterpret_cast<float *>(sm + OFF_GQ);
    float *gk_s = reinterpret_cast<float *>(sm + OFF_GK);
    bool failed = false;

    if (tid == 0) {
        for (int i = 0; i < 5; ++i) mbar_init(bar_full0 + 8 * i, 1);
        fence_mbar_init();
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
        tma_prefetch_desc(&tm_g);
    }
    if (warp == 0) tmem_alloc(base + OFF_TMEM, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(sm + OFF_TMEM);
    const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;   // this warp's TMEM lane quarter
    const int colhalf = warp >> 2;                                   // which 64 state / output columns

    auto issue_tma = [&](int n, int s) {
        const uint32_t bar = bar_full0 + 8 * s, st = base + s * STAGE;
        mbar_expect_tx(bar, STAGE);
        const int t0 = n * C;
        tma_load_4d(st + OFF_Q, &tm_q, 0, h, t0, b, bar);
        tma_load_4d(st + OFF_Q + HALF_BF16, &tm_q, 64, h, t0, b, bar);
        tma_load_4d(st + OFF_K, &tm_k, 0, h, t0, b, bar);
        tma_load_4d(st + OFF_K + HALF_BF16, &tm_k, 64, h, t0, b, bar);
        tma_load_4d(st + OFF_V, &tm_v, 0, h, t0, b, bar);
        tma_load_4d(st + OFF_V + HALF_BF16, &tm_v, 64, h, t0, b, bar);
        tma_load_4d(st + OFF_G, &tm_g, 0, h, t0, b, bar);
    };
    if (tid == 0) issue_tma(0, 0);

    {   // initial state: fp32 into TMEM, bf16 copy into shared memory (row = key dimension)
        const int row = 32 * (warp & 3) + lane;
        const float *src = p.h0 ? p.h0 + ((size_t)bh * D + row) * D + 64 * colhalf : nullptr;
#pragma unroll
        for (int part = 0; part < 2; ++part) {
            float v[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = src ? src[32 * part + j] : 0.f;
            tmem_st32(tmem + lane_base + COL_S + 64 * colhalf + 32 * part, v);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint4 w;
                w.x = pack_bf16(v[8 * c + 0], v[8 * c + 1]);
                w.y = pack_bf16(v[8 * c + 2], v[8 * c + 3]);
                w.z = pack_bf16(v[8 * c + 4], v[8 * c + 5]);
                w.w = pack_bf16(v[8 * c + 6], v[8 * c + 7]);
                *reinterpret_cast<uint4 *>(sm + OFF_S + colhalf * (D * 128) + swz(row, 4 * part + c)) = w;
            }
        }
        tmem_wait_st();
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();

    constexpr uint32_t ID_A = idesc_bf16(64, 64, 0, 0);      // qh (K-major) x kh (K-major)
    constexpr uint32_t ID_O1 = idesc_bf16(64, 128, 0, 1);    // qh (K-major) x S (MN-major)
    constexpr uint32_t ID_O2 = idesc_bf16(64, 128, 0, 1);    // A (K-major) x V (MN-major)
    constexpr uint32_t ID_Z = idesc_bf16(128, 128, 1, 1);    // kh^T (MN-major) x V (MN-major)
    uint32_t ph_full[2] = {0, 0}, ph_a = 0, ph_z = 0, ph_o = 0;
    const int rg = tid >> 4, cj = tid & 15;                   // prologue: rows 4rg..4rg+3, columns 8cj..8cj+7

    for (int n = 0; n < p.NT; ++n) {
        const int s = n & 1;
        const uint32_t st = base + s * STAGE;
        uint8_t *stp = sm + s * STAGE;
        const int t0 = n * C, cn = min(C, p.T - t0);
        if (tid == 0 && n + 1 < p.NT) issue_tma(n + 1, s ^ 1);
        SLA_TS(0);

        if (tid < C) {   // a1: head-softmax gates of this chunk's tokens (Eq. 4)
            float gq = 0.f, gk = 0.f;
            if (tid < cn) {
                const float *l1 = p.lq + ((size_t)b * p.T + t0 + tid) * p.H;
                const float *l2 = p.lk + ((size_t)b * p.T + t0 + tid) * p.H;
                float m1 = -INFINITY, m2 = -INFINITY;
                for (int j = 0; j < p.H; ++j) { m1 = fmaxf(m1, l1[j]); m2 = fmaxf(m2, l2[j]); }
                float s1 = 0.f, s2 = 0.f;
                for (int j = 0; j < p.H; ++j) { s1 += expf(l1[j] - m1); s2 += expf(l2[j] - m2); }
                gq = p.scale * expf(l1[h] - m1) / s1;
                gk = expf(l2[h] - m2) / s2;
            }
            gq_s[tid] = gq;
            gk_s[tid] = gk;
        }
        if (!failed && !mbar_wait_bounded(bar_full0 + 8 * s, ph_full[s])) failed = true;
        ph_full[s] ^= 1;
        SLA_TS(1);

        // a2: chunk-local cumulative log-decay, two-level: per-4-row partial sums, then a running sum
        const float *gs = reinterpret_cast<const float *>(stp + OFF_G);
        {
            float acc[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = 0.f;
#pragma unroll
            for (int rr = 0; rr < 4; ++rr) {
                const float4 g0 = *reinterpret_cast<const float4 *>(gs + (4 * rg + rr) * D + 8 * cj);
                const float4 g1 = *reinterpret_cast<const float4 *>(gs + (4 * rg + rr) * D + 8 * cj + 4);
                acc[0] += g0.x; acc[1] += g0.y; acc[2] += g0.z; acc[3] += g0.w;
                acc[4] += g1.x; acc[5] += g1.y; acc[6] += g1.z; acc[7] += g1.w;
            }
            *reinterpret_cast<float4 *>(tot + rg * D + 8 * cj) = make_float4(acc[0], acc[1], acc[2], acc[3]);
            *reinterpret_cast<float4 *>(tot + rg * D + 8 * cj + 4) = make_float4(acc[4], acc[5], acc[6], acc[7]);
        }
        __syncthreads();
        {
            float bsum[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) bsum[e] = 0.f;
            for (int g = 0; g < rg; ++g) {
                const float4 a0 = *reinterpret_cast<const float4 *>(tot + g * D + 8 * cj);
                const float4 a1 = *reinterpret_cast<const float4 *>(tot + g * D + 8 * cj + 4);
                bsum[0] += a0.x; bsum[1] += a0.y; bsum[2] += a0.z; bsum[3] += a0.w;
                bsum[4] += a1.x; bsum[5] += a1.y; bsum[6] += a1.z; bsum[7] += a1.w;
            }
            const uint32_t half = cj >> 3, chunk = cj & 7;
#pragma unroll
            for (int rr = 0; rr < 4; ++rr) {
                const int r = 4 * rg + rr;
                const float4 g0 = *reinterpret_cast<const float4 *>(gs + r * D + 8 * cj);
                const float4 g1 = *reinterpret_cast<const float4 *>(gs + r * D + 8 * cj + 4);
                bsum[0] += g0.x; bsum[1] += g0.y; bsum[2] += g0.z; bsum[3] += g0.w;
                bsum[4] += g1.x; bsum[5] += g1.y; bsum[6] += g1.z; bsum[7] += g1.w;
                const float gq = gq_s[r], gk = gk_s[r];
                uint4 *qp = reinterpret_cast<uint4 *>(stp + OFF_Q + half * HALF_BF16 + swz(r, chunk));
                uint4 *kp = reinterpret_cast<uint4 *>(stp + OFF_K + half * HALF_BF16 + swz(r, chunk));
                uint4 qv = *qp, kv = *kp;
                uint32_t *qw = reinterpret_cast<uint32_t *>(&qv), *kw = reinterpret_cast<uint32_t *>(&kv);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float e0 = __expf(bsum[2 * e]), e1 = __expf(bsum[2 * e + 1]);
                    const float i0 = __expf(-bsum[2 * e]), i1 = __expf(-bsum[2 * e + 1]);
                    float2 qf = unpack_bf16(qw[e]), kf = unpack_bf16(kw[e]);
                    qw[e] = pack_bf16(qf.x * gq * e0, qf.y * gq * e1);
                    kw[e] = pack_bf16(kf.x * gk * i0, kf.y * gk * i1);
                }
                *qp = qv;
                *kp = kv;
            }
            if (rg == 15) {
#pragma unroll
                for (int e = 0; e < 8; ++e) eblast[8 * cj + e] = __expf(bsum[e]);
            }
        }
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();
        SLA_TS(2);

        if (tid == 0) {
            tc_fence_after();
            // A = qh kh^T
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint32_t off = (kk >> 2) * HALF_BF16 + (kk & 3) * 32;
                tc_mma_bf16(tmem + COL_A, smem_desc_sw128(st + OFF_Q + off, 16, 1024),
                            smem_desc_sw128(st + OFF_K + off, 16, 1024), ID_A, kk > 0);
            }
            tc_commit(bar_a);
            // O = qh S_prev   (S operand: [K = d_k rows][N = d_v], two 64-column halves 16 KiB apart)
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
                const uint32_t off = (kk >> 2) * HALF_BF16 + (kk & 3) * 32;
                tc_mma_bf16(tmem + COL_O, smem_desc_sw128(st + OFF_Q + off, 16, 1024),
                            smem_desc_sw128(base + OFF_S + kk * 2048, D * 128, 1024), ID_O1, kk > 0);
            }
            // S += kh^T V   (both operands token-major: MN-major descriptors, halves 8 KiB apart)
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                tc_mma_bf16(tmem + COL_S, smem_desc_sw128(st + OFF_K + kk * 2048, HALF_BF16, 1024),
                            smem_desc_sw128(st + OFF_V + kk * 2048, HALF_BF16, 1024), ID_Z, 1);
            tc_commit(bar_z);
        }

        // A: TMEM -> causal mask -> bf16 -> shared memory (row i of the M=64 tile sits in lane 32*(i/16) + i%16)
        if (!failed && !mbar_wait_bounded(bar_a, ph_a)) failed = true;
        ph_a ^= 1;
        tc_fence_after();
        SLA_TS(3);
        if (warp < 4) {
            const int i = 16 * warp + lane;
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                float v[32];
                tmem_ld32(tmem + lane_base + COL_A + 32 * part, v);
                tmem_wait_ld();
                if (lane < 16) {
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const int j0 = 32 * part + 8 * c;
                        uint4 w;
                        w.x = pack_bf16(j0 + 0 <= i ? v[8 * c + 0] : 0.f, j0 + 1 <= i ? v[8 * c + 1] : 0.f);
                        w.y = pack_bf16(j0 + 2 <= i ? v[8 * c + 2] : 0.f, j0 + 3 <= i ? v[8 * c + 3] : 0.f);
                        w.z = pack_bf16(j0 + 4 <= i ? v[8 * c + 4] : 0.f, j0 + 5 <= i ? v[8 * c + 5] : 0.f);
                        w.w = pack_bf16(j0 + 6 <= i ? v[8 * c + 6] : 0.f, j0 + 7 <= i ? v[8 * c + 7] : 0.f);
                        *reinterpret_cast<uint4 *>(sm + OFF_A + swz(i, 4 * part + c)) = w;
                    }
                }
            }
        }
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();
        SLA_TS(4);
        if (tid == 0) {
            tc_fence_after();
            // O += A V
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                tc_mma_bf16(tmem + COL_O, smem_desc_sw128(base + OFF_A + kk * 32, 16, 1024),
                            smem_desc_sw128(st + OFF_V + kk * 2048, HALF_BF16, 1024), ID_O2, 1);
            tc_commit(bar_o);
        }

        // S <- diag(e^{b_last}) S : fp32 back into TMEM, bf16 copy for the next chunk's qh S product
        if (!failed && !mbar_wait_bounded(bar_z, ph_z)) failed = true;
        ph_z ^= 1;
        tc_fence_after();
        SLA_TS(5);
        {
            const int row = 32 * (warp & 3) + lane;
            const float e = eblast[row];
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                float v[32];
                const uint32_t ta = tmem + lane_base + COL_S + 64 * colhalf + 32 * part;
                tmem_ld32(ta, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] *= e;
                tmem_st32(ta, v);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint4 w;
                    w.x = pack_bf16(v[8 * c + 0], v[8 * c + 1]);
                    w.y = pack_bf16(v[8 * c + 2], v[8 * c + 3]);
                    w.z = pack_bf16(v[8 * c + 4], v[8 * c + 5]);
                    w.w = pack_bf16(v[8 * c + 6], v[8 * c + 7]);
                    *reinterpret_cast<uint4 *>(sm + OFF_S + colhalf * (D * 128) + swz(row, 4 * part + c)) = w;
                }
            }
            tmem_wait_st();
        }

        // O: TMEM -> bf16 -> HBM (heads concatenated: row stride H*d_v)
        if (!failed && !mbar_wait_bounded(bar_o, ph_o)) failed = true;
        SLA_TS(6);
        ph_o ^= 1;
        tc_fence_after();
        SLA_TS(7);
        {
            const int i = 16 * (warp & 3) + lane;
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                float v[32];
                tmem_ld32(tmem + lane_base + COL_O + 64 * colhalf + 32 * part, v);
                tmem_wait_ld();
                if (lane < 16 && i < cn) {
                    __nv_bfloat16 *dst = p.o + (((size_t)b * p.T + t0 + i) * p.H + h) * D + 64 * colhalf + 32 * part;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint4 w;
                        w.x = pack_bf16(v[8 * c + 0], v[8 * c + 1]);
                        w.y = pack_bf16(v[8 * c + 2], v[8 * c + 3]);
                        w.z = pack_bf16(v[8 * c + 4], v[8 * c + 5]);
                        w.w = pack_bf16(v[8 * c + 6], v[8 * c + 7]);
                        reinterpret_cast<uint4 *>(dst)[c] = w;
                    }
                }
            }
        }
        SLA_TS(8);
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        SLA_TS(9);
    }

    if (p.ht) {   // final state, fp32
        const int row = 32 * (warp & 3) + lane;
        float *dst = p.ht + ((size_t)bh * D + row) * D + 64 * colhalf;
#pragma unroll
        for (int part = 0; part < 2; ++part) {
            float v[32];
            tmem_ld32(tmem + lane_base + COL_S + 64 * colhalf + 32 * part, v);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; j += 4)
                *reinterpret_cast<float4 *>(dst + 32 * part + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
        }
    }
    if (failed) atomicExch(p.status, 1);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, TMEM_COLS);
}

// ---- host side ----
unsigned long long *g_phase_ts = nullptr;   // set by sla_debug_set_phase_timestamps (profiling aid)
}  // namespace

void gla_tc_set_phase_ts(unsigned long long *p) { g_phase_ts = p; }

bool gla_tc_supported(const Dims &d) {
    return d.variant == SLA_GLA && d.io_bf16 && d.dk == 128 && d.dv == 128 && d.C == 64;
}

int gla_tc_configure() {
    if (!encode_fn()) return -1;
    return cudaFuncSetAttribute(k_gla_fwd_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES) ==
                   cudaSuccess ? 0 : -1;
}

int gla_tc_forward(const Dims &d, const FwdArgs &a, int *status, cudaStream_t st, Tracer &tr) {
    CUtensorMap mq, mk, mv, mg;
    if (!make_map(&mq, a.q, d.B, d.T, d.H, d.dk, false, 64) || !make_map(&mk, a.k, d.B, d.T, d.H, d.dk, false, 64) ||
        !make_map(&mv, a.v, d.B, d.T, d.H, d.dv, false, 64) || !make_map(&mg, a.log_decay, d.B, d.T, d.H, d.dk, true, 128))
        return -1;
    FwdParams p{a.lq, a.lk, a.h0, (__nv_bfloat16 *)a.o, a.ht, status, d.T, d.H, d.NT, d.scale, g_phase_ts};
    k_gla_fwd_tc<<<d.B * d.H, 256, SMEM_BYTES, st>>>(mq, mk, mv, mg, p);
    tr.mark("gla_fwd_tc");
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace sla
