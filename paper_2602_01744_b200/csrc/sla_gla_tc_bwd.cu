// Softmax-GLA backward on the 5th-generation tensor cores (bf16 I/O, d_k = d_v = 128, chunk 64).
//
// The paper states no gradients; these are the chain rule applied to Eq. 4, 12-13, evaluated chunkwise.
// Two sweeps per (batch, head) sequence, one CTA each, chunk after chunk:
//
//   k_gla_states_tc   forward order.  Recomputes the state S_n at the start of every chunk
//                     (S_{n+1} = diag(e^{b_last})(S_n + kh^T V), Eq. 12 re-associated) with S in TMEM, and
//                     leaves each S_n in global memory as a bf16 image in MMA-operand layout (32 KiB per chunk).
//   k_gla_bwd_tc      reverse order.  Carries dS (fp32, TMEM).  Per chunk, with qh = scale*Gq*q*e^b,
//                     kh = Gk*k*e^-b, dZ = diag(e^{b_last}) dS_{n+1}:
//                       A = tril(qh kh^T)            dA = tril(dO V^T)
//                       dqh^T = kh^T dA^T + S_n dO^T        (128 x 64: key dimension x token)
//                       dkh^T = qh^T dA   + dZ V^T
//                       dV^T  = dO^T A    + dZ^T kh^T
//                       dS_n  = dZ + qh^T dO
//                     The three gradient tiles are produced transposed so that one thread owns one key (value)
//                     dimension and walks the tokens: the log-decay gradient is the in-chunk suffix sum of
//                     qh*dqh - kh*dkh plus rowsum(dS_{n+1} * S_{n+1}) carried from the chunk to the right.
//                     Gate gradients leave as the products Gq*dGq = sum_d qh*dqh, Gk*dGk = sum_d kh*dkh per
//                     (token, head); the softmax backward over heads runs afterwards on [B,T,H].
#include "sla_gla_tc.cuh"

namespace sla {
namespace {

using namespace ptx;
using namespace tc;

// ------------------------------------------------------------------------------------------------
// sweep 1: chunk states
namespace st1 {
constexpr uint32_t STAGE = 2 * TILE_BF16 + TILE_G;      // k, v, log-decay: 64 KiB
constexpr uint32_t OFF_K = 0, OFF_V = TILE_BF16, OFF_G = 2 * TILE_BF16;
constexpr uint32_t OFF_TOT = 2 * STAGE;                 // [16][128] fp32 partial column sums
constexpr uint32_t OFF_EB = OFF_TOT + 16 * D * 4;       // [128] exp(b_last)
constexpr uint32_t OFF_GK = OFF_EB + D * 4;             // [64] Gk
constexpr uint32_t OFF_BAR = OFF_GK + C * 4;            // full[2], z
constexpr uint32_t OFF_TMEM = OFF_BAR + 3 * 8;
constexpr uint32_t SMEM_BYTES = OFF_TMEM + 16 + 1024;
constexpr uint32_t TMEM_COLS = 128;
}  // namespace st1

struct StatesParams {
    const float *lq, *lk, *h0;
    uint8_t *simg;          // [B*H][NT+1][32 KiB] bf16 state images
    int *status;
    int T, H, NT;
};

// thread (row, colhalf) holds 32 consecutive state values of its row: bf16 them into the operand image
__device__ __forceinline__ void store_state_part(uint8_t *img, int row, int colhalf, int part, const float (&v)[32]) {
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        uint4 w;
        w.x = pack_bf16(v[8 * c + 0], v[8 * c + 1]);
        w.y = pack_bf16(v[8 * c + 2], v[8 * c + 3]);
        w.z = pack_bf16(v[8 * c + 4], v[8 * c + 5]);
        w.w = pack_bf16(v[8 * c + 6], v[8 * c + 7]);
        *reinterpret_cast<uint4 *>(img + colhalf * STATE_HALF + swz(row, 4 * part + c)) = w;
    }
}

__global__ void __launch_bounds__(256, 1)
k_gla_states_tc(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                const __grid_constant__ CUtensorMap tm_g, StatesParams p) {
    using namespace st1;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *sm = smem_raw + (base - raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.x, b = bh / p.H, h = bh % p.H;
    const uint32_t bar_full0 = base + OFF_BAR, bar_z = bar_full0 + 16;
    float *tot = reinterpret_cast<float *>(sm + OFF_TOT);
    float *eblast = reinterpret_cast<float *>(sm + OFF_EB);
    float *gk_s = reinterpret_cast<float *>(sm + OFF_GK);
    bool failed = false;

    if (tid == 0) {
        for (int i = 0; i < 3; ++i) mbar_init(bar_full0 + 8 * i, 1);
        fence_mbar_init();
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
        tma_prefetch_desc(&tm_g);
    }
    if (warp == 0) tmem_alloc(base + OFF_TMEM, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(sm + OFF_TMEM);
    const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;
    const int colhalf = warp >> 2;
    const int row = 32 * (warp & 3) + lane;
    uint8_t *img0 = p.simg + (size_t)bh * (p.NT + 1) * STATE_BF16;

    auto issue_tma = [&](int n, int s) {
        const uint32_t bar = bar_full0 + 8 * s, st = base + s * STAGE;
        mbar_expect_tx(bar, STAGE);
        const int t0 = n * C;
        tma_load_4d(st + OFF_K, &tm_k, 0, h, t0, b, bar);
        tma_load_4d(st + OFF_K + HALF_BF16, &tm_k, 64, h, t0, b, bar);
        tma_load_4d(st + OFF_V, &tm_v, 0, h, t0, b, bar);
        tma_load_4d(st + OFF_V + HALF_BF16, &tm_v, 64, h, t0, b, bar);
        tma_load_4d(st + OFF_G, &tm_g, 0, h, t0, b, bar);
    };
    if (tid == 0) issue_tma(0, 0);

    {   // S_0: fp32 into TMEM, bf16 image into slot 0
        const float *src = p.h0 ? p.h0 + ((size_t)bh * D + row) * D + 64 * colhalf : nullptr;
#pragma unroll
        for (int part = 0; part < 2; ++part) {
            float v[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = src ? src[32 * part + j] : 0.f;
            tmem_st32(tmem + lane_base + 64 * colhalf + 32 * part, v);
            store_state_part(img0, row, colhalf, part, v);
        }
        tmem_wait_st();
    }
    tc_fence_before();
    __syncthreads();

    constexpr uint32_t ID_Z = idesc_bf16(128, 128, 1, 1);
    uint32_t ph_full[2] = {0, 0}, ph_z = 0;
    const int rg = tid >> 4, cj = tid & 15;

    for (int n = 0; n < p.NT; ++n) {
        const int s = n & 1;
        const uint32_t st = base + s * STAGE;
        uint8_t *stp = sm + s * STAGE;
        const int t0 = n * C, cn = min(C, p.T - t0);
        if (tid == 0 && n + 1 < p.NT) issue_tma(n + 1, s ^ 1);
        if (tid < C) {
            float gk = 0.f;
            if (tid < cn) {
                const size_t tok = (size_t)b * p.T + t0 + tid;
                gk = head_gates(p.lq + tok * p.H, p.lk + tok * p.H, p.H, h).y;
            }
            gk_s[tid] = gk;
        }
        if (!failed && !mbar_wait_bounded(bar_full0 + 8 * s, ph_full[s])) failed = true;
        ph_full[s] ^= 1;

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
                const float gk = gk_s[r];
                uint4 *kp = reinterpret_cast<uint4 *>(stp + OFF_K + half * HALF_BF16 + swz(r, chunk));
                uint4 kv = *kp;
                uint32_t *kw = reinterpret_cast<uint32_t *>(&kv);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float i0 = __expf(-bsum[2 * e]), i1 = __expf(-bsum[2 * e + 1]);
                    float2 kf = unpack_bf16(kw[e]);
                    kw[e] = pack_bf16(kf.x * gk * i0, kf.y * gk * i1);
                }
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

        if (tid == 0) {
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                tc_mma_bf16(tmem, desc_mnmajor(st + OFF_K, kk, HALF_BF16), desc_mnmajor(st + OFF_V, kk, HALF_BF16), ID_Z, 1);
            tc_commit(bar_z);
        }
        if (!failed && !mbar_wait_bounded(bar_z, ph_z)) failed = true;
        ph_z ^= 1;
        tc_fence_after();
        {   // S_{n+1} = diag(e^{b_last}) (S_n + kh^T V): fp32 back into TMEM, bf16 image into slot n+1
            const float e = eblast[row];
            uint8_t *img = img0 + (size_t)(n + 1) * STATE_BF16;
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                float v[32];
                const uint32_t ta = tmem + lane_base + 64 * colhalf + 32 * part;
                tmem_ld32(ta, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] *= e;
                tmem_st32(ta, v);
                store_state_part(img, row, colhalf, part, v);
            }
            tmem_wait_st();
        }
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    }
    if (failed) atomicExch(p.status, 1);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, TMEM_COLS);
}

// ------------------------------------------------------------------------------------------------
// sweep 2: gradients
namespace st2 {
constexpr uint32_t OFF_Q = 0, OFF_K = TILE_BF16, OFF_V = 2 * TILE_BF16, OFF_DO = 3 * TILE_BF16;
constexpr uint32_t OFF_G = 4 * TILE_BF16;               // fp32 log-decay tile
constexpr uint32_t OFF_E = OFF_G + TILE_G;              // bf16 e^b, laid out like the q tile
constexpr uint32_t OFF_S = OFF_E + TILE_BF16;           // bf16 S_n image
constexpr uint32_t OFF_DZ = OFF_S + STATE_BF16;         // bf16 dZ, same layout
constexpr uint32_t OFF_A = OFF_DZ + STATE_BF16;         // masked A, [64 rows][128 B]
constexpr uint32_t OFF_DA = OFF_A + HALF_BF16;          // masked dA
constexpr uint32_t OFF_TOT = OFF_DA + HALF_BF16;        // [16][128] fp32 partial column sums
constexpr uint32_t OFF_EB = OFF_TOT + 16 * D * 4;       // [128] exp(b_last)
constexpr uint32_t OFF_GQ = OFF_EB + D * 4;             // [64] scale*Gq
constexpr uint32_t OFF_GK = OFF_GQ + C * 4;             // [64] Gk
constexpr uint32_t OFF_R = OFF_GK + C * 4;              // [2 buffers][2 column halves][128] rowsum(dS*S) partials
constexpr uint32_t OFF_UP = OFF_R + 4 * D * 4;          // [128] suffix total of the upper 32 tokens
constexpr uint32_t OFF_RED = OFF_UP + D * 4;            // [2][8 warps][32] gate partial sums
constexpr uint32_t OFF_BAR = OFF_RED + 2 * 8 * 32 * 4;  // g, qk, vdo, s, a, m
constexpr uint32_t OFF_TMEM = OFF_BAR + 6 * 8;
constexpr uint32_t SMEM_BYTES = OFF_TMEM + 16 + 1024;
constexpr uint32_t COL_DS = 0, COL_A = 128, COL_DA = 192, COL_DQ = 256, COL_DK = 320, COL_DV = 384, TMEM_COLS = 512;
static_assert(SMEM_BYTES <= 232448, "shared memory budget");
}  // namespace st2

struct BwdParams {
    const float *lq, *lk, *dht;
    const uint8_t *simg;
    __nv_bfloat16 *dq, *dk, *dv;
    float *dg, *pq, *pk, *dh0;     // pq = Gq*dGq, pk = Gk*dGk per (token, head)
    int *status;
    int T, H, NT;
    float scale;
    unsigned long long *phase_ts;   // optional: block 0 / thread 0 stamps the phases of one chunk
};
#define SLA_TS(k) do { if (p.phase_ts && bh == 0 && tid == 0 && n == 8) p.phase_ts[k] = globaltimer_ns(); } while (0)

// Sum v[j] over the 32 lanes for every j: afterwards lane l holds the total of v[l] in v[0].
__device__ __forceinline__ float warp_transpose_sum(float (&v)[32], int lane) {
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        const bool upper = (lane & off) != 0;
#pragma unroll
        for (int j = 0; j < off; ++j) {
            const float send = upper ? v[j] : v[j + off];
            const float keep = upper ? v[j + off] : v[j];
            v[j] = keep + __shfl_xor_sync(0xffffffffu, send, off);
        }
    }
    return v[0];
}

__global__ void __launch_bounds__(256, 1)
k_gla_bwd_tc(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
             const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
             const __grid_constant__ CUtensorMap tm_g, BwdParams p) {
    using namespace st2;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *sm = smem_raw + (base - raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.x, b = bh / p.H, h = bh % p.H;
    const uint32_t bar_g = base + OFF_BAR, bar_qk = bar_g + 8, bar_vdo = bar_g + 16, bar_s = bar_g + 24,
                   bar_a = bar_g + 32, bar_m = bar_g + 40;
    float *tot = reinterpret_cast<float *>(sm + OFF_TOT);
    float *eblast = reinterpret_cast<float *>(sm + OFF_EB);
    float *gq_s = reinterpret_cast<float *>(sm + OFF_GQ);
    float *gk_s = reinterpret_cast<float *>(sm + OFF_GK);
    float *Rs = reinterpret_cast<float *>(sm + OFF_R);
    float *up = reinterpret_cast<float *>(sm + OFF_UP);
    float *red = reinterpret_cast<float *>(sm + OFF_RED);
    bool failed = false;

    if (tid == 0) {
        for (int i = 0; i < 6; ++i) mbar_init(bar_g + 8 * i, 1);
        fence_mbar_init();
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
        tma_prefetch_desc(&tm_do);
        tma_prefetch_desc(&tm_g);
    }
    if (warp == 0) tmem_alloc(base + OFF_TMEM, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(sm + OFF_TMEM);
    const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;
    const int wh = warp >> 2;                       // column half (state passes) / token half (gradient tiles)
    const int row = 32 * (warp & 3) + lane;         // TMEM lane = key (value) dimension owned by this thread
    const uint8_t *img0 = p.simg + (size_t)bh * (p.NT + 1) * STATE_BF16;
    uint32_t ph_g = 0, ph_qk = 0, ph_vdo = 0, ph_s = 0, ph_a = 0, ph_m = 0;

    auto issue_g = [&](int n) {
        mbar_expect_tx(bar_g, TILE_G);
        tma_load_4d(base + OFF_G, &tm_g, 0, h, n * C, b, bar_g);
    };
    auto issue_rest = [&](int n) {
        const int t0 = n * C;
        mbar_expect_tx(bar_qk, 2 * TILE_BF16);
        tma_load_4d(base + OFF_Q, &tm_q, 0, h, t0, b, bar_qk);
        tma_load_4d(base + OFF_Q + HALF_BF16, &tm_q, 64, h, t0, b, bar_qk);
        tma_load_4d(base + OFF_K, &tm_k, 0, h, t0, b, bar_qk);
        tma_load_4d(base + OFF_K + HALF_BF16, &tm_k, 64, h, t0, b, bar_qk);
        mbar_expect_tx(bar_vdo, 2 * TILE_BF16);
        tma_load_4d(base + OFF_V, &tm_v, 0, h, t0, b, bar_vdo);
        tma_load_4d(base + OFF_V + HALF_BF16, &tm_v, 64, h, t0, b, bar_vdo);
        tma_load_4d(base + OFF_DO, &tm_do, 0, h, t0, b, bar_vdo);
        tma_load_4d(base + OFF_DO + HALF_BF16, &tm_do, 64, h, t0, b, bar_vdo);
        mbar_expect_tx(bar_s, STATE_BF16);
        bulk_load(base + OFF_S, img0 + (size_t)n * STATE_BF16, STATE_HALF, bar_s);
        bulk_load(base + OFF_S + STATE_HALF, img0 + (size_t)n * STATE_BF16 + STATE_HALF, STATE_HALF, bar_s);
    };

    // rowsum(dS * S) over this thread's 64 columns, with dS in registers part by part
    auto rowdot_part = [&](const float (&v)[32], int part) {
        float acc = 0.f;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const uint4 w = *reinterpret_cast<const uint4 *>(sm + OFF_S + wh * STATE_HALF + swz(row, 4 * part + c));
            const uint32_t *ww = reinterpret_cast<const uint32_t *>(&w);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 sf = unpack_bf16(ww[e]);
                acc = fmaf(v[8 * c + 2 * e], sf.x, acc);
                acc = fmaf(v[8 * c + 2 * e + 1], sf.y, acc);
            }
        }
        return acc;
    };

    const int nlast = p.NT - 1;
    if (tid == 0) issue_g(nlast);
    {   // dS_NT = dht (or zero) into TMEM; R_{NT-1} = rowsum(dht * S_NT)
        float rpart = 0.f;
        if (p.dht) {
            if (tid == 0) {
                mbar_expect_tx(bar_s, STATE_BF16);
                bulk_load(base + OFF_S, img0 + (size_t)p.NT * STATE_BF16, STATE_HALF, bar_s);
                bulk_load(base + OFF_S + STATE_HALF, img0 + (size_t)p.NT * STATE_BF16 + STATE_HALF, STATE_HALF, bar_s);
            }
            if (!mbar_wait_bounded(bar_s, ph_s)) failed = true;
            ph_s ^= 1;
        }
        const float *src = p.dht ? p.dht + ((size_t)bh * D + row) * D + 64 * wh : nullptr;
#pragma unroll
        for (int part = 0; part < 2; ++part) {
            float v[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = src ? src[32 * part + j] : 0.f;
            tmem_st32(tmem + lane_base + COL_DS + 64 * wh + 32 * part, v);
            if (p.dht) rpart += rowdot_part(v, part);
        }
        tmem_wait_st();
        Rs[(nlast & 1) * 2 * D + wh * D + row] = rpart;
    }
    tc_fence_before();
    __syncthreads();
    if (tid == 0) issue_rest(nlast);

    constexpr uint32_t ID_A = idesc_bf16(64, 64, 0, 0);
    const int rg = tid >> 4, cj = tid & 15;

    for (int n = nlast; n >= 0; --n) {
        const int t0 = n * C, cn = min(C, p.T - t0);
        SLA_TS(0);
        if (tid < C) {   // head-softmax gates of this chunk's tokens (Eq. 4)
            float gq = 0.f, gk = 0.f;
            if (tid < cn) {
                const size_t tok = (size_t)b * p.T + t0 + tid;
                const float2 g = head_gates(p.lq + tok * p.H, p.lk + tok * p.H, p.H, h);
                gq = p.scale * g.x;
                gk = g.y;
            }
            gq_s[tid] = gq;
            gk_s[tid] = gk;
        }
        if (!failed && !mbar_wait_bounded(bar_g, ph_g)) failed = true;
        ph_g ^= 1;
        if (!failed && !mbar_wait_bounded(bar_qk, ph_qk)) failed = true;
        ph_qk ^= 1;
        SLA_TS(1);

        // cumulative log-decay; qh, kh in place; e^b kept as bf16 for the epilogue
        const float *gs = reinterpret_cast<const float *>(sm + OFF_G);
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
                const uint32_t off = half * HALF_BF16 + swz(r, chunk);
                uint4 *qp = reinterpret_cast<uint4 *>(sm + OFF_Q + off);
                uint4 *kp = reinterpret_cast<uint4 *>(sm + OFF_K + off);
                uint4 qv = *qp, kv = *kp, ev;
                uint32_t *qw = reinterpret_cast<uint32_t *>(&qv), *kw = reinterpret_cast<uint32_t *>(&kv);
                uint32_t *ew = reinterpret_cast<uint32_t *>(&ev);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float e0 = __expf(bsum[2 * e]), e1 = __expf(bsum[2 * e + 1]);
                    const float i0 = __expf(-bsum[2 * e]), i1 = __expf(-bsum[2 * e + 1]);
                    float2 qf = unpack_bf16(qw[e]), kf = unpack_bf16(kw[e]);
                    qw[e] = pack_bf16(qf.x * gq * e0, qf.y * gq * e1);
                    kw[e] = pack_bf16(kf.x * gk * i0, kf.y * gk * i1);
                    ew[e] = pack_bf16(e0, e1);
                }
                *qp = qv;
                *kp = kv;
                *reinterpret_cast<uint4 *>(sm + OFF_E + off) = ev;
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
            if (n > 0) issue_g(n - 1);       // the log-decay tile is consumed: fetch the next one early
            if (!failed && !mbar_wait_bounded(bar_vdo, ph_vdo)) failed = true;
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)   // A = qh kh^T
                tc_mma_bf16(tmem + COL_A, desc_kmajor(base + OFF_Q, kk, HALF_BF16), desc_kmajor(base + OFF_K, kk, HALF_BF16),
                            ID_A, kk > 0);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)   // dA = dO V^T
                tc_mma_bf16(tmem + COL_DA, desc_kmajor(base + OFF_DO, kk, HALF_BF16), desc_kmajor(base + OFF_V, kk, HALF_BF16),
                            ID_A, kk > 0);
            tc_commit(bar_a);
        }
        ph_vdo ^= 1;

        {   // dZ = diag(e^{b_last}) dS_{n+1}: fp32 back into TMEM (dS_n accumulates on it), bf16 operand copy
            const float e = eblast[row];
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                float v[32];
                const uint32_t ta = tmem + lane_base + COL_DS + 64 * wh + 32 * part;
                tmem_ld32(ta, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] *= e;
                tmem_st32(ta, v);
                store_state_part(sm + OFF_DZ, row, wh, part, v);
            }
            tmem_wait_st();
        }
        SLA_TS(3);

        // A, dA: TMEM -> causal mask -> bf16 -> shared memory (row i of an M=64 tile sits in lane 32*(i/16) + i%16)
        if (!failed && !mbar_wait_bounded(bar_a, ph_a)) failed = true;
        ph_a ^= 1;
        tc_fence_after();
        SLA_TS(4);
        {
            const int i = 16 * (warp & 3) + lane;
            const uint32_t col = wh ? COL_DA : COL_A;
            uint8_t *dst = sm + (wh ? OFF_DA : OFF_A);
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                float v[32];
                tmem_ld32(tmem + lane_base + col + 32 * part, v);
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
                        *reinterpret_cast<uint4 *>(dst + swz(i, 4 * part + c)) = w;
                    }
                }
            }
        }
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();
        SLA_TS(5);

        if (tid == 0) {
            if (!failed && !mbar_wait_bounded(bar_s, ph_s)) failed = true;
            tc_fence_after();
            const uint32_t sQ = base + OFF_Q, sK = base + OFF_K, sV = base + OFF_V, sDO = base + OFF_DO,
                           sS = base + OFF_S, sDZ = base + OFF_DZ, sA = base + OFF_A, sDA = base + OFF_DA;
            // dqh^T = kh^T dA^T + S_n dO^T
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                tc_mma_bf16(tmem + COL_DQ, desc_mnmajor(sK, kk, HALF_BF16), desc_kmajor(sDA, kk, 0),
                            idesc_bf16(128, 64, 1, 0), kk > 0);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
                tc_mma_bf16(tmem + COL_DQ, desc_kmajor(sS, kk, STATE_HALF), desc_kmajor(sDO, kk, HALF_BF16),
                            idesc_bf16(128, 64, 0, 0), 1);
            // dkh^T = qh^T dA + dZ V^T
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                tc_mma_bf16(tmem + COL_DK, desc_mnmajor(sQ, kk, HALF_BF16), desc_mnmajor(sDA, kk, HALF_BF16),
                            idesc_bf16(128, 64, 1, 1), kk > 0);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
                tc_mma_bf16(tmem + COL_DK, desc_kmajor(sDZ, kk, STATE_HALF), desc_kmajor(sV, kk, HALF_BF16),
                            idesc_bf16(128, 64, 0, 0), 1);
            // dV^T = dO^T A + dZ^T kh^T
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                tc_mma_bf16(tmem + COL_DV, desc_mnmajor(sDO, kk, HALF_BF16), desc_mnmajor(sA, kk, HALF_BF16),
                            idesc_bf16(128, 64, 1, 1), kk > 0);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
                tc_mma_bf16(tmem + COL_DV, desc_mnmajor(sDZ, kk, STATE_HALF), desc_kmajor(sK, kk, HALF_BF16),
                            idesc_bf16(128, 64, 1, 0), 1);
            // dS_n = dZ + qh^T dO
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                tc_mma_bf16(tmem + COL_DS, desc_mnmajor(sQ, kk, HALF_BF16), desc_mnmajor(sDO, kk, HALF_BF16),
                            idesc_bf16(128, 128, 1, 1), 1);
            tc_commit(bar_m);
        }
        ph_s ^= 1;

        if (!failed && !mbar_wait_bounded(bar_m, ph_m)) failed = true;
        ph_m ^= 1;
        tc_fence_after();
        SLA_TS(6);

        const float *Rcur = Rs + (n & 1) * 2 * D;
        {   // R_{n-1} = rowsum(dS_n * S_n), this thread's 64 columns
            float rpart = 0.f;
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                float v[32];
                tmem_ld32(tmem + lane_base + COL_DS + 64 * wh + 32 * part, v);
                tmem_wait_ld();
                rpart += rowdot_part(v, part);
            }
            Rs[((n & 1) ^ 1) * 2 * D + wh * D + row] = rpart;
        }

        SLA_TS(7);
        // gradient tiles: this thread owns key dimension `row` and tokens 32*wh .. 32*wh+31
        const size_t tok0 = (size_t)b * p.T + t0;
        float sfx[32];
        {
            float dqh[32], dkh[32];
            tmem_ld32(tmem + lane_base + COL_DQ + 32 * wh, dqh);
            tmem_ld32(tmem + lane_base + COL_DK + 32 * wh, dkh);
            tmem_wait_ld();
            const uint32_t dhalf = (uint32_t)(row >> 6) * HALF_BF16, dchunk = (uint32_t)(row & 63) >> 3, dbyte = (row & 7) * 2;
            float run = 0.f;
#pragma unroll
            for (int ii = 31; ii >= 0; --ii) {
                const int i = 32 * wh + ii;
                const uint32_t off = dhalf + swz(i, dchunk) + dbyte;
                const float qh = __bfloat162float(*reinterpret_cast<const __nv_bfloat16 *>(sm + OFF_Q + off));
                const float kh = __bfloat162float(*reinterpret_cast<const __nv_bfloat16 *>(sm + OFF_K + off));
                const float eb = __bfloat162float(*reinterpret_cast<const __nv_bfloat16 *>(sm + OFF_E + off));
                const float pq = qh * dqh[ii], pk = kh * dkh[ii];
                run += pq - pk;
                sfx[ii] = run;
                if (i < cn) {
                    const size_t o = ((tok0 + i) * p.H + h) * D + row;
                    p.dq[o] = __float2bfloat16_rn(gq_s[i] * eb * dqh[ii]);
                    p.dk[o] = __float2bfloat16_rn(gk_s[i] * __fdividef(dkh[ii], eb));
                }
                dqh[ii] = pq;
                dkh[ii] = pk;
            }
            if (wh == 1) up[row] = run + Rcur[row] + Rcur[D + row];
            const float sq = warp_transpose_sum(dqh, lane);
            const float sk = warp_transpose_sum(dkh, lane);
            red[warp * 32 + lane] = sq;
            red[8 * 32 + warp * 32 + lane] = sk;
        }
        SLA_TS(8);
        {   // dV^T -> dv
            float dvt[32];
            tmem_ld32(tmem + lane_base + COL_DV + 32 * wh, dvt);
            tmem_wait_ld();
#pragma unroll
            for (int ii = 0; ii < 32; ++ii) {
                const int i = 32 * wh + ii;
                if (i < cn) p.dv[((tok0 + i) * p.H + h) * D + row] = __float2bfloat16_rn(dvt[ii]);
            }
        }
        SLA_TS(9);
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();
        SLA_TS(10);
        if (tid == 0 && n > 0) issue_rest(n - 1);      // every operand buffer is free again
        tc_fence_after();
        {   // log-decay gradient: in-chunk suffix sum + what flows in from the right of the chunk
            const float offs = wh == 1 ? Rcur[row] + Rcur[D + row] : up[row];
#pragma unroll
            for (int ii = 0; ii < 32; ++ii) {
                const int i = 32 * wh + ii;
                if (i < cn) p.dg[((tok0 + i) * p.H + h) * D + row] = sfx[ii] + offs;
            }
        }
        if (tid < C && tid < cn) {   // Gq*dGq and Gk*dGk of token tid: sum over the four key-dimension quarters
            const int w0 = 4 * (tid >> 5), l = tid & 31;
            float sq = 0.f, sk = 0.f;
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                sq += red[(w0 + w) * 32 + l];
                sk += red[8 * 32 + (w0 + w) * 32 + l];
            }
            p.pq[(tok0 + tid) * p.H + h] = sq;
            p.pk[(tok0 + tid) * p.H + h] = sk;
        }
        __syncthreads();     // red, up, Rs are rewritten by the next chunk
        SLA_TS(11);
    }

    if (p.dh0) {   // dS_0, fp32
        float *dst = p.dh0 + ((size_t)bh * D + row) * D + 64 * wh;
#pragma unroll
        for (int part = 0; part < 2; ++part) {
            float v[32];
            tmem_ld32(tmem + lane_base + COL_DS + 64 * wh + 32 * part, v);
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

// dl_h = P_h - G_h sum_h' P_h'  with P = G * dG  (softmax backward over the heads, Eq. 4), HP lanes per token
template <int HP>
__global__ void k_gate_bwd_prod(const float *__restrict__ lq, const float *__restrict__ lk,
                                const float *__restrict__ Pq, const float *__restrict__ Pk,
                                float *__restrict__ dlq, float *__restrict__ dlk, long n_tok, int H) {
    const float *l = blockIdx.y ? lk : lq;
    const float *P = blockIdx.y ? Pk : Pq;
    float *dl = blockIdx.y ? dlk : dlq;
    long gt = (long)blockIdx.x * blockDim.x + threadIdx.x;
    long tok = gt / HP;
    int h = (int)(gt % HP);
    bool valid = tok < n_tok && h < H;
    float x = valid ? l[tok * H + h] : -INFINITY;
    float m = x;
#pragma unroll
    for (int o = HP / 2; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float e = valid ? expf(x - m) : 0.f;
    float s = e;
#pragma unroll
    for (int o = HP / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    float pv = valid ? P[tok * H + h] : 0.f;
    float ps = pv;
#pragma unroll
    for (int o = HP / 2; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
    if (valid) dl[tok * H + h] = pv - (e / s) * ps;
}

template <int HP>
void launch_gate_bwd_prod(const float *lq, const float *lk, const float *Pq, const float *Pk, float *dlq, float *dlk,
                          long n_tok, int H, cudaStream_t st) {
    long threads = n_tok * HP;
    dim3 grid((unsigned)((threads + 255) / 256), 2);
    k_gate_bwd_prod<HP><<<grid, 256, 0, st>>>(lq, lk, Pq, Pk, dlq, dlk, n_tok, H);
}

}  // namespace

int gla_tc_bwd_configure() {
    if (cudaFuncSetAttribute(k_gla_states_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)st1::SMEM_BYTES) != cudaSuccess)
        return -1;
    if (cudaFuncSetAttribute(k_gla_bwd_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)st2::SMEM_BYTES) != cudaSuccess)
        return -1;
    return 0;
}

int gla_tc_backward(const Dims &d, const BwdArgs &a, int *status, cudaStream_t st, Tracer &tr) {
    CUtensorMap mq, mk, mv, mdo, mg;
    if (!make_map(&mq, a.q, d.B, d.T, d.H, d.dk, false, 64) || !make_map(&mk, a.k, d.B, d.T, d.H, d.dk, false, 64) ||
        !make_map(&mv, a.v, d.B, d.T, d.H, d.dv, false, 64) || !make_map(&mdo, a.dO, d.B, d.T, d.H, d.dv, false, 64) ||
        !make_map(&mg, a.log_decay, d.B, d.T, d.H, d.dk, true, 128))
        return -1;
    // workspace: state images, then the two [B,T,H] gate products
    const size_t bth = (size_t)d.B * d.T * d.H;
    const size_t img_floats = (size_t)d.B * d.H * (d.NT + 1) * (STATE_BF16 / 4);
    uint8_t *simg = reinterpret_cast<uint8_t *>(a.ws);
    float *pq = a.ws + img_floats;
    float *pk = pq + ((bth + 63) & ~(size_t)63);

    StatesParams sp{a.lq, a.lk, a.h0, simg, status, d.T, d.H, d.NT};
    k_gla_states_tc<<<d.B * d.H, 256, st1::SMEM_BYTES, st>>>(mk, mv, mg, sp);
    tr.mark("gla_states_tc");
    BwdParams bp{a.lq, a.lk, a.dht, simg, (__nv_bfloat16 *)a.dq, (__nv_bfloat16 *)a.dk, (__nv_bfloat16 *)a.dv,
                 a.dlog_decay, pq, pk, a.dh0, status, d.T, d.H, d.NT, d.scale, gla_tc_phase_ts()};
    k_gla_bwd_tc<<<d.B * d.H, 256, st2::SMEM_BYTES, st>>>(mq, mk, mv, mdo, mg, bp);
    tr.mark("gla_bwd_tc");
    const long n_tok = (long)d.B * d.T;
    int hp = 1;
    while (hp < d.H) hp <<= 1;
    switch (hp) {
        case 1: launch_gate_bwd_prod<1>(a.lq, a.lk, pq, pk, a.dlq, a.dlk, n_tok, d.H, st); break;
        case 2: launch_gate_bwd_prod<2>(a.lq, a.lk, pq, pk, a.dlq, a.dlk, n_tok, d.H, st); break;
        case 4: launch_gate_bwd_prod<4>(a.lq, a.lk, pq, pk, a.dlq, a.dlk, n_tok, d.H, st); break;
        case 8: launch_gate_bwd_prod<8>(a.lq, a.lk, pq, pk, a.dlq, a.dlk, n_tok, d.H, st); break;
        case 16: launch_gate_bwd_prod<16>(a.lq, a.lk, pq, pk, a.dlq, a.dlk, n_tok, d.H, st); break;
        default: launch_gate_bwd_prod<32>(a.lq, a.lk, pq, pk, a.dlq, a.dlk, n_tok, d.H, st); break;
    }
    tr.mark("gate_bwd");
    return cudaGetLastError() == cudaSuccess ? 3 : -1;
}

}  // namespace sla
