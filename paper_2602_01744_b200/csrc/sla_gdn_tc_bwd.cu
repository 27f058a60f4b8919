// Softmax-GatedDeltaNet backward on the 5th-generation tensor cores (bf16 I/O, d_k and d_v 128 - or 64, run as 128 with zero padding supplied by the tensor maps -, chunk 64).
//
// The paper states no gradients; these are the chain rule applied to Eq. 4, 14-16 in the chunkwise WY form of the
// forward kernel (sla_gdn_tc.cu), which in save mode leaves per chunk the bf16 state image S_n, U and T.
// One CTA per (batch, head) sequence walks the chunks in reverse order with dS (fp32) in TMEM.  Per chunk, with
//   Gam = e^b, ig = e^{-b}, Qg = scale Gq Gam q, Ke = ig k, Vg = Gk v, dZ = e^{b_last} dS_{n+1},
//   Pq = tril((Qg K^T) ig_j), Lnb = strict_tril(Gam_i ig_j (k_i.k_j)), W = T diag(beta Gam) K, U0 = T diag(beta) Vg:
//   dU   = Pq^T dO + Ke dZ                      dPq = tril(dO U^T)
//   dW   = -dU S_n^T        dKbg = T^T dW       dVb = T^T dU
//   dL   = -strict_tril(dKbg W^T + dVb U0^T)
//   aq   = dO S_n^T + dPq Ke                                  dq = scale Gq Gam aq
//   ak1  = U dZ^T + dPq^T Qg + (beta Gam dL)^T K              dk = ig ak1 + beta Gam (dKbg + dL Ke)
//   dv   = beta Gk dVb          dbeta = rowsum(dL*Lnb) + Gam (dKbg.k) + (dVb.Vg)
//   db   = (Qg.aq) + beta Gam (dKbg.k) + beta rowsum(dL*Lnb) - (Ke.ak1)   (+ <dS_{n+1}, S_{n+1}> on the last row)
//   dlog_decay = suffix sum of db;   dS_n = dZ + Qg^T dO - W^T dU;   Gq dGq = (Qg.aq),  Gk dGk = beta (dVb.Vg).
// Every matrix product is a tcgen05.mma; the operands are bf16 tiles in shared memory that the compute warps
// produce from the accumulators stage by stage (six MMA groups per chunk).  Buffers and TMEM regions are reused as
// their contents die, see the maps below.
#include "sla_gla_tc.cuh"

namespace sla {
namespace {

using namespace ptx;
using namespace tc;

namespace gb {
// shared memory (bytes): name = first content -> later contents
constexpr uint32_t B_Q = 0;                         // q -> Qg -> dk staged for the store
constexpr uint32_t B_K = B_Q + TILE_BF16;           // k
constexpr uint32_t B_V = B_K + TILE_BF16;           // v -> Vg -> dv staged
constexpr uint32_t B_DO = B_V + TILE_BF16;          // dO -> dq staged
constexpr uint32_t B_S = B_DO + TILE_BF16;          // S_n -> [dKbg bf16 | dVb bf16]
constexpr uint32_t B_T = B_S + STATE_BF16;          // T -> beta Gam dL
constexpr uint32_t B_U = B_T + HALF_BF16;           // U -> [dPq | dL]
constexpr uint32_t B_KE = B_U + TILE_BF16;          // Ke
constexpr uint32_t B_DZ = B_KE + TILE_BF16;         // dZ bf16 -> [dU bf16 | -dW bf16]
constexpr uint32_t B_T1 = B_DZ + STATE_BF16;        // T diag(beta Gam) -> Pq
constexpr uint32_t B_T2 = B_T1 + HALF_BF16;         // T diag(beta) -> Lnb
constexpr uint32_t B_WN = B_T2 + HALF_BF16;         // -W
constexpr uint32_t B_U0N = B_WN + TILE_BF16;        // -U0
constexpr uint32_t OFF_SC = B_U0N + TILE_BF16;      // per-token scalars: 18 arrays of 64 floats
constexpr uint32_t OFF_GATE = OFF_SC + 18 * C * 4;  // [4 chunks][4][64]: scale*Gq, Gk, log-decay, beta
constexpr uint32_t OFF_RED = OFF_GATE + 4 * 4 * C * 4;   // [16] CTA-wide reduction scratch, [2] carried <dS,S>
constexpr uint32_t OFF_BAR = OFF_RED + 32 * 4;
constexpr uint32_t OFF_TMEM = OFF_BAR + 48 * 8;     // TMEM base address, then the abort flag
constexpr uint32_t SMEM_BYTES = OFF_TMEM + 16 + 1024;
static_assert(SMEM_BYTES <= 232448, "shared memory budget");
// TMEM regions of 128 columns: R0 = dS; R1: KK|QK -> dU -> dW -> dKbg (+ dL Ke); R2: W -> dPq -> aq -> dVb -> dL;
// R3: U0 -> ak1
constexpr uint32_t R0 = 0, R1 = 128, R2 = 256, R3 = 384, TMEM_COLS = 512;
constexpr int NTHREADS = NCOMPUTE + 32 + NGATE + 32;
enum Bar { FULL_Q = 0, FULL_K, FULL_V, FULL_DO, FULL_S, FULL_T, FULL_U, GREADY /*[4]*/, GFREE = GREADY + 4 /*[4]*/,
           OPR = GFREE + 4, S1R, S2R, S3R, S4R, S5R, S6R, INIT_DONE, C1, C2, C3, C4, C5, C6, SFREE, KFREE, INIT_FULL,
           DRAIN, NBAR };
static_assert(NBAR <= 48, "barrier slots");
enum Sc { SC_B = 0, SC_GAM, SC_IGAM, SC_FQ, SC_BG, SC_BETA, SC_FVB, SC_GK, SC_PQ /*[2]*/, SC_PV = SC_PQ + 2 /*[2]*/,
          SC_RK = SC_PV + 2 /*[2]*/, SC_RL = SC_RK + 2 /*[2]*/, SC_CK = SC_RL + 2 /*[2]*/ };
static_assert(SC_CK + 2 <= 18, "scalar arrays");
}  // namespace gb

constexpr uint32_t REC_S = 0, REC_U = STATE_BF16, REC_T = STATE_BF16 + TILE_BF16, REC_BYTES = STATE_BF16 + TILE_BF16 + HALF_BF16;

struct GdnBwdParams {
    const float *lq, *lk, *g, *beta, *dht;
    const uint8_t *save;            // records of the forward sweep
    float *dg, *dbeta, *pq, *pk, *dh0;
    int *status;
    int T, H, NT;
    float scale;
    const SeqInfo *seqs;            // packed variable-length batch: per-sequence table and tensor maps (the seven below), else nullptr
    const CUtensorMap *vmaps;
    int dk, dv;             // head widths, each 128 or 64 (the upper half of a 128-wide tile is then zero padding)
};

__global__ void __launch_bounds__(gb::NTHREADS, 1)
k_gdn_bwd_tc(const __grid_constant__ CUtensorMap gm_q, const __grid_constant__ CUtensorMap gm_k,
             const __grid_constant__ CUtensorMap gm_v, const __grid_constant__ CUtensorMap gm_do,
             const __grid_constant__ CUtensorMap gm_dq, const __grid_constant__ CUtensorMap gm_dk,
             const __grid_constant__ CUtensorMap gm_dv, GdnBwdParams p) {
    using namespace gb;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *sm = smem_raw + (base - raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.x, h = bh % p.H;
    int b = bh / p.H;
    size_t tokb = (size_t)b * p.T, slot = (size_t)bh * (p.NT + 1);
    size_t sbh = (size_t)bh;                                // (sequence, head) index into h0 / ht / dht / dh0
    const CUtensorMap *vm = nullptr;
    if (p.seqs) {                                           // packed batch: see k_gdn_fwd_tc
        const SeqInfo si = p.seqs[b];
        vm = p.vmaps + (size_t)b * Varlen::MAPS_PER_SEQ;
        p.T = si.T; p.NT = si.NT;
        tokb = (size_t)si.t0;
        slot = (size_t)si.slot0 * p.H + (size_t)h * (si.NT + 1);
        sbh = (size_t)si.id * p.H + h;                      // (the table is ordered longest first, the state tensors as the caller gave them)
        b = 0;
    }
    const CUtensorMap &tm_q = vm ? vm[0] : gm_q, &tm_k = vm ? vm[1] : gm_k, &tm_v = vm ? vm[2] : gm_v, &tm_do = vm ? vm[3] : gm_do,
                      &tm_dq = vm ? vm[4] : gm_dq, &tm_dk = vm ? vm[5] : gm_dk, &tm_dv = vm ? vm[6] : gm_dv;
    const int NT = p.NT;
    auto bar = [&](int i) { return base + OFF_BAR + 8u * i; };
    float *sc = reinterpret_cast<float *>(sm + OFF_SC);
    float *gate_s = reinterpret_cast<float *>(sm + OFF_GATE);
    float *red = reinterpret_cast<float *>(sm + OFF_RED);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(sm + OFF_TMEM + 8);
    bool failed = false;
    auto wait = [&](int i, uint32_t parity) {
        if (!failed && !mbar_wait_bounded(bar(i), parity, abort_flag)) { failed = true; *abort_flag = 1; }
    };
    auto wait_relaxed = [&](int i, uint32_t parity) {
        if (!failed && !mbar_wait_bounded<128>(bar(i), parity, abort_flag)) { failed = true; *abort_flag = 1; }
    };

    if (tid == 0) {
        *abort_flag = 0;
        for (int i = 0; i < NBAR; ++i) {
            const bool all = (i >= GFREE && i <= INIT_DONE);
            mbar_init(bar(i), all ? NCOMPUTE : (i >= GREADY && i < GFREE) ? NGATE / 32 : 1);
        }
        fence_mbar_init();
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
        tma_prefetch_desc(&tm_do);
        tma_prefetch_desc(&tm_dq);
        tma_prefetch_desc(&tm_dk);
        tma_prefetch_desc(&tm_dv);
    }
    if (warp == 0) tmem_alloc(base + OFF_TMEM, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(sm + OFF_TMEM);
    const uint8_t *rec0 = p.save + slot * REC_BYTES;
    // chunks are visited in the order n = NT-1 ... 0; k = NT-1-n is the visit number that drives every barrier parity

    if (warp == 8) {
        // ---------------- MMA issue (one lane) ----------------
        if (lane == 0) {
            constexpr uint32_t I64 = idesc_bf16(64, 64, 0, 0);        // K-major x K-major, 64 x 64
            constexpr uint32_t IKK = idesc_bf16(64, 128, 0, 0);       // K-major x K-major
            constexpr uint32_t IKM = idesc_bf16(64, 128, 0, 1);       // K-major x MN-major
            constexpr uint32_t IMM = idesc_bf16(64, 128, 1, 1);       // MN-major x MN-major
            constexpr uint32_t ISS = idesc_bf16(128, 128, 1, 1);      // state update
            const uint64_t kQ = desc_kmajor(base + B_Q), mQ = desc_mnmajor(base + B_Q, HALF_BF16),
                           kK = desc_kmajor(base + B_K), mK = desc_mnmajor(base + B_K, HALF_BF16),
                           mV = desc_mnmajor(base + B_V, HALF_BF16),
                           kDO = desc_kmajor(base + B_DO), mDO = desc_mnmajor(base + B_DO, HALF_BF16),
                           kS = desc_kmajor(base + B_S), kDK = desc_kmajor(base + B_S), kDV = desc_kmajor(base + B_S + TILE_BF16),
                           mT = desc_mnmajor(base + B_T, HALF_BF16),
                           kU = desc_kmajor(base + B_U), kDP = desc_kmajor(base + B_U), mDP = desc_mnmajor(base + B_U, HALF_BF16),
                           kDL = desc_kmajor(base + B_U + HALF_BF16),
                           kKE = desc_kmajor(base + B_KE), mKE = desc_mnmajor(base + B_KE, HALF_BF16),
                           mDZ = desc_mnmajor(base + B_DZ, STATE_HALF), kDZ = desc_kmajor(base + B_DZ),
                           kDU = desc_kmajor(base + B_DZ), mDU = desc_mnmajor(base + B_DZ, HALF_BF16),
                           mDW = desc_mnmajor(base + B_DZ + TILE_BF16, HALF_BF16),
                           kT1 = desc_kmajor(base + B_T1), mPQ = desc_mnmajor(base + B_T1, HALF_BF16),
                           kT2 = desc_kmajor(base + B_T2),
                           kWN = desc_kmajor(base + B_WN), mWN = desc_mnmajor(base + B_WN, HALF_BF16),
                           kU0 = desc_kmajor(base + B_U0N);
            auto k8 = [](uint32_t kk, uint32_t hs) { return kstep_kmajor(kk, hs); };
            for (int k = 0; k < NT; ++k) {
                const uint32_t par = k & 1;
                // ---- group 1: K K^T | Qg K^T ; W = (T beta Gam) K ; U0 = (T beta) Vg ----
                wait(OPR, par);
                if (failed) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) tc_mma_bf16(tmem + R1, kK + k8(kk, HALF_BF16), kK + k8(kk, HALF_BF16), I64, kk > 0);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) tc_mma_bf16(tmem + R1 + 64, kQ + k8(kk, HALF_BF16), kK + k8(kk, HALF_BF16), I64, kk > 0);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) tc_mma_bf16(tmem + R2, kT1 + k8(kk, 0), mK + kstep_mnmajor(kk), IKM, kk > 0);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) tc_mma_bf16(tmem + R3, kT2 + k8(kk, 0), mV + kstep_mnmajor(kk), IKM, kk > 0);
                tc_commit(bar(C1));
                // ---- group 2: dU = Ke dZ + Pq^T dO ; dPq = dO U^T ; ak1 = U dZ^T ----
                wait(S1R, par);
                wait(FULL_DO, par);
                wait(FULL_U, par);
                if (failed) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) tc_mma_bf16(tmem + R1, kKE + k8(kk, HALF_BF16), mDZ + kstep_mnmajor(kk), IKM, kk > 0);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) tc_mma_bf16(tmem + R1, mPQ + kstep_mnmajor(kk), mDO + kstep_mnmajor(kk), IMM, 1);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) tc_mma_bf16(tmem + R2, kDO + k8(kk, HALF_BF16), kU + k8(kk, HALF_BF16), I64, kk > 0);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) tc_mma_bf16(tmem + R3, kU + k8(kk, HALF_BF16), kDZ + k8(kk, STATE_HALF), IKK, kk > 0);
                tc_commit(bar(C2));
                // ---- group 3: dW = dU S^T ; aq = dO S^T + dPq Ke ; ak1 += dPq^T Qg ; dS += Qg^T dO - W^T dU ----
                wait(S2R, par);
                wait(FULL_S, par);
                if (failed) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) tc_mma_bf16(tmem + R1, kDU + k8(kk, HALF_BF16), kS + k8(kk, STATE_HALF), IKK, kk > 0);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) tc_mma_bf16(tmem + R2, kDO + k8(kk, HALF_BF16), kS + k8(kk, STATE_HALF), IKK, kk > 0);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) tc_mma_bf16(tmem + R2, kDP + k8(kk, 0), mKE + kstep_mnmajor(kk), IKM, 1);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) tc_mma_bf16(tmem + R3, mDP + kstep_mnmajor(kk), mQ + kstep_mnmajor(kk), IMM, 1);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) tc_mma_bf16(tmem + R0, mQ + kstep_mnmajor(kk), mDO + kstep_mnmajor(kk), ISS, 1);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) tc_mma_bf16(tmem + R0, mWN + kstep_mnmajor(kk), mDU + kstep_mnmajor(kk), ISS, 1);
                tc_commit(bar(C3));
                // ---- group 4: dKbg = T^T dW ; dVb = T^T dU ----
                wait(S3R, par);
                if (failed) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) tc_mma_bf16(tmem + R1, mT + kstep_mnmajor(kk), mDW + kstep_mnmajor(kk), IMM, kk > 0);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) tc_mma_bf16(tmem + R2, mT + kstep_mnmajor(kk), mDU + kstep_mnmajor(kk), IMM, kk > 0);
                tc_commit(bar(C4));
                // ---- group 5: dL = dKbg (-W)^T + dVb (-U0)^T ----
                wait(S4R, par);
                if (failed) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) tc_mma_bf16(tmem + R2, kDK + k8(kk, HALF_BF16), kWN + k8(kk, HALF_BF16), I64, kk > 0);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) tc_mma_bf16(tmem + R2, kDV + k8(kk, HALF_BF16), kU0 + k8(kk, HALF_BF16), I64, 1);
                tc_commit(bar(C5));
                tc_commit(bar(SFREE));
                // ---- group 6: dKbg += dL Ke ; ak1 += (beta Gam dL)^T K ----
                wait(S5R, par);
                if (failed) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) tc_mma_bf16(tmem + R1, kDL + k8(kk, 0), mKE + kstep_mnmajor(kk), IKM, 1);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) tc_mma_bf16(tmem + R3, mT + kstep_mnmajor(kk), mK + kstep_mnmajor(kk), IMM, 1);
                tc_commit(bar(C6));
                tc_commit(bar(KFREE));
                wait(S6R, par);                        // the accumulators have been read out before the next chunk reuses them
            }
            tc_commit(bar(DRAIN));
            mbar_wait_bounded(bar(DRAIN), 0, nullptr, 20000000ull);
        }
    } else if (warp == 13) {
        // ---------------- TMA (one lane): loads for the next chunk as buffers die, gradient stores ----------------
        if (lane == 0) {
            auto load_tile = [&](int which, const CUtensorMap *map, uint32_t dst, int n) {
                mbar_expect_tx(bar(which), TILE_BF16);
                tma_load_5d(base + dst, map, 0, n * C, 0, h, b, bar(which));
            };
            auto load_rec = [&](int which, uint32_t dst, int n, uint32_t off, uint32_t bytes) {
                mbar_expect_tx(bar(which), bytes);
                bulk_load(base + dst, rec0 + (size_t)n * REC_BYTES + off, bytes, bar(which));
            };
            const int nl = NT - 1;
            if (p.dht) load_rec(INIT_FULL, B_S, NT, REC_S, STATE_BF16);      // S_NT, for <dht, S_NT>
            load_tile(FULL_Q, &tm_q, B_Q, nl);
            load_tile(FULL_K, &tm_k, B_K, nl);
            load_tile(FULL_V, &tm_v, B_V, nl);
            load_tile(FULL_DO, &tm_do, B_DO, nl);
            load_rec(FULL_T, B_T, nl, REC_T, HALF_BF16);
            load_rec(FULL_U, B_U, nl, REC_U, TILE_BF16);
            if (p.dht) wait(INIT_DONE, 0);
            if (!failed) load_rec(FULL_S, B_S, nl, REC_S, STATE_BF16);
            for (int k = 0; k < NT && !failed; ++k) {
                const int n = NT - 1 - k;
                const uint32_t par = k & 1;
                if (n > 0) {   // the next chunk's q, k and record can only be loaded late in this chunk: have them in L2 by then
                    tma_prefetch_l2_5d(&tm_q, 0, (n - 1) * C, 0, h, b);
                    tma_prefetch_l2_5d(&tm_k, 0, (n - 1) * C, 0, h, b);
                    bulk_prefetch_l2(rec0 + (size_t)(n - 1) * REC_BYTES, REC_BYTES);                        // S, U, T
                }
                wait_relaxed(S3R, par);                // dq staged over dO
                if (failed) break;
                tma_store_5d(&tm_dq, base + B_DO, 0, n * C, 0, h, b);
                bulk_commit();
                wait_relaxed(S4R, par);                // dv staged over Vg
                if (failed) break;
                tma_store_5d(&tm_dv, base + B_V, 0, n * C, 0, h, b);
                bulk_commit();
                bulk_wait_read0();
                if (n > 0) {
                    load_tile(FULL_DO, &tm_do, B_DO, n - 1);
                    load_tile(FULL_V, &tm_v, B_V, n - 1);
                    wait(SFREE, par);                  // group 5 done: the S buffer (dKbg | dVb tiles) is free
                    if (failed) break;
                    load_rec(FULL_S, B_S, n - 1, REC_S, STATE_BF16);
                }
                wait_relaxed(S6R, par);                // dk staged over Qg; every MMA of the chunk is done
                if (failed) break;
                tma_store_5d(&tm_dk, base + B_Q, 0, n * C, 0, h, b);
                bulk_commit();
                if (n > 0) {
                    wait(KFREE, par);
                    if (failed) break;
                    load_tile(FULL_K, &tm_k, B_K, n - 1);
                    load_rec(FULL_T, B_T, n - 1, REC_T, HALF_BF16);
                    load_rec(FULL_U, B_U, n - 1, REC_U, TILE_BF16);
                    bulk_wait_read0();
                    load_tile(FULL_Q, &tm_q, B_Q, n - 1);
                }
            }
            bulk_wait0();
            if (failed) {
                const uint64_t t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
            }
        }
    } else if (warp >= 9) {
        // ---------------- gates and per-token scalars, up to four chunks ahead ----------------
        const int g = tid - (NCOMPUTE + 32), t = g & (C - 1);
        for (int k = 0; k < NT; ++k) {
            const int n = NT - 1 - k;
            if (k >= 4) wait_relaxed(GFREE + (k & 3), ((k >> 2) - 1) & 1);
            if (failed) break;
            const int cn = min(C, p.T - n * C);
            const size_t tok = tokb + (size_t)n * C + t;
            float *dst = gate_s + (k & 3) * 4 * C;
            if (g < C) {
                chunk_gate(p.lq + (tok - t) * p.H, p.H, cn, h, p.scale, dst, t);
                dst[2 * C + t] = t < cn ? p.g[tok * p.H + h] : 0.f;
            } else {
                chunk_gate(p.lk + (tok - t) * p.H, p.H, cn, h, 1.f, dst + C, t);
                dst[3 * C + t] = t < cn ? p.beta[tok * p.H + h] : 0.f;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(GREADY + (k & 3)));
        }
    } else {
        // ---------------- compute warps ----------------
        const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;   // this warp's TMEM lane quarter
        const int ch = warp >> 2;                                        // column half of a 128-column tile
        const int row = 32 * (warp & 3) + lane;                          // state row (M = 128 tiles)
        const int ti = 16 * (warp & 3) + lane;                           // token row (M = 64 tiles; lanes 0..15 only)
        const bool act = lane < 16;

        // this thread's 64 columns of a token-major 128-column accumulator
        auto ld64 = [&](uint32_t col, float (&v0)[32], float (&v1)[32]) {
            tmem_ld32(tmem + lane_base + col + 64 * ch, v0);
            tmem_ld32(tmem + lane_base + col + 64 * ch + 32, v1);
            tmem_wait_ld();
        };
        // f * (v0 | v1) as bf16 into row ti, half ch of a swizzled tile
        auto st_tile = [&](uint8_t *tile, const float (&v0)[32], const float (&v1)[32], float f) {
            if (!act) return;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint4 w;
                w.x = pack_bf16(f * v0[8 * c + 0], f * v0[8 * c + 1]);
                w.y = pack_bf16(f * v0[8 * c + 2], f * v0[8 * c + 3]);
                w.z = pack_bf16(f * v0[8 * c + 4], f * v0[8 * c + 5]);
                w.w = pack_bf16(f * v0[8 * c + 6], f * v0[8 * c + 7]);
                *reinterpret_cast<uint4 *>(tile + ch * HALF_BF16 + swz(ti, c)) = w;
                w.x = pack_bf16(f * v1[8 * c + 0], f * v1[8 * c + 1]);
                w.y = pack_bf16(f * v1[8 * c + 2], f * v1[8 * c + 3]);
                w.z = pack_bf16(f * v1[8 * c + 4], f * v1[8 * c + 5]);
                w.w = pack_bf16(f * v1[8 * c + 6], f * v1[8 * c + 7]);
                *reinterpret_cast<uint4 *>(tile + ch * HALF_BF16 + swz(ti, 4 + c)) = w;
            }
        };
        // sum over this thread's 64 columns of (v0 | v1) * tile[ti][.]
        auto dot_tile = [&](const uint8_t *tile, const float (&v0)[32], const float (&v1)[32]) {
            float acc = 0.f;
            if (!act) return acc;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint4 a = *reinterpret_cast<const uint4 *>(tile + ch * HALF_BF16 + swz(ti, c));
                const uint4 bq = *reinterpret_cast<const uint4 *>(tile + ch * HALF_BF16 + swz(ti, 4 + c));
                const uint32_t *aw = reinterpret_cast<const uint32_t *>(&a), *bw = reinterpret_cast<const uint32_t *>(&bq);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 x = unpack_bf16(aw[e]), y = unpack_bf16(bw[e]);
                    acc = fmaf(v0[8 * c + 2 * e], x.x, acc);
                    acc = fmaf(v0[8 * c + 2 * e + 1], x.y, acc);
                    acc = fmaf(v1[8 * c + 2 * e], y.x, acc);
                    acc = fmaf(v1[8 * c + 2 * e + 1], y.y, acc);
                }
            }
            return acc;
        };
        // <dS, S> over this thread's 64 state columns (dS in registers, S = bf16 image in B_S), summed over the warp
        auto state_dot = [&](const float (&v0)[32], const float (&v1)[32]) {
            float acc = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint4 a = *reinterpret_cast<const uint4 *>(sm + B_S + ch * STATE_HALF + swz(row, c));
                const uint4 bq = *reinterpret_cast<const uint4 *>(sm + B_S + ch * STATE_HALF + swz(row, 4 + c));
                const uint32_t *aw = reinterpret_cast<const uint32_t *>(&a), *bw = reinterpret_cast<const uint32_t *>(&bq);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 x = unpack_bf16(aw[e]), y = unpack_bf16(bw[e]);
                    acc = fmaf(v0[8 * c + 2 * e], x.x, acc);
                    acc = fmaf(v0[8 * c + 2 * e + 1], x.y, acc);
                    acc = fmaf(v1[8 * c + 2 * e], y.x, acc);
                    acc = fmaf(v1[8 * c + 2 * e + 1], y.y, acc);
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            return acc;
        };

        {   // dS_NT = dht (or zero) into TMEM; carried scalar <dht, S_NT>
            float v0[32], v1[32];
            if (p.dht) wait(INIT_FULL, 0);
            const float *src = state_row(p.dht, sbh, row, ch, p.dk, p.dv);
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                v0[j] = src ? src[j] : 0.f;
                v1[j] = src ? src[32 + j] : 0.f;
            }
            tmem_st32(tmem + lane_base + R0 + 64 * ch, v0);
            tmem_st32(tmem + lane_base + R0 + 64 * ch + 32, v1);
            const float part = p.dht ? state_dot(v0, v1) : 0.f;
            if (lane == 0) red[warp] = part;
            tmem_wait_st();
            named_bar_sync(1, NCOMPUTE);
            if (tid == 0) {
                float s = 0.f;
                for (int w = 0; w < 8; ++w) s += red[w];
                red[16] = s;
            }
            if (p.dht) mbar_arrive(bar(INIT_DONE));
        }

        for (int k = 0; k < NT; ++k) {
            const int n = NT - 1 - k, t0 = n * C;
            const uint32_t par = k & 1;
            // ---- stage 0: scalars, row-scaled tiles, T variants, dZ ----
            wait(GREADY + (k & 3), (k >> 2) & 1);
            const float *gt = gate_s + (k & 3) * 4 * C;
            if (warp == 0) {      // inclusive scan of the 64 log-decays: lane l owns tokens 2l, 2l+1
                const float g0 = gt[2 * C + 2 * lane], g1 = gt[2 * C + 2 * lane + 1];
                float incl = g0 + g1;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const float t = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += t;
                }
                sc[SC_B * C + 2 * lane] = incl - g1;
                sc[SC_B * C + 2 * lane + 1] = incl;
            }
            named_bar_sync(1, NCOMPUTE);
            if (tid < C) {
                const float bi = sc[SC_B * C + tid], beta = gt[3 * C + tid], gk = gt[C + tid];
                const float gam = __expf(bi), igam = __expf(-bi);
                sc[SC_GAM * C + tid] = gam;
                sc[SC_IGAM * C + tid] = igam;
                sc[SC_FQ * C + tid] = gt[tid] * gam;               // scale Gq Gam
                sc[SC_BG * C + tid] = beta * gam;
                sc[SC_BETA * C + tid] = beta;
                sc[SC_FVB * C + tid] = beta * gk;
                sc[SC_GK * C + tid] = gk;
                if (tid == C - 1) {
                    red[20] = gam;                                  // e^{b_last}
                    if (bi < -SLA_MAX_CHUNK_DECAY) atomicOr(p.status, STATUS_RANGE);
                }
            }
            named_bar_sync(1, NCOMPUTE);
            mbar_arrive(bar(GFREE + (k & 3)));
            wait(FULL_Q, par);
            wait(FULL_K, par);
            wait(FULL_V, par);
            wait(FULL_T, par);
            {
                const int rg = warp, cj = lane;
                const uint32_t half = cj >> 4, chunk = (cj & 15) >> 1, sub = (cj & 1) * 8;
#pragma unroll
                for (int rr = 0; rr < 8; ++rr) {
                    const int r = 8 * rg + rr;
                    const uint32_t off = half * HALF_BF16 + swz(r, chunk) + sub;
                    const float fq = sc[SC_FQ * C + r], fke = sc[SC_IGAM * C + r], fv = sc[SC_GK * C + r];
                    uint2 qv = *reinterpret_cast<uint2 *>(sm + B_Q + off), kv = *reinterpret_cast<uint2 *>(sm + B_K + off),
                          vv = *reinterpret_cast<uint2 *>(sm + B_V + off), ke;
                    uint32_t *qw = reinterpret_cast<uint32_t *>(&qv), *kw = reinterpret_cast<uint32_t *>(&kv),
                             *vw = reinterpret_cast<uint32_t *>(&vv), *kew = reinterpret_cast<uint32_t *>(&ke);
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const float2 qf = unpack_bf16(qw[e]), kf = unpack_bf16(kw[e]), vf = unpack_bf16(vw[e]);
                        qw[e] = pack_bf16(qf.x * fq, qf.y * fq);
                        vw[e] = pack_bf16(vf.x * fv, vf.y * fv);
                        kew[e] = pack_bf16(kf.x * fke, kf.y * fke);
                    }
                    *reinterpret_cast<uint2 *>(sm + B_Q + off) = qv;
                    *reinterpret_cast<uint2 *>(sm + B_V + off) = vv;
                    *reinterpret_cast<uint2 *>(sm + B_KE + off) = ke;
                }
            }
            {   // T diag(beta Gam) and T diag(beta): thread = (row i, 16 columns)
                const int i = tid >> 2, jq = tid & 3;
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const uint32_t off = swz(i, 2 * jq + hh);
                    const uint4 tv = *reinterpret_cast<const uint4 *>(sm + B_T + off);
                    const uint32_t *tw = reinterpret_cast<const uint32_t *>(&tv);
                    uint4 w1, w2;
                    uint32_t *w1w = reinterpret_cast<uint32_t *>(&w1), *w2w = reinterpret_cast<uint32_t *>(&w2);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int j = 16 * jq + 8 * hh + 2 * e;
                        const float2 t = unpack_bf16(tw[e]);
                        w1w[e] = pack_bf16(t.x * sc[SC_BG * C + j], t.y * sc[SC_BG * C + j + 1]);
                        w2w[e] = pack_bf16(t.x * sc[SC_BETA * C + j], t.y * sc[SC_BETA * C + j + 1]);
                    }
                    *reinterpret_cast<uint4 *>(sm + B_T1 + off) = w1;
                    *reinterpret_cast<uint4 *>(sm + B_T2 + off) = w2;
                }
            }
            {   // dZ = e^{b_last} dS_{n+1}: fp32 back into TMEM (dS_n accumulates on it), bf16 operand copy
                const float e = red[20];
                float v0[32], v1[32];
                const uint32_t ta = tmem + lane_base + R0 + 64 * ch;
                tmem_ld32(ta, v0);
                tmem_ld32(ta + 32, v1);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) { v0[j] *= e; v1[j] *= e; }
                tmem_st32(ta, v0);
                tmem_st32(ta + 32, v1);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint4 w;
                    w.x = pack_bf16(v0[8 * c + 0], v0[8 * c + 1]);
                    w.y = pack_bf16(v0[8 * c + 2], v0[8 * c + 3]);
                    w.z = pack_bf16(v0[8 * c + 4], v0[8 * c + 5]);
                    w.w = pack_bf16(v0[8 * c + 6], v0[8 * c + 7]);
                    *reinterpret_cast<uint4 *>(sm + B_DZ + ch * STATE_HALF + swz(row, c)) = w;
                    w.x = pack_bf16(v1[8 * c + 0], v1[8 * c + 1]);
                    w.y = pack_bf16(v1[8 * c + 2], v1[8 * c + 3]);
                    w.z = pack_bf16(v1[8 * c + 4], v1[8 * c + 5]);
                    w.w = pack_bf16(v1[8 * c + 6], v1[8 * c + 7]);
                    *reinterpret_cast<uint4 *>(sm + B_DZ + ch * STATE_HALF + swz(row, 4 + c)) = w;
                }
                tmem_wait_st();
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(OPR));

            // ---- stage 1: Lnb, Pq, -W, -U0 as bf16 tiles ----
            wait(C1, par);
            tc_fence_after();
            {
                float a[32], c[32];
                tmem_ld32(tmem + lane_base + R1 + 32 * ch, a);            // (K K^T) columns 32ch .. 32ch+31
                tmem_ld32(tmem + lane_base + R1 + 64 + 32 * ch, c);       // (Qg K^T) same columns
                tmem_wait_ld();
                if (act) {
                    const float gi = sc[SC_GAM * C + ti];
                    const float *ig = sc + SC_IGAM * C + 32 * ch;
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        uint4 wl, wp;
                        uint32_t *wlw = reinterpret_cast<uint32_t *>(&wl), *wpw = reinterpret_cast<uint32_t *>(&wp);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int jl = 8 * cc + 2 * e, j = 32 * ch + jl;
                            wlw[e] = pack_bf16(j < ti ? gi * ig[jl] * a[jl] : 0.f, j + 1 < ti ? gi * ig[jl + 1] * a[jl + 1] : 0.f);
                            wpw[e] = pack_bf16(j <= ti ? ig[jl] * c[jl] : 0.f, j + 1 <= ti ? ig[jl + 1] * c[jl + 1] : 0.f);
                        }
                        *reinterpret_cast<uint4 *>(sm + B_T2 + swz(ti, 4 * ch + cc)) = wl;
                        *reinterpret_cast<uint4 *>(sm + B_T1 + swz(ti, 4 * ch + cc)) = wp;
                    }
                }
                float v0[32], v1[32];
                ld64(R2, v0, v1);
                st_tile(sm + B_WN, v0, v1, -1.f);
                ld64(R3, v0, v1);
                st_tile(sm + B_U0N, v0, v1, -1.f);
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(S1R));

            // ---- stage 2: dU and dPq as bf16 tiles ----
            wait(C2, par);
            tc_fence_after();
            {
                float v0[32], v1[32], a[32];
                ld64(R1, v0, v1);
                tmem_ld32(tmem + lane_base + R2 + 32 * ch, a);            // (dO U^T) columns 32ch .. 32ch+31
                tmem_wait_ld();
                st_tile(sm + B_DZ, v0, v1, 1.f);                          // dU over the first half of the dZ buffer
                if (act) {
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        uint4 w;
                        uint32_t *ww = reinterpret_cast<uint32_t *>(&w);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int jl = 8 * cc + 2 * e, j = 32 * ch + jl;
                            ww[e] = pack_bf16(j <= ti ? a[jl] : 0.f, j + 1 <= ti ? a[jl + 1] : 0.f);
                        }
                        *reinterpret_cast<uint4 *>(sm + B_U + swz(ti, 4 * ch + cc)) = w;
                    }
                }
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(S2R));

            // ---- stage 3: <dS_n, S_n>; -dW tile; dq out of aq ----
            wait(C3, par);
            tc_fence_after();
            {
                float v0[32], v1[32];
                tmem_ld32(tmem + lane_base + R0 + 64 * ch, v0);
                tmem_ld32(tmem + lane_base + R0 + 64 * ch + 32, v1);
                tmem_wait_ld();
                const float part = state_dot(v0, v1);
                if (lane == 0) red[warp] = part;
                ld64(R1, v0, v1);
                st_tile(sm + B_DZ + TILE_BF16, v0, v1, -1.f);             // -dW over the second half of the dZ buffer
                ld64(R2, v0, v1);
                const float pq = dot_tile(sm + B_Q, v0, v1);               // (Qg . aq)
                if (act) sc[(SC_PQ + ch) * C + ti] = pq;
                st_tile(sm + B_DO, v0, v1, act ? sc[SC_FQ * C + ti] : 0.f);   // dq staged over dO
            }
            named_bar_sync(1, NCOMPUTE);                                  // everybody is done with S_n; red[] complete
            if (tid == 0) {
                float s = 0.f;
                for (int w = 0; w < 8; ++w) s += red[w];
                red[16 + ((k + 1) & 1)] = s;                              // carried to the next chunk's last row
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(S3R));

            // ---- stage 4: dKbg, dVb as bf16 tiles; dv ----
            wait(C4, par);
            tc_fence_after();
            {
                float v0[32], v1[32];
                ld64(R1, v0, v1);
                const float rk = dot_tile(sm + B_K, v0, v1);               // (dKbg . k)
                if (act) sc[(SC_RK + ch) * C + ti] = rk;
                st_tile(sm + B_S, v0, v1, 1.f);
                ld64(R2, v0, v1);
                const float pv = dot_tile(sm + B_V, v0, v1);               // (dVb . Gk v)
                if (act) sc[(SC_PV + ch) * C + ti] = pv;
                st_tile(sm + B_S + TILE_BF16, v0, v1, 1.f);
                st_tile(sm + B_V, v0, v1, act ? sc[SC_FVB * C + ti] : 0.f);   // dv = beta Gk dVb staged over Vg
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(S4R));

            // ---- stage 5: dL (strictly lower), its row sums against Lnb, the two dL tiles ----
            wait(C5, par);
            tc_fence_after();
            {
                float a[32];
                tmem_ld32(tmem + lane_base + R2 + 32 * ch, a);
                tmem_wait_ld();
                if (act) {
                    const float bg = sc[SC_BG * C + ti];
                    float rl = 0.f;
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        const uint4 lv = *reinterpret_cast<const uint4 *>(sm + B_T2 + swz(ti, 4 * ch + cc));
                        const uint32_t *lw = reinterpret_cast<const uint32_t *>(&lv);
                        uint4 w1, w2;
                        uint32_t *w1w = reinterpret_cast<uint32_t *>(&w1), *w2w = reinterpret_cast<uint32_t *>(&w2);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int jl = 8 * cc + 2 * e, j = 32 * ch + jl;
                            const float d0 = j < ti ? a[jl] : 0.f, d1 = j + 1 < ti ? a[jl + 1] : 0.f;
                            const float2 l = unpack_bf16(lw[e]);
                            rl = fmaf(d0, l.x, rl);
                            rl = fmaf(d1, l.y, rl);
                            w1w[e] = pack_bf16(d0, d1);
                            w2w[e] = pack_bf16(bg * d0, bg * d1);
                        }
                        *reinterpret_cast<uint4 *>(sm + B_U + HALF_BF16 + swz(ti, 4 * ch + cc)) = w1;
                        *reinterpret_cast<uint4 *>(sm + B_T + swz(ti, 4 * ch + cc)) = w2;
                    }
                    sc[(SC_RL + ch) * C + ti] = rl;
                }
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(S5R));

            // ---- stage 6: dk; per-token scalars ----
            wait(C6, par);
            tc_fence_after();
            {
                float v0[32], v1[32], w0[32], w1[32];
                ld64(R3, v0, v1);                                          // ak1
                const float ck = dot_tile(sm + B_KE, v0, v1);              // (Ke . ak1)
                if (act) sc[(SC_CK + ch) * C + ti] = ck;
                ld64(R1, w0, w1);                                          // dKbg + dL Ke
                const float fi = act ? sc[SC_IGAM * C + ti] : 0.f, fb = act ? sc[SC_BG * C + ti] : 0.f;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    v0[j] = fmaf(fi, v0[j], fb * w0[j]);
                    v1[j] = fmaf(fi, v1[j], fb * w1[j]);
                }
                st_tile(sm + B_Q, v0, v1, 1.f);                            // dk staged over Qg
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(S6R));
            named_bar_sync(1, NCOMPUTE);                                  // the per-token partial sums are complete
            if (warp == 0) {      // lane l owns tokens 2l, 2l+1
                float db[2], dbt[2], pqv[2], pkv[2];
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int i = 2 * lane + e;
                    const float pq = sc[SC_PQ * C + i] + sc[(SC_PQ + 1) * C + i], pv = sc[SC_PV * C + i] + sc[(SC_PV + 1) * C + i];
                    const float rk = sc[SC_RK * C + i] + sc[(SC_RK + 1) * C + i], rl = sc[SC_RL * C + i] + sc[(SC_RL + 1) * C + i];
                    const float ck = sc[SC_CK * C + i] + sc[(SC_CK + 1) * C + i];
                    const float beta = sc[SC_BETA * C + i], bg = sc[SC_BG * C + i], gam = sc[SC_GAM * C + i];
                    db[e] = pq + bg * rk + beta * rl - ck;
                    dbt[e] = rl + gam * rk + pv;
                    pqv[e] = pq;
                    pkv[e] = beta * pv;
                }
                if (lane == 31) db[1] += red[16 + (k & 1)];               // <dS_{n+1}, S_{n+1}> enters at the last token
                float suf = db[0] + db[1];                                // inclusive suffix sum over the lanes
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const float t = __shfl_down_sync(0xffffffffu, suf, o);
                    if (lane + o < 32) suf += t;
                }
                const float dg1 = suf - db[0], dg0 = suf;
                const int cn = min(C, p.T - t0);
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int i = 2 * lane + e;
                    if (i < cn) {
                        const size_t o = (tokb + t0 + i) * p.H + h;
                        p.dg[o] = e ? dg1 : dg0;
                        p.dbeta[o] = dbt[e];
                        p.pq[o] = pqv[e];
                        p.pk[o] = pkv[e];
                    }
                }
            }
        }

        if (p.dh0) {   // dS_0, fp32 (complete since the last chunk's group 3)
            float *dst = state_row(p.dh0, sbh, row, ch, p.dk, p.dv);
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                float v[32];
                tmem_ld32(tmem + lane_base + R0 + 64 * ch + 32 * part, v);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; j += 4)
                    if (dst) *reinterpret_cast<float4 *>(dst + 32 * part + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
            }
        }
    }
    if (failed) atomicOr(p.status, STATUS_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, TMEM_COLS);
}

}  // namespace

int gdn_tc_bwd_configure() {
    return cudaFuncSetAttribute(k_gdn_bwd_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gb::SMEM_BYTES) ==
                   cudaSuccess ? 0 : -1;
}

// record slots (one per chunk plus one per sequence) over all (sequence, head) pairs
static size_t record_slots(const Dims &d, const Varlen *vl) {
    return (vl && vl->n_seq) ? (size_t)vl->slots * d.H : (size_t)d.B * d.H * (d.NT + 1);
}

size_t gdn_tc_backward_workspace_bytes(const Dims &d, const Varlen *vl) {
    const size_t bth = (size_t)d.B * d.T * d.H;
    return record_slots(d, vl) * REC_BYTES + 2 * ((bth + 63) & ~(size_t)63) * sizeof(float);
}

uint8_t *gdn_tc_records(float *ws) { return reinterpret_cast<uint8_t *>(ws); }

int gdn_tc_backward(const Dims &d, const BwdArgs &a, bool have_records, int *status, cudaStream_t st, Tracer &tr) {
    CUtensorMap mq, mk, mv, mdo, mdq, mdk, mdv;
    if (!make_tile_map(&mq, a.q, d.B, d.T, d.H, d.dk) || !make_tile_map(&mk, a.k, d.B, d.T, d.H, d.dk) ||
        !make_tile_map(&mv, a.v, d.B, d.T, d.H, d.dv) || !make_tile_map(&mdo, a.dO, d.B, d.T, d.H, d.dv) ||
        !make_tile_map(&mdq, a.dq, d.B, d.T, d.H, d.dk) || !make_tile_map(&mdk, a.dk, d.B, d.T, d.H, d.dk) ||
        !make_tile_map(&mdv, a.dv, d.B, d.T, d.H, d.dv))
        return -1;
    Varlen *vl = (a.vl && a.vl->n_seq) ? a.vl : nullptr;
    const size_t bth = (size_t)d.B * d.T * d.H;
    uint8_t *save = reinterpret_cast<uint8_t *>(a.ws);
    float *pq = reinterpret_cast<float *>(save + record_slots(d, vl) * REC_BYTES);
    float *pk = pq + ((bth + 63) & ~(size_t)63);
    FwdArgs f{a.q, a.k, a.v, a.log_decay, a.beta, a.lq, a.lk, a.h0, nullptr, nullptr, a.ws, a.status, vl};
    // (with have_records the forward pass of the same inputs has left the records in this workspace)
    if (!have_records && gdn_tc_forward_save(d, f, save, status, st, tr) < 0) return -1;
    const CUtensorMap *vm = nullptr;
    if (vl) {
        const void *key[] = {a.q, a.k, a.v, a.dO, a.dq, a.dk, a.dv};
        vm = varlen_maps(*vl, 2, key, 7, st, [&](const SeqInfo &si, CUtensorMap *m) {
            const size_t tok = (size_t)si.t0 * d.H;      // (q, k are d_k wide, v, o and their gradients d_v)
            const void *src[7] = {a.q, a.k, a.v, a.dO, a.dq, a.dk, a.dv};
            for (int i = 0; i < 7; ++i)
                if (!make_tile_map(m + i, (const __nv_bfloat16 *)src[i] + tok * (i == 2 || i == 3 || i == 6 ? d.dv : d.dk), 1, si.T, d.H, (i == 2 || i == 3 || i == 6 ? d.dv : d.dk))) return false;
            return true;
        });
        if (!vm) return -1;
    }
    GdnBwdParams bp{a.lq, a.lk, a.log_decay, a.beta, a.dht, save, a.dlog_decay, a.dbeta, pq, pk, a.dh0, status,
                    d.T, d.H, d.NT, d.scale, vl ? vl->d_seqs : nullptr, vm, d.dk, d.dv};
    k_gdn_bwd_tc<<<vl ? vl->n_seq * d.H : d.B * d.H, gb::NTHREADS, gb::SMEM_BYTES, st>>>(mq, mk, mv, mdo, mdq, mdk, mdv, bp);
    tr.mark("gdn_bwd_tc");
    if (gate_bwd_prod(a.lq, a.lk, pq, pk, a.dlq, a.dlk, (long)d.B * d.T, d.H, st) < 0) return -1;
    tr.mark("gate_bwd");
    return cudaGetLastError() == cudaSuccess ? (have_records ? 2 : 3) : -1;
}

}  // namespace sla
