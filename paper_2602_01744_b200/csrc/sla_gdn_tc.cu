// Softmax-GatedDeltaNet forward on the 5th-generation tensor cores (bf16 I/O, d_k and d_v 128 - or 64, run as 128 with zero padding supplied by the tensor maps -, chunk 64):
// Eq. 14-16 with a scalar decay per (token, head), evaluated chunkwise in WY form.
//
// Per chunk (local token i, b_i = cumulative log-decay, Gam_i = e^{b_i}, S = state at the chunk start):
//   L   = strict_tril(beta_i e^{b_i - b_j} (k_i . k_j))              T = (I + L)^{-1}
//   W   = T diag(beta Gam) K        U0 = T diag(beta Gk) V           U = U0 - W S
//   Pq  = tril((scale Gq Gam q) K^T e^{-b_j})                        O = (scale Gq Gam q) S + Pq U
//   S'  = e^{b_last} (S + (e^{-b} K)^T U)
// which is an exact re-association of  Sb = e^{g_t} S_{t-1};  u = beta_t (Gk v_t - k_t Sb);  S_t = Sb + k_t^T u.
// The decay is a scalar per token, so it acts on the 64x64 products K K^T and q K^T after the MMA, and the operand
// tiles only need row scalings.  The 64x64 unit-triangular inverse is formed in fp32 in shared memory (16x16 diagonal
// blocks by forward substitution, off-diagonal blocks level by level) and handed to the tensor core as bf16.
// One CTA per (batch, head) sequence; roles as in the GLA kernels: MMA lane, TMA lane, gate warps, compute warps.
#include "sla_gla_tc.cuh"

namespace sla {
namespace {

using namespace ptx;
using namespace tc;

namespace gd {
constexpr uint32_t STAGE = 3 * TILE_BF16;               // q (-> -W), k (-> U), v (-> beta Gk v -> staged O)
constexpr uint32_t OFF_Q = 0, OFF_K = TILE_BF16, OFF_V = 2 * TILE_BF16;
constexpr uint32_t OFF_KB = 2 * STAGE;                  // beta Gam k
constexpr uint32_t OFF_KE = OFF_KB + TILE_BF16;         // e^{-b} k
constexpr uint32_t OFF_S = OFF_KE + TILE_BF16;          // bf16 state operand
constexpr uint32_t OFF_T = OFF_S + STATE_BF16;          // bf16 T, [64 rows][128 B]
constexpr uint32_t OFF_PQ = OFF_T + HALF_BF16;          // bf16 Pq
constexpr int LDL = 68;                                 // row stride (floats) of the fp32 64x64 work arrays
constexpr uint32_t OFF_LS = OFF_PQ + HALF_BF16;         // fp32 L
constexpr uint32_t OFF_TS = OFF_LS + 64 * LDL * 4;      // fp32 T
constexpr uint32_t OFF_XS = OFF_TS + 64 * LDL * 4;      // fp32 block-product scratch, [6 warps][16][8] (816 floats reserved)
constexpr uint32_t OFF_SC = OFF_XS + 3 * 16 * 17 * 4;   // per-token scalars of the chunk: 8 arrays of 64 floats
constexpr uint32_t OFF_GATE = OFF_SC + 8 * C * 4;       // [4 chunks][4][64]: scale*Gq, Gk, log-decay, beta
constexpr uint32_t OFF_BAR = OFF_GATE + 4 * 4 * C * 4;
constexpr uint32_t OFF_TMEM = OFF_BAR + 32 * 8;         // TMEM base address, then the abort flag
constexpr uint32_t SMEM_BYTES = OFF_TMEM + 16 + 1024;
static_assert(SMEM_BYTES <= 232448, "shared memory budget");
constexpr uint32_t COL_KK = 0, COL_QK = 64, COL_W = 0, COL_U = 128, COL_O = 256, COL_S = 384, TMEM_COLS = 512;
constexpr int NTHREADS = NCOMPUTE + 32 + NGATE + 32;    // warps 0..7 compute, 8 MMA issue, 9..12 gates, 13 TMA
enum Bar { FULL = 0 /*[2]*/, GREADY = 2 /*[4]*/, GFREE = 6 /*[4]*/, OPR = 10, TREADY, WREADY, UREADY, SREADY, OSTAGED /*[2]*/,
           BAR_1 = OSTAGED + 2, BAR_2, BAR_3, BAR_4, DRAIN, SAVED, NBAR };
static_assert(NBAR <= 32, "barrier slots");
// scalar arrays in OFF_SC
enum Sc { SC_B = 0, SC_GAM, SC_IGAM, SC_FQ, SC_FKB, SC_FVB, SC_BETA, SC_MISC };
}  // namespace gd

// Per-chunk record the forward leaves for the gradient sweep (save mode): bf16 S_n image, bf16 U tile, bf16 T tile,
// each in MMA-operand layout.  Record n of sequence bh sits at save + (bh * (NT + 1) + n) * GDN_REC_BYTES; record NT
// holds only S_NT.
constexpr uint32_t REC_S = 0, REC_U = STATE_BF16, REC_T = STATE_BF16 + TILE_BF16, REC_BYTES = STATE_BF16 + TILE_BF16 + HALF_BF16;

struct GdnParams {
    const float *lq, *lk, *g, *beta, *h0;
    float *ht;
    uint8_t *save;          // not nullptr: the per-chunk records are written
    int write_o;            // 0: o is not stored (the gradient sweep's own recomputation)
    int *status;
    int T, H, NT;
    float scale;
    const SeqInfo *seqs;    // packed variable-length batch: per-sequence table and tensor maps (q, k, v, o), else nullptr
    const CUtensorMap *vmaps;
    int dk, dv;             // head widths, each 128 or 64 (the upper half of a 128-wide tile is then zero padding)
};

__global__ void __launch_bounds__(gd::NTHREADS, 1)
k_gdn_fwd_tc(const __grid_constant__ CUtensorMap gm_q, const __grid_constant__ CUtensorMap gm_k,
             const __grid_constant__ CUtensorMap gm_v, const __grid_constant__ CUtensorMap gm_o, GdnParams p) {
    using namespace gd;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *sm = smem_raw + (base - raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.x, h = bh % p.H;
    int b = bh / p.H;
    // A packed batch: this CTA's sequence has its own length, chunk count, first token, record slots and tensor maps
    // (based at its first token, so token coordinates stay relative and the batch coordinate is 0).
    size_t tokb = (size_t)b * p.T, slot = (size_t)bh * (p.NT + 1);
    size_t sbh = (size_t)bh;                                // (sequence, head) index into h0 / ht / dht / dh0
    const CUtensorMap *vm = nullptr;
    if (p.seqs) {
        const SeqInfo si = p.seqs[b];
        vm = p.vmaps + (size_t)b * Varlen::MAPS_PER_SEQ;
        p.T = si.T; p.NT = si.NT;
        tokb = (size_t)si.t0;
        slot = (size_t)si.slot0 * p.H + (size_t)h * (si.NT + 1);
        sbh = (size_t)si.id * p.H + h;                      // (the table is ordered longest first, the state tensors as the caller gave them)
        b = 0;
    }
    const CUtensorMap &tm_q = vm ? vm[0] : gm_q, &tm_k = vm ? vm[1] : gm_k, &tm_v = vm ? vm[2] : gm_v, &tm_o = vm ? vm[3] : gm_o;
    const int NT = p.NT;
    auto bar = [&](int i) { return base + OFF_BAR + 8u * i; };
    float *Ls = reinterpret_cast<float *>(sm + OFF_LS);
    float *Ts = reinterpret_cast<float *>(sm + OFF_TS);
    float *Xs = reinterpret_cast<float *>(sm + OFF_XS);
    float *sc = reinterpret_cast<float *>(sm + OFF_SC);
    float *gate_s = reinterpret_cast<float *>(sm + OFF_GATE);
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
            const bool all = (i >= GFREE && i < BAR_1);
            mbar_init(bar(i), all ? NCOMPUTE : (i >= GREADY && i < GFREE) ? NGATE / 32 : 1);
        }
        fence_mbar_init();
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
        tma_prefetch_desc(&tm_o);
    }
    if (warp == 0) tmem_alloc(base + OFF_TMEM, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(sm + OFF_TMEM);

    if (warp == 8) {
        // ---------------- MMA issue (one lane) ----------------
        if (lane == 0) {
            constexpr uint32_t ID_64 = idesc_bf16(64, 64, 0, 0);     // K-major x K-major
            constexpr uint32_t ID_N = idesc_bf16(64, 128, 0, 1);     // K-major x MN-major
            constexpr uint32_t ID_S = idesc_bf16(128, 128, 1, 1);    // MN-major x MN-major
            const uint64_t mS = desc_mnmajor(base + OFF_S, STATE_HALF), kT = desc_kmajor(base + OFF_T),
                           kPQ = desc_kmajor(base + OFF_PQ), mKB = desc_mnmajor(base + OFF_KB, HALF_BF16),
                           mKE = desc_mnmajor(base + OFF_KE, HALF_BF16);
            for (int n = 0; n < NT; ++n) {
                const uint32_t par = n & 1, st = base + (n & 1) * STAGE;
                const uint64_t kQ = desc_kmajor(st + OFF_Q), kK = desc_kmajor(st + OFF_K),
                               mU = desc_mnmajor(st + OFF_K, HALF_BF16), mV = desc_mnmajor(st + OFF_V, HALF_BF16);
                wait(OPR, par);                        // scaled operand tiles in place
                wait(SREADY, par);                     // S_n: fp32 in TMEM, bf16 in shared memory
                if (failed) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)         // K K^T
                    tc_mma_bf16(tmem + COL_KK, kK + kstep_kmajor(kk, HALF_BF16), kK + kstep_kmajor(kk, HALF_BF16), ID_64, kk > 0);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)         // (scale Gq Gam q) K^T
                    tc_mma_bf16(tmem + COL_QK, kQ + kstep_kmajor(kk, HALF_BF16), kK + kstep_kmajor(kk, HALF_BF16), ID_64, kk > 0);
                tc_commit(bar(BAR_1));
                if (n > 0) wait(OSTAGED + ((n - 1) & 1), ((n - 1) >> 1) & 1);   // O of chunk n-1 has been read out
                if (failed) break;
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)         // O = (scale Gq Gam q) S
                    tc_mma_bf16(tmem + COL_O, kQ + kstep_kmajor(kk, HALF_BF16), mS + kstep_mnmajor(kk), ID_N, kk > 0);
                wait(TREADY, par);                     // bf16 T and Pq in shared memory; K K^T, q K^T read out
                if (failed) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)         // W = T (beta Gam K)
                    tc_mma_bf16(tmem + COL_W, kT + kstep_kmajor(kk, 0), mKB + kstep_mnmajor(kk), ID_N, kk > 0);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)         // U0 = T (beta Gk V)
                    tc_mma_bf16(tmem + COL_U, kT + kstep_kmajor(kk, 0), mV + kstep_mnmajor(kk), ID_N, kk > 0);
                tc_commit(bar(BAR_2));
                wait(WREADY, par);                     // -W as bf16 in the q buffer
                if (failed) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)         // U = U0 - W S
                    tc_mma_bf16(tmem + COL_U, kQ + kstep_kmajor(kk, HALF_BF16), mS + kstep_mnmajor(kk), ID_N, 1);
                tc_commit(bar(BAR_3));
                wait(UREADY, par);                     // U as bf16 in the k buffer
                if (failed) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)         // O += Pq U
                    tc_mma_bf16(tmem + COL_O, kPQ + kstep_kmajor(kk, 0), mU + kstep_mnmajor(kk), ID_N, 1);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)         // S += (e^{-b} K)^T U
                    tc_mma_bf16(tmem + COL_S, mKE + kstep_mnmajor(kk), mU + kstep_mnmajor(kk), ID_S, 1);
                tc_commit(bar(BAR_4));
            }
            tc_commit(bar(DRAIN));
            mbar_wait_bounded(bar(DRAIN), 0, nullptr, 20000000ull);
        }
    } else if (warp == 13) {
        // ---------------- TMA (one lane) ----------------
        if (lane == 0) {
            auto load = [&](int n) {
                const uint32_t bf = bar(FULL + (n & 1)), st = base + (n & 1) * STAGE;
                mbar_expect_tx(bf, STAGE);
                tma_load_5d(st + OFF_Q, &tm_q, 0, n * C, 0, h, b, bf);
                tma_load_5d(st + OFF_K, &tm_k, 0, n * C, 0, h, b, bf);
                tma_load_5d(st + OFF_V, &tm_v, 0, n * C, 0, h, b, bf);
            };
            load(0);
            if (NT > 1) load(1);
            for (int n = 0; n < NT && !failed; ++n) {
                wait_relaxed(OSTAGED + (n & 1), (n >> 1) & 1);   // O staged in the v buffer; every MMA of the chunk is done
                if (failed) break;
                if (p.write_o) {
                    tma_store_5d(&tm_o, base + (n & 1) * STAGE + OFF_V, 0, n * C, 0, h, b);
                    bulk_commit();
                }
                if (p.save) {   // the chunk's record: T, U and S_{n+1} stand in shared memory in exactly the record's layout
                    uint8_t *rec = p.save + (slot + n) * REC_BYTES;
                    bulk_store(rec + REC_T, base + OFF_T, HALF_BF16);
                    bulk_store(rec + REC_U, base + (n & 1) * STAGE + OFF_K, TILE_BF16);
                    bulk_store(rec + REC_BYTES + REC_S, base + OFF_S, STATE_BF16);
                    bulk_commit();
                }
                if (n + 2 < NT || p.save) bulk_wait_read0();
                if (p.save) mbar_arrive(bar(SAVED));   // T and the S copy may be overwritten
                if (n + 2 < NT) load(n + 2);
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
        for (int n = 0; n < NT; ++n) {
            if (n >= 4) wait_relaxed(GFREE + (n & 3), ((n >> 2) - 1) & 1);
            if (failed) break;
            const int cn = min(C, p.T - n * C);
            const size_t tok = tokb + (size_t)n * C + t;
            float *dst = gate_s + (n & 3) * 4 * C;
            if (g < C) {
                chunk_gate(p.lq + (tok - t) * p.H, p.H, cn, h, p.scale, dst, t);
                dst[2 * C + t] = t < cn ? p.g[tok * p.H + h] : 0.f;
            } else {
                chunk_gate(p.lk + (tok - t) * p.H, p.H, cn, h, 1.f, dst + C, t);
                dst[3 * C + t] = t < cn ? p.beta[tok * p.H + h] : 0.f;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(GREADY + (n & 3)));
        }
    } else {
        // ---------------- compute warps ----------------
        const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;   // this warp's TMEM lane quarter
        const int colhalf = warp >> 2;
        const int row = 32 * (warp & 3) + lane;                          // state row (M = 128 tiles)
        const int ti = 16 * (warp & 3) + lane;                           // token row (M = 64 tiles, lanes 0..15)

        uint8_t *rec0 = p.save ? p.save + slot * REC_BYTES : nullptr;   // this sequence's records
        {   // initial state: fp32 into TMEM, bf16 copy into shared memory (row = key dimension)
            const float *src = state_row(p.h0, sbh, row, colhalf, p.dk, p.dv);
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
                    *reinterpret_cast<uint4 *>(sm + OFF_S + colhalf * STATE_HALF + swz(row, 4 * part + c)) = w;
                    if (rec0) *reinterpret_cast<uint4 *>(rec0 + REC_S + colhalf * STATE_HALF + swz(row, 4 * part + c)) = w;
                }
            }
            tmem_wait_st();
        }
        fence_proxy_async();
        tc_fence_before();
        mbar_arrive(bar(SREADY));

        // a 64x128 accumulator tile (M = 64: row i in lane 32*(i/16) + i%16) -> sign * bf16 -> swizzled tile at dst
        auto tile_to_bf16 = [&](uint32_t col, uint8_t *dst, float sign) {
            float v0[32], v1[32];
            tmem_ld32(tmem + lane_base + col + 64 * colhalf, v0);
            tmem_ld32(tmem + lane_base + col + 64 * colhalf + 32, v1);
            tmem_wait_ld();
            if (lane < 16) {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint4 w;
                    w.x = pack_bf16(sign * v0[8 * c + 0], sign * v0[8 * c + 1]);
                    w.y = pack_bf16(sign * v0[8 * c + 2], sign * v0[8 * c + 3]);
                    w.z = pack_bf16(sign * v0[8 * c + 4], sign * v0[8 * c + 5]);
                    w.w = pack_bf16(sign * v0[8 * c + 6], sign * v0[8 * c + 7]);
                    *reinterpret_cast<uint4 *>(dst + colhalf * HALF_BF16 + swz(ti, c)) = w;
                    w.x = pack_bf16(sign * v1[8 * c + 0], sign * v1[8 * c + 1]);
                    w.y = pack_bf16(sign * v1[8 * c + 2], sign * v1[8 * c + 3]);
                    w.z = pack_bf16(sign * v1[8 * c + 4], sign * v1[8 * c + 5]);
                    w.w = pack_bf16(sign * v1[8 * c + 6], sign * v1[8 * c + 7]);
                    *reinterpret_cast<uint4 *>(dst + colhalf * HALF_BF16 + swz(ti, 4 + c)) = w;
                }
            }
        };

        for (int n = 0; n < NT; ++n) {
            const uint32_t par = n & 1;
            uint8_t *st = sm + (n & 1) * STAGE;
            // ---- A: cumulative decay, per-token factors, row-scaled operand tiles ----
            wait(GREADY + (n & 3), (n >> 2) & 1);
            const float *gt = gate_s + (n & 3) * 4 * C;
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
                const float bi = sc[SC_B * C + tid], beta = gt[3 * C + tid];
                const float gam = __expf(bi), igam = __expf(-bi);
                sc[SC_GAM * C + tid] = gam;
                sc[SC_IGAM * C + tid] = igam;
                sc[SC_FQ * C + tid] = gt[tid] * gam;               // scale Gq Gam
                sc[SC_FKB * C + tid] = beta * gam;
                sc[SC_FVB * C + tid] = beta * gt[C + tid];         // beta Gk
                sc[SC_BETA * C + tid] = beta;
                if (tid == C - 1) {
                    sc[SC_MISC * C] = gam;                          // e^{b_last}
                    if (bi < -SLA_MAX_CHUNK_DECAY) atomicOr(p.status, STATUS_RANGE);
                }
            }
            named_bar_sync(1, NCOMPUTE);
            mbar_arrive(bar(GFREE + (n & 3)));
            wait(FULL + (n & 1), (n >> 1) & 1);
            {
                const int rg = warp, cj = lane;
                const uint32_t half = cj >> 4, chunk = (cj & 15) >> 1, sub = (cj & 1) * 8;
#pragma unroll
                for (int rr = 0; rr < 8; ++rr) {
                    const int r = 8 * rg + rr;
                    const uint32_t off = half * HALF_BF16 + swz(r, chunk) + sub;
                    const float fq = sc[SC_FQ * C + r], fkb = sc[SC_FKB * C + r], fke = sc[SC_IGAM * C + r], fvb = sc[SC_FVB * C + r];
                    uint2 qv = *reinterpret_cast<uint2 *>(st + OFF_Q + off), kv = *reinterpret_cast<uint2 *>(st + OFF_K + off),
                          vv = *reinterpret_cast<uint2 *>(st + OFF_V + off), kb, ke;
                    uint32_t *qw = reinterpret_cast<uint32_t *>(&qv), *kw = reinterpret_cast<uint32_t *>(&kv),
                             *vw = reinterpret_cast<uint32_t *>(&vv), *kbw = reinterpret_cast<uint32_t *>(&kb),
                             *kew = reinterpret_cast<uint32_t *>(&ke);
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const float2 qf = unpack_bf16(qw[e]), kf = unpack_bf16(kw[e]), vf = unpack_bf16(vw[e]);
                        qw[e] = pack_bf16(qf.x * fq, qf.y * fq);
                        vw[e] = pack_bf16(vf.x * fvb, vf.y * fvb);
                        kbw[e] = pack_bf16(kf.x * fkb, kf.y * fkb);
                        kew[e] = pack_bf16(kf.x * fke, kf.y * fke);
                    }
                    *reinterpret_cast<uint2 *>(st + OFF_Q + off) = qv;
                    *reinterpret_cast<uint2 *>(st + OFF_V + off) = vv;
                    *reinterpret_cast<uint2 *>(sm + OFF_KB + off) = kb;
                    *reinterpret_cast<uint2 *>(sm + OFF_KE + off) = ke;
                }
            }
            fence_proxy_async();
            mbar_arrive(bar(OPR));

            // ---- B: L and Pq out of TMEM, T = (I + L)^{-1} in fp32, bf16 T ----
            wait(BAR_1, par);
            tc_fence_after();
            {
                float v0[32], v1[32];
                tmem_ld32(tmem + lane_base + (colhalf ? COL_QK : COL_KK), v0);
                tmem_ld32(tmem + lane_base + (colhalf ? COL_QK : COL_KK) + 32, v1);
                tmem_wait_ld();
                if (lane < 16) {
                    const float *ig = sc + SC_IGAM * C;
                    if (colhalf == 0) {      // L_ij = beta_i Gam_i e^{-b_j} (k_i . k_j), j < i
                        const float f = sc[SC_FKB * C + ti];
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            float4 a, c;
                            a.x = j + 0 < ti ? f * ig[j + 0] * v0[j + 0] : 0.f;
                            a.y = j + 1 < ti ? f * ig[j + 1] * v0[j + 1] : 0.f;
                            a.z = j + 2 < ti ? f * ig[j + 2] * v0[j + 2] : 0.f;
                            a.w = j + 3 < ti ? f * ig[j + 3] * v0[j + 3] : 0.f;
                            c.x = 32 + j + 0 < ti ? f * ig[32 + j + 0] * v1[j + 0] : 0.f;
                            c.y = 32 + j + 1 < ti ? f * ig[32 + j + 1] * v1[j + 1] : 0.f;
                            c.z = 32 + j + 2 < ti ? f * ig[32 + j + 2] * v1[j + 2] : 0.f;
                            c.w = 32 + j + 3 < ti ? f * ig[32 + j + 3] * v1[j + 3] : 0.f;
                            *reinterpret_cast<float4 *>(Ls + ti * LDL + j) = a;
                            *reinterpret_cast<float4 *>(Ls + ti * LDL + 32 + j) = c;
                        }
                    } else {                 // Pq_ij = (q K^T)_ij e^{-b_j}, j <= i   (the row factor is already in q)
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint4 w;
                            uint32_t *ww = reinterpret_cast<uint32_t *>(&w);
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const int j = 8 * c + 2 * e;
                                ww[e] = pack_bf16(j <= ti ? v0[j] * ig[j] : 0.f, j + 1 <= ti ? v0[j + 1] * ig[j + 1] : 0.f);
                            }
                            *reinterpret_cast<uint4 *>(sm + OFF_PQ + swz(ti, c)) = w;
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const int j = 8 * c + 2 * e;
                                ww[e] = pack_bf16(32 + j <= ti ? v1[j] * ig[32 + j] : 0.f, 33 + j <= ti ? v1[j + 1] * ig[33 + j] : 0.f);
                            }
                            *reinterpret_cast<uint4 *>(sm + OFF_PQ + swz(ti, 4 + c)) = w;
                        }
                    }
                }
            }
            named_bar_sync(1, NCOMPUTE);
            if (tid < C) {        // diagonal 16x16 blocks: column c of (I + L_bb)^{-1} by forward substitution
                const int bb = tid >> 4, c = tid & 15;
                const float *Lb = Ls + (16 * bb) * LDL + 16 * bb;
                float x[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    float acc = i == c ? 1.f : 0.f;
#pragma unroll
                    for (int j = 0; j < i; ++j) acc = fmaf(-Lb[i * LDL + j], x[j], acc);
                    x[i] = acc;
                }
#pragma unroll
                for (int i = 0; i < 16; ++i) Ts[(16 * bb + i) * LDL + 16 * bb + c] = x[i];
            }
            named_bar_sync(1, NCOMPUTE);
            // Off-diagonal blocks, top down within a block column a:  T_ba = -T_bb sum_{a <= c < b} L_bc T_ca,  b = a+1 .. 3.
            // A column of T depends on no other column, so two warps share a block column, eight columns each, and no
            // barrier is needed inside.  16x16x16 products on the warp-level tf32 MMA (T is rounded to bf16 afterwards, so
            // tf32 operands cost nothing).
            if (warp < 6) {
                const int a = warp >> 1, nh = warp & 1, g = lane >> 2, t = lane & 3;
                float *Xw = Xs + warp * 16 * 8;          // this warp's 16x8 scratch
                auto frag_a = [&](const float *M, uint32_t (&fa)[4]) {       // 16x8 slice at M (row stride LDL)
                    fa[0] = to_tf32(M[g * LDL + t]);
                    fa[1] = to_tf32(M[(g + 8) * LDL + t]);
                    fa[2] = to_tf32(M[g * LDL + t + 4]);
                    fa[3] = to_tf32(M[(g + 8) * LDL + t + 4]);
                };
                const int col0 = 16 * a + 8 * nh;        // this warp's columns of T
                for (int bI = a + 1; bI < 4; ++bI) {
                    float x[4] = {0.f, 0.f, 0.f, 0.f};
                    for (int cc = a; cc < bI; ++cc) {
#pragma unroll
                        for (int ks = 0; ks < 2; ++ks) {
                            uint32_t fa[4], fb[2];
                            frag_a(Ls + (16 * bI) * LDL + 16 * cc + 8 * ks, fa);
                            const float *Tb = Ts + (16 * cc + 8 * ks) * LDL + col0;
                            fb[0] = to_tf32(Tb[t * LDL + g]);
                            fb[1] = to_tf32(Tb[(t + 4) * LDL + g]);
                            mma_tf32_16x8x8(x, fa, fb);
                        }
                    }
                    Xw[g * 8 + 2 * t] = x[0];       Xw[g * 8 + 2 * t + 1] = x[1];
                    Xw[(g + 8) * 8 + 2 * t] = x[2]; Xw[(g + 8) * 8 + 2 * t + 1] = x[3];
                    __syncwarp();
                    float y[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int ks = 0; ks < 2; ++ks) {
                        uint32_t fa[4], fb[2];
                        frag_a(Ts + (16 * bI) * LDL + 16 * bI + 8 * ks, fa);
                        fb[0] = to_tf32(Xw[(8 * ks + t) * 8 + g]);
                        fb[1] = to_tf32(Xw[(8 * ks + t + 4) * 8 + g]);
                        mma_tf32_16x8x8(y, fa, fb);
                    }
                    float *To = Ts + (16 * bI) * LDL + col0;
                    To[g * LDL + 2 * t] = -y[0];       To[g * LDL + 2 * t + 1] = -y[1];
                    To[(g + 8) * LDL + 2 * t] = -y[2]; To[(g + 8) * LDL + 2 * t + 1] = -y[3];
                    __syncwarp();
                }
            }
            named_bar_sync(1, NCOMPUTE);
            if (p.save && n > 0) wait(SAVED, (n - 1) & 1);   // the previous chunk's record has left T and the S copy
            {   // bf16 T (A operand, K-major): thread = (row i, 16 columns)
                const int i = tid >> 2, jq = tid & 3;
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    uint4 w;
                    uint32_t *ww = reinterpret_cast<uint32_t *>(&w);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int j = 16 * jq + 8 * hh + 2 * e;
                        const float t0 = (jq <= (i >> 4)) ? Ts[i * LDL + j] : 0.f, t1 = (jq <= (i >> 4)) ? Ts[i * LDL + j + 1] : 0.f;
                        ww[e] = pack_bf16(t0, t1);
                    }
                    *reinterpret_cast<uint4 *>(sm + OFF_T + swz(i, 2 * jq + hh)) = w;
                }
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(TREADY));

            // ---- C: -W as bf16 over the q tile ----
            wait(BAR_2, par);
            tc_fence_after();
            tile_to_bf16(COL_W, st + OFF_Q, -1.f);
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(WREADY));

            // ---- D: U as bf16 over the k tile ----
            wait(BAR_3, par);
            tc_fence_after();
            tile_to_bf16(COL_U, st + OFF_K, 1.f);
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(UREADY));

            // ---- E: S_{n+1} = e^{b_last} (S_n + (e^{-b} K)^T U); O staged over the v tile ----
            wait(BAR_4, par);
            tc_fence_after();
            {
                const float e = sc[SC_MISC * C];
                float v0[32], v1[32];
                const uint32_t ta = tmem + lane_base + COL_S + 64 * colhalf;
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
                    *reinterpret_cast<uint4 *>(sm + OFF_S + colhalf * STATE_HALF + swz(row, c)) = w;
                    w.x = pack_bf16(v1[8 * c + 0], v1[8 * c + 1]);
                    w.y = pack_bf16(v1[8 * c + 2], v1[8 * c + 3]);
                    w.z = pack_bf16(v1[8 * c + 4], v1[8 * c + 5]);
                    w.w = pack_bf16(v1[8 * c + 6], v1[8 * c + 7]);
                    *reinterpret_cast<uint4 *>(sm + OFF_S + colhalf * STATE_HALF + swz(row, 4 + c)) = w;
                }
                tmem_wait_st();
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(SREADY));
            tile_to_bf16(COL_O, st + OFF_V, 1.f);
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(OSTAGED + (n & 1)));
        }

        if (p.ht) {   // final state, fp32 (each thread reads back what it wrote in the last rescale)
            float *dst = state_row(p.ht, sbh, row, colhalf, p.dk, p.dv);
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                float v[32];
                tmem_ld32(tmem + lane_base + COL_S + 64 * colhalf + 32 * part, v);
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

bool gdn_tc_supported(const Dims &d) {
    return d.variant == SLA_GDN && d.io_bf16 && (d.dk == 128 || d.dk == 64) && (d.dv == 128 || d.dv == 64) && d.C == 64;
}

int gdn_tc_configure() {
    if (!encode_fn()) return -1;
    return cudaFuncSetAttribute(k_gdn_fwd_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gd::SMEM_BYTES) ==
                   cudaSuccess ? 0 : -1;
}

// per-sequence tensor maps of a packed batch (q, k, v and, when given, o) into region `r`
static const CUtensorMap *gdn_varlen_maps(const Dims &d, const FwdArgs &a, int r, cudaStream_t st) {
    const void *key[] = {a.q, a.k, a.v, a.o};
    return varlen_maps(*a.vl, r, key, 4, st, [&](const SeqInfo &si, CUtensorMap *m) {
        const size_t tok = (size_t)si.t0 * d.H;      // (q, k are d_k wide, v, o and their gradients d_v)
        if (!make_tile_map(m + 0, (const __nv_bfloat16 *)a.q + tok * d.dk, 1, si.T, d.H, d.dk) ||
            !make_tile_map(m + 1, (const __nv_bfloat16 *)a.k + tok * d.dk, 1, si.T, d.H, d.dk) ||
            !make_tile_map(m + 2, (const __nv_bfloat16 *)a.v + tok * d.dv, 1, si.T, d.H, d.dv))
            return false;
        if (!a.o) { m[3] = m[0]; return true; }
        return make_tile_map(m + 3, (__nv_bfloat16 *)a.o + tok * d.dv, 1, si.T, d.H, d.dv);
    });
}

// Forward sweep in save mode, for the gradient sweep: writes the per-chunk records (S_n, U, T), stores no output.
int gdn_tc_forward_save(const Dims &d, const FwdArgs &a, uint8_t *save, int *status, cudaStream_t st, Tracer &tr) {
    CUtensorMap mq, mk, mv;
    if (!make_tile_map(&mq, a.q, d.B, d.T, d.H, d.dk) || !make_tile_map(&mk, a.k, d.B, d.T, d.H, d.dk) ||
        !make_tile_map(&mv, a.v, d.B, d.T, d.H, d.dv))
        return -1;
    const bool vl = a.vl && a.vl->n_seq;
    const CUtensorMap *vm = vl ? gdn_varlen_maps(d, a, 1, st) : nullptr;
    if (vl && !vm) return -1;
    GdnParams p{a.lq, a.lk, a.log_decay, a.beta, a.h0, nullptr, save, 0, status, d.T, d.H, d.NT, d.scale,
                vl ? a.vl->d_seqs : nullptr, vm, d.dk, d.dv};
    k_gdn_fwd_tc<<<vl ? a.vl->n_seq * d.H : d.B * d.H, gd::NTHREADS, gd::SMEM_BYTES, st>>>(mq, mk, mv, mq /* unused: nothing is stored */, p);
    tr.mark("gdn_states_tc");
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

// Forward; with `save` not null it also leaves the per-chunk records for a later gradient sweep over the same inputs.
int gdn_tc_forward(const Dims &d, const FwdArgs &a, uint8_t *save, int *status, cudaStream_t st, Tracer &tr) {
    CUtensorMap mq, mk, mv, mo;
    if (!make_tile_map(&mq, a.q, d.B, d.T, d.H, d.dk) || !make_tile_map(&mk, a.k, d.B, d.T, d.H, d.dk) ||
        !make_tile_map(&mv, a.v, d.B, d.T, d.H, d.dv) || !make_tile_map(&mo, a.o, d.B, d.T, d.H, d.dv))
        return -1;
    const bool vl = a.vl && a.vl->n_seq;
    const CUtensorMap *vm = vl ? gdn_varlen_maps(d, a, 0, st) : nullptr;
    if (vl && !vm) return -1;
    GdnParams p{a.lq, a.lk, a.log_decay, a.beta, a.h0, a.ht, save, 1, status, d.T, d.H, d.NT, d.scale,
                vl ? a.vl->d_seqs : nullptr, vm, d.dk, d.dv};
    k_gdn_fwd_tc<<<vl ? a.vl->n_seq * d.H : d.B * d.H, gd::NTHREADS, gd::SMEM_BYTES, st>>>(mq, mk, mv, mo, p);
    tr.mark("gdn_fwd_tc");
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace sla
