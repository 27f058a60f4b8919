// Softmax-GLA forward on the 5th-generation tensor cores (bf16 I/O, d_k and d_v 128 - or 64, run as 128 with zero padding supplied by the tensor maps -, chunk 64).
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

// shared memory: one log-decay buffer (dead right after the prologue), three q/k operand buffers (chunk n in the
// tensor core, n+1 in the prologue, n+2 in flight), two v buffers, the bf16 state operand, the masked A tile
constexpr uint32_t OFF_G = 0;                                   // 32 KiB fp32 log-decay tile
constexpr uint32_t QK_BYTES = 2 * TILE_BF16;                    // q then k
constexpr uint32_t OFF_QK = OFF_G + TILE_G;                     // [3]
constexpr uint32_t OFF_V = OFF_QK + 3 * QK_BYTES;               // [2]
constexpr uint32_t OFF_S = OFF_V + 2 * TILE_BF16;               // bf16 state operand: two halves of [128 rows][128 B]
constexpr uint32_t OFF_A = OFF_S + STATE_BF16;                  // masked A, [64 rows][128 B]
constexpr uint32_t OFF_OST = OFF_A + HALF_BF16;                 // bf16 output tile staged for the TMA store
constexpr uint32_t OFF_TOT = OFF_OST + TILE_BF16;               // prologue scratch
constexpr uint32_t OFF_EB = OFF_TOT + TOT_BYTES;                // [4][128] 2^{b_last} of four chunks
constexpr uint32_t OFF_GATE = OFF_EB + 4 * D * 4;               // [4][2][64]: scale*Gq, Gk of four chunks
constexpr uint32_t OFF_BAR = OFF_GATE + 4 * 2 * C * 4;          // mbarriers, see Bar
constexpr uint32_t OFF_TMEM = OFF_BAR + 40 * 8;                 // TMEM base address, then the abort flag
constexpr uint32_t SMEM_BYTES = OFF_TMEM + 16 + 1024;           // + slack to align the base to 1024 B
static_assert(SMEM_BYTES <= 232448, "shared memory budget");

constexpr uint32_t COL_A = 0, COL_O = 64, COL_S = 320, TMEM_COLS = 512;   // O: two buffers of 128 columns
constexpr int W_PRO = 8, W_MMA = 16, W_GATE = 17, W_TMA = 21;      // first warp of each role
constexpr int NTHREADS = 2 * NCOMPUTE + 32 + NGATE + 32;

// mbarrier slots (8 bytes each)
enum Bar { FULL_G = 0, FULL_QK = 1, FULL_V = 4, OPR = 6, GREADY = 9, GFREE = 13, SREADY = 17, OFREE, AREADY, BAR_A, BAR_Z,
           BAR_O /* [2], one per O accumulator */, OSTAGED = BAR_O + 2, OSFREE, DRAIN, QKFREE /* [3] */, SSAVED = QKFREE + 3, ATAKEN,
           OFREE2 /* OFREE, OFREE2: one per O accumulator (the output warps may be a chunk ahead of the waiter) */, NBAR };
static_assert(NBAR <= 40, "barrier slots");

struct FwdParams {
    const float *lq, *lk, *h0;
    const float *fin, *gam;         // segmented run (P > 1): per (sequence, segment) the state reached from zero and the total decay
    __nv_bfloat16 *o;
    float *ht;
    uint8_t *simg;                  // optional: [B*H][NT+1][32 KiB] bf16 images of the state before every chunk (P = 1 only)
    int *status;
    int T, H, NT;
    int P, L;                       // segments per sequence and chunks per segment (P = 1: L = NT)
    float scale;
    const float *log_gamma;         // Softmax-RetNet: [H] constant log-decays (no log-decay tensor is read); else nullptr
    const SeqInfo *seqs;            // packed variable-length batch: per-sequence table and tensor maps (q, k, v, g, o), else nullptr
    const CUtensorMap *vmaps;
    int dk, dv;             // head widths, each 128 or 64 (the upper half of a 128-wide tile is then zero padding)
};

// One CTA per (batch, head) sequence, five roles that only meet on mbarriers:
//   warps 8..15        prologue: cumulative decay, qh, kh of the chunks ahead (as far as the three q/k buffers allow)
//   warps 0..7         causal mask of A, state rescale, output staging (TMEM lane quarter = warp % 4)
//   warp 16 (one lane) every tcgen05.mma
//   warp 21 (one lane) TMA: loads (log-decay one chunk ahead, q/k three, v two) and the output store
//   warps 17..20       head-softmax gates (Eq. 4) up to four chunks ahead, one thread per (token, gate)
// The prologue of chunk n+1.. runs beside the mask / rescale / store work of chunk n, so the shared-memory,
// special-function and FMA phases of the two groups overlap instead of following one another.
__global__ void __launch_bounds__(NTHREADS, 1)
k_gla_fwd_tc(const __grid_constant__ CUtensorMap gm_q, const __grid_constant__ CUtensorMap gm_k,
             const __grid_constant__ CUtensorMap gm_v, const __grid_constant__ CUtensorMap gm_g,
             const __grid_constant__ CUtensorMap gm_o, FwdParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *sm = smem_raw + (base - raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // a sequence may be cut into p.P segments of p.L chunks, one CTA each, every segment starting from its own state
    const int bh = blockIdx.x / p.P, seg = blockIdx.x % p.P, h = bh % p.H;
    int b = bh / p.H;
    // A packed batch: this CTA's sequence has its own length, chunk count, first token, state slots and tensor maps
    // (based at its first token, so token coordinates stay relative and the batch coordinate is 0).
    size_t tokb = (size_t)b * p.T, slot = (size_t)bh * (p.NT + 1);
    size_t sbh = (size_t)bh;                                // (sequence, head) index into h0 / ht / dht / dh0
    const CUtensorMap *vm = nullptr;
    if (p.seqs) {
        const SeqInfo si = p.seqs[b];
        vm = p.vmaps + (size_t)b * Varlen::MAPS_PER_SEQ;
        p.T = si.T; p.NT = si.NT; p.L = si.NT;
        tokb = (size_t)si.t0;
        slot = (size_t)si.slot0 * p.H + (size_t)h * (si.NT + 1);
        sbh = (size_t)si.id * p.H + h;                      // (the table is ordered longest first, the state tensors as the caller gave them)
        b = 0;
    }
    const CUtensorMap &tm_q = vm ? vm[0] : gm_q, &tm_k = vm ? vm[1] : gm_k, &tm_v = vm ? vm[2] : gm_v,
                      &tm_g = vm ? vm[3] : gm_g, &tm_o = vm ? vm[4] : gm_o;
    const int n0 = seg * p.L, NT = min(p.L, p.NT - n0);     // this CTA's chunks: n0 .. n0+NT-1
    auto bar = [&](int i) { return base + OFF_BAR + 8u * i; };
    float *tot = reinterpret_cast<float *>(sm + OFF_TOT);
    float *eblast = reinterpret_cast<float *>(sm + OFF_EB);
    float *gate_s = reinterpret_cast<float *>(sm + OFF_GATE);
    // Every wait is bounded.  The first thread whose wait expires raises the CTA's abort flag; from then on nobody
    // waits any more, the control lane stops issuing and drains what is in flight, and the kernel reports the failure.
    volatile int *abort_flag = reinterpret_cast<volatile int *>(sm + OFF_TMEM + 8);
    bool failed = false;
    auto wait = [&](int i, uint32_t parity) {
        if (!failed && !mbar_wait_bounded(bar(i), parity, abort_flag)) { failed = true; *abort_flag = 1; }
    };
    auto wait_relaxed = [&](int i, uint32_t parity) {     // for the warps that run ahead: poll with a back-off
        if (!failed && !mbar_wait_bounded<128>(bar(i), parity, abort_flag)) { failed = true; *abort_flag = 1; }
    };

    if (tid == 0) {
        *abort_flag = 0;
        for (int i = 0; i < NBAR; ++i) {
            const bool all = (i >= OPR && i < GREADY) || (i >= GFREE && i <= AREADY) || i == OSTAGED || i == ATAKEN || i == OFREE2;   // 256 arrivals
            mbar_init(bar(i), all ? NCOMPUTE : (i >= GREADY && i < GFREE) ? NGATE / 32 : 1);
        }
        fence_mbar_init();
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
        tma_prefetch_desc(&tm_g);
        tma_prefetch_desc(&tm_o);
    }
    if (warp == 0) tmem_alloc(base + OFF_TMEM, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(sm + OFF_TMEM);

    if (warp == W_MMA) {
        // ---------------- MMA issue (one lane) ----------------
        if (lane == 0) {
            constexpr uint32_t ID_A = idesc_bf16(64, 64, 0, 0);      // qh (K-major) x kh (K-major)
            constexpr uint32_t ID_O = idesc_bf16(64, 128, 0, 1);     // qh x S, A x V (B operand MN-major)
            constexpr uint32_t ID_Z = idesc_bf16(128, 128, 1, 1);    // kh^T (MN-major) x V (MN-major)
            auto issue_a = [&](int n) {                              // A_n = qh kh^T, one chunk ahead of the recurrence
                const uint32_t sQ = base + OFF_QK + (n % 3) * QK_BYTES, sK = sQ + TILE_BF16;
                wait(OPR + n % 3, (n / 3) & 1);                      // qh, kh of chunk n are in place
                if (n > 0) wait(ATAKEN, (n - 1) & 1);                // A_{n-1} has been read out of tensor memory
                if (failed) return;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    tc_mma_bf16(tmem + COL_A, (desc_kmajor(sQ) + kstep_kmajor(kk, HALF_BF16)), (desc_kmajor(sK) + kstep_kmajor(kk, HALF_BF16)), ID_A, kk > 0);
                tc_commit(bar(BAR_A));
            };
            issue_a(0);
            for (int n = 0; n < NT && !failed; ++n) {
                const uint32_t par = n & 1;
                const uint32_t sQ = base + OFF_QK + (n % 3) * QK_BYTES, sK = sQ + TILE_BF16;
                const uint32_t sV = base + OFF_V + (n & 1) * TILE_BF16;
                const uint32_t tO = tmem + COL_O + (n & 1) * D;
                wait(SREADY, par);                     // S_n: fp32 in TMEM, bf16 in shared memory
                if (n > 1) wait((n & 1) ? OFREE2 : OFREE, ((n - 2) >> 1) & 1);   // O of chunk n-2 (same TMEM buffer) has been read out
                wait(FULL_V + (n & 1), (n >> 1) & 1);
                if (failed) break;
                tc_fence_after();
                // the recurrence: S += kh^T V and O = qh S_n; their commit releases the rescale
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    tc_mma_bf16(tmem + COL_S, (desc_mnmajor(sK, HALF_BF16) + kstep_mnmajor(kk)), (desc_mnmajor(sV, HALF_BF16) + kstep_mnmajor(kk)), ID_Z, 1);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    tc_mma_bf16(tO, (desc_kmajor(sQ) + kstep_kmajor(kk, HALF_BF16)), (desc_mnmajor(base + OFF_S, STATE_HALF) + kstep_mnmajor(kk)), ID_O, kk > 0);
                tc_commit(bar(BAR_Z));
                tc_commit(bar(QKFREE + n % 3));        // (same event, own barrier: the TMA lane may look at it much later)
                // beside the rescale: A of the next chunk, then A V of this one
                if (n + 1 < NT) issue_a(n + 1);
                wait(AREADY, par);                     // masked A_n is in shared memory
                if (failed) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)         // O += A V
                    tc_mma_bf16(tO, (desc_kmajor(base + OFF_A) + kstep_kmajor(kk, 0)), (desc_mnmajor(sV, HALF_BF16) + kstep_mnmajor(kk)), ID_O, 1);
                tc_commit(bar(BAR_O + (n & 1)));
            }
            // let the tensor core finish before TMEM goes away (after an abort some of its work may still be queued)
            tc_commit(bar(DRAIN));
            mbar_wait_bounded(bar(DRAIN), 0, nullptr, 20000000ull);
        }
    } else if (warp == W_TMA) {
        // ---------------- TMA (one lane): loads ahead of the compute warps, output stores behind them ----------------
        if (lane == 0) {
            auto load_qk = [&](int n) {
                const uint32_t bf = bar(FULL_QK + n % 3), dst = base + OFF_QK + (n % 3) * QK_BYTES;
                mbar_expect_tx(bf, QK_BYTES);
                tma_load_5d(dst, &tm_q, 0, (n0 + n) * C, 0, h, b, bf);
                tma_load_5d(dst + TILE_BF16, &tm_k, 0, (n0 + n) * C, 0, h, b, bf);
            };
            auto load_v = [&](int n) {
                const uint32_t bf = bar(FULL_V + (n & 1)), dst = base + OFF_V + (n & 1) * TILE_BF16;
                mbar_expect_tx(bf, TILE_BF16);
                tma_load_5d(dst, &tm_v, 0, (n0 + n) * C, 0, h, b, bf);
            };
            // save mode: S_m (the bf16 operand copy, as it stands in shared memory) -> image slot m, for the backward pass
            uint8_t *img0 = p.simg ? p.simg + slot * STATE_BF16 : nullptr;
            for (int n = 0; n < 3 && n < NT; ++n) load_qk(n);
            for (int n = 0; n < 2 && n < NT; ++n) load_v(n);
            // From here on the lane serves whichever buffer falls free or fills first (no fixed order: the prologue warps
            // run ahead of the tensor core by a varying distance).  Next chunk to load / store per stream:
            int nqk = 3, nv = 2, nst = 0, nsv = img0 ? 0 : NT + 1;
            auto ready = [&](int i, uint32_t parity) { return mbar_test_wait(bar(i), parity) != 0; };
            uint64_t t_idle = globaltimer_ns();
            for (uint32_t it = 0; !failed && (nst < NT || nsv <= NT); ++it) {
                bool progress = false;
                if (nqk < NT && ready(QKFREE + nqk % 3, ((nqk - 3) / 3) & 1)) { // A, qh S and kh^T V of chunk nqk-3 have read it
                    load_qk(nqk++);
                    progress = true;
                }
                if (nv < NT && ready(BAR_O + (nv & 1), ((nv - 2) >> 1) & 1)) {  // A V of chunk nv-2 has read it
                    load_v(nv++);
                    progress = true;
                }
                if (nsv <= NT && ready(SREADY, nsv & 1)) {                       // S_nsv stands in shared memory
                    bulk_store(img0 + (size_t)nsv * STATE_BF16, base + OFF_S, STATE_BF16);
                    bulk_commit();
                    bulk_wait_read0();
                    mbar_arrive(bar(SSAVED));
                    ++nsv;
                    progress = true;
                }
                if (nst < NT && ready(OSTAGED, nst & 1)) {                       // O of chunk nst is staged; rows past T are clipped
                    tma_store_5d(&tm_o, base + OFF_OST, 0, (n0 + nst) * C, 0, h, b);
                    bulk_commit();
                    bulk_wait_read0();
                    mbar_arrive(bar(OSFREE));
                    ++nst;
                    progress = true;
                }
                if (progress) {
                    t_idle = globaltimer_ns();
                } else if ((it & 31u) == 31u) {
                    if (*abort_flag || globaltimer_ns() - t_idle > 2000000000ull) { failed = true; *abort_flag = 1; }
                    __nanosleep(64);
                }
            }
            bulk_wait0();
            if (failed) {   // give loads that are still in flight time to land before shared memory goes away
                const uint64_t t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
            }
        }
    } else if (warp >= W_GATE) {
        // ---------------- gates: softmax over the heads, up to four chunks ahead ----------------
        const int g = tid - 32 * W_GATE, t = g & (C - 1);
        const float *l = g < C ? p.lq : p.lk;
        const float mult = g < C ? p.scale : 1.f;
        for (int n = 0; n < NT; ++n) {
            if (n >= 4) wait_relaxed(GFREE + (n & 3), ((n >> 2) - 1) & 1);
            if (failed) break;
            const int cn = min(C, p.T - (n0 + n) * C);
            chunk_gate(l + (tokb + (size_t)(n0 + n) * C) * p.H, p.H, cn, h, mult, gate_s + (n & 3) * 2 * C + (g < C ? 0 : C), t);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(GREADY + (n & 3)));
        }
    } else if (warp >= W_PRO) {
        // ---------------- prologue warps: qh, kh of every chunk, ahead of the tensor core ----------------
        const int ptid = tid - 32 * W_PRO;
        auto load_g = [&](int n) {                     // (one thread) log-decay tile of chunk n
            mbar_expect_tx(bar(FULL_G), TILE_G);
            tma_load_4d(base + OFF_G, &tm_g, 0, h, (n0 + n) * C, b, bar(FULL_G));
        };
        const bool retnet = p.log_gamma != nullptr;
        const float lgam = retnet ? p.log_gamma[h] : 0.f;
        if (ptid == 0 && !retnet) load_g(0);
        for (int n = 0; n < NT; ++n) {
            wait(GREADY + (n & 3), (n >> 2) & 1);
            if (!retnet) wait(FULL_G, n & 1);
            wait(FULL_QK + n % 3, (n / 3) & 1);
            if (failed) break;
            uint8_t *qk = sm + OFF_QK + (n % 3) * QK_BYTES;
            const float *g = gate_s + (n & 3) * 2 * C;
            // eblast has four slots: these warps are never more than three chunks ahead of the rescale that reads one
            chunk_prologue<true, false>(qk, qk + TILE_BF16, retnet ? nullptr : reinterpret_cast<const float *>(sm + OFF_G), tot, g, g + C,
                                        eblast + (n & 3) * D, nullptr, p.status, ptid, 2,
                                        [&]() { if (ptid == 0 && n + 1 < NT && !retnet) load_g(n + 1); },
                                        ScalarDecay{lgam, min(C, p.T - (n0 + n) * C)});
            fence_proxy_async();
            mbar_arrive(bar(OPR + n % 3));
            mbar_arrive(bar(GFREE + (n & 3)));
        }
    } else {
        // ---------------- mask / rescale / store warps ----------------
        const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;   // this warp's TMEM lane quarter
        const int colhalf = warp >> 2;                                   // which 64 state / output columns
        const int row = 32 * (warp & 3) + lane;

        {   // initial state: fp32 into TMEM, bf16 copy into shared memory (row = key dimension).  A segment that is not the
            // first starts from S <- diag(gam_s) S + fin_s taken over the segments s before it (a short scan over their
            // summaries, elementwise, done here rather than in a launch of its own).
            const float *src = state_row(p.h0, sbh, row, colhalf, p.dk, p.dv);
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = src ? src[32 * part + j] : 0.f;
                for (int sgm = 0; sgm < seg; ++sgm) {
                    const size_t c = (size_t)bh * p.P + sgm;
                    const float gmm = p.gam[c * D + row];
                    const float4 *f = reinterpret_cast<const float4 *>(p.fin + (c * D + row) * D + 64 * colhalf + 32 * part);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float4 x = f[j];
                        v[4 * j] = fmaf(gmm, v[4 * j], x.x);         v[4 * j + 1] = fmaf(gmm, v[4 * j + 1], x.y);
                        v[4 * j + 2] = fmaf(gmm, v[4 * j + 2], x.z); v[4 * j + 3] = fmaf(gmm, v[4 * j + 3], x.w);
                    }
                }
                tmem_st32(tmem + lane_base + COL_S + 64 * colhalf + 32 * part, v);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint4 w;
                    w.x = pack_bf16(v[8 * c + 0], v[8 * c + 1]);
                    w.y = pack_bf16(v[8 * c + 2], v[8 * c + 3]);
                    w.z = pack_bf16(v[8 * c + 4], v[8 * c + 5]);
                    w.w = pack_bf16(v[8 * c + 6], v[8 * c + 7]);
                    *reinterpret_cast<uint4 *>(sm + OFF_S + colhalf * STATE_HALF + swz(row, 4 * part + c)) = w;
                }
            }
            tmem_wait_st();
        }
        fence_proxy_async();
        tc_fence_before();
        mbar_arrive(bar(SREADY));

        // O of chunk m: TMEM -> bf16 -> staging tile (the TMA warp stores it)
        auto stage_o = [&](int m) {
            wait(BAR_O + (m & 1), (m >> 1) & 1);
            tc_fence_after();
            const int i = 16 * (warp & 3) + lane;
            float v0[32], v1[32];
            tmem_ld32(tmem + lane_base + COL_O + (m & 1) * D + 64 * colhalf, v0);
            tmem_ld32(tmem + lane_base + COL_O + (m & 1) * D + 64 * colhalf + 32, v1);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(bar((m & 1) ? OFREE2 : OFREE));
            if (m > 0) wait(OSFREE, (m - 1) & 1);      // the previous store has left the staging tile
            if (lane < 16) {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint4 w;
                    w.x = pack_bf16(v0[8 * c + 0], v0[8 * c + 1]);
                    w.y = pack_bf16(v0[8 * c + 2], v0[8 * c + 3]);
                    w.z = pack_bf16(v0[8 * c + 4], v0[8 * c + 5]);
                    w.w = pack_bf16(v0[8 * c + 6], v0[8 * c + 7]);
                    *reinterpret_cast<uint4 *>(sm + OFF_OST + colhalf * HALF_BF16 + swz(i, c)) = w;
                    w.x = pack_bf16(v1[8 * c + 0], v1[8 * c + 1]);
                    w.y = pack_bf16(v1[8 * c + 2], v1[8 * c + 3]);
                    w.z = pack_bf16(v1[8 * c + 4], v1[8 * c + 5]);
                    w.w = pack_bf16(v1[8 * c + 6], v1[8 * c + 7]);
                    *reinterpret_cast<uint4 *>(sm + OFF_OST + colhalf * HALF_BF16 + swz(i, 4 + c)) = w;
                }
            }
            fence_proxy_async();
            mbar_arrive(bar(OSTAGED));
        };
        // A_m: TMEM -> registers as soon as it is there (the tensor core may then start on A_{m+1}) -> causal mask -> bf16 ->
        // shared memory once A_{m-1} V has read the tile (row i of the M=64 tile sits in lane 32*(i/16) + i%16)
        auto mask_a = [&](int m) {
            wait(BAR_A, m & 1);
            tc_fence_after();
            const int i = 16 * (warp & 3) + lane, part = colhalf;
            float v[32];
            tmem_ld32(tmem + lane_base + COL_A + 32 * part, v);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(bar(ATAKEN));
            if (m > 0) {
                wait(BAR_O + ((m - 1) & 1), ((m - 1) >> 1) & 1);
                tc_fence_after();
            }
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
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(AREADY));
        };
        mask_a(0);
        for (int n = 0; n < NT; ++n) {
            const uint32_t par = n & 1;
            // the recurrence first: S_{n+1} = diag(2^{b_last}) (S_n + kh^T V), fp32 back into TMEM, bf16 copy for the next
            // chunk's qh S; the tensor core goes on with chunk n+1 the moment this is done
            wait(BAR_Z, par);
            tc_fence_after();
            if (p.simg) wait(SSAVED, par);             // the image store of S_n has read the operand copy
            {
                const float e = eblast[(n & 3) * D + row];
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
                        *reinterpret_cast<uint4 *>(sm + OFF_S + colhalf * STATE_HALF + swz(row, 4 * part + c)) = w;
                    }
                }
                tmem_wait_st();
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(SREADY));
            if (n + 1 < NT) mask_a(n + 1);             // beside the MMAs of chunk n+1: its A tile ...
            stage_o(n);                                // ... and this chunk's output
        }

        if (p.ht && seg == p.P - 1) {   // final state, fp32 (each thread reads back what it wrote in the last rescale)
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

// ---- host side ----
int sm_count() {
    static int n = 0;
    if (!n) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
    }
    return n;
}
// One CTA per sequence leaves most SMs idle when there are few sequences: then every sequence is cut into P segments
// of L chunks (at least 8), so that B*H*P comes close to the SM count.
void choose_segments(const Dims &d, int &P, int &L) {
    const int BH = d.B * d.H, sms = sm_count();
    P = 1;
    L = d.NT;
    if (BH > 0 && 2 * BH <= sms && d.NT >= 16) {
        const int want = sms / BH;
        L = (d.NT + want - 1) / want;
        if (L < 8) L = 8;
        P = (d.NT + L - 1) / L;
    }
}
}  // namespace

// Softmax-GLA (Eq. 12-13) and Softmax-RetNet (Eq. 10-11: the same recurrence with a constant decay per head, which the
// kernels generate instead of reading a [B,T,H,d_k] tensor).
bool gla_tc_supported(const Dims &d) {
    return (d.variant == SLA_GLA || d.variant == SLA_RETNET) && d.io_bf16 && (d.dk == 128 || d.dk == 64) && (d.dv == 128 || d.dv == 64) && d.C == 64;
}

int gla_tc_configure() {
    if (!encode_fn()) return -1;
    return cudaFuncSetAttribute(k_gla_fwd_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES) ==
                   cudaSuccess ? 0 : -1;
}

// The backward runs the gradient sweep twice when it is cut into segments (once for the state gradients that leave
// each segment, once for the results), so cutting pays only from three segments per sequence on.
void gla_tc_backward_choose_segments(const Dims &d, int &P, int &L) {
    choose_segments(d, P, L);
    if (P < 3) { P = 1; L = d.NT; }
}

size_t gla_tc_forward_workspace_bytes(const Dims &d, const Varlen *vl) {
    int P, L;
    choose_segments(d, P, L);
    if (P == 1 || (vl && vl->n_seq)) return 0;
    return (size_t)d.B * d.H * P * (D * D + D) * sizeof(float);
}

bool gla_tc_forward_can_save(const Dims &d, const Varlen *vl) {
    if (vl && vl->n_seq) return true;     // (a packed batch always runs one CTA per sequence)
    int P, L;
    choose_segments(d, P, L);
    return P == 1;
}

int gla_tc_forward(const Dims &d, const FwdArgs &a, uint8_t *simg, int *status, cudaStream_t st, Tracer &tr) {
    CUtensorMap mq, mk, mv, mg, mo;
    const bool retnet = d.variant == SLA_RETNET;
    if (a.vl && a.vl->n_seq) {          // packed batch: one CTA per (sequence, head), per-sequence tensor maps
        const void *key[] = {a.q, a.k, a.v, a.log_decay, a.o};
        const CUtensorMap *vm = varlen_maps(*a.vl, 0, key, 5, st, [&](const SeqInfo &si, CUtensorMap *m) {
            const size_t tok = (size_t)si.t0 * d.H;      // (q, k are d_k wide, v, o and their gradients d_v)
            const __nv_bfloat16 *q = (const __nv_bfloat16 *)a.q, *k = (const __nv_bfloat16 *)a.k, *v = (const __nv_bfloat16 *)a.v;
            if (!make_tile_map(m + 0, q + tok * d.dk, 1, si.T, d.H, d.dk) || !make_tile_map(m + 1, k + tok * d.dk, 1, si.T, d.H, d.dk) ||
                !make_tile_map(m + 2, v + tok * d.dv, 1, si.T, d.H, d.dv) || !make_tile_map(m + 4, (__nv_bfloat16 *)a.o + tok * d.dv, 1, si.T, d.H, d.dv))
                return false;
            if (retnet) { m[3] = m[0]; return true; }
            return make_map(m + 3, a.log_decay + tok * d.dk, 1, si.T, d.H, d.dk, true, 128);
        });
        if (!vm || !make_tile_map(&mq, a.q, d.B, d.T, d.H, d.dk)) return -1;
        FwdParams p{a.lq, a.lk, a.h0, nullptr, nullptr, (__nv_bfloat16 *)a.o, a.ht, simg, status, d.T, d.H, d.NT, 1, d.NT, d.scale,
                    retnet ? a.log_decay : nullptr, a.vl->d_seqs, vm, d.dk, d.dv};
        k_gla_fwd_tc<<<a.vl->n_seq * d.H, NTHREADS, SMEM_BYTES, st>>>(mq, mq, mq, mq, mq, p);
        tr.mark("gla_fwd_tc");
        return cudaGetLastError() == cudaSuccess ? 1 : -1;
    }
    if (!make_tile_map(&mq, a.q, d.B, d.T, d.H, d.dk) || !make_tile_map(&mk, a.k, d.B, d.T, d.H, d.dk) ||
        !make_tile_map(&mv, a.v, d.B, d.T, d.H, d.dv) || !make_tile_map(&mo, a.o, d.B, d.T, d.H, d.dv))
        return -1;
    if (retnet) mg = mq;   // (never used: the decay is generated in the kernel)
    else if (!make_map(&mg, a.log_decay, d.B, d.T, d.H, d.dk, true, 128)) return -1;
    int P, L, launches = 1;
    choose_segments(d, P, L);
    float *fin = nullptr, *gam = nullptr;
    if (P > 1) {   // segment summaries from a zero state, then the segments in parallel (each scans the summaries before it)
        const size_t nseg = (size_t)d.B * d.H * P;
        fin = a.ws;
        gam = fin + nseg * D * D;
        if (gla_tc_segment_summaries(d, a, P, L, fin, gam, status, st, tr) < 0) return -1;
        launches = 2;
        simg = nullptr;
    }
    FwdParams p{a.lq, a.lk, a.h0, fin, gam, (__nv_bfloat16 *)a.o, a.ht, simg, status, d.T, d.H, d.NT, P, L, d.scale, retnet ? a.log_decay : nullptr, nullptr, nullptr, d.dk, d.dv};
    k_gla_fwd_tc<<<d.B * d.H * P, NTHREADS, SMEM_BYTES, st>>>(mq, mk, mv, mg, mo, p);
    tr.mark("gla_fwd_tc");
    return cudaGetLastError() == cudaSuccess ? launches : -1;
}

}  // namespace sla
