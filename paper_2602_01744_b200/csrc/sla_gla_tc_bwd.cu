// Softmax-GLA backward on the 5th-generation tensor cores (bf16 I/O, d_k and d_v 128 - or 64, run as 128 with zero padding supplied by the tensor maps -, chunk 64).
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
// Few long sequences (at least three segments per sequence fit the SMs): gla_tc_backward_segmented runs both sweeps
// on segments of every sequence as the sequences of a packed batch, twice, with the states at the cuts and the state
// gradients across them folded from per-segment summaries (see there).
// Both kernels use the forward kernel's roles: one MMA-issuing lane, one TMA lane, gate warps running ahead and
// eight compute warps; every wait is bounded and abortable.
#include "sla_gla_tc.cuh"

namespace sla {
namespace {

using namespace ptx;
using namespace tc;

// ------------------------------------------------------------------------------------------------
// sweep 1: chunk states
namespace st1 {
constexpr uint32_t OFF_G = 0;                               // [2] fp32 log-decay tiles
constexpr uint32_t OFF_K = OFF_G + 2 * TILE_G;              // [3] k tiles (kh after the prologue)
constexpr uint32_t OFF_V = OFF_K + 3 * TILE_BF16;           // [2] v tiles
constexpr uint32_t OFF_IMG = OFF_V + 2 * TILE_BF16;         // bf16 state image staged for the bulk store
constexpr uint32_t OFF_TOT = OFF_IMG + STATE_BF16;          // prologue scratch
constexpr uint32_t OFF_EB = OFF_TOT + TOT_BYTES;            // [2][128] 2^{b_last}
constexpr uint32_t OFF_GATE = OFF_EB + 2 * D * 4;           // [4][64] Gk of four chunks
constexpr uint32_t OFF_BAR = OFF_GATE + 4 * C * 4;
constexpr uint32_t OFF_TMEM = OFF_BAR + 32 * 8;             // TMEM base address, then the abort flag
constexpr uint32_t SMEM_BYTES = OFF_TMEM + 16 + 1024;
constexpr uint32_t TMEM_COLS = 128;
constexpr int NGATE1 = 64;                                  // gate threads (Gk only)
constexpr int NTHREADS = NCOMPUTE + 32 + NGATE1 + 32;       // warps 0..7 compute, 8 MMA issue, 9..10 gates, 11 TMA
enum Bar { FULL_G = 0 /*[2]*/, FULL_K = 2 /*[3]*/, FULL_V = 5 /*[2]*/, OPR = 7 /*[3]*/, GREADY = 10 /*[4]*/, GFREE = 14 /*[4]*/,
           SREADY = 18, STAGED, STFREE, BAR_Z, KFREE /*[3]*/, VFREE = KFREE + 3 /*[2]*/, DRAIN = VFREE + 2, NBAR };
static_assert(NBAR <= 32, "barrier slots");
}  // namespace st1

struct StatesParams {
    const float *lq, *lk, *h0;
    uint8_t *simg;          // [B*H][NT+1][32 KiB] bf16 state images (image mode)
    float *fin, *gam;       // summary mode: per CTA the state reached from a zero start [128][128] and the total decay [128]
    int *status;
    int T, H, NT;
    int P, L;               // segments per sequence and chunks per segment (image mode: P = 1, L = NT)
    const float *log_gamma; // Softmax-RetNet: [H] constant log-decays (no log-decay tensor is read); else nullptr
    const SeqInfo *seqs;    // packed variable-length batch: per-sequence table and tensor maps (k, v, g), else nullptr
    const CUtensorMap *vmaps;
    int dk, dv;             // head widths, each 128 or 64 (the upper half of a 128-wide tile is then zero padding)
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

// Per chunk: prologue of chunk n+1 (kh only) while the tensor core adds kh^T V of chunk n to S; then S is rescaled in
// TMEM and its bf16 image goes to global memory through a staged bulk store (image mode, for the backward pass).
// Summary mode (simg == nullptr) serves the segmented forward of long sequences: every CTA runs one segment of a
// sequence from a zero state and leaves only where it ended and the segment's total decay; a scan over the segments
// then gives every segment its true starting state.
__global__ void __launch_bounds__(st1::NTHREADS, 1)
k_gla_states_tc(const __grid_constant__ CUtensorMap gm_k, const __grid_constant__ CUtensorMap gm_v,
                const __grid_constant__ CUtensorMap gm_g, StatesParams p) {
    using namespace st1;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *sm = smem_raw + (base - raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.x / p.P, seg = blockIdx.x % p.P, h = bh % p.H;
    int b = bh / p.H;
    size_t tokb = (size_t)b * p.T, slot = (size_t)bh * (p.NT + 1);
    size_t sbh = (size_t)bh;                                // (sequence, head) index into h0 / ht / dht / dh0
    const CUtensorMap *vm = nullptr;
    if (p.seqs) {                                           // packed batch: see k_gla_fwd_tc
        const SeqInfo si = p.seqs[b];
        vm = p.vmaps + (size_t)b * Varlen::MAPS_PER_SEQ;
        p.T = si.T; p.NT = si.NT; p.L = si.NT;
        tokb = (size_t)si.t0;
        slot = (size_t)si.slot0 * p.H + (size_t)h * (si.NT + 1);
        sbh = (size_t)si.id * p.H + h;                      // (the table is ordered longest first, the state tensors as the caller gave them)
        b = 0;
    }
    const CUtensorMap &tm_k = vm ? vm[0] : gm_k, &tm_v = vm ? vm[1] : gm_v, &tm_g = vm ? vm[2] : gm_g;
    const int n0 = seg * p.L, NT = min(p.L, p.NT - n0);     // this CTA's chunks: n0 .. n0+NT-1
    const bool images = p.simg != nullptr;
    auto bar = [&](int i) { return base + OFF_BAR + 8u * i; };
    float *tot = reinterpret_cast<float *>(sm + OFF_TOT);
    float *eblast = reinterpret_cast<float *>(sm + OFF_EB);
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
            const bool all = (i >= OPR && i < GREADY) || (i >= GFREE && i <= STAGED);
            mbar_init(bar(i), all ? NCOMPUTE : (i >= GREADY && i < GFREE) ? NGATE1 / 32 : 1);
        }
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
    uint8_t *img0 = p.simg + slot * STATE_BF16;                       // (image mode: one segment, NT = p.NT)

    if (warp == 8) {
        // ---------------- MMA issue (one lane) ----------------
        if (lane == 0) {
            constexpr uint32_t ID_Z = idesc_bf16(128, 128, 1, 1);    // kh^T (MN-major) x V (MN-major)
            for (int n = 0; n < NT; ++n) {
                const uint32_t sK = base + OFF_K + (n % 3) * TILE_BF16, sV = base + OFF_V + (n & 1) * TILE_BF16;
                wait(OPR + n % 3, (n / 3) & 1);        // kh of chunk n is in place
                wait(SREADY, n & 1);                   // S_n is in TMEM
                wait(FULL_V + (n & 1), (n >> 1) & 1);
                if (failed) break;
                tc_fence_after();
                const uint64_t dK = desc_mnmajor(sK, HALF_BF16), dV = desc_mnmajor(sV, HALF_BF16);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)         // S += kh^T V
                    tc_mma_bf16(tmem, dK + kstep_mnmajor(kk), dV + kstep_mnmajor(kk), ID_Z, 1);
                tc_commit(bar(BAR_Z));
                tc_commit(bar(KFREE + n % 3));         // (same event on per-buffer barriers for the TMA lane)
                tc_commit(bar(VFREE + (n & 1)));
            }
            tc_commit(bar(DRAIN));
            mbar_wait_bounded(bar(DRAIN), 0, nullptr, 20000000ull);
        }
    } else if (warp == 11) {
        // ---------------- TMA (one lane) ----------------
        if (lane == 0) {
            auto load_g = [&](int n) {
                mbar_expect_tx(bar(FULL_G + (n & 1)), TILE_G);
                tma_load_4d(base + OFF_G + (n & 1) * TILE_G, &tm_g, 0, h, (n0 + n) * C, b, bar(FULL_G + (n & 1)));
            };
            auto load_k = [&](int n) {
                const uint32_t bf = bar(FULL_K + n % 3);
                mbar_expect_tx(bf, TILE_BF16);
                tma_load_5d(base + OFF_K + (n % 3) * TILE_BF16, &tm_k, 0, (n0 + n) * C, 0, h, b, bf);
            };
            auto load_v = [&](int n) {
                const uint32_t bf = bar(FULL_V + (n & 1));
                mbar_expect_tx(bf, TILE_BF16);
                tma_load_5d(base + OFF_V + (n & 1) * TILE_BF16, &tm_v, 0, (n0 + n) * C, 0, h, b, bf);
            };
            const bool retnet = p.log_gamma != nullptr;
            for (int n = 0; n < 2 && n < NT && !retnet; ++n) load_g(n);
            for (int n = 0; n < 3 && n < NT; ++n) load_k(n);
            for (int n = 0; n < 2 && n < NT; ++n) load_v(n);
            for (int n = 0; n < NT && !failed; ++n) {
                if (n + 2 < NT && !retnet) {         // log-decay buffer: free once the prologue of chunk n is done
                    wait(OPR + n % 3, (n / 3) & 1);
                    if (failed) break;
                    load_g(n + 2);
                }
                if (n + 3 < NT) {
                    wait(KFREE + n % 3, (n / 3) & 1);
                    if (failed) break;
                    load_k(n + 3);
                }
                if (n + 2 < NT) {
                    wait(VFREE + (n & 1), (n >> 1) & 1);
                    if (failed) break;
                    load_v(n + 2);
                }
                if (!images) continue;
                wait_relaxed(STAGED, n & 1);           // image of S_{n+1} is staged
                if (failed) break;
                bulk_store(img0 + (size_t)(n + 1) * STATE_BF16, base + OFF_IMG, STATE_BF16);
                bulk_commit();
                bulk_wait_read0();
                mbar_arrive(bar(STFREE));
            }
            bulk_wait0();
            if (failed) {   // give loads that are still in flight time to land before shared memory goes away
                const uint64_t t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
            }
        }
    } else if (warp >= 9) {
        // ---------------- gates (Gk only), up to four chunks ahead ----------------
        const int t = tid - (NCOMPUTE + 32);
        for (int n = 0; n < NT; ++n) {
            if (n >= 4) wait_relaxed(GFREE + (n & 3), ((n >> 2) - 1) & 1);
            if (failed) break;
            const int cn = min(C, p.T - (n0 + n) * C);
            chunk_gate(p.lk + (tokb + (size_t)(n0 + n) * C) * p.H, p.H, cn, h, 1.f, gate_s + (n & 3) * C, t);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(GREADY + (n & 3)));
        }
    } else {
        // ---------------- compute warps ----------------
        const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;
        const int colhalf = warp >> 2;
        const int row = 32 * (warp & 3) + lane;
        {   // S_0: fp32 into TMEM, bf16 image into slot 0
            const float *src = images ? state_row(p.h0, sbh, row, colhalf, p.dk, p.dv) : nullptr;
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = src ? src[32 * part + j] : 0.f;
                tmem_st32(tmem + lane_base + 64 * colhalf + 32 * part, v);
                if (images) store_state_part(img0, row, colhalf, part, v);
            }
            tmem_wait_st();
        }
        tc_fence_before();
        mbar_arrive(bar(SREADY));

        const bool retnet = p.log_gamma != nullptr;
        const float lgam = retnet ? p.log_gamma[h] : 0.f;
        auto prologue = [&](int n) {
            wait(GREADY + (n & 3), (n >> 2) & 1);
            if (!retnet) wait(FULL_G + (n & 1), (n >> 1) & 1);
            wait(FULL_K + n % 3, (n / 3) & 1);
            chunk_prologue<false, false>(nullptr, sm + OFF_K + (n % 3) * TILE_BF16,
                                         retnet ? nullptr : reinterpret_cast<const float *>(sm + OFF_G + (n & 1) * TILE_G), tot, nullptr,
                                         gate_s + (n & 3) * C, eblast + (n & 1) * D, nullptr, p.status, tid, 1, NoHook(),
                                         ScalarDecay{lgam, min(C, p.T - (n0 + n) * C)});
            fence_proxy_async();
            mbar_arrive(bar(OPR + n % 3));
            mbar_arrive(bar(GFREE + (n & 3)));
        };
        prologue(0);
        float gam = 1.f;                               // product of the chunks' 2^{b_last} for key dimension `row`
        for (int n = 0; n < NT; ++n) {
            if (n + 1 < NT) prologue(n + 1);         // overlaps the MMA of chunk n
            wait(BAR_Z, n & 1);
            tc_fence_after();
            {   // S_{n+1} = diag(2^{b_last}) (S_n + kh^T V): fp32 back into TMEM, bf16 image staged for slot n+1
                const float e = eblast[(n & 1) * D + row];
                gam *= e;
                float v0[32], v1[32];
                const uint32_t ta = tmem + lane_base + 64 * colhalf;
                tmem_ld32(ta, v0);
                tmem_ld32(ta + 32, v1);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) { v0[j] *= e; v1[j] *= e; }
                tmem_st32(ta, v0);
                tmem_st32(ta + 32, v1);
                if (images) {
                    if (n > 0) wait(STFREE, (n - 1) & 1);  // the previous image has left the staging buffer
                    store_state_part(sm + OFF_IMG, row, colhalf, 0, v0);
                    store_state_part(sm + OFF_IMG, row, colhalf, 1, v1);
                } else if (n == NT - 1) {              // summary mode: where the segment ended, fp32
                    float *dst = p.fin + ((size_t)blockIdx.x * D + row) * D + 64 * colhalf;
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        *reinterpret_cast<float4 *>(dst + j) = make_float4(v0[j], v0[j + 1], v0[j + 2], v0[j + 3]);
                        *reinterpret_cast<float4 *>(dst + 32 + j) = make_float4(v1[j], v1[j + 1], v1[j + 2], v1[j + 3]);
                    }
                    if (colhalf == 0) p.gam[(size_t)blockIdx.x * D + row] = gam;
                }
                tmem_wait_st();
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(SREADY));
            mbar_arrive(bar(STAGED));
        }
    }
    if (failed) atomicOr(p.status, STATUS_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, TMEM_COLS);
}

// ------------------------------------------------------------------------------------------------
// sweep 2: gradients
namespace st2 {
// two 32 KiB operand buffers that swap roles every chunk: one holds (q, k) -> (qh, kh) -> (dq, dk staged for the
// store), the other (v, dO); the next chunk's q, k land in the (v, dO) buffer as soon as the MMAs have read it
constexpr uint32_t OFF_X = 0, OFF_Y = 2 * TILE_BF16;
constexpr uint32_t OFF_G = 4 * TILE_BF16;               // fp32 log-decay tile (dead after the prologue)
constexpr uint32_t OFF_E2 = OFF_G + TILE_G;             // [64][128] x (bf16 gq 2^b, bf16 gk 2^-b)
constexpr uint32_t OFF_S = OFF_E2 + TILE_G;             // bf16 S_n image
constexpr uint32_t OFF_DZ = OFF_S + STATE_BF16;         // bf16 dZ operand; afterwards the fp32 dlog_decay tile staged for the store
constexpr uint32_t OFF_A = OFF_DZ + STATE_BF16;         // masked A, [64 rows][128 B]
constexpr uint32_t OFF_DA = OFF_A + HALF_BF16;          // masked dA; afterwards A|dA hold the dv tile staged for the store
constexpr uint32_t OFF_TOT = OFF_DA + HALF_BF16;        // prologue scratch
constexpr uint32_t OFF_EB = OFF_TOT + TOT_BYTES;        // [128] 2^{b_last}
constexpr uint32_t OFF_GATE = OFF_EB + D * 4;           // [4][2][64]: scale*Gq, Gk of four chunks
constexpr uint32_t OFF_R = OFF_GATE + 4 * 2 * C * 4;    // [2 buffers][2 column halves][128] rowsum(dS*S) partials
constexpr uint32_t OFF_UP = OFF_R + 4 * D * 4;          // [128] suffix total of the upper 32 tokens
constexpr uint32_t OFF_RED = OFF_UP + D * 4;            // [2][8 warps][32] gate partial sums
constexpr uint32_t OFF_BAR = OFF_RED + 2 * 8 * 32 * 4;
constexpr uint32_t OFF_TMEM = OFF_BAR + 32 * 8;         // TMEM base address, then the abort flag
constexpr uint32_t SMEM_BYTES = OFF_TMEM + 16 + 1024;
constexpr uint32_t COL_DS = 0, COL_A = 128, COL_DA = 192, COL_DQ = 256, COL_DK = 320, COL_DV = 384, TMEM_COLS = 512;
constexpr int NTHREADS = NCOMPUTE + 32 + NGATE + 32;    // warps 0..7 compute, 8 MMA issue, 9..12 gates, 13 TMA
enum Bar { FULL_G = 0, FULL_QK, FULL_V, FULL_DO, FULL_S, OPR, GREADY /*[4]*/, GFREE = GREADY + 4 /*[4]*/, ZREADY = GFREE + 4,
           AREADY, OUT1, OUT2, SNFREE, INIT_DONE, DGFREE, BAR_A, BAR_M1, BAR_M2, DOFREE, INIT_FULL, DRAIN, BAR_DS, NBAR };
static_assert(SMEM_BYTES <= 232448, "shared memory budget");
static_assert(NBAR <= 32, "barrier slots");
}  // namespace st2

struct BwdParams {
    const float *lq, *lk, *dht;
    const uint8_t *simg;
    float *pq, *pk, *dh0;          // pq = Gq*dGq, pk = Gk*dGk per (token, head)
    int *status;
    int T, H, NT;
    float scale;
    const float *log_gamma;         // Softmax-RetNet: [H] constant log-decays (no log-decay read, no log-decay gradient)
    const SeqInfo *seqs;            // packed variable-length batch: per-sequence table and tensor maps (the nine below), else nullptr
    const CUtensorMap *vmaps;
    int dk, dv;             // head widths, each 128 or 64 (the upper half of a 128-wide tile is then zero padding)
};

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

// Chunks in reverse order.  Per chunk n the compute warps run: prologue -> dZ = diag(2^{b_last}) dS_{n+1} -> causal
// mask of A and dA -> gradient tiles out of TMEM.  The MMA lane issues each product as soon as its operands exist:
// A, dA and S_n dO^T after the prologue; dZ V^T, dZ^T kh^T and qh^T dO after the dZ pass; only the three products
// with the masked tiles wait for the mask.  All four gradient tensors leave through staged TMA stores (rows past T
// are clipped by the tensor map).
__global__ void __launch_bounds__(st2::NTHREADS, 1)
k_gla_bwd_tc(const __grid_constant__ CUtensorMap gm_q, const __grid_constant__ CUtensorMap gm_k,
             const __grid_constant__ CUtensorMap gm_v, const __grid_constant__ CUtensorMap gm_do,
             const __grid_constant__ CUtensorMap gm_g, const __grid_constant__ CUtensorMap gm_dq,
             const __grid_constant__ CUtensorMap gm_dk, const __grid_constant__ CUtensorMap gm_dv,
             const __grid_constant__ CUtensorMap gm_dg, BwdParams p) {
    using namespace st2;
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
    if (p.seqs) {                                           // packed batch: see k_gla_fwd_tc
        const SeqInfo si = p.seqs[b];
        vm = p.vmaps + (size_t)b * Varlen::MAPS_PER_SEQ;
        p.T = si.T; p.NT = si.NT;
        tokb = (size_t)si.t0;
        slot = (size_t)si.slot0 * p.H + (size_t)h * (si.NT + 1);
        sbh = (size_t)si.id * p.H + h;                      // (the table is ordered longest first, the state tensors as the caller gave them)
        b = 0;
    }
    const CUtensorMap &tm_q = vm ? vm[0] : gm_q, &tm_k = vm ? vm[1] : gm_k, &tm_v = vm ? vm[2] : gm_v,
                      &tm_do = vm ? vm[3] : gm_do, &tm_g = vm ? vm[4] : gm_g, &tm_dq = vm ? vm[5] : gm_dq,
                      &tm_dk = vm ? vm[6] : gm_dk, &tm_dv = vm ? vm[7] : gm_dv, &tm_dg = vm ? vm[8] : gm_dg;
    auto bar = [&](int i) { return base + OFF_BAR + 8u * i; };
    float *tot = reinterpret_cast<float *>(sm + OFF_TOT);
    float *eblast = reinterpret_cast<float *>(sm + OFF_EB);
    float *gate_s = reinterpret_cast<float *>(sm + OFF_GATE);
    float *Rs = reinterpret_cast<float *>(sm + OFF_R);
    float *up = reinterpret_cast<float *>(sm + OFF_UP);
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
            const bool all = i == OPR || (i >= GFREE && i <= INIT_DONE);
            mbar_init(bar(i), all ? NCOMPUTE : (i >= GREADY && i < GFREE) ? NGATE / 32 : 1);
        }
        fence_mbar_init();
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
        tma_prefetch_desc(&tm_do);
        tma_prefetch_desc(&tm_g);
        tma_prefetch_desc(&tm_dq);
        tma_prefetch_desc(&tm_dk);
        tma_prefetch_desc(&tm_dv);
        tma_prefetch_desc(&tm_dg);
    }
    if (warp == 0) tmem_alloc(base + OFF_TMEM, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(sm + OFF_TMEM);
    const uint8_t *img0 = p.simg + slot * STATE_BF16;
    const int NT = p.NT;
    // chunks are visited in the order n = NT-1 ... 0; k = NT-1-n is the visit number that drives every barrier parity

    if (warp == 8) {
        // ---------------- MMA issue (one lane) ----------------
        if (lane == 0) {
            constexpr uint32_t ID_A = idesc_bf16(64, 64, 0, 0);
            constexpr uint32_t ID_KK = idesc_bf16(128, 64, 0, 0), ID_MK = idesc_bf16(128, 64, 1, 0),
                               ID_MM = idesc_bf16(128, 64, 1, 1), ID_S = idesc_bf16(128, 128, 1, 1);
            const uint64_t kS = desc_kmajor(base + OFF_S), kDZ = desc_kmajor(base + OFF_DZ),
                           mDZ = desc_mnmajor(base + OFF_DZ, STATE_HALF), mA = desc_mnmajor(base + OFF_A, HALF_BF16),
                           kDA = desc_kmajor(base + OFF_DA), mDA = desc_mnmajor(base + OFF_DA, HALF_BF16);
            for (int k = 0; k < NT; ++k) {
                const uint32_t par = k & 1;
                const uint32_t sQ = base + ((k & 1) ? OFF_Y : OFF_X), sK = sQ + TILE_BF16;
                const uint32_t sV = base + ((k & 1) ? OFF_X : OFF_Y), sDO = sV + TILE_BF16;
                const uint64_t kQ = desc_kmajor(sQ), kK = desc_kmajor(sK), kV = desc_kmajor(sV), kDO = desc_kmajor(sDO),
                               mQ = desc_mnmajor(sQ, HALF_BF16), mK = desc_mnmajor(sK, HALF_BF16),
                               mDO = desc_mnmajor(sDO, HALF_BF16);
                // dA = dO V^T and S_n dO^T need no prologue: they are issued while the compute warps still scale q and k
                wait(FULL_V, par);
                wait(FULL_DO, par);
                if (failed) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)         // dA = dO V^T
                    tc_mma_bf16(tmem + COL_DA, kDO + kstep_kmajor(kk, HALF_BF16), kV + kstep_kmajor(kk, HALF_BF16), ID_A, kk > 0);
                bool sdo_done = false;
                auto issue_sdo = [&]() {               // dqh^T = S_n dO^T ...
                    if (k > 0) wait(OUT1, (k - 1) & 1);    // dqh^T, dkh^T of the previous chunk have been read out (long ago)
                    tc_fence_after();
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        tc_mma_bf16(tmem + COL_DQ, kS + kstep_kmajor(kk, STATE_HALF), kDO + kstep_kmajor(kk, HALF_BF16), ID_KK, kk > 0);
                    sdo_done = true;
                };
                {   // whichever comes first: S_n landed, or the prologue done
                    const uint64_t t0 = globaltimer_ns();
                    for (uint32_t it = 0; !failed && !mbar_test_wait(bar(OPR), par); ++it) {
                        if (!sdo_done && mbar_test_wait(bar(FULL_S), par)) issue_sdo();
                        if ((it & 63u) == 63u && (*abort_flag || globaltimer_ns() - t0 > 2000000000ull)) { failed = true; *abort_flag = 1; }
                    }
                }
                if (failed) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)         // A = qh kh^T
                    tc_mma_bf16(tmem + COL_A, kQ + kstep_kmajor(kk, HALF_BF16), kK + kstep_kmajor(kk, HALF_BF16), ID_A, kk > 0);
                tc_commit(bar(BAR_A));
                if (!sdo_done) {
                    wait(FULL_S, par);
                    if (failed) break;
                    issue_sdo();
                }
                if (k > 0) wait(OUT2, (k - 1) & 1);    // dV^T and dS of the previous chunk have been read out
                wait(ZREADY, par);                     // dZ: fp32 in TMEM, bf16 in shared memory
                if (failed) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {       // three independent accumulation chains, interleaved
                    tc_mma_bf16(tmem + COL_DK, kDZ + kstep_kmajor(kk, STATE_HALF), kV + kstep_kmajor(kk, HALF_BF16), ID_KK, kk > 0);   // dkh^T = dZ V^T ...
                    tc_mma_bf16(tmem + COL_DV, mDZ + kstep_mnmajor(kk), kK + kstep_kmajor(kk, HALF_BF16), ID_MK, kk > 0);            // dV^T = dZ^T kh^T ...
                    if (kk < 4) tc_mma_bf16(tmem + COL_DS, mQ + kstep_mnmajor(kk), mDO + kstep_mnmajor(kk), ID_S, 1);                // dS_n = dZ + qh^T dO
                }
                tc_commit(bar(BAR_DS));                // dS_n is complete (and S_n dO^T has read S_n)
                wait(AREADY, par);                     // masked A, dA in shared memory
                if (failed) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {       // ... + kh^T dA^T  and  ... + qh^T dA, interleaved
                    tc_mma_bf16(tmem + COL_DQ, mK + kstep_mnmajor(kk), kDA + kstep_kmajor(kk, 0), ID_MK, 1);
                    tc_mma_bf16(tmem + COL_DK, mQ + kstep_mnmajor(kk), mDA + kstep_mnmajor(kk), ID_MM, 1);
                }
                tc_commit(bar(BAR_M1));
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)         // ... + dO^T A
                    tc_mma_bf16(tmem + COL_DV, mDO + kstep_mnmajor(kk), mA + kstep_mnmajor(kk), ID_MM, 1);
                tc_commit(bar(BAR_M2));
                tc_commit(bar(DOFREE));                // (same event, for the TMA lane)
            }
            tc_commit(bar(DRAIN));
            mbar_wait_bounded(bar(DRAIN), 0, nullptr, 20000000ull);
        }
    } else if (warp == 13) {
        // ---------------- TMA (one lane) ----------------
        if (lane == 0) {
            auto load_g = [&](int n) {
                mbar_expect_tx(bar(FULL_G), TILE_G);
                tma_load_4d(base + OFF_G, &tm_g, 0, h, n * C, b, bar(FULL_G));
            };
            // visit k keeps (q, k) in buffer k&1 and (v, dO) in the other one
            auto load_qk = [&](int n, int k) {
                const uint32_t dst = base + ((k & 1) ? OFF_Y : OFF_X);
                mbar_expect_tx(bar(FULL_QK), 2 * TILE_BF16);
                tma_load_5d(dst, &tm_q, 0, n * C, 0, h, b, bar(FULL_QK));
                tma_load_5d(dst + TILE_BF16, &tm_k, 0, n * C, 0, h, b, bar(FULL_QK));
            };
            auto load_vdo = [&](int n, int k) {
                const uint32_t dst = base + ((k & 1) ? OFF_X : OFF_Y);
                mbar_expect_tx(bar(FULL_V), TILE_BF16);
                tma_load_5d(dst, &tm_v, 0, n * C, 0, h, b, bar(FULL_V));
                mbar_expect_tx(bar(FULL_DO), TILE_BF16);
                tma_load_5d(dst + TILE_BF16, &tm_do, 0, n * C, 0, h, b, bar(FULL_DO));
            };
            auto load_s = [&](int n) {
                mbar_expect_tx(bar(FULL_S), STATE_BF16);
                bulk_load(base + OFF_S, img0 + (size_t)n * STATE_BF16, STATE_BF16, bar(FULL_S));
            };
            const bool retnet = p.log_gamma != nullptr;
            if (p.dht) {                               // S_NT, for rowsum(dht * S_NT)
                mbar_expect_tx(bar(INIT_FULL), STATE_BF16);
                bulk_load(base + OFF_S, img0 + (size_t)NT * STATE_BF16, STATE_BF16, bar(INIT_FULL));
            }
            if (!retnet) load_g(NT - 1);
            load_qk(NT - 1, 0);
            load_vdo(NT - 1, 0);
            if (p.dht) wait(INIT_DONE, 0);             // the compute warps are done with S_NT
            if (!failed) load_s(NT - 1);
            for (int k = 0; k < NT && !failed; ++k) {
                const int n = NT - 1 - k;
                const uint32_t par = k & 1;
                const uint32_t sQK = base + ((k & 1) ? OFF_Y : OFF_X);
                if (n > 0) {
                    // the next chunk's tiles can only be loaded as this chunk's buffers fall free: have them in L2 by then
                    tma_prefetch_l2_5d(&tm_q, 0, (n - 1) * C, 0, h, b);
                    tma_prefetch_l2_5d(&tm_k, 0, (n - 1) * C, 0, h, b);
                    tma_prefetch_l2_5d(&tm_v, 0, (n - 1) * C, 0, h, b);
                    tma_prefetch_l2_5d(&tm_do, 0, (n - 1) * C, 0, h, b);
                    bulk_prefetch_l2(img0 + (size_t)(n - 1) * STATE_BF16, STATE_BF16);
                    wait(OPR, par);                    // prologue done: the log-decay buffer is free
                    if (failed) break;
                    if (!retnet) load_g(n - 1);
                    wait(DOFREE, par);                 // every MMA of the chunk is done: its (v, dO) buffer takes the next q, k
                    if (failed) break;
                    load_qk(n - 1, k + 1);
                }
                if (n > 0) {
                    wait(SNFREE, par);                 // rowsum(dS_n * S_n) done (and S_n dO^T issued long ago): S_n no longer needed
                    if (failed) break;
                    load_s(n - 1);
                }
                wait(OUT1, par);                       // dq, dk staged over qh, kh
                if (failed) break;
                tma_store_5d(&tm_dq, sQK, 0, n * C, 0, h, b);
                tma_store_5d(&tm_dk, sQK + TILE_BF16, 0, n * C, 0, h, b);
                bulk_commit();
                bulk_wait_read0();
                if (n > 0) load_vdo(n - 1, k + 1);     // ... and this buffer takes the next v, dO
                wait(OUT2, par);                       // dv, dlog_decay staged
                if (failed) break;
                tma_store_5d(&tm_dv, base + OFF_A, 0, n * C, 0, h, b);
                if (!retnet) tma_store_4d(&tm_dg, base + OFF_DZ, 0, h, n * C, b);
                bulk_commit();
                bulk_wait_read0();
                mbar_arrive(bar(DGFREE));
            }
            bulk_wait0();
            if (failed) {
                const uint64_t t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
            }
        }
    } else if (warp >= 9) {
        // ---------------- gates, up to four chunks ahead ----------------
        const int g = tid - (NCOMPUTE + 32), t = g & (C - 1);
        const float *l = g < C ? p.lq : p.lk;
        const float mult = g < C ? p.scale : 1.f;
        for (int k = 0; k < NT; ++k) {
            const int n = NT - 1 - k;
            if (k >= 4) wait_relaxed(GFREE + (k & 3), ((k >> 2) - 1) & 1);
            if (failed) break;
            const int cn = min(C, p.T - n * C);
            chunk_gate(l + (tokb + (size_t)n * C) * p.H, p.H, cn, h, mult, gate_s + (k & 3) * 2 * C + (g < C ? 0 : C), t);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(GREADY + (k & 3)));
        }
    } else {
        // ---------------- compute warps ----------------
        const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;
        const int wh = warp >> 2;                       // column half (state passes) / token half (gradient tiles)
        const int row = 32 * (warp & 3) + lane;         // TMEM lane = key (value) dimension owned by this thread
        const bool retnet = p.log_gamma != nullptr;
        const float lgam = retnet ? p.log_gamma[h] : 0.f;

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

        {   // dS_NT = dht (or zero) into TMEM; R_{NT-1} = rowsum(dht * S_NT)
            float rpart = 0.f;
            if (p.dht) wait(INIT_FULL, 0);
            const float *src = state_row(p.dht, sbh, row, wh, p.dk, p.dv);
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = src ? src[32 * part + j] : 0.f;
                tmem_st32(tmem + lane_base + COL_DS + 64 * wh + 32 * part, v);
                if (p.dht) rpart += rowdot_part(v, part);
            }
            tmem_wait_st();
            Rs[((NT - 1) & 1) * 2 * D + wh * D + row] = rpart;
            if (p.dht) mbar_arrive(bar(INIT_DONE));     // S_NT is no longer needed
        }

        for (int k = 0; k < NT; ++k) {
            const int n = NT - 1 - k, t0 = n * C;
            const uint32_t par = k & 1;
            uint8_t *qk = sm + ((k & 1) ? OFF_Y : OFF_X);          // this chunk's q, k tiles
            // ---- prologue: cumulative decay, qh, kh in place, the (gq 2^b, gk 2^-b) tile ----
            wait(GREADY + (k & 3), (k >> 2) & 1);
            if (!retnet) wait(FULL_G, par);
            wait(FULL_QK, par);
            {
                const float *g = gate_s + (k & 3) * 2 * C;
                chunk_prologue<true, true>(qk, qk + TILE_BF16, retnet ? nullptr : reinterpret_cast<const float *>(sm + OFF_G), tot, g, g + C,
                                           eblast, sm + OFF_E2, p.status, tid, 1, NoHook(),
                                           ScalarDecay{lgam, min(C, p.T - t0)});
            }
            fence_proxy_async();
            mbar_arrive(bar(OPR));
            mbar_arrive(bar(GFREE + (k & 3)));

            // ---- dZ = diag(2^{b_last}) dS_{n+1}: fp32 back into TMEM (dS_n accumulates on it), bf16 operand copy ----
            if (k > 0) wait(DGFREE, (k - 1) & 1);       // the staged tiles of the previous chunk have left dZ and A|dA
            {
                float bl = 0.f;                         // b_last of key dimension `row` from the prologue's 8-row sums
#pragma unroll
                for (int g8 = 0; g8 < 8; ++g8) bl += tot[g8 * D + row];
                const float e = ex2f(bl * LOG2E);
                float v0[32], v1[32];
                const uint32_t ta = tmem + lane_base + COL_DS + 64 * wh;
                tmem_ld32(ta, v0);
                tmem_ld32(ta + 32, v1);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) { v0[j] *= e; v1[j] *= e; }
                tmem_st32(ta, v0);
                tmem_st32(ta + 32, v1);
                store_state_part(sm + OFF_DZ, row, wh, 0, v0);
                store_state_part(sm + OFF_DZ, row, wh, 1, v1);
                tmem_wait_st();
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(ZREADY));

            // ---- A, dA: TMEM -> causal mask -> bf16 -> shared memory (row i of an M=64 tile sits in lane 32*(i/16) + i%16) ----
            wait(BAR_A, par);
            tc_fence_after();
            {
                // rows 16q..16q+15 of this warp: a block of 8 columns c is empty for c >= 2q+2, full for c < 2q
                const int q4 = warp & 3, i = 16 * q4 + lane;
                const uint32_t col = wh ? COL_DA : COL_A;
                uint8_t *dst = sm + (wh ? OFF_DA : OFF_A);
                float v0[32], v1[32];
                tmem_ld32(tmem + lane_base + col, v0);
                tmem_ld32(tmem + lane_base + col + 32, v1);
                tmem_wait_ld();
                if (lane < 16) {
#define SLA_MASK_BLOCK(V, CL, CB)                                                                                          \
    {                                                                                                                      \
        uint4 w = make_uint4(0u, 0u, 0u, 0u);                                                                              \
        if ((CB) < 2 * q4 + 2) {                                                                                           \
            const int j0 = 8 * (CB);                                                                                       \
            const bool full = (CB) < 2 * q4;                                                                               \
            w.x = pack_bf16(full || j0 + 0 <= i ? V[8 * (CL) + 0] : 0.f, full || j0 + 1 <= i ? V[8 * (CL) + 1] : 0.f);     \
            w.y = pack_bf16(full || j0 + 2 <= i ? V[8 * (CL) + 2] : 0.f, full || j0 + 3 <= i ? V[8 * (CL) + 3] : 0.f);     \
            w.z = pack_bf16(full || j0 + 4 <= i ? V[8 * (CL) + 4] : 0.f, full || j0 + 5 <= i ? V[8 * (CL) + 5] : 0.f);     \
            w.w = pack_bf16(full || j0 + 6 <= i ? V[8 * (CL) + 6] : 0.f, full || j0 + 7 <= i ? V[8 * (CL) + 7] : 0.f);     \
        }                                                                                                                  \
        *reinterpret_cast<uint4 *>(dst + swz(i, (CB))) = w;                                                                \
    }
#pragma unroll
                    for (int c = 0; c < 4; ++c) SLA_MASK_BLOCK(v0, c, c)
#pragma unroll
                    for (int c = 0; c < 4; ++c) SLA_MASK_BLOCK(v1, c, 4 + c)
#undef SLA_MASK_BLOCK
                }
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(AREADY));

            // ---- R_{n-1} = rowsum(dS_n * S_n), while the tensor core works on the products with the masked tiles ----
            // (it feeds the log-decay gradient only: Softmax-RetNet, whose decay is a constant, has none and skips it)
            wait(BAR_DS, par);
            tc_fence_after();
            if (!retnet) {
                float v0[32], v1[32];
                tmem_ld32(tmem + lane_base + COL_DS + 64 * wh, v0);
                tmem_ld32(tmem + lane_base + COL_DS + 64 * wh + 32, v1);
                tmem_wait_ld();
                Rs[((n & 1) ^ 1) * 2 * D + wh * D + row] = rowdot_part(v0, 0) + rowdot_part(v1, 1);
            }
            mbar_arrive(bar(SNFREE));                   // S_n is no longer needed: the next image may land

            // ---- dqh^T, dkh^T: this thread owns key dimension `row` and tokens 32*wh .. 32*wh+31 ----
            wait(BAR_M1, par);
            tc_fence_after();
            const float *Rcur = Rs + (n & 1) * 2 * D;
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
                    __nv_bfloat16 *qp = reinterpret_cast<__nv_bfloat16 *>(qk + off);
                    __nv_bfloat16 *kp = reinterpret_cast<__nv_bfloat16 *>(qk + TILE_BF16 + off);
                    const float2 ee = unpack_bf16(*reinterpret_cast<const uint32_t *>(sm + OFF_E2 + i * (D * 4) + row * 4));
                    const float pq = __bfloat162float(*qp) * dqh[ii], pk = __bfloat162float(*kp) * dkh[ii];
                    run += pq - pk;
                    sfx[ii] = run;
                    *qp = __float2bfloat16_rn(ee.x * dqh[ii]);       // dq = scale Gq 2^b dqh   (over qh, for the store)
                    *kp = __float2bfloat16_rn(ee.y * dkh[ii]);       // dk = Gk 2^-b dkh
                    dqh[ii] = pq;
                    dkh[ii] = pk;
                }
                if (wh == 1) up[row] = run + Rcur[row] + Rcur[D + row];
                const float sq = warp_transpose_sum(dqh, lane);
                const float sk = warp_transpose_sum(dkh, lane);
                red[warp * 32 + lane] = sq;
                red[8 * 32 + warp * 32 + lane] = sk;
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(OUT1));

            // ---- dV^T -> dv tile; dlog_decay tile; gate products ----
            wait(BAR_M2, par);
            tc_fence_after();
            {
                float dvt[32];
                tmem_ld32(tmem + lane_base + COL_DV + 32 * wh, dvt);
                tmem_wait_ld();
                const uint32_t dhalf = (uint32_t)(row >> 6) * HALF_BF16, dchunk = (uint32_t)(row & 63) >> 3, dbyte = (row & 7) * 2;
#pragma unroll
                for (int ii = 0; ii < 32; ++ii)
                    *reinterpret_cast<__nv_bfloat16 *>(sm + OFF_A + dhalf + swz(32 * wh + ii, dchunk) + dbyte) =
                        __float2bfloat16_rn(dvt[ii]);
            }
            named_bar_sync(1, NCOMPUTE);                // up, red and the R partials are complete
            {   // log-decay gradient: in-chunk suffix sum + what flows in from the right of the chunk
                const float offs = wh == 1 ? Rcur[row] + Rcur[D + row] : up[row];
                float *dgt = reinterpret_cast<float *>(sm + OFF_DZ);
#pragma unroll
                for (int ii = 0; ii < 32; ++ii) dgt[(32 * wh + ii) * D + row] = sfx[ii] + offs;
            }
            if (tid < C) {   // Gq*dGq and Gk*dGk of token tid: sum over the four key-dimension quarters
                const int cn = min(C, p.T - t0);
                if (tid < cn) {
                    const int w0 = 4 * (tid >> 5), l = tid & 31;
                    float sq = 0.f, sk = 0.f;
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        sq += red[(w0 + w) * 32 + l];
                        sk += red[8 * 32 + (w0 + w) * 32 + l];
                    }
                    p.pq[(tokb + t0 + tid) * p.H + h] = sq;
                    p.pk[(tokb + t0 + tid) * p.H + h] = sk;
                }
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bar(OUT2));
        }

        if (p.dh0) {   // dS_0, fp32 (the last chunk's MMAs were waited for above)
            float *dst = state_row(p.dh0, sbh, row, wh, p.dk, p.dv);
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                float v[32];
                tmem_ld32(tmem + lane_base + COL_DS + 64 * wh + 32 * part, v);
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

// Segmented backward, between the passes.  A batch row's P segments are sequences b*P .. b*P+P-1 of the packed batch;
// summaries are indexed by (b*H + h)*P + p as the summary kernel leaves them, states by ((b*P + p)*H + h) as the
// packed kernels read them.  One thread per state element, a short loop over the segments.
// Start states: S_0 = h0 (or zero), S_{p+1} = diag(gam_p) S_p + fin_p.
__global__ void k_fold_segment_states(int H, int P, int dk, int dv, const float *__restrict__ h0, const float *__restrict__ fin,
                                      const float *__restrict__ gam, float *__restrict__ h0seg) {
    const int bh = blockIdx.x, b = bh / H, h = bh % H, row = blockIdx.y, col = threadIdx.x;
    float sv = h0 ? h0[((size_t)bh * dk + row) * dv + col] : 0.f;
    for (int p = 0; p < P; ++p) {
        h0seg[((((size_t)b * P + p) * H + h) * dk + row) * dv + col] = sv;
        const size_t c = (size_t)bh * P + p;
        sv = fmaf(gam[c * D + row], sv, fin[(c * D + row) * D + col]);
    }
}
// State gradients entering each segment from its right: R_{P-1} = dht (or zero), R_p = diag(gam_{p+1}) R_{p+1} + F_{p+1},
// F_p being what segment p alone sends out of its left edge (its dh0 when run with a zero dht).
__global__ void k_fold_segment_dstates(int H, int P, int dk, int dv, const float *__restrict__ dht, const float *__restrict__ gam,
                                       const float *__restrict__ dsfin, float *__restrict__ dhtseg) {
    const int bh = blockIdx.x, b = bh / H, h = bh % H, row = blockIdx.y, col = threadIdx.x;
    float r = dht ? dht[((size_t)bh * dk + row) * dv + col] : 0.f;
    for (int p = P - 1; p >= 0; --p) {
        const size_t i = ((((size_t)b * P + p) * H + h) * dk + row) * dv + col;
        dhtseg[i] = r;
        r = fmaf(gam[((size_t)bh * P + p) * D + row], r, dsfin[i]);
    }
}

}  // namespace

int gla_tc_bwd_configure() {
    if (cudaFuncSetAttribute(k_gla_states_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)st1::SMEM_BYTES) != cudaSuccess)
        return -1;
    if (cudaFuncSetAttribute(k_gla_bwd_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)st2::SMEM_BYTES) != cudaSuccess)
        return -1;
    return 0;
}

// Softmax backward over the heads from the gate products P = G dG (shared by the GLA and GDN tensor-core paths).
int gate_bwd_prod(const float *lq, const float *lk, const float *pq, const float *pk, float *dlq, float *dlk, long n_tok,
                  int H, cudaStream_t st) {
    int hp = 1;
    while (hp < H) hp <<= 1;
    switch (hp) {
        case 1: launch_gate_bwd_prod<1>(lq, lk, pq, pk, dlq, dlk, n_tok, H, st); break;
        case 2: launch_gate_bwd_prod<2>(lq, lk, pq, pk, dlq, dlk, n_tok, H, st); break;
        case 4: launch_gate_bwd_prod<4>(lq, lk, pq, pk, dlq, dlk, n_tok, H, st); break;
        case 8: launch_gate_bwd_prod<8>(lq, lk, pq, pk, dlq, dlk, n_tok, H, st); break;
        case 16: launch_gate_bwd_prod<16>(lq, lk, pq, pk, dlq, dlk, n_tok, H, st); break;
        default: launch_gate_bwd_prod<32>(lq, lk, pq, pk, dlq, dlk, n_tok, H, st); break;
    }
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

// state slots (one per chunk plus one per sequence) over all (sequence, head) pairs
static size_t state_slots(const Dims &d, const Varlen *vl) {
    return (vl && vl->n_seq) ? (size_t)vl->slots * d.H : (size_t)d.B * d.H * (d.NT + 1);
}

size_t gla_tc_backward_workspace_bytes(const Dims &d, const Varlen *vl) {
    const size_t bth = (size_t)d.B * d.T * d.H;
    return state_slots(d, vl) * STATE_BF16 + 2 * ((bth + 63) & ~(size_t)63) * sizeof(float);
}

int gla_tc_segment_summaries(const Dims &d, const FwdArgs &a, int P, int L, float *fin, float *gam, int *status,
                             cudaStream_t st, Tracer &tr) {
    CUtensorMap mk, mv, mg;
    const bool retnet = d.variant == SLA_RETNET;
    if (!make_tile_map(&mk, a.k, d.B, d.T, d.H, d.dk) || !make_tile_map(&mv, a.v, d.B, d.T, d.H, d.dv)) return -1;
    if (retnet) mg = mk;   // (never used: the decay is generated in the kernel)
    else if (!make_map(&mg, a.log_decay, d.B, d.T, d.H, d.dk, true, 128)) return -1;
    StatesParams sp{a.lq, a.lk, nullptr, nullptr, fin, gam, status, d.T, d.H, d.NT, P, L, retnet ? a.log_decay : nullptr,
                    nullptr, nullptr, d.dk, d.dv};
    k_gla_states_tc<<<d.B * d.H * P, st1::NTHREADS, st1::SMEM_BYTES, st>>>(mk, mv, mg, sp);
    tr.mark("gla_segment_states_tc");
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

uint8_t *gla_tc_state_images(float *ws) { return reinterpret_cast<uint8_t *>(ws); }

int gla_tc_backward(const Dims &d, const BwdArgs &a, bool have_states, int *status, cudaStream_t st, Tracer &tr) {
    CUtensorMap mq, mk, mv, mdo, mg, mdq, mdk, mdv, mdg;
    const bool retnet = d.variant == SLA_RETNET;      // constant decay: no log-decay tensor to read, no gradient for it
    if (!make_tile_map(&mq, a.q, d.B, d.T, d.H, d.dk) || !make_tile_map(&mk, a.k, d.B, d.T, d.H, d.dk) ||
        !make_tile_map(&mv, a.v, d.B, d.T, d.H, d.dv) || !make_tile_map(&mdo, a.dO, d.B, d.T, d.H, d.dv) ||
        !make_tile_map(&mdq, a.dq, d.B, d.T, d.H, d.dk) || !make_tile_map(&mdk, a.dk, d.B, d.T, d.H, d.dk) ||
        !make_tile_map(&mdv, a.dv, d.B, d.T, d.H, d.dv))
        return -1;
    if (retnet) { mg = mq; mdg = mdq; }               // (never used)
    else if (!make_map(&mg, a.log_decay, d.B, d.T, d.H, d.dk, true, 128) ||
             !make_map(&mdg, a.dlog_decay, d.B, d.T, d.H, d.dk, true, 128))
        return -1;
    // workspace: state images, then the two [B,T,H] gate products
    Varlen *vl = (a.vl && a.vl->n_seq) ? a.vl : nullptr;
    const size_t bth = (size_t)d.B * d.T * d.H;
    const size_t img_floats = state_slots(d, vl) * (STATE_BF16 / 4);
    uint8_t *simg = reinterpret_cast<uint8_t *>(a.ws);
    float *pq = a.ws + img_floats;
    float *pk = pq + ((bth + 63) & ~(size_t)63);
    const int ctas = vl ? vl->n_seq * d.H : d.B * d.H;
    const SeqInfo *dseqs = vl ? vl->d_seqs : nullptr;
    const __nv_bfloat16 *q = (const __nv_bfloat16 *)a.q, *k = (const __nv_bfloat16 *)a.k, *v = (const __nv_bfloat16 *)a.v,
                        *dO = (const __nv_bfloat16 *)a.dO;

    if (!have_states) {   // (otherwise the forward pass of the same inputs has left the images in this workspace)
        const CUtensorMap *vm = nullptr;
        if (vl) {
            const void *key[] = {a.k, a.v, a.log_decay};
            vm = varlen_maps(*vl, 1, key, 3, st, [&](const SeqInfo &si, CUtensorMap *m) {
                const size_t tok = (size_t)si.t0 * d.H;      // (q, k are d_k wide, v, o and their gradients d_v)
                if (!make_tile_map(m + 0, k + tok * d.dk, 1, si.T, d.H, d.dk) || !make_tile_map(m + 1, v + tok * d.dv, 1, si.T, d.H, d.dv)) return false;
                if (retnet) { m[2] = m[0]; return true; }
                return make_map(m + 2, a.log_decay + tok * d.dk, 1, si.T, d.H, d.dk, true, 128);
            });
            if (!vm) return -1;
        }
        StatesParams sp{a.lq, a.lk, a.h0, simg, nullptr, nullptr, status, d.T, d.H, d.NT, 1, d.NT, retnet ? a.log_decay : nullptr,
                        dseqs, vm, d.dk, d.dv};
        k_gla_states_tc<<<ctas, st1::NTHREADS, st1::SMEM_BYTES, st>>>(mk, mv, mg, sp);
        tr.mark("gla_states_tc");
    }
    const CUtensorMap *vm = nullptr;
    if (vl) {
        const void *key[] = {a.q, a.k, a.v, a.dO, a.log_decay, a.dq, a.dk, a.dv, a.dlog_decay};
        vm = varlen_maps(*vl, 2, key, 9, st, [&](const SeqInfo &si, CUtensorMap *m) {
            const size_t tok = (size_t)si.t0 * d.H;      // (q, k are d_k wide, v, o and their gradients d_v)
            if (!make_tile_map(m + 0, q + tok * d.dk, 1, si.T, d.H, d.dk) || !make_tile_map(m + 1, k + tok * d.dk, 1, si.T, d.H, d.dk) ||
                !make_tile_map(m + 2, v + tok * d.dv, 1, si.T, d.H, d.dv) || !make_tile_map(m + 3, dO + tok * d.dv, 1, si.T, d.H, d.dv) ||
                !make_tile_map(m + 5, (__nv_bfloat16 *)a.dq + tok * d.dk, 1, si.T, d.H, d.dk) ||
                !make_tile_map(m + 6, (__nv_bfloat16 *)a.dk + tok * d.dk, 1, si.T, d.H, d.dk) ||
                !make_tile_map(m + 7, (__nv_bfloat16 *)a.dv + tok * d.dv, 1, si.T, d.H, d.dv))
                return false;
            if (retnet) { m[4] = m[0]; m[8] = m[5]; return true; }
            return make_map(m + 4, a.log_decay + tok * d.dk, 1, si.T, d.H, d.dk, true, 128) &&
                   make_map(m + 8, a.dlog_decay + tok * d.dk, 1, si.T, d.H, d.dk, true, 128);
        });
        if (!vm) return -1;
    }
    BwdParams bp{a.lq, a.lk, a.dht, simg, pq, pk, a.dh0, status, d.T, d.H, d.NT, d.scale, retnet ? a.log_decay : nullptr, dseqs, vm, d.dk, d.dv};
    k_gla_bwd_tc<<<ctas, st2::NTHREADS, st2::SMEM_BYTES, st>>>(mq, mk, mv, mdo, mg, mdq, mdk, mdv, mdg, bp);
    tr.mark("gla_bwd_tc");
    if (gate_bwd_prod(a.lq, a.lk, pq, pk, a.dlq, a.dlk, (long)d.B * d.T, d.H, st) < 0) return -1;
    tr.mark("gate_bwd");
    return cudaGetLastError() == cudaSuccess ? (have_states ? 2 : 3) : -1;
}


void gla_tc_backward_segment_table(const Dims &d, int P, int L, Varlen &segs) {
    segs.seqs.clear();
    long slots = 0;
    for (int b = 0; b < d.B; ++b)
        for (int p = 0; p < P; ++p) {
            const int t0 = p * L * C, len = std::min(L * C, d.T - t0), nt = (len + C - 1) / C;
            segs.seqs.push_back({b * d.T + t0, len, nt, (int)slots, b * P + p});
            slots += nt + 1;
        }
    segs.slots = slots;
    segs.n_seq = d.B * P;
    segs.seg_P = P;
    segs.seg_L = L;
}

// floats: [images of the segments' slots | pq | pk] as gla_tc_backward lays them out, then fin, gam, h0seg, dhtseg, dsfin
static size_t segmented_base_floats(const Dims &d, const Varlen &segs) {
    const size_t bth = (size_t)d.B * d.T * d.H;
    return state_slots(d, &segs) * (STATE_BF16 / 4) + 2 * ((bth + 63) & ~(size_t)63);
}
size_t gla_tc_backward_segmented_workspace_bytes(const Dims &d, const Varlen &segs) {
    const size_t nseg = (size_t)d.B * d.H * segs.seg_P, st = (size_t)segs.n_seq * d.H * d.dk * d.dv;
    return (segmented_base_floats(d, segs) + nseg * (D * D + D) + 3 * st) * sizeof(float);
}

int gla_tc_backward_segmented(const Dims &d, const BwdArgs &a, Varlen &segs, int *status, cudaStream_t st, Tracer &tr) {
    const int P = segs.seg_P, L = segs.seg_L;
    const size_t nseg = (size_t)d.B * d.H * P, stf = (size_t)segs.n_seq * d.H * d.dk * d.dv;
    float *fin = a.ws + segmented_base_floats(d, segs), *gam = fin + nseg * D * D;
    float *h0seg = gam + nseg * D, *dhtseg = h0seg + stf, *dsfin = dhtseg + stf;
    // the state every segment starts from
    FwdArgs f{a.q, a.k, a.v, a.log_decay, a.beta, a.lq, a.lk, a.h0, nullptr, nullptr, a.ws, a.status, nullptr};
    if (gla_tc_segment_summaries(d, f, P, L, fin, gam, status, st, tr) < 0) return -1;
    const dim3 grid(d.B * d.H, d.dk);
    k_fold_segment_states<<<grid, d.dv, 0, st>>>(d.H, P, d.dk, d.dv, a.h0, fin, gam, h0seg);
    tr.mark("fold_segment_states");
    // first pass over the segments as a packed batch, no state gradient entering: what each sends out of its left edge
    BwdArgs a1 = a;
    a1.h0 = h0seg;
    a1.dht = nullptr;
    a1.dh0 = dsfin;
    a1.vl = &segs;
    const int n1 = gla_tc_backward(d, a1, false, status, st, tr);
    if (n1 < 0) return -1;
    k_fold_segment_dstates<<<grid, d.dv, 0, st>>>(d.H, P, d.dk, d.dv, a.dht, gam, dsfin, dhtseg);
    tr.mark("fold_segment_dstates");
    // second pass with the true state gradient entering every segment (the state images of the first pass are in place)
    BwdArgs a2 = a1;
    a2.dht = dhtseg;
    a2.dh0 = a.dh0 ? dsfin : nullptr;
    const int n2 = gla_tc_backward(d, a2, true, status, st, tr);
    if (n2 < 0) return -1;
    if (a.dh0) {    // dS_0 of a batch row = what its first segment sends out
        const size_t row = (size_t)d.H * d.dk * d.dv * sizeof(float);
        if (cudaMemcpy2DAsync(a.dh0, row, dsfin, row * P, row, d.B, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return -1;
    }
    return cudaGetLastError() == cudaSuccess ? 3 + n1 + n2 : -1;
}

}  // namespace sla
