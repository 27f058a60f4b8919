// Output projection of Eq. 7, y = Concat_h(o_h) W^O, and its reverse, as dense bf16 contractions on the
// 5th-generation tensor cores (tcgen05.mma, fp32 accumulators in TMEM, operands staged by TMA).
//
// One persistent kernel, C[Mr, Nc] = sum_k A[Mr, k] B[k, Nc], serves the three products; they differ only in which
// index of each operand is contiguous in memory, which the shared-memory and instruction descriptors express:
//   y  [tok, Dm] = o  [tok, K ] W [K, Dm]      A K-major  (rows of o),        B N-major (rows of W)
//   do [tok, K ] = dy [tok, Dm] W^T            A K-major  (rows of dy),       B K-major (rows of W: Dm contiguous)
//   dW [K,  Dm ] = o^T dy                      A M-major  (rows of o: K contiguous),  B N-major (rows of dy)
// CTA tile 128 x 256, 64 contraction steps per stage (four MMAs of K = 16), four stages of 48 KiB, two 256-column
// accumulators in TMEM so that the epilogue of one tile runs under the MMAs of the next.  Roles: warp 0 TMA, warp 1
// MMA issue, warps 2..5 epilogue (TMEM -> registers -> swizzled staging blocks -> TMA stores for bf16 results; fp32 results
// go from registers to global memory, 128 contiguous bytes per thread and step).  Tiles are dealt round robin with the column tiles of a row panel next to each other, so that the CTAs
// running at a time share A panels and all of B in L2.  Tails: rows, columns and contraction steps past the edge
// read as zeros through the tensor maps, stores are predicated.  Every wait is bounded and abortable.
#include <algorithm>

#include "sla_gla_tc.cuh"

namespace sla {
namespace {

using namespace ptx;
using tc::desc_kmajor;
using tc::desc_mnmajor;
using tc::encode_fn;

namespace gm {
constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4;
constexpr uint32_t A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr uint32_t BLOCK64 = 64 * 128;                  // a [64 rows][128 B] swizzled block
constexpr uint32_t OFF_OUT = STAGES * STAGE_BYTES;       // bf16 output staging: [4 epilogue warps][2][32 rows][128 B], swizzled
constexpr uint32_t OUT_BYTES = 32 * 128;
constexpr uint32_t OFF_BAR = OFF_OUT + 4 * 2 * OUT_BYTES;
enum Bar { FULL = 0 /*[4]*/, EMPTY = 4 /*[4]*/, TFULL = 8 /*[2]*/, TEMPTY = 10 /*[2]*/, NBAR = 12 };
constexpr uint32_t OFF_TMEM = OFF_BAR + NBAR * 8;       // TMEM base address, then the abort flag
constexpr uint32_t SMEM_BYTES = OFF_TMEM + 16 + 1024;
constexpr uint32_t TMEM_COLS = 512;
constexpr int NTHREADS = 6 * 32;
static_assert(SMEM_BYTES <= 232448, "shared memory budget");
}  // namespace gm

struct GemmParams {
    void *c;            // [Mr, Nc] row-major, bf16 or fp32
    int Mr, Nc, Kc;     // output rows, output columns, contraction length
    int *status;
};

// A_MN / B_MN: the operand's M (N) index is the contiguous one in memory (else its contraction index).
template <bool A_MN, bool B_MN, typename TOUT>
__global__ void __launch_bounds__(gm::NTHREADS, 1)
k_dense_tc(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
           const __grid_constant__ CUtensorMap tm_c, GemmParams p) {
    using namespace gm;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *sm = smem_raw + (base - raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    auto bar = [&](int i) { return base + OFF_BAR + 8u * i; };
    volatile int *abort_flag = reinterpret_cast<volatile int *>(sm + OFF_TMEM + 8);
    bool failed = false;
    auto wait = [&](int i, uint32_t parity) {
        if (!failed && !mbar_wait_bounded(bar(i), parity, abort_flag)) { failed = true; *abort_flag = 1; }
    };
    if (tid == 0) {
        *abort_flag = 0;
        for (int i = 0; i < NBAR; ++i) mbar_init(bar(i), i >= TEMPTY ? 128 : 1);
        fence_mbar_init();
        tma_prefetch_desc(&tm_a);
        tma_prefetch_desc(&tm_b);
        if (sizeof(TOUT) == 2) tma_prefetch_desc(&tm_c);
    }
    if (warp == 0) tmem_alloc(base + OFF_TMEM, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(sm + OFF_TMEM);
    const int tiles_n = (p.Nc + BN - 1) / BN, tiles = ((p.Mr + BM - 1) / BM) * tiles_n;
    const int nkb = (p.Kc + BK - 1) / BK;

    if (warp == 0) {
        // ---------------- TMA (one lane) ----------------
        if (lane == 0) {
            uint32_t fill = 0;                              // stages filled so far
            for (int t = blockIdx.x; t < tiles && !failed; t += gridDim.x) {
                const int m0 = (t / tiles_n) * BM, n0 = (t % tiles_n) * BN;
                for (int kb = 0; kb < nkb && !failed; ++kb, ++fill) {
                    const uint32_t s = fill % STAGES;
                    if (fill >= STAGES) wait(EMPTY + s, ((fill / STAGES) - 1) & 1);
                    if (failed) break;
                    const uint32_t sa = base + s * STAGE_BYTES, sb = sa + A_BYTES, fb = bar(FULL + s);
                    mbar_expect_tx(fb, STAGE_BYTES);
                    if (A_MN) {                             // [64 contraction rows][64 m] blocks, map (m, contraction)
                        tma_load_2d(sa, &tm_a, m0, kb * BK, fb);
                        tma_load_2d(sa + BLOCK64, &tm_a, m0 + 64, kb * BK, fb);
                    } else {                                // [128 m rows][64 contraction], map (contraction, m)
                        tma_load_2d(sa, &tm_a, kb * BK, m0, fb);
                    }
                    if (B_MN) {
#pragma unroll
                        for (int j = 0; j < BN / 64; ++j) tma_load_2d(sb + j * BLOCK64, &tm_b, n0 + 64 * j, kb * BK, fb);
                    } else {
                        tma_load_2d(sb, &tm_b, kb * BK, n0, fb);
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issue (one lane) ----------------
        if (lane == 0) {
            constexpr uint32_t IDESC = idesc_bf16(BM, BN, A_MN ? 1 : 0, B_MN ? 1 : 0);
            uint32_t use = 0, it = 0;
            for (int t = blockIdx.x; t < tiles && !failed; t += gridDim.x, ++it) {
                const uint32_t acc = it & 1;
                if (it >= 2) wait(TEMPTY + acc, ((it >> 1) - 1) & 1);   // the epilogue has read this accumulator
                if (failed) break;
                tc_fence_after();
                for (int kb = 0; kb < nkb && !failed; ++kb, ++use) {
                    const uint32_t s = use % STAGES;
                    wait(FULL + s, (use / STAGES) & 1);
                    if (failed) break;
                    tc_fence_after();
                    const uint32_t sa = base + s * STAGE_BYTES, sb = sa + A_BYTES;
                    const uint64_t da = A_MN ? desc_mnmajor(sa, BLOCK64) : desc_kmajor(sa);
                    const uint64_t db = B_MN ? desc_mnmajor(sb, BLOCK64) : desc_kmajor(sb);
#pragma unroll
                    for (int kk = 0; kk < BK / 16; ++kk)    // k-step: 16 rows of 128 B (MN-major) or 32 B along the row (K-major)
                        tc_mma_bf16(tmem + acc * BN, da + (A_MN ? kk * 128 : kk * 2), db + (B_MN ? kk * 128 : kk * 2), IDESC,
                                    (kb | kk) != 0);
                    tc_commit(bar(EMPTY + s));              // the stage may be refilled once these MMAs have read it
                }
                tc_commit(bar(TFULL + acc));                // the tile's accumulator is complete
            }
        }
    } else {
        // ---------------- epilogue: TMEM lane = output row ----------------
        const uint32_t quad = warp & 3;                     // the TMEM lanes this warp may read: 32 quad .. 32 quad + 31
        const uint32_t lane_base = (32u * quad) << 16;
        uint32_t it = 0, nst = 0;                           // nst: staged blocks so far (bf16 output)
        for (int t = blockIdx.x; t < tiles; t += gridDim.x, ++it) {
            const uint32_t acc = it & 1;
            const int m0 = (t / tiles_n) * BM + 32 * quad, m = m0 + lane, n0 = (t % tiles_n) * BN;
            wait(TFULL + acc, (it >> 1) & 1);
            tc_fence_after();
            if (sizeof(TOUT) == 2) {
                // bf16: 64 columns of the warp's 32 rows at a time through a swizzled staging block and a TMA store
                // (which clips rows and columns past the edge); two blocks per warp, so a store runs under the next read-out
                for (int jj = 0; jj < BN / 64; ++jj, ++nst) {
                    float v0[32], v1[32];
                    tmem_ld32(tmem + lane_base + acc * BN + 64 * jj, v0);
                    tmem_ld32(tmem + lane_base + acc * BN + 64 * jj + 32, v1);
                    tmem_wait_ld();
                    const uint32_t blk = OFF_OUT + (quad * 2 + (nst & 1)) * OUT_BYTES;
                    if (lane == 0 && nst >= 2) bulk_wait_read1();   // the store that last used this block has read it
                    __syncwarp();
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint4 w;
                        w.x = pack_bf16(v0[8 * c + 0], v0[8 * c + 1]); w.y = pack_bf16(v0[8 * c + 2], v0[8 * c + 3]);
                        w.z = pack_bf16(v0[8 * c + 4], v0[8 * c + 5]); w.w = pack_bf16(v0[8 * c + 6], v0[8 * c + 7]);
                        *reinterpret_cast<uint4 *>(sm + blk + lane * 128 + ((c ^ (lane & 7)) << 4)) = w;
                        w.x = pack_bf16(v1[8 * c + 0], v1[8 * c + 1]); w.y = pack_bf16(v1[8 * c + 2], v1[8 * c + 3]);
                        w.z = pack_bf16(v1[8 * c + 4], v1[8 * c + 5]); w.w = pack_bf16(v1[8 * c + 6], v1[8 * c + 7]);
                        *reinterpret_cast<uint4 *>(sm + blk + lane * 128 + (((4 + c) ^ (lane & 7)) << 4)) = w;
                    }
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0 && !failed && m0 < p.Mr && n0 + 64 * jj < p.Nc) {
                        tma_store_2d(&tm_c, base + blk, n0 + 64 * jj, m0);
                        bulk_commit();
                    }
                }
            } else {
                float *crow = reinterpret_cast<float *>(p.c) + (size_t)m * p.Nc + n0;
#pragma unroll 2
                for (int j = 0; j < BN / 32; ++j) {
                    float v[32];
                    tmem_ld32(tmem + lane_base + acc * BN + 32 * j, v);
                    tmem_wait_ld();
                    if (failed || m >= p.Mr) continue;
#pragma unroll
                    for (int c = 0; c < 32; c += 8) {       // columns come in groups of 8 (Nc is a multiple of 8)
                        if (n0 + 32 * j + c >= p.Nc) break;
                        float4 *dst = reinterpret_cast<float4 *>(crow + 32 * j + c);
                        dst[0] = make_float4(v[c + 0], v[c + 1], v[c + 2], v[c + 3]);
                        dst[1] = make_float4(v[c + 4], v[c + 5], v[c + 6], v[c + 7]);
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(bar(TEMPTY + acc));
        }
        if (sizeof(TOUT) == 2 && lane == 0) bulk_wait0();   // the last stores have left shared memory and landed
    }
    if (failed) atomicOr(p.status, STATUS_TIMEOUT);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, TMEM_COLS);
}

// 2-D bf16 tensor map over a row-major [rows, cols] matrix: box = 64 columns (128 bytes, swizzled) x box_rows rows.
bool make_matrix_map(CUtensorMap *m, const void *ptr, int rows, int cols, int box_rows) {
    auto fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sm_count() {
    static int n = 0;
    if (!n) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) n = 148;
    }
    return n;
}

// C[Mr,Nc] = A B with A given as the row-major matrix a [a_rows, a_cols] (A_MN: a = A^T, i.e. [Kc, Mr]; else [Mr, Kc])
// and B as b (B_MN: b = B, [Kc, Nc]; else b = B^T, [Nc, Kc]).
template <bool A_MN, bool B_MN, typename TOUT>
int launch_dense(const void *a, const void *b, void *c, int Mr, int Nc, int Kc, int *status, cudaStream_t st) {
    CUtensorMap ma, mb, mc;
    if (sizeof(TOUT) == 2 ? !make_matrix_map(&mc, c, Mr, Nc, 32) : false) return -1;
    if (sizeof(TOUT) != 2) mc = CUtensorMap();
    if (!(A_MN ? make_matrix_map(&ma, a, Kc, Mr, 64) : make_matrix_map(&ma, a, Mr, Kc, gm::BM))) return -1;
    if (!(B_MN ? make_matrix_map(&mb, b, Kc, Nc, 64) : make_matrix_map(&mb, b, Nc, Kc, gm::BN))) return -1;
    const int tiles = ((Mr + gm::BM - 1) / gm::BM) * ((Nc + gm::BN - 1) / gm::BN);
    GemmParams gp{c, Mr, Nc, Kc, status};
    k_dense_tc<A_MN, B_MN, TOUT><<<std::min(tiles, sm_count()), gm::NTHREADS, gm::SMEM_BYTES, st>>>(ma, mb, mc, gp);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace

int out_proj_configure() {
    if (cudaFuncSetAttribute(k_dense_tc<false, true, __nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gm::SMEM_BYTES) != cudaSuccess ||
        cudaFuncSetAttribute(k_dense_tc<false, false, __nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gm::SMEM_BYTES) != cudaSuccess ||
        cudaFuncSetAttribute(k_dense_tc<true, true, float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gm::SMEM_BYTES) != cudaSuccess)
        return -1;
    return 0;
}

// y [n_tok, Dm] = o [n_tok, K] w [K, Dm]
int out_proj_forward(long n_tok, int K, int Dm, const void *o, const void *w, void *y, int *status, cudaStream_t st, Tracer &tr) {
    if (launch_dense<false, true, __nv_bfloat16>(o, w, y, (int)n_tok, Dm, K, status, st) < 0) return -1;
    tr.mark("out_proj_fwd_tc");
    return 1;
}

// do [n_tok, K] = dy [n_tok, Dm] w^T;  dw [K, Dm] (fp32) = o^T dy
int out_proj_backward(long n_tok, int K, int Dm, const void *o, const void *w, const void *dy, void *d_o, float *dw, int *status,
                      cudaStream_t st, Tracer &tr) {
    if (launch_dense<false, false, __nv_bfloat16>(dy, w, d_o, (int)n_tok, K, Dm, status, st) < 0) return -1;
    tr.mark("out_proj_dx_tc");
    if (launch_dense<true, true, float>(o, dy, dw, K, Dm, (int)n_tok, status, st) < 0) return -1;
    tr.mark("out_proj_dw_tc");
    return 2;
}

}  // namespace sla
