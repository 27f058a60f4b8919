// Recurrent decode (Eq. 5-6 with the instantiations of Eq. 10-16 at single tokens) as a streaming kernel.
//
// A decode step moves the whole fp32 state once in and once out and does two FLOP per byte: it is HBM-bound, so the
// kernel is built like a copy.  One work item is the [d_k x d_v] state of one (sequence, head), at most 64 KiB.  One
// persistent CTA per SM walks its items with a ring of three shared-memory stages and three roles:
//   TMA lane          tile loads up to three items ahead of the arithmetic; the updated state leaves through a TMA
//                     store from the same stage, and the stage takes the next load as soon as the store has read it
//   operand warp      per token: the H gate logits -> head-softmax gates (Eq. 4), decay factors exp(g), and the
//                     operand vectors scale*Gq*q, Gk*k (or k), v (or Gk*v) as fp32 in a double-buffered block, one
//                     token ahead; the raw operands arrive by asynchronous 4-byte copies requested three tokens ahead
//   arithmetic warps  the state in registers (warp w owns rows w, w+NW, ..; lane l columns 4l..4l+3): decay, the delta
//                     rule's k S (GDN), the rank-1 write, the read-out o = q S
// so loads, arithmetic and stores of neighbouring items overlap all the time.
// n_tok consecutive tokens of a sequence are applied while its state sits in registers (multi-token decode).
#include "sla_gla_tc.cuh"

namespace sla {
namespace {

using namespace ptx;

namespace dc {
constexpr int STAGES = 3;                // states in flight per CTA
constexpr int NW = 8;                    // arithmetic warps
constexpr int RPT = 128 / NW;            // state rows per arithmetic thread
constexpr int NCONS = NW * 32;
constexpr int W_TMA = NW, W_OPS = NW + 1;
constexpr int NTHREADS = NCONS + 64;
constexpr int DMAX = 128;
constexpr uint32_t TILE_BYTES = DMAX * DMAX * 4;        // 64 KiB
// operand block (floats): q'[128] k'[128] a[128] u[128] beta
constexpr int OP_Q = 0, OP_K = DMAX, OP_A = 2 * DMAX, OP_U = 3 * DMAX, OP_BETA = 4 * DMAX, OP_FLOATS = 4 * DMAX + 4;
// raw operand block (byte offsets): q, k (I/O dtype, up to 512 B each), log-decay vector (GLA), v, the two logit rows,
// then beta and the scalar log-decay (RETNET, GDN)
constexpr uint32_t RAW_Q = 0, RAW_K = 512, RAW_G = 1024, RAW_V = 1536, RAW_LQ = 2048, RAW_LK = 2176, RAW_BETA = 2304,
                   RAW_BYTES = 2320;
constexpr int AHEAD = 3;                 // raw operands are requested this many tokens before they are used
constexpr int RAWBLOCKS = AHEAD + 1;
constexpr uint32_t OFF_OP = STAGES * TILE_BYTES;                    // [2] operand blocks
constexpr uint32_t OFF_RAW = OFF_OP + 2 * OP_FLOATS * 4;            // [RAWBLOCKS] raw operand blocks
constexpr uint32_t OFF_RED = OFF_RAW + RAWBLOCKS * RAW_BYTES;       // [2][NW][32] float4 partial sums
constexpr uint32_t OFF_BAR = OFF_RED + 2 * NW * 32 * 16;            // STAGES "full" + STAGES "ready to store" barriers
constexpr uint32_t SMEM_BYTES = OFF_BAR + 2 * STAGES * 8 + 16 + 128;   // + abort flag, + slack to align the base to 128 B
static_assert(SMEM_BYTES <= 232448, "shared memory budget");
}  // namespace dc

// four consecutive outputs (16-byte aligned position)
template <typename T> __device__ __forceinline__ void st_io4(T *p, size_t i, float4 v);
template <> __device__ __forceinline__ void st_io4<float>(float *p, size_t i, float4 v) {
    *reinterpret_cast<float4 *>(p + i) = v;
}
template <> __device__ __forceinline__ void st_io4<__nv_bfloat16>(__nv_bfloat16 *p, size_t i, float4 v) {
    *reinterpret_cast<uint2 *>(p + i) = make_uint2(pack_bf16(v.x, v.y), pack_bf16(v.z, v.w));
}

// (states move by 2-D tiled TMA: coordinates are column, row of the [Bdec*H*d_k, d_v] view)
struct DecParams {
    const void *q, *k, *v;
    const float *log_decay, *beta, *lq, *lk;
    void *o;
    int *status;
    int variant, H, dk, dv, n_tok;
    int n_items;                                // Bdec * H
    float scale;
};

// ---- raw per-token operands: asynchronous 4-byte copies global -> shared by the operand warp, several tokens ahead ----
__device__ __forceinline__ void cp_async4(void *dst_smem, const void *src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_u32(dst_smem)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
template <typename TIO> __device__ __forceinline__ float io_at(const uint8_t *blk, int i) {
    if (sizeof(TIO) == 4) return reinterpret_cast<const float *>(blk)[i];
    return __bfloat162float(reinterpret_cast<const __nv_bfloat16 *>(blk)[i]);
}
// The operand warp's copies of the operands of token row `tok` = b*n_tok + t, head h into raw block `blk` (bytes in the
// I/O dtype for q, k, v; fp32 for decay, beta, logits).
template <typename TIO>
__device__ __forceinline__ void issue_raw(const DecParams &p, uint8_t *blk, size_t tok, int h, int lane) {
    const size_t th = tok * p.H + h;
    const int nq = p.dk * (int)sizeof(TIO) / 4, nv = p.dv * (int)sizeof(TIO) / 4;       // 4-byte words of a q / k row, a v row
    for (int i = lane; i < nq; i += 32) {
        cp_async4(blk + dc::RAW_Q + 4 * i, (const uint8_t *)p.q + (th * p.dk) * sizeof(TIO) + 4 * i);
        cp_async4(blk + dc::RAW_K + 4 * i, (const uint8_t *)p.k + (th * p.dk) * sizeof(TIO) + 4 * i);
    }
    for (int i = lane; i < nv; i += 32)
        cp_async4(blk + dc::RAW_V + 4 * i, (const uint8_t *)p.v + (th * p.dv) * sizeof(TIO) + 4 * i);
    if (p.variant == SLA_GLA)
        for (int i = lane; i < p.dk; i += 32) cp_async4(blk + dc::RAW_G + 4 * i, p.log_decay + th * p.dk + i);
    if (lane < p.H) {
        cp_async4(blk + dc::RAW_LQ + 4 * lane, p.lq + tok * p.H + lane);
        cp_async4(blk + dc::RAW_LK + 4 * lane, p.lk + tok * p.H + lane);
    }
    if (lane == 0) {
        if (p.variant == SLA_GDN) {
            cp_async4(blk + dc::RAW_BETA, p.beta + th);
            cp_async4(blk + dc::RAW_BETA + 4, p.log_decay + th);
        } else if (p.variant == SLA_RETNET) {
            cp_async4(blk + dc::RAW_BETA + 4, p.log_decay + h);
        }
    }
}
// Gates (Eq. 4) and the operand vectors the arithmetic warps use, from raw block `raw` into operand block `op`.
template <typename TIO>
__device__ __forceinline__ void cook_ops(const DecParams &p, const uint8_t *raw, float *op, int h, int lane) {
    const float *rf = reinterpret_cast<const float *>(raw);
    const float xq = lane < p.H ? rf[dc::RAW_LQ / 4 + lane] : -INFINITY, xk = lane < p.H ? rf[dc::RAW_LK / 4 + lane] : -INFINITY;
    float mq = xq, mk = xk;
#pragma unroll
    for (int o2 = 16; o2 > 0; o2 >>= 1) {
        mq = fmaxf(mq, __shfl_xor_sync(0xffffffffu, mq, o2));
        mk = fmaxf(mk, __shfl_xor_sync(0xffffffffu, mk, o2));
    }
    const float eq = expf(xq - mq), ek = expf(xk - mk);          // exp(-inf) = 0 on the padding lanes
    float sq = eq, sk = ek;
#pragma unroll
    for (int o2 = 16; o2 > 0; o2 >>= 1) {
        sq += __shfl_xor_sync(0xffffffffu, sq, o2);
        sk += __shfl_xor_sync(0xffffffffu, sk, o2);
    }
    const float Gq = __shfl_sync(0xffffffffu, eq, h) / sq, Gk = __shfl_sync(0xffffffffu, ek, h) / sk;
    const bool gdn = p.variant == SLA_GDN;
    const float fq = p.scale * Gq, fk = gdn ? 1.f : Gk, fv = gdn ? Gk : 1.f;
    const float a_scalar = p.variant == SLA_GLA ? 0.f : expf(rf[dc::RAW_BETA / 4 + 1]);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int i = lane + 32 * e;
        // (all 128 entries are written: the arithmetic warps read rows and columns past d_k, d_v as zeros)
        const bool rk = i < p.dk, rv = i < p.dv;
        op[dc::OP_Q + i] = rk ? fq * io_at<TIO>(raw + dc::RAW_Q, i) : 0.f;
        op[dc::OP_K + i] = rk ? fk * io_at<TIO>(raw + dc::RAW_K, i) : 0.f;
        op[dc::OP_A + i] = rk ? (p.variant == SLA_GLA ? expf(rf[dc::RAW_G / 4 + i]) : a_scalar) : 0.f;
        op[dc::OP_U + i] = rv ? fv * io_at<TIO>(raw + dc::RAW_V, i) : 0.f;
    }
    if (lane == 0) op[dc::OP_BETA] = gdn ? rf[dc::RAW_BETA / 4] : 0.f;
}

template <typename TIO>
__global__ void __launch_bounds__(dc::NTHREADS, 1)
k_decode_stream(const __grid_constant__ CUtensorMap tm_s, DecParams p) {
    using namespace dc;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 127u) & ~127u;
    uint8_t *sm = smem_raw + (base - raw);
    const int tid = threadIdx.x, w = tid >> 5, lane = tid & 31;
    float *ops = reinterpret_cast<float *>(sm + OFF_OP);
    float4 *red = reinterpret_cast<float4 *>(sm + OFF_RED);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(sm + OFF_BAR + 2 * STAGES * 8);
    auto bar = [&](int i) { return base + OFF_BAR + 8u * i; };       // FULL[s] = s, READY[s] = STAGES + s
    const uint32_t tile_bytes = (uint32_t)p.dk * p.dv * 4;

    // this CTA's items ((sequence, head) indices): blockIdx.x, + gridDim.x, ...
    const int first = blockIdx.x, stride = gridDim.x;
    const int nj = first < p.n_items ? (p.n_items - first + stride - 1) / stride : 0;
    const int nsteps = nj * p.n_tok;            // steps (item j, token t) in processing order: n = j * n_tok + t

    if (tid == 0) {
        *abort_flag = 0;
        for (int i = 0; i < STAGES; ++i) {
            mbar_init(bar(i), 1);
            mbar_init(bar(STAGES + i), NCONS);
        }
        fence_mbar_init();
        tma_prefetch_desc(&tm_s);
    }
    __syncthreads();

    if (w == W_TMA) {
        // ---------------- TMA lane: state loads ahead of the arithmetic, stores behind it ----------------
        if (lane == 0) {
            bool failed = false;
            auto issue_load = [&](int j) {          // state of item j -> stage j % STAGES
                const int s = j % STAGES;
                mbar_expect_tx(bar(s), tile_bytes);
                tma_load_2d(base + s * TILE_BYTES, &tm_s, 0, (first + j * stride) * p.dk, bar(s));
            };
            for (int j = 0; j < STAGES && j < nj; ++j) issue_load(j);
            for (int j = 0; j < nj; ++j) {
                const int s = j % STAGES;
                if (!mbar_wait_bounded(bar(STAGES + s), (uint32_t)(j / STAGES) & 1, abort_flag)) { failed = true; *abort_flag = 1; break; }
                tma_store_2d(&tm_s, base + s * TILE_BYTES, 0, (first + j * stride) * p.dk);     // the updated state goes back
                bulk_commit();
                if (j + STAGES < nj) {              // once the store has read the stage, the stage takes the next load
                    bulk_wait_read0();
                    issue_load(j + STAGES);
                }
            }
            bulk_wait0();
            if (failed) {   // give loads that are still in flight time to land before shared memory goes away
                atomicOr(p.status, STATUS_TIMEOUT);
                const uint64_t t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
            }
        }
        return;
    }
    if (w == W_OPS) {
        // ---------------- operand warp ----------------
        // Raw operands of step m are requested AHEAD steps before step m starts and land in raw block m % RAWBLOCKS;
        // the cooked block m % 2 is written during step m - 1 (all of the warp's earlier copies have landed by then).
        int ij = 0, it = 0, iraw = 0;               // item, token and raw block of the next step to request
        auto request = [&]() {                      // always commits a group, empty past the last step
            if (ij < nj) {
                const int bh = first + ij * stride;
                issue_raw<TIO>(p, sm + OFF_RAW + (uint32_t)iraw * RAW_BYTES, (size_t)(bh / p.H) * p.n_tok + it, bh % p.H, lane);
                if (++it == p.n_tok) { it = 0; ++ij; }
                if (++iraw == RAWBLOCKS) iraw = 0;
            }
            cp_async_commit();
        };
        int cj = 0, ct = 0, craw = 0;               // item, token and raw block of the next step to cook
        auto cook = [&](int m) {
            __syncwarp();
            cook_ops<TIO>(p, sm + OFF_RAW + (uint32_t)craw * RAW_BYTES, ops + (m & 1) * OP_FLOATS, (first + cj * stride) % p.H, lane);
            if (++ct == p.n_tok) { ct = 0; ++cj; }
            if (++craw == RAWBLOCKS) craw = 0;
        };
        for (int m = 0; m < AHEAD; ++m) request();             // steps 0 .. AHEAD-1
        if (nsteps > 0) {
            cp_async_wait<AHEAD - 1>();             // step 0 has landed
            cook(0);
        }
        for (int n = 0; n < nsteps; ++n) {
            named_bar_sync(1, NCONS + 32);          // step n starts; operand block (n + 1) % 2 was last read in step n - 1
            request();                              // step n + AHEAD (its raw block was cooked from a step ago)
            if (n + 1 < nsteps) {
                cp_async_wait<AHEAD - 1>();         // step n + 1 has landed
                cook(n + 1);
            }
        }
        cp_async_wait<0>();
        return;
    }

    // ---------------- arithmetic warps ----------------
    bool failed = false;
    const bool gdn = p.variant == SLA_GDN;
    const bool col_ok = 4 * lane < p.dv;
    const int ld4 = p.dv >> 2;                      // float4s per state row
    int n = 0;
    for (int j = 0; j < nj; ++j) {
        const int bh = first + j * stride, b = bh / p.H, h = bh % p.H, s = j % STAGES;
        float4 *tile = reinterpret_cast<float4 *>(sm + s * TILE_BYTES);
        if (!failed && !mbar_wait_bounded(bar(s), (uint32_t)(j / STAGES) & 1, abort_flag)) { failed = true; *abort_flag = 1; }
        float4 S[RPT];
#pragma unroll
        for (int i = 0; i < RPT; ++i) {
            const int r = w + NW * i;
            S[i] = (r < p.dk && col_ok) ? tile[r * ld4 + lane] : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        for (int t = 0; t < p.n_tok; ++t, ++n) {
            named_bar_sync(1, NCONS + 32);          // the operand block of this step is complete
            const float *op = ops + (n & 1) * OP_FLOATS;
            float4 u = col_ok ? *reinterpret_cast<const float4 *>(op + OP_U + 4 * lane) : make_float4(0.f, 0.f, 0.f, 0.f);
            float kr[RPT];
#pragma unroll
            for (int i = 0; i < RPT; ++i) {         // Sbar = diag(a) S
                const int r = w + NW * i;
                const float a = op[OP_A + r];
                kr[i] = op[OP_K + r];
                S[i].x *= a; S[i].y *= a; S[i].z *= a; S[i].w *= a;
            }
            if (gdn) {                              // u = beta (Gk v - k Sbar)
                float4 part = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int i = 0; i < RPT; ++i) {
                    part.x = fmaf(kr[i], S[i].x, part.x); part.y = fmaf(kr[i], S[i].y, part.y);
                    part.z = fmaf(kr[i], S[i].z, part.z); part.w = fmaf(kr[i], S[i].w, part.w);
                }
                red[w * 32 + lane] = part;
                named_bar_sync(2, NCONS);
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int ww = 0; ww < NW; ++ww) {
                    const float4 x = red[ww * 32 + lane];
                    acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
                }
                const float beta = op[OP_BETA];
                u.x = beta * (u.x - acc.x); u.y = beta * (u.y - acc.y); u.z = beta * (u.z - acc.z); u.w = beta * (u.w - acc.w);
            }
            float4 part = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int i = 0; i < RPT; ++i) {         // write: S = Sbar + k^T u ; read: o = q S
                const int r = w + NW * i;
                const float qr = op[OP_Q + r];
                S[i].x = fmaf(kr[i], u.x, S[i].x); S[i].y = fmaf(kr[i], u.y, S[i].y);
                S[i].z = fmaf(kr[i], u.z, S[i].z); S[i].w = fmaf(kr[i], u.w, S[i].w);
                part.x = fmaf(qr, S[i].x, part.x); part.y = fmaf(qr, S[i].y, part.y);
                part.z = fmaf(qr, S[i].z, part.z); part.w = fmaf(qr, S[i].w, part.w);
            }
            red[NW * 32 + w * 32 + lane] = part;
            if (t == p.n_tok - 1) {                 // after the last token the state goes back: registers -> stage
#pragma unroll
                for (int i = 0; i < RPT; ++i) {
                    const int r = w + NW * i;
                    if (r < p.dk && col_ok) tile[r * ld4 + lane] = S[i];
                }
                fence_proxy_async();
                mbar_arrive(bar(STAGES + s));       // (the TMA lane stores it and reloads the stage)
            }
            named_bar_sync(2, NCONS);
            if (w == 0 && col_ok) {
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int ww = 0; ww < NW; ++ww) {
                    const float4 x = red[NW * 32 + ww * 32 + lane];
                    acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
                }
                st_io4((TIO *)p.o, (((size_t)b * p.n_tok + t) * p.H + h) * p.dv + 4 * lane, acc);
            }
        }
    }
}

bool make_state_map(CUtensorMap *m, float *state, long rows, int dv, int dk) {
    tc::EncodeFn fn = tc::encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)dv, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)dv * 4};
    cuuint32_t box[2] = {(cuuint32_t)dv, (cuuint32_t)dk};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, state, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int decode_sm_count() {
    static int n = 0;
    if (!n) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
    }
    return n;
}

}  // namespace

int decode_configure() {
    if (!tc::encode_fn()) return -1;
    if (cudaFuncSetAttribute(k_decode_stream<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dc::SMEM_BYTES) != cudaSuccess)
        return -1;
    if (cudaFuncSetAttribute(k_decode_stream<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dc::SMEM_BYTES) != cudaSuccess)
        return -1;
    return 0;
}

int decode_step(const Dims &d, const DecArgs &a, int *status, cudaStream_t st, Tracer &tr) {
    CUtensorMap ms;
    const long rows = (long)a.Bdec * d.H * d.dk;
    if (!make_state_map(&ms, a.state, rows, d.dv, d.dk)) return -1;
    DecParams p{a.q, a.k, a.v, a.log_decay, a.beta, a.lq, a.lk, a.o, status, d.variant, d.H, d.dk, d.dv, a.n_tok,
                a.Bdec * d.H, d.scale};
    const long want = decode_sm_count();                 // one persistent CTA per SM
    const unsigned grid = (unsigned)(p.n_items < want ? p.n_items : want);
    if (d.io_bf16)
        k_decode_stream<__nv_bfloat16><<<grid, dc::NTHREADS, dc::SMEM_BYTES, st>>>(ms, p);
    else
        k_decode_stream<float><<<grid, dc::NTHREADS, dc::SMEM_BYTES, st>>>(ms, p);
    tr.mark("decode");
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace sla
