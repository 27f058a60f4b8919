// Constants and host helpers shared by the tensor-core (tcgen05 / TMEM / TMA) Softmax-GLA kernels:
// bf16 I/O, d_k = d_v = 128 (64-wide heads run padded), 64-token chunks.  Shared-memory tiles are rows of 128 bytes (64 bf16) in the
// 128-byte swizzle; a 128-wide tile is two such halves side by side.
#pragma once
#include <type_traits>
#include "sla_internal.h"
#include "sla_ptx.cuh"

#include <mutex>

namespace sla {
namespace tc {

constexpr int C = 64, D = 128;
constexpr uint32_t TILE_BF16 = C * D * 2;           // 16 KiB: two 64-column halves of [64 rows][128 B]
constexpr uint32_t HALF_BF16 = C * 128;             // 8 KiB
constexpr uint32_t TILE_G = C * D * 4;              // 32 KiB fp32 log-decay tile
constexpr uint32_t STATE_HALF = D * 128;            // 16 KiB: [128 rows][128 B], one 64-column half of a state
constexpr uint32_t STATE_BF16 = 2 * STATE_HALF;     // 32 KiB bf16 state as an MMA operand

// byte offset of 16-byte chunk `chunk` (0..7) of row `row` inside a 128-byte-swizzled tile
__device__ __forceinline__ uint32_t swz(uint32_t row, uint32_t chunk) { return row * 128 + ((chunk ^ (row & 7)) << 4); }

// Shared-memory matrix descriptors are built once per tile (k-step 0); a k-step only moves the start-address field,
// i.e. adds a small constant to the descriptor, so the issuing lane spends one add per operand per MMA.
// K-major operand whose 128-wide K extent is split in two halves `half_stride` bytes apart; k-step kk = 16 elements.
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t tile) { return ptx::smem_desc_sw128(tile, 16, 1024); }
__device__ __forceinline__ constexpr uint64_t kstep_kmajor(uint32_t kk, uint32_t half_stride) {
    return ((kk >> 2) * half_stride + (kk & 3) * 32) >> 4;
}
// MN-major operand ([K rows][MN contiguous]); 64-element MN blocks `mn_stride` bytes apart; k-step kk = 16 rows.
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t tile, uint32_t mn_stride) {
    return ptx::smem_desc_sw128(tile, mn_stride, 1024);
}
__device__ __forceinline__ constexpr uint64_t kstep_mnmajor(uint32_t kk) { return (kk * 2048) >> 4; }

typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                             const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeFn encode_fn() {
    static EncodeFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeFn)ptr;
    });
    return fn;
}

// Tensor map over a [B,T,H,d] tensor: box = 64 tokens x `box_d` features of one head (coordinates d, h, t, b).
// bf16 tiles land 128-byte swizzled, fp32 tiles unswizzled.  Rows past T read as zero.
inline bool make_map(CUtensorMap *m, const void *ptr, int B, int T, int H, int d, bool fp32, int box_d) {
    EncodeFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t es = fp32 ? 4 : 2;
    cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)H, (cuuint64_t)T, (cuuint64_t)B};
    cuuint64_t strides[3] = {(cuuint64_t)d * es, (cuuint64_t)H * d * es, (cuuint64_t)T * H * d * es};
    cuuint32_t box[4] = {(cuuint32_t)box_d, 1, (cuuint32_t)C, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(m, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4,
                    const_cast<void *>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    fp32 ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Tensor map over a bf16 [B,T,H,d] tensor (d = 128 or 64) that moves a whole 64-token x 128-feature tile of one head in
// ONE copy: the feature axis is split as (64 within a half, d/64 halves) and the halves are made the slowest box
// dimension, so the tile lands as two 128-byte-swizzled [64 rows][128 B] halves, 8 KiB apart - the layout the MMA
// descriptors expect.  With d = 64 the second half lies outside the tensor: it loads as zeros and is dropped by stores,
// so a 64-wide head runs through the 128-wide kernels as if padded with zero features, at no cost in memory traffic.
// Coordinates: (0, token, 0, head, batch).
inline bool make_tile_map(CUtensorMap *m, const void *ptr, int B, int T, int H, int d = D) {
    EncodeFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[5] = {64, (cuuint64_t)T, (cuuint64_t)(d / 64), (cuuint64_t)H, (cuuint64_t)B};
    cuuint64_t strides[4] = {(cuuint64_t)H * d * 2, 128, (cuuint64_t)d * 2, (cuuint64_t)T * H * d * 2};
    cuuint32_t box[5] = {64, (cuuint32_t)C, 2, 1, 1};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Row `row`, columns 64*half .. 64*half+63 of the fp32 [dk, dv] state of sequence-head bh inside a [.., dk, dv]
// tensor, as seen by the thread that owns that part of the kernels' 128 x 128 state; nullptr where a 64-wide head has
// no such part (the padded rows and columns stay zero) or the tensor is absent.
template <typename T>
__device__ __forceinline__ T *state_row(T *t, size_t bh, int row, int half, int dk, int dv) {
    return (t && row < dk && 64 * half < dv) ? t + (bh * dk + row) * dv + 64 * half : nullptr;
}

// Device array of the per-sequence tensor maps of region r of a packed batch: `make(seq, maps)` encodes one sequence's
// maps.  They are encoded and uploaded (stream-ordered, from a pinned mirror) only when `key`, the tensors they point
// at, differs from the last call's; a training loop that reuses its buffers encodes once.  nullptr on failure.
template <class Make>
inline const CUtensorMap *varlen_maps(Varlen &vl, int r, const void *const *key, int nkey, cudaStream_t st, Make make) {
    Varlen::Region &g = vl.reg[r];
    bool same = g.valid;
    for (int i = 0; i < nkey && same; ++i) same = g.key[i] == key[i];
    if (same) return g.dev;
    g.valid = false;
    if (cudaEventSynchronize(g.uploaded) != cudaSuccess) return nullptr;      // the mirror's last upload has been read
    for (int s = 0; s < vl.n_seq; ++s)
        if (!make(vl.seqs[s], g.host + (size_t)s * Varlen::MAPS_PER_SEQ)) return nullptr;
    const size_t bytes = (size_t)vl.n_seq * Varlen::MAPS_PER_SEQ * sizeof(CUtensorMap);
    if (cudaMemcpyAsync(g.dev, g.host, bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return nullptr;
    if (cudaEventRecord(g.uploaded, st) != cudaSuccess) return nullptr;
    for (int i = 0; i < nkey; ++i) g.key[i] = key[i];
    g.valid = true;
    return g.dev;
}

// Head-softmax gates (Eq. 4) of one token for head h: returns (Gq_h, Gk_h).
__device__ __forceinline__ float2 head_gates(const float *lq, const float *lk, int H, int h) {
    float m1 = -INFINITY, m2 = -INFINITY;
    for (int j = 0; j < H; ++j) { m1 = fmaxf(m1, lq[j]); m2 = fmaxf(m2, lk[j]); }
    float s1 = 0.f, s2 = 0.f;
    for (int j = 0; j < H; ++j) { s1 += expf(lq[j] - m1); s2 += expf(lk[j] - m2); }
    return make_float2(expf(lq[h] - m1) / s1, expf(lk[h] - m2) / s2);
}

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

constexpr uint32_t NCOMPUTE = 256;      // compute threads (warps 0..7); they meet on named barrier 1
constexpr float LOG2E = 1.4426950408889634f;

// Chunk prologue, run by 256 threads (tid 0..255, meeting on named barrier bar_id) on one landed stage (the decay of Eq. 12, or of
// Eq. 10 when gs is null, made chunk-local):
//   b_i = inclusive cumulative log-decay (kept in log2 units), two-level: per-8-row sums, then a running sum
//   qh_i = gq_i * q_i * 2^{b_i}   (gq_i = scale*Gq_i)      kh_i = gk_i * k_i * 2^{-b_i}
// written over q and k in place (the swizzled tiles are the MMA operands); eblast[d] = 2^{b_last,d}.
// With WITH_E also leaves the tile e2[i][d] = (bf16 gq_i 2^{b_i}, bf16 gk_i 2^{-b_i}), 4 bytes per element, rows of 512 B,
// unswizzled: the factors that turn dqh, dkh into dq, dk.  Thread (rg = warp, cj = lane) owns rows 8rg..8rg+7,
// columns 4cj..4cj+3.
// tot: [8][128] floats of scratch.  status: the plan's device status word (a chunk whose cumulative log-decay is
// beyond the representable range raises STATUS_RANGE there).
constexpr uint32_t TOT_BYTES = 8 * D * 4;
struct NoHook { __device__ __forceinline__ void operator()() const {} };
// Softmax-RetNet runs on the same kernels: with gs == nullptr the chunk's log-decay tile is not read but generated,
// log_gamma on each of the chunk's cn tokens (all key dimensions alike).
struct ScalarDecay { float log_gamma = 0.f; int cn = 0; };
template <bool WITH_Q, bool WITH_E, class Hook = NoHook>
__device__ __forceinline__ void chunk_prologue(uint8_t *q_tile, uint8_t *k_tile, const float *gs, float *tot,
                                               const float *gq_s, const float *gk_s, float *eblast,
                                               uint8_t *e2_tile, int *status, int tid, int bar_id = 1,
                                               Hook tile_read = Hook(), ScalarDecay sc = ScalarDecay()) {
    using namespace ptx;
    const int rg = tid >> 5, cj = tid & 31;
    float4 gl[8];                               // this thread's log-decay rows: read once, kept for the second pass
    {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int rr = 0; rr < 8; ++rr) {
            if (gs) {
                gl[rr] = *reinterpret_cast<const float4 *>(gs + (8 * rg + rr) * D + 4 * cj);
            } else {                            // Eq. 10: one constant log-decay per head, none past the sequence end
                const float v = 8 * rg + rr < sc.cn ? sc.log_gamma : 0.f;
                gl[rr] = make_float4(v, v, v, v);
            }
            acc.x += gl[rr].x; acc.y += gl[rr].y; acc.z += gl[rr].z; acc.w += gl[rr].w;
        }
        *reinterpret_cast<float4 *>(tot + rg * D + 4 * cj) = acc;
    }
    named_bar_sync(bar_id, NCOMPUTE);
    tile_read();                                // every thread has read its rows: the log-decay tile may be overwritten
    float bsum[4] = {0.f, 0.f, 0.f, 0.f};
    for (int g = 0; g < rg; ++g) {
        const float4 a = *reinterpret_cast<const float4 *>(tot + g * D + 4 * cj);
        bsum[0] += a.x; bsum[1] += a.y; bsum[2] += a.z; bsum[3] += a.w;
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) bsum[e] *= LOG2E;
    // columns 4cj..4cj+3 = 8 bytes of a bf16 row: half cj>>4, 16-byte chunk (cj&15)>>1, upper or lower 8 bytes
    const uint32_t half = cj >> 4, chunk = (cj & 15) >> 1, sub = (cj & 1) * 8;
#pragma unroll
    for (int rr = 0; rr < 8; ++rr) {
        const int r = 8 * rg + rr;
        const float4 g = gl[rr];
        bsum[0] = fmaf(g.x, LOG2E, bsum[0]); bsum[1] = fmaf(g.y, LOG2E, bsum[1]);
        bsum[2] = fmaf(g.z, LOG2E, bsum[2]); bsum[3] = fmaf(g.w, LOG2E, bsum[3]);
        const float gq = WITH_Q ? gq_s[r] : 0.f, gk = gk_s[r];
        const uint32_t off = half * HALF_BF16 + swz(r, chunk) + sub;
        uint2 qv, kv = *reinterpret_cast<uint2 *>(k_tile + off);
        uint4 e2v;
        if (WITH_Q) qv = *reinterpret_cast<uint2 *>(q_tile + off);
        uint32_t *qw = reinterpret_cast<uint32_t *>(&qv), *kw = reinterpret_cast<uint32_t *>(&kv);
        uint32_t *e2w = reinterpret_cast<uint32_t *>(&e2v);
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const float i0 = gk * ex2f(-bsum[2 * e]), i1 = gk * ex2f(-bsum[2 * e + 1]);
            const float2 kf = unpack_bf16(kw[e]);
            kw[e] = pack_bf16(kf.x * i0, kf.y * i1);
            if (WITH_Q) {
                const float e0 = gq * ex2f(bsum[2 * e]), e1 = gq * ex2f(bsum[2 * e + 1]);
                const float2 qf = unpack_bf16(qw[e]);
                qw[e] = pack_bf16(qf.x * e0, qf.y * e1);
                if (WITH_E) {
                    e2w[2 * e] = pack_bf16(e0, i0);
                    e2w[2 * e + 1] = pack_bf16(e1, i1);
                }
            }
        }
        *reinterpret_cast<uint2 *>(k_tile + off) = kv;
        if (WITH_Q) *reinterpret_cast<uint2 *>(q_tile + off) = qv;
        if (WITH_E) *reinterpret_cast<uint4 *>(e2_tile + r * (D * 4) + cj * 16) = e2v;
    }
    if (rg == 7) {
#pragma unroll
        for (int e = 0; e < 4; ++e) eblast[4 * cj + e] = ex2f(bsum[e]);
        // beyond this the factors 2^{b}, 2^{-b} leave the exponent range of their fp32 / bf16 carriers
        if (fminf(fminf(bsum[0], bsum[1]), fminf(bsum[2], bsum[3])) < -SLA_MAX_CHUNK_DECAY * LOG2E) atomicOr(status, STATUS_RANGE);
    }
}

// Head-softmax gate (Eq. 4) of ONE token for head h: the H <= HP logits are fetched before the first use (one memory
// round trip), then max, exp and sum run over registers.  Returns softmax(row[0..H))[h].
template <int HP>
__device__ __forceinline__ float token_gate(const float *__restrict__ row, int H, int h) {
    float x[HP];
#pragma unroll
    for (int j = 0; j < HP; ++j) x[j] = j < H ? row[j] : -INFINITY;
    float m = x[0];
#pragma unroll
    for (int j = 1; j < HP; ++j) m = fmaxf(m, x[j]);
    float sum = 0.f, eh = 0.f;
#pragma unroll
    for (int j = 0; j < HP; ++j) {
        const float e = __expf(x[j] - m);      // exp(-inf) = 0 for the padding lanes
        sum += e;
        eh = j == h ? e : eh;
    }
    return eh / sum;
}
__device__ __forceinline__ float token_gate_any(const float *row, int H, int h) {
    if (H <= 4) return token_gate<4>(row, H, h);
    if (H <= 8) return token_gate<8>(row, H, h);
    if (H <= 16) return token_gate<16>(row, H, h);
    return token_gate<32>(row, H, h);
}
// Gates of one chunk for head h, by the NTH threads (whole warps) that serve one of the two gates:
// dst[i] = mult * softmax(L[i*H .. i*H+H))[h] for token i < cn, 0 for cn <= i < 64.  L points at the chunk's first
// logit; consecutive tokens are consecutive rows of H floats, so for H = 4, 8, 16, 32 the block is read as whole
// float4s, fully coalesced, H/4 lanes per token, and max / sum travel over shuffles (one exponential per logit).
// Other H: one thread per token reads its own row.
// fetch: this thread's float4s of the chunk's logit block (LPT = H/4 lanes per token, NTH threads per gate)
template <int LPT, int NTH>
__device__ __forceinline__ void gate_fetch(const float *__restrict__ L, int cn, int t, float4 (&x)[LPT * 64 / NTH]) {
#pragma unroll
    for (int i = 0; i < LPT * 64 / NTH; ++i) {
        const int f = i * NTH + t;                     // float4 index inside the chunk's block; token f / LPT
        x[i] = f / LPT < cn ? __ldg(reinterpret_cast<const float4 *>(L) + f) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
}
// finish: softmax over the H/4 lanes of every token, dst[token] = mult * G[token][h].  Stage by stage over all of the
// thread's float4s, so that the shuffles and exponentials of different tokens overlap.
template <int LPT, int NTH>
__device__ __forceinline__ void gate_finish(float4 (&x)[LPT * 64 / NTH], int cn, int h, float mult, float *dst, int t) {
    constexpr int NF = LPT * 64 / NTH;
    float m[NF], sum[NF];
#pragma unroll
    for (int i = 0; i < NF; ++i) m[i] = fmaxf(fmaxf(x[i].x, x[i].y), fmaxf(x[i].z, x[i].w));
#pragma unroll
    for (int o = 1; o < LPT; o <<= 1) {
#pragma unroll
        for (int i = 0; i < NF; ++i) m[i] = fmaxf(m[i], __shfl_xor_sync(0xffffffffu, m[i], o));
    }
#pragma unroll
    for (int i = 0; i < NF; ++i) {
        x[i].x = __expf(x[i].x - m[i]); x[i].y = __expf(x[i].y - m[i]);
        x[i].z = __expf(x[i].z - m[i]); x[i].w = __expf(x[i].w - m[i]);
        sum[i] = (x[i].x + x[i].y) + (x[i].z + x[i].w);
    }
#pragma unroll
    for (int o = 1; o < LPT; o <<= 1) {
#pragma unroll
        for (int i = 0; i < NF; ++i) sum[i] += __shfl_xor_sync(0xffffffffu, sum[i], o);
    }
    if ((t % LPT) == (h >> 2)) {
        const int j = h & 3;
#pragma unroll
        for (int i = 0; i < NF; ++i) {
            const int token = (i * NTH + t) / LPT;
            const float eh = j == 0 ? x[i].x : j == 1 ? x[i].y : j == 2 ? x[i].z : x[i].w;
            dst[token] = token < cn ? mult * __fdividef(eh, sum[i]) : 0.f;
        }
    }
}
template <int LPT, int NTH>
__device__ __forceinline__ void chunk_gate_vec(const float *__restrict__ L, int cn, int h, float mult, float *dst, int t) {
    float4 x[LPT * 64 / NTH];
    gate_fetch<LPT, NTH>(L, cn, t, x);
    gate_finish<LPT, NTH>(x, cn, h, mult, dst, t);
}
// NTH = 64 (threads t = 0..63, two whole warps) or 32 (one warp) serve one gate of one chunk.
template <int NTH = 64>
__device__ __forceinline__ void chunk_gate(const float *L, int H, int cn, int h, float mult, float *dst, int t) {
    if (H == 16) chunk_gate_vec<4, NTH>(L, cn, h, mult, dst, t);
    else if (H == 8) chunk_gate_vec<2, NTH>(L, cn, h, mult, dst, t);
    else if (H == 4) chunk_gate_vec<1, NTH>(L, cn, h, mult, dst, t);
    else if (H == 32) chunk_gate_vec<8, NTH>(L, cn, h, mult, dst, t);
    else {
        for (int i = t; i < C; i += NTH) dst[i] = i < cn ? mult * token_gate_any(L + (size_t)i * H, H, h) : 0.f;
    }
}
constexpr int NGATE = 128;   // gate threads: g < 64 -> scale*Gq of token g, g >= 64 -> Gk of token g-64

}  // namespace tc
}  // namespace sla
