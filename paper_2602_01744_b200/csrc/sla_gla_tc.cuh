// Constants and host helpers shared by the tensor-core (tcgen05 / TMEM / TMA) Softmax-GLA kernels:
// bf16 I/O, d_k = d_v = 128, 64-token chunks.  Shared-memory tiles are rows of 128 bytes (64 bf16) in the
// 128-byte swizzle; a 128-wide tile is two such halves side by side.
#pragma once
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

// K-major operand whose 128-wide K extent is split in two halves `half_stride` bytes apart; k-step kk = 16 elements
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t tile, uint32_t kk, uint32_t half_stride) {
    return ptx::smem_desc_sw128(tile + (kk >> 2) * half_stride + (kk & 3) * 32, 16, 1024);
}
// MN-major operand ([K rows][MN contiguous]); 64-element MN blocks `mn_stride` bytes apart; k-step kk = 16 rows
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t tile, uint32_t kk, uint32_t mn_stride) {
    return ptx::smem_desc_sw128(tile + kk * 2048, mn_stride, 1024);
}

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

// Head-softmax gates (Eq. 4) of one token for head h: returns (Gq_h, Gk_h).
__device__ __forceinline__ float2 head_gates(const float *lq, const float *lk, int H, int h) {
    float m1 = -INFINITY, m2 = -INFINITY;
    for (int j = 0; j < H; ++j) { m1 = fmaxf(m1, lq[j]); m2 = fmaxf(m2, lk[j]); }
    float s1 = 0.f, s2 = 0.f;
    for (int j = 0; j < H; ++j) { s1 += expf(lq[j] - m1); s2 += expf(lk[j] - m2); }
    return make_float2(expf(lq[h] - m1) / s1, expf(lk[h] - m2) / s2);
}

}  // namespace tc
}  // namespace sla
