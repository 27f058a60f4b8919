// sla_forward_noalloc: the chunkwise forward with its scratch in a fixed device array that is part of
// the library image, for callers that must not allocate device memory.
#include "sla_internal.h"

#include <mutex>

namespace {

constexpr size_t kScratchBytes = SLA_NOALLOC_SCRATCH_BYTES;

// Lives in every GPU context that loads the library, from load until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void *g_scratch_addr[kMaxDevices] = {};     // device address of the array, per device ordinal

// In host code `g_noalloc_scratch` is only a handle: the address a kernel can use has to be asked
// for, once per device, while that device is current.
sla_status scratch_for_current_device(int dev, void **out) {
    if (dev < 0 || dev >= kMaxDevices) return SLA_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return SLA_ERR_CUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return SLA_OK;
}

bool aligned16(const void *p) { return ((uintptr_t)p & 15u) == 0; }

}  // namespace

extern "C" sla_status sla_forward_noalloc(sla_plan *plan, const void *q, const void *k, const void *v,
                                          const float *log_decay, const float *beta,
                                          const float *gq_logits, const float *gk_logits, const float *h0,
                                          void *o, float *ht, void *cuda_stream) {
    if (!plan) return SLA_ERR_INVALID_ARG;
    const sla::Dims &d = plan->dims;
    plan->last_launches = 0;
    if (d.B == 0 || d.T == 0) return SLA_OK;
    if (!q || !k || !v || !log_decay || !gq_logits || !gk_logits || !o) return SLA_ERR_INVALID_ARG;
    if (d.variant == SLA_GDN && !beta) return SLA_ERR_INVALID_ARG;
    const void *ptrs[] = {q, k, v, log_decay, beta, gq_logits, gk_logits, h0, o, ht};
    for (const void *p : ptrs)
        if (!aligned16(p)) return SLA_ERR_INVALID_ARG;
    // The built-in scratch has a fixed size: larger problems must use sla_forward with a caller workspace.
    if (plan->ws.fwd_floats * sizeof(float) > kScratchBytes) return SLA_ERR_WORKSPACE;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return SLA_ERR_CUDA;
    if (dev != plan->device) return SLA_ERR_INVALID_ARG;
    void *scratch = nullptr;
    sla_status s = scratch_for_current_device(dev, &scratch);
    if (s != SLA_OK) return s;
    // Every region of the scratch the kernels read (gates, cumulative decays, chunk states, WY factors)
    // is written earlier in the same call, so nothing has to be cleared between calls.
    sla::FwdArgs a{q, k, v, log_decay, beta, gq_logits, gk_logits, h0, o, ht, (float *)scratch, plan->d_status};
    plan->tracer.start((cudaStream_t)cuda_stream);
    int n = sla::generic_forward(d, plan->ws, a, true, (cudaStream_t)cuda_stream, plan->tracer);
    if (n < 0) return SLA_ERR_CUDA;
    plan->last_launches = n;
    return SLA_OK;
}
