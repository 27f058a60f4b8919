// Host side of the C ABI: plan validation, workspace carve-up, launch order.
#include "sla_internal.h"
#include "sla_ptx.cuh"

#include <algorithm>
#include <new>
#include <string.h>
#include <utility>
#include <vector>

namespace sla {

static size_t align64(size_t x) { return (x + 63) & ~(size_t)63; }

Workspace plan_workspace(const Dims &d) {
    Workspace w{};
    size_t bth = (size_t)d.B * d.T * d.H;
    size_t off = 0;
    auto take = [&](size_t n) { size_t o = off; off = align64(off + n); return o; };
    w.Gq = take(bth);
    w.Gk = take(bth);
    w.bcum = take(d.variant == SLA_GLA ? bth * d.dk : bth);
    w.states = take((size_t)d.B * d.H * (d.NT + 1) * d.dk * d.dv);
    if (d.variant == SLA_GDN) {
        w.W = take(bth * d.dk);
        w.U0 = take(bth * d.dv);
        w.U = take(bth * d.dv);
    }
    w.fwd_floats = off;
    w.dstates = take((size_t)d.B * d.H * d.NT * d.dk * d.dv);
    if (d.variant == SLA_GDN) {
        w.dU = take(bth * d.dv);
        w.dKbg = take(bth * d.dk);
        w.dVb = take(bth * d.dv);
        w.dbpart = take(bth);
    }
    w.dGq = take(bth);
    w.dGk = take(bth);
    w.bwd_floats = off;
    return w;
}

}  // namespace sla

static bool aligned16(const void *p) { return ((uintptr_t)p & 15u) == 0; }

// One warp waits on an mbarrier that nobody ever arrives at, with the same bounded wait the tensor-core kernels use
// but a limit of `limit_ns`; when the wait gives up it raises the plan's status word, exactly as those kernels do.
__global__ void k_selftest_bounded_wait(int *status, unsigned long long limit_ns) {
    __shared__ __align__(8) unsigned long long mbar;
    const uint32_t bar = sla::ptx::smem_u32(&mbar);
    if (threadIdx.x == 0) {
        sla::ptx::mbar_init(bar, 1);
        sla::ptx::fence_mbar_init();
    }
    __syncthreads();
    if (!sla::ptx::mbar_wait_bounded(bar, 0, nullptr, limit_ns) && threadIdx.x == 0) atomicOr(status, sla::STATUS_TIMEOUT);
}

// Can sla_forward of this plan leave what sla_backward needs (SLA_FLAG_SAVE_FOR_BACKWARD)?  Only the tensor-core
// paths do, and Softmax-GLA only where the forward runs each sequence in one piece.
static bool forward_can_save(const sla_plan &p) {
    if (p.flags & SLA_FLAG_FORCE_GENERIC) return false;
    if (sla::gla_tc_supported(p.dims)) return sla::gla_tc_forward_can_save(p.dims, &p.varlen);
    return sla::gdn_tc_supported(p.dims);
}

// What the kernels this plan selects need as workspace (regular batch, or the packed batch of sla_plan_set_sequences).
static void plan_workspace_sizes(sla_plan *p) {
    const sla::Dims &d = p->dims;
    const bool generic = p->flags & SLA_FLAG_FORCE_GENERIC;
    p->fwd_bytes = p->ws.fwd_floats * sizeof(float);
    p->bwd_bytes = p->ws.bwd_floats * sizeof(float);
    if (sla::gla_tc_supported(d) && !generic) {
        p->fwd_bytes = sla::gla_tc_forward_workspace_bytes(d, &p->varlen);
        p->bwd_bytes = (!p->varlen.n_seq && p->segs.n_seq) ? sla::gla_tc_backward_segmented_workspace_bytes(d, p->segs)
                                                           : sla::gla_tc_backward_workspace_bytes(d, &p->varlen);
    }
    if (sla::gdn_tc_supported(d) && !generic) {
        p->fwd_bytes = 0;
        p->bwd_bytes = sla::gdn_tc_backward_workspace_bytes(d, &p->varlen);
    }
    if ((p->flags & SLA_FLAG_SAVE_FOR_BACKWARD) && forward_can_save(*p) && p->bwd_bytes > p->fwd_bytes)
        p->fwd_bytes = p->bwd_bytes;     // the forward writes into the backward pass's workspace layout
}

static void varlen_release(sla::Varlen &v) {
    if (v.d_seqs) cudaFree(v.d_seqs);
    for (auto &g : v.reg) {
        if (g.dev) cudaFree(g.dev);
        if (g.host) cudaFreeHost(g.host);
        if (g.uploaded) cudaEventDestroy(g.uploaded);
        g = sla::Varlen::Region();
    }
    v = sla::Varlen();
}

// Device side of a filled sequence table: the table itself and, per kernel kind, room for the sequences' tensor maps.
static bool varlen_to_device(sla::Varlen &v) {
    const int n_seq = v.n_seq;
    bool ok = cudaMalloc((void **)&v.d_seqs, sizeof(sla::SeqInfo) * n_seq) == cudaSuccess &&
              cudaMemcpy(v.d_seqs, v.seqs.data(), sizeof(sla::SeqInfo) * n_seq, cudaMemcpyHostToDevice) == cudaSuccess;
    const size_t mb = (size_t)n_seq * sla::Varlen::MAPS_PER_SEQ * sizeof(CUtensorMap);
    for (auto &g : v.reg)
        ok = ok && cudaMalloc((void **)&g.dev, mb) == cudaSuccess && cudaMallocHost((void **)&g.host, mb) == cudaSuccess &&
             cudaEventCreateWithFlags(&g.uploaded, cudaEventDisableTiming) == cudaSuccess;
    return ok;
}

extern "C" {

const char *sla_status_string(sla_status s) {
    switch (s) {
        case SLA_OK: return "ok";
        case SLA_ERR_INVALID_ARG: return "invalid argument";
        case SLA_ERR_UNSUPPORTED: return "unsupported shape or option";
        case SLA_ERR_WORKSPACE: return "workspace missing or too small";
        case SLA_ERR_ARCH: return "device is not sm_100";
        case SLA_ERR_CUDA: return "CUDA runtime error";
        case SLA_ERR_TIMEOUT: return "device-side wait timed out";
        case SLA_ERR_RANGE: return "cumulative log-decay of a chunk beyond the representable range";
    }
    return "unknown status";
}

sla_status sla_plan_create(sla_plan **out, const sla_desc *desc) {
    if (!out) return SLA_ERR_INVALID_ARG;
    *out = nullptr;
    if (!desc || desc->struct_size != sizeof(sla_desc)) return SLA_ERR_INVALID_ARG;
    if (desc->variant < SLA_RETNET || desc->variant > SLA_GDN) return SLA_ERR_INVALID_ARG;
    if (desc->io_dtype != SLA_FP32 && desc->io_dtype != SLA_BF16) return SLA_ERR_INVALID_ARG;
    if (desc->B < 0 || desc->T < 0 || desc->H < 1) return SLA_ERR_INVALID_ARG;
    if (desc->H > 32) return SLA_ERR_UNSUPPORTED;
    if (desc->d_k < 16 || desc->d_k > 128 || desc->d_k % 16) return SLA_ERR_UNSUPPORTED;
    if (desc->d_v < 16 || desc->d_v > 128 || desc->d_v % 16) return SLA_ERR_UNSUPPORTED;
    if (desc->chunk != 16 && desc->chunk != 32 && desc->chunk != 64) return SLA_ERR_UNSUPPORTED;
    if ((uint64_t)desc->B * desc->H > 65535u) return SLA_ERR_UNSUPPORTED;   // grid.y limit
    if (!(desc->scale == desc->scale)) return SLA_ERR_INVALID_ARG;

    int dev = 0;
    cudaDeviceProp prop;
    if (cudaGetDevice(&dev) != cudaSuccess) return SLA_ERR_CUDA;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return SLA_ERR_CUDA;
    if (prop.major != 10) return SLA_ERR_ARCH;
    if (sla::generic_configure() != 0 || sla::gdn_configure() != 0 || sla::gla_tc_configure() != 0 ||
        sla::gla_tc_bwd_configure() != 0 || sla::gdn_tc_configure() != 0 ||
        sla::gdn_tc_bwd_configure() != 0 || sla::decode_configure() != 0 || sla::out_proj_configure() != 0)
        return SLA_ERR_CUDA;

    sla_plan *p = new (std::nothrow) sla_plan();
    if (!p) return SLA_ERR_CUDA;
    sla::Dims &d = p->dims;
    d.variant = desc->variant;
    d.io_bf16 = desc->io_dtype == SLA_BF16;
    d.B = desc->B; d.T = desc->T; d.H = desc->H;
    d.dk = desc->d_k; d.dv = desc->d_v; d.C = desc->chunk;
    d.NT = (desc->T + desc->chunk - 1) / desc->chunk;
    d.scale = desc->scale;
    p->ws = sla::plan_workspace(d);
    p->flags = desc->flags;
    // few long sequences on the tensor-core GLA / RetNet kernels: the table of segments the backward runs in
    if (sla::gla_tc_supported(d) && !(p->flags & SLA_FLAG_FORCE_GENERIC) && d.B > 0 && d.T > 0) {
        int P, L;
        sla::gla_tc_backward_choose_segments(d, P, L);
        if (P > 1) {
            sla::gla_tc_backward_segment_table(d, P, L, p->segs);
            if (!varlen_to_device(p->segs)) {
                varlen_release(p->segs);
                delete p;
                return SLA_ERR_CUDA;
            }
        }
    }
    plan_workspace_sizes(p);
    p->device = dev;
    p->last_launches = 0;
    p->d_status = nullptr;
    if (cudaMalloc((void **)&p->d_status, sizeof(int)) != cudaSuccess ||
        cudaMemset(p->d_status, 0, sizeof(int)) != cudaSuccess) {
        if (p->d_status) cudaFree(p->d_status);
        delete p;
        return SLA_ERR_CUDA;
    }
    *out = p;
    return SLA_OK;
}

sla_status sla_plan_destroy(sla_plan *plan) {
    if (!plan) return SLA_OK;
    if (plan->d_status) cudaFree(plan->d_status);
    varlen_release(plan->varlen);
    varlen_release(plan->segs);
    plan->tracer.destroy();
    delete plan;
    return SLA_OK;
}

sla_status sla_plan_set_sequences(sla_plan *plan, const int32_t *cu_seqlens, int32_t n_seq) {
    if (!plan || n_seq < 0 || (n_seq > 0 && !cu_seqlens)) return SLA_ERR_INVALID_ARG;
    const sla::Dims &d = plan->dims;
    plan->saved.valid = false;
    varlen_release(plan->varlen);
    if (n_seq == 0) {
        plan_workspace_sizes(plan);
        return SLA_OK;
    }
    // the tensor-core kernels only (they address a sequence through tensor maps of its own)
    if ((plan->flags & SLA_FLAG_FORCE_GENERIC) || !(sla::gla_tc_supported(d) || sla::gdn_tc_supported(d))) return SLA_ERR_UNSUPPORTED;
    if (d.B != 1 || cu_seqlens[0] != 0 || cu_seqlens[n_seq] != d.T) return SLA_ERR_INVALID_ARG;
    if ((uint64_t)n_seq * d.H > 0x7fffffffu) return SLA_ERR_UNSUPPORTED;
    sla::Varlen &v = plan->varlen;
    long slots = 0;
    for (int s = 0; s < n_seq; ++s) {
        const int len = cu_seqlens[s + 1] - cu_seqlens[s];
        if (len <= 0) { v.seqs.clear(); return SLA_ERR_INVALID_ARG; }      // (empty sequences are not allowed)
        const int nt = (len + d.C - 1) / d.C;
        v.seqs.push_back({cu_seqlens[s], len, nt, 0, s});
    }
    std::stable_sort(v.seqs.begin(), v.seqs.end(), [](const sla::SeqInfo &a, const sla::SeqInfo &b) { return a.NT > b.NT; });
    for (auto &si : v.seqs) {
        si.slot0 = (int)slots;
        slots += si.NT + 1;
    }
    v.slots = slots;
    v.n_seq = n_seq;
    if (!varlen_to_device(v)) {
        varlen_release(v);
        plan_workspace_sizes(plan);
        return SLA_ERR_CUDA;
    }
    plan_workspace_sizes(plan);
    return SLA_OK;
}

sla_status sla_plan_workspace_bytes(const sla_plan *plan, size_t *fwd, size_t *bwd) {
    if (!plan) return SLA_ERR_INVALID_ARG;
    if (fwd) *fwd = plan->fwd_bytes;
    if (bwd) *bwd = plan->bwd_bytes;
    return SLA_OK;
}

sla_status sla_plan_poll(sla_plan *plan) {
    if (!plan) return SLA_ERR_INVALID_ARG;
    int v = 0;
    if (cudaMemcpy(&v, plan->d_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return SLA_ERR_CUDA;
    if (v != 0) {
        cudaMemset(plan->d_status, 0, sizeof(int));
        return (v & sla::STATUS_TIMEOUT) ? SLA_ERR_TIMEOUT : SLA_ERR_RANGE;
    }
    return SLA_OK;
}

int32_t sla_plan_last_launch_count(const sla_plan *plan) { return plan ? plan->last_launches : 0; }

sla_status sla_plan_selftest_timeout(sla_plan *plan, void *cuda_stream) {
    if (!plan) return SLA_ERR_INVALID_ARG;
    k_selftest_bounded_wait<<<1, 32, 0, (cudaStream_t)cuda_stream>>>(plan->d_status, 2000000ull);   // 2 ms
    return cudaGetLastError() == cudaSuccess ? SLA_OK : SLA_ERR_CUDA;
}

sla_status sla_plan_set_kernel_timing(sla_plan *plan, int32_t enable) {
    if (!plan) return SLA_ERR_INVALID_ARG;
    plan->tracer.clear();
    plan->agg.clear();
    plan->tracer.on = enable != 0;
    return SLA_OK;
}

sla_status sla_plan_kernel_timing_collect(sla_plan *plan, int32_t *n_kernels) {
    if (!plan || !n_kernels) return SLA_ERR_INVALID_ARG;
    sla::Tracer &t = plan->tracer;
    if (t.used && cudaEventSynchronize(t.pool[t.used - 1]) != cudaSuccess) return SLA_ERR_CUDA;
    for (const auto &r : t.recs) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, t.pool[r.e0], t.pool[r.e1]) != cudaSuccess) return SLA_ERR_CUDA;
        bool found = false;
        for (auto &a : plan->agg)
            if (!strcmp(a.first, r.name)) { a.second.first += 1; a.second.second += ms; found = true; break; }
        if (!found) plan->agg.push_back({r.name, {1, ms}});
    }
    t.clear();
    *n_kernels = (int32_t)plan->agg.size();
    return SLA_OK;
}

sla_status sla_plan_kernel_timing_get(const sla_plan *plan, int32_t index, const char **name,
                                      int32_t *launches, float *total_ms) {
    if (!plan || index < 0 || (size_t)index >= plan->agg.size()) return SLA_ERR_INVALID_ARG;
    if (name) *name = plan->agg[index].first;
    if (launches) *launches = plan->agg[index].second.first;
    if (total_ms) *total_ms = plan->agg[index].second.second;
    return SLA_OK;
}

sla_status sla_forward(sla_plan *plan, const void *q, const void *k, const void *v,
                       const float *log_decay, const float *beta, const float *gq_logits,
                       const float *gk_logits, const float *h0, void *o, float *ht, void *workspace,
                       size_t workspace_bytes, void *cuda_stream) {
    if (!plan) return SLA_ERR_INVALID_ARG;
    const sla::Dims &d = plan->dims;
    plan->last_launches = 0;
    if (d.B == 0) return SLA_OK;
    if (d.T == 0) {     // nothing to read: the final state is the initial one
        if (!ht) return SLA_OK;
        if (!aligned16(ht) || !aligned16(h0)) return SLA_ERR_INVALID_ARG;
        const size_t bytes = (size_t)d.B * d.H * d.dk * d.dv * sizeof(float);
        cudaError_t e = h0 ? cudaMemcpyAsync(ht, h0, bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)cuda_stream)
                           : cudaMemsetAsync(ht, 0, bytes, (cudaStream_t)cuda_stream);
        return e == cudaSuccess ? SLA_OK : SLA_ERR_CUDA;
    }
    if (!q || !k || !v || !log_decay || !gq_logits || !gk_logits || !o) return SLA_ERR_INVALID_ARG;
    if (d.variant == SLA_GDN && !beta) return SLA_ERR_INVALID_ARG;
    const void *ptrs[] = {q, k, v, log_decay, beta, gq_logits, gk_logits, h0, o, ht, workspace};
    for (const void *p : ptrs)
        if (!aligned16(p)) return SLA_ERR_INVALID_ARG;
    if (plan->fwd_bytes > 0 && (!workspace || workspace_bytes < plan->fwd_bytes)) return SLA_ERR_WORKSPACE;
    sla::FwdArgs a{q, k, v, log_decay, beta, gq_logits, gk_logits, h0, o, ht, (float *)workspace, plan->d_status,
                   plan->varlen.n_seq ? &plan->varlen : nullptr};
    plan->tracer.start((cudaStream_t)cuda_stream);
    const bool generic = plan->flags & SLA_FLAG_FORCE_GENERIC;
    const bool save = (plan->flags & SLA_FLAG_SAVE_FOR_BACKWARD) && forward_can_save(*plan);
    plan->saved.valid = false;
    int n = (!generic && sla::gla_tc_supported(d))
                ? sla::gla_tc_forward(d, a, save ? sla::gla_tc_state_images(a.ws) : nullptr, plan->d_status,
                                      (cudaStream_t)cuda_stream, plan->tracer)
            : (!generic && sla::gdn_tc_supported(d))
                ? sla::gdn_tc_forward(d, a, save ? sla::gdn_tc_records(a.ws) : nullptr, plan->d_status,
                                      (cudaStream_t)cuda_stream, plan->tracer)
                : sla::generic_forward(d, plan->ws, a, true, (cudaStream_t)cuda_stream, plan->tracer);
    if (n < 0) return SLA_ERR_CUDA;
    plan->last_launches = n;
    if (save) {
        sla_plan::Saved &sv = plan->saved;
        sv.valid = true;
        sv.ws = workspace; sv.q = q; sv.k = k; sv.v = v; sv.log_decay = log_decay; sv.beta = beta;
        sv.lq = gq_logits; sv.lk = gk_logits; sv.h0 = h0; sv.stream = cuda_stream;
    }
    return SLA_OK;
}

sla_status sla_backward(sla_plan *plan, const void *q, const void *k, const void *v,
                        const float *log_decay, const float *beta, const float *gq_logits,
                        const float *gk_logits, const float *h0, const void *dO, const float *dht,
                        void *dq, void *dk, void *dv, float *dlog_decay, float *dbeta,
                        float *dgq_logits, float *dgk_logits, float *dh0, void *workspace,
                        size_t workspace_bytes, void *cuda_stream) {
    if (!plan) return SLA_ERR_INVALID_ARG;
    const sla::Dims &d = plan->dims;
    plan->last_launches = 0;
    if (d.B == 0) return SLA_OK;
    if (d.T == 0) {     // no tokens: the gradient of the initial state is the gradient of the final one
        if (!dh0) return SLA_OK;
        if (!aligned16(dh0) || !aligned16(dht)) return SLA_ERR_INVALID_ARG;
        const size_t bytes = (size_t)d.B * d.H * d.dk * d.dv * sizeof(float);
        cudaError_t e = dht ? cudaMemcpyAsync(dh0, dht, bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)cuda_stream)
                            : cudaMemsetAsync(dh0, 0, bytes, (cudaStream_t)cuda_stream);
        return e == cudaSuccess ? SLA_OK : SLA_ERR_CUDA;
    }
    if (!q || !k || !v || !log_decay || !gq_logits || !gk_logits || !dO || !dq || !dk || !dv ||
        !dgq_logits || !dgk_logits)
        return SLA_ERR_INVALID_ARG;
    if (dgq_logits == dgk_logits) return SLA_ERR_INVALID_ARG;
    if (d.variant == SLA_GDN && (!beta || !dbeta || !dlog_decay)) return SLA_ERR_INVALID_ARG;
    if (d.variant == SLA_GLA && !dlog_decay) return SLA_ERR_INVALID_ARG;
    if (d.variant == SLA_RETNET && dlog_decay) return SLA_ERR_INVALID_ARG;
    const void *ptrs[] = {q, k, v, log_decay, beta, gq_logits, gk_logits, h0, dO, dht, dq, dk, dv,
                          dlog_decay, dbeta, dgq_logits, dgk_logits, dh0, workspace};
    for (const void *p : ptrs)
        if (!aligned16(p)) return SLA_ERR_INVALID_ARG;
    if (plan->bwd_bytes > 0 && (!workspace || workspace_bytes < plan->bwd_bytes)) return SLA_ERR_WORKSPACE;
    sla::BwdArgs a{q, k, v, log_decay, beta, gq_logits, gk_logits, h0, dO, dht, dq, dk, dv,
                   dlog_decay, dbeta, dgq_logits, dgk_logits, dh0, (float *)workspace, plan->d_status,
                   plan->varlen.n_seq ? &plan->varlen : nullptr};
    plan->tracer.start((cudaStream_t)cuda_stream);
    const bool generic = plan->flags & SLA_FLAG_FORCE_GENERIC;
    // the states (GLA) or per-chunk records (GDN) are taken from the workspace only if the last sla_forward of this plan
    // left them there for exactly these inputs, on this stream; anything else recomputes them
    sla_plan::Saved &sv = plan->saved;
    const bool have = sv.valid && sv.ws == workspace && sv.q == q && sv.k == k && sv.v == v && sv.log_decay == log_decay &&
                      sv.beta == beta && sv.lq == gq_logits && sv.lk == gk_logits && sv.h0 == h0 && sv.stream == cuda_stream;
    // a backward pass that recomputes writes its own states into `workspace`: whatever an earlier forward left there
    // (for other inputs) is gone, and must not be taken for valid by a later call
    if (!have && sv.ws == workspace) sv.valid = false;
    int n = (!generic && sla::gla_tc_supported(d) && !a.vl && plan->segs.n_seq)
                ? sla::gla_tc_backward_segmented(d, a, plan->segs, plan->d_status, (cudaStream_t)cuda_stream, plan->tracer)
            : (!generic && sla::gla_tc_supported(d))
                ? sla::gla_tc_backward(d, a, have, plan->d_status, (cudaStream_t)cuda_stream, plan->tracer)
            : (!generic && sla::gdn_tc_supported(d))
                ? sla::gdn_tc_backward(d, a, have, plan->d_status, (cudaStream_t)cuda_stream, plan->tracer)
                : sla::generic_backward(d, plan->ws, a, (cudaStream_t)cuda_stream, plan->tracer);
    if (n == -2) return SLA_ERR_UNSUPPORTED;
    if (n < 0) return SLA_ERR_CUDA;
    plan->last_launches = n;
    return SLA_OK;
}

static bool conv_args_ok(int32_t d, int32_t K) { return d >= 16 && d <= 128 && d % 16 == 0 && K >= 1 && K <= 4; }

sla_status sla_plan_shortconv_workspace_bytes(const sla_plan *plan, int32_t d, size_t *bytes) {
    if (!plan || !bytes) return SLA_ERR_INVALID_ARG;
    if (!conv_args_ok(d, 1)) return SLA_ERR_UNSUPPORTED;
    *bytes = sla::shortconv_workspace_bytes(plan->dims, d);
    return SLA_OK;
}

sla_status sla_shortconv_forward(sla_plan *plan, const void *x, const float *w, int32_t d, int32_t K, int32_t normalize,
                                 void *out, void *cuda_stream) {
    if (!plan) return SLA_ERR_INVALID_ARG;
    if (!conv_args_ok(d, K)) return SLA_ERR_UNSUPPORTED;
    const sla::Dims &dm = plan->dims;
    plan->last_launches = 0;
    if (dm.B == 0 || dm.T == 0) return SLA_OK;
    if (!x || !w || !out || !aligned16(x) || !aligned16(w) || !aligned16(out)) return SLA_ERR_INVALID_ARG;
    plan->tracer.start((cudaStream_t)cuda_stream);
    int n = sla::shortconv_forward(dm, d, K, normalize != 0, SLA_SHORTCONV_EPS, x, w, out, (cudaStream_t)cuda_stream,
                                   plan->tracer);
    if (n < 0) return SLA_ERR_CUDA;
    plan->last_launches = n;
    return SLA_OK;
}

sla_status sla_shortconv_backward(sla_plan *plan, const void *x, const float *w, int32_t d, int32_t K, int32_t normalize,
                                  const void *dout, void *dx, float *dw, void *workspace, size_t workspace_bytes,
                                  void *cuda_stream) {
    if (!plan) return SLA_ERR_INVALID_ARG;
    if (!conv_args_ok(d, K)) return SLA_ERR_UNSUPPORTED;
    const sla::Dims &dm = plan->dims;
    plan->last_launches = 0;
    if (!dw || !aligned16(dw)) return SLA_ERR_INVALID_ARG;
    if (dm.B == 0 || dm.T == 0)
        return cudaMemsetAsync(dw, 0, (size_t)dm.H * d * K * sizeof(float), (cudaStream_t)cuda_stream) == cudaSuccess
                   ? SLA_OK : SLA_ERR_CUDA;
    if (!x || !w || !dout || !dx) return SLA_ERR_INVALID_ARG;
    const void *ptrs[] = {x, w, dout, dx, workspace};
    for (const void *p : ptrs)
        if (!aligned16(p)) return SLA_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < sla::shortconv_workspace_bytes(dm, d)) return SLA_ERR_WORKSPACE;
    plan->tracer.start((cudaStream_t)cuda_stream);
    int n = sla::shortconv_backward(dm, d, K, normalize != 0, SLA_SHORTCONV_EPS, x, w, dout, dx, dw, (float *)workspace,
                                    (cudaStream_t)cuda_stream, plan->tracer);
    if (n < 0) return SLA_ERR_CUDA;
    plan->last_launches = n;
    return SLA_OK;
}

static bool out_proj_args_ok(const sla::Dims &d, int32_t d_model) {
    return d.io_bf16 && d_model >= 8 && d_model % 8 == 0 && (d.H * d.dv) % 8 == 0;
}

sla_status sla_out_proj_forward(sla_plan *plan, const void *o, const void *w_o, int32_t d_model, void *y, void *cuda_stream) {
    if (!plan) return SLA_ERR_INVALID_ARG;
    const sla::Dims &d = plan->dims;
    if (!out_proj_args_ok(d, d_model)) return SLA_ERR_UNSUPPORTED;
    plan->last_launches = 0;
    if (d.B == 0 || d.T == 0) return SLA_OK;
    if (!o || !w_o || !y || !aligned16(o) || !aligned16(w_o) || !aligned16(y)) return SLA_ERR_INVALID_ARG;
    plan->tracer.start((cudaStream_t)cuda_stream);
    int n = sla::out_proj_forward((long)d.B * d.T, d.H * d.dv, d_model, o, w_o, y, plan->d_status, (cudaStream_t)cuda_stream,
                                  plan->tracer);
    if (n < 0) return SLA_ERR_CUDA;
    plan->last_launches = n;
    return SLA_OK;
}

sla_status sla_out_proj_backward(sla_plan *plan, const void *o, const void *w_o, const void *dy, int32_t d_model, void *d_o,
                                 float *dw_o, void *cuda_stream) {
    if (!plan) return SLA_ERR_INVALID_ARG;
    const sla::Dims &d = plan->dims;
    if (!out_proj_args_ok(d, d_model)) return SLA_ERR_UNSUPPORTED;
    plan->last_launches = 0;
    if (!dw_o || !aligned16(dw_o)) return SLA_ERR_INVALID_ARG;
    if (d.B == 0 || d.T == 0)           // no tokens: the weight gradient is zero
        return cudaMemsetAsync(dw_o, 0, (size_t)d.H * d.dv * d_model * sizeof(float), (cudaStream_t)cuda_stream) == cudaSuccess
                   ? SLA_OK : SLA_ERR_CUDA;
    if (!o || !w_o || !dy || !d_o || !aligned16(o) || !aligned16(w_o) || !aligned16(dy) || !aligned16(d_o))
        return SLA_ERR_INVALID_ARG;
    plan->tracer.start((cudaStream_t)cuda_stream);
    int n = sla::out_proj_backward((long)d.B * d.T, d.H * d.dv, d_model, o, w_o, dy, d_o, dw_o, plan->d_status,
                                   (cudaStream_t)cuda_stream, plan->tracer);
    if (n < 0) return SLA_ERR_CUDA;
    plan->last_launches = n;
    return SLA_OK;
}

sla_status sla_plan_gate_scores_workspace_bytes(const sla_plan *plan, size_t *bytes) {
    if (!plan || !bytes) return SLA_ERR_INVALID_ARG;
    *bytes = sla::gate_scores_workspace_bytes(plan->dims);
    return SLA_OK;
}

sla_status sla_gate_scores_forward(sla_plan *plan, const void *q, const void *k, const float *w_gq, const float *w_gk,
                                   float *gq_logits, float *gk_logits, void *cuda_stream) {
    if (!plan) return SLA_ERR_INVALID_ARG;
    const sla::Dims &d = plan->dims;
    plan->last_launches = 0;
    if (d.B == 0 || d.T == 0) return SLA_OK;
    if (!q || !k || !w_gq || !w_gk || !gq_logits || !gk_logits) return SLA_ERR_INVALID_ARG;
    const void *ptrs[] = {q, k, w_gq, w_gk, gq_logits, gk_logits};
    for (const void *p : ptrs)
        if (!aligned16(p)) return SLA_ERR_INVALID_ARG;
    plan->tracer.start((cudaStream_t)cuda_stream);
    int n = sla::gate_scores_forward(d, q, k, w_gq, w_gk, gq_logits, gk_logits, (cudaStream_t)cuda_stream, plan->tracer);
    if (n < 0) return SLA_ERR_CUDA;
    plan->last_launches = n;
    return SLA_OK;
}

sla_status sla_gate_scores_backward(sla_plan *plan, const void *q, const void *k, const float *w_gq, const float *w_gk,
                                    const float *dgq_logits, const float *dgk_logits, void *dq, void *dk,
                                    float *dw_gq, float *dw_gk, void *workspace, size_t workspace_bytes,
                                    void *cuda_stream) {
    if (!plan) return SLA_ERR_INVALID_ARG;
    const sla::Dims &d = plan->dims;
    plan->last_launches = 0;
    if (!dw_gq || !dw_gk || !aligned16(dw_gq) || !aligned16(dw_gk)) return SLA_ERR_INVALID_ARG;
    if (d.B == 0 || d.T == 0) {          // no tokens: the weight gradients are zero
        const size_t wb = (size_t)d.dk * d.H * sizeof(float);
        if (cudaMemsetAsync(dw_gq, 0, wb, (cudaStream_t)cuda_stream) != cudaSuccess ||
            cudaMemsetAsync(dw_gk, 0, wb, (cudaStream_t)cuda_stream) != cudaSuccess)
            return SLA_ERR_CUDA;
        return SLA_OK;
    }
    if (!q || !k || !w_gq || !w_gk || !dgq_logits || !dgk_logits || !dq || !dk) return SLA_ERR_INVALID_ARG;
    const void *ptrs[] = {q, k, w_gq, w_gk, dgq_logits, dgk_logits, dq, dk, workspace};
    for (const void *p : ptrs)
        if (!aligned16(p)) return SLA_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < sla::gate_scores_workspace_bytes(d)) return SLA_ERR_WORKSPACE;
    plan->tracer.start((cudaStream_t)cuda_stream);
    int n = sla::gate_scores_backward(d, q, k, w_gq, w_gk, dgq_logits, dgk_logits, dq, dk, dw_gq, dw_gk,
                                      (float *)workspace, (cudaStream_t)cuda_stream, plan->tracer);
    if (n < 0) return SLA_ERR_CUDA;
    plan->last_launches = n;
    return SLA_OK;
}

sla_status sla_decode_steps(sla_plan *plan, int32_t Bdec, int32_t n_tokens, const void *q, const void *k,
                            const void *v, const float *log_decay, const float *beta,
                            const float *gq_logits, const float *gk_logits, float *state, void *o,
                            void *cuda_stream) {
    if (!plan || Bdec < 0 || n_tokens < 0) return SLA_ERR_INVALID_ARG;
    const sla::Dims &d = plan->dims;
    plan->last_launches = 0;
    if (Bdec == 0 || n_tokens == 0) return SLA_OK;
    if ((uint64_t)Bdec * d.H * d.dk > 0x7fffffffu) return SLA_ERR_UNSUPPORTED;   // (row coordinate of the state's tensor map)
    if (!q || !k || !v || !log_decay || !gq_logits || !gk_logits || !state || !o) return SLA_ERR_INVALID_ARG;
    if (d.variant == SLA_GDN && !beta) return SLA_ERR_INVALID_ARG;
    const void *ptrs[] = {q, k, v, log_decay, beta, gq_logits, gk_logits, state, o};
    for (const void *p : ptrs)
        if (!aligned16(p)) return SLA_ERR_INVALID_ARG;
    sla::DecArgs a{q, k, v, log_decay, beta, gq_logits, gk_logits, state, o, Bdec, n_tokens};
    plan->tracer.start((cudaStream_t)cuda_stream);
    int n = sla::decode_step(d, a, plan->d_status, (cudaStream_t)cuda_stream, plan->tracer);
    if (n < 0) return SLA_ERR_CUDA;
    plan->last_launches = n;
    return SLA_OK;
}

sla_status sla_decode_step(sla_plan *plan, int32_t Bdec, const void *q_t, const void *k_t,
                           const void *v_t, const float *log_decay_t, const float *beta_t,
                           const float *gq_logits_t, const float *gk_logits_t, float *state, void *o_t,
                           void *cuda_stream) {
    return sla_decode_steps(plan, Bdec, 1, q_t, k_t, v_t, log_decay_t, beta_t, gq_logits_t, gk_logits_t, state, o_t,
                            cuda_stream);
}

}  // extern "C"
