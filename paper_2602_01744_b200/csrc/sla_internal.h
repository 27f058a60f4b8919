// Internal declarations shared by the host API and the kernel translation units.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include <utility>
#include <vector>

#include "sla.h"

namespace sla {

// bits of a plan's device status word
constexpr int STATUS_TIMEOUT = 1;    // a bounded wait expired
constexpr int STATUS_RANGE = 2;      // a chunk's cumulative log-decay went below -SLA_MAX_CHUNK_DECAY

struct Dims {
    int variant;      // sla_variant
    int io_bf16;      // 1: q,k,v,o are bf16, 0: fp32
    int B, T, H, dk, dv, C, NT;
    float scale;
};

// Packed variable-length batches (B = 1: sequences one after another along T, the state reset at every boundary,
// chunks cut from each sequence's own start).  Per sequence: first token, length, chunks, and the index of its first
// state slot (the sum of chunks + 1 over the sequences before it).  The table is kept longest sequence first, so that the
// CTAs of long sequences are dispatched first (one CTA per (sequence, head), in table order).
struct SeqInfo { int t0, T, NT, slot0, id; };     // id: the sequence's number as the caller counts them
// Host side of a plan's sequence table.  The tensor-core kernels address a sequence through tensor maps of its own
// (based at its first token, T = its length: loads past its end read zeros, stores are clipped there, exactly as at the
// end of a batch row); those live in device arrays, one region per kernel kind, encoded again only when the tensors
// they point at change.
struct Varlen {
    int n_seq = 0;
    long slots = 0;                     // sum over the sequences of (chunks + 1)
    std::vector<SeqInfo> seqs;
    SeqInfo *d_seqs = nullptr;
    struct Region {
        CUtensorMap *dev = nullptr, *host = nullptr;    // [n_seq][MAPS_PER_SEQ]; host: pinned mirror
        const void *key[10] = {};
        bool valid = false;
        cudaEvent_t uploaded = nullptr;
    } reg[3];                           // 0: forward, 1: state / record sweep, 2: gradient sweep
    static constexpr int MAPS_PER_SEQ = 9;
    int seg_P = 0, seg_L = 0;           // > 0: an internal table that cuts each of the B batch rows into seg_P segments of seg_L chunks
};

// Carve-up of the caller's workspace (all fp32, offsets in floats, each 64-float aligned).
struct Workspace {
    size_t Gq, Gk;          // [B,T,H] gates
    size_t bcum;            // GLA [B,T,H,dk]; RETNET/GDN [B,T,H]: chunk-local inclusive cumulative log-decay
    size_t states;          // [B,H,NT+1,dk,dv]: state before each chunk, last = final state
    size_t W, U0, U;        // GDN: W [B,T,H,dk]; U0 and U = U0 - W S [B,T,H,dv]
    size_t fwd_floats;
    size_t dstates;         // [B,H,NT,dk,dv]: gradient w.r.t. the state after each chunk
    size_t dU;              // GDN: [B,T,H,dv]
    size_t dKbg, dVb, dbpart;  // GDN: [B,T,H,dk], [B,T,H,dv], [B,T,H]
    size_t dGq, dGk;        // [B,T,H]
    size_t bwd_floats;
};

Workspace plan_workspace(const Dims &d);

// ---- generic (fp32 CUDA-core) chunk kernels: sla_generic.cu ----
struct FwdArgs {
    const void *q, *k, *v;
    const float *log_decay, *beta, *lq, *lk, *h0;
    void *o;
    float *ht;
    float *ws;
    int *status;            // the plan's device status word
    Varlen *vl = nullptr;   // packed variable-length batch (tensor-core kernels only), else nullptr
};
struct BwdArgs {
    const void *q, *k, *v;
    const float *log_decay, *beta, *lq, *lk, *h0;
    const void *dO;
    const float *dht;
    void *dq, *dk, *dv;
    float *dlog_decay, *dbeta, *dlq, *dlk, *dh0;
    float *ws;
    int *status;
    Varlen *vl = nullptr;
};
struct DecArgs {
    const void *q, *k, *v;
    const float *log_decay, *beta, *lq, *lk;
    float *state;
    void *o;
    int Bdec;
    int n_tok;              // consecutive tokens per sequence applied in one launch
};

// Optional per-kernel timing: one CUDA event before the first kernel of a call and one after every
// kernel, all on the launch stream.  Off by default (mark() is then a no-op).
struct Tracer {
    bool on = false;
    cudaStream_t st = nullptr;
    std::vector<cudaEvent_t> pool;
    size_t used = 0;
    struct Rec { const char *name; size_t e0, e1; };
    std::vector<Rec> recs;
    size_t last = 0;
    size_t record() {
        if (used == pool.size()) {
            cudaEvent_t e;
            cudaEventCreate(&e);
            pool.push_back(e);
        }
        cudaEventRecord(pool[used], st);
        return used++;
    }
    void start(cudaStream_t s) { if (on) { st = s; last = record(); } }
    void mark(const char *name) { if (on) { size_t e = record(); recs.push_back({name, last, e}); last = e; } }
    void clear() { used = 0; recs.clear(); }
    void destroy() { for (auto e : pool) cudaEventDestroy(e); pool.clear(); clear(); }
};

// Each returns the number of kernels launched (>0) or -1 after a CUDA launch error.
int generic_forward(const Dims &d, const Workspace &w, const FwdArgs &a, bool write_o, cudaStream_t st, Tracer &tr);
int generic_backward(const Dims &d, const Workspace &w, const BwdArgs &a, cudaStream_t st, Tracer &tr);
// recurrent decode (sla_decode.cu): streaming kernel over 32-column slices of the state
int decode_step(const Dims &d, const DecArgs &a, int *status, cudaStream_t st, Tracer &tr);
int decode_configure();
// Opt the kernels into the shared memory they need (once per device).
int generic_configure();
int gdn_configure();

// ---- tensor-core (tcgen05 / TMEM / TMA) Softmax-GLA kernels: sla_gla_tc.cu ----
bool gla_tc_supported(const Dims &d);
int gla_tc_configure();
// With `simg` not null (and gla_tc_forward_can_save) the forward also leaves the bf16 image of the state before every
// chunk there, in the layout the gradient sweep reads: the backward pass of the same inputs then needs no state sweep.
bool gla_tc_forward_can_save(const Dims &d, const Varlen *vl = nullptr);
uint8_t *gla_tc_state_images(float *ws);   // where in the backward workspace the images sit
int gla_tc_forward(const Dims &d, const FwdArgs &a, uint8_t *simg, int *status, cudaStream_t st, Tracer &tr);
// Backward: chunk-state sweep, gradient sweep, gate softmax backward.  Needs the first
// B*H*(NT+1)*32 KiB + 2*B*T*H*4 bytes (rounded up) of the workspace, less than the generic path.
int gla_tc_bwd_configure();
// Segmented forward of long sequences, first pass: every (sequence, segment of L chunks) from a zero state; leaves
// the state it reaches (fin [B*H*P][128][128]) and the segment's total decay (gam [B*H*P][128]).
int gla_tc_segment_summaries(const Dims &d, const FwdArgs &a, int P, int L, float *fin, float *gam, int *status,
                             cudaStream_t st, Tracer &tr);
// Bytes of workspace the tensor-core forward / backward need (the generic kernels need more).
size_t gla_tc_forward_workspace_bytes(const Dims &d, const Varlen *vl = nullptr);
size_t gla_tc_backward_workspace_bytes(const Dims &d, const Varlen *vl = nullptr);
int gla_tc_backward(const Dims &d, const BwdArgs &a, bool have_states, int *status, cudaStream_t st, Tracer &tr);
// Few long sequences: the backward in segments.  Every batch row is cut into P segments of L chunks that run as the
// sequences of a packed batch (`segs`, filled by gla_tc_backward_segment_table); the states at the segment starts and
// the state gradients at the segment ends come from summaries folded along each row.  P == 1: not worth it.
void gla_tc_backward_choose_segments(const Dims &d, int &P, int &L);
void gla_tc_backward_segment_table(const Dims &d, int P, int L, Varlen &segs);
size_t gla_tc_backward_segmented_workspace_bytes(const Dims &d, const Varlen &segs);
int gla_tc_backward_segmented(const Dims &d, const BwdArgs &a, Varlen &segs, int *status, cudaStream_t st, Tracer &tr);

// ---- tensor-core Softmax-GatedDeltaNet forward (WY form): sla_gdn_tc.cu.  Needs no workspace. ----
bool gdn_tc_supported(const Dims &d);
int gdn_tc_configure();
int gdn_tc_forward(const Dims &d, const FwdArgs &a, uint8_t *save, int *status, cudaStream_t st, Tracer &tr);
uint8_t *gdn_tc_records(float *ws);        // where in the backward workspace the per-chunk records sit
int gdn_tc_forward_save(const Dims &d, const FwdArgs &a, uint8_t *save, int *status, cudaStream_t st, Tracer &tr);
// backward: forward sweep in save mode (per-chunk S_n, U, T records), reverse gradient sweep, gate softmax backward
int gdn_tc_bwd_configure();
size_t gdn_tc_backward_workspace_bytes(const Dims &d, const Varlen *vl = nullptr);
int gdn_tc_backward(const Dims &d, const BwdArgs &a, bool have_records, int *status, cudaStream_t st, Tracer &tr);
int gate_bwd_prod(const float *lq, const float *lk, const float *pq, const float *pk, float *dlq, float *dlk, long n_tok,
                  int H, cudaStream_t st);

// ---- gate score projections of Eq. 4 and their reverse: sla_gate_scores.cu ----
size_t gate_scores_workspace_bytes(const Dims &d);
int gate_scores_forward(const Dims &d, const void *q, const void *k, const float *Wq, const float *Wk, float *lq,
                        float *lk, cudaStream_t st, Tracer &tr);
int gate_scores_backward(const Dims &d, const void *q, const void *k, const float *Wq, const float *Wk, const float *dlq,
                         const float *dlk, void *dq, void *dk, float *dWq, float *dWk, float *ws, cudaStream_t st,
                         Tracer &tr);

// ---- feature map of the Gated-DeltaNet instantiation (short causal convolution, SiLU, per-head L2 norm): sla_shortconv.cu ----
size_t shortconv_workspace_bytes(const Dims &d, int width);
int shortconv_forward(const Dims &d, int width, int K, bool normalize, float eps, const void *x, const float *w, void *out,
                      cudaStream_t st, Tracer &tr);
int shortconv_backward(const Dims &d, int width, int K, bool normalize, float eps, const void *x, const float *w,
                       const void *dout, void *dx, float *dw, float *ws, cudaStream_t st, Tracer &tr);

// Output projection (Eq. 7) and its reverse: dense bf16 contractions on the tensor cores (sla_out_proj.cu).
int out_proj_configure();
int out_proj_forward(long n_tok, int K, int Dm, const void *o, const void *w, void *y, int *status, cudaStream_t st, Tracer &tr);
int out_proj_backward(long n_tok, int K, int Dm, const void *o, const void *w, const void *dy, void *d_o, float *dw, int *status,
                      cudaStream_t st, Tracer &tr);

// GDN per-tile gradient kernels (after the recompute pass and the state-gradient scan).
int gdn_backward_tiles(const Dims &d, const Workspace &w, const BwdArgs &a, cudaStream_t st, Tracer &tr);

}  // namespace sla

// The opaque plan of the C ABI.
struct sla_plan {
    sla::Dims dims;
    sla::Workspace ws;          // carve-up for the generic kernels
    size_t fwd_bytes, bwd_bytes; // what the kernels this plan selects need (tensor-core plans need less than ws says)
    uint32_t flags;
    int device;
    int *d_status;          // device status word (bounded waits report here)
    int last_launches;
    // SLA_FLAG_SAVE_FOR_BACKWARD: what the last sla_forward left in its workspace, and for which inputs
    struct Saved {
        bool valid = false;
        const void *ws = nullptr, *q = nullptr, *k = nullptr, *v = nullptr, *log_decay = nullptr, *beta = nullptr, *lq = nullptr,
                   *lk = nullptr, *h0 = nullptr;
        void *stream = nullptr;
    } saved;
    sla::Varlen varlen;     // sla_plan_set_sequences: packed variable-length batch (n_seq == 0: regular batch)
    sla::Varlen segs;       // tensor-core GLA / RetNet plans with few long sequences: the segments the backward runs in
    sla::Tracer tracer;
    std::vector<std::pair<const char *, std::pair<int, float>>> agg;   // name -> (launches, total ms)
};
