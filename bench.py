#!/usr/bin/env python
"""Benchmark of the SLA hot path: SLA-GLA forward + backward tokens/s at B=8, T=4096, H=16, d=128, bf16.

One step = sla_forward followed by sla_backward over one batch of seeded synthetic input, through the
C-ABI binding.  Prints ONE JSON line (rank 0).  `--impl reference` times the fp64 CPU oracle on a
bounded sample of the same workload instead.  With --gpus N > 1 (under torchrun) every rank runs an
independent replica of the workload on its own GPU (the path has no exchange step): weak scaling.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

METRIC = "SLA-GLA fwd+bwd tokens/s (T=4K,H=16,d=128,bf16)"
UNIT = "tokens/s"
WORKLOAD = "C2"
CPU_ROWS = 2          # batch rows of the workload the CPU oracle is timed on (about 20 core-seconds)
# Algorithmic HBM bytes per (token, head) at d_k=d_v=128: bf16 q,k,v,o (+dO,dq,dk,dv), fp32 log-decay
# (+ its gradient), fp32 gate logits (+ their gradients).
FWD_BYTES_PER_TOKEN_HEAD = 4 * 256 + 512 + 8            # 1544
BWD_BYTES_PER_TOKEN_HEAD = 4 * 256 + 512 + 3 * 256 + 512 + 16   # 2832
# The gated delta rule has a scalar decay and beta per (token, head): 4 B each instead of 512 B.
GDN_FWD_BYTES_PER_TOKEN_HEAD = 4 * 256 + 8 + 8          # 1040
GDN_BWD_BYTES_PER_TOKEN_HEAD = 4 * 256 + 3 * 256 + 8 + 8 + 16   # 1824
# Tensor-core work per (token, head) at chunk 64, d_k = d_v = 128 (2 FLOP per multiply-add).  "algorithmic" counts the
# causal half of the 64x64 products only; "executed" is what the MMAs issue (full 64x64 tiles; the chunk-state
# recomputation of the backward is counted only when the plan recomputes).
GLA_FLOP = {"fwd_algorithmic": 82176, "bwd_algorithmic": 205440, "fwd_executed": 98304, "bwd_executed": 212992,
            "state_recompute_executed": 32768}
# Softmax-RetNet: the decay is a constant per head, so no decay tensor is read and no decay gradient written.
RETNET_FWD_BYTES_PER_TOKEN_HEAD = 4 * 256 + 8           # 1032
RETNET_BWD_BYTES_PER_TOKEN_HEAD = 4 * 256 + 3 * 256 + 16   # 1808
KERNEL_BYTES = {  # which share of the compulsory traffic each kernel is accountable for
    "output": FWD_BYTES_PER_TOKEN_HEAD, "grads_lin": BWD_BYTES_PER_TOKEN_HEAD,
    "gla_fwd_tc": FWD_BYTES_PER_TOKEN_HEAD, "gla_bwd_tc": BWD_BYTES_PER_TOKEN_HEAD,
    "gdn_fwd_tc": GDN_FWD_BYTES_PER_TOKEN_HEAD, "gdn_bwd_tc": GDN_BWD_BYTES_PER_TOKEN_HEAD,
}
KERNEL_BYTES_RETNET = {"gla_fwd_tc": RETNET_FWD_BYTES_PER_TOKEN_HEAD, "gla_bwd_tc": RETNET_BWD_BYTES_PER_TOKEN_HEAD}


def step_bytes_per_pair(variant: str, backward: bool) -> int:
    f, b = {"gla": (FWD_BYTES_PER_TOKEN_HEAD, BWD_BYTES_PER_TOKEN_HEAD),
            "gdn": (GDN_FWD_BYTES_PER_TOKEN_HEAD, GDN_BWD_BYTES_PER_TOKEN_HEAD),
            "retnet": (RETNET_FWD_BYTES_PER_TOKEN_HEAD, RETNET_BWD_BYTES_PER_TOKEN_HEAD)}[variant]
    return f + (b if backward else 0)


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            d = json.loads(p.read_text())
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


def measured_tensor_peaks():
    """(burst, sustained) dense bf16 TFLOP/s and where they come from."""
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            d = json.loads(p.read_text())
            return float(d["bf16_tflops"]), float(d["bf16_tflops_sustained"]), "measured"
        except Exception:
            pass
    return 1590.0, 1400.0, "fallback"


def sources_sha256(files) -> str:
    """Hash of the named files of the kernel source folder (the sources a profiled kernel is built from)."""
    import hashlib
    h = hashlib.sha256()
    for f in sorted(files):
        h.update((ROOT / "paper_2602_01744_b200" / "csrc" / f).read_bytes())
    return h.hexdigest()


def recorded_counters(workload: str, kernel: str, key: str = "bytes_per_launch_full_size"):
    """A figure from the committed ncu summary (DRAM bytes per launch, tensor-pipe activity), if one covers this kernel
    on this workload (full size, plan flags as in the default run).  Each record names the source files its kernel is
    built from and carries their hash: once one of them has changed, the figure is stale and None is reported."""
    p = ROOT / "profiles" / "dram_traffic.json"
    if not p.exists():
        return None
    try:
        e = json.loads(p.read_text()).get(workload, {}).get(kernel)
        if e is None or e.get("source_sha256") != sources_sha256(e["sources"]):
            return None
        return e.get(key)
    except Exception:
        return None


def recorded_traffic(workload: str, kernel: str):
    return recorded_counters(workload, kernel)


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=self.tmp, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.tmp.flush()
        rows = [r.split(",") for r in Path(self.tmp.name).read_text().strip().splitlines() if r.count(",") >= 6]
        os.unlink(self.tmp.name)
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm = [float(r[0]) for r in rows]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[3 + i].strip().lower() == "active" for r in rows)]
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": float(rows[0][1]), "samples": len(rows),
                "power_w_max": max(float(r[2]) for r in rows), "reasons": reasons}


def cpu_oracle_sample(cfg, x, steps=1, warmup=0):
    """fp64 oracle, forward (+ backward where the workload has one), on the first CPU_ROWS batch rows of the workload
    (all T tokens, all heads)."""
    from oracle import sla_oracle as orc
    s = lambda t: t if t.dim() == 1 else t[0:CPU_ROWS]      # (RetNet's log-decay is per head, not per batch row)
    args = (s(x["q"]), s(x["k"]), s(x["v"]), s(x["log_decay"]), s(x["gq_logits"]), s(x["gk_logits"]))
    # widen once outside the timed region, as the GPU arm holds its inputs resident
    args = tuple(a.double().numpy() for a in args)
    beta = None if x.get("beta") is None else s(x["beta"]).double().numpy()
    dO = s(x["dO"]).double().numpy() if cfg.backward else None
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        orc.forward(cfg.variant, *args, beta=beta, scale=cfg.scale)
        if cfg.backward:
            orc.backward(cfg.variant, *args, dO, beta=beta, scale=cfg.scale)
        dt = time.perf_counter() - t0
        if i >= warmup:
            times.append(dt)
    tokens = cfg.T * min(CPU_ROWS, cfg.B)
    return tokens, times, orc.num_threads()


def run_reference(args, cfg, rank):
    if rank != 0:
        return
    from paper_2602_01744_b200.inputs import make_inputs, small
    x = make_inputs(small(cfg, B=min(CPU_ROWS, cfg.B)))
    tokens, times, cores = cpu_oracle_sample(cfg, x, steps=args.steps, warmup=min(args.warmup, 1))
    total = sum(times)
    value = tokens * len(times) / total
    sample = (f"first {min(CPU_ROWS, cfg.B)} batch rows of {WORKLOAD}: T={cfg.T}, H={cfg.H}, d={cfg.d_k}, "
              f"{'forward+backward' if cfg.backward else 'forward'}, fp64 recurrent oracle")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "variant": cfg.variant, "B": min(CPU_ROWS, cfg.B), "T": cfg.T, "H": cfg.H,
                   "d_k": cfg.d_k, "d_v": cfg.d_v, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--generic", action="store_true", help="force the fp32 CUDA-core kernels")
    ap.add_argument("--recompute", action="store_true",
                    help="plan without SLA_FLAG_SAVE_FOR_BACKWARD: the backward pass recomputes the chunk states "
                         "instead of reading what the forward pass of the same step left in the workspace")
    ap.add_argument("--workload", default="C2", choices=["C1", "C2", "C3", "C4", "R2"],
                    help="C2 is the benchmark; the other configurations (C1, C3: forward only; C4: gated delta rule, "
                         "forward + backward; R2: Softmax-RetNet at the shapes of C2) are timed the same way for the "
                         "per-configuration figures and profiles")
    ap.add_argument("--packed", action="store_true",
                    help="the workload's B*T tokens as ONE packed row of variable-length sequences (a seeded mix of "
                         "lengths from 64 to 4096 tokens, the maximum training length of the paper; sla_plan_set_sequences) instead of B rows of T: not the "
                         "benchmark, labelled in config")
    ap.add_argument("--batch", type=int, default=0,
                    help="profiling aid: shrink the batch of the workload (0 = the full configuration; "
                         "a reduced batch is not the benchmark and is labelled in config)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "b200" else args.warmup

    from paper_2602_01744_b200.inputs import CONFIGS, make_inputs
    global WORKLOAD, METRIC
    WORKLOAD = args.workload
    cfg = CONFIGS[WORKLOAD]
    passes = "forward+backward" if cfg.backward else "forward"
    if WORKLOAD != "C2":
        METRIC = f"SLA-{cfg.variant.upper()} {passes} tokens/s ({WORKLOAD}: B={cfg.B},T={cfg.T},H={cfg.H},d={cfg.d_k},{cfg.dtype})"
    if args.batch > 0:
        from paper_2602_01744_b200.inputs import small
        cfg = small(cfg, B=args.batch)
    packed_cu = None
    if args.packed:
        import random
        from paper_2602_01744_b200.inputs import small
        total = cfg.B * cfg.T
        rng, cu = random.Random(7), [0]
        while cu[-1] < total:
            cu.append(min(total, cu[-1] + rng.choice([64, 200, 512, 1000, 2048, 4096])))
        packed_cu = cu
        cfg = small(cfg, B=1, T=total)
        METRIC += f" [packed: {len(cu) - 1} sequences of 64..4096 tokens in one row of {total}]"
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, cfg, rank)
        return

    import torch
    from paper_2602_01744_b200 import api

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the SLA library has no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    x = make_inputs(cfg)                        # every replica draws the same seeded batch
    names = ["q", "k", "v", "log_decay", "gq_logits", "gk_logits"] + (["beta"] if x.get("beta") is not None else []) + \
            (["dO"] if cfg.backward else [])
    host = {n: x[n].pin_memory() for n in names}
    dev = {n: host[n].cuda() for n in names}
    dev.setdefault("beta", None)
    flags = api.SLA_FLAG_FORCE_GENERIC if args.generic else 0
    saving = cfg.backward and not args.recompute and not args.generic
    if saving:      # a training step: the forward leaves the chunk states for the backward of the same step
        flags |= api.SLA_FLAG_SAVE_FOR_BACKWARD
    plan = api.sla_plan_create(cfg.variant, cfg.dtype, cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk,
                               cfg.scale, flags)
    if packed_cu is not None:
        plan.set_sequences(packed_cu)
    ws = plan.workspace(backward=cfg.backward)
    o = torch.empty_like(dev["v"])
    grads = None
    if cfg.backward:
        grads = dict(dq=torch.empty_like(dev["q"]), dk=torch.empty_like(dev["k"]), dv=torch.empty_like(dev["v"]),
                     dlog_decay=None if cfg.variant == "retnet" else torch.empty_like(dev["log_decay"]),
                     dbeta=None if dev["beta"] is None else torch.empty_like(dev["beta"]),
                     dgq_logits=torch.empty_like(dev["gq_logits"]), dgk_logits=torch.empty_like(dev["gk_logits"]),
                     dh0=None)
    launches = [0]

    def step(d, o_=None, grads_=None):
        api.sla_forward(plan, d["q"], d["k"], d["v"], d["log_decay"], d["gq_logits"], d["gk_logits"], beta=d.get("beta"),
                        o=o if o_ is None else o_, workspace=ws)
        launches[0] += plan.last_launch_count
        if cfg.backward:
            api.sla_backward(plan, d["q"], d["k"], d["v"], d["log_decay"], d["gq_logits"], d["gk_logits"], d["dO"],
                             beta=d.get("beta"), workspace=ws, out=grads if grads_ is None else grads_)
            launches[0] += plan.last_launch_count

    for _ in range(args.warmup):
        step(dev)
    barrier()
    plan.poll()

    # ---- device-resident timing (inputs in HBM; 0.77 GB of inputs per step, far beyond the 126 MB L2) ----
    launches[0] = 0
    sampler = ClockSampler(local)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        step(dev)
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop()
    plan.poll()
    n_launch = launches[0]
    # second pass of the same steps with one CUDA event after every kernel (on the launch stream, inside the library):
    # per-kernel durations and shares.  Kept out of the pass above so that `value` carries no measurement overhead.
    plan.set_kernel_timing(True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        step(dev)
    e1.record()
    barrier()
    ms_traced = e0.elapsed_time(e1)
    ktimes = plan.kernel_times()
    plan.set_kernel_timing(False)
    plan.poll()
    launches[0] = n_launch
    from paper_2602_01744_b200.replicas import whole_job_throughput
    tokens_step = cfg.B * cfg.T
    value, ms = whole_job_throughput(tokens_step, args.steps, ms, dist, "cuda")

    # ---- end to end: pinned host inputs -> device, run, results -> pinned host, every step ----
    # Every step copies all of its inputs in and all of its results out.  The three legs run on three streams with
    # double-buffered device staging, so that the copy-in of step i+1 and the copy-out of step i-1 overlap the compute
    # of step i (PCIe is full duplex); the kernels themselves still run one step after the other.
    def out_list(o_, g_):
        return [o_] + ([t for t in (g_["dq"], g_["dk"], g_["dv"], g_["dlog_decay"], g_["dbeta"], g_["dgq_logits"],
                                    g_["dgk_logits"]) if t is not None] if cfg.backward else [])

    o2 = [o, torch.empty_like(o)]
    g2 = [grads, None if grads is None else {n: (None if t is None else torch.empty_like(t)) for n, t in grads.items()}]
    outs2 = [out_list(o2[j], g2[j]) for j in range(2)]
    host_out = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in outs2[0]]
    stage2 = [{n: torch.empty_like(dev[n]) for n in names} for _ in range(2)]
    for st_ in stage2:
        st_.setdefault("beta", None)
    h2d = sum(host[n].numel() * host[n].element_size() for n in names)
    d2h = sum(t.numel() * t.element_size() for t in outs2[0])
    e2e_steps = max(3, min(args.steps, 10))
    s_in, s_out, s_c = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()

    def e2e_run(nsteps):
        in_ready, done, copied = [], [], []
        for i in range(nsteps):
            j = i % 2
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(done[i - 2])            # the staging buffer's previous step has been computed
                for n in names:
                    stage2[j][n].copy_(host[n], non_blocking=True)
                ev = torch.cuda.Event()
                ev.record(s_in)
                in_ready.append(ev)
            s_c.wait_event(in_ready[i])
            if i >= 2:
                s_c.wait_event(copied[i - 2])               # the output buffers' previous results are on the host
            step(stage2[j], o2[j], g2[j])
            ev = torch.cuda.Event()
            ev.record(s_c)
            done.append(ev)
            with torch.cuda.stream(s_out):
                s_out.wait_event(done[i])
                for src, dst in zip(outs2[j], host_out):
                    dst.copy_(src, non_blocking=True)
                ev = torch.cuda.Event()
                ev.record(s_out)
                copied.append(ev)
        s_c.wait_event(copied[-1])

    e2e_run(2)
    barrier()
    e0.record()
    e2e_run(e2e_steps)
    e1.record()
    barrier()
    e2e_value, ms_e2e = whole_job_throughput(tokens_step, e2e_steps, e0.elapsed_time(e1), dist, "cuda")

    # ---- the gate score projections of Eq. 4 (logits from q, k and W_GQ, W_GK) and their reverse: what it costs a step
    # whose logits are not handed in but computed inside the boundary ----
    scores = None
    if rank == 0 and cfg.backward and not args.generic:
        from paper_2602_01744_b200.inputs import make_gate_weights
        wq, wk = (w.cuda() for w in make_gate_weights(cfg, seed=99))
        sws = torch.empty(64 << 20, dtype=torch.uint8, device="cuda")
        lq_, lk_ = torch.empty_like(dev["gq_logits"]), torch.empty_like(dev["gk_logits"])
        tms = {}
        for name, fn in (("forward", lambda: api.sla_gate_scores_forward(plan, dev["q"], dev["k"], wq, wk, lq_, lk_)),
                         ("backward", lambda: api.sla_gate_scores_backward(plan, dev["q"], dev["k"], wq, wk, grads["dgq_logits"],
                                                                           grads["dgk_logits"], grads["dq"], grads["dk"], workspace=sws))):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            e0.record()
            for _ in range(20):
                fn()
            e1.record()
            torch.cuda.synchronize()
            tms[name] = e0.elapsed_time(e1) / 20
        pairs_ = cfg.B * cfg.T * cfg.H
        es = 2 if cfg.dtype == "bf16" else 4
        fb, bb = (2 * cfg.d_k * es + 8) * pairs_, (6 * cfg.d_k * es + 8) * pairs_
        hb, _ = measured_peaks()
        scores = {"what": "sla_gate_scores_forward / _backward on the workload's q, k (logits = per-head q, k through W [d_k,H])",
                  "forward_ms": tms["forward"], "backward_ms": tms["backward"],
                  "forward_hbm_frac": fb / (tms["forward"] * 1e-3) / 1e9 / hb, "backward_hbm_frac": bb / (tms["backward"] * 1e-3) / 1e9 / hb,
                  "algorithmic_bytes": {"forward": fb, "backward": bb},
                  "share_of_step": (tms["forward"] + tms["backward"]) / (ms / args.steps)}

    # ---- the output projection of Eq. 7 (y = Concat_h(o_h) W^O, d_model = H d_v) and its reverse: dense contractions, so
    # their roofline is the tensor core's ----
    out_proj = None
    if rank == 0 and cfg.dtype == "bf16" and not args.generic and not args.packed:
        from paper_2602_01744_b200.inputs import make_out_proj_inputs
        dm = cfg.H * cfg.d_v
        po, pw, pdy = (t.cuda() for t in make_out_proj_inputs(cfg, dm, seed=97))
        py = torch.empty_like(pdy)
        tms = {}
        for name, fn in (("forward", lambda: api.sla_out_proj_forward(plan, po, pw, y=py)),
                         ("backward", lambda: api.sla_out_proj_backward(plan, po, pw, pdy))):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            e0.record()
            for _ in range(20):
                fn()
            e1.record()
            torch.cuda.synchronize()
            tms[name] = e0.elapsed_time(e1) / 20
        flop = 2.0 * cfg.B * cfg.T * dm * dm                      # per product; the reverse pass runs two
        tb, tsus, tkind = measured_tensor_peaks()
        out_proj = {"what": "sla_out_proj_forward / _backward: [B*T, H*d_v] x [H*d_v, d_model] with d_model = H*d_v, bf16, fp32 accumulation",
                    "bound": "tensor", "forward_ms": tms["forward"], "backward_ms": tms["backward"],
                    "forward_tflops": flop / (tms["forward"] * 1e-3) / 1e12, "backward_tflops": 2 * flop / (tms["backward"] * 1e-3) / 1e12,
                    "peak": tb, "unit": "TFLOP/s", "peak_kind": f"bf16 burst, of {tkind}",
                    "forward_frac": flop / (tms["forward"] * 1e-3) / 1e12 / tb,
                    "backward_frac": 2 * flop / (tms["backward"] * 1e-3) / 1e12 / tb,
                    "flop": {"forward": flop, "backward": 2 * flop}}

    # ---- the feature map of the Gated-DeltaNet instantiation (short convolution, SiLU, L2 norm) and its reverse ----
    frontend = None
    if rank == 0 and cfg.variant == "gdn" and not args.generic:
        from paper_2602_01744_b200.inputs import make_frontend_inputs
        fe = {n: t.cuda() for n, t in make_frontend_inputs(cfg, 4, seed=98).items()}
        fws = torch.empty(64 << 20, dtype=torch.uint8, device="cuda")
        fout = torch.empty_like(fe["x_q"])
        tms = {}
        for name, fn in (("forward", lambda: api.sla_shortconv_forward(plan, fe["x_q"], fe["w_q"], True, out=fout)),
                         ("backward", lambda: api.sla_shortconv_backward(plan, fe["x_q"], fe["w_q"], fe["dout"], True, workspace=fws))):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            e0.record()
            for _ in range(20):
                fn()
            e1.record()
            torch.cuda.synchronize()
            tms[name] = e0.elapsed_time(e1) / 20
        nb = fe["x_q"].numel() * fe["x_q"].element_size()
        hb, _ = measured_peaks()
        frontend = {"what": "sla_shortconv_forward / _backward on one [B,T,H,d_k] tensor (K = 4, with L2 normalisation); a layer "
                            "applies it to q, k and v",
                    "forward_ms": tms["forward"], "backward_ms": tms["backward"],
                    "forward_hbm_frac": 2 * nb / (tms["forward"] * 1e-3) / 1e9 / hb,
                    "backward_hbm_frac": 3 * nb / (tms["backward"] * 1e-3) / 1e9 / hb,
                    "algorithmic_bytes": {"forward": 2 * nb, "backward": 3 * nb}}

    # ---- the decode step of the long-context configuration (C3): batch 64, fp32 state of 64 MiB, updated in place ----
    decode = None
    if rank == 0 and args.batch <= 0 and WORKLOAD == "C2":
        from paper_2602_01744_b200.inputs import C3_DECODE_BATCH, make_decode_inputs
        c3 = CONFIGS["C3"]
        dplan = api.sla_plan_create(c3.variant, c3.dtype, 1, 64, c3.H, c3.d_k, c3.d_v, c3.chunk)
        dec = {n: (None if t is None else t.cuda()) for n, t in make_decode_inputs(c3, C3_DECODE_BATCH, 8, seed=5).items()}
        # four independent 64 MiB states taken in turn: between two visits of one state 192 MiB of other states pass
        # through the 126 MB L2, so every step reads its state from HBM and its writes are evicted to HBM
        NSTATE = 4
        states = [torch.zeros((C3_DECODE_BATCH, c3.H, c3.d_k, c3.d_v), dtype=torch.float32, device="cuda")
                  for _ in range(NSTATE)]
        state = states[0]
        o_t = torch.empty((C3_DECODE_BATCH, c3.H, c3.d_v), dtype=torch.bfloat16, device="cuda")
        dsteps = 64

        def dstep(i):
            j = i % 8
            api.sla_decode_step(dplan, dec["q"][j], dec["k"][j], dec["v"][j], dec["log_decay"][j], dec["gq_logits"][j],
                                dec["gk_logits"][j], states[i % NSTATE], o_t=o_t)

        for i in range(8):
            dstep(i)
        torch.cuda.synchronize()
        e0.record()
        for i in range(dsteps):
            dstep(i)
        e1.record()
        torch.cuda.synchronize()
        us = 1e3 * e0.elapsed_time(e1) / dsteps
        dbytes = 2 * state.numel() * 4 + sum(dec[n][0].numel() * dec[n][0].element_size() for n in
                                             ("q", "k", "v", "log_decay", "gq_logits", "gk_logits")) + o_t.numel() * 2
        dpeak, _ = measured_peaks()
        decode = {"workload": f"C3 decode: batch {C3_DECODE_BATCH}, H={c3.H}, d={c3.d_k}, fp32 state updated in place",
                  "us_per_step": us, "tokens_per_s": C3_DECODE_BATCH / (us * 1e-6), "bound": "hbm",
                  "algorithmic_bytes_per_step": dbytes, "achieved": dbytes / (us * 1e-6) / 1e9, "peak": dpeak,
                  "unit": "GB/s", "frac": dbytes / (us * 1e-6) / 1e9 / dpeak,
                  "l2": f"{NSTATE} independent 64 MiB states visited in turn ({NSTATE * 64} MiB > 126 MB L2): no step "
                        "finds its state in L2",
                  "traffic": recorded_counters("C3_decode", "decode")}
        # a single sequence (1 MiB of state): launch bound, so the serving loop replays its steps as one CUDA graph
        s1 = torch.zeros((1, c3.H, c3.d_k, c3.d_v), dtype=torch.float32, device="cuda")
        o1 = torch.empty((1, c3.H, c3.d_v), dtype=torch.bfloat16, device="cuda")
        d1 = {n: (None if t is None else t[:, :1].contiguous()) for n, t in dec.items()}

        def steps1():
            for j in range(8):
                api.sla_decode_step(dplan, d1["q"][j], d1["k"][j], d1["v"][j], d1["log_decay"][j], d1["gq_logits"][j],
                                    d1["gk_logits"][j], s1, o_t=o1)

        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            steps1()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            steps1()
        timings = {}
        for name, fn in (("launched", steps1), ("graph", graph.replay)):
            fn()
            torch.cuda.synchronize()
            e0.record()
            for _ in range(16):
                fn()
            e1.record()
            torch.cuda.synchronize()
            timings[name] = 1e3 * e0.elapsed_time(e1) / (16 * 8)
        decode["batch_1"] = {"us_per_step_launched_one_by_one": timings["launched"],
                             "us_per_step_as_one_cuda_graph_of_8_steps": timings["graph"]}
        # multi-token decode (sla_decode_steps): n tokens per sequence per call, the state read and written once per call
        multi = {}
        for nt in (4, 16):
            md = make_decode_inputs(c3, C3_DECODE_BATCH, nt, seed=6)
            tm = lambda t: None if t is None else t.transpose(0, 1).contiguous().cuda()      # [batch, n, H, d]
            mq, mk, mv, mg, mlq, mlk = (tm(md[n]) for n in ("q", "k", "v", "log_decay", "gq_logits", "gk_logits"))
            mo = torch.empty((C3_DECODE_BATCH, nt, c3.H, c3.d_v), dtype=torch.bfloat16, device="cuda")
            row = {}
            for label, bsz in (("batch_64", C3_DECODE_BATCH), ("batch_1", 1)):
                sts = states if bsz > 1 else [st_[:1] for st_ in states]
                call = lambda i: api.sla_decode_steps(dplan, mq[:bsz], mk[:bsz], mv[:bsz], mg[:bsz], mlq[:bsz], mlk[:bsz],
                                                      sts[i % NSTATE], o=mo[:bsz])
                for i in range(4):
                    call(i)
                torch.cuda.synchronize()
                e0.record()
                for i in range(32):
                    call(i)
                e1.record()
                torch.cuda.synchronize()
                us_call = 1e3 * e0.elapsed_time(e1) / 32
                row[label] = {"us_per_call": us_call, "us_per_token": us_call / nt}
            multi[f"{nt}_tokens_per_call"] = row
        decode["multi_token"] = multi

    # ---- roofline of the dominant kernel, from the per-kernel CUDA events of the timed region ----
    peak, peak_kind = measured_peaks()
    roof = None
    if ktimes:
        top = max(ktimes, key=lambda k: ktimes[k][1])
        cnt, tot = ktimes[top]
        avg_ms = tot / cnt
        per_unit = (KERNEL_BYTES_RETNET if cfg.variant == "retnet" else KERNEL_BYTES).get(top)
        share = {k: round(v[1] / sum(t[1] for t in ktimes.values()), 4) for k, v in ktimes.items()}
        if per_unit is not None:
            alg = per_unit * cfg.B * cfg.T * cfg.H
            achieved = alg / (avg_ms * 1e-3) / 1e9
            roof = {"bound": "hbm", "kernel": top, "achieved": achieved, "peak": peak, "unit": "GB/s",
                    "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": recorded_traffic(WORKLOAD, top) if (args.batch <= 0 and saving) else None,
                    "algorithmic_bytes_per_launch": alg, "avg_launch_ms": avg_ms, "kernel_time_share": share}
        else:
            roof = {"bound": "hbm", "kernel": top, "achieved": None, "peak": peak, "unit": "GB/s", "frac": None,
                    "peak_kind": f"of {peak_kind}", "traffic": None, "avg_launch_ms": avg_ms,
                    "kernel_time_share": share}
    # whole-step figure against the same peak: all compulsory bytes of forward + backward / step time
    step_bytes = step_bytes_per_pair(cfg.variant, cfg.backward) * cfg.B * cfg.T * cfg.H
    step_gbs = step_bytes / (ms / args.steps * 1e-3) / 1e9

    # the tensor-core side of the metric: algorithmic MMA FLOP of a step / step time against the dense bf16 peaks.
    # The step is HBM-bound (66 FLOP/B against a ridge near 256), so the fraction it could reach at the HBM roofline
    # is stated beside it.
    tensor = None
    if cfg.variant in ("gla", "retnet") and cfg.d_k == 128 and cfg.d_v == 128 and not args.generic:
        pairs = cfg.B * cfg.T * cfg.H
        alg = GLA_FLOP["fwd_algorithmic"] + (GLA_FLOP["bwd_algorithmic"] if cfg.backward else 0)
        exe = GLA_FLOP["fwd_executed"] + ((GLA_FLOP["bwd_executed"] + (0 if saving else GLA_FLOP["state_recompute_executed"]))
                                          if cfg.backward else 0)
        burst, sustained, tkind = measured_tensor_peaks()
        sec = ms / args.steps * 1e-3
        tf_alg, tf_exe = alg * pairs / sec / 1e12, exe * pairs / sec / 1e12
        ceiling_s = step_bytes / (peak * 1e9)
        tensor = {"algorithmic_flop_per_step": alg * pairs, "executed_mma_flop_per_step": exe * pairs,
                  "achieved_tflops": tf_alg, "achieved_tflops_executed": tf_exe,
                  "peak_burst_tflops": burst, "peak_sustained_tflops": sustained, "peak_kind": f"of {tkind}",
                  "frac_of_burst": tf_alg / burst, "frac_of_sustained": tf_alg / sustained,
                  "frac_of_burst_executed": tf_exe / burst,
                  "hbm_bound_ceiling_frac_of_burst": alg * pairs / ceiling_s / 1e12 / burst,
                  "ncu_tensor_pipe_pct_of_elapsed": {k: recorded_counters(WORKLOAD, k, "tensor_pipe_pct_of_elapsed")
                                                     for k in ("gla_fwd_tc", "gla_bwd_tc")} if args.batch <= 0 else None}

    if rank == 0:
        cpu = None
        if world == 1 and not args.no_cpu_baseline and packed_cu is None:
            tokens, times, cores = cpu_oracle_sample(cfg, x, steps=1)
            cpu = {"value": tokens / times[0], "unit": UNIT, "cores": cores, "kind": "oracle",
                   "sample": f"first {min(CPU_ROWS, cfg.B)} batch rows of {WORKLOAD} (T={cfg.T}, H={cfg.H}), {passes}, "
                             f"{times[0]:.1f} s of fp64 recurrent oracle"}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD if args.batch <= 0 else f"{WORKLOAD} reduced to batch {cfg.B} (profiling only)",
                       "variant": cfg.variant, "B": cfg.B, "T": cfg.T, "H": cfg.H,
                       "d_k": cfg.d_k, "d_v": cfg.d_v, "chunk": cfg.chunk, "pass": passes,
                       "io": "bf16 q,k,v,o and gradients; fp32 decay, logits, state; fp32 accumulation",
                       "l2": f"inputs ({h2d / 1e9:.2f} GB per step) exceed the 126 MB L2; no flush needed",
                       "packed_sequences": None if packed_cu is None else len(packed_cu) - 1,
                       "parallelism": "replicas only" if world > 1 else "single GPU",
                       "kernels": "generic fp32 CUDA-core" if args.generic else "default",
                       "chunk_states": ("written by the forward pass of each step into the workspace, read by the backward "
                                        "pass of the same step" if saving else
                                        "recomputed by the backward pass" if cfg.backward else "not kept")},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps, "ms_per_step": ms_e2e / e2e_steps},
            "gpu_launches": n_launch,
            "roofline": roof,
            "tensor": tensor,
            "ms_per_step_with_kernel_events": ms_traced / args.steps,
            "step_hbm": {"algorithmic_bytes_per_step": step_bytes, "achieved_gbs": step_gbs, "frac": step_gbs / peak},
            "gate_scores": scores,
            "out_proj": out_proj,
            "gdn_feature_map": frontend,
            "decode_step": decode,
            "cpu_baseline": cpu,
        }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
