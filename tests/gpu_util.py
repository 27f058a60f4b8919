"""Helpers for the GPU parity tests: run the CUDA path through the C-ABI binding and the oracle on
the same seeded tensors, and compare per tensor by relative L2 error - once over the whole tensor (the stated
tolerance) and once row by row (so that a fault confined to one chunk, tail row or segment boundary cannot hide
in the global figure)."""
import numpy as np
import torch

from oracle import sla_oracle as orc
from paper_2602_01744_b200 import api
from paper_2602_01744_b200.inputs import make_inputs

TOL = {"bf16": 1e-2, "fp32": 1e-4}     # max relative L2 error per tensor (bf16 I/O / fp32 I/O)


def rel_l2(x, ref):
    x = x.detach().double().cpu().numpy() if hasattr(x, "detach") else np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.linalg.norm(ref)
    return float(np.linalg.norm(x - ref) / den) if den > 0 else float(np.abs(x).max())


# Per-row bound.  A row is a vector along the last axis (the d_k / d_v features of one (b, t, h), the H logits of one
# token, one state row).  Its error ||x_row - ref_row|| is measured against its own norm, or against the RMS row norm
# of the tensor where the row is smaller than that: every row is right to a few bf16 roundings at its own scale (the
# head gates make row norms heavy tailed - 15 to 25 times the RMS norm occur in the benchmark configurations - so an
# absolute bound would only bind on the largest rows), and a small row is right at the scale of a typical one.
# With operands and outputs rounded to bf16 (relative 2^-9 each, a handful of roundings per value) whole tensors sit at
# 3e-3..4e-3; single rows, over 10^5..10^6 of them, reach 1.5e-2 (o, dq, dk, dv) and 2.5e-2 (the logit, beta and decay
# gradients, which are sums with cancellation).  Four times the global tolerance bounds that with margin; a chunk, tail
# row or segment boundary that is off by more than a few per cent of its own size fails it.
ROW_TOL = {"bf16": 4e-2, "fp32": 4e-4}


def row_err(x, ref):
    """max over rows of ||x_row - ref_row|| / max(||ref_row||, rms_rows ||ref_row||); rows run along the last axis."""
    x = x.detach().double().cpu().numpy() if hasattr(x, "detach") else np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    if ref.size == 0:
        return 0.0
    x = x.reshape(-1, ref.shape[-1])
    r = ref.reshape(-1, ref.shape[-1])
    if not np.isfinite(x).all():
        return float("inf")
    norm = np.sqrt(np.sum(r * r, axis=1))
    rms = np.sqrt(np.mean(norm * norm))
    err = np.sqrt(np.sum((x - r) ** 2, axis=1))
    den = np.maximum(norm, rms)
    return float((err / den).max()) if rms > 0 else float(err.max())


def assert_close(errs_global, errs_row, dtype, what=""):
    tol, rtol = TOL[dtype], ROW_TOL[dtype]
    bad = {n: e for n, e in errs_global.items() if not (np.isfinite(e) and e <= tol)}
    bad_rows = {n: e for n, e in errs_row.items() if not (np.isfinite(e) and e <= rtol)}
    assert not bad and not bad_rows, (what, "global", bad, "worst row", bad_rows)


def to_dev(x):
    return {n: (None if t is None else t.cuda()) for n, t in x.items()}


def gpu_forward(cfg, x, h0=None, want_ht=True, flags=0):
    plan = api.sla_plan_create(cfg.variant, cfg.dtype, cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk,
                               cfg.scale, flags)
    ht = torch.empty((cfg.B, cfg.H, cfg.d_k, cfg.d_v), dtype=torch.float32, device="cuda") if want_ht else None
    o, ht = api.sla_forward(plan, x["q"], x["k"], x["v"], x["log_decay"], x["gq_logits"], x["gk_logits"],
                            beta=x["beta"], h0=h0, ht=ht)
    torch.cuda.synchronize()
    plan.poll()
    return o, ht, plan


def gpu_backward(cfg, x, h0=None, dht=None, want_dh0=False, flags=0):
    plan = api.sla_plan_create(cfg.variant, cfg.dtype, cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk,
                               cfg.scale, flags)
    g = api.sla_backward(plan, x["q"], x["k"], x["v"], x["log_decay"], x["gq_logits"], x["gk_logits"], x["dO"],
                         beta=x["beta"], h0=h0, dht=dht, want_dh0=want_dh0)
    torch.cuda.synchronize()
    plan.poll()
    return g, plan


def oracle_forward(cfg, x, h0=None, bsel=None):
    """Oracle on the same bits (optionally on a subset of batch rows: sequences are independent)."""
    s = (lambda t: t) if bsel is None else (lambda t: None if t is None else (t if t.dim() == 1 else t[bsel]))
    return orc.forward(cfg.variant, s(x["q"]), s(x["k"]), s(x["v"]), s(x["log_decay"]), s(x["gq_logits"]),
                       s(x["gk_logits"]), beta=s(x["beta"]), h0=s(h0) if h0 is not None else None,
                       scale=cfg.scale)


def oracle_backward(cfg, x, h0=None, dht=None, bsel=None):
    s = (lambda t: t) if bsel is None else (lambda t: None if t is None else (t if t.dim() == 1 else t[bsel]))
    return orc.backward(cfg.variant, s(x["q"]), s(x["k"]), s(x["v"]), s(x["log_decay"]), s(x["gq_logits"]),
                        s(x["gk_logits"]), s(x["dO"]), beta=s(x["beta"]),
                        h0=s(h0) if h0 is not None else None, dht=s(dht) if dht is not None else None,
                        scale=cfg.scale)


GRAD_NAMES = {"dq": "dq", "dk": "dk", "dv": "dv", "dlog_decay": "dlog_decay", "dbeta": "dbeta",
              "dgq_logits": "dlq", "dgk_logits": "dlk", "dh0": "dh0"}


def check_forward(cfg, with_h0=False, flags=0, bsel=None):
    x = make_inputs(cfg, with_dO=False, with_h0=with_h0)
    xd = to_dev(x)
    o, ht, _ = gpu_forward(cfg, xd, h0=xd.get("h0"), flags=flags)
    oref, htref = oracle_forward(cfg, x, h0=x.get("h0"), bsel=bsel)
    sel = slice(None) if bsel is None else bsel
    errs = {"o": rel_l2(o[sel], oref), "ht": rel_l2(ht[sel], htref)}
    rows = {"o": row_err(o[sel], oref), "ht": row_err(ht[sel], htref)}
    assert_close(errs, rows, cfg.dtype, cfg)
    return errs


def check_backward(cfg, with_h0=False, flags=0, bsel=None):
    x = make_inputs(cfg, with_dO=True, with_h0=with_h0)
    xd = to_dev(x)
    g, _ = gpu_backward(cfg, xd, h0=xd.get("h0"), dht=xd.get("dht"), want_dh0=with_h0, flags=flags)
    ref = oracle_backward(cfg, x, h0=x.get("h0"), dht=x.get("dht"), bsel=bsel)
    sel = slice(None) if bsel is None else bsel
    errs, rows = {}, {}
    for gname, rname in GRAD_NAMES.items():
        if g.get(gname) is None:
            continue
        t = g[gname][sel] if g[gname].dim() > 1 else g[gname]
        errs[gname] = rel_l2(t, ref[rname])
        rows[gname] = row_err(t, ref[rname])
    assert_close(errs, rows, cfg.dtype, cfg)
    return errs


def gpu_training_step(cfg, x, h0=None, dht=None, want_dh0=False):
    """Forward then backward on one SLA_FLAG_SAVE_FOR_BACKWARD plan and one workspace, as a training step runs them.
    Returns (o, ht, gradients, plan, launches of the forward, launches of the backward)."""
    plan = api.sla_plan_create(cfg.variant, cfg.dtype, cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk, cfg.scale,
                               api.SLA_FLAG_SAVE_FOR_BACKWARD)
    ws = plan.workspace(backward=True)
    ht = torch.empty((cfg.B, cfg.H, cfg.d_k, cfg.d_v), dtype=torch.float32, device="cuda")
    o, ht = api.sla_forward(plan, x["q"], x["k"], x["v"], x["log_decay"], x["gq_logits"], x["gk_logits"],
                            beta=x["beta"], h0=h0, ht=ht, workspace=ws)
    lf = plan.last_launch_count
    g = api.sla_backward(plan, x["q"], x["k"], x["v"], x["log_decay"], x["gq_logits"], x["gk_logits"], x["dO"],
                         beta=x["beta"], h0=h0, dht=dht, want_dh0=want_dh0, workspace=ws)
    lb = plan.last_launch_count
    torch.cuda.synchronize()
    plan.poll()
    return o, ht, g, plan, ws, lf, lb


def check_training_step(cfg, with_h0=False):
    """Parity of o, ht and every gradient when the backward reads what the forward left in the workspace."""
    x = make_inputs(cfg, with_dO=True, with_h0=with_h0)
    xd = to_dev(x)
    o, ht, g, plan, ws, lf, lb = gpu_training_step(cfg, xd, h0=xd.get("h0"), dht=xd.get("dht"), want_dh0=with_h0)
    oref, htref = oracle_forward(cfg, x, h0=x.get("h0"))
    ref = oracle_backward(cfg, x, h0=x.get("h0"), dht=x.get("dht"))
    errs = {"o": rel_l2(o, oref), "ht": rel_l2(ht, htref)}
    rows = {"o": row_err(o, oref), "ht": row_err(ht, htref)}
    for gname, rname in GRAD_NAMES.items():
        if g.get(gname) is not None:
            errs[gname] = rel_l2(g[gname], ref[rname])
            rows[gname] = row_err(g[gname], ref[rname])
    assert_close(errs, rows, cfg.dtype, cfg)
    return errs, lf, lb


class Guarded:
    """Device buffers carved out of one pattern-filled arena with guard bands on both sides of each, standing in
    for a memory checker: after the calls, `check()` asserts that not one guard byte changed."""
    GUARD = 1 << 16
    PATTERN = 0xA5

    def __init__(self, total_bytes):
        self.arena = torch.full((total_bytes,), self.PATTERN, dtype=torch.uint8, device="cuda")
        self.off = 0
        self.spans = []

    @classmethod
    def for_sizes(cls, sizes):
        return cls(sum(((n + 255) & ~255) + 2 * cls.GUARD for n in sizes) + 512)

    def take(self, nbytes, dtype=torch.uint8, shape=None, fill=None):
        base = self.arena.data_ptr()
        start = self.off + self.GUARD
        start += (-(base + start)) % 256                   # 256-byte aligned, as torch allocations are
        end = start + nbytes
        assert end + self.GUARD <= self.arena.numel()
        self.spans.append((start, end))
        self.off = end
        t = self.arena[start:end].view(dtype)
        if shape is not None:
            t = t.view(shape)
        if fill is not None:
            t.fill_(fill)
        return t

    def check(self):
        keep = torch.ones(self.arena.numel(), dtype=torch.bool, device="cuda")
        for a, b in self.spans:
            keep[a:b] = False
        touched = (self.arena != self.PATTERN) & keep
        n = int(touched.sum())
        where = int(torch.nonzero(touched)[0]) if n else -1
        assert n == 0, f"{n} bytes outside the buffers handed to the library were written (first at arena offset {where}; spans {self.spans})"
