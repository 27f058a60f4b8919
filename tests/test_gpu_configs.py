"""The five benchmark configurations at full size, in the launch configuration bench.py times
(default kernel selection, and for the training configurations the plan flags of the benchmark), against the
oracle on EVERY batch row (the oracle runs a few rows at a time to bound host memory: sequences are independent),
per tensor and per row."""
import numpy as np
import pytest
import torch

from oracle import sla_oracle as orc
from paper_2602_01744_b200 import api
from paper_2602_01744_b200.inputs import (C3_DECODE_BATCH, C3_DECODE_STEPS, CONFIGS, make_decode_inputs,
                                          make_inputs, small)
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def test_c0_retnet_fp32():
    errs = gu.check_forward(CONFIGS["C0"])
    assert max(errs.values()) <= 1e-4


def _all_rows(cfg, rows_per_pass):
    """One GPU pass over the whole configuration (a training step where it has a backward, as bench.py runs it), then
    the oracle over all batch rows, `rows_per_pass` at a time."""
    x = make_inputs(cfg)
    xd = gu.to_dev(x)
    if cfg.backward:
        o, ht, g, plan, ws, lf, lb = gu.gpu_training_step(cfg, xd)
        assert (lf, lb) == (1, 2)
    else:
        o, ht, plan = gu.gpu_forward(cfg, xd)
        g = {}
    worst, worst_row = {}, {}
    for b0 in range(0, cfg.B, rows_per_pass):
        sel = slice(b0, min(cfg.B, b0 + rows_per_pass))
        oref, htref = gu.oracle_forward(cfg, x, bsel=sel)
        pairs = {"o": (o[sel], oref), "ht": (ht[sel], htref)}
        if cfg.backward:
            ref = gu.oracle_backward(cfg, x, bsel=sel)
            for gname, rname in gu.GRAD_NAMES.items():
                if g.get(gname) is not None:
                    pairs[gname] = (g[gname][sel], ref[rname])
        errs = {n: gu.rel_l2(a, r) for n, (a, r) in pairs.items()}
        rows = {n: gu.row_err(a, r) for n, (a, r) in pairs.items()}
        gu.assert_close(errs, rows, cfg.dtype, (cfg.name, "batch rows", sel))
        for n in errs:
            worst[n] = max(worst.get(n, 0.0), errs[n])
            worst_row[n] = max(worst_row.get(n, 0.0), rows[n])
    print(cfg.name, "worst relative L2 per tensor:", {n: f"{e:.2e}" for n, e in worst.items()})
    print(cfg.name, "worst row:", {n: f"{e:.2e}" for n, e in worst_row.items()})


def test_c1_gla_forward_full_size_every_row():
    _all_rows(CONFIGS["C1"], 4)


def test_c2_gla_forward_backward_full_size_every_row():
    _all_rows(CONFIGS["C2"], 2)


def test_c4_gdn_forward_backward_full_size_every_row():
    _all_rows(CONFIGS["C4"], 2)


def test_r2_retnet_forward_backward_full_size_every_row():
    _all_rows(CONFIGS["R2"], 2)


def test_c3_long_context_prefill_then_decode():
    cfg = CONFIGS["C3"]
    tol = gu.TOL[cfg.dtype]
    x = make_inputs(cfg, with_dO=False)
    xd = gu.to_dev(x)
    o, ht, plan = gu.gpu_forward(cfg, xd)
    oref, htref = gu.oracle_forward(cfg, x)
    assert gu.rel_l2(o, oref) <= tol
    assert gu.rel_l2(ht, htref) <= tol
    # row by row: covers the tokens on both sides of every segment boundary of the segmented forward
    assert gu.row_err(o, oref) <= gu.ROW_TOL[cfg.dtype]
    assert gu.row_err(ht, htref) <= gu.ROW_TOL[cfg.dtype]
    # split-sequence property at full size: forward(T1) -> ht -> forward(T2, h0 = ht)
    T1 = 40000 - 40000 % cfg.chunk + 17                 # an uneven cut: ragged chunk on both sides
    parts = []
    state = None
    for sl in (slice(0, T1), slice(T1, cfg.T)):
        sub = {n: (None if t is None else t[:, sl].contiguous()) for n, t in xd.items()}
        c = small(cfg, T=sl.stop - sl.start)
        o_p, state, _ = gu.gpu_forward(c, sub, h0=state)
        parts.append(o_p)
    assert gu.rel_l2(torch.cat(parts, 1), oref) <= tol
    assert gu.row_err(torch.cat(parts, 1), oref) <= gu.ROW_TOL[cfg.dtype]
    assert gu.rel_l2(state, htref) <= tol

    # decode: the final state replicated into 64 slots, each continuing with its own tokens
    Bd, steps = C3_DECODE_BATCH, C3_DECODE_STEPS
    dec = make_decode_inputs(cfg, Bd, steps, seed=33)
    state = ht.expand(Bd, -1, -1, -1).contiguous()
    ref_state = np.ascontiguousarray(np.broadcast_to(htref, (Bd,) + htref.shape[1:]).copy())
    dd = {n: (None if t is None else t.cuda()) for n, t in dec.items()}
    outs = torch.empty((steps, Bd, cfg.H, cfg.d_v), dtype=torch.bfloat16, device="cuda")
    refs = np.empty((steps, Bd, cfg.H, cfg.d_v))
    for t in range(steps):
        api.sla_decode_step(plan, dd["q"][t], dd["k"][t], dd["v"][t], dd["log_decay"][t], dd["gq_logits"][t],
                            dd["gk_logits"][t], state, o_t=outs[t])
        refs[t] = orc.decode_step("gla", dec["q"][t], dec["k"][t], dec["v"][t], dec["log_decay"][t],
                                  dec["gq_logits"][t], dec["gk_logits"][t], ref_state)
    torch.cuda.synchronize()
    assert gu.rel_l2(outs, refs) <= tol
    assert gu.row_err(outs, refs) <= gu.ROW_TOL[cfg.dtype]
    assert gu.rel_l2(state, ref_state) <= tol
    # the same continuation through the chunkwise kernels with h0 = replicated prefill state
    tr = lambda t: t.transpose(0, 1).contiguous()
    cdec = small(cfg, B=Bd, T=steps)
    xdec = dict(q=tr(dd["q"]), k=tr(dd["k"]), v=tr(dd["v"]), log_decay=tr(dd["log_decay"]), beta=None,
                gq_logits=tr(dd["gq_logits"]), gk_logits=tr(dd["gk_logits"]))
    o2, ht2, _ = gu.gpu_forward(cdec, xdec, h0=ht.expand(Bd, -1, -1, -1).contiguous())
    assert gu.rel_l2(o2, refs.transpose(1, 0, 2, 3)) <= tol
    assert gu.rel_l2(ht2, ref_state) <= tol
    # slot 0 against one chunkwise pass over the concatenated 65536 + 256 tokens
    cat = {n: torch.cat([xd[n], xdec[n][0:1]], 1) for n in ("q", "k", "v", "log_decay", "gq_logits", "gk_logits")}
    cat["beta"] = None
    o3, _, _ = gu.gpu_forward(small(cfg, T=cfg.T + steps), cat)
    assert gu.rel_l2(o3[0, cfg.T:], refs[:, 0]) <= tol
