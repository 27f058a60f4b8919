"""Serving hand-off: a chunkwise prefill leaves the state, then a run of recurrent decode steps replays as ONE CUDA
graph (decode at small batch is launch bound: a step moves only batch * H * 64 KiB).  The replayed steps must equal the
same steps launched one by one, and the oracle."""
import numpy as np
import pytest
import torch

from oracle import sla_oracle as orc
from paper_2602_01744_b200 import api
from paper_2602_01744_b200.inputs import CONFIGS, make_decode_inputs, make_inputs, small
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("base", ["C1", "C4"])
def test_prefill_then_graphed_decode(base):
    cfg = small(CONFIGS[base], B=2, T=256, H=4, seed=940)
    steps = 12
    x = make_inputs(cfg)
    xd = gu.to_dev(x)
    o, ht, plan = gu.gpu_forward(cfg, xd)                       # prefill through the tensor-core path
    oref, htref = gu.oracle_forward(cfg, x)
    assert gu.rel_l2(ht, htref) <= 1e-2
    dec = make_decode_inputs(cfg, cfg.B, steps, seed=941)
    dd = {n: (None if t is None else t.cuda()) for n, t in dec.items()}
    outs = torch.empty((steps, cfg.B, cfg.H, cfg.d_v), dtype=o.dtype, device="cuda")

    def run_steps(state, out):
        for t in range(steps):
            api.sla_decode_step(plan, dd["q"][t], dd["k"][t], dd["v"][t], dd["log_decay"][t], dd["gq_logits"][t],
                                dd["gk_logits"][t], state, beta_t=None if dd["beta"] is None else dd["beta"][t],
                                o_t=out[t])

    # one by one
    state_eager = ht.clone()
    run_steps(state_eager, outs)
    torch.cuda.synchronize()
    eager = outs.clone()
    # captured once, replayed on a fresh copy of the prefill state
    state_graph = ht.clone()
    outs.zero_()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        run_steps(state_graph, outs)                            # warm-up on the capture stream
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    state_graph.copy_(ht)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        run_steps(state_graph, outs)
    state_graph.copy_(ht)
    outs.zero_()
    graph.replay()
    torch.cuda.synchronize()
    plan.poll()
    assert torch.equal(outs, eager) and torch.equal(state_graph, state_eager)
    # and the oracle, continuing from its own prefill state
    ref_state = np.ascontiguousarray(htref.copy())
    refs = [orc.decode_step(cfg.variant, dec["q"][t], dec["k"][t], dec["v"][t], dec["log_decay"][t], dec["gq_logits"][t],
                            dec["gk_logits"][t], ref_state, beta_t=None if dec["beta"] is None else dec["beta"][t])
            for t in range(steps)]
    assert gu.rel_l2(outs, np.stack(refs)) <= 1e-2
    assert gu.rel_l2(state_graph, ref_state) <= 1e-2


@pytest.mark.parametrize("variant,dtype", [("retnet", "fp32"), ("gla", "bf16"), ("gdn", "bf16"), ("gla", "fp32")])
@pytest.mark.parametrize("n_tok", [2, 5, 16])
def test_multi_token_decode_equals_single_steps_bit_for_bit_and_the_oracle(variant, dtype, n_tok):
    """sla_decode_steps keeps the state in registers over n tokens; it must give the bits of n sla_decode_step calls
    (outputs and state) and match the oracle's n recurrent steps."""
    base = {"retnet": CONFIGS["C0"], "gla": CONFIGS["C1"], "gdn": CONFIGS["C4"]}[variant]
    d = 128 if dtype == "bf16" else 48
    cfg = small(base, B=4, T=n_tok, H=4, d_k=d, d_v=d, dtype=dtype, seed=960)   # (B*H*4 bytes per step: slices stay 16-byte aligned)
    dec = make_decode_inputs(cfg, cfg.B, n_tok, seed=961)          # [n, B, H, d]
    h0 = torch.randn(cfg.B, cfg.H, cfg.d_k, cfg.d_v, generator=torch.Generator().manual_seed(8)) * 0.1
    plan = api.sla_plan_create(cfg.variant, cfg.dtype, cfg.B, 64, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk, 0.9)
    dd = {n: (None if t is None else t.cuda()) for n, t in dec.items()}
    s1 = h0.clone().cuda()
    outs = []
    for t in range(n_tok):
        ld = dd["log_decay"] if variant == "retnet" else dd["log_decay"][t]
        outs.append(api.sla_decode_step(plan, dd["q"][t], dd["k"][t], dd["v"][t], ld, dd["gq_logits"][t],
                                        dd["gk_logits"][t], s1, beta_t=None if dd["beta"] is None else dd["beta"][t]))
    tm = lambda t: None if t is None else t.transpose(0, 1).contiguous()     # token-major per sequence: [B, n, H, d]
    s2 = h0.clone().cuda()
    ld = dd["log_decay"] if variant == "retnet" else tm(dd["log_decay"])
    o2 = api.sla_decode_steps(plan, tm(dd["q"]), tm(dd["k"]), tm(dd["v"]), ld, tm(dd["gq_logits"]), tm(dd["gk_logits"]),
                              s2, beta=tm(dd["beta"]))
    torch.cuda.synchronize()
    assert plan.last_launch_count == 1
    assert torch.equal(o2, torch.stack(outs, 1)) and torch.equal(s1, s2)
    ref_state = np.ascontiguousarray(h0.double().numpy().copy())
    cm = lambda t: None if t is None else t.transpose(0, 1).contiguous()
    oref = orc.decode_steps(variant, cm(dec["q"]), cm(dec["k"]), cm(dec["v"]),
                            dec["log_decay"] if variant == "retnet" else cm(dec["log_decay"]), cm(dec["gq_logits"]),
                            cm(dec["gk_logits"]), ref_state, beta=cm(dec["beta"]), scale=0.9)
    tol = gu.TOL[dtype]
    assert gu.rel_l2(o2, oref) <= tol and gu.row_err(o2, oref) <= gu.ROW_TOL[dtype]
    assert gu.rel_l2(s2, ref_state) <= tol
