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
