"""GPU parity of the gate score projections (Eq. 4: logits = per-head q, k through W_GQ, W_GK in R^{d x H}) and of the
whole layer with projected gates - scores -> forward -> backward -> reverse of the scores - against the oracle."""
import numpy as np
import pytest
import torch

from oracle import sla_oracle as orc
from paper_2602_01744_b200 import api
from paper_2602_01744_b200.inputs import CONFIGS, make_inputs, make_gate_weights, small
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,B,T,H,d", [("bf16", 2, 200, 16, 128), ("bf16", 1, 67, 3, 48), ("fp32", 2, 130, 5, 64),
                                           ("fp32", 1, 1, 32, 128), ("bf16", 3, 1000, 4, 16)])
def test_scores_forward_and_backward_alone(dtype, B, T, H, d):
    cfg = small(CONFIGS["C2"], B=B, T=T, H=H, d_k=d, d_v=d, dtype=dtype, seed=1100 + T)
    xh = make_inputs(cfg, with_dO=False)
    wq, wk = make_gate_weights(cfg, seed=1101)
    plan = api.sla_plan_create(cfg.variant, cfg.dtype, B, T, H, d, d, cfg.chunk)
    x = gu.to_dev(xh)
    lq, lk = api.sla_gate_scores_forward(plan, x["q"], x["k"], wq.cuda(), wk.cuda())
    torch.cuda.synchronize()
    lq_ref, lk_ref = orc.gate_scores(xh["q"], wq), orc.gate_scores(xh["k"], wk)
    # fp32 accumulation of exactly representable products: far inside the I/O tolerance
    assert gu.rel_l2(lq, lq_ref) <= 1e-5 and gu.rel_l2(lk, lk_ref) <= 1e-5
    assert gu.row_err(lq, lq_ref) <= 1e-4 and gu.row_err(lk, lk_ref) <= 1e-4
    # reverse: random upstream logit gradients, dq / dk pre-filled (the call adds to them)
    gen = torch.Generator().manual_seed(1102)
    dlq, dlk = torch.randn(B, T, H, generator=gen), torch.randn(B, T, H, generator=gen)
    dq0 = torch.randn(B, T, H, d, generator=gen).to(x["q"].dtype)
    dk0 = torch.randn(B, T, H, d, generator=gen).to(x["q"].dtype)
    dq, dk = dq0.clone().cuda(), dk0.clone().cuda()
    dwq, dwk = api.sla_gate_scores_backward(plan, x["q"], x["k"], wq.cuda(), wk.cuda(), dlq.cuda(), dlk.cuda(), dq, dk)
    dwq2, dwk2 = api.sla_gate_scores_backward(plan, x["q"], x["k"], wq.cuda(), wk.cuda(), dlq.cuda(), dlk.cuda(),
                                              dq0.clone().cuda(), dk0.clone().cuda())
    torch.cuda.synchronize()
    assert torch.equal(dwq, dwq2) and torch.equal(dwk, dwk2)            # fixed summation order
    dq_ref = np.ascontiguousarray(dq0.double().numpy().copy())
    dk_ref = np.ascontiguousarray(dk0.double().numpy().copy())
    dwq_ref = orc.gate_scores_backward(xh["q"], wq, dlq, dq_ref)
    dwk_ref = orc.gate_scores_backward(xh["k"], wk, dlk, dk_ref)
    tol = gu.TOL[dtype]
    assert gu.rel_l2(dq, dq_ref) <= tol and gu.rel_l2(dk, dk_ref) <= tol
    assert gu.row_err(dq, dq_ref) <= gu.ROW_TOL[dtype] and gu.row_err(dk, dk_ref) <= gu.ROW_TOL[dtype]
    assert gu.rel_l2(dwq, dwq_ref) <= 1e-4 and gu.rel_l2(dwk, dwk_ref) <= 1e-4


@pytest.mark.parametrize("base,T,H", [("C2", 300, 4), ("C4", 200, 3), ("R2", 130, 16)])
def test_layer_with_projected_gates_end_to_end(base, T, H):
    """logits from the projections -> training step on the tensor-core kernels -> reverse of the projections; every
    gradient (q and k now carry both routes, plus dW_GQ, dW_GK) against the oracle's chained reverse sweeps."""
    cfg = small(CONFIGS[base], B=2, T=T, H=H, seed=1110 + T)
    xh = make_inputs(cfg, with_dO=True)
    wq, wk = make_gate_weights(cfg, seed=1111)
    x = gu.to_dev(xh)
    wqd, wkd = wq.cuda(), wk.cuda()
    plan = api.sla_plan_create(cfg.variant, cfg.dtype, cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk, cfg.scale,
                               api.SLA_FLAG_SAVE_FOR_BACKWARD)
    ws = plan.workspace(backward=True)
    lq, lk = api.sla_gate_scores_forward(plan, x["q"], x["k"], wqd, wkd)
    o, _ = api.sla_forward(plan, x["q"], x["k"], x["v"], x["log_decay"], lq, lk, beta=x["beta"], workspace=ws)
    g = api.sla_backward(plan, x["q"], x["k"], x["v"], x["log_decay"], lq, lk, x["dO"], beta=x["beta"], workspace=ws)
    dwq, dwk = api.sla_gate_scores_backward(plan, x["q"], x["k"], wqd, wkd, g["dgq_logits"], g["dgk_logits"],
                                            g["dq"], g["dk"])
    torch.cuda.synchronize()
    plan.poll()
    lq_ref, lk_ref = orc.gate_scores(xh["q"], wq), orc.gate_scores(xh["k"], wk)
    o_ref, _ = orc.forward(cfg.variant, xh["q"], xh["k"], xh["v"], xh["log_decay"], lq_ref, lk_ref, beta=xh["beta"],
                           scale=cfg.scale)
    r = orc.backward(cfg.variant, xh["q"], xh["k"], xh["v"], xh["log_decay"], lq_ref, lk_ref, xh["dO"], beta=xh["beta"],
                     scale=cfg.scale)
    dq_ref, dk_ref = np.ascontiguousarray(r["dq"].copy()), np.ascontiguousarray(r["dk"].copy())
    dwq_ref = orc.gate_scores_backward(xh["q"], wq, r["dlq"], dq_ref)
    dwk_ref = orc.gate_scores_backward(xh["k"], wk, r["dlk"], dk_ref)
    pairs = {"o": (o, o_ref), "dq": (g["dq"], dq_ref), "dk": (g["dk"], dk_ref), "dv": (g["dv"], r["dv"]),
             "dw_gq": (dwq, dwq_ref), "dw_gk": (dwk, dwk_ref)}
    gu.assert_close({n: gu.rel_l2(a, b) for n, (a, b) in pairs.items()},
                    {n: gu.row_err(a, b) for n, (a, b) in pairs.items()}, cfg.dtype, cfg)
