"""GPU parity of the Gated-DeltaNet feature map (short causal convolution, SiLU, per-head L2 normalisation) and of its
reverse pass against the oracle, alone and in front of the Softmax-GDN layer."""
import numpy as np
import pytest
import torch

from oracle import sla_oracle as orc
from paper_2602_01744_b200 import api
from paper_2602_01744_b200.inputs import CONFIGS, make_inputs, make_frontend_inputs, small
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,B,T,H,d,K", [("bf16", 2, 300, 16, 128, 4), ("bf16", 1, 67, 3, 48, 2), ("fp32", 2, 130, 5, 64, 4),
                                             ("fp32", 1, 1, 32, 128, 3), ("bf16", 3, 1000, 4, 16, 1), ("fp32", 1, 700, 2, 128, 4)])
@pytest.mark.parametrize("normalize", [True, False])
def test_feature_map_forward_and_backward(dtype, B, T, H, d, K, normalize):
    cfg = small(CONFIGS["C4"], B=B, T=T, H=H, d_k=d, d_v=d, dtype=dtype, seed=1200 + T)
    f = make_frontend_inputs(cfg, K, seed=1201)
    plan = api.sla_plan_create(cfg.variant, cfg.dtype, B, T, H, d, d, cfg.chunk)
    x, w, dout = f["x_q"].cuda(), f["w_q"].cuda(), f["dout"].cuda()
    out = api.sla_shortconv_forward(plan, x, w, normalize)
    dx, dw = api.sla_shortconv_backward(plan, x, w, dout, normalize)
    dx2, dw2 = api.sla_shortconv_backward(plan, x, w, dout, normalize)
    torch.cuda.synchronize()
    assert torch.equal(dw, dw2) and torch.equal(dx, dx2)
    ref = orc.shortconv(f["x_q"], f["w_q"], normalize)
    dx_ref, dw_ref = orc.shortconv_backward(f["x_q"], f["w_q"], f["dout"], normalize)
    tol, rtol = gu.TOL[dtype], gu.ROW_TOL[dtype]
    assert gu.rel_l2(out, ref) <= tol and gu.row_err(out, ref) <= rtol
    assert gu.rel_l2(dx, dx_ref) <= tol and gu.row_err(dx, dx_ref) <= rtol
    assert gu.rel_l2(dw, dw_ref) <= tol           # (fp32 sums of bf16-rounded inputs: well inside)


def test_feature_map_in_front_of_the_gdn_layer_end_to_end():
    """x -> conv/SiLU/norm -> Softmax-GDN training step -> reverse of the feature maps: gradients with respect to the raw
    inputs and the taps, against the oracle's chained sweeps (the GPU chain rounds q, k, v to bf16 between the stages,
    and so does the reference chain, stage by stage, on the same bits)."""
    cfg = small(CONFIGS["C4"], B=2, T=200, H=3, seed=1210)
    base = make_inputs(cfg, with_dO=True)
    f = make_frontend_inputs(cfg, 4, seed=1211)
    plan = api.sla_plan_create(cfg.variant, cfg.dtype, cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk, cfg.scale,
                               api.SLA_FLAG_SAVE_FOR_BACKWARD)
    dev = {n: t.cuda() for n, t in f.items()}
    q = api.sla_shortconv_forward(plan, dev["x_q"], dev["w_q"], True)
    k = api.sla_shortconv_forward(plan, dev["x_k"], dev["w_k"], True)
    v = api.sla_shortconv_forward(plan, dev["x_v"], dev["w_v"], False)
    b = gu.to_dev(base)
    ws = plan.workspace(backward=True)
    o, _ = api.sla_forward(plan, q, k, v, b["log_decay"], b["gq_logits"], b["gk_logits"], beta=b["beta"], workspace=ws)
    g = api.sla_backward(plan, q, k, v, b["log_decay"], b["gq_logits"], b["gk_logits"], b["dO"], beta=b["beta"], workspace=ws)
    dxq, dwq = api.sla_shortconv_backward(plan, dev["x_q"], dev["w_q"], g["dq"], True)
    dxk, dwk = api.sla_shortconv_backward(plan, dev["x_k"], dev["w_k"], g["dk"], True)
    dxv, dwv = api.sla_shortconv_backward(plan, dev["x_v"], dev["w_v"], g["dv"], False)
    torch.cuda.synchronize()
    plan.poll()
    # reference chain: every stage is the oracle on the bits the GPU stage received
    bf = lambda a: torch.from_numpy(a).to(torch.bfloat16)
    q_r, k_r, v_r = (bf(orc.shortconv(f[f"x_{n}"], f[f"w_{n}"], n != "v")) for n in "qkv")
    o_r, _ = orc.forward("gdn", q_r, k_r, v_r, base["log_decay"], base["gq_logits"], base["gk_logits"], beta=base["beta"])
    r = orc.backward("gdn", q_r, k_r, v_r, base["log_decay"], base["gq_logits"], base["gk_logits"], base["dO"], beta=base["beta"])
    pairs = {"q": (q, q_r.double().numpy()), "k": (k, k_r.double().numpy()), "o": (o, o_r)}
    for n, dxg, dwg in (("q", dxq, dwq), ("k", dxk, dwk), ("v", dxv, dwv)):
        dx_r, dw_r = orc.shortconv_backward(f[f"x_{n}"], f[f"w_{n}"], bf(r[f"d{n}"]), n != "v")
        pairs[f"dx_{n}"] = (dxg, dx_r)
        pairs[f"dw_{n}"] = (dwg, dw_r)
    gu.assert_close({n: gu.rel_l2(a, c) for n, (a, c) in pairs.items()},
                    {n: gu.row_err(a, c) for n, (a, c) in pairs.items()}, cfg.dtype, cfg)
