"""GPU parity of the output projection (Eq. 7: y = Concat_h(o_h) W^O) and its reverse - three dense bf16 contractions
on the tensor cores - against the oracle: small shapes that span several 128 x 256 tiles with ragged tails in every
dimension, and the benchmark configuration on sampled rows and columns."""
import numpy as np
import pytest
import torch

from oracle import sla_oracle as orc
from paper_2602_01744_b200 import api
from paper_2602_01744_b200.inputs import CONFIGS, make_out_proj_inputs, small
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

# fp32 accumulation of bf16 products, one rounding to bf16 at the end: y and d_o sit at 2^-9 relative per value;
# dw_o leaves in fp32 (only its operands are rounded), so it is held to 1e-4 like the other weight gradients.
TOL_DW = 1e-4


def run_case(B, T, H, dv, dm, seed):
    cfg = small(CONFIGS["C2"], B=B, T=T, H=H, d_k=dv, d_v=dv, seed=seed)
    o, w, dy = make_out_proj_inputs(cfg, dm, seed=seed + 1)
    plan = api.sla_plan_create(cfg.variant, cfg.dtype, B, T, H, dv, dv, cfg.chunk)
    od, wd, dyd = o.cuda(), w.cuda(), dy.cuda()
    y = api.sla_out_proj_forward(plan, od, wd)
    d_o, dw = api.sla_out_proj_backward(plan, od, wd, dyd)
    d_o2, dw2 = api.sla_out_proj_backward(plan, od, wd, dyd)
    torch.cuda.synchronize()
    plan.poll()
    assert torch.equal(dw, dw2) and torch.equal(d_o, d_o2)                 # fixed summation order
    o2 = o.reshape(B, T, H * dv)
    y_ref = orc.out_proj(o2, w)
    do_ref, dw_ref = orc.out_proj_backward(o2, w, dy)
    errs = {"y": gu.rel_l2(y, y_ref), "d_o": gu.rel_l2(d_o.reshape(B, T, H * dv), do_ref)}
    rows = {"y": gu.row_err(y, y_ref), "d_o": gu.row_err(d_o.reshape(B, T, H * dv), do_ref)}
    gu.assert_close(errs, rows, "bf16", (B, T, H, dv, dm))
    assert gu.rel_l2(dw, dw_ref) <= TOL_DW and gu.row_err(dw, dw_ref) <= 4 * TOL_DW, (gu.rel_l2(dw, dw_ref), gu.row_err(dw, dw_ref))
    return errs


@pytest.mark.parametrize("B,T,H,dv,dm", [
    (2, 200, 4, 64, 328),       # 400 tokens (3.1 row tiles), K = 256, 1.3 column tiles
    (1, 67, 3, 48, 72),         # everything smaller than a tile; K = 144 is 2.25 contraction blocks
    (3, 129, 16, 128, 520),     # K = 2048 (the benchmark's), 387 tokens, 2.03 column tiles
    (1, 1, 2, 16, 8),           # one token, the smallest widths
    (2, 1024, 2, 128, 256),     # exact multiples of every tile size
])
def test_against_oracle(B, T, H, dv, dm):
    run_case(B, T, H, dv, dm, seed=1300 + T)


def test_benchmark_size_on_samples():
    cfg = CONFIGS["C2"]
    dm = cfg.H * cfg.d_v
    o, w, dy = make_out_proj_inputs(cfg, dm, seed=1350)
    plan = api.sla_plan_create(cfg.variant, cfg.dtype, cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk)
    od, wd, dyd = o.cuda(), w.cuda(), dy.cuda()
    y = api.sla_out_proj_forward(plan, od, wd)
    d_o, dw = api.sla_out_proj_backward(plan, od, wd, dyd)
    torch.cuda.synchronize()
    plan.poll()
    K = cfg.H * cfg.d_v
    o2, dy2 = o.reshape(-1, K), dy.reshape(-1, dm)
    rng = np.random.default_rng(1351)
    # token rows: the first and last of the tensor, tile edges, and a random sample
    rows = np.unique(np.concatenate([[0, 127, 128, 255, 256, o2.shape[0] - 129, o2.shape[0] - 128, o2.shape[0] - 1],
                                     rng.integers(0, o2.shape[0], 500)]))
    y_ref = orc.out_proj(o2[rows], w)
    do_ref, _ = orc.out_proj_backward(o2[rows], w, dy2[rows])
    yg, dog = y.reshape(-1, dm)[rows], d_o.reshape(-1, K)[rows]
    gu.assert_close({"y": gu.rel_l2(yg, y_ref), "d_o": gu.rel_l2(dog, do_ref)},
                    {"y": gu.row_err(yg, y_ref), "d_o": gu.row_err(dog, do_ref)}, "bf16", "C2 sampled rows")
    # rows of dw_o (features c): each is a sum over all 32768 tokens
    feats = np.unique(np.concatenate([[0, 127, 128, K - 1], rng.integers(0, K, 28)]))
    _, dw_ref = orc.out_proj_backward(o2[:, feats], w[feats], dy2)
    assert gu.rel_l2(dw[feats], dw_ref) <= TOL_DW and gu.row_err(dw[feats], dw_ref) <= 4 * TOL_DW


def test_refusals():
    plan32 = api.sla_plan_create("gla", "fp32", 1, 64, 2, 64, 64, 64)
    o = torch.zeros(1, 64, 2, 64, device="cuda")
    w = torch.zeros(128, 64, device="cuda")
    with pytest.raises(api.SLAError):                       # fp32 plans have no tensor-core projection
        api.sla_out_proj_forward(plan32, o, w)
    plan = api.sla_plan_create("gla", "bf16", 1, 64, 2, 64, 64, 64)
    with pytest.raises(api.SLAError):                       # d_model must be a multiple of 8
        api.sla_out_proj_forward(plan, o.bfloat16(), torch.zeros(128, 12, device="cuda", dtype=torch.bfloat16))


@pytest.mark.parametrize("base,T,H", [("C2", 200, 4), ("C4", 130, 3)])
def test_layer_followed_by_the_projection(base, T, H):
    """sla_forward -> output projection, and back: dy -> d_o -> sla_backward.  The oracle runs the same chain in fp64
    (on the GPU's bf16 o, and its bf16 d_o, where the GPU rounds them: those are tensors of the interface)."""
    from paper_2602_01744_b200.inputs import make_inputs
    cfg = small(CONFIGS[base], B=2, T=T, H=H, seed=1360 + T)
    xh = make_inputs(cfg, with_dO=False)
    dm = 264
    _, w, dy = make_out_proj_inputs(cfg, dm, seed=1361)
    x = gu.to_dev(xh)
    plan = api.sla_plan_create(cfg.variant, cfg.dtype, cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk, cfg.scale)
    o, _ = api.sla_forward(plan, x["q"], x["k"], x["v"], x["log_decay"], x["gq_logits"], x["gk_logits"], beta=x["beta"])
    y = api.sla_out_proj_forward(plan, o, w.cuda())
    d_o, dw = api.sla_out_proj_backward(plan, o, w.cuda(), dy.cuda())
    g = api.sla_backward(plan, x["q"], x["k"], x["v"], x["log_decay"], x["gq_logits"], x["gk_logits"], d_o, beta=x["beta"])
    torch.cuda.synchronize()
    plan.poll()
    K = cfg.H * cfg.d_v
    o_ref, _ = orc.forward(cfg.variant, xh["q"], xh["k"], xh["v"], xh["log_decay"], xh["gq_logits"], xh["gk_logits"],
                           beta=xh["beta"], scale=cfg.scale)
    y_ref = orc.out_proj(o_ref.reshape(cfg.B, cfg.T, K), w)
    do_ref, dw_ref = orc.out_proj_backward(o_ref.reshape(cfg.B, cfg.T, K), w, dy)
    g_ref = orc.backward(cfg.variant, xh["q"], xh["k"], xh["v"], xh["log_decay"], xh["gq_logits"], xh["gk_logits"],
                         do_ref.reshape(cfg.B, cfg.T, cfg.H, cfg.d_v), beta=xh["beta"], scale=cfg.scale)
    names = {"dq": "dq", "dk": "dk", "dv": "dv"}
    errs = {"y": gu.rel_l2(y, y_ref), "d_o": gu.rel_l2(d_o.reshape(cfg.B, cfg.T, K), do_ref)}
    rows = {"y": gu.row_err(y, y_ref), "d_o": gu.row_err(d_o.reshape(cfg.B, cfg.T, K), do_ref)}
    for n, r in names.items():
        errs[n], rows[n] = gu.rel_l2(g[n], g_ref[r]), gu.row_err(g[n], g_ref[r])
    gu.assert_close(errs, rows, "bf16", (base, T, H))
    # dw_o is fed by the GPU's o (bf16-rounded, itself within 1e-2 of the oracle's): the chain carries that error
    assert gu.rel_l2(dw, dw_ref) <= gu.TOL["bf16"]
