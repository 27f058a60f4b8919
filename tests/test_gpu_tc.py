"""GPU parity of the tcgen05/TMEM/TMA Softmax-GLA and Softmax-GatedDeltaNet kernels (bf16, d_k = d_v = 128, chunk 64) against
the fp64 oracle, through the C ABI with default kernel selection."""
import pytest
import torch

from paper_2602_01744_b200 import api
from paper_2602_01744_b200.inputs import CONFIGS, make_inputs, small
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("B,T,H,with_h0", [(1, 64, 1, False), (2, 200, 3, True), (1, 1000, 16, True), (3, 65, 4, False),
                                           (1, 1297, 2, True), (2, 2048, 4, False)])    # the last two run segmented
def test_gla_forward_tc(B, T, H, with_h0):
    cfg = small(CONFIGS["C1"], B=B, T=T, H=H, seed=300 + T)
    errs = gu.check_forward(cfg, with_h0=with_h0)
    assert max(errs.values()) <= 1e-2


def test_gla_forward_tc_is_the_path_taken_and_agrees_with_generic():
    cfg = small(CONFIGS["C1"], B=2, T=300, H=4, seed=310, scale=0.5)
    x = gu.to_dev(make_inputs(cfg, with_h0=True))
    o1, ht1, plan = gu.gpu_forward(cfg, x, h0=x["h0"])
    assert plan.last_launch_count == 1                 # the fused kernel (a short batch: one CTA per sequence)
    o2, ht2, plan2 = gu.gpu_forward(cfg, x, h0=x["h0"], flags=api.SLA_FLAG_FORCE_GENERIC)
    assert plan2.last_launch_count > 1
    assert gu.rel_l2(o1, o2.double().cpu().numpy()) <= 1e-2
    assert gu.rel_l2(ht1, ht2.double().cpu().numpy()) <= 1e-2


@pytest.mark.parametrize("B,T,H,with_h0", [(1, 64, 1, False), (1, 128, 2, False), (2, 200, 3, True), (1, 1000, 16, True),
                                           (3, 65, 4, True)])
def test_gla_backward_tc(B, T, H, with_h0):
    cfg = small(CONFIGS["C2"], B=B, T=T, H=H, seed=400 + T)
    errs = gu.check_backward(cfg, with_h0=with_h0)
    assert max(errs.values()) <= 1e-2


def test_gla_backward_tc_is_the_path_taken_and_agrees_with_generic():
    cfg = small(CONFIGS["C2"], B=2, T=300, H=4, seed=410, scale=0.5)
    x = gu.to_dev(make_inputs(cfg, with_dO=True, with_h0=True))
    g1, plan = gu.gpu_backward(cfg, x, h0=x["h0"], dht=x["dht"], want_dh0=True)
    assert plan.last_launch_count == 3                 # state sweep, gradient sweep, gate softmax backward
    g2, plan2 = gu.gpu_backward(cfg, x, h0=x["h0"], dht=x["dht"], want_dh0=True, flags=api.SLA_FLAG_FORCE_GENERIC)
    assert plan2.last_launch_count > 3
    for name in ("dq", "dk", "dv", "dlog_decay", "dgq_logits", "dgk_logits", "dh0"):
        assert gu.rel_l2(g1[name], g2[name].double().cpu().numpy()) <= 1e-2, name


@pytest.mark.parametrize("B,T,H,with_h0", [(1, 64, 1, False), (2, 200, 3, True), (1, 1000, 16, True), (3, 65, 4, True)])
def test_gdn_forward_tc(B, T, H, with_h0):
    cfg = small(CONFIGS["C4"], B=B, T=T, H=H, seed=500 + T, backward=False)
    errs = gu.check_forward(cfg, with_h0=with_h0)
    assert max(errs.values()) <= 1e-2


def test_gdn_forward_tc_is_the_path_taken_and_agrees_with_generic():
    cfg = small(CONFIGS["C4"], B=2, T=300, H=4, seed=510, scale=0.5, backward=False)
    x = gu.to_dev(make_inputs(cfg, with_h0=True))
    o1, ht1, plan = gu.gpu_forward(cfg, x, h0=x["h0"])
    assert plan.last_launch_count == 1 and plan.forward_workspace_bytes == 0
    o2, ht2, plan2 = gu.gpu_forward(cfg, x, h0=x["h0"], flags=api.SLA_FLAG_FORCE_GENERIC)
    assert plan2.last_launch_count > 1
    assert gu.rel_l2(o1, o2.double().cpu().numpy()) <= 1e-2
    assert gu.rel_l2(ht1, ht2.double().cpu().numpy()) <= 1e-2


@pytest.mark.parametrize("B,T,H,with_h0", [(1, 64, 1, False), (1, 128, 2, False), (2, 200, 3, True), (1, 1000, 16, True),
                                           (3, 65, 4, True)])
def test_gdn_backward_tc(B, T, H, with_h0):
    cfg = small(CONFIGS["C4"], B=B, T=T, H=H, seed=600 + T)
    errs = gu.check_backward(cfg, with_h0=with_h0)
    assert max(errs.values()) <= 1e-2


def test_gdn_backward_tc_is_the_path_taken_and_agrees_with_generic():
    cfg = small(CONFIGS["C4"], B=2, T=300, H=4, seed=610, scale=0.5)
    x = gu.to_dev(make_inputs(cfg, with_dO=True, with_h0=True))
    g1, plan = gu.gpu_backward(cfg, x, h0=x["h0"], dht=x["dht"], want_dh0=True)
    assert plan.last_launch_count == 3                 # forward sweep in save mode, gradient sweep, gate softmax backward
    g2, plan2 = gu.gpu_backward(cfg, x, h0=x["h0"], dht=x["dht"], want_dh0=True, flags=api.SLA_FLAG_FORCE_GENERIC)
    assert plan2.last_launch_count > 3
    for name in ("dq", "dk", "dv", "dlog_decay", "dbeta", "dgq_logits", "dgk_logits", "dh0"):
        assert gu.rel_l2(g1[name], g2[name].double().cpu().numpy()) <= 1e-2, name


@pytest.mark.parametrize("base", ["C2", "C4"])
@pytest.mark.parametrize("T", [1, 5, 193])
def test_tc_paths_on_very_short_and_ragged_sequences(base, T):
    cfg = small(CONFIGS[base], B=2, T=T, H=2, seed=700 + T)
    assert max(gu.check_forward(small(cfg, backward=False), with_h0=True).values()) <= 1e-2
    assert max(gu.check_backward(cfg, with_h0=True).values()) <= 1e-2


def test_tc_paths_with_thirty_two_heads():
    for base in ("C2", "C4"):
        cfg = small(CONFIGS[base], B=1, T=130, H=32, seed=720)
        assert max(gu.check_forward(small(cfg, backward=False)).values()) <= 1e-2
        assert max(gu.check_backward(cfg).values()) <= 1e-2
