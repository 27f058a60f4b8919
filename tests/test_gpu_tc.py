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


@pytest.mark.parametrize("base", ["C2", "C4"])
@pytest.mark.parametrize("B,T,H,with_h0", [(1, 64, 1, False), (2, 200, 3, True), (1, 960, 8, True), (3, 65, 4, True), (1, 5, 2, False)])
def test_training_step_backward_reads_what_the_forward_left(base, B, T, H, with_h0):
    cfg = small(CONFIGS[base], B=B, T=T, H=H, seed=900 + T)
    errs, lf, lb = gu.check_training_step(cfg, with_h0=with_h0)
    assert (lf, lb) == (1, 2)                          # no state sweep (GLA) / no forward recomputation (GDN) in the backward
    assert max(errs.values()) <= 1e-2


@pytest.mark.parametrize("base", ["C2", "C4"])
def test_saved_states_are_used_only_for_the_same_inputs_and_never_change_the_result(base):
    cfg = small(CONFIGS[base], B=2, T=300, H=4, seed=910)
    x = gu.to_dev(make_inputs(cfg, with_dO=True))
    o, ht, g, plan, ws, lf, lb = gu.gpu_training_step(cfg, x)
    args = (x["q"], x["k"], x["v"], x["log_decay"], x["gq_logits"], x["gk_logits"], x["dO"])
    # another workspace: nothing was left there, so the backward recomputes (3 launches) and gives the same bits
    g2 = api.sla_backward(plan, *args, beta=x["beta"])
    assert plan.last_launch_count == 3
    # other inputs (a copy of k at another address) with the forward's workspace: recomputed as well
    k2 = x["k"].clone()
    g3 = api.sla_backward(plan, x["q"], k2, *args[2:], beta=x["beta"], workspace=ws)
    assert plan.last_launch_count == 3
    # a plan without the flag leaves nothing and asks for no forward workspace beyond its own
    plain = api.sla_plan_create(cfg.variant, cfg.dtype, cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk, cfg.scale)
    assert plain.forward_workspace_bytes == 0 and plan.forward_workspace_bytes == plan.backward_workspace_bytes
    api.sla_forward(plain, *args[:6], beta=x["beta"], workspace=ws)
    g4 = api.sla_backward(plain, *args, beta=x["beta"], workspace=ws)
    assert plain.last_launch_count == 3
    torch.cuda.synchronize()
    for other in (g2, g3, g4):
        for n, t in g.items():
            if t is not None:
                assert torch.equal(t, other[n]), n


def test_segmented_forward_leaves_nothing_and_the_backward_recomputes():
    cfg = small(CONFIGS["C2"], B=1, T=2048, H=4, seed=920)     # few long sequences: the forward runs in segments
    errs, lf, lb = gu.check_training_step(cfg)
    assert lf == 2 and lb == 3                       # (segment summaries + forward; state sweep + gradient sweep + gates)
    assert max(errs.values()) <= 1e-2


@pytest.mark.parametrize("base,B,T,H", [("C2", 8, 1024, 16), ("C2", 1, 4096, 4), ("C4", 4, 1024, 16)])
def test_training_step_is_reproducible_bit_for_bit(base, B, T, H):
    """The roles of a CTA hand tiles to one another through barriers only; a missing one shows up as a result that
    changes from run to run.  Twenty training steps on the same inputs must give the same bits every time."""
    cfg = small(CONFIGS[base], B=B, T=T, H=H, seed=930 + T)
    x = gu.to_dev(make_inputs(cfg, with_dO=True))
    first = None
    for _ in range(20):
        o, ht, g, plan, ws, lf, lb = gu.gpu_training_step(cfg, x)
        cur = [o, ht] + [t for t in g.values() if t is not None]
        if first is None:
            first = [t.clone() for t in cur]
        else:
            for a, b in zip(first, cur):
                assert torch.equal(a, b)
