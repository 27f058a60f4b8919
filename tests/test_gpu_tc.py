"""GPU parity of the tcgen05/TMEM/TMA Softmax-GLA and Softmax-GatedDeltaNet kernels (bf16, d_k = d_v = 128 or 64, chunk 64) against
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


@pytest.mark.parametrize("base", ["C2", "C4"])
def test_saved_states_are_not_reused_once_another_backward_has_overwritten_them(base):
    """forward(A) leaves A's chunk states in the workspace; a backward for OTHER contents through the same workspace
    recomputes and overwrites them; a backward for A's pointers afterwards must recompute too (not read B's states)."""
    cfg_a = small(CONFIGS[base], B=2, T=300, H=4, seed=911)
    cfg_b = small(cfg_a, seed=912)
    xa_host, xb_host = make_inputs(cfg_a, with_dO=True), make_inputs(cfg_b, with_dO=True)
    xa, xb = gu.to_dev(xa_host), gu.to_dev(xb_host)
    plan = api.sla_plan_create(cfg_a.variant, cfg_a.dtype, cfg_a.B, cfg_a.T, cfg_a.H, cfg_a.d_k, cfg_a.d_v, cfg_a.chunk,
                               cfg_a.scale, api.SLA_FLAG_SAVE_FOR_BACKWARD)
    ws = plan.workspace(backward=True)
    args = lambda x: (x["q"], x["k"], x["v"], x["log_decay"], x["gq_logits"], x["gk_logits"])
    api.sla_forward(plan, *args(xa), beta=xa["beta"], workspace=ws)
    g_a1 = api.sla_backward(plan, *args(xa), xa["dO"], beta=xa["beta"], workspace=ws)
    assert plan.last_launch_count == 2                 # read what the forward left
    api.sla_forward(plan, *args(xa), beta=xa["beta"], workspace=ws)
    g_b = api.sla_backward(plan, *args(xb), xb["dO"], beta=xb["beta"], workspace=ws)
    assert plan.last_launch_count == 3                 # other inputs: recomputed, into the same workspace
    g_a2 = api.sla_backward(plan, *args(xa), xa["dO"], beta=xa["beta"], workspace=ws)
    assert plan.last_launch_count == 3                 # A's states are gone from the workspace: recomputed again
    g_b2 = api.sla_backward(plan, *args(xb), xb["dO"], beta=xb["beta"], workspace=ws)
    assert plan.last_launch_count == 3
    torch.cuda.synchronize()
    plan.poll()
    for cfg, xh, grads in ((cfg_a, xa_host, (g_a1, g_a2)), (cfg_b, xb_host, (g_b, g_b2))):
        ref = gu.oracle_backward(cfg, xh)
        for g in grads:
            errs = {n: gu.rel_l2(g[n], ref[r]) for n, r in gu.GRAD_NAMES.items() if g.get(n) is not None}
            rows = {n: gu.row_err(g[n], ref[r]) for n, r in gu.GRAD_NAMES.items() if g.get(n) is not None}
            gu.assert_close(errs, rows, cfg.dtype, cfg)
    for n, t in g_a1.items():
        if t is not None:
            assert torch.equal(t, g_a2[n]) and torch.equal(g_b[n], g_b2[n]), n


@pytest.mark.parametrize("base,T,d", [("C2", 200, 128), ("C2", 64, 128), ("C4", 200, 128), ("C4", 65, 128),
                                      ("C2", 200, 64), ("C2", 65, 64), ("C4", 200, 64)])
def test_nothing_is_written_outside_the_buffers_handed_in(base, T, d):
    """In place of a memory checker: outputs and workspace are carved out of one pattern-filled arena with guard bands
    around each; after a training step and a recomputing backward no guard byte may differ, every output element must
    have been written (they start as NaN) and the results must still match the oracle."""
    cfg = small(CONFIGS[base], B=2, T=T, H=3, d_k=d, d_v=d, seed=940 + T)     # (d = 64: heads padded inside the kernels)
    xh = make_inputs(cfg, with_dO=True, with_h0=True)
    x = gu.to_dev(xh)
    plan = api.sla_plan_create(cfg.variant, cfg.dtype, cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk, cfg.scale,
                               api.SLA_FLAG_SAVE_FOR_BACKWARD)
    nio = cfg.B * cfg.T * cfg.H * cfg.d_k * 2
    nst = cfg.B * cfg.H * cfg.d_k * cfg.d_v * 4
    nl = cfg.B * cfg.T * cfg.H * 4
    ndec = x["log_decay"].numel() * 4
    wsb = max(plan.backward_workspace_bytes, plan.forward_workspace_bytes, 16)
    arena = gu.Guarded.for_sizes([wsb, nio, nst, nio, nio, nio, ndec, nl, nl, nl, nst])
    nan = float("nan")
    ws = arena.take(wsb)
    shape_io = (cfg.B, cfg.T, cfg.H, cfg.d_k)
    shape_st = (cfg.B, cfg.H, cfg.d_k, cfg.d_v)
    o = arena.take(nio, torch.bfloat16, shape_io, nan)
    ht = arena.take(nst, torch.float32, shape_st, nan)
    out = dict(dq=arena.take(nio, torch.bfloat16, shape_io, nan), dk=arena.take(nio, torch.bfloat16, shape_io, nan),
               dv=arena.take(nio, torch.bfloat16, shape_io, nan),
               dlog_decay=arena.take(ndec, torch.float32, tuple(x["log_decay"].shape), nan),
               dbeta=arena.take(nl, torch.float32, (cfg.B, cfg.T, cfg.H), nan) if cfg.variant == "gdn" else None,
               dgq_logits=arena.take(nl, torch.float32, (cfg.B, cfg.T, cfg.H), nan),
               dgk_logits=arena.take(nl, torch.float32, (cfg.B, cfg.T, cfg.H), nan),
               dh0=arena.take(nst, torch.float32, shape_st, nan))
    args = (x["q"], x["k"], x["v"], x["log_decay"], x["gq_logits"], x["gk_logits"])
    api.sla_forward(plan, *args, beta=x["beta"], h0=x["h0"], o=o, ht=ht, workspace=ws)
    api.sla_backward(plan, *args, x["dO"], beta=x["beta"], h0=x["h0"], dht=x["dht"], workspace=ws, out=out)
    assert plan.last_launch_count == 2
    torch.cuda.synchronize()
    plan.poll()
    arena.check()
    oref, htref = gu.oracle_forward(cfg, xh, h0=xh["h0"])
    ref = gu.oracle_backward(cfg, xh, h0=xh["h0"], dht=xh["dht"])
    pairs = {"o": (o, oref), "ht": (ht, htref)}
    pairs.update({n: (out[n], ref[r]) for n, r in gu.GRAD_NAMES.items() if out.get(n) is not None})
    gu.assert_close({n: gu.rel_l2(a, r) for n, (a, r) in pairs.items()},
                    {n: gu.row_err(a, r) for n, (a, r) in pairs.items()}, cfg.dtype, cfg)   # (a NaN left in place fails here)
    # the recomputing backward (state sweep / record sweep into the same workspace) under the same watch
    for t in out.values():
        if t is not None:
            t.fill_(nan)
    plain = api.sla_plan_create(cfg.variant, cfg.dtype, cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk, cfg.scale)
    assert plain.backward_workspace_bytes <= wsb
    api.sla_backward(plain, *args, x["dO"], beta=x["beta"], h0=x["h0"], dht=x["dht"], workspace=ws, out=out)
    assert plain.last_launch_count == 3
    torch.cuda.synchronize()
    plain.poll()
    arena.check()
    pairs = {n: (out[n], ref[r]) for n, r in gu.GRAD_NAMES.items() if out.get(n) is not None}
    gu.assert_close({n: gu.rel_l2(a, r) for n, (a, r) in pairs.items()},
                    {n: gu.row_err(a, r) for n, (a, r) in pairs.items()}, cfg.dtype, cfg)


def test_segmented_forward_leaves_nothing_and_the_backward_recomputes():
    cfg = small(CONFIGS["C2"], B=2, T=1024, H=16, seed=920)    # few long sequences: the forward runs in two segments
    errs, lf, lb = gu.check_training_step(cfg)
    assert lf == 2 and lb == 3                       # (segment summaries + forward; state sweep + gradient sweep + gates)
    assert max(errs.values()) <= 1e-2


@pytest.mark.parametrize("base,B,T,H,d,with_h0", [("C2", 1, 2048, 4, 128, True), ("C2", 2, 1990, 3, 128, False),
                                                   ("R2", 1, 4096, 2, 128, True), ("C2", 1, 2048, 4, 64, True)])
def test_backward_in_segments_for_few_long_sequences(base, B, T, H, d, with_h0):
    """From three segments per sequence on, the backward runs every sequence in segments too (as the sequences of a
    packed batch, twice: once for the state gradients that leave each segment, once for the results), with the
    initial state, the final-state gradient and dh0 carried across the cuts."""
    cfg = small(CONFIGS[base], B=B, T=T, H=H, d_k=d, d_v=d, seed=925 + T)
    x = make_inputs(cfg, with_dO=True, with_h0=with_h0)
    xd = gu.to_dev(x)
    o, ht, g, plan, ws, lf, lb = gu.gpu_training_step(cfg, xd, h0=xd.get("h0"), dht=xd.get("dht"), want_dh0=with_h0)
    assert lf == 2 and lb == 8, (lf, lb)    # summaries, fold, (states, sweep, gates), fold, (sweep, gates)
    oref, htref = gu.oracle_forward(cfg, x, h0=x.get("h0"))
    ref = gu.oracle_backward(cfg, x, h0=x.get("h0"), dht=x.get("dht"))
    pairs = {"o": (o, oref), "ht": (ht, htref)}
    pairs.update({n: (g[n], ref[r]) for n, r in gu.GRAD_NAMES.items() if g.get(n) is not None})
    gu.assert_close({n: gu.rel_l2(a, r) for n, (a, r) in pairs.items()},
                    {n: gu.row_err(a, r) for n, (a, r) in pairs.items()}, cfg.dtype, cfg)
    g2 = api.sla_backward(plan, xd["q"], xd["k"], xd["v"], xd["log_decay"], xd["gq_logits"], xd["gk_logits"], xd["dO"],
                          h0=xd.get("h0"), dht=xd.get("dht"), want_dh0=with_h0, workspace=ws)
    torch.cuda.synchronize()
    for n, t in g.items():
        if t is not None:
            assert torch.equal(t, g2[n]), n          # same bits on every run


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


# ---- Softmax-RetNet (Eq. 10-11) on the tensor-core kernels: the GLA kernels with the decay generated in the kernel ----
@pytest.mark.parametrize("B,T,H,with_h0", [(1, 64, 1, False), (2, 200, 3, True), (1, 1000, 16, True), (3, 65, 4, True),
                                           (1, 5, 2, False), (1, 2048, 4, False)])       # the last one runs segmented
def test_retnet_forward_and_backward_tc(B, T, H, with_h0):
    cfg = small(CONFIGS["R2"], B=B, T=T, H=H, seed=1000 + T)
    assert max(gu.check_forward(small(cfg, backward=False), with_h0=with_h0).values()) <= 1e-2
    assert max(gu.check_backward(cfg, with_h0=with_h0).values()) <= 1e-2


def test_retnet_takes_the_tensor_core_path_and_agrees_with_generic():
    cfg = small(CONFIGS["R2"], B=2, T=300, H=4, seed=1010, scale=0.5)
    x = gu.to_dev(make_inputs(cfg, with_dO=True, with_h0=True))
    o1, ht1, plan = gu.gpu_forward(cfg, x, h0=x["h0"])
    assert plan.last_launch_count == 1 and plan.forward_workspace_bytes == 0
    o2, ht2, plan2 = gu.gpu_forward(cfg, x, h0=x["h0"], flags=api.SLA_FLAG_FORCE_GENERIC)
    assert plan2.last_launch_count > 1
    assert gu.rel_l2(o1, o2.double().cpu().numpy()) <= 1e-2 and gu.rel_l2(ht1, ht2.double().cpu().numpy()) <= 1e-2
    g1, plan = gu.gpu_backward(cfg, x, h0=x["h0"], dht=x["dht"], want_dh0=True)
    assert plan.last_launch_count == 3
    g2, plan2 = gu.gpu_backward(cfg, x, h0=x["h0"], dht=x["dht"], want_dh0=True, flags=api.SLA_FLAG_FORCE_GENERIC)
    for name in ("dq", "dk", "dv", "dgq_logits", "dgk_logits", "dh0"):
        assert gu.rel_l2(g1[name], g2[name].double().cpu().numpy()) <= 1e-2, name
    assert g1["dlog_decay"] is None


@pytest.mark.parametrize("B,T,H,with_h0", [(2, 200, 3, True), (1, 960, 8, False)])
def test_retnet_training_step_reads_what_the_forward_left(B, T, H, with_h0):
    cfg = small(CONFIGS["R2"], B=B, T=T, H=H, seed=1020 + T)
    errs, lf, lb = gu.check_training_step(cfg, with_h0=with_h0)
    assert (lf, lb) == (1, 2)
    assert max(errs.values()) <= 1e-2


# ---- 64-wide heads: the same kernels, the upper half of every 128-wide tile being zero padding that the tensor maps
# supply on loads and drop on stores (no padded copies in memory)
@pytest.mark.parametrize("base", ["C2", "R2", "C4"])
@pytest.mark.parametrize("dk,dv", [(64, 64), (64, 128), (128, 64)])
@pytest.mark.parametrize("B,T,H,with_h0", [(2, 200, 3, True), (1, 1000, 16, True), (3, 65, 4, False), (2, 5, 2, True)])
def test_heads_of_width_64_take_the_tensor_core_kernels(base, dk, dv, B, T, H, with_h0):
    cfg = small(CONFIGS[base], B=B, T=T, H=H, d_k=dk, d_v=dv, seed=1400 + T)
    x = make_inputs(cfg, with_dO=True, with_h0=with_h0)
    xd = gu.to_dev(x)
    o, ht, g, plan, ws, lf, lb = gu.gpu_training_step(cfg, xd, h0=xd.get("h0"), dht=xd.get("dht"), want_dh0=with_h0)
    # fused forward and a backward that reads the states it left; or, for few long sequences, a forward in segments
    # (which leaves none) and a backward that recomputes them
    assert (lf, lb) in ((1, 2), (2, 3)), (lf, lb)
    oref, htref = gu.oracle_forward(cfg, x, h0=x.get("h0"))
    ref = gu.oracle_backward(cfg, x, h0=x.get("h0"), dht=x.get("dht"))
    pairs = {"o": (o, oref), "ht": (ht, htref)}
    pairs.update({n: (g[n], ref[r]) for n, r in gu.GRAD_NAMES.items() if g.get(n) is not None})
    gu.assert_close({n: gu.rel_l2(a, r) for n, (a, r) in pairs.items()},
                    {n: gu.row_err(a, r) for n, (a, r) in pairs.items()}, cfg.dtype, cfg)
    # the recomputing backward gives the same bits
    g2, plan2 = gu.gpu_backward(cfg, xd, h0=xd.get("h0"), dht=xd.get("dht"), want_dh0=with_h0)
    assert plan2.last_launch_count == 3
    for n, t in g.items():
        if t is not None:
            assert torch.equal(t, g2[n]), n


def test_other_widths_stay_on_the_generic_kernels():
    cfg = small(CONFIGS["C2"], B=1, T=130, H=2, d_k=96, d_v=128, seed=1410)
    x = gu.to_dev(make_inputs(cfg))
    o, ht, plan = gu.gpu_forward(cfg, x)
    assert plan.last_launch_count > 1
