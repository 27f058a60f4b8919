"""GPU parity of the fp32 CUDA-core chunk kernels against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2602_01744_b200 import api
from paper_2602_01744_b200.inputs import CONFIGS, make_inputs, small
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu
GEN = api.SLA_FLAG_FORCE_GENERIC


def test_c0_retnet_fp32_full_config():
    errs = gu.check_forward(CONFIGS["C0"], flags=GEN)
    assert max(errs.values()) <= 1e-4


@pytest.mark.parametrize("variant", ["retnet", "gla", "gdn"])
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_forward_small_ragged_tail_with_initial_state(variant, dtype):
    base = {"retnet": CONFIGS["C0"], "gla": CONFIGS["C1"], "gdn": CONFIGS["C4"]}[variant]
    cfg = small(base, B=2, T=200, H=3, dtype=dtype, seed=100)      # 200 = 3 chunks + a tail of 8
    gu.check_forward(cfg, with_h0=True, flags=GEN)


@pytest.mark.parametrize("chunk,dk,dv,H", [(16, 64, 128, 4), (32, 16, 48, 1), (64, 128, 64, 16), (64, 32, 32, 5)])
@pytest.mark.parametrize("variant", ["retnet", "gla", "gdn"])
def test_forward_shapes(variant, chunk, dk, dv, H):
    base = {"retnet": CONFIGS["C0"], "gla": CONFIGS["C1"], "gdn": CONFIGS["C4"]}[variant]
    cfg = small(base, B=1, T=150, H=H, d_k=dk, d_v=dv, chunk=chunk, dtype="fp32", seed=101, scale=0.5)
    gu.check_forward(cfg, flags=GEN)


@pytest.mark.parametrize("variant", ["retnet", "gla", "gdn"])
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_backward_small_ragged_tail_with_state_gradients(variant, dtype):
    base = {"retnet": CONFIGS["C0"], "gla": CONFIGS["C2"], "gdn": CONFIGS["C4"]}[variant]
    cfg = small(base, B=2, T=200, H=3, dtype=dtype, seed=102, backward=True)
    gu.check_backward(cfg, with_h0=True, flags=GEN)


@pytest.mark.parametrize("variant", ["retnet", "gla", "gdn"])
def test_backward_shapes(variant):
    base = {"retnet": CONFIGS["C0"], "gla": CONFIGS["C2"], "gdn": CONFIGS["C4"]}[variant]
    cfg = small(base, B=1, T=130, H=4, d_k=64, d_v=32, chunk=32, dtype="fp32", seed=103, scale=0.7)
    gu.check_backward(cfg, flags=GEN)


def test_single_token_and_single_chunk():
    for T in (1, 64):
        for base in (CONFIGS["C1"], CONFIGS["C4"]):
            cfg = small(base, B=1, T=T, H=2, dtype="fp32", seed=104)
            gu.check_forward(cfg, flags=GEN)
            gu.check_backward(small(cfg, backward=True), flags=GEN)


@pytest.mark.parametrize("variant", ["retnet", "gla", "gdn"])
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_decode_steps_match_oracle_and_chunkwise(variant, dtype):
    from oracle import sla_oracle as orc
    from paper_2602_01744_b200.inputs import make_decode_inputs
    base = {"retnet": CONFIGS["C0"], "gla": CONFIGS["C1"], "gdn": CONFIGS["C4"]}[variant]
    cfg = small(base, B=3, T=20, H=4, dtype=dtype, seed=105)
    steps = cfg.T
    dec = make_decode_inputs(cfg, cfg.B, steps, seed=106)
    h0 = torch.randn(cfg.B, cfg.H, cfg.d_k, cfg.d_v, generator=torch.Generator().manual_seed(7)) * 0.1
    plan = api.sla_plan_create(cfg.variant, cfg.dtype, cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk)
    state = h0.clone().cuda()
    ref_state = np.ascontiguousarray(h0.double().numpy().copy())
    outs, refs = [], []
    for t in range(steps):
        ld = dec["log_decay"] if variant == "retnet" else dec["log_decay"][t]
        bt = None if dec["beta"] is None else dec["beta"][t]
        o = api.sla_decode_step(plan, dec["q"][t].cuda(), dec["k"][t].cuda(), dec["v"][t].cuda(), ld.cuda(),
                                dec["gq_logits"][t].cuda(), dec["gk_logits"][t].cuda(), state,
                                beta_t=None if bt is None else bt.cuda())
        outs.append(o)
        refs.append(orc.decode_step(variant, dec["q"][t], dec["k"][t], dec["v"][t], ld, dec["gq_logits"][t],
                                    dec["gk_logits"][t], ref_state, beta_t=bt))
    torch.cuda.synchronize()
    tol = gu.TOL[dtype]
    assert gu.rel_l2(torch.stack(outs), np.stack(refs)) <= tol
    assert gu.rel_l2(state, ref_state) <= tol
    # the same tokens through the chunkwise forward with the same initial state
    x = dict(q=dec["q"].transpose(0, 1).contiguous(), k=dec["k"].transpose(0, 1).contiguous(),
             v=dec["v"].transpose(0, 1).contiguous(),
             log_decay=dec["log_decay"] if variant == "retnet" else dec["log_decay"].transpose(0, 1).contiguous(),
             beta=None if dec["beta"] is None else dec["beta"].transpose(0, 1).contiguous(),
             gq_logits=dec["gq_logits"].transpose(0, 1).contiguous(),
             gk_logits=dec["gk_logits"].transpose(0, 1).contiguous())
    o2, ht2, _ = gu.gpu_forward(cfg, gu.to_dev(x), h0=h0.cuda(), flags=GEN)
    assert gu.rel_l2(o2, torch.stack(outs, 1).double().cpu().numpy()) <= 2 * tol
    assert gu.rel_l2(ht2, state.double().cpu().numpy()) <= 2 * tol


def test_rejections():
    with pytest.raises(api.SLAError) as e:
        api.sla_plan_create("gla", "bf16", 1, 64, 33, 128, 128)
    assert e.value.status == 2
    with pytest.raises(api.SLAError):
        api.sla_plan_create("gla", "bf16", 1, 64, 4, 100, 128)
    plan = api.sla_plan_create("gla", "fp32", 1, 64, 2, 16, 16)
    x = gu.to_dev(make_inputs(small(CONFIGS["C1"], B=1, T=64, H=2, d_k=16, d_v=16, dtype="fp32")))
    tiny = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(api.SLAError) as e:
        api.sla_forward(plan, x["q"], x["k"], x["v"], x["log_decay"], x["gq_logits"], x["gk_logits"], workspace=tiny)
    assert e.value.status == 3
    # empty problem: nothing to do, no error
    p0 = api.sla_plan_create("gla", "fp32", 0, 64, 2, 16, 16)
    z = torch.empty(0, device="cuda")
    api.sla_forward(p0, z, z, z, z, z, z, o=z)
    assert p0.last_launch_count == 0


def _with_decay(cfg, per_step, **kw):
    x = make_inputs(cfg, **kw)
    x["log_decay"] = torch.full_like(x["log_decay"], per_step)
    return x


@pytest.mark.parametrize("variant,dtype,flags", [("gla", "bf16", 0), ("gdn", "bf16", 0), ("gla", "fp32", GEN),
                                                 ("gdn", "fp32", GEN), ("retnet", "fp32", GEN)])
def test_decay_beyond_the_chunk_range_is_reported(variant, dtype, flags):
    """log_decay = -2 per token puts the cumulative log-decay of a 64-token chunk at -128, beyond what the
    e^{b} e^{-b} split can carry: the call completes, sla_plan_poll answers SLA_ERR_RANGE once, and the same plan
    works again on inputs inside the range."""
    base = {"retnet": CONFIGS["C0"], "gla": CONFIGS["C2"], "gdn": CONFIGS["C4"]}[variant]
    cfg = small(base, B=1, T=130, H=2, d_k=128, d_v=128, dtype=dtype, seed=950, backward=True)
    plan = api.sla_plan_create(cfg.variant, cfg.dtype, cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk, cfg.scale, flags)
    args = lambda x: (x["q"], x["k"], x["v"], x["log_decay"], x["gq_logits"], x["gk_logits"])
    xs = gu.to_dev(_with_decay(cfg, -2.0, with_dO=True))
    for run in ("forward", "backward"):
        if run == "forward":
            api.sla_forward(plan, *args(xs), beta=xs["beta"])
        else:
            api.sla_backward(plan, *args(xs), xs["dO"], beta=xs["beta"])
        torch.cuda.synchronize()
        with pytest.raises(api.SLAError) as e:
            plan.poll()
        assert e.value.status == 7, run             # SLA_ERR_RANGE
        plan.poll()                                 # reported once, then clear
    xh = make_inputs(cfg, with_dO=True)
    x = gu.to_dev(xh)
    o, _ = api.sla_forward(plan, *args(x), beta=x["beta"])
    torch.cuda.synchronize()
    plan.poll()
    oref, _ = gu.oracle_forward(cfg, xh)
    assert gu.rel_l2(o, oref) <= gu.TOL[dtype]


@pytest.mark.parametrize("variant", ["retnet", "gla", "gdn"])
@pytest.mark.parametrize("per_step,chunk", [(-1.0, 64), (-4.0, 16)])
def test_strong_decay_inside_the_range_matches_the_oracle(variant, per_step, chunk):
    """Decays far stronger than the benchmark recipe's, still inside the range of the chunk size: -1 per token at
    chunk 64 (cumulative -64) and -4 per token at chunk 16 (cumulative -64), forward and backward."""
    base = {"retnet": CONFIGS["C0"], "gla": CONFIGS["C2"], "gdn": CONFIGS["C4"]}[variant]
    cfg = small(base, B=2, T=150, H=3, d_k=64, d_v=64, chunk=chunk, dtype="fp32", seed=951, backward=True)
    xh = _with_decay(cfg, per_step, with_dO=True, with_h0=True)
    x = gu.to_dev(xh)
    o, ht, plan = gu.gpu_forward(cfg, x, h0=x["h0"], flags=GEN)
    g, plan2 = gu.gpu_backward(cfg, x, h0=x["h0"], dht=x["dht"], want_dh0=True, flags=GEN)
    oref, htref = gu.oracle_forward(cfg, xh, h0=xh["h0"])
    ref = gu.oracle_backward(cfg, xh, h0=xh["h0"], dht=xh["dht"])
    pairs = {"o": (o, oref), "ht": (ht, htref)}
    pairs.update({n: (g[n], ref[r]) for n, r in gu.GRAD_NAMES.items() if g.get(n) is not None})
    gu.assert_close({n: gu.rel_l2(a, r) for n, (a, r) in pairs.items()},
                    {n: gu.row_err(a, r) for n, (a, r) in pairs.items()}, "fp32", (cfg, per_step))


@pytest.mark.parametrize("base", ["C2", "C4"])
def test_strong_decay_on_the_tensor_core_kernels(base):
    """-1 per token at chunk 64 (cumulative -64, inside the range) through the tcgen05 kernels."""
    cfg = small(CONFIGS[base], B=2, T=200, H=3, seed=952)
    xh = _with_decay(cfg, -1.0, with_dO=True, with_h0=True)
    x = gu.to_dev(xh)
    o, ht, g, plan, ws, lf, lb = gu.gpu_training_step(cfg, x, h0=x["h0"], dht=x["dht"], want_dh0=True)
    oref, htref = gu.oracle_forward(cfg, xh, h0=xh["h0"])
    ref = gu.oracle_backward(cfg, xh, h0=xh["h0"], dht=xh["dht"])
    pairs = {"o": (o, oref), "ht": (ht, htref)}
    pairs.update({n: (g[n], ref[r]) for n, r in gu.GRAD_NAMES.items() if g.get(n) is not None})
    gu.assert_close({n: gu.rel_l2(a, r) for n, (a, r) in pairs.items()},
                    {n: gu.row_err(a, r) for n, (a, r) in pairs.items()}, cfg.dtype, cfg)


def test_no_tokens_the_final_state_is_the_initial_state():
    plan = api.sla_plan_create("gla", "bf16", 2, 0, 3, 128, 128)
    h0 = torch.randn(2, 3, 128, 128, device="cuda")
    ht = torch.full_like(h0, float("nan"))
    z = torch.empty(0, device="cuda")
    api.sla_forward(plan, z, z, z, z, z, z, h0=h0, o=z, ht=ht)
    torch.cuda.synchronize()
    assert torch.equal(ht, h0) and plan.last_launch_count == 0
    api.sla_forward(plan, z, z, z, z, z, z, o=z, ht=ht)
    torch.cuda.synchronize()
    assert torch.count_nonzero(ht) == 0


@pytest.mark.parametrize("variant", ["retnet", "gla", "gdn"])
def test_generic_kernels_write_nothing_outside_their_buffers(variant):
    base = {"retnet": CONFIGS["C0"], "gla": CONFIGS["C2"], "gdn": CONFIGS["C4"]}[variant]
    cfg = small(base, B=2, T=150, H=3, d_k=64, d_v=48, chunk=32, dtype="fp32", seed=953, backward=True)
    xh = make_inputs(cfg, with_dO=True, with_h0=True)
    x = gu.to_dev(xh)
    plan = api.sla_plan_create(cfg.variant, cfg.dtype, cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk, cfg.scale, GEN)
    nq, nv = cfg.B * cfg.T * cfg.H * cfg.d_k * 4, cfg.B * cfg.T * cfg.H * cfg.d_v * 4
    nst, nl = cfg.B * cfg.H * cfg.d_k * cfg.d_v * 4, cfg.B * cfg.T * cfg.H * 4
    ndec = x["log_decay"].numel() * 4
    wsb = plan.backward_workspace_bytes
    arena = gu.Guarded.for_sizes([wsb, nv, nst, nq, nq, nv, ndec, nl, nl, nl, nst])
    nan = float("nan")
    f32 = torch.float32
    ws = arena.take(wsb)
    sq, sv, sst, sl = (cfg.B, cfg.T, cfg.H, cfg.d_k), (cfg.B, cfg.T, cfg.H, cfg.d_v), (cfg.B, cfg.H, cfg.d_k, cfg.d_v), (cfg.B, cfg.T, cfg.H)
    o, ht = arena.take(nv, f32, sv, nan), arena.take(nst, f32, sst, nan)
    out = dict(dq=arena.take(nq, f32, sq, nan), dk=arena.take(nq, f32, sq, nan), dv=arena.take(nv, f32, sv, nan),
               dlog_decay=None if variant == "retnet" else arena.take(ndec, f32, tuple(x["log_decay"].shape), nan),
               dbeta=arena.take(nl, f32, sl, nan) if variant == "gdn" else None,
               dgq_logits=arena.take(nl, f32, sl, nan), dgk_logits=arena.take(nl, f32, sl, nan),
               dh0=arena.take(nst, f32, sst, nan))
    args = (x["q"], x["k"], x["v"], x["log_decay"], x["gq_logits"], x["gk_logits"])
    api.sla_forward(plan, *args, beta=x["beta"], h0=x["h0"], o=o, ht=ht, workspace=ws)
    api.sla_backward(plan, *args, x["dO"], beta=x["beta"], h0=x["h0"], dht=x["dht"], workspace=ws, out=out)
    torch.cuda.synchronize()
    plan.poll()
    arena.check()
    oref, htref = gu.oracle_forward(cfg, xh, h0=xh["h0"])
    ref = gu.oracle_backward(cfg, xh, h0=xh["h0"], dht=xh["dht"])
    pairs = {"o": (o, oref), "ht": (ht, htref)}
    pairs.update({n: (out[n], ref[r]) for n, r in gu.GRAD_NAMES.items() if out.get(n) is not None})
    gu.assert_close({n: gu.rel_l2(a, r) for n, (a, r) in pairs.items()},
                    {n: gu.row_err(a, r) for n, (a, r) in pairs.items()}, "fp32", cfg)


def test_bounded_wait_expiry_is_reported_and_the_context_survives():
    plan = api.sla_plan_create("gla", "bf16", 1, 64, 2, 128, 128)
    plan.selftest_timeout()                     # a wait nobody satisfies: gives up after 2 ms
    torch.cuda.synchronize()
    with pytest.raises(api.SLAError) as e:
        plan.poll()
    assert e.value.status == 6                  # SLA_ERR_TIMEOUT
    plan.poll()                                 # reported once, then clear again
    x = gu.to_dev(make_inputs(small(CONFIGS["C1"], B=1, T=64, H=2)))
    o, _ = api.sla_forward(plan, x["q"], x["k"], x["v"], x["log_decay"], x["gq_logits"], x["gk_logits"])
    torch.cuda.synchronize()
    plan.poll()
    assert torch.isfinite(o.float()).all()
