"""Packed variable-length batches (sla_plan_set_sequences): sequences of mixed lengths laid one after another along T,
the state reset at every boundary.  Checked against the oracle run sequence by sequence, and bit for bit against the
same kernels run on each sequence alone (the packing is index work: it must not change a single bit)."""
import numpy as np
import pytest
import torch

from paper_2602_01744_b200 import api
from paper_2602_01744_b200.inputs import CONFIGS, make_inputs, small
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu
LENGTHS = (1, 63, 64, 65, 900, 130)      # (under 16 chunks each: run alone, such a sequence is not cut into segments)


def _packed(base, lengths, H, seed, with_h0, d=128):
    T = sum(lengths)
    dk, dv = d if isinstance(d, tuple) else (d, d)
    cfg = small(CONFIGS[base], B=1, T=T, H=H, d_k=dk, d_v=dv, seed=seed)
    x = make_inputs(cfg, with_dO=True)
    n = len(lengths)
    if with_h0:
        gen = torch.Generator().manual_seed(seed + 1)
        x["h0"] = torch.randn(n, H, cfg.d_k, cfg.d_v, generator=gen) * 0.1
        x["dht"] = torch.randn(n, H, cfg.d_k, cfg.d_v, generator=gen) * 0.1
    cu = np.concatenate([[0], np.cumsum(lengths)]).tolist()
    return cfg, x, cu


def _slice(x, s, a, b):
    """Sequence s (tokens a..b) of the packed inputs as a batch of one."""
    out = {}
    for n, t in x.items():
        if t is None:
            out[n] = None
        elif n in ("h0", "dht"):
            out[n] = t[s:s + 1].contiguous()
        elif t.dim() == 1:
            out[n] = t
        else:
            out[n] = t[:, a:b].contiguous()
    return out


@pytest.mark.parametrize("base,d", [("C2", 128), ("R2", 128), ("C4", 128), ("C2", 64), ("C4", 64), ("C2", (64, 128)), ("C4", (128, 64))])
@pytest.mark.parametrize("with_h0", [False, True])
def test_packed_batch_matches_the_oracle_and_the_single_sequence_runs(base, d, with_h0):
    H = 3
    cfg, xh, cu = _packed(base, LENGTHS, H, 1300, with_h0, d)
    x = gu.to_dev(xh)
    n = len(LENGTHS)
    plan = api.sla_plan_create(cfg.variant, cfg.dtype, 1, cfg.T, H, cfg.d_k, cfg.d_v, cfg.chunk, cfg.scale,
                               api.SLA_FLAG_SAVE_FOR_BACKWARD)
    plan.set_sequences(cu)
    ws = plan.workspace(backward=True)
    ht = torch.full((n, H, cfg.d_k, cfg.d_v), float("nan"), device="cuda")
    args = (x["q"], x["k"], x["v"], x["log_decay"], x["gq_logits"], x["gk_logits"])
    o, _ = api.sla_forward(plan, *args, beta=x["beta"], h0=x.get("h0"), ht=ht, workspace=ws)
    assert plan.last_launch_count == 1
    g = api.sla_backward(plan, *args, x["dO"], beta=x["beta"], h0=x.get("h0"), dht=x.get("dht"), want_dh0=with_h0, workspace=ws)
    assert plan.last_launch_count == 2                 # read what the forward left
    g2 = api.sla_backward(plan, *args, x["dO"], beta=x["beta"], h0=x.get("h0"), dht=x.get("dht"), want_dh0=with_h0)
    assert plan.last_launch_count == 3                 # other workspace: recomputed
    torch.cuda.synchronize()
    plan.poll()
    for name, t in g.items():
        if t is not None:
            assert torch.equal(t, g2[name]), name
    # reference: the oracle run on every sequence alone, put together in the packed layout (the error is measured over
    # the packed tensors: a one-token sequence on its own is a single ill-conditioned dot product, not a tensor)
    refs = {}
    for s in range(n):
        a, b = cu[s], cu[s + 1]
        c1 = small(cfg, T=b - a)
        xs_h = _slice(xh, s, a, b)
        oref, htref = gu.oracle_forward(c1, xs_h, h0=xs_h.get("h0"))
        ref = gu.oracle_backward(c1, xs_h, h0=xs_h.get("h0"), dht=xs_h.get("dht"))
        parts = {"o": oref, "ht": htref}
        parts.update({gname: ref[rname] for gname, rname in gu.GRAD_NAMES.items() if g.get(gname) is not None})
        for k, v in parts.items():
            refs.setdefault(k, []).append(v)
        # the same kernels on this sequence alone: identical bits
        xs = gu.to_dev(xs_h)
        o1, ht1, g1, p1, ws1, lf, lb = gu.gpu_training_step(c1, xs, h0=xs.get("h0"), dht=xs.get("dht"), want_dh0=with_h0)
        assert torch.equal(o1, o[:, a:b]) and torch.equal(ht1, ht[s:s + 1]), (s, "forward")
        for gname, t in g1.items():
            if t is None:
                continue
            packed = g[gname][s:s + 1] if gname == "dh0" else g[gname][:, a:b]
            assert torch.equal(t, packed), (s, gname)
    pairs = {}
    for k, parts in refs.items():
        axis = 0 if k in ("ht", "dh0") else 1
        got = ht if k == "ht" else o if k == "o" else g[k]
        pairs[k] = (got, np.concatenate(parts, axis=axis))
    gu.assert_close({k: gu.rel_l2(u, v) for k, (u, v) in pairs.items()},
                    {k: gu.row_err(u, v) for k, (u, v) in pairs.items()}, cfg.dtype, (base, with_h0))


def test_sequence_table_is_validated_and_can_be_cleared():
    plan = api.sla_plan_create("gla", "bf16", 1, 300, 2, 128, 128)
    for bad in ([0, 100, 100, 300], [0, 100, 200], [1, 300], [0, 200, 100, 300]):
        with pytest.raises(api.SLAError) as e:
            plan.set_sequences(bad)
        assert e.value.status == 1
    with pytest.raises(api.SLAError) as e:
        api.sla_plan_create("gla", "fp32", 1, 300, 2, 64, 64).set_sequences([0, 300])
    assert e.value.status == 2                          # only the tensor-core kernels take a table
    with pytest.raises(api.SLAError):
        api.sla_plan_create("gla", "bf16", 2, 300, 2, 128, 128).set_sequences([0, 300])      # B must be 1
    plan.set_sequences([0, 100, 300])
    w2 = plan.backward_workspace_bytes
    plan.set_sequences(None)
    assert plan.backward_workspace_bytes < w2           # (one state slot fewer)
    cfg = small(CONFIGS["C1"], B=1, T=300, H=2, seed=1310)
    xh = make_inputs(cfg)
    x = gu.to_dev(xh)
    o, _ = api.sla_forward(plan, x["q"], x["k"], x["v"], x["log_decay"], x["gq_logits"], x["gk_logits"])
    torch.cuda.synchronize()
    oref, _ = gu.oracle_forward(cfg, xh)
    assert gu.rel_l2(o, oref) <= 1e-2
