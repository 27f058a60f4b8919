"""Pins for the oracle's reverse sweep: central finite differences of the oracle's own forward
(itself pinned by brute force), plus identities that hold for the true gradient."""
import numpy as np
import pytest

from oracle import sla_oracle as orc
from tests.test_oracle_recurrence import draw


def loss_fn(variant, x, h0, dO, dht, scale):
    o, ht = orc.forward(variant, **x, h0=h0, scale=scale)
    return float((o * dO).sum() + (ht * dht).sum())


@pytest.mark.parametrize("variant", ["retnet", "gla", "gdn"])
def test_backward_matches_finite_differences(variant):
    x, h0 = draw(variant, B=2, T=70, H=3, dk=4, dv=3, seed=30)   # T > 64: crosses a checkpoint segment
    rng = np.random.default_rng(31)
    dO = rng.normal(size=x["v"].shape)
    dht = rng.normal(size=h0.shape)
    scale = 0.8
    g = orc.backward(variant, x["q"], x["k"], x["v"], x["log_decay"], x["lq"], x["lk"], dO,
                     beta=x["beta"], h0=h0, dht=dht, scale=scale)
    names = {"q": "dq", "k": "dk", "v": "dv", "log_decay": "dlog_decay", "lq": "dlq", "lk": "dlk"}
    if variant == "gdn":
        names["beta"] = "dbeta"
    eps = 1e-6
    for name, gname in names.items():
        arr = x[name]
        flat_idx = rng.choice(arr.size, size=min(12, arr.size), replace=False)
        for fi in flat_idx:
            idx = np.unravel_index(fi, arr.shape)
            old = arr[idx]
            arr[idx] = old + eps
            lp = loss_fn(variant, x, h0, dO, dht, scale)
            arr[idx] = old - eps
            lm = loss_fn(variant, x, h0, dO, dht, scale)
            arr[idx] = old
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - g[gname][idx]) <= 1e-6 * max(1.0, abs(fd)), (name, idx, fd, g[gname][idx])
    # dh0
    for fi in rng.choice(h0.size, size=10, replace=False):
        idx = np.unravel_index(fi, h0.shape)
        old = h0[idx]
        h0[idx] = old + eps
        lp = loss_fn(variant, x, h0, dO, dht, scale)
        h0[idx] = old - eps
        lm = loss_fn(variant, x, h0, dO, dht, scale)
        h0[idx] = old
        fd = (lp - lm) / (2 * eps)
        assert abs(fd - g["dh0"][idx]) <= 1e-6 * max(1.0, abs(fd))


@pytest.mark.parametrize("variant", ["retnet", "gla", "gdn"])
def test_gradient_identities(variant):
    x, h0 = draw(variant, B=2, T=20, H=4, dk=6, dv=5, seed=32)
    rng = np.random.default_rng(33)
    dO = rng.normal(size=x["v"].shape)
    g = orc.backward(variant, x["q"], x["k"], x["v"], x["log_decay"], x["lq"], x["lk"], dO,
                     beta=x["beta"])
    o, _ = orc.forward(variant, **x)
    # softmax shift invariance: logit gradients sum to zero over heads
    np.testing.assert_allclose(g["dlq"].sum(-1), 0.0, atol=1e-12)
    np.testing.assert_allclose(g["dlk"].sum(-1), 0.0, atol=1e-12)
    # o is linear in q (always) and, with h0 = 0, in v
    np.testing.assert_allclose((g["dq"] * x["q"]).sum(), (dO * o).sum(), rtol=1e-10)
    np.testing.assert_allclose((g["dv"] * x["v"]).sum(), (dO * o).sum(), rtol=1e-10)
    if variant == "gla":
        # dg_s = sum_{t>=s} (q_t dq_t - k_t dk_t) per key dimension
        d = x["q"] * g["dq"] - x["k"] * g["dk"]
        suffix = np.flip(np.cumsum(np.flip(d, 1), 1), 1)
        np.testing.assert_allclose(g["dlog_decay"], suffix, rtol=1e-9, atol=1e-12)


def test_single_head_has_zero_logit_gradient():
    x, _ = draw("gla", H=1, seed=34)
    dO = np.ones_like(x["v"])
    g = orc.backward("gla", x["q"], x["k"], x["v"], x["log_decay"], x["lq"], x["lk"], dO)
    assert np.abs(g["dlq"]).max() == 0.0 and np.abs(g["dlk"]).max() == 0.0
