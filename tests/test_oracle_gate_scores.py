"""Pins for the oracle's gate score projections (Eq. 4: G = softmax(Q W_GQ), W in R^{d x H}, d the per-head width;
the score of head h is that head's vector through column h of W)."""
import numpy as np
import pytest

from oracle import sla_oracle as orc
from tests.test_oracle_recurrence import draw


def test_scores_are_the_per_head_contraction():
    rng = np.random.default_rng(40)
    x, W = rng.normal(size=(2, 5, 3, 7)), rng.normal(size=(7, 3))
    s = orc.gate_scores(x, W)
    np.testing.assert_allclose(s, np.einsum("bthc,ch->bth", x, W), rtol=1e-13, atol=1e-14)
    for b, t, h in ((0, 0, 0), (1, 4, 2), (0, 3, 1)):           # written out: head h meets column h of W, nothing else
        assert abs(s[b, t, h] - sum(x[b, t, h, c] * W[c, h] for c in range(7))) < 1e-12
    # H = 1: a plain matrix-vector product per token
    x1, W1 = rng.normal(size=(4, 1, 6)), rng.normal(size=(6, 1))
    np.testing.assert_allclose(orc.gate_scores(x1, W1)[:, 0], x1[:, 0] @ W1[:, 0], rtol=1e-13, atol=1e-14)


def test_parameter_count_of_the_reading_matches_the_paper():
    # two d x H matrices per layer, 24 layers, hidden 1024 with 4 heads (d = 256): "approximately 0.05M"
    assert abs(2 * 256 * 4 * 24 - 0.05e6) / 0.05e6 < 0.02


def test_scaling_the_projection_sharpens_the_gates_to_one_hot():
    rng = np.random.default_rng(41)
    x, W = rng.normal(size=(6, 4, 8)), rng.normal(size=(8, 4))
    s = orc.gate_scores(x, W)
    ent = []
    for lam in (0.5, 1.0, 4.0, 64.0, 4096.0):
        G = orc.head_softmax(orc.gate_scores(x, lam * W))
        ent.append(float(-(G * np.log(G + 1e-300)).sum(-1).mean()))
    assert all(a > b for a, b in zip(ent, ent[1:]))            # Thm 3.2: entropy falls as lambda grows
    G = orc.head_softmax(orc.gate_scores(x, 4096.0 * W))
    np.testing.assert_allclose(G, np.eye(4)[s.argmax(-1)], atol=1e-9)


def test_backward_of_the_scores_alone():
    rng = np.random.default_rng(42)
    x, W, ds = rng.normal(size=(3, 4, 2, 5)), rng.normal(size=(5, 2)), rng.normal(size=(3, 4, 2))
    dx = np.ascontiguousarray(rng.normal(size=x.shape))
    dx0 = dx.copy()
    dW = orc.gate_scores_backward(x, W, ds, dx)
    np.testing.assert_allclose(dx - dx0, np.einsum("bth,ch->bthc", ds, W), rtol=1e-13, atol=1e-14)   # accumulated
    np.testing.assert_allclose(dW, np.einsum("bth,bthc->ch", ds, x), rtol=1e-13, atol=1e-14)


@pytest.mark.parametrize("variant", ["retnet", "gla", "gdn"])
def test_layer_with_projected_gates_against_finite_differences(variant):
    """The whole layer with gates computed from q and k: loss(q, k, W_GQ, W_GK) differentiated by the oracle's two
    reverse sweeps chained, against central differences (q and k now reach the loss on two routes)."""
    x, h0 = draw(variant, B=2, T=9, H=3, dk=4, dv=3, seed=43)
    rng = np.random.default_rng(44)
    Wq, Wk = rng.normal(size=(4, 3)), rng.normal(size=(4, 3))
    dO = rng.normal(size=x["v"].shape)

    def loss():
        lq, lk = orc.gate_scores(x["q"], Wq), orc.gate_scores(x["k"], Wk)
        o, _ = orc.forward(variant, x["q"], x["k"], x["v"], x["log_decay"], lq, lk, beta=x["beta"], h0=h0, scale=0.9)
        return float((o * dO).sum())

    lq, lk = orc.gate_scores(x["q"], Wq), orc.gate_scores(x["k"], Wk)
    g = orc.backward(variant, x["q"], x["k"], x["v"], x["log_decay"], lq, lk, dO, beta=x["beta"], h0=h0, scale=0.9)
    dq, dk = np.ascontiguousarray(g["dq"].copy()), np.ascontiguousarray(g["dk"].copy())
    dWq = orc.gate_scores_backward(x["q"], Wq, g["dlq"], dq)
    dWk = orc.gate_scores_backward(x["k"], Wk, g["dlk"], dk)
    eps = 1e-6
    for arr, grad in ((x["q"], dq), (x["k"], dk), (Wq, dWq), (Wk, dWk)):
        for fi in rng.choice(arr.size, size=10, replace=False):
            idx = np.unravel_index(fi, arr.shape)
            old = arr[idx]
            arr[idx] = old + eps
            lp = loss()
            arr[idx] = old - eps
            lm = loss()
            arr[idx] = old
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - grad[idx]) <= 1e-6 * max(1.0, abs(fd)), (idx, fd, grad[idx])
