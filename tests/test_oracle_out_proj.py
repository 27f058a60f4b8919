"""Pins for the oracle's output projection (Eq. 7: the heads' outputs of a token, concatenated, times W^O)."""
import numpy as np

from oracle import sla_oracle as orc


def test_written_out_on_a_tiny_case():
    rng = np.random.default_rng(70)
    o, W = rng.normal(size=(2, 3, 5)), rng.normal(size=(5, 4))
    y = orc.out_proj(o, W)
    assert y.shape == (2, 3, 4)
    for b in range(2):
        for t in range(3):
            for n in range(4):
                assert abs(y[b, t, n] - sum(o[b, t, c] * W[c, n] for c in range(5))) < 1e-13
    # not the transposed product: a rectangular W only fits one way, and a non-symmetric square one tells them apart
    Ws = rng.normal(size=(5, 5))
    assert np.abs(orc.out_proj(o, Ws) - o @ Ws.T).max() > 1e-2
    np.testing.assert_allclose(orc.out_proj(o, Ws), o @ Ws, rtol=1e-13, atol=1e-13)


def test_special_weights():
    rng = np.random.default_rng(71)
    o = rng.normal(size=(7, 6))
    np.testing.assert_array_equal(orc.out_proj(o, np.eye(6)), o)                 # identity
    perm = rng.permutation(6)
    np.testing.assert_array_equal(orc.out_proj(o, np.eye(6)[:, perm]), o[:, perm])   # column n picks feature perm[n]
    e = np.zeros((6, 3)); e[4, 1] = 2.5                                           # one weight: feature 4 -> output 1
    y = orc.out_proj(o, e)
    np.testing.assert_array_equal(y[:, 1], 2.5 * o[:, 4])
    assert not y[:, [0, 2]].any()
    # heads enter through their own row block of W: zeroing head 1's rows removes exactly that head's contribution
    H, dv = 3, 2
    W = rng.normal(size=(H * dv, 5))
    W0 = W.copy(); W0[dv:2 * dv] = 0
    oh = o.reshape(7, H, dv)
    np.testing.assert_allclose(orc.out_proj(o, W) - orc.out_proj(o, W0), oh[:, 1] @ W[dv:2 * dv], rtol=1e-12, atol=1e-13)


def test_linear_in_both_arguments():
    rng = np.random.default_rng(72)
    o1, o2, W1, W2 = rng.normal(size=(4, 6)), rng.normal(size=(4, 6)), rng.normal(size=(6, 3)), rng.normal(size=(6, 3))
    np.testing.assert_allclose(orc.out_proj(2 * o1 - o2, W1), 2 * orc.out_proj(o1, W1) - orc.out_proj(o2, W1), atol=1e-12)
    np.testing.assert_allclose(orc.out_proj(o1, W1 + 3 * W2), orc.out_proj(o1, W1) + 3 * orc.out_proj(o1, W2), atol=1e-12)


def test_backward_is_the_adjoint_and_matches_finite_differences():
    rng = np.random.default_rng(73)
    o, W, dy = rng.normal(size=(2, 5, 6)), rng.normal(size=(6, 4)), rng.normal(size=(2, 5, 4))
    d_o, dW = orc.out_proj_backward(o, W, dy)
    # <dy, y> is bilinear in (o, W): its derivatives are the two adjoint products
    loss = lambda oo, WW: float((dy * orc.out_proj(oo, WW)).sum())
    h = 1e-6
    for idx in ((0, 0, 0), (1, 4, 5), (0, 2, 3)):
        e = np.zeros_like(o); e[idx] = h
        assert abs((loss(o + e, W) - loss(o - e, W)) / (2 * h) - d_o[idx]) < 1e-8
    for idx in ((0, 0), (5, 3), (2, 1)):
        e = np.zeros_like(W); e[idx] = h
        assert abs((loss(o, W + e) - loss(o, W - e)) / (2 * h) - dW[idx]) < 1e-8
    # adjoint identities: <d_o, o> = <dy, y> = <dW, W>
    y = orc.out_proj(o, W)
    assert abs((d_o * o).sum() - (dy * y).sum()) < 1e-11 and abs((dW * W).sum() - (dy * y).sum()) < 1e-11
    # written out
    assert abs(d_o[1, 2, 3] - sum(dy[1, 2, n] * W[3, n] for n in range(4))) < 1e-13
    assert abs(dW[3, 2] - sum(o[b, t, 3] * dy[b, t, 2] for b in range(2) for t in range(5))) < 1e-13
