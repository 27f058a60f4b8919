"""Pins for the oracle's Gated-DeltaNet feature map (short causal convolution, SiLU, per-head L2 normalisation)."""
import numpy as np
import pytest

from oracle import sla_oracle as orc


def test_convolution_against_a_library_routine_and_silu_closed_form():
    rng = np.random.default_rng(50)
    B, T, H, d, K = 2, 13, 2, 3, 4
    x, w = rng.normal(size=(B, T, H, d)), rng.normal(size=(H * d, K))
    out = orc.shortconv(x, w, normalize=False)
    xf = x.reshape(B, T, H * d)
    for b in range(B):
        for c in range(H * d):
            # causal correlation with taps w[c, 0..K-1] on x[t-K+1 .. t] = full convolution with the reversed taps
            y = np.convolve(xf[b, :, c], w[c, ::-1])[:T]
            np.testing.assert_allclose(out.reshape(B, T, -1)[b, :, c], y / (1 + np.exp(-y)), rtol=1e-12, atol=1e-13)
    # one tap of weight one: the map is SiLU itself
    o1 = orc.shortconv(x, np.ones((H * d, 1)), normalize=False)
    np.testing.assert_allclose(o1, x / (1 + np.exp(-x)), rtol=1e-13, atol=1e-14)


def test_normalised_rows_have_unit_norm_and_keep_their_direction():
    rng = np.random.default_rng(51)
    x, w = rng.normal(size=(2, 9, 3, 8)), rng.normal(size=(24, 4))
    z = orc.shortconv(x, w, normalize=False)
    zn = orc.shortconv(x, w, normalize=True, eps=1e-12)
    np.testing.assert_allclose(np.linalg.norm(zn, axis=-1), 1.0, rtol=1e-9)
    np.testing.assert_allclose(zn * np.linalg.norm(z, axis=-1, keepdims=True), z, rtol=1e-9, atol=1e-12)
    # eps sits inside the root: a zero row stays zero instead of dividing by zero
    z0 = orc.shortconv(np.zeros((1, 3, 1, 4)), np.ones((4, 2)), normalize=True)
    assert np.all(z0 == 0.0)


def test_causality_and_independence_of_batch_rows():
    rng = np.random.default_rng(52)
    x, w = rng.normal(size=(2, 10, 2, 4)), rng.normal(size=(8, 3))
    a = orc.shortconv(x, w, normalize=True)
    x2 = x.copy()
    x2[0, 6:] += 1.0                      # the future of row 0 changes
    b = orc.shortconv(x2, w, normalize=True)
    np.testing.assert_array_equal(a[0, :6], b[0, :6])
    np.testing.assert_array_equal(a[1], b[1])
    assert not np.allclose(a[0, 6], b[0, 6])


@pytest.mark.parametrize("normalize", [False, True])
@pytest.mark.parametrize("K", [1, 2, 4])
def test_backward_against_finite_differences(normalize, K):
    rng = np.random.default_rng(53 + K)
    x, w = rng.normal(size=(2, 7, 2, 3)), rng.normal(size=(6, K))
    dout = rng.normal(size=x.shape)
    dx, dw = orc.shortconv_backward(x, w, dout, normalize)
    loss = lambda: float((orc.shortconv(x, w, normalize) * dout).sum())
    eps = 1e-6
    for arr, grad in ((x, dx), (w, dw)):
        for fi in rng.choice(arr.size, size=min(12, arr.size), replace=False):
            idx = np.unravel_index(fi, arr.shape)
            old = arr[idx]
            arr[idx] = old + eps
            lp = loss()
            arr[idx] = old - eps
            lm = loss()
            arr[idx] = old
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - grad[idx]) <= 1e-6 * max(1.0, abs(fd)), (idx, fd, grad[idx])
