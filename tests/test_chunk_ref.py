"""The chunkwise evaluation order (any chunk size, ragged tail included) reproduces the
token-by-token oracle: forward, final state and every gradient."""
import numpy as np
import pytest

from oracle import sla_oracle as orc
from tests import chunk_ref
from tests.test_oracle_recurrence import draw


@pytest.mark.parametrize("variant", ["retnet", "gla", "gdn"])
@pytest.mark.parametrize("chunk", [1, 2, 16, 64, 100])
def test_chunkwise_forward_equals_recurrent(variant, chunk):
    x, h0 = draw(variant, B=1, T=75, H=2, dk=6, dv=5, seed=40, unit_k=True)
    o, ht = orc.forward(variant, **x, h0=h0, scale=0.9)
    o2, ht2 = chunk_ref.forward(variant, x["q"], x["k"], x["v"], x["log_decay"], x["lq"], x["lk"],
                                beta=x["beta"], h0=h0, scale=0.9, chunk=chunk)
    np.testing.assert_allclose(o2, o, rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(ht2, ht, rtol=1e-9, atol=1e-11)


@pytest.mark.parametrize("variant", ["retnet", "gla", "gdn"])
@pytest.mark.parametrize("chunk", [4, 16, 64])
def test_chunkwise_backward_equals_recurrent(variant, chunk):
    x, h0 = draw(variant, B=1, T=50, H=2, dk=6, dv=5, seed=41, unit_k=True)
    rng = np.random.default_rng(42)
    dO, dht = rng.normal(size=x["v"].shape), rng.normal(size=h0.shape)
    g = orc.backward(variant, x["q"], x["k"], x["v"], x["log_decay"], x["lq"], x["lk"], dO,
                     beta=x["beta"], h0=h0, dht=dht, scale=0.9)
    g2 = chunk_ref.backward(variant, x["q"], x["k"], x["v"], x["log_decay"], x["lq"], x["lk"], dO,
                            beta=x["beta"], h0=h0, dht=dht, scale=0.9, chunk=chunk)
    for name in ("dq", "dk", "dv", "dlq", "dlk", "dh0", "dbeta", "dlog_decay"):
        if g[name] is None or (variant == "retnet" and name == "dlog_decay"):
            continue
        np.testing.assert_allclose(g2[name], g[name], rtol=1e-8, atol=1e-10, err_msg=name)
