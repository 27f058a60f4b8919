"""Pins for the oracle's head-softmax gates (Eq. 4, Thm 3.2, Thm 3.3)."""
import numpy as np

from oracle import sla_oracle as orc


def test_gates_sum_to_one_and_positive():
    rng = np.random.default_rng(0)
    for H in (1, 2, 4, 8, 16, 5):
        G = orc.head_softmax(rng.normal(size=(7, 11, H)) * 3)
        assert np.all(G > 0)
        np.testing.assert_allclose(G.sum(-1), 1.0, rtol=0, atol=1e-14)


def test_single_head_gate_is_one():
    G = orc.head_softmax(np.array([[3.7], [-100.0], [0.0]]))
    np.testing.assert_array_equal(G, 1.0)


def test_two_heads_closed_form_is_sigmoid_of_difference():
    rng = np.random.default_rng(1)
    l = rng.normal(size=(50, 2)) * 4
    G = orc.head_softmax(l)
    np.testing.assert_allclose(G[:, 0], 1.0 / (1.0 + np.exp(-(l[:, 0] - l[:, 1]))), rtol=1e-13)


def test_uniform_logits_give_one_over_H_and_shift_invariance():
    G = orc.head_softmax(np.full((3, 8), 2.5))
    np.testing.assert_allclose(G, 1.0 / 8, rtol=1e-15)
    rng = np.random.default_rng(2)
    l = rng.normal(size=(9, 4))
    np.testing.assert_allclose(orc.head_softmax(l + 1000.0), orc.head_softmax(l), rtol=1e-12)


def test_large_logits_do_not_overflow():
    G = orc.head_softmax(np.array([[800.0, 799.0, -800.0]]))
    e = np.exp(-1.0)
    np.testing.assert_allclose(G[0], [1 / (1 + e), e / (1 + e), 0.0], atol=1e-15)


def test_sharpening_limit_is_one_hot_of_argmax():
    """Thm 3.2: softmax(lambda s) -> one_hot(argmax s); entropy decreases with lambda."""
    rng = np.random.default_rng(3)
    s = rng.normal(size=(20, 8))
    G = orc.head_softmax(1e4 * s)
    onehot = np.eye(8)[s.argmax(-1)]
    np.testing.assert_allclose(G, onehot, atol=1e-12)
    ent = []
    for lam in (0.5, 1.0, 2.0, 4.0, 8.0):
        P = orc.head_softmax(lam * s)
        ent.append(-(P * np.log(P + 1e-300)).sum(-1))
    ent = np.array(ent)
    assert np.all(np.diff(ent, axis=0) < 0)


def test_information_flow_coefficient_limit_is_kronecker_delta():
    """Thm 3.3: C(lambda) = sum_h Gq_h Gk_h -> delta(argmax sQ, argmax sK)."""
    rng = np.random.default_rng(4)
    sq, sk = rng.normal(size=(64, 4)), rng.normal(size=(64, 4))
    C = (orc.head_softmax(1e4 * sq) * orc.head_softmax(1e4 * sk)).sum(-1)
    np.testing.assert_allclose(C, (sq.argmax(-1) == sk.argmax(-1)).astype(float), atol=1e-12)
