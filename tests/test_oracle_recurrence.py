"""Pins for the oracle's forward / decode: brute-force quadratic and transition-product forms,
closed forms, cross-variant reductions and state-carry identities (Eq. 2-3, 5-7, 10-16, App. A)."""
import numpy as np
import pytest

from oracle import sla_oracle as orc
from tests import bruteforce as bf


def draw(variant, B=2, T=12, H=3, dk=5, dv=4, seed=0, unit_k=False):
    rng = np.random.default_rng(seed)
    q, k = rng.normal(size=(B, T, H, dk)), rng.normal(size=(B, T, H, dk))
    v = rng.normal(size=(B, T, H, dv))
    lq, lk = rng.normal(size=(B, T, H)), rng.normal(size=(B, T, H))
    beta = None
    if variant == "retnet":
        ld = np.log(1.0 - 2.0 ** (-2.0 - np.arange(H)))
    elif variant == "gla":
        ld = -np.abs(rng.normal(size=(B, T, H, dk))) * 0.3
    else:
        ld = -np.abs(rng.normal(size=(B, T, H))) * 0.3
        beta = 1.0 / (1.0 + np.exp(-rng.normal(size=(B, T, H))))
        if unit_k:
            k = k / np.linalg.norm(k, axis=-1, keepdims=True)
    h0 = rng.normal(size=(B, H, dk, dv))
    return dict(q=q, k=k, v=v, log_decay=ld, lq=lq, lk=lk, beta=beta), h0


def head_decay(variant, ld, h):
    """log-decay of head h as a one-head tensor."""
    return ld[h:h + 1] if variant == "retnet" else ld[:, :, h:h + 1]


@pytest.mark.parametrize("variant", ["retnet", "gla", "gdn"])
@pytest.mark.parametrize("with_h0", [False, True])
def test_forward_matches_bruteforce(variant, with_h0):
    x, h0 = draw(variant, seed=10)
    h0 = h0 if with_h0 else None
    o, _ = orc.forward(variant, **x, h0=h0, scale=0.7)
    ref = bf.sla_bruteforce(variant, x["q"], x["k"], x["v"], x["log_decay"], x["lq"], x["lk"],
                            beta=x["beta"], h0=h0, scale=0.7)
    np.testing.assert_allclose(o, ref, rtol=1e-10, atol=1e-12)


def test_no_decay_uniform_gates_is_masked_matmul_over_H_squared():
    """g = 0 and equal logits: o = tril(Q K^T) V / H^2  (Eq. 2 with a causal mask)."""
    x, _ = draw("gla", B=1, T=9, H=4, seed=11)
    x["log_decay"][:] = 0.0
    x["lq"][:] = 0.3
    x["lk"][:] = -1.2
    o, ht = orc.forward("gla", **x)
    for h in range(4):
        Q, K, V = x["q"][0, :, h], x["k"][0, :, h], x["v"][0, :, h]
        np.testing.assert_allclose(o[0, :, h], np.tril(Q @ K.T) @ V / 16.0, rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(ht[0, h], K.T @ V / 4.0, rtol=1e-12, atol=1e-13)
    x["log_decay"] = np.zeros(4)
    o2, _ = orc.forward("retnet", **x)
    np.testing.assert_allclose(o2, o, rtol=1e-13)


def test_retnet_mask_closed_form_and_gla_with_constant_decay_is_retnet():
    x, h0 = draw("retnet", B=1, T=10, H=2, seed=12)
    o, ht = orc.forward("retnet", **x, h0=h0)
    Gq, Gk = bf.softmax_heads(x["lq"]), bf.softmax_heads(x["lk"])
    t = np.arange(10)
    for h in range(2):
        gam = np.exp(x["log_decay"][h])
        Dm = np.tril(gam ** (t[:, None] - t[None, :]).clip(0))
        Q = Gq[0, :, h, None] * x["q"][0, :, h]
        K = Gk[0, :, h, None] * x["k"][0, :, h]
        ref = ((Q @ K.T) * Dm) @ x["v"][0, :, h] + (gam ** (t + 1))[:, None] * (Q @ h0[0, h])
        np.testing.assert_allclose(o[0, :, h], ref, rtol=1e-11, atol=1e-12)
    g = dict(x)
    g["log_decay"] = np.broadcast_to(x["log_decay"][None, None, :, None], x["q"].shape).copy()
    o2, ht2 = orc.forward("gla", **g, h0=h0)
    np.testing.assert_allclose(o2, o, rtol=1e-13)
    np.testing.assert_allclose(ht2, ht, rtol=1e-13)


@pytest.mark.parametrize("variant", ["retnet", "gla", "gdn"])
def test_single_head_reduces_to_base_and_gates_absorb(variant):
    """H = 1: gates are 1.  H > 1: SLA-X(q,k,v) = X(Gq q, Gk k, v)  (GDN: X(Gq q, k, Gk v)), run
    head by head through the H = 1 oracle (App. A)."""
    x, h0 = draw(variant, seed=13)
    o, ht = orc.forward(variant, **x, h0=h0)
    Gq, Gk = bf.softmax_heads(x["lq"]), bf.softmax_heads(x["lk"])
    B, T, H, dk = x["q"].shape
    for h in range(H):
        q1 = (Gq[..., h, None] * x["q"][:, :, h])[:, :, None]
        k1 = x["k"][:, :, h][:, :, None]
        v1 = x["v"][:, :, h][:, :, None]
        if variant == "gdn":
            v1 = v1 * Gk[..., h, None, None]
        else:
            k1 = k1 * Gk[..., h, None, None]
        ld = head_decay(variant, x["log_decay"], h)
        bt = None if x["beta"] is None else x["beta"][:, :, h:h + 1]
        zeros = np.zeros((B, T, 1))
        o1, ht1 = orc.forward(variant, q1, k1, v1, ld, zeros + 5.0, zeros - 3.0, beta=bt,
                              h0=h0[:, h:h + 1])
        np.testing.assert_allclose(o1[:, :, 0], o[:, :, h], rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(ht1[:, 0], ht[:, h], rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("variant", ["retnet", "gla", "gdn"])
def test_uniform_logits_scale_output(variant):
    """All three variants are linear in q and in the key-side gated operand: equal logits give
    the H = 1-gate result divided by H^2."""
    x, _ = draw(variant, seed=14)
    H = x["q"].shape[2]
    x["lq"][:] = 1.0
    x["lk"][:] = 2.0
    o, _ = orc.forward(variant, **x)
    base = bf.sla_bruteforce(variant, x["q"], x["k"], x["v"], x["log_decay"], x["lq"], x["lk"],
                             beta=x["beta"])
    np.testing.assert_allclose(o, base, rtol=1e-10, atol=1e-12)
    # the same inputs with every gate forced to 1 (H separate single-head problems), over H^2
    for h in range(H):
        ld = head_decay(variant, x["log_decay"], h)
        bt = None if x["beta"] is None else x["beta"][:, :, h:h + 1]
        z = np.zeros(x["lq"].shape[:2] + (1,))
        o1, _ = orc.forward(variant, x["q"][:, :, h:h + 1], x["k"][:, :, h:h + 1],
                            x["v"][:, :, h:h + 1], ld, z, z, beta=bt)
        np.testing.assert_allclose(o[:, :, h], o1[:, :, 0] / (H * H), rtol=1e-11, atol=1e-13)


def test_one_hot_routing_blocks_mismatched_heads():
    """Thm 3.3 at the layer level: keys routed to head 0, queries to head 1 => o == 0."""
    x, _ = draw("gla", B=1, T=8, H=2, seed=15)
    x["lk"][..., 0], x["lk"][..., 1] = 800.0, -800.0
    x["lq"][..., 0], x["lq"][..., 1] = -800.0, 800.0
    o, _ = orc.forward("gla", **x)
    assert np.abs(o).max() < 1e-300 or np.abs(o).max() == 0.0


def test_gdn_zero_log_decay_is_the_printed_delta_rule():
    """g = 0: S_t = S_{t-1} + k^T beta (Gk v - k S_{t-1}) exactly as Eq. 14-16 print it."""
    x, h0 = draw("gdn", B=1, T=7, H=2, seed=16)
    x["log_decay"][:] = 0.0
    o, ht = orc.forward("gdn", **x, h0=h0)
    Gq, Gk = bf.softmax_heads(x["lq"]), bf.softmax_heads(x["lk"])
    for h in range(2):
        S = h0[0, h].copy()
        for t in range(7):
            kk, vv = x["k"][0, t, h], x["v"][0, t, h]
            vnew = x["beta"][0, t, h] * (Gk[0, t, h] * vv - kk @ S)
            S = S + np.outer(kk, vnew)
            np.testing.assert_allclose(o[0, t, h], (Gq[0, t, h] * x["q"][0, t, h]) @ S, rtol=1e-12)
        np.testing.assert_allclose(ht[0, h], S, rtol=1e-12)


def test_gdn_beta_zero_only_decays_and_overwrite_identity():
    x, h0 = draw("gdn", B=1, T=6, H=2, seed=17, unit_k=True)
    xb = dict(x)
    xb["beta"] = np.zeros_like(x["beta"])
    o, ht = orc.forward("gdn", **xb, h0=h0)
    tot = np.exp(x["log_decay"].sum(1))[0]                     # [H]
    np.testing.assert_allclose(ht[0], tot[:, None, None] * h0[0], rtol=1e-12)
    o0, _ = orc.forward("gdn", **xb)
    assert np.abs(o0).max() == 0.0
    # unit-norm keys: k_t S_t = (1 - beta_t) alpha_t k_t S_{t-1} + beta_t Gk v_t  (beta = 1: exact recall)
    Gk = bf.softmax_heads(x["lk"])
    S_prev = h0.copy()
    for t in range(6):
        xt = {n: (a[:, t:t + 1] if n != "beta" else a[:, t:t + 1]) for n, a in x.items()}
        _, S_t = orc.forward("gdn", **xt, h0=S_prev)
        for h in range(2):
            kk, al, bt = x["k"][0, t, h], np.exp(x["log_decay"][0, t, h]), x["beta"][0, t, h]
            lhs = kk @ S_t[0, h]
            rhs = (1 - bt) * al * (kk @ S_prev[0, h]) + bt * Gk[0, t, h] * x["v"][0, t, h]
            np.testing.assert_allclose(lhs, rhs, rtol=1e-11, atol=1e-13)
        S_prev = S_t


def test_gdn_orthonormal_keys_reduce_to_linear_attention():
    """Orthonormal keys, T <= d_k, h0 = 0, g = 0: the erase term vanishes, so
    o_t = sum_{j<=t} (q_t . k_j) beta_j Gk_j v_j."""
    rng = np.random.default_rng(18)
    T, dk, dv = 5, 6, 3
    Qm, _ = np.linalg.qr(rng.normal(size=(dk, dk)))
    k = Qm[:T][None, :, None, :]
    q, v = rng.normal(size=(1, T, 1, dk)), rng.normal(size=(1, T, 1, dv))
    beta = rng.uniform(0.1, 0.9, size=(1, T, 1))
    z = np.zeros((1, T, 1))
    o, _ = orc.forward("gdn", q, k, v, z, z, z, beta=beta)
    ref = np.tril(q[0, :, 0] @ k[0, :, 0].T) @ (beta[0, :, 0, None] * v[0, :, 0])
    np.testing.assert_allclose(o[0, :, 0], ref, rtol=1e-11, atol=1e-13)


@pytest.mark.parametrize("variant", ["retnet", "gla", "gdn"])
def test_state_carry_and_decode_agree_with_one_pass(variant):
    x, h0 = draw(variant, T=11, seed=19)
    o, ht = orc.forward(variant, **x, h0=h0, scale=1.3)
    cut = 4

    def part(a, sl):
        return a if (a is None or a.ndim == 1) else a[:, sl]

    o1, h1 = orc.forward(variant, **{n: part(a, slice(0, cut)) for n, a in x.items()}, h0=h0, scale=1.3)
    o2, h2 = orc.forward(variant, **{n: part(a, slice(cut, None)) for n, a in x.items()}, h0=h1, scale=1.3)
    np.testing.assert_allclose(np.concatenate([o1, o2], 1), o, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(h2, ht, rtol=1e-12, atol=1e-13)
    state = np.ascontiguousarray(h0.copy())
    for t in range(11):
        ld = x["log_decay"] if variant == "retnet" else x["log_decay"][:, t]
        bt = None if x["beta"] is None else x["beta"][:, t]
        ot = orc.decode_step(variant, x["q"][:, t], x["k"][:, t], x["v"][:, t], ld, x["lq"][:, t],
                             x["lk"][:, t], state, beta_t=bt, scale=1.3)
        np.testing.assert_allclose(ot, o[:, t], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(state, ht, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("variant", ["retnet", "gla", "gdn"])
def test_multi_token_decode_is_the_single_step_repeated(variant):
    """decode_steps over n tokens = n decode_step calls on the token slices (same state, same outputs), and two calls
    of 3 and 4 tokens = one call of 7."""
    x, h0 = draw(variant, T=7, seed=23)
    s_multi = np.ascontiguousarray(h0.copy())
    o_multi = orc.decode_steps(variant, x["q"], x["k"], x["v"], x["log_decay"], x["lq"], x["lk"], s_multi,
                               beta=x["beta"], scale=0.7)
    s_one = np.ascontiguousarray(h0.copy())
    for t in range(7):
        ld = x["log_decay"] if variant == "retnet" else x["log_decay"][:, t]
        bt = None if x["beta"] is None else x["beta"][:, t]
        ot = orc.decode_step(variant, x["q"][:, t], x["k"][:, t], x["v"][:, t], ld, x["lq"][:, t], x["lk"][:, t],
                             s_one, beta_t=bt, scale=0.7)
        np.testing.assert_allclose(o_multi[:, t], ot, rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(s_multi, s_one, rtol=1e-13, atol=1e-14)
    s_split = np.ascontiguousarray(h0.copy())
    part = lambda a, sl: a if (a is None or a.ndim == 1) else np.ascontiguousarray(a[:, sl])
    outs = []
    for sl in (slice(0, 3), slice(3, 7)):
        outs.append(orc.decode_steps(variant, part(x["q"], sl), part(x["k"], sl), part(x["v"], sl),
                                     part(x["log_decay"], sl), part(x["lq"], sl), part(x["lk"], sl), s_split,
                                     beta=part(x["beta"], sl), scale=0.7))
    np.testing.assert_allclose(np.concatenate(outs, 1), o_multi, rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(s_split, s_multi, rtol=1e-13, atol=1e-14)


def test_bad_arguments_are_rejected():
    z = np.zeros((1, 2, 1, 2))
    with pytest.raises(ValueError):
        orc.forward("gdn", z, z, z, np.zeros((1, 2, 1)), np.zeros((1, 2, 1)), np.zeros((1, 2, 1)))
