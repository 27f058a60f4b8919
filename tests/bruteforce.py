"""Independent numpy statements used to pin the oracle (tiny inputs only).

Nothing here calls the oracle or the CUDA library.  Each function writes out a
definition that differs in form from the token-by-token recurrence: an explicit
O(T^2) decay-masked sum (Eq. 3 with the causal sum of App. A and the decays of
Eq. 10/12 unrolled) and, for the delta rule, explicit products of the per-token
transition matrices implied by Eq. 14-15.
"""
import numpy as np


def softmax_heads(logits):
    z = np.exp(logits - logits.max(axis=-1, keepdims=True))
    return z / z.sum(axis=-1, keepdims=True)


def quadratic_decay_attention(q, k, v, logdecay, h0=None):
    """o_t = sum_{j<=t} sum_d q_td k_jd exp(Bc_td - Bc_jd) v_j  (+ (q_t*exp(Bc_t)) h0).

    q,k [T,dk]; v [T,dv]; logdecay [T,dk] (per token, per key dimension); Bc = inclusive
    cumulative sum over tokens.  One (batch, head) sequence, gates already folded in.
    """
    T, dk = q.shape
    Bc = np.cumsum(logdecay, axis=0)
    o = np.zeros((T, v.shape[1]))
    for t in range(T):
        for j in range(t + 1):
            w = np.sum(q[t] * k[j] * np.exp(Bc[t] - Bc[j]))
            o[t] += w * v[j]
        if h0 is not None:
            o[t] += (q[t] * np.exp(Bc[t])) @ h0
    return o


def delta_rule_by_transition_products(q, k, vw, g, beta, h0=None):
    """S_t = M_t S_{t-1} + beta_t k_t^T vw_t with M_t = exp(g_t)(I - beta_t k_t^T k_t), written as
    S_t = sum_{j<=t} (M_t ... M_{j+1}) beta_j k_j^T vw_j + (M_t ... M_1) h0 ; o_t = q_t S_t."""
    T, dk = k.shape
    dv = vw.shape[1]
    M = [np.exp(g[t]) * (np.eye(dk) - beta[t] * np.outer(k[t], k[t])) for t in range(T)]
    o = np.zeros((T, dv))
    S_last = None
    for t in range(T):
        S = np.zeros((dk, dv))
        for j in range(t + 1):
            P = np.eye(dk)
            for s in range(j + 1, t + 1):
                P = M[s] @ P
            S += P @ (beta[j] * np.outer(k[j], vw[j]))
        if h0 is not None:
            P = np.eye(dk)
            for s in range(0, t + 1):
                P = M[s] @ P
            S += P @ h0
        o[t] = q[t] @ S
        S_last = S
    return o, S_last


def sla_bruteforce(variant, q, k, v, log_decay, lq, lk, beta=None, h0=None, scale=1.0):
    """Whole layer [B,T,H,*] by the definitions above (Eq. 3-4 gates absorbed as in App. A)."""
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    Gq, Gk = softmax_heads(lq), softmax_heads(lk)
    o = np.zeros((B, T, H, dv))
    for b in range(B):
        for h in range(H):
            qt = scale * Gq[b, :, h, None] * q[b, :, h]
            hh = None if h0 is None else h0[b, h]
            if variant == "gdn":
                vw = Gk[b, :, h, None] * v[b, :, h]
                o[b, :, h], _ = delta_rule_by_transition_products(
                    qt, k[b, :, h], vw, log_decay[b, :, h], beta[b, :, h], hh)
            else:
                kt = Gk[b, :, h, None] * k[b, :, h]
                if variant == "retnet":
                    ld = np.full((T, dk), log_decay[h])
                else:
                    ld = log_decay[b, :, h]
                o[b, :, h] = quadratic_decay_attention(qt, kt, v[b, :, h], ld, hh)
    return o
