"""fp64 numpy statement of the chunkwise-parallel evaluation order (the paper's "Chunkwise
Parallel Training" paragraph) for the three variants, forward and backward.

It is a test-side cross-check that the chunk algebra the CUDA kernels implement is an exact
re-association of the recurrence: it is compared with the oracle in test_chunk_ref.py.  It
calls neither the oracle nor the CUDA library.

Notation per (batch, head) and chunk: b_i = inclusive cumulative log-decay inside the chunk,
S = state at the chunk start, qt = scale*Gq*q; RetNet/GLA: kt = Gk*k, vt = v; GDN: kt = k,
vt = Gk*v.
"""
import numpy as np


def softmax_heads(l):
    z = np.exp(l - l.max(-1, keepdims=True))
    return z / z.sum(-1, keepdims=True)


def _chunk_logdecay(variant, log_decay, b, h, sl, dk):
    n = sl.stop - sl.start
    if variant == "retnet":
        return np.full((n, dk), log_decay[h])
    if variant == "gla":
        return log_decay[b, sl, h]
    return np.repeat(log_decay[b, sl, h][:, None], dk, axis=1)


def _gdn_chunk_fwd(qt, kt, vt, bs, beta, S):
    """bs: scalar cumulative log-decay [c]."""
    c = qt.shape[0]
    Gam = np.exp(bs)
    D = np.tril(np.exp(bs[:, None] - bs[None, :]))                 # j <= i
    L = np.tril((beta[:, None] * kt) @ kt.T * D, -1)
    Tm = np.linalg.inv(np.eye(c) + L)
    Kbg = (beta * Gam)[:, None] * kt
    Vb = beta[:, None] * vt
    W, U0 = Tm @ Kbg, Tm @ Vb
    U = U0 - W @ S
    Pq = (qt @ kt.T) * D
    O = Gam[:, None] * (qt @ S) + Pq @ U
    E = np.exp(bs[-1] - bs)
    S_next = np.exp(bs[-1]) * S + (E[:, None] * kt).T @ U
    return O, S_next, dict(Gam=Gam, D=D, L=L, Tm=Tm, Kbg=Kbg, Vb=Vb, W=W, U0=U0, U=U, Pq=Pq, E=E)


def forward(variant, q, k, v, log_decay, lq, lk, beta=None, h0=None, scale=1.0, chunk=64,
            return_states=False):
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    Gq, Gk = softmax_heads(lq), softmax_heads(lk)
    o = np.zeros((B, T, H, dv))
    ht = np.zeros((B, H, dk, dv))
    states = {}
    for b in range(B):
        for h in range(H):
            S = np.zeros((dk, dv)) if h0 is None else h0[b, h].copy()
            for n, t0 in enumerate(range(0, T, chunk)):
                sl = slice(t0, min(t0 + chunk, T))
                states[(b, h, n)] = S.copy()
                qt = scale * Gq[b, sl, h, None] * q[b, sl, h]
                bb = np.cumsum(_chunk_logdecay(variant, log_decay, b, h, sl, dk), axis=0)
                if variant == "gdn":
                    vt = Gk[b, sl, h, None] * v[b, sl, h]
                    O, S, _ = _gdn_chunk_fwd(qt, k[b, sl, h], vt, bb[:, 0], beta[b, sl, h], S)
                else:
                    kt = Gk[b, sl, h, None] * k[b, sl, h]
                    Qh, Kh = qt * np.exp(bb), kt * np.exp(-bb)
                    A = np.tril(Qh @ Kh.T)
                    O = A @ v[b, sl, h] + Qh @ S
                    S = np.exp(bb[-1])[:, None] * (S + Kh.T @ v[b, sl, h])
                o[b, sl, h] = O
            ht[b, h] = S
    if return_states:
        return o, ht, states
    return o, ht


def backward(variant, q, k, v, log_decay, lq, lk, dO, beta=None, h0=None, dht=None, scale=1.0,
             chunk=64):
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    Gq, Gk = softmax_heads(lq), softmax_heads(lk)
    _, ht, states = forward(variant, q, k, v, log_decay, lq, lk, beta, h0, scale, chunk, True)
    dq, dk_, dv_ = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v)
    dg = np.zeros_like(log_decay)
    dbeta = np.zeros((B, T, H))
    dGq, dGk = np.zeros((B, T, H)), np.zeros((B, T, H))
    dh0 = np.zeros((B, H, dk, dv))
    starts = list(range(0, T, chunk))
    for b in range(B):
        for h in range(H):
            dS = np.zeros((dk, dv)) if dht is None else dht[b, h].copy()      # grad wrt S_next
            for n in reversed(range(len(starts))):
                sl = slice(starts[n], min(starts[n] + chunk, T))
                S = states[(b, h, n)]
                qt = scale * Gq[b, sl, h, None] * q[b, sl, h]
                bb = np.cumsum(_chunk_logdecay(variant, log_decay, b, h, sl, dk), axis=0)
                dOc = dO[b, sl, h]
                if variant != "gdn":
                    kt = Gk[b, sl, h, None] * k[b, sl, h]
                    V = v[b, sl, h]
                    Qh, Kh = qt * np.exp(bb), kt * np.exp(-bb)
                    A = np.tril(Qh @ Kh.T)
                    S_next = np.exp(bb[-1])[:, None] * (S + Kh.T @ V)
                    dA = np.tril(dOc @ V.T)
                    dZ = np.exp(bb[-1])[:, None] * dS
                    dQh = dA @ Kh + dOc @ S.T
                    dKh = dA.T @ Qh + V @ dZ.T
                    dV = A.T @ dOc + Kh @ dZ
                    db = Qh * dQh - Kh * dKh
                    db[-1] += (dS * S_next).sum(1)
                    dS = Qh.T @ dOc + dZ
                    dqt, dkt = dQh * np.exp(bb), dKh * np.exp(-bb)
                    dgc = np.flip(np.cumsum(np.flip(db, 0), 0), 0)
                    if variant == "gla":
                        dg[b, sl, h] = dgc
                    dk_[b, sl, h] = Gk[b, sl, h, None] * dkt
                    dGk[b, sl, h] = (k[b, sl, h] * dkt).sum(1)
                    dv_[b, sl, h] = dV
                else:
                    kt = k[b, sl, h]
                    vt = Gk[b, sl, h, None] * v[b, sl, h]
                    bt = beta[b, sl, h]
                    bs = bb[:, 0]
                    _, _, f = _gdn_chunk_fwd(qt, kt, vt, bs, bt, S)
                    Gam, D, E, Tm, W, U0, U, Pq, L = (f[n_] for n_ in
                                                     ("Gam", "D", "E", "Tm", "W", "U0", "U", "Pq", "L"))
                    KdS = kt @ dS                                   # [c, dv]
                    dU = Pq.T @ dOc + E[:, None] * KdS
                    dOS = dOc @ S.T                                 # [c, dk]
                    dPq = np.tril(dOc @ U.T)
                    dQK = dPq * D
                    dqt = Gam[:, None] * dOS + dQK @ kt
                    UdS = U @ dS.T                                  # [c, dk]
                    dkt = dQK.T @ qt + E[:, None] * UdS
                    dW = -dU @ S.T
                    dKbg, dVb = Tm.T @ dW, Tm.T @ dU
                    dL = -np.tril(dKbg @ W.T + dVb @ U0.T, -1)
                    dM = dL * D
                    KK = kt @ kt.T
                    dbt = (dM * KK).sum(1) + Gam * (dKbg * kt).sum(1) + (dVb * vt).sum(1)
                    dkt += bt[:, None] * (dM @ kt) + (bt[:, None] * dM).T @ kt + (bt * Gam)[:, None] * dKbg
                    dvt = bt[:, None] * dVb
                    db = Gam * (dOS * qt).sum(1) + bt * Gam * (dKbg * kt).sum(1)
                    X = dPq * Pq + dL * L
                    db += X.sum(1) - X.sum(0)
                    e = E * (kt * UdS).sum(1)
                    db -= e
                    db[-1] += e.sum() + np.exp(bs[-1]) * (dS * S).sum()
                    dS = (Gam[:, None] * qt).T @ dOc + np.exp(bs[-1]) * dS - W.T @ dU
                    dg[b, sl, h] = np.flip(np.cumsum(np.flip(db)))
                    dbeta[b, sl, h] = dbt
                    dk_[b, sl, h] = dkt
                    dv_[b, sl, h] = Gk[b, sl, h, None] * dvt
                    dGk[b, sl, h] = (v[b, sl, h] * dvt).sum(1)
                dq[b, sl, h] = scale * Gq[b, sl, h, None] * dqt
                dGq[b, sl, h] = scale * (q[b, sl, h] * dqt).sum(1)
            dh0[b, h] = dS
    dlq = Gq * (dGq - (Gq * dGq).sum(-1, keepdims=True))
    dlk = Gk * (dGk - (Gk * dGk).sum(-1, keepdims=True))
    return dict(dq=dq, dk=dk_, dv=dv_, dlog_decay=dg, dbeta=dbeta if variant == "gdn" else None,
                dlq=dlq, dlk=dlk, dh0=dh0)
