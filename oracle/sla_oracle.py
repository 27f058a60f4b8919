"""ctypes front end of the fp64 CPU oracle (TEST INFRASTRUCTURE, not the product).

Only tests, the smoke check and the benchmark's CPU-baseline leg import this module.
It compiles ``sla_oracle.c`` with gcc on first use and marshals numpy fp64 arrays;
it contains no arithmetic of its own and imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

RETNET, GLA, GDN = 0, 1, 2
VARIANTS = {"retnet": RETNET, "gla": GLA, "gdn": GDN}

_HERE = Path(__file__).resolve().parent
_SO = _HERE / "libsla_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (no fast-math: fp64 IEEE semantics throughout)."""
    src = _HERE / "sla_oracle.c"
    hdr = _HERE / "sla_oracle.h"
    stale = (not _SO.exists()) or _SO.stat().st_mtime < max(src.stat().st_mtime, hdr.stat().st_mtime)
    if force or stale:
        tmp = _SO.with_suffix(f".so.{os.getpid()}.tmp")
        subprocess.run(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", str(tmp), str(src), "-lm"],
            check=True,
        )
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(str(build()))
        dp = ctypes.POINTER(ctypes.c_double)
        i, d = ctypes.c_int, ctypes.c_double
        lib.sla_oracle_num_threads.restype = i
        lib.sla_oracle_head_softmax.argtypes = [dp, ctypes.c_long, i, dp]
        lib.sla_oracle_head_softmax.restype = None
        lib.sla_oracle_forward.argtypes = [i] * 6 + [d] + [dp] * 10
        lib.sla_oracle_forward.restype = i
        lib.sla_oracle_backward.argtypes = [i] * 6 + [d] + [dp] * 18
        lib.sla_oracle_backward.restype = i
        lib.sla_oracle_decode_step.argtypes = [i] * 5 + [d] + [dp] * 9
        lib.sla_oracle_decode_step.restype = i
        lib.sla_oracle_decode_steps.argtypes = [i] * 6 + [d] + [dp] * 9
        lib.sla_oracle_decode_steps.restype = i
        lib.sla_oracle_shortconv.argtypes = [i] * 6 + [d] + [dp] * 3
        lib.sla_oracle_shortconv.restype = None
        lib.sla_oracle_shortconv_backward.argtypes = [i] * 6 + [d] + [dp] * 5
        lib.sla_oracle_shortconv_backward.restype = None
        lib.sla_oracle_gate_scores.argtypes = [ctypes.c_long, i, i, dp, dp, dp]
        lib.sla_oracle_gate_scores.restype = None
        lib.sla_oracle_gate_scores_backward.argtypes = [ctypes.c_long, i, i, dp, dp, dp, dp, dp]
        lib.sla_oracle_gate_scores_backward.restype = None
        lib.sla_oracle_out_proj.argtypes = [ctypes.c_long, i, i, dp, dp, dp]
        lib.sla_oracle_out_proj.restype = None
        lib.sla_oracle_out_proj_backward.argtypes = [ctypes.c_long, i, i, dp, dp, dp, dp, dp]
        lib.sla_oracle_out_proj_backward.restype = None
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().sla_oracle_num_threads())


def _f64(x):
    if x is None:
        return None
    if hasattr(x, "detach"):          # torch tensor (bf16 has no numpy dtype: widen first)
        x = x.detach().cpu().double().numpy()
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def _p(x):
    if x is None:
        return ctypes.POINTER(ctypes.c_double)()
    return x.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def head_softmax(logits):
    lg = _f64(logits)
    H = lg.shape[-1]
    out = np.empty_like(lg)
    _load().sla_oracle_head_softmax(_p(lg), lg.size // H, H, _p(out))
    return out


def _decay_shape(variant, B, T, H, d_k):
    return {RETNET: (H,), GLA: (B, T, H, d_k), GDN: (B, T, H)}[variant]


def forward(variant, q, k, v, log_decay, lq, lk, beta=None, h0=None, scale=1.0, want_ht=True):
    """Returns (o [B,T,H,d_v], ht [B,H,d_k,d_v] or None), fp64."""
    variant = VARIANTS.get(variant, variant)
    q, k, v, log_decay, beta, lq, lk, h0 = map(_f64, (q, k, v, log_decay, beta, lq, lk, h0))
    B, T, H, d_k = q.shape
    d_v = v.shape[-1]
    assert k.shape == q.shape and v.shape == (B, T, H, d_v)
    assert log_decay.shape == _decay_shape(variant, B, T, H, d_k), log_decay.shape
    assert lq.shape == (B, T, H) and lk.shape == (B, T, H)
    assert beta is None or beta.shape == (B, T, H)
    assert h0 is None or h0.shape == (B, H, d_k, d_v)
    o = np.zeros((B, T, H, d_v))
    ht = np.zeros((B, H, d_k, d_v)) if want_ht else None
    rc = _load().sla_oracle_forward(variant, B, T, H, d_k, d_v, float(scale), _p(q), _p(k), _p(v),
                                    _p(log_decay), _p(beta), _p(lq), _p(lk), _p(h0), _p(o), _p(ht))
    if rc != 0:
        raise ValueError("sla_oracle_forward rejected its arguments")
    return o, ht


def backward(variant, q, k, v, log_decay, lq, lk, dO, beta=None, h0=None, dht=None, scale=1.0):
    """Returns a dict of fp64 gradients: dq dk dv dlog_decay dbeta dlq dlk dh0."""
    variant = VARIANTS.get(variant, variant)
    q, k, v, log_decay, beta, lq, lk, h0, dO, dht = map(
        _f64, (q, k, v, log_decay, beta, lq, lk, h0, dO, dht))
    B, T, H, d_k = q.shape
    d_v = v.shape[-1]
    assert dO.shape == (B, T, H, d_v)
    assert log_decay.shape == _decay_shape(variant, B, T, H, d_k)
    g = dict(
        dq=np.zeros_like(q), dk=np.zeros_like(k), dv=np.zeros_like(v),
        dlog_decay=np.zeros_like(log_decay),
        dbeta=np.zeros((B, T, H)) if variant == GDN else None,
        dlq=np.zeros((B, T, H)), dlk=np.zeros((B, T, H)), dh0=np.zeros((B, H, d_k, d_v)),
    )
    rc = _load().sla_oracle_backward(
        variant, B, T, H, d_k, d_v, float(scale), _p(q), _p(k), _p(v), _p(log_decay), _p(beta),
        _p(lq), _p(lk), _p(h0), _p(dO), _p(dht), _p(g["dq"]), _p(g["dk"]), _p(g["dv"]),
        _p(g["dlog_decay"]), _p(g["dbeta"]), _p(g["dlq"]), _p(g["dlk"]), _p(g["dh0"]))
    if rc != 0:
        raise ValueError("sla_oracle_backward rejected its arguments")
    return g


def decode_step(variant, q_t, k_t, v_t, log_decay_t, lq_t, lk_t, state, beta_t=None, scale=1.0):
    """Updates ``state`` (a contiguous fp64 numpy array [Bdec,H,d_k,d_v]) in place; returns o_t."""
    variant = VARIANTS.get(variant, variant)
    assert isinstance(state, np.ndarray) and state.dtype == np.float64 and state.flags.c_contiguous
    q_t, k_t, v_t, log_decay_t, beta_t, lq_t, lk_t = map(
        _f64, (q_t, k_t, v_t, log_decay_t, beta_t, lq_t, lk_t))
    Bd, H, d_k = q_t.shape
    d_v = v_t.shape[-1]
    assert state.shape == (Bd, H, d_k, d_v)
    o = np.zeros((Bd, H, d_v))
    rc = _load().sla_oracle_decode_step(variant, Bd, H, d_k, d_v, float(scale), _p(q_t), _p(k_t),
                                        _p(v_t), _p(log_decay_t), _p(beta_t), _p(lq_t), _p(lk_t),
                                        _p(state), _p(o))
    if rc != 0:
        raise ValueError("sla_oracle_decode_step rejected its arguments")
    return o


def decode_steps(variant, q, k, v, log_decay, lq, lk, state, beta=None, scale=1.0):
    """n consecutive steps per sequence: q, k [Bdec,n,H,d_k], v [Bdec,n,H,d_v].  Updates ``state`` in place;
    returns o [Bdec,n,H,d_v]."""
    variant = VARIANTS.get(variant, variant)
    assert isinstance(state, np.ndarray) and state.dtype == np.float64 and state.flags.c_contiguous
    q, k, v, log_decay, beta, lq, lk = map(_f64, (q, k, v, log_decay, beta, lq, lk))
    Bd, n, H, d_k = q.shape
    d_v = v.shape[-1]
    assert state.shape == (Bd, H, d_k, d_v)
    assert log_decay.shape == _decay_shape(variant, Bd, n, H, d_k)
    o = np.zeros((Bd, n, H, d_v))
    rc = _load().sla_oracle_decode_steps(variant, Bd, n, H, d_k, d_v, float(scale), _p(q), _p(k), _p(v),
                                         _p(log_decay), _p(beta), _p(lq), _p(lk), _p(state), _p(o))
    if rc != 0:
        raise ValueError("sla_oracle_decode_steps rejected its arguments")
    return o


def gate_scores(x, W):
    """Eq. 4's score projection: x [..., H, d], W [d, H] -> s [..., H] with s[.., h] = x[.., h, :] @ W[:, h]."""
    x, W = _f64(x), _f64(W)
    H, d = x.shape[-2], x.shape[-1]
    assert W.shape == (d, H)
    s = np.zeros(x.shape[:-1])
    _load().sla_oracle_gate_scores(x.size // (H * d), H, d, _p(x), _p(W), _p(s))
    return s


def gate_scores_backward(x, W, ds, dx):
    """Adds ds W^T (per head) into the fp64 array dx (in place) and returns dW [d, H]."""
    x, W, ds = _f64(x), _f64(W), _f64(ds)
    H, d = x.shape[-2], x.shape[-1]
    assert isinstance(dx, np.ndarray) and dx.dtype == np.float64 and dx.flags.c_contiguous and dx.shape == x.shape
    dW = np.zeros((d, H))
    _load().sla_oracle_gate_scores_backward(x.size // (H * d), H, d, _p(x), _p(W), _p(ds), _p(dx), _p(dW))
    return dW


def out_proj(o, W):
    """Eq. 7's output projection: o [..., K] (the heads' outputs concatenated), W [K, N] -> y [..., N]."""
    o, W = _f64(o), _f64(W)
    K, N = W.shape
    assert o.shape[-1] == K
    y = np.zeros(o.shape[:-1] + (N,))
    _load().sla_oracle_out_proj(o.size // K, K, N, _p(o), _p(W), _p(y))
    return y


def out_proj_backward(o, W, dy):
    """Reverse of out_proj: returns (d_o [..., K], dW [K, N])."""
    o, W, dy = _f64(o), _f64(W), _f64(dy)
    K, N = W.shape
    assert o.shape[-1] == K and dy.shape == o.shape[:-1] + (N,)
    d_o, dW = np.zeros(o.shape), np.zeros((K, N))
    _load().sla_oracle_out_proj_backward(o.size // K, K, N, _p(o), _p(W), _p(dy), _p(d_o), _p(dW))
    return d_o, dW


SHORTCONV_EPS = 1e-6


def shortconv(x, w, normalize, eps=SHORTCONV_EPS):
    """Depthwise causal convolution + SiLU (+ per-head L2 normalisation): x [B,T,H,d], w [H*d,K] -> [B,T,H,d]."""
    x, w = _f64(x), _f64(w)
    B, T, H, d = x.shape
    assert w.shape[0] == H * d
    out = np.zeros_like(x)
    _load().sla_oracle_shortconv(B, T, H, d, w.shape[1], int(bool(normalize)), float(eps), _p(x), _p(w), _p(out))
    return out


def shortconv_backward(x, w, dout, normalize, eps=SHORTCONV_EPS):
    """Returns (dx [B,T,H,d], dw [H*d,K])."""
    x, w, dout = _f64(x), _f64(w), _f64(dout)
    B, T, H, d = x.shape
    dx, dw = np.zeros_like(x), np.zeros_like(w)
    _load().sla_oracle_shortconv_backward(B, T, H, d, w.shape[1], int(bool(normalize)), float(eps), _p(x), _p(w),
                                          _p(dout), _p(dx), _p(dw))
    return dx, dw
