"""Thin ctypes binding of libsla.so: argument marshalling only, every step runs in the CUDA kernels.

The functions carry the names of the C entry points (include/sla.h).  Tensors are torch CUDA
tensors used purely as device memory; the current torch stream is passed to the library.
There is no fallback: if the shared library is missing or a call is refused, an exception is raised.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
_SO = _PKG / "libsla.so"

SLA_RETNET, SLA_GLA, SLA_GDN = 0, 1, 2
SLA_FP32, SLA_BF16 = 0, 1
SLA_FLAG_FORCE_GENERIC = 1
SLA_FLAG_SAVE_FOR_BACKWARD = 2
VARIANTS = {"retnet": SLA_RETNET, "gla": SLA_GLA, "gdn": SLA_GDN}
DTYPES = {"fp32": SLA_FP32, "bf16": SLA_BF16, torch.float32: SLA_FP32, torch.bfloat16: SLA_BF16}
EXPORTS = (
    "sla_plan_create", "sla_plan_destroy", "sla_plan_workspace_bytes", "sla_plan_poll",
    "sla_plan_last_launch_count", "sla_plan_set_kernel_timing", "sla_plan_kernel_timing_collect",
    "sla_plan_kernel_timing_get", "sla_status_string", "sla_forward", "sla_backward", "sla_decode_step",
    "sla_forward_noalloc", "sla_plan_selftest_timeout", "sla_decode_steps", "sla_gate_scores_forward",
    "sla_gate_scores_backward", "sla_plan_gate_scores_workspace_bytes", "sla_shortconv_forward",
    "sla_shortconv_backward", "sla_plan_shortconv_workspace_bytes", "sla_plan_set_sequences",
    "sla_out_proj_forward", "sla_out_proj_backward",
)
SLA_NOALLOC_SCRATCH_BYTES = 32 << 20


class SLAError(RuntimeError):
    def __init__(self, call: str, status: int, text: str):
        super().__init__(f"{call} failed: status {status} ({text})")
        self.status = status


class sla_desc(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32), ("variant", ctypes.c_int32), ("io_dtype", ctypes.c_int32),
        ("B", ctypes.c_int32), ("T", ctypes.c_int32), ("H", ctypes.c_int32),
        ("d_k", ctypes.c_int32), ("d_v", ctypes.c_int32), ("chunk", ctypes.c_int32),
        ("scale", ctypes.c_float), ("flags", ctypes.c_uint32),
    ]


_lib = None


def lib():
    """Load libsla.so (built in-tree by paper_2602_01744_b200.build); raises if it is absent."""
    global _lib
    if _lib is None:
        try:                                    # (re)build in-tree when the sources are newer than the library
            from . import build as _build
            _build.build()
        except Exception as e:                  # no nvcc here: an existing, current library is still fine
            if not _SO.exists():
                raise FileNotFoundError(
                    f"{_SO} is missing and could not be built ({e}): run `python -m paper_2602_01744_b200.build` "
                    "(there is no fallback path)") from e
        if not _SO.exists():
            raise FileNotFoundError(
                f"{_SO} is missing: run `python -m paper_2602_01744_b200.build` (there is no fallback path)")
        L = ctypes.CDLL(str(_SO))
        vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
        L.sla_plan_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(sla_desc)]
        L.sla_plan_destroy.argtypes = [vp]
        L.sla_plan_workspace_bytes.argtypes = [vp, ctypes.POINTER(sz), ctypes.POINTER(sz)]
        L.sla_plan_poll.argtypes = [vp]
        L.sla_plan_selftest_timeout.argtypes = [vp, vp]
        L.sla_plan_selftest_timeout.restype = ctypes.c_int
        L.sla_plan_last_launch_count.argtypes = [vp]
        L.sla_plan_last_launch_count.restype = i32
        L.sla_plan_set_kernel_timing.argtypes = [vp, i32]
        L.sla_plan_kernel_timing_collect.argtypes = [vp, ctypes.POINTER(i32)]
        L.sla_plan_kernel_timing_get.argtypes = [vp, i32, ctypes.POINTER(ctypes.c_char_p), ctypes.POINTER(i32),
                                                 ctypes.POINTER(ctypes.c_float)]
        L.sla_status_string.argtypes = [ctypes.c_int]
        L.sla_status_string.restype = ctypes.c_char_p
        L.sla_forward.argtypes = [vp] * 11 + [vp, sz, vp]
        L.sla_forward_noalloc.argtypes = [vp] * 12
        L.sla_forward_noalloc.restype = ctypes.c_int
        L.sla_backward.argtypes = [vp] * 19 + [vp, sz, vp]
        L.sla_decode_step.argtypes = [vp, i32] + [vp] * 10
        L.sla_decode_steps.argtypes = [vp, i32, i32] + [vp] * 10
        L.sla_decode_steps.restype = ctypes.c_int
        L.sla_plan_set_sequences.argtypes = [vp, ctypes.POINTER(i32), i32]
        L.sla_plan_set_sequences.restype = ctypes.c_int
        L.sla_shortconv_forward.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp]
        L.sla_shortconv_forward.restype = ctypes.c_int
        L.sla_shortconv_backward.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp, vp, vp, sz, vp]
        L.sla_shortconv_backward.restype = ctypes.c_int
        L.sla_out_proj_forward.argtypes = [vp, vp, vp, i32, vp, vp]
        L.sla_out_proj_forward.restype = ctypes.c_int
        L.sla_out_proj_backward.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp]
        L.sla_out_proj_backward.restype = ctypes.c_int
        L.sla_plan_shortconv_workspace_bytes.argtypes = [vp, i32, ctypes.POINTER(sz)]
        L.sla_plan_shortconv_workspace_bytes.restype = ctypes.c_int
        L.sla_gate_scores_forward.argtypes = [vp] * 8
        L.sla_gate_scores_forward.restype = ctypes.c_int
        L.sla_gate_scores_backward.argtypes = [vp] * 11 + [vp, sz, vp]
        L.sla_gate_scores_backward.restype = ctypes.c_int
        L.sla_plan_gate_scores_workspace_bytes.argtypes = [vp, ctypes.POINTER(sz)]
        L.sla_plan_gate_scores_workspace_bytes.restype = ctypes.c_int
        for name in ("sla_plan_create", "sla_plan_destroy", "sla_plan_workspace_bytes", "sla_plan_poll",
                     "sla_plan_set_kernel_timing", "sla_plan_kernel_timing_collect",
                     "sla_plan_kernel_timing_get", "sla_forward", "sla_backward", "sla_decode_step"):
            getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def _check(call: str, status: int):
    if status != 0:
        raise SLAError(call, status, lib().sla_status_string(status).decode())


def _ptr(t):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "tensors must be contiguous CUDA tensors"
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


class Plan:
    """Owns an sla_plan* (see sla_plan_create in include/sla.h)."""

    def __init__(self, variant, io_dtype, B, T, H, d_k, d_v, chunk=64, scale=1.0, flags=0):
        self.desc = sla_desc(ctypes.sizeof(sla_desc), VARIANTS.get(variant, variant),
                             DTYPES.get(io_dtype, io_dtype), B, T, H, d_k, d_v, chunk, scale, flags)
        self.handle = ctypes.c_void_p()
        _check("sla_plan_create", lib().sla_plan_create(ctypes.byref(self.handle), ctypes.byref(self.desc)))
        f, b = ctypes.c_size_t(), ctypes.c_size_t()
        _check("sla_plan_workspace_bytes",
               lib().sla_plan_workspace_bytes(self.handle, ctypes.byref(f), ctypes.byref(b)))
        self.forward_workspace_bytes, self.backward_workspace_bytes = f.value, b.value
        self.io_torch = torch.bfloat16 if self.desc.io_dtype == SLA_BF16 else torch.float32

    def close(self):
        h = getattr(self, "handle", None)
        if h is not None and h.value and _lib is not None:     # (at interpreter shutdown the module may be gone)
            try:
                _lib.sla_plan_destroy(h)
            except Exception:
                pass
            self.handle.value = None

    __del__ = close

    def set_sequences(self, cu_seqlens):
        """Packed variable-length batch (see sla_plan_set_sequences): cu_seqlens = n_seq + 1 ascending token offsets
        (a host sequence of ints), or None / [] for a regular batch.  Workspace sizes are queried again."""
        cu = list(cu_seqlens) if cu_seqlens is not None else []
        n = max(len(cu) - 1, 0)
        arr = (ctypes.c_int32 * max(len(cu), 1))(*cu)
        _check("sla_plan_set_sequences", lib().sla_plan_set_sequences(self.handle, arr, n))
        f, b = ctypes.c_size_t(), ctypes.c_size_t()
        _check("sla_plan_workspace_bytes", lib().sla_plan_workspace_bytes(self.handle, ctypes.byref(f), ctypes.byref(b)))
        self.forward_workspace_bytes, self.backward_workspace_bytes = f.value, b.value
        self.n_seq = n

    def poll(self):
        _check("sla_plan_poll", lib().sla_plan_poll(self.handle))

    def selftest_timeout(self):
        """Enqueue the bounded-wait self test (see sla_plan_selftest_timeout); poll() raises afterwards."""
        _check("sla_plan_selftest_timeout", lib().sla_plan_selftest_timeout(self.handle, _stream()))

    @property
    def last_launch_count(self) -> int:
        return int(lib().sla_plan_last_launch_count(self.handle))

    def set_kernel_timing(self, enable: bool):
        _check("sla_plan_set_kernel_timing", lib().sla_plan_set_kernel_timing(self.handle, int(enable)))

    def kernel_times(self) -> dict:
        """{kernel name: (launches, total ms)} accumulated since timing was enabled."""
        n = ctypes.c_int32()
        _check("sla_plan_kernel_timing_collect", lib().sla_plan_kernel_timing_collect(self.handle, ctypes.byref(n)))
        out = {}
        for i in range(n.value):
            name, cnt, ms = ctypes.c_char_p(), ctypes.c_int32(), ctypes.c_float()
            _check("sla_plan_kernel_timing_get", lib().sla_plan_kernel_timing_get(
                self.handle, i, ctypes.byref(name), ctypes.byref(cnt), ctypes.byref(ms)))
            out[name.value.decode()] = (cnt.value, ms.value)
        return out

    def workspace(self, backward=False, device="cuda"):
        n = self.backward_workspace_bytes if backward else self.forward_workspace_bytes
        return torch.empty(max(n, 16), dtype=torch.uint8, device=device)


def sla_plan_create(variant, io_dtype, B, T, H, d_k, d_v, chunk=64, scale=1.0, flags=0) -> Plan:
    return Plan(variant, io_dtype, B, T, H, d_k, d_v, chunk, scale, flags)


def sla_forward(plan: Plan, q, k, v, log_decay, gq_logits, gk_logits, beta=None, h0=None, o=None, ht=None,
                workspace=None):
    """Enqueue the chunkwise forward on the current stream.  Returns (o, ht)."""
    d = plan.desc
    if o is None:
        o = torch.empty((d.B, d.T, d.H, d.d_v), dtype=plan.io_torch, device=q.device)
    if workspace is None:
        workspace = plan.workspace(False, q.device)
    _check("sla_forward", lib().sla_forward(
        plan.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(log_decay), _ptr(beta), _ptr(gq_logits),
        _ptr(gk_logits), _ptr(h0), _ptr(o), _ptr(ht), _ptr(workspace), workspace.numel(), _stream()))
    return o, ht


def sla_forward_noalloc(plan: Plan, q, k, v, log_decay, gq_logits, gk_logits, o, beta=None, h0=None, ht=None):
    """sla_forward for callers that may not allocate device memory when they run the layer (a plugin
    inside a runtime that owns the allocator, a serving loop with a frozen memory budget).  The scratch
    is a fixed SLA_NOALLOC_SCRATCH_BYTES array inside the library, so `o` (and `ht`) must be passed in
    and nothing is allocated here either.  Problems whose forward workspace exceeds that size are
    refused (SLAError, status 3).  Calls share the array: do not let two of them overlap on the GPU."""
    _check("sla_forward_noalloc", lib().sla_forward_noalloc(
        plan.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(log_decay), _ptr(beta), _ptr(gq_logits),
        _ptr(gk_logits), _ptr(h0), _ptr(o), _ptr(ht), _stream()))
    return o, ht


def sla_backward(plan: Plan, q, k, v, log_decay, gq_logits, gk_logits, dO, beta=None, h0=None, dht=None,
                 want_dh0=False, workspace=None, out=None):
    """Enqueue the chunkwise backward on the current stream.  Returns a dict of gradients."""
    d = plan.desc
    dev = q.device
    if out is None:
        out = dict(
            dq=torch.empty_like(q), dk=torch.empty_like(k), dv=torch.empty_like(v),
            dlog_decay=None if d.variant == SLA_RETNET else torch.empty_like(log_decay),
            dbeta=torch.empty_like(beta) if d.variant == SLA_GDN else None,
            dgq_logits=torch.empty_like(gq_logits), dgk_logits=torch.empty_like(gk_logits),
            dh0=torch.empty((getattr(plan, "n_seq", 0) or d.B, d.H, d.d_k, d.d_v), dtype=torch.float32, device=dev) if want_dh0 else None,
        )
    if workspace is None:
        workspace = plan.workspace(True, dev)
    _check("sla_backward", lib().sla_backward(
        plan.handle, _ptr(q), _ptr(k), _ptr(v), _ptr(log_decay), _ptr(beta), _ptr(gq_logits),
        _ptr(gk_logits), _ptr(h0), _ptr(dO), _ptr(dht), _ptr(out["dq"]), _ptr(out["dk"]), _ptr(out["dv"]),
        _ptr(out["dlog_decay"]), _ptr(out["dbeta"]), _ptr(out["dgq_logits"]), _ptr(out["dgk_logits"]),
        _ptr(out["dh0"]), _ptr(workspace), workspace.numel(), _stream()))
    return out


def sla_decode_step(plan: Plan, q_t, k_t, v_t, log_decay_t, gq_logits_t, gk_logits_t, state, beta_t=None,
                    o_t=None):
    """One recurrent step on `state` ([Bdec,H,d_k,d_v] fp32, updated in place).  Returns o_t."""
    d = plan.desc
    Bdec = q_t.shape[0]
    if o_t is None:
        o_t = torch.empty((Bdec, d.H, d.d_v), dtype=plan.io_torch, device=q_t.device)
    _check("sla_decode_step", lib().sla_decode_step(
        plan.handle, Bdec, _ptr(q_t), _ptr(k_t), _ptr(v_t), _ptr(log_decay_t), _ptr(beta_t),
        _ptr(gq_logits_t), _ptr(gk_logits_t), _ptr(state), _ptr(o_t), _stream()))
    return o_t


def sla_decode_steps(plan: Plan, q, k, v, log_decay, gq_logits, gk_logits, state, beta=None, o=None):
    """n consecutive recurrent steps per sequence on `state` ([Bdec,H,d_k,d_v] fp32, updated in place): q, k
    [Bdec,n,H,d_k], v [Bdec,n,H,d_v].  Returns o [Bdec,n,H,d_v]."""
    d = plan.desc
    Bdec, n = q.shape[0], q.shape[1]
    if o is None:
        o = torch.empty((Bdec, n, d.H, d.d_v), dtype=plan.io_torch, device=q.device)
    _check("sla_decode_steps", lib().sla_decode_steps(
        plan.handle, Bdec, n, _ptr(q), _ptr(k), _ptr(v), _ptr(log_decay), _ptr(beta), _ptr(gq_logits),
        _ptr(gk_logits), _ptr(state), _ptr(o), _stream()))
    return o


def sla_gate_scores_forward(plan: Plan, q, k, w_gq, w_gk, gq_logits=None, gk_logits=None):
    """Eq. 4's score projections: returns (gq_logits, gk_logits), fp32 [B,T,H], from q, k and w_gq, w_gk [d_k,H]."""
    d = plan.desc
    if gq_logits is None:
        gq_logits = torch.empty((d.B, d.T, d.H), dtype=torch.float32, device=q.device)
    if gk_logits is None:
        gk_logits = torch.empty((d.B, d.T, d.H), dtype=torch.float32, device=q.device)
    _check("sla_gate_scores_forward", lib().sla_gate_scores_forward(
        plan.handle, _ptr(q), _ptr(k), _ptr(w_gq), _ptr(w_gk), _ptr(gq_logits), _ptr(gk_logits), _stream()))
    return gq_logits, gk_logits


def sla_gate_scores_backward(plan: Plan, q, k, w_gq, w_gk, dgq_logits, dgk_logits, dq, dk, workspace=None):
    """Reverse of the score projections: adds the logit route into dq, dk (in place) and returns (dw_gq, dw_gk)."""
    n = ctypes.c_size_t()
    _check("sla_plan_gate_scores_workspace_bytes", lib().sla_plan_gate_scores_workspace_bytes(plan.handle, ctypes.byref(n)))
    if workspace is None:
        workspace = torch.empty(max(n.value, 16), dtype=torch.uint8, device=q.device)
    dw_gq, dw_gk = torch.empty_like(w_gq), torch.empty_like(w_gk)
    _check("sla_gate_scores_backward", lib().sla_gate_scores_backward(
        plan.handle, _ptr(q), _ptr(k), _ptr(w_gq), _ptr(w_gk), _ptr(dgq_logits), _ptr(dgk_logits), _ptr(dq), _ptr(dk),
        _ptr(dw_gq), _ptr(dw_gk), _ptr(workspace), workspace.numel(), _stream()))
    return dw_gq, dw_gk


def sla_out_proj_forward(plan: Plan, o, w_o, y=None):
    """Eq. 7's output projection: o [B,T,H,d_v] (or [B,T,H*d_v]) bf16, w_o [H*d_v, d_model] bf16 -> y [B,T,d_model] bf16."""
    if y is None:
        y = torch.empty(o.shape[0], o.shape[1], w_o.shape[1], dtype=o.dtype, device=o.device)
    _check("sla_out_proj_forward", lib().sla_out_proj_forward(
        plan.handle, _ptr(o), _ptr(w_o), w_o.shape[1], _ptr(y), _stream()))
    return y


def sla_out_proj_backward(plan: Plan, o, w_o, dy):
    """Returns (d_o like o, dw_o fp32 [H*d_v, d_model]) of sla_out_proj_forward."""
    d_o = torch.empty_like(o)
    dw = torch.empty(w_o.shape, dtype=torch.float32, device=o.device)
    _check("sla_out_proj_backward", lib().sla_out_proj_backward(
        plan.handle, _ptr(o), _ptr(w_o), _ptr(dy), w_o.shape[1], _ptr(d_o), _ptr(dw), _stream()))
    return d_o, dw


def sla_shortconv_forward(plan: Plan, x, w, normalize, out=None):
    """Gated-DeltaNet feature map: causal depthwise convolution (w [H*d,K]) + SiLU (+ per-head L2 norm): x -> out [B,T,H,d]."""
    if out is None:
        out = torch.empty_like(x)
    _check("sla_shortconv_forward", lib().sla_shortconv_forward(
        plan.handle, _ptr(x), _ptr(w), x.shape[-1], w.shape[1], int(bool(normalize)), _ptr(out), _stream()))
    return out


def sla_shortconv_backward(plan: Plan, x, w, dout, normalize, workspace=None):
    """Returns (dx, dw) of sla_shortconv_forward."""
    n = ctypes.c_size_t()
    _check("sla_plan_shortconv_workspace_bytes",
           lib().sla_plan_shortconv_workspace_bytes(plan.handle, x.shape[-1], ctypes.byref(n)))
    if workspace is None:
        workspace = torch.empty(max(n.value, 16), dtype=torch.uint8, device=x.device)
    dx, dw = torch.empty_like(x), torch.empty_like(w)
    _check("sla_shortconv_backward", lib().sla_shortconv_backward(
        plan.handle, _ptr(x), _ptr(w), x.shape[-1], w.shape[1], int(bool(normalize)), _ptr(dout), _ptr(dx), _ptr(dw),
        _ptr(workspace), workspace.numel(), _stream()))
    return dx, dw
