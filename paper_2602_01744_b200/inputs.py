"""Seeded synthetic inputs for the five benchmark configurations.

This module holds input recipes only (random draws, the transforms the configurations
state for decay / beta / key normalisation, and rounding to the I/O dtype).  None of the
layer's arithmetic lives here; both the CUDA path and the CPU oracle are fed from it.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class SLAConfig:
    name: str
    variant: str            # "retnet" | "gla" | "gdn"
    B: int
    T: int
    H: int
    d_k: int
    d_v: int
    dtype: str              # "fp32" | "bf16"  (dtype of q, k, v, o and their gradients)
    chunk: int = 64
    seed: int = 0
    backward: bool = False
    scale: float = 1.0


CONFIGS = {
    "C0": SLAConfig("C0", "retnet", 1, 256, 4, 64, 64, "fp32", 64, 0, False),
    "C1": SLAConfig("C1", "gla", 4, 2048, 8, 128, 128, "bf16", 64, 1, False),
    "C2": SLAConfig("C2", "gla", 8, 4096, 16, 128, 128, "bf16", 64, 2, True),
    "C3": SLAConfig("C3", "gla", 1, 65536, 16, 128, 128, "bf16", 64, 3, False),
    "C4": SLAConfig("C4", "gdn", 4, 4096, 16, 128, 128, "bf16", 64, 4, True),
    # Softmax-RetNet at the shapes of C2 (the variant of Eq. 10-11 on the tensor-core kernels; not one of the five
    # benchmark configurations, timed by `bench.py --workload R2`)
    "R2": SLAConfig("R2", "retnet", 8, 4096, 16, 128, 128, "bf16", 64, 5, True),
}
C3_DECODE_BATCH = 64
C3_DECODE_STEPS = 256


def torch_dtype(name: str) -> torch.dtype:
    return {"fp32": torch.float32, "bf16": torch.bfloat16}[name]


def small(cfg: SLAConfig, **kw) -> SLAConfig:
    """A reduced copy of a configuration (same distributions, other sizes)."""
    return replace(cfg, **kw)


def make_inputs(cfg: SLAConfig, with_dO: bool | None = None, with_h0: bool = False) -> dict:
    """Draw the tensors of one configuration on the CPU, in a fixed order, from one generator.

    Returns a dict of CPU tensors: q, k [B,T,H,d_k], v [B,T,H,d_v] in the I/O dtype;
    log_decay fp32 (retnet [H], gla [B,T,H,d_k], gdn [B,T,H]); beta fp32 [B,T,H] (gdn) or None;
    gq_logits, gk_logits fp32 [B,T,H]; dO (I/O dtype) when asked; h0, dht fp32 [B,H,d_k,d_v] when asked.
    """
    gen = torch.Generator(device="cpu").manual_seed(cfg.seed)
    B, T, H, dk, dv = cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v
    io = torch_dtype(cfg.dtype)

    def randn(*shape):
        return torch.randn(*shape, generator=gen, dtype=torch.float32)

    q = randn(B, T, H, dk) / (dk ** 0.5)
    k = randn(B, T, H, dk) / (dk ** 0.5)
    v = randn(B, T, H, dv) / (dv ** 0.5)
    if cfg.variant == "retnet":
        h = torch.arange(H, dtype=torch.float64)
        log_decay = torch.log(1.0 - torch.pow(2.0, -5.0 - h)).float()
        beta = None
    elif cfg.variant == "gla":
        log_decay = torch.nn.functional.logsigmoid(randn(B, T, H, dk)) / 16.0
        beta = None
    else:
        log_decay = torch.nn.functional.logsigmoid(randn(B, T, H)) / 16.0
        beta = torch.sigmoid(randn(B, T, H))
        k = k / k.norm(dim=-1, keepdim=True)
    gq_logits = randn(B, T, H)
    gk_logits = randn(B, T, H)
    out = dict(
        q=q.to(io), k=k.to(io), v=v.to(io), log_decay=log_decay.contiguous(), beta=beta,
        gq_logits=gq_logits, gk_logits=gk_logits,
    )
    if with_dO is None:
        with_dO = cfg.backward
    if with_dO:
        out["dO"] = randn(B, T, H, dv).to(io)
    if with_h0:
        out["h0"] = randn(B, H, dk, dv) * 0.1
        out["dht"] = randn(B, H, dk, dv) * 0.1
    return out


def make_decode_inputs(cfg: SLAConfig, batch: int, steps: int, seed: int) -> dict:
    """Per-step decode tokens [steps, batch, H, d] drawn like the prefill tensors of cfg."""
    gen = torch.Generator(device="cpu").manual_seed(seed)
    H, dk, dv = cfg.H, cfg.d_k, cfg.d_v
    io = torch_dtype(cfg.dtype)

    def randn(*shape):
        return torch.randn(*shape, generator=gen, dtype=torch.float32)

    q = randn(steps, batch, H, dk) / (dk ** 0.5)
    k = randn(steps, batch, H, dk) / (dk ** 0.5)
    v = randn(steps, batch, H, dv) / (dv ** 0.5)
    beta = None
    if cfg.variant == "retnet":
        h = torch.arange(H, dtype=torch.float64)
        log_decay = torch.log(1.0 - torch.pow(2.0, -5.0 - h)).float()
    elif cfg.variant == "gla":
        log_decay = torch.nn.functional.logsigmoid(randn(steps, batch, H, dk)) / 16.0
    else:
        log_decay = torch.nn.functional.logsigmoid(randn(steps, batch, H)) / 16.0
        beta = torch.sigmoid(randn(steps, batch, H))
        k = k / k.norm(dim=-1, keepdim=True)
    return dict(q=q.to(io), k=k.to(io), v=v.to(io), log_decay=log_decay, beta=beta,
                gq_logits=randn(steps, batch, H), gk_logits=randn(steps, batch, H))


def make_gate_weights(cfg: SLAConfig, seed: int):
    """Gate score projection matrices W_GQ, W_GK (fp32 [d_k, H]) drawn N(0,1): with q, k ~ N(0,1)/sqrt(d_k) the scores
    q W come out ~ N(0,1) per (token, head), the distribution the configurations state for the gate logits."""
    gen = torch.Generator(device="cpu").manual_seed(seed)
    return (torch.randn(cfg.d_k, cfg.H, generator=gen, dtype=torch.float32),
            torch.randn(cfg.d_k, cfg.H, generator=gen, dtype=torch.float32))


def make_out_proj_inputs(cfg: SLAConfig, d_model: int, seed: int):
    """Inputs of the output projection (Eq. 7): head outputs o ~ N(0,1) [B,T,H,d_v] (the scale the layer's outputs
    have behind an output norm), W^O ~ N(0,1)/sqrt(H d_v) [H*d_v, d_model] (unit-scale y) and an upstream gradient
    dy ~ N(0,1) [B,T,d_model]; all in the I/O dtype."""
    gen = torch.Generator(device="cpu").manual_seed(seed)
    io = torch_dtype(cfg.dtype)
    K = cfg.H * cfg.d_v
    o = torch.randn(cfg.B, cfg.T, cfg.H, cfg.d_v, generator=gen, dtype=torch.float32).to(io)
    w = (torch.randn(K, d_model, generator=gen, dtype=torch.float32) / (K ** 0.5)).to(io)
    dy = torch.randn(cfg.B, cfg.T, d_model, generator=gen, dtype=torch.float32).to(io)
    return o, w, dy


def make_frontend_inputs(cfg: SLAConfig, K: int, seed: int) -> dict:
    """Raw inputs of the Gated-DeltaNet feature map: x_q, x_k, x_v ~ N(0,1) [B,T,H,d] in the I/O dtype (the layer's
    linear projections are upstream and leave unit-scale activations), taps w_* ~ N(0,1)/sqrt(K) fp32 [H*d,K], and an
    upstream gradient dout ~ N(0,1)."""
    gen = torch.Generator(device="cpu").manual_seed(seed)
    io = torch_dtype(cfg.dtype)
    B, T, H = cfg.B, cfg.T, cfg.H
    out = {}
    for n, d in (("q", cfg.d_k), ("k", cfg.d_k), ("v", cfg.d_v)):
        out[f"x_{n}"] = torch.randn(B, T, H, d, generator=gen, dtype=torch.float32).to(io)
        out[f"w_{n}"] = torch.randn(H * d, K, generator=gen, dtype=torch.float32) / (K ** 0.5)
    out["dout"] = torch.randn(B, T, H, cfg.d_k, generator=gen, dtype=torch.float32).to(io)
    return out
