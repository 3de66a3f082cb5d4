"""Seeded synthetic inputs for the Gated Slot Attention layer.

This module only draws random tensors; it holds none of the layer's arithmetic
and is the one piece of code that both the CPU oracle's tests and the CUDA
path's tests/benchmark use, so that both sides see bit-identical inputs.

Recipe (stand-in for the paper's workloads, whose datasets and weights are not
available: the shapes are those of the 1.3B model -- 4 heads of width 512, 64
slots -- of a 7B-attention geometry for the finetuning setting, and of batched
recurrent decoding; the gate statistics follow the layer's parameterisation
a = sigmoid(x)^(1/tau) with tau = 8):

  * one numpy Generator(PCG64) child stream per tensor, spawned from
    SeedSequence(seed) in the fixed order
        q, k, v, gate-noise, dO, K0, V0, channel-scale
    so adding or dropping an optional tensor never changes the others;
  * q, k, v, dO ~ N(0,1) drawn in float32; q is multiplied by d_k^-0.5;
  * optional per-(head, channel) log-normal scale exp(sigma * xi) on k;
  * gate a = sigmoid(mu + N(0,1)) ** (1/tau) in float32 (float64 intermediate);
  * K0, V0 ~ N(0, 0.1) float32 when requested;
  * for io == "bf16" the q, k, v, dO values are rounded to the nearest bfloat16
    (ties to even) and returned as float32 arrays holding exactly those values.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    T: int
    H: int
    d_k: int
    d_v: int
    m: int
    io: str = "bf16"            # "f32" or "bf16": dtype of q,k,v,o and their gradients
    seed: int = 0
    gate_mu: float = 0.0        # a = sigmoid(gate_mu + N(0,1)) ** (1/gate_tau)
    gate_tau: float = 8.0
    k_channel_sigma: float = 0.0
    init_state: bool = False    # draw K0, V0 ~ N(0, 0.1)
    with_dO: bool = True

    @property
    def tokens(self) -> int:
        return self.B * self.T

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five benchmark configurations (seed = configuration index, the first one
# uses seed 0) plus the two gate regimes of the long-context case.
CONFIGS = {
    "tiny_f32": Workload("tiny_f32", B=1, T=256, H=2, d_k=64, d_v=64, m=32, io="f32", seed=0),
    "train_1p3b": Workload("train_1p3b", B=8, T=2048, H=4, d_k=512, d_v=512, m=64, seed=1),
    # the 2.7B model's layer: 5 heads of width 512 (model width 2560), otherwise as the 1.3B one
    "train_2p7b": Workload("train_2p7b", B=8, T=2048, H=5, d_k=512, d_v=512, m=64, seed=5),
    # decoding with the whole 1.3B model's stack of GSA layers: one sequence, 24 layers of 4 heads of width 512
    "decode_1p3b": Workload("decode_1p3b", B=1, T=16384, H=4, d_k=512, d_v=512, m=64, seed=6,
                            init_state=True, with_dO=False),
    "t2r_7b": Workload("t2r_7b", B=4, T=4096, H=32, d_k=128, d_v=128, m=64, seed=2,
                       k_channel_sigma=0.5),
    "long_keep": Workload("long_keep", B=1, T=32768, H=16, d_k=128, d_v=128, m=64, seed=3,
                          gate_mu=2.0, gate_tau=16.0, init_state=True, with_dO=False),
    "long_forget": Workload("long_forget", B=1, T=32768, H=16, d_k=128, d_v=128, m=64, seed=3,
                            gate_mu=-2.0, gate_tau=1.0, init_state=True, with_dO=False),
    "decode": Workload("decode", B=256, T=1024, H=32, d_k=128, d_v=128, m=64, seed=4,
                       init_state=True, with_dO=False),
}


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest-even rounding of float32 values to bfloat16, returned as float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    bits = x.view(np.uint32)
    lsb = (bits >> np.uint32(16)) & np.uint32(1)
    rounded = (bits + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return rounded.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """The upper 16 bits (as int16) of float32 values that are already exactly
    representable in bfloat16 -- the raw storage of a bfloat16 tensor."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> np.uint32(16)).astype(np.uint16).view(np.int16)


def _streams(seed: int):
    names = ("q", "k", "v", "gate", "dO", "K0", "V0", "kscale")
    kids = np.random.SeedSequence(seed).spawn(len(names))
    return {n: np.random.Generator(np.random.PCG64(s)) for n, s in zip(names, kids)}


def _normal(rng, shape):
    return rng.standard_normal(shape, dtype=np.float32)


def make_gate(rng, shape, mu: float, tau: float) -> np.ndarray:
    x = rng.standard_normal(shape, dtype=np.float32).astype(np.float64) + mu
    a = (1.0 / (1.0 + np.exp(-x))) ** (1.0 / tau)
    return a.astype(np.float32)


def make_inputs(w: Workload) -> dict:
    """All tensors of a training/prefill call: q,k [B,T,H,d_k], v,dO [B,T,H,d_v],
    gate [B,T,H,m] (linear a, float32), optional K0 [B,H,m,d_k], V0 [B,H,m,d_v]."""
    r = _streams(w.seed)
    q = _normal(r["q"], (w.B, w.T, w.H, w.d_k)) * np.float32(w.d_k ** -0.5)
    k = _normal(r["k"], (w.B, w.T, w.H, w.d_k))
    v = _normal(r["v"], (w.B, w.T, w.H, w.d_v))
    if w.k_channel_sigma:
        xi = _normal(r["kscale"], (w.H, w.d_k))
        k = k * np.exp(np.float32(w.k_channel_sigma) * xi)[None, None]
    out = {"gate": make_gate(r["gate"], (w.B, w.T, w.H, w.m), w.gate_mu, w.gate_tau)}
    if w.with_dO:
        out["dO"] = _normal(r["dO"], (w.B, w.T, w.H, w.d_v))
    if w.init_state:
        out["K0"] = _normal(r["K0"], (w.B, w.H, w.m, w.d_k)) * np.float32(0.1)
        out["V0"] = _normal(r["V0"], (w.B, w.H, w.m, w.d_v)) * np.float32(0.1)
    out.update(q=q, k=k, v=v)
    if w.io == "bf16":
        for n in ("q", "k", "v", "dO"):
            if n in out:
                out[n] = round_to_bf16(out[n])
    return out


def make_decode_states(w: Workload) -> dict:
    """Initial slot memories for the decode workload: B sequences, [B,H,m,d] float32 ~ N(0, 0.1)."""
    r = _streams(w.seed)
    return {"K": _normal(r["K0"], (w.B, w.H, w.m, w.d_k)) * np.float32(0.1),
            "V": _normal(r["V0"], (w.B, w.H, w.m, w.d_v)) * np.float32(0.1)}


def make_decode_step_inputs(w: Workload, step: int) -> dict:
    """Fresh q,k [B,H,d_k], v [B,H,d_v], gate [B,H,m] for decode step `step`
    (its own stream family, keyed by (seed, step))."""
    kids = np.random.SeedSequence([w.seed, 1_000_003, step]).spawn(4)
    rq, rk, rv, rg = (np.random.Generator(np.random.PCG64(s)) for s in kids)
    q = _normal(rq, (w.B, w.H, w.d_k)) * np.float32(w.d_k ** -0.5)
    k = _normal(rk, (w.B, w.H, w.d_k))
    v = _normal(rv, (w.B, w.H, w.d_v))
    gate = make_gate(rg, (w.B, w.H, w.m), w.gate_mu, w.gate_tau)
    if w.io == "bf16":
        q, k, v = (round_to_bf16(x) for x in (q, k, v))
    return dict(q=q, k=k, v=v, gate=gate)
