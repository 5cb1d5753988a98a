"""Seeded synthetic inputs with the shapes of the paper's LLaMA workloads.

This module holds no arithmetic of the method: it only draws tensors.  It is
the one module that both the CUDA path's callers and the CPU oracle's callers
use, so that both see the same bytes.

Recipe: hidden states ~ N(0,1) multiplied by projection weights of variance
1/4096 give Q, K, V, Q', K' entries that are ~ N(0,1); the projections lie
outside the library, so those tensors are drawn directly as N(0,1).  Aligner
weights are N(0, 1/fan_in).  Each tensor has its own stream, keyed by
(seed, name), so adding a tensor never changes another.  For bf16 workloads the
fp32 draw is rounded to nearest-even bf16 and both sides consume the rounded
values.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass, field
from typing import Tuple

import numpy as np
import torch


def normal(name: str, shape, seed: int = 0, std: float = 1.0) -> np.ndarray:
    """fp32 N(0, std^2) tensor from the stream keyed by (seed, name)."""
    rng = np.random.default_rng([int(seed), zlib.crc32(name.encode())])
    out = rng.standard_normal(size=tuple(shape), dtype=np.float32)
    if std != 1.0:
        out *= np.float32(std)
    return out


def as_dtype(x: np.ndarray, dtype: str) -> torch.Tensor:
    """Host tensor in the workload's storage type ('f32' or 'bf16', RNE)."""
    t = torch.from_numpy(np.ascontiguousarray(x))
    return t.to(torch.bfloat16) if dtype == "bf16" else t.to(torch.float32)


def to_f64(t: torch.Tensor) -> np.ndarray:
    """The exact stored values, widened to fp64 (what the oracle consumes)."""
    return t.detach().to("cpu").to(torch.float64).numpy()


@dataclass(frozen=True)
class Workload:
    """Shape of one benchmark workload."""
    name: str
    dtype: str            # storage type of activations and weights
    B: int
    N: int                # prompt length (prefill) or context length L (decode)
    Hq: int
    Hkv: int
    d: int
    r: int
    m: int                # aligner hidden width
    act: str              # 'relu' | 'silu' | 'none'
    chain: int            # number of shared layers after the anchor
    decode: bool = False
    extra: Tuple = field(default_factory=tuple)


WORKLOADS = {
    "cfg1_tiny_fp32": Workload("cfg1_tiny_fp32", "f32", 1, 128, 4, 4, 32, 8, 16, "relu", 1),
    "cfg2_llama2_7b_prefill": Workload("cfg2_llama2_7b_prefill", "bf16", 1, 2048, 32, 32, 128, 21, 64, "silu", 1),
    "cfg3_llama3_8b_gqa_prefill": Workload("cfg3_llama3_8b_gqa_prefill", "bf16", 4, 8192, 32, 8, 128, 21, 64, "relu", 3),
    "cfg4_llama2_13b_decode": Workload("cfg4_llama2_13b_decode", "bf16", 64, 4096, 40, 40, 128, 21, 80, "relu", 1, True),
    "cfg5_llama2_7b_stack": Workload("cfg5_llama2_7b_stack", "bf16", 32, 2048, 32, 32, 128, 21, 64, "relu", 3, False,
                                     (("layers", 32), ("decode_steps", 256))),
}


def prefill_inputs(w: Workload, seed: int = 0, B=None, N=None):
    """Host tensors for an anchor layer followed by `w.chain` shared layers.

    Returns a dict: q0,k0,v0 and per link k=1..chain: qp{k},kp{k},v{k},w1_{k},w2_{k}.
    """
    B = w.B if B is None else B
    N = w.N if N is None else N
    t = {}
    t["q0"] = as_dtype(normal("q0", (B, N, w.Hq, w.d), seed), w.dtype)
    t["k0"] = as_dtype(normal("k0", (B, N, w.Hkv, w.d), seed), w.dtype)
    t["v0"] = as_dtype(normal("v0", (B, N, w.Hkv, w.d), seed), w.dtype)
    for k in range(1, w.chain + 1):
        t[f"qp{k}"] = as_dtype(normal(f"qp{k}", (B, N, w.Hq, w.r), seed), w.dtype)
        t[f"kp{k}"] = as_dtype(normal(f"kp{k}", (B, N, w.Hkv, w.r), seed), w.dtype)
        t[f"v{k}"] = as_dtype(normal(f"v{k}", (B, N, w.Hkv, w.d), seed), w.dtype)
        t[f"w1_{k}"] = as_dtype(normal(f"w1_{k}", (w.Hq, w.m), seed, std=w.Hq ** -0.5), w.dtype)
        t[f"w2_{k}"] = as_dtype(normal(f"w2_{k}", (w.m, w.Hq), seed, std=w.m ** -0.5), w.dtype)
    return t


def decode_inputs(w: Workload, seed: int = 0, B=None, L=None, seqs=None):
    """Host tensors for one decode step of a shared layer and of a standard layer.

    prev [B,Hq,L] fp32 score row; qp [B,1,Hq,r]; kp [B,L,Hkv,r]; v [B,L,Hkv,d]; aligner w1,w2;
    and q0 [B,1,Hq,d], k [B,L,Hkv,d] for the standard-attention comparison.  Every sequence has its own
    streams, so `seqs` (a list of sequence indices) yields exactly those sequences of the full batch.
    """
    B = w.B if B is None else B
    L = w.N if L is None else L
    seqs = list(range(B)) if seqs is None else list(seqs)

    def per_seq(name, shape, dtype):
        return torch.stack([as_dtype(normal("%s/%d" % (name, b), shape, seed), dtype) for b in seqs])

    t = {}
    t["prev"] = per_seq("prev", (w.Hq, L), "f32")
    t["qp"] = per_seq("qp", (1, w.Hq, w.r), w.dtype)
    t["kp"] = per_seq("kp", (L, w.Hkv, w.r), w.dtype)
    t["v"] = per_seq("v", (L, w.Hkv, w.d), w.dtype)
    t["w1"] = as_dtype(normal("w1", (w.Hq, w.m), seed, std=w.Hq ** -0.5), w.dtype)
    t["w2"] = as_dtype(normal("w2", (w.m, w.Hq), seed, std=w.m ** -0.5), w.dtype)
    t["q0"] = per_seq("q0", (1, w.Hq, w.d), w.dtype)
    t["k"] = per_seq("k", (L, w.Hkv, w.d), w.dtype)
    return t


def device_normal(name: str, shape, seed: int = 0, dtype: str = "bf16", device="cuda") -> torch.Tensor:
    """N(0,1) tensor drawn on the device from the stream keyed by (seed, name); for tensors too large to
    draw on the host in reasonable time.  Whoever needs the same bytes on the host copies them back."""
    g = torch.Generator(device=device)
    g.manual_seed((int(seed) << 32) ^ zlib.crc32(name.encode()))
    x = torch.randn(tuple(shape), generator=g, device=device, dtype=torch.float32)
    return x.to(torch.bfloat16) if dtype == "bf16" else x
