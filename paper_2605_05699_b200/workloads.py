"""Seeded synthetic inputs shaped like the paper's KV-cache workloads.

This module is the one piece shared by the CPU oracle's tests and the CUDA
path's tests and benchmark.  It holds none of the method's arithmetic: it only
draws random head-dim vectors, per-channel lambda vectors and shape tables.
Real model activations, weights and evaluation text are not available; these
generators stand in for them (Sec. 4.1 lists the model shapes; Sec. 5.6
describes the few persistent outlier channels of Qwen2.5 K projections that
the "k_outlier" recipe imitates).

Everything is generated with ``torch.Generator`` so the same recipe runs on
the host (small cases, fed to the oracle) and on the device (full-size cases,
from which rows are sampled back to the host).
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

GROUP = 32


@dataclass(frozen=True)
class CacheShape:
    """One KV-cache workload: ``layers * kv_heads * batch`` streams per K or V."""

    name: str
    layers: int
    kv_heads: int
    head_dim: int
    batch: int
    prefix: int
    dtype: str  # "f16" | "bf16"

    @property
    def streams(self) -> int:  # K and V streams together
        return 2 * self.layers * self.kv_heads * self.batch

    @property
    def vectors(self) -> int:
        return self.streams * self.prefix


# Model-shaped configurations (shapes from Sec. 4.1 and Table 3).
QWEN25_1P5B = CacheShape("qwen2.5-1.5b-shaped", 28, 2, 128, 1, 1024, "f16")
GEMMA3_1B = CacheShape("gemma-3-1b-shaped", 26, 1, 256, 1, 4096, "bf16")
LLAMA3_70B = CacheShape("llama-3-70b-shaped", 80, 8, 128, 4, 32768, "f16")


def torch_dtype(dtype: str) -> torch.dtype:
    return {"f16": torch.float16, "bf16": torch.bfloat16}[dtype]


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def channel_scales(D: int, seed: int, n_outliers: int, outlier_gain: float = 20.0,
                   device="cpu") -> torch.Tensor:
    """Per-channel scale exp(N(0,1)), with ``n_outliers`` random channels multiplied by the gain."""
    g = _gen(seed, device)
    s = torch.exp(torch.randn(D, generator=g, device=device, dtype=torch.float32))
    if n_outliers > 0:
        idx = torch.randperm(D, generator=g, device=device)[:n_outliers]
        s[idx] *= outlier_gain
    return s


def make_vectors(N: int, D: int, dtype: str, kind: str, seed: int, device="cpu") -> torch.Tensor:
    """``[N, D]`` vectors of the requested half-precision dtype.

    kind:
      "gaussian"   entries N(0,1)                                (V-like)
      "lognormal"  N(0,1) times a per-channel exp(N(0,1)) scale  (config 4)
      "c1"         lognormal plus 4 channels x20                 (config 1)
      "k_outlier"  lognormal plus 2 % of channels x20 (3 of 128) (K-like, configs 2, 3, 5)
    """
    g = _gen(seed, device)
    x = torch.randn(N, D, generator=g, device=device, dtype=torch.float32)
    if kind == "gaussian":
        pass
    elif kind == "lognormal":
        x *= channel_scales(D, seed + 7919, 0, device=device)
    elif kind == "c1":
        x *= channel_scales(D, seed + 7919, 4, device=device)
    elif kind == "k_outlier":
        x *= channel_scales(D, seed + 7919, max(1, round(0.02 * D)), device=device)
    else:
        raise ValueError("unknown kind %r" % kind)
    return x.to(torch_dtype(dtype))


def make_lambda(n_rows: int, D: int, seed: int, device="cpu") -> torch.Tensor:
    """Per-channel lambda rows, uniform on (0.5, 2), fp32 ``[n_rows, D]``."""
    g = _gen(seed, device)
    return 0.5 + 1.5 * torch.rand(n_rows, D, generator=g, device=device, dtype=torch.float32)


def make_rotation(D: int, seed: int, near_identity: float = 0.0) -> torch.Tensor:
    """A seeded orthogonal matrix, host fp32 ``[D, D]``: the stand-in for a learned rotation (no trained one exists
    here).  ``near_identity`` = 0 gives a Haar-like draw (QR of a Gaussian matrix, column signs fixed); a value t > 0
    gives exp(t (U - U^T)) for Gaussian U, the near-identity shape a short training run starts from and stays close to."""
    g = _gen(seed, "cpu")
    u = torch.randn(D, D, generator=g, dtype=torch.float64)
    if near_identity > 0.0:
        q = torch.linalg.matrix_exp(near_identity * (u - u.T))
    else:
        q, r = torch.linalg.qr(u)
        q = q * torch.sign(torch.diagonal(r))
    return q.to(torch.float32).contiguous()


def raw_bits(x: torch.Tensor):
    """Host uint16 bit patterns of a half-precision tensor (what the oracle consumes)."""
    return x.detach().cpu().contiguous().view(torch.int16).numpy().view("uint16")
