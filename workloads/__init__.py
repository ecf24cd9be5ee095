"""Seeded synthetic inputs shaped like the paper's LLM workloads.

This module only draws random tensors and lists layer shapes; it contains none of the
pruning method's arithmetic.  Both the CPU oracle's tests and the CUDA path's tests / the
benchmark take their inputs from here, so both sides see the same bits.

The paper calibrates on 128 text sequences and prunes trained checkpoints (Section 5.1);
neither is available offline, so activations are drawn from a heavy-tailed distribution with
a few high-energy "outlier" input channels (the structure real LLM activations show) and
weights from N(0, 0.02^2) (the usual initialisation scale).

Layout: activations are tokens-major ``[a, b]`` (the transpose of the paper's ``X``, which
is ``b x a``); weights are ``[c, b]`` row-major.
"""

from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import torch

TOKEN_CHUNK = 4096  # activations are drawn in chunks of this many tokens, one seed per chunk


@dataclass(frozen=True)
class LayerSpec:
    name: str
    c: int  # output features (rows of W)
    b: int  # input features (columns of W)
    input_id: int  # layers with the same input_id share one activation matrix / Hessian


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    layers: List[LayerSpec]
    a: int  # calibration tokens
    dtype: str  # "f32" | "bf16" (weights and activations)
    x_dist: str  # "normal" | "student_t4"
    outlier_frac: float  # fraction of input channels scaled up (0 -> use outlier_count)
    outlier_count: int
    outlier_scale: float
    mode: str  # "unstructured" | "nm"
    p: float = 0.0
    n: int = 0
    m: int = 0
    B: int = 128
    damp_rel: float = 0.01
    seed: int = 0
    extra_modes: tuple = field(default_factory=tuple)


def _L(name, c, b, i):
    return LayerSpec(name, c, b, i)


CONFIGS = {
    # single small layer: the oracle finishes in seconds
    "tiny": WorkloadConfig(
        "tiny", [_L("fc", 256, 256, 0)], a=2048, dtype="f32", x_dist="normal",
        outlier_frac=0.0, outlier_count=4, outlier_scale=20.0,
        mode="unstructured", p=0.5, B=64, seed=0),
    # OPT-125M-shaped layer set
    "opt125m": WorkloadConfig(
        "opt125m",
        [_L("q", 768, 768, 0), _L("k", 768, 768, 0), _L("v", 768, 768, 0),
         _L("o", 768, 768, 1), _L("fc1", 3072, 768, 2), _L("fc2", 768, 3072, 3)],
        a=262144, dtype="f32", x_dist="student_t4",
        outlier_frac=0.01, outlier_count=0, outlier_scale=20.0,
        mode="nm", n=2, m=4, B=128, seed=1),
    # LLaMA-2-7B-shaped transformer block
    "llama2_7b": WorkloadConfig(
        "llama2_7b",
        [_L("q", 4096, 4096, 0), _L("k", 4096, 4096, 0), _L("v", 4096, 4096, 0),
         _L("o", 4096, 4096, 1), _L("gate", 11008, 4096, 2), _L("up", 11008, 4096, 2),
         _L("down", 4096, 11008, 3)],
        a=262144, dtype="bf16", x_dist="student_t4",
        outlier_frac=0.005, outlier_count=0, outlier_scale=50.0,
        mode="unstructured", p=0.5, B=128, seed=2),
    # LLaMA-3-8B-shaped transformer block (grouped-query k, v)
    "llama3_8b": WorkloadConfig(
        "llama3_8b",
        [_L("q", 4096, 4096, 0), _L("k", 1024, 4096, 0), _L("v", 1024, 4096, 0),
         _L("o", 4096, 4096, 1), _L("gate", 14336, 4096, 2), _L("up", 14336, 4096, 2),
         _L("down", 4096, 14336, 3)],
        a=262144, dtype="bf16", x_dist="student_t4",
        outlier_frac=0.005, outlier_count=0, outlier_scale=50.0,
        mode="nm", n=4, m=8, B=256, seed=3),
    # LLaMA-2-70B-shaped layer set
    "llama2_70b": WorkloadConfig(
        "llama2_70b",
        [_L("q", 8192, 8192, 0), _L("k", 1024, 8192, 0), _L("gate", 28672, 8192, 1),
         _L("down", 8192, 28672, 2)],
        a=131072, dtype="bf16", x_dist="student_t4",
        outlier_frac=0.005, outlier_count=0, outlier_scale=50.0,
        mode="nm", n=2, m=4, B=128, seed=4,
        extra_modes=(("unstructured", 0.6),)),
}


def torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def _gen(device, *seed_parts) -> torch.Generator:
    g = torch.Generator(device=device)
    s = 0x9E3779B97F4A7C15
    for p in seed_parts:
        s = (s * 6364136223846793005 + int(p) + 1442695040888963407) % (1 << 63)
    g.manual_seed(s)
    return g


def make_weight(c: int, b: int, dtype: str, seed: int, layer_index: int = 0,
                device="cpu", std: float = 0.02) -> torch.Tensor:
    """``[c, b]`` weights ~ N(0, std^2), rounded to ``dtype``."""
    g = _gen(device, seed, 101, layer_index)
    w = torch.randn((c, b), generator=g, device=device, dtype=torch.float32) * std
    return w.to(torch_dtype(dtype)).contiguous()


def outlier_channels(b: int, frac: float, count: int, seed: int, input_id: int) -> torch.Tensor:
    k = count if count > 0 else max(1, int(round(frac * b)))
    g = _gen("cpu", seed, 202, input_id)
    return torch.randperm(b, generator=g)[:k].sort().values


def make_activations(a: int, b: int, dtype: str, x_dist: str, outlier_frac: float,
                     outlier_count: int, outlier_scale: float, seed: int, input_id: int = 0,
                     device="cpu", mix: float = 0.0, token_offset: int = 0) -> torch.Tensor:
    """Tokens-major activations ``[a, b]`` in ``dtype``.

    ``x_dist``: "normal" -> N(0,1); "student_t4" -> Student-t with 4 degrees of freedom.
    A seeded subset of channels is multiplied by ``outlier_scale``.  ``mix > 0`` additionally
    right-multiplies by ``I + mix * G / sqrt(b)`` (``G`` seeded N(0,1)) so that features are
    correlated and the pruning updates are not small; used for parity tests only.
    ``token_offset`` selects which chunk seeds are used (must be a multiple of TOKEN_CHUNK).
    """
    assert token_offset % TOKEN_CHUNK == 0
    scale = torch.ones(b, dtype=torch.float32)
    scale[outlier_channels(b, outlier_frac, outlier_count, seed, input_id)] = outlier_scale
    scale = scale.to(device)
    A = None
    if mix > 0.0:
        g = _gen("cpu", seed, 303, input_id)
        A = (torch.eye(b) + mix * torch.randn((b, b), generator=g) / (b ** 0.5)).to(device)
    out = torch.empty((a, b), dtype=torch_dtype(dtype), device=device)
    for t0 in range(0, a, TOKEN_CHUNK):
        t1 = min(a, t0 + TOKEN_CHUNK)
        g = _gen(device, seed, 404, input_id, (t0 + token_offset) // TOKEN_CHUNK)
        z = torch.randn((t1 - t0, b), generator=g, device=device, dtype=torch.float32)
        if x_dist == "student_t4":
            # chi-square with 4 degrees of freedom = -2 ln(U1 U2); one draw per element
            u = torch.rand((t1 - t0, b), generator=g, device=device, dtype=torch.float32)
            u = u * torch.rand((t1 - t0, b), generator=g, device=device, dtype=torch.float32)
            chi = -2.0 * torch.log(u.clamp_min(1e-30))
            z = z / torch.sqrt(chi / 4.0)
        elif x_dist != "normal":
            raise ValueError(x_dist)
        z = z * scale
        if A is not None:
            z = z @ A
        out[t0:t1] = z.to(out.dtype)
    return out


def config_activations(cfg: WorkloadConfig, input_id: int, b: int, device="cpu",
                       a: Optional[int] = None, mix: float = 0.0) -> torch.Tensor:
    return make_activations(a if a is not None else cfg.a, b, cfg.dtype, cfg.x_dist,
                            cfg.outlier_frac, cfg.outlier_count, cfg.outlier_scale,
                            cfg.seed, input_id, device=device, mix=mix)


def config_weight(cfg: WorkloadConfig, layer_index: int, device="cpu") -> torch.Tensor:
    L = cfg.layers[layer_index]
    return make_weight(L.c, L.b, cfg.dtype, cfg.seed, layer_index, device=device)
