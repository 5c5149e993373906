"""Seeded synthetic workloads for the CompAct compressed linear layer.

This module only describes layer shapes and draws input tensors (X, W, dY).
It holds none of the method's arithmetic: no projection, no Philox, no Adam.
Both the CPU oracle's tests and the CUDA path's tests/benchmarks draw their
inputs here so that the two sides consume identical bits.

The shapes and value distributions stand in for the paper's workloads
(LLaMA pre-training on C4 at sequence 256, RoBERTa-base fine-tuning on GLUE at
sequence 512; Section 4 and Appendix B/C).  Only shapes and distributions are
taken; no dataset item or trained weight is reproduced.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List

import numpy as np
import torch

KIND_X, KIND_W, KIND_DY = 1, 2, 3


@dataclass(frozen=True)
class LayerShape:
    name: str
    n: int            # in-features
    m: int            # out-features
    r: int            # projection rank
    x_dist: str = "normal"   # "normal" | "outlier" | "gelu"


@dataclass(frozen=True)
class Workload:
    name: str
    cfg_id: int
    dtype: str                 # "f32" | "bf16"
    tokens: int                # b*l
    layers: List[LayerShape] = field(default_factory=list)
    steps: int = 1
    refresh_T: int = 0
    lr: float = 1e-3
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    alpha: float = 1.0
    seed: int = 0
    x_scale_inv_sqrt_n: bool = False
    dy_std: float | None = None   # None: 1/sqrt(n)
    sparse_s: int = 0             # > 0: the layers use the sparse JL projection with this many terms per row

    def with_tokens(self, tokens: int) -> "Workload":
        return Workload(**{**self.__dict__, "tokens": tokens})


def _llama_set(n: int, ffn: int, frac: int, x_dist: str = "normal") -> List[LayerShape]:
    out = [LayerShape(f"{nm}_proj", n, n, n // frac, x_dist) for nm in ("q", "k", "v", "o")]
    out += [LayerShape(f"{nm}_proj", n, ffn, n // frac, x_dist) for nm in ("gate", "up")]
    out += [LayerShape("down_proj", ffn, n, ffn // frac, x_dist)]
    return out


def config1() -> Workload:
    return Workload("c1_single_fp32", 1, "f32", 256, [LayerShape("linear", 128, 512, 16)],
                    steps=3, refresh_T=2, dy_std=1e-2)


def config2() -> Workload:
    return Workload("c2_llama60m", 2, "bf16", 8192, _llama_set(512, 1376, 4),
                    steps=20, refresh_T=10, x_scale_inv_sqrt_n=True)


def config3(frac: int = 8) -> Workload:
    return Workload(f"c3_llama350m_r{frac}", 3, "bf16", 16384, _llama_set(1024, 2736, frac, "outlier"),
                    steps=50, refresh_T=25)


def config4() -> Workload:
    n, f = 768, 3072
    layers = [LayerShape(f"{nm}_proj", n, n, n // 2) for nm in ("q", "k", "v", "o")]
    layers += [LayerShape("ffn_up", n, f, n // 2), LayerShape("ffn_down", f, n, f // 2, "gelu")]
    return Workload("c4_roberta_base", 4, "bf16", 16384, layers, steps=30, refresh_T=10)


def config5() -> Workload:
    return Workload("c5_llama7b", 5, "bf16", 16384, _llama_set(4096, 11008, 8),
                    steps=10, refresh_T=200, x_scale_inv_sqrt_n=True)


def all_configs() -> List[Workload]:
    return [config1(), config2(), config3(8), config3(4), config4(), config5()]


def torch_dtype(wl_dtype: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[wl_dtype]


def _rng(cfg_id: int, layer_index: int, kind: int, step: int) -> np.random.Generator:
    return np.random.default_rng([0xDA7A, cfg_id, layer_index, kind, step])


def _finish(a: np.ndarray, dtype: str) -> torch.Tensor:
    # Values are drawn in fp32 and converted to the storage dtype by torch's
    # own round-to-nearest-even conversion; both sides read the stored bits.
    return torch.from_numpy(a).to(torch_dtype(dtype)).contiguous()


def draw_X(wl: Workload, layer_index: int, step: int, tokens: int | None = None,
           row_start: int = 0) -> torch.Tensor:
    """X_t for one layer and step, tokens x n, in the workload's storage dtype.

    Rows are drawn in blocks of 256 tokens from independent streams so that a
    row range can be drawn without drawing the rows before it.
    """
    L = wl.layers[layer_index]
    tokens = wl.tokens if tokens is None else tokens
    blk = 256
    out = np.empty((tokens, L.n), dtype=np.float32)
    t = 0
    while t < tokens:
        g = row_start + t
        b = g // blk
        off = g - b * blk
        take = min(blk - off, tokens - t)
        rng = np.random.default_rng([0xDA7A, wl.cfg_id, layer_index, KIND_X, step, b])
        a = rng.standard_normal((blk, L.n), dtype=np.float32)
        out[t:t + take] = a[off:off + take]
        t += take
    if L.x_dist == "outlier":
        cols = np.arange(L.n)
        out[:, (cols % 100) == 37] *= 20.0
    elif L.x_dist == "gelu":
        x64 = torch.from_numpy(out.astype(np.float64))
        out = torch.nn.functional.gelu(x64).numpy().astype(np.float32)
    if wl.x_scale_inv_sqrt_n:
        out = out * np.float32(1.0 / np.sqrt(L.n))
    return _finish(out, wl.dtype)


def draw_dY(wl: Workload, layer_index: int, step: int, tokens: int | None = None,
            row_start: int = 0) -> torch.Tensor:
    """dY_t for one layer and step, tokens x m."""
    L = wl.layers[layer_index]
    tokens = wl.tokens if tokens is None else tokens
    std = wl.dy_std if wl.dy_std is not None else 1.0 / np.sqrt(L.n)
    blk = 256
    out = np.empty((tokens, L.m), dtype=np.float32)
    t = 0
    while t < tokens:
        g = row_start + t
        b = g // blk
        off = g - b * blk
        take = min(blk - off, tokens - t)
        rng = np.random.default_rng([0xDA7A, wl.cfg_id, layer_index, KIND_DY, step, b])
        a = rng.standard_normal((blk, L.m), dtype=np.float32)
        out[t:t + take] = a[off:off + take]
        t += take
    return _finish(out * np.float32(std), wl.dtype)


def draw_W(wl: Workload, layer_index: int) -> torch.Tensor:
    """Initial weight, n x m row-major, N(0, 0.02^2)."""
    L = wl.layers[layer_index]
    a = _rng(wl.cfg_id, layer_index, KIND_W, 0).standard_normal((L.n, L.m), dtype=np.float32)
    return _finish(a * np.float32(0.02), wl.dtype)


def algorithmic_flops(tokens: int, n: int, m: int, r: int) -> float:
    """Flops of one fwd+bwd+update of one layer: Y, Z, dX, Gc and P.N (true r)."""
    return 2.0 * tokens * n * m + 2.0 * tokens * n * r + 2.0 * tokens * m * n \
        + 2.0 * tokens * r * m + 2.0 * n * r * m


def update_bytes(n: int, m: int, r: int, elem_bytes: int) -> float:
    """HBM bytes of one update: W read+write, Gc read, M and V read+write (fp32)."""
    return 2.0 * n * m * elem_bytes + 20.0 * r * m
