"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke check.

This module holds no arithmetic of the method (no quantizer, dictionary, coder
or product): it only manufactures floating-point weights and activations with
the shapes and value distribution of the workloads, identically on CPU and GPU.

Recipe
------
* Weights: Student-t(df=5) scaled to std 0.02, with 1 % of the input channels
  (columns) multiplied by 8.  A value is drawn by inverse-CDF sampling: a
  counter-based 32-bit integer hash of (matrix seed, flat element index) gives a
  24-bit uniform u; the top 16 bits pick an interval of a 65537-point quantile
  table (computed once on the CPU in fp64, stored as fp32) and the low 8 bits
  interpolate linearly inside it.  Only exact integer operations and separately
  rounded fp32 add/sub/mul are used, so a CPU tensor and a CUDA tensor built
  from the same seed are bit-identical.
* Activations: the same sampler with a standard-normal quantile table, rounded
  to bf16 (round to nearest even).
* Shapes: the linear layers of LLaMA-3.2-1B / 3B / 11B (q, k, v, o, gate, up, down per
  decoder layer, then lm_head), in that order.
"""
from __future__ import annotations

import functools
import math

import numpy as np
import torch

BASE_SEED = 250922951
_TABLE_BITS = 16
_EPS = 2.0 ** -18


@functools.lru_cache(maxsize=None)
def _quantile_table(kind: str) -> torch.Tensor:
    from scipy import stats

    n = 1 << _TABLE_BITS
    p = np.clip(np.arange(n + 1, dtype=np.float64) / n, _EPS, 1.0 - _EPS)
    if kind == "t5_std0.02":
        tab = stats.t.ppf(p, 5) * (0.02 / math.sqrt(5.0 / 3.0))
    elif kind == "normal":
        tab = stats.norm.ppf(p)
    else:
        raise ValueError(kind)
    return torch.from_numpy(tab.astype(np.float32))


def _mul32(x: torch.Tensor, c: int) -> torch.Tensor:
    """(x * c) mod 2**32 for 0 <= x < 2**32 held in int64, without int64 overflow."""
    lo = (x & 0xFFFF) * c
    hi = (((x >> 16) * c) & 0xFFFF) << 16
    return (lo + hi) & 0xFFFFFFFF


def _fmix32(h: torch.Tensor) -> torch.Tensor:
    h = h ^ (h >> 16)
    h = _mul32(h, 0x85EBCA6B)
    h = h ^ (h >> 13)
    h = _mul32(h, 0xC2B2AE35)
    h = h ^ (h >> 16)
    return h


def _fmix32_int(h: int) -> int:
    h &= 0xFFFFFFFF
    h ^= h >> 16
    h = (h * 0x85EBCA6B) & 0xFFFFFFFF
    h ^= h >> 13
    h = (h * 0xC2B2AE35) & 0xFFFFFFFF
    h ^= h >> 16
    return h


def _uniform24(seed: int, start: int, count: int, device) -> torch.Tensor:
    """24-bit uniforms for flat indices start..start+count-1 (int64 tensor)."""
    k0 = _fmix32_int(seed & 0xFFFFFFFF)
    k1 = _fmix32_int(((seed >> 32) ^ 0x9E3779B9) & 0xFFFFFFFF)
    idx = torch.arange(start, start + count, dtype=torch.int64, device=device)
    h = _fmix32(((idx & 0xFFFFFFFF) ^ k0))
    h = _fmix32((h + (idx >> 32) * 0x632BE5AB + k1) & 0xFFFFFFFF)
    return h >> 8


def _sample(kind: str, seed: int, count: int, device, chunk: int = 1 << 25) -> torch.Tensor:
    tab = _quantile_table(kind).to(device)
    out = torch.empty(count, dtype=torch.float32, device=device)
    for s in range(0, count, chunk):
        c = min(chunk, count - s)
        u = _uniform24(seed, s, c, device)
        i = u >> 8
        frac = (u & 0xFF).to(torch.float32) * (1.0 / 256.0)
        lo = tab[i]
        hi = tab[i + 1]
        d = hi - lo
        d = d * frac
        out[s:s + c] = lo + d
    return out


def matrix_seed(m: int, base: int = BASE_SEED) -> int:
    return base * 1000 + m


def outlier_columns(cols: int, seed: int) -> np.ndarray:
    rng = np.random.default_rng(seed ^ 0x5EED)
    k = int(round(0.01 * cols))
    return np.sort(rng.choice(cols, k, replace=False)) if k > 0 else np.zeros(0, dtype=np.int64)


def weight(rows: int, cols: int, seed: int, device="cpu") -> torch.Tensor:
    """fp32 [rows][cols]: t(5) scaled to std 0.02, 1 % of the columns times 8."""
    w = _sample("t5_std0.02", seed, rows * cols, device).view(rows, cols)
    colscale = torch.ones(cols, dtype=torch.float32)
    colscale[torch.from_numpy(outlier_columns(cols, seed))] = 8.0
    w *= colscale.to(device)
    return w


def activations(batch: int, cols: int, seed: int, device="cpu") -> torch.Tensor:
    """bf16 [batch][cols] ~ N(0,1)."""
    x = _sample("normal", seed + 10 ** 6, batch * cols, device).view(batch, cols)
    return x.to(torch.bfloat16)


def llama32_linear_shapes(model: str, n_layers: int | None = None, lm_head: bool = True):
    """[(name, out, in)] for every linear layer of one decode step, in model order."""
    cfg = {
        "1b": dict(h=2048, kv=512, ffn=8192, layers=16, vocab=128256),
        "3b": dict(h=3072, kv=1024, ffn=8192, layers=28, vocab=128256),
        # text decoder of LLaMA-3.2-11B-Vision (its self-attention layers): a second workload with long rows
        "11b": dict(h=4096, kv=1024, ffn=14336, layers=32, vocab=128256),
        # text decoder of LLaMA-3.2-90B-Vision (self-attention layers): the longest rows of the family
        "90b": dict(h=8192, kv=1024, ffn=28672, layers=80, vocab=128256),
    }[model.lower()]
    L = cfg["layers"] if n_layers is None else n_layers
    out = []
    for i in range(L):
        out += [
            (f"l{i}.q", cfg["h"], cfg["h"]),
            (f"l{i}.k", cfg["kv"], cfg["h"]),
            (f"l{i}.v", cfg["kv"], cfg["h"]),
            (f"l{i}.o", cfg["h"], cfg["h"]),
            (f"l{i}.gate", cfg["ffn"], cfg["h"]),
            (f"l{i}.up", cfg["ffn"], cfg["h"]),
            (f"l{i}.down", cfg["h"], cfg["ffn"]),
        ]
    if lm_head:
        out.append(("lm_head", cfg["vocab"], cfg["h"]))
    return out
