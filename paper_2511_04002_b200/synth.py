"""Seeded synthetic split-point hidden states.

These tensors stand in for the Llama-family split-layer activations the paper
compresses (its weights and evaluation data are not available here).  The module
only draws random numbers and casts them to 16 bits: it contains none of the
codec's arithmetic, and both the CUDA path and the CPU oracle are fed the very
same bytes it returns.

Every tensor is a pure function of (recipe, seed): numpy's Philox bit generator
is counter-based and its stream is fixed by the seed alone.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

_FP16_MAX = 65504.0


@dataclass(frozen=True)
class Recipe:
    """How one [tokens x hidden] tensor is drawn."""
    tokens: int
    hidden: int
    dtype: str = "f16"                   # "f16" | "bf16"
    base: str = "normal"                 # "normal" | "student_t"
    nu: float = 0.0                      # degrees of freedom for student_t
    token_scale_sigma: float = 0.0       # per-token factor exp(N(0, sigma)); 0 = none
    channel_outliers: Tuple[int, float] = (0, 1.0)   # (number of fixed channels, multiplier)
    random_outliers: Tuple[float, str, float, float] = (0.0, "none", 0.0, 0.0)
    # (rate, kind, p0, p1): kind "absnormal" -> +-|N(p0, p1)|, "uniform" -> +-U(p0, p1)
    kv_layers: int = 0                   # > 0: a KV cache, rows ordered [layer][key | value][token], tokens = 2 * kv_layers * w:
                                         # every layer's keys and values get their own factor exp(N(0, 0.3)), and the
                                         # fixed outlier channels exist in the key rows only


@dataclass(frozen=True)
class Workload:
    """A recipe plus the codec parameters it is run with."""
    name: str
    recipe: Recipe
    tau: float
    bits: Tuple[int, ...]
    delta: float = 0.2
    seed: int = 0
    steps: int = 1                       # >1: that many independent tensors, seed + i each
    note: str = ""


def torch_dtype(name: str) -> torch.dtype:
    return {"f16": torch.float16, "bf16": torch.bfloat16}[name]


def generate(recipe: Recipe, seed: int, row_chunk: int = 1024) -> torch.Tensor:
    """Draw one tensor. Returns a contiguous CPU tensor of the recipe's 16-bit dtype."""
    T, H = recipe.tokens, recipe.hidden
    rng = np.random.Generator(np.random.Philox(seed))
    out = torch.empty((T, H), dtype=torch_dtype(recipe.dtype))
    n_ch, ch_mult = recipe.channel_outliers
    channels = rng.choice(H, size=n_ch, replace=False) if n_ch > 0 else None
    rate, kind, p0, p1 = recipe.random_outliers
    layer_scale, is_key = None, None
    if recipe.kv_layers > 0:
        if T % (2 * recipe.kv_layers) != 0:
            raise ValueError("a KV cache of %d layers needs a multiple of %d rows" % (recipe.kv_layers, 2 * recipe.kv_layers))
        w = T // (2 * recipe.kv_layers)
        factors = np.exp(rng.standard_normal(2 * recipe.kv_layers) * 0.3).astype(np.float32)   # [layer][key | value]
        block = np.arange(T) // w
        layer_scale = factors[block][:, None]
        is_key = (block % 2 == 0)
    for t0 in range(0, T, row_chunk):
        t1 = min(T, t0 + row_chunk)
        n = t1 - t0
        if recipe.base == "normal":
            v = rng.standard_normal((n, H), dtype=np.float32)
        elif recipe.base == "student_t":
            v = rng.standard_t(recipe.nu, size=(n, H)).astype(np.float32)
        else:
            raise ValueError(recipe.base)
        if recipe.token_scale_sigma > 0:
            g = np.exp(rng.standard_normal((n, 1)) * recipe.token_scale_sigma).astype(np.float32)
            v *= g
        if layer_scale is not None:
            v *= layer_scale[t0:t1]
        if channels is not None:
            if is_key is None:
                v[:, channels] *= np.float32(ch_mult)
            else:
                rows = np.nonzero(is_key[t0:t1])[0]
                v[np.ix_(rows, channels)] *= np.float32(ch_mult)
        if rate > 0:
            hit = rng.random((n, H), dtype=np.float32) < np.float32(rate)
            k = int(hit.sum())
            if kind == "absnormal":
                mag = np.abs(rng.normal(p0, p1, size=k))
            elif kind == "uniform":
                mag = rng.uniform(p0, p1, size=k)
            else:
                raise ValueError(kind)
            sign = np.where(rng.random(k) < 0.5, -1.0, 1.0)
            v[hit] = (mag * sign).astype(np.float32)
        np.clip(v, -_FP16_MAX, _FP16_MAX, out=v)
        out[t0:t1] = torch.from_numpy(v).to(out.dtype)   # round-to-nearest-even cast
    return out


def raw_u16(x: torch.Tensor) -> np.ndarray:
    """The tensor's 16-bit patterns as a uint16 numpy array (no conversion)."""
    assert x.dtype in (torch.float16, torch.bfloat16) and x.is_contiguous()
    return x.cpu().view(torch.int16).numpy().view(np.uint16)


def from_raw_u16(a: np.ndarray, dtype: str) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch_dtype(dtype))


# ---- the five workloads -----------------------------------------------------------------

def c1_prefill() -> Workload:
    return Workload("c1_prefill_128x4096_f16",
                    Recipe(128, 4096, "f16", "normal", token_scale_sigma=0.5, channel_outliers=(8, 50.0)),
                    tau=6.0, bits=(2, 4, 8), seed=0)


def c2_decode_steps(steps: int = 512) -> Workload:
    return Workload("c2_decode_steps_64x4096_f16",
                    Recipe(64, 4096, "f16", "normal", token_scale_sigma=0.5,
                           random_outliers=(0.001, "absnormal", 40.0, 10.0)),
                    tau=6.0, bits=(2, 4, 8), seed=1000, steps=steps,
                    note="step i uses seed 1000 + i")


def c3_13b_prefill() -> Workload:
    return Workload("c3_llama2_13b_2048x5120_f16",
                    Recipe(2048, 5120, "f16", "student_t", nu=4.0, token_scale_sigma=0.5,
                           channel_outliers=(16, 30.0)),
                    tau=6.0, bits=(2, 3, 4, 8), seed=3)


def c4_70b_prefill(tokens: int = 8192) -> Workload:
    return Workload("c4_llama3_70b_%dx8192_bf16" % tokens,
                    Recipe(tokens, 8192, "bf16", "student_t", nu=3.0,
                           random_outliers=(0.001, "uniform", 20.0, 100.0)),
                    tau=8.0, bits=(2, 4, 8), seed=4)


def kv_cache(w: int = 256, layers: int = 20) -> Workload:
    """Keys and values of the first `layers` decoder layers for w tokens of a 7B-shaped model (4096 = heads x head
    dimension), the tensor Eq. "bkv" sizes: [2 * layers * w] rows through the same codec."""
    rows = 2 * layers * w
    return Workload("kv_llama2_7b_l%d_w%d_%dx4096_f16" % (layers, w, rows),
                    Recipe(rows, 4096, "f16", "normal", token_scale_sigma=0.2, channel_outliers=(8, 8.0), kv_layers=layers),
                    tau=6.0, bits=(2, 4, 8), seed=7)


C5_TOKENS = (1, 16, 256, 4096, 32768)
C5_RATES = (0.0, 0.001, 0.01)
C5_DTYPES = ("f16", "bf16")


def c5_sweep_point(i_tok: int, i_rate: int, i_dtype: int) -> Workload:
    tokens, rate, dt = C5_TOKENS[i_tok], C5_RATES[i_rate], C5_DTYPES[i_dtype]
    ro = (rate, "absnormal", 40.0, 10.0) if rate > 0 else (0.0, "none", 0.0, 0.0)
    return Workload("c5_sweep_%dx4096_%s_rate%g" % (tokens, dt, rate),
                    Recipe(tokens, 4096, dt, "normal", token_scale_sigma=0.5, random_outliers=ro),
                    tau=6.0, bits=(2, 4, 8), seed=5000 + 100 * i_tok + 10 * i_rate + i_dtype)


def c5_sweep() -> List[Workload]:
    return [c5_sweep_point(a, b, c) for a in range(len(C5_TOKENS)) for b in range(len(C5_RATES))
            for c in range(len(C5_DTYPES))]


def make(workload: Workload, step: int = 0) -> torch.Tensor:
    return generate(workload.recipe, workload.seed + step)
