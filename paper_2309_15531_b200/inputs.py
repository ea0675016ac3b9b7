"""Seeded synthetic layers and calibration activations.

This module only draws random tensors; it holds none of the quantization
arithmetic.  Both the CPU oracle's tests and the CUDA library's tests take
their inputs from here, so that the two sides always see the same bytes.

The tensors stand in for the trained LLaMA-family weights and the text
calibration sets of the paper (Section 4.1), which are not available offline.
Shapes follow LLaMA linear layers; the value structure follows the paper's
description of activation outliers: a small subset of hidden dimensions whose
magnitude is far above the rest (Section 2.2).

Every tensor is a pure function of (base seed, tensor id, shape, recipe) on a
given device type.  A tensor needed by both sides of a comparison is drawn
once and handed to both.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import torch

BASE_SEED = 230915531


@dataclasses.dataclass(frozen=True)
class WeightSpec:
    """Recipe for one linear layer's weight W[out, in]."""
    out: int
    inp: int
    dtype: str = "f16"            # "f16" | "f32"
    sigma: float = 0.02           # N(0, sigma^2) body
    heavy_frac: float = 0.0       # fraction of entries replaced by sigma * Student-t(3)
    seed: int = 0                 # added to BASE_SEED


@dataclasses.dataclass(frozen=True)
class CalibSpec:
    """Recipe for calibration activations X[n_tokens, in]."""
    n_tokens: int
    inp: int
    dtype: str = "bf16"           # "bf16" | "f32"
    kind: str = "normal"          # "normal": N(0,1);  "skew": |a| * silu(c), a,c ~ N(0,1)
    n_outlier: int = 0            # number of outlier channels (drawn without replacement)
    outlier_lo: float = 1.0       # outlier scale ~ U(lo, hi) per channel (lo == hi: constant)
    outlier_hi: float = 1.0
    seed: int = 0


_TORCH_DTYPE = {"f16": torch.float16, "f32": torch.float32, "bf16": torch.bfloat16}


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(BASE_SEED + int(seed))
    return g


def make_weight(spec: WeightSpec, device="cpu") -> torch.Tensor:
    """W[out, in], row-major contiguous, in spec.dtype."""
    g = _gen(spec.seed, device)
    w = torch.randn(spec.out, spec.inp, generator=g, device=device, dtype=torch.float32) * spec.sigma
    if spec.heavy_frac > 0.0:
        pick = torch.rand(spec.out, spec.inp, generator=g, device=device) < spec.heavy_frac
        z = torch.randn(spec.out, spec.inp, generator=g, device=device)
        chi = torch.randn(3, spec.out, spec.inp, generator=g, device=device).square_().sum(0)
        t3 = z / torch.sqrt(chi / 3.0)
        w = torch.where(pick, t3 * spec.sigma, w)
        del pick, z, chi, t3
    return w.to(_TORCH_DTYPE[spec.dtype]).contiguous()


def outlier_channels(spec: CalibSpec):
    """(channel ids int64[n_outlier], scales float32[n_outlier]); always drawn on CPU."""
    g = _gen(spec.seed + 500_000, "cpu")
    ids = torch.randperm(spec.inp, generator=g)[: spec.n_outlier].sort().values
    u = torch.rand(spec.n_outlier, generator=g)
    scales = spec.outlier_lo + (spec.outlier_hi - spec.outlier_lo) * u
    return ids, scales.to(torch.float32)


def make_calib(spec: CalibSpec, device="cpu", out: Optional[torch.Tensor] = None,
               chunk_tokens: int = 16384) -> torch.Tensor:
    """X[n_tokens, in], row-major contiguous, in spec.dtype.  Drawn in token chunks
    (the chunking is part of the recipe: it fixes the order of the random draws)."""
    g = _gen(spec.seed, device)
    dt = _TORCH_DTYPE[spec.dtype]
    if out is None:
        out = torch.empty(spec.n_tokens, spec.inp, device=device, dtype=dt)
    ids, scales = outlier_channels(spec)
    colscale = torch.ones(spec.inp, dtype=torch.float32)
    colscale[ids] = scales
    colscale = colscale.to(device)
    for t0 in range(0, spec.n_tokens, chunk_tokens):
        n = min(chunk_tokens, spec.n_tokens - t0)
        a = torch.randn(n, spec.inp, generator=g, device=device, dtype=torch.float32)
        if spec.kind == "skew":
            c = torch.randn(n, spec.inp, generator=g, device=device, dtype=torch.float32)
            a = a.abs_() * torch.nn.functional.silu(c)
        elif spec.kind != "normal":
            raise ValueError(f"unknown calibration kind {spec.kind!r}")
        a *= colscale
        out[t0:t0 + n].copy_(a)
    return out


# ---------------------------------------------------------------------------
# Named workloads.  `scale` shrinks token counts / shapes for quick tests while
# keeping the recipe; scale=1 is the full-size workload.
# ---------------------------------------------------------------------------

def _ceil_frac(n: int, frac: float) -> int:
    return int(math.ceil(n * frac))


def workload_small():
    """Single linear 512x512 fp32, 256 calibration tokens, 4 outlier channels x60.
    RTN 3-bit g128 in both dims, score, select."""
    w = WeightSpec(512, 512, "f32", 0.02, 0.0, seed=1000)
    x = CalibSpec(256, 512, "f32", "normal", 4, 60.0, 60.0, seed=1001)
    return {"name": "small_512", "layers": {"linear": (w, x)}, "bits": 3, "group": 128}


def workload_qproj(n_tokens: int = 128 * 2048, out: int = 4096, inp: int = 4096):
    """LLaMA-7B q_proj-shaped layer: fp16 N(0,0.02^2) with 0.1% Student-t(3) entries;
    bf16 N(0,1) activations with ceil(0.5%) outlier channels scaled by U(50,100)."""
    w = WeightSpec(out, inp, "f16", 0.02, 0.001, seed=2000)
    x = CalibSpec(n_tokens, inp, "bf16", "normal", _ceil_frac(inp, 0.005), 50.0, 100.0, seed=2001)
    return {"name": "llama7b_q_proj", "layers": {"q_proj": (w, x)}, "bits": 3, "group": 128}


def workload_downproj(n_tokens: int = 128 * 2048, out: int = 4096, inp: int = 11008):
    """LLaMA-7B down_proj-shaped layer: fp16 N(0,0.015^2); skewed non-negative-leaning
    activations |a|*silu(c) with ceil(0.2%) outlier channels x80."""
    w = WeightSpec(out, inp, "f16", 0.015, 0.0, seed=3000)
    x = CalibSpec(n_tokens, inp, "bf16", "skew", _ceil_frac(inp, 0.002), 80.0, 80.0, seed=3001)
    return {"name": "llama7b_down_proj", "layers": {"down_proj": (w, x)},
            "variants": [(4, 128), (3, 64)]}


def workload_block(n_tokens: int = 128 * 2048, hidden: int = 4096, ffn: int = 11008):
    """LLaMA-7B-shaped decoder block: q,k,v,o [h,h]; gate,up [ffn,h]; down [h,ffn].
    One activation tensor per distinct input width: the six hidden-input layers
    share one X (and therefore one Hessian); down_proj has its own."""
    xh = CalibSpec(n_tokens, hidden, "bf16", "normal", _ceil_frac(hidden, 0.005), 50.0, 100.0, seed=4001)
    xf = CalibSpec(n_tokens, ffn, "bf16", "skew", _ceil_frac(ffn, 0.002), 80.0, 80.0, seed=4002)
    layers = {}
    for k, name in enumerate(["q_proj", "k_proj", "v_proj", "o_proj"]):
        layers[name] = (WeightSpec(hidden, hidden, "f16", 0.02, 0.0, seed=4010 + k), xh)
    for k, name in enumerate(["gate_proj", "up_proj"]):
        layers[name] = (WeightSpec(ffn, hidden, "f16", 0.02, 0.0, seed=4020 + k), xh)
    layers["down_proj"] = (WeightSpec(hidden, ffn, "f16", 0.02, 0.0, seed=4030), xf)
    return {"name": "llama7b_block", "layers": layers, "bits": 3, "group": 128}


def workload_mlp70b(n_tokens: int = 128 * 2048, hidden: int = 8192, ffn: int = 28672):
    """LLaMA-2-70B-shaped MLP: gate/up [ffn,h], down [h,ffn]; fp16 N(0,0.01^2) with 0.1%
    heavy-tail entries; activations N(0,1) with ceil(0.5%) outlier channels x100."""
    xh = CalibSpec(n_tokens, hidden, "bf16", "normal", _ceil_frac(hidden, 0.005), 100.0, 100.0, seed=5001)
    xf = CalibSpec(n_tokens, ffn, "bf16", "normal", _ceil_frac(ffn, 0.005), 100.0, 100.0, seed=5002)
    layers = {
        "gate_proj": (WeightSpec(ffn, hidden, "f16", 0.01, 0.001, seed=5010), xh),
        "up_proj": (WeightSpec(ffn, hidden, "f16", 0.01, 0.001, seed=5011), xh),
        "down_proj": (WeightSpec(hidden, ffn, "f16", 0.01, 0.001, seed=5012), xf),
    }
    return {"name": "llama2_70b_mlp", "layers": layers, "bits": 4, "group": 128}
