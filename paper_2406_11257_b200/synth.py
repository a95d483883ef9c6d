"""Seeded synthetic checkpoints: tensor lists shaped like the models named in the
workload configurations, filled from the stated distributions.

This module only makes inputs.  It holds none of the compression arithmetic and
is the one piece of code that both the CUDA tests/benchmark and the CPU oracle
are fed from (the same bits go to both: tensors are generated once, on whatever
device is asked for, and copied).

Distributions (all fp32, all streams independent):
    W_prev ~ N(0, 0.02)
    delta  ~ Student-t(nu = 3) scaled to standard deviation 1e-4
             (t_3 = Z0 / sqrt((Z1^2 + Z2^2 + Z3^2) / 3), variance 3)
    W_t    = W_prev + delta
    ea     ~ N(0, 1e-4)                      (Adam first moment)
    eas    = (|N(0,1)| * 1e-4)^2 + 1e-12     (Adam second moment)
With `outlier_frac` > 0 an independent Bernoulli subset of delta is multiplied
by `outlier_scale` (the threshold-stress configuration).
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch


@dataclass(frozen=True)
class ModelShape:
    name: str
    family: str          # "neox" or "llama"
    layers: int
    d_model: int
    ffn: int
    vocab: int


CONFIG_SHAPES = {
    "tiny": ModelShape("tiny-neox", "neox", 2, 256, 1024, 4096),
    "pythia-410m": ModelShape("pythia-410m-shaped", "neox", 24, 1024, 4096, 50304),
    "pythia-1.4b": ModelShape("pythia-1.4b-shaped", "neox", 24, 2048, 8192, 50304),
    "llama-7b": ModelShape("llama-7b-shaped", "llama", 32, 4096, 11008, 32000),
}


def tensor_list(shape: ModelShape) -> list[tuple[str, int]]:
    """(name, numel) of every parameter tensor, in checkpoint order."""
    d, f, v = shape.d_model, shape.ffn, shape.vocab
    out: list[tuple[str, int]] = [("embed_in", v * d)]
    for i in range(shape.layers):
        p = f"layers.{i}."
        if shape.family == "neox":
            out += [(p + "ln1.w", d), (p + "ln1.b", d), (p + "ln2.w", d), (p + "ln2.b", d),
                    (p + "qkv.w", 3 * d * d), (p + "qkv.b", 3 * d),
                    (p + "attn_out.w", d * d), (p + "attn_out.b", d),
                    (p + "fc1.w", f * d), (p + "fc1.b", f),
                    (p + "fc2.w", d * f), (p + "fc2.b", d)]
        else:
            out += [(p + "q", d * d), (p + "k", d * d), (p + "v", d * d), (p + "o", d * d),
                    (p + "gate", f * d), (p + "up", f * d), (p + "down", d * f),
                    (p + "norm1", d), (p + "norm2", d)]
    if shape.family == "neox":
        out += [("final_ln.w", d), ("final_ln.b", d)]
    else:
        out += [("final_norm", d)]
    out.append(("embed_out", v * d))
    return out


def _seed_for(global_seed: int, step: int, tensor_index: int) -> int:
    # distinct streams per (seed, step, tensor); plain integer packing
    return (global_seed * 1_000_003 + step) * 1_000_003 + tensor_index


def _student_t3(n: int, gen: torch.Generator, device) -> torch.Tensor:
    z0 = torch.randn(n, generator=gen, device=device, dtype=torch.float32)
    chi = torch.randn(n, generator=gen, device=device, dtype=torch.float32).square_()
    for _ in range(2):
        chi += torch.randn(n, generator=gen, device=device, dtype=torch.float32).square_()
    return z0.div_(chi.div_(3.0).sqrt_())


def make_delta(numel: int, gen: torch.Generator, device, outlier_frac: float = 0.0,
               outlier_scale: float = 10.0) -> torch.Tensor:
    delta = _student_t3(numel, gen, device).mul_(1e-4 / math.sqrt(3.0))
    if outlier_frac > 0.0:
        hit = torch.rand(numel, generator=gen, device=device) < outlier_frac
        delta = torch.where(hit, delta * outlier_scale, delta)
    return delta


def make_moments(numel: int, gen: torch.Generator, device):
    ea = torch.randn(numel, generator=gen, device=device, dtype=torch.float32).mul_(1e-4)
    eas = torch.randn(numel, generator=gen, device=device, dtype=torch.float32).abs_().mul_(1e-4)
    eas = eas.square_().add_(1e-12)
    return ea, eas


def make_quad(numel: int, global_seed: int, tensor_index: int, device="cpu", step: int = 0,
              outlier_frac: float = 0.0, w_prev: torch.Tensor | None = None):
    """One tensor's (w_t, w_prev, ea, eas).  If `w_prev` is given (a chain step)
    it is used as W_(t-1) instead of a fresh draw."""
    gen = torch.Generator(device=device)
    gen.manual_seed(_seed_for(global_seed, step, tensor_index))
    if w_prev is None:
        w_prev = torch.randn(numel, generator=gen, device=device, dtype=torch.float32).mul_(0.02)
    delta = make_delta(numel, gen, device, outlier_frac)
    w_t = w_prev + delta
    ea, eas = make_moments(numel, gen, device)
    return w_t, w_prev, ea, eas


def make_checkpoint(config: str, global_seed: int = 0, device="cpu", step: int = 0,
                    outlier_frac: float = 0.0, max_tensors: int | None = None):
    """List of (name, w_t, w_prev, ea, eas) for a named configuration."""
    shapes = tensor_list(CONFIG_SHAPES[config])
    if max_tensors is not None:
        shapes = shapes[:max_tensors]
    out = []
    for i, (name, numel) in enumerate(shapes):
        out.append((name,) + make_quad(numel, global_seed, i, device, step, outlier_frac))
    return out
