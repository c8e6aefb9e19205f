"""Draws the synthetic tensors of a workload from a seed.

Every tensor is a function of (workload.seed, purpose, step, worker) only, so
any worker's gradient for any step can be regenerated alone.  A tensor is drawn
once, on whichever device is asked for, and then copied wherever it is needed:
the CPU and CUDA generators of torch do not produce the same stream, so
bit-identical inputs come from copying, not from re-drawing.

All tensors are returned in the *logical* layout: the workload's tensors
concatenated without padding, length workload.d.
"""
from __future__ import annotations

import math
from typing import Optional

import torch

from .workloads import Workload

_MASK = (1 << 64) - 1


def _splitmix64(x: int) -> int:
    x = (x + 0x9E3779B97F4A7C15) & _MASK
    z = x
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK
    return z ^ (z >> 31)


def _generator(device, seed: int, purpose: int, step: int, worker: int) -> torch.Generator:
    s = _splitmix64(seed & _MASK)
    for v in (purpose, step, worker):
        s = _splitmix64(s ^ (v & _MASK))
    g = torch.Generator(device=device)
    g.manual_seed(s & ((1 << 63) - 1))
    return g


def _tensor_scales(w: Workload, lo: float, hi: float) -> torch.Tensor:
    """One positive scale per tensor, log-uniform in [lo, hi], fixed by the seed."""
    g = _generator("cpu", w.seed, 7, 0, 0)
    u = torch.rand(len(w.seg_len), generator=g, dtype=torch.float64)
    return torch.exp(math.log(lo) + u * (math.log(hi) - math.log(lo))).to(torch.float32)


def _scale_tensors_(out: torch.Tensor, w: Workload, scales: torch.Tensor) -> None:
    off = 0
    for length, s in zip(w.seg_len, scales.tolist()):
        out[off:off + length].mul_(s)
        off += length


def gradients(w: Workload, step: int, worker: int, device="cpu",
              out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Worker `worker`'s stochastic gradient for step `step` (1-based), fp32 [d]."""
    d = w.d
    gen = _generator(device, w.seed, 1, step, worker)
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=device)
    out.normal_(0.0, 1.0, generator=gen)
    if w.grad == "gauss_worker":
        out.mul_(0.01 * (1.0 + 0.1 * worker))
    elif w.grad == "gauss_tensor":
        _scale_tensors_(out, w, _tensor_scales(w, 1e-4, 1e-1))
    elif w.grad == "student_t_tensor":
        # Student-t with 3 degrees of freedom: normal / sqrt(chi2_3 / 3), chunked
        chunk = 1 << 24
        for lo in range(0, d, chunk):
            hi = min(d, lo + chunk)
            c = torch.empty(3, hi - lo, dtype=torch.float32, device=device)
            c.normal_(0.0, 1.0, generator=gen)
            out[lo:hi].div_(c.square_().mean(dim=0).sqrt_())
        _scale_tensors_(out, w, _tensor_scales(w, 1e-5, 1e-2))
    elif w.grad == "mixture":
        # 99 % N(0, 1e-3^2) with 1 % N(0, 1e-1^2) outliers
        chunk = 1 << 24
        for lo in range(0, d, chunk):
            hi = min(d, lo + chunk)
            u = torch.empty(hi - lo, dtype=torch.float32, device=device)
            u.uniform_(0.0, 1.0, generator=gen)
            sig = torch.where(u < 0.01, 1e-1, 1e-3).to(torch.float32)
            out[lo:hi].mul_(sig)
    elif w.grad.startswith("gauss_clip:"):
        # N(0, 1e-3^2) clipped at C sigma: the max-abs scale is C sigma for every worker, so a
        # known share of the values lies above half of it (C = 5: 1.2 %, C = 4: 4.6 %, C = 2: 32 %):
        # gradients whose ternary codes have a chosen density
        c = float(w.grad.split(":")[1])
        out.clamp_(-c, c).mul_(1e-3)
    else:
        raise ValueError(w.grad)
    return out


def initial_weights(w: Workload, device="cpu") -> torch.Tensor:
    """x_1, fp32 [d]."""
    gen = _generator(device, w.seed, 2, 0, 0)
    out = torch.empty(w.d, dtype=torch.float32, device=device)
    out.normal_(0.0, 1.0, generator=gen)
    if w.w0.startswith("gauss:"):
        out.mul_(float(w.w0.split(":")[1]))
    elif w.w0 == "he":
        off = 0
        for length, fan, gamma in zip(w.seg_len, w.fan_in, w.is_gamma):
            if fan > 0:
                out[off:off + length].mul_(math.sqrt(2.0 / fan))
            else:
                out[off:off + length].fill_(1.0 if gamma else 0.0)
            off += length
    else:
        raise ValueError(w.w0)
    return out
