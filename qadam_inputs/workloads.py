"""The synthetic workloads: shapes, worker counts, step counts, distributions.

Each workload stands in for a training run of the kind the paper's Section 5
describes (a parameter set split into tensors, N workers each producing a
stochastic gradient per step).  Only sizes and value distributions are
described here; the tensors themselves are drawn in generate.py.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from math import prod
from typing import List, Optional, Tuple

from .shapes import bert_base_shapes, resnet18_shapes


@dataclass(frozen=True)
class Workload:
    name: str
    seg_len: Tuple[int, ...]          # elements per tensor, in order
    fan_in: Tuple[int, ...]           # per tensor; 0 for vectors
    is_gamma: Tuple[bool, ...]        # normalisation scale vectors (init 1)
    n: int                            # simulated workers
    steps: int                        # optimizer steps T
    grad: str                         # "gauss_worker" | "gauss_tensor" | "student_t_tensor" | "mixture" | "gauss_clip:<C>"
    w0: str                           # "gauss:<sigma>" | "he"
    kg: int = 0                       # gradient quantizer level parameter (-1: identity)
    kx: int = -1                      # weight quantizer level parameter (-1: none)
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    lr: float = 1e-3
    seed: int = 20200429
    per_tensor_scale: bool = True     # one max-abs scale per tensor (False: one per vector)
    scale_block: int = 0              # > 0: one scale per block of this many elements of a tensor

    @property
    def d(self) -> int:
        return sum(self.seg_len)

    @property
    def num_segments(self) -> int:
        return len(self.scale_seg_len)

    @property
    def scale_seg_len(self) -> Tuple[int, ...]:
        """Segment lengths as the quantizer sees them: the tensors (or the whole vector),
        each cut into blocks of `scale_block` elements when that is set (the last block of
        a tensor may be shorter)."""
        base = self.seg_len if self.per_tensor_scale else (self.d,)
        if self.scale_block <= 0:
            return base
        out = []
        for ln in base:
            full, rest = divmod(ln, self.scale_block)
            out.extend([self.scale_block] * full)
            if rest:
                out.append(rest)
        return tuple(out)

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


def _from_shapes(shapes):
    seg = tuple(prod(s) for _, s, _ in shapes)
    fan = tuple(f for _, _, f in shapes)
    gam = tuple(name.endswith(".gamma") for name, _, _ in shapes)
    return seg, fan, gam


def _flat(d):
    return (d,), (0,), (False,)


def get_workload(name: str, n: Optional[int] = None) -> Workload:
    """Workloads by name.  `n` overrides the worker count where a workload is
    defined as a sweep over worker counts ("flat28")."""
    if name == "flat20":
        seg, fan, gam = _flat(1 << 20)
        w = Workload("flat20", seg, fan, gam, n=4, steps=10, grad="gauss_worker",
                     w0="gauss:0.05", kg=0, kx=-1)
    elif name == "resnet18_qg":
        seg, fan, gam = _from_shapes(resnet18_shapes())
        w = Workload("resnet18_qg", seg, fan, gam, n=8, steps=100, grad="gauss_tensor",
                     w0="gauss:0.05", kg=0, kx=-1)
    elif name in ("resnet18_qg_qx", "resnet18_qg_qx_k0"):
        seg, fan, gam = _from_shapes(resnet18_shapes())
        w = Workload("resnet18_qg_qx_k0", seg, fan, gam, n=8, steps=100, grad="gauss_tensor",
                     w0="he", kg=0, kx=0)
    elif name == "resnet18_qg_qx_k1":
        seg, fan, gam = _from_shapes(resnet18_shapes())
        w = Workload("resnet18_qg_qx_k1", seg, fan, gam, n=8, steps=100, grad="gauss_tensor",
                     w0="he", kg=1, kx=1)
    elif name == "resnet18_qg_qx_8bit":
        seg, fan, gam = _from_shapes(resnet18_shapes())
        w = Workload("resnet18_qg_qx_8bit", seg, fan, gam, n=8, steps=100, grad="gauss_tensor",
                     w0="he", kg=0, kx=6)
    elif name == "bert_base":
        seg, fan, gam = _from_shapes(bert_base_shapes())
        w = Workload("bert_base", seg, fan, gam, n=16, steps=50, grad="student_t_tensor",
                     w0="gauss:0.02", kg=0, kx=0)
    elif name == "flat28":
        seg, fan, gam = _flat(1 << 28)
        w = Workload("flat28", seg, fan, gam, n=16, steps=20, grad="mixture",
                     w0="gauss:0.05", kg=0, kx=0)
    elif name.startswith("flat") and name[4:].isdigit() and 10 <= int(name[4:]) <= 30:
        # the flat28 recipe at another power-of-two length (profiling and sampling)
        seg, fan, gam = _flat(1 << int(name[4:]))
        w = Workload(name, seg, fan, gam, n=16, steps=20, grad="mixture",
                     w0="gauss:0.05", kg=0, kx=0)
    else:
        raise KeyError(f"unknown workload {name!r}; known: {WORKLOAD_NAMES}")
    if n is not None:
        w = w.with_(n=int(n))
    return w


WORKLOAD_NAMES = (
    "flat20", "resnet18_qg", "resnet18_qg_qx_k0", "resnet18_qg_qx_k1",
    "resnet18_qg_qx_8bit", "bert_base", "flat28",
)
