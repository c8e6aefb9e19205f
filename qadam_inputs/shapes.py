"""Parameter-tensor shape lists of two well-known network layouts.

The experiments of the paper (Section 5) train convolutional networks with
8 workers; the synthetic workloads used here only need the *shapes* of such
parameter sets (how many tensors, how uneven their sizes are), not the networks.
Each entry is (name, shape, fan_in); fan_in is 0 for normalisation scale/shift
and bias vectors.
"""
from __future__ import annotations

from math import prod
from typing import List, Tuple

Shape = Tuple[str, Tuple[int, ...], int]


def numel(shapes: List[Shape]) -> int:
    return sum(prod(s) for _, s, _ in shapes)


def _conv(name, cout, cin, k):
    return (name, (cout, cin, k, k), cin * k * k)


def _norm(name, c):
    return [(name + ".gamma", (c,), 0), (name + ".beta", (c,), 0)]


def resnet18_shapes() -> List[Shape]:
    """62 tensors, 11 689 512 elements: 7x7 stem, four stages of two basic
    blocks (3x3 convolutions, 64..512 channels), three 1x1 downsample
    convolutions, a scale and a shift vector per normalisation layer, and a
    1000x512 classifier with bias."""
    out: List[Shape] = [_conv("stem.conv", 64, 3, 7)] + _norm("stem.norm", 64)
    cin = 64
    for stage, cout in enumerate((64, 128, 256, 512), start=1):
        for block in range(2):
            p = f"stage{stage}.block{block}"
            out.append(_conv(p + ".conv1", cout, cin if block == 0 else cout, 3))
            out += _norm(p + ".norm1", cout)
            out.append(_conv(p + ".conv2", cout, cout, 3))
            out += _norm(p + ".norm2", cout)
            if block == 0 and cin != cout:
                out.append(_conv(p + ".down.conv", cout, cin, 1))
                out += _norm(p + ".down.norm", cout)
        cin = cout
    out.append(("fc.weight", (1000, 512), 512))
    out.append(("fc.bias", (1000,), 0))
    return out


def bert_base_shapes() -> List[Shape]:
    """199 tensors, 109 482 240 elements: token / position / type embeddings
    with their layer norm, 12 encoder layers (four 768x768 attention
    projections, a 768->3072->768 feed-forward pair, two layer norms, all with
    biases) and a 768x768 pooler."""
    h, ff = 768, 3072
    out: List[Shape] = [
        ("emb.word", (30522, h), h),
        ("emb.position", (512, h), h),
        ("emb.type", (2, h), h),
    ] + _norm("emb.norm", h)
    for layer in range(12):
        p = f"layer{layer}"
        for proj in ("q", "k", "v", "o"):
            out.append((f"{p}.attn.{proj}.weight", (h, h), h))
            out.append((f"{p}.attn.{proj}.bias", (h,), 0))
        out += _norm(p + ".attn.norm", h)
        out.append((p + ".ffn.in.weight", (ff, h), h))
        out.append((p + ".ffn.in.bias", (ff,), 0))
        out.append((p + ".ffn.out.weight", (h, ff), ff))
        out.append((p + ".ffn.out.bias", (h,), 0))
        out += _norm(p + ".ffn.norm", h)
    out.append(("pooler.weight", (h, h), h))
    out.append(("pooler.bias", (h,), 0))
    return out
