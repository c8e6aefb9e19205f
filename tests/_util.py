"""Shared helpers of the tests: golden-file reader, exact brute-force quantizers
written independently of the oracle, an independent generic-Adam loop."""
import os
from fractions import Fraction

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            key, vals = line.split("=", 1)
            out[key.strip()] = [float(v) for v in vals.split()]
    return out


def level_fractions(k, grid):
    """Non-negative levels of G as exact rationals, written from Section 5.1."""
    if grid == 1:      # uniform: c / 2^k
        return [Fraction(c, 2 ** k) for c in range(2 ** k + 1)]
    # geometric: 0, 2^-k, 2^-k+1, ..., 1
    return [Fraction(0)] + [Fraction(1, 2 ** (k - j)) for j in range(k + 1)]


def brute_nearest_level(y, levels):
    """argmin_c |y - levels[c]| over exact rationals; ties -> smaller level."""
    best, best_d = 0, None
    for c, lv in enumerate(levels):
        dist = abs(Fraction(y) - lv)
        if best_d is None or dist < best_d:
            best, best_d = c, dist
    return best


def brute_qg(u, k, grid):
    """Brute-force Q_g level indices for one segment: normalise by the max-abs
    in binary32, then exact nearest level."""
    u = np.asarray(u, dtype=np.float32)
    s = np.float32(np.max(np.abs(u))) if u.size else np.float32(0)
    levels = level_fractions(k, grid)
    q = np.zeros(u.size, dtype=np.int32)
    if s > 0:
        for j, uj in enumerate(u):
            y = np.float32(abs(uj)) / s          # one binary32 division
            c = brute_nearest_level(float(y), levels)
            q[j] = -c if uj < 0 else c
    return float(s), q


def brute_qx(x, kx):
    """Brute-force Q_x level indices: exact nearest point of c / 2^(kx+1),
    c in -2^kx..2^kx, ties toward zero."""
    x = np.asarray(x, dtype=np.float32)
    L = 2 ** kx
    grid = [Fraction(c, 2 ** (kx + 1)) for c in range(L + 1)]
    q = np.zeros(x.size, dtype=np.int32)
    for j, xj in enumerate(x):
        c = brute_nearest_level(abs(Fraction(float(xj))), grid)
        q[j] = -c if xj < 0 else c
    return q


def generic_adam_f32(x, grads, beta, theta, eps, lr):
    """Textbook 'generic Adam' (no bias correction, eps inside the root) in
    binary32 numpy, one rounding per operation.  grads: [T][d]."""
    f = np.float32
    x = np.array(x, dtype=np.float32)
    m = np.zeros_like(x)
    v = np.zeros_like(x)
    omb, omt = f(1) - f(beta), f(1) - f(theta)
    for g in grads:
        g = np.asarray(g, dtype=np.float32)
        v = f(theta) * v + omt * (g * g)
        m = f(beta) * m + omb * g
        x = x - (f(lr) * m) / np.sqrt(v + f(eps))
    return x, m, v


def generic_adam_f64(x, grads, beta, theta, eps, lr):
    """The same loop in binary64.  The hyper-parameters are the binary32 numbers
    the problem is given (0.999 and 1 - 0.999 are not binary32 numbers)."""
    beta, theta, eps, lr = (float(np.float32(h)) for h in (beta, theta, eps, lr))
    x = np.array(x, dtype=np.float64)
    m = np.zeros_like(x)
    v = np.zeros_like(x)
    for g in grads:
        g = np.asarray(g, dtype=np.float64)
        v = theta * v + (1 - theta) * g * g
        m = beta * m + (1 - beta) * g
        x = x - lr * m / np.sqrt(v + eps)
    return x, m, v


def pack_little_endian(codes, bits):
    """Independent statement of the packing: one big integer, element j at bit
    j*bits, written out least-significant byte first."""
    total = 0
    for j, c in enumerate(codes):
        total |= int(c) << (j * bits)
    nbytes = (len(codes) * bits + 7) // 8
    return np.frombuffer(total.to_bytes(nbytes, "little"), dtype=np.uint8)
