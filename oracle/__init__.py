"""ctypes front-end of the CPU oracle (oracle/qadam_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
CPU-baseline leg of the benchmark.  The product package never imports this.

`build()` compiles the C++ file with g++ into oracle/libqadam_oracle.so with
floating-point contraction switched off; every other function loads that
library.  `OracleState` holds the state of one parameter-server problem
(x, m, v, e for all workers) as numpy arrays in the padded layout and steps it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qadam_oracle.cpp")
_LIB = os.path.join(_HERE, "libqadam_oracle.so")

PLACE_SERVER = 0
PLACE_WORKER = 1
GRID_POW2 = 0
GRID_UNIFORM = 1
GRID_STOCHASTIC = 2     # kg = 0 only: the stochastic ternary operator (Philox4x32-10 coins)
ALIGN = 128


def build(force: bool = False) -> str:
    """Compile the oracle if the library is missing or older than its source."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math",
           "-fPIC", "-shared", "-o", _LIB, _SRC]
    subprocess.run(cmd, check=True)
    return _LIB


class _Problem(C.Structure):
    _fields_ = [
        ("d", C.c_int64), ("D", C.c_int64), ("n", C.c_int32), ("S", C.c_int32),
        ("seg_len", C.POINTER(C.c_int64)), ("seg_off", C.POINTER(C.c_int64)),
        ("kg", C.c_int32), ("kx", C.c_int32), ("grid_g", C.c_int32), ("placement", C.c_int32),
        ("beta", C.c_float), ("theta", C.c_float), ("eps", C.c_float),
        ("weight_decay", C.c_float), ("seed", C.c_uint64),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        f32p, i32p, u32p, u8p, i64p = (C.POINTER(C.c_float), C.POINTER(C.c_int32),
                                       C.POINTER(C.c_uint32), C.POINTER(C.c_uint8),
                                       C.POINTER(C.c_int64))
        pp = C.POINTER(_Problem)
        L.qo_layout.restype = C.c_int64
        L.qo_layout.argtypes = [C.c_int32, i64p, i64p]
        L.qo_grad_levels.restype = C.c_int32
        L.qo_grad_levels.argtypes = [C.c_int32, C.c_int32, f32p, C.c_int32]
        L.qo_grad_code_bits.restype = C.c_int32
        L.qo_grad_code_bits.argtypes = [C.c_int32, C.c_int32]
        L.qo_weight_code_bits.restype = C.c_int32
        L.qo_weight_code_bits.argtypes = [C.c_int32]
        L.qo_gcode_bytes.restype = C.c_int64
        L.qo_gcode_bytes.argtypes = [pp]
        L.qo_wcode_bytes.restype = C.c_int64
        L.qo_wcode_bytes.argtypes = [pp]
        L.qo_quantize_grad_segment.restype = C.c_int32
        L.qo_quantize_grad_segment.argtypes = [f32p, C.c_int64, C.c_int32, C.c_int32, f32p, i32p, f32p]
        L.qo_quantize_weights.restype = None
        L.qo_quantize_weights.argtypes = [f32p, C.c_int64, C.c_int32, i32p, f32p, f32p]
        L.qo_pack_bits.restype = None
        L.qo_pack_bits.argtypes = [u32p, C.c_int64, C.c_int32, u8p]
        L.qo_unpack_bits.restype = None
        L.qo_unpack_bits.argtypes = [u8p, C.c_int64, C.c_int32, u32p]
        L.qo_worker_step.restype = C.c_int32
        L.qo_worker_step.argtypes = [pp, f32p, f32p, f32p, f32p, f32p, C.c_float, f32p, u8p,
                                     C.c_int32, C.c_int64]
        L.qo_philox4x32_10.restype = None
        L.qo_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.qo_quantize_grad_segment_stochastic.restype = C.c_int32
        L.qo_quantize_grad_segment_stochastic.argtypes = [f32p, C.c_int64, C.c_int64, C.c_uint64, C.c_uint32,
                                                          C.c_uint32, f32p, i32p, f32p]
        L.qo_broadcast_weights.restype = C.c_int32
        L.qo_broadcast_weights.argtypes = [pp, f32p, u8p, f32p, f32p]
        L.qo_server_step.restype = C.c_int32
        L.qo_server_step.argtypes = [pp, f32p, u8p, f32p, f32p, f32p, C.c_float, u8p, f32p, f32p]
        L.qo_decode_weights.restype = C.c_int32
        L.qo_decode_weights.argtypes = [pp, u8p, f32p]
        _lib = L
    return _lib


def _p(a: Optional[np.ndarray], ctype):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(C.POINTER(ctype))


# ------------------------------------------------------------------ primitives

def layout(seg_len: Sequence[int]):
    """Padded offsets of the segments and the padded total D."""
    sl = np.ascontiguousarray(seg_len, dtype=np.int64)
    off = np.zeros(len(sl), dtype=np.int64)
    D = lib().qo_layout(len(sl), _p(sl, C.c_int64), _p(off, C.c_int64))
    return off, int(D)


def grad_levels(kg: int, grid: int = GRID_POW2) -> np.ndarray:
    buf = np.zeros(1 << 15, dtype=np.float32)
    L = lib().qo_grad_levels(kg, grid, _p(buf, C.c_float), buf.size)
    if L < 0:
        raise ValueError("bad (kg, grid)")
    return buf[:L + 1].copy()


def grad_code_bits(kg: int, grid: int = GRID_POW2) -> int:
    return int(lib().qo_grad_code_bits(kg, grid))


def weight_code_bits(kx: int) -> int:
    return int(lib().qo_weight_code_bits(kx))


def quantize_grad_segment(u: np.ndarray, kg: int, grid: int = GRID_POW2):
    """-> (scale, q[int32], resid[float32]) for one segment."""
    u = np.ascontiguousarray(u, dtype=np.float32)
    q = np.zeros(u.size, dtype=np.int32)
    r = np.zeros(u.size, dtype=np.float32)
    s = np.zeros(1, dtype=np.float32)
    rc = lib().qo_quantize_grad_segment(_p(u, C.c_float), u.size, kg, grid,
                                        _p(s, C.c_float), _p(q, C.c_int32), _p(r, C.c_float))
    if rc != 0:
        raise ValueError("bad (kg, grid)")
    return float(s[0]), q, r


def philox4x32_10(ctr, key) -> np.ndarray:
    """One block of Philox4x32-10: ctr four and key two 32-bit words -> four words."""
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().qo_philox4x32_10(_p(c, C.c_uint32), _p(k, C.c_uint32), _p(out, C.c_uint32))
    return out


def quantize_grad_segment_stochastic(u: np.ndarray, first_elem: int, seed: int, step: int, worker: int):
    """Stochastic ternary operator on one segment -> (scale, q[int32], resid[float32])."""
    u = np.ascontiguousarray(u, dtype=np.float32)
    q = np.zeros(u.size, dtype=np.int32)
    r = np.zeros(u.size, dtype=np.float32)
    s = np.zeros(1, dtype=np.float32)
    lib().qo_quantize_grad_segment_stochastic(_p(u, C.c_float), u.size, first_elem, seed, step, worker,
                                              _p(s, C.c_float), _p(q, C.c_int32), _p(r, C.c_float))
    return float(s[0]), q, r


def quantize_weights(x: np.ndarray, kx: int):
    """-> (q[int32], xhat[float32], resid[float32])."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    q = np.zeros(x.size, dtype=np.int32)
    xh = np.zeros(x.size, dtype=np.float32)
    r = np.zeros(x.size, dtype=np.float32)
    lib().qo_quantize_weights(_p(x, C.c_float), x.size, kx, _p(q, C.c_int32),
                              _p(xh, C.c_float), _p(r, C.c_float))
    return q, xh, r


def pack_bits(code: np.ndarray, bits: int) -> np.ndarray:
    code = np.ascontiguousarray(code, dtype=np.uint32)
    out = np.zeros((code.size * bits + 7) // 8, dtype=np.uint8)
    lib().qo_pack_bits(_p(code, C.c_uint32), code.size, bits, _p(out, C.c_uint8))
    return out


def unpack_bits(stream: np.ndarray, count: int, bits: int) -> np.ndarray:
    stream = np.ascontiguousarray(stream, dtype=np.uint8)
    assert stream.size * 8 >= count * bits
    out = np.zeros(count, dtype=np.uint32)
    lib().qo_unpack_bits(_p(stream, C.c_uint8), count, bits, _p(out, C.c_uint32))
    return out


# ------------------------------------------------------------------ whole problem

class OracleState:
    """State of one parameter-server problem, stepped by the oracle.

    Arrays are in the padded layout ([D], pads zero): x; m, v ([D] with the
    moments on the server, [n][D] with the moments on the workers); e [n][D];
    and the last step's outputs scales [n][S], gcodes [n][gcode_bytes],
    wcodes [wcode_bytes], wresid [D].
    """

    def __init__(self, seg_len: Sequence[int], n: int, kg: int, kx: int, placement: int,
                 beta1: float, beta2: float, eps: float, grid_g: int = GRID_POW2,
                 want_wresid: bool = False, seed: int = 0, want_wfeedback: bool = False):
        self.seg_len = np.ascontiguousarray(seg_len, dtype=np.int64)
        self.seg_off, self.D = layout(self.seg_len)
        self.d = int(self.seg_len.sum())
        self.n, self.S = int(n), len(self.seg_len)
        self.kg, self.kx, self.grid_g, self.placement = kg, kx, grid_g, placement
        self._prob = _Problem(self.d, self.D, self.n, self.S,
                              _p(self.seg_len, C.c_int64), _p(self.seg_off, C.c_int64),
                              kg, kx, grid_g, placement, beta1, beta2, eps, 0.0, seed)
        self.step_no = 0                  # completed steps; the next worker step is step_no + 1
        self.gcode_bytes = int(lib().qo_gcode_bytes(C.byref(self._prob)))
        self.wcode_bytes = int(lib().qo_wcode_bytes(C.byref(self._prob)))
        D = self.D
        self.x = np.zeros(D, np.float32)
        mv_shape = (self.n, D) if placement == PLACE_WORKER else (D,)
        self.m = np.zeros(mv_shape, np.float32)
        self.v = np.zeros(mv_shape, np.float32)
        self.e = np.zeros((self.n, D), np.float32)
        self.scales = np.zeros((self.n, self.S), np.float32)
        self.gcodes = np.zeros((self.n, self.gcode_bytes), np.uint8)
        self.wcodes = np.zeros(self.wcode_bytes, np.uint8)
        self.wresid = np.zeros(D, np.float32) if want_wresid else None
        # optional error buffer of the broadcast (sigma-delta form, beyond the paper): starts at zero
        self.wfeedback = np.zeros(D, np.float32) if want_wfeedback else None

    # layout helpers -------------------------------------------------------
    def to_padded(self, logical: np.ndarray) -> np.ndarray:
        """[..., d] logical -> [..., D] padded (pads zero)."""
        logical = np.asarray(logical, dtype=np.float32)
        out = np.zeros(logical.shape[:-1] + (self.D,), np.float32)
        lo = 0
        for off, ln in zip(self.seg_off.tolist(), self.seg_len.tolist()):
            out[..., off:off + ln] = logical[..., lo:lo + ln]
            lo += ln
        return out

    def to_logical(self, padded: np.ndarray) -> np.ndarray:
        out = np.zeros(padded.shape[:-1] + (self.d,), padded.dtype)
        lo = 0
        for off, ln in zip(self.seg_off.tolist(), self.seg_len.tolist()):
            out[..., lo:lo + ln] = padded[..., off:off + ln]
            lo += ln
        return out

    def set_weights(self, x_logical: np.ndarray) -> None:
        """Install x_1 and emit the first broadcast Q_x(x_1)."""
        self.x[:] = self.to_padded(x_logical)
        self.broadcast()

    def broadcast(self) -> None:
        lib().qo_broadcast_weights(C.byref(self._prob), _p(self.x, C.c_float),
                                   _p(self.wcodes, C.c_uint8) if self.kx >= 0 else None,
                                   _p(self.wresid, C.c_float), _p(self.wfeedback, C.c_float))

    # step-dependent parameters -------------------------------------------------
    def set_moment_rates(self, beta_t: float, theta_t: float) -> None:
        """beta_t, theta_t of Algorithm 1 for the steps that follow."""
        self._prob.beta, self._prob.theta = beta_t, theta_t

    def set_regularization(self, weight_decay: float) -> None:
        """lambda of the l2 term (Section 5.1) for the steps that follow."""
        self._prob.weight_decay = weight_decay

    def held_weights(self) -> np.ndarray:
        """What the workers hold during a step: the decoded broadcast, or x itself
        when the weights are not quantized."""
        return self.decoded_weights() if self.kx >= 0 else self.x

    # steps -------------------------------------------------------------------
    def worker_step(self, i: int, g_padded: np.ndarray, lr: float, xhat: np.ndarray = None) -> None:
        g = np.ascontiguousarray(g_padded, dtype=np.float32)
        assert g.shape == (self.D,)
        wm = self.placement == PLACE_WORKER
        if xhat is None and self._prob.weight_decay != 0.0:
            xhat = self.held_weights()
        rc = lib().qo_worker_step(
            C.byref(self._prob), _p(g, C.c_float), _p(xhat, C.c_float),
            _p(self.m[i], C.c_float) if wm else None,
            _p(self.v[i], C.c_float) if wm else None,
            _p(self.e[i], C.c_float), lr,
            _p(self.scales[i], C.c_float), _p(self.gcodes[i], C.c_uint8), i, self.step_no + 1)
        if rc != 0:
            raise RuntimeError(f"qo_worker_step failed: {rc}")

    def workers_step(self, g_padded: np.ndarray, lr: float, threads: int = 1) -> None:
        """All n workers.  The oracle itself is single-threaded; `threads` > 1
        only runs independent workers side by side."""
        assert g_padded.shape == (self.n, self.D)
        xhat = self.held_weights() if self._prob.weight_decay != 0.0 else None
        if threads <= 1:
            for i in range(self.n):
                self.worker_step(i, g_padded[i], lr, xhat)
        else:
            with ThreadPoolExecutor(max_workers=threads) as ex:
                list(ex.map(lambda i: self.worker_step(i, g_padded[i], lr, xhat), range(self.n)))

    def server_step(self, lr: float) -> None:
        sm = self.placement == PLACE_SERVER
        rc = lib().qo_server_step(
            C.byref(self._prob), _p(self.scales, C.c_float), _p(self.gcodes, C.c_uint8),
            _p(self.x, C.c_float),
            _p(self.m, C.c_float) if sm else None,
            _p(self.v, C.c_float) if sm else None, lr,
            _p(self.wcodes, C.c_uint8) if self.kx >= 0 else None,
            _p(self.wresid, C.c_float), _p(self.wfeedback, C.c_float))
        if rc != 0:
            raise RuntimeError(f"qo_server_step failed: {rc}")
        self.step_no += 1

    def step(self, g_padded: np.ndarray, lr: float, threads: int = 1) -> None:
        self.workers_step(g_padded, lr, threads)
        self.server_step(lr)

    def decoded_weights(self) -> np.ndarray:
        out = np.zeros(self.D, np.float32)
        rc = lib().qo_decode_weights(C.byref(self._prob), _p(self.wcodes, C.c_uint8),
                                     _p(out, C.c_float))
        if rc != 0:
            raise RuntimeError("no packed weights (kx < 0)")
        return out
