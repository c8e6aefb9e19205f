"""ctypes binding of include/qadam.h.

Module-level functions carry the C names and do nothing but convert arguments.
`QAdam` is a convenience holder that allocates the caller-owned device buffers
as torch tensors and keeps them alive for the lifetime of the context.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

PLACE_SERVER, PLACE_WORKER = 0, 1
GRID_POW2, GRID_UNIFORM, GRID_STOCHASTIC = 0, 1, 2
ST_NONFINITE, ST_TIMEOUT = 1, 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libqadam.so")

exported_symbols = (
    "qadam_query_sizes", "qadam_grad_code_bits", "qadam_weight_code_bits", "qadam_create",
    "qadam_worker_compress", "qadam_server_step", "qadam_step_host", "qadam_poll_status",
    "qadam_launch_count", "qadam_destroy", "qadam_strerror", "qadam_last_cuda_error",
    "qadam_profile_enable", "qadam_profile_read", "qadam_worker_scales_static",
    "qadam_worker_pass_model", "qadam_set_moment_rates", "qadam_set_regularization",
    "qadam_create_ex", "qadam_server_step_range", "qadam_finish_step", "qadam_shard_cuts",
)

SERVER_AUTO, SERVER_PLAIN = 0, 1
WORKER_AUTO, WORKER_STREAMING = 0, 1
HANDOVER_AUTO, HANDOVER_COUNTERS = 0, 1

STATIC_MAX_ELEMENTS = 1 << 26
STATIC_MAX_WORKERS = 1024

KERNEL_NAMES = ("absmax", "quantize", "identity", "server", "broadcast", "worker_fused")


class QAdamError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = qadam_strerror(code)
        if code == -9:
            msg += f" (cudaError {load_library().qadam_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{code}]")


class QAdamConfig(C.Structure):
    _fields_ = [
        ("d", C.c_int64), ("n", C.c_int32), ("num_segments", C.c_int32),
        ("seg_len", C.POINTER(C.c_int64)),
        ("kg", C.c_int32), ("kx", C.c_int32), ("grid_g", C.c_int32), ("placement", C.c_int32),
        ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float), ("lr", C.c_float),
        ("stream", C.c_void_p), ("seed", C.c_uint64),
    ]


class QAdamOptions(C.Structure):
    _fields_ = [
        ("server_kernel", C.c_int32), ("worker_kernel", C.c_int32), ("hand_over", C.c_int32),
        ("wait_polls", C.c_uint32), ("test_missing_tiles", C.c_int32), ("reserved", C.c_int32 * 3),
    ]


class QAdamBuffers(C.Structure):
    _fields_ = [
        ("x", C.c_void_p), ("m", C.c_void_p), ("v", C.c_void_p), ("e", C.c_void_p),
        ("scales", C.c_void_p), ("gcodes", C.c_void_p), ("wcodes", C.c_void_p),
        ("wresid", C.c_void_p), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
        ("status", C.c_void_p), ("wfeedback", C.c_void_p),
    ]


_lib = None


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Loads libqadam.so.  Raises if it has not been built: there is no fallback."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2004_14180_b200.build` "
            "(nvcc, sm_100a).  This package has no other implementation.")
    L = C.CDLL(_LIB_PATH)
    cfgp, bufp = C.POINTER(QAdamConfig), C.POINTER(QAdamBuffers)
    L.qadam_query_sizes.restype = C.c_int
    L.qadam_query_sizes.argtypes = [cfgp, C.POINTER(C.c_int64), C.POINTER(C.c_int64),
                                    C.POINTER(C.c_size_t), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    L.qadam_grad_code_bits.restype = C.c_int
    L.qadam_grad_code_bits.argtypes = [C.c_int32, C.c_int32]
    L.qadam_weight_code_bits.restype = C.c_int
    L.qadam_weight_code_bits.argtypes = [C.c_int32]
    L.qadam_create.restype = C.c_int
    L.qadam_create.argtypes = [cfgp, bufp, C.POINTER(C.c_void_p)]
    L.qadam_create_ex.restype = C.c_int
    L.qadam_create_ex.argtypes = [cfgp, bufp, C.POINTER(QAdamOptions), C.POINTER(C.c_void_p)]
    L.qadam_server_step_range.restype = C.c_int
    L.qadam_server_step_range.argtypes = [C.c_void_p, C.c_int64, C.c_float, C.c_int64, C.c_int64]
    L.qadam_finish_step.restype = C.c_int
    L.qadam_finish_step.argtypes = [C.c_void_p, C.c_int64]
    L.qadam_shard_cuts.restype = C.c_int
    L.qadam_shard_cuts.argtypes = [cfgp, C.c_int32, C.POINTER(C.c_int64)]
    L.qadam_worker_compress.restype = C.c_int
    L.qadam_worker_compress.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_int32, C.c_int32, C.c_float]
    L.qadam_server_step.restype = C.c_int
    L.qadam_server_step.argtypes = [C.c_void_p, C.c_int64, C.c_float]
    L.qadam_step_host.restype = C.c_int
    L.qadam_step_host.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_float]
    L.qadam_poll_status.restype = C.c_int
    L.qadam_poll_status.argtypes = [C.c_void_p, C.POINTER(C.c_uint32)]
    L.qadam_profile_enable.restype = C.c_int
    L.qadam_profile_enable.argtypes = [C.c_void_p, C.c_int]
    L.qadam_profile_read.restype = C.c_int
    L.qadam_profile_read.argtypes = [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_int64)]
    L.qadam_worker_scales_static.restype = C.c_int
    L.qadam_worker_scales_static.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int32, C.c_void_p, C.c_void_p]
    L.qadam_worker_pass_model.restype = C.c_int
    L.qadam_worker_pass_model.argtypes = [C.c_void_p, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
    L.qadam_set_moment_rates.restype = C.c_int
    L.qadam_set_moment_rates.argtypes = [C.c_void_p, C.c_float, C.c_float]
    L.qadam_set_regularization.restype = C.c_int
    L.qadam_set_regularization.argtypes = [C.c_void_p, C.c_float]
    L.qadam_launch_count.restype = C.c_int64
    L.qadam_launch_count.argtypes = [C.c_void_p]
    L.qadam_destroy.restype = C.c_int
    L.qadam_destroy.argtypes = [C.c_void_p]
    L.qadam_strerror.restype = C.c_char_p
    L.qadam_strerror.argtypes = [C.c_int]
    L.qadam_last_cuda_error.restype = C.c_int
    L.qadam_last_cuda_error.argtypes = []
    _lib = L
    return L


def _check(rc: int, where: str) -> None:
    if rc != 0:
        raise QAdamError(rc, where)


# ---------------------------------------------------------------- the C calls

def qadam_strerror(code: int) -> str:
    return load_library().qadam_strerror(code).decode()


def qadam_grad_code_bits(kg: int, grid_g: int = GRID_POW2) -> int:
    return int(load_library().qadam_grad_code_bits(kg, grid_g))


def qadam_weight_code_bits(kx: int) -> int:
    return int(load_library().qadam_weight_code_bits(kx))


def qadam_query_sizes(cfg: QAdamConfig):
    """-> dict(D, seg_off, gcode_bytes, wcode_bytes, workspace_bytes)"""
    D = C.c_int64()
    S = max(1, int(cfg.num_segments))
    seg_off = (C.c_int64 * S)()
    gb, wb, ws = C.c_size_t(), C.c_size_t(), C.c_size_t()
    _check(load_library().qadam_query_sizes(C.byref(cfg), C.byref(D), seg_off, C.byref(gb),
                                            C.byref(wb), C.byref(ws)), "qadam_query_sizes")
    return dict(D=D.value, seg_off=list(seg_off), gcode_bytes=gb.value, wcode_bytes=wb.value,
                workspace_bytes=ws.value)


def qadam_create(cfg: QAdamConfig, bufs: QAdamBuffers) -> int:
    ctx = C.c_void_p()
    _check(load_library().qadam_create(C.byref(cfg), C.byref(bufs), C.byref(ctx)), "qadam_create")
    return ctx.value


def qadam_create_ex(cfg: QAdamConfig, bufs: QAdamBuffers, opt: Optional[QAdamOptions]) -> int:
    ctx = C.c_void_p()
    _check(load_library().qadam_create_ex(C.byref(cfg), C.byref(bufs),
                                          C.byref(opt) if opt is not None else None, C.byref(ctx)),
           "qadam_create_ex")
    return ctx.value


def qadam_server_step_range(ctx: int, step: int, lr_t: float, elem_begin: int, elem_end: int) -> None:
    _check(load_library().qadam_server_step_range(ctx, step, lr_t, elem_begin, elem_end),
           "qadam_server_step_range")


def qadam_finish_step(ctx: int, step: int) -> None:
    _check(load_library().qadam_finish_step(ctx, step), "qadam_finish_step")


def qadam_shard_cuts(cfg: QAdamConfig, shards: int):
    """-> shards + 1 element offsets, the ranges a sharded server may be cut into (host only)."""
    cuts = (C.c_int64 * (max(0, shards) + 1))()
    _check(load_library().qadam_shard_cuts(C.byref(cfg), shards, cuts), "qadam_shard_cuts")
    return list(cuts)


def qadam_worker_compress(ctx: int, step: int, g_ptr: int, worker_begin: int, worker_count: int,
                          lr_t: float = -1.0) -> None:
    _check(load_library().qadam_worker_compress(ctx, step, g_ptr, worker_begin, worker_count, lr_t),
           "qadam_worker_compress")


def qadam_server_step(ctx: int, step: int, lr_t: float = -1.0) -> None:
    _check(load_library().qadam_server_step(ctx, step, lr_t), "qadam_server_step")


def qadam_step_host(ctx: int, step: int, g_host_ptr: int, g_stage_ptr: int, out_host_ptr: Optional[int],
                    lr_t: float = -1.0) -> None:
    _check(load_library().qadam_step_host(ctx, step, g_host_ptr, g_stage_ptr, out_host_ptr, lr_t),
           "qadam_step_host")


def qadam_poll_status(ctx: int) -> int:
    st = C.c_uint32()
    _check(load_library().qadam_poll_status(ctx, C.byref(st)), "qadam_poll_status")
    return st.value


def qadam_set_moment_rates(ctx: int, beta_t: float, theta_t: float) -> None:
    _check(load_library().qadam_set_moment_rates(ctx, beta_t, theta_t), "qadam_set_moment_rates")


def qadam_set_regularization(ctx: int, weight_decay: float) -> None:
    _check(load_library().qadam_set_regularization(ctx, weight_decay), "qadam_set_regularization")


def qadam_profile_enable(ctx: int, enable: bool) -> None:
    _check(load_library().qadam_profile_enable(ctx, int(bool(enable))), "qadam_profile_enable")


def qadam_profile_read(ctx: int):
    """-> {kernel name: (total ms, launches)} since the last read."""
    n = len(KERNEL_NAMES)
    ms, cnt = (C.c_double * n)(), (C.c_int64 * n)()
    _check(load_library().qadam_profile_read(ctx, ms, cnt), "qadam_profile_read")
    return {KERNEL_NAMES[i]: (ms[i], cnt[i]) for i in range(n)}


def qadam_worker_scales_static(g_ptr: int, e_ptr: int, D: int, n: int, scales_ptr: int,
                               stream_ptr: Optional[int] = None) -> None:
    """Max-abs scales of n workers without a context, a workspace or any allocation
    (for callers that cannot allocate device memory); see include/qadam.h."""
    _check(load_library().qadam_worker_scales_static(g_ptr, e_ptr, D, n, scales_ptr, stream_ptr),
           "qadam_worker_scales_static")


def qadam_worker_pass_model(ctx: int):
    """-> (one_pass, two_pass): (worker, element) pairs read from HBM once / twice by the worker side."""
    a, b = C.c_int64(), C.c_int64()
    _check(load_library().qadam_worker_pass_model(ctx, C.byref(a), C.byref(b)), "qadam_worker_pass_model")
    return a.value, b.value


def qadam_launch_count(ctx: int) -> int:
    return int(load_library().qadam_launch_count(ctx))


def qadam_destroy(ctx: int) -> None:
    _check(load_library().qadam_destroy(ctx), "qadam_destroy")


# ---------------------------------------------------------------- convenience holder

class QAdam:
    """Owns the device buffers of one problem (as torch tensors) and its context.

    seg_len: logical tensor lengths (one max-abs scale per tensor and worker).
    x1: logical initial weights [d] (any device), or None for zeros.
    """

    def __init__(self, seg_len: Sequence[int], n: int, kg: int = 0, kx: int = -1,
                 placement: int = PLACE_SERVER, beta1: float = 0.9, beta2: float = 0.999,
                 eps: float = 1e-8, lr: float = 1e-3, grid_g: int = GRID_POW2,
                 x1: Optional[torch.Tensor] = None, want_wresid: bool = False,
                 device: Optional[torch.device] = None, stream: Optional[torch.cuda.Stream] = None,
                 seed: int = 0, options: Optional[QAdamOptions] = None, want_wfeedback: bool = False):
        load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2004_14180_b200 needs a CUDA device; there is no CPU path")
        self.device = torch.device(device if device is not None else f"cuda:{torch.cuda.current_device()}")
        self.stream = stream
        self.seg_len = [int(s) for s in seg_len]
        self.n, self.kg, self.kx, self.placement, self.grid_g = int(n), kg, kx, placement, grid_g
        self._seg_arr = (C.c_int64 * len(self.seg_len))(*self.seg_len)
        self.cfg = QAdamConfig(
            d=sum(self.seg_len), n=self.n, num_segments=len(self.seg_len), seg_len=self._seg_arr,
            kg=kg, kx=kx, grid_g=grid_g, placement=placement, beta1=beta1, beta2=beta2, eps=eps,
            lr=lr, stream=(stream.cuda_stream if stream is not None else
                           torch.cuda.current_stream(self.device).cuda_stream), seed=seed)
        sz = qadam_query_sizes(self.cfg)
        self.d, self.D, self.S = sum(self.seg_len), sz["D"], len(self.seg_len)
        self.seg_off = sz["seg_off"]
        self.gcode_bytes, self.wcode_bytes = sz["gcode_bytes"], sz["wcode_bytes"]
        with torch.cuda.device(self.device):
            z = lambda *shape, dtype=torch.float32: torch.zeros(*shape, dtype=dtype, device=self.device)
            D = self.D
            self.x = z(D)
            mv_shape = (self.n, D) if placement == PLACE_WORKER else (D,)
            self.m, self.v = z(*mv_shape), z(*mv_shape)
            self.e = z(self.n, D)
            self.scales = z(self.n, self.S)
            self.gcodes = z(self.n, self.gcode_bytes, dtype=torch.uint8)
            self.wcodes = z(max(self.wcode_bytes, 16), dtype=torch.uint8)
            self.wresid = z(D) if want_wresid else None
            self.wfeedback = z(D) if want_wfeedback else None      # error buffer of the broadcast (optional)
            self.workspace = z(sz["workspace_bytes"] + 256, dtype=torch.uint8)
            self.status = z(4, dtype=torch.int32)
            if x1 is not None:
                self.x.copy_(self.to_padded(x1.to(self.device, torch.float32)))
            ws_ptr = (self.workspace.data_ptr() + 255) // 256 * 256
            self.bufs = QAdamBuffers(
                x=self.x.data_ptr(), m=self.m.data_ptr(), v=self.v.data_ptr(), e=self.e.data_ptr(),
                scales=self.scales.data_ptr(), gcodes=self.gcodes.data_ptr(),
                wcodes=self.wcodes.data_ptr() if kx >= 0 else None,
                wresid=self.wresid.data_ptr() if want_wresid else None,
                workspace=ws_ptr, workspace_bytes=sz["workspace_bytes"],
                status=self.status.data_ptr(),
                wfeedback=self.wfeedback.data_ptr() if want_wfeedback else None)
            # buffers were filled on torch's current stream; the context may use another
            torch.cuda.current_stream(self.device).synchronize()
            self.ctx = (qadam_create(self.cfg, self.bufs) if options is None
                        else qadam_create_ex(self.cfg, self.bufs, options))

    # layout -------------------------------------------------------------------
    def to_padded(self, logical: torch.Tensor) -> torch.Tensor:
        """[..., d] logical -> [..., D] padded layout (pads zero)."""
        if self.D == self.d:
            return logical
        out = torch.zeros(logical.shape[:-1] + (self.D,), dtype=logical.dtype, device=logical.device)
        lo = 0
        for off, ln in zip(self.seg_off, self.seg_len):
            out[..., off:off + ln] = logical[..., lo:lo + ln]
            lo += ln
        return out

    def to_logical(self, padded: torch.Tensor) -> torch.Tensor:
        if self.D == self.d:
            return padded
        out = torch.empty(padded.shape[:-1] + (self.d,), dtype=padded.dtype, device=padded.device)
        lo = 0
        for off, ln in zip(self.seg_off, self.seg_len):
            out[..., lo:lo + ln] = padded[..., off:off + ln]
            lo += ln
        return out

    # steps --------------------------------------------------------------------
    def worker_compress(self, step: int, g: torch.Tensor, worker_begin: int = 0,
                        worker_count: Optional[int] = None, lr: float = -1.0) -> None:
        """g: [worker_count][D] fp32 on the device, padded layout."""
        wc = self.n - worker_begin if worker_count is None else worker_count
        assert g.is_cuda and g.dtype == torch.float32 and g.is_contiguous()
        assert g.numel() == wc * self.D, "g must be [worker_count][D] in the padded layout"
        qadam_worker_compress(self.ctx, step, g.data_ptr(), worker_begin, wc, lr)

    def server_step(self, step: int, lr: float = -1.0) -> None:
        qadam_server_step(self.ctx, step, lr)

    def server_step_range(self, step: int, elem_begin: int, elem_end: int, lr: float = -1.0) -> None:
        qadam_server_step_range(self.ctx, step, lr, elem_begin, elem_end)

    def finish_step(self, step: int) -> None:
        qadam_finish_step(self.ctx, step)

    def shard_cuts(self, shards: int):
        return qadam_shard_cuts(self.cfg, shards)

    def step(self, step: int, g: torch.Tensor, lr: float = -1.0) -> None:
        self.worker_compress(step, g, 0, self.n, lr)
        self.server_step(step, lr)

    def step_host(self, step: int, g_host: torch.Tensor, g_stage: torch.Tensor,
                  out_host: Optional[torch.Tensor], lr: float = -1.0) -> None:
        assert not g_host.is_cuda and g_host.is_contiguous() and g_host.numel() == self.n * self.D
        assert g_stage.is_cuda and g_stage.numel() == self.n * self.D
        qadam_step_host(self.ctx, step, g_host.data_ptr(), g_stage.data_ptr(),
                        out_host.data_ptr() if out_host is not None else None, lr)

    def profile(self, enable: bool) -> None:
        qadam_profile_enable(self.ctx, enable)

    def profile_read(self):
        return qadam_profile_read(self.ctx)

    def worker_pass_model(self):
        return qadam_worker_pass_model(self.ctx)

    def poll_status(self) -> int:
        return qadam_poll_status(self.ctx)

    def set_moment_rates(self, beta_t: float, theta_t: float) -> None:
        """beta_t, theta_t of Algorithm 1 for the steps that follow."""
        qadam_set_moment_rates(self.ctx, beta_t, theta_t)

    def set_regularization(self, weight_decay: float) -> None:
        """lambda of the l2 term (Section 5.1) for the steps that follow; 0 switches it off."""
        qadam_set_regularization(self.ctx, weight_decay)

    @property
    def launches(self) -> int:
        return qadam_launch_count(self.ctx)

    def sent_bytes_per_step(self) -> int:
        """What the n workers send per step: codes plus one fp32 scale per segment."""
        return self.n * (self.gcode_bytes + 4 * self.S)

    def compression_ratio(self) -> float:
        return 4.0 * self.d * self.n / self.sent_bytes_per_step()

    def close(self) -> None:
        if getattr(self, "ctx", None):
            qadam_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
