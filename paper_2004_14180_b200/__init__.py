"""Quantized Adam with error feedback: one parameter-server step on a B200.

Thin Python binding over the C interface of include/qadam.h (libqadam.so, built
from csrc/ by build.py).  Every step of the method runs in the library's CUDA
kernels; this package only marshals arguments and uses PyTorch for device
memory and streams.  There is no CPU fallback: importing the binding without
the built library, or calling it without a CUDA device, raises.
"""
from .binding import (  # noqa: F401
    PLACE_SERVER, PLACE_WORKER, GRID_POW2, GRID_UNIFORM, GRID_STOCHASTIC,
    ST_NONFINITE, ST_TIMEOUT,
    QAdamError, QAdamConfig, QAdamBuffers, QAdamOptions, QAdam,
    SERVER_AUTO, SERVER_PLAIN, WORKER_AUTO, WORKER_STREAMING, HANDOVER_AUTO, HANDOVER_COUNTERS,
    qadam_create_ex, qadam_server_step_range, qadam_finish_step, qadam_shard_cuts,
    library_path, load_library, exported_symbols,
    qadam_query_sizes, qadam_grad_code_bits, qadam_weight_code_bits,
    qadam_create, qadam_worker_compress, qadam_server_step, qadam_step_host,
    qadam_worker_scales_static, STATIC_MAX_ELEMENTS, STATIC_MAX_WORKERS,
    qadam_worker_pass_model, qadam_set_moment_rates, qadam_set_regularization,
    qadam_poll_status, qadam_profile_enable, qadam_profile_read, KERNEL_NAMES, qadam_launch_count, qadam_destroy, qadam_strerror,
)
