"""Host-side checks of the C interface that need no GPU: the library loads, it
exports every function the header declares, and argument validation that happens
before any CUDA call returns the documented error codes."""
import ctypes as C
import os
import re

import pytest

import paper_2004_14180_b200 as qb
from paper_2004_14180_b200 import build as qbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    qbuild.build()
    return qb.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "qadam.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qadam_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_function(lib):
    names = _declared_functions()
    assert "qadam_create" in names and "qadam_worker_compress" in names
    assert "qadam_server_step" in names and "qadam_destroy" in names
    for name in names:
        assert hasattr(lib, name), f"{name} declared in qadam.h but not exported"
    assert sorted(qb.exported_symbols) == names


def _cfg(**kw):
    base = dict(d=1000, n=2, num_segments=1, seg_len=None, kg=0, kx=0, grid_g=0, placement=0,
                beta1=0.9, beta2=0.999, eps=1e-8, lr=1e-3, stream=None, seed=0)
    base.update(kw)
    return qb.QAdamConfig(**base)


def test_query_sizes_layout_and_bytes(lib):
    seg = (C.c_int64 * 4)(64, 129, 4096, 1)
    sz = qb.qadam_query_sizes(_cfg(d=64 + 129 + 4096 + 1, num_segments=4, seg_len=seg, kg=1, kx=6))
    assert sz["seg_off"] == [0, 128, 384, 384 + 4096]
    assert sz["D"] == 384 + 4096 + 128
    assert sz["gcode_bytes"] == sz["D"] * 3 // 8
    assert sz["wcode_bytes"] == sz["D"]
    assert sz["workspace_bytes"] % 256 == 0 and sz["workspace_bytes"] > 0
    ident = qb.qadam_query_sizes(_cfg(kg=-1, kx=-1))
    assert ident["gcode_bytes"] == 4 * ident["D"] and ident["wcode_bytes"] == 0


def test_code_widths(lib):
    assert qb.qadam_grad_code_bits(0) == 2 and qb.qadam_grad_code_bits(1) == 3
    assert qb.qadam_grad_code_bits(2, qb.GRID_POW2) == 3        # 7 levels
    assert qb.qadam_grad_code_bits(2, qb.GRID_UNIFORM) == 4     # 9 levels
    assert qb.qadam_grad_code_bits(6, qb.GRID_UNIFORM) == 8     # 129 levels
    assert qb.qadam_grad_code_bits(-1) == 32
    assert qb.qadam_grad_code_bits(7, qb.GRID_UNIFORM) < 0
    assert qb.qadam_weight_code_bits(6) == 8 and qb.qadam_weight_code_bits(14) == 16
    assert qb.qadam_weight_code_bits(-1) == 0 and qb.qadam_weight_code_bits(15) < 0


@pytest.mark.parametrize("kw,code", [
    (dict(d=0), -2), (dict(n=0), -2), (dict(num_segments=0), -2),
    (dict(num_segments=3), -1),                      # seg_len NULL with S > 1
    (dict(kg=-2), -3), (dict(kg=15), -3), (dict(kg=7, grid_g=1), -3), (dict(grid_g=3), -3),
    (dict(kg=1, grid_g=2), -3), (dict(kg=-1, grid_g=2), -3),      # the stochastic operator is ternary only
    (dict(kx=15), -3), (dict(kx=-2), -3),
    (dict(placement=2), -10),
    (dict(beta1=1.0), -8), (dict(beta2=-0.1), -8), (dict(eps=0.0), -8), (dict(lr=float("nan")), -8),
])
def test_invalid_configurations_are_rejected(lib, kw, code):
    with pytest.raises(qb.QAdamError) as ei:
        qb.qadam_query_sizes(_cfg(**kw))
    assert ei.value.code == code


def test_segment_lengths_must_sum_to_d(lib):
    seg = (C.c_int64 * 2)(10, 20)
    with pytest.raises(qb.QAdamError) as ei:
        qb.qadam_query_sizes(_cfg(d=31, num_segments=2, seg_len=seg))
    assert ei.value.code == -2
    seg = (C.c_int64 * 2)(31, 0)
    with pytest.raises(qb.QAdamError):
        qb.qadam_query_sizes(_cfg(d=31, num_segments=2, seg_len=seg))


def test_null_arguments(lib):
    assert lib.qadam_create(None, None, None) == -1
    assert lib.qadam_worker_compress(None, 1, None, 0, 1, C.c_float(0.1)) == -1
    assert lib.qadam_server_step(None, 1, C.c_float(0.1)) == -1
    assert lib.qadam_destroy(None) == -1
    assert qb.qadam_strerror(-6) == "step out of order"


def test_options_are_checked_before_anything_else_happens(lib):
    # unknown enumerators, a negative test hook and non-zero reserved fields: QADAM_ERR_SIZE,
    # decided on the host before any CUDA call (so this runs without a GPU)
    cfg, bufs, ctx = _cfg(), qb.QAdamBuffers(), C.c_void_p()
    bad = [qb.QAdamOptions(server_kernel=2), qb.QAdamOptions(worker_kernel=5), qb.QAdamOptions(hand_over=-1),
           qb.QAdamOptions(test_missing_tiles=-3)]
    r = qb.QAdamOptions()
    r.reserved[1] = 1
    bad.append(r)
    for opt in bad:
        assert lib.qadam_create_ex(C.byref(cfg), C.byref(bufs), C.byref(opt), C.byref(ctx)) == -2
        assert not ctx.value
    assert lib.qadam_create_ex(None, C.byref(bufs), None, C.byref(ctx)) == -1
    # valid options, missing buffers: the next check in line answers
    assert lib.qadam_create_ex(C.byref(cfg), C.byref(bufs), C.byref(qb.QAdamOptions()), C.byref(ctx)) == -1


def test_range_and_shard_calls_reject_bad_arguments(lib):
    assert lib.qadam_server_step_range(None, 1, C.c_float(0.1), 0, 128) == -1
    assert lib.qadam_finish_step(None, 1) == -1
    cuts = (C.c_int64 * 3)()
    assert lib.qadam_shard_cuts(None, 2, cuts) == -1
    assert lib.qadam_shard_cuts(C.byref(_cfg()), 0, cuts) == -2
    assert lib.qadam_shard_cuts(C.byref(_cfg(d=0)), 2, cuts) == -2
    assert lib.qadam_shard_cuts(C.byref(_cfg(d=10000)), 2, cuts) == 0
    assert list(cuts) == [0, 8192, 10112]          # tiles of 4096; D = 10000 padded to 10112


def test_stochastic_operator_sizes(lib):
    sz = qb.qadam_query_sizes(_cfg(grid_g=qb.GRID_STOCHASTIC))
    assert sz["gcode_bytes"] == sz["D"] // 4       # ternary codes
    assert qb.qadam_grad_code_bits(0, qb.GRID_STOCHASTIC) == 2
    assert qb.qadam_grad_code_bits(1, qb.GRID_STOCHASTIC) < 0


def test_layout_agrees_with_the_oracle(lib, oracle):
    # two independent implementations of the padded layout must agree
    lens = [64, 129, 4096, 1, 1000, 128, 127]
    seg = (C.c_int64 * len(lens))(*lens)
    sz = qb.qadam_query_sizes(_cfg(d=sum(lens), num_segments=len(lens), seg_len=seg))
    off, D = oracle.layout(lens)
    assert sz["seg_off"] == off.tolist() and sz["D"] == D


def test_no_cpu_fallback_without_cuda():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError):
        qb.QAdam([100], 2)
