"""Parity at the full sizes of the two large workloads, over several steps, in the launch
configuration the benchmark times (same context parameters, same kernels, same grids).

The oracle cannot step 2^28 x 16 elements through its server in reasonable time, so the
check is split the way the sizes allow:
  * worker side: the oracle runs EVERY worker in full, step after step (workers are
    independent and, without the l2 term, need nothing from the server, so they run side by
    side on the host cores); scales and packed codes of all workers are compared after every
    step, the error buffers (and worker moments) of sampled workers after every step and of
    all workers after the last one;
  * server side: the oracle carries 64 slices of the vector as problems of their own across
    the steps, fed with the ORACLE's codes and scales of that step; the GPU's x, m, v and
    packed weights must be bit-identical on those slices after every step.
From step 2 on the error-feedback add and the moment recursions see non-zero state.
Gradients are drawn on the GPU, one batch per step, and copied to the host for the oracle.

Streams beyond 2^31 and 2^32 bytes: the worker-side arrays g, e (m, v) are [n][D] and cross
those offsets at worker boundaries; the sampled workers sit on both sides of each.  x, m, v
of the server and each worker's code stream stay below 2^31 bytes at these sizes."""
import os

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import oracle  # noqa: E402
import paper_2004_14180_b200 as qb  # noqa: E402
import qadam_inputs as qi  # noqa: E402

THREADS = max(1, min(16, os.cpu_count() or 1))


def _bits(a):
    return np.ascontiguousarray(a).view(np.uint32)


def _pick_slices(cpu, count, slice_len):
    """`count` slices [lo, hi) spread over the vector, each inside one segment's padded run
    (multiples of 128): the first and the last elements of the vector and evenly spaced
    positions in between."""
    seg_off = cpu.seg_off.tolist()
    seg_plen = [(ln + 127) // 128 * 128 for ln in cpu.seg_len.tolist()]
    out = []
    for k in range(count):
        pos = min(cpu.D - 128, (cpu.D * k // (count - 1)) // 128 * 128)
        s = int(np.searchsorted(cpu.seg_off, pos, side="right")) - 1
        take = min(seg_plen[s], slice_len)
        lo = min(max(pos, seg_off[s]), seg_off[s] + seg_plen[s] - take)
        out.append((s, lo, lo + take))
    return out


class _SliceOracle:
    """One slice of the vector carried by the oracle as a single-segment problem."""

    def __init__(self, cpu, w, seg, lo, hi):
        self.seg, self.lo, self.hi = seg, lo, hi
        self.bits_g = oracle.grad_code_bits(w.kg)
        self.bits_x = oracle.weight_code_bits(w.kx) if w.kx >= 0 else 0
        self.sub = oracle.OracleState([hi - lo], cpu.n, w.kg, w.kx, cpu.placement, w.beta1, w.beta2, w.eps)
        self.sub.x[:] = cpu.x[lo:hi]

    def step_and_compare(self, cpu, gpu, lr, tag):
        sub, lo, hi = self.sub, self.lo, self.hi
        sub.scales[:, 0] = cpu.scales[:, self.seg]
        sub.gcodes[:] = cpu.gcodes[:, lo * self.bits_g // 8: hi * self.bits_g // 8]
        sub.server_step(lr)
        assert np.array_equal(_bits(gpu.x[lo:hi].cpu().numpy()), _bits(sub.x)), ("x", tag, lo)
        if cpu.placement == oracle.PLACE_SERVER:
            assert np.array_equal(_bits(gpu.m[lo:hi].cpu().numpy()), _bits(sub.m)), ("m", tag, lo)
            assert np.array_equal(_bits(gpu.v[lo:hi].cpu().numpy()), _bits(sub.v)), ("v", tag, lo)
        if self.bits_x:
            got = gpu.wcodes[lo * self.bits_x // 8: hi * self.bits_x // 8].cpu().numpy()
            assert np.array_equal(got, sub.wcodes), ("wcodes", tag, lo)


def _compare_worker(gpu, cpu, i, placement, tag):
    assert np.array_equal(_bits(gpu.e[i].cpu().numpy()), _bits(cpu.e[i])), ("e", i, tag)
    if placement == qb.PLACE_WORKER:
        assert np.array_equal(_bits(gpu.m[i].cpu().numpy()), _bits(cpu.m[i])), ("m", i, tag)
        assert np.array_equal(_bits(gpu.v[i].cpu().numpy()), _bits(cpu.v[i])), ("v", i, tag)


def _run_full(w, placement, steps, sample_workers, nslices=64, slice_len=1 << 14):
    dev = torch.device("cuda")
    x1 = qi.initial_weights(w, dev)
    gpu = qb.QAdam(w.scale_seg_len, w.n, kg=w.kg, kx=w.kx, placement=placement, beta1=w.beta1,
                   beta2=w.beta2, eps=w.eps, lr=w.lr, x1=x1, device=dev)
    cpu = oracle.OracleState(w.scale_seg_len, w.n, w.kg, w.kx, placement, w.beta1, w.beta2, w.eps)
    cpu.set_weights(x1.cpu().numpy())
    del x1
    assert gpu.D == cpu.D
    slices = [_SliceOracle(cpu, w, *s) for s in _pick_slices(cpu, nslices, slice_len)]
    g_dev = torch.zeros(w.n, gpu.D, dtype=torch.float32, device=dev)
    g_host = np.zeros((w.n, cpu.D), np.float32)
    for t in range(1, steps + 1):
        for i in range(w.n):
            gi = qi.gradients(w, t, i, dev)
            g_dev[i].copy_(gpu.to_padded(gi))
            g_host[i] = g_dev[i].cpu().numpy()
            del gi
        gpu.worker_compress(t, g_dev)
        cpu.workers_step(g_host, w.lr, threads=THREADS)
        torch.cuda.synchronize()
        assert np.array_equal(_bits(gpu.scales.cpu().numpy()), _bits(cpu.scales)), ("scales", t)
        for i in range(w.n):
            assert np.array_equal(gpu.gcodes[i].cpu().numpy(), cpu.gcodes[i]), ("gcodes", i, t)
        for i in (range(w.n) if t == steps else sample_workers):
            _compare_worker(gpu, cpu, i, placement, t)
        gpu.server_step(t)
        torch.cuda.synchronize()
        assert gpu.poll_status() == 0
        for s in slices:
            s.step_and_compare(cpu, gpu, w.lr, t)
    gpu.close()


def test_flat28_n16_server_moments_full_size():
    # worker rows of 1 GiB: rows 1|2 meet at 2^31 bytes of g and e, rows 3|4 at 2^32
    _run_full(qi.get_workload("flat28", n=16), qb.PLACE_SERVER, steps=3, sample_workers=(0, 1, 2, 3, 4, 15))


def test_flat28_n4_worker_moments_full_size():
    _run_full(qi.get_workload("flat28", n=4), qb.PLACE_WORKER, steps=3, sample_workers=(1, 2, 3))


def test_flat28_worker_count_sweep_ends_full_size():
    # the ends of the worker-count sweep: n = 32 (moments on the server), n = 1 (on the worker)
    _run_full(qi.get_workload("flat28", n=32), qb.PLACE_SERVER, steps=2, sample_workers=(3, 4, 31))
    _run_full(qi.get_workload("flat28", n=1), qb.PLACE_WORKER, steps=2, sample_workers=(0,))


def test_flat28_block_scales_full_size():
    # one scale per 2^20 elements: every (worker, block) pair fits on chip, so the whole
    # worker side of the 2^28-element vector goes through the on-chip kernel
    w = qi.get_workload("flat28", n=4).with_(scale_block=1 << 20)
    _run_full(w, qb.PLACE_SERVER, steps=2, sample_workers=(1, 2))
    _run_full(w, qb.PLACE_WORKER, steps=2, sample_workers=(3,))


def test_bert_base_n16_full_size_both_placements():
    # worker rows of 0.44 GB: row 4 straddles 2^31 bytes of g and e, row 9 straddles 2^32
    w = qi.get_workload("bert_base")
    _run_full(w, qb.PLACE_SERVER, steps=3, sample_workers=(0, 4, 5, 9, 10))
    _run_full(w, qb.PLACE_WORKER, steps=3, sample_workers=(4, 9))
