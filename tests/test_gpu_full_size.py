"""Parity at the full sizes of the two large workloads, in the launch configuration
the benchmark times (same context parameters, same kernels, same grids).

The oracle cannot step 2^28 x 16 elements through its server in reasonable time,
so the check is split the way the sizes allow:
  * worker side: the oracle runs EVERY worker in full (workers are independent, so
    they run side by side on the host cores); scales and packed codes of all
    workers and the error buffers of sampled workers must be bit-identical;
  * server side: the oracle steps sampled slices of the vector, fed with the
    oracle's own codes and scales, and the GPU's x, m, v and packed weights must be
    bit-identical on those slices.
Gradients are drawn once on the GPU and copied to the host for the oracle."""
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


def _server_slices(cpu, gpu, w, slices, lr):
    """Oracle server step on [lo, hi) slices (multiples of 128 inside one segment),
    from the oracle's worker outputs; compare with the GPU's result there."""
    bits_g = oracle.grad_code_bits(w.kg)
    bits_x = oracle.weight_code_bits(w.kx) if w.kx >= 0 else 0
    gx, gm, gv = gpu.x.cpu().numpy(), gpu.m.cpu().numpy(), gpu.v.cpu().numpy()
    gw = gpu.wcodes.cpu().numpy()
    for seg, lo, hi in slices:
        ln = hi - lo
        sub = oracle.OracleState([ln], cpu.n, w.kg, w.kx, cpu.placement, w.beta1, w.beta2, w.eps)
        sub.x[:] = cpu.x[lo:hi]
        if cpu.placement == oracle.PLACE_SERVER:
            sub.m[:] = cpu.m[lo:hi]
            sub.v[:] = cpu.v[lo:hi]
        sub.scales[:, 0] = cpu.scales[:, seg]
        sub.gcodes[:] = cpu.gcodes[:, lo * bits_g // 8: hi * bits_g // 8]
        sub.server_step(lr)
        assert np.array_equal(_bits(gx[lo:hi]), _bits(sub.x)), ("x", seg, lo)
        if cpu.placement == oracle.PLACE_SERVER:
            assert np.array_equal(_bits(gm[lo:hi]), _bits(sub.m)), ("m", seg, lo)
            assert np.array_equal(_bits(gv[lo:hi]), _bits(sub.v)), ("v", seg, lo)
        if w.kx >= 0:
            assert np.array_equal(gw[lo * bits_x // 8: hi * bits_x // 8], sub.wcodes), ("wcodes", seg, lo)


def _run_full(w, placement, sample_e_workers, slice_len=1 << 16, nslices=6):
    dev = torch.device("cuda")
    x1 = qi.initial_weights(w, dev)
    gpu = qb.QAdam(w.scale_seg_len, w.n, kg=w.kg, kx=w.kx, placement=placement, beta1=w.beta1,
                   beta2=w.beta2, eps=w.eps, lr=w.lr, x1=x1, device=dev)
    cpu = oracle.OracleState(w.scale_seg_len, w.n, w.kg, w.kx, placement, w.beta1, w.beta2, w.eps)
    cpu.set_weights(x1.cpu().numpy())
    del x1
    assert gpu.D == cpu.D
    g_dev = torch.zeros(w.n, gpu.D, dtype=torch.float32, device=dev)
    g_host = np.zeros((w.n, cpu.D), np.float32)
    for i in range(w.n):
        gi = qi.gradients(w, 1, i, dev)
        g_dev[i].copy_(gpu.to_padded(gi))
        g_host[i] = g_dev[i].cpu().numpy()
        del gi
    gpu.worker_compress(1, g_dev)
    cpu.workers_step(g_host, w.lr, threads=THREADS)
    torch.cuda.synchronize()
    assert np.array_equal(_bits(gpu.scales.cpu().numpy()), _bits(cpu.scales)), "scales"
    for i in range(w.n):
        assert np.array_equal(gpu.gcodes[i].cpu().numpy(), cpu.gcodes[i]), ("gcodes", i)
    for i in sample_e_workers:
        assert np.array_equal(_bits(gpu.e[i].cpu().numpy()), _bits(cpu.e[i])), ("e", i)
        if placement == qb.PLACE_WORKER:
            assert np.array_equal(_bits(gpu.m[i].cpu().numpy()), _bits(cpu.m[i])), ("m", i)
            assert np.array_equal(_bits(gpu.v[i].cpu().numpy()), _bits(cpu.v[i])), ("v", i)
    # server on sampled slices: first and last of the vector, and inside other segments
    rng = np.random.default_rng(0)
    segs = list(zip(cpu.seg_off.tolist(), cpu.seg_len.tolist()))
    picks = [0, len(segs) - 1] + rng.integers(0, len(segs), nslices).tolist()
    slices = []
    for j, s in enumerate(picks):
        off, ln = segs[s]
        plen = (ln + 127) // 128 * 128
        take = min(plen, slice_len)
        start = 0 if j == 0 else (plen - take if j == 1 else int(rng.integers(0, (plen - take) // 128 + 1)) * 128)
        slices.append((s, off + start, off + start + take))
    gpu.server_step(1)
    torch.cuda.synchronize()
    assert gpu.poll_status() == 0
    _server_slices(cpu, gpu, w, slices, w.lr)
    gpu.close()


def test_flat28_n16_server_moments_full_size():
    _run_full(qi.get_workload("flat28", n=16), qb.PLACE_SERVER, sample_e_workers=(0, 7, 15))


def test_flat28_worker_count_sweep_ends_full_size():
    # the ends of the worker-count sweep: n = 32 (server moments), n = 1 and n = 4 (worker moments)
    _run_full(qi.get_workload("flat28", n=32), qb.PLACE_SERVER, sample_e_workers=(31,))
    _run_full(qi.get_workload("flat28", n=1), qb.PLACE_WORKER, sample_e_workers=(0,))
    _run_full(qi.get_workload("flat28", n=4), qb.PLACE_WORKER, sample_e_workers=(2,))


def test_flat28_block_scales_full_size():
    # one scale per 2^20 elements: every (worker, block) pair fits on chip, so the whole
    # worker side of the 2^28-element vector goes through the on-chip kernel
    w = qi.get_workload("flat28", n=4).with_(scale_block=1 << 20)
    _run_full(w, qb.PLACE_SERVER, sample_e_workers=(1,))
    _run_full(w, qb.PLACE_WORKER, sample_e_workers=(3,))


def test_bert_base_n16_full_size_both_placements():
    w = qi.get_workload("bert_base")
    _run_full(w, qb.PLACE_SERVER, sample_e_workers=(0, 9))
    _run_full(w, qb.PLACE_WORKER, sample_e_workers=(3,))
