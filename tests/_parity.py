"""Runs the CUDA library and the CPU oracle side by side on the same inputs and
compares everything they produce.  Used by the GPU parity tests only."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2004_14180_b200 as qb

REL_TOL = 1e-5      # the stated bound on fp32 state (max relative error, see rel_err)


def rel_err(a: np.ndarray, b: np.ndarray) -> float:
    """max_j |a_j - b_j| / max(|b_j|, 1e-3 * |b|_inf): relative error that stays
    meaningful for buffers holding exact zeros (e is 0 at each segment's arg-max)."""
    a = a.astype(np.float64).ravel()
    b = b.astype(np.float64).ravel()
    if a.size == 0:
        return 0.0
    floor = 1e-3 * np.max(np.abs(b)) if np.max(np.abs(b)) > 0 else 1.0
    return float(np.max(np.abs(a - b) / np.maximum(np.abs(b), floor)))


def bits_equal(a: np.ndarray, b: np.ndarray) -> bool:
    return np.array_equal(np.ascontiguousarray(a).view(np.uint32), np.ascontiguousarray(b).view(np.uint32))


class Pair:
    """One problem held twice: `gpu` (qb.QAdam) and `cpu` (oracle.OracleState)."""

    def __init__(self, seg_len, n, kg, kx, placement, x1=None, grid_g=0, beta1=0.9, beta2=0.999,
                 eps=1e-8, lr=1e-3, want_wresid=False, options=None, seed=0, want_wfeedback=False):
        self.lr = lr
        x1_t = None if x1 is None else torch.as_tensor(x1, dtype=torch.float32)
        self.gpu = qb.QAdam(seg_len, n, kg=kg, kx=kx, placement=placement, beta1=beta1, beta2=beta2,
                            eps=eps, lr=lr, grid_g=grid_g, x1=x1_t, want_wresid=want_wresid,
                            options=options, seed=seed, want_wfeedback=want_wfeedback)
        self.cpu = oracle.OracleState(seg_len, n, kg, kx, placement, beta1, beta2, eps,
                                      grid_g=grid_g, want_wresid=want_wresid, seed=seed,
                                      want_wfeedback=want_wfeedback)
        if x1 is not None:
            self.cpu.set_weights(np.asarray(x1, dtype=np.float32))
        else:
            self.cpu.broadcast()
        assert self.gpu.D == self.cpu.D and list(self.gpu.seg_off) == self.cpu.seg_off.tolist()
        assert self.gpu.gcode_bytes == self.cpu.gcode_bytes
        assert self.gpu.wcode_bytes == self.cpu.wcode_bytes
        self.step_no = 0

    def step(self, g_logical: np.ndarray, lr=None, threads: int = 1, split_workers: bool = False):
        """g_logical: [n][d] float32.  Runs one full step on both sides."""
        lr = self.lr if lr is None else lr
        self.step_no += 1
        gp = self.cpu.to_padded(g_logical)
        g_dev = torch.from_numpy(gp).to(self.gpu.device)
        if split_workers and self.gpu.n > 1:
            h = self.gpu.n // 2
            self.gpu.worker_compress(self.step_no, g_dev[h:].contiguous(), h, self.gpu.n - h, lr)
            self.gpu.worker_compress(self.step_no, g_dev[:h].contiguous(), 0, h, lr)
        else:
            self.gpu.worker_compress(self.step_no, g_dev, 0, self.gpu.n, lr)
        self.cpu.workers_step(gp, lr, threads)
        self.compare_worker_outputs()
        self.gpu.server_step(self.step_no, lr)
        self.cpu.server_step(lr)

    def set_moment_rates(self, beta_t: float, theta_t: float):
        self.gpu.set_moment_rates(beta_t, theta_t)
        self.cpu.set_moment_rates(beta_t, theta_t)

    def set_regularization(self, weight_decay: float):
        self.gpu.set_regularization(weight_decay)
        self.cpu.set_regularization(weight_decay)

    # ------------------------------------------------------------------ checks
    def compare_worker_outputs(self):
        g, c = self.gpu, self.cpu
        torch.cuda.synchronize()
        assert bits_equal(g.scales.cpu().numpy(), c.scales), "scales differ"
        gc = g.gcodes.cpu().numpy()
        if not np.array_equal(gc, c.gcodes):
            bad = np.argwhere(gc != c.gcodes)
            raise AssertionError(f"gcodes differ at {len(bad)} bytes, first {bad[:5].tolist()}")

    def compare_state(self, exact: bool = True):
        g, c = self.gpu, self.cpu
        torch.cuda.synchronize()
        assert g.poll_status() == 0
        for name in ("x", "m", "v", "e"):
            a = getattr(g, name).cpu().numpy()
            b = getattr(c, name)
            r = rel_err(a, b)
            assert r <= REL_TOL, f"{name}: relative error {r}"
            if exact:
                assert bits_equal(a, b), f"{name}: not bit-identical (rel err {r})"
        if c.kx >= 0:
            assert np.array_equal(g.wcodes.cpu().numpy()[:c.wcode_bytes], c.wcodes), "wcodes differ"
        if c.wresid is not None:
            assert bits_equal(g.wresid.cpu().numpy(), c.wresid), "wresid differs"
        if c.wfeedback is not None:
            assert bits_equal(g.wfeedback.cpu().numpy(), c.wfeedback), "wfeedback differs"

    def close(self):
        self.gpu.close()
