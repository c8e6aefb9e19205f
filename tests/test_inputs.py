"""The synthetic-input module: shape totals, determinism, stated distributions."""
import numpy as np
import torch

import qadam_inputs as qi


def test_shape_totals():
    r = qi.resnet18_shapes()
    assert len(r) == 62 and qi.numel(r) == 11_689_512
    b = qi.bert_base_shapes()
    assert len(b) == 199 and qi.numel(b) == 109_482_240
    assert max(np.prod(s) for _, s, _ in b) == 30522 * 768


def test_workloads_are_the_stated_configurations():
    w = qi.get_workload("flat20")
    assert (w.d, w.n, w.steps, w.kg, w.kx, w.num_segments) == (1 << 20, 4, 10, 0, -1, 1)
    w = qi.get_workload("resnet18_qg")
    assert (w.d, w.n, w.steps, w.kx, w.num_segments) == (11_689_512, 8, 100, -1, 62)
    assert qi.get_workload("resnet18_qg_qx_k1").kg == 1
    w = qi.get_workload("bert_base")
    assert (w.d, w.n, w.steps, w.kg, w.kx) == (109_482_240, 16, 50, 0, 0)
    for n in (1, 4, 16, 32):
        w = qi.get_workload("flat28", n=n)
        assert (w.d, w.n, w.steps) == (1 << 28, n, 20)
    assert w.with_(per_tensor_scale=False).num_segments == 1


def _small(grad, w0="gauss:0.05"):
    return qi.Workload("t", (3000, 64, 500), (27, 0, 0), (False, True, False), n=3, steps=2,
                       grad=grad, w0=w0)


def test_gradients_are_deterministic_and_distinct():
    w = _small("gauss_worker")
    a = qi.gradients(w, 1, 0)
    assert torch.equal(a, qi.gradients(w, 1, 0))
    assert not torch.equal(a, qi.gradients(w, 2, 0))
    assert not torch.equal(a, qi.gradients(w, 1, 1))
    assert a.dtype == torch.float32 and a.shape == (w.d,)


def test_distributions_have_the_stated_scales():
    w = qi.Workload("t", (200000,), (0,), (False,), n=4, steps=1, grad="gauss_worker", w0="gauss:0.05")
    for i in range(4):
        s = qi.gradients(w, 1, i).std().item()
        assert abs(s / (0.01 * (1 + 0.1 * i)) - 1) < 0.02
    assert abs(qi.initial_weights(w).std().item() / 0.05 - 1) < 0.02
    m = qi.gradients(w.with_(grad="mixture"), 1, 0)
    frac_out = (m.abs() > 6e-3).float().mean().item()       # 6 sigma of the narrow part
    assert 0.007 < frac_out < 0.011
    t = qi.gradients(_small("student_t_tensor"), 1, 0)
    assert torch.isfinite(t).all()
    g = qi.gradients(_small("gauss_tensor"), 1, 0)
    sig = [g[:3000].std().item(), g[3000:3064].std().item(), g[3064:].std().item()]
    assert all(5e-5 < s < 2e-1 for s in sig)


def test_he_init():
    x = qi.initial_weights(_small("gauss_worker", w0="he"))
    assert abs(x[:3000].std().item() / np.sqrt(2 / 27) - 1) < 0.05
    assert torch.all(x[3000:3064] == 1) and torch.all(x[3064:] == 0)


def test_scale_blocks_cut_every_tensor():
    w = qi.get_workload("flat20").with_(scale_block=1 << 18)
    assert w.scale_seg_len == (1 << 18,) * 4 and w.num_segments == 4
    r = qi.get_workload("resnet18_qg").with_(scale_block=100000)
    assert sum(r.scale_seg_len) == r.d and max(r.scale_seg_len) == 100000
    assert r.num_segments == sum(-(-ln // 100000) for ln in r.seg_len)
