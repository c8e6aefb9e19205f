"""Checkpoint and resume.  The state of a run is exactly x, m, v, e and the step number
(every other buffer is an output of the step that writes it): T steps in one go and
T/2 steps + save + a NEW context loaded from the save + T/2 steps must give the same bits
in the state and in everything the last step emits."""
import io

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import paper_2004_14180_b200 as qb  # noqa: E402


def _grads(seed, t, n, D, seg_mask):
    gen = torch.Generator(device="cuda").manual_seed(seed * 1000 + t)
    return torch.randn(n, D, device="cuda", generator=gen) * 0.01 * seg_mask


@pytest.mark.parametrize("placement", [qb.PLACE_SERVER, qb.PLACE_WORKER])
@pytest.mark.parametrize("kg,kx", [(0, 0), (1, 6)])
def test_resume_is_bit_identical(kg, kx, placement):
    seg, n, T = [5000, 64, 3 * 4096 + 130, 70000], 4, 6
    rng = np.random.default_rng(3)
    x1 = torch.from_numpy((rng.standard_normal(sum(seg)) * 0.1).astype(np.float32))

    def fresh():
        return qb.QAdam(seg, n, kg=kg, kx=kx, placement=placement, x1=x1)

    a = fresh()
    mask = (a.to_padded(torch.ones(sum(seg), device="cuda")) != 0).float()     # pads stay zero
    for t in range(1, T + 1):
        a.step(t, _grads(kg + kx, t, n, a.D, mask))
    torch.cuda.synchronize()

    b = fresh()
    for t in range(1, T // 2 + 1):
        b.step(t, _grads(kg + kx, t, n, b.D, mask))
    torch.cuda.synchronize()
    blob = io.BytesIO()
    torch.save({"x": b.x.cpu(), "m": b.m.cpu(), "v": b.v.cpu(), "e": b.e.cpu(), "step": T // 2}, blob)
    b.close()
    del b

    blob.seek(0)
    ck = torch.load(blob)
    # a new context starts at step 1: the caller keeps the global step number and passes the
    # learning rate of that step; nothing else in the library depends on it
    c = fresh()
    for name in ("x", "m", "v", "e"):
        getattr(c, name).copy_(ck[name])
    torch.cuda.synchronize()
    for k, t in enumerate(range(ck["step"] + 1, T + 1), start=1):
        c.step(k, _grads(kg + kx, t, n, c.D, mask))
    torch.cuda.synchronize()
    assert a.poll_status() == 0 and c.poll_status() == 0
    for name in ("x", "m", "v", "e", "scales", "gcodes", "wcodes"):
        assert torch.equal(getattr(a, name).view(torch.uint8), getattr(c, name).view(torch.uint8)), name
    a.close()
    c.close()
