"""The allocation-free entry point, through the C interface, on a GPU.

qadam_worker_scales_static is for hosts that cannot allocate device memory once
they run (all device memory sized at start-up, cudaMalloc forbidden afterwards), so
they cannot hand the library the workspace its context-based calls need.  Its
scratch is a fixed array inside the library.  Here its output is compared, bit for
bit (the bar the other parity tests use for scales), with what the regular
qadam_worker_compress writes into `scales`, on two calls in a row of different
shapes: the second call must not see anything the first one left in the shared
scratch.  The file name sorts last so that a run that stops at the first failure
has already run every other test."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _regular_scales(qb, D, n, g, steps_before=1):
    """Scales from the regular path for gradients g at a step where e is non-zero;
    returns (scales, e as it was before that step)."""
    q = qb.QAdam([D], n, kg=0, kx=-1, placement=qb.PLACE_SERVER)
    gen = torch.Generator(device="cuda").manual_seed(1234 + D + n)
    for t in range(1, steps_before + 1):
        warm = torch.randn(n, D, device="cuda", generator=gen) * 0.02
        q.step(t, warm)
    e_before = q.e.clone()
    q.worker_compress(steps_before + 1, g)
    torch.cuda.synchronize()
    scales = q.scales.clone().view(-1)
    q.close()
    return scales, e_before


def test_static_scratch_entry_point_matches_worker_compress_twice_in_a_row():
    import paper_2004_14180_b200 as qb
    stream = torch.cuda.current_stream().cuda_stream
    gen = torch.Generator(device="cuda").manual_seed(7)
    shapes = [(3 * 4096 + 640, 5), (4096 + 128, 3)]      # second call is smaller: stale scratch must not leak
    cases = []
    for D, n in shapes:
        g = torch.randn(n, D, device="cuda", generator=gen) * 0.01
        want, e_before = _regular_scales(qb, D, n, g)
        cases.append((D, n, g, e_before, want))
    assert any(c[3].abs().max().item() > 0 for c in cases)       # error feedback is in play
    outs = []
    for D, n, g, e_before, want in cases:                        # two calls in a row
        out = torch.full((n,), -1.0, device="cuda")
        qb.qadam_worker_scales_static(g.data_ptr(), e_before.data_ptr(), D, n, out.data_ptr(), stream)
        outs.append(out)
    torch.cuda.synchronize()
    for (D, n, g, e_before, want), out in zip(cases, outs):
        got = out.cpu().numpy().view(np.uint32)
        assert np.array_equal(got, want.cpu().numpy().view(np.uint32)), (D, n)
        # and it is the plain definition: max |g + e| per worker
        ref = (g + e_before).abs().amax(dim=1)
        assert torch.equal(out, ref)


def test_static_scratch_entry_point_rejects_what_does_not_fit():
    import paper_2004_14180_b200 as qb
    buf = torch.zeros(256, device="cuda")
    out = torch.zeros(4, device="cuda")
    for D, n, code in [(qb.STATIC_MAX_ELEMENTS + 128, 1, -11), (128, qb.STATIC_MAX_WORKERS + 1, -11),
                       (100, 1, -2), (0, 1, -2), (128, 0, -2)]:
        with pytest.raises(qb.QAdamError) as ei:
            qb.qadam_worker_scales_static(buf.data_ptr(), buf.data_ptr(), D, n, out.data_ptr(), None)
        assert ei.value.code == code
    with pytest.raises(qb.QAdamError) as ei:
        qb.qadam_worker_scales_static(None, buf.data_ptr(), 128, 1, out.data_ptr(), None)
    assert ei.value.code == -1
    assert "capacity" in qb.qadam_strerror(-11)
