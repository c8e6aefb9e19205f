"""Conditions the kernels report through the status word, made to happen without a fault.

A wait inside the persistent worker kernel is given something that never comes (the tile
tables claim one more tile per pair than exists: the test_missing_tiles option) and a small
poll limit; the kernel must return, the status word must carry the TIMEOUT bit, and the GPU
must go on working: a fresh context then passes an ordinary parity step."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import paper_2004_14180_b200 as qb  # noqa: E402
from _parity import Pair  # noqa: E402


@pytest.mark.parametrize("placement", [qb.PLACE_SERVER, qb.PLACE_WORKER])
@pytest.mark.parametrize("hand_over", [qb.HANDOVER_AUTO, qb.HANDOVER_COUNTERS])
def test_bounded_wait_runs_out_and_the_device_stays_usable(placement, hand_over):
    seg, n = [3 * 4096 + 300, 5000, 129], 2
    opt = qb.QAdamOptions(wait_polls=1 << 12, test_missing_tiles=1, hand_over=hand_over)
    q = qb.QAdam(seg, n, kg=0, kx=0, placement=placement, options=opt)
    one, two = q.worker_pass_model()
    assert one > 0 and two == 0                      # everything goes through the persistent kernel
    g = torch.randn(n, q.D, device="cuda") * 0.01
    q.worker_compress(1, g)                          # returns: every wait is bounded
    status = q.poll_status()
    assert status & qb.ST_TIMEOUT, status
    q.close()
    # the device is fine: the same problem without the hook matches the oracle
    rng = np.random.default_rng(5)
    d = sum(seg)
    p = Pair(seg, n, 0, 0, placement, x1=(rng.standard_normal(d) * 0.1).astype(np.float32),
             options=qb.QAdamOptions(hand_over=hand_over))
    for _ in range(2):
        p.step((rng.standard_normal((n, d)) * 0.01).astype(np.float32))
        p.compare_state()
    p.close()


def test_options_are_validated():
    for bad in (qb.QAdamOptions(server_kernel=2), qb.QAdamOptions(worker_kernel=-1),
                qb.QAdamOptions(hand_over=7), qb.QAdamOptions(test_missing_tiles=-1)):
        with pytest.raises(qb.QAdamError) as ei:
            qb.QAdam([1000], 1, options=bad)
        assert ei.value.code == -2
