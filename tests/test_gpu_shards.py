"""The server pass range by range (qadam_server_step_range), on one GPU.

A sharded server gives each shard a contiguous range of the vector.  Here one GPU
serves G ranges one after the other, in a shuffled order, and the result must be the
same bits as one pass over the whole vector and as the oracle: x, m, v and the packed
weights on every range, nothing touched outside the range being served.  The last
test runs the sharded step's driver with real NCCL collectives on a group of one rank."""
import os
import socket

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

import paper_2004_14180_b200 as qb  # noqa: E402
from _parity import Pair  # noqa: E402

SEG = [3 * 4096 + 640, 130, 70000, 4096, 9000, 1]


@pytest.mark.parametrize("placement", [qb.PLACE_SERVER, qb.PLACE_WORKER])
@pytest.mark.parametrize("shards", [2, 4, 8])
@pytest.mark.parametrize("kg,grid,n", [(0, 0, 4), (1, 0, 5), (3, 1, 3), (0, 0, 70), (-1, 0, 2)])
def test_virtual_shards_match_the_whole_pass(kg, grid, n, shards, placement):
    rng = np.random.default_rng(1000 + 10 * kg + n + shards)
    d = sum(SEG)
    x1 = (rng.standard_normal(d) * 0.2).astype(np.float32)
    p = Pair(SEG, n, kg, 1, placement, x1=x1, grid_g=grid, want_wresid=True)
    whole = qb.QAdam(SEG, n, kg=kg, kx=1, placement=placement, grid_g=grid,
                     x1=torch.from_numpy(x1), want_wresid=True)
    cuts = p.gpu.shard_cuts(shards)
    assert cuts[0] == 0 and cuts[-1] == p.gpu.D
    for t in range(1, 4):
        g = (rng.standard_normal((n, d)) * 0.01).astype(np.float32)
        gp = p.cpu.to_padded(g)
        g_dev = torch.from_numpy(gp).cuda()
        whole.step(t, g_dev)
        p.gpu.worker_compress(t, g_dev)
        p.cpu.workers_step(gp, p.lr)
        p.compare_worker_outputs()
        order = rng.permutation(shards)
        before = p.gpu.x.clone()
        for k, r in enumerate(order):
            p.gpu.server_step_range(t, cuts[r], cuts[r + 1])
            if k == 0:
                torch.cuda.synchronize()
                untouched = torch.ones(p.gpu.D, dtype=torch.bool, device="cuda")
                untouched[cuts[r]:cuts[r + 1]] = False
                assert torch.equal(p.gpu.x[untouched], before[untouched]), "a range wrote outside itself"
        p.gpu.finish_step(t)
        p.cpu.server_step(p.lr)
        p.compare_state()
        torch.cuda.synchronize()
        for name in ("x", "m", "v", "e", "wcodes", "wresid"):
            assert torch.equal(getattr(p.gpu, name).view(torch.uint8), getattr(whole, name).view(torch.uint8)), name
    p.close()
    whole.close()


def test_range_calls_check_their_arguments():
    q = qb.QAdam(SEG, 2, kg=0, kx=0)
    g = torch.zeros(2, q.D, device="cuda")
    cuts = q.shard_cuts(2)
    q.worker_compress(1, g)
    for lo, hi in [(128, cuts[1]), (0, cuts[1] + 128), (cuts[1], 0), (0, q.D + 4096), (-4096, cuts[1])]:
        with pytest.raises(qb.QAdamError) as ei:
            q.server_step_range(1, lo, hi)
        assert ei.value.code == -2
    with pytest.raises(qb.QAdamError) as ei:
        q.server_step_range(2, 0, cuts[1])
    assert ei.value.code == -6
    q.server_step_range(1, 0, cuts[1])
    with pytest.raises(qb.QAdamError) as ei:
        q.server_step(1)                         # the step is being served by ranges
    assert ei.value.code == -6
    with pytest.raises(qb.QAdamError) as ei:
        q.finish_step(2)
    assert ei.value.code == -6
    q.server_step_range(1, cuts[1], cuts[2])
    q.server_step_range(1, q.D, q.D)             # an empty range is fine
    q.finish_step(1)
    q.step(2, g)                                 # and the context goes on
    assert q.poll_status() == 0
    q.close()


def test_sharded_step_driver_with_nccl_on_one_rank():
    """ShardedStep with the collectives forced on (all-to-all, all-gather, broadcast over
    NCCL, group of one rank): same bits as the oracle."""
    import torch.distributed as dist
    from paper_2004_14180_b200 import ps
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    created = not dist.is_initialized()
    if created:
        dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                                device_id=torch.device("cuda", torch.cuda.current_device()))
    try:
        rng = np.random.default_rng(21)
        n, d = 3, sum(SEG)
        x1 = (rng.standard_normal(d) * 0.2).astype(np.float32)
        p = Pair(SEG, n, 0, 0, qb.PLACE_SERVER, x1=x1)
        drv = ps.ShardedStep(p.gpu, always_communicate=True)
        assert drv.plan.world == 1 and drv.plan.workers_per_rank == n
        for t in range(1, 4):
            g = (rng.standard_normal((n, d)) * 0.01).astype(np.float32)
            gp = p.cpu.to_padded(g)
            drv.step(t, torch.from_numpy(gp).cuda())
            p.cpu.step(gp, p.lr)
            p.compare_worker_outputs()
            p.compare_state()
        p.close()
    finally:
        if created:
            dist.destroy_process_group()
