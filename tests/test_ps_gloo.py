"""The sharded parameter server's exchange bookkeeping, on CPU tensors over gloo.

Two and three processes stand in for as many GPUs.  Every rank knows what all code
streams, scales and packed weights should be (drawn from one seed), holds only its own
workers' rows and its own range of the weights, runs the exchange and must end up with
exactly the bytes the plan says it needs: every worker's codes inside its range, all
scales, the whole packed broadcast.  The cuts come from the library (host call)."""
import ctypes as C
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _problem(qb, n, kg=0, kx=0):
    lens = [3 * 4096 + 640, 130, 70000, 4096, 9000, 1]
    seg = (C.c_int64 * len(lens))(*lens)
    cfg = qb.QAdamConfig(d=sum(lens), n=n, num_segments=len(lens), seg_len=seg, kg=kg, kx=kx, grid_g=0,
                         placement=0, beta1=0.9, beta2=0.999, eps=1e-8, lr=1e-3, stream=None, seed=0)
    return cfg, seg, len(lens)


def _rank_main(rank, world, port, k, kg, kx):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import paper_2004_14180_b200 as qb
    from paper_2004_14180_b200 import ps
    dist.init_process_group("gloo", rank=rank, world_size=world)
    n = world * k
    cfg, _seg, S = _problem(qb, n, kg, kx)
    sz = qb.qadam_query_sizes(cfg)
    cuts = qb.qadam_shard_cuts(cfg, world)
    gbits, xbits = qb.qadam_grad_code_bits(kg), qb.qadam_weight_code_bits(kx)
    plan = ps.ShardPlan(world, rank, n, cuts, gbits, xbits)
    gen = torch.Generator().manual_seed(99)
    full_codes = torch.randint(0, 256, (n, sz["gcode_bytes"]), dtype=torch.uint8, generator=gen)
    full_scales = torch.rand(n, S, generator=gen)
    full_w = torch.randint(0, 256, (sz["wcode_bytes"],), dtype=torch.uint8, generator=gen)

    mine = range(rank * k, (rank + 1) * k)
    codes = torch.zeros_like(full_codes)
    codes[mine.start:mine.stop] = full_codes[mine.start:mine.stop]
    ps.exchange_codes(plan, codes)
    lo, hi = plan.code_span(rank)
    assert torch.equal(codes[:, lo:hi], full_codes[:, lo:hi]), "codes of my range"
    others = [i for i in range(n) if i not in mine]
    outside = torch.ones(sz["gcode_bytes"], dtype=torch.bool)
    outside[lo:hi] = False
    assert not codes[others][:, outside].any(), "bytes outside my range were not sent to me"
    assert torch.equal(codes[mine.start:mine.stop], full_codes[mine.start:mine.stop]), "my own rows"

    scales = torch.zeros_like(full_scales)
    scales[mine.start:mine.stop] = full_scales[mine.start:mine.stop]
    ps.gather_scales(plan, scales)
    assert torch.equal(scales, full_scales)

    w = torch.zeros_like(full_w)
    wlo, whi = plan.weight_span(rank)
    w[wlo:whi] = full_w[wlo:whi]
    ps.broadcast_weights(plan, w)
    assert torch.equal(w, full_w)

    # the accounting: what the ranks send adds up to every stream minus the ranges that stay home
    wire = ps.wire_bytes_per_step(plan, S)
    sent = torch.tensor([plan.sent_code_bytes()], dtype=torch.int64)
    dist.all_reduce(sent)
    assert int(sent) == wire["codes_up"]
    assert sum(plan.send_splits()) == k * sz["gcode_bytes"]
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world,k,kg,kx", [(2, 1, 0, 0), (2, 2, 1, 6), (3, 1, 0, 1), (3, 2, 3, 0)])
def test_exchange_delivers_exactly_what_each_shard_needs(world, k, kg, kx):
    mp.spawn(_rank_main, args=(world, _free_port(), k, kg, kx), nprocs=world, join=True)


def test_cuts_and_plan_properties():
    import paper_2004_14180_b200 as qb
    from paper_2004_14180_b200 import ps
    cfg, _seg, S = _problem(qb, 8)
    sz = qb.qadam_query_sizes(cfg)
    for shards in (1, 2, 3, 4, 8, 64, 1000):
        cuts = qb.qadam_shard_cuts(cfg, shards)
        assert cuts[0] == 0 and cuts[-1] == sz["D"] and cuts == sorted(cuts) and len(cuts) == shards + 1
        # every cut is a tile boundary: a multiple of 4096 counted from its segment's start
        for c in cuts[1:-1]:
            seg = max(i for i, o in enumerate(sz["seg_off"]) if o <= c) if c < sz["D"] else None
            if seg is not None:
                assert (c - sz["seg_off"][seg]) % 4096 == 0
        if shards <= 8:
            sizes = [b - a for a, b in zip(cuts, cuts[1:])]
            assert max(sizes) - min(sizes) <= 70000 + 4096          # balanced up to one tensor / tile
    with pytest.raises(qb.QAdamError):
        qb.qadam_shard_cuts(cfg, 0)
    plan = ps.ShardPlan(4, 1, 8, qb.qadam_shard_cuts(cfg, 4), 2, 2)
    assert plan.workers_of(1) == range(2, 4)
    wire = ps.wire_bytes_per_step(plan, S)
    assert 15.0 < wire["up_ratio"] <= 16.0 and abs(wire["down_ratio"] - 16.0) < 1e-9
    with pytest.raises(ValueError):
        ps.ShardPlan(3, 0, 8, qb.qadam_shard_cuts(cfg, 3), 2, 2)       # 8 workers, 3 ranks
