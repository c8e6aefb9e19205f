"""The parameter server across processes: one process per GPU, the server sharded.

Algorithm 2 ("Broadcasting Q_x(x_t) to all workers", "Gathering all updates") and
Algorithm 3 ("Receiving", "Sending") with the workers spread over the ranks of a
torch.distributed group and the server's vector cut into one contiguous range per rank
(qadam_shard_cuts).  Per step a rank

  1. compresses its own workers (qadam_worker_compress on its worker range),
  2. sends every other rank the bytes of its workers' code streams that fall into that
     rank's range and receives the same from everyone (one all-to-all), and gathers all
     workers' scales (one all-gather),
  3. serves its range (qadam_server_step_range): x, m, v and the packed Q_x(x) there,
  4. broadcasts its piece of the packed weights, so that every rank holds the whole
     broadcast for the next step, and closes the step (qadam_finish_step).

What crosses the wire is what the paper counts in its "Comm" column: packed codes and
one scale per (worker, segment) up, packed weights down.  Everything received lands in
this rank's own buffers before any kernel reads it; no kernel is handed another GPU's
memory.

This module holds the bookkeeping (who sends which bytes where) and the collectives; all
arithmetic stays in the library's kernels.  It works on any tensors, so its logic is
testable with CPU tensors over the gloo backend.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence

import torch
import torch.distributed as dist


@dataclass(frozen=True)
class ShardPlan:
    """Who owns what.  Workers are dealt out in equal consecutive blocks; rank r serves
    elements [cuts[r], cuts[r + 1]) of the padded vector."""
    world: int
    rank: int
    n: int                      # workers in all
    cuts: Sequence[int]         # world + 1 element offsets (qadam_shard_cuts)
    gbits: int                  # bits per gradient code (32: identity)
    xbits: int                  # bits per weight code (0: weights are not quantized)

    def __post_init__(self):
        if self.n % self.world != 0:
            raise ValueError(f"{self.n} workers cannot be dealt out evenly to {self.world} ranks")
        if len(self.cuts) != self.world + 1 or list(self.cuts) != sorted(self.cuts):
            raise ValueError("cuts must be world + 1 non-decreasing offsets")
        for c in self.cuts:
            if (c * self.gbits) % 8 or (c * self.xbits) % 8:
                raise ValueError("a cut does not fall on a byte boundary of the packed streams")

    @property
    def workers_per_rank(self) -> int:
        return self.n // self.world

    def workers_of(self, rank: int) -> range:
        k = self.workers_per_rank
        return range(rank * k, (rank + 1) * k)

    def code_span(self, shard: int):
        """Byte range of shard `shard` inside ONE worker's code stream."""
        return self.cuts[shard] * self.gbits // 8, self.cuts[shard + 1] * self.gbits // 8

    def weight_span(self, shard: int):
        """Byte range of shard `shard` inside the packed weights."""
        return self.cuts[shard] * self.xbits // 8, self.cuts[shard + 1] * self.xbits // 8

    def sent_code_bytes(self) -> int:
        """Bytes of codes this rank puts on the wire per step (its own range stays local)."""
        k = self.workers_per_rank
        lo, hi = self.code_span(self.rank)
        total = (self.cuts[-1] * self.gbits // 8) * k
        return total - (hi - lo) * k

    def send_splits(self) -> List[int]:
        k = self.workers_per_rank
        return [k * (self.code_span(j)[1] - self.code_span(j)[0]) for j in range(self.world)]

    def recv_splits(self) -> List[int]:
        k = self.workers_per_rank
        lo, hi = self.code_span(self.rank)
        return [k * (hi - lo)] * self.world


def exchange_codes(plan: ShardPlan, gcodes: torch.Tensor, group=None, always: bool = False) -> None:
    """gcodes: [n][gcode_bytes] uint8.  On entry the rows of this rank's workers are
    complete; on return the columns of this rank's range are complete in EVERY row.
    With one rank there is nothing to exchange and no collective is called, unless
    `always` asks for it (the collective then copies the rank's own bytes onto themselves)."""
    k, world, rank = plan.workers_per_rank, plan.world, plan.rank
    mine = gcodes[rank * k:(rank + 1) * k]
    if world == 1 and not always:
        return
    # destination-major send buffer: for rank j, my workers' bytes of j's range
    if k == 1:
        send = mine.reshape(-1)                           # one stream: already in shard order
    else:
        send = torch.cat([mine[:, plan.code_span(j)[0]:plan.code_span(j)[1]].reshape(-1)
                          for j in range(world)])
    lo, hi = plan.code_span(rank)
    recv = torch.empty(world * k * (hi - lo), dtype=gcodes.dtype, device=gcodes.device)
    dist.all_to_all_single(recv, send.contiguous(), output_split_sizes=plan.recv_splits(),
                           input_split_sizes=plan.send_splits(), group=group)
    # source-major receive buffer: rank i's k workers, each (hi - lo) bytes
    gcodes[:, lo:hi].copy_(recv.view(world * k, hi - lo))


def gather_scales(plan: ShardPlan, scales: torch.Tensor, group=None, always: bool = False) -> None:
    """scales: [n][S] float32; this rank's workers' rows are complete on entry, all rows on return."""
    if plan.world == 1 and not always:
        return
    k, rank = plan.workers_per_rank, plan.rank
    mine = scales[rank * k:(rank + 1) * k].contiguous().clone()
    dist.all_gather_into_tensor(scales.view(-1), mine.view(-1), group=group)


def broadcast_weights(plan: ShardPlan, wcodes: torch.Tensor, group=None, always: bool = False) -> None:
    """wcodes: packed Q_x(x), uint8; this rank's range is fresh on entry, everything on return."""
    if (plan.world == 1 and not always) or plan.xbits == 0:
        return
    for r in range(plan.world):
        lo, hi = plan.weight_span(r)
        if hi > lo:
            dist.broadcast(wcodes[lo:hi], src=dist.get_global_rank(group, r) if group is not None else r,
                           group=group)


def wire_bytes_per_step(plan: ShardPlan, S: int) -> dict:
    """What one step moves between ranks, summed over ranks, against fp32 both ways."""
    world, k = plan.world, plan.workers_per_rank
    D = plan.cuts[-1]
    stream = D * plan.gbits // 8
    codes = sum(k * (stream - (plan.code_span(r)[1] - plan.code_span(r)[0])) for r in range(world))
    scales = world * (world - 1) * k * S * 4
    wbytes = D * plan.xbits // 8 if plan.xbits else 4 * D
    weights = sum((world - 1) * (plan.weight_span(r)[1] - plan.weight_span(r)[0]) for r in range(world)) \
        if plan.xbits else (world - 1) * 4 * D
    fp32_up = sum(k * 4 * (D - (plan.cuts[r + 1] - plan.cuts[r])) for r in range(world))
    fp32_down = (world - 1) * 4 * D
    return {"codes_up": codes, "scales_up": scales, "weights_down": weights,
            "fp32_up": fp32_up, "fp32_down": fp32_down, "packed_weight_bytes": wbytes,
            "up_ratio": fp32_up / max(1, codes + scales), "down_ratio": fp32_down / max(1, weights)}


class ShardedStep:
    """Drives one rank of the sharded parameter server on top of a QAdam context.

    q: binding.QAdam with n = total workers (only this rank's workers' rows of e, and this
    rank's range of x, m, v, are live).  g_local: [workers_per_rank][D] gradients of this
    rank's workers."""

    def __init__(self, q, group=None, always_communicate: bool = False):
        self.q = q
        self.group = group
        self.always = always_communicate      # call the collectives even with a single rank
        world = dist.get_world_size(group) if dist.is_initialized() else 1
        rank = dist.get_rank(group) if dist.is_initialized() else 0
        gbits = q.gcode_bytes * 8 // q.D
        xbits = q.wcode_bytes * 8 // q.D
        self.plan = ShardPlan(world, rank, q.n, q.shard_cuts(world), gbits, xbits)

    def step(self, step: int, g_local: torch.Tensor, lr: float = -1.0) -> None:
        q, plan = self.q, self.plan
        k = plan.workers_per_rank
        q.worker_compress(step, g_local, plan.rank * k, k, lr)
        talk = plan.world > 1 or self.always
        if talk:
            # the collectives run on torch's stream for this device: order them after the kernels
            self._sync_streams()
            exchange_codes(plan, q.gcodes, self.group, self.always)
            gather_scales(plan, q.scales, self.group, self.always)
            self._sync_streams()
        q.server_step_range(step, plan.cuts[plan.rank], plan.cuts[plan.rank + 1], lr)
        if talk and q.kx >= 0:
            self._sync_streams()
            broadcast_weights(plan, q.wcodes[:q.wcode_bytes], self.group, self.always)
            self._sync_streams()
        q.finish_step(step)

    def _sync_streams(self) -> None:
        # the context's stream and torch's current stream are the same unless the caller
        # gave the context a stream of its own; then each waits for the other
        if self.q.stream is not None:
            cur = torch.cuda.current_stream(self.q.device)
            if cur != self.q.stream:
                cur.wait_stream(self.q.stream)
                self.q.stream.wait_stream(cur)
