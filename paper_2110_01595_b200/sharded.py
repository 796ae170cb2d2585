"""Column-sharded encode / decode: one gradient problem spread over several GPUs.

The chunks of Section 3.4 are independent in the encoder and in the block decoder; only the locator of
Equation (1) looks at the whole coded vector, and it does so through the projected values rho = f R, which
are a sum over columns.  So device i keeps the coordinates [lo_i, hi_i) of every partition gradient (and
the matching columns of every coded vector), projects them with its own random f, and ONE all-reduce of
(K + 1) * P float64 values (a few KB: latency-bound) gives every device the same rho and nu.  Each device
then runs the same locator and recovers its own coordinates.  No other data crosses devices.

Argument marshalling and the collective only; every arithmetic step runs in the library's kernels.
"""

from __future__ import annotations

import torch
import torch.distributed as dist

from . import binding


def column_shares(d: int, m: int, world: int) -> list[tuple[int, int]]:
    """Coordinate ranges [lo, hi) of the `world` devices: whole chunks of m coordinates, as even as possible,
    the ragged last chunk (if m does not divide d) on the last device that owns anything."""
    if d < 1 or m < 1 or world < 1:
        raise ValueError("d, m and world must be positive")
    d_c = -(-d // m)
    base, extra = divmod(d_c, world)
    shares, chunk = [], 0
    for i in range(world):
        n = base + (1 if i < extra else 0)
        lo, hi = min(chunk * m, d), min((chunk + n) * m, d)
        shares.append((lo, hi))
        chunk += n
    return shares


class ShardedPlan:
    """The plan of one device for its share of the coordinates.

    All ranks pass the same (P, s, m, r, d, seed); rank i builds a library plan for d_i = hi_i - lo_i with seed
    seed + i, so the projection vectors of different shares are independent draws.  There must be at least as
    many chunks as devices.
    """

    def __init__(self, P: int, s: int, m: int, r: int, d: int, seed: int = 0, rank: int | None = None,
                 world: int | None = None, group=None):
        if rank is None:
            rank = dist.get_rank(group) if dist.is_initialized() else 0
        if world is None:
            world = dist.get_world_size(group) if dist.is_initialized() else 1
        self.rank, self.world, self.group = rank, world, group
        self.P, self.s, self.m, self.r, self.d = P, s, m, r, d
        self.lo, self.hi = column_shares(d, m, world)[rank]
        self.d_local = self.hi - self.lo
        if self.d_local <= 0:
            raise ValueError(f"{world} devices but only {-(-d // m)} chunks: every device needs at least one")
        self.plan = binding.Plan(P, s, m, r, self.d_local, seed=seed + rank)
        self.K = self.plan.K
        self._sums = None

    def _buffer(self, like):
        if self._sums is None:
            self._sums = torch.zeros((self.K + 1, self.P), dtype=torch.float64, device=like.device)
        return self._sums

    def encode(self, partition_grads_local, coded=None):
        """partition_grads_local: P x d_local (this device's coordinates of every partition gradient)."""
        return self.plan.encode(partition_grads_local, coded)

    def decode(self, received_local, agg_grad=None, byz_mask=None, all_reduce=None):
        """received_local: P x d_c_local.  Returns (aggregate of this device's coordinates, mask).

        all_reduce(tensor) sums a float64 device tensor in place over the devices; the default is
        torch.distributed.all_reduce on self.group (a no-op without a process group).  The plan must run on
        torch's current stream so that the collective is ordered between the two halves.
        """
        sums = self._buffer(received_local)
        rho, nu = sums[: self.K], sums[self.K]
        if received_local.is_cuda and self.plan.stream_handle != torch.cuda.current_stream().cuda_stream:
            raise RuntimeError("ShardedPlan.decode: the plan's stream is not torch's current stream, so the all-reduce "
                               "would not be ordered between the two halves of the decode (use plan.set_stream)")
        if self.s > 0:
            self.plan.decode_project(received_local, rho, nu)
            if all_reduce is not None:
                all_reduce(sums)
            elif dist.is_initialized() and self.world > 1:
                dist.all_reduce(sums, op=dist.ReduceOp.SUM, group=self.group)
        return self.plan.decode_finish(rho, nu, received_local, agg_grad, byz_mask)

    def close(self):
        if self.plan is not None:
            self.plan.close()
            self.plan = None
