"""Closed loop: least-squares gradient descent in which every step's gradient sum goes through Solon.

Per step: partition gradients (solon_lsq_grads) -> coded vectors (solon_encode) -> an adversary overwrites the
rows of a freshly drawn set of nodes (Section 5: a new Byzantine set every iteration) -> robust decode
(solon_decode) -> w <- w - lr * u.  The decode returns the exact gradient sum whatever the adversary sent, so the
iterates equal those of an attack-free run (Section 3.2).

The library's kernels do the method's arithmetic; this module is the harness around them: it draws the
attackers, lets them write (device-side tensor operations standing in for whatever arrives over the network) and
applies the update.  One step can be captured in a CUDA graph: the attackers' indices live in a device tensor
that is refreshed between replays, so the graph's shape is fixed while the Byzantine set changes.
"""

from __future__ import annotations

import numpy as np
import torch

from . import binding

ATTACKS = ("flip10", "neg_mean", "alie")


def draw_attackers(plan: binding.Plan, rng: np.random.Generator, per_group: int) -> list[int]:
    """`per_group` distinct nodes of every group (per_group <= s), sorted."""
    if per_group > plan.s:
        raise ValueError("more attackers per group than the plan tolerates")
    nodes = []
    start = 0
    for size in plan.group_sizes():
        nodes += (start + rng.permutation(size)[:per_group]).tolist()
        start += size
    return sorted(nodes)


def attack_rows(coded: torch.Tensor, idx: torch.Tensor, kind: str) -> torch.Tensor:
    """What the nodes idx send instead of their coded vectors (device-side, no host synchronisation).

    flip10: -10 z_k.  neg_mean: -(1/P) sum_k z_k.  alie: per-coordinate mean + 1.5 population standard
    deviations of the P honest coded vectors.
    """
    n = idx.numel()
    if kind == "flip10":
        return coded.index_select(0, idx) * (-10.0)
    if kind == "neg_mean":
        return (-coded.mean(dim=0, keepdim=True)).expand(n, coded.shape[1]).contiguous()
    if kind == "alie":
        mu = coded.mean(dim=0, keepdim=True)
        sd = coded.std(dim=0, unbiased=False, keepdim=True)
        return (mu + 1.5 * sd).expand(n, coded.shape[1]).contiguous()
    raise ValueError(f"unknown attack {kind!r}")


class ClosedLoop:
    """State of one run: data, iterate, and the buffers every step reuses."""

    def __init__(self, plan: binding.Plan, X: torch.Tensor, y: torch.Tensor, w0: torch.Tensor, lr: float, rows: int,
                 attackers_per_group: int = 0, attack: str = "flip10"):
        self.plan, self.X, self.y, self.lr = plan, X, y, float(lr)
        plan.set_lsq_rows(rows)
        plan.set_fresh_projections(True)      # a fresh Byzantine set every step may adapt to what it saw: new vectors f per decode
        self.w = w0.clone()
        dev = X.device
        self.grads = torch.empty((plan.P, plan.d), dtype=torch.float32, device=dev)
        self.coded = torch.empty((plan.P, plan.d_c), dtype=torch.float32, device=dev)
        self.agg = torch.empty(plan.d, dtype=torch.float32, device=dev)
        self.mask = torch.empty(plan.P, dtype=torch.uint8, device=dev)
        self.per_group = attackers_per_group
        self.attack = attack
        self.idx = torch.zeros(attackers_per_group * plan.q, dtype=torch.long, device=dev)
        self._idx_host = torch.zeros(attackers_per_group * plan.q, dtype=torch.long).pin_memory()
        self.graph = None

    def set_attackers(self, nodes: list[int]) -> None:
        """This step's Byzantine set (as many nodes as the loop was built for)."""
        if len(nodes) != self.idx.numel():
            raise ValueError("the number of attackers is fixed per loop")
        if nodes:
            self._idx_host.copy_(torch.tensor(nodes, dtype=torch.long))
            self.idx.copy_(self._idx_host, non_blocking=True)

    def _step_body(self) -> None:
        self.plan.lsq_grads(self.X, self.y, self.w, self.grads)
        self.plan.encode(self.grads, self.coded)
        if self.idx.numel():
            self.coded.index_copy_(0, self.idx, attack_rows(self.coded, self.idx, self.attack))
        self.plan.decode(self.coded, self.agg, self.mask)
        self.w.add_(self.agg, alpha=-self.lr)

    def step(self) -> None:
        """One iteration, launched eagerly (or by replaying the captured graph)."""
        if self.graph is not None:
            self.graph.replay()
        else:
            self._step_body()

    def capture(self) -> None:
        """Capture one iteration in a CUDA graph; later step() calls replay it.  The iterate is restored afterwards."""
        w_saved = self.w.clone()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            self.plan.set_stream(side)
            for _ in range(2):              # warm-up on the capture stream, as graph capture wants
                self._step_body()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.plan.set_stream(torch.cuda.current_stream())
            self._step_body()
        self.plan.set_stream(torch.cuda.current_stream())
        self.w.copy_(w_saved)
        self.graph = graph
