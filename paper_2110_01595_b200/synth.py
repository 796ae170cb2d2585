"""Seeded synthetic workloads and Byzantine attacks for Solon's encode/decode path.

This module only makes inputs: partition gradients shaped like the paper's
models (Table 1) and the vectors that Byzantine nodes send instead of their
coded vectors (Section 4, "Attacks").  It contains none of the method's
arithmetic and imports neither the CUDA binding nor the CPU oracle, so both
can be fed from it.  Everything is a pure function of the seed.

The synthetic gradients stand in for the CIFAR-10 / SVHN / WikiText-2
gradients of the paper's experiments, which need datasets and training.
"""

from __future__ import annotations

import dataclasses
import math

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    """One configuration: plan parameters, gradient recipe, attack recipe."""

    name: str
    P: int
    s: int
    m: int          # compression ratio r_c
    d: int
    grads: str      # "normal" | "layered" | "lsq"
    sigma: float    # std of "normal" gradients
    attack: str     # "none" | "gaussian" | "flip10" | "neg_mean" | "alie"
    n_byz: int      # attackers actually present (<= s)
    seed: int
    fixed_byz: tuple = ()   # explicit attacker nodes, else drawn from the seed
    lsq_rows: int = 256

    @property
    def r(self) -> int:
        """Minimum group size allowed by the redundancy bound r >= 2 s + r_c (Theorem 2)."""
        return 2 * self.s + self.m

    @property
    def d_c(self) -> int:
        return -(-self.d // self.m)


WORKLOADS = {
    # P=8, s=1, m=2: two groups of four; node 3 sends N(0, 100^2) noise.
    "tiny": Workload("tiny", 8, 1, 2, 4096, "normal", 1.0, "gaussian", 1, 1000, fixed_byz=(3,)),
    # One least-squares SGD step; one node flips the sign of its coded vector and scales it by 10.
    "lsq": Workload("lsq", 15, 1, 3, 100_000, "lsq", 1.0, "flip10", 1, 2000),
    # ResNet-18-sized (Table 1: 11,173k parameters); two nodes send the negated mean coded vector.
    "resnet18": Workload("resnet18", 15, 2, 5, 11_173_962, "layered", 1.0, "neg_mean", 2, 3000),
    # VGG-13-sized; three nodes send mean + 1.5 std of the coded vectors (ALIE-style).
    "vgg13": Workload("vgg13", 45, 3, 5, 28_332_000, "normal", 0.1, "alie", 3, 4000),
    # Same without any attacker: detection must be a no-op.
    "vgg13_clean": Workload("vgg13_clean", 45, 3, 5, 28_332_000, "normal", 0.1, "none", 0, 4001),
}


def sweep_points(ds=(1_000_000, 10_000_000, 50_000_000)):
    """The (P, s, m, d) grid: P in {15,45,105}, s in {1,3,5}, m in {1,2,5,10}; infeasible points skipped."""
    points = []
    index = 0
    for d in ds:
        for P in (15, 45, 105):
            for s in (1, 3, 5):
                for m in (1, 2, 5, 10):
                    index += 1
                    if 2 * s + m > P:
                        continue
                    points.append(Workload(f"sweep_P{P}_s{s}_m{m}_d{d}", P, s, m, d, "normal", 1.0,
                                           "gaussian", s, 5000 + index))
    return points


def small_variant(wl: Workload, d: int) -> Workload:
    """Same plan and recipes at a smaller gradient length (for cases an oracle finishes in seconds)."""
    return dataclasses.replace(wl, name=f"{wl.name}_d{d}", d=d)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def layer_profile(d: int, seed: int, n_layers: int = 62):
    """Split d coordinates into contiguous layer blocks with log-uniform sizes and
    per-layer std drawn log-uniformly from [1e-4, 1e-1].  Returns (sizes, sigmas)."""
    g = _gen(seed, "cpu")
    u = torch.rand(n_layers, generator=g, dtype=torch.float64)
    weights = torch.exp(u * math.log(1e4))
    sizes = torch.clamp((weights / weights.sum() * d).floor().long(), min=1)
    sizes[-1] += d - int(sizes.sum())
    if sizes[-1] < 1:
        raise ValueError("d too small for the layer profile")
    v = torch.rand(n_layers, generator=g, dtype=torch.float64)
    sigmas = torch.exp(math.log(1e-4) + v * (math.log(1e-1) - math.log(1e-4)))
    return sizes, sigmas


def make_grads(wl: Workload, device="cpu") -> torch.Tensor:
    """Partition gradients G as a P x d float32 tensor on ``device`` ("normal" and "layered" recipes)."""
    g = _gen(wl.seed, device)
    if wl.grads == "normal":
        G = torch.empty((wl.P, wl.d), dtype=torch.float32, device=device)
        G.normal_(0.0, wl.sigma, generator=g)
        return G
    if wl.grads == "layered":
        sizes, sigmas = layer_profile(wl.d, wl.seed + 1)
        scale = torch.repeat_interleave(sigmas.to(torch.float32), sizes).to(device)
        G = torch.empty((wl.P, wl.d), dtype=torch.float32, device=device)
        G.normal_(0.0, 1.0, generator=g)
        G.mul_(scale[None, :])
        return G
    raise ValueError(f"recipe {wl.grads!r} has no direct gradient generator")


def make_lsq_problem(wl: Workload, device="cpu"):
    """Least-squares data: X (P*rows x d) ~ N(0,1), y = X w* + N(0, 0.01^2), iterate w = 0."""
    g = _gen(wl.seed, device)
    n = wl.P * wl.lsq_rows
    X = torch.empty((n, wl.d), dtype=torch.float32, device=device)
    X.normal_(0.0, 1.0, generator=g)
    w_star = torch.empty(wl.d, dtype=torch.float32, device=device).normal_(0.0, 1.0, generator=g)
    noise = torch.empty(n, dtype=torch.float32, device=device).normal_(0.0, 0.01, generator=g)
    y = X @ w_star + noise
    w = torch.zeros(wl.d, dtype=torch.float32, device=device)
    return X, y, w


def byzantine_nodes(wl: Workload) -> list[int]:
    """The attackers of this workload: explicit, or n_byz distinct nodes drawn from the seed."""
    if wl.n_byz == 0:
        return []
    if wl.fixed_byz:
        return list(wl.fixed_byz)
    g = _gen(wl.seed + 7, "cpu")
    return sorted(torch.randperm(wl.P, generator=g)[:wl.n_byz].tolist())


def byzantine_rows(wl: Workload, coded: torch.Tensor, nodes: list[int]) -> torch.Tensor:
    """The len(nodes) x d_c vectors the attackers send, computed from the honest coded matrix.

    gaussian: N(0, 100^2) noise.  flip10: -10 z_k.  neg_mean: every attacker sends
    -(1/P) sum_k z_k.  alie: per-coordinate mean + 1.5 population std of the P
    honest coded vectors (the "a little is enough" form mu + z sigma).
    """
    n = len(nodes)
    d_c = coded.shape[1]
    if n == 0 or wl.attack == "none":
        return coded.new_empty((0, d_c))
    if wl.attack == "gaussian":
        g = _gen(wl.seed + 13, coded.device)
        return torch.empty((n, d_c), dtype=coded.dtype, device=coded.device).normal_(0.0, 100.0, generator=g)
    if wl.attack == "flip10":
        return -10.0 * coded[nodes]
    if wl.attack == "neg_mean":
        return (-coded.mean(dim=0, keepdim=True)).expand(n, d_c).contiguous()
    if wl.attack == "alie":
        mu = coded.mean(dim=0, keepdim=True)
        sd = coded.std(dim=0, unbiased=False, keepdim=True)
        return (mu + 1.5 * sd).expand(n, d_c).contiguous()
    raise ValueError(f"unknown attack {wl.attack!r}")


def apply_attack(wl: Workload, coded: torch.Tensor):
    """Return (received, nodes): a copy of ``coded`` with the attackers' rows replaced."""
    nodes = byzantine_nodes(wl)
    received = coded.clone()
    if nodes and wl.attack != "none":
        received[nodes] = byzantine_rows(wl, coded, nodes)
    return received, nodes
