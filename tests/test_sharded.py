"""Column-sharded decode (the chunks of Section 3.4 are independent; the locator of Equation (1) needs only
the sum over devices of the projected values).

CPU: the share layout, and two gloo ranks that each project their columns, all-reduce the K x P sums and run
the host build of the locator: both ranks locate the same, true, set and their recovered shares concatenate
to the plain sum.  GPU (one device, the ranks' kernels run one after another, none waits on another): the
library's two decode halves around an emulated all-reduce, against the oracle and the unsharded decode.
"""

import os
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

from oracle import solon_oracle as so
from paper_2110_01595_b200 import binding, build, sharded, synth


def test_column_shares_cover_and_align():
    for d in (1, 7, 64, 1000, 11_173_962):
        for m in (1, 2, 5, 10):
            d_c = -(-d // m)
            for world in (1, 2, 3, 8):
                shares = sharded.column_shares(d, m, world)
                assert len(shares) == world and shares[0][0] == 0 and shares[-1][1] == d
                for (lo, hi), (lo2, _) in zip(shares, shares[1:]):
                    assert hi == lo2
                widths = [-(-(hi - lo) // m) for lo, hi in shares]
                assert sum(widths) == d_c and max(widths) - min(widths) <= 1
                assert all(lo % m == 0 for lo, hi in shares if hi > lo)
    with pytest.raises(ValueError):
        sharded.column_shares(0, 1, 1)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _problem():
    P, s, m, r, d = 15, 2, 5, 15, 2003
    rng = np.random.default_rng(42)
    G = rng.normal(size=(P, d)).astype(np.float32)
    return P, s, m, r, d, G, [3, 11]


def _gloo_worker(rank, world, port, out):
    import torch.distributed as dist
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo")
    build.build()
    P, s, m, r, d, G, nodes = _problem()
    lo, hi = sharded.column_shares(d, m, world)[rank]
    sizes = so.group_sizes(P, r)
    w = so.node_scalars(sizes)
    Z = so.encode(G[:, lo:hi], m, sizes, w).astype(np.float32).astype(np.float64)
    R = Z.copy()
    if rank == 0:
        R[nodes[0]] = -10.0 * Z[nodes[0]]       # this node lies only in the columns of rank 0
    R[nodes[1]] = 50.0 + Z[nodes[1]]            # this one everywhere
    rng = np.random.default_rng(100 + rank)     # every rank draws its own f
    f = 1.0 + rng.normal(size=(2, R.shape[1]))
    sums = torch.from_numpy(np.concatenate([so.project(R, f), so.row_energy(R)[None]], axis=0))
    dist.all_reduce(sums)
    sums = sums.numpy()
    status, mask, t, rows, coeff = binding.solon_locate_host(sums[:2], sums[2], w, m, s, 1e-5)
    u = (coeff.T @ R[rows]).T.reshape(-1)[: hi - lo]
    out.put((rank, status, mask.tolist(), t, lo, u))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_locate_the_same_set_and_recover_their_shares():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_gloo_worker, args=(rk, 2, port, out)) for rk in range(2)]
    for p in procs:
        p.start()
    results = sorted((out.get(timeout=180) for _ in procs), key=lambda x: x[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    P, s, m, r, d, G, nodes = _problem()
    want = so.plain_sum(G)
    truth = [1 if k in nodes else 0 for k in range(P)]
    for rank, status, mask, t, lo, u in results:
        assert status == 0 and mask == truth and t == 2
    got = np.concatenate([res[5] for res in results])
    assert got.shape == want.shape
    assert np.abs(got - want).max() <= 1e-4 * np.abs(want).max()


# ------------------------------------------------------------------ GPU


def _sharded_case(wl, world, partial_attack):
    sizes = so.group_sizes(wl.P, wl.r)
    G_cpu = synth.make_grads(wl, "cpu")
    want = so.plain_sum(G_cpu.numpy().astype(np.float64))
    nodes = synth.byzantine_nodes(wl)
    plans = [sharded.ShardedPlan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=wl.seed, rank=i, world=world) for i in range(world)]
    try:
        received = []
        for i, sp in enumerate(plans):
            G_i = G_cpu[:, sp.lo:sp.hi].contiguous().cuda()
            coded = sp.encode(G_i)
            if nodes and not (partial_attack and i > 0):
                coded[nodes] = synth.byzantine_rows(wl, coded, nodes)
            received.append(coded)
        # the all-reduce, emulated: first every rank's projections, then their sum handed to each rank
        total = None
        for sp, R in zip(plans, received):
            buf = torch.zeros((sp.K + 1, wl.P), dtype=torch.float64, device="cuda")
            sp.plan.decode_project(R, buf[: sp.K], buf[sp.K])
            total = buf if total is None else total + buf
        parts, masks = [], []
        for sp, R in zip(plans, received):
            agg, mask = sp.decode(R, all_reduce=lambda t: t.copy_(total))
            assert sp.plan.decode_status() == 0
            parts.append(agg.cpu().numpy().astype(np.float64))
            masks.append(mask.cpu().numpy())
        truth = np.zeros(wl.P, dtype=np.uint8)
        truth[nodes] = 1
        for mk in masks:
            assert np.array_equal(mk, truth)
        got = np.concatenate(parts)
        assert got.shape == want.shape
        assert np.abs(got - want).max() <= 1e-4 * np.abs(want).max()
    finally:
        for sp in plans:
            sp.close()


@pytest.mark.gpu
@pytest.mark.parametrize("world", [1, 2, 3])
@pytest.mark.parametrize("name", ["tiny", "resnet18", "vgg13"])
def test_sharded_decode_matches_oracle(name, world):
    build.build()
    wl = synth.WORKLOADS[name]
    if wl.d > 1_000_000:
        wl = synth.small_variant(wl, 200_003)
    _sharded_case(wl, world, partial_attack=False)


@pytest.mark.gpu
def test_attack_confined_to_one_share_is_located_on_every_share():
    build.build()
    wl = synth.small_variant(synth.WORKLOADS["resnet18"], 100_001)
    _sharded_case(wl, 3, partial_attack=True)


@pytest.mark.gpu
def test_two_halves_equal_the_whole():
    build.build()
    wl = synth.small_variant(synth.WORKLOADS["vgg13"], 300_007)
    G = synth.make_grads(wl, "cuda")
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=wl.seed) as plan:
        coded, nodes = synth.apply_attack(wl, plan.encode(G))
        assert nodes
        agg, mask = plan.decode(coded)
        rho = torch.zeros((plan.K, wl.P), dtype=torch.float64, device="cuda")
        nu = torch.zeros(wl.P, dtype=torch.float64, device="cuda")
        plan.decode_project(coded, rho, nu)
        agg2, mask2 = plan.decode_finish(rho, nu, coded)
        assert plan.decode_status() == 0
        assert torch.equal(mask, mask2) and torch.equal(agg, agg2)
