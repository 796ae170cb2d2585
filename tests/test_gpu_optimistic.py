"""Optimistic decode (solon_plan_set_optimistic): the projection pass recovers the aggregate from the rows that are read
when no node is corrupt, and the recovery kernel is skipped when the locator confirms them.  Results must not depend on
the mode: bit for bit the same aggregate, the same mask, with and without attackers, and against the oracle."""

import dataclasses

import numpy as np
import pytest
import torch

from oracle import solon_oracle as so
from paper_2110_01595_b200 import binding, build, synth

pytestmark = pytest.mark.gpu

AGG_TOL = 1e-4


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def _decode(plan, received):
    agg, mask = plan.decode(received)
    status = plan.decode_status()
    return status, agg.clone(), mask.clone(), plan.optimistic_outcome()


@pytest.mark.parametrize("name,d", [("vgg13_clean", 283_321), ("resnet18", 150_003), ("tiny", 4096), ("vgg13", 1_000_000)])
@pytest.mark.parametrize("early", [0, 2])
def test_modes_agree_with_and_without_attackers(name, d, early):
    wl = synth.small_variant(synth.WORKLOADS[name], d)
    G_cpu = synth.make_grads(wl, "cpu")
    want = so.plain_sum(G_cpu.numpy())
    scale = np.abs(want).max()
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=wl.seed) as plan:
        plan.set_early_locator(early)
        coded = plan.encode(G_cpu.cuda())
        attacked, nodes = synth.apply_attack(dataclasses.replace(wl, attack="gaussian", n_byz=wl.s), coded)
        plan.set_optimistic(0)
        ref_clean = _decode(plan, coded)
        ref_attacked = _decode(plan, attacked)
        assert ref_clean[0] == 0 and ref_attacked[0] == 0 and not ref_clean[3] and not ref_attacked[3]
        assert int(ref_clean[2].sum()) == 0 and ref_attacked[2].nonzero().flatten().tolist() == nodes
        assert np.abs(ref_clean[1].cpu().numpy() - want).max() <= AGG_TOL * scale
        assert np.abs(ref_attacked[1].cpu().numpy() - want).max() <= AGG_TOL * scale

        def same(got, ref):
            return got[0] == ref[0] and torch.equal(got[1], ref[1]) and torch.equal(got[2], ref[2])

        # mode 1: optimistic only after a decode that found every node honest
        plan.set_optimistic(1)
        first = _decode(plan, coded)            # nothing known yet: the ordinary path
        second = _decode(plan, coded)           # the projection pass recovers, the locator confirms, the recovery skips
        third = _decode(plan, attacked)         # it recovers again, but nodes are corrupt: the recovery kernel overwrites
        fourth = _decode(plan, attacked)        # the last decode was not clean: the ordinary path
        fifth = _decode(plan, coded)            # still the ordinary path (the last decode was not clean), but clean again
        sixth = _decode(plan, coded)            # optimistic again
        assert [x[3] for x in (first, second, third, fourth, fifth, sixth)] == [False, True, False, False, False, True]
        for got in (first, second, fifth, sixth):
            assert same(got, ref_clean)
        for got in (third, fourth):
            assert same(got, ref_attacked)
        # mode 2: always
        plan.set_optimistic(2)
        a = _decode(plan, attacked)
        b = _decode(plan, coded)
        c = _decode(plan, attacked)
        assert [x[3] for x in (a, b, c)] == [False, True, False]
        assert same(a, ref_attacked) and same(b, ref_clean) and same(c, ref_attacked)
        # and the oracle's own decode of the clean matrix
        u, o_mask, o_status = so.decode(coded.cpu().numpy(), wl.d, wl.m, wl.s, so.group_sizes(wl.P, wl.r),
                                        so.node_scalars(so.group_sizes(wl.P, wl.r)), plan.projection_vectors(), tau=1e-5)
        assert o_status == 0 and int(o_mask.sum()) == 0
        assert np.abs(b[1].cpu().numpy() - u).max() <= AGG_TOL * scale


@pytest.mark.parametrize("P,s,m,r,d", [
    (15, 2, 5, 9, 11_173),      # d % m != 0, odd d_c: rows off 16-byte boundaries
    (8, 1, 2, 4, 7),            # a handful of columns
    (45, 3, 1, 11, 50_001),     # m = 1
    (30, 2, 6, 10, 60_005),     # m = 6, three groups
    (16, 2, 4, 8, 4096),
])
def test_edge_shapes(P, s, m, r, d):
    wl = synth.Workload("opt_edge", P, s, m, d, "normal", 1.0, "none", 0, 31 + P)
    G_cpu = synth.make_grads(wl, "cpu")
    want = so.plain_sum(G_cpu.numpy())
    with binding.Plan(P, s, m, r, d, seed=3) as plan:
        coded = plan.encode(G_cpu.cuda())
        guard = torch.full((d + 64,), -7.0, dtype=torch.float32, device="cuda")     # the aggregate between two guard zones
        agg = guard[32:32 + d]
        if agg.data_ptr() % 16:
            pytest.skip("unaligned view")
        mask = torch.empty(P, dtype=torch.uint8, device="cuda")
        plan.set_optimistic(0)
        plan.decode(coded, agg, mask)
        ref = agg.clone()
        plan.set_optimistic(2)
        agg.fill_(float("nan"))
        plan.decode(coded, agg, mask)
        assert plan.decode_status() == 0 and plan.optimistic_outcome() and int(mask.sum()) == 0
        assert torch.equal(agg, ref)
        assert bool((guard[:32] == -7.0).all()) and bool((guard[32 + d:] == -7.0).all())
        assert np.abs(agg.cpu().numpy() - want).max() <= AGG_TOL * max(np.abs(want).max(), 1e-30)


def test_plans_that_are_not_eligible_ignore_the_mode():
    for P, s, m, dtype in ((15, 1, 10, "f32"), (105, 1, 1, "f32"), (15, 2, 5, "f64")):
        wl = synth.Workload("inel", P, s, m, 30_000, "normal", 1.0, "none", 0, 5)
        G = synth.make_grads(wl, "cuda")
        if dtype == "f64":
            G = G.double()
        with binding.Plan(P, s, m, wl.r, wl.d, dtype=dtype) as plan:
            plan.set_optimistic(2)
            coded = plan.encode(G)
            for _ in range(2):
                agg, mask = plan.decode(coded)
                assert plan.decode_status() == 0 and not plan.optimistic_outcome() and int(mask.sum()) == 0
            ref = G.sum(dim=0, dtype=torch.float64)
            assert float((agg.double() - ref).abs().max()) <= AGG_TOL * float(ref.abs().max())
