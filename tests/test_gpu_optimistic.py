"""Optimistic decode (solon_plan_set_optimistic): the projection pass recovers the aggregate from the rows of the previous
decode's recovery table, and the recovery kernel is skipped when the locator finds all of them trusted.  Results must not
depend on the mode: the same mask, the same aggregate (bit for bit whenever the same table is used, within the tolerance
otherwise), with and without attackers, with attackers that stay and attackers that move, and against the oracle."""

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

        # attackers that move onto a row the table for `nodes` reads: in group 0 the first trusted node (m >= 2: the rows are
        # spread over the trusted nodes from the first to the last), the middle one for m = 1
        n0 = so.group_sizes(wl.P, wl.r)[0]
        trusted0 = [k for k in range(n0) if k not in nodes]
        moved_to = [trusted0[0] if wl.m >= 2 else trusted0[(len(trusted0) - 1) // 2]]
        attacked_b = coded.clone()
        attacked_b[moved_to] = synth.byzantine_rows(dataclasses.replace(wl, attack="gaussian", n_byz=1), coded, moved_to)
        ref_moved = _decode(plan, attacked_b)
        assert ref_moved[0] == 0 and ref_moved[2].nonzero().flatten().tolist() == moved_to

        def same(got, ref):
            return got[0] == ref[0] and torch.equal(got[1], ref[1]) and torch.equal(got[2], ref[2])

        def agrees(got, ref):
            # another table (other trusted rows) gives the same sum up to rounding; the recovery kernel itself always uses
            # the table of its own decode
            ok = got[0] == ref[0] and torch.equal(got[2], ref[2]) and np.abs(got[1].cpu().numpy() - want).max() <= AGG_TOL * scale
            return ok and (got[3] or same(got, ref))

        # mode 1: optimistic when in each of the last two decodes the table of the decode before would have served
        plan.set_optimistic(1)
        clean = [_decode(plan, coded) for _ in range(4)]
        # nothing known at first; the third recovers from the table of the second, the locator confirms, the recovery skips
        assert [x[3] for x in clean] == [False, False, True, True]
        assert all(same(x, ref_clean) for x in clean)
        # attackers arrive and stay: from the fourth decode on at the latest the table of the decode before avoids them
        runs = [_decode(plan, attacked) for _ in range(5)]
        assert all(agrees(got, ref_attacked) for got in runs)
        assert runs[3][3] and runs[4][3] and same(runs[3], ref_attacked) and same(runs[4], ref_attacked)
        # they move onto a row of that table: the speculation fails, the recovery kernel runs as usual
        moved = _decode(plan, attacked_b)
        assert not moved[3] and same(moved, ref_moved)
        after = [_decode(plan, attacked_b) for _ in range(2)]       # no speculation until two tables in a row have held
        assert not after[0][3] and not after[1][3] and all(same(got, ref_moved) for got in after)
        settled = [_decode(plan, attacked_b) for _ in range(2)]
        assert settled[0][3] and settled[1][3] and all(same(got, ref_moved) for got in settled)
        # mode 2: always (from whatever table the last decode left)
        plan.set_optimistic(2)
        a = _decode(plan, attacked)
        b = _decode(plan, coded)
        c = _decode(plan, coded)
        assert agrees(a, ref_attacked) and agrees(b, ref_clean) and b[3] and c[3] and same(c, ref_clean)
        # a decode that fails (more liars than s in a group) leaves nothing behind that the next one trips over
        too_many = list(range(wl.s + 1))
        broken = coded.clone()
        broken[too_many] = synth.byzantine_rows(dataclasses.replace(wl, attack="gaussian", n_byz=wl.s + 1), coded, too_many)
        failed = _decode(plan, broken)
        assert failed[0] != 0 and not failed[3]
        d1 = _decode(plan, coded)
        d2 = _decode(plan, coded)
        assert agrees(d1, ref_clean) and d2[3] and same(d2, ref_clean)
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


@pytest.mark.parametrize("P,s,m,r,d", [
    (15, 2, 5, 9, 150_003),     # one batch of rows, d_c odd: rows off 16-byte boundaries
    (45, 3, 5, 11, 283_321),    # two batches of rows: the speculated rows are taken first
    (30, 2, 6, 10, 60_005),
    (16, 1, 1, 3, 4099),
])
def test_float64_plans(P, s, m, r, d):
    """The same decode for float64 elements: float64 weights and sums as in the float64 recovery kernel."""
    wl = synth.Workload("opt_f64", P, s, m, d, "normal", 1.0, "gaussian", s, 17 + P)
    G = synth.make_grads(wl, "cuda").double()
    want = so.plain_sum(G.cpu().numpy())
    scale = np.abs(want).max()
    with binding.Plan(P, s, m, r, d, seed=3, dtype="f64") as plan:
        coded = plan.encode(G)
        attacked, nodes = synth.apply_attack(wl, coded)
        plan.set_optimistic(0)
        ref_clean = _decode(plan, coded)
        ref_attacked = _decode(plan, attacked)
        assert ref_clean[0] == 0 and ref_attacked[0] == 0 and not ref_clean[3] and not ref_attacked[3]
        assert ref_attacked[2].nonzero().flatten().tolist() == nodes
        assert np.abs(ref_attacked[1].cpu().numpy() - want).max() <= 1e-9 * scale

        def same(got, ref):
            return got[0] == ref[0] and torch.equal(got[1], ref[1]) and torch.equal(got[2], ref[2])

        plan.set_optimistic(1)
        runs = [_decode(plan, attacked) for _ in range(5)]
        for got in runs:
            assert got[0] == 0 and torch.equal(got[2], ref_attacked[2])
            assert np.abs(got[1].cpu().numpy() - want).max() <= 1e-9 * scale
            assert got[3] or same(got, ref_attacked)
        assert not runs[0][3] and not runs[1][3] and runs[3][3] and runs[4][3]
        assert same(runs[3], ref_attacked) and same(runs[4], ref_attacked)
        plan.set_optimistic(2)
        a = _decode(plan, coded)
        b = _decode(plan, coded)
        assert a[3] and b[3] and same(b, ref_clean)
        assert np.abs(a[1].cpu().numpy() - want).max() <= 1e-9 * scale


def test_random_plans_with_attackers_that_stay_and_move():
    """Random (P, s, m, r, d), a random walk of Byzantine sets (stay for a few decodes, then move; sometimes none): every
    decode, speculated or not, gives the exact mask and the aggregate within the tolerance; single-pass decodes do occur."""
    rng = np.random.default_rng(2024)
    seen_single_pass = 0
    for trial in range(24):
        m = int(rng.choice([1, 2, 3, 4, 5, 6]))
        s = int(rng.integers(1, 4))
        r = 2 * s + m + int(rng.integers(0, 3))
        q = int(rng.integers(1, 5))
        P = q * r + int(rng.integers(0, r))
        d = int(rng.integers(3_000, 60_000))
        dtype = "f64" if trial % 4 == 3 else "f32"
        wl = synth.Workload("opt_rand", P, s, m, d, "normal", 1.0, "gaussian", 0, 100 + trial)
        G = synth.make_grads(wl, "cuda")
        if dtype == "f64":
            G = G.double()
        ref = G.sum(dim=0, dtype=torch.float64)
        scale = float(ref.abs().max())
        tol = (1e-9 if dtype == "f64" else AGG_TOL) * scale
        sizes = so.group_sizes(P, r)
        starts = np.concatenate([[0], np.cumsum(sizes)])
        with binding.Plan(P, s, m, r, d, seed=trial, dtype=dtype) as plan:
            coded = plan.encode(G)
            nodes = []
            for step in range(14):
                if step % 4 == 0:          # the Byzantine set moves: up to s nodes in each group, or nobody
                    nodes = []
                    if rng.random() < 0.8:
                        for g in range(len(sizes)):
                            k = int(rng.integers(0, s + 1))
                            nodes += sorted((starts[g] + rng.choice(sizes[g], size=k, replace=False)).tolist())
                received = coded.clone()
                if nodes:
                    received[nodes] = synth.byzantine_rows(dataclasses.replace(wl, n_byz=len(nodes)), coded, nodes)
                agg, mask = plan.decode(received)
                assert plan.decode_status() == 0, (trial, step)
                assert mask.nonzero().flatten().tolist() == sorted(nodes), (trial, step)
                assert float((agg.double() - ref).abs().max()) <= tol, (trial, step)
                seen_single_pass += int(plan.optimistic_outcome())
    assert seen_single_pass >= 24


def test_replayed_graph_goes_over_to_the_single_pass_decode():
    """The decision lives on the device: a decode captured in a CUDA graph before anything was known speculates in later
    replays once two tables in a row have held, and falls back when the attackers move (the received matrix is rewritten
    in place between replays)."""
    wl = synth.small_variant(synth.WORKLOADS["vgg13"], 400_003)
    G = synth.make_grads(wl, "cuda")
    want = so.plain_sum(G.cpu().numpy())
    scale = np.abs(want).max()
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=11) as plan:
        coded = plan.encode(G)
        attacked, nodes = synth.apply_attack(dataclasses.replace(wl, attack="gaussian", n_byz=wl.s), coded)
        plan.set_optimistic(0)
        ref_clean = _decode(plan, coded)
        ref_attacked = _decode(plan, attacked)
        received = coded.clone()
        agg = torch.empty(wl.d, dtype=torch.float32, device="cuda")
        mask = torch.empty(wl.P, dtype=torch.uint8, device="cuda")
        plan.set_optimistic(1)                        # the mode in force at capture decides whether the captured kernel can speculate at all
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            plan.set_stream(side)
            plan.decode(received, agg, mask)          # warm-up on the capture stream, as graph capture wants
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            plan.set_stream(torch.cuda.current_stream())
            plan.decode(received, agg, mask)
        plan.set_stream(torch.cuda.current_stream())
        plan.set_optimistic(1)                        # again: the flags start from nothing

        def replay():
            graph.replay()
            torch.cuda.synchronize()
            return plan.decode_status(), agg.clone(), mask.clone(), plan.optimistic_outcome()

        clean = [replay() for _ in range(4)]
        assert [x[3] for x in clean] == [False, False, True, True]
        assert all(x[0] == 0 and torch.equal(x[1], ref_clean[1]) and torch.equal(x[2], ref_clean[2]) for x in clean)
        received.copy_(attacked)                      # attackers arrive and stay
        runs = [replay() for _ in range(5)]
        for x in runs:
            assert x[0] == 0 and torch.equal(x[2], ref_attacked[2])
            assert np.abs(x[1].cpu().numpy() - want).max() <= AGG_TOL * scale
        assert runs[3][3] and runs[4][3] and torch.equal(runs[4][1], ref_attacked[1])
        assert mask.nonzero().flatten().tolist() == nodes


def test_finish_with_given_projections_after_a_single_pass_decode():
    """solon_decode_finish with projections that did not come from this plan's own projection kernel just before: the
    recovery kernel must run, whatever the last whole decode of the plan did."""
    wl = synth.small_variant(synth.WORKLOADS["resnet18"], 120_007)
    G_a = synth.make_grads(wl, "cuda")
    G_b = synth.make_grads(dataclasses.replace(wl, seed=wl.seed + 1), "cuda")
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=9) as plan, binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=9) as other:
        coded_a, coded_b = plan.encode(G_a), plan.encode(G_b)
        for _ in range(4):
            agg_a, _ = plan.decode(coded_a)
        assert plan.optimistic_outcome()                     # the plan's last decode was a single-pass one
        rho = torch.empty(plan.K, wl.P, dtype=torch.float64, device="cuda")
        nu = torch.empty(wl.P, dtype=torch.float64, device="cuda")
        other.decode_project(coded_b, rho, nu)               # same seed: the same vectors f
        agg_b = torch.full((wl.d,), float("nan"), dtype=torch.float32, device="cuda")
        _, mask = plan.decode_finish(rho, nu, coded_b, agg_b)
        assert plan.decode_status() == 0 and int(mask.sum()) == 0 and not plan.optimistic_outcome()
        ref = G_b.sum(dim=0, dtype=torch.float64)
        assert float((agg_b.double() - ref).abs().max()) <= AGG_TOL * float(ref.abs().max())


def test_mode_argument_is_checked():
    with binding.Plan(8, 1, 2, 4, 4096) as plan:
        lib = binding.lib()
        for bad in (-1, 3, 17):
            assert lib.solon_plan_set_optimistic(plan._h, bad) == binding.ERR_INVALID_ARG
        assert lib.solon_plan_set_optimistic(None, 1) == binding.ERR_INVALID_ARG
        assert plan.status() == 0
        G = torch.randn(8, 4096, device="cuda")
        coded = plan.encode(G)
        for _ in range(4):                       # the default mode is still in force
            agg, mask = plan.decode(coded)
        assert plan.decode_status() == 0 and plan.optimistic_outcome() and int(mask.sum()) == 0
        ref = G.sum(dim=0, dtype=torch.float64)
        assert float((agg.double() - ref).abs().max()) <= AGG_TOL * float(ref.abs().max())


def test_plans_that_are_not_eligible_ignore_the_mode():
    for P, s, m, dtype in ((15, 1, 10, "f32"), (105, 1, 1, "f32"), (15, 1, 8, "f64")):
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
