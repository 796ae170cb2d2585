"""The early locator (solon_plan_set_early_locator): the locator kernel starts on the projection of the first
part of every column range and the final pass only checks the set it found.  Results must not depend on the mode,
whether the attackers touch those first columns or not."""

import dataclasses

import numpy as np
import pytest
import torch

from oracle import solon_oracle as so
from paper_2110_01595_b200 import binding, build, synth

pytestmark = pytest.mark.gpu

AGG_TOL = 1e-4
SEEN = set()          # early outcomes observed over the module (1 confirmed, 2 rejected, 4 started too late)


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def _decode_all_modes(plan, received):
    out = []
    for mode in (0, 2, 1):
        plan.set_early_locator(mode)
        agg, mask = plan.decode(received)
        status = plan.decode_status()
        n_rec, t_acc, rows, coeff = plan.recovery()
        out.append((status, agg.clone(), mask.clone(), n_rec.copy(), t_acc.copy(), rows.copy(), coeff.copy(),
                    plan.early_outcome().tolist()))
    assert set(out[0][7]) == {0}                       # mode 0 never runs early
    assert set(out[1][7]) <= {1, 2, 4}                 # mode 2 always tries (small solvers); the wait never expires
    SEEN.update(out[1][7])
    return out


def _same(a, b):
    return (a[0] == b[0] and torch.equal(a[1], b[1]) and torch.equal(a[2], b[2]) and np.array_equal(a[3], b[3])
            and np.array_equal(a[4], b[4]) and np.array_equal(a[5], b[5]) and np.array_equal(a[6], b[6]))


@pytest.mark.parametrize("name,d", [("tiny", 4096), ("resnet18", 150_003), ("vgg13", 400_000), ("vgg13_clean", 100_000)])
def test_modes_agree_on_named_workloads(name, d):
    wl = synth.small_variant(synth.WORKLOADS[name], d)
    G_cpu = synth.make_grads(wl, "cpu")
    want = so.plain_sum(G_cpu.numpy())
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=wl.seed) as plan:
        received, nodes = synth.apply_attack(wl, plan.encode(G_cpu.cuda()))
        res = _decode_all_modes(plan, received)
        assert _same(res[0], res[1]) and _same(res[0], res[2])
        assert res[0][0] == 0
        assert res[0][2].cpu().numpy().nonzero()[0].tolist() == nodes
        assert np.abs(res[0][1].cpu().numpy() - want).max() <= AGG_TOL * np.abs(want).max()
        assert set(res[1][7]) <= {1, 4}                # whole rows are replaced: an early run sees every attacker


@pytest.mark.parametrize("P,s,m", [(15, 1, 1), (15, 3, 5), (15, 5, 2), (45, 5, 10), (105, 3, 5), (45, 1, 8)])
def test_modes_agree_on_sweep_shapes(P, s, m):
    wl = synth.Workload(f"early_{P}_{s}_{m}", P, s, m, 60_000 + 7 * m + 1, "normal", 1.0, "gaussian", s, 1000 + P + s + m)
    G_cpu = synth.make_grads(wl, "cpu")
    want = so.plain_sum(G_cpu.numpy())
    with binding.Plan(wl.P, wl.s, wl.m, 2 * s + m, wl.d, seed=wl.seed) as plan:
        received, nodes = synth.apply_attack(wl, plan.encode(G_cpu.cuda()))
        res = _decode_all_modes(plan, received)
        assert _same(res[0], res[1]) and _same(res[0], res[2])
        assert res[0][0] == 0 and res[0][2].cpu().numpy().nonzero()[0].tolist() == nodes
        assert np.abs(res[0][1].cpu().numpy() - want).max() <= AGG_TOL * np.abs(want).max()


@pytest.mark.parametrize("where", ["first", "last", "middle", "nan_last", "first_and_last"])
def test_corruption_confined_to_a_few_columns(where):
    """One corrupt entry is enough to be located; whether it sits in the columns the early run sees (the final pass
    confirms the early answer) or not (the final pass finds it itself) must not matter."""
    # m = 1 and 600 000 columns: every CTA of the projection kernel owns about 2048 columns, of which the first
    # 832 are its part A, so the last column of the matrix lies in a part B and column 0 in a part A
    wl = synth.Workload("confined", 15, 2, 1, 600_000, "normal", 1.0, "none", 0, 77)
    G_cpu = synth.make_grads(wl, "cpu")
    want = so.plain_sum(G_cpu.numpy())
    with binding.Plan(wl.P, wl.s, wl.m, 5, wl.d, seed=3) as plan:
        coded = plan.encode(G_cpu.cuda())
        d_c = plan.d_c
        received = coded.clone()
        if where == "first":
            received[2, 0] += 1.0
            nodes = [2]
        elif where == "last":
            received[2, d_c - 1] += 1.0
            nodes = [2]
        elif where == "middle":
            received[10, d_c // 2 + 11] -= 3.0
            received[11, d_c // 3] += 2.0
            nodes = [10, 11]
        elif where == "nan_last":
            received[14, d_c - 1] = float("nan")
            nodes = [14]
        else:
            received[6, 1] += 5.0            # seen by the early run
            received[7, d_c - 2] += 5.0      # not seen by it: the early answer {6} must be rejected
            nodes = [6, 7]
        res = _decode_all_modes(plan, received)
        assert _same(res[0], res[1]) and _same(res[0], res[2])
        assert res[0][0] == 0 and res[0][2].cpu().numpy().nonzero()[0].tolist() == nodes
        assert np.abs(res[0][1].cpu().numpy() - want).max() <= AGG_TOL * np.abs(want).max()
        # groups are nodes 0-4, 5-9, 10-14; a group whose attackers the early run saw all of is confirmed
        expect = {"first": [1, 1, 1], "last": [2, 1, 1], "nan_last": [1, 1, 2], "first_and_last": [1, 2, 1]}
        if where in expect:       # 4: that group's CTA became resident only after the projections and ran no early pass
            assert all(got in (want_g, 4) for got, want_g in zip(res[1][7], expect[where]))


def test_undecodable_and_reuse_with_the_early_locator():
    wl = synth.Workload("over", 9, 2, 5, 30_000, "normal", 1.0, "gaussian", 3, 5, fixed_byz=(1, 4, 7))
    G_cpu = synth.make_grads(wl, "cpu")
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d) as plan:
        plan.set_early_locator(2)
        coded = plan.encode(G_cpu.cuda())
        received, _ = synth.apply_attack(wl, coded)
        plan.decode(received)
        assert plan.decode_status() == binding.ERR_UNDECODABLE
        for _ in range(3):
            agg, mask = plan.decode(coded)
            assert plan.decode_status() == 0 and int(mask.sum()) == 0
        # the two-call form never uses it and still agrees
        rho = torch.zeros((plan.K, wl.P), dtype=torch.float64, device="cuda")
        nu = torch.zeros(wl.P, dtype=torch.float64, device="cuda")
        plan.decode_project(coded, rho, nu)
        agg2, mask2 = plan.decode_finish(rho, nu, coded)
        assert plan.decode_status() == 0 and torch.equal(agg, agg2) and torch.equal(mask, mask2)


def test_the_bounded_wait_for_partial_sums_runs_out_and_the_decode_is_unchanged():
    """Mode 3 lets the locator wait for partial sums that the projection kernel never announces: the wait (2 ms) gives
    up, the locator takes its ordinary path after the projections, reports outcome 3, and every output equals what
    mode 0 gives; the next decode in an ordinary mode is unaffected."""
    wl = synth.small_variant(synth.WORKLOADS["resnet18"], 150_003)
    G_cpu = synth.make_grads(wl, "cpu")
    want = so.plain_sum(G_cpu.numpy())
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=wl.seed) as plan:
        received, nodes = synth.apply_attack(wl, plan.encode(G_cpu.cuda()))
        out = []
        for mode in (0, 3, 3, 2):
            plan.set_early_locator(mode)
            agg, mask = plan.decode(received)
            status = plan.decode_status()
            n_rec, t_acc, rows, coeff = plan.recovery()
            out.append((status, agg.clone(), mask.clone(), n_rec.copy(), t_acc.copy(), rows.copy(), coeff.copy(),
                        plan.early_outcome().tolist()))
        assert set(out[0][7]) == {0}
        assert set(out[1][7]) == {3} and set(out[2][7]) == {3}          # the wait expired, twice in a row
        assert set(out[3][7]) <= {1, 4}                                 # and the counters were left clean
        for other in out[1:]:
            assert _same(out[0], other)
        assert out[0][0] == 0 and out[0][2].cpu().numpy().nonzero()[0].tolist() == nodes
        assert np.abs(out[0][1].cpu().numpy() - want).max() <= AGG_TOL * np.abs(want).max()


def test_both_early_outcomes_were_exercised():
    """Runs after the cases above (same module, file order): the early answer was confirmed somewhere and rejected
    somewhere, so both branches of the final pass are covered by the comparisons above."""
    assert {1, 2} <= SEEN
