"""GPU parity: the CUDA path, called through the C-ABI binding, against the float64 oracle on the same
seeded inputs.  Bars: Byzantine mask bit-exact; aggregate within 1e-4 of ||sum||_inf; coded vectors within
one float32 rounding of the oracle's float64 values; projections within the float32 runs the kernel states."""

import dataclasses

import numpy as np
import pytest
import torch

from oracle import solon_oracle as so
from paper_2110_01595_b200 import binding, build, synth

pytestmark = pytest.mark.gpu

AGG_TOL = 1e-4          # max |agg_gpu - agg*| / ||agg*||_inf
TAU = 1e-5              # the library's default detection tolerance, also given to the oracle
RHO_TOL = 8 * 2.0 ** -24 * 1.01   # projections: worst case of the kernel's float32 runs, relative to ||f|| ||R_k||
# Coded values against the oracle's float64 encoding, in float32 roundings (2^-24) of the sum of |terms|.  The largest
# error seen over this suite's shapes is 3.8 roundings (m <= 6: float32 group sum and Horner steps), 3.0 (m = 8, 10) and
# 3.1 (other m: float32 group sum, float64 evaluation); the bar is about twice that, far below the worst case (r_g + m).
CODED_ROUNDINGS = 8.0
OBSERVED = {"coded_roundings": 0.0}


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()
    assert torch.cuda.is_available()


def _oracle_plan(wl):
    sizes = so.group_sizes(wl.P, wl.r)
    return sizes, so.node_scalars(sizes)


def _check_encode(plan, G_cpu, coded_gpu, m, sizes, w):
    """Coded vectors against the oracle's float64 values.

    Every m: float32 group sums and (m <= 6) float32 Horner steps stay within CODED_ROUNDINGS roundings of the sum of
    absolute terms (about twice the largest error observed; the worst case would be r_g + m).  m > 6 in addition: the group sum is the float32 left-to-right sum ybar' of the group's rows
    (its rounding is common to all nodes of the group, so the decoder returns it unamplified), and the coded
    values are the float64 evaluation of the polynomial with coefficients ybar', rounded once: half an ulp from
    the oracle's encoding of ybar'."""
    G_np = G_cpu.numpy()
    Z = so.encode(G_np, m, sizes, w)
    got = coded_gpu.cpu().numpy().astype(np.float64)
    bound = so.encode(np.abs(G_np), m, sizes, np.abs(w))          # sum of |terms| of every entry
    err = np.abs(got - Z)
    worst = float((err / (2.0 ** -24 * bound + 1e-300)).max())
    OBSERVED["coded_roundings"] = max(OBSERVED["coded_roundings"], worst)
    assert np.all(err <= CODED_ROUNDINGS * 2.0 ** -24 * bound + 1e-45), worst
    if m > 6:
        G_sum = np.zeros_like(G_np)                                # row `start` of each group: ybar', the others 0
        for start, size in zip(so.group_starts(sizes), sizes):
            acc = np.zeros(G_np.shape[1], dtype=np.float32)
            for k in range(start, start + size):
                acc = acc + G_np[k]                                # float32 adds, rows in order
            G_sum[start] = acc
        Z32 = so.encode(G_sum, m, sizes, w)
        bound32 = so.encode(np.abs(G_sum), m, sizes, np.abs(w))
        err32 = np.abs(got - Z32)
        assert np.all(err32 <= 2.0 ** -24 * np.abs(Z32) * 1.0001 + 1e-14 * bound32 + 1e-45), \
            float((err32 / (np.abs(Z32) + 1e-30)).max())
    return Z


def _run_case(wl, n_byz=None, check_intermediates=True):
    """Encode on the GPU, attack, decode on the GPU; compare everything with the oracle."""
    if n_byz is not None:
        wl = dataclasses.replace(wl, n_byz=n_byz, fixed_byz=(), attack=wl.attack if n_byz else "none")
    sizes, w = _oracle_plan(wl)
    G_cpu = synth.make_grads(wl, "cpu")
    G = G_cpu.cuda()
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=wl.seed) as plan:
        assert plan.group_sizes() == sizes
        assert np.allclose(plan.node_scalars(), w, rtol=0, atol=1e-15)
        coded = plan.encode(G)
        torch.cuda.synchronize()
        if check_intermediates:
            _check_encode(plan, G_cpu, coded, wl.m, sizes, w)
        received, nodes = synth.apply_attack(wl, coded)
        agg, mask = plan.decode(received)
        status = plan.decode_status()
        assert status == 0, binding.strerror(status)
        R = received.cpu().numpy()
        want_mask = so.true_mask(R, coded.cpu().numpy())
        assert want_mask.nonzero()[0].tolist() == nodes
        assert np.array_equal(mask.cpu().numpy(), want_mask)                       # bit-exact
        want = so.plain_sum(G_cpu.numpy())
        scale = np.abs(want).max()
        got = agg.cpu().numpy().astype(np.float64)
        assert np.abs(got - want).max() <= AGG_TOL * scale, np.abs(got - want).max() / scale
        # the oracle's own decode of the very same received matrix (Algorithm 1 in float64)
        f = plan.projection_vectors()
        u, o_mask, o_status = so.decode(R, wl.d, wl.m, wl.s, sizes, w, f, tau=TAU)
        assert o_status == 0 and np.array_equal(o_mask, want_mask)
        assert np.abs(got - u).max() <= AGG_TOL * scale
        if check_intermediates and wl.s > 0:
            rho, nu = plan.projections()
            o_rho = so.project(R, f)
            o_nu = so.row_energy(R)
            f64 = f.astype(np.float64)
            lim = np.sqrt((f64 ** 2).sum(1))[:, None] * np.sqrt(o_nu)[None, :]
            # products and runs of eight terms in float32, the rest in float64: |error| <= 8 * 2^-24 * sum |f_p R_kp|,
            # and sum |f_p R_kp| <= ||f|| ||R_k||
            assert np.all(np.abs(rho - o_rho) <= RHO_TOL * lim + 1e-300)
            assert np.allclose(nu, o_nu, rtol=1e-4)
            # what matters to the locator: on rows of ordinary size (honest ones) the error stays below a tenth of the
            # detection tolerance tau * sqrt(2 median nu) of the row's group, so it cannot flip a decision
            for start, size in zip(so.group_starts(sizes), sizes):
                grp = slice(start, start + size)
                tol = so.detection_tolerance(o_nu[grp], TAU)
                ordinary = o_nu[grp] <= 4.0 * np.median(o_nu[grp])
                assert np.all(np.abs(rho - o_rho)[:, grp][:, ordinary] <= 0.1 * tol + 1e-300)
            n_rec, t_acc, rows, coeff = plan.recovery()
            starts = so.group_starts(sizes)
            off = 0
            for g, (start, size) in enumerate(zip(starts, sizes)):
                in_group = [k for k in nodes if start <= k < start + size]
                assert t_acc[g] == len(in_group)
                rg = rows[off:off + n_rec[g]]
                assert n_rec[g] == (wl.m if wl.m <= 6 else size - len(in_group))
                assert all(start <= k < start + size and k not in nodes for k in rg)
                Wm = so.w_hat(w[start:start + size], wl.m - 1)[rg - start]
                assert np.allclose(coeff[off:off + n_rec[g]].T @ Wm, np.eye(wl.m), atol=1e-8)
                off += n_rec[g]
        return np.abs(got - want).max() / scale


# ---------------------------------------------------------------- the five configurations, small


def test_config_tiny():
    _run_case(synth.WORKLOADS["tiny"])


def test_config_resnet18_shape_small():
    # same plan, layered sigma profile and attack; spans many encode tiles and a ragged tail (d % m != 0)
    _run_case(synth.small_variant(synth.WORKLOADS["resnet18"], 1_117_397))


def test_config_vgg13_shape_small():
    _run_case(synth.small_variant(synth.WORKLOADS["vgg13"], 283_321))
    _run_case(synth.small_variant(synth.WORKLOADS["vgg13_clean"], 283_321))


@pytest.mark.parametrize("P,s,m", [(15, 1, 1), (15, 1, 2), (15, 1, 5), (15, 1, 10), (15, 3, 5), (15, 5, 2), (15, 5, 5),
                                   (45, 1, 10), (45, 3, 1), (45, 3, 10), (45, 5, 5), (45, 5, 10), (105, 1, 1),
                                   (105, 3, 5), (105, 5, 10), (105, 5, 2)])
def test_config_sweep_small(P, s, m):
    wl = synth.Workload(f"sweep_P{P}_s{s}_m{m}", P, s, m, 100_003, "normal", 1.0, "gaussian", s, 5000 + P + 10 * s + m)
    _run_case(wl)


@pytest.mark.parametrize("d", [5_003, 5_004])          # rows off and on 16-byte boundaries: scalar and 128-bit-load kernels
@pytest.mark.parametrize("iterate", ["zero", "random"])
def test_config_lsq_small(d, iterate):
    wl = dataclasses.replace(synth.WORKLOADS["lsq"], d=d, lsq_rows=64)
    sizes, w = _oracle_plan(wl)
    X, y, wvec = synth.make_lsq_problem(wl, "cpu")
    if iterate == "random":
        wvec = torch.empty(d, dtype=torch.float32).normal_(0.0, 1.0, generator=torch.Generator().manual_seed(77))
    want_G = so.lsq_grads(X.numpy(), y.numpy(), wvec.numpy(), wl.lsq_rows)
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=wl.seed) as plan:
        G = plan.lsq_grads(X.cuda(), y.cuda(), wvec.cuda(), rows=wl.lsq_rows)
        got_G = G.cpu().numpy().astype(np.float64)
        Xa = np.abs(X.numpy()).astype(np.float64)
        e = np.abs(X.numpy().astype(np.float64) @ wvec.numpy().astype(np.float64) - y.numpy())
        # residuals: float32 products summed in float64 and one rounding to float32; gradients likewise
        e_err = 2.0 ** -24 * (Xa @ np.abs(wvec.numpy()).astype(np.float64)) + 2.0 ** -24 * e
        for i in range(wl.P):
            rows = slice(i * wl.lsq_rows, (i + 1) * wl.lsq_rows)
            bound = Xa[rows].T @ e[rows]                      # sum of |terms|
            assert np.all(np.abs(got_G[i] - want_G[i]) <= 3e-7 * bound + 1.01 * Xa[rows].T @ e_err[rows] + 1e-30)
        coded = plan.encode(G)
        received, nodes = synth.apply_attack(wl, coded)
        agg, mask = plan.decode(received)
        assert plan.decode_status() == 0
        assert mask.cpu().numpy().nonzero()[0].tolist() == nodes and len(nodes) == 1
        want = want_G.sum(0)                                   # the oracle's own float64 gradients
        assert np.abs(agg.cpu().numpy() - want).max() <= AGG_TOL * np.abs(want).max()


# ---------------------------------------------------------------- edge cases


@pytest.mark.parametrize("P,s,m,r,d", [
    (4, 1, 2, 4, 2),          # the introduction's example: d_c = 1
    (5, 1, 3, 5, 1),          # d < m: one padded chunk
    (5, 0, 5, 5, 23),         # s = 0: pure compression code, no locator
    (9, 2, 1, 5, 1000),       # m = 1: repetition code
    (7, 3, 1, 7, 255),        # maximal s for P
    (16, 2, 4, 8, 4096),      # r divides P (the paper's layout), m = 4
    (11, 1, 7, 9, 1234),      # m without a specialised kernel
    (23, 1, 3, 23, 777),      # r = P, one odd-sized group
    (40, 2, 12, 20, 3000),    # m = 12 (generic kernels), two groups of 20
    (128, 1, 2, 128, 513),    # largest group the locator handles
    (256, 1, 2, 4, 10_007),   # 64 groups of four
    (1024, 1, 1, 3, 517),     # most nodes allowed: 341 groups of three (one of four)
    (126, 16, 1, 126, 300),   # most adversaries per group allowed
    (40, 3, 8, 20, 4_001),    # m = 8: float64 paths, all-rows inverse
])
def test_edge_shapes(P, s, m, r, d):
    wl = synth.Workload("edge", P, s, m, d, "normal", 1.0, "gaussian", s, 99)
    wl_r = dataclasses.replace(wl)
    sizes = so.group_sizes(P, r)
    w = so.node_scalars(sizes)
    G_cpu = synth.make_grads(wl, "cpu")
    with binding.Plan(P, s, m, r, d, seed=7) as plan:
        assert plan.group_sizes() == sizes
        coded = plan.encode(G_cpu.cuda())
        _check_encode(plan, G_cpu, coded, m, sizes, w)
        received, nodes = synth.apply_attack(wl_r, coded)
        agg, mask = plan.decode(received)
        assert plan.decode_status() == 0
        assert mask.cpu().numpy().nonzero()[0].tolist() == nodes
        want = so.plain_sum(G_cpu.numpy())
        tol = AGG_TOL if m <= 10 else 1e-2      # m = 12 is past the float32 budget (the paper warns above 14)
        assert np.abs(agg.cpu().numpy() - want).max() <= tol * max(np.abs(want).max(), 1e-30)


def _random_plan(rng):
    """A feasible (P, s, m, r, d): m up to 12, s up to 5, r anywhere from the bound 2 s + m to P, ragged d."""
    while True:
        P = int(rng.integers(3, 70))
        m = int(rng.integers(1, 13))
        if m > P:
            continue
        s = int(rng.integers(0, min(5, (P - m) // 2) + 1))
        r = int(rng.integers(2 * s + m, P + 1))
        d = int(rng.integers(1, 40_000))
        return P, s, m, r, d


@pytest.mark.parametrize("case", range(24))
def test_random_plans_and_placements(case):
    """Seeded random plans (group size above the bound too, d not a multiple of m or of 4), a random number of
    attackers (0..s) in every group, random attack kinds: mask bit-exact, aggregate within the bar of the plain
    float64 sum and of the oracle's own decode of the same received matrix."""
    rng = np.random.default_rng(9000 + case)
    P, s, m, r, d = _random_plan(rng)
    sizes = so.group_sizes(P, r)
    w = so.node_scalars(sizes)
    g = torch.Generator().manual_seed(9000 + case)
    G_cpu = torch.empty((P, d), dtype=torch.float32).normal_(0.0, float(10.0 ** rng.uniform(-3, 1)), generator=g)
    with binding.Plan(P, s, m, r, d, seed=case) as plan:
        assert plan.group_sizes() == sizes
        coded = plan.encode(G_cpu.cuda())
        _check_encode(plan, G_cpu, coded, m, sizes, w)
        Z = coded.cpu().numpy()
        R = Z.copy()
        nodes = []
        scale_z = float(np.abs(Z).max()) + 1e-30
        for start, size in zip(so.group_starts(sizes), sizes):
            n_byz = int(rng.integers(0, s + 1))
            for k in sorted((start + rng.permutation(size)[:n_byz]).tolist()):
                kind = rng.integers(0, 4)
                if kind == 0:
                    R[k] = rng.normal(scale=100.0 * scale_z, size=Z.shape[1])
                elif kind == 1:
                    R[k] = -10.0 * Z[k]
                elif kind == 2:
                    R[k] = -Z.mean(0) + scale_z          # shifted so that it cannot coincide with the honest row
                else:
                    R[k, rng.integers(Z.shape[1])] += 1000.0 * scale_z
                nodes.append(k)
        R = R.astype(np.float32)
        want_mask = so.true_mask(R, Z)
        assert want_mask.nonzero()[0].tolist() == nodes
        agg, mask = plan.decode(torch.from_numpy(R).cuda())
        assert plan.decode_status() == 0
        assert np.array_equal(mask.cpu().numpy(), want_mask)
        want = so.plain_sum(G_cpu.numpy())
        scale = np.abs(want).max()
        got = agg.cpu().numpy().astype(np.float64)
        assert np.abs(got - want).max() <= AGG_TOL * scale, (P, s, m, r, d, np.abs(got - want).max() / scale)
        if s > 0:
            u, o_mask, o_status = so.decode(R, d, m, s, sizes, w, plan.projection_vectors(), tau=TAU)
            assert o_status == 0 and np.array_equal(o_mask, want_mask)
            assert np.abs(got - u).max() <= AGG_TOL * scale


def test_all_attackers_in_one_group_and_every_count():
    base = synth.Workload("placement", 45, 3, 5, 50_001, "normal", 1.0, "alie", 3, 321)
    sizes, w = _oracle_plan(base)
    G_cpu = synth.make_grads(base, "cpu")
    want = so.plain_sum(G_cpu.numpy())
    with binding.Plan(base.P, base.s, base.m, base.r, base.d, seed=1) as plan:
        coded = plan.encode(G_cpu.cuda())
        for nodes in ([], [0], [44], [12, 13], [33, 34, 35], [12, 22, 23], [0, 11, 44], [1, 5, 9, 13, 20, 25, 34, 40, 44]):
            wl = dataclasses.replace(base, n_byz=len(nodes), fixed_byz=tuple(nodes), attack="alie" if nodes else "none")
            received, _ = synth.apply_attack(wl, coded)
            agg, mask = plan.decode(received)
            assert plan.decode_status() == 0      # up to s = 3 per group, nine in total in the last case
            assert mask.cpu().numpy().nonzero()[0].tolist() == nodes
            assert np.abs(agg.cpu().numpy() - want).max() <= AGG_TOL * np.abs(want).max()


@pytest.mark.parametrize("P,s,d", [(9, 2, 20_001), (45, 3, 100_003), (105, 5, 30_000)])
def test_m1_is_the_repetition_code_with_majority_vote(P, s, d):
    """r_c = 1: W_j = I_d, every node of a group sends the same vector (bit for bit), and the decode equals the
    oracle's majority vote over the very same received matrix: same flagged set, the sum of the groups' majority
    vectors within the float32 roundings of adding q terms."""
    wl = synth.Workload("rep", P, s, 1, d, "normal", 1.0, "gaussian", s, 4242 + P)
    sizes, w = _oracle_plan(wl)
    G_cpu = synth.make_grads(wl, "cpu")
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=3) as plan:
        coded = plan.encode(G_cpu.cuda())
        for start, size in zip(so.group_starts(sizes), sizes):
            assert bool((coded[start:start + size] == coded[start]).all())
        received, nodes = synth.apply_attack(wl, coded)
        agg, mask = plan.decode(received)
        assert plan.decode_status() == 0
        R = received.cpu().numpy()
        u, o_mask, o_status = so.majority_decode(R, wl.s, sizes)
        assert o_status == 0 and o_mask.nonzero()[0].tolist() == nodes
        assert np.array_equal(mask.cpu().numpy(), o_mask)
        bound = 1.001 * len(sizes) * 2.0 ** -24 * np.abs(G_cpu.numpy().astype(np.float64)).sum(0)
        assert np.all(np.abs(agg.cpu().numpy().astype(np.float64) - u) <= bound + 1e-30)


def test_non_finite_rows_are_located():
    wl = synth.Workload("nan", 15, 2, 5, 20_000, "normal", 1.0, "none", 0, 11)
    G_cpu = synth.make_grads(wl, "cpu")
    want = so.plain_sum(G_cpu.numpy())
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d) as plan:
        coded = plan.encode(G_cpu.cuda())
        received = coded.clone()
        received[4] = float("nan")
        received[9, 17] = float("inf")
        agg, mask = plan.decode(received)
        assert plan.decode_status() == 0
        assert mask.cpu().numpy().nonzero()[0].tolist() == [4, 9]
        assert np.abs(agg.cpu().numpy() - want).max() <= AGG_TOL * np.abs(want).max()


def test_more_than_s_attackers_reports_undecodable():
    wl = synth.Workload("over", 9, 2, 5, 10_000, "normal", 1.0, "gaussian", 3, 5, fixed_byz=(1, 4, 7))
    G_cpu = synth.make_grads(wl, "cpu")
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d) as plan:
        coded = plan.encode(G_cpu.cuda())
        received, _ = synth.apply_attack(wl, coded)
        plan.decode(received)
        assert plan.decode_status() == binding.ERR_UNDECODABLE
        # the plan stays usable: a clean decode afterwards succeeds
        agg, mask = plan.decode(coded)
        assert plan.decode_status() == 0 and int(mask.sum()) == 0


def test_decode_is_bit_reproducible_and_reusable():
    wl = synth.small_variant(synth.WORKLOADS["vgg13"], 200_000)
    G = synth.make_grads(wl, "cuda")
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d) as plan:
        coded = plan.encode(G)
        received, nodes = synth.apply_attack(wl, coded)
        # with fresh projections every decode draws new vectors f: different projections, the same results
        plan.set_fresh_projections(True)
        a0, m0 = plan.decode(received)
        a0, m0 = a0.clone(), m0.clone()
        f0, r0 = plan.projection_vectors(), plan.projections()
        a1, m1 = plan.decode(received)
        a1, m1 = a1.clone(), m1.clone()
        f1, r1 = plan.projection_vectors(), plan.projections()
        assert not np.array_equal(f0, f1) and not np.array_equal(r0[0], r1[0])
        assert abs(f1.mean() - 1.0) < 0.02 and abs(f1.std() - 1.0) < 0.02 and abs(np.corrcoef(f0[0], f1[0])[0, 1]) < 0.02
        assert torch.equal(a0, a1) and torch.equal(m0, m1) and np.array_equal(r0[1], r1[1])
        # with the draw switched off the vectors stay and everything is bit-reproducible run to run
        plan.set_fresh_projections(False)
        a1, m1 = plan.decode(received)
        a1, m1 = a1.clone(), m1.clone()
        r1, f_kept = plan.projections(), plan.projection_vectors()
        a2, m2 = plan.decode(received)
        r2 = plan.projections()
        assert np.array_equal(plan.projection_vectors(), f_kept) and not np.array_equal(f_kept, f1)
        assert torch.equal(a1, a2) and torch.equal(m1, m2) and torch.equal(a0, a2)
        assert np.array_equal(r1[0], r2[0]) and np.array_equal(r1[1], r2[1])
        c2 = plan.encode(G)
        assert torch.equal(coded, c2)


def test_a_replayed_graph_of_a_decode_draws_new_vectors_each_time():
    """The count of the draws lives on the device: every replay of a captured decode projects with vectors of its own."""
    wl = synth.small_variant(synth.WORKLOADS["resnet18"], 90_001)
    G = synth.make_grads(wl, "cuda")
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=5) as plan:
        coded = plan.encode(G)
        received, nodes = synth.apply_attack(wl, coded)
        agg = torch.empty(wl.d, dtype=torch.float32, device="cuda")
        mask = torch.empty(wl.P, dtype=torch.uint8, device="cuda")
        plan.set_fresh_projections(True)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            plan.set_stream(side)
            for _ in range(2):
                plan.decode(received, agg, mask)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            plan.set_stream(torch.cuda.current_stream())
            plan.decode(received, agg, mask)
        plan.set_stream(torch.cuda.current_stream())
        seen = []
        for _ in range(3):
            graph.replay()
            torch.cuda.synchronize()
            assert plan.decode_status() == 0 and mask.nonzero().flatten().tolist() == nodes
            f = plan.projection_vectors()
            rho, _ = plan.projections()
            assert np.allclose(rho, so.project(received.cpu().numpy(), f), rtol=0, atol=1e-5 * np.abs(rho).max())   # these are the vectors it used
            seen.append(f)
        assert not np.array_equal(seen[0], seen[1]) and not np.array_equal(seen[1], seen[2]) and not np.array_equal(seen[0], seen[2])


def test_plan_status_after_encode_and_argument_errors_leave_the_plan_usable():
    """solon_plan_status reports the sticky wait-expired bit without a decode (OK here: no wait ever runs out), and calls
    refused for their arguments enqueue nothing: the next decode is unaffected."""
    wl = synth.small_variant(synth.WORKLOADS["vgg13"], 120_000)
    G = synth.make_grads(wl, "cuda")
    want = so.plain_sum(G.cpu().numpy())
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d) as plan:
        coded = plan.encode(G)
        assert plan.status() == binding.OK
        received, nodes = synth.apply_attack(wl, coded)
        from ctypes import c_void_p
        lib = binding.lib()
        agg = torch.empty(wl.d, dtype=torch.float32, device="cuda")
        mask = torch.empty(wl.P, dtype=torch.uint8, device="cuda")
        assert lib.solon_decode(plan._h, c_void_p(received.data_ptr()), c_void_p(agg.data_ptr()), c_void_p(0)) == binding.ERR_INVALID_ARG
        assert lib.solon_decode(plan._h, c_void_p(received.data_ptr() + 4), c_void_p(agg.data_ptr()), c_void_p(mask.data_ptr())) == binding.ERR_INVALID_ARG
        for _ in range(2):
            plan.decode(received, agg, mask)
            assert plan.decode_status() == 0 and plan.status() == binding.OK
            assert mask.nonzero().flatten().tolist() == nodes
            assert np.abs(agg.cpu().numpy() - want).max() <= AGG_TOL * np.abs(want).max()


def test_projection_settings():
    wl = synth.small_variant(synth.WORKLOADS["resnet18"], 60_000)
    G = synth.make_grads(wl, "cuda")
    want = so.plain_sum(G.cpu().numpy())
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=3) as plan:
        coded = plan.encode(G)
        received, nodes = synth.apply_attack(wl, coded)
        f2 = plan.projection_vectors()
        assert abs(f2.mean() - 1.0) < 0.02 and abs(f2.std() - 1.0) < 0.02     # f ~ N(1, I)
        for K in (1, 3, 4, 2):
            plan.set_num_projections(K)
            assert plan.projection_vectors().shape == (K, plan.d_c)
            agg, mask = plan.decode(received)
            assert plan.decode_status() == 0 and mask.cpu().numpy().nonzero()[0].tolist() == nodes
            assert np.abs(agg.cpu().numpy() - want).max() <= AGG_TOL * np.abs(want).max()
        plan.reseed(12345)
        f_new = plan.projection_vectors()
        assert not np.array_equal(f_new, f2)
        agg, mask = plan.decode(received)
        assert plan.decode_status() == 0 and mask.cpu().numpy().nonzero()[0].tolist() == nodes


def test_step_host_matches_device_path():
    wl = synth.small_variant(synth.WORKLOADS["resnet18"], 300_007)
    G_cpu = synth.make_grads(wl, "cpu").pin_memory()
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d) as plan:
        coded = plan.encode(G_cpu.cuda())
        nodes = synth.byzantine_nodes(wl)
        rows = synth.byzantine_rows(wl, coded, nodes).cpu().pin_memory()
        agg_h = torch.empty(wl.d, dtype=torch.float32).pin_memory()
        mask_h = torch.empty(wl.P, dtype=torch.uint8).pin_memory()
        status = plan.step_host(G_cpu, nodes, rows, agg_h, mask_h)
        assert status == 0
        assert mask_h.numpy().nonzero()[0].tolist() == nodes
        want = so.plain_sum(G_cpu.numpy())
        assert np.abs(agg_h.numpy() - want).max() <= AGG_TOL * np.abs(want).max()


@pytest.mark.parametrize("dtype", ["f32", "f64"])
@pytest.mark.parametrize("d", [40_000, 40_001, 40_002, 40_003, 77, 70, 66, 5])
def test_overwrite_rows(d, dtype):
    """Rows that start on 16-byte boundaries or not: every offset between a source row's and a destination row's boundaries
    occurs among the rows below for the odd widths (the copy realigns), and short rows go element by element."""
    tdtype = torch.float32 if dtype == "f32" else torch.float64
    with binding.Plan(15, 2, 1, 5, d, dtype=dtype) as plan:      # m = 1: d_c = d
        g = torch.Generator(device="cuda").manual_seed(3)
        matrix = torch.randn(15, d, device="cuda", generator=g, dtype=tdtype)
        before = matrix.clone()
        rows = torch.randn(6, d, device="cuda", generator=g, dtype=tdtype)
        nodes = torch.tensor([14, 0, 99, 7, 9, 2], dtype=torch.int32, device="cuda")      # 99: out of range, skipped
        plan.overwrite_rows(matrix, nodes, rows)
        torch.cuda.synchronize()
        want = before.clone()
        want[14], want[0], want[7], want[9], want[2] = rows[0], rows[1], rows[3], rows[4], rows[5]
        assert torch.equal(matrix, want)
        plan.overwrite_rows(matrix, nodes[:0], rows[:0])                             # nothing to do
        assert torch.equal(matrix, want)


def test_argument_checks():
    with binding.Plan(8, 1, 2, 4, 64) as plan:
        lib = binding.lib()
        assert lib.solon_encode(plan._h, None, None) == binding.ERR_INVALID_ARG
        assert lib.solon_decode(plan._h, None, None, None) == binding.ERR_INVALID_ARG
        buf = torch.zeros(8 * 64 + 4, dtype=torch.float32, device="cuda")
        out = torch.zeros(8 * 32, dtype=torch.float32, device="cuda")
        import ctypes
        misaligned = ctypes.c_void_p(buf.data_ptr() + 4)
        assert lib.solon_encode(plan._h, misaligned, ctypes.c_void_p(out.data_ptr())) == binding.ERR_INVALID_ARG
    for args in ((15, 5, 10, 15, 100), (8, 1, 2, 3, 64), (8, 1, 2, 9, 64), (0, 0, 1, 1, 1), (300, 1, 2, 200, 64)):
        with pytest.raises(binding.SolonError):
            binding.Plan(*args)
