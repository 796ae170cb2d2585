"""GPU parity of the float64 boundary (solon_plan_create_ex with SOLON_F64; the paper's wire format, Table 2) against the
float64 oracle.  Bars: mask bit-exact; aggregate within 1e-9 of ||sum||_inf for m <= 5, 1e-6 at m = 10 (the oracle's own
agreement with the definition), 1e-4 at m = 12 and 14; coded values within a few float64 roundings of the sum of |terms|;
projections within float64 accumulation error."""

import dataclasses

import numpy as np
import pytest
import torch

from oracle import solon_oracle as so
from paper_2110_01595_b200 import binding, build, synth

pytestmark = pytest.mark.gpu

TAU = 1e-10                       # the library's default tolerance for float64 plans, also given to the oracle
EPS = 2.0 ** -53


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def _agg_tol(m):
    return 1e-9 if m <= 6 else (1e-6 if m <= 10 else 1e-4)


def _grads64(wl, device="cpu"):
    """The workload's float32 recipe widened to float64 and perturbed in the low bits, so that the values are not
    float32-representable (a path that narrowed them anywhere would lose nine digits)."""
    G = synth.make_grads(wl, device).double()
    gen = torch.Generator(device=device).manual_seed(wl.seed + 99)
    noise = torch.empty(G.shape, dtype=torch.float64, device=device).normal_(0.0, 1.0, generator=gen)
    return G * (1.0 + 1e-9 * noise)


def _check_encode(G_np, coded_gpu, m, sizes, w):
    Z = so.encode(G_np, m, sizes, w)
    bound = so.encode(np.abs(G_np), m, sizes, np.abs(w))          # sum of |terms| of every entry
    err = np.abs(coded_gpu.cpu().numpy() - Z)
    ops = np.zeros((Z.shape[0], 1))
    for start, size in zip(so.group_starts(sizes), sizes):
        ops[start:start + size] = size + m
    # float64 group sum (r_g - 1 roundings), Horner (m), final rounding; the oracle itself rounds as often
    assert np.all(err <= 2.0 * ops * EPS * bound + 1e-300), float((err / (EPS * bound + 1e-300)).max())
    return Z


def _run_case(wl, check_intermediates=True):
    sizes = so.group_sizes(wl.P, wl.r)
    w = so.node_scalars(sizes)
    G_cpu = _grads64(wl)
    G_np = G_cpu.numpy()
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=wl.seed, dtype="f64") as plan:
        assert plan.group_sizes() == sizes
        coded = plan.encode(G_cpu.cuda())
        assert coded.dtype == torch.float64
        if check_intermediates:
            _check_encode(G_np, coded, wl.m, sizes, w)
        received, nodes = synth.apply_attack(wl, coded)
        agg, mask = plan.decode(received)
        status = plan.decode_status()
        assert status == 0, binding.strerror(status)
        R = received.cpu().numpy()
        want_mask = so.true_mask(R, coded.cpu().numpy())
        assert want_mask.nonzero()[0].tolist() == nodes
        assert np.array_equal(mask.cpu().numpy(), want_mask)                       # bit-exact
        want = so.plain_sum(G_np)
        scale = np.abs(want).max()
        got = agg.cpu().numpy()
        assert got.dtype == np.float64
        err = np.abs(got - want).max() / scale
        assert err <= _agg_tol(wl.m), err
        f = plan.projection_vectors()
        u, o_mask, o_status = so.decode(R, wl.d, wl.m, wl.s, sizes, w, f, tau=TAU)
        assert o_status == 0 and np.array_equal(o_mask, want_mask)
        assert np.abs(got - u).max() <= _agg_tol(wl.m) * scale
        if check_intermediates and wl.s > 0:
            rho, nu = plan.projections()
            o_rho, o_nu = so.project(R, f), so.row_energy(R)
            lim = np.sqrt((f.astype(np.float64) ** 2).sum(1))[:, None] * np.sqrt(o_nu)[None, :]
            assert np.all(np.abs(rho - o_rho) <= 1e-12 * lim + 1e-300)             # float64 products and sums, another order
            assert np.allclose(nu, o_nu, rtol=1e-12)
        return err


def test_config_tiny():
    _run_case(synth.WORKLOADS["tiny"])


def test_config_resnet18_shape_small():
    _run_case(synth.small_variant(synth.WORKLOADS["resnet18"], 1_117_397))      # many tiles, d % m != 0, rows off 16 bytes


def test_config_vgg13_shape_small():
    _run_case(synth.small_variant(synth.WORKLOADS["vgg13"], 283_321))
    _run_case(synth.small_variant(synth.WORKLOADS["vgg13_clean"], 283_321))


def test_config_lsq_shape():
    """The least-squares configuration's plan and attack on float64 gradients (the gradients themselves come from the
    oracle here: solon_lsq_grads is a float32 call)."""
    wl = dataclasses.replace(synth.WORKLOADS["lsq"], d=20_003, lsq_rows=32)
    sizes = so.group_sizes(wl.P, wl.r)
    w = so.node_scalars(sizes)
    X, y, wvec = synth.make_lsq_problem(wl, "cpu")
    G_np = so.lsq_grads(X.numpy(), y.numpy(), wvec.numpy(), wl.lsq_rows)
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=wl.seed, dtype="f64") as plan:
        coded = plan.encode(torch.from_numpy(G_np).cuda())
        _check_encode(G_np, coded, wl.m, sizes, w)
        received, nodes = synth.apply_attack(wl, coded)
        agg, mask = plan.decode(received)
        assert plan.decode_status() == 0
        assert mask.cpu().numpy().nonzero()[0].tolist() == nodes and len(nodes) == 1
        want = so.plain_sum(G_np)
        assert np.abs(agg.cpu().numpy() - want).max() <= 1e-9 * np.abs(want).max()


@pytest.mark.parametrize("P,s,m", [(15, 1, 1), (15, 1, 2), (15, 1, 5), (15, 1, 10), (15, 3, 5), (15, 5, 2), (45, 1, 10),
                                   (45, 3, 1), (45, 5, 10), (105, 1, 1), (105, 3, 5), (105, 5, 10), (30, 2, 3), (30, 2, 4),
                                   (30, 1, 6), (40, 2, 8), (45, 1, 12), (45, 2, 14), (15, 0, 14)])
def test_sweep_shapes(P, s, m):
    wl = synth.Workload(f"f64_P{P}_s{s}_m{m}", P, s, m, 100_003, "normal", 1.0, "gaussian" if s else "none", s, 6000 + P + 10 * s + m)
    _run_case(wl)


@pytest.mark.parametrize("P,s,m,r,d", [
    (4, 1, 2, 4, 2),          # the introduction's example: d_c = 1
    (5, 1, 3, 5, 1),          # d < m: one padded chunk
    (9, 2, 1, 5, 1001),       # m = 1, odd d: rows start off 16-byte boundaries
    (16, 2, 4, 8, 4096),      # r divides P
    (23, 1, 3, 23, 777),      # one odd-sized group
    (256, 1, 2, 4, 10_007),   # 64 groups of four
    (126, 16, 1, 126, 301),   # most adversaries per group allowed
])
def test_edge_shapes(P, s, m, r, d):
    wl = synth.Workload("edge64", P, s, m, d, "normal", 1.0, "gaussian", s, 199)
    sizes = so.group_sizes(P, r)
    w = so.node_scalars(sizes)
    G_cpu = _grads64(wl)
    with binding.Plan(P, s, m, r, d, seed=7, dtype="f64") as plan:
        coded = plan.encode(G_cpu.cuda())
        _check_encode(G_cpu.numpy(), coded, m, sizes, w)
        received, nodes = synth.apply_attack(wl, coded)
        agg, mask = plan.decode(received)
        assert plan.decode_status() == 0
        assert mask.cpu().numpy().nonzero()[0].tolist() == nodes
        want = so.plain_sum(G_cpu.numpy())
        assert np.abs(agg.cpu().numpy() - want).max() <= _agg_tol(m) * max(np.abs(want).max(), 1e-300)


def test_dtype_is_a_property_of_the_plan():
    lib = binding.lib()
    assert [m for m in range(1, 17) if lib.solon_float64_m_supported(m)] == [1, 2, 3, 4, 5, 6, 8, 10, 12, 14]
    with pytest.raises(binding.SolonError) as err:
        binding.Plan(15, 1, 7, 9, 1000, dtype="f64")                 # no float64 kernel for m = 7
    assert err.value.status == binding.ERR_INVALID_ARG
    G32 = torch.zeros((8, 64), dtype=torch.float32, device="cuda")
    G64 = G32.double()
    with binding.Plan(8, 1, 2, 4, 64, dtype="f64") as p64, binding.Plan(8, 1, 2, 4, 64) as p32:
        assert lib.solon_plan_dtype(p64._h) == binding.F64 and lib.solon_plan_dtype(p32._h) == binding.F32
        with pytest.raises(ValueError):
            p64.encode(G32)                                          # the binding checks tensor types against the plan
        c64 = torch.zeros((8, 32), dtype=torch.float64, device="cuda")
        c32 = torch.zeros((8, 32), dtype=torch.float32, device="cuda")
        from ctypes import c_void_p
        # and the library refuses the calls of the other element type
        assert lib.solon_encode(p64._h, c_void_p(G32.data_ptr()), c_void_p(c32.data_ptr())) == binding.ERR_INVALID_ARG
        assert lib.solon_encode_f64(p32._h, c_void_p(G64.data_ptr()), c_void_p(c64.data_ptr())) == binding.ERR_INVALID_ARG
        agg = torch.zeros(64, dtype=torch.float32, device="cuda")
        mask = torch.zeros(8, dtype=torch.uint8, device="cuda")
        assert lib.solon_decode(p64._h, c_void_p(c32.data_ptr()), c_void_p(agg.data_ptr()), c_void_p(mask.data_ptr())) == binding.ERR_INVALID_ARG


def test_undecodable_and_host_step():
    wl = synth.Workload("over64", 9, 2, 5, 30_000, "normal", 1.0, "gaussian", 3, 5, fixed_byz=(1, 4, 7))
    G_cpu = _grads64(wl)
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, dtype="f64") as plan:
        coded = plan.encode(G_cpu.cuda())
        received, _ = synth.apply_attack(wl, coded)
        plan.decode(received)
        assert plan.decode_status() == binding.ERR_UNDECODABLE       # s + 1 attackers in a group of 2 s + m
        # the host-buffer step with two attackers
        nodes = [1, 7]
        rows_host = received[nodes].cpu().contiguous()
        agg_host = torch.empty(wl.d, dtype=torch.float64)
        mask_host = torch.empty(wl.P, dtype=torch.uint8)
        status = plan.step_host(G_cpu.contiguous(), nodes, rows_host, agg_host, mask_host)
        assert status == 0 and mask_host.nonzero().flatten().tolist() == nodes
        want = so.plain_sum(G_cpu.numpy())
        assert np.abs(agg_host.numpy() - want).max() <= 1e-9 * np.abs(want).max()


def test_full_size_resnet18_float64():
    """The ResNet-18-sized configuration with 8-byte elements (the 89.6 MB per worker of the paper's Table 2), in the
    launch configuration the benchmark times: mask exact, sampled coded chunks and aggregate coordinates against the
    oracle, the whole aggregate against a device-side float64 sum."""
    wl = synth.WORKLOADS["resnet18"]
    sizes = so.group_sizes(wl.P, wl.r)
    w = so.node_scalars(sizes)
    G = _grads64(wl, "cuda")
    with binding.Plan(wl.P, wl.s, wl.m, wl.r, wl.d, seed=wl.seed, dtype="f64") as plan:
        coded = plan.encode(G)
        received, nodes = synth.apply_attack(wl, coded)
        agg, mask = plan.decode(received)
        assert plan.decode_status() == 0
        assert mask.cpu().numpy().nonzero()[0].tolist() == nodes
        ref = G.sum(dim=0)
        scale = float(ref.abs().max())
        assert float((agg - ref).abs().max()) <= 1e-9 * scale
        rng = np.random.default_rng(wl.seed)
        chunks = np.unique(np.concatenate([rng.integers(0, plan.d_c, size=2000), [0, 1, 255, 256, plan.d_c - 2, plan.d_c - 1]]))
        cols = (chunks[:, None] * wl.m + np.arange(wl.m)[None, :]).reshape(-1)
        in_range = cols < wl.d
        G_s = np.zeros((wl.P, cols.size))
        G_s[:, in_range] = G[:, torch.from_numpy(cols[in_range]).cuda()].cpu().numpy()
        Z_s = so.encode(G_s, wl.m, sizes, w)
        bound = so.encode(np.abs(G_s), wl.m, sizes, np.abs(w))
        got_Z = coded[:, torch.from_numpy(chunks).cuda()].cpu().numpy()
        assert np.all(np.abs(got_Z - Z_s) <= 2.0 * (max(sizes) + wl.m) * EPS * bound + 1e-300)
        got = agg[torch.from_numpy(cols[in_range]).cuda()].cpu().numpy()
        assert np.abs(got - so.plain_sum(G_s)[in_range]).max() <= 1e-9 * scale
