"""CPU-only checks of the C-ABI library: it loads, exports what the header declares, and its host-side
logic (feasibility, group layout, node scalars, the host build of the locator) agrees with the oracle."""

import os
import re

import numpy as np
import pytest

from oracle import solon_oracle as so
from paper_2110_01595_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "solon.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(solon_[a-z_0-9]+)\s*\(", header))
    assert declared, "no declarations found"
    lib = binding.lib()
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in solon.h but not exported"
    assert declared == set(binding.SIGNATURES), declared ^ set(binding.SIGNATURES)


def test_strerror_and_missing_device():
    import torch
    assert binding.strerror(0) == "ok"
    assert "infeasible" in binding.strerror(binding.ERR_INFEASIBLE)
    if not torch.cuda.is_available():
        # without a device the plan must fail loudly, never fall back
        with pytest.raises(binding.SolonError) as err:
            binding.Plan(8, 1, 2, 4, 64)
        assert err.value.status == binding.ERR_CUDA


def test_check_params_matches_oracle_feasibility():
    for P in range(1, 20):
        for s in range(0, 6):
            for m in range(1, 8):
                for r in range(1, P + 2):
                    try:
                        so.check_plan(P, s, m, r, 10)
                        want_ok = True
                    except ValueError:
                        want_ok = False
                    got = binding.solon_check_params(P, s, m, r, 10)
                    assert (got == 0) == want_ok, (P, s, m, r, got)
                    if 2 * s + m > P:
                        assert got == binding.ERR_INFEASIBLE
    assert binding.solon_check_params(4, 1, 2, 4, 2) == 0          # the introduction's example
    assert binding.solon_check_params(4, 1, 2, 3, 2) == binding.ERR_INVALID_ARG
    assert binding.solon_check_params(15, 5, 10, 15, 100) == binding.ERR_INFEASIBLE


def test_group_layout_and_node_scalars_match_oracle():
    for P in (4, 8, 15, 45, 100, 105):
        for r in range(1, min(P, 40) + 1):
            sizes = so.group_sizes(P, r)
            starts = binding.solon_group_layout(P, r)
            assert starts == so.group_starts(sizes) + [P]
            assert np.allclose(binding.solon_node_scalars(P, r), so.node_scalars(sizes), rtol=0, atol=1e-15)


def _attack(kind, Z, nodes, rng):
    R = Z.copy()
    if kind == "gaussian":
        R[nodes] = rng.normal(scale=100.0, size=(len(nodes), Z.shape[1]))
    elif kind == "flip10":
        R[nodes] = -10.0 * Z[nodes]
    elif kind == "neg_mean":
        R[nodes] = -Z.mean(0)
    elif kind == "alie":
        R[nodes] = Z.mean(0) + 1.5 * Z.std(0)
    elif kind == "nan":
        R[nodes] = np.nan
    elif kind == "inf":
        R[nodes, 0] = np.inf
    return R


CASES = [(15, 2, 5), (12, 1, 10), (20, 5, 10), (11, 3, 5), (4, 1, 2), (15, 5, 2), (9, 2, 1), (23, 5, 10), (14, 1, 8)]


@pytest.mark.parametrize("n,s,m", CASES)
def test_host_locator_matches_oracle_on_fp32_coded_vectors(n, s, m):
    """Same projected values in, same located set out as the oracle's incremental locator and the truth;
    the recovery table reproduces the group sum within the float32 error budget."""
    rng = np.random.default_rng(1000 * n + 10 * s + m)
    sizes = [n]
    w = so.node_scalars(sizes)
    d = 600 * m + 1
    G = rng.normal(size=(n, d)).astype(np.float32)
    Z = so.encode(G, m, sizes, w).astype(np.float32)
    f = (1.0 + rng.normal(size=(2, Z.shape[1]))).astype(np.float32)
    want = so.plain_sum(G)
    for kind in ("gaussian", "flip10", "neg_mean", "alie", "nan", "inf"):
        if kind == "alie" and m == 1:
            continue
        for n_byz in range(0, s + 1):
            nodes = sorted(rng.permutation(n)[:n_byz].tolist())
            R = _attack(kind, Z.astype(np.float64), nodes, rng).astype(np.float32)
            with np.errstate(invalid="ignore", over="ignore"):
                rho = so.project(R, f)
                nu = so.row_energy(R)
            status, mask, t, rows, coeff = binding.solon_locate_host(rho, nu, w, m, s, 1e-5)
            assert status == 0, (kind, nodes)
            assert mask.nonzero()[0].tolist() == nodes, (kind, nodes, mask)
            assert t == len(nodes)
            if kind not in ("nan", "inf"):
                tol = so.detection_tolerance(nu, 1e-5)
                V, t_or = so.phi_incremental(rho, w, m, s, tol)
                assert V == nodes and t_or == t
            # recovery rows are trusted nodes only, and the table inverts the code
            assert not set(rows.tolist()) & set(nodes)
            assert len(rows) == (m if m <= 6 else n - len(nodes))
            Wm = so.w_hat(w, m - 1)[rows]
            assert np.allclose(coeff.T @ Wm, np.eye(m), atol=1e-8)
            u = (coeff.T @ R[rows].astype(np.float64)).T.reshape(-1)[:d]
            assert np.abs(u - want).max() <= 1e-4 * np.abs(want).max(), (kind, nodes)


def test_host_locator_projection_count_and_exact_data():
    """K = 1 (the paper's single f) and K = 4 give the same answer; exact float64 coded vectors pass tau = 1e-9."""
    rng = np.random.default_rng(77)
    n, s, m = 13, 3, 4
    w = so.node_scalars([n])
    G = rng.normal(size=(n, 40 * m))
    Z = so.encode(G, m, [n], w)
    nodes = [1, 6, 12]
    R = _attack("gaussian", Z, nodes, rng)
    for K in (1, 2, 3, 4):
        f = 1.0 + rng.normal(size=(K, Z.shape[1]))
        status, mask, t, rows, coeff = binding.solon_locate_host(so.project(R, f), so.row_energy(R), w, m, s, 1e-9)
        assert status == 0 and mask.nonzero()[0].tolist() == nodes and t == 3


def test_host_locator_rejects_more_than_s_attackers():
    rng = np.random.default_rng(5)
    for n, s, m in ((8, 2, 4), (4, 1, 2), (12, 5, 2), (9, 2, 5)):
        w = so.node_scalars([n])
        G = rng.normal(size=(n, 50 * m)).astype(np.float32)
        Z = so.encode(G, m, [n], w).astype(np.float32)
        f = (1.0 + rng.normal(size=(2, Z.shape[1]))).astype(np.float32)
        for trial in range(10):
            nodes = sorted(rng.permutation(n)[:s + 1].tolist())
            R = _attack("gaussian", Z.astype(np.float64), nodes, rng).astype(np.float32)
            status, mask, t, rows, coeff = binding.solon_locate_host(so.project(R, f), so.row_energy(R), w, m, s, 1e-5)
            assert status == binding.ERR_UNDECODABLE and t == -1


def test_host_locator_all_zero_data():
    n, s, m = 8, 2, 4
    w = so.node_scalars([n])
    rho = np.zeros((2, n))
    nu = np.zeros(n)
    status, mask, t, rows, coeff = binding.solon_locate_host(rho, nu, w, m, s, 1e-5)
    assert status == 0 and mask.sum() == 0 and t == 0
    rho[:, 3] = 1e-12                      # any deviation from all-zero honest data is a corruption
    nu[3] = 1e-24
    status, mask, t, rows, coeff = binding.solon_locate_host(rho, nu, w, m, s, 1e-5)
    assert status == 0 and mask.nonzero()[0].tolist() == [3]
