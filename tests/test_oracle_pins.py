"""Pins for the float64 oracle: what the paper and the mathematics fix, independent of the oracle's code."""

import itertools
import math
import os

import numpy as np
import pytest

from oracle import solon_oracle as so

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _plan(P, s, m, r=None):
    r = so.redundancy_bound(s, m) if r is None else r
    sizes = so.group_sizes(P, r)
    return sizes, so.node_scalars(sizes)


def _rows(path):
    with open(path) as fh:
        return [ln.split() for ln in fh if ln.strip() and not ln.startswith("#")]


# ---------------------------------------------------------------- feasibility


def test_intro_example_feasibility():
    """Introduction's example: P=4, d=2, r=4, r_c=2 tolerates s=1 because 4 >= 2*1+2."""
    for P, d, r, r_c, s, ok in _rows(os.path.join(GOLDEN, "intro_example.txt")):
        P, d, r, r_c, s, ok = map(int, (P, d, r, r_c, s, ok))
        if ok:
            so.check_plan(P, s, r_c, r, d)
        else:
            with pytest.raises(ValueError):
                so.check_plan(P, s, r_c, r, d)


def test_redundancy_bound_and_corollary():
    """Theorem 2: r >= 2s + r_c; corollary: s <= (P - r_c)/2."""
    for P in range(1, 24):
        for m in range(1, P + 1):
            s_max = so.max_adversaries(P, m)
            assert 2 * s_max + m <= P < 2 * (s_max + 1) + m
            for s in range(0, s_max + 2):
                r = so.redundancy_bound(s, m)
                if s <= s_max:
                    so.check_plan(P, s, m, r, 10)
                    with pytest.raises(ValueError):
                        so.check_plan(P, s, m, r - 1, 10)
                else:
                    with pytest.raises(ValueError):
                        so.check_plan(P, s, m, min(r, P), 10)


def test_table2_message_sizes():
    """Table 2: a worker sends size / r_c bytes, i.e. d_c = d / r_c elements."""
    for model, size, rc6, rc8, rc10 in _rows(os.path.join(GOLDEN, "table2_message_sizes.txt")):
        d = round(float(size) * 1e6 / 8)
        for r_c, printed in ((6, rc6), (8, rc8), (10, rc10)):
            mb = so.coded_length(d, r_c) * 8 / 1e6
            decimals = len(printed.split(".")[1])
            # the printed rows are rounded to three digits and not mutually consistent beyond 0.3 %
            slack = 3e-3 * float(printed) + 0.5 * 10.0 ** (-decimals)
            assert abs(mb - float(printed)) <= slack, (model, r_c, mb, printed)


def test_groups_reduce_to_paper_when_r_divides_P():
    assert so.group_sizes(100, 20) == [20] * 5          # Section 4: 5 groups of 20
    assert so.group_sizes(45, 11) == [12, 11, 11, 11]
    assert so.group_sizes(15, 9) == [15]
    for P in range(1, 60):
        for r in range(1, P + 1):
            sizes = so.group_sizes(P, r)
            assert sum(sizes) == P and min(sizes) >= r and max(sizes) - min(sizes) <= 1
            assert len(sizes) == P // r
    A = so.allocation_matrix(8, [4, 4])
    assert np.array_equal(A, np.kron(np.eye(2), np.ones((4, 4))))


def test_node_scalars_distinct_nonzero():
    for r_j in range(1, 130):
        w = so.node_scalars([r_j])
        assert np.all(w != 0.0) and len(set(np.round(w, 14))) == r_j
        assert np.all(np.abs(w) < 1.0)


# ---------------------------------------------------------------- encoder


def test_encode_equals_dense_kronecker():
    """z_j = W_j Y_j 1_P with W_j = I (x) [1, w_j, ...] built by numpy.kron and Y_j by the allocation matrix."""
    rng = np.random.default_rng(1)
    P, s, m, d = 8, 1, 2, 10
    sizes, w = _plan(P, s, m)
    G = rng.normal(size=(P, d))
    Z = so.encode(G, m, sizes, w)
    A = so.allocation_matrix(P, sizes)
    d_c = d // m
    for j in range(P):
        Y_j = (np.ones((d, 1)) @ A[j:j + 1]) * G.T            # d x P, zero where not allocated
        W_j = np.kron(np.eye(d_c), (w[j] ** np.arange(m))[None, :])
        assert np.allclose(Z[j], W_j @ (Y_j @ np.ones(P)), rtol=1e-13, atol=1e-13)


def test_encode_m1_is_group_sum():
    """r_c = 1: W_j = I_d, every node of a group sends the group's summed gradient (repetition code)."""
    rng = np.random.default_rng(2)
    P, s, m, d = 9, 1, 1, 17
    sizes, w = _plan(P, s, m)
    G = rng.normal(size=(P, d)).astype(np.float32)
    Z = so.encode(G, m, sizes, w)
    for start, size in zip(so.group_starts(sizes), sizes):
        ybar = G[start:start + size].astype(np.float64).sum(0)
        for k in range(start, start + size):
            assert np.array_equal(Z[k], ybar)


@pytest.mark.parametrize("P,s", [(9, 1), (7, 3), (15, 2), (10, 0)])
def test_majority_vote_is_the_m1_decoder(P, s):
    """r_c = 1: the repetition code.  The majority vote returns the plain sum (Definition 1) and the exact set of
    nodes that sent something else, and agrees with the general decoder (Algorithm 1) on the same received matrix;
    one attacker too many in a group leaves no majority."""
    rng = np.random.default_rng(40 + P + s)
    m, d = 1, 29
    sizes, w = _plan(P, s, m)
    G = rng.normal(size=(P, d)).astype(np.float32)
    Z = so.encode(G, m, sizes, w)
    f = 1.0 + rng.normal(size=(2, d))
    want = so.plain_sum(G)
    starts = so.group_starts(sizes)
    for n_byz in range(s + 1):
        nodes = sorted((starts[-1] + rng.permutation(sizes[-1])[:n_byz]).tolist())
        R = Z.copy()
        R[nodes] = rng.normal(scale=100.0, size=(len(nodes), d))
        u, mask, status = so.majority_decode(R, s, sizes)
        assert status == 0
        assert mask.nonzero()[0].tolist() == nodes
        assert np.abs(u - want).max() <= 1e-12 * np.abs(want).max()
        if s > 0:
            u2, mask2, status2 = so.decode(R, d, m, s, sizes, w, f)
            assert status2 == 0 and np.array_equal(mask2, mask)
            assert np.abs(u2 - u).max() <= 1e-9 * np.abs(want).max()
    if s > 0 and sizes[-1] == 2 * s + 1:
        # s + 1 different liars in a group of 2 s + 1: only s honest copies remain, fewer than r - s
        nodes = list(range(starts[-1], starts[-1] + s + 1))
        R = Z.copy()
        R[nodes] = rng.normal(scale=100.0, size=(len(nodes), d))
        assert so.majority_decode(R, s, sizes)[2] == -1
    # a colluding majority is believed: the vote itself cannot tell (the bound r >= 2 s + 1 is what rules it out)
    if s > 0:
        liars = list(range(starts[0], starts[0] + sizes[0] - s))
        R = Z.copy()
        R[liars] = 7.0
        u, mask, status = so.majority_decode(R, s, sizes)
        assert status == 0 and mask.nonzero()[0].tolist() == [k for k in range(starts[0], starts[0] + sizes[0]) if k not in liars]


def test_encode_padding_and_chunk_order():
    """d not divisible by r_c: the last chunk is zero padded; chunk p covers coordinates p r_c .. p r_c + r_c - 1."""
    P, s, m, d = 5, 1, 3, 7
    sizes, w = _plan(P, s, m)
    G = np.zeros((P, d))
    G[2, 4] = 1.0                              # coordinate 4 = chunk 1, offset 1
    G[0, 6] = 2.0                              # coordinate 6 = chunk 2, offset 0 (last, padded chunk)
    Z = so.encode(G, m, sizes, w)
    assert Z.shape == (P, 3)
    for k in range(P):
        assert np.allclose(Z[k], [0.0, w[k], 2.0])


def test_projection_is_the_polynomial_of_lemma9():
    """Lemma 9: f z_k = Q(w_k), Q(w) = sum_l u_{l+1} w^l, u_{l+1} = sum_p f_p ybar[l + p r_c] (explicit loops)."""
    rng = np.random.default_rng(3)
    P, s, m, d = 14, 2, 3, 31
    sizes, w = _plan(P, s, m)
    G = rng.normal(size=(P, d))
    d_c = so.coded_length(d, m)
    f = 1.0 + rng.normal(size=d_c)
    Z = so.encode(G, m, sizes, w)
    rho = so.project(Z, f)[0]
    for start, size in zip(so.group_starts(sizes), sizes):
        ybar = np.zeros(m * d_c)
        for i in range(start, start + size):
            for c in range(d):
                ybar[c] += G[i, c]
        u = [sum(f[p] * ybar[l + p * m] for p in range(d_c)) for l in range(m)]
        for k in range(start, start + size):
            Q = sum(u[l] * w[k] ** l for l in range(m))
            assert abs(rho[k] - Q) <= 1e-12 * (1 + abs(Q))


# ---------------------------------------------------------------- locator and decoder


ATTACKS = ("gaussian", "flip10", "neg_mean", "alie", "one_coordinate")


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
    elif kind == "one_coordinate":
        for k in nodes:
            R[k, rng.integers(Z.shape[1])] += 1.0
    return R


CASES = [  # P, s, m, d
    (8, 1, 2, 64), (15, 2, 5, 103), (45, 3, 5, 200), (15, 1, 3, 50), (12, 5, 2, 40),
    (20, 5, 10, 95), (7, 3, 1, 33), (15, 1, 10, 120), (9, 0, 4, 30),
]


@pytest.mark.parametrize("P,s,m,d", CASES)
def test_decode_recovers_plain_sum_under_any_attack(P, s, m, d):
    """Definition 1 / Theorem 5: D(Z + N) = G 1_P for every N with at most s non-zero columns."""
    rng = np.random.default_rng(100 * P + 10 * s + m)
    sizes, w = _plan(P, s, m)
    G = rng.normal(size=(P, d))
    Z = so.encode(G, m, sizes, w)
    f = 1.0 + rng.normal(size=(2, Z.shape[1]))
    want = so.plain_sum(G)
    scale = np.abs(want).max()
    bound = 1e-9 if m <= 5 else 1e-6
    for kind in ATTACKS:
        if kind == "alie" and m == 1:
            continue        # honest rows of a group coincide: mean + 1.5 * 0 is the honest vector up to rounding
        for n_byz in range(0, s + 1):
            # worst placement: all attackers inside one group
            start = so.group_starts(sizes)[-1]
            nodes = sorted((start + rng.permutation(sizes[-1])[:n_byz]).tolist())
            R = _attack(kind, Z, nodes, rng)
            u, mask, status = so.decode(R, d, m, s, sizes, w, f)
            assert status == 0
            assert np.array_equal(mask, so.true_mask(R, Z)), (kind, nodes, mask)
            assert np.abs(u - want).max() <= bound * scale, (kind, nodes)


@pytest.mark.parametrize("P,s,m", [(8, 1, 2), (15, 2, 5), (12, 3, 2), (20, 5, 10), (9, 2, 1)])
def test_paper_locator_matches_incremental_and_truth(P, s, m):
    """Section 3.4's fixed-s system (minimum-norm solve, polynomial division) finds {i : n_i != 0},
    also with fewer than s attackers (case (ii) of Lemma 9), and agrees with the incremental variant."""
    rng = np.random.default_rng(7 * P + s)
    sizes, w = _plan(P, s, m)
    d = 12 * m
    G = rng.normal(size=(P, d))
    Z = so.encode(G, m, sizes, w)
    f = 1.0 + rng.normal(size=(1, Z.shape[1]))
    for n_byz in range(0, s + 1):
        nodes = sorted(rng.permutation(sizes[0])[:n_byz].tolist())       # group 0
        R = _attack("gaussian", Z, nodes, rng)
        rho = so.project(R, f)[:, :sizes[0]]
        w_g = w[:sizes[0]]
        tol = 1e-7 * np.median(np.abs(rho))
        V_paper = so.phi_paper(rho[0], w_g, m, s, tol)
        V_inc, t = so.phi_incremental(rho, w_g, m, s, tol)
        assert V_paper == nodes and V_inc == nodes and t == n_byz


def test_locator_denominator_roots_are_corrupt_scalars():
    """Reed-Solomon view (proof of Lemma 9): with exactly t corrupt nodes the monic denominator
    is prod (w - w_{i_k}); its roots, found by numpy.roots, are the corrupt nodes' scalars."""
    rng = np.random.default_rng(11)
    P, s, m = 15, 3, 4
    sizes, w = _plan(P, s, m, r=15)
    G = rng.normal(size=(P, 40))
    Z = so.encode(G, m, sizes, w)
    f = 1.0 + rng.normal(size=(2, Z.shape[1]))
    nodes = [2, 7, 13]
    R = _attack("flip10", Z, nodes, rng)
    rho = so.project(R, f)
    A, b = so.locator_system(rho, w, m, 3)
    a = np.linalg.lstsq(A, b, rcond=None)[0]
    theta = a[-3:]
    roots = np.sort(np.roots(np.concatenate([[1.0], theta[::-1]])).real)
    assert np.allclose(roots, np.sort(w[nodes]), atol=1e-9)
    # numerator / denominator is the honest polynomial Q of Lemma 9 for each projection
    for kappa in range(2):
        num = a[kappa * (m + 3):(kappa + 1) * (m + 3)]
        quo, rem = np.polydiv(num[::-1], np.concatenate([[1.0], theta[::-1]]))
        honest = [k for k in range(P) if k not in nodes]
        assert np.allclose(np.polyval(quo, w[honest]), rho[kappa, honest], rtol=1e-9, atol=1e-9)
        assert np.abs(rem).max() < 1e-8 * np.abs(num).max()


def test_locator_matches_brute_force_on_tiny_groups():
    """Appendix C: enumerating subsets on the full received block gives the same set as the projected locator."""
    rng = np.random.default_rng(5)
    for P, s, m in ((8, 1, 2), (6, 2, 2), (7, 1, 5), (5, 2, 1)):
        sizes, w = _plan(P, s, m)
        G = rng.normal(size=(P, 8 * m))
        Z = so.encode(G, m, sizes, w)
        f = 1.0 + rng.normal(size=(2, Z.shape[1]))
        for g, (start, size) in enumerate(zip(so.group_starts(sizes), sizes)):
            for n_byz in range(0, s + 1):
                for nodes in itertools.combinations(range(size), n_byz):
                    R = _attack("gaussian", Z, [start + k for k in nodes], rng)
                    R_g = R[start:start + size]
                    w_g = w[start:start + size]
                    brute = so.brute_force_locate(R_g, w_g, m, s, 1e-9)
                    rho = so.project(R_g, f)
                    tol = so.detection_tolerance(so.row_energy(R_g), 1e-9)
                    V, _ = so.phi_incremental(rho, w_g, m, s, tol)
                    assert brute == list(nodes) == V


def test_more_than_s_attackers_is_never_silently_accepted():
    """s + 1 attackers in a group of size exactly 2 s + r_c: the decoder must not return status 0 with
    at most s flagged nodes AND a wrong sum."""
    rng = np.random.default_rng(9)
    for P, s, m in ((8, 1, 2), (9, 2, 5), (12, 5, 2)):
        sizes, w = _plan(P, s, m)
        G = rng.normal(size=(P, 10 * m))
        Z = so.encode(G, m, sizes, w)
        f = 1.0 + rng.normal(size=(2, Z.shape[1]))
        want = so.plain_sum(G)
        for trial in range(20):
            nodes = sorted(rng.permutation(sizes[0])[:s + 1].tolist())
            R = _attack("gaussian", Z, nodes, rng)
            u, mask, status = so.decode(R, G.shape[1], m, s, sizes, w, f)
            wrong = np.abs(u - want).max() > 1e-6 * np.abs(want).max()
            assert not (status == 0 and wrong)
            assert status == -1


def test_psi_same_result_for_every_admissible_U():
    """Lemma 4: any trusted set of at least r - s honest nodes gives the group's summed gradient;
    and C = ([W-hat]_{U'})^{-1} satisfies W-hat_{U'} C = I."""
    rng = np.random.default_rng(13)
    P, s, m, d = 9, 2, 5, 45
    sizes, w = _plan(P, s, m)
    G = rng.normal(size=(P, d))
    Z = so.encode(G, m, sizes, w)
    ybar = so.group_sum(G, 0, P, m)
    for U in itertools.combinations(range(P), P - s):
        assert np.allclose(so.psi(Z, w, m, list(U)), ybar, rtol=1e-9, atol=1e-9)
    for U_prime in itertools.combinations(range(P), m):
        C = so.inverse_rows(w, m, list(U_prime))
        assert np.allclose(so.w_hat(w, m - 1)[list(U_prime)] @ C, np.eye(m), atol=1e-9)
        chunks = (C @ Z[list(U_prime)]).T.reshape(-1)
        assert np.allclose(chunks, ybar, rtol=1e-8, atol=1e-8)


def test_honest_sender_is_not_flagged():
    """A node that sends exactly its honest vector is not in {i : n_i != 0}."""
    rng = np.random.default_rng(17)
    P, s, m = 8, 1, 2
    sizes, w = _plan(P, s, m)
    G = rng.normal(size=(P, 32))
    Z = so.encode(G, m, sizes, w)
    f = 1.0 + rng.normal(size=(2, Z.shape[1]))
    u, mask, status = so.decode(Z.copy(), 32, m, s, sizes, w, f)
    assert status == 0 and mask.sum() == 0
    assert np.allclose(u, so.plain_sum(G), rtol=1e-10, atol=1e-10)


def test_fp32_rounded_coded_vectors_still_decode():
    """The CUDA path moves float32 coded vectors: with tau = 1e-5 the oracle locates the attackers and
    recovers the sum to well within 1e-4 of its largest entry (the acceptance bound of the GPU tests)."""
    rng = np.random.default_rng(19)
    for P, s, m in ((15, 2, 5), (45, 3, 5), (20, 5, 10), (15, 1, 10), (15, 5, 2)):
        sizes, w = _plan(P, s, m)
        d = 2000 * m + 3
        G = rng.normal(size=(P, d)).astype(np.float32)
        Z = so.encode(G, m, sizes, w).astype(np.float32)
        f = (1.0 + rng.normal(size=(2, Z.shape[1]))).astype(np.float32)
        want = so.plain_sum(G)
        for kind in ("gaussian", "alie", "neg_mean", "flip10"):
            for n_byz in (0, s):
                nodes = sorted(rng.permutation(P)[:n_byz].tolist())
                R = _attack(kind, Z.astype(np.float64), nodes, rng).astype(np.float32)
                u, mask, status = so.decode(R, d, m, s, sizes, w, f, tau=1e-5)
                assert status == 0
                assert np.array_equal(mask, so.true_mask(R, Z)), (P, s, m, kind)
                assert np.abs(u - want).max() <= 1e-4 * np.abs(want).max(), (P, s, m, kind)


def test_row_energy_is_the_sum_of_squares_along_a_row():
    """nu[k] = sum_p R[k, p]^2, added up entry by entry on a 3 x 4 matrix whose rows, columns and signs all differ
    (a sum of absolute values, a sum down the columns or a squared sum would each give other numbers)."""
    R = np.array([[1.0, -2.0, 3.0, 0.5], [0.0, 4.0, -1.0, 2.0], [-3.0, 0.25, 0.0, 1.0]], dtype=np.float32)
    want = []
    for k in range(3):
        acc = 0.0
        for p in range(4):
            acc += float(R[k, p]) * float(R[k, p])
        want.append(acc)
    assert want == [14.25, 21.0, 10.0625]
    assert np.array_equal(so.row_energy(R), np.array(want))


def test_detection_tolerance_value_and_threshold():
    """The floating-point reading of the locator's "!=" (Section 3.4): a node is off the fitted polynomial when its
    projected value misses it by more than tau * sqrt(2 * median row energy).  The number itself on a hand-made
    energy vector, then the decision through Algorithm 1: one coordinate of one honest coded vector is moved so that
    the node's projected value moves by half the tolerance (not located, nothing to locate: Lemma 3's set is about
    exact inequality, the floating-point test cannot see it) and by twice the tolerance (located)."""
    assert so.detection_tolerance(np.array([8.0, 2.0, 18.0]), 0.5) == 2.0          # median 8: 0.5 * sqrt(16)
    assert so.detection_tolerance(np.array([50.0, 2.0, 2.0, 50.0]), 1e-3) == pytest.approx(1e-3 * math.sqrt(52.0))
    rng = np.random.default_rng(29)
    P, s, m, d = 8, 1, 2, 64
    sizes, w = _plan(P, s, m, r=8)                       # one group of eight: leverage of a node about m / 8
    G = 300.0 * rng.normal(size=(P, d))                  # far from 1, so that sum R^2 and sum |R| differ by orders
    Z = so.encode(G, m, sizes, w)
    f = 1.0 + rng.normal(size=(1, Z.shape[1]))
    tau = 1e-6
    nu = [sum(float(v) * float(v) for v in Z[k]) for k in range(P)]
    tol = tau * math.sqrt(2.0 * sorted(nu)[3] / 2.0 + 2.0 * sorted(nu)[4] / 2.0)   # median of eight: mean of the middle two
    k, p0 = 5, 17
    for factor, located in ((0.5, False), (2.0, True)):
        R = Z.copy()
        R[k, p0] += factor * tol / f[0, p0]
        u, mask, status = so.decode(R, d, m, s, sizes, w, f, tau=tau)
        assert status == 0
        assert mask.nonzero()[0].tolist() == ([k] if located else []), factor
    # the same two deviations straight through the locator with an explicit tolerance
    rho = so.project(Z, f)
    for factor, want_V in ((0.5, []), (2.0, [k])):
        moved = rho.copy()
        moved[0, k] += factor * tol
        V, t = so.phi_incremental(moved, w, m, s, tol)
        assert V == want_V and t == len(want_V)


# ---------------------------------------------------------------- least-squares gradients


def test_lsq_grads_match_finite_differences():
    """g_i is the gradient of 1/2 ||X_i w - y_i||^2: central differences of that loss (exact for a quadratic)."""
    rng = np.random.default_rng(23)
    P, rows, d = 3, 5, 7
    X = rng.normal(size=(P * rows, d))
    y = rng.normal(size=P * rows)
    w = rng.normal(size=d)
    G = so.lsq_grads(X, y, w, rows)
    h = 1e-3
    for i in range(P):
        X_i, y_i = X[i * rows:(i + 1) * rows], y[i * rows:(i + 1) * rows]
        loss = lambda v: 0.5 * np.sum((X_i @ v - y_i) ** 2)
        for c in range(d):
            e = np.zeros(d)
            e[c] = h
            fd = (loss(w + e) - loss(w - e)) / (2 * h)
            assert math.isclose(G[i, c], fd, rel_tol=1e-8, abs_tol=1e-8)
