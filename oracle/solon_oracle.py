"""Float64 CPU oracle for Solon's encode and robust decode (arXiv 2110.01595).

THIS MODULE IS TEST INFRASTRUCTURE.  It is a plain, slow, obviously-correct
restatement of what the paper's mechanism (A, E, D) computes, written from the
paper's definitions.  It shares no code, tables or helpers with the CUDA
library and never imports it.  Only the test-suite, the smoke check and the
benchmark's CPU-baseline leg may call it; the product path never does.

Notation follows the paper (Section 3), with the shorter letters used by this
library's C interface in brackets:

    P     compute nodes = partition gradients (the paper takes B = P)
    s     Byzantine nodes tolerated (per group, see ``decode``)
    r_c   compression ratio                                   [m]
    d_c   ceil(d / r_c), length of one coded vector
    r     redundancy ratio = group size, r >= 2 s + r_c  (Theorem 2)
    q     number of groups ("blocks" of the linear block code, Section 3.4)
    w_k   the distinct non-zero scalar of node k (Section 3.4)
    f     the random row vector of the locator (Section 3.4)

Every function names the passage it follows.  Arithmetic is float64
throughout; the inputs may be float32 arrays (they are widened first).

Pins (tests/test_oracle_*.py): encode against a dense Kronecker product built
with ``numpy.kron``; the m = 1 special case; the closed form of Lemma 9 for
the projected values; exact recovery of the plain sum (Definition 1) under
0..s attackers of several kinds; the locator against brute-force subset
enumeration (Appendix C) and against the Reed-Solomon property that the
denominator's roots are the corrupt nodes' scalars; the fixed-s system of
Section 3.4 against the incremental variant; the r_c = 1 majority vote against
the general decoder and the plain sum; Theorem 2 / its corollary and the
introduction's 4-node example for feasibility; Table 2 for d_c; the
least-squares gradient against finite differences of the loss; the row
energies against an entry-by-entry sum on a hand-made matrix and the
floating-point tolerance by its value and by a deviation of half and of twice
the tolerance sent through Algorithm 1.
No function here is "parity unpinned".
"""

from __future__ import annotations

import itertools
import math

import numpy as np

# --------------------------------------------------------------------------
# Plan: feasibility, groups, node scalars
# --------------------------------------------------------------------------


def redundancy_bound(s: int, r_c: int) -> int:
    """Smallest redundancy ratio that tolerates s adversaries: 2 s + r_c (Theorem 2)."""
    return 2 * s + r_c


def max_adversaries(P: int, r_c: int) -> int:
    """Largest tolerable s for P nodes: floor((P - r_c) / 2) (corollary of Theorem 2)."""
    return (P - r_c) // 2


def check_plan(P: int, s: int, r_c: int, r: int, d: int) -> None:
    """Raise ValueError unless (P, s, r_c, r, d) is a feasible Solon plan.

    Theorem 2 requires r >= 2 s + r_c; its corollary requires 2 s + r_c <= P;
    a group cannot be larger than the cluster, so r <= P.
    """
    if P < 1 or s < 0 or r_c < 1 or d < 1:
        raise ValueError("P, r_c, d must be >= 1 and s >= 0")
    if redundancy_bound(s, r_c) > P:
        raise ValueError("infeasible: 2 s + r_c > P (corollary of Theorem 2)")
    if r < redundancy_bound(s, r_c):
        raise ValueError("r < 2 s + r_c violates Theorem 2")
    if r > P:
        raise ValueError("r > P")


def coded_length(d: int, r_c: int) -> int:
    """d_c = d / r_c (Section 3.1), rounded up when r_c does not divide d."""
    return -(-d // r_c)


def group_sizes(P: int, r: int) -> list[int]:
    """Sizes of the q = floor(P / r) groups of the linear block code (Section 3.4).

    The paper treats r | P.  Otherwise the P - q r left-over nodes are dealt to
    the groups one at a time, first groups first, so every group keeps at least
    r >= 2 s + r_c members (all that the locator lemma needs).  With r | P this
    is the paper's layout exactly.
    """
    q = P // r
    extra = P - q * r
    return [r + extra // q + (1 if j < extra % q else 0) for j in range(q)]


def group_starts(sizes: list[int]) -> list[int]:
    """First node of every group; groups occupy consecutive node indices (A = I_q (x) 1_{r x r})."""
    starts = [0]
    for size in sizes[:-1]:
        starts.append(starts[-1] + size)
    return starts


def node_scalars(sizes: list[int]) -> np.ndarray:
    """The scalars w_1..w_P: "any distinct nonzero scalars" (Section 3.4).

    Only distinctness inside a group is ever used.  Each group of size r_j takes
    the first r_j of the n' Chebyshev points cos((2k-1) pi / (2 n')), k = 1..n',
    with n' = r_j rounded up to an even number so that 0 is not among them.
    """
    w = []
    for r_j in sizes:
        n_prime = r_j if r_j % 2 == 0 else r_j + 1
        for k in range(1, r_j + 1):
            w.append(math.cos((2 * k - 1) * math.pi / (2 * n_prime)))
    return np.array(w, dtype=np.float64)


def allocation_matrix(P: int, sizes: list[int]) -> np.ndarray:
    """A = I_q (x) 1_{r x r}: node j computes the gradients of its own group (Section 3.4)."""
    A = np.zeros((P, P), dtype=np.float64)
    for start, size in zip(group_starts(sizes), sizes):
        A[start:start + size, start:start + size] = 1.0
    return A


# --------------------------------------------------------------------------
# Encoder E  (Section 3.4: z_j = W_j Y_j 1_P)
# --------------------------------------------------------------------------


def encoder_matrix(w_j: float, r_c: int, d_c: int) -> np.ndarray:
    """W_j = I_{d_c} (x) [1, w_j, ..., w_j^{r_c-1}], dense (tiny sizes only)."""
    return np.kron(np.eye(d_c), w_j ** np.arange(r_c, dtype=np.float64)[None, :])


def group_sum(G: np.ndarray, start: int, size: int, r_c: int) -> np.ndarray:
    """ybar = Y_j 1_P: the sum of the group's gradients, zero-padded to r_c d_c entries."""
    d = G.shape[1]
    d_c = coded_length(d, r_c)
    ybar = np.zeros(r_c * d_c, dtype=np.float64)
    ybar[:d] = G[start:start + size].astype(np.float64).sum(axis=0)
    return ybar


def encode(G: np.ndarray, r_c: int, sizes: list[int], w: np.ndarray) -> np.ndarray:
    """All P coded vectors z_k = W_k ybar_g, as the rows of a P x d_c matrix.

    Entry p of z_k is sum_l w_k^l ybar_g[p r_c + l]: chunk p of ybar_g is its
    r_c consecutive coordinates starting at p r_c (Kronecker structure of W_k;
    the index pattern [ybar]_{l+1+(p-1) r_c} in the proof of Lemma 9).
    """
    P, d = G.shape
    d_c = coded_length(d, r_c)
    Z = np.zeros((P, d_c), dtype=np.float64)
    for start, size in zip(group_starts(sizes), sizes):
        chunks = group_sum(G, start, size, r_c).reshape(d_c, r_c)
        for k in range(start, start + size):
            Z[k] = chunks @ (w[k] ** np.arange(r_c, dtype=np.float64))
    return Z


# --------------------------------------------------------------------------
# Locator phi  (Section 3.4)
# --------------------------------------------------------------------------


def project(R: np.ndarray, f: np.ndarray) -> np.ndarray:
    """r_{j,c} = f R_j for every projection vector: rho[kappa, k] = sum_p f[kappa, p] R[k, p]."""
    return np.atleast_2d(f).astype(np.float64) @ R.astype(np.float64).T


def row_energy(R: np.ndarray) -> np.ndarray:
    """nu[k] = sum_p R[k, p]^2, used only to scale the floating-point tolerance."""
    R64 = R.astype(np.float64)
    return np.einsum("kp,kp->k", R64, R64)


def w_hat(w_g: np.ndarray, v: int) -> np.ndarray:
    """W-hat_{j,v}: rows [1, w, w^2, ..., w^v] for the nodes of one group."""
    return np.vander(w_g, v + 1, increasing=True)


def phi_paper(rho: np.ndarray, w_g: np.ndarray, r_c: int, s: int, tol: float) -> list[int]:
    """The locator exactly as Section 3.4 states it, for one projection.

    Solve  [ W-hat_{r_c+s-1} , -W-hat_{s-1} (.) (rho 1_s^T) ] a = rho (.) w^s
    (minimum-norm least squares, as a rank-deficient system arises whenever
    fewer than s nodes are corrupt: case (ii) in the proof of Lemma 9), form
    P_j(w) = (sum_i a_{i+1} w^i) / (w^s + sum_i a_{i+r_c+s+1} w^i) by polynomial
    division, and return V = {i : P_j(w_i) != rho_i}; "!=" is read as
    "differs by more than tol".
    """
    rho = np.asarray(rho, dtype=np.float64)
    if s == 0:
        A = w_hat(w_g, r_c - 1)
    else:
        A = np.hstack([w_hat(w_g, r_c + s - 1), -w_hat(w_g, s - 1) * rho[:, None]])
    b = rho * w_g ** s
    a = np.linalg.lstsq(A, b, rcond=None)[0]
    numerator = a[:r_c + s]                                 # ascending powers
    denominator = np.concatenate([a[r_c + s:], [1.0]])      # monic, ascending
    quotient, _ = np.polydiv(numerator[::-1], denominator[::-1])   # descending
    P_j = np.polyval(quotient, w_g)
    return [i for i in range(len(w_g)) if abs(P_j[i] - rho[i]) > tol]


def locator_system(rho: np.ndarray, w_g: np.ndarray, r_c: int, t: int):
    """The Section 3.4 system for t errors, stacked over the K projections.

    Unknowns: K numerators of r_c + t coefficients each, then the t lower
    coefficients theta of ONE monic denominator w^t + sum theta_i w^i shared by
    all projections (every projection sees the same corrupt nodes).  With K = 1
    and t = s this is the paper's system.
    """
    K, r = rho.shape
    n_num = r_c + t
    A = np.zeros((K * r, K * n_num + t), dtype=np.float64)
    b = np.zeros(K * r, dtype=np.float64)
    for kappa in range(K):
        rows = slice(kappa * r, (kappa + 1) * r)
        A[rows, kappa * n_num:(kappa + 1) * n_num] = w_hat(w_g, n_num - 1)
        if t > 0:
            A[rows, K * n_num:] = -w_hat(w_g, t - 1) * rho[kappa][:, None]
        b[rows] = rho[kappa] * w_g ** t
    return A, b


def refit_residuals(rho: np.ndarray, w_g: np.ndarray, r_c: int, U: list[int]) -> np.ndarray:
    """Fit a degree-(r_c - 1) polynomial to every projection on the nodes U; residual at all nodes.

    Honest projected values lie on such a polynomial (Lemma 9: rho_k = Q(w_k)).
    """
    Wm = w_hat(w_g, r_c - 1)
    coeff = np.linalg.lstsq(Wm[U], rho[:, U].T, rcond=None)[0]      # r_c x K
    return rho - (Wm @ coeff).T


def phi_incremental(rho: np.ndarray, w_g: np.ndarray, r_c: int, s: int, tol: np.ndarray):
    """Locator for floating-point data: try t = 0, 1, ..., s errors in turn.

    For each t solve the t-error system (unique when exactly t nodes are
    corrupt), take the t nodes where the denominator is smallest as candidates,
    refit on the rest and accept if every remaining node agrees with the fit
    within tol[kappa].  Returns (V, t) or (None, s) when no t <= s is accepted;
    V holds the candidates that disagree with the accepted polynomial (a node
    whose values fit is not corrupt, whoever sent them).
    """
    rho = np.atleast_2d(np.asarray(rho, dtype=np.float64))
    tol = np.broadcast_to(np.asarray(tol, dtype=np.float64), (rho.shape[0],))
    r = rho.shape[1]
    candidates: list[int] = []
    for t in range(s + 1):
        if t > 0:
            A, b = locator_system(rho, w_g, r_c, t)
            a = np.linalg.lstsq(A, b, rcond=None)[0]
            theta = a[len(a) - t:]
            E = w_g ** t + w_hat(w_g, t - 1) @ theta
            candidates = sorted(np.argsort(np.abs(E), kind="stable")[:t].tolist())
        U = [k for k in range(r) if k not in candidates]
        res = np.abs(refit_residuals(rho, w_g, r_c, U))
        if np.all(res[:, U] <= tol[:, None]):
            V = [k for k in candidates if np.any(res[:, k] > tol)]
            return V, t
    return None, s


def brute_force_locate(R_g: np.ndarray, w_g: np.ndarray, r_c: int, s: int, tol: float):
    """Appendix C: enumerate subsets S, smallest first, until R restricted to the
    complement lies in the span of the code there.  Works on the full received
    block (no projection), so it does not depend on f.  Tiny groups only.

    A complement row set is "in the span" when every column of R_g[S^c] is a
    combination of the columns of W-hat_{r_c-1}[S^c] up to ``tol`` (absolute).
    Returns the members of S that are themselves off the fitted code word.
    """
    R64 = R_g.astype(np.float64)
    r = R64.shape[0]
    Wm = w_hat(w_g, r_c - 1)
    for size in range(s + 1):
        for S in itertools.combinations(range(r), size):
            keep = [k for k in range(r) if k not in S]
            coeff = np.linalg.lstsq(Wm[keep], R64[keep], rcond=None)[0]
            res = np.abs(R64 - Wm @ coeff).max(axis=1)
            if np.all(res[keep] <= tol):
                return [k for k in S if res[k] > tol]
    return None


# --------------------------------------------------------------------------
# Block decoder psi and decoder D  (Section 3.4, Algorithm 1)
# --------------------------------------------------------------------------


def psi(R_g: np.ndarray, w_g: np.ndarray, r_c: int, U: list[int]) -> np.ndarray:
    """vec( [R_j]_{.,U} [W-hat_{j,r_c-1}]_{U,.}^{-1,T} ): the group's summed gradient, length r_c d_c.

    With more than r_c trusted nodes the inverse is read as the least-squares
    solution over all of U (identical in exact arithmetic, Lemma 4).
    """
    Wm = w_hat(w_g, r_c - 1)
    chunks = np.linalg.lstsq(Wm[U], R_g[U].astype(np.float64), rcond=None)[0]   # r_c x d_c
    return chunks.T.reshape(-1)


def inverse_rows(w_g: np.ndarray, r_c: int, U_prime: list[int]) -> np.ndarray:
    """C = ([W-hat_{r_c-1}]_{U',.})^{-1}: C[l, j] weights trusted node U'[j] in coordinate l of a chunk."""
    if len(U_prime) != r_c:
        raise ValueError("need exactly r_c trusted nodes for a square inverse")
    return np.linalg.inv(w_hat(w_g, r_c - 1)[U_prime])


def detection_tolerance(nu_g: np.ndarray, tau: float) -> float:
    """Floating-point reading of the "!=" test: tau * sqrt(2 * median row energy).

    sqrt(2 nu_k) is the size of f z_k for f ~ N(1, I); rounding of the coded
    values perturbs an honest projection by about one unit roundoff times that.
    """
    return tau * math.sqrt(2.0 * float(np.median(nu_g)))


def decode(R: np.ndarray, d: int, r_c: int, s: int, sizes: list[int], w: np.ndarray,
           f: np.ndarray, tau: float = 1e-9):
    """Algorithm 1.  Returns (u, mask, status).

    For each group: V = phi(R_j), U = complement, u_j = psi(R_j, U); u = sum u_j
    truncated to d.  mask[k] = 1 for located nodes.  status is 0, or -1 if some
    group admits no consistent set of at most s corrupt nodes (then u is built
    from the last candidates tried and must not be trusted).  The budget of s
    applies to each group separately, which contains the paper's "at most s in
    total".  With s = 0 the locator is skipped.
    """
    P, d_c = R.shape
    f = np.atleast_2d(f)
    u = np.zeros(r_c * d_c, dtype=np.float64)
    mask = np.zeros(P, dtype=np.uint8)
    status = 0
    rho_all = project(R, f)
    nu = row_energy(R)
    for start, size in zip(group_starts(sizes), sizes):
        grp = slice(start, start + size)
        w_g = w[grp]
        if s == 0:
            V = []
        else:
            tol = detection_tolerance(nu[grp], tau)
            V, _ = phi_incremental(rho_all[:, grp], w_g, r_c, s, tol)
            if V is None:
                status = -1
                V = []
        U = [k for k in range(size) if k not in V]
        mask[[start + k for k in V]] = 1
        u += psi(R[grp], w_g, r_c, U)
    return u[:d], mask, status


def majority_decode(R: np.ndarray, s: int, sizes: list[int]):
    """The r_c = 1 special case written out: repetition code and majority vote.

    With r_c = 1 the encoder matrix W_j = I_d (x) [1] is the identity (Section 3.4), so every node of a group
    sends the same vector, the group's summed gradient: Solon's code is then the repetition code, and locating
    at most s < r / 2 corrupt nodes is a majority vote among the group's received vectors.  For each group the
    vector held by at least r_j - s nodes is taken (rows are compared exactly), the nodes that sent anything
    else are flagged, and the groups' vectors are added up.  Returns (u, mask, status); status is -1 if some
    group has no such majority.
    """
    P, d = R.shape
    u = np.zeros(d, dtype=np.float64)
    mask = np.zeros(P, dtype=np.uint8)
    status = 0
    for start, size in zip(group_starts(sizes), sizes):
        rows = R[start:start + size]
        winner = None
        for k in range(size):
            same = [j for j in range(size) if np.array_equal(rows[j], rows[k])]
            if len(same) >= size - s:
                winner = (k, same)
                break
        if winner is None:
            status = -1
            continue
        k, same = winner
        u += rows[k].astype(np.float64)
        for j in range(size):
            if j not in same:
                mask[start + j] = 1
    return u, mask, status


# --------------------------------------------------------------------------
# Definitions the mechanism must reproduce
# --------------------------------------------------------------------------


def plain_sum(G: np.ndarray) -> np.ndarray:
    """G 1_P: the sum of all partition gradients (Definition 1), in float64."""
    return G.astype(np.float64).sum(axis=0)


def true_mask(received: np.ndarray, honest: np.ndarray) -> np.ndarray:
    """{k : n_k != 0}: nodes whose received vector differs from their honest coded vector (Lemma 3)."""
    return np.any(received != honest, axis=1).astype(np.uint8)


def lsq_grads(X: np.ndarray, y: np.ndarray, w: np.ndarray, rows: int) -> np.ndarray:
    """Partition gradients of 1/2 ||X_i w - y_i||^2: g_i = X_i^T (X_i w - y_i), one row per partition.

    Not in the paper, which accepts any method that needs a sum of functions
    (Section 1); partition i owns rows [i rows, (i+1) rows) of X and y.
    """
    P = X.shape[0] // rows
    X64 = X.astype(np.float64)
    w64 = w.astype(np.float64)
    G = np.zeros((P, X.shape[1]), dtype=np.float64)
    for i in range(P):
        X_i = X64[i * rows:(i + 1) * rows]
        G[i] = X_i.T @ (X_i @ w64 - y[i * rows:(i + 1) * rows].astype(np.float64))
    return G
