// Locator (phi) and recovery-table (psi) arithmetic of Solon's decoder, Section 3.4, in float64.
//
// One source, two builds.  On the device every function is executed by one CTA: matrices live in
// shared memory column by column, a warp owns columns (SOLON_FOR_WARPS), its lanes own rows
// (SOLON_FOR_LANES, partial sums combined by lane_sum), element-wise work is spread over all threads
// (SOLON_FOR_THREADS) and SOLON_SYNC is the CTA barrier.  On the host the same code runs serially
// (one warp of one lane), which is what solon_locate_host exposes for CPU tests.
//
// Reading of the paper's exact-arithmetic locator used here:
//   * the error count is tried incrementally, t = 0..s; for each t the rational-interpolation
//     system of Section 3.4 is solved with the K projections sharing one denominator;
//   * polynomials are expanded in Chebyshev polynomials T_i instead of monomials (the same
//     rational function, a better conditioned system); the denominator is T_t + sum theta_i T_i;
//   * the t nodes where the denominator is smallest are the candidates; a degree-(m-1) fit on the
//     remaining nodes must reproduce every remaining node within tau (relative to
//     sqrt(2 median nu)), which replaces the paper's "P_j(w_i) != r_i" test;
//   * the inverse of the block decoder is the least-squares inverse over the rows it reads:
//     m well-spread trusted rows when m <= SOLON_SUBSET_MAX_M, all trusted rows otherwise.
#pragma once

#include <math.h>
#include <stdint.h>

#if defined(__CUDA_ARCH__)
#define SOLON_TID ((int)threadIdx.x)
#define SOLON_NTHREADS ((int)blockDim.x)
#define SOLON_LANE ((int)(threadIdx.x & 31))
#define SOLON_NLANES 32
#define SOLON_WARP ((int)(threadIdx.x >> 5))
#define SOLON_NWARPS ((int)(blockDim.x >> 5))
#define SOLON_SYNC() __syncthreads()
#else
#define SOLON_TID 0
#define SOLON_NTHREADS 1
#define SOLON_LANE 0
#define SOLON_NLANES 1
#define SOLON_WARP 0
#define SOLON_NWARPS 1
#define SOLON_SYNC() ((void)0)
#endif
#define SOLON_FOR_THREADS(i, n) for (int i = SOLON_TID; i < (n); i += SOLON_NTHREADS)
#define SOLON_FOR_WARPS(i, n) for (int i = SOLON_WARP; i < (n); i += SOLON_NWARPS)
#define SOLON_FOR_LANES(i, n) for (int i = SOLON_LANE; i < (n); i += SOLON_NLANES)

#if defined(__CUDACC__)
#define SOLON_HD __host__ __device__
#define SOLON_HD_NOINLINE __host__ __device__ __noinline__   /* one copy of the code: the locator runs once per
                                                                decode from a cold instruction cache */
#else
#define SOLON_HD
#define SOLON_HD_NOINLINE
#endif

#define SOLON_SUBSET_MAX_M 6
#define SOLON_THETA_MAX 16   /* largest error count per group (SOLON_MAX_S) */

namespace solon {

// Sum of x over the lanes of the calling warp, returned to every lane (the value itself on the host).
SOLON_HD inline double lane_sum(double x) {
#if defined(__CUDA_ARCH__)
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
#endif
  return x;
}

// One (group, t) record written by locate_task and read by the group's epilogue.
struct TaskRecord {
  int accept;      // 1 if every node outside the candidates fits the polynomial
  int n_flagged;   // candidates that do not fit
  double max_fit;  // largest |residual| / tolerance over the non-candidates (best-guess ranking)
};

// Doubles of workspace one task needs (group of n nodes, K projections, t errors).
SOLON_HD inline size_t locate_task_ws_doubles(int n, int m, int K, int t) {
  size_t ncheb = (size_t)m + t + 1;
  size_t ncol = (size_t)K * (m + t) + t;
  size_t rows = (size_t)K * n;
  size_t solve = rows * (ncol + 1) + (ncol + 1) + (size_t)t * (t + 1) + ncol + n;
  size_t fit = (size_t)n * (m + K) + (m + K) + (size_t)m * (m + K) + m + (size_t)K * m + n + (size_t)n / 2 + 2;
  return (size_t)n * ncheb + (solve > fit ? solve : fit) + 8;
}

// Doubles of workspace the epilogue needs.
SOLON_HD inline size_t locate_epilogue_ws_doubles(int n, int m) {
  return (size_t)n * m + (size_t)m * m + 2 * (size_t)m + 64;
}

// T_i(x) for i = 0..count-1 into out[0..count).
SOLON_HD inline void chebyshev_row(double x, int count, double* out) {
  double t0 = 1.0, t1 = x;
  for (int i = 0; i < count; ++i) {
    out[i] = t0;
    double t2 = 2.0 * x * t1 - t0;
    t0 = t1;
    t1 = t2;
  }
}

// norm0[c] = squared norm of column c of the column-major matrix A (rows x ncols, column stride ldc).
SOLON_HD_NOINLINE inline void column_norms(const double* A, int rows, int ldc, int ncols, double* norm0) {
  SOLON_FOR_WARPS(c, ncols) {
    double acc = 0.0;
    SOLON_FOR_LANES(i, rows) acc = fma(A[(size_t)c * ldc + i], A[(size_t)c * ldc + i], acc);
    acc = lane_sum(acc);
    if (SOLON_LANE == 0) norm0[c] = acc;
  }
  SOLON_SYNC();
}

// Modified Gram-Schmidt on the first `nq` columns of the column-major matrix A, applied to all
// `ncols` columns (the trailing ones are right-hand sides).  Columns stay un-normalised.
// R (row-major, leading dimension ldr) receives the rows j >= r_first of the triangular factor,
// right-hand-side columns included, with entry (j, c) stored at R[(j - r_first) * ldr + c - r_first];
// diag[j] = ||q_j|| (0 for a numerically dependent column).
SOLON_HD_NOINLINE inline void mgs_factor(double* A, int rows, int ldc, int nq, int ncols, const double* norm0,
                                double* R, int ldr, int r_first, double* diag) {
  for (int j = 0; j < nq; ++j) {
    const double* qj = A + (size_t)j * ldc;
    double acc = 0.0;
    SOLON_FOR_LANES(i, rows) acc = fma(qj[i], qj[i], acc);
    const double nrm2 = lane_sum(acc);               // every warp computes the same value
    const bool dead = !(nrm2 > norm0[j] * 1e-26) || !(nrm2 > 0.0);
    const double nrm = dead ? 0.0 : sqrt(nrm2);
    const double inv2 = dead ? 0.0 : 1.0 / nrm2;
    if (SOLON_TID == 0) {
      diag[j] = nrm;
      if (j >= r_first) R[(size_t)(j - r_first) * ldr + (j - r_first)] = nrm;
    }
    const int todo = ncols - (j + 1);
    SOLON_FOR_WARPS(cc, todo) {
      const int c = j + 1 + cc;
      double* ac = A + (size_t)c * ldc;
      double dot = 0.0;
      if (!dead) {
        SOLON_FOR_LANES(i, rows) dot = fma(qj[i], ac[i], dot);
        dot = lane_sum(dot);
        const double coef = dot * inv2;
        SOLON_FOR_LANES(i, rows) ac[i] = fma(-coef, qj[i], ac[i]);
      }
      if (j >= r_first && SOLON_LANE == 0) R[(size_t)(j - r_first) * ldr + (c - r_first)] = dot * (nrm * inv2);
    }
    SOLON_SYNC();
  }
}

// Verification: fit a degree-(m-1) polynomial to every projection on the non-candidates and test
// all nodes.  cheb: n x ncheb table of T_i(w_k); rho_n: K x n projected values divided by the
// scale; cand[k] != 0 marks the n_cand candidates.  bad[k] receives 1 where some projection is off by
// more than tau (or is not a number).  Returns through rec.
SOLON_HD inline void locate_verify(int n, int m, int K, const double* cheb, int ncheb, const double* rho_n,
                                   double tau, const uint8_t* cand, int n_cand, uint8_t* bad, double* ws,
                                   TaskRecord* rec) {
  const int ld = m + K;          // columns: m basis polynomials, K right-hand sides
  const int n_u = n - n_cand;    // rows: the non-candidates
  double* B = ws;                            // column-major, ld columns of n_u rows
  double* norm0 = B + (size_t)n * ld;        // ld
  double* Rf = norm0 + ld;                   // m x ld
  double* diag = Rf + (size_t)m * ld;        // m
  double* coef = diag + m;                   // K x m
  double* ratio = coef + (size_t)K * m;      // n
  int* ulist = reinterpret_cast<int*>(ratio + n);   // n
  SOLON_FOR_THREADS(k, n) {
    if (!cand[k]) {
      int pos = 0;
      for (int o = 0; o < k; ++o) pos += cand[o] ? 0 : 1;
      ulist[pos] = k;
    }
  }
  SOLON_SYNC();
  SOLON_FOR_THREADS(idx, n_u * ld) {
    const int c = idx / n_u, i = idx - c * n_u, k = ulist[i];
    B[(size_t)c * n_u + i] = c < m ? cheb[(size_t)k * ncheb + c] : rho_n[(size_t)(c - m) * n + k];
  }
  SOLON_SYNC();
  column_norms(B, n_u, n_u, ld, norm0);
  mgs_factor(B, n_u, n_u, m, ld, norm0, Rf, ld, 0, diag);
  SOLON_FOR_THREADS(kappa, K) {             // back substitution, one projection per thread
    for (int i = m - 1; i >= 0; --i) {
      double acc = Rf[(size_t)i * ld + m + kappa];
      for (int c = i + 1; c < m; ++c) acc = fma(-Rf[(size_t)i * ld + c], coef[(size_t)kappa * m + c], acc);
      coef[(size_t)kappa * m + i] = diag[i] > 0.0 ? acc / diag[i] : 0.0;
    }
  }
  SOLON_SYNC();
  SOLON_FOR_THREADS(k, n) {
    double worst = 0.0;
    for (int kappa = 0; kappa < K; ++kappa) {
      double q = 0.0;
      for (int i = 0; i < m; ++i) q = fma(coef[(size_t)kappa * m + i], cheb[(size_t)k * ncheb + i], q);
      double res = fabs(rho_n[(size_t)kappa * n + k] - q);
      if (!(res == res)) res = INFINITY;
      worst = res > worst ? res : worst;
    }
    ratio[k] = tau > 0.0 ? worst / tau : (worst > 0.0 ? INFINITY : 0.0);
    bad[k] = ratio[k] > 1.0 ? 1 : 0;
  }
  SOLON_SYNC();
  if (SOLON_TID == 0) {
    int accept = 1, n_flagged = 0;
    double max_fit = 0.0;
    for (int k = 0; k < n; ++k) {
      if (cand[k]) {
        n_flagged += bad[k];
      } else {
        if (bad[k]) accept = 0;
        max_fit = ratio[k] > max_fit ? ratio[k] : max_fit;
      }
    }
    rec->accept = accept;
    rec->n_flagged = n_flagged;
    rec->max_fit = max_fit;
  }
  SOLON_SYNC();
}

// One task: assume exactly t corrupt nodes among the n (finite) nodes of a group.
//   rho_n   K x n projected values divided by the scale (so honest values are O(1))
//   w       n node scalars;  tau  tolerance in the same normalised units
//   flags   n bytes out: 1 for candidates that do not fit (the located nodes if accepted)
//   cand, bad: n bytes of scratch each;  ws: locate_task_ws_doubles(n, m, K, t) doubles
SOLON_HD inline void locate_task(int n, int m, int K, int t, const double* rho_n, const double* w, double tau,
                                 uint8_t* flags, uint8_t* cand, uint8_t* bad, double* ws, TaskRecord* rec) {
  const int ncheb = m + t + 1;
  double* cheb = ws;                         // n x ncheb
  double* rest = cheb + (size_t)n * ncheb;
  SOLON_FOR_THREADS(k, n) {
    chebyshev_row(w[k], ncheb, cheb + (size_t)k * ncheb);
    cand[k] = 0;
  }
  SOLON_SYNC();
  if (t > 0) {
    const int n_num = m + t;
    const int ncol = K * n_num + t;            // unknowns: K numerators, then theta
    const int ld = ncol + 1;                   // + right-hand side
    const int rows = K * n;
    double* A = rest;                          // column-major, ld columns of `rows` rows
    double* norm0 = A + (size_t)rows * ld;     // ld
    double* Rt = norm0 + ld;                   // t x (t+1): trailing rows of R, rhs in the last column
    double* diag = Rt + (size_t)t * (t + 1);   // ncol
    double* absE = diag + ncol;                // n
    SOLON_FOR_THREADS(idx, rows * ld) {
      const int c = idx / rows, row = idx - c * rows;
      const int kappa = row / n, k = row - kappa * n;
      const double rv = rho_n[(size_t)kappa * n + k];
      const double sc = 1.0 / sqrt(1.0 + rv * rv);     // balance rows of very large (corrupt) values
      double val;
      if (c < K * n_num) {
        const int blk = c / n_num, i = c - blk * n_num;
        val = blk == kappa ? sc * cheb[(size_t)k * ncheb + i] : 0.0;
      } else if (c < ncol) {
        val = -sc * rv * cheb[(size_t)k * ncheb + (c - K * n_num)];
      } else {
        val = sc * rv * cheb[(size_t)k * ncheb + t];
      }
      A[idx] = val;
    }
    SOLON_SYNC();
    column_norms(A, rows, rows, ld, norm0);
    const int r_first = ncol - t;
    mgs_factor(A, rows, rows, ncol, ld, norm0, Rt, t + 1, r_first, diag);
    // back substitution for the last t unknowns (theta); every thread does the same arithmetic
    double theta[SOLON_THETA_MAX];
    for (int i = t - 1; i >= 0; --i) {
      double acc = Rt[(size_t)i * (t + 1) + t];
      for (int c = i + 1; c < t; ++c) acc = fma(-Rt[(size_t)i * (t + 1) + c], theta[c], acc);
      theta[i] = diag[r_first + i] > 0.0 ? acc / diag[r_first + i] : 0.0;
    }
    SOLON_FOR_THREADS(k, n) {
      double e = cheb[(size_t)k * ncheb + t];
      for (int i = 0; i < t; ++i) e = fma(theta[i], cheb[(size_t)k * ncheb + i], e);
      const double ae = fabs(e);
      absE[k] = (ae == ae) ? ae : INFINITY;
    }
    SOLON_SYNC();
    SOLON_FOR_THREADS(k, n) {
      int rank = 0;
      const double mine = absE[k];
      for (int o = 0; o < n; ++o) rank += (absE[o] < mine || (absE[o] == mine && o < k)) ? 1 : 0;
      cand[k] = rank < t ? 1 : 0;
    }
    SOLON_SYNC();
  }
  locate_verify(n, m, K, cheb, ncheb, rho_n, tau, cand, t, bad, rest, rec);
  SOLON_FOR_THREADS(k, n) flags[k] = (cand[k] && bad[k]) ? 1 : 0;
  SOLON_SYNC();
}

// Recovery table for one group: given the trusted nodes (trusted[k] != 0 among n), choose the rows
// the recovery reads and the weights coeff[j*m + l] of row rec_rows[j] in coordinate l of a chunk,
// i.e. the least-squares inverse of [W-hat_{m-1}]_{rows,.} (monomial basis, as the encoder used).
// ws: locate_epilogue_ws_doubles(n, m).  Returns the number of rows (same value in every thread).
SOLON_HD inline int recovery_table(int n, int m, const double* w, const uint8_t* trusted, int* rec_rows,
                                   double* coeff, double* ws) {
  int n_u = 0;
  for (int k = 0; k < n; ++k) n_u += trusted[k] ? 1 : 0;
  if (n_u < m) return 0;
  const int n_rec = (m <= SOLON_SUBSET_MAX_M) ? m : n_u;
  {
    // every thread derives the same list; thread 0 stores it
    int seen = 0, next = 0;
    for (int k = 0; k < n && next < n_rec; ++k) {
      if (!trusted[k]) continue;
      const int want = (n_rec == n_u) ? next
                       : (m == 1 ? (n_u - 1) / 2 : (int)(((long long)next * (n_u - 1) + (m - 1) / 2) / (m - 1)));
      if (seen == want) {
        if (SOLON_TID == 0) rec_rows[next] = k;
        ++next;
      }
      ++seen;
    }
  }
  SOLON_SYNC();
  double* V = ws;                          // column-major: m columns of n_rec rows (becomes Q, un-normalised)
  double* norm0 = V + (size_t)n_rec * m;   // m
  double* R = norm0 + m;                   // m x m
  double* diag = R + (size_t)m * m;        // m
  SOLON_FOR_THREADS(j, n_rec) {
    const double x = w[rec_rows[j]];
    double p = 1.0;
    for (int l = 0; l < m; ++l) {
      V[(size_t)l * n_rec + j] = p;
      p *= x;
    }
  }
  SOLON_SYNC();
  column_norms(V, n_rec, n_rec, m, norm0);
  mgs_factor(V, n_rec, n_rec, m, m, norm0, R, m, 0, diag);
  // C = R^{-1} Q^T, one trusted row per thread
  SOLON_FOR_THREADS(j, n_rec) {
    double* c = coeff + (size_t)j * m;
    for (int l = m - 1; l >= 0; --l) {
      double acc = diag[l] > 0.0 ? V[(size_t)l * n_rec + j] / diag[l] : 0.0;
      for (int i = l + 1; i < m; ++i) acc = fma(-R[(size_t)l * m + i], c[i], acc);
      c[l] = diag[l] > 0.0 ? acc / diag[l] : 0.0;
    }
  }
  SOLON_SYNC();
  return n_rec;
}

// Group preparation shared by all tasks of a group: drop nodes whose projected values or energy are
// not finite (such nodes are corrupt by inspection), scale the rest.
//   rho: K rows with leading dimension ld_rho, this group's n entries each;  nu, w: n entries
//   idx[n_eff] original positions of the kept nodes; rho_n (K x n_eff) = rho / scale; w_c their scalars
//   *tau_eff = tau, or 0 when the median energy is 0 (all-zero data: any deviation counts)
// scratch: n doubles.  Returns n_eff (same in every thread).
SOLON_HD inline int locate_prepare(int n, int K, const double* rho, int ld_rho, const double* nu, const double* w,
                                   double tau, int* idx, double* rho_n, double* w_c, double* tau_eff,
                                   double* scratch) {
  int n_eff = 0;
  for (int k = 0; k < n; ++k) {
    bool finite = isfinite(nu[k]);
    for (int kappa = 0; kappa < K; ++kappa) finite = finite && isfinite(rho[(size_t)kappa * ld_rho + k]);
    if (finite) {
      if (SOLON_TID == 0) idx[n_eff] = k;
      ++n_eff;
    }
  }
  SOLON_SYNC();
  // lower median of the kept energies by rank counting
  SOLON_FOR_THREADS(i, n_eff) {
    const double mine = nu[idx[i]];
    int rank = 0;
    for (int o = 0; o < n_eff; ++o) {
      const double other = nu[idx[o]];
      rank += (other < mine || (other == mine && o < i)) ? 1 : 0;
    }
    if (rank == (n_eff - 1) / 2) scratch[0] = mine;
  }
  SOLON_SYNC();
  const double med = n_eff > 0 ? scratch[0] : 0.0;
  const double scale = med > 0.0 ? sqrt(2.0 * med) : 1.0;
  *tau_eff = med > 0.0 ? tau : 0.0;
  SOLON_FOR_THREADS(i, n_eff) {
    w_c[i] = w[idx[i]];
    for (int kappa = 0; kappa < K; ++kappa) rho_n[(size_t)kappa * n_eff + i] = rho[(size_t)kappa * ld_rho + idx[i]] / scale;
  }
  SOLON_SYNC();
  return n_eff;
}

// Group epilogue: pick the smallest accepted error count (else the best-fitting guess), write the
// mask over the group's n original nodes, and build the recovery table from the trusted nodes.
//   recs[s_eff+1], flags[(s_eff+1) x flags_ld] from the tasks (s_eff < 0: more non-finite nodes than s)
//   trusted: n bytes scratch; ws: locate_epilogue_ws_doubles(n, m)
// Returns 1 if the group decoded, 0 if not.  *t_out: corrupt nodes assumed (-1 if undecodable).
SOLON_HD inline int locate_epilogue(int n, int m, int s_eff, int n_eff, const int* idx, const double* w,
                                    const TaskRecord* recs, const uint8_t* flags, int flags_ld, uint8_t* mask,
                                    int* t_out, int* rec_rows, int* n_rec_out, double* coeff, uint8_t* trusted,
                                    double* ws) {
  int chosen = -1, ok = 0;
  if (s_eff >= 0) {
    for (int t = 0; t <= s_eff; ++t) {
      if (recs[t].accept) {
        chosen = t;
        ok = 1;
        break;
      }
    }
    if (!ok) {
      double best = INFINITY;
      chosen = 0;
      for (int t = 0; t <= s_eff; ++t) {
        if (recs[t].max_fit < best) {
          best = recs[t].max_fit;
          chosen = t;
        }
      }
    }
  }
  SOLON_FOR_THREADS(k, n) trusted[k] = 0;
  SOLON_SYNC();
  if (chosen >= 0) {
    SOLON_FOR_THREADS(i, n_eff) trusted[idx[i]] = flags[(size_t)chosen * flags_ld + i] ? 0 : 1;
  } else {
    SOLON_FOR_THREADS(i, n_eff) trusted[idx[i]] = 1;
  }
  SOLON_SYNC();
  SOLON_FOR_THREADS(k, n) mask[k] = trusted[k] ? 0 : 1;
  const int n_rec = recovery_table(n, m, w, trusted, rec_rows, coeff, ws);
  if (n_rec == 0) ok = 0;
  if (SOLON_TID == 0) {
    *n_rec_out = n_rec;
    *t_out = ok ? chosen + (n - n_eff) : -1;
  }
  SOLON_SYNC();
  return ok;
}

}  // namespace solon
