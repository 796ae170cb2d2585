// Locator (phi) and recovery-table (psi) arithmetic of Solon's decoder, Section 3.4, in float64.
//
// One source, two builds.  On the device every function is executed by one CTA: a warp owns columns
// (SOLON_FOR_WARPS), its lanes own rows (SOLON_FOR_LANES, partial sums combined by lane_sum),
// element-wise work is spread over all threads (SOLON_FOR_THREADS) and SOLON_SYNC is the CTA barrier.
// On the host the same code runs serially (one warp of one lane), which is what solon_locate_host
// exposes for CPU tests.
//
// Reading of the paper's exact-arithmetic locator used here:
//   * the error count is tried incrementally, t = 0..s; for each t the rational-interpolation system
//     of Section 3.4, N_kappa(w_k) = rho_kappa,k E(w_k) with deg N_kappa < m + t and E monic of degree t,
//     is solved in the least-squares sense with the K projections sharing E;
//   * the node scalars are fixed by the plan, so an orthonormal basis q_0, q_1, ... of the polynomials
//     on a group's nodes (q_i of degree i) is tabulated once.  The numerators are eliminated by
//     projecting on the complement of the polynomials of degree < m + t (columns m+t.. of the table):
//     only the t coefficients of E remain unknown, E = T_t + sum_i theta_i T_i in Chebyshev polynomials;
//   * the t nodes where E is smallest are the candidates; a degree-(m-1) fit on the remaining nodes
//     must reproduce every remaining node within tau (relative to sqrt(2 median nu)), which replaces
//     the paper's "P_j(w_i) != r_i" test.  The refit is obtained from the fit over all nodes by the
//     deletion (downdating) identity  r = e + H[:,V] (I - H[V,V])^{-1} e[V],  H = Q_m Q_m^T;
//   * the inverse of the block decoder is the least-squares inverse over the rows it reads:
//     m well-spread trusted rows when m <= SOLON_SUBSET_MAX_M (Lagrange form), all trusted rows
//     otherwise (the same deletion identity applied to the coefficient map).
#pragma once

#include <math.h>
#include <stdint.h>

#if defined(__CUDACC__)
#define SOLON_HD __host__ __device__
#define SOLON_NOINLINE __noinline__   /* one copy of the code, whoever calls it: a rehearsal warms it for the real call */
#else
#define SOLON_HD
#define SOLON_NOINLINE
#endif

// The threads that execute a routine together: a whole CTA, one warp of it, or (host) a single thread.
struct Team {
  int tid, nthreads;   // index and count of the threads of the team
  int lane, nlanes;    // lane inside the warp
  int warp, nwarps;    // warp inside the team
  SOLON_HD void sync() const {
#if defined(__CUDA_ARCH__)
    if (nwarps == 1) __syncwarp();
    else __syncthreads();   // a team of several warps is always the whole CTA
#endif
  }
#if defined(__CUDACC__)
  static __device__ Team cta() {
    return Team{(int)threadIdx.x, (int)blockDim.x, (int)(threadIdx.x & 31), 32, (int)(threadIdx.x >> 5), (int)(blockDim.x >> 5)};
  }
  static __device__ Team own_warp() { return Team{(int)(threadIdx.x & 31), 32, (int)(threadIdx.x & 31), 32, 0, 1}; }
#endif
  static Team serial() { return Team{0, 1, 0, 1, 0, 1}; }
};
#define SOLON_TID (tm.tid)
#define SOLON_NTHREADS (tm.nthreads)
#define SOLON_LANE (tm.lane)
#define SOLON_NLANES (tm.nlanes)
#define SOLON_WARP (tm.warp)
#define SOLON_NWARPS (tm.nwarps)
#define SOLON_SYNC() tm.sync()
#define SOLON_FOR_THREADS(i, n) for (int i = SOLON_TID; i < (n); i += SOLON_NTHREADS)
#define SOLON_FOR_WARPS(i, n) for (int i = SOLON_WARP; i < (n); i += SOLON_NWARPS)
#define SOLON_FOR_LANES(i, n) for (int i = SOLON_LANE; i < (n); i += SOLON_NLANES)

#define SOLON_SUBSET_MAX_M 6
#define SOLON_THETA_MAX 16   /* largest error count per group (SOLON_MAX_S) */
#define SOLON_RHO_CLAMP 1e8  /* projected values beyond this multiple of the group's median are clamped */

namespace solon {

// Sum of x over the lanes of the calling warp, returned to every lane (the value itself on the host).
SOLON_HD inline double lane_sum(double x) {
#if defined(__CUDA_ARCH__)
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) x += __shfl_xor_sync(0xffffffffu, x, off);
#endif
  return x;
}

// Tables of one group, fixed at plan time (functions of the node scalars only).
struct GroupTables {
  const double* Qb;    // n x n, column-major: Qb[j * n + k] = q_j(w_k), orthonormal columns, deg q_j = j
  const double* Hm;    // n x n, row-major: H = Q_m Q_m^T, the projector on the polynomials of degree < m
  const double* Mt;    // m x m, row-major: q_i(w) = sum_l Mt[l * m + i] w^l  (i < m)
  const double* Tch;   // n x (s + 1), row-major: Tch[k * (s + 1) + i] = T_i(w_k)
  const double* w;     // n node scalars
  // Recovery tables tabulated per corrupt set (n_sets = 0: not tabulated, recovery_table runs at decode time): entry
  // corrupt_set_index(V) holds what recovery_table returns when exactly the nodes V are untrusted - tab_count rows,
  // their indices at tab_rows[i * tab_ld ..], their weights at tab_coeff[i * tab_ld * m ..].
  const int* tab_count;
  const int* tab_rows;
  const double* tab_coeff;
  int n_sets;
  int tab_ld;
};

#define SOLON_MAX_SETS 4096   /* corrupt sets tabulated per group at most */

// C(a, b), saturating at 2^20 (callers only need exact values up to SOLON_MAX_SETS; 32-bit arithmetic throughout).
SOLON_HD inline int binomial(int a, int b) {
  if (b < 0 || b > a) return 0;
  int c = 1;
  for (int i = 1; i <= b; ++i) {
    if (c > (1 << 20)) return 1 << 20;
    c = c * (a - b + i) / i;       // exact (c = C(a - b + i - 1, i - 1), so the product is i C(a - b + i, i)) and below 2^31 for a <= 1024
  }
  return c;
}

// Number of subsets of at most s of n nodes (saturating above SOLON_MAX_SETS).
SOLON_HD inline int count_corrupt_sets(int n, int s) {
  int total = 0;
  for (int t = 0; t <= s && t <= n; ++t) {
    total += binomial(n, t);
    if (total > SOLON_MAX_SETS) return SOLON_MAX_SETS + 1;
  }
  return total;
}

// Position of the set {k : trusted[k] == 0} among all subsets of at most s of n nodes: sets are ordered by size and,
// within a size t, by sum_i C(v_i, i + 1) over their nodes v_0 < v_1 < ... (the combinatorial number system).
SOLON_HD inline int corrupt_set_index(int n, const uint8_t* trusted) {
  int t = 0, rank = 0;
  for (int k = 0; k < n; ++k) {
    if (trusted[k]) continue;
    rank += binomial(k, t + 1);
    ++t;
  }
  int offset = 0, c = 1;         // c = C(n, u)
  for (int u = 0; u < t; ++u) {
    offset += c;
    c = c * (n - u) / (u + 1);
  }
  return offset + rank;
}

// One (group, t) record written by locate_task and read by the group's epilogue.
struct TaskRecord {
  int accept;      // 1 if every node outside the candidates fits the polynomial
  int n_flagged;   // candidates that do not fit
  double max_fit;  // largest |residual| / tolerance over the non-candidates (best-guess ranking)
};

// Doubles of workspace one task needs (group of n nodes, K projections, up to t errors).
SOLON_HD inline size_t locate_task_ws_doubles(int n, int m, int K, int t) {
  (void)m;
  size_t rows = (size_t)K * n;                              // upper bound of K (n - m - t)
  size_t solve = rows * (t + 1) + (t + 1) + (size_t)t * (t + 1) + t;
  size_t fit = (size_t)K * n + 3 * (size_t)t * t + (size_t)K * t + n;
  return (size_t)n + (size_t)(t + n) / 2 + 1 + (solve > fit ? solve : fit) + 16;
}

// Doubles of workspace the epilogue needs.
SOLON_HD inline size_t locate_epilogue_ws_doubles(int n, int m, int s) {
  size_t t = (size_t)s;     // untrusted nodes the all-rows table is built for: at most s
  return 3 * t * t + t * (size_t)n + (size_t)m * n + (size_t)n + 64;
}

// norm0[c] = squared norm of column c of the column-major matrix A (rows x ncols, column stride ldc).
SOLON_HD inline void column_norms(const Team& tm, const double* A, int rows, int ldc, int ncols, double* norm0) {
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
// R (row-major, leading dimension ldr) receives the triangular factor, right-hand sides included;
// diag[j] = ||q_j|| (0 for a numerically dependent column).
SOLON_HD inline void mgs_factor(const Team& tm, double* A, int rows, int ldc, int nq, int ncols, const double* norm0, double* R,
                                int ldr, double* diag) {
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
      R[(size_t)j * ldr + j] = nrm;
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
      if (SOLON_LANE == 0) R[(size_t)j * ldr + c] = dot * (nrm * inv2);
    }
    SOLON_SYNC();
  }
}

// In-place inverse of the symmetric positive definite t x t matrix S (row-major) by Gauss-Jordan
// elimination on [S | I] held in `aug` (t x 2t, row-major); one thread per column of the pair.
// No pivoting is needed for a positive definite matrix.
SOLON_HD inline void spd_inverse(const Team& tm, double* S, int t, double* aug) {
  const int w2 = 2 * t;
  SOLON_FOR_THREADS(idx, t * w2) {
    const int r = idx / w2, c = idx - r * w2;
    aug[idx] = c < t ? S[(size_t)r * t + c] : (c - t == r ? 1.0 : 0.0);
  }
  SOLON_SYNC();
  for (int p = 0; p < t; ++p) {
    const double piv = aug[(size_t)p * w2 + p];
    const double inv = piv != 0.0 ? 1.0 / piv : 0.0;
    // columns other than p: scale the pivot row, eliminate column p from the other rows
    SOLON_FOR_THREADS(c, w2) {
      if (c == p) continue;
      const double top = aug[(size_t)p * w2 + c] * inv;
      for (int r = 0; r < t; ++r) {
        if (r == p) continue;
        aug[(size_t)r * w2 + c] = fma(-aug[(size_t)r * w2 + p], top, aug[(size_t)r * w2 + c]);
      }
      aug[(size_t)p * w2 + c] = top;
    }
    SOLON_SYNC();       // column p has been read by everyone
    SOLON_FOR_THREADS(r, t) aug[(size_t)r * w2 + p] = r == p ? 1.0 : 0.0;
    SOLON_SYNC();
  }
  SOLON_FOR_THREADS(idx, t * t) {
    const int r = idx / t, c = idx - r * t;
    S[idx] = aug[(size_t)r * w2 + t + c];
  }
  SOLON_SYNC();
}

// S <- (I - H[V,V])^{-1} for the node list V (nv nodes), H = Q_m Q_m^T (tabulated).
SOLON_HD inline void deletion_inverse(const Team& tm, const GroupTables& tb, int n, const int* V, int nv, double* S, double* aug) {
  SOLON_FOR_THREADS(idx, nv * nv) {
    const int a = idx / nv, b = idx - a * nv;
    S[idx] = (a == b ? 1.0 : 0.0) - tb.Hm[(size_t)V[a] * n + V[b]];
  }
  SOLON_SYNC();
  spd_inverse(tm, S, nv, aug);
}

// Verification: fit a degree-(m-1) polynomial to every projection on the non-candidates and test
// all nodes.  cand[k] != 0 marks the t candidates, vlist[0..t) lists them and vpos[k] is a candidate's
// position in that list; forced[k] != 0 marks nodes that are corrupt by inspection (they never fit).
// bad[k] receives 1 where some projection is off by more than tau.
SOLON_HD inline void locate_verify(const Team& tm, const GroupTables& tb, int n, int K, const double* rho_n, double tau,
                                   const uint8_t* cand, int t, const int* vlist, const int* vpos, const uint8_t* forced,
                                   uint8_t* bad, double* ws, TaskRecord* rec) {
  double* e = ws;                            // K x n   residual of the fit over all nodes: rho - H rho
  double* S = e + (size_t)K * n;             // t x t
  double* aug = S + (size_t)t * t;           // t x 2t
  double* x = aug + 2 * (size_t)t * t;       // K x t   leave-out residuals of the candidates
  double* ratio = x + (size_t)K * t;         // n
  SOLON_FOR_THREADS(idx, K * n) {
    const int kappa = idx / n, k = idx - kappa * n;
    const double* h = tb.Hm + (size_t)k * n;
    const double* r = rho_n + (size_t)kappa * n;
    double a0 = r[k], a1 = 0.0;
    int j = 0;
    for (; j + 1 < n; j += 2) {
      a0 = fma(-h[j], r[j], a0);
      a1 = fma(-h[j + 1], r[j + 1], a1);
    }
    if (j < n) a0 = fma(-h[j], r[j], a0);
    e[idx] = a0 + a1;
  }
  SOLON_SYNC();
  if (t == 1) {
    // one deleted node v: x = e_v / (1 - H_vv), every thread computes it for itself
    const int v = vlist[0];
    const double sinv = 1.0 / (1.0 - tb.Hm[(size_t)v * n + v]);
    SOLON_FOR_THREADS(kappa, K) x[kappa] = sinv * e[(size_t)kappa * n + v];
    SOLON_SYNC();
  } else if (t == 2) {
    const int v0 = vlist[0], v1 = vlist[1];
    const double s00 = 1.0 - tb.Hm[(size_t)v0 * n + v0], s11 = 1.0 - tb.Hm[(size_t)v1 * n + v1];
    const double s01 = -tb.Hm[(size_t)v0 * n + v1];
    const double idet = 1.0 / (s00 * s11 - s01 * s01);
    SOLON_FOR_THREADS(kappa, K) {
      const double e0 = e[(size_t)kappa * n + v0], e1 = e[(size_t)kappa * n + v1];
      x[(size_t)kappa * 2] = (s11 * e0 - s01 * e1) * idet;
      x[(size_t)kappa * 2 + 1] = (s00 * e1 - s01 * e0) * idet;
    }
    SOLON_SYNC();
  } else if (t > 2) {
    deletion_inverse(tm, tb, n, vlist, t, S, aug);
    SOLON_FOR_THREADS(idx, K * t) {
      const int kappa = idx / t, a = idx - kappa * t;
      double acc = 0.0;
      for (int b = 0; b < t; ++b) acc = fma(S[(size_t)a * t + b], e[(size_t)kappa * n + vlist[b]], acc);
      x[idx] = acc;
    }
    SOLON_SYNC();
  }
  const double inv_tau = tau > 0.0 ? 1.0 / tau : 0.0;
  SOLON_FOR_THREADS(k, n) {
    double worst = 0.0;
    for (int kappa = 0; kappa < K; ++kappa) {
      double res;
      if (cand[k]) {
        res = x[(size_t)kappa * t + vpos[k]];
      } else {
        res = e[(size_t)kappa * n + k];
        for (int b = 0; b < t; ++b) res = fma(tb.Hm[(size_t)k * n + vlist[b]], x[(size_t)kappa * t + b], res);
      }
      res = fabs(res);
      if (!(res == res)) res = INFINITY;
      worst = res > worst ? res : worst;
    }
    double rt = tau > 0.0 ? worst * inv_tau : (worst > 0.0 ? INFINITY : 0.0);
    if (forced[k]) rt = INFINITY;
    ratio[k] = rt;
    bad[k] = rt > 1.0 ? 1 : 0;
  }
  SOLON_SYNC();
  // every thread scans the verdicts (no branches on loaded values); thread 0 stores the record
  int rejected = 0, n_flagged = 0;
  double max_fit = 0.0;
  for (int k = 0; k < n; ++k) {
    const int c = cand[k] ? 1 : 0, b = bad[k] ? 1 : 0;
    n_flagged += c & b;
    rejected += (1 - c) & b;
    const double rk = c ? 0.0 : ratio[k];
    max_fit = rk > max_fit ? rk : max_fit;
  }
  if (SOLON_TID == 0) {
    rec->accept = rejected == 0 ? 1 : 0;
    rec->n_flagged = n_flagged;
    rec->max_fit = max_fit;
  }
}

#define SOLON_FAST_T 5         /* largest error count handled by the register-resident solver (locate_task<FT>, FT <= this) */
#if defined(__CUDA_ARCH__)
#define SOLON_FAST_RPL 2       /* rows per lane it can hold */
#else
#define SOLON_FAST_RPL 64
#endif

// One task: assume exactly t corrupt nodes among the n nodes of a group.  FT: the register-resident solver is
// compiled for error counts up to FT (the arithmetic does not depend on FT; a small FT is simply less code to
// fetch for plans with a small s).
//   rho_n   K x n projected values divided by the scale (0 for forced nodes)
//   s       the plan's s (row stride of tb.Tch is s + 1);  tau  tolerance in the same normalised units
//   flags   n bytes out: 1 for candidates that do not fit (the located nodes if accepted)
//   cand, bad: n bytes of scratch each;  ws: locate_task_ws_doubles(n, m, K, t) doubles
template <int FT>
SOLON_HD inline void locate_task(const Team& tm, const GroupTables& tb, int n, int m, int K, int t, int s, const double* rho_n,
                                 const uint8_t* forced, double tau, uint8_t* flags, uint8_t* cand, uint8_t* bad,
                                 double* ws, TaskRecord* rec) {
  const int ldt = s + 1;
  double* absE = ws;                         // n
  int* vlist = reinterpret_cast<int*>(absE + n);   // t
  int* vpos = vlist + t;                            // n
  double* rest = absE + n + (size_t)(t + n) / 2 + 1;
  SOLON_FOR_THREADS(k, n) {
    cand[k] = 0;
    vpos[k] = 0;
  }
  SOLON_SYNC();
  if (t > 0) {
    const int nperp = n - m - t;               // complement of the polynomials of degree < m + t
    const int rows = K * nperp;
    double theta[SOLON_THETA_MAX];
    if (tm.nwarps == 1 && t <= FT && rows <= SOLON_FAST_RPL * tm.nlanes) {
      // Small system: every lane keeps its rows of [A | b] in registers.  Row (kappa, j), column i:
      //   sum_k q_{m+t+j}(w_k) rho_kappa,k T_i(w_k);  the last column carries -(...) T_t.
      // One combined lane reduction per Gram-Schmidt step yields the norm and all inner products.
      double a[SOLON_FAST_RPL][FT + 1];
      const int rpl = (rows + tm.nlanes - 1) / tm.nlanes;
#pragma unroll
      for (int rr = 0; rr < SOLON_FAST_RPL; ++rr) {
        const int row = tm.lane + rr * tm.nlanes;
#pragma unroll
        for (int i = 0; i <= FT; ++i) a[rr][i] = 0.0;
        if (rr < rpl && row < rows) {
          const int kappa = row / nperp, j = row - kappa * nperp;
          const double* q = tb.Qb + (size_t)(m + t + j) * n;
          for (int k = 0; k < n; ++k) {
            const double qr = q[k] * rho_n[(size_t)kappa * n + k];
#pragma unroll
            for (int i = 0; i <= FT; ++i)
              if (i <= t) a[rr][i] = fma(qr, tb.Tch[(size_t)k * ldt + i], a[rr][i]);
          }
#pragma unroll
          for (int i = 0; i <= FT; ++i)
            if (i == t) a[rr][i] = -a[rr][i];
        }
      }
      double R[FT][FT + 1], diag[FT], norm0[FT];
#pragma unroll
      for (int j = 0; j < FT; ++j) {
        double v = 0.0;
#pragma unroll
        for (int rr = 0; rr < SOLON_FAST_RPL; ++rr) v = fma(a[rr][j], a[rr][j], v);
        norm0[j] = v;
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
#if defined(__CUDA_ARCH__)
        double tmp[FT];
#pragma unroll
        for (int j = 0; j < FT; ++j) tmp[j] = __shfl_xor_sync(0xffffffffu, norm0[j], off);
#pragma unroll
        for (int j = 0; j < FT; ++j) norm0[j] += tmp[j];
#endif
      }
#pragma unroll
      for (int j = 0; j < FT; ++j) {
        diag[j] = 0.0;
#pragma unroll
        for (int c = 0; c <= FT; ++c) R[j][c] = 0.0;
        if (j < t) {
          double d[FT + 1];      // d[c] = a_j . a_c for c >= j (d[j] is the squared norm)
#pragma unroll
          for (int c = 0; c <= FT; ++c) {
            double v = 0.0;
            if (c >= j && c <= t) {
#pragma unroll
              for (int rr = 0; rr < SOLON_FAST_RPL; ++rr) v = fma(a[rr][j], a[rr][c], v);
            }
            d[c] = v;
          }
#if defined(__CUDA_ARCH__)
#pragma unroll
          for (int off = 16; off > 0; off >>= 1) {
            double tmp[FT + 1];
#pragma unroll
            for (int c = 0; c <= FT; ++c) tmp[c] = __shfl_xor_sync(0xffffffffu, d[c], off);
#pragma unroll
            for (int c = 0; c <= FT; ++c) d[c] += tmp[c];
          }
#endif
          const double nrm2 = d[j];
          const bool dead = !(nrm2 > norm0[j] * 1e-26) || !(nrm2 > 0.0);
          const double nrm = dead ? 0.0 : sqrt(nrm2);
          const double inv2 = dead ? 0.0 : 1.0 / nrm2;
          diag[j] = nrm;
#pragma unroll
          for (int c = 0; c <= FT; ++c) {
            if (c > j && c <= t) {
              const double coef = d[c] * inv2;
#pragma unroll
              for (int rr = 0; rr < SOLON_FAST_RPL; ++rr) a[rr][c] = fma(-coef, a[rr][j], a[rr][c]);
              R[j][c] = d[c] * (nrm * inv2);
            }
          }
        }
      }
#pragma unroll
      for (int i = FT - 1; i >= 0; --i) {
        if (i < t) {
          double acc = 0.0;
#pragma unroll
          for (int c = 0; c <= FT; ++c)
            if (c == t) acc = R[i][c];
#pragma unroll
          for (int c = 0; c < FT; ++c)
            if (c > i && c < t) acc = fma(-R[i][c], theta[c], acc);
          theta[i] = diag[i] > 0.0 ? acc / diag[i] : 0.0;
        }
      }
    } else {
      const int ld = t + 1;                      // t unknowns theta, then the right-hand side
      double* A = rest;                          // column-major, ld columns of `rows` rows
      double* norm0 = A + (size_t)rows * ld;     // ld
      double* Rt = norm0 + ld;                   // t x (t + 1)
      double* diag = Rt + (size_t)t * (t + 1);   // t
      SOLON_FOR_THREADS(idx, rows * ld) {
        const int i = idx / rows, row = idx - i * rows;
        const int kappa = row / nperp, j = row - kappa * nperp;
        const double* q = tb.Qb + (size_t)(m + t + j) * n;
        double acc = 0.0;
        for (int k = 0; k < n; ++k) acc = fma(q[k] * rho_n[(size_t)kappa * n + k], tb.Tch[(size_t)k * ldt + i], acc);
        A[idx] = i < t ? acc : -acc;
      }
      SOLON_SYNC();
      column_norms(tm, A, rows, rows, ld, norm0);
      mgs_factor(tm, A, rows, rows, t, ld, norm0, Rt, t + 1, diag);
      // back substitution for theta; every thread does the same arithmetic
      for (int i = t - 1; i >= 0; --i) {
        double acc = Rt[(size_t)i * (t + 1) + t];
        for (int c = i + 1; c < t; ++c) acc = fma(-Rt[(size_t)i * (t + 1) + c], theta[c], acc);
        theta[i] = diag[i] > 0.0 ? acc / diag[i] : 0.0;
      }
      SOLON_SYNC();     // A is reused by the verification below
    }
    SOLON_FOR_THREADS(k, n) {
      double ev = tb.Tch[(size_t)k * ldt + t];
      for (int i = 0; i < t; ++i) ev = fma(theta[i], tb.Tch[(size_t)k * ldt + i], ev);
      const double ae = fabs(ev);
      absE[k] = (ae == ae) ? ae : INFINITY;
    }
    SOLON_SYNC();
    SOLON_FOR_THREADS(k, n) {
      int rank = 0;
      const double mine = absE[k];
      for (int o = 0; o < n; ++o) {
        const double other = absE[o];
        rank += (other < mine || (other == mine && o < k)) ? 1 : 0;
      }
      if (rank < t) {
        cand[k] = 1;
        vlist[rank] = k;
        vpos[k] = rank;
      }
    }
    SOLON_SYNC();
  }
  locate_verify(tm, tb, n, K, rho_n, tau, cand, t, vlist, vpos, forced, bad, rest, rec);
  SOLON_FOR_THREADS(k, n) flags[k] = (cand[k] && bad[k]) ? 1 : 0;
  SOLON_SYNC();
}

// Check of a given set: is `mask_in` (n bytes, at most s set) exactly the set of nodes that do not fit the
// polynomial refitted on all the others?  This is the acceptance test of locate_task for candidates that are known
// in advance.  cand, bad: n bytes of scratch each; ws: locate_task_ws_doubles(n, m, K, s) doubles.
// Every thread gets the same answer.
SOLON_HD inline int locate_check(const Team& tm, const GroupTables& tb, int n, int K, int s, const double* rho_n,
                                 const uint8_t* forced, double tau, const uint8_t* mask_in, uint8_t* cand, uint8_t* bad,
                                 double* ws, TaskRecord* rec) {
  int t = 0;
  for (int k = 0; k < n; ++k) t += mask_in[k] ? 1 : 0;
  if (t > s) return 0;
  double* absE = ws;                                // same layout as locate_task
  int* vlist = reinterpret_cast<int*>(absE + n);    // t
  int* vpos = vlist + t;                            // n
  double* rest = absE + n + (size_t)(t + n) / 2 + 1;
  SOLON_FOR_THREADS(k, n) {
    int pos = 0;
    for (int o = 0; o < k; ++o) pos += mask_in[o] ? 1 : 0;
    cand[k] = mask_in[k] ? 1 : 0;
    vpos[k] = mask_in[k] ? pos : 0;
    if (mask_in[k]) vlist[pos] = k;
  }
  SOLON_SYNC();
  locate_verify(tm, tb, n, K, rho_n, tau, cand, t, vlist, vpos, forced, bad, rest, rec);
  SOLON_SYNC();
  return (rec->accept && rec->n_flagged == t) ? 1 : 0;
}

// Recovery table for one group: given the trusted nodes (trusted[k] != 0 among n), choose the rows
// the recovery reads and the weights coeff[j*m + l] of row rec_rows[j] in coordinate l of a chunk,
// i.e. the least-squares inverse of [W-hat_{m-1}]_{rows,.} (monomial basis, as the encoder used).
// ws: locate_epilogue_ws_doubles(n, m, s).  Returns the number of rows (same value in every thread),
// 0 if fewer than m nodes are trusted or (all-rows form) more than s are not.
SOLON_HD SOLON_NOINLINE inline int recovery_table(const Team& tm, const GroupTables& tb, int n, int m, int s, const uint8_t* trusted,
                                                  int* rec_rows, double* coeff, double* ws) {
  int n_u = 0;
  for (int k = 0; k < n; ++k) n_u += trusted[k] ? 1 : 0;
  if (n_u < m) return 0;
  const bool subset = m <= SOLON_SUBSET_MAX_M;
  if (!subset && n - n_u > s) return 0;
  const int n_rec = subset ? m : n_u;
  {
    // every thread derives the same list; thread 0 stores it
    // the j-th of the n_rec rows is the trusted node number want(j) (in node order): all of them in the all-rows
    // form, m of them spread evenly over the trusted nodes in the subset form; want is only recomputed (an integer
    // division) when j moves on
    int seen = 0, next = 0;
    int want = !subset ? 0 : (m == 1 ? (n_u - 1) / 2 : ((m - 1) / 2) / (m - 1));
    for (int k = 0; k < n && next < n_rec; ++k) {
      if (!trusted[k]) continue;
      if (seen == want) {
        if (SOLON_TID == 0) rec_rows[next] = k;
        ++next;
        want = !subset ? next : (m == 1 ? n : (next * (n_u - 1) + (m - 1) / 2) / (m - 1));
      }
      ++seen;
    }
  }
  SOLON_SYNC();
  if (subset) {
    // Lagrange form of the inverse Vandermonde: row j holds the monomial coefficients of
    // L_j(w) = prod_{i != j} (w - x_i) / (x_j - x_i), built by multiplying one factor at a time.
    SOLON_FOR_THREADS(j, m) {
      double c[SOLON_SUBSET_MAX_M];
#pragma unroll
      for (int l = 0; l < SOLON_SUBSET_MAX_M; ++l) c[l] = l == 0 ? 1.0 : 0.0;
      const double xj = tb.w[rec_rows[j]];
      double denom = 1.0;
      for (int i = 0; i < m; ++i) {
        if (i == j) continue;
        const double xi = tb.w[rec_rows[i]];
#pragma unroll
        for (int l = SOLON_SUBSET_MAX_M - 1; l >= 1; --l) c[l] = fma(-xi, c[l], c[l - 1]);   // times (w - x_i)
        c[0] = -xi * c[0];
        denom *= xj - xi;
      }
      const double inv = 1.0 / denom;
#pragma unroll
      for (int l = 0; l < SOLON_SUBSET_MAX_M; ++l)
        if (l < m) coeff[(size_t)j * m + l] = c[l] * inv;
    }
    SOLON_SYNC();
    return n_rec;
  }
  // All trusted rows: coefficients in the orthonormal basis after deleting the untrusted nodes V,
  //   c' = (Q_U^T + Q_V^T (I - H_VV)^{-1} H_VU) z_U,  then monomial coefficients  y = Mt c'.
  const int nv = n - n_u;
  double* S = ws;                               // nv x nv
  double* aug = S + (size_t)nv * nv;            // nv x 2nv
  double* Z = aug + 2 * (size_t)nv * nv;        // nv x n_u:  S^{-1} H_VU
  double* Wc = Z + (size_t)nv * n_u;            // m x n_u:   Q_U^T + Q_V^T Z
  int* vlist = reinterpret_cast<int*>(Wc + (size_t)m * n_u);   // nv
  SOLON_FOR_THREADS(k, n) {
    if (!trusted[k]) {
      int pos = 0;
      for (int o = 0; o < k; ++o) pos += trusted[o] ? 0 : 1;
      vlist[pos] = k;
    }
  }
  SOLON_SYNC();
  if (nv > 0) {
    deletion_inverse(tm, tb, n, vlist, nv, S, aug);
    SOLON_FOR_THREADS(idx, nv * n_u) {
      const int a = idx / n_u, u = idx - a * n_u;
      double acc = 0.0;
      for (int b = 0; b < nv; ++b) {
        double h = 0.0;
        for (int i = 0; i < m; ++i) h = fma(tb.Qb[(size_t)i * n + vlist[b]], tb.Qb[(size_t)i * n + rec_rows[u]], h);
        acc = fma(S[(size_t)a * nv + b], h, acc);
      }
      Z[idx] = acc;
    }
    SOLON_SYNC();
  }
  SOLON_FOR_THREADS(idx, m * n_u) {
    const int i = idx / n_u, u = idx - i * n_u;
    double acc = tb.Qb[(size_t)i * n + rec_rows[u]];
    for (int a = 0; a < nv; ++a) acc = fma(tb.Qb[(size_t)i * n + vlist[a]], Z[(size_t)a * n_u + u], acc);
    Wc[idx] = acc;
  }
  SOLON_SYNC();
  SOLON_FOR_THREADS(idx, n_u * m) {
    const int u = idx / m, l = idx - u * m;
    double acc = 0.0;
    for (int i = 0; i < m; ++i) acc = fma(tb.Mt[(size_t)l * m + i], Wc[(size_t)i * n_u + u], acc);
    coeff[(size_t)u * m + l] = acc;
  }
  SOLON_SYNC();
  return n_rec;
}

// Group preparation shared by all tasks of a group.
//   rho (K x n), nu (n): this group's projected values and energies
//   forced[k] = 1 for nodes whose values are not finite (corrupt by inspection; their rho_n is 0)
//   rho_n = rho / sqrt(2 median nu), clamped to +-SOLON_RHO_CLAMP medians of |rho| per projection
//   *tau_eff = tau, or (median energy 0: all-zero data, any deviation counts) 1e-10 of the largest |rho|
// scratch: K + 2 doubles.
SOLON_HD inline void locate_prepare(const Team& tm, int n, int K, const double* rho, const double* nu, double tau, uint8_t* forced,
                                    double* rho_n, double* tau_eff, double* scratch) {
  SOLON_FOR_THREADS(k, n) {
    bool finite = isfinite(nu[k]);
    for (int kappa = 0; kappa < K; ++kappa) finite = finite && isfinite(rho[(size_t)kappa * n + k]);
    forced[k] = finite ? 0 : 1;
  }
  SOLON_FOR_THREADS(i, K + 1) scratch[i] = 0.0;
  SOLON_SYNC();
  int n_fin = 0;
  for (int k = 0; k < n; ++k) n_fin += forced[k] ? 0 : 1;
  // lower medians by rank counting among the finite nodes: scratch[0] <- median nu,
  // scratch[1 + kappa] <- median |rho_kappa|
  SOLON_FOR_THREADS(idx, (K + 1) * n) {
    const int which = idx / n, i = idx - which * n;
    if (!forced[i]) {
      const double* src = which == 0 ? nu : rho + (size_t)(which - 1) * n;
      const double mine = fabs(src[i]);
      int rank = 0;
      for (int o = 0; o < n; ++o) {
        if (forced[o]) continue;
        const double other = fabs(src[o]);
        rank += (other < mine || (other == mine && o < i)) ? 1 : 0;
      }
      if (rank == (n_fin - 1) / 2) scratch[which] = mine;
    }
  }
  SOLON_SYNC();
  const double med = n_fin > 0 ? scratch[0] : 0.0;
  const double scale = med > 0.0 ? sqrt(2.0 * med) : 1.0;
  if (med > 0.0) {
    *tau_eff = tau;
  } else {
    // all-zero honest data: any deviation counts, down to the rounding of the largest value present
    double big = 0.0;
    for (int idx = 0; idx < K * n; ++idx) {
      const double v = forced[idx % n] ? 0.0 : fabs(rho[idx]);
      big = v > big ? v : big;
    }
    *tau_eff = 1e-10 * big;
  }
  SOLON_FOR_THREADS(idx, K * n) {
    const int kappa = idx / n, i = idx - kappa * n;
    double v = forced[i] ? 0.0 : rho[idx];
    const double cap = scratch[1 + kappa] * SOLON_RHO_CLAMP;
    if (cap > 0.0) v = v > cap ? cap : (v < -cap ? -cap : v);
    rho_n[idx] = v / scale;
  }
  SOLON_SYNC();
}

// Group epilogue: pick the smallest accepted error count (else the best-fitting guess), write the
// mask over the group's n nodes, and build the recovery table from the trusted nodes.
//   recs[s+1], flags[(s+1) x flags_ld] from the tasks; forced from locate_prepare
//   trusted: n bytes scratch; ws: locate_epilogue_ws_doubles(n, m, s)
// Returns 1 if the group decoded, 0 if not.  *t_out: corrupt nodes located (-1 if undecodable).
SOLON_HD inline int locate_epilogue(const Team& tm, const GroupTables& tb, int n, int m, int s, const uint8_t* forced,
                                    const TaskRecord* recs, const uint8_t* flags, int flags_ld, uint8_t* mask,
                                    int* t_out, int* rec_rows, int* n_rec_out, double* coeff, uint8_t* trusted,
                                    double* ws) {
  int chosen = 0, ok = 0;
  for (int t = 0; t <= s; ++t) {
    if (recs[t].accept) {
      chosen = t;
      ok = 1;
      break;
    }
  }
  if (!ok) {
    double best = INFINITY;
    for (int t = 0; t <= s; ++t) {
      if (recs[t].max_fit < best) {
        best = recs[t].max_fit;
        chosen = t;
      }
    }
  }
  SOLON_FOR_THREADS(k, n) {
    const uint8_t corrupt = (flags[(size_t)chosen * flags_ld + k] || forced[k]) ? 1 : 0;
    trusted[k] = corrupt ? 0 : 1;
    mask[k] = corrupt;
  }
  SOLON_SYNC();
  int n_bad = 0;
  for (int k = 0; k < n; ++k) n_bad += trusted[k] ? 0 : 1;
  if (n_bad > s) ok = 0;
  int n_rec;
  if (tb.n_sets > 0 && n_bad <= s) {
    // tabulated at plan time for every set of at most s untrusted nodes
    const int idx = corrupt_set_index(n, trusted);
    n_rec = m <= SOLON_SUBSET_MAX_M ? m : n - n_bad;      // what recovery_table returns for at most s untrusted nodes
    const int* rows_t = tb.tab_rows + (size_t)idx * tb.tab_ld;
    const double* coeff_t = tb.tab_coeff + (size_t)idx * tb.tab_ld * m;
    SOLON_FOR_THREADS(j, n_rec) rec_rows[j] = rows_t[j];
    SOLON_FOR_THREADS(i, n_rec * m) coeff[i] = coeff_t[i];
    SOLON_SYNC();
  } else {
    n_rec = recovery_table(tm, tb, n, m, s, trusted, rec_rows, coeff, ws);
  }
  if (n_rec == 0) ok = 0;
  if (SOLON_TID == 0) {
    *n_rec_out = n_rec;
    *t_out = ok ? n_bad : -1;
  }
  SOLON_SYNC();
  return ok;
}

}  // namespace solon
