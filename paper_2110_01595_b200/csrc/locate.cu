// Locator kernel (phi of Section 3.4) and recovery table (the inverse inside psi), on the device, plus
// the host mirror solon_locate_host built from the same source (locate_core.cuh).
//
// One CTA per group; warp t of it assumes exactly t corrupt nodes, so all error counts are tried
// concurrently.  The CTA then picks the smallest accepted count, writes the group's part of the mask and
// builds the recovery table.  The kernel is launched as a programmatic dependent of the projection kernel
// and can do all of that ahead of time on a partial projection, leaving only a check for afterwards (see the
// comment on the passes inside the kernel).
#include <vector>

#include "locate_core.cuh"
#include "projection_draw.cuh"
#include "solon_internal.h"

namespace solon {

struct LocateParams {
  const int* group_start;
  const double* w;       // P node scalars
  const double* rho;     // K x P
  const double* nu;      // P
  const double* qb;      // per group n_g x n_g orthonormal polynomial tables, group g at qb_off[g]
  const double* hm;      // per group n_g x n_g projector tables, same offsets
  const int64_t* qb_off; // q
  const double* mt;      // q x m x m
  const double* tch;     // P x (s + 1)
  const int* tab_count;       // recovery tables per corrupt set, all groups: rows in use per set
  const int* tab_rows;        // tab_ld ints per set
  const double* tab_coeff;    // tab_ld x m doubles per set
  const int64_t* tab_off;     // q: first set of group g
  const int* tab_sets;        // q: number of sets of group g (0: not tabulated)
  int tab_ld;
  int use_tabs;               // look recovery tables up (else compute them): pays when the tables survive in L2 between decodes
  int P, m, s, K;
  double tau;
  double* ws_global;     // q x ws_stride doubles, used when shared memory is too small
  size_t ws_stride;
  int use_smem;
  const double* bunch_sums;   // n_bunches x (K + 1) x P partial sums of the projection kernel (rho rows, then nu)
  int n_bunches;              // 0: rho and nu are final
  double* rho_w;              // with n_bunches > 0 the sums are also written here (K x P) and to nu_w (P)
  double* nu_w;
  const double* bunch_a;      // same shape as bunch_sums: the sums over part A of the projection kernel's column ranges
  const unsigned long long* progress;   // bunches whose part-A sums [0] and final sums [1] are complete in this decode
  unsigned long long progress_target;   // its value once part A is complete
  int* early;                 // q: outcome of the early run per group (see solon_plan_get_early_outcome)
  int spec;                   // work on part A while the projection kernel streams part B, then only check the result
  unsigned long long* tile_counter;   // work counter of the recovery kernel, zeroed here
  int stage_tables;      // copy the group's tables to shared memory (they follow the workspace)
  uint8_t* mask;         // P (caller's buffer)
  int* t_acc;            // q
  int* n_rec;            // q
  int* rec_rows;         // P
  double* coeff;         // P x m
  int* status;
  int* opt;              // optimistic decode: opt[8 + g] counts (up to 2) the decodes in a row in which the rows of group g's previous
                         // recovery table were all trusted (0: not in this decode)
  int opt_track;         // the plan can decode optimistically (m <= 6): keep opt[8 + g] (else it is written as 0)
  int opt_given_projections;      // this decode's projections did not come from the plan's own projection kernel just before (given by the
                         // caller): no aggregate was recovered ahead, whatever opt[1] still says from an earlier decode
  DrawParams draw;       // the vectors f of the next decode, written by the CTAs beyond the q locator CTAs (n_draw_ctas of them)
  int n_draw_ctas;
};

DrawParams draw_params(const solon_plan* plan);   // plan.cu

// Workspace of one group, shared by the device kernel and the host mirror.
struct GroupScratch {
  int* rows_l;           // n      recovery rows (local copy, written out at the end)
  uint8_t* trusted;      // n
  uint8_t* mask_l;       // n
  uint8_t* forced;       // n
  uint8_t* flags;        // (s + 1) x n   located nodes per error count
  TaskRecord* recs;      // s + 1
  double* rho_in;        // K x n  staged inputs
  double* nu_in;         // n
  double* rho_n;         // K x n
  double* scratch;       // K + 2
  double* coeff_l;       // n x m
  uint8_t* warm_trusted; // n      outputs and workspace of the recovery table's rehearsal (never read)
  int* warm_rows;        // n
  double* warm_coeff;    // n x m
  double* warm_ws;       // locate_epilogue_ws_doubles
  double* tasks;         // (s + 1) x task_stride, reused by the epilogue
  size_t task_stride;
};

// cand / bad bytes followed by the task's doubles
SOLON_HD static inline size_t task_stride_doubles(int n, int m, int K, int s) {
  return 2 * ((size_t)n / 8 + 1) + locate_task_ws_doubles(n, m, K, s);
}

SOLON_HD static inline size_t group_ws_doubles(int n, int m, int K, int s) {
  size_t tasks = (size_t)(s + 1) * task_stride_doubles(n, m, K, s);
  size_t epi = locate_epilogue_ws_doubles(n, m, s);
  size_t warm = ((size_t)n / 8 + 1) + ((size_t)(n + 1) / 2 + 1) + (size_t)n * m + epi;
  return ((size_t)(n + 1) / 2 + 1) + 3 * ((size_t)n / 8 + 1) + ((size_t)(s + 1) * n / 8 + 1) + 2 * (size_t)(s + 1) +
         (size_t)(2 * K + 1) * n + K + 2 + (size_t)n * m + warm + (tasks > epi ? tasks : epi) + 8;
}

SOLON_HD static inline GroupScratch carve(double* ws, int n, int m, int K, int s) {
  GroupScratch sc;
  double* p = ws;
  sc.rows_l = reinterpret_cast<int*>(p);         p += (n + 1) / 2 + 1;
  sc.trusted = reinterpret_cast<uint8_t*>(p);    p += n / 8 + 1;
  sc.mask_l = reinterpret_cast<uint8_t*>(p);     p += n / 8 + 1;
  sc.forced = reinterpret_cast<uint8_t*>(p);     p += n / 8 + 1;
  sc.flags = reinterpret_cast<uint8_t*>(p);      p += (size_t)(s + 1) * n / 8 + 1;
  sc.recs = reinterpret_cast<TaskRecord*>(p);    p += 2 * (size_t)(s + 1);
  sc.rho_in = p;                                 p += (size_t)K * n;
  sc.nu_in = p;                                  p += n;
  sc.rho_n = p;                                  p += (size_t)K * n;
  sc.scratch = p;                                p += K + 2;
  sc.coeff_l = p;                                p += (size_t)n * m;
  sc.warm_trusted = reinterpret_cast<uint8_t*>(p); p += n / 8 + 1;
  sc.warm_rows = reinterpret_cast<int*>(p);      p += (n + 1) / 2 + 1;
  sc.warm_coeff = p;                             p += (size_t)n * m;
  sc.warm_ws = p;                                p += locate_epilogue_ws_doubles(n, m, s);
  sc.tasks = p;
  sc.task_stride = task_stride_doubles(n, m, K, s);
  return sc;
}

// One CTA per group, one warp per error count: warp t assumes exactly t corrupt nodes, all counts are tried
// at the same time with warp-level synchronisation only; afterwards the whole CTA picks the smallest
// accepted count, writes the group's part of the mask and builds the recovery table.  No CTA waits on
// another one.
__device__ __forceinline__ unsigned long long pipe_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Optimistic decode: 1 if the m rows of the group's previous recovery table are all trusted by this decode's mask (then an
// aggregate recovered from them is this decode's aggregate, and the table would have served this decode too).
__device__ __forceinline__ int old_rows_trusted(const LocateParams& prm, const int* old_row, int old_n, int t_acc, const uint8_t* mask_l,
                                                int row0, int n) {
  if (!prm.opt_track || t_acc < 0 || old_n != prm.m) return 0;
  for (int j = 0; j < prm.m; ++j) {
    const int k = old_row[j] - row0;
    if (k < 0 || k >= n || mask_l[k]) return 0;
  }
  return 1;
}

constexpr int kGatherBatch = 20;   // bunch sums fetched at once per column (the projection kernel leaves 37 on 148 SMs: two rounds)

__global__ void __launch_bounds__(32 * (SOLON_MAX_S + 1)) locate_kernel(LocateParams prm) {
  extern __shared__ __align__(16) double smem_ws[];
  const int g = blockIdx.x;
  const int tid = threadIdx.x, n_threads = blockDim.x;
  if (g >= (int)gridDim.x - prm.n_draw_ctas) {
    // Not a locator CTA: these draw the vectors f of the NEXT decode (Algorithm 1 draws its random vector anew in every
    // decode) into the buffer the projection kernel just before this one did not read, while the locator's few CTAs
    // work and the rest of the GPU would be idle.  The projection kernel must be done with the draw count first.
    pdl_trigger();
    pdl_wait();
    draw_projection_vectors(prm.draw, 1, g - ((int)gridDim.x - prm.n_draw_ctas), prm.n_draw_ctas, tid, n_threads);
    return;
  }
  if (g == 0 && tid == 0 && prm.opt_given_projections) prm.opt[1] = 0;     // (the recovery kernel reads it after this grid)
  const int row0 = prm.group_start[g];
  const int n = prm.group_start[g + 1] - row0;
  double* ws = prm.use_smem ? smem_ws : prm.ws_global + (size_t)g * prm.ws_stride;
  GroupScratch sc = carve(ws, n, prm.m, prm.K, prm.s);
  __shared__ int s_n_rec, s_t_acc;
  // Optimistic decode: the rows of this group's recovery table as the previous decode left it - the rows the projection
  // kernel of THIS decode may have recovered from - are read before anything here overwrites them.
  __shared__ int s_old_row[SOLON_SUBSET_MAX_M], s_old_n, s_old_streak;
  if (prm.opt_track) {
    if (tid < prm.m) s_old_row[tid] = prm.rec_rows[row0 + tid];
    if (tid == 0) {
      s_old_n = prm.n_rec[g];
      s_old_streak = prm.opt[8 + g];
    }
  }
  GroupTables tb;
  tb.Qb = prm.qb + prm.qb_off[g];
  tb.Hm = prm.hm + prm.qb_off[g];
  tb.Mt = prm.mt + (size_t)g * prm.m * prm.m;
  tb.Tch = prm.tch + (size_t)row0 * (prm.s + 1);
  tb.w = prm.w + row0;
  tb.n_sets = prm.use_tabs ? prm.tab_sets[g] : 0;
  tb.tab_ld = prm.tab_ld;
  tb.tab_count = prm.tab_count + prm.tab_off[g];
  tb.tab_rows = prm.tab_rows + (size_t)prm.tab_off[g] * prm.tab_ld;
  tb.tab_coeff = prm.tab_coeff + (size_t)prm.tab_off[g] * prm.tab_ld * prm.m;
  if (prm.stage_tables) {
    // small groups: one coalesced pass brings the plan's tables on chip, so the dependent reads of the
    // solver never wait on L2 or HBM (the tables are evicted by the streaming kernels between decodes)
    double* qb_s = smem_ws + prm.ws_stride;
    double* hm_s = qb_s + (size_t)n * n;
    double* tch_s = hm_s + (size_t)n * n;
    double* w_s = tch_s + (size_t)n * (prm.s + 1);
    for (int i = tid; i < n * n; i += n_threads) {
      qb_s[i] = tb.Qb[i];
      hm_s[i] = tb.Hm[i];
    }
    for (int i = tid; i < n * (prm.s + 1); i += n_threads) tch_s[i] = tb.Tch[i];
    for (int i = tid; i < n; i += n_threads) w_s[i] = tb.w[i];
    tb.Qb = qb_s;
    tb.Hm = hm_s;
    tb.Tch = tch_s;
    tb.w = w_s;
  }
  const Team cta = Team::cta();
  pdl_trigger();   // the recovery kernel may be scheduled early; it waits for this grid before reading the table
  // Up to three passes over the same code; the last one is the decode proper, after the projections are complete.
  // The others (prm.spec) run while the projection kernel is still streaming and write nothing outside this CTA's
  // scratch.  Pass 0: that kernel announces the sums over part A of its column ranges early - a random projection
  // of those columns, as good as any for locating whoever lies there - and the whole locator runs on them.  The last
  // pass then only checks, on the final sums, that the set found is exactly the set of nodes that do not fit
  // (locate_check): the mask and the recovery table depend on that set alone.  If the check fails (an attacker who
  // spared part A, a timed-out wait) it runs the whole locator as usual.  Pass 1 rehearses that check on the part-A
  // sums: between decodes gigabytes stream through L2, and pass 0's solver has pushed the few instructions of the
  // check out of the SM's instruction cache again, so without it each step of the check would wait for HBM.
  __shared__ int s_ready, s_spec_ok;
  if (tid == 0) {
    s_spec_ok = 0;
    s_ready = 0;
  }
#pragma unroll 1
  for (int pass = prm.spec ? 0 : 2; pass < 3; ++pass) {
    const bool spec0 = pass == 0;
    const bool last = pass == 2;
    if (pass == 1 && !s_spec_ok) continue;     // nothing to rehearse
    if (last) {
      pdl_wait();   // the projections are complete and visible (everything above only read plan tables)
      if (g == 0 && tid == 0) *prm.tile_counter = 0ULL;   // the recovery kernel reads it only after this grid is done
    }
    if (spec0) {
      // wait (bounded: 2 ms) until every bunch of the projection kernel has added up its part A.  That kernel was
      // resident as a whole before this one could start and never waits for anything, so the count always comes.
      if (tid == 0) {
        int ready = 0;
        unsigned long long seen;
        asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(seen) : "l"(prm.progress + 1) : "memory");
        if (seen >= prm.progress_target) {
          ready = -1;      // this CTA became resident only after the projections were complete: nothing to gain
        } else {
          const unsigned long long t_start = pipe_timer_ns();
          for (;;) {
            asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(seen) : "l"(prm.progress) : "memory");
            if (seen >= prm.progress_target) {
              ready = 1;
              break;
            }
            if (pipe_timer_ns() - t_start > 2000000ull) break;
            __nanosleep(200);
          }
        }
        s_ready = ready;
      }
      __syncthreads();
      if (s_ready <= 0) continue;      // nothing to go on: the last pass does all the work
    }
    if (prm.s == 0) {
      // pure compression code: nothing to locate, every node is trusted
      for (int k = tid; k < n; k += n_threads) {
        sc.forced[k] = 0;
        sc.flags[k] = 0;
      }
      if (tid == 0) {
        sc.recs[0].accept = 1;
        sc.recs[0].n_flagged = 0;
        sc.recs[0].max_fit = 0.0;
      }
    } else {
      // one parallel round trip brings the group's projected values on chip
      if (prm.n_bunches > 0) {
        // last level of the projection kernel's reduction, for this group's columns only: a thread fetches all
        // bunch sums of its column at once and adds them in bunch order
        const int n_cols = (prm.K + 1) * n;
        const size_t n_acc = (size_t)(prm.K + 1) * prm.P;
        const double* sums = last ? prm.bunch_sums : prm.bunch_a;
        for (int c = tid; c < n_cols; c += n_threads) {
          const int which = c / n, i = c - which * n;
          const double* src = sums + (size_t)which * prm.P + row0 + i;
          double acc = 0.0;
          for (int b0 = 0; b0 < prm.n_bunches; b0 += kGatherBatch) {
            double v[kGatherBatch];
#pragma unroll
            for (int u = 0; u < kGatherBatch; ++u) v[u] = b0 + u < prm.n_bunches ? __ldcg(src + (size_t)(b0 + u) * n_acc) : 0.0;
#pragma unroll
            for (int u = 0; u < kGatherBatch; ++u) acc += v[u];
          }
          if (which < prm.K) {
            sc.rho_in[(size_t)which * n + i] = acc;
            if (last) prm.rho_w[(size_t)which * prm.P + row0 + i] = acc;
          } else {
            sc.nu_in[i] = acc;
            if (last) prm.nu_w[row0 + i] = acc;
          }
        }
        __syncthreads();
      }
      for (int i = tid; i < n; i += n_threads) {
        if (last) {
          if (prm.n_bunches > 0) continue;
          sc.nu_in[i] = prm.nu[row0 + i];
          for (int kappa = 0; kappa < prm.K; ++kappa) sc.rho_in[(size_t)kappa * n + i] = prm.rho[(size_t)kappa * prm.P + row0 + i];
        }
      }
      __syncthreads();
      double tau_eff = 0.0;
      locate_prepare(cta, n, prm.K, sc.rho_in, sc.nu_in, prm.tau, sc.forced, sc.rho_n, &tau_eff, sc.scratch);
      bool confirmed = false;
      if (pass >= 1 && s_spec_ok) {
        // the set found on part A, checked on the final sums by the whole CTA
        uint8_t* cand = reinterpret_cast<uint8_t*>(sc.tasks);
        uint8_t* bad = cand + 8 * ((size_t)n / 8 + 1);
        confirmed = locate_check(cta, tb, n, prm.K, prm.s, sc.rho_n, sc.forced, tau_eff, sc.mask_l, cand, bad,
                                 sc.tasks + 2 * ((size_t)n / 8 + 1), &sc.recs[0]) != 0;
      }
      if (pass == 1) continue;     // the rehearsal ends here, whatever the check said
      if (confirmed) {
        // mask, recovery rows and weights of pass 0 stand as they are
        for (int k = tid; k < n; k += n_threads) prm.mask[row0 + k] = sc.mask_l[k];
        const int n_rec = s_n_rec;
        for (int j = tid; j < n_rec; j += n_threads) prm.rec_rows[row0 + j] = sc.rows_l[j] + row0;
        for (int i = tid; i < n_rec * prm.m; i += n_threads) prm.coeff[(size_t)row0 * prm.m + i] = sc.coeff_l[i];
        if (tid == 0) {
          prm.n_rec[g] = n_rec;
          prm.t_acc[g] = s_t_acc;
          prm.early[g] = 1;
          prm.opt[8 + g] = old_rows_trusted(prm, s_old_row, s_old_n, s_t_acc, sc.mask_l, row0, n) ? min(s_old_streak + 1, 2) : 0;
        }
        return;
      }
      const int t = tid >> 5;                       // this warp's error count
      double* task = sc.tasks + (size_t)t * sc.task_stride;
      uint8_t* cand = reinterpret_cast<uint8_t*>(task);
      uint8_t* bad = cand + 8 * ((size_t)n / 8 + 1);
      if (t <= prm.s) {    // warps beyond s + 1 only help with the CTA-wide steps
        double* tws = task + 2 * ((size_t)n / 8 + 1);
        uint8_t* tflags = sc.flags + (size_t)t * n;
        if (prm.s <= 2)
          locate_task<2>(Team::own_warp(), tb, n, prm.m, prm.K, t, prm.s, sc.rho_n, sc.forced, tau_eff, tflags, cand, bad, tws,
                         &sc.recs[t]);
        else if (prm.s <= 3)
          locate_task<3>(Team::own_warp(), tb, n, prm.m, prm.K, t, prm.s, sc.rho_n, sc.forced, tau_eff, tflags, cand, bad, tws,
                         &sc.recs[t]);
        else
          locate_task<SOLON_FAST_T>(Team::own_warp(), tb, n, prm.m, prm.K, t, prm.s, sc.rho_n, sc.forced, tau_eff, tflags, cand,
                                    bad, tws, &sc.recs[t]);
      }
      // Rehearsal of the recovery table.  The epilogue below runs that code once, after all the tasks, and between
      // decodes gigabytes stream through L2: fetched from HBM it takes about 10 us, for a few hundred operations.  A
      // warp with nothing else to do (else warp 0, whose task - no corrupt node - is the shortest) runs the very same
      // code now, on a made-up trusted set and into scratch that nobody reads, so that the SM's instruction cache
      // holds it when the epilogue comes.  Only for the subset form (m <= 6): the all-rows form takes a single warp
      // longer than the tasks last, and the CTA would wait for it.
      const int idle_warp = prm.s + 1 < (n_threads >> 5) ? prm.s + 1 : 0;
      if (tb.n_sets == 0 && t == idle_warp && prm.m <= SOLON_SUBSET_MAX_M) {
        const Team own = Team::own_warp();
        for (int k = own.lane; k < n; k += 32) sc.warm_trusted[k] = (k == 0 && prm.s > 0) ? 0 : 1;   // one node deleted
        __syncwarp();
        (void)recovery_table(own, tb, n, prm.m, prm.s, sc.warm_trusted, sc.warm_rows, sc.warm_coeff, sc.warm_ws);
      }
    }
    __syncthreads();
    const int ok = locate_epilogue(cta, tb, n, prm.m, prm.s, sc.forced, sc.recs, sc.flags, n, sc.mask_l, &s_t_acc, sc.rows_l,
                                   &s_n_rec, sc.coeff_l, sc.trusted, sc.tasks);
    if (pass == 0) {
      if (tid == 0) s_spec_ok = (spec0 && ok && prm.s > 0) ? 1 : 0;
      __syncthreads();
      continue;
    }
    // write the group's results: mask, recovery rows as global node indices, weights
    const int n_rec = s_n_rec;
    for (int k = tid; k < n; k += n_threads) prm.mask[row0 + k] = sc.mask_l[k];
    for (int j = tid; j < n_rec; j += n_threads) prm.rec_rows[row0 + j] = sc.rows_l[j] + row0;
    for (int i = tid; i < n_rec * prm.m; i += n_threads) prm.coeff[(size_t)row0 * prm.m + i] = sc.coeff_l[i];
    if (tid == 0) {
      prm.n_rec[g] = n_rec;
      prm.t_acc[g] = s_t_acc;
      prm.early[g] = !prm.spec ? 0 : (s_ready > 0 ? 2 : (s_ready == 0 ? 3 : 4));
      prm.opt[8 + g] = old_rows_trusted(prm, s_old_row, s_old_n, s_t_acc, sc.mask_l, row0, n) ? min(s_old_streak + 1, 2) : 0;
      (void)ok;      // an undecodable group is reported through t_acc[g] = -1
    }
  }
}

size_t locate_ws_doubles(int n, int m, int K, int s) { return group_ws_doubles(n, m, K, s); }

// Tables of one group (host, once per plan): the orthonormal polynomials q_0..q_{n-1} on the nodes
// (Gram-Schmidt, twice, of the Chebyshev polynomials T_0..T_{n-1} evaluated at the nodes), the monomial
// coefficients of q_0..q_{m-1}, and T_0..T_s at the nodes.
void build_group_tables(int n, int m, int s, const double* w, double* Qb, double* Hm, double* Mt, double* Tch) {
  typedef long double real;
  std::vector<real> T((size_t)n * n), Q((size_t)n * n), R((size_t)n * n, 0.0L);   // column-major n x n
  for (int k = 0; k < n; ++k) {
    real t0 = 1.0L, t1 = (real)w[k];
    for (int i = 0; i < n; ++i) {
      T[(size_t)i * n + k] = t0;
      real t2 = 2.0L * (real)w[k] * t1 - t0;
      t0 = t1;
      t1 = t2;
    }
  }
  Q = T;
  for (int j = 0; j < n; ++j) {
    for (int pass = 0; pass < 2; ++pass) {
      for (int i = 0; i < j; ++i) {
        real dot = 0.0L;
        for (int k = 0; k < n; ++k) dot += Q[(size_t)i * n + k] * Q[(size_t)j * n + k];
        for (int k = 0; k < n; ++k) Q[(size_t)j * n + k] -= dot * Q[(size_t)i * n + k];
        R[(size_t)i * n + j] += dot;           // R[i][j], row-major
      }
    }
    real nrm = 0.0L;
    for (int k = 0; k < n; ++k) nrm += Q[(size_t)j * n + k] * Q[(size_t)j * n + k];
    nrm = sqrtl(nrm);
    R[(size_t)j * n + j] = nrm;
    for (int k = 0; k < n; ++k) Q[(size_t)j * n + k] = nrm > 0.0L ? Q[(size_t)j * n + k] / nrm : 0.0L;
  }
  for (size_t i = 0; i < (size_t)n * n; ++i) Qb[i] = (double)Q[i];
  for (int a = 0; a < n; ++a)
    for (int b = 0; b < n; ++b) {
      real h = 0.0L;
      for (int i = 0; i < m && i < n; ++i) h += Q[(size_t)i * n + a] * Q[(size_t)i * n + b];
      Hm[(size_t)a * n + b] = (double)h;
    }
  // q_i = sum_{j<=i} Rinv[j][i] T_j (T = Q R); T_j = sum_l C[l][j] w^l with integer C from the recurrence
  std::vector<real> Rinv((size_t)m * m, 0.0L), C((size_t)m * m, 0.0L);
  for (int i = 0; i < m; ++i) {
    Rinv[(size_t)i * m + i] = 1.0L / R[(size_t)i * n + i];
    for (int r = i - 1; r >= 0; --r) {
      real acc = 0.0L;
      for (int c = r + 1; c <= i; ++c) acc += R[(size_t)r * n + c] * Rinv[(size_t)c * m + i];
      Rinv[(size_t)r * m + i] = -acc / R[(size_t)r * n + r];
    }
  }
  for (int j = 0; j < m; ++j) {
    if (j == 0) C[0] = 1.0L;
    else if (j == 1) C[(size_t)1 * m + 1] = 1.0L;
    else
      for (int l = 0; l <= j; ++l)
        C[(size_t)l * m + j] = (l > 0 ? 2.0L * C[(size_t)(l - 1) * m + (j - 1)] : 0.0L) - C[(size_t)l * m + (j - 2)];
  }
  for (int l = 0; l < m; ++l)
    for (int i = 0; i < m; ++i) {
      real acc = 0.0L;
      for (int j = 0; j <= i; ++j) acc += C[(size_t)l * m + j] * Rinv[(size_t)j * m + i];
      Mt[(size_t)l * m + i] = (double)acc;
    }
  for (int k = 0; k < n; ++k)
    for (int i = 0; i <= s; ++i) Tch[(size_t)k * (s + 1) + i] = i < n ? (double)T[(size_t)i * n + k] : 0.0;
}

// Recovery table of one group when every node is trusted (host, once per plan): what the locator writes after a decode
// that found no corrupt node.  rows: n ints, coeff: n x m doubles; returns the rows in use.
int clean_recovery_table(int n, int m, int s, const GroupTables& tb, int* rows, double* coeff) {
  std::vector<uint8_t> trusted((size_t)n, 1);
  std::vector<double> ws(locate_epilogue_ws_doubles(n, m, s) + 8);
  return recovery_table(Team::serial(), tb, n, m, s, trusted.data(), rows, coeff, ws.data());
}

// Recovery tables of one group for every set of at most s untrusted nodes (host, once per plan): entry
// corrupt_set_index(V) holds what recovery_table gives for the trusted set = complement of V.  Leaves the vectors empty
// when there are more than SOLON_MAX_SETS such sets.  ld = rows reserved per set (m in the subset form, n otherwise).
void build_recovery_tabs(int n, int m, int s, const GroupTables& tb, int ld, std::vector<int>* count, std::vector<int>* rows,
                         std::vector<double>* coeff) {
  count->clear();
  rows->clear();
  coeff->clear();
  const int n_sets = count_corrupt_sets(n, s);
  if (n_sets > SOLON_MAX_SETS) return;
  count->assign((size_t)n_sets, 0);
  rows->assign((size_t)n_sets * ld, 0);
  coeff->assign((size_t)n_sets * ld * m, 0.0);
  std::vector<uint8_t> trusted((size_t)n);
  std::vector<int> r((size_t)n), V;
  std::vector<double> c((size_t)n * m), ws(locate_epilogue_ws_doubles(n, m, s) + 8);
  const Team tm = Team::serial();
  for (int t = 0; t <= s && t <= n; ++t) {
    V.resize(t);
    for (int i = 0; i < t; ++i) V[i] = i;
    for (;;) {
      for (int k = 0; k < n; ++k) trusted[k] = 1;
      for (int i = 0; i < t; ++i) trusted[V[i]] = 0;
      const int idx = corrupt_set_index(n, trusted.data());
      const int n_rec = recovery_table(tm, tb, n, m, s, trusted.data(), r.data(), c.data(), ws.data());
      (*count)[idx] = n_rec;
      for (int j = 0; j < n_rec; ++j) (*rows)[(size_t)idx * ld + j] = r[j];
      for (int i = 0; i < n_rec * m; ++i) (*coeff)[(size_t)idx * ld * m + i] = c[i];
      int i = t - 1;                       // next combination
      while (i >= 0 && V[i] == n - t + i) --i;
      if (i < 0) break;
      ++V[i];
      for (int j = i + 1; j < t; ++j) V[j] = V[j - 1] + 1;
    }
  }
}

int launch_locate(solon_plan* plan, uint8_t* byz_mask, const double* rho, const double* nu) {
  LocateParams prm;
  prm.group_start = plan->d_group_start;
  prm.w = plan->d_w;
  prm.rho = rho ? rho : plan->d_rho;
  prm.nu = nu ? nu : plan->d_nu;
  // the decode proper: the projection kernel stopped one level short and left its bunch sums
  const bool fused = !rho && !nu && plan->s > 0 && plan->proj_bunches > 0;
  prm.bunch_sums = fused ? plan->proj_bunch_sums : nullptr;
  prm.n_bunches = fused ? plan->proj_bunches : 0;
  prm.rho_w = plan->d_rho;
  prm.nu_w = plan->d_nu;
  prm.bunch_a = fused ? plan->proj_bunch_a : nullptr;
  prm.progress = plan->d_proj_progress;
  prm.progress_target = plan->proj_progress_target;
  prm.early = plan->d_early;
  prm.qb = plan->d_qb;
  prm.hm = plan->d_hm;
  prm.qb_off = plan->d_qb_off;
  prm.mt = plan->d_mt;
  prm.tch = plan->d_tch;
  prm.tab_count = plan->d_tab_count;
  prm.tab_rows = plan->d_tab_rows;
  prm.tab_coeff = plan->d_tab_coeff;
  prm.tab_off = plan->d_tab_off;
  prm.tab_sets = plan->d_tab_sets;
  prm.tab_ld = plan->tab_ld;
  prm.use_tabs = plan->stream_hints;
  prm.P = plan->P; prm.m = plan->m; prm.s = plan->s; prm.K = plan->K;
  prm.tau = plan->tau;
  prm.ws_global = plan->d_locate_ws;
  prm.ws_stride = plan->locate_ws_stride;
  prm.mask = byz_mask;
  prm.t_acc = plan->d_t_acc;
  prm.n_rec = plan->d_n_rec;
  prm.rec_rows = plan->d_rec_rows;
  prm.coeff = plan->d_coeff;
  prm.status = plan->d_status;
  prm.tile_counter = plan->d_tile_counter;
  size_t need = locate_ws_doubles(plan->max_group, plan->m, plan->K, plan->s) * sizeof(double);
  if (need > plan->locate_ws_stride * sizeof(double)) return SOLON_ERR_INTERNAL;
  prm.use_smem = need <= 128 * 1024 ? 1 : 0;
  // working ahead on part A pays for a small solver beside a long projection pass (about 6 GB per ms); otherwise it
  // would still be at it when the projections end
  prm.spec = (fused && (plan->proj_two_parts || (early_locator_starved(plan) && uses_early_locator(plan)))) ? 1 : 0;
  size_t smem = prm.use_smem ? need : 0;
  const size_t tables = (2 * (size_t)plan->max_group * plan->max_group + (size_t)plan->max_group * (plan->s + 2)) * sizeof(double);
  prm.stage_tables = (prm.use_smem && smem + tables <= 200 * 1024) ? 1 : 0;
  if (prm.stage_tables) {
    prm.ws_stride = need / sizeof(double);      // the tables follow the workspace in shared memory
    smem += tables;
  }
  if (smem > 48 * 1024)
    SOLON_CUDA_TRY(cudaFuncSetAttribute(locate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  prm.opt = plan->d_opt;
  prm.opt_track = plan->opt_rows > 0 ? 1 : 0;
  prm.opt_given_projections = (rho || nu) ? 1 : 0;
  // CTAs that draw the next decode's vectors beside the locator's: a few per SM, a thread per several quads
  prm.draw = draw_params(plan);
  prm.n_draw_ctas = 0;
  if (plan->fresh_f && plan->s > 0) {
    const int64_t quads = ((plan->d_c + 3) / 4) * plan->K;
    int64_t want = (quads + 127) / 128;
    const int64_t cap = (int64_t)plan->num_sms * 8;      // more CTAs per SM than eight bought nothing
    prm.n_draw_ctas = (int)(want < cap ? (want < 1 ? 1 : want) : cap);
  }
  plan->last_decode_advanced = prm.n_draw_ctas > 0 ? 1 : 0;
  if (prm.n_draw_ctas > 0) plan->draw_parity = -1;      // the count moves on the device from here on
  plan->launches += 1;
  // one warp per error count, at least four for the CTA-wide steps (four still fit, at 128 registers a thread, in the
  // slot the projection kernel leaves free, so the CTA is resident early)
  const int warps = plan->s + 1 < 4 ? 4 : plan->s + 1;
  return launch_dependent(locate_kernel, dim3(plan->q + prm.n_draw_ctas), dim3(32 * warps), smem, plan->stream, prm);
}

}  // namespace solon

using namespace solon;

extern "C" int solon_locate_host(int n, int m, int s, int K, const double* rho, const double* nu, const double* w_g,
                                 double tau, uint8_t* mask, int* t_out, int* rec_rows, int* n_rec, double* coeff) {
  if (!rho || !nu || !w_g || !mask || !t_out || !rec_rows || !n_rec || !coeff) return SOLON_ERR_INVALID_ARG;
  if (n < 1 || n > SOLON_MAX_GROUP || m < 1 || m > SOLON_MAX_M || s < 0 || s > SOLON_MAX_S || K < 1 ||
      K > SOLON_MAX_PROJECTIONS || n < 2 * s + m)
    return SOLON_ERR_INVALID_ARG;
  std::vector<double> Qb((size_t)n * n), Hm((size_t)n * n), Mt((size_t)m * m), Tch((size_t)n * (s + 1));
  build_group_tables(n, m, s, w_g, Qb.data(), Hm.data(), Mt.data(), Tch.data());
  GroupTables tb;
  tb.Qb = Qb.data();
  tb.Hm = Hm.data();
  tb.Mt = Mt.data();
  tb.Tch = Tch.data();
  tb.w = w_g;
  tb.n_sets = 0;
  tb.tab_ld = m <= SOLON_SUBSET_MAX_M ? m : n;
  tb.tab_count = nullptr;
  tb.tab_rows = nullptr;
  tb.tab_coeff = nullptr;
  std::vector<int> tab_count, tab_rows;
  std::vector<double> tab_coeff;
  build_recovery_tabs(n, m, s, tb, tb.tab_ld, &tab_count, &tab_rows, &tab_coeff);
  tb.n_sets = (int)tab_count.size();
  tb.tab_count = tab_count.data();
  tb.tab_rows = tab_rows.data();
  tb.tab_coeff = tab_coeff.data();
  std::vector<double> ws(group_ws_doubles(n, m, K, s) + 64);
  GroupScratch sc = carve(ws.data(), n, m, K, s);
  const Team tm = Team::serial();
  double tau_eff = 0.0;
  if (s > 0) {
    locate_prepare(tm, n, K, rho, nu, tau, sc.forced, sc.rho_n, &tau_eff, sc.scratch);
    for (int t = 0; t <= s; ++t) {
      double* task = sc.tasks + (size_t)t * sc.task_stride;
      uint8_t* cand = reinterpret_cast<uint8_t*>(task);
      uint8_t* bad = cand + 8 * ((size_t)n / 8 + 1);
      locate_task<SOLON_FAST_T>(tm, tb, n, m, K, t, s, sc.rho_n, sc.forced, tau_eff, sc.flags + (size_t)t * n, cand, bad,
                  task + 2 * ((size_t)n / 8 + 1), &sc.recs[t]);
    }
  } else {
    for (int k = 0; k < n; ++k) sc.forced[k] = sc.flags[k] = 0;
    sc.recs[0].accept = 1;
    sc.recs[0].n_flagged = 0;
    sc.recs[0].max_fit = 0.0;
  }
  const int ok = locate_epilogue(tm, tb, n, m, s, sc.forced, sc.recs, sc.flags, n, mask, t_out, rec_rows, n_rec, coeff,
                                 sc.trusted, sc.tasks);
  return ok ? SOLON_OK : SOLON_ERR_UNDECODABLE;
}
