// Internal definitions shared by the translation units of libsolon (not part of the C interface).
#pragma once

#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>
#include <stdint.h>

#include <vector>

#include "../../include/solon.h"

#define SOLON_CUDA_TRY(expr)                   \
  do {                                         \
    cudaError_t solon_err__ = (expr);          \
    if (solon_err__ != cudaSuccess) {          \
      (void)cudaGetLastError();                \
      return SOLON_ERR_CUDA;                   \
    }                                          \
  } while (0)

namespace solon {

// Device-side view of the group layout, passed by value to kernels.
struct GroupTable {
  const int* start;   // q + 1 entries, device
  const double* w;    // P node scalars, device
  int q;
  int P;
};

// Bit positions of the device status word.
enum : int {
  kStatusUndecodable = 1,  // some group had no consistent set of <= s corrupt nodes
  kStatusWaitExpired = 2,  // a bounded wait on a shared-memory barrier ran out
};

}  // namespace solon

struct solon_plan {
  int P, s, m, r, K;
  int dtype;               // SOLON_F32 or SOLON_F64: element type of gradients, coded vectors and aggregate
  int64_t d, d_c;
  uint64_t seed;
  double tau;
  int lsq_rows;
  cudaStream_t stream;
  int device;
  int num_sms;
  int64_t launches;
  int stream_hints;        // the streaming kernels mark what they move evict-first in L2 (see keeps_l2_for_code)

  // host copies
  std::vector<int> group_start;   // q + 1
  std::vector<int> group_of;      // P
  std::vector<double> w;          // P
  int q;
  int max_group;

  // device tables
  int* d_group_start;      // q + 1
  int* d_group_of;         // P
  double* d_w;             // P (float64 node scalars)
  double* d_qb;            // per group n_g x n_g orthonormal polynomial tables (locator)
  double* d_hm;            // per group n_g x n_g projectors on the polynomials of degree < m (same offsets)
  int64_t* d_qb_off;       // q offsets into d_qb
  double* d_mt;            // q x m x m monomial coefficients of the first m orthonormal polynomials
  double* d_tch;           // P x (s + 1) Chebyshev polynomials at the nodes
  int* d_tab_count;        // recovery tables tabulated per corrupt set, all groups: rows in use per set
  int* d_tab_rows;         // tab_ld ints per set
  double* d_tab_coeff;     // tab_ld x m doubles per set
  int64_t* d_tab_off;      // q: first set of group g
  int* d_tab_sets;         // q: sets of group g (0: not tabulated, the table is computed at decode time)
  int tab_ld;              // rows reserved per set: m in the subset form, the largest group otherwise

  // optimistic decode (solon_plan_set_optimistic): the projection pass also writes the aggregate, recovered from the rows
  // of the locator's last recovery table (d_rec_rows, d_coeff: what the previous decode's recovery read; before the first
  // decode the table for no corrupt node), and the recovery kernel is skipped when the locator finds all of them trusted
  int optimistic;          // 0 never, 1 when in each of the last two decodes the table of the decode before would have served (default), 2 always
  int opt_rows;            // rows speculated on over all groups: q m (0: the plan is not eligible)
  std::vector<int> opt_src_host;   // their positions in d_rec_rows (and rows of d_coeff): group_start[g] + j, j < m
  int* d_opt;              // [1] the projection pass of this decode recovered too, [4] mode (copied from `optimistic`),
                           // [8 + g] decodes in a row (up to 2) in which the rows group g could have speculated on were all trusted
  int draw_parity;         // which buffer holds the current draw of f (0, 1), or -1: only the device knows (decodes draw anew)
  float* d_f;              // K x f_pitch projection vectors: the draws with an even index
  float* d_f2;             // the draws with an odd index
  int last_decode_advanced;    // the most recent decode drew new vectors for the next one (the count is one ahead of what it used)
  int64_t f_pitch;         // row pitch of d_f in floats (multiple of 4)
  int fresh_f;             // every decode draws new vectors first (solon_plan_set_fresh_projections)
  unsigned long long* d_draw;   // [0] index of the draw now in d_f, [1] ticket of the fill kernel

  // projection workspace
  int proj_grid;           // CTAs of the projection kernel = number of partial sums
  double* d_partials;      // proj_grid x (K + 1) x P
  int proj_two_parts;      // the last projection launch announced part A
  int early_locator;       // 0 never, 1 by size, 2 whenever the solver is small, 3 diagnostic (solon_plan_set_early_locator)
  int proj_bunches;        // > 0: the last projection launch left this many bunch sums for the locator to add
  const double* proj_bunch_sums;   // proj_bunches x (K + 1) x P: final sums
  const double* proj_bunch_a;      // same shape: sums over part A of the column ranges only
  unsigned long long* d_proj_progress;          // [0] bunches done with part A in the current decode (the recovery kernel zeroes it)
  unsigned long long proj_progress_target;      // its value once part A is complete
  double* d_rho;           // K x P
  double* d_nu;            // P
  unsigned int* d_proj_ticket;   // 1

  // locator workspace / outputs
  double* d_locate_ws;     // q x locate_ws_stride doubles (workspace of groups too large for shared memory)
  size_t locate_ws_stride;
  int* d_t_acc;            // q
  int* d_n_rec;            // q
  int* d_rec_rows;         // P   (global node index of the j-th recovery row of group g at start[g] + j)
  double* d_coeff;         // P x m
  int* d_early;            // q: 0 no early run, 1 early answer confirmed, 2 not confirmed, 3 the wait for part A expired, 4 started too late
  int* d_status;           // [0] status bits of the last decode, [1] sticky bits (expired waits)
  unsigned long long* d_tile_counter;   // [0] the recovery kernel's next tile (the locator kernel zeroes it);
                                        // [1], [2] the encode kernel's next tile and departed CTAs (it zeroes them itself)

  // optional per-kernel timing: events [0,1] around encode, [2..5] before/after the decode kernels
  int profiling;
  cudaEvent_t ev[6];
  int ev_valid[6];

  // lsq workspace
  float* d_resid;          // P * lsq_rows
  int64_t resid_capacity;

  // host-step staging (allocated on first use)
  float* d_stage_grads;
  float* d_stage_coded;
  float* d_stage_agg;
  uint8_t* d_stage_mask;
};

namespace solon {

// Programmatic dependent launch (sm_90+): a kernel launched with launch_dependent may start while the kernel
// before it in the stream is still running, once every CTA of that kernel has called pdl_trigger (or exited);
// it must call pdl_wait before it reads anything the earlier kernel wrote or writes anything it may still
// read.  pdl_wait returns when the earlier kernel has completed and its writes are visible.
#if defined(__CUDACC__)
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
static inline int launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                   Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...) != cudaSuccess) {
    (void)cudaGetLastError();
    return SOLON_ERR_CUDA;
  }
  return SOLON_OK;
}
#endif

// A named range on the calling host thread while `on` (plans with profiling switched on): timeline tools show the
// library's calls and, inside solon_decode, its three launches under their names.  Header-only NVTX: costs nothing
// measurable when no tool is attached.
struct TraceRange {
  bool on;
  TraceRange(bool on_, const char* name) : on(on_) {
    if (on) nvtxRangePushA(name);
  }
  ~TraceRange() {
    if (on) nvtxRangePop();
  }
  TraceRange(const TraceRange&) = delete;
  TraceRange& operator=(const TraceRange&) = delete;
};

// Kernel launchers (each enqueues on plan->stream and returns a solon_status).
// Whether solon_decode lets the locator work ahead on a partial projection (solon_plan_set_early_locator): a small
// solver, and either mode 2 or a projection pass long enough to hide the early run, which takes 60-80 us beside
// a streaming kernel (the projection kernel moves about 6 GB per ms).
inline bool uses_early_locator(const solon_plan* plan) {
  const bool small_solver = plan->s > 0 && plan->max_group <= 64 && plan->s <= 5;
  // (a locator with a single error count to try is through sooner: 300 MB suffice at s = 1 - 101 -> 89 us per decode on 15
  // nodes x 10 M at m = 2 - where s = 3 and s = 5 lose 2 and 8 us)
  const bool long_pass = (double)plan->P * (double)plan->d_c * 4.0 >= (plan->s <= 1 ? 250e6 : 350e6);
  return small_solver && (plan->early_locator >= 2 || (plan->early_locator == 1 && long_pass));
}
// Mode 3 (diagnostic): the locator works ahead as in mode 2 but the projection kernel announces no partial sums,
// so the locator's bounded wait for them runs out and it falls back to its ordinary path.
inline bool early_locator_starved(const solon_plan* plan) { return plan->early_locator == 3; }

// Between two decodes the encode step and the recovery move gigabytes through L2 and push out everything else - the
// locator kernel's instructions and tables included, whose re-fetch from device memory (about a microsecond per 128
// bytes of code) is most of a short decode's serial time.  When every streamed byte is marked evict-first the code
// survives in L2; a single unmarked stream undoes it.  The marks have a price: the encode kernel loses 2-4 % of its
// bandwidth, the recovery kernel's streaming stores are slower than plain ones (33 -> 41 us at m = 2, 49 -> 70 us at
// m = 1 on 15 nodes x 10 M), and the coded matrix no longer lingers in L2 for the projection pass of a decode that
// follows an encode.  Measured per case (same box, switch in the environment): worth it where the locator is long
// and the streams are short - m > 6 (all-rows recovery tables, 89 -> 67 us per decode on 15 nodes x 10 M at m = 10) -
// and for m = 4 .. 6 when the decode's own pass is short: at 600 - 670 MB of gradients on 15 nodes (m = 5, a projection
// pass over 120 - 134 MB) the decode gains 4 - 9 us in the single-pass form and 0 - 6 us in the two-pass form while the encode
// loses 0 - 2; with m = 1, 2 at the same sizes (a projection pass over 300 - 600 MB, which evicts the code whatever the
// marks) the locator gains nothing.  Small steps gain at every m: over the 30 grid points with 1 M coordinates (60 - 420 MB
// of gradients) the step is 3 - 28 % shorter with the marks at m = 1, 2 and 6 - 25 % at m = 5, 10, and longer at none by
// more than 3 %.  How much may stream before the code is gone whatever the marks: at 1.8 GB of gradients per step (45 nodes
// x 10 M, m = 10) the decode still gains 14 - 22 us and the encode loses 2 - 8; at 4.2 GB (105 nodes) the decode gains
// nothing and the encode loses 20.  So: at most 450 MB of gradients per step, or m = 4 .. 6 with at most 1 GB of gradients
// and 160 MB of coded vectors, or m > 6 and at most 2 GB of gradients.
inline bool keeps_l2_for_code(int P, int m, int64_t d) {
  const double grads = (double)P * (double)d * 4.0;
  if (grads <= 450e6) return true;
  if (m > 6) return grads <= 2.0e9;
  return m >= 4 && grads <= 1.0e9 && grads / m <= 160e6;
}

int launch_fill_projection(solon_plan* plan, int advance);   // advance = 1: the next draw (device-side count), 0: redo the current one
int launch_encode(solon_plan* plan, const float* grads, float* coded);
int launch_encode_f64(solon_plan* plan, const double* grads, double* coded);
// rho_out / nu_out (and rho / nu below): device buffers, or nullptr for the plan's own
// agg: where the optimistic decode may write the aggregate (the whole decode only; nullptr: never)
int launch_project(solon_plan* plan, const float* received, double* rho_out = nullptr, double* nu_out = nullptr, float* agg = nullptr);
int launch_project_f64(solon_plan* plan, const double* received, double* rho_out = nullptr, double* nu_out = nullptr, double* agg = nullptr);
int launch_locate(solon_plan* plan, uint8_t* byz_mask, const double* rho = nullptr, const double* nu = nullptr);
int launch_recover(solon_plan* plan, const float* received, float* agg);
int launch_recover_f64(solon_plan* plan, const double* received, double* agg);
int launch_lsq(solon_plan* plan, const float* X, const float* y, const float* w, float* grads);

// Doubles of workspace one locator CTA needs for a group of n nodes.
size_t locate_ws_doubles(int n, int m, int K, int s);

// Host: locator tables of one group (n x n Qb column-major, n x n Hm, m x m Mt, n x (s + 1) Tch).
void build_group_tables(int n, int m, int s, const double* w, double* Qb, double* Hm, double* Mt, double* Tch);

// Host-side layout rules (also used by the plan-free helpers).
int check_params(int P, int s, int m, int r, int64_t d);
void group_layout(int P, int r, std::vector<int>* start);
void node_scalars(const std::vector<int>& start, std::vector<double>* w);

}  // namespace solon
