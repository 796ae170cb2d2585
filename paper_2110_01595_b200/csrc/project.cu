// Detection projections (Section 3.4): rho[kappa][k] = f_kappa . R_k for the K random vectors f_kappa
// and all P received rows, plus the row energies nu[k] = ||R_k||^2 that scale the locator's tolerance.
//
// One pass over the P x d_c received matrix.  Every CTA owns one contiguous range of the chunk axis.
// Two forms: the plan's decode uses the streaming kernel (rows and f brought through a shared-memory ring by
// bulk copies, float32 products in short runs, float64 sums: see project_pipe_kernel); the entry point that
// allocates nothing uses the direct kernel (each warp loads its own rows, the tile of f in shared memory as
// float64, every product and sum of rho in float64; nu is added in float32 inside a lane for one tile at a time
// and in float64 beyond).  Per-CTA partial sums go to global memory and are added in a
// fixed order by the last CTAs to finish (atomic tickets, no waiting), so results are bit-reproducible.
#include <mutex>

#include "solon_internal.h"
#include "stream_pipe.cuh"

namespace solon {

constexpr int kProjThreads = 256;
constexpr int kProjWarps = kProjThreads / 32;
constexpr int kProjBunch = 16;   // CTAs per first-level reduction

template <int K>
struct ProjAcc {
  double rho[K];
  float nu;
};

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  return v;
}

// Two-level, fixed-order reduction of the per-CTA partial sums with atomic tickets (nobody waits): every CTA
// has written its n_acc sums to partials[blockIdx.x]; the last CTA of every bunch of kProjBunch adds that
// bunch, and (final_reduce) the last bunch adds the bunch sums into rho_out / nu_out.  Called by all threads.
__device__ __forceinline__ void reduce_partials(double* __restrict__ partials, int n_acc, int KP, double* __restrict__ rho_out,
                                                double* __restrict__ nu_out, unsigned int* ticket, int final_reduce) {
  __shared__ unsigned int s_ticket;
  const int tid = threadIdx.x, n_threads = blockDim.x;
  const unsigned int bunch = blockIdx.x / kProjBunch;
  const unsigned int n_bunches = (gridDim.x + kProjBunch - 1) / kProjBunch;
  const unsigned int first = bunch * kProjBunch;
  const unsigned int members = min((unsigned int)kProjBunch, gridDim.x - first);
  double* bunch_sums = partials + (size_t)gridDim.x * n_acc;
  __threadfence();
  __syncthreads();
  if (tid == 0) s_ticket = atomicAdd(ticket + 1 + bunch, 1u);
  __syncthreads();
  if (s_ticket != members - 1) return;
  __threadfence();
  for (int i = tid; i < n_acc; i += n_threads) {
    double v[kProjBunch];
#pragma unroll
    for (unsigned int b = 0; b < (unsigned int)kProjBunch; ++b)     // all loads in flight at once, then a fixed order
      v[b] = b < members ? __ldcg(partials + (size_t)(first + b) * n_acc + i) : 0.0;
    double acc = 0.0;
#pragma unroll
    for (unsigned int b = 0; b < (unsigned int)kProjBunch; ++b) acc += v[b];
    bunch_sums[(size_t)bunch * n_acc + i] = acc;
  }
  if (!final_reduce) {
    // the locator kernel adds the bunch sums itself (it needs them on chip anyway): nothing more to do here
    __syncthreads();
    if (tid == 0) ticket[1 + bunch] = 0u;   // ready for the next decode
    return;
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    ticket[1 + bunch] = 0u;   // ready for the next decode
    s_ticket = atomicAdd(ticket, 1u);
  }
  __syncthreads();
  if (s_ticket != n_bunches - 1) return;
  __threadfence();
  for (int i = tid; i < n_acc; i += n_threads) {
    double acc = 0.0;
#pragma unroll 4
    for (unsigned int b = 0; b < n_bunches; ++b) acc += __ldcg(bunch_sums + (size_t)b * n_acc + i);
    if (i < KP) rho_out[i] = acc;
    else nu_out[i - KP] = acc;
  }
  if (tid == 0) *ticket = 0u;
}

template <int K>
__global__ void __launch_bounds__(kProjThreads, 4) project_kernel(const float* __restrict__ R, const float* __restrict__ f,
                                                               int64_t f_pitch, int P, int64_t d_c, int64_t range_len,
                                                               int tile_cols, double* __restrict__ partials,
                                                               double* __restrict__ rho_out, double* __restrict__ nu_out,
                                                               unsigned int* ticket, int final_reduce) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  double* fs = reinterpret_cast<double*>(smem_raw);            // K x tile_cols
  double* sacc = fs + (size_t)K * tile_cols;                  // P x (K + 1)
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_acc = (K + 1) * P;
  pdl_trigger();   // the locator may be scheduled early; it waits for this grid before reading rho
  for (int i = tid; i < n_acc; i += kProjThreads) sacc[i] = 0.0;

  const int64_t c_begin = (int64_t)blockIdx.x * range_len;
  int64_t c_end = c_begin + range_len;
  if (c_end > d_c) c_end = d_c;

  for (int64_t c0 = c_begin; c0 < c_end; c0 += tile_cols) {
    const int cols = (int)((c_end - c0) < tile_cols ? (c_end - c0) : tile_cols);
    __syncthreads();   // previous tile fully consumed (also orders the zeroing of sacc)
    // f tile -> float64 shared memory; c0 is a multiple of 4 and f rows are 16-byte aligned
    for (int i = tid * 4; i < cols; i += kProjThreads * 4) {
#pragma unroll
      for (int kappa = 0; kappa < K; ++kappa) {
        const float* src = f + (int64_t)kappa * f_pitch + c0 + i;
        float4 v = *reinterpret_cast<const float4*>(src);     // pitch padding keeps this in bounds
        double* dst = fs + (size_t)kappa * tile_cols + i;
        dst[0] = (double)v.x;
        if (i + 1 < cols) dst[1] = (double)v.y;
        if (i + 2 < cols) dst[2] = (double)v.z;
        if (i + 3 < cols) dst[3] = (double)v.w;
      }
    }
    __syncthreads();
    // rows in batches of two; batch b belongs to warp b mod kProjWarps
    for (int row = warp * 2; row < P; row += kProjWarps * 2) {
      const bool two = row + 1 < P;
      const float* ra = R + (int64_t)row * d_c + c0;
      const float* rb = two ? ra + d_c : ra;
      double a_rho[K], b_rho[K];
      float a_nu = 0.f, b_nu = 0.f;
#pragma unroll
      for (int kappa = 0; kappa < K; ++kappa) a_rho[kappa] = b_rho[kappa] = 0.0;
      int c = lane;
      // software pipeline: the loads of the next 8 x 32 columns are in flight while this batch is used
      float va[8], vb[8], na_[8], nb_[8];
      bool have = c + 7 * 32 < cols;
      if (have) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          va[u] = __ldcs(ra + c + u * 32);
          vb[u] = __ldcs(rb + c + u * 32);
        }
      }
      while (have) {
        const int cn = c + 8 * 32;
        const bool more = cn + 7 * 32 < cols;
        if (more) {
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            na_[u] = __ldcs(ra + cn + u * 32);
            nb_[u] = __ldcs(rb + cn + u * 32);
          }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const double da = (double)va[u], db = (double)vb[u];
#pragma unroll
          for (int kappa = 0; kappa < K; ++kappa) {
            const double fv = fs[(size_t)kappa * tile_cols + c + u * 32];
            a_rho[kappa] = fma(fv, da, a_rho[kappa]);
            b_rho[kappa] = fma(fv, db, b_rho[kappa]);
          }
          a_nu = fmaf(va[u], va[u], a_nu);
          b_nu = fmaf(vb[u], vb[u], b_nu);
        }
        if (more) {
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            va[u] = na_[u];
            vb[u] = nb_[u];
          }
        }
        c = cn;
        have = more;
      }
      for (; c < cols; c += 32) {
        const float va = __ldcs(ra + c), vb = __ldcs(rb + c);
        const double da = (double)va, db = (double)vb;
#pragma unroll
        for (int kappa = 0; kappa < K; ++kappa) {
          const double fv = fs[(size_t)kappa * tile_cols + c];
          a_rho[kappa] = fma(fv, da, a_rho[kappa]);
          b_rho[kappa] = fma(fv, db, b_rho[kappa]);
        }
        a_nu = fmaf(va, va, a_nu);
        b_nu = fmaf(vb, vb, b_nu);
      }
#pragma unroll
      for (int kappa = 0; kappa < K; ++kappa) {
        const double sa = warp_sum(a_rho[kappa]);
        const double sb = warp_sum(b_rho[kappa]);
        if (lane == 0) {
          sacc[(size_t)kappa * P + row] += sa;
          if (two) sacc[(size_t)kappa * P + row + 1] += sb;
        }
      }
      const double na = warp_sum((double)a_nu), nb = warp_sum((double)b_nu);
      if (lane == 0) {
        sacc[(size_t)K * P + row] += na;
        if (two) sacc[(size_t)K * P + row + 1] += nb;
      }
    }
  }
  __syncthreads();
  double* mine = partials + (size_t)blockIdx.x * n_acc;
  for (int i = tid; i < n_acc; i += kProjThreads) mine[i] = sacc[i];
  reduce_partials(partials, n_acc, K * P, rho_out, nu_out, ticket, final_reduce);
}

// ---- streaming form: rows and f come through shared memory by bulk copies ------------------------------------
//
// A producer warp moves, per stage, one column slice of up to kPipeRows received rows plus the same slice of the
// K projection vectors into a shared-memory ring (cp.async.bulk, completion on an mbarrier), so hundreds of KB
// per SM are in flight without occupying registers.  The P rows are cut into equal batches of at most kPipeRows;
// within a batch consumer warp w owns rows w, w + 8, w + 16, w + 24 (those that exist), walks the slice 32 columns
// at a time reusing each f value for all its rows, and keeps its sums across all slices of the CTA's column range:
// products and short runs (8 steps) in float32, everything else in float64.  The rounding this adds (at most
// 8 * 2^-24 of sum |f_p R_kp|, the size of the float32 rounding the coded vectors already carry) is a hundred times
// below the locator's tolerance.  A row is summed by exactly one warp in a fixed order: bit-reproducible.
constexpr int kPipeRows = 32;                       // rows per stage: up to four per consumer warp
constexpr int kPipeConsumers = 256;
constexpr int kPipeWarps = kPipeConsumers / 32;
constexpr int kPipeThreads = kPipeConsumers + 32;   // + one producer warp
constexpr int kPipeStages = 2;
#ifndef SOLON_PIPE_CTAS
#define SOLON_PIPE_CTAS 2
#endif
constexpr int kPipeCtasPerSm = SOLON_PIPE_CTAS;

struct ProjPipe {
  int slice_cols;     // columns per stage (multiple of 32)
  int slot_floats;    // slice_cols + 8: room for the alignment shift and the rounded-up end
  int batch_rows;     // rows per batch (<= kPipeRows), the same for all batches but the last
  int64_t part_a_cols;                // columns of part A in every CTA's range (whole slices)
  unsigned long long* progress;       // bunches whose part-A sums [0] and final sums [1] are complete (zeroed by the recovery kernel)
  int* status;
  // Optimistic decode.  The rows of the locator's last recovery table (m per group: what the previous decode's recovery
  // read; opt_rows of them over all groups, ascending) are the ones this decode speculates on.  When the device flags say
  // so (mode 2, or mode 1 and every group's count at 2: the last two decodes' previous tables both held) the consumers also recover the aggregate of every
  // column slice from them, exactly as the recovery kernel would with that table.  They must all lie in one stage of the
  // ring: with a single batch of rows the order stays the natural one and nothing has to come from device memory before
  // the first loads are issued; with several batches they are taken first (the other rows follow in ascending order),
  // and the kernel starts by fetching the list.
  int opt_rows;                       // 0: rows in natural order, never optimistic
  int multi_batch;                    // more than one batch of rows
  int opt_ch;                         // chunks per consumer thread and pass of the recovery (1..4): slice_cols is a multiple of 256 opt_ch
  uint16_t spec_src[kPipeRows];       // positions of those rows in rec_rows and rec_coeff: group_start[g] + j, j < m
  int q;                              // groups (their flags are opt_flags[8 + g])
  const int* rec_rows;                // P: the locator's last recovery table (rows as node indices, per group from group_start[g])
  const double* rec_coeff;            // P x m: its weights
  const int* n_rec;                   // q: rows in use per group (m after a decode that succeeded)
  int* opt_flags;                     // [1] this pass recovered (written here), [4] mode, [8 + g] see the locator kernel
  void* agg;                          // d elements of the plan's type: the aggregate (written only when this pass recovers)
  int m;
  int64_t d;
};

// The row taken at position pos of the kernel's order: the n_first rows of first_rows (ascending), then all others in
// ascending order.
__device__ __forceinline__ int pipe_row_at(int pos, int n_first, const int* first_rows) {
  if (pos < n_first) return first_rows[pos];
  int r = pos - n_first;
  for (int j = 0; j < n_first; ++j)
    if (first_rows[j] <= r) ++r;
  return r;
}

// Two float32 values in one 64-bit register, and the packed fused multiply-add of sm_100 (fma.rn.f32x2: each half is an
// ordinary IEEE fma.rn, so results equal those of two scalar instructions bit for bit, in one issue slot).
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
  f32x2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
  f32x2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}

// Aggregate of one column slice from the n_def rows speculated on (row j starts s_off[j] floats into the stage), in the
// recovery kernel's arithmetic and order: acc = fma(weight, value, acc) over the rows, group by group.  A lane owns the
// chunks c + i * 256, i < ch, of each 256 ch, two chunks to a packed multiply-add, and shares a row's weights (eight
// pairs (w_l, w_l) per row in shared memory, fetched with 128-bit loads) between them; it writes each chunk's m floats
// itself (routing them through shared memory into 128-bit stores, as the recovery kernel does, made this kernel 20 %
// slower: its consumer warps are bound by instruction issue).
constexpr int kOptChunks = 4;
// NP: pairs of chunks per lane and pass held in registers (ch <= 2 NP)
template <int M, int NP>
__device__ __forceinline__ void opt_recover_slice(const float* base, const int* s_off, const f32x2* s_coeff2, int n_def,
                                                  int cols, int ch, int64_t c0, float* __restrict__ agg, int64_t d, int warp, int lane) {
  // ch (1..4): chunks per lane and pass; the slice width is a multiple of 256 ch where that costs little, so that every
  // pass but the one at the ragged end of a range keeps all lanes busy
  for (int cb = warp * 32; cb < cols; cb += ch * kPipeConsumers) {
    const int c = cb + lane;
    f32x2 acc[NP][M];
#pragma unroll
    for (int h = 0; h < NP; ++h)
#pragma unroll
      for (int l = 0; l < M; ++l) acc[h][l] = 0ULL;          // (+0.0f, +0.0f)
    for (int j = 0; j < n_def; ++j) {
      const float* row = base + s_off[j];
      f32x2 w[(M + 1) / 2 * 2];
#pragma unroll
      for (int t = 0; t < (M + 1) / 2; ++t) {
        const ulonglong2 ww = *reinterpret_cast<const ulonglong2*>(s_coeff2 + j * 8 + 2 * t);
        w[2 * t] = ww.x;
        w[2 * t + 1] = ww.y;
      }
      float v[2 * NP];
#pragma unroll
      for (int i = 0; i < 2 * NP; ++i) v[i] = (i < ch && c + i * kPipeConsumers < cols) ? row[c + i * kPipeConsumers] : 0.0f;
#pragma unroll
      for (int h = 0; h < NP; ++h) {
        if (2 * h < ch) {
          const f32x2 vv = pack2(v[2 * h], v[2 * h + 1]);
#pragma unroll
          for (int l = 0; l < M; ++l) acc[h][l] = fma2(w[l], vv, acc[h][l]);
        }
      }
    }
#pragma unroll
    for (int i = 0; i < 2 * NP; ++i) {
      const int ci = cb + i * kPipeConsumers + lane;
      if (i < ch && ci < cols) {
        const int64_t o = (c0 + ci) * M;
#pragma unroll
        for (int l = 0; l < M; ++l) {
          float lo, hi;
          unpack2(acc[i / 2][l], lo, hi);
          if (o + l < d) __stcs(agg + o + l, (i & 1) ? hi : lo);
        }
      }
    }
  }
}

template <int M>
__device__ __forceinline__ void opt_recover_slice_m(const float* base, const int* s_off, const f32x2* s_coeff2, int n_def,
                                                    int cols, int ch, int64_t c0, float* __restrict__ agg, int64_t d, int warp, int lane) {
  // fewer accumulators in registers when the passes are narrow (the kernel is at its register limit)
  if (ch <= 2) opt_recover_slice<M, 1>(base, s_off, s_coeff2, n_def, cols, ch, c0, agg, d, warp, lane);
  else opt_recover_slice<M, 2>(base, s_off, s_coeff2, n_def, cols, ch, c0, agg, d, warp, lane);
}

// The same for float64 plans: float64 weights and sums as in the float64 recovery kernel, one or two chunks per lane and pass.
template <int M>
__device__ __forceinline__ void opt_recover_slice_m(const double* base, const int* s_off, const f32x2* s_coeff2, int n_def,
                                                    int cols, int ch, int64_t c0, double* __restrict__ agg, int64_t d, int warp, int lane) {
  const double* s_coeff = reinterpret_cast<const double*>(s_coeff2);     // eight weights per row
  for (int cb = warp * 32; cb < cols; cb += ch * kPipeConsumers) {
    const int c = cb + lane;
    double acc[2][M];
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int l = 0; l < M; ++l) acc[i][l] = 0.0;
    for (int j = 0; j < n_def; ++j) {
      const double* row = base + s_off[j];
      double w[(M + 1) / 2 * 2];
#pragma unroll
      for (int t = 0; t < (M + 1) / 2; ++t) {
        const double2 ww = *reinterpret_cast<const double2*>(s_coeff + j * 8 + 2 * t);
        w[2 * t] = ww.x;
        w[2 * t + 1] = ww.y;
      }
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        if (i < ch) {
          const double v = c + i * kPipeConsumers < cols ? row[c + i * kPipeConsumers] : 0.0;
#pragma unroll
          for (int l = 0; l < M; ++l) acc[i][l] = fma(w[l], v, acc[i][l]);
        }
      }
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int ci = cb + i * kPipeConsumers + lane;
      if (i < ch && ci < cols) {
        const int64_t o = (c0 + ci) * M;
#pragma unroll
        for (int l = 0; l < M; ++l)
          if (o + l < d) __stcs(agg + o + l, acc[i][l]);
      }
    }
  }
}

// One slice for the NR rows of this warp: rows[j] point at column 0 of the slice in the warp's j-th row.
template <int K, int NR>
__device__ __forceinline__ void pipe_consume(const float* const* rows, const float* fs, int slot_floats, int cols, int lane,
                                             double (*rho)[K], double* nu) {
  for (int c = lane; c < cols; c += 8 * 32) {
    float sr[NR][K], sn[NR];
#pragma unroll
    for (int j = 0; j < NR; ++j) {
      sn[j] = 0.f;
#pragma unroll
      for (int kappa = 0; kappa < K; ++kappa) sr[j][kappa] = 0.f;
    }
    const int steps = (cols - c + 31) / 32;      // 8 except at the ragged end of the range
    if (steps >= 8) {
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int cc = c + u * 32;
        float fv[K];
#pragma unroll
        for (int kappa = 0; kappa < K; ++kappa) fv[kappa] = fs[(size_t)kappa * slot_floats + cc];
#pragma unroll
        for (int j = 0; j < NR; ++j) {
          const float v = rows[j][cc];
#pragma unroll
          for (int kappa = 0; kappa < K; ++kappa) sr[j][kappa] = fmaf(fv[kappa], v, sr[j][kappa]);
          sn[j] = fmaf(v, v, sn[j]);
        }
      }
    } else {
      for (int cc = c; cc < cols; cc += 32) {
        float fv[K];
#pragma unroll
        for (int kappa = 0; kappa < K; ++kappa) fv[kappa] = fs[(size_t)kappa * slot_floats + cc];
#pragma unroll
        for (int j = 0; j < NR; ++j) {
          const float v = rows[j][cc];
#pragma unroll
          for (int kappa = 0; kappa < K; ++kappa) sr[j][kappa] = fmaf(fv[kappa], v, sr[j][kappa]);
          sn[j] = fmaf(v, v, sn[j]);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < NR; ++j) {
#pragma unroll
      for (int kappa = 0; kappa < K; ++kappa) rho[j][kappa] += (double)sr[j][kappa];
      nu[j] += (double)sn[j];
    }
  }
}

// The same for float64 rows: exact products and sums in float64 (f is widened), four independent steps in flight.
template <int K, int NR>
__device__ __forceinline__ void pipe_consume(const double* const* rows, const float* fs, int slot_floats, int cols, int lane,
                                             double (*rho)[K], double* nu) {
#pragma unroll 4
  for (int c = lane; c < cols; c += 32) {
    double fv[K];
#pragma unroll
    for (int kappa = 0; kappa < K; ++kappa) fv[kappa] = (double)fs[(size_t)kappa * slot_floats + c];
#pragma unroll
    for (int j = 0; j < NR; ++j) {
      const double v = rows[j][c];
#pragma unroll
      for (int kappa = 0; kappa < K; ++kappa) rho[j][kappa] = fma(fv[kappa], v, rho[j][kappa]);
      nu[j] = fma(v, v, nu[j]);
    }
  }
}

// Sums of one bunch of kProjBunch CTAs, added in a fixed order by the last of them to arrive (atomic ticket, nobody
// waits).  Called by n_threads threads of the CTA that synchronise through Sync; every one of them gets the same
// answer: whether this CTA was the one that completed the bunch.  bunch_out[i] = add_in[i] + sum over members.
struct SyncAll {
  __device__ __forceinline__ static void sync() { __syncthreads(); }
};
struct SyncConsumers {
  __device__ __forceinline__ static void sync() { pipe::named_barrier_sync(1, 256); }
};

template <class Sync>
__device__ __forceinline__ bool bunch_reduce(const double* __restrict__ partials, const double* add_in, double* __restrict__ bunch_out,
                                             int n_acc, unsigned int* bunch_ticket, unsigned int* s_flag, int tid, int n_threads) {
  const unsigned int bunch = blockIdx.x / kProjBunch;
  const unsigned int first = bunch * kProjBunch;
  const unsigned int members = min((unsigned int)kProjBunch, gridDim.x - first);
  __threadfence();
  Sync::sync();
  if (tid == 0) *s_flag = atomicAdd(bunch_ticket + bunch, 1u);
  Sync::sync();
  const bool last = *s_flag == members - 1;
  if (!last) return false;
  __threadfence();
  for (int i = tid; i < n_acc; i += n_threads) {
    double v[kProjBunch];
#pragma unroll
    for (unsigned int b = 0; b < (unsigned int)kProjBunch; ++b)     // all loads in flight at once, then a fixed order
      v[b] = b < members ? __ldcg(partials + (size_t)(first + b) * n_acc + i) : 0.0;
    double acc = add_in ? __ldcg(add_in + (size_t)bunch * n_acc + i) : 0.0;
#pragma unroll
    for (unsigned int b = 0; b < (unsigned int)kProjBunch; ++b) acc += v[b];
    bunch_out[(size_t)bunch * n_acc + i] = acc;
  }
  __threadfence();
  Sync::sync();
  if (tid == 0) bunch_ticket[bunch] = 0u;   // ready for the next launch
  return true;
}

// The CTA's column range is walked in two parts.  Part A (the first eighth or so) is summed, reduced over the
// bunches and announced (progress[0]) on its own, so that the locator kernel can already work on a projection of
// those columns - it is a random projection like any other - while part B streams; the final sums are A + B.
template <int K, typename T>
__global__ void __launch_bounds__(kPipeThreads, kPipeCtasPerSm) project_pipe_kernel(const T* __restrict__ R, const float* __restrict__ f_even,
                                                                     const float* __restrict__ f_odd,
                                                                     const unsigned long long* __restrict__ draw,
                                                                     int64_t f_pitch, int P, int64_t d_c, int64_t range_len,
                                                                     ProjPipe pp, double* __restrict__ partials,
                                                                     double* __restrict__ rho_out, double* __restrict__ nu_out,
                                                                     unsigned int* ticket, int final_reduce) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ unsigned int s_flag;
  __shared__ __align__(16) f32x2 s_opt_coeff[kPipeRows * 8];     // eight pairs per speculated row: (w_l, w_l) for l < m, then zeros
  __shared__ int s_opt_off[kPipeRows];                           // where that row starts in a stage of the first batch
  __shared__ int s_first_row[kPipeRows];                         // rows taken first (several batches of rows only)
  __shared__ int s_n_first, s_opt_on;
  const int tid = threadIdx.x;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem_raw);
  uint64_t* empty_bar = full_bar + kPipeStages;
  int* abort_flag = reinterpret_cast<int*>(empty_bar + kPipeStages);
  constexpr int64_t kVec = 16 / sizeof(T);                    // elements per 16 bytes
  unsigned char* ring = smem_raw + 128;
  const size_t rows_bytes = (size_t)pp.batch_rows * pp.slot_floats * sizeof(T);
  const size_t stage_bytes = rows_bytes + (size_t)K * pp.slot_floats * sizeof(float);   // the rows of a batch, then f
  const int n_acc = (K + 1) * P;
  pdl_trigger();   // the locator may be scheduled early; it waits for this grid before reading the final sums
  // the vectors of draw n live in the buffer n & 1 (the count moves on only after this kernel has completed); when the
  // host knows which buffer that is it passes it as f_even and no count
  const float* __restrict__ f = f_even;
  if (draw != nullptr) f = (draw[0] & 1ULL) ? f_odd : f_even;
  if (tid == 0) {
    for (int s = 0; s < kPipeStages; ++s) {
      pipe::mbar_init(&full_bar[s], 32);
      pipe::mbar_init(&empty_bar[s], kPipeWarps);
    }
    *abort_flag = 0;
    pipe::fence_barrier_init();
  }
  // Optimistic decode: does this pass also recover the aggregate, from the rows of the last recovery table?
  // Mode 2, or mode 1 and every group's count at 2 (two decodes in a row whose previous table held); and only if that table is whole (m rows in every group,
  // ascending node indices).  Flags, rows and weights are fetched here - one load per thread - and looked at only when the
  // first stage's projection work is done (see below), so that their round trip to device memory hides behind it; with
  // several batches of rows the row order depends on the list, and the kernel waits for it here.  CTA 0 records the
  // answer for this decode's recovery kernel (0 until it is known).
  int opt_mode = 0, opt_flag = 2, spec_row = 0;      // raw values: nothing is computed from them before they are needed
  bool spec_whole = false;
  double spec_coeff = 0.0;
  {
    if (pp.opt_rows > 0) {
      if (tid < 32) {
        opt_mode = pp.opt_flags[4];
        if (tid < pp.q) opt_flag = pp.opt_flags[8 + tid];                           // q <= 32 when opt_rows > 0
        const int rows_g = tid < pp.q ? pp.n_rec[tid] : pp.m;
        spec_row = tid < pp.opt_rows ? pp.rec_rows[pp.spec_src[tid]] : 0x7fffffff;  // opt_rows <= 32
        if (pp.multi_batch) {
          const int below = __shfl_up_sync(0xffffffffu, spec_row, 1);
          const bool lane_ok = rows_g == pp.m && (tid >= pp.opt_rows || (spec_row >= 0 && spec_row < P && (tid == 0 || spec_row > below)));
          spec_whole = __all_sync(0xffffffffu, lane_ok);
          s_first_row[tid] = spec_row;
          if (tid == 0) s_n_first = spec_whole ? pp.opt_rows : 0;
        } else {
          spec_whole = rows_g == pp.m;      // this lane's part; completed when the flags are looked at
        }
      }
      if (tid < pp.opt_rows * 8 && (tid & 7) < pp.m)                                // opt_rows * 8 <= 256 consumer threads
        spec_coeff = pp.rec_coeff[(size_t)pp.spec_src[tid >> 3] * pp.m + (tid & 7)];
    }
  }
  if (tid == 0 && !(pp.opt_rows > 0 && pp.multi_batch)) s_n_first = 0;
  if (blockIdx.x == 0 && tid == 0) pp.opt_flags[1] = 0;
  __syncthreads();
  const int n_first = s_n_first;
  bool opt = false, opt_resolved = false;

  const int64_t c_begin = (int64_t)blockIdx.x * range_len;     // multiple of 4
  int64_t c_end = c_begin + range_len;
  if (c_end > d_c) c_end = d_c;
  int64_t c_mid = c_begin + pp.part_a_cols;                    // part_a_cols is a multiple of the slice width (0: one part)
  if (c_mid > c_end) c_mid = c_end;
  const int64_t total_floats = (int64_t)P * d_c;
  const unsigned int n_bunches = (gridDim.x + kProjBunch - 1) / kProjBunch;
  double* part_sums[2] = {partials + (size_t)blockIdx.x * n_acc, partials + ((size_t)gridDim.x + blockIdx.x) * n_acc};
  double* bunch_a = partials + 2 * (size_t)gridDim.x * n_acc;
  double* bunch_f = bunch_a + (size_t)n_bunches * n_acc;

  if (tid >= kPipeConsumers) {
    const int lane = tid - kPipeConsumers;
    const uint64_t row_policy = pipe::policy_evict_first();   // the recovery pass re-reads only a few of these rows
    const uint64_t f_policy = pipe::policy_evict_last();      // every decode reads the projection vectors again
    uint32_t it = 0;
    for (int part = pp.part_a_cols > 0 ? 0 : 1; part < 2; ++part) {
      const int64_t lo = part ? c_mid : c_begin, hi = part ? c_end : c_mid;
      for (int b0 = 0; b0 < P && lo < hi; b0 += pp.batch_rows) {
        const int nb = min(pp.batch_rows, P - b0);
        const int lane_row = lane < nb ? pipe_row_at(b0 + lane, n_first, s_first_row) : 0;
        for (int64_t c0 = lo; c0 < hi; c0 += pp.slice_cols, ++it) {
          const int stage = it % kPipeStages;
          const uint32_t phase = (it / kPipeStages) & 1;
          if (it >= (uint32_t)kPipeStages) pipe::mbar_wait(&empty_bar[stage], phase ^ 1, abort_flag, pp.status + 1);
          const int64_t cols = (hi - c0) < pp.slice_cols ? (hi - c0) : pp.slice_cols;
          unsigned char* stage_base = ring + stage * stage_bytes;
          uint32_t row_bytes = 0, f_bytes = 0;
          const T* row_src = nullptr;
          T* slot = reinterpret_cast<T*>(stage_base) + (size_t)lane * pp.slot_floats;
          if (lane < nb) {
            const int64_t first = (int64_t)lane_row * d_c + c0;
            const int64_t last = first + cols;
            const int64_t a0 = first & ~(kVec - 1);                   // enclosing 16-byte boundary
            int64_t a1 = (last + kVec - 1) & ~(kVec - 1);
            const int64_t safe_end = total_floats & ~(kVec - 1);      // bulk copies stay inside the matrix
            if (a1 > safe_end) a1 = safe_end;
            row_bytes = a1 > a0 ? (uint32_t)((a1 - a0) * sizeof(T)) : 0u;
            row_src = R + a0;
            for (int64_t e = (a1 > a0 ? a1 : a0); e < last; ++e) slot[e - a0] = R[e];   // fewer than 16 bytes
          }
          // the first K lanes also bring the slice of f (16-byte aligned rows padded to a multiple of 4 floats)
          if (lane < K) f_bytes = (uint32_t)(((cols + 3) & ~(int64_t)3) * 4);
          if (row_bytes + f_bytes) pipe::mbar_arrive_expect_tx(&full_bar[stage], row_bytes + f_bytes);
          else pipe::mbar_arrive(&full_bar[stage]);
          if (row_bytes) pipe::bulk_load_hint(slot, row_src, row_bytes, &full_bar[stage], row_policy);
          if (f_bytes)
            pipe::bulk_load_hint(reinterpret_cast<float*>(stage_base + rows_bytes) + (size_t)lane * pp.slot_floats,
                                 f + (int64_t)lane * f_pitch + c0, f_bytes, &full_bar[stage], f_policy);
        }
      }
    }
    if (*(volatile int*)abort_flag) pipe::drain_delay();
  } else {
    const int lane = tid & 31, warp = tid >> 5;
    const int dc_mod4 = (int)(d_c & (kVec - 1));
    uint32_t it = 0;
    for (int part = pp.part_a_cols > 0 ? 0 : 1; part < 2; ++part) {
      const int64_t lo = part ? c_mid : c_begin, hi = part ? c_end : c_mid;
      double* mine = part_sums[part];
      if (lo >= hi) {
        for (int i = tid; i < n_acc; i += kPipeConsumers) mine[i] = 0.0;      // nothing of this part in this CTA's range
      }
      for (int b0 = 0; b0 < P && lo < hi; b0 += pp.batch_rows) {
        const int nb = min(pp.batch_rows, P - b0);
        const int nr = warp < nb ? (nb - warp + kPipeWarps - 1) / kPipeWarps : 0;    // rows warp, warp + 8, ... below nb
        int shift[4], row_of[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          row_of[j] = j < nr ? pipe_row_at(b0 + warp + 8 * j, n_first, s_first_row) : 0;
          shift[j] = (int)(((row_of[j] & (kVec - 1)) * dc_mod4) & (kVec - 1));   // (row * d_c + c0) mod (elements per 16 bytes)
        }
        double rho[4][K], nu[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          nu[j] = 0.0;
#pragma unroll
          for (int kappa = 0; kappa < K; ++kappa) rho[j][kappa] = 0.0;
        }
        for (int64_t c0 = lo; c0 < hi; c0 += pp.slice_cols, ++it) {
          const int stage = it % kPipeStages;
          const uint32_t phase = (it / kPipeStages) & 1;
          pipe::mbar_wait(&full_bar[stage], phase, abort_flag, pp.status + 1);
          const int cols = (int)((hi - c0) < pp.slice_cols ? (hi - c0) : pp.slice_cols);
          const unsigned char* base = ring + stage * stage_bytes;
          const float* fs = reinterpret_cast<const float*>(base + rows_bytes);
          const T* rows[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) rows[j] = reinterpret_cast<const T*>(base) + (size_t)(warp + 8 * j) * pp.slot_floats + shift[j];
          if (nr == 4) pipe_consume<K, 4>(rows, fs, pp.slot_floats, cols, lane, rho, nu);
          else if (nr == 3) pipe_consume<K, 3>(rows, fs, pp.slot_floats, cols, lane, rho, nu);
          else if (nr == 2) pipe_consume<K, 2>(rows, fs, pp.slot_floats, cols, lane, rho, nu);
          else if (nr == 1) pipe_consume<K, 1>(rows, fs, pp.slot_floats, cols, lane, rho, nu);
          {
            if (pp.opt_rows > 0 && b0 == 0 && !opt_resolved) {
              // first stage of this CTA: flags, rows and weights have long arrived; all consumer warps pass here together
              if (tid < 32) {
                if (!pp.multi_batch) {
                  const int below = __shfl_up_sync(0xffffffffu, spec_row, 1);
                  const bool lane_ok = spec_whole && (tid >= pp.opt_rows || (spec_row >= 0 && spec_row < P && (tid == 0 || spec_row > below)));
                  spec_whole = __all_sync(0xffffffffu, lane_ok);
                }
                const bool all_clean = __all_sync(0xffffffffu, opt_flag >= 2);     // two decodes in a row whose previous table held
                if (tid == 0) {
                  s_opt_on = (spec_whole && (opt_mode == 2 || (opt_mode == 1 && all_clean))) ? 1 : 0;
                  if (blockIdx.x == 0) pp.opt_flags[1] = s_opt_on;
                }
                if (tid < pp.opt_rows && spec_whole) {
                  // slot of the row in a stage of the first batch: its position in the kernel's order
                  const int slot = pp.multi_batch ? tid : spec_row;
                  s_opt_off[tid] = slot * pp.slot_floats + (int)((((int64_t)spec_row & (kVec - 1)) * (d_c & (kVec - 1))) & (kVec - 1));
                }
              }
              if (tid < pp.opt_rows * 8) {     // rounded as the recovery kernel of the plan's type rounds it
                if constexpr (sizeof(T) == 4) s_opt_coeff[tid] = pack2((float)spec_coeff, (float)spec_coeff);
                else s_opt_coeff[tid] = (f32x2)__double_as_longlong(spec_coeff);
              }
              pipe::named_barrier_sync(1, kPipeConsumers);
              opt = s_opt_on != 0;
              opt_resolved = true;
            }
            if (opt && b0 == 0) {
              const T* rows0 = reinterpret_cast<const T*>(base);
              T* agg_t = reinterpret_cast<T*>(pp.agg);
              switch (pp.m) {
                case 1: opt_recover_slice_m<1>(rows0, s_opt_off, s_opt_coeff, pp.opt_rows, cols, pp.opt_ch, c0, agg_t, pp.d, warp, lane); break;
                case 2: opt_recover_slice_m<2>(rows0, s_opt_off, s_opt_coeff, pp.opt_rows, cols, pp.opt_ch, c0, agg_t, pp.d, warp, lane); break;
                case 3: opt_recover_slice_m<3>(rows0, s_opt_off, s_opt_coeff, pp.opt_rows, cols, pp.opt_ch, c0, agg_t, pp.d, warp, lane); break;
                case 4: opt_recover_slice_m<4>(rows0, s_opt_off, s_opt_coeff, pp.opt_rows, cols, pp.opt_ch, c0, agg_t, pp.d, warp, lane); break;
                case 5: opt_recover_slice_m<5>(rows0, s_opt_off, s_opt_coeff, pp.opt_rows, cols, pp.opt_ch, c0, agg_t, pp.d, warp, lane); break;
                default: opt_recover_slice_m<6>(rows0, s_opt_off, s_opt_coeff, pp.opt_rows, cols, pp.opt_ch, c0, agg_t, pp.d, warp, lane); break;
              }
            }
          }
          __syncwarp();
          if (lane == 0) pipe::mbar_arrive(&empty_bar[stage]);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (j < nr) {
            const int row = row_of[j];
#pragma unroll
            for (int kappa = 0; kappa < K; ++kappa) {
              const double t = warp_sum(rho[j][kappa]);
              if (lane == 0) mine[(size_t)kappa * P + row] = t;
            }
            const double t = warp_sum(nu[j]);
            if (lane == 0) mine[(size_t)K * P + row] = t;
          }
        }
      }
      if (part == 0) {
        // part A is complete in this CTA: the consumers alone (the producer is already fetching part B) add their
        // bunch if they are the last of it, and tell the locator kernel
        const bool done = bunch_reduce<SyncConsumers>(partials, nullptr, bunch_a, n_acc, ticket + 1 + n_bunches, &s_flag, tid,
                                                      kPipeConsumers);
        if (done && tid == 0) atomicAdd(pp.progress, 1ULL);
      }
    }
  }
  // final sums of a bunch = its part-A sums + its members' part-B sums
  const bool done = bunch_reduce<SyncAll>(partials + (size_t)gridDim.x * n_acc, pp.part_a_cols > 0 ? bunch_a : nullptr, bunch_f, n_acc,
                                          ticket + 1, &s_flag, tid,
                                          kPipeThreads);
  if (done && tid == 0 && pp.part_a_cols > 0) atomicAdd(pp.progress + 1, 1ULL);   // a locator CTA that starts this late skips its early run
  if (!done || !final_reduce) return;
  // the last bunch to finish adds the bunch sums
  if (tid == 0) s_flag = atomicAdd(ticket, 1u);
  __syncthreads();
  if (s_flag != n_bunches - 1) return;
  __threadfence();
  for (int i = tid; i < n_acc; i += kPipeThreads) {
    double acc = 0.0;
#pragma unroll 4
    for (unsigned int b = 0; b < n_bunches; ++b) acc += __ldcg(bunch_f + (size_t)b * n_acc + i);
    if (i < K * P) rho_out[i] = acc;
    else nu_out[i - K * P] = acc;
  }
  if (tid == 0) *ticket = 0u;
}

template <int K, typename T>
static int launch_project_pipe_k(solon_plan* plan, const T* received, double* rho_out, double* nu_out, int final_reduce, T* agg) {
  ProjPipe pp;
  pp.status = plan->d_status;
  pp.progress = plan->d_proj_progress;
  // optimistic decode: only in the whole decode (the aggregate's buffer is known) of a plan that is eligible
  pp.opt_rows = (!final_reduce && agg && plan->optimistic != 0) ? plan->opt_rows : 0;
  for (int j = 0; j < kPipeRows; ++j) pp.spec_src[j] = j < pp.opt_rows ? (uint16_t)plan->opt_src_host[(size_t)j] : 0;
  pp.q = plan->q;
  pp.rec_rows = plan->d_rec_rows;
  pp.rec_coeff = plan->d_coeff;
  pp.n_rec = plan->d_n_rec;
  pp.opt_flags = plan->d_opt;
  pp.agg = agg;
  pp.m = plan->m;
  pp.d = plan->d;
  // two CTAs per SM: the widest slice (multiple of 32 columns) whose ring fits in half of the shared memory
  // (the kernel's static shared memory - the optimistic decode's weights above all - is 2.4 KB)
  const size_t per_cta = (size_t)227 * 1024 / kPipeCtasPerSm - 1024 - 128 - 2560;
  const int n_batches = (plan->P + kPipeRows - 1) / kPipeRows;
  pp.batch_rows = (plan->P + n_batches - 1) / n_batches;
  pp.multi_batch = n_batches > 1 ? 1 : 0;
  int slice = (int)(per_cta / ((size_t)kPipeStages * (pp.batch_rows * sizeof(T) + K * sizeof(float)))) - 8;
  slice = slice / 32 * 32;
  if (slice > 2048) slice = 2048;
  int grid = plan->num_sms * kPipeCtasPerSm;
  if (grid > plan->proj_grid) grid = plan->proj_grid;
  // leave one slot per group free: the locator's CTAs (launched as dependents) then become resident while this
  // kernel streams and use the time to stage their tables and work on part A
  if (plan->q <= plan->num_sms / 2 && grid >= 4 * plan->q) grid -= plan->q;
  int64_t range_len = (plan->d_c + grid - 1) / grid;
  range_len = (range_len + 3) / 4 * 4;
  if (range_len < slice) slice = (int)((range_len + 31) / 32 * 32);
  // the optimistic recovery hands a slice out in passes of 256 opt_ch columns (opt_ch chunks per consumer thread): a
  // width that is a multiple of that keeps every lane busy; when that would cost more than an eighth of the slice (more
  // stages, each with its overhead) the width stays and opt_ch is the one that pads the last pass least
  const int max_ch = sizeof(T) == 8 ? 2 : kOptChunks;     // float64: two chunks per lane at most (registers)
  pp.opt_ch = max_ch;
  if (pp.opt_rows > 0 && slice >= kPipeConsumers) {
    int best_ch = 0, best_slice = 0;
    for (int ch = 1; ch <= max_ch; ++ch) {
      const int rounded = slice / (kPipeConsumers * ch) * (kPipeConsumers * ch);
      if (rounded >= best_slice && rounded > 0) { best_slice = rounded; best_ch = ch; }
    }
    if (best_slice * 8 >= slice * 7) {
      slice = best_slice;
      pp.opt_ch = best_ch;
    } else {
      int best_work = 1 << 30;
      for (int ch = 1; ch <= max_ch; ++ch) {
        const int work = (slice + kPipeConsumers * ch - 1) / (kPipeConsumers * ch) * ch;
        if (work <= best_work) { best_work = work; pp.opt_ch = ch; }
      }
    }
  }
  pp.slice_cols = slice;
  pp.slot_floats = slice + 8;
  // part A (only when the locator kernel will work ahead on it): about an eighth of the range, whole slices, at least one
  int64_t a_slices = range_len / slice / 8;
  if (a_slices < 1) a_slices = 1;
  const bool two_parts = !final_reduce && uses_early_locator(plan) && !early_locator_starved(plan);
  pp.part_a_cols = two_parts ? a_slices * slice : 0;
  const size_t smem = 128 + (size_t)kPipeStages * (pp.batch_rows * sizeof(T) + K * sizeof(float)) * pp.slot_floats;
  // which buffer holds the current draw: known on the host while decodes do not draw (the count then stands still)
  const bool host_knows = !plan->fresh_f && plan->draw_parity >= 0;
  const float* f_first = host_knows ? (plan->draw_parity ? plan->d_f2 : plan->d_f) : plan->d_f;
  const unsigned long long* draw_count = host_knows ? nullptr : plan->d_draw;
  SOLON_CUDA_TRY(cudaFuncSetAttribute(project_pipe_kernel<K, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  project_pipe_kernel<K, T><<<grid, kPipeThreads, smem, plan->stream>>>(received, f_first, plan->d_f2, draw_count, plan->f_pitch, plan->P, plan->d_c,
                                                                     range_len, pp, plan->d_partials, rho_out, nu_out,
                                                                     plan->d_proj_ticket, final_reduce);
  const int n_bunches = (grid + kProjBunch - 1) / kProjBunch;
  const size_t n_acc = (size_t)(K + 1) * plan->P;
  plan->proj_bunches = final_reduce ? 0 : n_bunches;
  plan->proj_bunch_a = plan->d_partials + 2 * (size_t)grid * n_acc;
  plan->proj_bunch_sums = plan->proj_bunch_a + (size_t)n_bunches * n_acc;
  plan->proj_progress_target = (unsigned long long)n_bunches;     // progress[0] once part A is complete (the recovery kernel zeroes it)
  plan->proj_two_parts = two_parts ? 1 : 0;
  SOLON_CUDA_TRY(cudaGetLastError());
  return SOLON_OK;
}

template <typename T>
static int launch_project_t(solon_plan* plan, const T* received, double* rho_out, double* nu_out, T* agg) {
  // no output buffers: the decode proper, whose locator kernel adds the last level of partial sums itself
  const int final_reduce = (rho_out || nu_out) ? 1 : 0;
  if (!rho_out) rho_out = plan->d_rho;
  if (!nu_out) nu_out = plan->d_nu;
  plan->launches += 1;
  switch (plan->K) {
    case 1: return launch_project_pipe_k<1, T>(plan, received, rho_out, nu_out, final_reduce, agg);
    case 2: return launch_project_pipe_k<2, T>(plan, received, rho_out, nu_out, final_reduce, agg);
    case 3: return launch_project_pipe_k<3, T>(plan, received, rho_out, nu_out, final_reduce, agg);
    case 4: return launch_project_pipe_k<4, T>(plan, received, rho_out, nu_out, final_reduce, agg);
    default: return SOLON_ERR_INVALID_ARG;
  }
}

int launch_project(solon_plan* plan, const float* received, double* rho_out, double* nu_out, float* agg) {
  return launch_project_t<float>(plan, received, rho_out, nu_out, agg);
}
int launch_project_f64(solon_plan* plan, const double* received, double* rho_out, double* nu_out, double* agg) {
  return launch_project_t<double>(plan, received, rho_out, nu_out, agg);
}

// ---- projections without any allocation ------------------------------------------------------------
//
// Scratch for solon_project_noalloc: the per-CTA partial sums, the per-bunch sums and the tickets of
// project_kernel, in a file-scope device array instead of plan-owned cudaMalloc memory.  Every GPU that
// loads the library holds these bytes until the process exits.
constexpr int kNoAllocMaxCtas = 296;                                   // grid cap of the no-allocation variant
constexpr int kNoAllocMaxSums = 512;                                   // (K + 1) * P
constexpr int kNoAllocBunches = kNoAllocMaxCtas / kProjBunch + 1;
constexpr size_t kNoAllocPartialBytes = (size_t)(kNoAllocMaxCtas + kNoAllocBunches) * kNoAllocMaxSums * sizeof(double);
constexpr size_t kNoAllocTicketBytes = 256;                            // 1 + kNoAllocBunches counters, padded
static_assert((1 + kNoAllocBunches) * sizeof(unsigned int) <= kNoAllocTicketBytes, "ticket area too small");
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocPartialBytes + kNoAllocTicketBytes];

constexpr int kNoAllocMaxDevices = 64;
static std::mutex g_noalloc_mutex;
static unsigned char* g_noalloc_ptr[kNoAllocMaxDevices];               // device address of the array, per device

// In host code the array's name is only a handle; the device address comes from cudaGetSymbolAddress,
// asked once per device while that device is current.
static int noalloc_scratch_address(unsigned char** out) {
  int device = -1;
  SOLON_CUDA_TRY(cudaGetDevice(&device));
  if (device < 0 || device >= kNoAllocMaxDevices) return SOLON_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (!g_noalloc_ptr[device]) {
    void* ptr = nullptr;
    SOLON_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
    if (!ptr) return SOLON_ERR_CUDA;
    g_noalloc_ptr[device] = static_cast<unsigned char*>(ptr);
  }
  *out = g_noalloc_ptr[device];
  return SOLON_OK;
}

template <int K>
static int launch_project_noalloc_k(const float* received, const float* f, int64_t f_pitch, int P, int64_t d_c,
                                    double* rho, double* nu, cudaStream_t stream, unsigned char* scratch) {
  int tile_cols = K <= 2 ? 2048 : 1024;
  size_t smem = (size_t)K * tile_cols * sizeof(double) + (size_t)(K + 1) * P * sizeof(double);
  SOLON_CUDA_TRY(cudaFuncSetAttribute(project_kernel<K>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  int device = 0, num_sms = 0, per_sm = 1;
  SOLON_CUDA_TRY(cudaGetDevice(&device));
  SOLON_CUDA_TRY(cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, device));
  SOLON_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, project_kernel<K>, kProjThreads, smem));
  int grid = num_sms * (per_sm < 1 ? 1 : per_sm);
  if (grid > kNoAllocMaxCtas) grid = kNoAllocMaxCtas;
  int64_t range_len = (d_c + grid - 1) / grid;
  range_len = (range_len + 3) / 4 * 4;
  if (range_len < tile_cols) tile_cols = (int)range_len;
  double* partials = reinterpret_cast<double*>(scratch);
  unsigned int* ticket = reinterpret_cast<unsigned int*>(scratch + kNoAllocPartialBytes);
  // the tickets must start at zero; the partial sums are fully rewritten by every launch
  SOLON_CUDA_TRY(cudaMemsetAsync(ticket, 0, kNoAllocTicketBytes, stream));
  project_kernel<K><<<grid, kProjThreads, smem, stream>>>(received, f, f_pitch, P, d_c, range_len, tile_cols, partials,
                                                          rho, nu, ticket, 1);
  SOLON_CUDA_TRY(cudaGetLastError());
  return SOLON_OK;
}

}  // namespace solon

extern "C" int solon_project_noalloc(const float* received, const float* f, int64_t f_pitch, int P, int64_t d_c, int K,
                                     double* rho, double* nu, void* cuda_stream) {
  using namespace solon;
  if (!received || !f || !rho || !nu) return SOLON_ERR_INVALID_ARG;
  if (P < 1 || d_c < 1 || K < 1 || K > SOLON_MAX_PROJECTIONS) return SOLON_ERR_INVALID_ARG;
  if ((int64_t)(K + 1) * P > kNoAllocMaxSums) return SOLON_ERR_INVALID_ARG;      // beyond the static scratch
  if (f_pitch < d_c || (f_pitch & 3) || ((uintptr_t)f & 15) || ((uintptr_t)received & 3)) return SOLON_ERR_INVALID_ARG;
  unsigned char* scratch = nullptr;
  int rc = noalloc_scratch_address(&scratch);
  if (rc) return rc;
  cudaStream_t stream = (cudaStream_t)cuda_stream;
  switch (K) {
    case 1: return launch_project_noalloc_k<1>(received, f, f_pitch, P, d_c, rho, nu, stream, scratch);
    case 2: return launch_project_noalloc_k<2>(received, f, f_pitch, P, d_c, rho, nu, stream, scratch);
    case 3: return launch_project_noalloc_k<3>(received, f, f_pitch, P, d_c, rho, nu, stream, scratch);
    default: return launch_project_noalloc_k<4>(received, f, f_pitch, P, d_c, rho, nu, stream, scratch);
  }
}
