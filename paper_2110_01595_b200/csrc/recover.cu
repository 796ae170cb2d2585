// Recovery kernel: the block decoder psi of Section 3.4 applied to every chunk, fused with the final sum
// of Algorithm 1:  agg[p m + l] = sum_g sum_{j in rows_g} coeff_g[j][l] * R[rows_g[j]][p],  truncated to d.
//
// One pass over the trusted rows the locator selected (m per group when m <= 6, else all trusted rows),
// streamed through shared memory with bulk asynchronous copies (see recover_kernel).  The m outputs of
// each chunk are accumulated in registers: float32 for m <= 6, where the weights are small; float64
// above, where they reach 10^3 and cancel.  The rows and weights come from device memory written by the
// locator kernel, so no host round trip separates the two.
#include "solon_internal.h"
#include "stream_pipe.cuh"

namespace solon {

constexpr int kRecThreads = 256;

template <typename T>
struct RecoverParamsT {
  const T* R;
  T* agg;
  int64_t d, d_c;
  int q, m, P;
  const int* group_start;
  const int* n_rec;      // q
  const int* rec_rows;   // P, group g's rows at [group_start[g], +n_rec[g])
  const double* coeff;   // P x m, same indexing
  unsigned long long* proj_progress;   // the projection kernel's part-A count, zeroed here for the next decode
  const int* opt;        // optimistic decode: opt[1] - the projection pass of this decode recovered too; opt[8 + g] - group g is clean
};
typedef RecoverParamsT<float> RecoverParams;

// Copy the locator's tables (group layout, rows per group, row indices, weights) into shared memory.
template <typename Acc, typename Prm>
__device__ __forceinline__ void load_tables(const Prm& prm, Acc* coeff_s, int* rows_s, int* start_s,
                                            int* n_rec_s) {
  for (int i = threadIdx.x; i < prm.P * prm.m; i += blockDim.x) coeff_s[i] = (Acc)prm.coeff[i];
  for (int i = threadIdx.x; i < prm.P; i += blockDim.x) rows_s[i] = prm.rec_rows[i];
  for (int i = threadIdx.x; i <= prm.q; i += blockDim.x) start_s[i] = prm.group_start[i];
  for (int i = threadIdx.x; i < prm.q; i += blockDim.x) n_rec_s[i] = prm.n_rec[i];
  __syncthreads();
}

// The locator's tables, brought on chip in ONE parallel round trip (every load is independent of every other),
// then packed in order of use from the on-chip copies: the i-th row in use (all groups, in group order) has its
// matrix row and its offset from a 16-byte boundary in rowsh_c[i] = (row << 2) | ((row * d_c) & 3) and its M
// weights at coeff_c[i * STRIDE .. + M) (STRIDE: M rounded up so that every row of weights starts on a 16-byte
// boundary and can be fetched with 128-bit loads).  Returns the number of rows in use.
// coeff_s (P x M), rows_s, slots_s (P each), start_s (q + 1), n_rec_s (q): staging.
// nothing_to_do: this thread's view of "the aggregate is already there" (optimistic decode); when every thread of the CTA
// says so the routine returns -1 at its first barrier, before it packs anything.
template <typename Acc, int M, int STRIDE, int VEC, typename Prm>
__device__ __forceinline__ int pack_tables(const Prm& prm, int* rows_s, Acc* coeff_s, int* slots_s, int* start_s,
                                           int* n_rec_s, int* count_s, Acc* coeff_c, int* rowsh_c, int nothing_to_do) {
  for (int i = threadIdx.x; i < prm.P * M; i += blockDim.x) coeff_s[i] = (Acc)prm.coeff[i];
  for (int i = threadIdx.x; i < prm.P; i += blockDim.x) rows_s[i] = prm.rec_rows[i];
  for (int i = threadIdx.x; i <= prm.q; i += blockDim.x) start_s[i] = prm.group_start[i];
  for (int i = threadIdx.x; i < prm.q; i += blockDim.x) n_rec_s[i] = prm.n_rec[i];
  if (__syncthreads_and(nothing_to_do)) return -1;
  for (int g = threadIdx.x; g < prm.q; g += blockDim.x) {
    int base = 0;
    for (int o = 0; o < g; ++o) base += min(max(n_rec_s[o], 0), start_s[o + 1] - start_s[o]);
    const int src = start_s[g];
    const int n = min(max(n_rec_s[g], 0), start_s[g + 1] - src);   // never more than the group has nodes
    for (int j = 0; j < n; ++j) slots_s[base + j] = src + j;
    if (g == prm.q - 1) *count_s = base + n;
  }
  __syncthreads();
  const int n_rows = *count_s;
  const int dc_mod4 = (int)(prm.d_c & (VEC - 1));       // VEC: elements per 16 bytes
  for (int i = threadIdx.x; i < n_rows; i += blockDim.x) {
    const int row = rows_s[slots_s[i]];
    rowsh_c[i] = (row << 2) | (((row & (VEC - 1)) * dc_mod4) & (VEC - 1));
  }
  for (int i = threadIdx.x; i < n_rows * STRIDE; i += blockDim.x) {
    const int r = i / STRIDE, l = i - r * STRIDE;
    coeff_c[i] = l < M ? coeff_s[(size_t)slots_s[r] * M + l] : (Acc)0;
  }
  __syncthreads();
  return n_rows;
}

// Bytes reserved for a P x M table of doubles in shared memory, rounded up to 16.
__host__ __device__ inline size_t recover_coeff_bytes(int P, int M) { return ((size_t)P * M * sizeof(double) + 15) & ~(size_t)15; }
// Weights per packed row: M rounded up to a whole number of 16-byte words.
template <typename Acc, int M>
struct PackedStride { static constexpr int value = (int)(((M * sizeof(Acc) + 15) / 16) * 16 / sizeof(Acc)); };

// One packed row of weights from shared memory, 16 bytes per load.
template <int STRIDE>
__device__ __forceinline__ void load_weights(const float* __restrict__ src, float (&c)[STRIDE]) {
#pragma unroll
  for (int t = 0; t < STRIDE / 4; ++t) {
    const float4 v = reinterpret_cast<const float4*>(src)[t];
    c[4 * t] = v.x;
    c[4 * t + 1] = v.y;
    c[4 * t + 2] = v.z;
    c[4 * t + 3] = v.w;
  }
}
template <int STRIDE>
__device__ __forceinline__ void load_weights(const double* __restrict__ src, double (&c)[STRIDE]) {
#pragma unroll
  for (int t = 0; t < STRIDE / 2; ++t) {
    const double2 v = reinterpret_cast<const double2*>(src)[t];
    c[2 * t] = v.x;
    c[2 * t + 1] = v.y;
  }
}

constexpr int kRecConsumers = 256;   // consumer threads per CTA of the float32 kernels (template parameter NC)

struct RecoverPipe {
  int row_batch;     // rows per stage
  int stages;
  int slot_floats;   // shared-memory floats per row slot (multiple of 4)
  unsigned long long* tile_counter;   // next tile to hand out; zero at launch
  int* status;
};

// Streaming kernel: a producer warp moves the selected rows, tile by tile and a few rows at a time, into a
// shared-memory ring with bulk asynchronous copies; consumer threads own CPT chunks each, take one float per
// row from the ring, apply the row's m weights, and every consumer warp writes its runs of chunks back
// through its own shared buffer as contiguous 128-bit stores.
// kStreamStores: write the aggregate with streaming stores (evict-first in L2; a template parameter, not a run-time
// branch: with both forms in one kernel the compiler kept 94 registers instead of 72 and the kernel ran 7 - 40 % longer).
template <int M, int CPT, typename Acc, int NC, int kCtasPerSm, typename T, bool kStreamStores>
__global__ void __launch_bounds__(NC + 32, kCtasPerSm) recover_kernel(RecoverParamsT<T> prm, RecoverPipe pp) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  constexpr int kTileChunks = NC * CPT;
  constexpr int64_t kVec = 16 / sizeof(T);     // elements per 16 bytes
  const int tid = threadIdx.x;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem_raw);
  uint64_t* empty_bar = full_bar + pp.stages;
  long long* tile_of = reinterpret_cast<long long*>(empty_bar + pp.stages);   // per stage: tile of the batch it holds
  int* b0_of = reinterpret_cast<int*>(tile_of + pp.stages);                  // per stage: first row of that batch
  int* abort_flag = b0_of + pp.stages;
  int* count_s = abort_flag + 1;
  // every region starts on a 16-byte boundary (128-bit shared loads, bulk-copy destinations)
  constexpr int kStride = PackedStride<Acc, M>::value;
  Acc* coeff_p = reinterpret_cast<Acc*>(smem_raw + 256);                                  // P x M (staging)
  Acc* coeff_c = reinterpret_cast<Acc*>(smem_raw + 256 + recover_coeff_bytes(prm.P, M));  // P x kStride (packed)
  int* rows_p = reinterpret_cast<int*>(smem_raw + 256 + recover_coeff_bytes(prm.P, M) + recover_coeff_bytes(prm.P, kStride));
  int* slots_p = rows_p + ((prm.P + 3) & ~3);                                             // P
  int* rowsh_c = slots_p + ((prm.P + 3) & ~3);                                            // P (packed)
  int* start_s = rowsh_c + ((prm.P + 3) & ~3);                                            // q + 1
  int* n_rec_s = start_s + ((prm.q + 4) & ~3);                                            // q
  T* out_all = reinterpret_cast<T*>(n_rec_s + ((prm.q + 3) & ~3));                        // one buffer of 32 x M per consumer warp
  T* ring = out_all + (size_t)(NC / 32) * 32 * M;                              // 32 M elements: a multiple of 16 bytes
  const size_t stage_floats = (size_t)pp.row_batch * pp.slot_floats;

  if (tid == 0) {
    for (int s = 0; s < pp.stages; ++s) {
      pipe::mbar_init(&full_bar[s], 32);
      pipe::mbar_init(&empty_bar[s], NC / 32);
    }
    *abort_flag = 0;
    pipe::fence_barrier_init();
  }
  pdl_wait();   // the locator's mask and table are complete and visible; nothing above touched global memory
  if (blockIdx.x == 0 && tid == 0) {   // every locator CTA is done with them: ready for the next decode
    prm.proj_progress[0] = 0ULL;
    prm.proj_progress[1] = 0ULL;
  }
  // optimistic decode: the projection pass has already written the aggregate, and it stands if every group is clean
  // (no branch on the first word before the other loads: they all go out together with the table loads below)
  int clean = prm.opt[1] != 0 ? 1 : 0;
  for (int g = tid; g < prm.q; g += blockDim.x) clean &= prm.opt[8 + g] != 0 ? 1 : 0;
  const int n_rows = pack_tables<Acc, M, kStride, (int)kVec>(prm, rows_p, coeff_p, slots_p, start_s, n_rec_s, count_s, coeff_c, rowsh_c, clean);
  if (n_rows < 0) return;   // the rows the projection pass recovered from were all confirmed: the aggregate stands
  const int64_t n_tiles = (prm.d_c + kTileChunks - 1) / kTileChunks;
  const int64_t total_floats = (int64_t)prm.P * prm.d_c;

  // Tiles are handed out through a global counter (zeroed by the locator kernel), not by a fixed stride: SMs do
  // not all draw the same bandwidth (those of the fuller GPCs get about a third less), and with equal shares the
  // slow ones finish long after the rest.  The producer announces every batch's tile in tile_of[stage]; a
  // negative tile ends the stream.
  if (tid >= NC) {
    const int lane = tid - NC;
    const uint64_t stream_policy = pipe::policy_evict_first();   // last use of the received rows
    uint32_t it = 0;
    long long tile = 0;
    if (lane == 0) tile = (long long)atomicAdd(pp.tile_counter, 1ULL);
    tile = __shfl_sync(0xffffffffu, tile, 0);
    while (tile < n_tiles) {
      const int64_t c0 = tile * kTileChunks;
      int64_t c1 = c0 + kTileChunks;
      if (c1 > prm.d_c) c1 = prm.d_c;
      int b0 = 0;
      do {
        const int stage = it % pp.stages;
        const uint32_t phase = (it / pp.stages) & 1;
        if (it >= (uint32_t)pp.stages) pipe::mbar_wait(&empty_bar[stage], phase ^ 1, abort_flag, pp.status + 1);
        const int nb = min(pp.row_batch, n_rows - b0);
        if (lane == 0) {
          tile_of[stage] = tile;
          b0_of[stage] = b0;
        }
        if (lane < nb) {
          const int64_t first = (int64_t)(rowsh_c[b0 + lane] >> 2) * prm.d_c + c0;
          const int64_t last = first + (c1 - c0);
          const int64_t a0 = first & ~(kVec - 1);                   // enclosing 16-byte boundary
          int64_t a1 = (last + kVec - 1) & ~(kVec - 1);
          const int64_t safe_end = total_floats & ~(kVec - 1);      // bulk copies stay inside the matrix
          if (a1 > safe_end) a1 = safe_end;
          T* slot = ring + stage * stage_floats + (size_t)lane * pp.slot_floats;
          const uint32_t bytes = a1 > a0 ? (uint32_t)((a1 - a0) * sizeof(T)) : 0u;
          for (int64_t e = (a1 > a0 ? a1 : a0); e < last; ++e) slot[e - a0] = prm.R[e];   // fewer than 16 bytes
          if (bytes) {
            pipe::mbar_arrive_expect_tx(&full_bar[stage], bytes);
            pipe::bulk_load_hint(slot, prm.R + a0, bytes, &full_bar[stage], stream_policy);
          } else {
            pipe::mbar_arrive(&full_bar[stage]);
          }
        } else {
          pipe::mbar_arrive(&full_bar[stage]);
        }
        b0 += pp.row_batch;
        ++it;
      } while (b0 < n_rows);
      // claim late: a tile claimed ahead of time is a tile a faster SM can no longer take
      if (lane == 0) tile = (long long)atomicAdd(pp.tile_counter, 1ULL);
      tile = __shfl_sync(0xffffffffu, tile, 0);
    }
    {
      const int stage = it % pp.stages;
      const uint32_t phase = (it / pp.stages) & 1;
      if (it >= (uint32_t)pp.stages) pipe::mbar_wait(&empty_bar[stage], phase ^ 1, abort_flag, pp.status + 1);
      if (lane == 0) tile_of[stage] = -1;
      pipe::mbar_arrive(&full_bar[stage]);
    }
    if (*(volatile int*)abort_flag) pipe::drain_delay();
    return;
  }

  const int lane = tid & 31, warp = tid >> 5;
  T* out_s = out_all + (size_t)warp * 32 * M;
  Acc acc[CPT][M];
  for (uint32_t it = 0;; ++it) {
    const int stage = it % pp.stages;
    const uint32_t phase = (it / pp.stages) & 1;
    pipe::mbar_wait(&full_bar[stage], phase, abort_flag, pp.status + 1);
    const long long tile = *(volatile long long*)&tile_of[stage];
    if (tile < 0 || *(volatile int*)abort_flag) break;
    const int b0 = *(volatile int*)&b0_of[stage];
    const int64_t c0 = tile * kTileChunks;   // a multiple of 4: a row's offset from a 16-byte boundary is the same in every tile
    if (b0 == 0) {
#pragma unroll
      for (int i = 0; i < CPT; ++i)
#pragma unroll
        for (int l = 0; l < M; ++l) acc[i][l] = (Acc)0;
    }
    // Chunks past the end of the matrix (last tile only) read whatever an earlier tile left in the ring: finite
    // values, whose sums are never written back.
    const int nb = min(pp.row_batch, n_rows - b0);
    const T* slot = ring + stage * stage_floats + tid;
    const int* rs = rowsh_c + b0;
    const Acc* cj = coeff_c + (size_t)b0 * kStride;
#pragma unroll(sizeof(Acc) == 8 ? 1 : 2)
    for (int j = 0; j < nb; ++j) {
      const T* src = slot + (rs[j] & 3);
      Acc v[CPT];
#pragma unroll
      for (int i = 0; i < CPT; ++i) v[i] = (Acc)src[i * NC];
      Acc c[kStride];
      load_weights<kStride>(cj, c);
#pragma unroll
      for (int l = 0; l < M; ++l) {
#pragma unroll
        for (int i = 0; i < CPT; ++i) acc[i][l] = fma(c[l], v[i], acc[i][l]);
      }
      slot += pp.slot_floats;
      cj += kStride;
    }
    __syncwarp();
    if (lane == 0) pipe::mbar_arrive(&empty_bar[stage]);
    if (b0 + pp.row_batch < n_rows) continue;
    // last batch of the tile: write back; for each i the warp's 32 chunks are contiguous, 32 M floats starting
    // on a 16-byte boundary
#pragma unroll
    for (int i = 0; i < CPT; ++i) {
#pragma unroll
      for (int l = 0; l < M; ++l) out_s[lane * M + l] = (T)acc[i][l];
      __syncwarp();
      const int64_t o0 = (c0 + (int64_t)i * NC + warp * 32) * M;
      int64_t o1 = o0 + 32 * M;
      if (o1 > prm.d) o1 = prm.d;
      const int count = o1 > o0 ? (int)(o1 - o0) : 0;
      const int vec = count / (int)kVec;                          // whole 16-byte words
      float4* dst4 = reinterpret_cast<float4*>(prm.agg + o0);
      const float4* src4 = reinterpret_cast<const float4*>(out_s);
      if constexpr (kStreamStores) {
        for (int e = lane; e < vec; e += 32) __stcs(dst4 + e, src4[e]);
        for (int e = vec * (int)kVec + lane; e < count; e += 32) __stcs(prm.agg + o0 + e, out_s[e]);
      } else {
        for (int e = lane; e < vec; e += 32) dst4[e] = src4[e];
        for (int e = vec * (int)kVec + lane; e < count; e += 32) prm.agg[o0 + e] = out_s[e];
      }
      __syncwarp();
    }
  }
}

// Any m: one thread per output coordinate (slower; used for compression ratios without a specialisation).
__global__ void __launch_bounds__(kRecThreads) recover_generic_kernel(RecoverParams prm) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  double* coeff_s = reinterpret_cast<double*>(smem_raw);
  int* rows_s = reinterpret_cast<int*>(coeff_s + (size_t)prm.P * prm.m);
  int* start_s = rows_s + prm.P;
  int* n_rec_s = start_s + prm.q + 1;
  load_tables(prm, coeff_s, rows_s, start_s, n_rec_s);
  if (blockIdx.x == 0 && threadIdx.x == 0) {   // ready for the next decode
    prm.proj_progress[0] = 0ULL;
    prm.proj_progress[1] = 0ULL;
  }
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < prm.d; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t p = e / prm.m;
    const int l = (int)(e - p * prm.m);
    double acc = 0.0;
    for (int g = 0; g < prm.q; ++g) {
      const int base = start_s[g], n = n_rec_s[g];
      for (int j = 0; j < n; ++j)
        acc = fma(coeff_s[(size_t)(base + j) * prm.m + l], (double)prm.R[(int64_t)rows_s[base + j] * prm.d_c + p], acc);
    }
    prm.agg[e] = (float)acc;
  }
}

template <int M, int CPT, typename Acc, int NC, int kCtasPerSm, typename T, bool kStreamStores>
static int launch_recover_hint(solon_plan* plan, RecoverParamsT<T>& prm) {
  constexpr int kTileChunks = NC * CPT;
  RecoverPipe pp;
  pp.status = plan->d_status;
  pp.slot_floats = kTileChunks + 8;
  const size_t slot_bytes = (size_t)pp.slot_floats * sizeof(T);
  const size_t fixed = 256 + recover_coeff_bytes(plan->P, M) + recover_coeff_bytes(plan->P, PackedStride<Acc, M>::value) +
                       3 * (size_t)((plan->P + 3) & ~3) * sizeof(int) +
                       (size_t)(((plan->q + 4) & ~3) + ((plan->q + 3) & ~3)) * sizeof(int) +
                       (size_t)(NC / 32) * 32 * M * sizeof(T);
  // the locator may select up to all P rows (large m) or as few as q m; batches of about 20 KB (40 KB when one
  // CTA has the SM's shared memory to itself)
  int row_batch = (int)((size_t)(kCtasPerSm == 1 ? 40 : 20) * 1024 / slot_bytes);
  if (row_batch < 1) row_batch = 1;
  if (row_batch > 32) row_batch = 32;
  const int max_rows = M <= 6 ? plan->q * M : plan->P;
  if (row_batch > max_rows) row_batch = max_rows;
  {
    int nb = (max_rows + row_batch - 1) / row_batch;     // an even split of the expected row count
    row_batch = (max_rows + nb - 1) / nb;
  }
  const size_t per_cta = (size_t)227 * 1024 / kCtasPerSm - 1024;
  int stages = 4;
  while (stages > 2 && fixed + (size_t)stages * row_batch * slot_bytes > per_cta) --stages;
  while (row_batch > 1 && fixed + (size_t)stages * row_batch * slot_bytes > per_cta) --row_batch;
  {
    // few tiles per CTA: a deep ring would claim most of them up front and leave the counter nothing to balance
    const int64_t n_tiles_all = (plan->d_c + kTileChunks - 1) / kTileChunks;
    const int batches_per_tile = (max_rows + row_batch - 1) / row_batch;
    if (n_tiles_all < (int64_t)plan->num_sms * 4 * 16 && stages > batches_per_tile + 1) stages = batches_per_tile + 1;
  }
  const size_t smem = fixed + (size_t)stages * row_batch * slot_bytes;
  if (smem > (size_t)226 * 1024) return SOLON_ERR_INVALID_ARG;
  pp.row_batch = row_batch;
  pp.stages = stages;
  auto kernel = recover_kernel<M, CPT, Acc, NC, kCtasPerSm, T, kStreamStores>;
  SOLON_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  static_assert((32 * M * sizeof(T)) % 16 == 0, "warp runs must start on a 16-byte boundary of the output");
  int64_t tiles = (plan->d_c + kTileChunks - 1) / kTileChunks;
  int per_sm = 1;
  SOLON_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, (NC + 32), smem));
  if (per_sm < 1) per_sm = 1;
  int64_t cap = (int64_t)plan->num_sms * per_sm;
  int grid = (int)(tiles < cap ? tiles : cap);
  pp.tile_counter = plan->d_tile_counter;
  return launch_dependent(kernel, dim3(grid), dim3((NC + 32)), smem, plan->stream, prm, pp);
}

template <int M, int CPT, typename Acc, int NC, int kCtasPerSm, typename T>
static int launch_recover_m(solon_plan* plan, RecoverParamsT<T>& prm) {
  if (plan->stream_hints) return launch_recover_hint<M, CPT, Acc, NC, kCtasPerSm, T, true>(plan, prm);
  return launch_recover_hint<M, CPT, Acc, NC, kCtasPerSm, T, false>(plan, prm);
}

template <typename T>
static void fill_recover_params(solon_plan* plan, const T* received, T* agg, RecoverParamsT<T>* prm) {
  prm->R = received;
  prm->agg = agg;
  prm->d = plan->d;
  prm->d_c = plan->d_c;
  prm->q = plan->q;
  prm->m = plan->m;
  prm->P = plan->P;
  prm->group_start = plan->d_group_start;
  prm->n_rec = plan->d_n_rec;
  prm->rec_rows = plan->d_rec_rows;
  prm->coeff = plan->d_coeff;
  prm->proj_progress = plan->d_proj_progress;
  prm->opt = plan->d_opt;
}

// float64 received vectors and aggregate: weights and sums in float64 for every compression ratio.
int launch_recover_f64(solon_plan* plan, const double* received, double* agg) {
  RecoverParamsT<double> prm;
  fill_recover_params(plan, received, agg, &prm);
  plan->launches += 1;
  switch (plan->m) {
    case 1: return launch_recover_m<1, 4, double, kRecConsumers, 2>(plan, prm);
    case 2: return launch_recover_m<2, 4, double, kRecConsumers, 2>(plan, prm);
    case 3: return launch_recover_m<3, 4, double, kRecConsumers, 2>(plan, prm);
    case 4: return launch_recover_m<4, 2, double, kRecConsumers, 2>(plan, prm);
    case 5: return launch_recover_m<5, 2, double, kRecConsumers, 2>(plan, prm);
    case 6: return launch_recover_m<6, 2, double, kRecConsumers, 2>(plan, prm);
    case 8: return launch_recover_m<8, 4, double, 480, 1>(plan, prm);
    case 10: return launch_recover_m<10, 4, double, 480, 1>(plan, prm);
    case 12: return launch_recover_m<12, 2, double, 480, 1>(plan, prm);
    case 14: return launch_recover_m<14, 2, double, 480, 1>(plan, prm);
    default: return SOLON_ERR_INVALID_ARG;
  }
}

int launch_recover(solon_plan* plan, const float* received, float* agg) {
  RecoverParams prm;
  fill_recover_params(plan, received, agg, &prm);
  plan->launches += 1;
#define SOLON_RECOVER_CASE(M_, CPT_, ACC_, NC_, BLOCKS_) \
  case M_:                                               \
    return launch_recover_m<M_, CPT_, ACC_, NC_, BLOCKS_>(plan, prm);
  switch (plan->m) {
    SOLON_RECOVER_CASE(1, 4, float, kRecConsumers, 2)
    SOLON_RECOVER_CASE(2, 4, float, kRecConsumers, 2)
    SOLON_RECOVER_CASE(3, 4, float, kRecConsumers, 2)
    SOLON_RECOVER_CASE(4, 4, float, kRecConsumers, 2)
    SOLON_RECOVER_CASE(5, 4, float, kRecConsumers, 2)
    SOLON_RECOVER_CASE(6, 2, float, kRecConsumers, 2)
    SOLON_RECOVER_CASE(8, 4, double, 480, 1)
    SOLON_RECOVER_CASE(10, 4, double, 480, 1)
    default: break;
  }
#undef SOLON_RECOVER_CASE
  size_t smem = (size_t)plan->P * plan->m * sizeof(double) + (size_t)(plan->P + 2 * plan->q + 2) * sizeof(int);
  if (smem > 200 * 1024) return SOLON_ERR_INVALID_ARG;
  SOLON_CUDA_TRY(cudaFuncSetAttribute(recover_generic_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  int64_t want = (plan->d + kRecThreads - 1) / kRecThreads;
  int64_t cap = (int64_t)plan->num_sms * 8;
  int grid = (int)(want < cap ? want : cap);
  recover_generic_kernel<<<grid, kRecThreads, smem, plan->stream>>>(prm);
  SOLON_CUDA_TRY(cudaGetLastError());
  return SOLON_OK;
}

}  // namespace solon
