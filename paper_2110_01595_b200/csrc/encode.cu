// Encode kernel (Section 3.4): z_k = W_k (Y_k 1_P), W_k = I_{d_c} (x) [1, w_k, ..., w_k^{m-1}].
//
// One pass over the P x d gradient matrix.  A tile is (group g, a run of chunks); the r_g rows of the
// group are streamed through shared memory in batches by a producer warp that issues one bulk
// asynchronous copy (cp.async.bulk, completion on an mbarrier) per row segment, so every gradient
// byte is read from HBM exactly once and many kilobytes per SM are in flight without occupying
// registers.  In the specialised kernels (m = 1..6, 8, 10) each consumer thread owns whole chunks:
// it adds the r_g rows of its chunks into registers straight from the staged rows, then evaluates the
// r_g polynomials sum_l w_k^l ybar[p m + l] by Horner's rule and stores one float32 per node (coalesced
// along the chunk axis); no CTA-wide barrier is needed.  The group sum ybar is accumulated in float32
// in every specialised kernel: whatever rounding it carries is common to all nodes of the group, so the
// coded values still lie on ONE polynomial (with coefficients ybar + delta) and the decoder returns
// ybar + delta without amplifying delta.  Only the rounding that differs from node to node - the Horner
// evaluation and the final rounding to float32 - is amplified by the decoder (about 2^(m-1)), so for
// m > 6 the polynomials are evaluated in float64 and rounded once; for m <= 6 float32 is enough.  The
// generic kernel (any m) sums into a float32 ybar tile in shared memory first (rows in node order, like the
// specialised kernels) and evaluates in float64.
//
// Row segments start at arbitrary 4-byte offsets (d need not be a multiple of 4): the copy starts at
// the enclosing 16-byte boundary and consumers index from the remainder; the last few floats of the
// whole matrix, where rounding the end up would leave the buffer, are fetched with ordinary loads.
#include "solon_internal.h"
#include "stream_pipe.cuh"

namespace solon {

constexpr int kEncConsumers = 256;                 // consumer threads per CTA
constexpr int kEncThreads = kEncConsumers + 32;    // + one producer warp
constexpr int kEncMaxBatch = 32;                   // rows per pipeline stage (one per producer lane)

template <typename T>
struct EncodeParamsT {
  const T* grads;
  T* coded;
  const int* group_start;
  const double* w;
  int q, m, P;
  int64_t d, d_c;
  int64_t total_floats;   // P * d (elements)
  int chunks_per_thread;  // tile = kEncConsumers * chunks_per_thread chunks
  int row_batch;          // rows per stage
  int stages;
  int slot_floats;        // shared-memory floats per row slot (multiple of 4)
  int64_t tiles_per_group;
  unsigned long long* tile_counter;   // [0] next tile to hand out, [1] CTAs that have left; both zero at launch
  int* status;            // device status words: [1] collects wait-expiry bits
  int stream_hints;       // mark the gradients read and the coded values written evict-first in L2
};
typedef EncodeParamsT<float> EncodeParams;

// Elements per 16 bytes (the granularity of bulk copies): 4 floats or 2 doubles.
template <typename T>
struct Vec16 { static constexpr int64_t n = 16 / sizeof(T); };

// Horner evaluation for all nodes of the group with the chunk held in registers.
template <int M>
__device__ __forceinline__ void mix_chunk(const float* __restrict__ y, const double* __restrict__ w_g, int r_g,
                                          float* __restrict__ out, int64_t out_stride) {
  double c[M];
#pragma unroll
  for (int l = 0; l < M; ++l) c[l] = (double)y[l];
  for (int k = 0; k < r_g; ++k) {
    double wk = w_g[k];
    double acc = c[M - 1];
#pragma unroll
    for (int l = M - 2; l >= 0; --l) acc = fma(acc, wk, c[l]);
    out[(int64_t)k * out_stride] = (float)acc;
  }
}

__device__ __forceinline__ void mix_chunk_generic(const float* __restrict__ y, int m, const double* __restrict__ w_g,
                                                  int r_g, float* __restrict__ out, int64_t out_stride) {
  for (int k = 0; k < r_g; ++k) {
    double wk = w_g[k];
    double acc = (double)y[m - 1];
    for (int l = m - 2; l >= 0; --l) acc = fma(acc, wk, (double)y[l]);
    out[(int64_t)k * out_stride] = (float)acc;
  }
}

template <int M>
__global__ void __launch_bounds__(kEncThreads, 2) encode_kernel(EncodeParams prm) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int tid = threadIdx.x;
  const int m = (M > 0) ? M : prm.m;
  const int tile_chunks = kEncConsumers * prm.chunks_per_thread;
  const int tile_floats = tile_chunks * m;

  // shared memory: [barriers][w_g x 2][ybar x 2][stages x row_batch x slot]; w_g and ybar (float32, added up
  // row by row in node order like in the specialised kernels) are double buffered by tile parity so that one
  // consumer barrier per tile suffices
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem_raw);
  uint64_t* empty_bar = full_bar + prm.stages;
  int* abort_flag = reinterpret_cast<int*>(empty_bar + prm.stages);
  double* w_s = reinterpret_cast<double*>(smem_raw + 256);
  float* ybar = reinterpret_cast<float*>(w_s + 2 * SOLON_MAX_GROUP);
  float* ring = ybar + 2 * (size_t)((tile_floats + 3) & ~3);
  const size_t stage_floats = (size_t)prm.row_batch * prm.slot_floats;

  if (tid == 0) {
    for (int s = 0; s < prm.stages; ++s) {
      pipe::mbar_init(&full_bar[s], 32);                     // every producer lane arrives
      pipe::mbar_init(&empty_bar[s], kEncConsumers / 32);    // one arrival per consumer warp
    }
    *abort_flag = 0;
    pipe::fence_barrier_init();
  }
  __syncthreads();

  const int64_t total_tiles = prm.tiles_per_group * prm.q;
  const bool is_producer = tid >= kEncConsumers;

  if (is_producer) {
    const int lane = tid - kEncConsumers;
    uint32_t it = 0;   // running stage counter
    for (int64_t tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
      const int g = (int)(tile / prm.tiles_per_group);
      const int64_t ct = tile - (int64_t)g * prm.tiles_per_group;
      const int row0 = prm.group_start[g], r_g = prm.group_start[g + 1] - row0;
      const int64_t e0 = ct * tile_floats;
      int64_t e1 = e0 + tile_floats;
      if (e1 > prm.d) e1 = prm.d;
      for (int b0 = 0; b0 < r_g; b0 += prm.row_batch, ++it) {
        const int stage = it % prm.stages;
        const uint32_t phase = (it / prm.stages) & 1;
        if (it >= (uint32_t)prm.stages) pipe::mbar_wait(&empty_bar[stage], phase ^ 1, abort_flag, prm.status + 1);
        const int nb = min(prm.row_batch, r_g - b0);
        if (lane < nb && e1 > e0) {
          const int64_t first = (int64_t)(row0 + b0 + lane) * prm.d + e0;    // float index of the segment
          const int64_t last = first + (e1 - e0);
          const int64_t a0 = first & ~(int64_t)3;                            // enclosing 16-byte boundary
          int64_t a1 = (last + 3) & ~(int64_t)3;
          const int64_t safe_end = prm.total_floats & ~(int64_t)3;           // bulk copies stay inside the matrix
          if (a1 > safe_end) a1 = safe_end;
          float* slot = ring + stage * stage_floats + (size_t)lane * prm.slot_floats;
          uint32_t bytes = a1 > a0 ? (uint32_t)((a1 - a0) * 4) : 0u;
          for (int64_t e = (a1 > a0 ? a1 : a0); e < last; ++e) slot[e - a0] = prm.grads[e];   // <= 3 floats
          if (bytes) {
            pipe::mbar_arrive_expect_tx(&full_bar[stage], bytes);
            pipe::bulk_load(slot, prm.grads + a0, bytes, &full_bar[stage]);
          } else {
            pipe::mbar_arrive(&full_bar[stage]);
          }
        } else {
          pipe::mbar_arrive(&full_bar[stage]);
        }
      }
    }
    // Every copy issued above is awaited by the consumers before they finish, unless a wait expired;
    // in that case drain here so no copy is in flight into shared memory when the CTA exits.
    if (*(volatile int*)abort_flag) pipe::drain_delay();
  } else {
    uint32_t it = 0;
    int parity = 0;   // ybar double buffer
    for (int64_t tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, parity ^= 1) {
      const int g = (int)(tile / prm.tiles_per_group);
      const int64_t ct = tile - (int64_t)g * prm.tiles_per_group;
      const int row0 = prm.group_start[g], r_g = prm.group_start[g + 1] - row0;
      const int64_t e0 = ct * tile_floats;
      int64_t e1 = e0 + tile_floats;
      if (e1 > prm.d) e1 = prm.d;
      const int valid = (int)(e1 > e0 ? e1 - e0 : 0);
      float* y = ybar + (size_t)parity * ((tile_floats + 3) & ~3);
      double* w_g = w_s + (size_t)parity * SOLON_MAX_GROUP;
      for (int k = tid; k < r_g; k += kEncConsumers) w_g[k] = prm.w[row0 + k];
      const int d_mod4 = (int)(prm.d & 3), e0_mod4 = (int)(e0 & 3);

      for (int b0 = 0; b0 < r_g; b0 += prm.row_batch, ++it) {
        const int stage = it % prm.stages;
        const uint32_t phase = (it / prm.stages) & 1;
        pipe::mbar_wait(&full_bar[stage], phase, abort_flag, prm.status + 1);
        const int nb = min(prm.row_batch, r_g - b0);
        const float* base = ring + stage * stage_floats;
        // each thread owns elements tid + i * 256 of the tile, four at a time
        for (int eb = tid; eb < tile_floats; eb += 4 * kEncConsumers) {
          const bool i1 = eb + kEncConsumers < tile_floats, i2 = eb + 2 * kEncConsumers < tile_floats,
                     i3 = eb + 3 * kEncConsumers < tile_floats;
          float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
          if (b0 > 0) {   // carry on from the rows of the earlier batches
            acc0 = y[eb];
            if (i1) acc1 = y[eb + kEncConsumers];
            if (i2) acc2 = y[eb + 2 * kEncConsumers];
            if (i3) acc3 = y[eb + 3 * kEncConsumers];
          }
          const bool v0 = eb < valid, v1 = eb + kEncConsumers < valid, v2 = eb + 2 * kEncConsumers < valid,
                     v3 = eb + 3 * kEncConsumers < valid;
          for (int j = 0; j < nb; ++j) {
            const int shift = ((((row0 + b0 + j) & 3) * d_mod4) + e0_mod4) & 3;   // (row * d + e0) mod 4
            const float* src = base + (size_t)j * prm.slot_floats + shift + eb;
            if (v0) acc0 += src[0];
            if (v1) acc1 += src[kEncConsumers];
            if (v2) acc2 += src[2 * kEncConsumers];
            if (v3) acc3 += src[3 * kEncConsumers];
          }
          y[eb] = acc0;
          if (i1) y[eb + kEncConsumers] = acc1;
          if (i2) y[eb + 2 * kEncConsumers] = acc2;
          if (i3) y[eb + 3 * kEncConsumers] = acc3;
        }
        __syncwarp();
        if ((tid & 31) == 0) pipe::mbar_arrive(&empty_bar[stage]);
      }
      pipe::named_barrier_sync(1, kEncConsumers);   // ybar (and w_s) complete

      const int64_t c0 = ct * tile_chunks;
      for (int i = 0; i < prm.chunks_per_thread; ++i) {
        const int p = tid + i * kEncConsumers;
        if (c0 + p < prm.d_c) {
          float* out = prm.coded + (int64_t)row0 * prm.d_c + c0 + p;
          if (M > 0) mix_chunk<(M > 0 ? M : 1)>(y + (size_t)p * m, w_g, r_g, out, prm.d_c);
          else mix_chunk_generic(y + (size_t)p * m, m, w_g, r_g, out, prm.d_c);
        }
      }
    }
  }
}


// ---- specialised kernels: a thread owns CPT whole chunks of M coordinates ---------------------------

template <typename Acc>
__device__ __forceinline__ Acc acc_fma(Acc a, Acc b, Acc c);
template <>
__device__ __forceinline__ float acc_fma<float>(float a, float b, float c) { return fmaf(a, b, c); }
template <>
__device__ __forceinline__ double acc_fma<double>(double a, double b, double c) { return fma(a, b, c); }

template <int M, int CPT, typename Acc, int kMinBlocks, typename T>
__global__ void __launch_bounds__(kEncThreads, kMinBlocks) encode_direct_kernel(EncodeParamsT<T> prm) {
  constexpr int64_t kVec = Vec16<T>::n;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int tid = threadIdx.x;
  constexpr int kTileChunks = kEncConsumers * CPT;
  constexpr int kTileFloats = kTileChunks * M;

  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem_raw);
  uint64_t* empty_bar = full_bar + prm.stages;
  long long* tile_of = reinterpret_cast<long long*>(empty_bar + prm.stages);   // per stage: tile of the batch it holds
  int* b0_of = reinterpret_cast<int*>(tile_of + prm.stages);                  // per stage: first row of that batch
  int* abort_flag = b0_of + prm.stages;
  Acc* w_s = reinterpret_cast<Acc*>(smem_raw + 256);                       // all P node scalars
  T* ring = reinterpret_cast<T*>(smem_raw + 256 + (((size_t)prm.P * sizeof(Acc) + 15) & ~(size_t)15));
  const size_t stage_floats = (size_t)prm.row_batch * prm.slot_floats;

  if (tid == 0) {
    for (int s = 0; s < prm.stages; ++s) {
      pipe::mbar_init(&full_bar[s], 32);
      pipe::mbar_init(&empty_bar[s], kEncConsumers / 32);
    }
    *abort_flag = 0;
    pipe::fence_barrier_init();
  }
  for (int k = tid; k < prm.P; k += kEncThreads) w_s[k] = (Acc)prm.w[k];
  __syncthreads();

  const int64_t total_tiles = prm.tiles_per_group * prm.q;

  // Tiles are handed out through a global counter, not by a fixed stride: the SMs do not all draw the same
  // bandwidth (those of the fuller GPCs get less), and with equal shares the slow ones finish long after the
  // rest.  The producer announces every batch's tile in tile_of[stage]; a negative tile ends the stream.  The
  // last CTA to leave puts the counters back to zero for the next launch.
  if (tid >= kEncConsumers) {
    const int lane = tid - kEncConsumers;
    const uint64_t stream_policy = pipe::policy_evict_first();
    uint32_t it = 0;
    long long tile = 0;
    if (lane == 0) tile = (long long)atomicAdd(prm.tile_counter, 1ULL);
    tile = __shfl_sync(0xffffffffu, tile, 0);
    while (tile < total_tiles) {
      const int g = (int)(tile / prm.tiles_per_group);
      const int64_t ct = tile - (int64_t)g * prm.tiles_per_group;
      const int row0 = prm.group_start[g], r_g = prm.group_start[g + 1] - row0;
      const int64_t e0 = ct * kTileFloats;
      int64_t e1 = e0 + kTileFloats;
      if (e1 > prm.d) e1 = prm.d;
      for (int b0 = 0; b0 < r_g; b0 += prm.row_batch, ++it) {
        const int stage = it % prm.stages;
        const uint32_t phase = (it / prm.stages) & 1;
        if (it >= (uint32_t)prm.stages) pipe::mbar_wait(&empty_bar[stage], phase ^ 1, abort_flag, prm.status + 1);
        const int nb = min(prm.row_batch, r_g - b0);
        if (lane == 0) {
          tile_of[stage] = tile;
          b0_of[stage] = b0;
        }
        if (lane < nb) {
          const int64_t first = (int64_t)(row0 + b0 + lane) * prm.d + e0;
          const int64_t last = first + (e1 - e0);
          const int64_t a0 = first & ~(kVec - 1);
          int64_t a1 = (last + kVec - 1) & ~(kVec - 1);
          const int64_t safe_end = prm.total_floats & ~(kVec - 1);
          if (a1 > safe_end) a1 = safe_end;
          T* slot = ring + stage * stage_floats + (size_t)lane * prm.slot_floats;
          const uint32_t bytes = a1 > a0 ? (uint32_t)((a1 - a0) * sizeof(T)) : 0u;
          for (int64_t e = (a1 > a0 ? a1 : a0); e < last; ++e) slot[e - a0] = prm.grads[e];   // fewer than 16 bytes
          if (bytes) {
            pipe::mbar_arrive_expect_tx(&full_bar[stage], bytes);
            if (prm.stream_hints) pipe::bulk_load_hint(slot, prm.grads + a0, bytes, &full_bar[stage], stream_policy);
            else pipe::bulk_load(slot, prm.grads + a0, bytes, &full_bar[stage]);
          } else {
            pipe::mbar_arrive(&full_bar[stage]);
          }
        } else {
          pipe::mbar_arrive(&full_bar[stage]);
        }
      }
      if (lane == 0) tile = (long long)atomicAdd(prm.tile_counter, 1ULL);
      tile = __shfl_sync(0xffffffffu, tile, 0);
    }
    {
      const int stage = it % prm.stages;
      const uint32_t phase = (it / prm.stages) & 1;
      if (it >= (uint32_t)prm.stages) pipe::mbar_wait(&empty_bar[stage], phase ^ 1, abort_flag, prm.status + 1);
      if (lane == 0) tile_of[stage] = -1;
      pipe::mbar_arrive(&full_bar[stage]);
    }
    if (lane == 0) {
      __threadfence();   // this CTA's last claim is ordered before its departure
      if (atomicAdd(prm.tile_counter + 1, 1ULL) == (unsigned long long)gridDim.x - 1) {
        prm.tile_counter[0] = 0ULL;   // every CTA has made its last claim
        prm.tile_counter[1] = 0ULL;
      }
    }
    if (*(volatile int*)abort_flag) pipe::drain_delay();
    return;
  }

  const int d_mod4 = (int)(prm.d & (kVec - 1));
  T acc[CPT][M];   // the group sum of this thread's chunks (in the element type)
  int row0 = 0, r_g = 0, valid = 0;
  int64_t e0 = 0, ct = 0;
  for (uint32_t it = 0;; ++it) {
    const int stage = it % prm.stages;
    const uint32_t phase = (it / prm.stages) & 1;
    pipe::mbar_wait(&full_bar[stage], phase, abort_flag, prm.status + 1);
    const long long tile = *(volatile long long*)&tile_of[stage];
    if (tile < 0 || *(volatile int*)abort_flag) break;
    const int b0 = *(volatile int*)&b0_of[stage];
    if (b0 == 0) {
      const int g = (int)(tile / prm.tiles_per_group);
      ct = tile - (int64_t)g * prm.tiles_per_group;
      row0 = prm.group_start[g];
      r_g = prm.group_start[g + 1] - row0;
      e0 = ct * kTileFloats;
      valid = (int)((prm.d - e0) < kTileFloats ? (prm.d - e0) : kTileFloats);
#pragma unroll
      for (int i = 0; i < CPT; ++i)
#pragma unroll
        for (int l = 0; l < M; ++l) acc[i][l] = (T)0;
    }
    const bool full_tile = valid == kTileFloats;
    const int nb = min(prm.row_batch, r_g - b0);
    const T* slot = ring + stage * stage_floats + tid * M;
    int shift = (int)(((((row0 + b0) & (kVec - 1)) * d_mod4) + (e0 & (kVec - 1))) & (kVec - 1));   // (row * d + e0) mod (elements per 16 bytes)
    if (full_tile) {
      for (int j = 0; j < nb; ++j) {
        const T* src = slot + shift;
#pragma unroll
        for (int i = 0; i < CPT; ++i)
#pragma unroll
          for (int l = 0; l < M; ++l) acc[i][l] += src[i * kEncConsumers * M + l];
        slot += prm.slot_floats;
        shift = (int)((shift + d_mod4) & (kVec - 1));
      }
    } else {
      for (int j = 0; j < nb; ++j) {
        const T* src = slot + shift;
#pragma unroll
        for (int i = 0; i < CPT; ++i)
#pragma unroll
          for (int l = 0; l < M; ++l)
            if ((tid + i * kEncConsumers) * M + l < valid) acc[i][l] += src[i * kEncConsumers * M + l];
        slot += prm.slot_floats;
        shift = (int)((shift + d_mod4) & (kVec - 1));
      }
    }
    __syncwarp();
    if ((tid & 31) == 0) pipe::mbar_arrive(&empty_bar[stage]);
    if (b0 + prm.row_batch < r_g) continue;

    // last batch of the tile: one Horner evaluation per node of the group, coalesced stores
    const int64_t c0 = ct * kTileChunks;
    T* out = prm.coded + (int64_t)row0 * prm.d_c + c0 + tid;
    bool ok[CPT];
#pragma unroll
    for (int i = 0; i < CPT; ++i) ok[i] = c0 + tid + i * kEncConsumers < prm.d_c;
    Acc c[CPT][M];   // the polynomial's coefficients in the precision of the evaluation
#pragma unroll
    for (int i = 0; i < CPT; ++i)
#pragma unroll
      for (int l = 0; l < M; ++l) c[i][l] = (Acc)acc[i][l];
    for (int k = 0; k < r_g; ++k) {
      const Acc wk = w_s[row0 + k];
#pragma unroll
      for (int i = 0; i < CPT; ++i) {
        Acc z = c[i][M - 1];
#pragma unroll
        for (int l = M - 2; l >= 0; --l) z = acc_fma<Acc>(z, wk, c[i][l]);
        if (ok[i]) {
          if (prm.stream_hints) __stcs(out + i * kEncConsumers, (T)z);
          else out[i * kEncConsumers] = (T)z;
        }
      }
      out += prm.d_c;
    }
  }
}

static size_t encode_smem_bytes(int m, int cpt, int row_batch, int stages, int slot_floats) {
  size_t tile_floats = (size_t)kEncConsumers * cpt * m;
  return 256 + 2 * SOLON_MAX_GROUP * sizeof(double) + 2 * ((tile_floats + 3) & ~(size_t)3) * sizeof(float) +
         (size_t)stages * row_batch * slot_floats * sizeof(float);
}

template <int M>
static int launch_encode_generic(solon_plan* plan, EncodeParams& prm) {
  // tile: about 1024..2048 floats per row for small m, one chunk per thread otherwise
  int cpt = 1;
  while (cpt < 8 && kEncConsumers * cpt * plan->m < 1024) cpt *= 2;
  prm.chunks_per_thread = cpt;
  int tile_floats = kEncConsumers * cpt * plan->m;
  prm.slot_floats = ((tile_floats + 3) / 4) * 4 + 8;
  size_t slot_bytes = (size_t)prm.slot_floats * 4;
  int row_batch = (int)((size_t)24 * 1024 / slot_bytes);
  if (row_batch < 1) row_batch = 1;
  if (row_batch > kEncMaxBatch) row_batch = kEncMaxBatch;
  if (row_batch > plan->max_group) row_batch = plan->max_group;
  {
    int nb = (plan->max_group + row_batch - 1) / row_batch;   // batches that divide the group evenly
    row_batch = (plan->max_group + nb - 1) / nb;
  }
  prm.row_batch = row_batch;
  const size_t budget = 200 * 1024;
  int stages = 4;
  while (stages > 2 && encode_smem_bytes(plan->m, cpt, row_batch, stages, prm.slot_floats) > budget) --stages;
  while (prm.row_batch > 1 && encode_smem_bytes(plan->m, cpt, prm.row_batch, stages, prm.slot_floats) > budget) --prm.row_batch;
  if (encode_smem_bytes(plan->m, cpt, prm.row_batch, stages, prm.slot_floats) > budget) return SOLON_ERR_INVALID_ARG;
  prm.stages = stages;
  size_t smem = encode_smem_bytes(plan->m, cpt, prm.row_batch, stages, prm.slot_floats);
  prm.tiles_per_group = (plan->d_c + (int64_t)kEncConsumers * cpt - 1) / ((int64_t)kEncConsumers * cpt);
  int64_t total_tiles = prm.tiles_per_group * plan->q;
  int per_sm = (int)((size_t)220 * 1024 / (smem + 1024));
  if (per_sm > 2) per_sm = 2;
  if (per_sm < 1) per_sm = 1;
  int64_t resident = (int64_t)plan->num_sms * per_sm;
  int grid = (int)(total_tiles < resident ? total_tiles : resident);
  SOLON_CUDA_TRY(cudaFuncSetAttribute(encode_kernel<M>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  encode_kernel<M><<<grid, kEncThreads, smem, plan->stream>>>(prm);
  SOLON_CUDA_TRY(cudaGetLastError());
  return SOLON_OK;
}

template <int M, int CPT, typename Acc, int kMinBlocks, typename T>
static int launch_encode_direct(solon_plan* plan, EncodeParamsT<T>& prm) {
  constexpr int kTileFloats = kEncConsumers * CPT * M;
  constexpr int kVec = (int)Vec16<T>::n;
  prm.chunks_per_thread = CPT;
  prm.slot_floats = ((kTileFloats + kVec - 1) / kVec) * kVec + 2 * kVec;   // elements: room for the alignment shift and the rounded-up end
  const size_t slot_bytes = (size_t)prm.slot_floats * sizeof(T);
  const size_t fixed = 256 + (((size_t)plan->P * sizeof(Acc) + 15) & ~(size_t)15);
  const size_t per_cta = (size_t)227 * 1024 / kMinBlocks - 1024;      // shared memory one CTA may take
  // rows per stage: about 20 KB per stage, an even split of the largest group
  int row_batch = (int)((size_t)20 * 1024 / slot_bytes);
  if (row_batch < 1) row_batch = 1;
  if (row_batch > kEncMaxBatch) row_batch = kEncMaxBatch;
  if (row_batch > plan->max_group) row_batch = plan->max_group;
  {
    int nb = (plan->max_group + row_batch - 1) / row_batch;
    row_batch = (plan->max_group + nb - 1) / nb;
  }
  int stages = 4;
  while (stages > 2 && fixed + (size_t)stages * row_batch * slot_bytes > per_cta) --stages;
  while (row_batch > 1 && fixed + (size_t)stages * row_batch * slot_bytes > per_cta) --row_batch;
  const size_t smem = fixed + (size_t)stages * row_batch * slot_bytes;
  if (smem > (size_t)226 * 1024) return SOLON_ERR_INVALID_ARG;
  prm.row_batch = row_batch;
  prm.stages = stages;
  prm.tiles_per_group = (plan->d_c + (int64_t)kEncConsumers * CPT - 1) / ((int64_t)kEncConsumers * CPT);
  const int64_t total_tiles = prm.tiles_per_group * plan->q;
  int per_sm = (int)((size_t)227 * 1024 / (smem + 1024));
  if (per_sm > kMinBlocks) per_sm = kMinBlocks;
  if (per_sm < 1) per_sm = 1;
  const int64_t resident = (int64_t)plan->num_sms * per_sm;
  const int grid = (int)(total_tiles < resident ? total_tiles : resident);
  auto kernel = encode_direct_kernel<M, CPT, Acc, kMinBlocks, T>;
  SOLON_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  kernel<<<grid, kEncThreads, smem, plan->stream>>>(prm);
  SOLON_CUDA_TRY(cudaGetLastError());
  return SOLON_OK;
}

template <typename T>
static void fill_encode_params(solon_plan* plan, const T* grads, T* coded, EncodeParamsT<T>* prm) {
  prm->grads = grads;
  prm->coded = coded;
  prm->group_start = plan->d_group_start;
  prm->w = plan->d_w;
  prm->q = plan->q;
  prm->m = plan->m;
  prm->P = plan->P;
  prm->d = plan->d;
  prm->d_c = plan->d_c;
  prm->total_floats = (int64_t)plan->P * plan->d;
  prm->status = plan->d_status;
  prm->tile_counter = plan->d_tile_counter + 1;
  prm->stream_hints = plan->stream_hints;
}

int launch_encode(solon_plan* plan, const float* grads, float* coded) {
  EncodeParams prm;
  fill_encode_params(plan, grads, coded, &prm);
  plan->launches += 1;
  switch (plan->m) {
    case 1: return launch_encode_direct<1, 4, float, 3>(plan, prm);
    case 2:   // small groups: wider tiles, or the per-tile work (claim, group lookup) shows; large groups: more tiles to hand out
      return plan->max_group <= 6 ? launch_encode_direct<2, 4, float, 3>(plan, prm) : launch_encode_direct<2, 2, float, 3>(plan, prm);
    case 3: return launch_encode_direct<3, 2, float, 3>(plan, prm);
    case 4: return launch_encode_direct<4, 1, float, 3>(plan, prm);
    case 5: return launch_encode_direct<5, 1, float, 3>(plan, prm);
    case 6: return launch_encode_direct<6, 1, float, 3>(plan, prm);
    case 8: return launch_encode_direct<8, 1, double, 3>(plan, prm);
    case 10: return launch_encode_direct<10, 1, double, 3>(plan, prm);
    default: return launch_encode_generic<0>(plan, prm);
  }
}

// float64 gradients (the paper's wire format, Table 2): group sums and polynomial evaluation in float64 throughout.
// Compression ratios with a kernel of their own only (solon_float64_m_supported).
int launch_encode_f64(solon_plan* plan, const double* grads, double* coded) {
  EncodeParamsT<double> prm;
  fill_encode_params(plan, grads, coded, &prm);
  plan->launches += 1;
  switch (plan->m) {
    case 1: return launch_encode_direct<1, 2, double, 3>(plan, prm);
    case 2: return launch_encode_direct<2, 2, double, 3>(plan, prm);
    case 3: return launch_encode_direct<3, 1, double, 3>(plan, prm);
    case 4: return launch_encode_direct<4, 1, double, 3>(plan, prm);
    case 5: return launch_encode_direct<5, 1, double, 3>(plan, prm);
    case 6: return launch_encode_direct<6, 1, double, 3>(plan, prm);
    case 8: return launch_encode_direct<8, 1, double, 2>(plan, prm);
    case 10: return launch_encode_direct<10, 1, double, 2>(plan, prm);
    case 12: return launch_encode_direct<12, 1, double, 2>(plan, prm);
    case 14: return launch_encode_direct<14, 1, double, 2>(plan, prm);
    default: return SOLON_ERR_INVALID_ARG;
  }
}

}  // namespace solon

extern "C" int solon_encode(solon_plan* plan, const float* partition_grads, float* coded) {
  if (!plan || !partition_grads || !coded || plan->dtype != SOLON_F32) return SOLON_ERR_INVALID_ARG;
  if (((uintptr_t)partition_grads & 15) || ((uintptr_t)coded & 3)) return SOLON_ERR_INVALID_ARG;
  solon::TraceRange range(plan->profiling != 0, "solon_encode");
  if (plan->profiling) {
    SOLON_CUDA_TRY(cudaEventRecord(plan->ev[0], plan->stream));
    plan->ev_valid[0] = 1;
  }
  int rc = solon::launch_encode(plan, partition_grads, coded);
  if (rc == SOLON_OK && plan->profiling) {
    SOLON_CUDA_TRY(cudaEventRecord(plan->ev[1], plan->stream));
    plan->ev_valid[1] = 1;
  }
  return rc;
}

extern "C" int solon_encode_f64(solon_plan* plan, const double* partition_grads, double* coded) {
  if (!plan || !partition_grads || !coded || plan->dtype != SOLON_F64) return SOLON_ERR_INVALID_ARG;
  if (((uintptr_t)partition_grads & 15) || ((uintptr_t)coded & 7)) return SOLON_ERR_INVALID_ARG;
  solon::TraceRange range(plan->profiling != 0, "solon_encode");
  if (plan->profiling) {
    SOLON_CUDA_TRY(cudaEventRecord(plan->ev[0], plan->stream));
    plan->ev_valid[0] = 1;
  }
  int rc = solon::launch_encode_f64(plan, partition_grads, coded);
  if (rc == SOLON_OK && plan->profiling) {
    SOLON_CUDA_TRY(cudaEventRecord(plan->ev[1], plan->stream));
    plan->ev_valid[1] = 1;
  }
  return rc;
}
