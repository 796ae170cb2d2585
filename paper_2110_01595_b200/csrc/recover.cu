// Recovery kernel: the block decoder psi of Section 3.4 applied to every chunk, fused with the final sum
// of Algorithm 1:  agg[p m + l] = sum_g sum_{j in rows_g} coeff_g[j][l] * R[rows_g[j]][p],  truncated to d.
//
// One pass over the trusted rows the locator selected (m per group when m <= 6, else all trusted rows).
// Each thread owns a few chunks, loads one float per row and chunk (coalesced along the chunk axis),
// accumulates the m outputs of each chunk in float64 registers, and the tile is written back through
// shared memory as contiguous 128-bit stores.  The rows and weights come from device memory written by
// the locator kernel, so no host round trip separates the two.
#include "solon_internal.h"

namespace solon {

constexpr int kRecThreads = 256;
constexpr int kRowBlock = 5;   // rows whose loads are in flight together

struct RecoverParams {
  const float* R;
  float* agg;
  int64_t d, d_c;
  int q, m, P;
  const int* group_start;
  const int* n_rec;      // q
  const int* rec_rows;   // P, group g's rows at [group_start[g], +n_rec[g])
  const double* coeff;   // P x m, same indexing
};

// Copy the locator's tables (group layout, rows per group, row indices, weights) into shared memory.
__device__ __forceinline__ void load_tables(const RecoverParams& prm, double* coeff_s, int* rows_s, int* start_s,
                                            int* n_rec_s) {
  for (int i = threadIdx.x; i < prm.P * prm.m; i += blockDim.x) coeff_s[i] = prm.coeff[i];
  for (int i = threadIdx.x; i < prm.P; i += blockDim.x) rows_s[i] = prm.rec_rows[i];
  for (int i = threadIdx.x; i <= prm.q; i += blockDim.x) start_s[i] = prm.group_start[i];
  for (int i = threadIdx.x; i < prm.q; i += blockDim.x) n_rec_s[i] = prm.n_rec[i];
  __syncthreads();
}

template <int M, int CPT>
__global__ void __launch_bounds__(kRecThreads) recover_kernel(RecoverParams prm) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  constexpr int kTileChunks = kRecThreads * CPT;
  float* out_s = reinterpret_cast<float*>(smem_raw);                                 // kTileChunks x M
  double* coeff_s = reinterpret_cast<double*>(smem_raw + (size_t)kTileChunks * M * sizeof(float));
  int* rows_s = reinterpret_cast<int*>(coeff_s + (size_t)prm.P * M);
  int* start_s = rows_s + prm.P;
  int* n_rec_s = start_s + prm.q + 1;
  load_tables(prm, coeff_s, rows_s, start_s, n_rec_s);
  const int tid = threadIdx.x;

  for (int64_t c0 = (int64_t)blockIdx.x * kTileChunks; c0 < prm.d_c; c0 += (int64_t)gridDim.x * kTileChunks) {
    double acc[CPT][M];
#pragma unroll
    for (int i = 0; i < CPT; ++i)
#pragma unroll
      for (int l = 0; l < M; ++l) acc[i][l] = 0.0;
    bool ok[CPT];
#pragma unroll
    for (int i = 0; i < CPT; ++i) ok[i] = c0 + tid + i * kRecThreads < prm.d_c;

    for (int g = 0; g < prm.q; ++g) {
      const int base = start_s[g], n = n_rec_s[g];
      // rows in blocks of kRowBlock: all loads of a block are issued before its arithmetic
      for (int j0 = 0; j0 < n; j0 += kRowBlock) {
        float v[kRowBlock][CPT];
#pragma unroll
        for (int jj = 0; jj < kRowBlock; ++jj) {
          const int j = j0 + jj < n ? j0 + jj : n - 1;
          const float* row = prm.R + (int64_t)rows_s[base + j] * prm.d_c + c0 + tid;
#pragma unroll
          for (int i = 0; i < CPT; ++i) v[jj][i] = ok[i] ? __ldcs(row + i * kRecThreads) : 0.f;
        }
#pragma unroll
        for (int jj = 0; jj < kRowBlock; ++jj) {
          if (j0 + jj < n) {
            const double* cj = coeff_s + (size_t)(base + j0 + jj) * M;
            double dv[CPT];
#pragma unroll
            for (int i = 0; i < CPT; ++i) dv[i] = (double)v[jj][i];
#pragma unroll
            for (int l = 0; l < M; ++l) {
              const double c = cj[l];
#pragma unroll
              for (int i = 0; i < CPT; ++i) acc[i][l] = fma(c, dv[i], acc[i][l]);
            }
          }
        }
      }
    }
#pragma unroll
    for (int i = 0; i < CPT; ++i)
#pragma unroll
      for (int l = 0; l < M; ++l) out_s[(size_t)(tid + i * kRecThreads) * M + l] = (float)acc[i][l];
    __syncthreads();
    // contiguous write-back of the tile: floats [c0 M, min((c0 + tile) M, d))
    const int64_t o0 = c0 * M;
    int64_t o1 = o0 + (int64_t)kTileChunks * M;
    if (o1 > prm.d) o1 = prm.d;
    const int count = (int)(o1 - o0);
    const int vec = count / 4;                       // o0 is a multiple of 4 (tile of 256 * CPT chunks)
    float4* dst4 = reinterpret_cast<float4*>(prm.agg + o0);
    const float4* src4 = reinterpret_cast<const float4*>(out_s);
    for (int i = tid; i < vec; i += kRecThreads) dst4[i] = src4[i];
    for (int i = vec * 4 + tid; i < count; i += kRecThreads) prm.agg[o0 + i] = out_s[i];
    __syncthreads();
  }
}

// Any m: one thread per output coordinate (slower; used for compression ratios without a specialisation).
__global__ void __launch_bounds__(kRecThreads) recover_generic_kernel(RecoverParams prm) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double* coeff_s = reinterpret_cast<double*>(smem_raw);
  int* rows_s = reinterpret_cast<int*>(coeff_s + (size_t)prm.P * prm.m);
  int* start_s = rows_s + prm.P;
  int* n_rec_s = start_s + prm.q + 1;
  load_tables(prm, coeff_s, rows_s, start_s, n_rec_s);
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

template <int M, int CPT>
static int launch_recover_m(solon_plan* plan, RecoverParams& prm) {
  size_t smem = (size_t)kRecThreads * CPT * M * sizeof(float) + (size_t)plan->P * M * sizeof(double) +
                (size_t)(plan->P + 2 * plan->q + 2) * sizeof(int);
  if (smem > 200 * 1024) return SOLON_ERR_INVALID_ARG;
  SOLON_CUDA_TRY(cudaFuncSetAttribute(recover_kernel<M, CPT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  int64_t tiles = (plan->d_c + (int64_t)kRecThreads * CPT - 1) / ((int64_t)kRecThreads * CPT);
  int per_sm = 1;
  SOLON_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, recover_kernel<M, CPT>, kRecThreads, smem));
  if (per_sm < 1) per_sm = 1;
  int64_t cap = (int64_t)plan->num_sms * per_sm;
  int grid = (int)(tiles < cap ? tiles : cap);
  recover_kernel<M, CPT><<<grid, kRecThreads, smem, plan->stream>>>(prm);
  SOLON_CUDA_TRY(cudaGetLastError());
  return SOLON_OK;
}

int launch_recover(solon_plan* plan, const float* received, float* agg) {
  RecoverParams prm;
  prm.R = received;
  prm.agg = agg;
  prm.d = plan->d;
  prm.d_c = plan->d_c;
  prm.q = plan->q;
  prm.m = plan->m;
  prm.P = plan->P;
  prm.group_start = plan->d_group_start;
  prm.n_rec = plan->d_n_rec;
  prm.rec_rows = plan->d_rec_rows;
  prm.coeff = plan->d_coeff;
  plan->launches += 1;
  switch (plan->m) {
    case 1: return launch_recover_m<1, 4>(plan, prm);
    case 2: return launch_recover_m<2, 4>(plan, prm);
    case 3: return launch_recover_m<3, 4>(plan, prm);
    case 4: return launch_recover_m<4, 4>(plan, prm);
    case 5: return launch_recover_m<5, 4>(plan, prm);
    case 6: return launch_recover_m<6, 2>(plan, prm);
    case 8: return launch_recover_m<8, 2>(plan, prm);
    case 10: return launch_recover_m<10, 2>(plan, prm);
    default: break;
  }
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
