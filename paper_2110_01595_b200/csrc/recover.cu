// Recovery kernel: the block decoder psi of Section 3.4 applied to every chunk, fused with the final sum
// of Algorithm 1:  agg[p m + l] = sum_g sum_{j in rows_g} coeff_g[j][l] * R[rows_g[j]][p],  truncated to d.
//
// One pass over the trusted rows the locator selected (m per group when m <= 6, else all trusted rows).
// Each thread owns a few chunks, loads one float per row and chunk (coalesced along the chunk axis),
// accumulates the m outputs of each chunk in registers (float32 for m <= 6, where the weights are small;
// float64 above, where they reach 10^3 and cancel), and every warp writes its run of chunks
// back through its own shared-memory buffer as contiguous 128-bit stores.  The rows and weights come from device memory written by
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
template <typename Acc>
__device__ __forceinline__ void load_tables(const RecoverParams& prm, Acc* coeff_s, int* rows_s, int* start_s,
                                            int* n_rec_s) {
  for (int i = threadIdx.x; i < prm.P * prm.m; i += blockDim.x) coeff_s[i] = (Acc)prm.coeff[i];
  for (int i = threadIdx.x; i < prm.P; i += blockDim.x) rows_s[i] = prm.rec_rows[i];
  for (int i = threadIdx.x; i <= prm.q; i += blockDim.x) start_s[i] = prm.group_start[i];
  for (int i = threadIdx.x; i < prm.q; i += blockDim.x) n_rec_s[i] = prm.n_rec[i];
  __syncthreads();
}

template <int M, int CPT, typename Acc>
__global__ void __launch_bounds__(kRecThreads) recover_kernel(RecoverParams prm) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  constexpr int kWarpChunks = 32 * CPT;                      // chunks one warp handles per step
  constexpr int kWarps = kRecThreads / 32;
  float* out_all = reinterpret_cast<float*>(smem_raw);       // per warp: kWarpChunks x M
  Acc* coeff_s = reinterpret_cast<Acc*>(smem_raw + (size_t)kWarps * kWarpChunks * M * sizeof(float));
  int* rows_s = reinterpret_cast<int*>(smem_raw + (size_t)kWarps * kWarpChunks * M * sizeof(float) +
                                       (size_t)prm.P * M * sizeof(double));
  int* start_s = rows_s + prm.P;
  int* n_rec_s = start_s + prm.q + 1;
  load_tables(prm, coeff_s, rows_s, start_s, n_rec_s);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float* out_s = out_all + (size_t)warp * kWarpChunks * M;

  // Warps run independently of each other (no CTA barrier below): while one waits for its loads another
  // does arithmetic or stores.
  const int64_t stride = (int64_t)gridDim.x * kWarps * kWarpChunks;
  for (int64_t c0 = ((int64_t)blockIdx.x * kWarps + warp) * kWarpChunks; c0 < prm.d_c; c0 += stride) {
    Acc acc[CPT][M];
#pragma unroll
    for (int i = 0; i < CPT; ++i)
#pragma unroll
      for (int l = 0; l < M; ++l) acc[i][l] = (Acc)0;
    bool ok[CPT];
#pragma unroll
    for (int i = 0; i < CPT; ++i) ok[i] = c0 + lane + i * 32 < prm.d_c;

    for (int g = 0; g < prm.q; ++g) {
      const int base = start_s[g], n = n_rec_s[g];
      // rows in blocks of kRowBlock: all loads of a block are issued before its arithmetic
      for (int j0 = 0; j0 < n; j0 += kRowBlock) {
        float v[kRowBlock][CPT];
#pragma unroll
        for (int jj = 0; jj < kRowBlock; ++jj) {
          const int j = j0 + jj < n ? j0 + jj : n - 1;
          const float* row = prm.R + (int64_t)rows_s[base + j] * prm.d_c + c0 + lane;
#pragma unroll
          for (int i = 0; i < CPT; ++i) v[jj][i] = ok[i] ? __ldcs(row + i * 32) : 0.f;
        }
#pragma unroll
        for (int jj = 0; jj < kRowBlock; ++jj) {
          if (j0 + jj < n) {
            const Acc* cj = coeff_s + (size_t)(base + j0 + jj) * M;
            Acc dv[CPT];
#pragma unroll
            for (int i = 0; i < CPT; ++i) dv[i] = (Acc)v[jj][i];
#pragma unroll
            for (int l = 0; l < M; ++l) {
              const Acc c = cj[l];
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
      for (int l = 0; l < M; ++l) out_s[(size_t)(lane + i * 32) * M + l] = (float)acc[i][l];
    __syncwarp();
    // contiguous write-back: floats [c0 M, min((c0 + kWarpChunks) M, d)); c0 M is a multiple of 4
    const int64_t o0 = c0 * M;
    int64_t o1 = o0 + (int64_t)kWarpChunks * M;
    if (o1 > prm.d) o1 = prm.d;
    const int count = (int)(o1 - o0);
    const int vec = count / 4;
    float4* dst4 = reinterpret_cast<float4*>(prm.agg + o0);
    const float4* src4 = reinterpret_cast<const float4*>(out_s);
    for (int i = lane; i < vec; i += 32) dst4[i] = src4[i];
    for (int i = vec * 4 + lane; i < count; i += 32) prm.agg[o0 + i] = out_s[i];
    __syncwarp();
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

template <int M, int CPT, typename Acc>
static int launch_recover_m(solon_plan* plan, RecoverParams& prm) {
  size_t smem = (size_t)kRecThreads * CPT * M * sizeof(float) + (size_t)plan->P * M * sizeof(double) +
                (size_t)(plan->P + 2 * plan->q + 2) * sizeof(int);
  if (smem > 200 * 1024) return SOLON_ERR_INVALID_ARG;
  SOLON_CUDA_TRY(cudaFuncSetAttribute(recover_kernel<M, CPT, Acc>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  static_assert((32 * CPT) % 4 == 0, "warp tiles must start on a 16-byte boundary of the output");
  int64_t tiles = (plan->d_c + (int64_t)kRecThreads * CPT - 1) / ((int64_t)kRecThreads * CPT);
  int per_sm = 1;
  SOLON_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, recover_kernel<M, CPT, Acc>, kRecThreads, smem));
  if (per_sm < 1) per_sm = 1;
  int64_t cap = (int64_t)plan->num_sms * per_sm;
  int grid = (int)(tiles < cap ? tiles : cap);
  recover_kernel<M, CPT, Acc><<<grid, kRecThreads, smem, plan->stream>>>(prm);
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
    case 1: return launch_recover_m<1, 4, float>(plan, prm);
    case 2: return launch_recover_m<2, 4, float>(plan, prm);
    case 3: return launch_recover_m<3, 4, float>(plan, prm);
    case 4: return launch_recover_m<4, 4, float>(plan, prm);
    case 5: return launch_recover_m<5, 4, float>(plan, prm);
    case 6: return launch_recover_m<6, 2, float>(plan, prm);
    case 8: return launch_recover_m<8, 2, double>(plan, prm);
    case 10: return launch_recover_m<10, 2, double>(plan, prm);
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
