// Detection projections (Section 3.4): rho[kappa][k] = f_kappa . R_k for the K random vectors f_kappa
// and all P received rows, plus the row energies nu[k] = ||R_k||^2 that scale the locator's tolerance.
//
// One pass over the P x d_c received matrix.  Every CTA owns one contiguous range of the chunk axis,
// walks it in tiles, keeps the tile of f in shared memory as float64 and lets each warp stream its own
// rows (two at a time) against it, so each received byte is read once and f is read once per CTA.
// Products are exact in float64 and accumulated in float64; nu is accumulated in float32 per lane and
// in float64 across lanes and tiles.  Per-CTA partial sums go to global memory and are added in a fixed
// order by the last CTAs to finish (atomic tickets, no waiting), so results are bit-reproducible.
#include <mutex>

#include "solon_internal.h"

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

template <int K>
__global__ void __launch_bounds__(kProjThreads, 4) project_kernel(const float* __restrict__ R, const float* __restrict__ f,
                                                               int64_t f_pitch, int P, int64_t d_c, int64_t range_len,
                                                               int tile_cols, double* __restrict__ partials,
                                                               double* __restrict__ rho_out, double* __restrict__ nu_out,
                                                               unsigned int* ticket, int final_reduce) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double* fs = reinterpret_cast<double*>(smem_raw);            // K x tile_cols
  double* sacc = fs + (size_t)K * tile_cols;                  // P x (K + 1)
  __shared__ unsigned int s_ticket;
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
  // Two-level, fixed-order reduction of the per-CTA partial sums with atomic tickets (nobody waits):
  // the last CTA of every bunch of kProjBunch adds that bunch, the last bunch adds the bunch sums.
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
  for (int i = tid; i < n_acc; i += kProjThreads) {
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
  for (int i = tid; i < n_acc; i += kProjThreads) {
    double acc = 0.0;
#pragma unroll 4
    for (unsigned int b = 0; b < n_bunches; ++b) acc += __ldcg(bunch_sums + (size_t)b * n_acc + i);
    if (i < K * P) rho_out[i] = acc;
    else nu_out[i - K * P] = acc;
  }
  if (tid == 0) *ticket = 0u;
}

template <int K>
static int launch_project_k(solon_plan* plan, const float* received, double* rho_out, double* nu_out, int final_reduce) {
  int tile_cols = K <= 2 ? 2048 : 1024;
  size_t smem = (size_t)K * tile_cols * sizeof(double) + (size_t)(K + 1) * plan->P * sizeof(double);
  if (smem > 200 * 1024) return SOLON_ERR_INVALID_ARG;
  SOLON_CUDA_TRY(cudaFuncSetAttribute(project_kernel<K>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  // one wave: as many CTAs as are resident at once (the partial-sum buffer holds plan->proj_grid of them)
  int per_sm = 1;
  SOLON_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, project_kernel<K>, kProjThreads, smem));
  int grid = plan->num_sms * (per_sm < 1 ? 1 : per_sm);
  if (grid > plan->proj_grid) grid = plan->proj_grid;
  // leave one slot per group free: the locator's CTAs (launched as dependents) then become resident while this
  // kernel streams and use the time to stage their tables and fetch their code
  if (plan->q <= plan->num_sms && grid >= 4 * plan->q) grid -= plan->q;
  int64_t range_len = (plan->d_c + grid - 1) / grid;
  range_len = (range_len + 3) / 4 * 4;
  if (range_len < tile_cols) tile_cols = (int)range_len;
  project_kernel<K><<<grid, kProjThreads, smem, plan->stream>>>(
      received, plan->d_f, plan->f_pitch, plan->P, plan->d_c, range_len, tile_cols, plan->d_partials, rho_out,
      nu_out, plan->d_proj_ticket, final_reduce);
  plan->proj_bunches = final_reduce ? 0 : (grid + kProjBunch - 1) / kProjBunch;
  plan->proj_bunch_sums = plan->d_partials + (size_t)grid * (K + 1) * plan->P;
  SOLON_CUDA_TRY(cudaGetLastError());
  return SOLON_OK;
}

int launch_project(solon_plan* plan, const float* received, double* rho_out, double* nu_out) {
  // no output buffers: the decode proper, whose locator kernel adds the last level of partial sums itself
  const int final_reduce = (rho_out || nu_out) ? 1 : 0;
  if (!rho_out) rho_out = plan->d_rho;
  if (!nu_out) nu_out = plan->d_nu;
  plan->launches += 1;
  switch (plan->K) {
    case 1: return launch_project_k<1>(plan, received, rho_out, nu_out, final_reduce);
    case 2: return launch_project_k<2>(plan, received, rho_out, nu_out, final_reduce);
    case 3: return launch_project_k<3>(plan, received, rho_out, nu_out, final_reduce);
    case 4: return launch_project_k<4>(plan, received, rho_out, nu_out, final_reduce);
    default: return SOLON_ERR_INVALID_ARG;
  }
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
