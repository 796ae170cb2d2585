// Least-squares partition gradients g_i = X_i^T (X_i w - y_i): two streaming passes over X, no tensor
// cores (both are matrix-vector products with one right-hand side, bound by HBM bandwidth).
//   pass 1  e[row] = X[row] . w - y[row]            one CTA per row of X, float64 accumulation
//   pass 2  g_i[c] = sum_{row in partition i} X[row][c] e[row]     one thread per column, coalesced
#include "solon_internal.h"

namespace solon {

constexpr int kLsqThreads = 256;

__global__ void __launch_bounds__(kLsqThreads) lsq_residual_kernel(const float* __restrict__ X, const float* __restrict__ y,
                                                                  const float* __restrict__ w, int64_t d, int64_t n_rows,
                                                                  float* __restrict__ resid) {
  __shared__ double warp_part[kLsqThreads / 32];
  for (int64_t row = blockIdx.x; row < n_rows; row += gridDim.x) {
    const float* x = X + row * d;
    double acc = 0.0;
    for (int64_t c = threadIdx.x; c < d; c += kLsqThreads) acc = fma((double)__ldcs(x + c), (double)__ldg(w + c), acc);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
      double total = 0.0;
      for (int i = 0; i < kLsqThreads / 32; ++i) total += warp_part[i];
      resid[row] = (float)(total - (double)y[row]);
    }
    __syncthreads();
  }
}

__global__ void __launch_bounds__(kLsqThreads) lsq_gradient_kernel(const float* __restrict__ X, const float* __restrict__ resid,
                                                                  int64_t d, int rows, float* __restrict__ grads) {
  extern __shared__ float e_s[];   // rows
  const int part = blockIdx.y;
  for (int i = threadIdx.x; i < rows; i += kLsqThreads) e_s[i] = resid[(int64_t)part * rows + i];
  __syncthreads();
  const float* Xi = X + (int64_t)part * rows * d;
  for (int64_t c = (int64_t)blockIdx.x * kLsqThreads + threadIdx.x; c < d; c += (int64_t)gridDim.x * kLsqThreads) {
    double acc = 0.0;
    int r = 0;
    for (; r + 8 <= rows; r += 8) {
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = __ldcs(Xi + (int64_t)(r + u) * d + c);
#pragma unroll
      for (int u = 0; u < 8; ++u) acc = fma((double)v[u], (double)e_s[r + u], acc);
    }
    for (; r < rows; ++r) acc = fma((double)__ldcs(Xi + (int64_t)r * d + c), (double)e_s[r], acc);
    grads[(int64_t)part * d + c] = (float)acc;
  }
}

int launch_lsq(solon_plan* plan, const float* X, const float* y, const float* w, float* grads) {
  const int64_t n_rows = (int64_t)plan->P * plan->lsq_rows;
  if (plan->resid_capacity < n_rows) {
    cudaFree(plan->d_resid);
    plan->d_resid = nullptr;
    plan->resid_capacity = 0;
    if (cudaMalloc((void**)&plan->d_resid, n_rows * sizeof(float)) != cudaSuccess) {
      (void)cudaGetLastError();
      return SOLON_ERR_NOMEM;
    }
    plan->resid_capacity = n_rows;
  }
  int grid1 = (int)(n_rows < (int64_t)plan->num_sms * 8 ? n_rows : (int64_t)plan->num_sms * 8);
  lsq_residual_kernel<<<grid1, kLsqThreads, 0, plan->stream>>>(X, y, w, plan->d, n_rows, plan->d_resid);
  SOLON_CUDA_TRY(cudaGetLastError());
  int64_t col_blocks = (plan->d + kLsqThreads - 1) / kLsqThreads;
  int64_t cap = ((int64_t)plan->num_sms * 8 + plan->P - 1) / plan->P;
  dim3 grid2((unsigned)(col_blocks < cap ? col_blocks : cap), plan->P);
  size_t smem = (size_t)plan->lsq_rows * sizeof(float);
  if (smem > 48 * 1024) return SOLON_ERR_INVALID_ARG;
  lsq_gradient_kernel<<<grid2, kLsqThreads, smem, plan->stream>>>(X, plan->d_resid, plan->d, plan->lsq_rows, grads);
  SOLON_CUDA_TRY(cudaGetLastError());
  plan->launches += 2;
  return SOLON_OK;
}

}  // namespace solon

extern "C" int solon_lsq_grads(solon_plan* plan, const float* X, const float* y, const float* w, float* grads) {
  if (!plan || !X || !y || !w || !grads) return SOLON_ERR_INVALID_ARG;
  return solon::launch_lsq(plan, X, y, w, grads);
}
