// Least-squares partition gradients g_i = X_i^T (X_i w - y_i): two streaming passes over X, no tensor
// cores (both are matrix-vector products with one right-hand side, bound by HBM bandwidth).
//   pass 1  e[row] = X[row] . w - y[row]            one CTA per row of X, float64 accumulation
//   pass 2  g_i[c] = sum_{row in partition i} X[row][c] e[row]     one thread per column (four in the fast form), coalesced
// Rows that start on 16-byte boundaries take the fast forms (128-bit loads); any other layout the scalar ones.
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

// Fast forms of the two passes for rows that start on 16-byte boundaries (d a multiple of 4, X and w 16-byte
// aligned): 128-bit loads, several per thread in flight; products in float32 (one rounding each), sums in float64.

// 128-bit streaming load whose place in the instruction stream is fixed (volatile): a batch of these is issued
// back to back before the first use, whatever the register allocator would prefer.
__device__ __forceinline__ float4 load_stream_pinned(const float4* p) {
  float4 v;
  asm volatile("ld.global.cs.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
}

// e[row] = X[row] . w - y[row]: one CTA per row, each thread four 128-bit loads of X ahead.
__global__ void __launch_bounds__(kLsqThreads, 4) lsq_residual_vec_kernel(const float4* __restrict__ X4, const float* __restrict__ y,
                                                                      const float4* __restrict__ w4, int64_t d4, int64_t n_rows,
                                                                      float* __restrict__ resid) {
  __shared__ double warp_part[kLsqThreads / 32];
  for (int64_t row = blockIdx.x; row < n_rows; row += gridDim.x) {
    const float4* x = X4 + row * d4;
    double acc = 0.0;
    int64_t c = threadIdx.x;
    for (; c + 3 * kLsqThreads < d4; c += 4 * kLsqThreads) {
      float4 xv[4], wv[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) xv[u] = load_stream_pinned(x + c + u * kLsqThreads);
#pragma unroll
      for (int u = 0; u < 4; ++u) wv[u] = __ldg(w4 + c + u * kLsqThreads);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        acc += (double)(xv[u].x * wv[u].x);
        acc += (double)(xv[u].y * wv[u].y);
        acc += (double)(xv[u].z * wv[u].z);
        acc += (double)(xv[u].w * wv[u].w);
      }
    }
    for (; c < d4; c += kLsqThreads) {
      const float4 xv = __ldcs(x + c), wv = __ldg(w4 + c);
      acc += (double)(xv.x * wv.x);
      acc += (double)(xv.y * wv.y);
      acc += (double)(xv.z * wv.z);
      acc += (double)(xv.w * wv.w);
    }
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

// g_i[c..c+3] = sum_row X[row][c..c+3] e[row]: one thread per four columns, eight rows of 128-bit loads in flight.
__global__ void __launch_bounds__(kLsqThreads, 4) lsq_gradient_vec_kernel(const float4* __restrict__ X4, const float* __restrict__ resid,
                                                                      int64_t d4, int rows, float4* __restrict__ grads4) {
  extern __shared__ float e_s[];   // rows
  const int part = blockIdx.y;
  for (int i = threadIdx.x; i < rows; i += kLsqThreads) e_s[i] = resid[(int64_t)part * rows + i];
  __syncthreads();
  const float4* Xi = X4 + (int64_t)part * rows * d4;
  for (int64_t c = (int64_t)blockIdx.x * kLsqThreads + threadIdx.x; c < d4; c += (int64_t)gridDim.x * kLsqThreads) {
    double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
    int r = 0;
    for (; r + 8 <= rows; r += 8) {
      float4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = load_stream_pinned(Xi + (int64_t)(r + u) * d4 + c);
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const float e = e_s[r + u];
        a0 += (double)(v[u].x * e);
        a1 += (double)(v[u].y * e);
        a2 += (double)(v[u].z * e);
        a3 += (double)(v[u].w * e);
      }
    }
    for (; r < rows; ++r) {
      const float4 v = __ldcs(Xi + (int64_t)r * d4 + c);
      const float e = e_s[r];
      a0 += (double)(v.x * e);
      a1 += (double)(v.y * e);
      a2 += (double)(v.z * e);
      a3 += (double)(v.w * e);
    }
    grads4[(int64_t)part * d4 + c] = make_float4((float)a0, (float)a1, (float)a2, (float)a3);
  }
}

// Finer-grained form of the gradient pass: a work item is (partition, block of 64 x four columns); the CTA's four
// groups of 64 threads each take a quarter of the partition's rows for those columns and their sums are added up
// through shared memory.  About ten items per CTA instead of two or three, so no CTA is left with half the kernel
// to do alone.  All residuals (P * rows floats) are staged in shared memory once.
constexpr int kLsqItemCols4 = 64;
__global__ void __launch_bounds__(kLsqThreads, 4) lsq_gradient_items_kernel(const float4* __restrict__ X4, const float* __restrict__ resid,
                                                                        int64_t d4, int rows, int P, float4* __restrict__ grads4) {
  extern __shared__ __align__(16) unsigned char lsq_smem[];
  double* part_s = reinterpret_cast<double*>(lsq_smem);                    // 3 x 64 x 4 partial sums (quarters 1..3)
  float* e_s = reinterpret_cast<float*>(part_s + 3 * kLsqItemCols4 * 4);   // P x rows residuals
  for (int i = threadIdx.x; i < P * rows; i += kLsqThreads) e_s[i] = resid[i];
  __syncthreads();
  const int cq = threadIdx.x & (kLsqItemCols4 - 1), rq = threadIdx.x / kLsqItemCols4;
  const int quarter = (rows + 3) / 4;
  const int r_begin = rq * quarter < rows ? rq * quarter : rows;
  const int r_end = r_begin + quarter < rows ? r_begin + quarter : rows;
  const int64_t blocks = (d4 + kLsqItemCols4 - 1) / kLsqItemCols4;
  const int64_t items = blocks * P;
  for (int64_t item = blockIdx.x; item < items; item += gridDim.x) {
    const int part = (int)(item / blocks);
    const int64_t c = (item - (int64_t)part * blocks) * kLsqItemCols4 + cq;
    const float4* Xi = X4 + (int64_t)part * rows * d4;
    const float* e = e_s + (size_t)part * rows;
    double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
    if (c < d4) {
      int r = r_begin;
      for (; r + 8 <= r_end; r += 8) {
        float4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = load_stream_pinned(Xi + (int64_t)(r + u) * d4 + c);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const float ev = e[r + u];
          a0 += (double)(v[u].x * ev);
          a1 += (double)(v[u].y * ev);
          a2 += (double)(v[u].z * ev);
          a3 += (double)(v[u].w * ev);
        }
      }
      for (; r < r_end; ++r) {
        const float4 v = __ldcs(Xi + (int64_t)r * d4 + c);
        const float ev = e[r];
        a0 += (double)(v.x * ev);
        a1 += (double)(v.y * ev);
        a2 += (double)(v.z * ev);
        a3 += (double)(v.w * ev);
      }
    }
    if (rq > 0) {
      double* dst = part_s + ((size_t)(rq - 1) * kLsqItemCols4 + cq) * 4;
      dst[0] = a0; dst[1] = a1; dst[2] = a2; dst[3] = a3;
    }
    __syncthreads();
    if (rq == 0 && c < d4) {
#pragma unroll
      for (int o = 0; o < 3; ++o) {      // quarters in row order: the sum does not depend on which CTA ran the item
        const double* src = part_s + ((size_t)o * kLsqItemCols4 + cq) * 4;
        a0 += src[0]; a1 += src[1]; a2 += src[2]; a3 += src[3];
      }
      grads4[(int64_t)part * d4 + c] = make_float4((float)a0, (float)a1, (float)a2, (float)a3);
    }
    __syncthreads();
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
  size_t smem = (size_t)plan->lsq_rows * sizeof(float);
  if (smem > 48 * 1024) return SOLON_ERR_INVALID_ARG;
  const bool vec = (plan->d & 3) == 0 && (((uintptr_t)X | (uintptr_t)w | (uintptr_t)grads) & 15) == 0;
  if (vec) {
    const int64_t d4 = plan->d / 4;
    const int64_t resident = (int64_t)plan->num_sms * 4;     // four CTAs per SM (64 registers a thread)
    grid1 = (int)(n_rows < resident ? n_rows : resident);
    lsq_residual_vec_kernel<<<grid1, kLsqThreads, 0, plan->stream>>>(reinterpret_cast<const float4*>(X), y,
                                                                      reinterpret_cast<const float4*>(w), d4, n_rows, plan->d_resid);
    SOLON_CUDA_TRY(cudaGetLastError());
    const size_t smem_items = 3 * kLsqItemCols4 * 4 * sizeof(double) + (size_t)n_rows * sizeof(float);
    if (smem_items <= 40 * 1024) {
      const int64_t items = ((d4 + kLsqItemCols4 - 1) / kLsqItemCols4) * plan->P;
      const int grid2 = (int)(items < resident ? items : resident);
      lsq_gradient_items_kernel<<<grid2, kLsqThreads, smem_items, plan->stream>>>(
          reinterpret_cast<const float4*>(X), plan->d_resid, d4, plan->lsq_rows, plan->P, reinterpret_cast<float4*>(grads));
    } else {
      int64_t col_blocks = (d4 + kLsqThreads - 1) / kLsqThreads;
      int64_t cap = (resident + plan->P - 1) / plan->P;
      dim3 grid2((unsigned)(col_blocks < cap ? col_blocks : cap), plan->P);
      lsq_gradient_vec_kernel<<<grid2, kLsqThreads, smem, plan->stream>>>(reinterpret_cast<const float4*>(X), plan->d_resid, d4,
                                                                          plan->lsq_rows, reinterpret_cast<float4*>(grads));
    }
    SOLON_CUDA_TRY(cudaGetLastError());
  } else {
    lsq_residual_kernel<<<grid1, kLsqThreads, 0, plan->stream>>>(X, y, w, plan->d, n_rows, plan->d_resid);
    SOLON_CUDA_TRY(cudaGetLastError());
    int64_t col_blocks = (plan->d + kLsqThreads - 1) / kLsqThreads;
    int64_t cap = ((int64_t)plan->num_sms * 8 + plan->P - 1) / plan->P;
    dim3 grid2((unsigned)(col_blocks < cap ? col_blocks : cap), plan->P);
    lsq_gradient_kernel<<<grid2, kLsqThreads, smem, plan->stream>>>(X, plan->d_resid, plan->d, plan->lsq_rows, grads);
    SOLON_CUDA_TRY(cudaGetLastError());
  }
  plan->launches += 2;
  return SOLON_OK;
}

}  // namespace solon

extern "C" int solon_lsq_grads(solon_plan* plan, const float* X, const float* y, const float* w, float* grads) {
  if (plan && plan->dtype != SOLON_F32) return SOLON_ERR_INVALID_ARG;
  if (!plan || !X || !y || !w || !grads) return SOLON_ERR_INVALID_ARG;
  return solon::launch_lsq(plan, X, y, w, grads);
}
