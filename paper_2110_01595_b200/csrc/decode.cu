// solon_decode (Algorithm 1: locate, then decode every group from its trusted nodes, then sum) and the
// host-buffer convenience call solon_step_host.
#include "solon_internal.h"

using namespace solon;

template <typename T>
static int decode_t(solon_plan* plan, const T* received, T* agg_grad, uint8_t* byz_mask) {
  if (!plan || !received || !agg_grad || !byz_mask) return SOLON_ERR_INVALID_ARG;
  if (plan->dtype != (sizeof(T) == 8 ? SOLON_F64 : SOLON_F32)) return SOLON_ERR_INVALID_ARG;
  if (((uintptr_t)received & 15) || ((uintptr_t)agg_grad & 15)) return SOLON_ERR_INVALID_ARG;
  int rc;
  const bool prof = plan->profiling != 0;
  auto mark = [&](int i) -> int {
    if (!prof) return SOLON_OK;
    SOLON_CUDA_TRY(cudaEventRecord(plan->ev[i], plan->stream));
    plan->ev_valid[i] = 1;
    return SOLON_OK;
  };
  auto project = [&]() -> int {
    if constexpr (sizeof(T) == 8) return launch_project_f64(plan, received, nullptr, nullptr, agg_grad);
    else return launch_project(plan, received, nullptr, nullptr, agg_grad);
  };
  auto recover = [&]() -> int {
    if constexpr (sizeof(T) == 8) return launch_recover_f64(plan, received, agg_grad);
    else return launch_recover(plan, received, agg_grad);
  };
  TraceRange range(prof, "solon_decode");
  if ((rc = mark(2))) return rc;
  {
    TraceRange step(prof, "project");
    if (plan->s > 0 && (rc = project())) return rc;   // s = 0: nothing to locate
  }
  // from here on the projection kernel may have announced partial sums on the progress counters, which only the
  // recovery kernel puts back to zero: a failure before that kernel is enqueued clears them here instead
  auto fail = [&](int code) -> int {
    if (plan->s > 0) (void)cudaMemsetAsync(plan->d_proj_progress, 0, 2 * sizeof(unsigned long long), plan->stream);
    (void)cudaGetLastError();
    return code;
  };
  if ((rc = mark(3))) return fail(rc);
  {
    TraceRange step(prof, "locate");
    if ((rc = launch_locate(plan, byz_mask))) return fail(rc);
  }
  if ((rc = mark(4))) return fail(rc);
  {
    TraceRange step(prof, "recover");
    if ((rc = recover())) return fail(rc);
  }
  return mark(5);
}

extern "C" int solon_decode(solon_plan* plan, const float* received, float* agg_grad, uint8_t* byz_mask) {
  return decode_t<float>(plan, received, agg_grad, byz_mask);
}

extern "C" int solon_decode_f64(solon_plan* plan, const double* received, double* agg_grad, uint8_t* byz_mask) {
  return decode_t<double>(plan, received, agg_grad, byz_mask);
}

extern "C" int solon_decode_project(solon_plan* plan, const float* received, double* rho, double* nu) {
  if (!plan || !received || !rho || !nu || plan->dtype != SOLON_F32) return SOLON_ERR_INVALID_ARG;
  if (((uintptr_t)received & 15) || ((uintptr_t)rho & 7) || ((uintptr_t)nu & 7)) return SOLON_ERR_INVALID_ARG;
  if (plan->s == 0) return SOLON_OK;
  return launch_project(plan, received, rho, nu);
}

extern "C" int solon_decode_finish(solon_plan* plan, const double* rho, const double* nu, const float* received,
                                   float* agg_grad, uint8_t* byz_mask) {
  if (!plan || !rho || !nu || !received || !agg_grad || !byz_mask || plan->dtype != SOLON_F32) return SOLON_ERR_INVALID_ARG;
  if (((uintptr_t)received & 15) || ((uintptr_t)agg_grad & 15) || ((uintptr_t)rho & 7) || ((uintptr_t)nu & 7))
    return SOLON_ERR_INVALID_ARG;
  int rc;
  if ((rc = launch_locate(plan, byz_mask, rho, nu))) return rc;
  return launch_recover(plan, received, agg_grad);
}

// Row overwrite for device-resident simulations: one streaming copy for all rows.
template <typename T>
__global__ void __launch_bounds__(256) overwrite_rows_kernel(T* __restrict__ matrix, const T* __restrict__ rows,
                                                             const int* __restrict__ nodes, int P, int64_t d_c, int vec, int stream_hints) {
  constexpr int kVec = 16 / sizeof(T);     // elements per 16 bytes
  const int node = nodes[blockIdx.y];
  if (node < 0 || node >= P) return;
  T* dst = matrix + (int64_t)node * d_c;
  const T* src = rows + (int64_t)blockIdx.y * d_c;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  const int64_t t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (vec) {   // d_c a multiple of 16 bytes and both bases 16-byte aligned: every row starts on a 16-byte boundary
    const int64_t n4 = d_c / kVec;
    float4* d4 = reinterpret_cast<float4*>(dst);
    const float4* s4 = reinterpret_cast<const float4*>(src);
    int64_t i = t0;
    for (; i + 7 * stride < n4; i += 8 * stride) {     // eight loads in flight per thread
      float4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = __ldcs(s4 + i + u * stride);
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        if (stream_hints) __stcs(d4 + i + u * stride, v[u]);
        else d4[i + u * stride] = v[u];
      }
    }
    for (; i < n4; i += stride) {
      if (stream_hints) __stcs(d4 + i, __ldcs(s4 + i));
      else d4[i] = __ldcs(s4 + i);
    }
  } else {
    int64_t i = t0;
    for (; i + 7 * stride < d_c; i += 8 * stride) {
      T v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) v[u] = __ldcs(src + i + u * stride);
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        if (stream_hints) __stcs(dst + i + u * stride, v[u]);
        else dst[i + u * stride] = v[u];
      }
    }
    for (; i < d_c; i += stride) {
      if (stream_hints) __stcs(dst + i, __ldcs(src + i));
      else dst[i] = __ldcs(src + i);
    }
  }
}

// The same when rows do not start on 16-byte boundaries (d_c not a multiple of 16 bytes): 16-byte stores at the destination
// row's own boundaries, each taking its values from the two 16-byte words of the source row that hold them (the offset
// between the two rows' boundaries is the same along the whole row); the elements before the first and after the last
// whole word, and the first and last word themselves, go one by one.
template <typename T>
__global__ void __launch_bounds__(256) overwrite_rows_shifted_kernel(T* __restrict__ matrix, const T* __restrict__ rows,
                                                                     const int* __restrict__ nodes, int P, int64_t d_c, int stream_hints) {
  constexpr int kVec = 16 / sizeof(T);     // elements per 16 bytes
  union Word {
    float4 v;
    T e[kVec];
  };
  const int node = nodes[blockIdx.y];
  if (node < 0 || node >= P) return;
  T* dst = matrix + (int64_t)node * d_c;
  const T* src = rows + (int64_t)blockIdx.y * d_c;
  int64_t head = (int64_t)((kVec - (((uintptr_t)dst / sizeof(T)) & (kVec - 1))) & (kVec - 1));    // elements before dst's first boundary
  if (head > d_c) head = d_c;
  const int64_t n_words = (d_c - head) / kVec;
  const int64_t body_end = head + n_words * kVec;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  if (blockIdx.x == 0) {
    const int64_t first_end = n_words > 0 ? head + kVec : head;
    const int64_t last_begin = n_words > 1 ? body_end - kVec : body_end;
    for (int64_t i = threadIdx.x; i < first_end; i += blockDim.x) dst[i] = src[i];
    for (int64_t i = last_begin + threadIdx.x; i < d_c; i += blockDim.x) dst[i] = src[i];
  }
  if (n_words < 3) return;
  const T* s0 = src + head;                                                      // source of dst's first whole word
  const int delta = (int)(((uintptr_t)s0 / sizeof(T)) & (kVec - 1));           // its offset from a 16-byte boundary of its own
  const float4* sw = reinterpret_cast<const float4*>(s0 - delta);              // word i of dst comes from sw[i] and sw[i + 1]
  float4* dw = reinterpret_cast<float4*>(dst + head);
  // words 1 .. n_words - 2: both source words lie inside the row; four words (eight loads) in flight per thread
  for (int64_t i = 1 + (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_words - 1; i += 4 * stride) {
    Word a[4], b[4], o[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int64_t w = i + u * stride;
      if (w < n_words - 1) {
        a[u].v = __ldcs(sw + w);
        if (delta) b[u].v = __ldcs(sw + w + 1);
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int64_t w = i + u * stride;
      if (w < n_words - 1) {
#pragma unroll
        for (int k = 0; k < kVec; ++k) {
          T val = a[u].e[k];                                   // delta == 0
#pragma unroll
          for (int dlt = 1; dlt < kVec; ++dlt)
            if (delta == dlt) val = dlt + k < kVec ? a[u].e[(dlt + k) % kVec] : b[u].e[(dlt + k) % kVec];
          o[u].e[k] = val;
        }
        if (stream_hints) __stcs(dw + w, o[u].v);
        else dw[w] = o[u].v;
      }
    }
  }
}

template <typename T>
static int overwrite_rows_t(solon_plan* plan, T* matrix, int n_rows, const int* nodes, const T* rows) {
  if (!plan || n_rows < 0 || n_rows > plan->P) return SOLON_ERR_INVALID_ARG;
  if (plan->dtype != (sizeof(T) == 8 ? SOLON_F64 : SOLON_F32)) return SOLON_ERR_INVALID_ARG;
  if (n_rows == 0) return SOLON_OK;
  if (!matrix || !nodes || !rows) return SOLON_ERR_INVALID_ARG;
  constexpr int kVec = 16 / sizeof(T);
  const int vec = (plan->d_c % kVec == 0 && !((uintptr_t)matrix & 15) && !((uintptr_t)rows & 15)) ? 1 : 0;
  // one wave of CTAs (eight per SM) shared by the rows; every thread then has several batches of eight accesses
  const bool shifted = !vec && plan->d_c >= 64;      // rows off 16-byte boundaries: realign (element pointers are element-aligned)
  int64_t per_row = (plan->d_c / ((vec || shifted) ? kVec : 1) + 256 * 8 - 1) / (256 * 8);
  int64_t cap = ((int64_t)plan->num_sms * 8 + n_rows - 1) / n_rows;
  if (per_row > cap) per_row = cap;
  if (per_row < 1) per_row = 1;
  if (shifted)
    overwrite_rows_shifted_kernel<T><<<dim3((unsigned)per_row, (unsigned)n_rows), 256, 0, plan->stream>>>(matrix, rows, nodes, plan->P, plan->d_c,
                                                                                                         plan->stream_hints);
  else
    overwrite_rows_kernel<T><<<dim3((unsigned)per_row, (unsigned)n_rows), 256, 0, plan->stream>>>(matrix, rows, nodes, plan->P, plan->d_c, vec,
                                                                                                 plan->stream_hints);
  SOLON_CUDA_TRY(cudaGetLastError());
  plan->launches += 1;
  return SOLON_OK;
}

extern "C" int solon_overwrite_rows(solon_plan* plan, float* matrix, int n_rows, const int* nodes, const float* rows) {
  return overwrite_rows_t<float>(plan, matrix, n_rows, nodes, rows);
}

extern "C" int solon_overwrite_rows_f64(solon_plan* plan, double* matrix, int n_rows, const int* nodes, const double* rows) {
  return overwrite_rows_t<double>(plan, matrix, n_rows, nodes, rows);
}

template <typename T>
static int stage_alloc(T** ptr, size_t count) {
  if (*ptr) return SOLON_OK;
  cudaError_t err = cudaMalloc((void**)ptr, count * sizeof(T));
  if (err != cudaSuccess) {
    (void)cudaGetLastError();
    *ptr = nullptr;
    return err == cudaErrorMemoryAllocation ? SOLON_ERR_NOMEM : SOLON_ERR_CUDA;
  }
  return SOLON_OK;
}

template <typename T>
static int step_host_t(solon_plan* plan, const T* grads_host, int n_byz, const int* byz_nodes, const T* byz_rows_host, T* agg_host,
                       uint8_t* mask_host) {
  if (!plan || !grads_host || !agg_host || !mask_host || n_byz < 0) return SOLON_ERR_INVALID_ARG;
  if (plan->dtype != (sizeof(T) == 8 ? SOLON_F64 : SOLON_F32)) return SOLON_ERR_INVALID_ARG;
  if (n_byz > 0 && (!byz_nodes || !byz_rows_host)) return SOLON_ERR_INVALID_ARG;
  for (int i = 0; i < n_byz; ++i)
    if (byz_nodes[i] < 0 || byz_nodes[i] >= plan->P) return SOLON_ERR_INVALID_ARG;
  int rc;
  const size_t n_grad = (size_t)plan->P * plan->d, n_coded = (size_t)plan->P * plan->d_c;
  // the staging buffers are typed by the plan's element type (allocated in bytes)
  T** grads_dev = reinterpret_cast<T**>(&plan->d_stage_grads);
  T** coded_dev = reinterpret_cast<T**>(&plan->d_stage_coded);
  T** agg_dev = reinterpret_cast<T**>(&plan->d_stage_agg);
  if ((rc = stage_alloc(grads_dev, n_grad))) return rc;
  if ((rc = stage_alloc(coded_dev, n_coded))) return rc;
  if ((rc = stage_alloc(agg_dev, (size_t)plan->d))) return rc;
  if ((rc = stage_alloc(&plan->d_stage_mask, (size_t)plan->P))) return rc;
  cudaStream_t st = plan->stream;
  SOLON_CUDA_TRY(cudaMemcpyAsync(*grads_dev, grads_host, n_grad * sizeof(T), cudaMemcpyHostToDevice, st));
  if constexpr (sizeof(T) == 8) rc = solon_encode_f64(plan, *grads_dev, *coded_dev);
  else rc = solon_encode(plan, *grads_dev, *coded_dev);
  if (rc) return rc;
  for (int i = 0; i < n_byz; ++i) {
    SOLON_CUDA_TRY(cudaMemcpyAsync(*coded_dev + (size_t)byz_nodes[i] * plan->d_c, byz_rows_host + (size_t)i * plan->d_c,
                                   (size_t)plan->d_c * sizeof(T), cudaMemcpyHostToDevice, st));
  }
  if ((rc = decode_t<T>(plan, *coded_dev, *agg_dev, plan->d_stage_mask))) return rc;
  SOLON_CUDA_TRY(cudaMemcpyAsync(agg_host, *agg_dev, (size_t)plan->d * sizeof(T), cudaMemcpyDeviceToHost, st));
  SOLON_CUDA_TRY(cudaMemcpyAsync(mask_host, plan->d_stage_mask, (size_t)plan->P, cudaMemcpyDeviceToHost, st));
  return solon_decode_status(plan);
}

extern "C" int solon_step_host(solon_plan* plan, const float* grads_host, int n_byz, const int* byz_nodes,
                               const float* byz_rows_host, float* agg_host, uint8_t* mask_host) {
  return step_host_t<float>(plan, grads_host, n_byz, byz_nodes, byz_rows_host, agg_host, mask_host);
}

extern "C" int solon_step_host_f64(solon_plan* plan, const double* grads_host, int n_byz, const int* byz_nodes,
                                   const double* byz_rows_host, double* agg_host, uint8_t* mask_host) {
  return step_host_t<double>(plan, grads_host, n_byz, byz_nodes, byz_rows_host, agg_host, mask_host);
}
