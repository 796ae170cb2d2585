// Plan construction (Section 3.4: allocation, node scalars, projection vectors), queries, and the
// plan-free host helpers of the C interface.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "locate_core.cuh"
#include <vector>

#include "projection_draw.cuh"
#include "solon_internal.h"

namespace solon {

void build_recovery_tabs(int n, int m, int s, const GroupTables& tb, int ld, std::vector<int>* count, std::vector<int>* rows,
                         std::vector<double>* coeff);   // locate.cu
int clean_recovery_table(int n, int m, int s, const GroupTables& tb, int* rows, double* coeff);   // locate.cu

int check_params(int P, int s, int m, int r, int64_t d) {
  if (P < 1 || s < 0 || m < 1 || d < 1 || r < 1) return SOLON_ERR_INVALID_ARG;
  if (P > SOLON_MAX_NODES || m > SOLON_MAX_M || s > SOLON_MAX_S) return SOLON_ERR_INVALID_ARG;
  if ((int64_t)2 * s + m > P) return SOLON_ERR_INFEASIBLE;   // corollary of Theorem 2
  if (r < 2 * s + m) return SOLON_ERR_INVALID_ARG;            // Theorem 2
  if (r > P) return SOLON_ERR_INVALID_ARG;
  return SOLON_OK;
}

// q = floor(P / r) groups of consecutive nodes; left-over nodes dealt to the first groups.
void group_layout(int P, int r, std::vector<int>* start) {
  int q = P / r;
  int extra = P - q * r;
  start->assign(q + 1, 0);
  for (int g = 0; g < q; ++g) {
    int size = r + extra / q + (g < extra % q ? 1 : 0);
    (*start)[g + 1] = (*start)[g] + size;
  }
}

// Chebyshev points of the first kind, n' = group size rounded up to even (so none is zero).
void node_scalars(const std::vector<int>& start, std::vector<double>* w) {
  const double pi = 3.14159265358979323846;
  int q = (int)start.size() - 1;
  w->assign(start[q], 0.0);
  for (int g = 0; g < q; ++g) {
    int size = start[g + 1] - start[g];
    int n_prime = size + (size & 1);
    for (int k = 1; k <= size; ++k) (*w)[start[g] + k - 1] = cos((2 * k - 1) * pi / (2.0 * n_prime));
  }
}

// ---- projection vectors: see projection_draw.cuh ------------------------------------------------------

__global__ void __launch_bounds__(256) fill_projection_kernel(DrawParams dp, int advance) {
  draw_projection_vectors(dp, advance, blockIdx.x, gridDim.x, threadIdx.x, blockDim.x);
}

DrawParams draw_params(const solon_plan* plan) {
  DrawParams dp;
  dp.f[0] = plan->d_f;
  dp.f[1] = plan->d_f2;
  dp.d_c = plan->d_c;
  dp.pitch = plan->f_pitch;
  dp.K = plan->K;
  dp.seed = plan->seed;
  dp.draw = plan->d_draw;
  return dp;
}

int launch_fill_projection(solon_plan* plan, int advance) {
  int64_t total = ((plan->d_c + 3) / 4) * plan->K;
  int threads = 256;
  int64_t want = (total + threads - 1) / threads;
  int blocks = (int)(want < (int64_t)plan->num_sms * 8 ? (want < 1 ? 1 : want) : (int64_t)plan->num_sms * 8);
  fill_projection_kernel<<<blocks, threads, 0, plan->stream>>>(draw_params(plan), advance);
  plan->launches += 1;
  plan->last_decode_advanced = 0;
  SOLON_CUDA_TRY(cudaGetLastError());
  return SOLON_OK;
}

template <typename T>
static int dev_alloc(T** ptr, size_t count) {
  *ptr = nullptr;
  if (count == 0) count = 1;
  cudaError_t err = cudaMalloc((void**)ptr, count * sizeof(T));
  if (err != cudaSuccess) {
    (void)cudaGetLastError();
    return err == cudaErrorMemoryAllocation ? SOLON_ERR_NOMEM : SOLON_ERR_CUDA;
  }
  return SOLON_OK;
}

static void free_device(solon_plan* p) {
  cudaFree(p->d_group_start); cudaFree(p->d_group_of); cudaFree(p->d_w); cudaFree(p->d_f); cudaFree(p->d_f2);
  cudaFree(p->d_qb); cudaFree(p->d_hm); cudaFree(p->d_qb_off); cudaFree(p->d_mt); cudaFree(p->d_tch);
  cudaFree(p->d_tab_count); cudaFree(p->d_tab_rows); cudaFree(p->d_tab_coeff); cudaFree(p->d_tab_off); cudaFree(p->d_tab_sets);
  cudaFree(p->d_opt);
  cudaFree(p->d_partials); cudaFree(p->d_rho); cudaFree(p->d_nu); cudaFree(p->d_proj_ticket);
  cudaFree(p->d_locate_ws);
  cudaFree(p->d_t_acc); cudaFree(p->d_n_rec); cudaFree(p->d_rec_rows); cudaFree(p->d_coeff); cudaFree(p->d_status); cudaFree(p->d_early); cudaFree(p->d_tile_counter); cudaFree(p->d_proj_progress); cudaFree(p->d_draw);
  cudaFree(p->d_resid);
  for (int i = 0; i < 6; ++i)
    if (p->ev[i]) cudaEventDestroy(p->ev[i]);
  cudaFree(p->d_stage_grads); cudaFree(p->d_stage_coded); cudaFree(p->d_stage_agg); cudaFree(p->d_stage_mask);
  (void)cudaGetLastError();
}

static int alloc_projection(solon_plan* p) {
  int rc;
  cudaFree(p->d_f); cudaFree(p->d_f2); cudaFree(p->d_partials); cudaFree(p->d_rho);
  cudaFree(p->d_locate_ws);
  (void)cudaGetLastError();
  p->d_f2 = nullptr;
  p->d_f = nullptr; p->d_partials = nullptr; p->d_rho = nullptr; p->d_locate_ws = nullptr;
  if ((rc = dev_alloc(&p->d_f, (size_t)p->K * p->f_pitch))) return rc;
  if ((rc = dev_alloc(&p->d_f2, (size_t)p->K * p->f_pitch))) return rc;
  // per-CTA partial sums of the two parts of every column range, then the per-bunch sums of part A and of the whole
  if ((rc = dev_alloc(&p->d_partials, 2 * (size_t)(p->proj_grid + p->proj_grid / 16 + 1) * (p->K + 1) * p->P))) return rc;
  if ((rc = dev_alloc(&p->d_rho, (size_t)p->K * p->P))) return rc;
  p->locate_ws_stride = locate_ws_doubles(p->max_group, p->m, p->K, p->s);
  if ((rc = dev_alloc(&p->d_locate_ws, (size_t)p->q * p->locate_ws_stride))) return rc;
  return SOLON_OK;
}

}  // namespace solon

using namespace solon;

extern "C" {

int solon_check_params(int P, int s, int m, int r, int64_t d) { return check_params(P, s, m, r, d); }

int solon_group_layout(int P, int r, int* starts, int starts_capacity, int* q_out) {
  if (!starts || !q_out || P < 1 || r < 1 || r > P) return SOLON_ERR_INVALID_ARG;
  std::vector<int> start;
  group_layout(P, r, &start);
  if ((int)start.size() > starts_capacity) return SOLON_ERR_INVALID_ARG;
  memcpy(starts, start.data(), start.size() * sizeof(int));
  *q_out = (int)start.size() - 1;
  return SOLON_OK;
}

int solon_node_scalars(int P, int r, double* w) {
  if (!w || P < 1 || r < 1 || r > P) return SOLON_ERR_INVALID_ARG;
  std::vector<int> start;
  std::vector<double> ws;
  group_layout(P, r, &start);
  node_scalars(start, &ws);
  memcpy(w, ws.data(), ws.size() * sizeof(double));
  return SOLON_OK;
}

const char* solon_strerror(int status) {
  switch (status) {
    case SOLON_OK: return "ok";
    case SOLON_ERR_INVALID_ARG: return "invalid argument";
    case SOLON_ERR_INFEASIBLE: return "infeasible: 2 s + m > P";
    case SOLON_ERR_CUDA: return "CUDA error or no CUDA device";
    case SOLON_ERR_UNDECODABLE: return "undecodable: more than s inconsistent nodes in a group";
    case SOLON_ERR_INTERNAL: return "internal error: bounded device wait expired";
    case SOLON_ERR_NOMEM: return "out of memory";
    default: return "unknown status";
  }
}

int solon_float64_m_supported(int m) { return (m >= 1 && m <= 6) || m == 8 || m == 10 || m == 12 || m == 14; }

int solon_plan_create(int P, int s, int m, int r, int64_t d, uint64_t seed, solon_plan** out) {
  return solon_plan_create_ex(P, s, m, r, d, seed, SOLON_F32, out);
}

int solon_plan_dtype(const solon_plan* plan) { return plan ? plan->dtype : SOLON_ERR_INVALID_ARG; }

int solon_plan_create_ex(int P, int s, int m, int r, int64_t d, uint64_t seed, int dtype, solon_plan** out) {
  if (!out) return SOLON_ERR_INVALID_ARG;
  *out = nullptr;
  if (dtype != SOLON_F32 && dtype != SOLON_F64) return SOLON_ERR_INVALID_ARG;
  int rc = check_params(P, s, m, r, d);
  if (rc) return rc;
  if (dtype == SOLON_F64 && !solon_float64_m_supported(m)) return SOLON_ERR_INVALID_ARG;
  std::vector<int> start;
  group_layout(P, r, &start);
  int q = (int)start.size() - 1;
  int max_group = 0;
  for (int g = 0; g < q; ++g) max_group = start[g + 1] - start[g] > max_group ? start[g + 1] - start[g] : max_group;
  if (max_group > SOLON_MAX_GROUP) return SOLON_ERR_INVALID_ARG;
  if ((int64_t)P * m > 16384) return SOLON_ERR_INVALID_ARG;   // recovery table must fit in shared memory

  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || n_dev < 1) {
    (void)cudaGetLastError();
    return SOLON_ERR_CUDA;
  }
  solon_plan* p = new (std::nothrow) solon_plan();
  if (!p) return SOLON_ERR_NOMEM;
  p->P = P; p->s = s; p->m = m; p->r = r; p->K = 2; p->d = d; p->d_c = (d + m - 1) / m;
  p->dtype = dtype;
  p->seed = seed; p->tau = dtype == SOLON_F64 ? 1e-10 : 1e-5; p->lsq_rows = 256; p->stream = 0; p->launches = 0;
  p->group_start = start; p->q = q; p->max_group = max_group;
  p->group_of.assign(P, 0);
  for (int g = 0; g < q; ++g)
    for (int k = start[g]; k < start[g + 1]; ++k) p->group_of[k] = g;
  node_scalars(start, &p->w);
  p->f_pitch = (p->d_c + 3) / 4 * 4;

  cudaDeviceProp prop;
  if (cudaGetDevice(&p->device) != cudaSuccess || cudaGetDeviceProperties(&prop, p->device) != cudaSuccess) {
    (void)cudaGetLastError();
    delete p;
    return SOLON_ERR_CUDA;
  }
  p->num_sms = prop.multiProcessorCount;
  p->proj_grid = p->num_sms * 4;
  p->early_locator = 1;
  if (const char* env = getenv("SOLON_EARLY_LOCATOR")) {     // for measurements, like SOLON_STREAM_HINTS below
    if (env[0] >= '0' && env[0] <= '2') p->early_locator = env[0] - '0';
  }
  p->fresh_f = 0;
  p->draw_parity = 0;
  p->stream_hints = keeps_l2_for_code(P, m, dtype == SOLON_F64 ? 2 * d : d) ? 1 : 0;
  if (const char* env = getenv("SOLON_STREAM_HINTS")) p->stream_hints = env[0] == '1' ? 1 : (env[0] == '0' ? 0 : p->stream_hints);

  rc = SOLON_OK;
  do {
    if ((rc = dev_alloc(&p->d_group_start, q + 1))) break;
    if ((rc = dev_alloc(&p->d_group_of, P))) break;
    if ((rc = dev_alloc(&p->d_w, P))) break;
    // locator tables, one set per group
    std::vector<int64_t> qb_off(q);
    int64_t qb_total = 0;
    for (int g = 0; g < q; ++g) {
      int n_g = start[g + 1] - start[g];
      qb_off[g] = qb_total;
      qb_total += (int64_t)n_g * n_g;
    }
    std::vector<double> h_qb(qb_total), h_hm(qb_total), h_mt((size_t)q * m * m), h_tch((size_t)P * (s + 1));
    for (int g = 0; g < q; ++g)
      build_group_tables(start[g + 1] - start[g], m, s, p->w.data() + start[g], h_qb.data() + qb_off[g],
                         h_hm.data() + qb_off[g], h_mt.data() + (size_t)g * m * m, h_tch.data() + (size_t)start[g] * (s + 1));
    if ((rc = dev_alloc(&p->d_qb, (size_t)qb_total))) break;
    if ((rc = dev_alloc(&p->d_hm, (size_t)qb_total))) break;
    if ((rc = dev_alloc(&p->d_qb_off, q))) break;
    if ((rc = dev_alloc(&p->d_mt, h_mt.size()))) break;
    if ((rc = dev_alloc(&p->d_tch, h_tch.size()))) break;
    if (cudaMemcpy(p->d_qb, h_qb.data(), h_qb.size() * sizeof(double), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(p->d_hm, h_hm.data(), h_hm.size() * sizeof(double), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(p->d_qb_off, qb_off.data(), q * sizeof(int64_t), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(p->d_mt, h_mt.data(), h_mt.size() * sizeof(double), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(p->d_tch, h_tch.data(), h_tch.size() * sizeof(double), cudaMemcpyHostToDevice) != cudaSuccess) {
      (void)cudaGetLastError();
      rc = SOLON_ERR_CUDA;
      break;
    }
    std::vector<int> rec_rows_init((size_t)P, 0), n_rec_init((size_t)q, 0);
    std::vector<double> coeff_init((size_t)P * m, 0.0);
    {
      // recovery tables for every set of at most s untrusted nodes, where those sets are few enough to tabulate
      std::vector<int> all_count, all_rows, count, rows;
      std::vector<double> all_coeff, coeff;
      std::vector<int64_t> tab_off(q);
      std::vector<int> tab_sets(q);
      p->tab_ld = m <= SOLON_SUBSET_MAX_M ? m : max_group;
      for (int g = 0; g < q; ++g) {
        const int n_g = start[g + 1] - start[g];
        GroupTables tb = {};
        tb.Qb = h_qb.data() + qb_off[g];
        tb.Hm = h_hm.data() + qb_off[g];
        tb.Mt = h_mt.data() + (size_t)g * m * m;
        tb.Tch = h_tch.data() + (size_t)start[g] * (s + 1);
        tb.w = p->w.data() + start[g];
        build_recovery_tabs(n_g, m, s, tb, p->tab_ld, &count, &rows, &coeff);
        tab_off[g] = (int64_t)all_count.size();
        tab_sets[g] = (int)count.size();
        all_count.insert(all_count.end(), count.begin(), count.end());
        all_rows.insert(all_rows.end(), rows.begin(), rows.end());
        all_coeff.insert(all_coeff.end(), coeff.begin(), coeff.end());
      }
      {
        // Optimistic decode: the projection pass may recover the aggregate from the rows the previous decode's recovery
        // read (subset form: m per group), i.e. from the locator's last recovery table; eligible when those rows all fit
        // in the projection kernel's first batch of rows, which then takes them first.  Before the first decode that
        // table is the one for no corrupt node.
        std::vector<int> opt_src;
        const int n_batches = (P + 31) / 32;
        const int batch_rows = (P + n_batches - 1) / n_batches;
        bool eligible = s > 0 && m <= SOLON_SUBSET_MAX_M && q * m <= batch_rows;
        std::vector<int> rows_g((size_t)max_group);
        std::vector<double> coeff_g((size_t)max_group * m);
        for (int g = 0; g < q && eligible; ++g) {
          const int n_g = start[g + 1] - start[g];
          GroupTables tb = {};
          tb.Qb = h_qb.data() + qb_off[g];
          tb.Hm = h_hm.data() + qb_off[g];
          tb.Mt = h_mt.data() + (size_t)g * m * m;
          tb.Tch = h_tch.data() + (size_t)start[g] * (s + 1);
          tb.w = p->w.data() + start[g];
          if (clean_recovery_table(n_g, m, s, tb, rows_g.data(), coeff_g.data()) != m) { eligible = false; break; }
          n_rec_init[(size_t)g] = m;
          for (int j = 0; j < m; ++j) {
            opt_src.push_back(start[g] + j);
            rec_rows_init[(size_t)start[g] + j] = start[g] + rows_g[(size_t)j];
            for (int l = 0; l < m; ++l) coeff_init[((size_t)start[g] + j) * m + l] = coeff_g[(size_t)j * m + l];
          }
        }
        if (!eligible) opt_src.clear();
        p->opt_rows = (int)opt_src.size();
        p->opt_src_host = opt_src;
        p->optimistic = 1;
        if (const char* env = getenv("SOLON_OPTIMISTIC")) {     // for measurements
          if (env[0] >= '0' && env[0] <= '2') p->optimistic = env[0] - '0';
        }
        if ((rc = dev_alloc(&p->d_opt, (size_t)8 + q))) break;
        std::vector<int> opt_init((size_t)8 + q, 0);
        opt_init[4] = p->optimistic;
        if (cudaMemcpy(p->d_opt, opt_init.data(), opt_init.size() * sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess) {
          (void)cudaGetLastError();
          rc = SOLON_ERR_CUDA;
          break;
        }
      }
      if ((rc = dev_alloc(&p->d_tab_count, all_count.size()))) break;
      if ((rc = dev_alloc(&p->d_tab_rows, all_rows.size()))) break;
      if ((rc = dev_alloc(&p->d_tab_coeff, all_coeff.size()))) break;
      if ((rc = dev_alloc(&p->d_tab_off, q))) break;
      if ((rc = dev_alloc(&p->d_tab_sets, q))) break;
      if ((!all_count.empty() && cudaMemcpy(p->d_tab_count, all_count.data(), all_count.size() * sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess) ||
          (!all_rows.empty() && cudaMemcpy(p->d_tab_rows, all_rows.data(), all_rows.size() * sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess) ||
          (!all_coeff.empty() && cudaMemcpy(p->d_tab_coeff, all_coeff.data(), all_coeff.size() * sizeof(double), cudaMemcpyHostToDevice) != cudaSuccess) ||
          cudaMemcpy(p->d_tab_off, tab_off.data(), q * sizeof(int64_t), cudaMemcpyHostToDevice) != cudaSuccess ||
          cudaMemcpy(p->d_tab_sets, tab_sets.data(), q * sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess) {
        (void)cudaGetLastError();
        rc = SOLON_ERR_CUDA;
        break;
      }
    }
    if ((rc = alloc_projection(p))) break;
    if ((rc = dev_alloc(&p->d_nu, P))) break;
    if ((rc = dev_alloc(&p->d_proj_ticket, 2 * ((size_t)p->proj_grid / 16 + 2)))) break;
    if ((rc = dev_alloc(&p->d_t_acc, q))) break;
    if ((rc = dev_alloc(&p->d_n_rec, q))) break;
    if ((rc = dev_alloc(&p->d_rec_rows, P))) break;
    if ((rc = dev_alloc(&p->d_coeff, (size_t)P * m))) break;
    if (cudaMemcpy(p->d_n_rec, n_rec_init.data(), (size_t)q * sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(p->d_rec_rows, rec_rows_init.data(), (size_t)P * sizeof(int), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(p->d_coeff, coeff_init.data(), coeff_init.size() * sizeof(double), cudaMemcpyHostToDevice) != cudaSuccess) {
      (void)cudaGetLastError();
      rc = SOLON_ERR_CUDA;
      break;
    }
    if ((rc = dev_alloc(&p->d_status, 2))) break;
    if ((rc = dev_alloc(&p->d_tile_counter, 4))) break;
    if ((rc = dev_alloc(&p->d_early, (size_t)q))) break;
    if ((rc = dev_alloc(&p->d_proj_progress, 2))) break;
    if ((rc = dev_alloc(&p->d_draw, 2))) break;
    cudaError_t e = cudaSuccess;
    if (e == cudaSuccess) e = cudaMemcpy(p->d_group_start, start.data(), (q + 1) * sizeof(int), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(p->d_group_of, p->group_of.data(), P * sizeof(int), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(p->d_w, p->w.data(), P * sizeof(double), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemset(p->d_proj_ticket, 0, 2 * ((size_t)p->proj_grid / 16 + 2) * sizeof(unsigned int));
    if (e == cudaSuccess) e = cudaMemset(p->d_status, 0, 2 * sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(p->d_tile_counter, 0, 4 * sizeof(unsigned long long));
    if (e == cudaSuccess) e = cudaMemset(p->d_early, 0, q * sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(p->d_proj_progress, 0, 2 * sizeof(unsigned long long));
    if (e == cudaSuccess) e = cudaMemset(p->d_draw, 0, 2 * sizeof(unsigned long long));
    if (e == cudaSuccess) e = cudaMemset(p->d_n_rec, 0, q * sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(p->d_t_acc, 0, q * sizeof(int));
    if (e != cudaSuccess) { (void)cudaGetLastError(); rc = SOLON_ERR_CUDA; break; }
    if ((rc = launch_fill_projection(p, 0))) break;
    if (cudaDeviceSynchronize() != cudaSuccess) { (void)cudaGetLastError(); rc = SOLON_ERR_CUDA; break; }
  } while (0);
  if (rc) {
    free_device(p);
    delete p;
    return rc;
  }
  *out = p;
  return SOLON_OK;
}

int solon_plan_destroy(solon_plan* plan) {
  if (!plan) return SOLON_ERR_INVALID_ARG;
  cudaStreamSynchronize(plan->stream);
  free_device(plan);
  delete plan;
  return SOLON_OK;
}

int solon_plan_set_stream(solon_plan* plan, void* cuda_stream) {
  if (!plan) return SOLON_ERR_INVALID_ARG;
  plan->stream = (cudaStream_t)cuda_stream;
  return SOLON_OK;
}

int solon_plan_set_num_projections(solon_plan* plan, int K) {
  if (!plan || K < 1 || K > SOLON_MAX_PROJECTIONS) return SOLON_ERR_INVALID_ARG;
  SOLON_CUDA_TRY(cudaStreamSynchronize(plan->stream));
  plan->K = K;
  int rc = alloc_projection(plan);
  if (rc) return rc;
  SOLON_CUDA_TRY(cudaMemsetAsync(plan->d_draw, 0, 2 * sizeof(unsigned long long), plan->stream));
  plan->draw_parity = 0;
  if ((rc = launch_fill_projection(plan, 0))) return rc;
  SOLON_CUDA_TRY(cudaStreamSynchronize(plan->stream));
  return SOLON_OK;
}

int solon_plan_reseed(solon_plan* plan, uint64_t seed) {
  if (!plan) return SOLON_ERR_INVALID_ARG;
  plan->seed = seed;
  SOLON_CUDA_TRY(cudaMemsetAsync(plan->d_draw, 0, 2 * sizeof(unsigned long long), plan->stream));   // draw 0 of the new seed
  plan->draw_parity = 0;
  return launch_fill_projection(plan, 0);
}

int solon_plan_set_fresh_projections(solon_plan* plan, int on) {
  if (!plan) return SOLON_ERR_INVALID_ARG;
  plan->fresh_f = on ? 1 : 0;
  if (!on && plan->draw_parity < 0) {
    // decodes stop drawing: the count now stands still, so the host may know which buffer holds the current draw
    unsigned long long n = 0;
    SOLON_CUDA_TRY(cudaMemcpyAsync(&n, plan->d_draw, sizeof(n), cudaMemcpyDeviceToHost, plan->stream));
    SOLON_CUDA_TRY(cudaStreamSynchronize(plan->stream));
    plan->draw_parity = (int)(n & 1ULL);
  }
  return SOLON_OK;
}

int solon_plan_set_optimistic(solon_plan* plan, int mode) {
  if (!plan || mode < 0 || mode > 2) return SOLON_ERR_INVALID_ARG;
  plan->optimistic = mode;
  // the mode is read on the device by the projection kernel; a change also forgets what the last decode found
  std::vector<int> init((size_t)8 + plan->q, 0);
  init[4] = mode;
  SOLON_CUDA_TRY(cudaMemcpyAsync(plan->d_opt, init.data(), init.size() * sizeof(int), cudaMemcpyHostToDevice, plan->stream));
  SOLON_CUDA_TRY(cudaStreamSynchronize(plan->stream));
  return SOLON_OK;
}

int solon_plan_get_optimistic_outcome(solon_plan* plan, int* skipped) {
  if (!plan || !skipped) return SOLON_ERR_INVALID_ARG;
  std::vector<int> word((size_t)8 + plan->q, 0);
  SOLON_CUDA_TRY(cudaMemcpyAsync(word.data(), plan->d_opt, word.size() * sizeof(int), cudaMemcpyDeviceToHost, plan->stream));
  SOLON_CUDA_TRY(cudaStreamSynchronize(plan->stream));
  int all_clean = 1;
  for (int g = 0; g < plan->q; ++g) all_clean &= word[(size_t)8 + g] != 0 ? 1 : 0;
  *skipped = (word[1] != 0 && all_clean) ? 1 : 0;      // what the recovery kernel itself evaluates
  return SOLON_OK;
}

int solon_plan_set_early_locator(solon_plan* plan, int mode) {
  if (!plan || mode < 0 || mode > 3) return SOLON_ERR_INVALID_ARG;
  plan->early_locator = mode;
  return SOLON_OK;
}

int solon_plan_get_early_outcome(solon_plan* plan, int* outcome) {
  if (!plan || !outcome) return SOLON_ERR_INVALID_ARG;
  SOLON_CUDA_TRY(cudaMemcpyAsync(outcome, plan->d_early, (size_t)plan->q * sizeof(int), cudaMemcpyDeviceToHost, plan->stream));
  SOLON_CUDA_TRY(cudaStreamSynchronize(plan->stream));
  return SOLON_OK;
}

int solon_plan_set_tolerance(solon_plan* plan, double tau) {
  if (!plan || !(tau >= 0.0)) return SOLON_ERR_INVALID_ARG;
  plan->tau = tau;
  return SOLON_OK;
}

int solon_plan_set_lsq_rows(solon_plan* plan, int rows) {
  if (!plan || rows < 1) return SOLON_ERR_INVALID_ARG;
  plan->lsq_rows = rows;
  return SOLON_OK;
}

int64_t solon_plan_dc(const solon_plan* plan) { return plan ? plan->d_c : SOLON_ERR_INVALID_ARG; }
int solon_plan_num_groups(const solon_plan* plan) { return plan ? plan->q : SOLON_ERR_INVALID_ARG; }
int solon_plan_num_projections(const solon_plan* plan) { return plan ? plan->K : SOLON_ERR_INVALID_ARG; }
int solon_plan_group_of(const solon_plan* plan, int node) {
  if (!plan || node < 0 || node >= plan->P) return SOLON_ERR_INVALID_ARG;
  return plan->group_of[node];
}
int solon_plan_group_start(const solon_plan* plan, int group) {
  if (!plan || group < 0 || group >= plan->q) return SOLON_ERR_INVALID_ARG;
  return plan->group_start[group];
}
int solon_plan_group_size(const solon_plan* plan, int group) {
  if (!plan || group < 0 || group >= plan->q) return SOLON_ERR_INVALID_ARG;
  return plan->group_start[group + 1] - plan->group_start[group];
}
int solon_plan_get_node_scalars(const solon_plan* plan, double* w) {
  if (!plan || !w) return SOLON_ERR_INVALID_ARG;
  memcpy(w, plan->w.data(), plan->P * sizeof(double));
  return SOLON_OK;
}
int solon_plan_get_projection_vectors(solon_plan* plan, float* f) {
  if (!plan || !f) return SOLON_ERR_INVALID_ARG;
  // draw n lives in buffer n & 1; a decode that drew anew has already advanced the count past the draw it used
  unsigned long long n = 0;
  SOLON_CUDA_TRY(cudaMemcpyAsync(&n, plan->d_draw, sizeof(n), cudaMemcpyDeviceToHost, plan->stream));
  SOLON_CUDA_TRY(cudaStreamSynchronize(plan->stream));
  if (plan->last_decode_advanced && n > 0) n -= 1;
  const float* src = (n & 1ULL) ? plan->d_f2 : plan->d_f;
  SOLON_CUDA_TRY(cudaMemcpy2DAsync(f, plan->d_c * sizeof(float), src, plan->f_pitch * sizeof(float),
                                   plan->d_c * sizeof(float), plan->K, cudaMemcpyDeviceToHost, plan->stream));
  SOLON_CUDA_TRY(cudaStreamSynchronize(plan->stream));
  return SOLON_OK;
}

int solon_plan_get_projections(solon_plan* plan, double* rho, double* nu) {
  if (!plan || !rho || !nu) return SOLON_ERR_INVALID_ARG;
  SOLON_CUDA_TRY(cudaMemcpyAsync(rho, plan->d_rho, (size_t)plan->K * plan->P * sizeof(double), cudaMemcpyDeviceToHost, plan->stream));
  SOLON_CUDA_TRY(cudaMemcpyAsync(nu, plan->d_nu, (size_t)plan->P * sizeof(double), cudaMemcpyDeviceToHost, plan->stream));
  SOLON_CUDA_TRY(cudaStreamSynchronize(plan->stream));
  return SOLON_OK;
}

int solon_plan_get_recovery(solon_plan* plan, int* n_rec, int* t, int* rec_rows, double* coeff) {
  if (!plan || !n_rec || !t || !rec_rows || !coeff) return SOLON_ERR_INVALID_ARG;
  std::vector<int> rows(plan->P);
  std::vector<double> cf((size_t)plan->P * plan->m);
  SOLON_CUDA_TRY(cudaMemcpyAsync(n_rec, plan->d_n_rec, plan->q * sizeof(int), cudaMemcpyDeviceToHost, plan->stream));
  SOLON_CUDA_TRY(cudaMemcpyAsync(t, plan->d_t_acc, plan->q * sizeof(int), cudaMemcpyDeviceToHost, plan->stream));
  SOLON_CUDA_TRY(cudaMemcpyAsync(rows.data(), plan->d_rec_rows, plan->P * sizeof(int), cudaMemcpyDeviceToHost, plan->stream));
  SOLON_CUDA_TRY(cudaMemcpyAsync(cf.data(), plan->d_coeff, cf.size() * sizeof(double), cudaMemcpyDeviceToHost, plan->stream));
  SOLON_CUDA_TRY(cudaStreamSynchronize(plan->stream));
  size_t out = 0;
  for (int g = 0; g < plan->q; ++g) {
    int base = plan->group_start[g];
    for (int j = 0; j < n_rec[g]; ++j, ++out) {
      rec_rows[out] = rows[base + j];
      memcpy(coeff + out * plan->m, cf.data() + (size_t)(base + j) * plan->m, plan->m * sizeof(double));
    }
  }
  return SOLON_OK;
}

int solon_plan_set_profiling(solon_plan* plan, int on) {
  if (!plan) return SOLON_ERR_INVALID_ARG;
  if (on && !plan->ev[0]) {
    for (int i = 0; i < 6; ++i) SOLON_CUDA_TRY(cudaEventCreate(&plan->ev[i]));
  }
  plan->profiling = on ? 1 : 0;
  return SOLON_OK;
}

int solon_plan_get_timings(solon_plan* plan, float* ms) {
  if (!plan || !ms) return SOLON_ERR_INVALID_ARG;
  for (int i = 0; i < 4; ++i) ms[i] = 0.f;
  if (!plan->ev[0]) return SOLON_OK;
  SOLON_CUDA_TRY(cudaStreamSynchronize(plan->stream));
  if (plan->ev_valid[0] && plan->ev_valid[1]) SOLON_CUDA_TRY(cudaEventElapsedTime(&ms[0], plan->ev[0], plan->ev[1]));
  for (int i = 0; i < 3; ++i)
    if (plan->ev_valid[2 + i] && plan->ev_valid[3 + i])
      SOLON_CUDA_TRY(cudaEventElapsedTime(&ms[1 + i], plan->ev[2 + i], plan->ev[3 + i]));
  return SOLON_OK;
}

int64_t solon_plan_kernel_launches(const solon_plan* plan) { return plan ? plan->launches : SOLON_ERR_INVALID_ARG; }

int solon_plan_status(solon_plan* plan) {
  if (!plan) return SOLON_ERR_INVALID_ARG;
  int word[2] = {0, 0};
  SOLON_CUDA_TRY(cudaMemcpyAsync(word, plan->d_status, 2 * sizeof(int), cudaMemcpyDeviceToHost, plan->stream));
  SOLON_CUDA_TRY(cudaStreamSynchronize(plan->stream));
  return ((word[0] | word[1]) & kStatusWaitExpired) ? SOLON_ERR_INTERNAL : SOLON_OK;
}

int solon_decode_status(solon_plan* plan) {
  if (!plan) return SOLON_ERR_INVALID_ARG;
  // the locator leaves the accepted error count of every group (-1: none); expired waits leave a sticky bit
  std::vector<int> t_acc((size_t)plan->q, 0);
  int word[2] = {0, 0};
  SOLON_CUDA_TRY(cudaMemcpyAsync(word, plan->d_status, 2 * sizeof(int), cudaMemcpyDeviceToHost, plan->stream));
  SOLON_CUDA_TRY(cudaMemcpyAsync(t_acc.data(), plan->d_t_acc, (size_t)plan->q * sizeof(int), cudaMemcpyDeviceToHost, plan->stream));
  SOLON_CUDA_TRY(cudaStreamSynchronize(plan->stream));
  if ((word[0] | word[1]) & kStatusWaitExpired) return SOLON_ERR_INTERNAL;
  for (int g = 0; g < plan->q; ++g)
    if (t_acc[(size_t)g] < 0) return SOLON_ERR_UNDECODABLE;
  return SOLON_OK;
}

}  // extern "C"
