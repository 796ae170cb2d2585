/*
 * solon.h - C interface of libsolon: the encode step and the robust decode step of Solon
 * (arXiv 2110.01595, Section 3), for all P simulated compute nodes on one sm_100a GPU.
 *
 * Notation (paper -> this header): compression ratio r_c -> m; coded length d_c = ceil(d / m);
 * redundancy ratio r = group size; s = Byzantine nodes tolerated; P nodes = P partition
 * gradients (the paper takes B = P); q groups ("blocks" of the linear block code).
 *
 * Conventions for every call
 *   - Returns 0 (SOLON_OK) or a negative solon_status.  Nothing is printed, thrown or aborted.
 *   - "device" pointers are CUDA device memory owned by the caller, float32, contiguous,
 *     row-major, and 16-byte aligned at their base; the library never frees or resizes them and
 *     never writes its inputs.  "host" pointers are ordinary host memory.
 *   - Work is enqueued on the plan's stream (default: the legacy default stream) and the call
 *     returns without synchronising, unless stated otherwise.
 *   - A plan is not thread-safe; use one plan per host thread / stream.
 *   - There is no CPU fallback: without a CUDA device every call that needs one fails with
 *     SOLON_ERR_CUDA.
 */
#ifndef SOLON_H_
#define SOLON_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum solon_status {
  SOLON_OK = 0,
  SOLON_ERR_INVALID_ARG = -1, /* null pointer, misaligned pointer, value out of range          */
  SOLON_ERR_INFEASIBLE = -2,  /* 2 s + m > P: no mechanism exists (corollary of Theorem 2)     */
  SOLON_ERR_CUDA = -3,        /* a CUDA runtime call failed or no device is present            */
  SOLON_ERR_UNDECODABLE = -4, /* some group has no consistent set of <= s corrupt nodes        */
  SOLON_ERR_INTERNAL = -5,    /* a bounded device-side wait expired (should not happen)        */
  SOLON_ERR_NOMEM = -6        /* host or device allocation failed                              */
} solon_status;

/* Limits of this implementation. */
#define SOLON_MAX_NODES 1024      /* P; also P * m <= 16384 (recovery table in shared memory) */
#define SOLON_MAX_GROUP 128       /* largest group size the locator handles                   */
#define SOLON_MAX_M 32            /* compression ratio (the paper reports trouble above 14)   */
#define SOLON_MAX_S 16            /* adversaries per group                                    */
#define SOLON_MAX_PROJECTIONS 4   /* random projections K                                     */

/* Element type of partition gradients, coded vectors and aggregate (a property of the plan). */
typedef enum solon_dtype {
  SOLON_F32 = 0, /* float32 at the boundary (solon_encode, solon_decode, ...)                                   */
  SOLON_F64 = 1  /* float64 at the boundary, the paper's wire format (Table 2): the calls with the suffix _f64 */
} solon_dtype;

typedef struct solon_plan solon_plan;

/* ------------------------------------------------------------------------------------------
 * Plan-free host helpers (no device needed).
 * ---------------------------------------------------------------------------------------- */

/* Feasibility of a mechanism (Theorem 2: r >= 2 s + m; its corollary: 2 s + m <= P; r <= P).
 * Returns SOLON_OK, SOLON_ERR_INFEASIBLE (2 s + m > P) or SOLON_ERR_INVALID_ARG (anything else,
 * including the limits above). */
int solon_check_params(int P, int s, int m, int r, int64_t d);

/* Group layout of the linear block code (Section 3.4, A = I_q (x) 1_{r x r}): q = floor(P / r)
 * groups of consecutive nodes; when r does not divide P the P - q r left-over nodes are dealt
 * one at a time to the first groups, so every group has at least r members.
 * starts: host array of q + 1 ints (capacity given by starts_capacity), group g owns nodes
 * [starts[g], starts[g+1]).  *q_out receives q. */
int solon_group_layout(int P, int r, int* starts, int starts_capacity, int* q_out);

/* The "distinct nonzero scalars w_1..w_P" of Section 3.4.  Each group of size r_g uses the first
 * r_g of the n' Chebyshev points cos((2k-1) pi / (2 n')), k = 1..n', n' = r_g rounded up to even.
 * w: host array of P doubles. */
int solon_node_scalars(int P, int r, double* w);

/* Host mirror of the device locator (the same source compiled for the CPU), for one group:
 * the floating-point reading of the locator phi of Section 3.4 and of the block decoder's
 * inverse (psi).
 *   rho   host, K x n row-major: projected values f_kappa . R_k of the group's n nodes
 *   nu    host, n: row energies sum_p R_k[p]^2
 *   w_g   host, n: the group's node scalars
 *   tau   relative tolerance of the "!=" test (see solon_plan_set_tolerance)
 * Outputs (host): mask[n] (1 = located as corrupt); *t_out the accepted error count;
 * rec_rows[n] / *n_rec the nodes (indices inside the group) whose rows the recovery reads;
 * coeff[n_rec * m], coeff[j*m + l] = weight of row rec_rows[j] in coordinate l of a chunk.
 * Returns SOLON_OK or SOLON_ERR_UNDECODABLE (outputs then hold the best guess). */
int solon_locate_host(int n, int m, int s, int K, const double* rho, const double* nu,
                      const double* w_g, double tau, uint8_t* mask, int* t_out, int* rec_rows,
                      int* n_rec, double* coeff);

const char* solon_strerror(int status);

/* ------------------------------------------------------------------------------------------
 * Plan.
 * ---------------------------------------------------------------------------------------- */

/* Build the mechanism (A, E, D) of Section 3.4 for P nodes, s adversaries per group,
 * compression ratio m, minimum group size r (>= 2 s + m) and gradient length d: group layout,
 * node scalars, K = 2 projection vectors f_kappa[p] = 1 + N(0,1) drawn on the device from
 * `seed` (f ~ N(1, I) in Section 3.4; solon_plan_set_fresh_projections makes every decode draw anew),
 * and all device workspace.  Uses the current CUDA device.
 * Synchronises the device once.  *out receives the plan, to be released by solon_plan_destroy. */
int solon_plan_create(int P, int s, int m, int r, int64_t d, uint64_t seed, solon_plan** out);
int solon_plan_destroy(solon_plan* plan);

/* The same with the element type chosen (solon_plan_create is dtype = SOLON_F32).  A SOLON_F64 plan moves 8-byte
 * gradients, coded vectors and aggregates - what the paper's implementation sent (Table 2: 89.6 MB for ResNet-18's
 * 11,173k parameters) and the precision for which it reports decoding trouble only "when r_c > 14" (appendix on
 * limitations) - through solon_encode_f64, solon_decode_f64, solon_overwrite_rows_f64 and solon_step_host_f64; the
 * float32 calls, solon_lsq_grads and the two-call decode return SOLON_ERR_INVALID_ARG on such a plan, and the _f64 calls
 * on a float32 plan.  Group sums, polynomial evaluation, projections and recovery are all float64 then; the locator's
 * default tolerance is 1e-10.  Compression ratios with a float64 kernel: m = 1..6, 8, 10, 12, 14
 * (solon_float64_m_supported); any other m gives SOLON_ERR_INVALID_ARG. */
int solon_plan_create_ex(int P, int s, int m, int r, int64_t d, uint64_t seed, int dtype, solon_plan** out);
int solon_float64_m_supported(int m);
int solon_plan_dtype(const solon_plan* plan);          /* SOLON_F32 or SOLON_F64 */

/* Stream on which later calls enqueue (a cudaStream_t passed as void*). */
int solon_plan_set_stream(solon_plan* plan, void* cuda_stream);

/* Number of random projections K in 1..SOLON_MAX_PROJECTIONS (default 2; 1 is the paper's
 * single f).  All projections share one error-locator polynomial.  Redraws f; synchronises. */
int solon_plan_set_num_projections(solon_plan* plan, int K);

/* Restart the sequence of draws from a new seed: the vectors in memory become draw 0 of that seed.
 * Enqueued on the plan's stream. */
int solon_plan_reseed(solon_plan* plan, uint64_t seed);

/* Algorithm 1 draws its random vector inside the decoder, and the proof that every corrupt node is located with
 * probability 1 (Lemma 3) needs f independent of what the adversary sent.  on = 0 (default): the vectors in memory
 * are reused by every decode until solon_plan_reseed; that is sound against an adversary that can neither read nor
 * infer them (they are drawn on the device from the plan's seed and never leave it), but one that knows f can send a
 * deviation orthogonal to all K vectors and stay unseen.  on = 1: every decode projects with vectors no earlier decode
 * used - draw n of the plan's seed, n counted on the device, so that a replayed CUDA graph of a decode moves on as well.
 * The next decode's vectors are written, into a second buffer, by spare CTAs of the locator kernel (solon_decode,
 * solon_decode_finish), before the adversary's next vectors exist: no kernel is added, but the recovery kernel can only
 * be scheduled once those CTAs have all started, which costs 5 us on a decode of 15 nodes x 2.2 M coded values and
 * 12 - 45 us (the higher figure under the power cap) on one of 45 x 5.7 M.  A closed training loop that faces an adaptive
 * adversary should switch it on (sgd.ClosedLoop does).
 * solon_plan_get_projection_vectors returns the vectors the most recent decode used. */
int solon_plan_set_fresh_projections(solon_plan* plan, int on);

/* tau of the floating-point "!=" test of the locator: node k is inconsistent with a fitted
 * polynomial Q when |rho_k - Q(w_k)| > tau * sqrt(2 * median_k nu_k).  Default 1e-5, about
 * thirty times the rounding noise of float32 coded vectors. */
int solon_plan_set_tolerance(solon_plan* plan, double tau);

/* Early locator.  Any subset of the columns gives a valid random projection, so solon_decode lets
 * the locator kernel start on the projection of the first eighth (about) of every column range
 * while the projection kernel is still streaming the rest, and afterwards only checks, on the final
 * projections, that the set it found is exactly the set of nodes that do not fit; if that check
 * fails (an attacker who spared those columns) the whole locator runs as it would have anyway.
 * Results do not depend on the mode.  mode 0: never; 1 (default): when the projection pass is long
 * enough to hide the early run (P * d_c * 4 bytes >= 350 MB; 250 MB when s = 1) and the solver is small (groups of at
 * most 64 nodes, s <= 5); 2: whenever the solver is small; 3: diagnostic - as 2, but the projection
 * kernel announces no partial sums, so the locator's bounded wait for them (2 ms) runs out and it
 * takes its ordinary path afterwards (outcome 3 of solon_plan_get_early_outcome; results unchanged). */
int solon_plan_set_early_locator(solon_plan* plan, int mode);

/* Optimistic decode (Algorithm 1 with the block decoder's work done ahead of the locator's verdict).  For m <= 6 the
 * recovery reads m trusted rows per group and applies the inverse of their Vandermonde block (Section 4.2's block
 * decoder); any m trusted rows give the same sum.  The projection kernel, which has every row on chip anyway, can apply
 * the inverse for the rows the PREVIOUS decode's recovery read (the locator's last table; before the first decode the
 * table for no corrupt node) to each column slice as it passes and write the aggregate itself.  If the locator then
 * finds all of those rows trusted in THIS decode, the recovery kernel returns at once and the decode has read the
 * received matrix once instead of 1 + q m / P times: with no attackers, or with attackers that stay where they were,
 * every decode from the third or fourth on.  If one of those rows is corrupt now, the recovery kernel runs as usual and
 * overwrites the aggregate.  The mask never depends on the mode.  The aggregate is computed in the recovery kernel's
 * arithmetic and order: bit for bit what mode 0 gives whenever the previous table is also this decode's table (same
 * corrupt set), and the same sum up to the rounding of the plan's element type when it came from other trusted rows - so with mode 1 or 2 the
 * last bits of an aggregate can depend on the decode before it; mode 0 gives history-independent bits.
 * mode 0: never; 1 (default): when in each of the last two decodes the table of the decode before would have served (its
 * rows were all trusted: the attackers, if any, stay where they are; decided on the device, no host round trip); 2: always.  Eligible plans (either element type): s > 0, m <= 6
 * and q m rows fitting in the projection kernel's first batch of rows (at most 32); other plans ignore the mode.
 * A decode captured in a CUDA graph keeps deciding on the device at every replay; only a graph captured in mode 0
 * never speculates, whatever the mode set later (its projection kernel was launched without the rows to recover from). */
int solon_plan_set_optimistic(solon_plan* plan, int mode);
/* *skipped = 1 if the recovery kernel of the most recent solon_decode had nothing to do.  Synchronises. */
int solon_plan_get_optimistic_outcome(solon_plan* plan, int* skipped);

/* Rows per partition for solon_lsq_grads (default 256). */
int solon_plan_set_lsq_rows(solon_plan* plan, int rows_per_partition);

/* Queries (host, no synchronisation unless stated). */
int64_t solon_plan_dc(const solon_plan* plan);          /* d_c = ceil(d / m)                    */
int solon_plan_num_groups(const solon_plan* plan);      /* q                                    */
int solon_plan_group_of(const solon_plan* plan, int node);
int solon_plan_group_start(const solon_plan* plan, int group);
int solon_plan_group_size(const solon_plan* plan, int group);
int solon_plan_num_projections(const solon_plan* plan);
int solon_plan_get_node_scalars(const solon_plan* plan, double* w /* host, P */);
/* Copies f (K x d_c, row-major) to the host; synchronises the plan's stream. */
int solon_plan_get_projection_vectors(solon_plan* plan, float* f /* host, K * d_c */);

/* ------------------------------------------------------------------------------------------
 * The hot path.
 * ---------------------------------------------------------------------------------------- */

/* Encode (Section 3.4, z_j = W_j Y_j 1_P with W_j = I_{d_c} (x) [1, w_j, ..., w_j^{m-1}]).
 *   partition_grads  device, P x d: row i is partition gradient g_i
 *   coded            device, P x d_c: row k receives node k's coded vector,
 *                    coded[k][p] = sum_{l<m} w_k^l * ybar_g[p m + l], where ybar_g is the sum of
 *                    the gradients of k's group, zero-padded to m d_c entries.
 * Arithmetic: ybar_g is added up in float32, the group's rows in node order (its rounding is
 * common to all nodes of the group, so the decoder returns it unamplified).  The mix is
 * evaluated in float32 for m <= 6; for larger m (and for m without a specialised kernel) in
 * float64 and rounded once to float32, because the decoder amplifies rounding that differs
 * from node to node by a factor that grows like 2^m. */
int solon_encode(solon_plan* plan, const float* partition_grads, float* coded);

/* Robust decode (Algorithm 1 with the locator phi and block decoder psi of Section 3.4).
 *   received  device, P x d_c: what the P nodes sent (coded vectors, up to s rows per group
 *             replaced by arbitrary values, non-finite values included); may alias `coded`
 *   agg_grad  device, d: receives u = sum over groups of the recovered group sums = G 1_P
 *   byz_mask  device, P bytes: 1 for every node located as Byzantine, else 0
 * Three kernels: projections rho = f R and row energies (one pass over `received`), the locator
 * (tiny, on device; see solon_plan_set_early_locator for how it overlaps the first), the recovery
 * (one pass over the trusted rows it needs).  The projections are computed with float32
 * products and float32 sums of eight terms at a time, float64 beyond (error at most
 * 8 * 2^-24 of sum |f_p R_kp|, far below the locator's tolerance).  If some group has
 * no consistent set of at most s corrupt nodes the outputs hold a best guess and
 * solon_decode_status reports SOLON_ERR_UNDECODABLE. */
int solon_decode(solon_plan* plan, const float* received, float* agg_grad, uint8_t* byz_mask);

/* Encode and decode of a SOLON_F64 plan: as solon_encode / solon_decode with float64 buffers of the same shapes (bases
 * 16-byte aligned).  The group sum, the mix and the recovery are float64 throughout, the projections exact float64
 * products of the (float32-valued) vectors f with the received values. */
int solon_encode_f64(solon_plan* plan, const double* partition_grads, double* coded);
int solon_decode_f64(solon_plan* plan, const double* received, double* agg_grad, uint8_t* byz_mask);

/* Status of the most recent solon_decode: synchronises the plan's stream, then returns SOLON_OK,
 * SOLON_ERR_UNDECODABLE, SOLON_ERR_INTERNAL or SOLON_ERR_CUDA. */
int solon_decode_status(solon_plan* plan);

/* Health of the plan's kernels so far, for callers that encode without decoding: synchronises the
 * plan's stream, then returns SOLON_OK, SOLON_ERR_INTERNAL (a bounded wait inside one of the plan's
 * kernels - solon_encode's included - ran out at some point; the bit is sticky) or SOLON_ERR_CUDA. */
int solon_plan_status(solon_plan* plan);

/* The decode in two halves, for a coded matrix whose COLUMNS are spread over several devices.
 * Equation (1)'s locator needs only the projected values rho = f R, and f R is a sum over
 * columns; so each device projects the columns it holds with its own f, the K x P values (and
 * the P row energies) are summed over the devices by whatever collective the caller has, and
 * every device then runs the same locator on the same sums and recovers its own columns
 * (Algorithm 1 applied to a column block of Y_j; the chunks of Section 3.4 are independent).
 * Each device uses a plan built for the columns it owns (same P, s, m, r; d = its share, a
 * multiple of m except on the last device; different seeds).
 *
 * solon_decode_project: first kernel only.
 *   received  device, P x d_c        rho  device, K x P float64 (output)    nu  device, P float64 (output)
 * With s = 0 nothing is launched and rho, nu are left untouched.
 * solon_decode_finish: locator and recovery from the given rho and nu (device; the caller's sums).
 *   received, agg_grad, byz_mask as in solon_decode.
 * solon_decode(plan, R, u, mask) equals solon_decode_project followed by solon_decode_finish on
 * the same buffers.  Status is read with solon_decode_status after solon_decode_finish. */
int solon_decode_project(solon_plan* plan, const float* received, double* rho, double* nu);
int solon_decode_finish(solon_plan* plan, const double* rho, const double* nu, const float* received,
                        float* agg_grad, uint8_t* byz_mask);

/* Least-squares partition gradients g_i = X_i^T (X_i w - y_i) (the paper accepts any method that
 * needs a sum of per-partition functions, Section 1; this one feeds the encode step).
 *   X      device, (P * rows) x d; partition i owns rows [i rows, (i+1) rows)
 *   y      device, P * rows
 *   w      device, d
 *   grads  device, P x d (output)
 * Two streaming passes over X (residuals, then gradients), sums in float64.  When d is a multiple
 * of 4 and X, w and grads are 16-byte aligned the passes use 128-bit loads and float32 products
 * (one rounding per term); any other layout takes scalar loads and float64 products.  Allocates
 * the residual buffer (P * rows floats) on first use or when rows grows: returns SOLON_ERR_NOMEM
 * if that fails. */
int solon_lsq_grads(solon_plan* plan, const float* X, const float* y, const float* w, float* grads);

/* One whole step with HOST buffers: copies the gradients to the device, encodes, overwrites the
 * rows of the n_byz listed nodes with the given vectors (the adversary sits between encode and
 * decode), decodes, copies the aggregate and the mask back, and synchronises.
 *   grads_host     host, P x d          byz_nodes      host, n_byz node indices (may be NULL if 0)
 *   byz_rows_host  host, n_byz x d_c    agg_host       host, d (output)
 *   mask_host      host, P bytes (output)
 * Device staging buffers are owned by the plan and allocated on the first call.  Returns the
 * decode status.  Pinned host memory makes the copies asynchronous to each other but the call
 * still returns only when everything is done. */
int solon_step_host(solon_plan* plan, const float* grads_host, int n_byz, const int* byz_nodes,
                    const float* byz_rows_host, float* agg_host, uint8_t* mask_host);

/* The adversary of a device-resident simulation: overwrites rows of a P x d_c matrix in place,
 * matrix[nodes[i]][:] = rows[i][:], on the plan's stream (what solon_step_host does from host
 * buffers).  Not part of the method: it stands in for whatever the Byzantine nodes send.
 *   matrix  device, P x d_c          nodes  device, n_rows ints in [0, P) (checked on the device:
 *   rows    device, n_rows x d_c            out-of-range entries are skipped)
 * n_rows = 0 does nothing. */
int solon_overwrite_rows(solon_plan* plan, float* matrix, int n_rows, const int* nodes, const float* rows);

/* solon_step_host and solon_overwrite_rows for a SOLON_F64 plan (float64 buffers, same shapes and rules). */
int solon_step_host_f64(solon_plan* plan, const double* grads_host, int n_byz, const int* byz_nodes,
                        const double* byz_rows_host, double* agg_host, uint8_t* mask_host);
int solon_overwrite_rows_f64(solon_plan* plan, double* matrix, int n_rows, const int* nodes, const double* rows);

/* ------------------------------------------------------------------------------------------
 * Introspection of the last decode (for parity tests and diagnostics; each synchronises).
 * ---------------------------------------------------------------------------------------- */

/* rho (K x P, row-major) and nu (P) computed by the projection kernel. */
int solon_plan_get_projections(solon_plan* plan, double* rho /* host, K * P */, double* nu /* host, P */);

/* Recovery table chosen by the locator: n_rec[g] rows for group g, their node indices in
 * rec_rows (concatenated over groups), coefficients coeff (concatenated, n_rec[g] * m each,
 * coeff[j*m + l]), and the accepted error count t[g] (-1 if the group was undecodable).
 * Capacities: n_rec and t hold q ints, rec_rows P ints, coeff P * m doubles. */
int solon_plan_get_recovery(solon_plan* plan, int* n_rec, int* t, int* rec_rows, double* coeff);

/* Outcome of the early locator in the last solon_decode, one int per group (host, q entries):
 * 0 no early run, 1 the early answer was confirmed on the final projections, 2 it was not (the
 * whole locator ran), 3 the bounded wait for the partial projection expired (the whole locator
 * ran), 4 the group's CTA became resident only after the projections were complete and skipped
 * the early run. */
int solon_plan_get_early_outcome(solon_plan* plan, int* outcome);

/* Projections without any allocation.  (The paper has no counterpart: this entry point exists for
 * callers of this library that are not allowed to allocate device memory at the moment they need
 * the projections - for example a service whose whole device memory has already been handed to its
 * own pool, or a step loop that must not run into the device-wide synchronisation an allocation
 * implies.  solon_plan_create allocates, so such callers cannot use a plan.)
 *
 * Computes what the first kernel of solon_decode computes: rho[kappa * P + k] = sum_p
 * f[kappa * f_pitch + p] * received[k * d_c + p] and nu[k] = sum_p received[k * d_c + p]^2.
 *   received  device, P x d_c float32          f    device, K rows of f_pitch floats (f_pitch >= d_c,
 *   rho       device, K x P float64 (output)        a multiple of 4; base 16-byte aligned; entries
 *   nu        device, P float64 (output)            beyond d_c in a row are ignored)
 * The kernel's scratch (per-block partial sums and completion counters, about 1.3 MB) is a fixed
 * array inside the library's device image, so every GPU that loads the library holds it until the
 * process exits.  Limits: (K + 1) * P <= 512 and K <= 4; larger problems get SOLON_ERR_INVALID_ARG.
 * No allocation routine is called, here or in anything this calls.  One thing is outside the library's
 * hands: the CUDA runtime places the library's device code, this array included, on a device the first
 * time anything of the library runs there.  A caller about to hand all device memory to its own pool
 * should therefore make one call of this entry point (or create and destroy a plan) on each device at
 * start-up, before the memory is given away.
 * That first call on each device also looks up the array's device address (with that device current);
 * make it outside any stream capture.  All calls on a device share the one array: two
 * calls whose kernels may overlap on the GPU (different streams, no ordering) race on it and
 * corrupt each other's sums; calls on one stream, or otherwise ordered, are fine.  The counters are
 * cleared at the start of every call; the partial sums are fully rewritten by every call.
 * Enqueued on `cuda_stream`; does not synchronise. */
int solon_project_noalloc(const float* received, const float* f, int64_t f_pitch, int P, int64_t d_c,
                          int K, double* rho, double* nu, void* cuda_stream);

/* Per-kernel timing with CUDA events on the plan's stream.  When switched on, solon_encode and
 * solon_decode record an event before and after each of their kernels; solon_plan_get_timings
 * synchronises the stream and returns the durations of the most recent calls in milliseconds:
 * ms[0] encode, ms[1] projections, ms[2] locator, ms[3] recovery (0 for a kernel not yet run).
 * While it is on, the two calls also open NVTX ranges on the calling thread ("solon_encode";
 * "solon_decode" with "project", "locate", "recover" inside) for timeline tools.
 * Off by default (the events cost a few microseconds per call). */
int solon_plan_set_profiling(solon_plan* plan, int on);
int solon_plan_get_timings(solon_plan* plan, float* ms /* host, 4 */);

/* Number of kernels the library launched on behalf of this plan since creation. */
int64_t solon_plan_kernel_launches(const solon_plan* plan);

#ifdef __cplusplus
}
#endif
#endif /* SOLON_H_ */
