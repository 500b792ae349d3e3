/* wpsgd.h -- C ABI of the B200 (sm_100a) library for the hot path of weighted parallel SGD.
 *
 * Method: Cheng, Li, Zhang, "Weighted parallel SGD for distributed unbalanced-workload
 * training system" (WP-SGD). The library runs Algorithm 1 on one GPU:
 *
 *   - k simulated nodes; node j owns the rows [shard_off[j], shard_off[j+1]) of the data and
 *     runs n_steps[j] sequential SGD steps (Eq. 5) on the regularised loss of Eq. 4,
 *         w_n = w_{n-1} - eta_n ( lambda w_{n-1} + L'(y, w_{n-1}.x) x ),
 *     starting from a shared w0 (zeros if not given). Chains of different nodes are independent.
 *   - the final models are combined with the weights of Eq. 6 (default rate r = 1 - eta lambda)
 *     or Eq. 8 (caller's rate r):  v = sum_j weight_j w_j,  weight_j = r^{T_j} / sum_i r^{T_i},
 *     where T_j = max_i n_steps[i] - n_steps[j] is the paper's delay of node j.
 *
 * Conventions fixed here because the paper leaves them open:
 *   - The n-th example (n = 1, 2, ...) of node j is row shard_off[j] + floor(u m_j / 2^32), where
 *     m_j is the shard's row count and u is output word (n-1) mod 4 of Philox4x32-10 with key
 *     (seed low 32 bits, seed high 32 bits) and counter ((n-1)/4 low, (n-1)/4 high, j, 0):
 *     i.i.d. uniform draws with replacement, a pure function of (seed, j, n).
 *   - Losses, with z = w.x: hinge L = max(0, 1 - y z), L' = -y if y z < 1 else 0;
 *     logistic L = log(1 + exp(-y z)), L' = -y / (1 + exp(y z)); squared L = (z - y)^2 / 2,
 *     L' = z - y. Labels for hinge and logistic are +1 / -1 floats.
 *   - Step size: constant eta0, or eta_n = eta0 / sqrt(n). For the decaying schedule the default
 *     weight of node j is the product of (1 - eta_s lambda) over the steps s = n_j+1 .. t it did
 *     not run (this equals Eq. 6 when eta is constant; the paper has constant eta only).
 *   - A node with n_steps[j] == 0 keeps w0 and still takes part in the combination.
 *
 * Arithmetic: features fp32 or bf16 (widened exactly), model and accumulation fp32, the scale
 * factor of the sparse path and all weights fp64.
 *
 * Memory: every pointer is tagged DEVICE or HOST below. Device buffers belong to the caller and
 * must stay valid until the work enqueued on the context's stream has finished. The context owns
 * the k x d model matrix, the index stream and small tables. All functions except the *_host one
 * and the queries documented as synchronous only enqueue work on the stream given at creation.
 *
 * Errors: every function returns a wpsgd_status; a text for the last failure on a context is
 * available from wpsgd_last_error(). Nothing throws or aborts. Kernels never spin without bound:
 * a wait that exceeds its limit sets a device status word, reported as WPSGD_ERR_TIMEOUT by the
 * next wpsgd_check().
 */
#ifndef WPSGD_H_
#define WPSGD_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct wpsgd_ctx wpsgd_ctx; /* opaque; created and destroyed by the library */

typedef enum {
  WPSGD_OK = 0,
  WPSGD_ERR_INVALID_ARG = 1,
  WPSGD_ERR_ALLOC = 2,
  WPSGD_ERR_CUDA = 3,
  WPSGD_ERR_STATE = 4,       /* call out of order, e.g. combine before run */
  WPSGD_ERR_UNSUPPORTED = 5,
  WPSGD_ERR_TIMEOUT = 6      /* a bounded device-side wait gave up */
} wpsgd_status;

typedef enum { WPSGD_LOSS_HINGE = 0, WPSGD_LOSS_LOGISTIC = 1, WPSGD_LOSS_SQUARED = 2 } wpsgd_loss;
typedef enum { WPSGD_X_F32 = 0, WPSGD_X_BF16 = 1 } wpsgd_xtype;
typedef enum { WPSGD_LR_CONST = 0, WPSGD_LR_INV_SQRT = 1 } wpsgd_lr;

/* Create a context for k nodes and d features on CUDA device `device`; all work is enqueued on
 * `cuda_stream` (a cudaStream_t; NULL = the legacy default stream). Allocates the k x d fp32
 * model matrix. (Algorithm 1: inputs "nodes k", model w in R^d.) */
wpsgd_status wpsgd_create(int device, void* cuda_stream, int32_t k, int64_t d, wpsgd_ctx** out);

/* Release everything the context owns. Synchronises the stream first. NULL is accepted. */
wpsgd_status wpsgd_destroy(wpsgd_ctx* ctx);

/* Options by name. Unknown name or bad value: WPSGD_ERR_INVALID_ARG. Except for "sampling", the result of a run
 * never depends on an option beyond rounding order.
 *
 *   "sampling"        order of the examples. 0 (default): independent uniform draws as in the header comment.
 *                     1: the literal reading of Algorithm 1 ("randomly shuffle the data on machine i", then "get the
 *                     n-th example"): one fixed pseudo-random permutation pi_j of the shard per node, cycled, i.e. the
 *                     n-th example is row pi_j((n-1) mod m_j). pi_j is a 4-round balanced Feistel network on the even
 *                     bit count covering m_j - 1 with cycle walking, keyed by the Philox block at counter (0, 0, j, 1)
 *                     under the seed; round function mix(R ^ key) = multiply 0x85EBCA6B, xor-shift 13, multiply
 *                     0xC2B2AE35, xor-shift 16, masked to half the bits.
 *   "dense_variant"   kernel for dense rows. 0 (default): chosen from the shape. 1: any shape and alignment, model in
 *                     global memory. 2: one CTA per node, one step per round trip, model in registers. 3: the same with
 *                     one warp per node. 4: blocked form (8 samples per synchronisation), one CTA per node. 5: blocked
 *                     form, one warp per node (rows of at most 64 16-byte chunks). 8: blocked form for bf16 rows, Gram
 *                     block and margins from mma.sync tensor-core instructions, columns of a node split over a
 *                     thread-block cluster (what 0 picks for aligned bf16 rows of 2048 columns and more). 9: blocked
 *                     form (16 samples) for fp32 rows with a node's columns split over a cluster, at most 256 columns
 *                     per CTA (what 0 picks for rows of 512 columns and more when the nodes are few enough for clusters
 *                     of 4 or 8 on the GPU's SMs). The blocked forms (4, 5, 8, 9) take both step-size schedules and
 *                     need eta0 * lambda <= 0.25.
 *   "sparse_variant"  kernel for CSR rows. 0 (default) and 2: blocks of up to 64 steps run in a shared-memory cache of
 *                     the model entries they touch. 1: one step per round trip to the model in global memory.
 *   "cluster"         CTAs per node of variants 8 and 9: 0 (default) chosen from d (and the node count), else 1, 2, 4 or 8.
 *   "block_samples"   samples per block of variant 8: 0 (default) 16 when the rows fit, else 8; 8 or 16 to force one.
 *   "threads"         threads per node of variants 2 and 4, warps x 32 per CTA of variant 5; 0 (default): chosen from d.
 *   "prefetch"        rows in flight per chain of variants 2, 3 and of sparse variant 1; 0 (default): chosen.
 *   "stages"          blocks of rows in the shared-memory ring of the blocked kernels; 0 (default): as many as fit
 *                     (up to 4), else 2..8.
 *   "host_pipeline"   wpsgd_solve_host: 1 (default) copies the shards in up to four groups of nodes, longest chains
 *                     first, on a stream of the context and starts the chains of a group when its rows have arrived;
 *                     0 copies everything first.
 *   "spin_limit"      polls after which a device-side wait gives up (default 2^20).
 *   "timing"          1: record events around the chain kernel (see wpsgd_last_chain_ms). Default 0.
 *   "test_drop_block" test hook of the bounded waits, not for production use: the rows of that block of every chain
 *                     are never requested, so the wait for them runs out and WPSGD_ERR_TIMEOUT is reported by
 *                     wpsgd_check; -1 (default) = off. */
wpsgd_status wpsgd_set_option(wpsgd_ctx* ctx, const char* name, int64_t value);

/* Node numbers that enter the sample stream in place of 0..k-1 (HOST [k], >= 0; NULL restores the
 * default). A GPU that holds a subset of a larger cluster's nodes passes their global numbers, so
 * that every node draws the same examples wherever it is placed. Takes effect at the next run. */
wpsgd_status wpsgd_set_node_ids(wpsgd_ctx* ctx, const int32_t* ids);

/* Algorithm 1, the per-node loops (Eq. 5), on dense rows.
 *   X          DEVICE  [N, ld_elems] row-major, fp32 or bf16 per `xt`; only the first d columns
 *                      of a row are read. N = shard_off[k].
 *   y          DEVICE  [N] fp32 labels / targets.
 *   shard_off  HOST    [k+1] non-decreasing row offsets; node j owns rows [off[j], off[j+1]).
 *   n_steps    HOST    [k] steps of each node (>= 0). A node with steps needs >= 1 row, < 2^32 rows.
 *   eta0, sched, lambda, loss   as in the header comment; requires 0 <= eta_n lambda < 1.
 *   seed       seed of the sample stream.
 *   w0         DEVICE  [d] shared initial model, or NULL for zeros (Algorithm 1 initialises to 0;
 *                      the paper's experiments start from a constant vector).
 * After the call the context holds the k final models. Host arrays are copied before return. */
wpsgd_status wpsgd_run(wpsgd_ctx* ctx, const void* X, wpsgd_xtype xt, int64_t ld_elems, const float* y,
                       const int64_t* shard_off, const int64_t* n_steps, float eta0, wpsgd_lr sched,
                       float lambda, wpsgd_loss loss, uint64_t seed, const float* w0);

/* Continue every chain from the models the context holds: node j runs n_more[j] further steps,
 * numbered after the ones it has already run (so it draws examples step_done+1, ...). Data and
 * hyper-parameters must be the ones given to the wpsgd_run / wpsgd_run_csr that started the
 * chains. Gives the paper's snapshots "after 100000 x i updates of the fastest node"
 * (Section "Numerical experiments", Approach) without restarting. Dense rows; chains that were started on CSR
 * rows continue with wpsgd_continue_csr. */
wpsgd_status wpsgd_continue(wpsgd_ctx* ctx, const void* X, wpsgd_xtype xt, int64_t ld_elems, const float* y,
                            const int64_t* shard_off, const int64_t* n_more);

/* The same loops on sparse rows in CSR form (the paper's data: a few tens of features per row).
 *   row_ptr    DEVICE  [N+1] int64, col_idx DEVICE [nnz] int32 (unique within a row, < d),
 *   val        DEVICE  [nnz] fp32.  Other arguments as wpsgd_run.
 * The model of node j is kept as s_j * u_j with an fp64 scalar s_j, so that the regulariser costs
 * one scalar multiply per step instead of a pass over d (same iterates as Eq. 5). */
wpsgd_status wpsgd_run_csr(wpsgd_ctx* ctx, const int64_t* row_ptr, const int32_t* col_idx, const float* val,
                           const float* y, const int64_t* shard_off, const int64_t* n_steps, float eta0,
                           wpsgd_lr sched, float lambda, wpsgd_loss loss, uint64_t seed, const float* w0);

/* wpsgd_continue on CSR rows: node j runs n_more[j] further steps from the model (u_j and its scale) the context
 * holds; arrays as wpsgd_run_csr, hyper-parameters and seed those of the run that started the chains. With
 * wpsgd_combine and wpsgd_set_models this is averaging every `span` fastest-node steps on the paper's kind of data
 * (Section "Combining WP-SGD with bucket SGD"). */
wpsgd_status wpsgd_continue_csr(wpsgd_ctx* ctx, const int64_t* row_ptr, const int32_t* col_idx, const float* val,
                                const float* y, const int64_t* shard_off, const int64_t* n_more);

/* Read-only check of a CSR matrix against the preconditions of wpsgd_run_csr, enqueued on the context's stream:
 * row_ptr DEVICE [n_rows+1] within [0, nnz] and non-decreasing, col_idx DEVICE [nnz] in [0, d) and strictly increasing
 * within a row (no column twice: the sparse update of Eq. 5 writes each nonzero's model entry once). Nothing outside
 * [0, nnz) is read. A violation is reported by the next wpsgd_check as WPSGD_ERR_CUDA with the row in the message. */
wpsgd_status wpsgd_validate_csr(wpsgd_ctx* ctx, const int64_t* row_ptr, const int32_t* col_idx, int64_t n_rows,
                                int64_t nnz);

/* Algorithm 1, the aggregation: v = sum_j weight_j w_j (j ascending) with Eq. 6 weights, or Eq. 8
 * weights when r > 0 is given (r <= 0 or NaN selects the default; r = 1 is plain averaging).
 *   v_out      DEVICE  [d] fp32.
 * WPSGD_ERR_STATE if no run has been made on the context. */
wpsgd_status wpsgd_combine(wpsgd_ctx* ctx, double r, float* v_out);

/* The same aggregation with weights given by the caller (HOST [k] fp64): v = sum_j weights[j] w_j.
 * For a cluster of GPUs that each hold a subset of the nodes: every GPU passes the Eq. 6 weights of
 * its own nodes, computed over all nodes with wpsgd_weights, and the partial sums are then added
 * across GPUs (the single exchange of Algorithm 1's last line). */
wpsgd_status wpsgd_combine_weighted(wpsgd_ctx* ctx, const double* weights, float* v_out);

/* Copy the k final models (W^{j, t - T_j} of Lemma 3), scale applied, to W_out DEVICE [k, d] fp32. */
wpsgd_status wpsgd_get_models(wpsgd_ctx* ctx, float* W_out);

/* Replace every node's model by v (DEVICE [d]): the broadcast step of averaging every `span`
 * fastest-node steps (Section "Combining WP-SGD with bucket SGD"); follow with wpsgd_continue. */
wpsgd_status wpsgd_set_models(wpsgd_ctx* ctx, const float* v);

/* Eq. 6 / Eq. 8 weights of the last run, to weights HOST [k] (fp64), and whether the condition of
 * Corollary 3 / 4 (Eq. 7 / Eq. 9), 2 sum_j r^{T_j} > sqrt(k) + k, holds (cond_holds may be NULL).
 * Host-only computation; synchronous. */
wpsgd_status wpsgd_get_weights(wpsgd_ctx* ctx, double r, double* weights, int* cond_holds);

/* The weights for given step counts without a context (HOST arrays). sum_rT (may be NULL) receives
 * sum_j r^{T_j}, the quantity in Eq. 7 / Eq. 9 and in the validity bound of averaging every span. */
wpsgd_status wpsgd_weights(const int64_t* n_steps, int32_t k, float eta0, wpsgd_lr sched, float lambda,
                           double r, double* weights, int* cond_holds, double* sum_rT);

/* Condition the paper gives for averaging every `span` fastest-node steps on an unbalanced system (Section "Combining
 * WP-SGD with bucket SGD", after Deduction 2): (k / sum_j r^{T_j}) (1 - eta lambda)^span < 1, with r = 1 - eta lambda
 * unless r > 0 is given. n_steps HOST [k]. lhs (may be NULL) receives the left-hand side, holds (may be NULL) whether
 * it is below 1. Constant step size. Host-only computation. */
wpsgd_status wpsgd_span_valid(const int64_t* n_steps, int32_t k, float eta0, float lambda, double r, int64_t span,
                              double* lhs, int* holds);

/* The sample stream of Algorithm 1's "get the n-th example" as defined in the header comment, computed on the host by
 * the same function the kernels call: row indices (within a shard of m rows) of steps n_begin+1 .. n_begin+count of
 * node `node`, to out HOST [count] uint32. sampling as the option of that name (0 draws, 1 shuffled order). Needs no
 * context and no GPU. */
wpsgd_status wpsgd_sample_indices_host(uint64_t seed, int32_t node, int64_t m, int64_t n_begin, int64_t count,
                                       int32_t sampling, uint32_t* out);

/* The sample stream exactly as the chain kernels draw it: row indices (within the shard of m rows)
 * of steps n_begin+1 .. n_begin+count of node `node`, to out DEVICE [count] uint32. */
wpsgd_status wpsgd_sample_indices(wpsgd_ctx* ctx, uint64_t seed, int32_t node, int64_t m, int64_t n_begin,
                                  int64_t count, uint32_t* out);

/* Objective of Eq. 3-4 and 0/1 error of sign(w.x) on dense rows (the paper's evaluation measures):
 *   objective = (lambda/2)|w|^2 + mean_i L(y_i, w.x_i);  error = share of rows with sign(w.x) != sign(y).
 *   X DEVICE [n_rows, ld_elems], y DEVICE [n_rows], w DEVICE [d]; out DEVICE [2] fp64 = {objective, error}. */
wpsgd_status wpsgd_objective(wpsgd_ctx* ctx, const void* X, wpsgd_xtype xt, int64_t ld_elems, const float* y,
                             int64_t n_rows, const float* w, float lambda, wpsgd_loss loss, double* out);

/* The same two measures on CSR rows (the paper's data are sparse): row_ptr DEVICE [n_rows+1] int64, col_idx DEVICE
 * int32 (< d), val DEVICE fp32, y DEVICE [n_rows], w DEVICE [d]; out DEVICE [2] fp64 = {objective, error}. */
wpsgd_status wpsgd_objective_csr(wpsgd_ctx* ctx, const int64_t* row_ptr, const int32_t* col_idx, const float* val,
                                 const float* y, int64_t n_rows, const float* w, float lambda, wpsgd_loss loss,
                                 double* out);

/* Whole path from HOST buffers: copies X HOST [N, d] (dense, contiguous), y HOST [N] and w0 HOST [d]
 * (or NULL) to the device, runs the chains and the combination, copies v back to v_out HOST [d], and
 * waits for completion. Page-locked host buffers give full copy speed. Device staging buffers are
 * owned by the context and reused across calls. r as in wpsgd_combine. */
wpsgd_status wpsgd_solve_host(wpsgd_ctx* ctx, const void* X, wpsgd_xtype xt, const float* y,
                              const int64_t* shard_off, const int64_t* n_steps, float eta0, wpsgd_lr sched,
                              float lambda, wpsgd_loss loss, uint64_t seed, const float* w0, double r,
                              float* v_out);

/* The same from HOST buffers for CSR rows (the paper's kind of data): row_ptr HOST [N+1], col_idx HOST [nnz], val HOST
 * [nnz], y HOST [N], w0 HOST [d] or NULL, v_out HOST [d]; other arguments as wpsgd_run_csr and wpsgd_combine. Copies
 * the arrays to staging buffers of the context, runs the chains and the combination, copies v back and waits. */
wpsgd_status wpsgd_solve_host_csr(wpsgd_ctx* ctx, const int64_t* row_ptr, const int32_t* col_idx, const float* val,
                                  const float* y, const int64_t* shard_off, const int64_t* n_steps, float eta0,
                                  wpsgd_lr sched, float lambda, wpsgd_loss loss, uint64_t seed, const float* w0, double r,
                                  float* v_out);

/* An entry point for callers that must not allocate device memory. (The paper has no counterpart:
 * this is a convenience of the library.) It does what wpsgd_run followed by wpsgd_combine does on
 * dense rows, but takes no context and calls no cudaMalloc / cudaFree or any other allocating
 * routine: the model matrix, the sample stream and the small tables that a context would own live in
 * one array built into the library (about 5.4 MiB of device memory on every GPU that loads it, held
 * until the process exits). Meant for code that runs where allocation is forbidden or would stall:
 * inside another framework's memory pool that has reserved the whole device, in a latency-critical
 * loop that cannot afford cudaMalloc's device-wide synchronisation, or in a process whose memory
 * budget is fixed at start-up.
 *   device, cuda_stream   where to run; the work is enqueued on the stream and the call returns.
 *   X, y, w0, v_out       DEVICE buffers of the caller, as in wpsgd_run / wpsgd_combine.
 *   shard_off, n_steps    HOST [k+1] / [k], as in wpsgd_run.
 * Limits (WPSGD_ERR_UNSUPPORTED with a message naming the limit when exceeded): k <=
 * WPSGD_STATIC_MAX_NODES, k * d <= WPSGD_STATIC_MAX_MODEL_ELEMS, sum of n_steps <=
 * WPSGD_STATIC_MAX_STEPS. Other argument errors as wpsgd_run.
 * The first call on a device looks up the array's device address (once per device); make that
 * first call before starting any stream capture. All calls on a device share the one array, which
 * still holds what the previous call left there; each call rewrites what it uses and clears its
 * status word, so calls in sequence on one stream are independent, but two calls whose GPU work
 * overlaps (different streams, or different host threads) race on it and give wrong results.
 * The kernels' status word (a bounded wait that gave up, a failed bounds check) lives in the same array;
 * wpsgd_check_static reads it. */
#define WPSGD_STATIC_MAX_NODES 1024
#define WPSGD_STATIC_MAX_MODEL_ELEMS (1 << 18)
#define WPSGD_STATIC_MAX_STEPS (1 << 20)
wpsgd_status wpsgd_solve_static(int device, void* cuda_stream, const void* X, wpsgd_xtype xt, int64_t ld_elems,
                                const float* y, const int64_t* shard_off, const int64_t* n_steps, int32_t k,
                                int64_t d, float eta0, wpsgd_lr sched, float lambda, wpsgd_loss loss, uint64_t seed,
                                const float* w0, double r, float* v_out);

/* wpsgd_check for wpsgd_solve_static: waits for the stream and reads the status word inside the built-in array
 * (no allocation). Same return values as wpsgd_check; the text is available from wpsgd_last_error(NULL). */
wpsgd_status wpsgd_check_static(int device, void* cuda_stream);

/* Wait for the stream and read the device status word. WPSGD_OK, WPSGD_ERR_TIMEOUT (a bounded wait
 * gave up), or WPSGD_ERR_CUDA (a launch or copy failed, or a kernel's own bounds check fired). */
wpsgd_status wpsgd_check(wpsgd_ctx* ctx);

/* Device time of the most recent chain kernel launch (the per-node loops only, without the sample
 * stream kernel and the combination), in milliseconds, from events recorded on the context's
 * stream around it. Needs wpsgd_set_option(ctx, "timing", 1) before the run; waits for the kernel. */
wpsgd_status wpsgd_last_chain_ms(wpsgd_ctx* ctx, float* ms);

/* Number of kernels this context has launched so far (for launch accounting). */
int64_t wpsgd_launch_count(const wpsgd_ctx* ctx);

/* Text of the last error on the context (or of the last context-free call when ctx is NULL).
 * The pointer stays valid until the next call on that context. */
const char* wpsgd_last_error(const wpsgd_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* WPSGD_H_ */
