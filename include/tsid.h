/*
 * tsid.h - C ABI of the B200 (sm_100a) template-recovery factorization.
 *
 * Problem (Sec. 1 and Def. 1 of the paper; Sec. 3.2, Eq. (rmf-obj)): a template
 * R in R^{m x n} is known on an index set Omega (|Omega| = nnz).  Stage I of
 * TSID matrix completion fits factors P in R^{m x k}, Q in R^{n x k} to
 *
 *     L(P, Q) = sum_{(i,j) in Omega} (r_ij - p_i . q_j)^2 + lambda (|P|_F^2 + |Q|_F^2)
 *
 * by full-batch gradient steps.  One step (Sec. 5.1, Eqs. (update-p), (update-q), Eq. 9;
 * Sec. 5.3 for the clip) computes, from the SAME (P, Q) for both sides:
 *
 *     e_ij = r_ij - p_i . q_j                          for (i,j) in Omega
 *     G_P  = E Q   (m x k),   G_Q = E^T P   (n x k)    E = sparse residual matrix
 *     D_P[i,:] = 2 G_P[i,:] / s_i  - 2 lambda P[i,:]   s_i  = 1 or max(1, |Omega_i|)
 *     D_Q[j,:] = 2 G_Q[j,:] / s'_j - 2 lambda Q[j,:]   s'_j = 1 or max(1, |Omega^j|)
 *     D <- clip(D)                                     ASYM_STEP: min(D, xi)
 *     P <- P + eta D_P,   Q <- Q + eta D_Q
 *
 * The sums are accumulated warp -> block -> grid in a fixed order (no floating
 * point atomics): identical inputs give bitwise identical outputs.
 *
 * Conventions for every entry point
 *   - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  The library
 *     never allocates device memory: all device state lives in the caller's
 *     `workspace` (size from tsid_workspace_bytes), which must stay valid and
 *     untouched until tsid_destroy.  The handle owns host bookkeeping only.
 *   - P is row-major m x k fp32, Q is row-major n x k fp32, caller-owned, 16-byte
 *     aligned, updated in place.
 *   - All work is enqueued on cfg.stream.  tsid_grad_step and tsid_fit with
 *     loss_every == 0 do not synchronise; tsid_template_create, tsid_loss,
 *     tsid_fit with loss_every > 0 and tsid_check synchronise the stream.
 *   - Every call returns a status; nothing throws, aborts or traps.  Argument
 *     errors are detected before any launch.  tsid_last_error gives a message.
 *   - Limits: 1 <= k <= 256, k a multiple of 4 (TSID_F32) or 8 (TSID_BF16_SHADOW);
 *     0 <= nnz <= 2^31 - 1; m, n >= 1.
 */
#ifndef TSID_H_
#define TSID_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tsid_template tsid_template_t; /* opaque */

typedef enum {
  TSID_OK = 0,
  TSID_ERR_INVALID_ARG = 1,  /* null pointer, bad size, bad enum, misaligned pointer      */
  TSID_ERR_INDEX_RANGE = 2,  /* a row index outside [0,m) or column index outside [0,n)   */
  TSID_ERR_DUPLICATE = 3,    /* TSID_VALIDATE: the same (row, col) appears twice          */
  TSID_ERR_UNSORTED = 4,     /* TSID_INPUT_ROW_SORTED promised but the input is not       */
  TSID_ERR_OOM = 5,          /* workspace smaller than tsid_workspace_bytes               */
  TSID_ERR_CUDA = 6,         /* a CUDA runtime call failed (message in tsid_last_error)   */
  TSID_ERR_UNSUPPORTED = 7,  /* configuration outside the limits above                    */
  TSID_ERR_NONFINITE = 8,    /* an updated factor became inf/nan (reported by tsid_check, */
                             /* tsid_loss and tsid_fit with loss_every > 0)               */
  TSID_ERR_TOO_LARGE = 9     /* tsid_sse_noalloc: more entries than its built-in scratch   */
                             /* covers (the call did nothing)                             */
} tsid_status_t;

/* Storage precision of the factor values the two gradient passes READ.  The
 * caller's P, Q are always the fp32 master copy.  TSID_BF16_SHADOW keeps a
 * bfloat16 copy (round to nearest even) refreshed by the update kernel; products
 * are exact in fp32 and all sums are fp32 (Sec. 5.1 mixed precision: 16-bit
 * multiplicands, 32-bit accumulation). */
typedef enum { TSID_F32 = 0, TSID_BF16_SHADOW = 1 } tsid_precision_t;

/* TSID_PATH_SPARSE: CSR/CSC gather-reduce passes (HBM bound).
 * TSID_PATH_DENSE_TC: tcgen05 masked-GEMM variant (Sec. 5.1, "Regularizing Sparse RMF
 * Updates for Tensor Cores"): P Q^T, then E Q and E^T P with bf16 operands and fp32
 * accumulation; requires TSID_BF16_SHADOW, k a multiple of 16 and m, n multiples of 128.
 * TSID_PATH_HYBRID: both, each where it fits.  Under skewed popularity the observed cells crowd into
 * nearly full blocks once rows and columns are ordered by their number of entries.  At create the rows and
 * columns are ranked by degree (ties by index), the template is cut into 128 x 128 tiles in that order,
 * and every tile with at least ~3 % of its cells observed (480 entries; more if the tiles would not fit
 * the 16 bytes per entry of workspace reserved for them) is kept as a dense fp16 block and goes through
 * the tensor-core pass; every other entry goes through the gather-reduce passes on a CSR / CSC of the
 * remainder; the two partial sums of a factor row are added in a fixed order.  Needs TSID_BF16_SHADOW,
 * k in {64, 128}, no entry-wise clip, no TSID_VALUES_U8, and nnz >= max(m, n, ceil(m/128) ceil(n/128)).
 * If no tile reaches the threshold, if Omega holds a duplicate, or if a value in a stored tile is beyond
 * the fp16 range, the handle runs TSID_PATH_SPARSE instead (tsid_get_info tells).
 * TSID_PATH_AUTO picks DENSE_TC when the template qualifies and nnz / (m n) >= 0.05, else HYBRID when
 * it qualifies and nnz >= 4,000,000, else SPARSE. */
typedef enum { TSID_PATH_AUTO = 0, TSID_PATH_SPARSE = 1, TSID_PATH_DENSE_TC = 2, TSID_PATH_HYBRID = 3 } tsid_path_t;

/* Sec. 5.3.  ASYM_STEP (default reading): D <- min(max(xi, -D), D) = min(D, xi): increases
 * of a coordinate are capped at eta*xi, decreases are free.  ASYM_GRAD: the same formula
 * applied to the loss gradient g = -D, i.e. D <- max(D, -xi).  ASYM_ENTRY: the equation of
 * Sec. 5.3 taken entry by entry, as printed: every observed (i,j) contributes its own clipped
 * direction c_ij = min(2 e_ij q_j - 2 lambda p_i, xi) (for p_i; symmetrically for q_j), the
 * contributions of a factor row are added, divided by s (Eq. 9's 1/n) and applied with eta.
 * In this mode the regulariser sits inside every entry's term, a row without entries does not
 * move, the values read are those of the template's precision, and d_gradP / d_gradQ receive
 * the sums of the c_ij.  Sparse path only, and with TSID_F32 factors k <= 128 (TSID_ERR_UNSUPPORTED
 * otherwise, from tsid_workspace_bytes and tsid_template_create). */
typedef enum {
  TSID_CLIP_NONE = 0, TSID_CLIP_ASYM_STEP = 1, TSID_CLIP_ASYM_GRAD = 2, TSID_CLIP_ASYM_ENTRY = 3
} tsid_clip_t;

/* Eq. 9's 1/n factor: divide the summed gradient of a factor row by the number of
 * observed entries that contribute to it (COUNT) or not at all (NONE). */
typedef enum { TSID_NORM_NONE = 0, TSID_NORM_COUNT = 1 } tsid_norm_t;

enum {
  TSID_VALIDATE = 1u,         /* also check Omega for duplicate (row, col) pairs            */
  TSID_INPUT_ROW_SORTED = 2u, /* promise: COO is sorted by (row, col); checked, skips a sort */
  TSID_VALUES_U8 = 4u         /* promise: every value is an integer in [0, 255] (ratings); checked
                                 (else TSID_ERR_UNSUPPORTED).  The gradient passes then stream one byte
                                 per value instead of four; results are bitwise the same.            */
};

typedef struct {
  int32_t m, n, k;
  int64_t nnz;
  int32_t precision; /* tsid_precision_t */
  int32_t path;      /* tsid_path_t      */
  float eta, lambda, xi;
  int32_t clip;      /* tsid_clip_t */
  int32_t norm_p;    /* tsid_norm_t */
  int32_t norm_q;    /* tsid_norm_t */
  uint32_t flags;
  void *stream;           /* cudaStream_t owned by the caller (0 = legacy default stream) */
  void *workspace;        /* DEVICE memory owned by the caller, 256-byte aligned          */
  size_t workspace_bytes; /* its size                                                     */
} tsid_config_t;

/* Bytes of device workspace a template needs (no counterpart in the paper: the library allocates nothing, the
 * caller brings the memory).  The size depends on m, n, k, nnz, precision, path (AUTO resolves from these and
 * clip), and flags (TSID_VALUES_U8 adds two byte streams); the whole cfg is validated as by
 * tsid_template_create, so fill every field the way the create call will see it (stream, workspace and
 * workspace_bytes are not read).  Host-only, no CUDA call.  Errors: INVALID_ARG, UNSUPPORTED. */
tsid_status_t tsid_workspace_bytes(const tsid_config_t *cfg, size_t *h_bytes_out);

/* Layout pass + handle creation: takes the problem as Def. 1 / Sec. 1 state it - R in R^{m x n} known on the
 * index set Omega - with Omega given as COO triples (Sec. 6.1, "Data Model").  d_rows, d_cols (int32[nnz]) and d_vals (fp32[nnz]) are
 * the COO triples of Omega on the DEVICE, in any order; they are only read, and may be
 * freed when the call returns (it synchronises cfg.stream).  Builds in the workspace:
 * CSR sorted by (row, col), CSC sorted by (col, row), perm (CSC position -> CSR position),
 * the equal-length work segments of both passes, gradient / shadow / partial buffers.
 * Duplicates, when not rejected by TSID_VALIDATE, are each counted; ties keep input order.  A dense cell
 * holds one value, so TSID_PATH_DENSE_TC refuses a template with a duplicate (TSID_ERR_DUPLICATE, whatever
 * the flags say) and TSID_PATH_HYBRID runs such a template on the sparse path.
 * On error *out is NULL. */
tsid_status_t tsid_template_create(const tsid_config_t *cfg, const int32_t *d_rows,
                                   const int32_t *d_cols, const float *d_vals,
                                   tsid_template_t **out);

/* One full-batch step (Sec. 5.1 Eqs. (update-p), (update-q) summed over Omega, aggregated as in Eq. 9 with its
 * 1/n normalisation; clip of Sec. 5.3), in place on d_P (m x k) and d_Q (n x k).  If d_gradP / d_gradQ are
 * non-null they receive the raw sums G_P = E Q (m x k) and G_Q = E^T P (n x k), fp32,
 * computed from the factors as they were BEFORE the update.  Asynchronous. */
tsid_status_t tsid_grad_step(tsid_template_t *t, float *d_P, float *d_Q, float *d_gradP_or_null,
                             float *d_gradQ_or_null);

/* The two halves of tsid_grad_step, for a template whose rows are sharded over several GPUs
 * (the paper keeps template recovery on one GPU and names multi-GPU recovery as future work,
 * Sec. 7; the full-batch step itself splits exactly: with the rows of Omega partitioned over the
 * ranks, each rank's G_P rows are complete and the G_Q of all ranks add up, so one sum-exchange of
 * G_Q per step is the only communication).
 *   tsid_grad: the raw sums G_P = E Q (m x k) and G_Q = E^T P (n x k) of THIS template's entries
 *     at (d_P, d_Q); nothing is updated.  With TSID_CLIP_ASYM_ENTRY the sums are those of the
 *     clipped per-entry directions, which add up over shards in the same way.
 *   tsid_apply: direction, clip and update of tsid_grad_step from given sums (for example d_GQ
 *     summed over the ranks), in place on d_P, d_Q; refreshes the bf16 shadows.
 *   tsid_get_counts: |Omega_i| (int32[m]) and |Omega^j| (int32[n]) of this template; either may be NULL.
 *   tsid_set_norm_counts: replaces the counts that TSID_NORM_COUNT divides by (a shard sees only
 *     its part of every column: pass the counts summed over the ranks); NULL leaves a side as it is.
 *     Lasts until destroy.
 * All four are asynchronous on cfg.stream; every pointer is a 16-byte aligned DEVICE pointer.
 * Errors: TSID_ERR_INVALID_ARG. */
tsid_status_t tsid_grad(tsid_template_t *t, const float *d_P, const float *d_Q, float *d_GP, float *d_GQ);
tsid_status_t tsid_apply(tsid_template_t *t, float *d_P, float *d_Q, const float *d_GP, const float *d_GQ);
tsid_status_t tsid_get_counts(tsid_template_t *t, int32_t *d_cnt_p_or_null, int32_t *d_cnt_q_or_null);
/* tsid_apply with the exchange of G_Q folded into the update kernel (no counterpart in the paper).
 * h_GQ_parts and h_Q_replicas are HOST arrays of `world` DEVICE pointers: part r is rank r's partial
 * G_Q (n x k fp32, written by its tsid_grad), replica r is rank r's copy of Q; pointers of other ranks
 * must be mapped into this process (peer access, symmetric or IPC memory) and are used with plain
 * loads and stores only.  Updates P (this rank's rows) from d_GP, and the rows
 * [n rank / world, n (rank + 1) / world) of Q: their parts are added in rank order, the update is
 * applied once and the result is stored into EVERY replica.  The caller synchronises the ranks before
 * the call (all parts complete) and after it (all slices stored) before anything reads Q or rewrites
 * a part; the bf16 shadows are refreshed by the next tsid_grad.  world <= 16.  Asynchronous.
 * Errors: TSID_ERR_INVALID_ARG. */
tsid_status_t tsid_apply_sliced(tsid_template_t *t, float *d_P, const float *d_GP, float *const *h_Q_replicas,
                                const float *const *h_GQ_parts, int32_t rank, int32_t world);
tsid_status_t tsid_set_norm_counts(tsid_template_t *t, const int32_t *d_cnt_p_or_null,
                                   const int32_t *d_cnt_q_or_null);

/* The iteration of Sec. 5.1, "Stage I Execution Example" (repeat the step until R* ~ P Q^T; here a fixed number
 * of epochs): `epochs` steps in place.  loss_every > 0: after every loss_every-th step (and before the
 * first) the SSE is computed and stored in h_sse_history_or_null (host, capacity
 * 1 + epochs / loss_every doubles); this synchronises.  loss_every == 0: asynchronous.
 *   With loss_every == 0 and epochs >= 4 the steps are replayed from an executable CUDA graph (the
 * whole call when epochs <= 16, else 8 steps per launch and the rest step by step): captured once on
 * a stream of the library's own, launched into cfg.stream, kept with the template while d_P, d_Q and
 * the step count stay the same.  The results are bitwise those of the same number of tsid_grad_step
 * calls.  If the capture fails, the steps launch one by one, in this and every later call; they also do
 * while cfg.stream is itself being captured by the caller (the call can be part of a caller's graph). */
tsid_status_t tsid_fit(tsid_template_t *t, float *d_P, float *d_Q, int32_t epochs,
                       int32_t loss_every, double *h_sse_history_or_null);

/* SSE = sum_Omega e^2 and objective = SSE + lambda (|P|_F^2 + |Q|_F^2) (Eq. (rmf-obj)).
 * Residuals are taken at the template's precision (bf16 shadows if so configured), squares
 * are summed in double in a fixed order; the norms use the fp32 values.  Synchronises. */
tsid_status_t tsid_loss(tsid_template_t *t, const float *d_P, const float *d_Q, double *h_sse,
                        double *h_objective);

/* Synchronises the stream and reports a pending device-side condition
 * (TSID_ERR_NONFINITE, TSID_ERR_CUDA) or TSID_OK. */
tsid_status_t tsid_check(tsid_template_t *t);

/* The whole of Stage I from HOST arrays in one call (Sec. 5.1, "Stage I Execution Example":
 * move the COO triples to the device, initialise from the given P, Q, iterate, return the
 * factors).  h_rows/h_cols/h_vals (nnz each) and h_P (m x k), h_Q (n x k) are HOST pointers
 * (pinned memory makes the copies asynchronous); h_P, h_Q are overwritten with the fitted
 * factors.  cfg.workspace must hold tsid_workspace_bytes_host(cfg) bytes of DEVICE memory:
 * the template's workspace followed by the staged triples and factors.  Copies in, builds the
 * layout, runs `epochs` steps, optionally evaluates the SSE (host double), copies the factors
 * back and synchronises.  Errors as in tsid_template_create / tsid_fit; message via
 * tsid_last_error(NULL). */
tsid_status_t tsid_workspace_bytes_host(const tsid_config_t *cfg, size_t *h_bytes_out);
tsid_status_t tsid_fit_host(const tsid_config_t *cfg, const int32_t *h_rows, const int32_t *h_cols,
                            const float *h_vals, float *h_P, float *h_Q, int32_t epochs,
                            double *h_sse_or_null);

/* Releases the host handle (no counterpart in the paper).  The workspace belongs to the caller.  NULL is accepted. */
tsid_status_t tsid_destroy(tsid_template_t *t);

/* ---- debug / test surface ------------------------------------------------------------ */

/* Device pointers into the workspace (valid until destroy): row_ptr int64[m+1], col_idx
 * int32[nnz] and val_csr fp32[nnz] in CSR order; col_ptr int64[n+1], row_idx int32[nnz] and
 * val_csc fp32[nnz] in CSC order; perm uint32[nnz].  Any out pointer may be NULL. */
tsid_status_t tsid_get_layout(tsid_template_t *t, const int64_t **d_row_ptr,
                              const int32_t **d_col_idx, const float **d_val_csr,
                              const int64_t **d_col_ptr, const int32_t **d_row_idx,
                              const float **d_val_csc, const uint32_t **d_perm);

/* e in CSR order (fp32[nnz], device), at the template's precision.  Asynchronous. */
tsid_status_t tsid_residuals(tsid_template_t *t, const float *d_P, const float *d_Q,
                             float *d_e_csr);

/* Which path the handle runs (tsid_path_t, never AUTO) and how many kernels one
 * tsid_grad_step launches. */
tsid_status_t tsid_get_info(const tsid_template_t *t, int32_t *h_path, int32_t *h_launches_per_step);

/* How many kernels one tsid_fit(t, P, Q, epochs, 0, NULL) enqueues (replayed from a captured graph or
 * launched one by one, the kernels are the same): the shadow refresh of the call, and per epoch the
 * passes and the update.  On the hybrid path tsid_fit's epochs launch fewer kernels than tsid_grad_step:
 * the rank-ordered shadow copies are made once per call and kept current by the update kernel, which also
 * adds the tile passes' sums to the gather-reduce passes' sums (same order of additions, same bits).
 * h_launches: host int64. */
tsid_status_t tsid_get_fit_launches(const tsid_template_t *t, int32_t epochs, int64_t *h_launches);

/* Mini-batch form (Sec. 5.1: the updates run over mini-batches of observed entries, aggregated per factor row and divided
 * by the number of contributors, Eq. 9; a mini-batch step is the full-batch step above restricted to the batch's entries,
 * with Eq. 9's n counted inside the batch).  ONE template holds all batches: d_batch (DEVICE, int32[nnz]) gives the batch of
 * every COO triple, 0 <= batch < n_batches; the layout pass sorts by (batch, row, col) and (batch, col, row) in one go, so
 * every batch owns a contiguous range of work segments in one workspace (tsid_workspace_bytes_batched bytes).  cfg.m, cfg.n
 * are the sizes of P and Q as usual.  tsid_grad_step_batch runs one step on batch `batch` (the other arguments as in
 * tsid_grad_step; the raw sums returned are those of the batch); an epoch is one call per batch, in the caller's order.
 * Sparse path only (cfg.path AUTO or SPARSE), fp32 value streams, n_batches * m and n_batches * n below 2^31,
 * n_batches <= 65536.  The other stepping, loss and count calls refuse such a handle (TSID_ERR_UNSUPPORTED).
 * Errors: as tsid_template_create; TSID_ERR_INDEX_RANGE also for a batch number out of range. */
tsid_status_t tsid_workspace_bytes_batched(const tsid_config_t *cfg, int32_t n_batches, size_t *h_bytes_out);
tsid_status_t tsid_template_create_batched(const tsid_config_t *cfg, const int32_t *d_rows, const int32_t *d_cols,
                                           const float *d_vals, const int32_t *d_batch, int32_t n_batches,
                                           tsid_template_t **out);
tsid_status_t tsid_grad_step_batch(tsid_template_t *t, int32_t batch, float *d_P, float *d_Q, float *d_gradP_or_null,
                                   float *d_gradQ_or_null);

/* What the hybrid path stored (debug / bench surface): the number of 128 x 128 tiles kept densely, the
 * smallest number of entries such a tile holds, and how many entries stayed on the gather-reduce passes.
 * On a handle of another path all three are 0 (tail = nnz).  Any out pointer may be NULL. */
tsid_status_t tsid_get_hybrid_info(const tsid_template_t *t, int64_t *h_tiles, int32_t *h_min_tile_entries,
                                   int64_t *h_tail_entries);

/* Test hook for the failure path of the tensor-core kernel (no counterpart in the paper).  Every wait of that
 * kernel on one of its barriers is bounded by a cycle budget; when it runs out the CTA raises a flag, stops
 * issuing work, frees its tensor memory and returns, and the next synchronising call reports TSID_ERR_CUDA
 * ("a bounded device-side wait expired").  This call makes that happen on purpose, without faulting anything:
 * from now on the kernels of this handle (TSID_PATH_DENSE_TC only, else TSID_ERR_UNSUPPORTED) use a budget of
 * `wait_cycles` clock cycles and their load-issuing thread stops before work item `item` of each CTA, so the
 * consumers of that item wait for loads that were never issued (nothing is outstanding).  wait_cycles = 0
 * restores normal operation.  The gradients of a stalled step are meaningless. */
tsid_status_t tsid_debug_stall_tile_pass(tsid_template_t *t, int64_t wait_cycles, int32_t item);

/* Template sampling (Sec. 5.1, "Sampling the TSID Template Submatrix"): the step before the
 * factorization.  Chooses d = ceil(alpha n) of the n columns uniformly at random without replacement
 * and extracts the template R* = { r_ij : j chosen, (i,j) in Omega } as COO triples with the chosen
 * columns re-indexed 0..d-1 in ascending order of their original index (rows unchanged, kept entries
 * in input order), ready for tsid_template_create with n = d.  The draw is counter-based and
 * reproducible: column j gets the key SplitMix64(seed + (j+1) * 0x9E3779B97F4A7C15) and the d columns
 * with the smallest (key, j) are taken.
 *   - d_rows, d_cols, d_vals: DEVICE, the COO triples of the full matrix (m x n, nnz entries, any order).
 *   - d_colmap: DEVICE int32[n], out: new index of each column, or -1 if it is not in the template.
 *   - d_rows_out, d_cols_out, d_vals_out: DEVICE, capacity nnz each, out: the template's triples.
 *   - h_d_out, h_nnz_out: HOST, out: d and the number of template entries.
 *   - workspace: DEVICE, 256-byte aligned, tsid_sample_workspace_bytes(n, nnz) bytes; nothing is allocated.
 * 0 < alpha <= 1.  Work is enqueued on `stream`; the call synchronises it before writing the host outputs.
 * Errors: TSID_ERR_INVALID_ARG, TSID_ERR_OOM (workspace too small), TSID_ERR_INDEX_RANGE (a column index
 * outside [0, n)), TSID_ERR_CUDA. */
tsid_status_t tsid_sample_workspace_bytes(int32_t n, int64_t nnz, size_t *h_bytes_out);
tsid_status_t tsid_sample_template(int32_t m, int32_t n, int64_t nnz, double alpha, uint64_t seed,
                                   const int32_t *d_rows, const int32_t *d_cols, const float *d_vals,
                                   void *stream, void *workspace, size_t workspace_bytes,
                                   int32_t *d_colmap, int32_t *d_rows_out, int32_t *d_cols_out,
                                   float *d_vals_out, int32_t *h_d_out, int64_t *h_nnz_out);

/* Stage II, the template-conditioned extension (Sec. 5.2, Eq. 10).  With the template estimate
 * Rhat* = P Q^T (m x d) fixed, every column j of the matrix being completed gets coefficients C_j in R^d
 * minimising  sum_{i in Omega^j} (R_ij - Rhat*_i C_j)^2 + lambda |C_j|^2  by `iters` Adam steps
 * (Kingma & Ba, Algorithm 1, bias-corrected; beta1, beta2, eps as given).  Columns are processed in
 * chunks of `chunk_cols`: the matrix and C stay in HOST memory (pinned memory makes the copies
 * asynchronous), the template factors stay on the device, and while one chunk computes the next one is
 * copied in and the previous one's coefficients are copied out.
 *   - d_P (m x k), d_Q (d x k): DEVICE, fp32 row-major, the fitted template factors; only read.
 *   - h_col_ptr (int64[n_cols + 1]), h_row_idx (int32[nnz]), h_vals (fp32[nnz]): HOST, the observed
 *     entries in column-compressed order (entries of column j at positions [col_ptr[j], col_ptr[j+1])).
 *   - h_C: HOST, fp32 [n_cols x d], column j's coefficients at h_C + j*d; read as the starting point
 *     (zeros for a cold start) and overwritten with the result.
 *   - h_sse_or_null: HOST, receives sum_Omega e^2 at the returned coefficients.
 *   - cfg.workspace: DEVICE, tsid_extend_workspace_bytes(cfg, h_col_ptr) bytes (it depends on the
 *     largest chunk); nothing is allocated on the device.  The call creates two helper streams, a few
 *     events and 64 bytes of pinned host memory (released before it returns), and synchronises before
 *     it returns.
 * Limits: k a multiple of 4 in [4, 128]; at most 2^31 - 3 entries per chunk.  Errors: INVALID_ARG,
 * UNSUPPORTED (k, or a shape TSID_EXTEND_TC does not take), OOM (workspace), INDEX_RANGE (a row index
 * outside [0, m)), CUDA (also when a bounded device-side wait of the tensor-core kernels expired). */
enum {
  TSID_EXTEND_COLD_START = 1u,   /* start from C = 0, h_C is only written */
  TSID_EXTEND_TC = 2u            /* mixed precision as in the paper's Stage II (Sec. 5.2): both products of a
                                    step (W = C Q and U Q^T) run on the tensor cores with bf16 operands and
                                    fp32 accumulation; C and the Adam moments stay fp32 (a bf16 copy of C is
                                    kept beside it).  Needs k in {64, 128}, d a multiple of 8 and >= 128
                                    (else TSID_ERR_UNSUPPORTED). */
};
typedef struct {
  int32_t m, d, k;     /* rows; template columns (rows of Q); rank                      */
  int32_t n_cols;      /* columns handled by this call                                  */
  int32_t chunk_cols;  /* chunk width (Delta c)                                         */
  int32_t iters;       /* Adam steps per chunk                                          */
  float eta, lambda, beta1, beta2, eps;
  uint32_t flags;      /* TSID_EXTEND_COLD_START | TSID_EXTEND_TC (above)                */
  void *stream;           /* compute stream (cudaStream_t) owned by the caller          */
  void *workspace;        /* DEVICE memory owned by the caller, 256-byte aligned        */
  size_t workspace_bytes;
} tsid_extend_config_t;
tsid_status_t tsid_extend_workspace_bytes(const tsid_extend_config_t *cfg, const int64_t *h_col_ptr,
                                          size_t *h_bytes_out);
tsid_status_t tsid_extend(const tsid_extend_config_t *cfg, const float *d_P, const float *d_Q,
                          const int64_t *h_col_ptr, const int32_t *h_row_idx, const float *h_vals,
                          float *h_C, double *h_sse_or_null);

/* Per-kernel timing for benchmarks.  tsid_set_profiling(t, 1) makes every following step record
 * CUDA events on the template's stream right before and after its row pass, its column pass
 * and its update kernel (at most 256 steps are kept); 0 turns it off and frees the events.
 * tsid_get_pass_times synchronises, returns the number of recorded steps and the summed
 * milliseconds of each of the three kernels over them, and restarts the recording. */
tsid_status_t tsid_set_profiling(tsid_template_t *t, int32_t enable);
/* The same with a fourth figure: h_ms4 = { row pass, column pass, update, tile passes } summed over the
 * recorded steps; the fourth is the hybrid path's tensor-core part (rank-ordered shadow copies, the two
 * tile-list passes and the two adds), 0 on the other paths. */
tsid_status_t tsid_get_step_times(tsid_template_t *t, int32_t *h_steps, float *h_ms4);
tsid_status_t tsid_get_pass_times(tsid_template_t *t, int32_t *h_steps, float *h_row_ms,
                                  float *h_col_ms, float *h_update_ms);

/* (The paper has no counterpart for this call; it exists for callers that cannot allocate.)
 * SSE = sum_Omega (r_ij - p_i . q_j)^2 of a template given as raw COO triples, with fp32 factors,
 * WITHOUT a handle, a workspace or any allocation.  It is meant for code that is handed device
 * pointers and a stream but may not create device memory: a monitoring hook inside a process
 * whose framework owns the whole GPU through its own pool, a latency-critical loop that cannot
 * afford the device-wide synchronisation an allocate/free pair brings, a plug-in with no
 * allocator access.  The partial sums the reduction needs live in a fixed 512 KiB array that is
 * part of the library image on every GPU that loads it (until the process exits).
 *   - All d_* pointers are device memory of the CURRENT device: d_rows, d_cols (int32[nnz],
 *     indices must be in range: they are not checked), d_vals (fp32[nnz]), d_P (m x k), d_Q
 *     (n x k) fp32 row-major and 16-byte aligned, k a multiple of 4 in [4, 256].  The result is
 *     written to d_sse_out (one double, device memory, 8-byte aligned) by work enqueued on
 *     `stream`; the call does not synchronise.  Residuals are fp32, squares are added in double
 *     in a fixed order (deterministic).
 *   - Limit: nnz <= 67,108,864 (65,536 partial sums of 1,024 entries).  Larger templates are
 *     refused with TSID_ERR_TOO_LARGE before anything is launched; use tsid_loss for those.
 *   - The first call on each device looks up the device address of the built-in array (a
 *     runtime query, no allocation).  Make that first call at start-up, with the device current,
 *     before any stream capture is begun on the thread.
 *   - Every call on a device uses the same array.  Calls whose GPU work can overlap (two
 *     streams, two host threads) race on it: serialise them.  The array keeps the previous
 *     call's contents, which is harmless: each call overwrites every slot it reads.
 *   - Other statuses: TSID_ERR_INVALID_ARG (null or misaligned pointer, bad size),
 *     TSID_ERR_UNSUPPORTED (k outside the limits, device ordinal above 63), TSID_ERR_CUDA. */
tsid_status_t tsid_sse_noalloc(int32_t m, int32_t n, int32_t k, int64_t nnz, const int32_t *d_rows,
                               const int32_t *d_cols, const float *d_vals, const float *d_P,
                               const float *d_Q, void *stream, double *d_sse_out);

/* Message of the last failing call on this handle (or of the last failing create when
 * t == NULL).  Never NULL; valid until the next call on the same handle / thread. */
const char *tsid_last_error(const tsid_template_t *t);

#ifdef __cplusplus
}
#endif
#endif /* TSID_H_ */
