// Host side of the C ABI declared in include/tsid.h: argument checks, workspace carving,
// and the order of kernel launches of each entry point.  No device allocation happens here.
#include <new>
#include <stdlib.h>
#include <string.h>

#include "tsid_internal.cuh"

using namespace tsid;

namespace {

thread_local char g_create_err[256] = "";

tsid_status_t fail(tsid_template *t, tsid_status_t st, const char *fmt, const char *detail = "") {
  char *dst = t ? t->err : g_create_err;
  snprintf(dst, 256, fmt, detail);
  return st;
}

tsid_status_t check_cfg(const tsid_config_t *c, char *err) {
  if (!c) { snprintf(err, 256, "cfg is null"); return TSID_ERR_INVALID_ARG; }
  if (c->m < 1 || c->n < 1 || c->nnz < 0) { snprintf(err, 256, "m, n must be >= 1 and nnz >= 0"); return TSID_ERR_INVALID_ARG; }
  if (c->nnz > 2147483647LL) { snprintf(err, 256, "nnz exceeds 2^31-1"); return TSID_ERR_UNSUPPORTED; }
  if (c->precision != TSID_F32 && c->precision != TSID_BF16_SHADOW) { snprintf(err, 256, "bad precision"); return TSID_ERR_INVALID_ARG; }
  if (c->path < TSID_PATH_AUTO || c->path > TSID_PATH_HYBRID) { snprintf(err, 256, "bad path"); return TSID_ERR_INVALID_ARG; }
  if (c->clip < TSID_CLIP_NONE || c->clip > TSID_CLIP_ASYM_ENTRY) { snprintf(err, 256, "bad clip mode"); return TSID_ERR_INVALID_ARG; }
  if (c->norm_p < 0 || c->norm_p > 1 || c->norm_q < 0 || c->norm_q > 1) { snprintf(err, 256, "bad norm mode"); return TSID_ERR_INVALID_ARG; }
  const int mult = c->precision == TSID_BF16_SHADOW ? 8 : 4;
  if (c->k < 1 || c->k > 256 || c->k % mult) { snprintf(err, 256, "k must be in [1,256] and a multiple of %d", mult); return TSID_ERR_UNSUPPORTED; }
  if (c->clip == TSID_CLIP_ASYM_ENTRY &&
      (c->path == TSID_PATH_DENSE_TC || c->path == TSID_PATH_HYBRID || (c->precision == TSID_F32 && c->k > 128))) {
    snprintf(err, 256, "entry-wise clipping runs on the sparse path only (fp32 factors: k <= 128)");
    return TSID_ERR_UNSUPPORTED;
  }
  if (c->clip != TSID_CLIP_NONE && !(c->xi > 0.f)) { snprintf(err, 256, "xi must be > 0 when clipping"); return TSID_ERR_INVALID_ARG; }
  return TSID_OK;
}

// Below this many entries AUTO does not try the hybrid path: its extra launches per step cost more than
// the tiles save.
constexpr int64_t kHybridAutoMinEntries = 4000000;

// AUTO takes the dense tensor-core variant when the template qualifies for it and at least 5 % of
// its cells are observed; the answer depends on cfg alone, so the workspace size is predictable.
int resolve_path(const tsid_config_t &c) {
  if (c.path != TSID_PATH_AUTO) return c.path;
  if (dense_qualifies(c) && c.clip != TSID_CLIP_ASYM_ENTRY && (double)c.nnz >= 0.05 * (double)c.m * (double)c.n)
    return TSID_PATH_DENSE_TC;
  if (hybrid_qualifies(c) && c.nnz >= kHybridAutoMinEntries) return TSID_PATH_HYBRID;
  return TSID_PATH_SPARSE;
}

// Carves (or, with a null base, measures) every device buffer of a template.
void carve_all(tsid_template *t, const tsid_config_t &c, Carver &cv, LayoutScratch &ls) {
  const size_t nnz = (size_t)c.nnz, k = (size_t)c.k;
  const size_t mr = (size_t)c.m, nr = (size_t)c.n;                       // sizes of the factor matrices
  const size_t m = t->vm ? (size_t)t->vm : mr, n = t->vn ? (size_t)t->vn : nr;   // sizes of the layout (virtual for mini-batches)
  const size_t nz = nnz ? nnz : 1;
  t->flags = cv.take<int32_t>(FLAG_COUNT);
  t->row_ptr = cv.take<int64_t>(m + 1);
  t->col_ptr = cv.take<int64_t>(n + 1);
  if (t->n_batches) { t->vrows = cv.take<int32_t>(nz); t->vcols = cv.take<int32_t>(nz); }
  t->col_idx = cv.take<int32_t>(nz);
  t->val_csr = cv.take<float>(nz);
  t->row_idx = cv.take<int32_t>(nz);
  t->val_csc = cv.take<float>(nz);
  t->perm = cv.take<uint32_t>(nz);
  const size_t per = nnz / kSegLen;
  Side *sides[2] = {&t->rowside, &t->colside};
  for (int i = 0; i < 2; ++i) {
    Side &sd = *sides[i];
    sd.nrows = (int32_t)(i == 0 ? m : n);
    sd.cap_seg = (int32_t)(sd.nrows + per + 1);
    sd.cap_split = (int32_t)(per + 1);
    sd.cap_slot = (int32_t)(2 * per + 2);
    sd.segs = cv.take<Segment>(sd.cap_seg);
    sd.splits = cv.take<SplitRow>(sd.cap_split);
    sd.scale = cv.take<float>(sd.nrows);
    const size_t real_rows = i == 0 ? mr : nr;
    sd.G = cv.take<float>(real_rows * k);
    sd.shadow = c.precision == TSID_BF16_SHADOW ? cv.take<__nv_bfloat16>(real_rows * k) : nullptr;
  }
  t->rowside.ptr = t->row_ptr; t->rowside.idx = t->col_idx; t->rowside.val = t->val_csr;
  t->colside.ptr = t->col_ptr; t->colside.idx = t->row_idx; t->colside.val = t->val_csc;
  if (c.flags & TSID_VALUES_U8) {
    t->rowside.val8 = cv.take<uint8_t>(nz);
    t->colside.val8 = cv.take<uint8_t>(nz);
  }
  t->partial = cv.take<float>((2 * per + 2) * k);
  t->red_cap = (int32_t)(2 + 2 * 256 + t->rowside.cap_seg);
  t->red = cv.take<double>(t->red_cap);
  if (t->path == TSID_PATH_DENSE_TC) dense_carve(t, c, cv);
  if (t->path == TSID_PATH_HYBRID) hybrid_carve(t, c, cv);
  // buffers of the layout pass (one spare slot for the scans' totals); the hybrid path keeps its tail
  // layout in four of them afterwards
  ls.kA = cv.take<uint32_t>(nz + 64); ls.kB = cv.take<uint32_t>(nz + 64);
  ls.vA = cv.take<uint32_t>(nz + 64); ls.vB = cv.take<uint32_t>(nz + 64);
  ls.wA = cv.take<uint32_t>(nz + 64); ls.wB = cv.take<uint32_t>(nz + 64);
  ls.xA = cv.take<uint32_t>(nz + 64); ls.xB = cv.take<uint32_t>(nz + 64);
  ls.hist = cv.take<uint32_t>(256 * (size_t)kSortBlocksMax);
  const size_t mx = (m > n ? m : n) + 2;
  ls.scanA = cv.take<uint32_t>(mx); ls.scanB = cv.take<uint32_t>(mx); ls.scanC = cv.take<uint32_t>(mx);
  ls.blocksums = cv.take<uint32_t>(kScanBlocksMax);
}

cudaError_t grad_any(tsid_template *t, const float *d_P, const float *d_Q, float *GP, float *GQ) {
  if (t->path == TSID_PATH_HYBRID) return hybrid_grad(t, d_P, d_Q, GP, GQ);
  return t->path == TSID_PATH_DENSE_TC ? dense_grad(t, GP, GQ) : sparse_grad(t, d_P, d_Q, GP, GQ);
}

// One step of tsid_fit on the internal gradient buffers.  The hybrid path leaves the tile passes' sums in their
// partial blocks and lets the update kernel add them (same order, same bits as hybrid_grad + sparse_update).
cudaError_t fit_step(tsid_template *t, float *P, float *Q) {
  if (t->path == TSID_PATH_HYBRID) {
    cudaError_t e = hybrid_grad_partial(t, t->rowside.G, t->colside.G);
    return e == cudaSuccess ? hybrid_update(t, P, Q, t->rowside.G, t->colside.G) : e;
  }
  cudaError_t e = grad_any(t, P, Q, t->rowside.G, t->colside.G);
  return e == cudaSuccess ? sparse_update(t, P, Q, t->rowside.G, t->colside.G) : e;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

tsid_status_t cuda_fail(tsid_template *t, cudaError_t e) {
  return fail(t, TSID_ERR_CUDA, "CUDA error: %s", cudaGetErrorString(e));
}

// Steps per captured graph: the whole call when it has 4 .. 16 epochs, else 8 (the rest launches step by
// step).  A step is three to five launches; replaying them from a graph removes the per-launch host cost
// and most of the gap between kernels, which is what bounds small templates (tens of microseconds per step)
// and still shows on the dense path (7 % of a 0.3 ms step).
constexpr int kFitGraphMin = 4, kFitGraphMax = 16, kFitGraphEpochs = 8;

void fit_graph_release(tsid_template *t) {
  if (t->fit_exec) cudaGraphExecDestroy(t->fit_exec);  // in-flight launches finish first
  if (t->fit_cap) cudaStreamDestroy(t->fit_cap);
  t->fit_exec = nullptr;
  t->fit_cap = nullptr;
  t->fit_P = t->fit_Q = nullptr;
}

// The executable graph of `steps` steps on (P, Q): the cached one, or a fresh capture.  The capture
// runs on a stream of the library's own (the caller's may be the legacy default stream, which cannot capture);
// the graph is launched into the caller's stream.
cudaError_t fit_graph_get(tsid_template *t, float *P, float *Q, int steps) {
  if (t->fit_exec && t->fit_P == P && t->fit_Q == Q && t->fit_steps == steps) return cudaSuccess;
  if (t->fit_exec) { cudaGraphExecDestroy(t->fit_exec); t->fit_exec = nullptr; }
  cudaError_t e = cudaSuccess;
  if (!t->fit_cap) e = cudaStreamCreateWithFlags(&t->fit_cap, cudaStreamNonBlocking);
  if (e != cudaSuccess) return e;
  e = cudaStreamBeginCapture(t->fit_cap, cudaStreamCaptureModeRelaxed);
  if (e != cudaSuccess) return e;
  cudaStream_t user = t->stream;
  t->stream = t->fit_cap;
  cudaError_t el = cudaSuccess;
  for (int u = 0; u < steps && el == cudaSuccess; ++u) el = fit_step(t, P, Q);
  t->stream = user;
  cudaGraph_t g = nullptr;
  e = cudaStreamEndCapture(t->fit_cap, &g);
  if (el != cudaSuccess) e = el;
  if (e == cudaSuccess) e = cudaGraphInstantiate(&t->fit_exec, g, 0);
  if (g) cudaGraphDestroy(g);
  if (e != cudaSuccess) { t->fit_exec = nullptr; return e; }
  t->fit_P = P;
  t->fit_Q = Q;
  t->fit_steps = steps;
  return cudaSuccess;
}

tsid_status_t check_factors(tsid_template *t, const float *P, const float *Q, bool batch_call = false) {
  if (!t) return TSID_ERR_INVALID_ARG;
  if (t->n_batches && !batch_call)
    return fail(t, TSID_ERR_UNSUPPORTED, "a mini-batch template is stepped with tsid_grad_step_batch only");
  if (!P || !Q) return fail(t, TSID_ERR_INVALID_ARG, "P or Q is null");
  if (!aligned16(P) || !aligned16(Q)) return fail(t, TSID_ERR_INVALID_ARG, "P and Q must be 16-byte aligned");
  return TSID_OK;
}

}  // namespace

extern "C" {

tsid_status_t tsid_workspace_bytes(const tsid_config_t *cfg, size_t *h_bytes_out) {
  if (!h_bytes_out) return fail(nullptr, TSID_ERR_INVALID_ARG, "bytes_out is null");
  tsid_status_t st = check_cfg(cfg, g_create_err);
  if (st != TSID_OK) return st;
  tsid_template tmp;
  memset(static_cast<void *>(&tmp), 0, sizeof(tmp));
  tmp.path = resolve_path(*cfg);
  if (tmp.path == TSID_PATH_DENSE_TC && !dense_qualifies(*cfg)) {
    snprintf(g_create_err, 256, "dense path needs bf16 shadows, k in {64, 128}, m and n multiples of 128");
    return TSID_ERR_UNSUPPORTED;
  }
  if (tmp.path == TSID_PATH_HYBRID && !hybrid_qualifies(*cfg)) {
    snprintf(g_create_err, 256, "hybrid path needs bf16 shadows, k in {64, 128}, no entry-wise clip or byte values, "
                                "and at least max(m, n, ceil(m/128) * ceil(n/128)) entries");
    return TSID_ERR_UNSUPPORTED;
  }
  Carver cv(nullptr);
  LayoutScratch ls;
  carve_all(&tmp, *cfg, cv, ls);
  *h_bytes_out = cv.off;
  return TSID_OK;
}

tsid_status_t tsid_template_create(const tsid_config_t *cfg, const int32_t *d_rows, const int32_t *d_cols,
                                   const float *d_vals, tsid_template_t **out) {
  if (!out) return fail(nullptr, TSID_ERR_INVALID_ARG, "out is null");
  *out = nullptr;
  tsid_status_t st = check_cfg(cfg, g_create_err);
  if (st != TSID_OK) return st;
  if (cfg->nnz > 0 && (!d_rows || !d_cols || !d_vals)) return fail(nullptr, TSID_ERR_INVALID_ARG, "COO pointer is null");
  if (!cfg->workspace || (reinterpret_cast<uintptr_t>(cfg->workspace) & 255u))
    return fail(nullptr, TSID_ERR_INVALID_ARG, "workspace is null or not 256-byte aligned");
  size_t need = 0;
  tsid_workspace_bytes(cfg, &need);
  if (cfg->workspace_bytes < need) return fail(nullptr, TSID_ERR_OOM, "workspace smaller than tsid_workspace_bytes");
  const int path = resolve_path(*cfg);

  tsid_template *t = new (std::nothrow) tsid_template;
  if (!t) return fail(nullptr, TSID_ERR_OOM, "host allocation failed");
  memset(static_cast<void *>(t), 0, sizeof(*t));
  t->cfg = *cfg;
  t->stream = static_cast<cudaStream_t>(cfg->stream);
  t->path = path;
  if (path == TSID_PATH_DENSE_TC) {
    t->dense = dense_new();
    if (!t->dense) { delete t; return fail(nullptr, TSID_ERR_OOM, "host allocation failed"); }
  }
  if (path == TSID_PATH_HYBRID) {
    t->hybrid = hybrid_new();
    if (!t->hybrid) { delete t; return fail(nullptr, TSID_ERR_OOM, "host allocation failed"); }
  }
  Carver cv(cfg->workspace);
  LayoutScratch ls;
  carve_all(t, *cfg, cv, ls);

  int32_t hf[FLAG_COUNT] = {0};
  cudaError_t e = layout_build(t, d_rows, d_cols, d_vals, ls, hf);
  if (e != cudaSuccess) { st = cuda_fail(nullptr, e); delete t; return st; }
  if (hf[FLAG_RANGE]) { delete t; return fail(nullptr, TSID_ERR_INDEX_RANGE, "a row or column index is out of range"); }
  if (hf[FLAG_UNSORTED] && (cfg->flags & TSID_INPUT_ROW_SORTED)) { delete t; return fail(nullptr, TSID_ERR_UNSORTED, "input promised row-sorted but is not"); }
  if (hf[FLAG_DUP] && (cfg->flags & TSID_VALIDATE)) { delete t; return fail(nullptr, TSID_ERR_DUPLICATE, "duplicate (row, col) in Omega"); }
  e = build_segments(t, t->rowside, cfg->norm_p, ls);
  if (e == cudaSuccess) e = build_segments(t, t->colside, cfg->norm_q, ls);
  if (e != cudaSuccess) { st = cuda_fail(nullptr, e); tsid_destroy(t); return st; }
  if (cfg->flags & TSID_VALUES_U8) {
    int32_t bad = 0;
    e = sparse_pack_values_u8(t, &bad);
    if (e != cudaSuccess) { st = cuda_fail(nullptr, e); tsid_destroy(t); return st; }
    if (bad) { tsid_destroy(t); return fail(nullptr, TSID_ERR_UNSUPPORTED, "TSID_VALUES_U8 promised but a value is not an integer in [0, 255]"); }
  }
  if (path == TSID_PATH_DENSE_TC) {
    // a dense cell holds one value: a template that lists a cell twice cannot run here (the loss, the counts and
    // the sparse passes would count both occurrences, the dense matrix only one)
    int32_t dup = 0;
    e = csr_has_duplicates(t, &dup);
    if (e != cudaSuccess) { st = cuda_fail(nullptr, e); tsid_destroy(t); return st; }
    if (dup) { tsid_destroy(t); return fail(nullptr, TSID_ERR_DUPLICATE, "the dense path cannot hold a (row, col) that occurs twice"); }
    int32_t bad = 0;
    e = dense_build(t, &bad);
    if (e != cudaSuccess) { st = cuda_fail(nullptr, e); tsid_destroy(t); return st; }
    if (bad) { tsid_destroy(t); return fail(nullptr, TSID_ERR_UNSUPPORTED, "a value is outside the fp16 range of the dense path"); }
  }
  if (path == TSID_PATH_HYBRID) {
    int32_t fallback = 0;
    e = hybrid_build(t, ls, &fallback);
    if (e != cudaSuccess) { st = cuda_fail(nullptr, e); tsid_destroy(t); return st; }
    if (fallback) t->path = TSID_PATH_SPARSE;   // no tile worth storing (or duplicates, or a value beyond fp16)
  }
  snprintf(t->err, 256, "ok");
  *out = t;
  return TSID_OK;
}

tsid_status_t tsid_grad_step(tsid_template_t *t, float *d_P, float *d_Q, float *d_gradP_or_null,
                             float *d_gradQ_or_null) {
  tsid_status_t st = check_factors(t, d_P, d_Q);
  if (st != TSID_OK) return st;
  if ((d_gradP_or_null && !aligned16(d_gradP_or_null)) || (d_gradQ_or_null && !aligned16(d_gradQ_or_null)))
    return fail(t, TSID_ERR_INVALID_ARG, "gradient outputs must be 16-byte aligned");
  float *GP = d_gradP_or_null ? d_gradP_or_null : t->rowside.G;
  float *GQ = d_gradQ_or_null ? d_gradQ_or_null : t->colside.G;
  cudaError_t e = sparse_convert_shadow(t, d_P, d_Q);
  if (e == cudaSuccess) e = grad_any(t, d_P, d_Q, GP, GQ);
  if (e == cudaSuccess) e = sparse_update(t, d_P, d_Q, GP, GQ);
  return e == cudaSuccess ? TSID_OK : cuda_fail(t, e);
}

tsid_status_t tsid_grad(tsid_template_t *t, const float *d_P, const float *d_Q, float *d_GP, float *d_GQ) {
  tsid_status_t st = check_factors(t, d_P, d_Q);
  if (st != TSID_OK) return st;
  if (!d_GP || !d_GQ || !aligned16(d_GP) || !aligned16(d_GQ))
    return fail(t, TSID_ERR_INVALID_ARG, "gradient outputs must be non-null and 16-byte aligned");
  cudaError_t e = sparse_convert_shadow(t, d_P, d_Q);
  if (e == cudaSuccess) e = grad_any(t, d_P, d_Q, d_GP, d_GQ);
  return e == cudaSuccess ? TSID_OK : cuda_fail(t, e);
}

tsid_status_t tsid_apply(tsid_template_t *t, float *d_P, float *d_Q, const float *d_GP, const float *d_GQ) {
  tsid_status_t st = check_factors(t, d_P, d_Q);
  if (st != TSID_OK) return st;
  if (!d_GP || !d_GQ || !aligned16(d_GP) || !aligned16(d_GQ))
    return fail(t, TSID_ERR_INVALID_ARG, "gradient inputs must be non-null and 16-byte aligned");
  cudaError_t e = sparse_update(t, d_P, d_Q, d_GP, d_GQ);
  return e == cudaSuccess ? TSID_OK : cuda_fail(t, e);
}

tsid_status_t tsid_apply_sliced(tsid_template_t *t, float *d_P, const float *d_GP, float *const *h_Q_replicas,
                                const float *const *h_GQ_parts, int32_t rank, int32_t world) {
  if (!t) return TSID_ERR_INVALID_ARG;
  if (t->n_batches) return fail(t, TSID_ERR_UNSUPPORTED, "not for a mini-batch template");
  if (!d_P || !d_GP || !h_Q_replicas || !h_GQ_parts || !aligned16(d_P) || !aligned16(d_GP))
    return fail(t, TSID_ERR_INVALID_ARG, "P, G_P and the pointer arrays must be non-null (P, G_P 16-byte aligned)");
  if (world < 1 || world > kMaxRanks || rank < 0 || rank >= world)
    return fail(t, TSID_ERR_INVALID_ARG, "need 1 <= world <= 16 and 0 <= rank < world");
  for (int r = 0; r < world; ++r)
    if (!h_Q_replicas[r] || !h_GQ_parts[r] || !aligned16(h_Q_replicas[r]) || !aligned16(h_GQ_parts[r]))
      return fail(t, TSID_ERR_INVALID_ARG, "every Q replica and G_Q part must be a non-null, 16-byte aligned device pointer");
  cudaError_t e = sparse_apply_sliced(t, d_P, d_GP, h_Q_replicas, h_GQ_parts, rank, world);
  return e == cudaSuccess ? TSID_OK : cuda_fail(t, e);
}

tsid_status_t tsid_get_counts(tsid_template_t *t, int32_t *d_cnt_p_or_null, int32_t *d_cnt_q_or_null) {
  if (!t) return TSID_ERR_INVALID_ARG;
  if (t->n_batches) return fail(t, TSID_ERR_UNSUPPORTED, "not for a mini-batch template");
  cudaError_t e = cudaSuccess;
  if (d_cnt_p_or_null) e = sparse_counts(t, t->rowside, d_cnt_p_or_null);
  if (e == cudaSuccess && d_cnt_q_or_null) e = sparse_counts(t, t->colside, d_cnt_q_or_null);
  return e == cudaSuccess ? TSID_OK : cuda_fail(t, e);
}

tsid_status_t tsid_set_norm_counts(tsid_template_t *t, const int32_t *d_cnt_p_or_null, const int32_t *d_cnt_q_or_null) {
  if (!t) return TSID_ERR_INVALID_ARG;
  if (t->n_batches) return fail(t, TSID_ERR_UNSUPPORTED, "not for a mini-batch template");
  cudaError_t e = cudaSuccess;
  if (d_cnt_p_or_null) e = sparse_scale_from_counts(t, t->rowside, t->cfg.norm_p, d_cnt_p_or_null);
  if (e == cudaSuccess && d_cnt_q_or_null) e = sparse_scale_from_counts(t, t->colside, t->cfg.norm_q, d_cnt_q_or_null);
  return e == cudaSuccess ? TSID_OK : cuda_fail(t, e);
}

static tsid_status_t loss_sync(tsid_template *t, const float *d_P, const float *d_Q, double *sse, double *sq) {
  cudaError_t e = sparse_loss(t, d_P, d_Q, t->red);
  double h[2] = {0, 0};
  if (e == cudaSuccess) e = cudaMemcpyAsync(h, t->red, 2 * sizeof(double), cudaMemcpyDeviceToHost, t->stream);
  int32_t hf[FLAG_COUNT] = {0};
  if (e == cudaSuccess) e = cudaMemcpyAsync(hf, t->flags, sizeof(hf), cudaMemcpyDeviceToHost, t->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(t->stream);
  if (e != cudaSuccess) return cuda_fail(t, e);
  *sse = h[0];
  *sq = h[1];
  if (hf[FLAG_TIMEOUT]) return fail(t, TSID_ERR_CUDA, "a bounded device-side wait expired ");
  if (hf[FLAG_NONFINITE] || !(h[0] == h[0]) || !(h[1] == h[1]))
    return fail(t, TSID_ERR_NONFINITE, "a factor became non-finite");
  return TSID_OK;
}

tsid_status_t tsid_fit(tsid_template_t *t, float *d_P, float *d_Q, int32_t epochs, int32_t loss_every,
                       double *h_sse_history_or_null) {
  tsid_status_t st = check_factors(t, d_P, d_Q);
  if (st != TSID_OK) return st;
  if (epochs < 0 || loss_every < 0) return fail(t, TSID_ERR_INVALID_ARG, "epochs and loss_every must be >= 0");
  int nh = 0;
  double sse, sq;
  if (loss_every > 0) {
    st = loss_sync(t, d_P, d_Q, &sse, &sq);
    if (h_sse_history_or_null) h_sse_history_or_null[nh] = sse;
    ++nh;
    if (st != TSID_OK) return st;
  }
  cudaError_t e = sparse_convert_shadow(t, d_P, d_Q);
  if (e == cudaSuccess && t->path == TSID_PATH_HYBRID) e = hybrid_refresh_ranked(t);
  int ep = 0;
  // a caller that is capturing cfg.stream into a graph of its own gets plain launches
  cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
  if (e == cudaSuccess && cudaStreamIsCapturing(t->stream, &capturing) != cudaSuccess) {
    cudaGetLastError();
    capturing = cudaStreamCaptureStatusActive;
  }
  if (e == cudaSuccess && loss_every == 0 && !t->prof.on && !t->fit_graph_off && epochs >= kFitGraphMin &&
      capturing == cudaStreamCaptureStatusNone) {
    const int per = epochs <= kFitGraphMax ? epochs : kFitGraphEpochs;
    if (fit_graph_get(t, d_P, d_Q, per) == cudaSuccess) {
      for (; ep + per <= epochs && e == cudaSuccess; ep += per) e = cudaGraphLaunch(t->fit_exec, t->stream);
    } else {
      cudaGetLastError();  // the capture's error is not the call's: the steps below launch one by one
      t->fit_graph_off = true;
    }
  }
  for (; ep < epochs && e == cudaSuccess; ++ep) {
    // the update kernel refreshes the shadows, so they stay current between epochs
    e = fit_step(t, d_P, d_Q);
    if (e == cudaSuccess && loss_every > 0 && (ep + 1) % loss_every == 0) {
      st = loss_sync(t, d_P, d_Q, &sse, &sq);
      if (h_sse_history_or_null) h_sse_history_or_null[nh] = sse;
      ++nh;
      if (st != TSID_OK) return st;
    }
  }
  return e == cudaSuccess ? TSID_OK : cuda_fail(t, e);
}

tsid_status_t tsid_loss(tsid_template_t *t, const float *d_P, const float *d_Q, double *h_sse, double *h_objective) {
  tsid_status_t st = check_factors(t, d_P, d_Q);
  if (st != TSID_OK) return st;
  double sse = 0, sq = 0;
  st = loss_sync(t, d_P, d_Q, &sse, &sq);
  if (h_sse) *h_sse = sse;
  if (h_objective) *h_objective = sse + (double)t->cfg.lambda * sq;
  return st;
}

tsid_status_t tsid_check(tsid_template_t *t) {
  if (!t) return TSID_ERR_INVALID_ARG;
  int32_t hf[FLAG_COUNT] = {0};
  cudaError_t e = cudaMemcpyAsync(hf, t->flags, sizeof(hf), cudaMemcpyDeviceToHost, t->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(t->stream);
  if (e != cudaSuccess) return cuda_fail(t, e);
  if (hf[FLAG_TIMEOUT]) return fail(t, TSID_ERR_CUDA, "a bounded device-side wait expired ");
  if (hf[FLAG_NONFINITE]) return fail(t, TSID_ERR_NONFINITE, "a factor became non-finite");
  return TSID_OK;
}

static void prof_release(tsid_template *t) {
  if (t->prof.ev) {
    for (int i = 0; i < kProfSteps * EV_PER_STEP; ++i) cudaEventDestroy(t->prof.ev[i]);
    delete[] t->prof.ev;
    t->prof.ev = nullptr;
  }
  t->prof.on = false;
  t->prof.nsteps = 0;
}

tsid_status_t tsid_destroy(tsid_template_t *t) {
  if (t) { prof_release(t); fit_graph_release(t); dense_delete(t->dense); hybrid_delete(t->hybrid); free(t->bseg_row); }
  delete t;
  return TSID_OK;
}

tsid_status_t tsid_set_profiling(tsid_template_t *t, int32_t enable) {
  if (!t) return TSID_ERR_INVALID_ARG;
  if (!enable) { prof_release(t); return TSID_OK; }
  if (!t->prof.ev) {
    t->prof.ev = new (std::nothrow) cudaEvent_t[kProfSteps * EV_PER_STEP];
    if (!t->prof.ev) return fail(t, TSID_ERR_OOM, "host allocation failed");
    for (int i = 0; i < kProfSteps * EV_PER_STEP; ++i) {
      cudaError_t e = cudaEventCreate(&t->prof.ev[i]);
      if (e != cudaSuccess) return cuda_fail(t, e);
    }
  }
  t->prof.on = true;
  t->prof.nsteps = 0;
  return TSID_OK;
}

tsid_status_t tsid_get_step_times(tsid_template_t *t, int32_t *h_steps, float *h_ms4) {
  if (!t) return TSID_ERR_INVALID_ARG;
  if (!t->prof.on) return fail(t, TSID_ERR_INVALID_ARG, "profiling is off");
  cudaError_t e = cudaStreamSynchronize(t->stream);
  if (e != cudaSuccess) return cuda_fail(t, e);
  double acc[4] = {0, 0, 0, 0};
  const int nq = t->path == TSID_PATH_HYBRID ? 4 : 3;   // the fourth pair brackets the tile passes of the hybrid path
  for (int sidx = 0; sidx < t->prof.nsteps; ++sidx) {
    for (int q = 0; q < nq; ++q) {
      float ms = 0.f;
      e = cudaEventElapsedTime(&ms, t->prof.ev[sidx * EV_PER_STEP + 2 * q], t->prof.ev[sidx * EV_PER_STEP + 2 * q + 1]);
      if (e != cudaSuccess) return cuda_fail(t, e);
      acc[q] += ms;
    }
  }
  if (h_steps) *h_steps = t->prof.nsteps;
  if (h_ms4) for (int q = 0; q < 4; ++q) h_ms4[q] = (float)acc[q];
  t->prof.nsteps = 0;
  return TSID_OK;
}

tsid_status_t tsid_get_pass_times(tsid_template_t *t, int32_t *h_steps, float *h_row_ms, float *h_col_ms,
                                  float *h_update_ms) {
  float ms[4] = {0.f, 0.f, 0.f, 0.f};
  tsid_status_t st = tsid_get_step_times(t, h_steps, ms);
  if (st != TSID_OK) return st;
  if (h_row_ms) *h_row_ms = ms[0];
  if (h_col_ms) *h_col_ms = ms[1];
  if (h_update_ms) *h_update_ms = ms[2];
  return TSID_OK;
}

// Device memory the host-buffer call needs: the template's own workspace, then the staged COO
// triples and the two factor matrices.
static size_t host_extra_bytes(const tsid_config_t &c) {
  Carver cv(nullptr);
  const size_t nz = c.nnz ? (size_t)c.nnz : 1;
  cv.take<int32_t>(nz); cv.take<int32_t>(nz); cv.take<float>(nz);
  cv.take<float>((size_t)c.m * c.k); cv.take<float>((size_t)c.n * c.k);
  return cv.off;
}

tsid_status_t tsid_workspace_bytes_host(const tsid_config_t *cfg, size_t *h_bytes_out) {
  size_t base = 0;
  tsid_status_t st = tsid_workspace_bytes(cfg, &base);
  if (st != TSID_OK) return st;
  *h_bytes_out = base + host_extra_bytes(*cfg);
  return TSID_OK;
}

tsid_status_t tsid_fit_host(const tsid_config_t *cfg, const int32_t *h_rows, const int32_t *h_cols,
                            const float *h_vals, float *h_P, float *h_Q, int32_t epochs, double *h_sse_or_null) {
  size_t base = 0, total = 0;
  tsid_status_t st = tsid_workspace_bytes(cfg, &base);
  if (st != TSID_OK) return st;
  tsid_workspace_bytes_host(cfg, &total);
  if (!h_P || !h_Q || (cfg->nnz > 0 && (!h_rows || !h_cols || !h_vals)))
    return fail(nullptr, TSID_ERR_INVALID_ARG, "host pointer is null");
  if (epochs < 0) return fail(nullptr, TSID_ERR_INVALID_ARG, "epochs must be >= 0");
  if (!cfg->workspace || (reinterpret_cast<uintptr_t>(cfg->workspace) & 255u))
    return fail(nullptr, TSID_ERR_INVALID_ARG, "workspace is null or not 256-byte aligned");
  if (cfg->workspace_bytes < total) return fail(nullptr, TSID_ERR_OOM, "workspace smaller than tsid_workspace_bytes_host");
  cudaStream_t s = static_cast<cudaStream_t>(cfg->stream);
  Carver cv(static_cast<char *>(cfg->workspace) + base);
  const size_t nnz = (size_t)cfg->nnz, nz = nnz ? nnz : 1;
  int32_t *d_rows = cv.take<int32_t>(nz), *d_cols = cv.take<int32_t>(nz);
  float *d_vals = cv.take<float>(nz);
  const size_t pb = (size_t)cfg->m * cfg->k * sizeof(float), qb = (size_t)cfg->n * cfg->k * sizeof(float);
  float *d_P = cv.take<float>(pb / 4), *d_Q = cv.take<float>(qb / 4);
  cudaError_t e = cudaSuccess;
  if (nnz) {
    e = cudaMemcpyAsync(d_rows, h_rows, nnz * 4, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d_cols, h_cols, nnz * 4, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d_vals, h_vals, nnz * 4, cudaMemcpyHostToDevice, s);
  }
  // The factors travel on a second stream, behind the triples on the bus but beside the layout pass on
  // the device: the layout only needs the triples.
  cudaStream_t s2 = nullptr;
  cudaEvent_t coo_in = nullptr, fac_in = nullptr;
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&s2, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&coo_in, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&fac_in, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventRecord(coo_in, s);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(s2, coo_in, 0);
  if (e == cudaSuccess) e = cudaMemcpyAsync(d_P, h_P, pb, cudaMemcpyHostToDevice, s2);
  if (e == cudaSuccess) e = cudaMemcpyAsync(d_Q, h_Q, qb, cudaMemcpyHostToDevice, s2);
  if (e == cudaSuccess) e = cudaEventRecord(fac_in, s2);
  auto release = [&]() {
    if (s2) { cudaStreamSynchronize(s2); cudaStreamDestroy(s2); }
    if (coo_in) cudaEventDestroy(coo_in);
    if (fac_in) cudaEventDestroy(fac_in);
  };
  if (e != cudaSuccess) { release(); return cuda_fail(nullptr, e); }
  tsid_config_t c2 = *cfg;
  c2.workspace_bytes = base;
  tsid_template *t = nullptr;
  st = tsid_template_create(&c2, d_rows, d_cols, d_vals, &t);
  if (st != TSID_OK) { release(); return st; }
  e = cudaStreamWaitEvent(s, fac_in, 0);
  if (e != cudaSuccess) { release(); tsid_destroy(t); return cuda_fail(nullptr, e); }
  st = tsid_fit(t, d_P, d_Q, epochs, 0, nullptr);
  if (st == TSID_OK && h_sse_or_null) st = tsid_loss(t, d_P, d_Q, h_sse_or_null, nullptr);
  if (st == TSID_OK) {
    e = cudaMemcpyAsync(h_P, d_P, pb, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h_Q, d_Q, qb, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) st = tsid_check(t);
    if (e != cudaSuccess) st = cuda_fail(nullptr, e);
  }
  if (st != TSID_OK) snprintf(g_create_err, 256, "%s", t->err);
  tsid_destroy(t);
  release();
  return st;
}

tsid_status_t tsid_get_layout(tsid_template_t *t, const int64_t **d_row_ptr, const int32_t **d_col_idx,
                              const float **d_val_csr, const int64_t **d_col_ptr, const int32_t **d_row_idx,
                              const float **d_val_csc, const uint32_t **d_perm) {
  if (!t) return TSID_ERR_INVALID_ARG;
  if (d_row_ptr) *d_row_ptr = t->row_ptr;
  if (d_col_idx) *d_col_idx = t->col_idx;
  if (d_val_csr) *d_val_csr = t->val_csr;
  if (d_col_ptr) *d_col_ptr = t->col_ptr;
  if (d_row_idx) *d_row_idx = t->row_idx;
  if (d_val_csc) *d_val_csc = t->val_csc;
  if (d_perm) *d_perm = t->perm;
  return TSID_OK;
}

tsid_status_t tsid_residuals(tsid_template_t *t, const float *d_P, const float *d_Q, float *d_e_csr) {
  tsid_status_t st = check_factors(t, d_P, d_Q);
  if (st != TSID_OK) return st;
  if (!d_e_csr && t->cfg.nnz > 0) return fail(t, TSID_ERR_INVALID_ARG, "e output is null");
  cudaError_t e = sparse_residuals(t, d_P, d_Q, d_e_csr);
  return e == cudaSuccess ? TSID_OK : cuda_fail(t, e);
}

tsid_status_t tsid_get_info(const tsid_template_t *t, int32_t *h_path, int32_t *h_launches_per_step) {
  if (!t) return TSID_ERR_INVALID_ARG;
  if (h_path) *h_path = t->path;
  if (h_launches_per_step) {
    if (t->path == TSID_PATH_HYBRID) *h_launches_per_step = 1 + hybrid_launches_per_step(t) + 1;   // + shadow refresh, update
    else *h_launches_per_step = t->path == TSID_PATH_DENSE_TC ? dense_launches_per_step(t) : sparse_launches_per_step(t);
  }
  return TSID_OK;
}

tsid_status_t tsid_get_fit_launches(const tsid_template_t *t, int32_t epochs, int64_t *h_launches) {
  if (!t || !h_launches || epochs < 0) return TSID_ERR_INVALID_ARG;
  const int64_t shadow = t->cfg.precision == TSID_BF16_SHADOW ? 1 : 0;
  if (t->path == TSID_PATH_HYBRID) *h_launches = shadow + 1 + (int64_t)epochs * (hybrid_launches_per_fit_step(t) + 2);   // one update launch per side
  else if (t->path == TSID_PATH_DENSE_TC) *h_launches = shadow + (int64_t)epochs * (dense_launches_per_step(t) - shadow);
  else *h_launches = shadow + (int64_t)epochs * (sparse_launches_per_step(t) - shadow);
  return TSID_OK;
}

tsid_status_t tsid_debug_stall_tile_pass(tsid_template_t *t, int64_t wait_cycles, int32_t item) {
  if (!t) return TSID_ERR_INVALID_ARG;
  if (t->path != TSID_PATH_DENSE_TC) return fail(t, TSID_ERR_UNSUPPORTED, "only handles on the dense tensor-core path have bounded waits");
  if (wait_cycles < 0 || item < 0) return fail(t, TSID_ERR_INVALID_ARG, "wait_cycles and item must be >= 0");
  t->dbg_wait_cycles = wait_cycles;
  t->dbg_stall_item = item;
  fit_graph_release(t);   // a captured graph holds the old launch parameters
  return TSID_OK;
}

// ---- mini-batch template -----------------------------------------------------------------------------
static tsid_status_t check_batched(const tsid_config_t *cfg, int32_t n_batches, char *err) {
  tsid_status_t st = check_cfg(cfg, err);
  if (st != TSID_OK) return st;
  if (n_batches < 1 || n_batches > 65536) { snprintf(err, 256, "n_batches must be in [1, 65536]"); return TSID_ERR_INVALID_ARG; }
  if (cfg->path == TSID_PATH_DENSE_TC || cfg->path == TSID_PATH_HYBRID || (cfg->flags & TSID_VALUES_U8)) {
    snprintf(err, 256, "a mini-batch template runs the sparse path with fp32 value streams");
    return TSID_ERR_UNSUPPORTED;
  }
  if ((int64_t)cfg->m * n_batches > 2147483647LL || (int64_t)cfg->n * n_batches > 2147483647LL) {
    snprintf(err, 256, "n_batches * m and n_batches * n must stay below 2^31");
    return TSID_ERR_UNSUPPORTED;
  }
  return TSID_OK;
}

tsid_status_t tsid_workspace_bytes_batched(const tsid_config_t *cfg, int32_t n_batches, size_t *h_bytes_out) {
  if (!h_bytes_out) return fail(nullptr, TSID_ERR_INVALID_ARG, "bytes_out is null");
  tsid_status_t st = check_batched(cfg, n_batches, g_create_err);
  if (st != TSID_OK) return st;
  tsid_template tmp;
  memset(static_cast<void *>(&tmp), 0, sizeof(tmp));
  tmp.path = TSID_PATH_SPARSE;
  tmp.n_batches = n_batches; tmp.vm = cfg->m * n_batches; tmp.vn = cfg->n * n_batches;
  Carver cv(nullptr);
  LayoutScratch ls;
  carve_all(&tmp, *cfg, cv, ls);
  *h_bytes_out = cv.off;
  return TSID_OK;
}

tsid_status_t tsid_template_create_batched(const tsid_config_t *cfg, const int32_t *d_rows, const int32_t *d_cols,
                                           const float *d_vals, const int32_t *d_batch, int32_t n_batches,
                                           tsid_template_t **out) {
  if (!out) return fail(nullptr, TSID_ERR_INVALID_ARG, "out is null");
  *out = nullptr;
  tsid_status_t st = check_batched(cfg, n_batches, g_create_err);
  if (st != TSID_OK) return st;
  if (cfg->nnz > 0 && (!d_rows || !d_cols || !d_vals || !d_batch)) return fail(nullptr, TSID_ERR_INVALID_ARG, "COO or batch pointer is null");
  if (!cfg->workspace || (reinterpret_cast<uintptr_t>(cfg->workspace) & 255u))
    return fail(nullptr, TSID_ERR_INVALID_ARG, "workspace is null or not 256-byte aligned");
  size_t need = 0;
  tsid_workspace_bytes_batched(cfg, n_batches, &need);
  if (cfg->workspace_bytes < need) return fail(nullptr, TSID_ERR_OOM, "workspace smaller than tsid_workspace_bytes_batched");
  tsid_template *t = new (std::nothrow) tsid_template;
  int32_t *hb = static_cast<int32_t *>(malloc(sizeof(int32_t) * 4 * ((size_t)n_batches + 1)));
  if (!t || !hb) { delete t; free(hb); return fail(nullptr, TSID_ERR_OOM, "host allocation failed"); }
  memset(static_cast<void *>(t), 0, sizeof(*t));
  t->cfg = *cfg;
  t->cfg.flags &= ~(uint32_t)TSID_INPUT_ROW_SORTED;   // the promise is about (row, col); the layout sorts (batch, row, col)
  t->stream = static_cast<cudaStream_t>(cfg->stream);
  t->path = TSID_PATH_SPARSE;
  t->n_batches = n_batches; t->vm = cfg->m * n_batches; t->vn = cfg->n * n_batches;
  t->bseg_row = hb; t->bseg_col = hb + (n_batches + 1); t->bsplit_row = hb + 2 * (n_batches + 1); t->bsplit_col = hb + 3 * (n_batches + 1);
  Carver cv(cfg->workspace);
  LayoutScratch ls;
  carve_all(t, t->cfg, cv, ls);
  int32_t hf[FLAG_COUNT] = {0};
  cudaError_t e = batch_virtual_coo(t, d_rows, d_cols, d_batch);
  if (e == cudaSuccess) e = layout_build(t, t->vrows, t->vcols, d_vals, ls, hf);
  if (e != cudaSuccess) { st = cuda_fail(nullptr, e); tsid_destroy(t); return st; }
  if (hf[FLAG_RANGE]) { tsid_destroy(t); return fail(nullptr, TSID_ERR_INDEX_RANGE, "a row, column or batch index is out of range"); }
  if (hf[FLAG_DUP] && (cfg->flags & TSID_VALIDATE)) { tsid_destroy(t); return fail(nullptr, TSID_ERR_DUPLICATE, "duplicate (batch, row, col)"); }
  e = build_segments(t, t->rowside, cfg->norm_p, ls);
  if (e == cudaSuccess) e = batch_ranges(t, ls, false);
  if (e == cudaSuccess) e = build_segments(t, t->colside, cfg->norm_q, ls);
  if (e == cudaSuccess) e = batch_ranges(t, ls, true);
  if (e != cudaSuccess) { st = cuda_fail(nullptr, e); tsid_destroy(t); return st; }
  snprintf(t->err, 256, "ok");
  *out = t;
  return TSID_OK;
}

tsid_status_t tsid_grad_step_batch(tsid_template_t *t, int32_t batch, float *d_P, float *d_Q, float *d_gradP_or_null,
                                   float *d_gradQ_or_null) {
  tsid_status_t st = check_factors(t, d_P, d_Q, true);
  if (st != TSID_OK) return st;
  if (!t->n_batches) return fail(t, TSID_ERR_UNSUPPORTED, "not a mini-batch template");
  if (batch < 0 || batch >= t->n_batches) return fail(t, TSID_ERR_INVALID_ARG, "batch out of range");
  if ((d_gradP_or_null && !aligned16(d_gradP_or_null)) || (d_gradQ_or_null && !aligned16(d_gradQ_or_null)))
    return fail(t, TSID_ERR_INVALID_ARG, "gradient outputs must be 16-byte aligned");
  float *GP = d_gradP_or_null ? d_gradP_or_null : t->rowside.G;
  float *GQ = d_gradQ_or_null ? d_gradQ_or_null : t->colside.G;
  cudaError_t e = sparse_batch_step(t, batch, d_P, d_Q, GP, GQ);
  return e == cudaSuccess ? TSID_OK : cuda_fail(t, e);
}

tsid_status_t tsid_get_hybrid_info(const tsid_template_t *t, int64_t *h_tiles, int32_t *h_min_tile_entries,
                                   int64_t *h_tail_entries) {
  if (!t) return TSID_ERR_INVALID_ARG;
  int64_t tiles = 0, tail = t->cfg.nnz;
  int32_t mine = 0;
  if (t->path == TSID_PATH_HYBRID) hybrid_info(t, &tiles, &mine, &tail);
  if (h_tiles) *h_tiles = tiles;
  if (h_min_tile_entries) *h_min_tile_entries = mine;
  if (h_tail_entries) *h_tail_entries = tail;
  return TSID_OK;
}

const char *tsid_last_error(const tsid_template_t *t) { return t ? t->err : g_create_err; }

}  // extern "C"
