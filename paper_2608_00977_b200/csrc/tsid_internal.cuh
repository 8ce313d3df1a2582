// Internal declarations shared by the translation units of libtsid (host side of the
// C ABI, layout pass, sparse passes, dense tensor-core variant).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stdio.h>

#include "../../include/tsid.h"

namespace tsid {

// Longest run of entries one warp reduces in registers before the result goes through the
// grid-level (fixed order) reduction.  Also the unit of load balance under skewed degrees
// (measured on the 1e9-entry template: 512 is 1 - 2 % faster than 1024, 256 and 4096 are slower).
constexpr int kSegLen = 512;

// One unit of work of a gather-reduce pass: `len` consecutive entries of one row (CSR pass)
// or one column (CSC pass).  slot < 0: the row has a single segment and the warp writes the
// gradient row directly; slot >= 0: index of the partial row the fix-up kernel sums later.
struct __align__(16) Segment {
  int32_t row;
  uint32_t begin;
  int32_t len;
  int32_t slot;
};

// A row (column) that spans several segments: partial rows [slot0, slot0 + nseg).
struct __align__(16) SplitRow {
  int32_t row;
  int32_t slot0;
  int32_t nseg;
  int32_t pad;
};

// One side (rows for the CSR pass, columns for the CSC pass).
struct Side {
  int32_t nrows = 0;       // m or n
  const int64_t *ptr = nullptr;   // [nrows+1]
  const int32_t *idx = nullptr;   // [nnz] opposite-side index of each entry
  const float *val = nullptr;     // [nnz]
  const uint8_t *val8 = nullptr;  // [nnz] the same values as bytes (TSID_VALUES_U8), else null
  Segment *segs = nullptr;
  SplitRow *splits = nullptr;
  float *scale = nullptr;  // [nrows] 2 / s_i
  float *G = nullptr;      // [nrows * k] internal gradient buffer
  __nv_bfloat16 *shadow = nullptr;  // [nrows * k] or null
  int32_t nseg = 0, nsplit = 0, nslot = 0;
  int32_t cap_seg = 0, cap_split = 0, cap_slot = 0;
};

struct DenseState;   // dense_tc.cu
struct HybridState;  // hybrid.cu

// One CTA's share of a tile-list pass of the tensor-core kernel: the stored tiles [t0, t0 + nt) of row
// block ib; the CTA's partial gradient block goes to slot `slot` of the partial buffer.
struct __align__(16) DenseChunk {
  int32_t ib, t0, nt, slot;
};

// Optional per-kernel timing: CUDA events recorded on the template's stream right around the
// row pass, the column pass and the update kernel of each step (up to kProfSteps steps).
constexpr int kProfSteps = 256;
enum { EV_ROW0 = 0, EV_ROW1, EV_COL0, EV_COL1, EV_UPD0, EV_UPD1, EV_DNS0, EV_DNS1, EV_PER_STEP };
struct Prof {
  bool on = false;
  int nsteps = 0;
  cudaEvent_t *ev = nullptr;  // [kProfSteps * EV_PER_STEP], host-side handles
};

}  // namespace tsid

struct tsid_template {
  tsid_config_t cfg;
  cudaStream_t stream;
  int path;  // resolved tsid_path_t
  tsid::Side rowside, colside;
  // layout arrays (device, in the workspace)
  int64_t *row_ptr, *col_ptr;
  int32_t *col_idx, *row_idx;
  float *val_csr, *val_csc;
  uint32_t *perm;
  float *partial;     // [max(nslot_row, nslot_col) * k]
  double *red;        // reduction scratch for the loss
  int32_t red_cap;
  int32_t *flags;     // device flags: [0] range, [1] unsorted, [2] duplicate, [3] non-finite
  tsid::DenseState *dense;
  tsid::HybridState *hybrid;
  // Mini-batch template (tsid_template_create_batched): the layout is that of the block-diagonal matrix whose block b
  // holds batch b, i.e. rows b * m + i and columns b * n + j, so one sort gives (batch, row, col) and (batch, col, row)
  // order; vm, vn are those virtual sizes (0: an ordinary template).  bseg_* / bsplit_*: first segment / split row of
  // each batch on either side (host arrays of n_batches + 1 entries).
  int32_t n_batches, vm, vn;
  int32_t *bseg_row, *bseg_col, *bsplit_row, *bsplit_col;
  int32_t *vrows, *vcols;   // device: the virtual COO indices (read by the layout pass only)
  tsid::Prof prof;
  // tsid_fit replays its epochs from an executable graph: fit_steps steps on the factor arrays
  // fit_P / fit_Q, captured on fit_cap (no work ever runs there) and kept until arrays or count change
  cudaGraphExec_t fit_exec;
  cudaStream_t fit_cap;
  const float *fit_P, *fit_Q;
  int fit_steps;
  bool fit_graph_off;  // a capture failed once: launch step by step from then on
  // test hook (tsid_debug_stall_tile_pass): cycle budget of the dense kernel's waits and the work item whose
  // loads its producer never issues; 0 = normal operation
  long long dbg_wait_cycles;
  int dbg_stall_item;
  char err[256];
};

namespace tsid {

enum { FLAG_RANGE = 0, FLAG_UNSORTED = 1, FLAG_DUP = 2, FLAG_NONFINITE = 3, FLAG_TIMEOUT = 4, FLAG_COUNT = 8 };

// Carves 256-byte aligned pieces out of the caller's workspace; with base == nullptr it
// only measures.
struct Carver {
  char *base;
  size_t off = 0;
  explicit Carver(void *b) : base(static_cast<char *>(b)) {}
  template <typename T>
  T *take(size_t count) {
    size_t bytes = (count * sizeof(T) + 255) & ~size_t(255);
    T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
    off += bytes;
    return p;
  }
};

// Transient buffers of the layout pass (also carved from the workspace).
struct LayoutScratch {
  uint32_t *kA, *kB, *vA, *vB;  // [nnz] each: key and first payload of the two sort buffer sets
  uint32_t *wA, *wB, *xA, *xB;  // [nnz] each or null: second and third payload (layout pass only)
  uint32_t *hist;               // [256 * kSortBlocks]
  uint32_t *scanA, *scanB, *scanC;  // [max(m,n)+1] each
  uint32_t *blocksums;          // [kScanBlocksMax]
  // Optional 64-byte pinned host buffer mapped into the device (host address, device alias).  When set,
  // the few words the host needs back (segment totals, flags) are stored there by a kernel instead of
  // going through the copy engine, where they would queue behind any large device-to-host transfer
  // already submitted on another stream.
  uint32_t *hmap = nullptr, *hmap_dev = nullptr;
};
constexpr int kSortBlocksMax = 148 * 6;
constexpr int kScanBlocksMax = 1 << 20;

cudaError_t layout_build(tsid_template *t, const int32_t *d_rows, const int32_t *d_cols,
                         const float *d_vals, LayoutScratch &s, int32_t h_flags[FLAG_COUNT]);
cudaError_t build_segments(tsid_template *t, Side &side, int norm_mode, LayoutScratch &s);
// stable LSD radix sort of (key, payload) pairs on key bits [0, nbits) (vin == nullptr: payload = position);
// ping-pongs between (s.kA, s.vA) and (s.kB, s.vB), first writing the pair that holds no input
cudaError_t sort_pairs_u32(const uint32_t *kin, const uint32_t *vin, int64_t n, int nbits, LayoutScratch &s,
                           cudaStream_t st, uint32_t **kres, uint32_t **vres);
// out[0..n) = exclusive scan of in[0..n), out[n] = total; in[n] must be 0; in may alias out
cudaError_t scan_u32(const uint32_t *in, uint32_t *out, int64_t n, LayoutScratch &s, cudaStream_t st);

// Stage II (extend.cu, extend_tc.cu)
struct AdamArgs {
  float lr, lam2, b1, b2, eps, c1, c2;   // c1 = 1/(1-b1^t), c2 = 1/(1-b2^t)
};
struct ExtendTcMaps {                       // host copies of the tensor maps of the bf16 Q (128 bytes each)
  alignas(64) unsigned char q128[128];
  alignas(64) unsigned char q64[128];
};
bool extend_tc_qualifies(int32_t d, int32_t k);
cudaError_t extend_tc_prepare(cudaStream_t st, const float *d_Q, int32_t d, int32_t k, __nv_bfloat16 *qb, ExtendTcMaps *maps);
cudaError_t extend_tc_map_c(__nv_bfloat16 *cb, int32_t rows, int32_t d, void *map);
cudaError_t extend_tc_to_bf16(cudaStream_t st, const float *src, __nv_bfloat16 *dst, size_t n);
cudaError_t extend_tc_w(cudaStream_t st, const void *map_c, const ExtendTcMaps *maps, int32_t nc, int32_t d, int32_t k,
                        float *Wpart, int max_split, int *nsplit_out, int32_t *flags);
cudaError_t extend_tc_adam(cudaStream_t st, const float *U, const ExtendTcMaps *maps, int32_t nc, int32_t d, int32_t k,
                           float *Cm, float *Mo, float *Vo, __nv_bfloat16 *Cb, const AdamArgs &aa, int32_t *flags);

// sparse passes (sparse.cu)
cudaError_t sparse_convert_shadow(tsid_template *t, const float *d_P, const float *d_Q);
cudaError_t sparse_grad(tsid_template *t, const float *d_P, const float *d_Q, float *GP, float *GQ);
cudaError_t sparse_update(tsid_template *t, float *d_P, float *d_Q, const float *GP, const float *GQ);
// What the update kernel adds to one side when the tile passes of the hybrid path left their sums in partial
// blocks: row i has popularity rank r = rank_of[i]; the chunks [first_chunk[r / 128], first_chunk[r / 128 + 1]) of
// its block hold row r % 128 of their sums; `ranked` (or null) is the rank-ordered copy of the bf16 shadow,
// refreshed in the same kernel.
struct UpdHot {
  const int32_t *rank_of = nullptr;
  const int32_t *first_chunk = nullptr;
  const float *part = nullptr;
  __nv_bfloat16 *ranked = nullptr;
};
cudaError_t sparse_update_hot(tsid_template *t, float *d_P, float *d_Q, const float *GP, const float *GQ,
                              const UpdHot &hot_p, const UpdHot &hot_q);
cudaError_t sparse_update_scaled(tsid_template *t, float *d_P, float *d_Q, const float *GP, const float *GQ,
                                 const float *scale_p, const float *scale_q);
// one batch of a mini-batch template: the passes over the batch's segments (factor and gradient pointers shifted so that
// the layout's virtual row b * m + i lands on row i), then the update with the batch's own counts
cudaError_t sparse_batch_step(tsid_template *t, int batch, float *d_P, float *d_Q, float *GP, float *GQ);
cudaError_t batch_virtual_coo(tsid_template *t, const int32_t *d_rows, const int32_t *d_cols, const int32_t *d_batch);
cudaError_t batch_ranges(tsid_template *t, const LayoutScratch &s, bool colside);
cudaError_t sparse_residuals(tsid_template *t, const float *d_P, const float *d_Q, float *d_e);
cudaError_t sparse_loss(tsid_template *t, const float *d_P, const float *d_Q, double *d_out2);
int sparse_launches_per_step(const tsid_template *t);
cudaError_t sparse_pack_values_u8(tsid_template *t, int32_t *h_bad);
cudaError_t sparse_apply_sliced(tsid_template *t, float *d_P, const float *GP, float *const *h_Q, const float *const *h_GQ,
                                int rank, int world);
constexpr int kMaxRanks = 16;
cudaError_t sparse_counts(tsid_template *t, const Side &sd, int32_t *d_cnt);
cudaError_t sparse_scale_from_counts(tsid_template *t, Side &sd, int norm_mode, const int32_t *d_cnt);
cudaError_t sparse_side_grad(tsid_template *t, const Side &sd, const void *stage, const void *gather, float *G);
cudaError_t sparse_side_sse(tsid_template *t, const Side &sd, const void *stage, const void *gather, double *red,
                            double *d_out);

// dense tensor-core variant (dense_tc.cu)
bool dense_qualifies(const tsid_config_t &c);
DenseState *dense_new();
void dense_delete(DenseState *d);
void dense_carve(tsid_template *t, const tsid_config_t &c, Carver &cv);
cudaError_t dense_build(tsid_template *t, int32_t *h_range_flag);
int dense_launches_per_step(const tsid_template *t);
cudaError_t dense_grad(tsid_template *t, float *GP, float *GQ);
// tensor map (128 bytes at `map`) of a 16-bit matrix [rows][cols], box = box_rows x 64 columns, 128-byte swizzle
cudaError_t dense_make_map(void *map, bool half_not_bf16, void *base, uint64_t rows, uint64_t cols, uint32_t box_rows);
// tile-list pass: partial[chunk.slot] = sum over the chunk's tiles of (M .* (R_tile - X_blk Y_blk^T)) Y_blk
cudaError_t dense_tiles_pass(cudaStream_t st, int k, const __nv_bfloat16 *X, const void *map_y, const void *map_r,
                             const DenseChunk *chunks, int nchunks, const int32_t *ylist, float *partial, int32_t *flags);

// hybrid path (hybrid.cu): the populated 128 x 128 tiles of the degree-ordered template on the tensor cores,
// every other entry through the gather-reduce passes
cudaError_t csr_has_duplicates(tsid_template *t, int32_t *h_dup);
bool hybrid_qualifies(const tsid_config_t &c);
HybridState *hybrid_new();
void hybrid_delete(HybridState *h);
void hybrid_carve(tsid_template *t, const tsid_config_t &c, Carver &cv);
// builds the tiles and the tail layout; *h_status: 0 ok, 1 no tile worth it (or duplicates / fp16 range): run sparse
cudaError_t hybrid_build(tsid_template *t, LayoutScratch &s, int32_t *h_status);
cudaError_t hybrid_grad(tsid_template *t, const float *d_P, const float *d_Q, float *GP, float *GQ);
// The step as tsid_fit runs it: hybrid_refresh_ranked once after the shadows were refreshed, then per step
// hybrid_grad_partial (tail sums in GP / GQ, tile sums left in their partial blocks) and hybrid_update (which adds
// the two in the order hybrid_grad adds them and keeps the rank-ordered shadow copies current).
cudaError_t hybrid_refresh_ranked(tsid_template *t);
cudaError_t hybrid_grad_partial(tsid_template *t, float *GP, float *GQ);
cudaError_t hybrid_update(tsid_template *t, float *d_P, float *d_Q, const float *GP, const float *GQ);
int hybrid_launches_per_fit_step(const tsid_template *t);
int hybrid_launches_per_step(const tsid_template *t);
void hybrid_info(const tsid_template *t, int64_t *tiles, int32_t *min_entries, int64_t *tail);

inline int bits_for(uint32_t maxval) {  // number of bits needed to represent values <= maxval
  int b = 0;
  while (b < 32 && (maxval >> b) != 0) ++b;
  return b < 1 ? 1 : b;
}

}  // namespace tsid
