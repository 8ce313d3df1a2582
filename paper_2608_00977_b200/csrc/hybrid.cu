// Hybrid path of the gradient step (Sec. 5.1, "Regularizing Sparse RMF Updates for Tensor Cores", applied
// where the template really is dense): under skewed popularity the populated part of Omega is a staircase
// of nearly full blocks once rows and columns are ordered by their number of observed entries.  At create
// time the rows and the columns are ranked by degree, the template is cut into 128 x 128 tiles in that
// order, and every tile that holds at least a threshold of entries is stored densely (fp16, NaN =
// unobserved, once as it is and once transposed).  Per step those tiles go through the tensor-core pass
// (dense_tc.cu, tile-list form: S = X Y^T, E = M .* (R - S), G += E Y with bf16 operands and fp32
// accumulation), all other entries through the gather-reduce passes on a CSR / CSC of their own, and the
// two partial sums of every factor row are added in a fixed order (tail first, then the row block's chunks
// in chunk order).  No floating-point atomics; integer atomics only in the tile histogram, whose result
// does not depend on their order.
#include <cuda_fp16.h>

#include <new>
#include <vector>

#include "tsid_internal.cuh"

namespace tsid {

namespace {

#define CK(x)                         \
  do {                                \
    cudaError_t e_ = (x);             \
    if (e_ != cudaSuccess) return e_; \
  } while (0)

constexpr int HB = 128;               // tile edge
constexpr int HCELLS = HB * HB;
constexpr int kChunkTiles = 64;       // tiles one CTA of a tile-list pass walks
constexpr uint32_t kMinTileEntries = 480;   // a tile is stored densely from this many entries on (about 3 %)
constexpr int kBytesPerEntryForTiles = 16;  // workspace reserved for tiles: this many bytes per entry of Omega

inline int grid_for(int64_t n, int threads) {
  int64_t g = (n + threads - 1) / threads;
  if (g < 1) g = 1;
  if (g > 148 * 16) g = 148 * 16;
  return (int)g;
}

// key = other_dim - degree: ascending keys = descending degree; the sort is stable, so ties keep ascending id
__global__ void deg_key_kernel(const int64_t *__restrict__ ptr, int32_t nrows, uint32_t other_dim, uint32_t *__restrict__ key) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nrows; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t d = ptr[i + 1] - ptr[i];
    key[i] = d >= (int64_t)other_dim ? 0u : other_dim - (uint32_t)d;
  }
}
__global__ void rank_tables_kernel(const uint32_t *__restrict__ ids, int32_t nrows, int32_t *__restrict__ of_rank,
                                   int32_t *__restrict__ rank_of) {
  for (int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; r < nrows; r += (int64_t)gridDim.x * blockDim.x) {
    const uint32_t id = ids[r];
    of_rank[r] = (int32_t)id;
    rank_of[id] = (int32_t)r;
  }
}
__global__ void dup_csr_kernel(const Segment *__restrict__ segs, int nseg, const int32_t *__restrict__ col_idx, int32_t *flags) {
  const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (w >= nseg) return;
  const Segment sg = segs[w];
  bool dup = false;
  for (int q = lane + 1; q < sg.len; q += 32) {   // neighbours inside the segment (the CSR is sorted by column within a row)
    const int64_t p = (int64_t)sg.begin + q;
    if (col_idx[p] == col_idx[p - 1]) dup = true;
  }
  if (dup) flags[FLAG_DUP] = 1;
}
// duplicates across segment borders of one row: first entry of a later segment against its predecessor
__global__ void dup_border_kernel(const Segment *__restrict__ segs, int nseg, const int64_t *__restrict__ row_ptr,
                                  const int32_t *__restrict__ col_idx, int32_t *flags) {
  for (int64_t w = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; w < nseg; w += (int64_t)gridDim.x * blockDim.x) {
    const Segment sg = segs[w];
    if (sg.len > 0 && (int64_t)sg.begin > row_ptr[sg.row] && col_idx[sg.begin] == col_idx[sg.begin - 1]) flags[FLAG_DUP] = 1;
  }
}

// cnt[tile] = entries of Omega in the tile, tiles taken in the degree order of rows and columns
__global__ void tile_count_kernel(const Segment *__restrict__ segs, int nseg, const int32_t *__restrict__ col_idx,
                                  const int32_t *__restrict__ rank_of_row, const int32_t *__restrict__ rank_of_col, int JB,
                                  uint32_t *__restrict__ cnt) {
  const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (w >= nseg) return;
  const Segment sg = segs[w];
  if (sg.len <= 0) return;
  const size_t rb = (size_t)(rank_of_row[sg.row] >> 7) * JB;
  for (int q = lane; q < sg.len; q += 32) {
    const int jb = rank_of_col[__ldcs(col_idx + sg.begin + q)] >> 7;
    atomicAdd(&cnt[rb + jb], 1u);
  }
}
// hist[c] = number of tiles that hold exactly c entries, for c = minc .. 16384 (the thin tiles, which are most
// of them and would all hit the same few counters, are of no interest to the threshold search)
__global__ void count_hist_kernel(const uint32_t *__restrict__ cnt, int64_t ntile, uint32_t minc, uint32_t *__restrict__ hist) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < ntile; i += (int64_t)gridDim.x * blockDim.x) {
    const uint32_t c = cnt[i];
    if (c >= minc) atomicAdd(&hist[c > (uint32_t)HCELLS ? (uint32_t)HCELLS : c], 1u);
  }
}
// flagA[ib * JB + jb] = flagB[jb * IB + ib] = tile stored; one extra zero behind each (the scans need it)
__global__ void tile_flag_kernel(const uint32_t *__restrict__ cnt, int IB, int JB, uint32_t thresh, uint32_t *__restrict__ flagA,
                                 uint32_t *__restrict__ flagB) {
  const int64_t nt = (int64_t)IB * JB;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i <= nt; i += (int64_t)gridDim.x * blockDim.x) {
    if (i == nt) { flagA[i] = 0; flagB[i] = 0; continue; }
    const int ib = (int)(i / JB), jb = (int)(i % JB);
    const uint32_t f = cnt[i] >= thresh ? 1u : 0u;
    flagA[i] = f;
    flagB[(size_t)jb * IB + ib] = f;
  }
}
// after the scans: tabA / tabB hold the tile's index in the row-major / column-major tile array
__global__ void tile_lists_kernel(const uint32_t *__restrict__ cnt, int IB, int JB, uint32_t thresh, const uint32_t *__restrict__ tabA,
                                  const uint32_t *__restrict__ tabB, int32_t *__restrict__ ylistA, int32_t *__restrict__ ylistB) {
  const int64_t nt = (int64_t)IB * JB;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nt; i += (int64_t)gridDim.x * blockDim.x) {
    if (cnt[i] < thresh) continue;
    const int ib = (int)(i / JB), jb = (int)(i % JB);
    ylistA[tabA[i]] = jb;
    ylistB[tabB[(size_t)jb * IB + ib]] = ib;
  }
}
// out[b] = tab[b * stride] for b = 0 .. nb (the last one is tab[nb * stride] = the total)
__global__ void block_ptr_kernel(const uint32_t *__restrict__ tab, int nb, int64_t stride, uint32_t *__restrict__ out) {
  for (int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; b <= nb; b += (int64_t)gridDim.x * blockDim.x)
    out[b] = tab[b * stride];
}
__global__ void fill_u32_kernel(uint32_t *p, size_t n, uint32_t v) {
  size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) p[i] = v;
}
// warp per CSR segment: the entries of stored tiles go into the tile arrays (RA as they are, RB transposed),
// keep[p] = 1 for every other entry.  flags[FLAG_RANGE] if a stored value is beyond fp16.
__global__ void scatter_tiles_kernel(const Segment *__restrict__ segs, int nseg, const int32_t *__restrict__ col_idx,
                                     const float *__restrict__ val, const int32_t *__restrict__ rank_of_row,
                                     const int32_t *__restrict__ rank_of_col, int IB, int JB, const uint32_t *__restrict__ cnt,
                                     uint32_t thresh, const uint32_t *__restrict__ tabA, const uint32_t *__restrict__ tabB,
                                     __half *__restrict__ RA, __half *__restrict__ RB, uint32_t *__restrict__ keep, int32_t *flags) {
  const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (w >= nseg) return;
  const Segment sg = segs[w];
  if (sg.len <= 0) return;
  const int rr = rank_of_row[sg.row], ib = rr >> 7, ri = rr & 127;
  for (int q = lane; q < sg.len; q += 32) {
    const size_t p = (size_t)sg.begin + q;
    const int rc = rank_of_col[col_idx[p]], jb = rc >> 7, ci = rc & 127;
    const size_t tile = (size_t)ib * JB + jb;
    const bool sel = cnt[tile] >= thresh;
    keep[p] = sel ? 0u : 1u;
    if (sel) {
      const float r = val[p];
      if (!(fabsf(r) <= 65504.f)) flags[FLAG_RANGE] = 1;
      const __half hv = __float2half_rn(r);
      RA[(size_t)tabA[tile] * HCELLS + ri * HB + ci] = hv;
      RB[(size_t)tabB[(size_t)jb * IB + ib] * HCELLS + ci * HB + ri] = hv;
    }
  }
}
// warp per CSC segment: keep[p] for the entries in CSC order
__global__ void keep_csc_kernel(const Segment *__restrict__ segs, int nseg, const int32_t *__restrict__ row_idx,
                                const int32_t *__restrict__ rank_of_row, const int32_t *__restrict__ rank_of_col, int JB,
                                const uint32_t *__restrict__ cnt, uint32_t thresh, uint32_t *__restrict__ keep) {
  const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (w >= nseg) return;
  const Segment sg = segs[w];
  if (sg.len <= 0) return;
  const int jb = rank_of_col[sg.row] >> 7;
  for (int q = lane; q < sg.len; q += 32) {
    const size_t p = (size_t)sg.begin + q;
    const int ib = rank_of_row[row_idx[p]] >> 7;
    keep[p] = cnt[(size_t)ib * JB + jb] >= thresh ? 0u : 1u;
  }
}
// pos = exclusive scan of keep (pos[nnz] = number kept): kept entries move to pos[p], in order
__global__ void compact_kernel(const uint32_t *__restrict__ pos, int64_t nnz, const int32_t *__restrict__ idx,
                               const float *__restrict__ val, int32_t *__restrict__ idx_t, float *__restrict__ val_t) {
  for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < nnz; p += (int64_t)gridDim.x * blockDim.x) {
    const uint32_t a = pos[p];
    if (pos[p + 1] != a) { idx_t[a] = __ldcs(idx + p); val_t[a] = __ldcs(val + p); }
  }
}
__global__ void tail_ptr_kernel(const uint32_t *__restrict__ pos, const int64_t *__restrict__ ptr, int32_t nrows,
                                int64_t *__restrict__ ptr_t) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i <= nrows; i += (int64_t)gridDim.x * blockDim.x)
    ptr_t[i] = (int64_t)pos[ptr[i]];
}

// rank-ordered copies of the two shadows (16-byte pieces)
__global__ void __launch_bounds__(256)
gather_rows_kernel(const uint4 *__restrict__ A, const int32_t *__restrict__ a_of_rank, int64_t na, uint4 *__restrict__ Ah,
                   const uint4 *__restrict__ Bm, const int32_t *__restrict__ b_of_rank, int64_t nb, uint4 *__restrict__ Bh,
                   int pieces) {
  const int64_t total = (na + nb) * pieces;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
    int64_t r = i / pieces;
    const int pc = (int)(i % pieces);
    if (r < na) Ah[r * pieces + pc] = __ldg(A + (int64_t)a_of_rank[r] * pieces + pc);
    else { r -= na; Bh[r * pieces + pc] = __ldg(Bm + (int64_t)b_of_rank[r] * pieces + pc); }
  }
}
// G[of_rank[r]] += part[c0] + part[c0 + 1] + ...   (the chunks of r's row block, in chunk order)
__global__ void __launch_bounds__(256)
hot_add_kernel(float4 *__restrict__ G, const int32_t *__restrict__ of_rank, int32_t nrows, int k4,
               const float4 *__restrict__ part, const int32_t *__restrict__ first_chunk) {
  const int ib = blockIdx.x;
  const int c0 = first_chunk[ib], c1 = first_chunk[ib + 1];
  if (c1 <= c0) return;
  const int rows_per = HB / gridDim.y;
  const int r0 = blockIdx.y * rows_per;
  for (int e = threadIdx.x; e < rows_per * k4; e += blockDim.x) {
    const int rl = r0 + e / k4, l = e % k4;
    const int r = ib * HB + rl;
    if (r >= nrows) continue;
    float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int c = c0; c < c1; ++c) {
      const float4 a = __ldcs(part + ((size_t)c * HB + rl) * k4 + l);
      sum.x += a.x; sum.y += a.y; sum.z += a.z; sum.w += a.w;
    }
    float4 *g = G + (size_t)of_rank[r] * k4 + l;
    float4 v = *g;
    v.x += sum.x; v.y += sum.y; v.z += sum.z; v.w += sum.w;
    *g = v;
  }
}

int64_t hybrid_max_tiles(const tsid_config_t &c) {
  const int64_t IB = (c.m + HB - 1) / HB, JB = (c.n + HB - 1) / HB;
  int64_t mt = (int64_t)kBytesPerEntryForTiles * c.nnz / (2 * HCELLS * (int64_t)sizeof(__half));
  if (mt > IB * JB) mt = IB * JB;
  if (mt > (1 << 23)) mt = 1 << 23;   // tile row coordinates of the tensor map stay below 2^31
  return mt < 1 ? 1 : mt;
}

}  // namespace

struct HybridState {
  int IB = 0, JB = 0, n_tiles = 0, max_tiles = 0;
  uint32_t thresh = 0;
  int64_t nnz_tail = 0;
  int32_t *row_of_rank = nullptr, *rank_of_row = nullptr, *col_of_rank = nullptr, *rank_of_col = nullptr;
  __nv_bfloat16 *Ph = nullptr, *Qh = nullptr;   // [IB * 128 * k], [JB * 128 * k]: shadows in rank order, padding rows zero
  __half *RA = nullptr, *RB = nullptr;          // [n_tiles][128][128]: tiles in (ib, jb) order; transposed tiles in (jb, ib) order
  int32_t *ylistA = nullptr, *ylistB = nullptr; // column block of tile t (A); row block of transposed tile t (B)
  DenseChunk *chunksA = nullptr, *chunksB = nullptr;
  int32_t *rbc = nullptr, *cbc = nullptr;       // first chunk of each row block [IB + 1] / column block [JB + 1]
  int nchA = 0, nchB = 0, capA = 0, capB = 0;
  float *gpartA = nullptr, *gpartB = nullptr;   // [capA][128][k], [capB][128][k]: sums of the chunks of the two tile passes
  int64_t *tail_row_ptr = nullptr, *tail_col_ptr = nullptr;
  Side tailrow, tailcol;
  alignas(64) unsigned char mapPh[128], mapQh[128], mapRA[128], mapRB[128];
};

// *h_dup = 1 if some (row, col) occurs twice in the CSR arrays (neighbours: the CSR is sorted by column within a row)
cudaError_t csr_has_duplicates(tsid_template *t, int32_t *h_dup) {
  cudaStream_t st = t->stream;
  const int gr = (int)(((int64_t)t->rowside.nseg * 32 + 255) / 256);
  CK(cudaMemsetAsync(t->flags + FLAG_DUP, 0, sizeof(int32_t), st));
  if (t->rowside.nseg > 0) {
    dup_csr_kernel<<<gr, 256, 0, st>>>(t->rowside.segs, t->rowside.nseg, t->col_idx, t->flags);
    dup_border_kernel<<<grid_for(t->rowside.nseg, 256), 256, 0, st>>>(t->rowside.segs, t->rowside.nseg, t->row_ptr, t->col_idx, t->flags);
  }
  CK(cudaGetLastError());
  CK(cudaMemcpyAsync(h_dup, t->flags + FLAG_DUP, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  if (*h_dup) CK(cudaMemsetAsync(t->flags + FLAG_DUP, 0, sizeof(int32_t), st));
  return cudaSuccess;
}

bool hybrid_qualifies(const tsid_config_t &c) {
  if (c.precision != TSID_BF16_SHADOW || (c.k != 64 && c.k != 128)) return false;
  if (c.clip == TSID_CLIP_ASYM_ENTRY || (c.flags & TSID_VALUES_U8)) return false;
  const int64_t IB = (c.m + HB - 1) / HB, JB = (c.n + HB - 1) / HB;
  return c.nnz >= 1 && IB * JB <= c.nnz && c.m <= c.nnz && c.n <= c.nnz;
}

HybridState *hybrid_new() { return new (std::nothrow) HybridState; }
void hybrid_delete(HybridState *h) { delete h; }

void hybrid_carve(tsid_template *t, const tsid_config_t &c, Carver &cv) {
  HybridState tmp, *h = t->hybrid ? t->hybrid : &tmp;
  const size_t m = (size_t)c.m, n = (size_t)c.n, k = (size_t)c.k;
  h->IB = (int)((m + HB - 1) / HB);
  h->JB = (int)((n + HB - 1) / HB);
  h->max_tiles = (int)hybrid_max_tiles(c);
  h->capA = h->IB + h->max_tiles / kChunkTiles + 1;
  h->capB = h->JB + h->max_tiles / kChunkTiles + 1;
  h->row_of_rank = cv.take<int32_t>(m); h->rank_of_row = cv.take<int32_t>(m);
  h->col_of_rank = cv.take<int32_t>(n); h->rank_of_col = cv.take<int32_t>(n);
  h->Ph = cv.take<__nv_bfloat16>((size_t)h->IB * HB * k);
  h->Qh = cv.take<__nv_bfloat16>((size_t)h->JB * HB * k);
  h->RA = cv.take<__half>((size_t)h->max_tiles * HCELLS);
  h->RB = cv.take<__half>((size_t)h->max_tiles * HCELLS);
  h->ylistA = cv.take<int32_t>(h->max_tiles); h->ylistB = cv.take<int32_t>(h->max_tiles);
  h->chunksA = cv.take<DenseChunk>(h->capA); h->chunksB = cv.take<DenseChunk>(h->capB);
  h->rbc = cv.take<int32_t>(h->IB + 1); h->cbc = cv.take<int32_t>(h->JB + 1);
  h->gpartA = cv.take<float>((size_t)h->capA * HB * k);
  h->gpartB = cv.take<float>((size_t)h->capB * HB * k);
  h->tail_row_ptr = cv.take<int64_t>(m + 1); h->tail_col_ptr = cv.take<int64_t>(n + 1);
  const size_t per = (size_t)c.nnz / kSegLen;
  Side *sides[2] = {&h->tailrow, &h->tailcol};
  for (int i = 0; i < 2; ++i) {
    Side &sd = *sides[i];
    sd.nrows = (int32_t)(i == 0 ? m : n);
    sd.cap_seg = (int32_t)(sd.nrows + per + 1);
    sd.cap_split = (int32_t)(per + 1);
    sd.cap_slot = (int32_t)(2 * per + 2);
    sd.segs = cv.take<Segment>(sd.cap_seg);
    sd.splits = cv.take<SplitRow>(sd.cap_split);
  }
}

cudaError_t hybrid_build(tsid_template *t, LayoutScratch &s, int32_t *h_status) {
  HybridState *h = t->hybrid;
  const tsid_config_t &c = t->cfg;
  cudaStream_t st = t->stream;
  *h_status = 1;
  const int32_t m = c.m, n = c.n;
  const int64_t nnz = c.nnz;
  const int IB = h->IB, JB = h->JB;
  const int64_t NT = (int64_t)IB * JB;
  const int segthreads = 256;
  const int gr_row = (int)(((int64_t)t->rowside.nseg * 32 + segthreads - 1) / segthreads);
  const int gr_col = (int)(((int64_t)t->colside.nseg * 32 + segthreads - 1) / segthreads);

  // a cell observed twice cannot live in a dense tile: such templates stay on the gather-reduce passes
  CK(cudaMemsetAsync(t->flags + FLAG_DUP, 0, sizeof(int32_t), st));
  CK(cudaMemsetAsync(t->flags + FLAG_RANGE, 0, sizeof(int32_t), st));
  dup_csr_kernel<<<gr_row, segthreads, 0, st>>>(t->rowside.segs, t->rowside.nseg, t->col_idx, t->flags);
  dup_border_kernel<<<grid_for(t->rowside.nseg, 256), 256, 0, st>>>(t->rowside.segs, t->rowside.nseg, t->row_ptr, t->col_idx, t->flags);

  // 1. rows and columns ranked by degree (descending; ties by ascending index)
  uint32_t *kres, *vres;
  deg_key_kernel<<<grid_for(m, 256), 256, 0, st>>>(t->row_ptr, m, (uint32_t)n, s.kA);
  CK(sort_pairs_u32(s.kA, nullptr, m, bits_for((uint32_t)n), s, st, &kres, &vres));
  rank_tables_kernel<<<grid_for(m, 256), 256, 0, st>>>(vres, m, h->row_of_rank, h->rank_of_row);
  deg_key_kernel<<<grid_for(n, 256), 256, 0, st>>>(t->col_ptr, n, (uint32_t)m, s.kA);
  CK(sort_pairs_u32(s.kA, nullptr, n, bits_for((uint32_t)m), s, st, &kres, &vres));
  rank_tables_kernel<<<grid_for(n, 256), 256, 0, st>>>(vres, n, h->col_of_rank, h->rank_of_col);
  CK(cudaGetLastError());

  // 2. entries per tile, and how many tiles hold how many
  uint32_t *cnt = s.kA, *tabA = s.kB, *tabB = s.vA, *keep = s.vB;
  CK(cudaMemsetAsync(cnt, 0, sizeof(uint32_t) * (size_t)NT, st));
  tile_count_kernel<<<gr_row, segthreads, 0, st>>>(t->rowside.segs, t->rowside.nseg, t->col_idx, h->rank_of_row,
                                                   h->rank_of_col, JB, cnt);
  const uint32_t minc = kMinTileEntries;
  CK(cudaMemsetAsync(s.hist, 0, sizeof(uint32_t) * (HCELLS + 1), st));
  count_hist_kernel<<<grid_for(NT, 256), 256, 0, st>>>(cnt, NT, minc, s.hist);
  CK(cudaGetLastError());
  std::vector<uint32_t> hist(HCELLS + 1);
  int32_t hf[FLAG_COUNT];
  CK(cudaMemcpyAsync(hist.data(), s.hist, sizeof(uint32_t) * (HCELLS + 1), cudaMemcpyDeviceToHost, st));
  CK(cudaMemcpyAsync(hf, t->flags, sizeof(hf), cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  if (hf[FLAG_DUP]) { CK(cudaMemsetAsync(t->flags + FLAG_DUP, 0, sizeof(int32_t), st)); return cudaSuccess; }

  // 3. threshold: at least kMinTileEntries, raised until the stored tiles fit the reserved memory
  int64_t ntl = 0, ent = 0;
  uint32_t thresh = HCELLS + 1;
  for (int cc = HCELLS; cc >= (int)minc; --cc) {
    if (ntl + hist[cc] > (int64_t)h->max_tiles) break;
    ntl += hist[cc];
    ent += (int64_t)hist[cc] * cc;
    thresh = (uint32_t)cc;
  }
  if (ntl == 0) return cudaSuccess;   // nothing dense enough: the caller runs the sparse path
  h->thresh = thresh;
  h->n_tiles = (int)ntl;

  // 4. tile indices in row-major (pass over R) and column-major (pass over R^T) order
  tile_flag_kernel<<<grid_for(NT + 1, 256), 256, 0, st>>>(cnt, IB, JB, thresh, tabA, tabB);
  CK(scan_u32(tabA, tabA, NT, s, st));
  CK(scan_u32(tabB, tabB, NT, s, st));
  tile_lists_kernel<<<grid_for(NT, 256), 256, 0, st>>>(cnt, IB, JB, thresh, tabA, tabB, h->ylistA, h->ylistB);
  block_ptr_kernel<<<grid_for(IB + 1, 256), 256, 0, st>>>(tabA, IB, JB, s.scanA);
  block_ptr_kernel<<<grid_for(JB + 1, 256), 256, 0, st>>>(tabB, JB, IB, s.scanB);
  CK(cudaGetLastError());
  std::vector<uint32_t> rb(IB + 1), cb(JB + 1);
  CK(cudaMemcpyAsync(rb.data(), s.scanA, sizeof(uint32_t) * (IB + 1), cudaMemcpyDeviceToHost, st));
  CK(cudaMemcpyAsync(cb.data(), s.scanB, sizeof(uint32_t) * (JB + 1), cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  if ((int64_t)rb[IB] != ntl || (int64_t)cb[JB] != ntl) return cudaErrorUnknown;

  // 5. chunks: at most kChunkTiles consecutive tiles of one row (column) block per CTA
  std::vector<DenseChunk> chA, chB;
  std::vector<int32_t> rbc(IB + 1), cbc(JB + 1);
  auto cut = [](const std::vector<uint32_t> &bp, int nb, std::vector<DenseChunk> &ch, std::vector<int32_t> &first) {
    for (int b = 0; b < nb; ++b) {
      first[b] = (int32_t)ch.size();
      const int nt = (int)(bp[b + 1] - bp[b]);
      for (int o = 0; o < nt; o += kChunkTiles) {
        DenseChunk dc;
        dc.ib = b; dc.t0 = (int32_t)bp[b] + o; dc.nt = nt - o < kChunkTiles ? nt - o : kChunkTiles; dc.slot = (int32_t)ch.size();
        ch.push_back(dc);
      }
    }
    first[nb] = (int32_t)ch.size();
  };
  cut(rb, IB, chA, rbc);
  cut(cb, JB, chB, cbc);
  if ((int)chA.size() > h->capA || (int)chB.size() > h->capB) return cudaErrorMemoryAllocation;
  h->nchA = (int)chA.size();
  h->nchB = (int)chB.size();
  CK(cudaMemcpyAsync(h->chunksA, chA.data(), sizeof(DenseChunk) * chA.size(), cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(h->chunksB, chB.data(), sizeof(DenseChunk) * chB.size(), cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(h->rbc, rbc.data(), sizeof(int32_t) * (IB + 1), cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(h->cbc, cbc.data(), sizeof(int32_t) * (JB + 1), cudaMemcpyHostToDevice, st));

  // 6. the tiles themselves, and which entries stay on the gather-reduce passes
  const size_t words = (size_t)ntl * HCELLS / 2;
  fill_u32_kernel<<<148 * 8, 256, 0, st>>>(reinterpret_cast<uint32_t *>(h->RA), words, 0x7e007e00u);
  fill_u32_kernel<<<148 * 8, 256, 0, st>>>(reinterpret_cast<uint32_t *>(h->RB), words, 0x7e007e00u);
  CK(cudaMemsetAsync(keep + nnz, 0, sizeof(uint32_t), st));
  scatter_tiles_kernel<<<gr_row, segthreads, 0, st>>>(t->rowside.segs, t->rowside.nseg, t->col_idx, t->val_csr, h->rank_of_row,
                                                      h->rank_of_col, IB, JB, cnt, thresh, tabA, tabB, h->RA, h->RB, keep, t->flags);
  CK(cudaGetLastError());

  // 7. tail CSR (rows) and tail CSC (columns): stable compaction of the full arrays
  int32_t *idx_r = reinterpret_cast<int32_t *>(s.wA), *idx_c = reinterpret_cast<int32_t *>(s.xA);
  float *val_r = reinterpret_cast<float *>(s.wB), *val_c = reinterpret_cast<float *>(s.xB);
  CK(scan_u32(keep, keep, nnz, s, st));
  tail_ptr_kernel<<<grid_for((int64_t)m + 1, 256), 256, 0, st>>>(keep, t->row_ptr, m, h->tail_row_ptr);
  compact_kernel<<<grid_for(nnz, 256), 256, 0, st>>>(keep, nnz, t->col_idx, t->val_csr, idx_r, val_r);
  uint32_t kept_r = 0, kept_c = 0;
  CK(cudaMemcpyAsync(&kept_r, keep + nnz, sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));   // (also keeps the host vectors above alive until their copies are done)
  CK(cudaMemsetAsync(keep + nnz, 0, sizeof(uint32_t), st));
  keep_csc_kernel<<<gr_col, segthreads, 0, st>>>(t->colside.segs, t->colside.nseg, t->row_idx, h->rank_of_row, h->rank_of_col, JB,
                                                 cnt, thresh, keep);
  CK(scan_u32(keep, keep, nnz, s, st));
  tail_ptr_kernel<<<grid_for((int64_t)n + 1, 256), 256, 0, st>>>(keep, t->col_ptr, n, h->tail_col_ptr);
  compact_kernel<<<grid_for(nnz, 256), 256, 0, st>>>(keep, nnz, t->row_idx, t->val_csc, idx_c, val_c);
  CK(cudaMemcpyAsync(&kept_c, keep + nnz, sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
  CK(cudaMemcpyAsync(hf, t->flags, sizeof(hf), cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  if (kept_r != kept_c || (int64_t)kept_r + ent != nnz) return cudaErrorUnknown;
  if (hf[FLAG_RANGE]) { CK(cudaMemsetAsync(t->flags + FLAG_RANGE, 0, sizeof(int32_t), st)); return cudaSuccess; }
  h->nnz_tail = kept_r;

  h->tailrow.ptr = h->tail_row_ptr; h->tailrow.idx = idx_r; h->tailrow.val = val_r;
  h->tailcol.ptr = h->tail_col_ptr; h->tailcol.idx = idx_c; h->tailcol.val = val_c;
  h->tailrow.scale = nullptr; h->tailcol.scale = nullptr;
  h->tailrow.shadow = t->rowside.shadow; h->tailcol.shadow = t->colside.shadow;
  CK(build_segments(t, h->tailrow, TSID_NORM_NONE, s));
  CK(build_segments(t, h->tailcol, TSID_NORM_NONE, s));

  // 8. rank-ordered shadows (padding rows stay zero) and the tensor maps
  CK(cudaMemsetAsync(h->Ph, 0, sizeof(__nv_bfloat16) * (size_t)IB * HB * c.k, st));
  CK(cudaMemsetAsync(h->Qh, 0, sizeof(__nv_bfloat16) * (size_t)JB * HB * c.k, st));
  CK(dense_make_map(h->mapPh, false, h->Ph, (uint64_t)IB * HB, c.k, HB));
  CK(dense_make_map(h->mapQh, false, h->Qh, (uint64_t)JB * HB, c.k, HB));
  CK(dense_make_map(h->mapRA, true, h->RA, (uint64_t)ntl * HB, HB, HB));
  CK(dense_make_map(h->mapRB, true, h->RB, (uint64_t)ntl * HB, HB, HB));
  CK(cudaStreamSynchronize(st));
  *h_status = 0;
  return cudaSuccess;
}

// gather shadows + tail passes (+ fix-ups) + two tile-list passes + two adds
int hybrid_launches_per_step(const tsid_template *t) {
  const HybridState *h = t->hybrid;
  return 1 + 2 + (h->tailrow.nsplit > 0) + (h->tailcol.nsplit > 0) + 4;
}

void hybrid_info(const tsid_template *t, int64_t *tiles, int32_t *min_entries, int64_t *tail) {
  const HybridState *h = t->hybrid;
  *tiles = h->n_tiles;
  *min_entries = (int32_t)h->thresh;
  *tail = h->nnz_tail;
}

namespace {
// tail passes into GP / GQ, tile passes into their partial blocks; with_adds: the blocks are added to GP / GQ too
cudaError_t hybrid_passes(tsid_template *t, float *GP, float *GQ, bool with_adds) {
  HybridState *h = t->hybrid;
  const tsid_config_t &c = t->cfg;
  cudaStream_t st = t->stream;
  const int k4 = c.k / 4;
  auto mark = [&](int which) {
    if (t->prof.on && t->prof.nsteps < kProfSteps) cudaEventRecord(t->prof.ev[t->prof.nsteps * EV_PER_STEP + which], st);
  };
  mark(EV_ROW0);
  CK(sparse_side_grad(t, h->tailrow, t->rowside.shadow, t->colside.shadow, GP));
  mark(EV_ROW1);
  mark(EV_COL0);
  CK(sparse_side_grad(t, h->tailcol, t->colside.shadow, t->rowside.shadow, GQ));
  mark(EV_COL1);
  mark(EV_DNS0);
  CK(dense_tiles_pass(st, c.k, h->Ph, h->mapQh, h->mapRA, h->chunksA, h->nchA, h->ylistA, h->gpartA, t->flags));
  if (with_adds)
    hot_add_kernel<<<dim3(h->IB, 8), 256, 0, st>>>(reinterpret_cast<float4 *>(GP), h->row_of_rank, c.m, k4,
                                                   reinterpret_cast<const float4 *>(h->gpartA), h->rbc);
  CK(dense_tiles_pass(st, c.k, h->Qh, h->mapPh, h->mapRB, h->chunksB, h->nchB, h->ylistB, h->gpartB, t->flags));
  if (with_adds)
    hot_add_kernel<<<dim3(h->JB, 8), 256, 0, st>>>(reinterpret_cast<float4 *>(GQ), h->col_of_rank, c.n, k4,
                                                   reinterpret_cast<const float4 *>(h->gpartB), h->cbc);
  mark(EV_DNS1);
  return cudaGetLastError();
}
}  // namespace

// rank-ordered copies of the current bf16 shadows
cudaError_t hybrid_refresh_ranked(tsid_template *t) {
  HybridState *h = t->hybrid;
  const tsid_config_t &c = t->cfg;
  const int pieces = c.k / 8;
  gather_rows_kernel<<<grid_for(((int64_t)c.m + c.n) * pieces, 256), 256, 0, t->stream>>>(
      reinterpret_cast<const uint4 *>(t->rowside.shadow), h->row_of_rank, c.m, reinterpret_cast<uint4 *>(h->Ph),
      reinterpret_cast<const uint4 *>(t->colside.shadow), h->col_of_rank, c.n, reinterpret_cast<uint4 *>(h->Qh), pieces);
  return cudaGetLastError();
}

// complete gradient sums in GP / GQ (what tsid_grad_step and tsid_grad hand out)
cudaError_t hybrid_grad(tsid_template *t, const float *d_P, const float *d_Q, float *GP, float *GQ) {
  (void)d_P; (void)d_Q;   // bf16 shadows only
  CK(hybrid_refresh_ranked(t));
  return hybrid_passes(t, GP, GQ, true);
}

cudaError_t hybrid_grad_partial(tsid_template *t, float *GP, float *GQ) { return hybrid_passes(t, GP, GQ, false); }

cudaError_t hybrid_update(tsid_template *t, float *d_P, float *d_Q, const float *GP, const float *GQ) {
  HybridState *h = t->hybrid;
  UpdHot hp, hq;
  hp.rank_of = h->rank_of_row; hp.first_chunk = h->rbc; hp.part = h->gpartA; hp.ranked = h->Ph;
  hq.rank_of = h->rank_of_col; hq.first_chunk = h->cbc; hq.part = h->gpartB; hq.ranked = h->Qh;
  return sparse_update_hot(t, d_P, d_Q, GP, GQ, hp, hq);
}

// tail passes (+ fix-ups) + two tile-list passes; the update kernel is counted by the caller
int hybrid_launches_per_fit_step(const tsid_template *t) {
  const HybridState *h = t->hybrid;
  return 2 + (h->tailrow.nsplit > 0) + (h->tailcol.nsplit > 0) + 2;
}

}  // namespace tsid
