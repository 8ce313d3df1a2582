// Template sampling (Sec. 5.1, "Sampling the TSID Template Submatrix"): choose d = ceil(alpha n)
// columns uniformly at random without replacement, keep the observed entries that fall in them, and
// re-index the columns to 0..d-1 in ascending order of the original index.
//
// The draw is counter-based so that it can be reproduced anywhere: column j gets the 64-bit key
// SplitMix64(seed + (j+1) * 0x9E3779B97F4A7C15) (the (j+1)-th output of the SplitMix64 stream seeded
// with `seed`), and the template takes the d columns with the smallest (key, j).  Integer work only:
// the key sort is the library's stable radix sort (low word, then high word), the column map and
// the entry compaction are exclusive scans, so the kept entries stay in input order.
#include "tsid_internal.cuh"

namespace tsid {
namespace {

#define CK(x)                         \
  do {                                \
    cudaError_t e_ = (x);             \
    if (e_ != cudaSuccess) return e_; \
  } while (0)

__host__ __device__ inline uint64_t splitmix64_at(uint64_t seed, uint64_t index1) {
  uint64_t z = seed + index1 * 0x9E3779B97F4A7C15ULL;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}

__global__ void keys_kernel(uint64_t seed, int32_t n, uint32_t *lo, uint32_t *hi) {
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < n; j += stride) {
    const uint64_t key = splitmix64_at(seed, (uint64_t)j + 1);
    lo[j] = (uint32_t)key;
    hi[j] = (uint32_t)(key >> 32);
  }
}
__global__ void gather_u32_kernel(const uint32_t *src, const uint32_t *pos, uint32_t *dst, int64_t n) {
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) dst[i] = src[pos[i]];
}
__global__ void copy_u32_kernel(const uint32_t *src, uint32_t *dst, int64_t n) {
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) dst[i] = src[i];
}
__global__ void fill_zero_kernel(uint32_t *p, int64_t n) {
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) p[i] = 0u;
}
// flag[col] = 1 for the first d columns of the key order
__global__ void mark_kernel(const uint32_t *order, int32_t d, uint32_t *flag) {
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < d; i += stride) flag[order[i]] = 1u;
}
// colmap[j] = rank of j among the chosen columns, or -1
__global__ void colmap_kernel(const uint32_t *flag, const uint32_t *rank, int32_t n, int32_t *colmap) {
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < n; j += stride)
    colmap[j] = flag[j] ? (int32_t)rank[j] : -1;
}
__global__ void keep_kernel(const int32_t *cols, const int32_t *colmap, int64_t nnz, int32_t n, uint32_t *keep,
                            int32_t *flags) {
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  bool bad = false;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t <= nnz; t += stride) {
    if (t == nnz) { keep[t] = 0u; continue; }
    const int32_t c = cols[t];
    if (c < 0 || c >= n) { bad = true; keep[t] = 0u; continue; }
    keep[t] = colmap[c] >= 0 ? 1u : 0u;
  }
  if (bad) flags[FLAG_RANGE] = 1;
}
__global__ void compact_kernel(const int32_t *rows, const int32_t *cols, const float *vals, const int32_t *colmap,
                               const uint32_t *pos, int64_t nnz, int32_t n, int32_t *rows_out, int32_t *cols_out,
                               float *vals_out) {
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < nnz; t += stride) {
    if (pos[t + 1] != pos[t]) {   // kept (out-of-range columns were given keep = 0)
      const uint32_t o = pos[t];
      rows_out[o] = rows[t];
      cols_out[o] = colmap[cols[t]];
      vals_out[o] = vals[t];
    }
  }
}

// ---- fused selection of the entries (used when the column bitmap fits shared memory) -----------------
// Every block owns a contiguous range of the entries.  The chosen columns are a bitmap in shared memory
// (one bit per column) with the rank of the first column of every 256-column group beside it, so both
// "is this column chosen" and "which new index does it get" are answered without touching global memory.
// Sweep 1 counts the kept entries of each block; sweep 2 re-reads the range tile by tile, ranks the kept
// entries of a tile in input order (ballots, then a scan of the per-warp counts) and writes them to their
// final places: no flag array and no position array travel through HBM.
constexpr int FS_THREADS = 1024, FS_ITEMS = 4, FS_TILE = FS_THREADS * FS_ITEMS, FS_WARPS = FS_THREADS / 32;
constexpr int FS_MAX_SMEM = 200 * 1024;
constexpr int kFusedBlocks = 148;

__host__ __device__ inline size_t fused_smem_bytes(int32_t n) {
  const size_t nw = ((size_t)n + 31) / 32, ng = (nw + 7) / 8;
  return (nw + ng + FS_ITEMS * FS_WARPS + 8) * sizeof(uint32_t);
}

// bm[w] = bits of flag[32 w .. 32 w + 31]; gp[g] = rank of column 256 g (rank = exclusive scan of flag)
__global__ void bitmap_kernel(const uint32_t *__restrict__ flag, const uint32_t *__restrict__ rank, int32_t n,
                              uint32_t *__restrict__ bm, uint32_t *__restrict__ gp) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  const int64_t n32 = ((int64_t)n + 31) / 32 * 32;
  for (int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < n32; j += stride) {
    const uint32_t b = __ballot_sync(0xffffffffu, j < n && flag[j] != 0u);
    if ((j & 31) == 0) bm[j >> 5] = b;
    if ((j & 255) == 0) gp[j >> 8] = rank[j < n ? j : n];
  }
}

__device__ __forceinline__ void load_bitmap(uint32_t *sbm, uint32_t *sgp, const uint32_t *bm, const uint32_t *gp,
                                            int32_t n) {
  const int nw = (n + 31) / 32, ng = (nw + 7) / 8;
  for (int i = threadIdx.x; i < nw; i += blockDim.x) sbm[i] = bm[i];
  for (int i = threadIdx.x; i < ng; i += blockDim.x) sgp[i] = gp[i];
  __syncthreads();
}

__global__ void __launch_bounds__(FS_THREADS, 1)
count_keep_kernel(const int32_t *__restrict__ cols, int64_t nnz, int32_t n, const uint32_t *__restrict__ bm,
                  const uint32_t *__restrict__ gp, uint32_t *__restrict__ cnt, int32_t *flags) {
  extern __shared__ uint32_t fs_sm[];
  const int nw = (n + 31) / 32, ng = (nw + 7) / 8;
  uint32_t *sbm = fs_sm, *sgp = sbm + nw, *swc = sgp + ng;
  load_bitmap(sbm, sgp, bm, gp, n);
  const int64_t lo = nnz * blockIdx.x / gridDim.x, hi = nnz * (blockIdx.x + 1) / gridDim.x;
  uint32_t c = 0;
  bool bad = false;
  for (int64_t t = lo + threadIdx.x; t < hi; t += FS_THREADS) {
    const int32_t col = __ldcs(cols + t);
    if (col < 0 || col >= n) bad = true;
    else c += (sbm[col >> 5] >> (col & 31)) & 1u;
  }
  if (bad) flags[FLAG_RANGE] = 1;
  for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
  if ((threadIdx.x & 31) == 0) swc[threadIdx.x >> 5] = c;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t tot = 0;
    for (int w = 0; w < FS_WARPS; ++w) tot += swc[w];
    cnt[blockIdx.x] = tot;
  }
}

__global__ void __launch_bounds__(FS_THREADS, 1)
compact_fused_kernel(const int32_t *__restrict__ rows, const int32_t *__restrict__ cols, const float *__restrict__ vals,
                     int64_t nnz, int32_t n, const uint32_t *__restrict__ bm, const uint32_t *__restrict__ gp,
                     const uint32_t *__restrict__ cnt, int32_t *__restrict__ rows_out, int32_t *__restrict__ cols_out,
                     float *__restrict__ vals_out, uint32_t *__restrict__ total_out) {
  extern __shared__ uint32_t fs_sm[];
  const int nw = (n + 31) / 32, ng = (nw + 7) / 8;
  uint32_t *sbm = fs_sm, *sgp = sbm + nw, *swc = sgp + ng, *sbase = swc + FS_ITEMS * FS_WARPS;
  load_bitmap(sbm, sgp, bm, gp, n);
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  if (threadIdx.x == 0) {   // kept entries of all earlier blocks (and, by the last block, the grand total)
    uint32_t before = 0;
    for (unsigned b = 0; b < blockIdx.x; ++b) before += cnt[b];
    sbase[0] = before;
    if (blockIdx.x == gridDim.x - 1) *total_out = before + cnt[blockIdx.x];
  }
  __syncthreads();
  uint32_t run = sbase[0];
  const int64_t lo = nnz * blockIdx.x / gridDim.x, hi = nnz * (blockIdx.x + 1) / gridDim.x;
  // the triples of the next tile are fetched while this one is ranked and written
  int32_t ncol[FS_ITEMS], nrow[FS_ITEMS];
  float nval[FS_ITEMS];
  auto fetch = [&](int64_t tile) {
#pragma unroll
    for (int i = 0; i < FS_ITEMS; ++i) {
      const int64_t t = tile + i * FS_THREADS + threadIdx.x;
      const bool in = t < hi;
      ncol[i] = in ? __ldcs(cols + t) : -1;
      nrow[i] = in ? __ldcs(rows + t) : 0;
      nval[i] = in ? __ldcs(vals + t) : 0.f;
    }
  };
  fetch(lo);
  for (int64_t tile = lo; tile < hi; tile += FS_TILE) {
    int32_t col[FS_ITEMS], row[FS_ITEMS];
    float val[FS_ITEMS];
    bool kept[FS_ITEMS];
    uint32_t pre[FS_ITEMS];
#pragma unroll
    for (int i = 0; i < FS_ITEMS; ++i) { col[i] = ncol[i]; row[i] = nrow[i]; val[i] = nval[i]; }
    fetch(tile + FS_TILE);
#pragma unroll
    for (int i = 0; i < FS_ITEMS; ++i) {
      kept[i] = col[i] >= 0 && col[i] < n && ((sbm[col[i] >> 5] >> (col[i] & 31)) & 1u);
      const uint32_t b = __ballot_sync(0xffffffffu, kept[i]);
      pre[i] = __popc(b & ((1u << lane) - 1u));
      if (lane == 0) swc[i * FS_WARPS + w] = __popc(b);
    }
    __syncthreads();
    if (w == 0) {   // exclusive scan of the FS_ITEMS * FS_WARPS per-warp counts, in entry order
      uint32_t v[FS_ITEMS], sum = 0;
#pragma unroll
      for (int i = 0; i < FS_ITEMS; ++i) { v[i] = swc[lane * FS_ITEMS + i]; sum += v[i]; }
      uint32_t inc = sum;
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t u = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += u;
      }
      uint32_t ex = inc - sum;
#pragma unroll
      for (int i = 0; i < FS_ITEMS; ++i) { swc[lane * FS_ITEMS + i] = ex; ex += v[i]; }
      if (lane == 31) sbase[1] = inc;   // kept entries of the tile
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < FS_ITEMS; ++i) {
      if (kept[i]) {
        const uint32_t o = run + swc[i * FS_WARPS + w] + pre[i];
        const int c = col[i], wd = c >> 5, g = wd >> 3;
        uint32_t r = sgp[g] + __popc(sbm[wd] & ((1u << (c & 31)) - 1u));
        for (int q = g << 3; q < wd; ++q) r += __popc(sbm[q]);
        rows_out[o] = row[i];
        cols_out[o] = (int32_t)r;
        vals_out[o] = val[i];
      }
    }
    run += sbase[1];
    __syncthreads();
  }
}

inline int grid_of(int64_t n) {
  int64_t g = (n + 255) / 256;
  if (g < 1) g = 1;
  if (g > 148 * 16) g = 148 * 16;
  return (int)g;
}

struct SampleCarve {
  LayoutScratch ls;
  uint32_t *klo, *khi, *flag, *keep;
  uint32_t *bm, *gp, *cnt, *total;   // fused selection: column bitmap, group ranks, per-block counts, kept total
  int32_t *dflags;
  size_t bytes;
};

SampleCarve carve(void *base, int32_t n, int64_t nnz) {
  Carver cv(base);
  SampleCarve c;
  const size_t nn = (size_t)n + 2, nz = (size_t)nnz + 2;
  c.dflags = cv.take<int32_t>(FLAG_COUNT);
  c.ls.kA = cv.take<uint32_t>(nn); c.ls.kB = cv.take<uint32_t>(nn);
  c.ls.vA = cv.take<uint32_t>(nn); c.ls.vB = cv.take<uint32_t>(nn);
  c.ls.wA = c.ls.wB = c.ls.xA = c.ls.xB = nullptr;
  c.ls.hist = cv.take<uint32_t>(256 * (size_t)kSortBlocksMax);
  c.ls.scanA = c.ls.scanB = c.ls.scanC = nullptr;
  c.ls.blocksums = cv.take<uint32_t>(kScanBlocksMax);
  c.klo = cv.take<uint32_t>(nn); c.khi = cv.take<uint32_t>(nn);
  c.flag = cv.take<uint32_t>(nn);
  c.keep = cv.take<uint32_t>(nz);
  c.bm = cv.take<uint32_t>(nn / 32 + 2);
  c.gp = cv.take<uint32_t>(nn / 256 + 2);
  c.cnt = cv.take<uint32_t>(kFusedBlocks);
  c.total = cv.take<uint32_t>(4);
  c.bytes = cv.off;
  return c;
}

}  // namespace
}  // namespace tsid

using namespace tsid;

extern "C" {

tsid_status_t tsid_sample_workspace_bytes(int32_t n, int64_t nnz, size_t *h_bytes_out) {
  if (!h_bytes_out || n < 1 || nnz < 0 || nnz > 2147483647LL - 2) return TSID_ERR_INVALID_ARG;
  *h_bytes_out = carve(nullptr, n, nnz).bytes;
  return TSID_OK;
}

tsid_status_t tsid_sample_template(int32_t m, int32_t n, int64_t nnz, double alpha, uint64_t seed,
                                   const int32_t *d_rows, const int32_t *d_cols, const float *d_vals, void *stream,
                                   void *workspace, size_t workspace_bytes, int32_t *d_colmap, int32_t *d_rows_out,
                                   int32_t *d_cols_out, float *d_vals_out, int32_t *h_d_out, int64_t *h_nnz_out) {
  if (m < 1 || n < 1 || nnz < 0 || nnz > 2147483647LL - 2 || !(alpha > 0.0) || !(alpha <= 1.0) || !d_colmap ||
      !h_d_out || !h_nnz_out || !workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
      (nnz > 0 && (!d_rows || !d_cols || !d_vals || !d_rows_out || !d_cols_out || !d_vals_out)))
    return TSID_ERR_INVALID_ARG;
  SampleCarve c = carve(workspace, n, nnz);
  if (workspace_bytes < c.bytes) return TSID_ERR_OOM;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  double dd = ceil(alpha * (double)n);
  int32_t d = dd < 1.0 ? 1 : (dd > (double)n ? n : (int32_t)dd);

  const bool fused = nnz > 0 && fused_smem_bytes(n) <= (size_t)FS_MAX_SMEM;
  auto run = [&]() -> cudaError_t {
    CK(cudaMemsetAsync(c.dflags, 0, sizeof(int32_t) * FLAG_COUNT, st));
    keys_kernel<<<grid_of(n), 256, 0, st>>>(seed, n, c.klo, c.khi);
    // stable sort by the low word, then by the high word => order by (key, column)
    uint32_t *k1, *v1, *k2, *v2;
    CK(sort_pairs_u32(c.klo, nullptr, n, 32, c.ls, st, &k1, &v1));
    uint32_t *gk = c.ls.kB;   // the second sort writes (kA, vA) first: keep its input in the B buffers
    gather_u32_kernel<<<grid_of(n), 256, 0, st>>>(c.khi, v1, gk, n);
    if (v1 == c.ls.vA) { copy_u32_kernel<<<grid_of(n), 256, 0, st>>>(v1, c.ls.vB, n); v1 = c.ls.vB; }
    CK(sort_pairs_u32(gk, v1, n, 32, c.ls, st, &k2, &v2));
    fill_zero_kernel<<<grid_of(n + 1), 256, 0, st>>>(c.flag, (int64_t)n + 1);
    mark_kernel<<<grid_of(d), 256, 0, st>>>(v2, d, c.flag);
    // rank of each chosen column = exclusive scan of the flags (reuse klo for the scan output)
    CK(scan_u32(c.flag, c.klo, n, c.ls, st));
    colmap_kernel<<<grid_of(n), 256, 0, st>>>(c.flag, c.klo, n, d_colmap);
    if (fused) {
      // the chosen columns as a shared-memory bitmap: count per block, then rank and write in one sweep
      const size_t smem = fused_smem_bytes(n);
      CK(cudaFuncSetAttribute(count_keep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      CK(cudaFuncSetAttribute(compact_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      bitmap_kernel<<<grid_of(n), 256, 0, st>>>(c.flag, c.klo, n, c.bm, c.gp);
      count_keep_kernel<<<kFusedBlocks, FS_THREADS, smem, st>>>(d_cols, nnz, n, c.bm, c.gp, c.cnt, c.dflags);
      compact_fused_kernel<<<kFusedBlocks, FS_THREADS, smem, st>>>(d_rows, d_cols, d_vals, nnz, n, c.bm, c.gp, c.cnt,
                                                                   d_rows_out, d_cols_out, d_vals_out, c.total);
      return cudaGetLastError();
    }
    keep_kernel<<<grid_of(nnz + 1), 256, 0, st>>>(d_cols, d_colmap, nnz, n, c.keep, c.dflags);
    CK(scan_u32(c.keep, c.keep, nnz, c.ls, st));
    if (nnz > 0)
      compact_kernel<<<grid_of(nnz), 256, 0, st>>>(d_rows, d_cols, d_vals, d_colmap, c.keep, nnz, n, d_rows_out,
                                                   d_cols_out, d_vals_out);
    return cudaGetLastError();
  };
  cudaError_t e = run();
  uint32_t kept = 0;
  int32_t hf[FLAG_COUNT] = {0};
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(&kept, fused ? c.total : c.keep + nnz, sizeof(uint32_t), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(hf, c.dflags, sizeof(hf), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return TSID_ERR_CUDA;
  if (hf[FLAG_RANGE]) return TSID_ERR_INDEX_RANGE;
  *h_d_out = d;
  *h_nnz_out = (int64_t)kept;
  return TSID_OK;
}

}  // extern "C"
