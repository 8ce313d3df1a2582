// Layout pass: COO -> CSR sorted by (row, col), CSC sorted by (col, row), perm, and the
// equal-length work segments of the two gather-reduce passes.  Integer work only; every
// output is unique (stable sorts), so it can be compared bit for bit with a CPU sort.
//
// The sort is a hand-written stable LSD radix sort of a uint32 key with one to three uint32
// payload words: per pass a per-block digit histogram, an exclusive scan over the
// (digit, block) matrix and a scatter that ranks the items of each tile in input order (warp
// match + per-warp digit counters) and writes them out digit by digit from shared memory.
// The index and the value of an entry travel with its key, so no pass gathers through a
// permutation.  Integer atomics appear only in shared-memory histograms; nothing here depends
// on their order.
#include "tsid_internal.cuh"

namespace tsid {

namespace {

constexpr int RS_HIST_THREADS = 256;
constexpr int RS_THREADS = 512;  // scatter kernel
constexpr int RS_WARPS = RS_THREADS / 32;
constexpr int RS_ITEMS = 8;
constexpr int RS_TILE = RS_THREADS * RS_ITEMS;  // 4096 items per tile
constexpr int RS_RADIX = 256;
constexpr int RS_MAXP = 3;  // payload words carried per key

#define CK(x)                        \
  do {                               \
    cudaError_t e_ = (x);            \
    if (e_ != cudaSuccess) return e_; \
  } while (0)

// ---- radix sort ---------------------------------------------------------------------------
// hist[d * nb + b] = number of keys of block b's range whose digit is d, for d <= mask.
__global__ void __launch_bounds__(RS_HIST_THREADS)
rs_hist_kernel(const uint32_t *__restrict__ keys, int64_t n, int64_t per_block, int shift,
               uint32_t mask, uint32_t *__restrict__ hist, int nb) {
  __shared__ uint32_t h[RS_RADIX];
  for (int d = threadIdx.x; d < RS_RADIX; d += RS_HIST_THREADS) h[d] = 0;
  __syncthreads();
  int64_t lo = (int64_t)blockIdx.x * per_block;
  int64_t hi = lo + per_block < n ? lo + per_block : n;
  for (int64_t p = lo + threadIdx.x; p < hi; p += RS_HIST_THREADS)
    atomicAdd(&h[(keys[p] >> shift) & mask], 1u);
  __syncthreads();
  for (int d = threadIdx.x; d <= (int)mask; d += RS_HIST_THREADS) hist[(size_t)d * nb + blockIdx.x] = h[d];
}

// In-place exclusive scan of a short array by one block (four items per thread and sweep).
__global__ void __launch_bounds__(1024) rs_scan_kernel(uint32_t *a, int n) {
  __shared__ uint32_t warp_tot[32];
  __shared__ uint32_t carry_s;
  if (threadIdx.x == 0) carry_s = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  for (int base = 0; base < n; base += 4096) {
    int i = base + threadIdx.x * 4;
    uint32_t v[4], sum = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      v[j] = i + j < n ? a[i + j] : 0u;
      sum += v[j];
    }
    uint32_t inc = sum;
    for (int o = 1; o < 32; o <<= 1) {
      uint32_t u = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += u;
    }
    if (lane == 31) warp_tot[w] = inc;
    __syncthreads();
    if (w == 0) {
      uint32_t t = warp_tot[lane];
      uint32_t ti = t;
      for (int o = 1; o < 32; o <<= 1) {
        uint32_t u = __shfl_up_sync(0xffffffffu, ti, o);
        if (lane >= o) ti += u;
      }
      warp_tot[lane] = ti - t;  // exclusive prefix of the warp totals
    }
    __syncthreads();
    uint32_t run = carry_s + warp_tot[w] + inc - sum;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (i + j < n) a[i + j] = run;
      run += v[j];
    }
    __syncthreads();
    if (threadIdx.x == 1023) carry_s = run;
    __syncthreads();
  }
}

// One key stream and NP payload streams of a sort pass.  pin[q] == nullptr: payload q is the
// position of the item in the input (a sort that starts from the identity permutation).
template <int NP>
struct SortIO {
  const uint32_t *kin;
  uint32_t *kout;
  const uint32_t *pin[NP];
  uint32_t *pout[NP];
};

constexpr size_t rs_scatter_smem(int np) {
  return sizeof(uint32_t) * ((size_t)RS_WARPS * RS_RADIX + 2 * RS_RADIX + 32 + (size_t)(1 + np) * RS_TILE);
}

// Stable scatter of one pass.  Each block owns a contiguous range of the input and walks it in
// tiles.  Within a tile every item gets its rank among the tile's items of the same digit in
// input order (warp match + per-warp digit counters + a scan over the warps); the tile is
// then put in digit order in shared memory, so that the copy to global memory writes each
// digit's items to consecutive addresses from consecutive threads.
template <int NP>
__global__ void __launch_bounds__(RS_THREADS, 2)
rs_scatter_kernel(SortIO<NP> io, int64_t n, int64_t per_block, int shift, uint32_t mask,
                  const uint32_t *__restrict__ offs, int nb) {
  extern __shared__ uint32_t rs_sm[];
  uint32_t(*wc)[RS_RADIX] = reinterpret_cast<uint32_t(*)[RS_RADIX]>(rs_sm);
  uint32_t *lstart = rs_sm + RS_WARPS * RS_RADIX;  // first staged slot of each digit
  uint32_t *gadj = lstart + RS_RADIX;              // global position of a staged slot = gadj[digit] + slot
  uint32_t *wtot = gadj + RS_RADIX;
  uint32_t *skey = wtot + 32;
  uint32_t *sval = skey + RS_TILE;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const uint32_t lt = (1u << lane) - 1u;
  // thread d keeps the running global offset of digit d for this block
  uint32_t run_off = (uint32_t)threadIdx.x <= mask ? offs[(size_t)threadIdx.x * nb + blockIdx.x] : 0u;
  int64_t lo = (int64_t)blockIdx.x * per_block;
  int64_t hi = lo + per_block < n ? lo + per_block : n;
  // The keys of the next tile are fetched while this tile is ranked and written, and the
  // payload words of this tile while it is ranked, so that no load is waited for in place.
  uint32_t nkey[RS_ITEMS];
#pragma unroll
  for (int it = 0; it < RS_ITEMS; ++it) {
    int64_t p = lo + (int64_t)w * 32 * RS_ITEMS + it * 32 + lane;
    nkey[it] = p < hi ? io.kin[p] : 0u;
  }
  for (int64_t tile = lo; tile < hi; tile += RS_TILE) {
    for (int d = lane; d < RS_RADIX; d += 32) wc[w][d] = 0;
    __syncwarp();
    uint32_t key[RS_ITEMS], rank[RS_ITEMS], pay[NP][RS_ITEMS];
    const int64_t wbase = tile + (int64_t)w * 32 * RS_ITEMS;
#pragma unroll
    for (int it = 0; it < RS_ITEMS; ++it) {
      key[it] = nkey[it];
      int64_t p = wbase + RS_TILE + it * 32 + lane;
      nkey[it] = p < hi ? io.kin[p] : 0u;
    }
#pragma unroll
    for (int q = 0; q < NP; ++q) {
#pragma unroll
      for (int it = 0; it < RS_ITEMS; ++it) {
        int64_t p = wbase + it * 32 + lane;
        pay[q][it] = (p < hi && io.pin[q]) ? io.pin[q][p] : (uint32_t)p;
      }
    }
#pragma unroll
    for (int it = 0; it < RS_ITEMS; ++it) {
      const bool ok = wbase + it * 32 + lane < hi;
      const uint32_t dig = ok ? ((key[it] >> shift) & mask) : 0xffffffffu;
      // lanes with the same digit, from one ballot per digit bit (the match instruction takes time in
      // proportion to the number of distinct values in the warp, which is ~28 for a 7-bit digit)
      uint32_t peers = __ballot_sync(0xffffffffu, ok);
      if (!ok) peers = ~peers;
#pragma unroll
      for (int b = 0; b < 8; ++b) {
        if ((mask >> b) == 0) break;
        const uint32_t bal = __ballot_sync(0xffffffffu, (dig >> b) & 1u);
        peers &= ((dig >> b) & 1u) ? bal : ~bal;
      }
      int leader = __ffs(peers) - 1;
      uint32_t base = 0;
      if (lane == leader && ok) {
        base = wc[w][dig];
        wc[w][dig] = base + __popc(peers);
      }
      base = __shfl_sync(0xffffffffu, base, leader);
      rank[it] = base + __popc(peers & lt);
      __syncwarp();
    }
    __syncthreads();
    // thread d < RS_RADIX: scan digit d over the warps, then the digit totals over d
    uint32_t tot = 0, inc = 0;
    if (threadIdx.x < RS_RADIX) {
      const int d = threadIdx.x;
#pragma unroll
      for (int ww = 0; ww < RS_WARPS; ++ww) {
        uint32_t c = wc[ww][d];
        wc[ww][d] = tot;
        tot += c;
      }
      inc = tot;
      for (int o = 1; o < 32; o <<= 1) {
        uint32_t u = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += u;
      }
      if (lane == 31) wtot[w] = inc;
    }
    __syncthreads();
    if (threadIdx.x < RS_RADIX) {
      uint32_t pre = 0;
      for (int ww = 0; ww < w; ++ww) pre += wtot[ww];
      const uint32_t ls = pre + inc - tot;
      lstart[threadIdx.x] = ls;
      gadj[threadIdx.x] = run_off - ls;
      run_off += tot;
    }
    __syncthreads();
#pragma unroll
    for (int it = 0; it < RS_ITEMS; ++it) {
      const int64_t p = wbase + it * 32 + lane;
      if (p < hi) {
        const uint32_t dig = (key[it] >> shift) & mask;
        const uint32_t slot = lstart[dig] + wc[w][dig] + rank[it];
        skey[slot] = key[it];
#pragma unroll
        for (int q = 0; q < NP; ++q) sval[q * RS_TILE + slot] = pay[q][it];
      }
    }
    __syncthreads();
    const int cnt = (int)(hi - tile < RS_TILE ? hi - tile : RS_TILE);
#pragma unroll 4
    for (int i = threadIdx.x; i < cnt; i += RS_THREADS) {
      const uint32_t k = skey[i];
      const uint32_t g = gadj[(k >> shift) & mask] + (uint32_t)i;
      io.kout[g] = k;
#pragma unroll
      for (int q = 0; q < NP; ++q) io.pout[q][g] = sval[q * RS_TILE + i];
    }
    __syncthreads();
  }
}

// The two buffer sets a sort ping-pongs between.
struct SortSet {
  uint32_t *k;
  uint32_t *p[RS_MAXP];
};
inline SortSet set_a(const LayoutScratch &s) { return SortSet{s.kA, {s.vA, s.wA, s.xA}}; }
inline SortSet set_b(const LayoutScratch &s) { return SortSet{s.kB, {s.vB, s.wB, s.xB}}; }
inline bool in_set(const SortSet &x, const void *ptr) {
  if (!ptr) return false;
  if (ptr == x.k) return true;
  for (int q = 0; q < RS_MAXP; ++q)
    if (ptr == x.p[q]) return true;
  return false;
}

// Stable sort of n items (key + NP payload words) on key bits [0, nbits).  The passes
// ping-pong between the two buffer sets of the scratch, starting with the set that holds none
// of the inputs; where kfin / pfin[q] is not null the last pass writes that stream there
// instead (it must not alias an input of that pass).  *kres / pres[q] receive the location of
// each result stream.
template <int NP>
cudaError_t radix_sort_multi(const uint32_t *kin, const uint32_t *const *pin, int64_t n, int nbits,
                             LayoutScratch &s, cudaStream_t st, uint32_t *kfin, uint32_t *const *pfin,
                             uint32_t **kres, uint32_t **pres) {
  static_assert(NP >= 1 && NP <= RS_MAXP, "payload count");
  int npass = (nbits + 7) / 8;
  if (npass < 1) npass = 1;
  int64_t tiles = (n + RS_TILE - 1) / RS_TILE;
  int nb = (int)(tiles < kSortBlocksMax ? tiles : kSortBlocksMax);
  if (nb < 1) nb = 1;
  int64_t per_block = ((tiles + nb - 1) / nb) * RS_TILE;
  const SortSet A = set_a(s), B = set_b(s);
  bool inA = in_set(A, kin), inB = in_set(B, kin);
  for (int q = 0; q < NP; ++q) {
    inA = inA || in_set(A, pin[q]);
    inB = inB || in_set(B, pin[q]);
  }
  if (inA && inB) return cudaErrorInvalidValue;
  CK(cudaFuncSetAttribute(rs_scatter_kernel<NP>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                          (int)rs_scatter_smem(NP)));
  SortSet out = inA ? B : A, other = inA ? A : B;
  SortIO<NP> io;
  io.kin = kin;
  for (int q = 0; q < NP; ++q) io.pin[q] = pin[q];
  int shift = 0;
  for (int p = 0; p < npass; ++p) {
    int bits = (nbits - shift + (npass - p) - 1) / (npass - p);  // spread the bits evenly
    if (bits < 1) bits = 1;
    uint32_t mask = (1u << bits) - 1u;
    const bool last = p == npass - 1;
    io.kout = (last && kfin) ? kfin : out.k;
    for (int q = 0; q < NP; ++q) io.pout[q] = (last && pfin && pfin[q]) ? pfin[q] : out.p[q];
    rs_hist_kernel<<<nb, RS_HIST_THREADS, 0, st>>>(io.kin, n, per_block, shift, mask, s.hist, nb);
    rs_scan_kernel<<<1, 1024, 0, st>>>(s.hist, (int)(mask + 1) * nb);
    rs_scatter_kernel<NP><<<nb, RS_THREADS, rs_scatter_smem(NP), st>>>(io, n, per_block, shift, mask, s.hist, nb);
    CK(cudaGetLastError());
    io.kin = io.kout;
    for (int q = 0; q < NP; ++q) io.pin[q] = io.pout[q];
    SortSet tmp = out; out = other; other = tmp;
    shift += bits;
  }
  *kres = const_cast<uint32_t *>(io.kin);
  for (int q = 0; q < NP; ++q) pres[q] = const_cast<uint32_t *>(io.pin[q]);
  return cudaSuccess;
}

// ---- generic exclusive scan of uint32 (three kernels; block sums scanned by one block) -----
constexpr int SC_THREADS = 256, SC_ITEMS = 8, SC_TILE = SC_THREADS * SC_ITEMS;

__global__ void __launch_bounds__(SC_THREADS)
scan_tile_kernel(const uint32_t *in, uint32_t *out, int64_t n,  // in may alias out
                 uint32_t *__restrict__ blocksums, const uint32_t *__restrict__ blockoffs) {
  __shared__ uint32_t wt[SC_THREADS / 32];
  int64_t base = (int64_t)blockIdx.x * SC_TILE + (int64_t)threadIdx.x * SC_ITEMS;
  uint32_t v[SC_ITEMS], sum = 0;
#pragma unroll
  for (int i = 0; i < SC_ITEMS; ++i) {
    v[i] = (base + i < n) ? in[base + i] : 0u;
    sum += v[i];
  }
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  uint32_t inc = sum;
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t u = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += u;
  }
  if (lane == 31) wt[w] = inc;
  __syncthreads();
  uint32_t woff = 0;
  for (int ww = 0; ww < w; ++ww) woff += wt[ww];
  if (blockoffs == nullptr) {  // first sweep: only the block total is needed
    if (threadIdx.x == SC_THREADS - 1) blocksums[blockIdx.x] = woff + inc;
    return;
  }
  uint32_t run = blockoffs[blockIdx.x] + woff + inc - sum;
#pragma unroll
  for (int i = 0; i < SC_ITEMS; ++i) {
    if (base + i < n) out[base + i] = run;
    run += v[i];
  }
}

// out[0..n) = exclusive scan of in[0..n); out[n] = total.  in and out may alias.
cudaError_t exclusive_scan_u32(const uint32_t *in, uint32_t *out, int64_t n, LayoutScratch &s,
                               cudaStream_t st) {
  int64_t n1 = n + 1;  // scan n+1 slots so that out[n] receives the total (in[n] must be 0)
  int nb = (int)((n1 + SC_TILE - 1) / SC_TILE);
  if (nb > kScanBlocksMax) return cudaErrorInvalidValue;
  scan_tile_kernel<<<nb, SC_THREADS, 0, st>>>(in, nullptr, n1, s.blocksums, nullptr);
  rs_scan_kernel<<<1, 1024, 0, st>>>(s.blocksums, nb);
  scan_tile_kernel<<<nb, SC_THREADS, 0, st>>>(in, out, n1, nullptr, s.blocksums);
  return cudaGetLastError();
}

// ---- checks, copies, pointer arrays ------------------------------------------------------------
__global__ void check_coo_kernel(const int32_t *__restrict__ rows, const int32_t *__restrict__ cols,
                                 int64_t nnz, int32_t m, int32_t n, int32_t *flags) {
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  bool bad = false, unsorted = false, dup = false;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < nnz; t += stride) {
    int32_t r = rows[t], c = cols[t];
    if (r < 0 || r >= m || c < 0 || c >= n) bad = true;
    if (t > 0) {
      int32_t r0 = rows[t - 1], c0 = cols[t - 1];
      if (r0 > r || (r0 == r && c0 > c)) unsorted = true;
      if (r0 == r && c0 == c) dup = true;
    }
  }
  if (bad) flags[FLAG_RANGE] = 1;
  if (unsorted) flags[FLAG_UNSORTED] = 1;
  if (dup) flags[FLAG_DUP] = 1;  // only meaningful when the input is sorted
}

__global__ void check_dup_kernel(const uint32_t *__restrict__ rowkey, const int32_t *__restrict__ col_idx,
                                 int64_t nnz, int32_t *flags) {
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  bool dup = false;
  for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x + 1; p < nnz; p += stride)
    if (rowkey[p] == rowkey[p - 1] && col_idx[p] == col_idx[p - 1]) dup = true;
  if (dup) flags[FLAG_DUP] = 1;
}

template <typename TI, typename TO>
__global__ void copy_kernel(const TI *__restrict__ src, TO *__restrict__ dst, int64_t n) {
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < n; p += stride) dst[p] = (TO)src[p];
}

// ptr[r] = first position p with key[p] >= r, for r in [0, nrows]; keys are sorted.
__global__ void ptr_from_sorted_kernel(const uint32_t *__restrict__ key, int64_t nnz, int32_t nrows,
                                       int64_t *__restrict__ ptr) {
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p <= nnz; p += stride) {
    int64_t lo = (p == 0) ? 0 : (int64_t)key[p - 1] + 1;       // rows (key[p-1], key[p]] start at p
    int64_t hi = (p == nnz) ? (int64_t)nrows : (int64_t)key[p];
    for (int64_t r = lo; r <= hi; ++r) ptr[r] = p;
  }
}

// ---- segments ---------------------------------------------------------------------------------------
__global__ void seg_count_kernel(const int64_t *__restrict__ ptr, int32_t nrows, int norm_count,
                                 uint32_t *__restrict__ nseg, uint32_t *__restrict__ nslot,
                                 uint32_t *__restrict__ nsplit, float *__restrict__ scale) {
  int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i <= nrows; i += stride) {
    if (i == nrows) { nseg[i] = 0; nslot[i] = 0; nsplit[i] = 0; continue; }
    int64_t cnt = ptr[i + 1] - ptr[i];
    uint32_t s = cnt <= kSegLen ? 1u : (uint32_t)((cnt + kSegLen - 1) / kSegLen);
    nseg[i] = s;
    nslot[i] = s > 1 ? s : 0u;
    nsplit[i] = s > 1 ? 1u : 0u;
    float sc = (norm_count && cnt > 1) ? (float)cnt : 1.0f;
    if (scale) scale[i] = 2.0f / sc;   // null: segments of a side whose normalisation is kept elsewhere
  }
}

__global__ void seg_fill_kernel(const int64_t *__restrict__ ptr, int32_t nrows,
                                const uint32_t *__restrict__ seg_off, const uint32_t *__restrict__ slot_off,
                                const uint32_t *__restrict__ split_off, Segment *__restrict__ segs,
                                SplitRow *__restrict__ splits) {
  // one warp per row: the lanes stride over the row's segments
  int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  int lane = threadIdx.x & 31;
  int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t i = warp; i < nrows; i += nwarps) {
    int64_t b = ptr[i], cnt = ptr[i + 1] - b;
    uint32_t s0 = seg_off[i], ns = seg_off[i + 1] - s0;
    bool split = ns > 1;
    uint32_t sl0 = slot_off[i];
    for (uint32_t q = lane; q < ns; q += 32) {
      Segment sg;
      sg.row = (int32_t)i;
      sg.begin = (uint32_t)(b + (int64_t)q * kSegLen);
      int64_t rem = cnt - (int64_t)q * kSegLen;
      sg.len = (int32_t)(rem < kSegLen ? rem : kSegLen);
      sg.slot = split ? (int32_t)(sl0 + q) : -1;
      segs[s0 + q] = sg;
    }
    if (split && lane == 0) {
      SplitRow sr;
      sr.row = (int32_t)i; sr.slot0 = (int32_t)sl0; sr.nseg = (int32_t)ns; sr.pad = 0;
      splits[split_off[i]] = sr;
    }
  }
}

// three words to a host-mapped buffer (visible to the host once the stream has been synchronised)
__global__ void store3_kernel(const uint32_t *a, const uint32_t *b, const uint32_t *c, uint32_t *out) {
  if (threadIdx.x == 0) {
    out[0] = *a; out[1] = *b; out[2] = *c;
    __threadfence_system();
  }
}

inline int grid_for(int64_t n, int threads) {
  int64_t g = (n + threads - 1) / threads;
  if (g < 1) g = 1;
  if (g > 148 * 16) g = 148 * 16;
  return (int)g;
}

}  // namespace

cudaError_t layout_build(tsid_template *t, const int32_t *d_rows, const int32_t *d_cols,
                         const float *d_vals, LayoutScratch &s, int32_t h_flags[FLAG_COUNT]) {
  cudaStream_t st = t->stream;
  const int64_t nnz = t->cfg.nnz;
  const int32_t m = t->vm ? t->vm : t->cfg.m, n = t->vn ? t->vn : t->cfg.n;   // a mini-batch template sorts its virtual indices
  if (!t->n_batches) CK(cudaMemsetAsync(t->flags, 0, sizeof(int32_t) * FLAG_COUNT, st));   // (whose range flag is already set)
  if (nnz > 0) check_coo_kernel<<<grid_for(nnz, 256), 256, 0, st>>>(d_rows, d_cols, nnz, m, n, t->flags);
  CK(cudaGetLastError());
  CK(cudaMemcpyAsync(h_flags, t->flags, sizeof(int32_t) * FLAG_COUNT, cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  if (h_flags[FLAG_RANGE]) return cudaSuccess;  // caller reports TSID_ERR_INDEX_RANGE
  if (h_flags[FLAG_UNSORTED] && (t->cfg.flags & TSID_INPUT_ROW_SORTED)) return cudaSuccess;

  const int g = grid_for(nnz, 256);
  const uint32_t *rowkey = reinterpret_cast<const uint32_t *>(d_rows);  // row of each entry in CSR order
  if (nnz > 0) {
    if (!h_flags[FLAG_UNSORTED]) {
      // already in (row, col) order: CSR is the input
      copy_kernel<int32_t, int32_t><<<g, 256, 0, st>>>(d_cols, t->col_idx, nnz);
      copy_kernel<float, float><<<g, 256, 0, st>>>(d_vals, t->val_csr, nnz);
    } else {
      h_flags[FLAG_DUP] = 0;  // the adjacent-pair test of check_coo only holds for sorted input
      CK(cudaMemsetAsync(t->flags + FLAG_DUP, 0, sizeof(int32_t), st));
      // stable by column, then stable by row  =>  (row, col, input position) order; the other
      // index and the value travel with the key, so nothing is gathered afterwards
      uint32_t *k1, *p1[2], *k2, *p2[2];
      const uint32_t *in1[2] = {reinterpret_cast<const uint32_t *>(d_rows), reinterpret_cast<const uint32_t *>(d_vals)};
      CK(radix_sort_multi<2>(reinterpret_cast<const uint32_t *>(d_cols), in1, nnz, bits_for(n - 1), s, st, nullptr,
                             nullptr, &k1, p1));
      const uint32_t *in2[2] = {k1, p1[1]};
      uint32_t *fin2[2] = {reinterpret_cast<uint32_t *>(t->col_idx), reinterpret_cast<uint32_t *>(t->val_csr)};
      CK(radix_sort_multi<2>(p1[0], in2, nnz, bits_for(m - 1), s, st, nullptr, fin2, &k2, p2));
      rowkey = k2;
      if (t->cfg.flags & TSID_VALIDATE) check_dup_kernel<<<g, 256, 0, st>>>(rowkey, t->col_idx, nnz, t->flags);
    }
    CK(cudaGetLastError());
  }
  ptr_from_sorted_kernel<<<grid_for(nnz + 1, 256), 256, 0, st>>>(rowkey, nnz, m, t->row_ptr);
  CK(cudaGetLastError());

  // CSC: stable sort of the CSR entries by column, carrying (CSR position, row, value)
  if (nnz > 0) {
    uint32_t *k3, *p3[3];
    const uint32_t *in3[3] = {nullptr, rowkey, reinterpret_cast<const uint32_t *>(t->val_csr)};
    uint32_t *fin3[3] = {t->perm, reinterpret_cast<uint32_t *>(t->row_idx), reinterpret_cast<uint32_t *>(t->val_csc)};
    CK(radix_sort_multi<3>(reinterpret_cast<const uint32_t *>(t->col_idx), in3, nnz, bits_for(n - 1), s, st, nullptr,
                           fin3, &k3, p3));
    ptr_from_sorted_kernel<<<grid_for(nnz + 1, 256), 256, 0, st>>>(k3, nnz, n, t->col_ptr);
    CK(cudaGetLastError());
  } else {
    ptr_from_sorted_kernel<<<1, 256, 0, st>>>(nullptr, 0, n, t->col_ptr);
    CK(cudaGetLastError());
  }
  int32_t dupflag = 0;
  CK(cudaMemcpyAsync(&dupflag, t->flags + FLAG_DUP, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  h_flags[FLAG_DUP] = dupflag;
  return cudaSuccess;
}

cudaError_t build_segments(tsid_template *t, Side &side, int norm_mode, LayoutScratch &s) {
  cudaStream_t st = t->stream;
  const int32_t nr = side.nrows;
  seg_count_kernel<<<grid_for((int64_t)nr + 1, 256), 256, 0, st>>>(side.ptr, nr, norm_mode == TSID_NORM_COUNT,
                                                                 s.scanA, s.scanB, s.scanC, side.scale);
  CK(cudaGetLastError());
  CK(exclusive_scan_u32(s.scanA, s.scanA, nr, s, st));
  CK(exclusive_scan_u32(s.scanB, s.scanB, nr, s, st));
  CK(exclusive_scan_u32(s.scanC, s.scanC, nr, s, st));
  uint32_t tot[3];
  if (s.hmap_dev) {
    store3_kernel<<<1, 32, 0, st>>>(s.scanA + nr, s.scanB + nr, s.scanC + nr, s.hmap_dev);
    CK(cudaGetLastError());
    CK(cudaStreamSynchronize(st));
    tot[0] = s.hmap[0]; tot[1] = s.hmap[1]; tot[2] = s.hmap[2];
  } else {
    CK(cudaMemcpyAsync(&tot[0], s.scanA + nr, 4, cudaMemcpyDeviceToHost, st));
    CK(cudaMemcpyAsync(&tot[1], s.scanB + nr, 4, cudaMemcpyDeviceToHost, st));
    CK(cudaMemcpyAsync(&tot[2], s.scanC + nr, 4, cudaMemcpyDeviceToHost, st));
    CK(cudaStreamSynchronize(st));
  }
  side.nseg = (int32_t)tot[0];
  side.nslot = (int32_t)tot[1];
  side.nsplit = (int32_t)tot[2];
  if (side.nseg > side.cap_seg || side.nslot > side.cap_slot || side.nsplit > side.cap_split)
    return cudaErrorMemoryAllocation;
  int64_t threads = (int64_t)nr * 32;
  seg_fill_kernel<<<grid_for(threads, 256), 256, 0, st>>>(side.ptr, nr, s.scanA, s.scanB, s.scanC, side.segs,
                                                         side.splits);
  CK(cudaGetLastError());
  return cudaStreamSynchronize(st);
}

// The sort and the scan, for the other translation units (template sampling).
cudaError_t sort_pairs_u32(const uint32_t *kin, const uint32_t *vin, int64_t n, int nbits, LayoutScratch &s,
                           cudaStream_t st, uint32_t **kres, uint32_t **vres) {
  const uint32_t *pin[1] = {vin};
  return radix_sort_multi<1>(kin, pin, n, nbits, s, st, nullptr, nullptr, kres, vres);
}
cudaError_t scan_u32(const uint32_t *in, uint32_t *out, int64_t n, LayoutScratch &s, cudaStream_t st) {
  return exclusive_scan_u32(in, out, n, s, st);
}

}  // namespace tsid
