// Stage II, the template-conditioned extension (Sec. 5.2, Eq. 10): with Rhat* = P Q^T fixed, every column
// j of the full matrix gets coefficients C_j in R^d minimising
//       sum_{i in Omega^j} (R_ij - Rhat*_i C_j)^2 + lambda |C_j|^2
// by `iters` Adam steps.  Columns are processed in chunks of `chunk_cols`; the full matrix and C stay in
// host memory, the template factors stay in HBM.  While chunk c computes, the entries of chunk c+1 are
// copied in and the coefficients of chunk c-1 are copied out (three streams, two buffer sets).
//
// Factored form used on the device (Rhat* is never materialised):
//       W_j = Q^T C_j  (k)        pred_ij = p_i . W_j        e_ij = R_ij - pred_ij
//       U_j = sum_i e_ij p_i (k)  grad C_j = -2 Q U_j + 2 lambda C_j
// i.e. per step one tall-skinny GEMM (W = C^T Q), the same gather-reduce pass the template factorization
// uses on the chunk's entries (staged row = W_j, gathered rows = p_i), and one GEMM (U Q^T) fused with the
// Adam update of C and its moments.
#include <string.h>

#include "tsid_internal.cuh"

namespace tsid {
namespace {

#define CK(x)                         \
  do {                                \
    cudaError_t e_ = (x);             \
    if (e_ != cudaSuccess) return e_; \
  } while (0)

// Register-tiled fp32 GEMM: BM x BN output tile per 256-thread block, 8 x 8 outputs per thread (two 4-wide
// halves in each direction so that shared-memory reads are conflict-free float4s), BK-deep slices, two
// shared-memory buffers: the next slice travels global -> registers while the current one is multiplied.
// A is [M][K] row-major.  B is [K][N] row-major, or with B_NK = true [N][K] row-major.  VEC = every row
// of A, B and of the epilogue's matrices starts 16-byte aligned and K, N are multiples of 4 (then global
// memory is read and written as float4).
constexpr int BM = 128, BK = 16;   // BN (128 or 64) is a template parameter
constexpr int kSplitW = 8;         // K-splits of the tall-skinny first GEMM (K = d is long, M x N is small)

struct SplitEpi {       // partial[z][m][n] = acc   (z = K-split index; summed in order by sum_splits_kernel)
  float *part;
  size_t plane;
  __device__ __forceinline__ void operator()(int gm, int gn, int N, float acc) const {
    part[blockIdx.z * plane + (size_t)gm * N + gn] = acc;
  }
  __device__ __forceinline__ void vec4(int gm, int gn, int N, float4 acc) const {
    *reinterpret_cast<float4 *>(part + blockIdx.z * plane + (size_t)gm * N + gn) = acc;
  }
  __device__ __forceinline__ void prefetch(int, int, int) const {}
};
struct AdamEpi {        // g = -2 acc + 2 lambda C; Adam update of C and its moments in place
  float *Cm, *Mo, *Vo;
  AdamArgs a;
  __device__ __forceinline__ float one(float acc, float c, float &mo, float &vo) const {
    const float g = fmaf(a.lam2, c, -2.f * acc);
    mo = fmaf(a.b1, mo, (1.f - a.b1) * g);
    vo = fmaf(a.b2, vo, (1.f - a.b2) * g * g);
    // (the quotient uses the fast reciprocal: 2 ulp on a step that is itself ~lr in size)
    return c - __fdividef(a.lr * (mo * a.c1), sqrtf(vo * a.c2) + a.eps);
  }
  __device__ __forceinline__ void operator()(int gm, int gn, int N, float acc) const {
    const size_t o = (size_t)gm * N + gn;
    float mo = Mo[o], vo = Vo[o];
    Cm[o] = one(acc, Cm[o], mo, vo);
    Mo[o] = mo;
    Vo[o] = vo;
  }
  __device__ __forceinline__ void vec4(int gm, int gn, int N, float4 acc) const {
    const size_t o = (size_t)gm * N + gn;
    float4 c = *reinterpret_cast<const float4 *>(Cm + o), mo = *reinterpret_cast<const float4 *>(Mo + o),
           vo = *reinterpret_cast<const float4 *>(Vo + o);
    c.x = one(acc.x, c.x, mo.x, vo.x);
    c.y = one(acc.y, c.y, mo.y, vo.y);
    c.z = one(acc.z, c.z, mo.z, vo.z);
    c.w = one(acc.w, c.w, mo.w, vo.w);
    *reinterpret_cast<float4 *>(Cm + o) = c;
    *reinterpret_cast<float4 *>(Mo + o) = mo;
    *reinterpret_cast<float4 *>(Vo + o) = vo;
  }
  // asks L2 for the three 16-byte pieces this thread will update, so that they arrive during the main loop
  __device__ __forceinline__ void prefetch(int gm, int gn, int N) const {
    const size_t o = (size_t)gm * N + gn;
    asm volatile("prefetch.global.L2 [%0];" ::"l"(Cm + o));
    asm volatile("prefetch.global.L2 [%0];" ::"l"(Mo + o));
    asm volatile("prefetch.global.L2 [%0];" ::"l"(Vo + o));
  }
};

// four consecutive elements of row `row` of a row-major matrix with leading dimension ld, zero outside
// [0, nrows) x [0, colend)
template <bool VEC>
__device__ __forceinline__ float4 fetch4(const float *__restrict__ P, int row, int col, int nrows, int ld, int colend) {
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (row < nrows) {
    const float *src = P + (size_t)row * ld + col;
    if (VEC) {
      if (col < colend) v = __ldg(reinterpret_cast<const float4 *>(src));
    } else {
      if (col < colend) v.x = __ldg(src);
      if (col + 1 < colend) v.y = __ldg(src + 1);
      if (col + 2 < colend) v.z = __ldg(src + 2);
      if (col + 3 < colend) v.w = __ldg(src + 3);
    }
  }
  return v;
}

template <int BN, bool B_NK, bool VEC, class Epi>
__global__ void __launch_bounds__(256, BN == 64 ? 3 : 2)
gemm_kernel(const float *__restrict__ A, const float *__restrict__ B, int M, int N, int K, int kper, Epi epi) {
  constexpr int TH = BN / 32;   // half of the thread's columns: 4 (BN = 128) or 2 (BN = 64)
  constexpr int NA = BM * BK / 4 / 256, NB = BN * BK / 4 / 256;   // float4 loads per thread and slice
  __shared__ __align__(16) float As[2][BK][BM], Bs[2][BK][BN];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
  const int kbeg = blockIdx.z * kper, kend = kbeg + kper < K ? kbeg + kper : K;
  float acc[8][2 * TH] = {};
  float4 ra[NA], rb[NB];
  auto load_slice = [&](int k0) {
#pragma unroll
    for (int i = 0; i < NA; ++i) {   // lanes run along the rows, so the transposed store below is conflict-free
      const int q = threadIdx.x + i * 256;
      ra[i] = fetch4<VEC>(A, m0 + q % BM, k0 + (q / BM) * 4, M, K, kend);
    }
#pragma unroll
    for (int i = 0; i < NB; ++i) {
      const int q = threadIdx.x + i * 256;
      if (B_NK) rb[i] = fetch4<VEC>(B, n0 + q % BN, k0 + (q / BN) * 4, N, K, kend);
      else rb[i] = fetch4<VEC>(B, k0 + q / (BN / 4), n0 + (q % (BN / 4)) * 4, kend, N, N);
    }
  };
  auto store_slice = [&](int buf) {
#pragma unroll
    for (int i = 0; i < NA; ++i) {
      const int q = threadIdx.x + i * 256, r = q % BM, c = (q / BM) * 4;
      As[buf][c][r] = ra[i].x; As[buf][c + 1][r] = ra[i].y; As[buf][c + 2][r] = ra[i].z; As[buf][c + 3][r] = ra[i].w;
    }
#pragma unroll
    for (int i = 0; i < NB; ++i) {
      const int q = threadIdx.x + i * 256;
      if (B_NK) {
        const int r = q % BN, c = (q / BN) * 4;
        Bs[buf][c][r] = rb[i].x; Bs[buf][c + 1][r] = rb[i].y; Bs[buf][c + 2][r] = rb[i].z; Bs[buf][c + 3][r] = rb[i].w;
      } else {
        *reinterpret_cast<float4 *>(&Bs[buf][q / (BN / 4)][(q % (BN / 4)) * 4]) = rb[i];
      }
    }
  };
  if (kbeg < kend) {
    load_slice(kbeg);
    store_slice(0);
  }
  if (VEC && TH == 4) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int gm = m0 + (i < 4 ? ty * 4 + i : BM / 2 + ty * 4 + i - 4);
#pragma unroll
      for (int hcol = 0; hcol < 2; ++hcol) {
        const int gn = n0 + hcol * (BN / 2) + tx * 4;
        if (gm < M && gn < N) epi.prefetch(gm, gn, N);
      }
    }
  }
  __syncthreads();
  int buf = 0;
  for (int k0 = kbeg; k0 < kend; k0 += BK, buf ^= 1) {
    const bool more = k0 + BK < kend;
    if (more) load_slice(k0 + BK);
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      const float4 a0 = *reinterpret_cast<const float4 *>(&As[buf][kk][ty * 4]);
      const float4 a1 = *reinterpret_cast<const float4 *>(&As[buf][kk][BM / 2 + ty * 4]);
      const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      float b[2 * TH];
#pragma unroll
      for (int j = 0; j < TH; ++j) { b[j] = Bs[buf][kk][tx * TH + j]; b[TH + j] = Bs[buf][kk][BN / 2 + tx * TH + j]; }
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 2 * TH; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    if (more) store_slice(buf ^ 1);   // the other buffer was last read before the previous barrier
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int gm = m0 + (i < 4 ? ty * 4 + i : BM / 2 + ty * 4 + i - 4);
    if (gm >= M) continue;
    if (VEC && TH == 4) {
#pragma unroll
      for (int hcol = 0; hcol < 2; ++hcol) {
        const int gn = n0 + hcol * (BN / 2) + tx * 4;
        if (gn < N) epi.vec4(gm, gn, N, make_float4(acc[i][hcol * 4], acc[i][hcol * 4 + 1], acc[i][hcol * 4 + 2], acc[i][hcol * 4 + 3]));
      }
    } else {
#pragma unroll
      for (int j = 0; j < 2 * TH; ++j) {
        const int gn = n0 + (j < TH ? tx * TH + j : BN / 2 + tx * TH + j - TH);
        if (gn < N) epi(gm, gn, N, acc[i][j]);
      }
    }
  }
}

__global__ void store_flag_kernel(const int32_t *flag, uint32_t *out) {
  if (threadIdx.x == 0) {
    *out = (uint32_t)*flag;
    __threadfence_system();
  }
}

// W = sum of the K-split partial planes, in split order
__global__ void sum_splits_kernel(const float *__restrict__ part, size_t plane, int nsplit, float *__restrict__ W) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < plane; i += (size_t)gridDim.x * blockDim.x) {
    float sacc = 0.f;
    for (int z = 0; z < nsplit; ++z) sacc += part[z * plane + i];
    W[i] = sacc;
  }
}

__global__ void rebase_ptr_kernel(const int64_t *__restrict__ in, int64_t *__restrict__ out, int n1) {
  const int64_t base = in[0];
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n1; i += gridDim.x * blockDim.x) out[i] = in[i] - base;
}

__global__ void check_rows_kernel(const int32_t *__restrict__ rows, int64_t n, int32_t m, int32_t *flags) {
  bool bad = false;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    if (rows[i] < 0 || rows[i] >= m) bad = true;
  if (bad) flags[FLAG_RANGE] = 1;
}

struct Slot {           // buffers of one chunk in flight
  int64_t *ptr_raw;     // [cc+1] as copied from the host
  int32_t *rows;        // [cap]
  float *vals;          // [cap]
  float *CT;            // [cc * d]
  __nv_bfloat16 *Cb;    // [cc * d] bf16 copy of CT (tensor-core form) or null
  alignas(64) unsigned char mapC[128];   // its tensor map (host copy)
  cudaEvent_t in_done, out_done;
};

struct ExtCarve {
  Slot slot[2];
  int64_t *ptr;         // [cc+1] rebased
  Segment *segs;
  SplitRow *splits;
  float *scale, *partial, *Mo, *Vo, *W, *U, *Wpart;
  __nv_bfloat16 *Qb;    // [d * k] bf16 copy of Q (tensor-core form) or null
  double *red, *sse;
  int32_t *flags;
  LayoutScratch ls;
  int32_t cap_seg, cap_split, cap_slot;
  size_t bytes;
};

ExtCarve carve(void *base, const tsid_extend_config_t &c, int64_t cap) {
  Carver cv(base);
  ExtCarve e;
  const size_t cc = (size_t)c.chunk_cols, d = (size_t)c.d, k = (size_t)c.k, cp = (size_t)(cap > 0 ? cap : 1);
  for (int s = 0; s < 2; ++s) {
    e.slot[s].ptr_raw = cv.take<int64_t>(cc + 1);
    e.slot[s].rows = cv.take<int32_t>(cp);
    e.slot[s].vals = cv.take<float>(cp);
    e.slot[s].CT = cv.take<float>(cc * d);
    e.slot[s].Cb = (c.flags & TSID_EXTEND_TC) ? cv.take<__nv_bfloat16>(cc * d) : nullptr;
  }
  e.ptr = cv.take<int64_t>(cc + 1);
  const size_t per = cp / kSegLen;
  e.cap_seg = (int32_t)(cc + per + 1);
  e.cap_split = (int32_t)(per + 1);
  e.cap_slot = (int32_t)(2 * per + 2);
  e.segs = cv.take<Segment>(e.cap_seg);
  e.splits = cv.take<SplitRow>(e.cap_split);
  e.scale = cv.take<float>(cc);
  e.partial = cv.take<float>((size_t)e.cap_slot * k);
  e.Mo = cv.take<float>(cc * d);
  e.Vo = cv.take<float>(cc * d);
  e.W = cv.take<float>(cc * k);
  e.U = cv.take<float>(cc * k);
  e.Wpart = cv.take<float>((size_t)kSplitW * cc * k);
  e.Qb = (c.flags & TSID_EXTEND_TC) ? cv.take<__nv_bfloat16>(d * k) : nullptr;
  e.red = cv.take<double>(2 + 2 * 256 + (size_t)e.cap_seg);
  e.sse = cv.take<double>(1);
  e.flags = cv.take<int32_t>(FLAG_COUNT);
  e.ls.kA = e.ls.kB = e.ls.vA = e.ls.vB = e.ls.wA = e.ls.wB = e.ls.xA = e.ls.xB = nullptr;
  e.ls.hist = nullptr;
  e.ls.scanA = cv.take<uint32_t>(cc + 2);
  e.ls.scanB = cv.take<uint32_t>(cc + 2);
  e.ls.scanC = cv.take<uint32_t>(cc + 2);
  e.ls.blocksums = cv.take<uint32_t>(kScanBlocksMax);
  e.bytes = cv.off;
  return e;
}

tsid_status_t check(const tsid_extend_config_t *c, const int64_t *h_col_ptr, int64_t *cap_out) {
  if (!c || !h_col_ptr) return TSID_ERR_INVALID_ARG;
  if (c->m < 1 || c->d < 1 || c->n_cols < 1 || c->chunk_cols < 1 || c->iters < 0) return TSID_ERR_INVALID_ARG;
  if (c->k < 4 || c->k > 128 || (c->k & 3)) return TSID_ERR_UNSUPPORTED;
  if ((c->flags & TSID_EXTEND_TC) && !extend_tc_qualifies(c->d, c->k)) return TSID_ERR_UNSUPPORTED;
  if (!(c->beta1 >= 0.f && c->beta1 < 1.f) || !(c->beta2 >= 0.f && c->beta2 < 1.f) || !(c->eps > 0.f))
    return TSID_ERR_INVALID_ARG;
  int64_t cap = 0;
  for (int32_t j0 = 0; j0 < c->n_cols; j0 += c->chunk_cols) {
    const int32_t j1 = j0 + c->chunk_cols < c->n_cols ? j0 + c->chunk_cols : c->n_cols;
    const int64_t cnt = h_col_ptr[j1] - h_col_ptr[j0];
    if (cnt < 0 || cnt > 2147483647LL - 2) return TSID_ERR_INVALID_ARG;
    if (cnt > cap) cap = cnt;
  }
  *cap_out = cap;
  return TSID_OK;
}

}  // namespace
}  // namespace tsid

using namespace tsid;

extern "C" {

tsid_status_t tsid_extend_workspace_bytes(const tsid_extend_config_t *cfg, const int64_t *h_col_ptr,
                                          size_t *h_bytes_out) {
  int64_t cap = 0;
  tsid_status_t st = check(cfg, h_col_ptr, &cap);
  if (st != TSID_OK) return st;
  if (!h_bytes_out) return TSID_ERR_INVALID_ARG;
  *h_bytes_out = carve(nullptr, *cfg, cap).bytes;
  return TSID_OK;
}

tsid_status_t tsid_extend(const tsid_extend_config_t *cfg, const float *d_P, const float *d_Q,
                          const int64_t *h_col_ptr, const int32_t *h_row_idx, const float *h_vals, float *h_C,
                          double *h_sse_or_null) {
  int64_t cap = 0;
  tsid_status_t st = check(cfg, h_col_ptr, &cap);
  if (st != TSID_OK) return st;
  if (!d_P || !d_Q || !h_C || (cap > 0 && (!h_row_idx || !h_vals))) return TSID_ERR_INVALID_ARG;
  if (!cfg->workspace || (reinterpret_cast<uintptr_t>(cfg->workspace) & 255u)) return TSID_ERR_INVALID_ARG;
  ExtCarve e = carve(cfg->workspace, *cfg, cap);
  if (cfg->workspace_bytes < e.bytes) return TSID_ERR_OOM;
  const int32_t d = cfg->d, k = cfg->k, cc = cfg->chunk_cols;
  // 64 bytes of pinned, device-mapped host memory for the words that come back every chunk (see LayoutScratch)
  uint32_t *hmap = nullptr, *hmap_dev = nullptr;
  if (cudaHostAlloc(reinterpret_cast<void **>(&hmap), 64, cudaHostAllocMapped) != cudaSuccess ||
      cudaHostGetDevicePointer(reinterpret_cast<void **>(&hmap_dev), hmap, 0) != cudaSuccess) {
    if (hmap) cudaFreeHost(hmap);
    (void)cudaGetLastError();
    return TSID_ERR_CUDA;
  }
  memset(hmap, 0, 64);
  e.ls.hmap = hmap;
  e.ls.hmap_dev = hmap_dev;
  const bool use_tc = (cfg->flags & TSID_EXTEND_TC) != 0;   // check() made sure the shape qualifies
  ExtendTcMaps tc_maps;                                     // tensor maps of the bf16 copy of Q

  // a template object that only carries what the pass launchers read
  tsid_template ctx;
  memset(static_cast<void *>(&ctx), 0, sizeof(ctx));
  ctx.cfg.m = cc; ctx.cfg.n = cfg->m; ctx.cfg.k = k;
  ctx.cfg.precision = TSID_F32; ctx.cfg.clip = TSID_CLIP_NONE;
  ctx.stream = static_cast<cudaStream_t>(cfg->stream);
  ctx.partial = e.partial;
  ctx.flags = e.flags;

  cudaStream_t s_cmp = ctx.stream, s_in = nullptr, s_out = nullptr;
  cudaError_t err = cudaStreamCreateWithFlags(&s_in, cudaStreamNonBlocking);
  if (err == cudaSuccess) err = cudaStreamCreateWithFlags(&s_out, cudaStreamNonBlocking);
  for (int s = 0; s < 2 && err == cudaSuccess; ++s) {
    err = cudaEventCreateWithFlags(&e.slot[s].in_done, cudaEventDisableTiming);
    if (err == cudaSuccess) err = cudaEventCreateWithFlags(&e.slot[s].out_done, cudaEventDisableTiming);
  }
  cudaEvent_t cmp_done = nullptr;
  if (err == cudaSuccess) err = cudaEventCreateWithFlags(&cmp_done, cudaEventDisableTiming);

  const int nchunks = (cfg->n_cols + cc - 1) / cc;
  auto copy_in = [&](int c) -> cudaError_t {
    Slot &sl = e.slot[c & 1];
    const int32_t j0 = c * cc, j1 = j0 + cc < cfg->n_cols ? j0 + cc : cfg->n_cols;
    const int64_t p0 = h_col_ptr[j0], cnt = h_col_ptr[j1] - p0;
    // the slot's previous coefficients must have left for the host before they are overwritten
    CK(cudaStreamWaitEvent(s_in, sl.out_done, 0));
    CK(cudaMemcpyAsync(sl.ptr_raw, h_col_ptr + j0, sizeof(int64_t) * (size_t)(j1 - j0 + 1), cudaMemcpyHostToDevice, s_in));
    if (cnt > 0) {
      CK(cudaMemcpyAsync(sl.rows, h_row_idx + p0, sizeof(int32_t) * (size_t)cnt, cudaMemcpyHostToDevice, s_in));
      CK(cudaMemcpyAsync(sl.vals, h_vals + p0, sizeof(float) * (size_t)cnt, cudaMemcpyHostToDevice, s_in));
    }
    if (cfg->flags & TSID_EXTEND_COLD_START) {
      CK(cudaMemsetAsync(sl.CT, 0, sizeof(float) * (size_t)(j1 - j0) * d, s_in));
      if (use_tc) CK(cudaMemsetAsync(sl.Cb, 0, sizeof(__nv_bfloat16) * (size_t)(j1 - j0) * d, s_in));
    } else {
      CK(cudaMemcpyAsync(sl.CT, h_C + (size_t)j0 * d, sizeof(float) * (size_t)(j1 - j0) * d, cudaMemcpyHostToDevice, s_in));
      if (use_tc) CK(extend_tc_to_bf16(s_in, sl.CT, sl.Cb, (size_t)(j1 - j0) * d));
    }
    return cudaEventRecord(sl.in_done, s_in);
  };

  auto run_chunk = [&](int c) -> cudaError_t {
    Slot &sl = e.slot[c & 1];
    const int32_t j0 = c * cc, j1 = j0 + cc < cfg->n_cols ? j0 + cc : cfg->n_cols, nc = j1 - j0;
    const int64_t cnt = h_col_ptr[j1] - h_col_ptr[j0];
    CK(cudaStreamWaitEvent(s_cmp, sl.in_done, 0));
    rebase_ptr_kernel<<<(nc + 256) / 256, 256, 0, s_cmp>>>(sl.ptr_raw, e.ptr, nc + 1);
    if (cnt > 0) check_rows_kernel<<<148 * 4, 256, 0, s_cmp>>>(sl.rows, cnt, cfg->m, e.flags);
    Side side;
    side.nrows = nc; side.ptr = e.ptr; side.idx = sl.rows; side.val = sl.vals;
    side.segs = e.segs; side.splits = e.splits; side.scale = e.scale;
    side.cap_seg = e.cap_seg; side.cap_split = e.cap_split; side.cap_slot = e.cap_slot;
    // the range flag rides along with the segment totals (same host-mapped words, same synchronisation)
    store_flag_kernel<<<1, 32, 0, s_cmp>>>(e.flags + FLAG_RANGE, e.ls.hmap_dev + 8);
    CK(build_segments(&ctx, side, TSID_NORM_NONE, e.ls));   // synchronises the compute stream
    if (e.ls.hmap[8]) return cudaErrorInvalidValue;
    const size_t cd = (size_t)nc * d;
    CK(cudaMemsetAsync(e.Mo, 0, sizeof(float) * cd, s_cmp));
    CK(cudaMemsetAsync(e.Vo, 0, sizeof(float) * cd, s_cmp));
    // first GEMM: W (nc x k) = C^T (nc x d) Q (d x k), K = d split kSplitW ways; second: (nc x d) tiles
    const int kper = (((d + kSplitW - 1) / kSplitW) + BK - 1) / BK * BK;
    const int nsplit = (d + kper - 1) / kper;
    const dim3 gw((nc + BM - 1) / BM, (k + 63) / 64, nsplit), ga((nc + BM - 1) / BM, (d + 127) / 128, 1);
    const size_t plane = (size_t)nc * k;
    // float4 paths need every matrix row 16-byte aligned: k is a multiple of 4 by contract, d need not be
    const bool vec = d % 4 == 0 && k % 4 == 0 && ((reinterpret_cast<uintptr_t>(sl.CT) | reinterpret_cast<uintptr_t>(d_Q) |
                                                  reinterpret_cast<uintptr_t>(e.U) | reinterpret_cast<uintptr_t>(e.Mo) |
                                                  reinterpret_cast<uintptr_t>(e.Vo) | reinterpret_cast<uintptr_t>(e.Wpart)) & 15u) == 0;
    auto gemm_w = [&]() {
      if (use_tc) {   // C (bf16 copy) x Q (bf16) on the tensor cores, split over d
        int ns = 1;
        (void)extend_tc_w(s_cmp, sl.mapC, &tc_maps, nc, d, k, e.Wpart, kSplitW, &ns, e.flags);
        sum_splits_kernel<<<148 * 2, 256, 0, s_cmp>>>(e.Wpart, plane, ns, e.W);
        return;
      }
      if (vec) gemm_kernel<64, false, true, SplitEpi><<<gw, 256, 0, s_cmp>>>(sl.CT, d_Q, nc, k, d, kper, SplitEpi{e.Wpart, plane});
      else gemm_kernel<64, false, false, SplitEpi><<<gw, 256, 0, s_cmp>>>(sl.CT, d_Q, nc, k, d, kper, SplitEpi{e.Wpart, plane});
      sum_splits_kernel<<<148 * 2, 256, 0, s_cmp>>>(e.Wpart, plane, nsplit, e.W);
    };
    double p1 = 1.0, p2 = 1.0;
    for (int it = 1; it <= cfg->iters; ++it) {
      gemm_w();
      CK(sparse_side_grad(&ctx, side, e.W, d_P, e.U));
      p1 *= cfg->beta1; p2 *= cfg->beta2;
      AdamArgs aa{cfg->eta, 2.f * cfg->lambda, cfg->beta1, cfg->beta2, cfg->eps, (float)(1.0 / (1.0 - p1)),
                  (float)(1.0 / (1.0 - p2))};
      if (use_tc) CK(extend_tc_adam(s_cmp, e.U, &tc_maps, nc, d, k, sl.CT, e.Mo, e.Vo, sl.Cb, aa, e.flags));
      else if (vec) gemm_kernel<128, true, true, AdamEpi><<<ga, 256, 0, s_cmp>>>(e.U, d_Q, nc, d, k, k, AdamEpi{sl.CT, e.Mo, e.Vo, aa});
      else gemm_kernel<128, true, false, AdamEpi><<<ga, 256, 0, s_cmp>>>(e.U, d_Q, nc, d, k, k, AdamEpi{sl.CT, e.Mo, e.Vo, aa});
    }
    if (h_sse_or_null) {
      gemm_w();
      CK(sparse_side_sse(&ctx, side, e.W, d_P, e.red, e.sse));
    }
    CK(cudaGetLastError());
    CK(cudaEventRecord(cmp_done, s_cmp));
    // coefficients of this chunk go home on the third stream
    CK(cudaStreamWaitEvent(s_out, cmp_done, 0));
    // in pieces: the few-byte reads of the next chunk's layout (segment totals, flags) go through the same
    // copy engine and would otherwise queue behind this whole transfer, holding the compute stream up
    const size_t piece = (size_t)2 << 20;   // floats: 8 MB per copy
    for (size_t off = 0; off < cd; off += piece) {
      const size_t cnt_f = cd - off < piece ? cd - off : piece;
      CK(cudaMemcpyAsync(h_C + (size_t)j0 * d + off, sl.CT + off, sizeof(float) * cnt_f, cudaMemcpyDeviceToHost, s_out));
    }
    return cudaEventRecord(sl.out_done, s_out);
  };

  if (err == cudaSuccess && use_tc) err = extend_tc_prepare(s_cmp, d_Q, d, k, e.Qb, &tc_maps);
  for (int s = 0; s < 2 && err == cudaSuccess && use_tc; ++s) err = extend_tc_map_c(e.slot[s].Cb, cc, d, e.slot[s].mapC);
  if (err == cudaSuccess) err = cudaMemsetAsync(e.flags, 0, sizeof(int32_t) * FLAG_COUNT, s_cmp);
  if (err == cudaSuccess) err = cudaMemsetAsync(e.sse, 0, sizeof(double), s_cmp);
  if (err == cudaSuccess) err = cudaStreamSynchronize(s_cmp);
  bool bad_index = false;
  if (err == cudaSuccess) err = copy_in(0);
  for (int c = 0; c < nchunks && err == cudaSuccess; ++c) {
    if (c + 1 < nchunks) err = copy_in(c + 1);          // prefetch the next chunk while this one computes
    if (err == cudaSuccess) err = run_chunk(c);
    if (err == cudaErrorInvalidValue) { bad_index = true; break; }
  }
  double sse = 0.0;
  if (err == cudaSuccess && h_sse_or_null)
    err = cudaMemcpyAsync(&sse, e.sse, sizeof(double), cudaMemcpyDeviceToHost, s_cmp);
  int32_t hflags[FLAG_COUNT] = {0};
  if (err == cudaSuccess) err = cudaMemcpyAsync(hflags, e.flags, sizeof(hflags), cudaMemcpyDeviceToHost, s_cmp);
  cudaError_t e2 = cudaStreamSynchronize(s_cmp);
  if (hflags[FLAG_TIMEOUT] && err == cudaSuccess) err = cudaErrorLaunchTimeout;   // a bounded device-side wait expired
  cudaError_t e3 = s_out ? cudaStreamSynchronize(s_out) : cudaSuccess;
  cudaError_t e4 = s_in ? cudaStreamSynchronize(s_in) : cudaSuccess;
  if (h_sse_or_null) *h_sse_or_null = sse;
  for (int s = 0; s < 2; ++s) {
    if (e.slot[s].in_done) cudaEventDestroy(e.slot[s].in_done);
    if (e.slot[s].out_done) cudaEventDestroy(e.slot[s].out_done);
  }
  if (cmp_done) cudaEventDestroy(cmp_done);
  cudaFreeHost(hmap);
  if (s_in) cudaStreamDestroy(s_in);
  if (s_out) cudaStreamDestroy(s_out);
  if (bad_index) { (void)cudaGetLastError(); return TSID_ERR_INDEX_RANGE; }
  if (err != cudaSuccess || e2 != cudaSuccess || e3 != cudaSuccess || e4 != cudaSuccess) return TSID_ERR_CUDA;
  return TSID_OK;
}

}  // extern "C"
