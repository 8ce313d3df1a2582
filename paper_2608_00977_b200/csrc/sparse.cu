// Sparse path: the two gather-reduce passes (CSR pass -> G_P = E Q, CSC pass -> G_Q = E^T P,
// each recomputing e_ij = r_ij - p_i . q_j), the fixed-order fix-up of rows that span several
// segments, and the fused normalise + regularise + clip + update kernel
// (Sec. 5.1 Eqs. (update-p), (update-q), Eq. 9; Sec. 5.3).
//
// Work mapping of a pass.  One warp owns one segment (<= kSegLen consecutive entries of one
// row).  The warp is cut into groups of GROUP lanes; a group owns one entry at a time and each
// of its lanes owns EPL = KP / GROUP coordinates of the factor rows, so that the lanes of a
// group read one gathered factor row as contiguous 16-byte vectors.  The owning row p_i is
// staged once per segment in registers.  Per entry: partial dot over the lane's coordinates,
// log2(GROUP) shuffles -> e, then e * q_j into the lane's accumulators.  At the end of the
// segment the accumulators of the groups are added by shuffles (warp level), written either
// to the gradient row or to a partial row; partial rows are summed in segment order by the
// fix-up kernel (grid level).  No floating-point atomics anywhere: results are deterministic.
#include "tsid_internal.cuh"

namespace tsid {

namespace {

#define CK(x)                         \
  do {                                \
    cudaError_t e_ = (x);             \
    if (e_ != cudaSuccess) return e_; \
  } while (0)

template <int KP>
struct Geo {
  static constexpr int GROUP = KP >= 128 ? KP / 16 : (KP >= 32 ? 8 : 4);
  static constexpr int EPL = KP / GROUP;  // coordinates per lane: 4, 4, 8, 16, 16
  static constexpr int EPW = 32 / GROUP;  // entries a warp handles per iteration
};

// ---- 16-byte (or 8-byte) vectors of factor values -----------------------------------------------
template <bool BF16, int VE>
struct Raw;
template <>
struct Raw<false, 4> {
  float4 v;
  __device__ __forceinline__ void zero() { v = make_float4(0.f, 0.f, 0.f, 0.f); }
  __device__ __forceinline__ void load(const float *p) { v = __ldg(reinterpret_cast<const float4 *>(p)); }
  __device__ __forceinline__ void unpack(float *o) const { o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w; }
};
__device__ __forceinline__ void bf2(uint32_t w, float &lo, float &hi) {
  lo = __uint_as_float(w << 16);
  hi = __uint_as_float(w & 0xffff0000u);
}
template <>
struct Raw<true, 8> {
  uint4 v;
  __device__ __forceinline__ void zero() { v = make_uint4(0u, 0u, 0u, 0u); }
  __device__ __forceinline__ void load(const __nv_bfloat16 *p) { v = __ldg(reinterpret_cast<const uint4 *>(p)); }
  __device__ __forceinline__ void unpack(float *o) const {
    bf2(v.x, o[0], o[1]); bf2(v.y, o[2], o[3]); bf2(v.z, o[4], o[5]); bf2(v.w, o[6], o[7]);
  }
};
template <>
struct Raw<true, 4> {
  uint2 v;
  __device__ __forceinline__ void zero() { v = make_uint2(0u, 0u); }
  __device__ __forceinline__ void load(const __nv_bfloat16 *p) { v = __ldg(reinterpret_cast<const uint2 *>(p)); }
  __device__ __forceinline__ void unpack(float *o) const { bf2(v.x, o[0], o[1]); bf2(v.y, o[2], o[3]); }
};

enum { MODE_GRAD = 0, MODE_RESID = 1, MODE_LOSS = 2 };

template <int KP, bool BF16, int MODE>
__global__ void __launch_bounds__(256)
pass_kernel(const Segment *__restrict__ segs, int nseg, const int32_t *__restrict__ idx,
            const float *__restrict__ val, const void *__restrict__ stage_v,
            const void *__restrict__ gather_v, int k, float *__restrict__ G,
            float *__restrict__ partial, float *__restrict__ e_out, double *__restrict__ red) {
  using T = typename std::conditional<BF16, __nv_bfloat16, float>::type;
  constexpr int GROUP = Geo<KP>::GROUP, EPL = Geo<KP>::EPL, EPW = Geo<KP>::EPW;
  constexpr int VE = BF16 ? (EPL >= 8 ? 8 : 4) : 4;
  constexpr int NV = EPL / VE;
  using R = Raw<BF16, VE>;
  const T *stage = static_cast<const T *>(stage_v);
  const T *gat = static_cast<const T *>(gather_v);

  const int warp = (int)(((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
  if (warp >= nseg) return;
  const int lane = threadIdx.x & 31;
  const int g = lane / GROUP, s = lane % GROUP;
  const Segment sg = segs[warp];

  // coordinates owned by this lane: chunk c covers [c*GROUP*VE + s*VE, +VE)
  bool cv[NV];
  int co[NV];
#pragma unroll
  for (int c = 0; c < NV; ++c) {
    co[c] = c * GROUP * VE + s * VE;
    cv[c] = co[c] < k;
  }

  float x[EPL], acc[EPL];
  {
    const T *xr = stage + (size_t)sg.row * k;
#pragma unroll
    for (int c = 0; c < NV; ++c) {
      R r;
      r.zero();
      if (cv[c]) r.load(xr + co[c]);
      r.unpack(x + c * VE);
    }
  }
#pragma unroll
  for (int i = 0; i < EPL; ++i) acc[i] = 0.f;
  double sq = 0.0;

  const int32_t *ip = idx + sg.begin;
  const float *vp = val + sg.begin;
  const int len = sg.len;

  int32_t nj = 0;
  float nr = 0.f;
  if (lane < len) { nj = __ldcs(ip + lane); nr = __ldcs(vp + lane); }

  for (int base = 0; base < len; base += 32) {
    const int32_t myj = nj;
    const float myr = nr;
    const int nv = len - base < 32 ? len - base : 32;
    if (base + 32 + lane < len) { nj = __ldcs(ip + base + 32 + lane); nr = __ldcs(vp + base + 32 + lane); }
    const int iters = (nv + EPW - 1) / EPW;
    for (int it = 0; it < iters; it += 2) {
      const int sa = it * EPW + g, sb = sa + EPW;
      const int32_t ja = __shfl_sync(0xffffffffu, myj, sa & 31);
      const int32_t jb = __shfl_sync(0xffffffffu, myj, sb & 31);
      const float ra = __shfl_sync(0xffffffffu, myr, sa & 31);
      const float rb = __shfl_sync(0xffffffffu, myr, sb & 31);
      const bool va = sa < nv, vb = sb < nv;
      R ya[NV], yb[NV];
      const T *pa = gat + (size_t)ja * k, *pb = gat + (size_t)jb * k;
#pragma unroll
      for (int c = 0; c < NV; ++c) {
        ya[c].zero();
        yb[c].zero();
        if (va && cv[c]) ya[c].load(pa + co[c]);
        if (vb && cv[c]) yb[c].load(pb + co[c]);
      }
      float fa[EPL], fb[EPL];
#pragma unroll
      for (int c = 0; c < NV; ++c) { ya[c].unpack(fa + c * VE); yb[c].unpack(fb + c * VE); }
      float da = 0.f, db = 0.f;
#pragma unroll
      for (int i = 0; i < EPL; ++i) { da = fmaf(x[i], fa[i], da); db = fmaf(x[i], fb[i], db); }
#pragma unroll
      for (int o = GROUP / 2; o > 0; o >>= 1) {
        da += __shfl_xor_sync(0xffffffffu, da, o);
        db += __shfl_xor_sync(0xffffffffu, db, o);
      }
      const float ea = va ? ra - da : 0.f;
      const float eb = vb ? rb - db : 0.f;
      if (MODE == MODE_GRAD) {
#pragma unroll
        for (int i = 0; i < EPL; ++i) acc[i] = fmaf(ea, fa[i], acc[i]);
#pragma unroll
        for (int i = 0; i < EPL; ++i) acc[i] = fmaf(eb, fb[i], acc[i]);
      } else if (MODE == MODE_RESID) {
        if (s == 0 && va) e_out[(size_t)sg.begin + base + sa] = ea;
        if (s == 0 && vb) e_out[(size_t)sg.begin + base + sb] = eb;
      } else {
        if (s == 0) sq += (double)ea * (double)ea + (double)eb * (double)eb;
      }
    }
  }

  if (MODE == MODE_GRAD) {
#pragma unroll
    for (int o = GROUP; o < 32; o <<= 1) {
#pragma unroll
      for (int i = 0; i < EPL; ++i) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], o);
    }
    if (g == 0) {
      float *dst = sg.slot < 0 ? G + (size_t)sg.row * k : partial + (size_t)sg.slot * k;
#pragma unroll
      for (int c = 0; c < NV; ++c) {
        if (cv[c]) {
#pragma unroll
          for (int q = 0; q < VE / 4; ++q)
            *reinterpret_cast<float4 *>(dst + co[c] + 4 * q) =
                make_float4(acc[c * VE + 4 * q], acc[c * VE + 4 * q + 1], acc[c * VE + 4 * q + 2],
                            acc[c * VE + 4 * q + 3]);
        }
      }
    }
  } else if (MODE == MODE_LOSS) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    if (lane == 0) red[warp] = sq;
  }
}

// Rows that span several segments: add their partial rows in segment order.
__global__ void __launch_bounds__(128)
fixup_kernel(const SplitRow *__restrict__ splits, int nsplit, const float *__restrict__ partial,
             float *__restrict__ G, int k) {
  const int r = blockIdx.x;
  if (r >= nsplit) return;
  const SplitRow sr = splits[r];
  for (int l = threadIdx.x; l < k; l += blockDim.x) {
    float sum = 0.f;
    const float *p = partial + (size_t)sr.slot0 * k + l;
    for (int q = 0; q < sr.nseg; ++q) sum += p[(size_t)q * k];
    G[(size_t)sr.row * k + l] = sum;
  }
}

struct UpdSide {
  float *X;
  const float *G;
  const float *scale;
  __nv_bfloat16 *shadow;
  int64_t n4;  // rows * k / 4
  UpdHot hot;  // hybrid path: sums of the tile passes still to be added, rank-ordered shadow copy
};

__device__ __forceinline__ float clip_dir(float d, float xi, int clip) {
  if (clip == TSID_CLIP_ASYM_STEP) return fminf(fmaxf(xi, -d), d);
  if (clip == TSID_CLIP_ASYM_GRAD) return -fminf(fmaxf(xi, d), -d);
  return d;
}

// D = G * (2/s) - 2 lambda X; clip; X += eta D; refresh the bf16 shadow; flag non-finite values.
// HOT: the side carries sums of the hybrid path's tile passes (UpdHot); launched per side (side b unused), which
// keeps it at 48 registers.
template <bool HOT>
__global__ void __launch_bounds__(256, HOT ? 5 : 8)
update_kernel(UpdSide a, UpdSide b, int k4, float eta, float lam2, float xi, int clip, float gmul, int32_t *flags) {
  const int64_t total = HOT ? a.n4 : a.n4 + b.n4;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  bool bad = false;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
    const bool first = HOT || i < a.n4;
    const UpdSide &sd = first ? a : b;
    const int64_t j = first ? i : i - a.n4;
    const float sc = __ldg(sd.scale + j / k4) * gmul;
    float4 x = reinterpret_cast<float4 *>(sd.X)[j];
    float4 gv = __ldcs(reinterpret_cast<const float4 *>(sd.G) + j);
    int r = 0;
    if (HOT && sd.hot.rank_of) {
      // + the sums of the row block's chunks, added among themselves first, in chunk order
      r = __ldg(sd.hot.rank_of + j / k4);
      const int l = (int)(j % k4), c0 = __ldg(sd.hot.first_chunk + (r >> 7)), c1 = __ldg(sd.hot.first_chunk + (r >> 7) + 1);
      if (c1 > c0) {
        float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int c = c0; c < c1; ++c) {
          const float4 p = __ldcs(reinterpret_cast<const float4 *>(sd.hot.part) + ((size_t)c * 128 + (r & 127)) * k4 + l);
          sum.x += p.x; sum.y += p.y; sum.z += p.z; sum.w += p.w;
        }
        gv.x += sum.x; gv.y += sum.y; gv.z += sum.z; gv.w += sum.w;
      }
    }
    float xs[4] = {x.x, x.y, x.z, x.w};
    const float gs[4] = {gv.x, gv.y, gv.z, gv.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float d = fmaf(gs[q], sc, -lam2 * xs[q]);
      bad |= !isfinite(d);
      d = clip_dir(d, xi, clip);
      xs[q] = fmaf(eta, d, xs[q]);
      bad |= !isfinite(xs[q]);
    }
    reinterpret_cast<float4 *>(sd.X)[j] = make_float4(xs[0], xs[1], xs[2], xs[3]);
    if (sd.shadow) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(xs[0], xs[1]);
      __nv_bfloat162 hi = __floats2bfloat162_rn(xs[2], xs[3]);
      uint2 pk;
      pk.x = *reinterpret_cast<uint32_t *>(&lo);
      pk.y = *reinterpret_cast<uint32_t *>(&hi);
      reinterpret_cast<uint2 *>(sd.shadow)[j] = pk;
      if (HOT && sd.hot.ranked) reinterpret_cast<uint2 *>(sd.hot.ranked)[(size_t)r * k4 + j % k4] = pk;
    }
  }
  if (bad) flags[FLAG_NONFINITE] = 1;
}

// Exchange + update of one slice of Q for a row-sharded template, in one kernel.  The slice's rows of
// every rank's partial G_Q are read with plain loads (this GPU's memory or a peer's mapped memory) and
// added in rank order, the update is applied once, and the new values are stored with plain stores into
// every rank's replica of Q: a reduce-scatter and an all-gather folded into the update, with no
// intermediate buffer.  Since one rank computes a row and all receive the same bits, the replicas cannot
// drift.  (Nothing waits inside the kernel: the ranks synchronise before and after it.)
constexpr int kMaxPeers = 16;
struct PeerPtrs {
  const float *gq[kMaxPeers];
  float *q[kMaxPeers];
};
__global__ void __launch_bounds__(256)
apply_slice_kernel(PeerPtrs pp, int world, int self, const float *__restrict__ scale, int64_t j0, int64_t j1, int k4,
                   float eta, float lam2, float xi, int clip, float gmul, int32_t *flags) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  bool bad = false;
  for (int64_t j = j0 + (int64_t)blockIdx.x * blockDim.x + threadIdx.x; j < j1; j += stride) {
    const float sc = __ldg(scale + j / k4) * gmul;
    float4 gv = *(reinterpret_cast<const float4 *>(pp.gq[0]) + j);
    for (int r = 1; r < world; ++r) {
      const float4 a = *(reinterpret_cast<const float4 *>(pp.gq[r]) + j);
      gv.x += a.x; gv.y += a.y; gv.z += a.z; gv.w += a.w;
    }
    const float4 x = reinterpret_cast<const float4 *>(pp.q[self])[j];
    float xs[4] = {x.x, x.y, x.z, x.w};
    const float gs[4] = {gv.x, gv.y, gv.z, gv.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float d = fmaf(gs[q], sc, -lam2 * xs[q]);
      bad |= !isfinite(d);
      d = clip_dir(d, xi, clip);
      xs[q] = fmaf(eta, d, xs[q]);
      bad |= !isfinite(xs[q]);
    }
    const float4 nx = make_float4(xs[0], xs[1], xs[2], xs[3]);
    for (int r = 0; r < world; ++r) reinterpret_cast<float4 *>(pp.q[r])[j] = nx;
  }
  if (bad) flags[FLAG_NONFINITE] = 1;
}

__global__ void __launch_bounds__(256)
convert_kernel(const float *__restrict__ A, __nv_bfloat16 *__restrict__ Ab, int64_t na4,
               const float *__restrict__ B, __nv_bfloat16 *__restrict__ Bb, int64_t nb4) {
  const int64_t total = na4 + nb4;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
    const bool first = i < na4;
    const int64_t j = first ? i : i - na4;
    const float4 x = __ldg(reinterpret_cast<const float4 *>(first ? A : B) + j);
    __nv_bfloat162 lo = __floats2bfloat162_rn(x.x, x.y);
    __nv_bfloat162 hi = __floats2bfloat162_rn(x.z, x.w);
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t *>(&lo);
    pk.y = *reinterpret_cast<uint32_t *>(&hi);
    reinterpret_cast<uint2 *>(first ? Ab : Bb)[j] = pk;
  }
}

// ---- loss reductions (double, fixed order) ----------------------------------------------------------
constexpr int RED_BLOCKS = 256;

__device__ __forceinline__ double block_sum(double v) {
  __shared__ double ws[32];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if (lane == 0) ws[w] = v;
  __syncthreads();
  double t = 0.0;
  if (w == 0) {
    t = lane < (int)(blockDim.x >> 5) ? ws[lane] : 0.0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
  }
  return t;  // valid in warp 0
}

// out[blockIdx.x] = sum of in over this block's contiguous slice
__global__ void __launch_bounds__(256) reduce_slices_kernel(const double *__restrict__ in, int64_t n,
                                                             double *__restrict__ out) {
  const int64_t per = (n + gridDim.x - 1) / gridDim.x;
  const int64_t lo = (int64_t)blockIdx.x * per, hi = lo + per < n ? lo + per : n;
  double v = 0.0;
  for (int64_t i = lo + threadIdx.x; i < hi; i += blockDim.x) v += in[i];
  v = block_sum(v);
  if (threadIdx.x == 0) out[blockIdx.x] = v;
}

__global__ void __launch_bounds__(256) sqnorm_slices_kernel(const float *__restrict__ A, int64_t na,
                                                             const float *__restrict__ B, int64_t nb,
                                                             double *__restrict__ out) {
  const int64_t n = na + nb;
  const int64_t per = (n + gridDim.x - 1) / gridDim.x;
  const int64_t lo = (int64_t)blockIdx.x * per, hi = lo + per < n ? lo + per : n;
  double v = 0.0;
  for (int64_t i = lo + threadIdx.x; i < hi; i += blockDim.x) {
    const double x = (double)(i < na ? A[i] : B[i - na]);
    v += x * x;
  }
  v = block_sum(v);
  if (threadIdx.x == 0) out[blockIdx.x] = v;
}

// out2[0] = sum a[0..RED_BLOCKS), out2[1] = sum b[0..RED_BLOCKS)
__global__ void __launch_bounds__(256) reduce_final_kernel(const double *__restrict__ a,
                                                            const double *__restrict__ b,
                                                            double *__restrict__ out2) {
  double va = threadIdx.x < RED_BLOCKS ? a[threadIdx.x] : 0.0;
  double vb = threadIdx.x < RED_BLOCKS ? b[threadIdx.x] : 0.0;
  va = block_sum(va);
  vb = block_sum(vb);
  if (threadIdx.x == 0) { out2[0] = va; out2[1] = vb; }
}

// *out += sum a[0..RED_BLOCKS)
__global__ void __launch_bounds__(256) reduce_add_kernel(const double *__restrict__ a, double *__restrict__ out) {
  double v = threadIdx.x < RED_BLOCKS ? a[threadIdx.x] : 0.0;
  v = block_sum(v);
  if (threadIdx.x == 0) *out += v;
}

// ---- dispatch -------------------------------------------------------------------------------------------
template <int KP, bool BF16, int MODE>
cudaError_t launch_pass_t(cudaStream_t st, const Side &sd, const void *stage, const void *gather, int k,
                          float *G, float *partial, float *e_out, double *red) {
  if (sd.nseg <= 0) return cudaSuccess;
  const int wpb = 2;  // small CTAs: segments differ in length, a CTA lives as long as its longest one
  const int grid = (sd.nseg + wpb - 1) / wpb;
  pass_kernel<KP, BF16, MODE><<<grid, wpb * 32, 0, st>>>(sd.segs, sd.nseg, sd.idx, sd.val, stage, gather, k, G,
                                                         partial, e_out, red);
  return cudaGetLastError();
}

template <bool BF16, int MODE>
cudaError_t launch_pass_k(cudaStream_t st, const Side &sd, const void *stage, const void *gather, int k,
                          float *G, float *partial, float *e_out, double *red) {
  if (k <= 16) return launch_pass_t<16, BF16, MODE>(st, sd, stage, gather, k, G, partial, e_out, red);
  if (k <= 32) return launch_pass_t<32, BF16, MODE>(st, sd, stage, gather, k, G, partial, e_out, red);
  if (k <= 64) return launch_pass_t<64, BF16, MODE>(st, sd, stage, gather, k, G, partial, e_out, red);
  if (k <= 128) return launch_pass_t<128, BF16, MODE>(st, sd, stage, gather, k, G, partial, e_out, red);
  return launch_pass_t<256, BF16, MODE>(st, sd, stage, gather, k, G, partial, e_out, red);
}

#include "pass_staged.cuh"

// Staged gradient pass for every (KP, precision) whose factor row fits the copy mapping (<= 512 B).
// Chunk depth measured on B200: two stages; 16-row chunks for 256-byte rows and wider (more CTAs
// per SM matter more than deeper chunks), 32-row chunks below.  Returns cudaErrorNotSupported when
// there is no staged instantiation (fp32 with k > 128): the caller then uses the direct kernel.
template <bool ENTRY>
cudaError_t launch_staged_e(tsid_template *t, const Side &sd, const void *stage, const void *gather, float *G) {
  if (sd.nseg <= 0) return cudaSuccess;
  const int k = t->cfg.k;
  if (t->cfg.precision == TSID_BF16_SHADOW) {
    if (k <= 16) return launch_staged_v<16, true, 2, 32, ENTRY>(t, sd, stage, gather, G);
    if (k <= 32) return launch_staged_v<32, true, 2, 32, ENTRY>(t, sd, stage, gather, G);
    if (k <= 64) return launch_staged_v<64, true, 2, 32, ENTRY>(t, sd, stage, gather, G);
    if (k <= 128) return launch_staged_v<128, true, 2, 16, ENTRY>(t, sd, stage, gather, G);
    return launch_staged_v<256, true, 2, 16, ENTRY>(t, sd, stage, gather, G);
  }
  if (k <= 16) return launch_staged_v<16, false, 2, 32, ENTRY>(t, sd, stage, gather, G);
  if (k <= 32) return launch_staged_v<32, false, 2, 32, ENTRY>(t, sd, stage, gather, G);
  if (k <= 64) return launch_staged_v<64, false, 2, 16, ENTRY>(t, sd, stage, gather, G);
  if (k <= 128) return launch_staged_v<128, false, 2, 16, ENTRY>(t, sd, stage, gather, G);
  return cudaErrorNotSupported;
}

cudaError_t launch_staged(tsid_template *t, const Side &sd, const void *stage, const void *gather, float *G) {
  if (t->cfg.clip == TSID_CLIP_ASYM_ENTRY) return launch_staged_e<true>(t, sd, stage, gather, G);
  return launch_staged_e<false>(t, sd, stage, gather, G);
}

template <int MODE>
cudaError_t launch_pass(tsid_template *t, const Side &sd, const void *stage, const void *gather, float *G,
                        float *e_out, double *red) {
  if (MODE == MODE_GRAD) {
    cudaError_t e = launch_staged(t, sd, stage, gather, G);
    if (e != cudaErrorNotSupported) return e;
  }
  const int k = t->cfg.k;
  if (t->cfg.precision == TSID_BF16_SHADOW)
    return launch_pass_k<true, MODE>(t->stream, sd, stage, gather, k, G, t->partial, e_out, red);
  return launch_pass_k<false, MODE>(t->stream, sd, stage, gather, k, G, t->partial, e_out, red);
}

inline void prof_mark(tsid_template *t, int which) {
  if (t->prof.on && t->prof.nsteps < kProfSteps)
    cudaEventRecord(t->prof.ev[t->prof.nsteps * EV_PER_STEP + which], t->stream);
}

inline int ew_grid(int64_t n) {
  int64_t g = (n + 255) / 256;
  if (g < 1) g = 1;
  if (g > 148 * 8) g = 148 * 8;
  return (int)g;
}

}  // namespace

cudaError_t sparse_convert_shadow(tsid_template *t, const float *d_P, const float *d_Q) {
  if (t->cfg.precision != TSID_BF16_SHADOW) return cudaSuccess;
  const int64_t a4 = (int64_t)t->cfg.m * t->cfg.k / 4, b4 = (int64_t)t->cfg.n * t->cfg.k / 4;
  convert_kernel<<<ew_grid(a4 + b4), 256, 0, t->stream>>>(d_P, t->rowside.shadow, a4, d_Q, t->colside.shadow, b4);
  return cudaGetLastError();
}

// Reads the shadows when the precision says so (they must be current), else d_P / d_Q.
cudaError_t sparse_grad(tsid_template *t, const float *d_P, const float *d_Q, float *GP, float *GQ) {
  const bool bf = t->cfg.precision == TSID_BF16_SHADOW;
  const void *Ps = bf ? (const void *)t->rowside.shadow : (const void *)d_P;
  const void *Qs = bf ? (const void *)t->colside.shadow : (const void *)d_Q;
  prof_mark(t, EV_ROW0);
  CK(launch_pass<MODE_GRAD>(t, t->rowside, Ps, Qs, GP, nullptr, nullptr));
  prof_mark(t, EV_ROW1);
  if (t->rowside.nsplit > 0)
    fixup_kernel<<<t->rowside.nsplit, 128, 0, t->stream>>>(t->rowside.splits, t->rowside.nsplit, t->partial, GP,
                                                           t->cfg.k);
  prof_mark(t, EV_COL0);
  CK(launch_pass<MODE_GRAD>(t, t->colside, Qs, Ps, GQ, nullptr, nullptr));
  prof_mark(t, EV_COL1);
  if (t->colside.nsplit > 0)
    fixup_kernel<<<t->colside.nsplit, 128, 0, t->stream>>>(t->colside.splits, t->colside.nsplit, t->partial, GQ,
                                                           t->cfg.k);
  return cudaGetLastError();
}

cudaError_t sparse_update(tsid_template *t, float *d_P, float *d_Q, const float *GP, const float *GQ) {
  return sparse_update_scaled(t, d_P, d_Q, GP, GQ, t->rowside.scale, t->colside.scale);
}

cudaError_t update_launch(tsid_template *t, float *d_P, float *d_Q, const float *GP, const float *GQ,
                          const float *scale_p, const float *scale_q, const UpdHot &hot_p, const UpdHot &hot_q);

// the update with the 2 / s factors taken from the given arrays (one per row of P, one per row of Q)
cudaError_t sparse_update_scaled(tsid_template *t, float *d_P, float *d_Q, const float *GP, const float *GQ,
                                 const float *scale_p, const float *scale_q) {
  return update_launch(t, d_P, d_Q, GP, GQ, scale_p, scale_q, UpdHot(), UpdHot());
}

// the update that also adds the hybrid path's tile sums (see UpdHot)
cudaError_t sparse_update_hot(tsid_template *t, float *d_P, float *d_Q, const float *GP, const float *GQ,
                              const UpdHot &hot_p, const UpdHot &hot_q) {
  return update_launch(t, d_P, d_Q, GP, GQ, t->rowside.scale, t->colside.scale, hot_p, hot_q);
}

cudaError_t update_launch(tsid_template *t, float *d_P, float *d_Q, const float *GP, const float *GQ,
                          const float *scale_p, const float *scale_q, const UpdHot &hot_p, const UpdHot &hot_q) {
  const tsid_config_t &c = t->cfg;
  UpdSide a{d_P, GP, scale_p, t->rowside.shadow, (int64_t)c.m * c.k / 4, hot_p};
  UpdSide b{d_Q, GQ, scale_q, t->colside.shadow, (int64_t)c.n * c.k / 4, hot_q};
  prof_mark(t, EV_UPD0);
  // entry-wise clip: the passes already delivered the sum of clipped per-entry directions (regulariser
  // included), so the update is x += eta * G / s   (scale holds 2 / s)
  const bool entry = c.clip == TSID_CLIP_ASYM_ENTRY;
  if (hot_p.rank_of || hot_q.rank_of) {
    if (a.n4 > 0)
      update_kernel<true><<<ew_grid(a.n4), 256, 0, t->stream>>>(a, a, c.k / 4, c.eta, entry ? 0.f : 2.0f * c.lambda, c.xi,
                                                                entry ? (int)TSID_CLIP_NONE : c.clip, entry ? 0.5f : 1.0f, t->flags);
    if (b.n4 > 0)
      update_kernel<true><<<ew_grid(b.n4), 256, 0, t->stream>>>(b, b, c.k / 4, c.eta, entry ? 0.f : 2.0f * c.lambda, c.xi,
                                                                entry ? (int)TSID_CLIP_NONE : c.clip, entry ? 0.5f : 1.0f, t->flags);
  } else
    update_kernel<false><<<ew_grid(a.n4 + b.n4), 256, 0, t->stream>>>(a, b, c.k / 4, c.eta, entry ? 0.f : 2.0f * c.lambda, c.xi,
                                                                      entry ? (int)TSID_CLIP_NONE : c.clip, entry ? 0.5f : 1.0f,
                                                                      t->flags);
  prof_mark(t, EV_UPD1);
  if (t->prof.on && t->prof.nsteps < kProfSteps) t->prof.nsteps++;
  return cudaGetLastError();
}

__global__ void counts_kernel(const int64_t *__restrict__ ptr, int32_t nrows, int32_t *__restrict__ cnt) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nrows; i += (int64_t)gridDim.x * blockDim.x)
    cnt[i] = (int32_t)(ptr[i + 1] - ptr[i]);
}
// scale = 2 / s with s = max(1, count) under NORM_COUNT, 1 otherwise (the same rule as at create)
__global__ void scale_kernel(const int32_t *__restrict__ cnt, int32_t nrows, int norm_count, float *__restrict__ scale) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nrows; i += (int64_t)gridDim.x * blockDim.x) {
    const int32_t c = cnt[i];
    scale[i] = 2.0f / ((norm_count && c > 1) ? (float)c : 1.0f);
  }
}

// byte copies of the value streams; flags[FLAG_RANGE] if a value is not an integer in [0, 255]
__global__ void pack_u8_kernel(const float *__restrict__ v, int64_t n, uint8_t *__restrict__ o, int32_t *flags) {
  bool bad = false;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const float x = v[i];
    const int q = (int)x;
    if (!(x >= 0.f && x <= 255.f) || (float)q != x) bad = true;
    o[i] = (uint8_t)q;
  }
  if (bad) flags[FLAG_RANGE] = 1;
}

cudaError_t sparse_pack_values_u8(tsid_template *t, int32_t *h_bad) {
  const int64_t nnz = t->cfg.nnz;
  CK(cudaMemsetAsync(t->flags + FLAG_RANGE, 0, sizeof(int32_t), t->stream));
  if (nnz > 0) {
    pack_u8_kernel<<<ew_grid(nnz), 256, 0, t->stream>>>(t->rowside.val, nnz, const_cast<uint8_t *>(t->rowside.val8), t->flags);
    pack_u8_kernel<<<ew_grid(nnz), 256, 0, t->stream>>>(t->colside.val, nnz, const_cast<uint8_t *>(t->colside.val8), t->flags);
  }
  CK(cudaGetLastError());
  CK(cudaMemcpyAsync(h_bad, t->flags + FLAG_RANGE, sizeof(int32_t), cudaMemcpyDeviceToHost, t->stream));
  CK(cudaStreamSynchronize(t->stream));
  if (*h_bad) CK(cudaMemsetAsync(t->flags + FLAG_RANGE, 0, sizeof(int32_t), t->stream));
  return cudaSuccess;
}

cudaError_t sparse_counts(tsid_template *t, const Side &sd, int32_t *d_cnt) {
  counts_kernel<<<ew_grid(sd.nrows), 256, 0, t->stream>>>(sd.ptr, sd.nrows, d_cnt);
  return cudaGetLastError();
}
cudaError_t sparse_scale_from_counts(tsid_template *t, Side &sd, int norm_mode, const int32_t *d_cnt) {
  scale_kernel<<<ew_grid(sd.nrows), 256, 0, t->stream>>>(d_cnt, sd.nrows, norm_mode == TSID_NORM_COUNT, sd.scale);
  return cudaGetLastError();
}

// P side: the usual update from the local sums.  Q side: rows [n rank / world, n (rank + 1) / world) through
// apply_slice_kernel.
cudaError_t sparse_apply_sliced(tsid_template *t, float *d_P, const float *GP, float *const *h_Q, const float *const *h_GQ,
                                int rank, int world) {
  const tsid_config_t &c = t->cfg;
  const bool entry = c.clip == TSID_CLIP_ASYM_ENTRY;
  const float lam2 = entry ? 0.f : 2.0f * c.lambda, gmul = entry ? 0.5f : 1.0f;
  const int clip = entry ? (int)TSID_CLIP_NONE : (int)c.clip;
  UpdSide a{d_P, GP, t->rowside.scale, t->rowside.shadow, (int64_t)c.m * c.k / 4, UpdHot()};
  UpdSide none{nullptr, nullptr, nullptr, nullptr, 0, UpdHot()};
  prof_mark(t, EV_UPD0);
  if (a.n4 > 0) update_kernel<false><<<ew_grid(a.n4), 256, 0, t->stream>>>(a, none, c.k / 4, c.eta, lam2, c.xi, clip, gmul, t->flags);
  PeerPtrs pp;
  for (int r = 0; r < kMaxPeers; ++r) { pp.gq[r] = nullptr; pp.q[r] = nullptr; }
  for (int r = 0; r < world; ++r) { pp.gq[r] = h_GQ[r]; pp.q[r] = h_Q[r]; }
  const int k4 = c.k / 4;
  const int64_t r0 = (int64_t)c.n * rank / world, r1 = (int64_t)c.n * (rank + 1) / world;
  if (r1 > r0)
    apply_slice_kernel<<<ew_grid((r1 - r0) * k4), 256, 0, t->stream>>>(pp, world, rank, t->colside.scale, r0 * k4, r1 * k4,
                                                                     k4, c.eta, lam2, c.xi, clip, gmul, t->flags);
  prof_mark(t, EV_UPD1);
  if (t->prof.on && t->prof.nsteps < kProfSteps) t->prof.nsteps++;
  return cudaGetLastError();
}

cudaError_t sparse_residuals(tsid_template *t, const float *d_P, const float *d_Q, float *d_e) {
  const bool bf = t->cfg.precision == TSID_BF16_SHADOW;
  CK(sparse_convert_shadow(t, d_P, d_Q));
  const void *Ps = bf ? (const void *)t->rowside.shadow : (const void *)d_P;
  const void *Qs = bf ? (const void *)t->colside.shadow : (const void *)d_Q;
  return launch_pass<MODE_RESID>(t, t->rowside, Ps, Qs, nullptr, d_e, nullptr);
}

// d_out2[0] = SSE, d_out2[1] = |P|_F^2 + |Q|_F^2 (device doubles inside t->red)
cudaError_t sparse_loss(tsid_template *t, const float *d_P, const float *d_Q, double *d_out2) {
  const bool bf = t->cfg.precision == TSID_BF16_SHADOW;
  CK(sparse_convert_shadow(t, d_P, d_Q));
  const void *Ps = bf ? (const void *)t->rowside.shadow : (const void *)d_P;
  const void *Qs = bf ? (const void *)t->colside.shadow : (const void *)d_Q;
  double *warp_part = t->red + 2 + 2 * RED_BLOCKS;
  double *sl_a = t->red + 2, *sl_b = t->red + 2 + RED_BLOCKS;
  CK(launch_pass<MODE_LOSS>(t, t->rowside, Ps, Qs, nullptr, nullptr, warp_part));
  reduce_slices_kernel<<<RED_BLOCKS, 256, 0, t->stream>>>(warp_part, t->rowside.nseg, sl_a);
  sqnorm_slices_kernel<<<RED_BLOCKS, 256, 0, t->stream>>>(d_P, (int64_t)t->cfg.m * t->cfg.k, d_Q,
                                                         (int64_t)t->cfg.n * t->cfg.k, sl_b);
  reduce_final_kernel<<<1, 256, 0, t->stream>>>(sl_a, sl_b, d_out2);
  return cudaGetLastError();
}

// One side's gather-reduce pass on its own (used by the Stage II extension): G[row] = sum over the
// row's entries of e * gathered row, e = val - staged row . gathered row; fp32 or bf16 per t->cfg.
cudaError_t sparse_side_grad(tsid_template *t, const Side &sd, const void *stage, const void *gather, float *G) {
  CK(launch_pass<MODE_GRAD>(t, sd, stage, gather, G, nullptr, nullptr));
  if (sd.nsplit > 0) fixup_kernel<<<sd.nsplit, 128, 0, t->stream>>>(sd.splits, sd.nsplit, t->partial, G, t->cfg.k);
  return cudaGetLastError();
}

// d_out[0] += sum over the side's entries of e^2 (fixed order inside; `red` needs 2 + 2*256 + nseg doubles)
cudaError_t sparse_side_sse(tsid_template *t, const Side &sd, const void *stage, const void *gather, double *red,
                            double *d_out) {
  double *warp_part = red + 2 + 2 * RED_BLOCKS, *sl_a = red + 2;
  CK(launch_pass<MODE_LOSS>(t, sd, stage, gather, nullptr, nullptr, warp_part));
  reduce_slices_kernel<<<RED_BLOCKS, 256, 0, t->stream>>>(warp_part, sd.nseg, sl_a);
  reduce_add_kernel<<<1, 256, 0, t->stream>>>(sl_a, d_out);
  return cudaGetLastError();
}

// ---- mini-batch template -------------------------------------------------------------------------------
// rows' = batch * m + row, cols' = batch * n + col; flags[FLAG_RANGE] if a row, column or batch number is out of range
__global__ void virtual_coo_kernel(const int32_t *__restrict__ rows, const int32_t *__restrict__ cols,
                                   const int32_t *__restrict__ batch, int64_t nnz, int32_t m, int32_t n, int32_t nb,
                                   int32_t *__restrict__ vrows, int32_t *__restrict__ vcols, int32_t *flags) {
  bool bad = false;
  for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < nnz; t += (int64_t)gridDim.x * blockDim.x) {
    const int32_t r = rows[t], c = cols[t], b = batch[t];
    const bool ok = r >= 0 && r < m && c >= 0 && c < n && b >= 0 && b < nb;
    bad |= !ok;
    vrows[t] = ok ? b * m + r : 0;
    vcols[t] = ok ? b * n + c : 0;
  }
  if (bad) flags[FLAG_RANGE] = 1;
}
// out[b] = scan[b * stride], b = 0 .. nb
__global__ void sample_scan_kernel(const uint32_t *__restrict__ scan, int nb, int64_t stride, int32_t *__restrict__ out) {
  for (int b = blockIdx.x * blockDim.x + threadIdx.x; b <= nb; b += gridDim.x * blockDim.x) out[b] = (int32_t)scan[(int64_t)b * stride];
}

cudaError_t batch_virtual_coo(tsid_template *t, const int32_t *d_rows, const int32_t *d_cols, const int32_t *d_batch) {
  const tsid_config_t &c = t->cfg;
  CK(cudaMemsetAsync(t->flags, 0, sizeof(int32_t) * FLAG_COUNT, t->stream));
  if (c.nnz > 0)
    virtual_coo_kernel<<<ew_grid(c.nnz), 256, 0, t->stream>>>(d_rows, d_cols, d_batch, c.nnz, c.m, c.n, t->n_batches, t->vrows,
                                                               t->vcols, t->flags);
  return cudaGetLastError();
}

// Right after build_segments of one side: where each batch's segments and split rows begin (the scans of that call are
// still in the scratch).  The side's rows are the virtual ones, batch b owning [b * rows, (b + 1) * rows).
cudaError_t batch_ranges(tsid_template *t, const LayoutScratch &s, bool colside) {
  const int nb = t->n_batches;
  const int64_t stride = colside ? t->cfg.n : t->cfg.m;
  int32_t *d_tmp = reinterpret_cast<int32_t *>(s.hist);   // 2 (nb + 1) words of a scratch array nothing else uses now
  sample_scan_kernel<<<(nb + 256) / 256, 256, 0, t->stream>>>(s.scanA, nb, stride, d_tmp);
  sample_scan_kernel<<<(nb + 256) / 256, 256, 0, t->stream>>>(s.scanC, nb, stride, d_tmp + nb + 1);
  CK(cudaGetLastError());
  CK(cudaMemcpyAsync(colside ? t->bseg_col : t->bseg_row, d_tmp, sizeof(int32_t) * (nb + 1), cudaMemcpyDeviceToHost, t->stream));
  CK(cudaMemcpyAsync(colside ? t->bsplit_col : t->bsplit_row, d_tmp + nb + 1, sizeof(int32_t) * (nb + 1), cudaMemcpyDeviceToHost,
                     t->stream));
  return cudaStreamSynchronize(t->stream);
}

cudaError_t sparse_batch_step(tsid_template *t, int b, float *d_P, float *d_Q, float *GP, float *GQ) {
  const tsid_config_t &c = t->cfg;
  const bool bf = c.precision == TSID_BF16_SHADOW;
  CK(sparse_convert_shadow(t, d_P, d_Q));
  const size_t esz = bf ? sizeof(__nv_bfloat16) : sizeof(float);
  const char *Ps = bf ? reinterpret_cast<const char *>(t->rowside.shadow) : reinterpret_cast<const char *>(d_P);
  const char *Qs = bf ? reinterpret_cast<const char *>(t->colside.shadow) : reinterpret_cast<const char *>(d_Q);
  // the layout numbers this batch's rows b * m + i and its columns b * n + j: shift the bases by that many rows so that
  // the kernels' row arithmetic lands on row i of the real arrays (the shifted pointers are only ever used with those offsets)
  const ptrdiff_t ro = (ptrdiff_t)b * c.m * c.k, co = (ptrdiff_t)b * c.n * c.k;
  const void *Pv = Ps - ro * (ptrdiff_t)esz, *Qv = Qs - co * (ptrdiff_t)esz;
  Side rs = t->rowside, cs = t->colside;
  rs.segs += t->bseg_row[b]; rs.nseg = t->bseg_row[b + 1] - t->bseg_row[b];
  rs.splits += t->bsplit_row[b]; rs.nsplit = t->bsplit_row[b + 1] - t->bsplit_row[b];
  cs.segs += t->bseg_col[b]; cs.nseg = t->bseg_col[b + 1] - t->bseg_col[b];
  cs.splits += t->bsplit_col[b]; cs.nsplit = t->bsplit_col[b + 1] - t->bsplit_col[b];
  CK(sparse_side_grad(t, rs, Pv, Qv, GP - ro));
  CK(sparse_side_grad(t, cs, Qv, Pv, GQ - co));
  return sparse_update_scaled(t, d_P, d_Q, GP, GQ, t->rowside.scale + (size_t)b * c.m, t->colside.scale + (size_t)b * c.n);
}

int sparse_launches_per_step(const tsid_template *t) {
  return (t->cfg.precision == TSID_BF16_SHADOW ? 1 : 0) + 2 + (t->rowside.nsplit > 0) + (t->colside.nsplit > 0) + 1;
}

}  // namespace tsid
