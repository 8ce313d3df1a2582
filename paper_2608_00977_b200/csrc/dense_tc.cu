// Dense tensor-core variant of the gradient step (Sec. 5.1, "Regularizing Sparse RMF Updates for
// Tensor Cores": the dominant work becomes dense tiles S = P Q^T around which the sparse structure
// is only a mask).  For templates dense enough that this really is a dense contraction:
//
//   pass A (CTA per block of 128 rows i, loop over blocks of 128 columns j):
//       S = P_blk Q_blk^T            tcgen05.mma, A = the CTA's own factor block held in TMEM for the whole
//                                    kernel, B = the Q tile in shared memory (TMA), fp32 accumulator in TMEM
//       E = M .* (R - S)             epilogue warps: S from TMEM, the R tile (fp16, NaN = unobserved) from
//                                    shared memory (TMA); E goes back to TMEM as packed bf16, in place
//       G_P_blk += E Q_blk           tcgen05.mma with A = E read from TMEM, accumulating in TMEM over the
//                                    whole j loop
//   pass B: the same kernel on (Q, P, R^T) gives G_Q.
//
// S is computed in both passes (four GEMMs instead of three) so that each gradient block has one
// owner and a fixed summation order: no atomics.  Both products take their A operand from TMEM: a
// 128 x 128 x 16 MMA whose A comes from shared memory was measured at ~129 clocks on this part against
// ~73 with A in TMEM (64 is the tensor pipe's own time), so the owner block is copied to TMEM once
// and E never leaves it.  The Y tile (128 rows j x K columns, 128-byte-swizzled as TMA writes it)
// serves both products: K-major as B of the first (contraction over the factor index) and MN-major as
// B of the second (contraction over j), so no transposed copy of the factors exists.  When there are
// fewer row blocks than SMs the column range is split over several CTAs per row block; each writes its
// own partial gradient block and a small kernel adds them in a fixed order.  Every mbarrier wait is
// bounded by a cycle budget; on expiry the CTA raises FLAG_TIMEOUT, stops issuing, and still frees its
// TMEM before it returns.
#include <cuda.h>
#include <cuda_fp16.h>

#include <new>

#include "tsid_internal.cuh"

namespace tsid {

struct DenseState {
  __half *R = nullptr, *RT = nullptr;              // [m*n], [n*m]; NaN = not observed
  float *gpart = nullptr;                          // [(MAX_SPLIT - 1) * max(m, n) * k] partial gradient blocks
  CUtensorMap tmP, tmQ, tmR, tmRT;
};

namespace {

#define CK(x)                         \
  do {                                \
    cudaError_t e_ = (x);             \
    if (e_ != cudaSuccess) return e_; \
  } while (0)

constexpr int BLK = 128;                 // tile edge (rows of one X half, rows of Y per iteration)
constexpr int MAX_SPLIT = 4;             // CTAs sharing one row block (each takes a range of column blocks)
#include "tc_common.cuh"

template <int K>
struct Smem {
  static constexpr int NSY = 3;                   // stages of the Y tile ring
  static constexpr int NSR = 4;                   // stages of the R tile ring
  static constexpr int XB = BLK * 128;            // one 64-column block of a 128-row tile: 16 KB
  static constexpr int Y_BYTES = (K / 64) * XB;   // Y block (128 x K bf16)
  static constexpr int R_BYTES = 2 * XB;          // R tile (128 x 128 fp16)
  static constexpr int OFF_Y = 0;
  static constexpr int OFF_R = OFF_Y + NSY * Y_BYTES;
  static constexpr int OFF_BAR = OFF_R + NSR * R_BYTES;
  static constexpr int TOTAL = OFF_BAR + 256 + 1024;  // barriers + slack for 1024-byte alignment
  // barrier indices
  static constexpr int B_XFULL = 0, B_YFULL = 1, B_YEMPTY = B_YFULL + NSY, B_RFULL = B_YEMPTY + NSY,
                       B_REMPTY = B_RFULL + NSR, B_SFULL = B_REMPTY + NSR, B_EFULL = B_SFULL + 2,
                       B_GFULL = B_EFULL + 2, B_COUNT = B_GFULL + 1;
  static_assert(B_COUNT * 8 <= 192, "barriers overlap the TMEM address slot");
  static_assert(TOTAL <= 232448, "shared memory of one CTA");
};

// TMEM columns (512 allocated): the CTA's X block as packed bf16 at 0 (K / 2 columns used), S tiles at
// 64 and 192 (fp32; the epilogue overwrites the first 32 columns of each 64-column half with the packed
// bf16 E values of that half), G block at 320 (fp32, K columns used).
constexpr uint32_t TM_X = 0, TM_S0 = 64, TM_S1 = 192, TM_G = 320;

// One pass: G_X[rows_x x K] = (M .* (R - X Y^T)) Y, R given as fp16 [rows_x][rows_y] with NaN = unobserved.
// CTA (ib, sp) owns rows [128 ib, 128 ib + 128) of X and the column blocks [NJ sp / nsplit,
// NJ (sp + 1) / nsplit) of Y; split 0 writes to G, split sp > 0 to its partial buffer.  Work item w is
// the w-th column block of the CTA; it uses S buffer and epilogue team w & 1, so the TMEM round trips of
// one item overlap with the tensor work of the next.
// Warps: 0 = TMA producer, 1 = MMA issuer (one thread), 2..17 = two epilogue teams of eight warps (two
// warps per TMEM lane quarter; a thread owns one row of the tile and half of its columns).
// TMEM reuse needs no barrier of its own: the MMAs of one CTA execute in issue order, and the first
// product of item w + 2 is issued after the second product of item w, which is the last reader of that
// S / E buffer.
template <int K>
__global__ void __launch_bounds__(576, 1)
dense_pass_kernel(const __nv_bfloat16 *__restrict__ Xg, const __grid_constant__ CUtensorMap tmY,
                  const __grid_constant__ CUtensorMap tmR, int rows_x, int rows_y, int nsplit,
                  float *__restrict__ G, float *__restrict__ Gpart, int32_t *__restrict__ flags,
                  const DenseChunk *__restrict__ chunks, const int32_t *__restrict__ ylist, long long wait_budget,
                  int stall_item) {
  using L = Smem<K>;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t sm0 = (s32(smem_dyn) + 1023u) & ~1023u;   // tiles need 1024-byte alignment
  unsigned char *smp = smem_dyn + (sm0 - s32(smem_dyn));
  const uint32_t bar0 = sm0 + L::OFF_BAR;
  volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smp + L::OFF_BAR + 192);
  auto bar = [&](int i) { return bar0 + 8u * i; };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Whole-matrix form: CTA (ib, sp) walks the column blocks [jb0, jb0 + NW) of a dense R.  Tile-list form
  // (chunks != nullptr): the CTA walks the NW stored tiles [t0, t0 + NW) of row block ib; tile t holds the
  // cells of (ib, ylist[t]) as one 128 x 128 block of the tile array behind tmR, and the CTA's result is a
  // partial gradient block of its own (the caller adds the blocks of a row block in chunk order).
  int row0, jb0, NW, t0 = 0;
  float *Gout;           // where row `row0 + r` of this CTA's result goes: Gout + (grow0 + r) * K
  int grow0;
  if (chunks) {
    const DenseChunk ck = chunks[blockIdx.x];
    row0 = ck.ib * BLK; jb0 = 0; NW = ck.nt; t0 = ck.t0;
    Gout = Gpart + (size_t)ck.slot * BLK * K; grow0 = 0;
  } else {
    const int ib = blockIdx.x / nsplit, sp = blockIdx.x % nsplit;
    row0 = ib * BLK;
    const int NJ = rows_y / BLK;
    jb0 = (int)((long long)NJ * sp / nsplit);
    NW = (int)((long long)NJ * (sp + 1) / nsplit) - jb0;
    Gout = sp == 0 ? G : Gpart + (size_t)(sp - 1) * rows_x * K; grow0 = row0;
  }

  if (threadIdx.x == 0) {
    mbar_init(bar(L::B_XFULL), 8);
    for (int s = 0; s < L::NSY; ++s) { mbar_init(bar(L::B_YFULL + s), 1); mbar_init(bar(L::B_YEMPTY + s), 1); }
    for (int s = 0; s < L::NSR; ++s) { mbar_init(bar(L::B_RFULL + s), 1); mbar_init(bar(L::B_REMPTY + s), 8); }
    for (int b = 0; b < 2; ++b) { mbar_init(bar(L::B_SFULL + b), 1); mbar_init(bar(L::B_EFULL + b), 8); }
    mbar_init(bar(L::B_GFULL), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(bar0 + 192u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tmX = tmem + TM_X;
  const uint32_t tmS[2] = {tmem + TM_S0, tmem + TM_S1};
  const uint32_t tmG = tmem + TM_G;
  bool ok = true;

  if (warp == 0) {
    // ---- TMA producer ---------------------------------------------------------------------------
    if (lane == 0) {
      int jb_next = (ylist && NW > 0) ? __ldg(ylist + t0) : jb0;
      for (int w = 0; w < NW && ok; ++w) {
        if (w == stall_item) break;   // test hook: the loads of this item and of all later ones are never issued
        const int jb = jb_next, ys = w % L::NSY, rs = w % L::NSR;
        if (w + 1 < NW) jb_next = ylist ? __ldg(ylist + t0 + w + 1) : jb + 1;
        if (w >= L::NSY) ok = mbar_wait(bar(L::B_YEMPTY + ys), ((w / L::NSY) - 1) & 1, wait_budget);
        if (!ok) break;
        mbar_expect_tx(bar(L::B_YFULL + ys), L::Y_BYTES);
        for (int c = 0; c < K / 64; ++c)
          tma_load_2d(sm0 + L::OFF_Y + ys * L::Y_BYTES + c * L::XB, &tmY, bar(L::B_YFULL + ys), c * 64, jb * BLK);
        if (w >= L::NSR) ok = mbar_wait(bar(L::B_REMPTY + rs), ((w / L::NSR) - 1) & 1, wait_budget);
        if (!ok) break;
        mbar_expect_tx(bar(L::B_RFULL + rs), L::R_BYTES);
        for (int c = 0; c < 2; ++c) {
          if (chunks) tma_load_2d(sm0 + L::OFF_R + rs * L::R_BYTES + c * L::XB, &tmR, bar(L::B_RFULL + rs), c * 64, (t0 + w) * BLK);
          else tma_load_2d(sm0 + L::OFF_R + rs * L::R_BYTES + c * L::XB, &tmR, bar(L::B_RFULL + rs), jb * BLK + c * 64, row0);
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---- MMA issuer -----------------------------------------------------------------------------
    if (lane == 0) {
      constexpr uint32_t ID1 = idesc_bf16(BLK), ID2 = idesc_bf16(K) | (1u << 16);   // second product: B is MN-major
      auto mma1 = [&](int w) -> bool {
        const int ys = w % L::NSY, b = w & 1;
        if (!mbar_wait(bar(L::B_YFULL + ys), (w / L::NSY) & 1, wait_budget)) return false;
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < K / 16; ++ks) {   // A: 16 factor columns = 8 TMEM columns of the X block
          const uint32_t off = (ks / 4) * L::XB + (ks % 4) * 32;
          tc_mma_ts(tmS[b], tmX + ks * 8, smem_desc(sm0 + L::OFF_Y + ys * L::Y_BYTES + off), ID1, ks > 0);
        }
        tc_commit(bar(L::B_SFULL + b));
        return true;
      };
      ok = mbar_wait(bar(L::B_XFULL), 0, wait_budget);
      if (ok && NW > 0) ok = mma1(0);
      for (int w = 0; w < NW && ok; ++w) {
        const int ys = w % L::NSY, b = w & 1;
        if (w + 1 < NW) ok = mma1(w + 1);
        if (ok) ok = mbar_wait(bar(L::B_EFULL + b), (w >> 1) & 1, wait_budget);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < BLK / 16; ++ks) {   // K of this product = the 128 columns j: 8 TMEM columns per step
          // A: E of column half ks / 4 sits in the first 32 columns of that half of the S buffer;
          // B[K = j][N = l] is the Y tile itself read MN-major: 16 rows j per step = 2048 B
          tc_mma_ts(tmG, tmS[b] + (ks / 4) * 64 + (ks % 4) * 8,
                    smem_desc_mn(sm0 + L::OFF_Y + ys * L::Y_BYTES + ks * 2048, L::XB), ID2, (w > 0 || ks > 0));
        }
        tc_commit(bar(L::B_YEMPTY + ys));
      }
      if (ok) tc_commit(bar(L::B_GFULL));
    }
    __syncwarp();
  } else {
    // ---- epilogue warps ---------------------------------------------------------------------------
    const int q = warp & 3;                 // TMEM lane quarter this warp may access
    const int team = (warp - 2) >> 3;       // which epilogue team
    const int h = ((warp - 2) & 7) >> 2;    // which half of the columns
    const int row = q * 32 + lane;          // row inside the tile
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    const uint32_t rrow0 = sm0 + L::OFF_R + h * L::XB + row * 128;   // this row in the R tile (block h)
    if (team == 0) {
      // the CTA's X block goes to TMEM once: lane = row, 32-bit column c = factor columns 2c, 2c + 1
      const uint4 *xrow = reinterpret_cast<const uint4 *>(Xg + (size_t)(row0 + row) * K + h * (K / 2));
#pragma unroll
      for (int c = 0; c < K / 64; ++c) {
        uint32_t xw[16];
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          const uint4 x4 = xrow[c * 4 + v];
          xw[4 * v] = x4.x; xw[4 * v + 1] = x4.y; xw[4 * v + 2] = x4.z; xw[4 * v + 3] = x4.w;
        }
        tc_st16(tmX + lane_off + h * (K / 4) + c * 16, xw);
      }
      tc_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(L::B_XFULL));
    }
    for (int w = team; w < NW && ok; w += 2) {
      const int b = w & 1, rs = w % L::NSR;
      ok = mbar_wait(bar(L::B_RFULL + rs), (w / L::NSR) & 1, wait_budget);                 // R tile has landed
      if (ok) ok = mbar_wait(bar(L::B_SFULL + b), (w >> 1) & 1, wait_budget);              // S is complete
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t rrow = rrow0 + rs * L::R_BYTES;
      uint32_t sv[2][32];
      tc_ld32_nowait(tmS[b] + lane_off + h * 64, sv[0]);
      tc_ld32_nowait(tmS[b] + lane_off + h * 64 + 32, sv[1]);
      tc_wait_ld();
#pragma unroll
      for (int c2 = 0; c2 < 2; ++c2) {
        uint32_t ew[16];
#pragma unroll
        for (int v = 0; v < 4; ++v) {   // 8 columns per 16-byte chunk of the swizzled R row
          const int chunk = c2 * 4 + v;
          uint32_t rw[4];
          asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                       : "=r"(rw[0]), "=r"(rw[1]), "=r"(rw[2]), "=r"(rw[3])
                       : "r"(rrow + (((uint32_t)chunk ^ (uint32_t)(row & 7)) << 4)));
#pragma unroll
          for (int p = 0; p < 4; ++p) {
            const float2 r2 = __half22float2(*reinterpret_cast<const __half2 *>(&rw[p]));
            float e0 = r2.x - __uint_as_float(sv[c2][v * 8 + 2 * p]);
            float e1 = r2.y - __uint_as_float(sv[c2][v * 8 + 2 * p + 1]);
            e0 = (e0 == e0) ? e0 : 0.f;   // unobserved cells carry NaN in R
            e1 = (e1 == e1) ? e1 : 0.f;
            __nv_bfloat162 pk = __floats2bfloat162_rn(e0, e1);
            ew[v * 4 + p] = *reinterpret_cast<uint32_t *>(&pk);
          }
        }
        // in place: this thread has already read all 64 S columns of its half
        tc_st16(tmS[b] + lane_off + h * 64 + c2 * 16, ew);
      }
      __syncwarp();   // every lane has its R values in registers: the stage can be refilled
      if (lane == 0) mbar_arrive(bar(L::B_REMPTY + rs));
      tc_wait_st();
      // one arrival per warp: every lane orders its TMEM accesses, then lane 0 signals for the warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(L::B_EFULL + b));
    }
    const bool writer = team == 0 && NW > 0;
    if (ok && writer) ok = __all_sync(0xffffffffu, mbar_wait(bar(L::B_GFULL), 0, wait_budget));
    if (ok && writer) {
      tc_fence_after();
      float *grow = Gout + (size_t)(grow0 + row) * K + h * (K / 2);
#pragma unroll
      for (int c = 0; c < K / 64; ++c) {
        uint32_t gv[32];
        tc_ld32(tmG + lane_off + h * (K / 2) + c * 32, gv);
#pragma unroll
        for (int v = 0; v < 8; ++v)
          *reinterpret_cast<uint4 *>(grow + c * 32 + v * 4) = make_uint4(gv[4 * v], gv[4 * v + 1], gv[4 * v + 2], gv[4 * v + 3]);
      }
    }
  }
  if (!ok && lane == 0) flags[FLAG_TIMEOUT] = 1;
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
}

// G[i] += part_0[i] + ... in this order (the partial blocks of the CTAs that shared a row block)
__global__ void add_partials_kernel(float4 *__restrict__ G, const float4 *__restrict__ part, size_t n4, int nparts) {
  size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
    float4 g = G[i];
    for (int p = 0; p < nparts; ++p) {
      const float4 a = part[(size_t)p * n4 + i];
      g.x += a.x; g.y += a.y; g.z += a.z; g.w += a.w;
    }
    G[i] = g;
  }
}

// ---- helpers: dense R, transposed shadows -----------------------------------------------------------
__global__ void fill_u32_kernel(uint32_t *p, size_t n, uint32_t v) {
  size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) p[i] = v;
}

// warp per CSR row: R[i][j] = fp16(r), RT[j][i] = fp16(r); flags[FLAG_RANGE] if |r| is beyond fp16
__global__ void scatter_dense_kernel(const int64_t *__restrict__ row_ptr, const int32_t *__restrict__ col_idx,
                                     const float *__restrict__ val, int m, int n, __half *__restrict__ R,
                                     __half *__restrict__ RT, int32_t *flags) {
  const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const int64_t nw = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t i = warp; i < m; i += nw) {
    for (int64_t p = row_ptr[i] + lane; p < row_ptr[i + 1]; p += 32) {
      const float r = val[p];
      if (!(fabsf(r) <= 65504.f)) flags[FLAG_RANGE] = 1;
      const __half hv = __float2half_rn(r);
      const int j = col_idx[p];
      R[(size_t)i * n + j] = hv;
      RT[(size_t)j * m + i] = hv;
    }
  }
}

// Number of CTAs per row block: fill the SMs when there are fewer row blocks than SMs, but leave every
// CTA at least four column blocks.
int dense_split(int rows_x, int rows_y) {
  const int nrb = rows_x / BLK, nj = rows_y / BLK;
  int sp = 148 / nrb;
  if (sp > MAX_SPLIT) sp = MAX_SPLIT;
  if (sp > nj / 4) sp = nj / 4;
  return sp < 1 ? 1 : sp;
}

template <int K>
cudaError_t launch_dense_pass(cudaStream_t st, const __nv_bfloat16 *X, const CUtensorMap &tmY,
                              const CUtensorMap &tmR, int rows_x, int rows_y, float *G, float *Gpart,
                              int32_t *flags, long long wait_budget, int stall_item) {
  auto kern = dense_pass_kernel<K>;
  CK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<K>::TOTAL));
  const int nrb = rows_x / BLK, nsplit = dense_split(rows_x, rows_y);
  kern<<<nrb * nsplit, 576, Smem<K>::TOTAL, st>>>(X, tmY, tmR, rows_x, rows_y, nsplit, G, Gpart, flags, nullptr, nullptr,
                                                  wait_budget, stall_item);
  if (nsplit > 1) {
    const size_t n4 = (size_t)rows_x * K / 4;
    add_partials_kernel<<<148 * 4, 256, 0, st>>>(reinterpret_cast<float4 *>(G), reinterpret_cast<const float4 *>(Gpart),
                                                n4, nsplit - 1);
  }
  return cudaGetLastError();
}

}  // namespace

bool dense_qualifies(const tsid_config_t &c) {
  return c.precision == TSID_BF16_SHADOW && (c.k == 64 || c.k == 128) && c.m % BLK == 0 && c.n % BLK == 0 &&
         (int64_t)c.m * c.n <= (int64_t)1 << 34;
}

void dense_carve(tsid_template *t, const tsid_config_t &c, Carver &cv) {
  DenseState *d = t->dense;
  const size_t mn = (size_t)c.m * c.n;
  __half *R = cv.take<__half>(mn), *RT = cv.take<__half>(mn);
  float *gpart = cv.take<float>((size_t)(MAX_SPLIT - 1) * (c.m > c.n ? c.m : c.n) * c.k);
  if (d) { d->R = R; d->RT = RT; d->gpart = gpart; }
}

DenseState *dense_new() { return new (std::nothrow) DenseState; }
void dense_delete(DenseState *d) { delete d; }

// After the layout pass: dense fp16 copies of R and R^T, tensor maps of the shadows and of R, R^T.
cudaError_t dense_build(tsid_template *t, int32_t *h_range_flag) {
  DenseState *d = t->dense;
  const tsid_config_t &c = t->cfg;
  cudaStream_t st = t->stream;
  const size_t words = (size_t)c.m * c.n / 2;   // m*n is a multiple of 128*128
  fill_u32_kernel<<<148 * 8, 256, 0, st>>>(reinterpret_cast<uint32_t *>(d->R), words, 0x7e007e00u);
  fill_u32_kernel<<<148 * 8, 256, 0, st>>>(reinterpret_cast<uint32_t *>(d->RT), words, 0x7e007e00u);
  scatter_dense_kernel<<<148 * 8, 256, 0, st>>>(t->row_ptr, t->col_idx, t->val_csr, c.m, c.n, d->R, d->RT, t->flags);
  CK(cudaGetLastError());
  CK(cudaMemcpyAsync(h_range_flag, t->flags + FLAG_RANGE, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  const CUtensorMapDataType BF = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, HF = CU_TENSOR_MAP_DATA_TYPE_FLOAT16;
  CK(make_map(&d->tmP, BF, t->rowside.shadow, c.m, c.k, BLK));
  CK(make_map(&d->tmQ, BF, t->colside.shadow, c.n, c.k, BLK));
  CK(make_map(&d->tmR, HF, d->R, c.m, c.n, BLK));
  CK(make_map(&d->tmRT, HF, d->RT, c.n, c.m, BLK));
  return cudaSuccess;
}

// two passes + the update kernels of the two sides, + one add per pass whose column range is split
int dense_launches_per_step(const tsid_template *t) {
  const tsid_config_t &c = t->cfg;
  return 4 + (dense_split(c.m, c.n) > 1) + (dense_split(c.n, c.m) > 1);
}

cudaError_t dense_make_map(void *map, bool half_not_bf16, void *base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  static_assert(sizeof(CUtensorMap) == 128, "tensor map size");
  return make_map(reinterpret_cast<CUtensorMap *>(map),
                  half_not_bf16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, base, rows, cols, box_rows);
}

cudaError_t dense_tiles_pass(cudaStream_t st, int k, const __nv_bfloat16 *X, const void *map_y, const void *map_r,
                             const DenseChunk *chunks, int nchunks, const int32_t *ylist, float *partial, int32_t *flags) {
  if (nchunks <= 0) return cudaSuccess;
  const CUtensorMap &tmY = *reinterpret_cast<const CUtensorMap *>(map_y);
  const CUtensorMap &tmR = *reinterpret_cast<const CUtensorMap *>(map_r);
  if (k == 128) {
    auto kern = dense_pass_kernel<128>;
    CK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<128>::TOTAL));
    kern<<<nchunks, 576, Smem<128>::TOTAL, st>>>(X, tmY, tmR, 0, 0, 1, nullptr, partial, flags, chunks, ylist, WAIT_CYCLES, -1);
  } else {
    auto kern = dense_pass_kernel<64>;
    CK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<64>::TOTAL));
    kern<<<nchunks, 576, Smem<64>::TOTAL, st>>>(X, tmY, tmR, 0, 0, 1, nullptr, partial, flags, chunks, ylist, WAIT_CYCLES, -1);
  }
  return cudaGetLastError();
}

// G_P and G_Q from the current bf16 shadows (which must be up to date).
cudaError_t dense_grad(tsid_template *t, float *GP, float *GQ) {
  DenseState *d = t->dense;
  const tsid_config_t &c = t->cfg;
  cudaStream_t st = t->stream;
  if (t->prof.on && t->prof.nsteps < kProfSteps) cudaEventRecord(t->prof.ev[t->prof.nsteps * EV_PER_STEP + EV_ROW0], st);
  const long long wb = t->dbg_wait_cycles > 0 ? t->dbg_wait_cycles : WAIT_CYCLES;
  const int stall = t->dbg_wait_cycles > 0 ? t->dbg_stall_item : -1;
  if (c.k == 128) CK(launch_dense_pass<128>(st, t->rowside.shadow, d->tmQ, d->tmR, c.m, c.n, GP, d->gpart, t->flags, wb, stall));
  else CK(launch_dense_pass<64>(st, t->rowside.shadow, d->tmQ, d->tmR, c.m, c.n, GP, d->gpart, t->flags, wb, stall));
  if (t->prof.on && t->prof.nsteps < kProfSteps) {
    cudaEventRecord(t->prof.ev[t->prof.nsteps * EV_PER_STEP + EV_ROW1], st);
    cudaEventRecord(t->prof.ev[t->prof.nsteps * EV_PER_STEP + EV_COL0], st);
  }
  if (c.k == 128) CK(launch_dense_pass<128>(st, t->colside.shadow, d->tmP, d->tmRT, c.n, c.m, GQ, d->gpart, t->flags, wb, stall));
  else CK(launch_dense_pass<64>(st, t->colside.shadow, d->tmP, d->tmRT, c.n, c.m, GQ, d->gpart, t->flags, wb, stall));
  if (t->prof.on && t->prof.nsteps < kProfSteps) cudaEventRecord(t->prof.ev[t->prof.nsteps * EV_PER_STEP + EV_COL1], st);
  return cudaSuccess;
}

}  // namespace tsid
