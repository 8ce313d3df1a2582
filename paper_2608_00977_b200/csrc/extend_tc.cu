// Stage II (Sec. 5.2, Eq. 10), the gradient GEMM fused with the Adam update, on the tensor cores:
//       G = U Q^T   (chunk columns x template columns, contraction over the rank k)
//       g = -2 G + 2 lambda C;  Adam update of C and its moments
// The paper runs Stage II's products in mixed precision (Sec. 5.2, Tensor Core acceleration of Stage II:
// half-precision operands, fp32 accumulation); this is that variant: U and Q are
// rounded to bf16, the products accumulate in fp32 in TMEM, and C and the Adam moments stay fp32.
//
// CTA = 128 rows of the chunk (its U block is converted and copied to TMEM once) x a range of
// 128-column tiles of C.  Warp 0 streams the Q tiles (bf16, TMA, 128-byte swizzle), warp 1's lane 0
// issues tcgen05.mma (A = U block from TMEM, B = Q tile, K-major), and two teams of eight warps take
// the finished 128 x 128 tiles alternately: a thread owns one row and 64 columns, reads G from TMEM
// sixteen columns at a time and streams C, m, v through it as float4s (a full 128-byte line per
// array and thread every two steps).  The kernel is bound by that stream (24 B per coefficient):
// the 8 MMAs of a tile cost ~800 clocks against ~17,000 clocks of HBM time per tile and SM.
// Every mbarrier wait is bounded by a cycle budget; on expiry the CTA raises FLAG_TIMEOUT, stops
// issuing and still frees its TMEM.
#include <cuda.h>

#include "tsid_internal.cuh"

namespace tsid {
namespace {

#define CK(x)                         \
  do {                                \
    cudaError_t e_ = (x);             \
    if (e_ != cudaSuccess) return e_; \
  } while (0)

#include "tc_common.cuh"

// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void tc_mma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

constexpr int BLK = 128;
constexpr int NSY = 4;   // stages of the Q tile ring
constexpr int STG_LD = 36;   // floats per staged row (32 + 4: float4-aligned, rows four banks apart)

template <int K>
struct ESmem {
  static constexpr int XB = BLK * 128;            // one 64-column block of a 128-row tile: 16 KB
  static constexpr int Y_BYTES = (K / 64) * XB;   // Q tile (128 x K bf16)
  static constexpr int OFF_STG = NSY * Y_BYTES;                     // per-warp staging of G: 16 warps x 32 x STG_LD floats
  static constexpr int OFF_BAR = OFF_STG + 16 * 32 * STG_LD * 4;
  static constexpr int TOTAL = OFF_BAR + 256 + 1024;
  static constexpr int B_XFULL = 0, B_YFULL = 1, B_YEMPTY = B_YFULL + NSY, B_SFULL = B_YEMPTY + NSY,
                       B_SEMPTY = B_SFULL + 2, B_COUNT = B_SEMPTY + 2;
  static_assert(B_COUNT * 8 <= 192, "barriers overlap the TMEM address slot");
};

// TMEM columns: U block (packed bf16, K / 2 columns) at 0, G tiles (fp32) at 64 and 192
constexpr uint32_t TM_U = 0, TM_G0 = 64, TM_G1 = 192;

__device__ __forceinline__ float adam_one(const AdamArgs &a, float acc, float c, float &mo, float &vo) {
  const float g = fmaf(a.lam2, c, -2.f * acc);
  mo = fmaf(a.b1, mo, (1.f - a.b1) * g);
  vo = fmaf(a.b2, vo, (1.f - a.b2) * g * g);
  return c - __fdividef(a.lr * (mo * a.c1), sqrtf(vo * a.c2) + a.eps);
}

template <int K>
__global__ void __launch_bounds__(576, 1)
adam_gemm_tc_kernel(const float *__restrict__ U, const __grid_constant__ CUtensorMap tmQ, int nc, int d, int nsplit,
                    float *__restrict__ Cm, float *__restrict__ Mo, float *__restrict__ Vo,
                    __nv_bfloat16 *__restrict__ Cb, AdamArgs aa, int32_t *__restrict__ flags) {
  using L = ESmem<K>;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t sm0 = (s32(smem_dyn) + 1023u) & ~1023u;
  unsigned char *smp = smem_dyn + (sm0 - s32(smem_dyn));
  const uint32_t bar0 = sm0 + L::OFF_BAR;
  volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smp + L::OFF_BAR + 192);
  auto bar = [&](int i) { return bar0 + 8u * i; };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ib = blockIdx.x / nsplit, sp = blockIdx.x % nsplit;
  const int row0 = ib * BLK;
  const int NJ = (d + BLK - 1) / BLK;
  const int jb0 = (int)((long long)NJ * sp / nsplit), jb1 = (int)((long long)NJ * (sp + 1) / nsplit);
  const int NW = jb1 - jb0;

  if (threadIdx.x == 0) {
    mbar_init(bar(L::B_XFULL), 8);
    for (int s = 0; s < NSY; ++s) { mbar_init(bar(L::B_YFULL + s), 1); mbar_init(bar(L::B_YEMPTY + s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(bar(L::B_SFULL + b), 1); mbar_init(bar(L::B_SEMPTY + b), 8); }
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
  const uint32_t tmU = tmem + TM_U;
  const uint32_t tmG[2] = {tmem + TM_G0, tmem + TM_G1};
  bool ok = true;

  if (warp == 0) {
    // ---- TMA producer: the Q tiles of this CTA's column range (rows past d arrive as zeros) -------
    if (lane == 0) {
      for (int w = 0; w < NW && ok; ++w) {
        const int ys = w % NSY;
        if (w >= NSY) ok = mbar_wait(bar(L::B_YEMPTY + ys), ((w / NSY) - 1) & 1);
        if (!ok) break;
        mbar_expect_tx(bar(L::B_YFULL + ys), L::Y_BYTES);
        for (int c = 0; c < K / 64; ++c)
          tma_load_2d(sm0 + ys * L::Y_BYTES + c * L::XB, &tmQ, bar(L::B_YFULL + ys), c * 64, (jb0 + w) * BLK);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---- MMA issuer -----------------------------------------------------------------------------
    if (lane == 0) {
      constexpr uint32_t ID = idesc_bf16(BLK);
      ok = mbar_wait(bar(L::B_XFULL), 0);
      for (int w = 0; w < NW && ok; ++w) {
        const int ys = w % NSY, b = w & 1;
        ok = mbar_wait(bar(L::B_YFULL + ys), (w / NSY) & 1);
        if (ok && w >= 2) ok = mbar_wait(bar(L::B_SEMPTY + b), ((w >> 1) - 1) & 1);   // the tile two back has been read
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < K / 16; ++ks) {
          const uint32_t off = (ks / 4) * L::XB + (ks % 4) * 32;
          tc_mma_ts(tmG[b], tmU + ks * 8, smem_desc(sm0 + ys * L::Y_BYTES + off), ID, ks > 0);
        }
        tc_commit(bar(L::B_SFULL + b));
        tc_commit(bar(L::B_YEMPTY + ys));
      }
    }
    __syncwarp();
  } else {
    // ---- epilogue warps ---------------------------------------------------------------------------
    const int q = warp & 3;
    const int team = (warp - 2) >> 3;
    const int h = ((warp - 2) & 7) >> 2;
    const int row = q * 32 + lane;
    const int gr = row0 + row;   // the row this thread converts into the U block
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    if (team == 0) {
      // the U block goes to TMEM as bf16: lane = row, 32-bit column c = rank columns 2c, 2c + 1
      const float4 *urow = reinterpret_cast<const float4 *>(U + (size_t)(gr < nc ? gr : 0) * K + h * (K / 2));
#pragma unroll
      for (int c = 0; c < K / 64; ++c) {
        uint32_t xw[16];
#pragma unroll
        for (int v = 0; v < 8; ++v) {
          float4 u4 = urow[c * 8 + v];
          if (gr >= nc) u4 = make_float4(0.f, 0.f, 0.f, 0.f);
          __nv_bfloat162 lo = __floats2bfloat162_rn(u4.x, u4.y), hi = __floats2bfloat162_rn(u4.z, u4.w);
          xw[2 * v] = *reinterpret_cast<uint32_t *>(&lo);
          xw[2 * v + 1] = *reinterpret_cast<uint32_t *>(&hi);
        }
        tc_st16(tmU + lane_off + h * (K / 4) + c * 16, xw);
      }
      tc_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(L::B_XFULL));
    }
    // each warp turns its 32 rows x 32 columns of G through shared memory, so that C, m and v are
    // streamed with the lanes along a row (four full 128-byte lines per instruction)
    float *stg = reinterpret_cast<float *>(smp + L::OFF_STG) + (warp - 2) * (32 * STG_LD);
    for (int w = team; w < NW && ok; w += 2) {
      const int b = w & 1;
      ok = __all_sync(0xffffffffu, mbar_wait(bar(L::B_SFULL + b), (w >> 1) & 1));
      if (!ok) break;
      tc_fence_after();
#pragma unroll
      for (int c32 = 0; c32 < 2; ++c32) {
        uint32_t gv[32];
        tc_ld32(tmG[b] + lane_off + h * 64 + c32 * 32, gv);
        if (c32 == 1) {   // this warp holds all it needs of the tile: the buffer may be overwritten
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar(L::B_SEMPTY + b));
        }
#pragma unroll
        for (int v = 0; v < 8; ++v)
          *reinterpret_cast<float4 *>(stg + lane * STG_LD + 4 * v) =
              make_float4(__uint_as_float(gv[4 * v]), __uint_as_float(gv[4 * v + 1]), __uint_as_float(gv[4 * v + 2]),
                          __uint_as_float(gv[4 * v + 3]));
        __syncwarp();
        const int col = (jb0 + w) * BLK + h * 64 + c32 * 32 + (lane & 7) * 4;
#pragma unroll
        for (int r0 = 0; r0 < 8; r0 += 4) {   // four rows per lane in flight: twelve independent 16-byte loads
          float4 c[4], mo[4], vo[4];
          bool in[4];
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            const int grow = row0 + q * 32 + (r0 + r) * 4 + (lane >> 3);
            in[r] = grow < nc && col < d;
            if (in[r]) {
              const size_t o = (size_t)grow * d + col;
              c[r] = __ldcs(reinterpret_cast<const float4 *>(Cm + o));
              mo[r] = __ldcs(reinterpret_cast<const float4 *>(Mo + o));
              vo[r] = __ldcs(reinterpret_cast<const float4 *>(Vo + o));
            }
          }
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            if (in[r]) {
              const int rr = (r0 + r) * 4 + (lane >> 3);
              const float4 g4 = *reinterpret_cast<const float4 *>(stg + rr * STG_LD + (lane & 7) * 4);
              const size_t o = (size_t)(row0 + q * 32 + rr) * d + col;
              c[r].x = adam_one(aa, g4.x, c[r].x, mo[r].x, vo[r].x);
              c[r].y = adam_one(aa, g4.y, c[r].y, mo[r].y, vo[r].y);
              c[r].z = adam_one(aa, g4.z, c[r].z, mo[r].z, vo[r].z);
              c[r].w = adam_one(aa, g4.w, c[r].w, mo[r].w, vo[r].w);
              __stcs(reinterpret_cast<float4 *>(Cm + o), c[r]);
              __stcs(reinterpret_cast<float4 *>(Mo + o), mo[r]);
              __stcs(reinterpret_cast<float4 *>(Vo + o), vo[r]);
              // the bf16 copy the next step's first product reads
              __nv_bfloat162 lo = __floats2bfloat162_rn(c[r].x, c[r].y), hi = __floats2bfloat162_rn(c[r].z, c[r].w);
              uint2 pk;
              pk.x = *reinterpret_cast<uint32_t *>(&lo);
              pk.y = *reinterpret_cast<uint32_t *>(&hi);
              __stcs(reinterpret_cast<uint2 *>(Cb + o), pk);
            }
          }
        }
        __syncwarp();   // the staging rows are rewritten by the next round
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

// ---- first product of a step: W = C Q (chunk columns x rank, contraction over the d template columns) --
// CTA = 128 rows of the chunk x one slice of d (split-K; the partial planes are added in split order by
// the caller).  Per 64 template columns: the C tile (128 x 64 bf16, K-major) and the Q tile (64 rows x
// K rank columns, read MN-major: its rows are the contraction index) arrive by TMA; four tcgen05.mma
// of 128 x K x 16 accumulate into one fp32 block in TMEM; after the slice, four warps store the block.
constexpr int WST = 6;   // stages of the (C tile, Q tile) ring

template <int K>
struct WSmem {
  static constexpr int A_BYTES = BLK * 128;        // 128 rows x 64 bf16
  static constexpr int B_BYTES = (K / 64) * 64 * 128;   // 64 rows x K bf16, in 64-column blocks
  static constexpr int STAGE = A_BYTES + B_BYTES;
  static constexpr int OFF_BAR = WST * STAGE;
  static constexpr int TOTAL = OFF_BAR + 256 + 1024;
  static constexpr int B_FULL = 0, B_EMPTY = WST, B_DONE = 2 * WST, B_COUNT = 2 * WST + 1;
  static_assert(B_COUNT * 8 <= 192, "barriers overlap the TMEM address slot");
};

template <int K>
__global__ void __launch_bounds__(192, 1)
w_gemm_tc_kernel(const __grid_constant__ CUtensorMap tmC, const __grid_constant__ CUtensorMap tmQ64, int nc, int d,
                 int nsplit, float *__restrict__ Wpart, size_t plane, int32_t *__restrict__ flags) {
  using L = WSmem<K>;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t sm0 = (s32(smem_dyn) + 1023u) & ~1023u;
  unsigned char *smp = smem_dyn + (sm0 - s32(smem_dyn));
  const uint32_t bar0 = sm0 + L::OFF_BAR;
  volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smp + L::OFF_BAR + 192);
  auto bar = [&](int i) { return bar0 + 8u * i; };
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ib = blockIdx.x / nsplit, sp = blockIdx.x % nsplit;
  const int NS = (d + 63) / 64;                                   // 64-column steps over d
  const int s0 = (int)((long long)NS * sp / nsplit), s1 = (int)((long long)NS * (sp + 1) / nsplit);
  const int NW = s1 - s0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < WST; ++s) { mbar_init(bar(L::B_FULL + s), 1); mbar_init(bar(L::B_EMPTY + s), 1); }
    mbar_init(bar(L::B_DONE), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 128;" ::"r"(bar0 + 192u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  bool ok = true;

  if (warp == 0) {
    if (lane == 0) {
      for (int w = 0; w < NW && ok; ++w) {
        const int st = w % WST;
        if (w >= WST) ok = mbar_wait(bar(L::B_EMPTY + st), ((w / WST) - 1) & 1);
        if (!ok) break;
        mbar_expect_tx(bar(L::B_FULL + st), L::STAGE);
        const uint32_t a = sm0 + st * L::STAGE;
        tma_load_2d(a, &tmC, bar(L::B_FULL + st), (s0 + w) * 64, ib * BLK);              // columns beyond d: zeros
        for (int c = 0; c < K / 64; ++c)
          tma_load_2d(a + L::A_BYTES + c * 64 * 128, &tmQ64, bar(L::B_FULL + st), c * 64, (s0 + w) * 64);   // rows beyond d: zeros
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t ID = idesc_bf16(K) | (1u << 16);   // B is MN-major
      for (int w = 0; w < NW && ok; ++w) {
        const int st = w % WST;
        ok = mbar_wait(bar(L::B_FULL + st), (w / WST) & 1);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a = sm0 + st * L::STAGE, b = a + L::A_BYTES;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)   // 16 template columns per step: 32 B along a C row, 16 rows (2048 B) of the Q tile
          tc_mma_ss(tmem, smem_desc(a + ks * 32), smem_desc_mn(b + ks * 2048, 64 * 128), ID, (w > 0 || ks > 0));
        tc_commit(bar(L::B_EMPTY + st));
      }
      if (ok) tc_commit(bar(L::B_DONE));
    }
    __syncwarp();
  } else {
    // ---- four warps store the accumulated block (a slice with no steps stores zeros) --------------------
    const int q = warp & 3;
    const int row = q * 32 + lane, gr = ib * BLK + row;
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    if (NW > 0) ok = __all_sync(0xffffffffu, mbar_wait(bar(L::B_DONE), 0));
    if (ok) {
      tc_fence_after();
      float *dst = Wpart + (size_t)sp * plane + (size_t)gr * K;
#pragma unroll
      for (int c = 0; c < K / 32; ++c) {
        uint32_t gv[32];
        if (NW > 0) tc_ld32(tmem + lane_off + c * 32, gv);
        else {
#pragma unroll
          for (int v = 0; v < 32; ++v) gv[v] = 0u;
        }
        if (gr < nc) {
#pragma unroll
          for (int v = 0; v < 8; ++v)
            *reinterpret_cast<uint4 *>(dst + c * 32 + v * 4) = make_uint4(gv[4 * v], gv[4 * v + 1], gv[4 * v + 2], gv[4 * v + 3]);
        }
      }
    }
  }
  if (!ok && lane == 0) flags[FLAG_TIMEOUT] = 1;
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 128;" ::"r"(tmem) : "memory");
  }
}

__global__ void to_bf16_kernel(const float *__restrict__ src, __nv_bfloat16 *__restrict__ dst, size_t n) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    dst[i] = __float2bfloat16_rn(src[i]);
}

template <int K>
cudaError_t launch_adam_tc(cudaStream_t st, const float *U, const CUtensorMap &tmQ, int nc, int d, float *Cm, float *Mo,
                           float *Vo, __nv_bfloat16 *Cb, const AdamArgs &aa, int32_t *flags) {
  auto kern = adam_gemm_tc_kernel<K>;
  CK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ESmem<K>::TOTAL));
  const int nrb = (nc + BLK - 1) / BLK, nj = (d + BLK - 1) / BLK;
  int nsplit = 148 / nrb;
  if (nsplit > nj / 4) nsplit = nj / 4;
  if (nsplit < 1) nsplit = 1;
  kern<<<nrb * nsplit, 576, ESmem<K>::TOTAL, st>>>(U, tmQ, nc, d, nsplit, Cm, Mo, Vo, Cb, aa, flags);
  return cudaGetLastError();
}

}  // namespace

// Whether the tensor-core form exists for this shape: rank 64 or 128, every row of C 16-byte aligned in both
// its fp32 and its bf16 copy.
bool extend_tc_qualifies(int32_t d, int32_t k) { return (k == 64 || k == 128) && d % 8 == 0 && d >= 128; }

// Per call: the bf16 copy of Q (d x k) and its two tensor maps (128-row tiles for the gradient product,
// 64-row tiles for the first product).  `maps` is host memory for the ExtendTcMaps of this call.
cudaError_t extend_tc_prepare(cudaStream_t st, const float *d_Q, int32_t d, int32_t k, __nv_bfloat16 *qb, ExtendTcMaps *maps) {
  to_bf16_kernel<<<148 * 4, 256, 0, st>>>(d_Q, qb, (size_t)d * k);
  CK(cudaGetLastError());
  CK(make_map(reinterpret_cast<CUtensorMap *>(maps->q128), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, qb, (uint64_t)d, (uint64_t)k, BLK));
  return make_map(reinterpret_cast<CUtensorMap *>(maps->q64), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, qb, (uint64_t)d, (uint64_t)k, 64);
}

// Per slot: the tensor map of the bf16 coefficient buffer (rows = chunk capacity, d columns).
cudaError_t extend_tc_map_c(__nv_bfloat16 *cb, int32_t rows, int32_t d, void *map) {
  return make_map(static_cast<CUtensorMap *>(map), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, cb, (uint64_t)rows, (uint64_t)d, BLK);
}

cudaError_t extend_tc_to_bf16(cudaStream_t st, const float *src, __nv_bfloat16 *dst, size_t n) {
  to_bf16_kernel<<<148 * 4, 256, 0, st>>>(src, dst, n);
  return cudaGetLastError();
}

// W partial planes [nsplit][nc x k] = C Q over the slices of d; returns the number of planes in *nsplit_out.
cudaError_t extend_tc_w(cudaStream_t st, const void *map_c, const ExtendTcMaps *maps, int32_t nc, int32_t d, int32_t k,
                        float *Wpart, int max_split, int *nsplit_out, int32_t *flags) {
  const int nrb = (nc + BLK - 1) / BLK, ns = (d + 63) / 64;
  int nsplit = 148 / nrb;
  if (nsplit > max_split) nsplit = max_split;
  if (nsplit > ns) nsplit = ns;
  if (nsplit < 1) nsplit = 1;
  *nsplit_out = nsplit;
  const CUtensorMap &tmC = *static_cast<const CUtensorMap *>(map_c);
  const CUtensorMap &tmQ = *reinterpret_cast<const CUtensorMap *>(maps->q64);
  const size_t plane = (size_t)nc * k;
  if (k == 128) {
    auto kern = w_gemm_tc_kernel<128>;
    CK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, WSmem<128>::TOTAL));
    kern<<<nrb * nsplit, 192, WSmem<128>::TOTAL, st>>>(tmC, tmQ, nc, d, nsplit, Wpart, plane, flags);
  } else {
    auto kern = w_gemm_tc_kernel<64>;
    CK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, WSmem<64>::TOTAL));
    kern<<<nrb * nsplit, 192, WSmem<64>::TOTAL, st>>>(tmC, tmQ, nc, d, nsplit, Wpart, plane, flags);
  }
  return cudaGetLastError();
}

cudaError_t extend_tc_adam(cudaStream_t st, const float *U, const ExtendTcMaps *maps, int32_t nc, int32_t d, int32_t k,
                           float *Cm, float *Mo, float *Vo, __nv_bfloat16 *Cb, const AdamArgs &aa, int32_t *flags) {
  const CUtensorMap &tmQ = *reinterpret_cast<const CUtensorMap *>(maps->q128);
  if (k == 128) return launch_adam_tc<128>(st, U, tmQ, nc, d, Cm, Mo, Vo, Cb, aa, flags);
  return launch_adam_tc<64>(st, U, tmQ, nc, d, Cm, Mo, Vo, Cb, aa, flags);
}

}  // namespace tsid
