// Dense tensor-core variant of the gradient step (Sec. 5.1, "Regularizing Sparse RMF Updates for
// Tensor Cores": the dominant work becomes dense tiles S = P Q^T around which the sparse structure
// is only a mask).  For templates dense enough that this really is a dense contraction:
//
//   pass A (CTA per block of 128 rows i, loop over blocks of 128 columns j):
//       S = P_blk Q_blk^T            tcgen05.mma, bf16 operands from shared memory (TMA), fp32 in TMEM
//       E = M .* (R - S)             epilogue warps: S from TMEM, the R tile (fp16, NaN = unobserved) from
//                                    shared memory (TMA); E goes back to TMEM as packed bf16
//       G_P_blk += E Q_blk           tcgen05.mma with A = E read from TMEM, accumulating in TMEM over the
//                                    whole j loop
//   pass B: the same kernel on (Q, P, R^T) gives G_Q.
//
// S is computed in both passes (four GEMMs instead of three) so that each gradient block has one
// owner CTA and a fixed summation order: no atomics, no partial buffers.  A 128x128x16 MMA with both
// operands in shared memory reads 128 B per clock, the whole shared-memory bandwidth of an SM; keeping
// E in TMEM removes its round trip through shared memory and halves what the second MMA reads there.
// The Y tile (128 rows j x K columns, 128-byte-swizzled as TMA writes it) serves both products: K-major
// as B of the first (contraction over the factor index) and MN-major as B of the second (contraction
// over j), so no transposed copy of the factors exists.  Every mbarrier wait is bounded by a cycle budget; on
// expiry the CTA raises FLAG_TIMEOUT, stops issuing, and still frees its TMEM before it returns.
#include <cuda.h>
#include <cuda_fp16.h>

#include <new>

#include "tsid_internal.cuh"

namespace tsid {

struct DenseState {
  __half *R = nullptr, *RT = nullptr;              // [m*n], [n*m]; NaN = not observed
  CUtensorMap tmP, tmQ, tmR, tmRT;
};

namespace {

#define CK(x)                         \
  do {                                \
    cudaError_t e_ = (x);             \
    if (e_ != cudaSuccess) return e_; \
  } while (0)

constexpr int BLK = 128;                 // tile edge (rows of X per CTA, rows of Y per iteration)
constexpr int NSTAGE = 3;                // stages of the Y and R tiles
constexpr long long WAIT_CYCLES = 4000000000LL;  // ~2 s at 2 GHz: bound of every wait

// ---- PTX wrappers ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t s32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false when the cycle budget ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity))
    if (clock64() - t0 > WAIT_CYCLES) return false;
  return true;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tm, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
      "l"(reinterpret_cast<uint64_t>(tm)), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void tc_mma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]   (A: lane = row, 32-bit column = two consecutive bf16 along K)
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_ld32_nowait(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
        "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
        "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_st16(uint32_t taddr, const uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]),
      "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
      : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile stored as 128-byte-swizzled rows (what a TMA
// box of 64 16-bit elements x rows writes): 8-row groups are 1024 B apart, descriptor version 1,
// swizzle 128B.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Descriptor of an MN-major operand read from the same kind of tile: rows of the tile are the K index
// (8-row groups 1024 B apart), the 64 contiguous elements of a row are the MN index, and the next 64
// MN elements live in the next 64-column block, `mn_block_bytes` further.
__device__ __forceinline__ uint64_t smem_desc_mn(uint32_t saddr, uint32_t mn_block_bytes) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(mn_block_bytes >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// kind::f16 instruction descriptor: fp32 accumulate, bf16 A and B, both K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t idesc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

template <int K>
struct Smem {
  static constexpr int XB = BLK * 128;            // one 64-column block of a 128-row tile: 16 KB
  static constexpr int X_BYTES = (K / 64) * XB;   // X block (128 x K bf16)
  static constexpr int Y_BYTES = (K / 64) * XB;   // Y block (128 x K bf16)
  static constexpr int R_BYTES = 2 * XB;          // R tile (128 x 128 fp16)
  static constexpr int STAGE_BYTES = Y_BYTES + R_BYTES;
  static constexpr int OFF_X = 0;
  static constexpr int OFF_Y = OFF_X + X_BYTES;
  static constexpr int OFF_R = OFF_Y + NSTAGE * Y_BYTES;
  static constexpr int OFF_BAR = OFF_R + NSTAGE * R_BYTES;
  static constexpr int TOTAL = OFF_BAR + 256 + 1024;  // barriers + slack for 1024-byte alignment
};

enum { B_XFULL = 0, B_QFULL = 1, B_QEMPTY = 1 + NSTAGE, B_SFULL = 1 + 2 * NSTAGE, B_SEMPTY = B_SFULL + 2, B_EFULL = B_SFULL + 4,
       B_EEMPTY = B_SFULL + 6, B_GFULL = B_SFULL + 8, B_COUNT = B_SFULL + 9 };
static_assert(B_COUNT * 8 <= 192, "barriers overlap the TMEM address slot");

// TMEM columns (512 allocated): S tiles 0..127 and 128..255 (fp32), G block 256..383 (fp32, K used),
// E tiles 384..447 and 448..511 (packed bf16: 64 columns hold 128 values per row).
constexpr uint32_t TM_S0 = 0, TM_S1 = 128, TM_G = 256, TM_E0 = 384, TM_E1 = 448;

// One pass: G_X[rows_x x K] = (M .* (R - X Y^T)) Y, R given as fp16 [rows_x][rows_y] with NaN = unobserved.
// Warps: 0 = TMA producer, 1 = MMA issuer (one thread), 2..17 = two epilogue teams of eight warps (two
// warps per TMEM lane quarter; a thread owns one row of the tile and half of its columns).  Team 0 takes
// the even column blocks (S0 / E0 / stage 0), team 1 the odd ones, so that the TMEM round trips of one
// tile overlap with the arithmetic of the next.
template <int K>
__global__ void __launch_bounds__(576, 1)
dense_pass_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmY,
                  const __grid_constant__ CUtensorMap tmR, int rows_y,
                  float *__restrict__ G, int32_t *__restrict__ flags) {
  using L = Smem<K>;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t sm0 = (s32(smem_dyn) + 1023u) & ~1023u;   // tiles need 1024-byte alignment
  unsigned char *smp = smem_dyn + (sm0 - s32(smem_dyn));
  const uint32_t bar0 = sm0 + L::OFF_BAR;
  volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smp + L::OFF_BAR + 192);
  auto bar = [&](int i) { return bar0 + 8u * i; };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ib = blockIdx.x;
  const int NJ = rows_y / BLK;

  if (threadIdx.x == 0) {
    mbar_init(bar(B_XFULL), 1);
    for (int s = 0; s < NSTAGE; ++s) { mbar_init(bar(B_QFULL + s), 1); mbar_init(bar(B_QEMPTY + s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(bar(B_SFULL + b), 1); mbar_init(bar(B_SEMPTY + b), 8); }
    for (int b = 0; b < 2; ++b) { mbar_init(bar(B_EFULL + b), 8); mbar_init(bar(B_EEMPTY + b), 1); }
    mbar_init(bar(B_GFULL), 1);
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
  const uint32_t tmS[2] = {tmem + TM_S0, tmem + TM_S1};
  const uint32_t tmE[2] = {tmem + TM_E0, tmem + TM_E1};
  const uint32_t tmG = tmem + TM_G;
  bool ok = true;

  if (warp == 0) {
    // ---- TMA producer ---------------------------------------------------------------------------
    if (lane == 0) {
      mbar_expect_tx(bar(B_XFULL), L::X_BYTES);
      for (int h = 0; h < K / 64; ++h) tma_load_2d(sm0 + L::OFF_X + h * L::XB, &tmX, bar(B_XFULL), h * 64, ib * BLK);
      for (int jb = 0; jb < NJ && ok; ++jb) {
        const int st = jb % NSTAGE;
        if (jb >= NSTAGE) ok = mbar_wait(bar(B_QEMPTY + st), ((jb / NSTAGE) - 1) & 1);
        if (!ok) break;
        mbar_expect_tx(bar(B_QFULL + st), L::STAGE_BYTES);
        for (int h = 0; h < K / 64; ++h)
          tma_load_2d(sm0 + L::OFF_Y + st * L::Y_BYTES + h * L::XB, &tmY, bar(B_QFULL + st), h * 64, jb * BLK);
        for (int h = 0; h < 2; ++h)
          tma_load_2d(sm0 + L::OFF_R + st * L::R_BYTES + h * L::XB, &tmR, bar(B_QFULL + st), jb * BLK + h * 64, ib * BLK);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---- MMA issuer -----------------------------------------------------------------------------
    if (lane == 0) {
      constexpr uint32_t ID1 = idesc_bf16(BLK), ID2 = idesc_bf16(K) | (1u << 16);   // second product: B is MN-major
      auto mma1 = [&](int jb) -> bool {
        const int st = jb % NSTAGE, b = jb & 1;
        if (!mbar_wait(bar(B_QFULL + st), (jb / NSTAGE) & 1)) return false;
        if (jb >= 2 && !mbar_wait(bar(B_SEMPTY + b), ((jb >> 1) - 1) & 1)) return false;
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < K / 16; ++ks) {
          const uint32_t off = (ks / 4) * L::XB + (ks % 4) * 32;
          tc_mma_ss(tmS[b], smem_desc(sm0 + L::OFF_X + off), smem_desc(sm0 + L::OFF_Y + st * L::Y_BYTES + off), ID1,
                    ks > 0);
        }
        tc_commit(bar(B_SFULL + b));
        return true;
      };
      ok = mbar_wait(bar(B_XFULL), 0);
      if (ok) ok = mma1(0);
      for (int jb = 0; jb < NJ && ok; ++jb) {
        const int st = jb % NSTAGE, b = jb & 1;
        if (jb + 1 < NJ) ok = mma1(jb + 1);
        if (ok) ok = mbar_wait(bar(B_EFULL + b), (jb >> 1) & 1);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < BLK / 16; ++ks) {   // K of this product = the 128 columns j: 8 TMEM columns per step
          // B[K = j][N = l] is the Y tile itself read MN-major: 16 rows j per step = 2048 B
          tc_mma_ts(tmG, tmE[b] + ks * 8, smem_desc_mn(sm0 + L::OFF_Y + st * L::Y_BYTES + ks * 2048, L::XB), ID2,
                    (jb > 0 || ks > 0));
        }
        tc_commit(bar(B_EEMPTY + b));
        tc_commit(bar(B_QEMPTY + st));
      }
      if (ok) tc_commit(bar(B_GFULL));
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
    for (int jb = team; jb < NJ && ok; jb += 2) {
      const int b = jb & 1, st = jb % NSTAGE;
      ok = mbar_wait(bar(B_QFULL + st), (jb / NSTAGE) & 1);                   // R tile has landed
      if (ok) ok = mbar_wait(bar(B_SFULL + b), (jb >> 1) & 1);                // S is complete
      if (ok && jb >= 2) ok = mbar_wait(bar(B_EEMPTY + b), ((jb >> 1) - 1) & 1);  // E buffer is free again
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t rrow = rrow0 + st * L::R_BYTES;
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
        tc_st16(tmE[b] + lane_off + h * 32 + c2 * 16, ew);
      }
      tc_wait_st();
      // one arrival per warp: every lane orders its TMEM accesses, then lane 0 signals for the warp
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(bar(B_SEMPTY + b));
        mbar_arrive(bar(B_EFULL + b));
      }
    }
    if (ok && team == 0) ok = __all_sync(0xffffffffu, mbar_wait(bar(B_GFULL), 0));
    if (ok && team == 0) {
      tc_fence_after();
      float *grow = G + (size_t)(ib * BLK + row) * K + h * (K / 2);
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

typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                             const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 16-bit matrix [rows][cols] (cols contiguous), box = box_rows x 64 columns, 128-byte swizzle
cudaError_t make_map(CUtensorMap *tm, CUtensorMapDataType dt, void *base, uint64_t rows, uint64_t cols,
                     uint32_t box_rows) {
  static EncodeFn fn = nullptr;
  if (!fn) {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    CK(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr));
    if (!p || qr != cudaDriverEntryPointSuccess) return cudaErrorNotSupported;
    fn = reinterpret_cast<EncodeFn>(p);
  }
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {64, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(tm, dt, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <int K>
cudaError_t launch_dense_pass(cudaStream_t st, const CUtensorMap &tmX, const CUtensorMap &tmY,
                              const CUtensorMap &tmR, int rows_x, int rows_y, float *G, int32_t *flags) {
  auto kern = dense_pass_kernel<K>;
  CK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<K>::TOTAL));
  kern<<<rows_x / BLK, 576, Smem<K>::TOTAL, st>>>(tmX, tmY, tmR, rows_y, G, flags);
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
  if (d) { d->R = R; d->RT = RT; }
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

// G_P and G_Q from the current bf16 shadows (which must be up to date).
cudaError_t dense_grad(tsid_template *t, float *GP, float *GQ) {
  DenseState *d = t->dense;
  const tsid_config_t &c = t->cfg;
  cudaStream_t st = t->stream;
  if (t->prof.on && t->prof.nsteps < kProfSteps) cudaEventRecord(t->prof.ev[t->prof.nsteps * EV_PER_STEP + EV_ROW0], st);
  if (c.k == 128) CK(launch_dense_pass<128>(st, d->tmP, d->tmQ, d->tmR, c.m, c.n, GP, t->flags));
  else CK(launch_dense_pass<64>(st, d->tmP, d->tmQ, d->tmR, c.m, c.n, GP, t->flags));
  if (t->prof.on && t->prof.nsteps < kProfSteps) {
    cudaEventRecord(t->prof.ev[t->prof.nsteps * EV_PER_STEP + EV_ROW1], st);
    cudaEventRecord(t->prof.ev[t->prof.nsteps * EV_PER_STEP + EV_COL0], st);
  }
  if (c.k == 128) CK(launch_dense_pass<128>(st, d->tmQ, d->tmP, d->tmRT, c.n, c.m, GQ, t->flags));
  else CK(launch_dense_pass<64>(st, d->tmQ, d->tmP, d->tmRT, c.n, c.m, GQ, t->flags));
  if (t->prof.on && t->prof.nsteps < kProfSteps) cudaEventRecord(t->prof.ev[t->prof.nsteps * EV_PER_STEP + EV_COL1], st);
  return cudaSuccess;
}

}  // namespace tsid
