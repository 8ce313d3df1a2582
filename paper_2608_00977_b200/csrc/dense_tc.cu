// Dense tensor-core variant of the gradient step (Sec. 5.1, "Regularizing Sparse RMF Updates for
// Tensor Cores": the dominant work becomes dense tiles S = P Q^T around which the sparse structure
// is only a mask).  For templates dense enough that this really is a dense contraction:
//
//   pass A (CTA per block of 128 rows i, loop over blocks of 128 columns j):
//       S = P_blk Q_blk^T            tcgen05.mma, bf16 operands from shared memory (TMA), fp32 in TMEM
//       E = M .* (R - S)             epilogue warps: TMEM -> registers, R as fp16 with NaN = unobserved,
//                                    E written to shared memory as a bf16 MMA operand
//       G_P_blk += E Q_blk           tcgen05.mma accumulating in TMEM over the whole j loop
//   pass B: the same kernel on (Q, P, R^T) gives G_Q.
//
// S is computed in both passes (four GEMMs instead of three) so that each gradient block has one
// owner CTA and a fixed summation order: no atomics, no partial buffers.  All MMA operands are
// K-major 128-byte-swizzled tiles; that is why transposed bf16 shadows (k x rows) are kept next to
// the row-major ones.  Every mbarrier wait is bounded by a cycle budget; on expiry the CTA raises
// FLAG_TIMEOUT, stops issuing, and still frees its TMEM before it returns.
#include <cuda.h>
#include <cuda_fp16.h>

#include <new>

#include "tsid_internal.cuh"

namespace tsid {

struct DenseState {
  __half *R = nullptr, *RT = nullptr;              // [m*n], [n*m]; NaN = not observed
  __nv_bfloat16 *PbT = nullptr, *QbT = nullptr;    // [k*m], [k*n]
  CUtensorMap tmP, tmQ, tmPT, tmQT;
};

namespace {

#define CK(x)                         \
  do {                                \
    cudaError_t e_ = (x);             \
    if (e_ != cudaSuccess) return e_; \
  } while (0)

constexpr int BLK = 128;                 // tile edge (rows of X per CTA, rows of Y per iteration)
constexpr int NSTAGE = 2;                // Y / Y^T stages
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
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
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

// Shared-memory matrix descriptor of a K-major tile stored as 128-byte-swizzled rows (what a TMA
// box of 64 bf16 x rows writes): 8-row groups are 1024 B apart, descriptor version 1, swizzle 128B.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// kind::f16 instruction descriptor: fp32 accumulate, bf16 A and B, both K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t idesc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

template <int K>
struct Smem {
  static constexpr int XB = BLK * 128;            // one 64-column block of a 128-row tile: 16 KB
  static constexpr int X_BYTES = (K / 64) * XB;   // X block (128 x K)
  static constexpr int Y_BYTES = (K / 64) * XB;   // Y block (128 x K)
  static constexpr int YTB = K * 128;             // one 64-column block of the K-row Y^T tile
  static constexpr int YT_BYTES = 2 * YTB;        // Y^T block (K x 128)
  static constexpr int E_BYTES = 2 * XB;          // E tile (128 x 128 bf16)
  static constexpr int OFF_X = 0;
  static constexpr int OFF_Y = OFF_X + X_BYTES;
  static constexpr int OFF_YT = OFF_Y + NSTAGE * Y_BYTES;
  static constexpr int OFF_E = OFF_YT + NSTAGE * YT_BYTES;
  static constexpr int OFF_BAR = OFF_E + E_BYTES;
  static constexpr int TOTAL = OFF_BAR + 256 + 1024;  // barriers + slack for 1024-byte alignment
};

enum { B_XFULL = 0, B_QFULL = 1, B_QEMPTY = 3, B_SFULL = 5, B_SEMPTY = 7, B_EFULL = 9, B_EEMPTY = 10, B_GFULL = 11, B_COUNT = 12 };

// One pass: G_X[rows_x x K] = (M .* (R - X Y^T)) Y, R given as fp16 [rows_x][rows_y] with NaN = unobserved.
template <int K>
__global__ void __launch_bounds__(192, 1)
dense_pass_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmY,
                  const __grid_constant__ CUtensorMap tmYT, const __half *__restrict__ R, int rows_y,
                  float *__restrict__ G, int32_t *__restrict__ flags) {
  using L = Smem<K>;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t sm0 = (s32(smem_dyn) + 1023u) & ~1023u;   // tiles need 1024-byte alignment
  unsigned char *smp = smem_dyn + (sm0 - s32(smem_dyn));
  const uint32_t bar0 = sm0 + L::OFF_BAR;
  volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smp + L::OFF_BAR + 128);
  auto bar = [&](int i) { return bar0 + 8u * i; };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ib = blockIdx.x;
  const int NJ = rows_y / BLK;

  if (threadIdx.x == 0) {
    mbar_init(bar(B_XFULL), 1);
    for (int s = 0; s < NSTAGE; ++s) { mbar_init(bar(B_QFULL + s), 1); mbar_init(bar(B_QEMPTY + s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(bar(B_SFULL + b), 1); mbar_init(bar(B_SEMPTY + b), 128); }
    mbar_init(bar(B_EFULL), 128);
    mbar_init(bar(B_EEMPTY), 1);
    mbar_init(bar(B_GFULL), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(bar0 + 128u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tmS[2] = {tmem, tmem + 128u};
  const uint32_t tmG = tmem + 256u;
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
        mbar_expect_tx(bar(B_QFULL + st), L::Y_BYTES + L::YT_BYTES);
        for (int h = 0; h < K / 64; ++h)
          tma_load_2d(sm0 + L::OFF_Y + st * L::Y_BYTES + h * L::XB, &tmY, bar(B_QFULL + st), h * 64, jb * BLK);
        for (int h = 0; h < 2; ++h)
          tma_load_2d(sm0 + L::OFF_YT + st * L::YT_BYTES + h * L::YTB, &tmYT, bar(B_QFULL + st), jb * BLK + h * 64, 0);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---- MMA issuer -----------------------------------------------------------------------------
    if (lane == 0) {
      constexpr uint32_t ID1 = idesc_bf16(BLK), ID2 = idesc_bf16(K);
      auto mma1 = [&](int jb) -> bool {
        const int st = jb % NSTAGE, b = jb & 1;
        if (!mbar_wait(bar(B_QFULL + st), (jb / NSTAGE) & 1)) return false;
        if (jb >= 2 && !mbar_wait(bar(B_SEMPTY + b), ((jb >> 1) - 1) & 1)) return false;
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < K / 16; ++ks) {
          const uint32_t off = (ks / 4) * L::XB + (ks % 4) * 32;
          tc_mma_bf16(tmS[b], smem_desc(sm0 + L::OFF_X + off), smem_desc(sm0 + L::OFF_Y + st * L::Y_BYTES + off), ID1,
                      ks > 0);
        }
        tc_commit(bar(B_SFULL + b));
        return true;
      };
      ok = mbar_wait(bar(B_XFULL), 0);
      if (ok) ok = mma1(0);
      for (int jb = 0; jb < NJ && ok; ++jb) {
        const int st = jb % NSTAGE;
        if (jb + 1 < NJ) ok = mma1(jb + 1);
        if (ok) ok = mbar_wait(bar(B_EFULL), jb & 1);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < BLK / 16; ++ks) {
          const uint32_t offa = (ks / 4) * L::XB + (ks % 4) * 32;
          const uint32_t offb = (ks / 4) * L::YTB + (ks % 4) * 32;
          tc_mma_bf16(tmG, smem_desc(sm0 + L::OFF_E + offa), smem_desc(sm0 + L::OFF_YT + st * L::YT_BYTES + offb), ID2,
                      (jb > 0 || ks > 0));
        }
        tc_commit(bar(B_EEMPTY));
        tc_commit(bar(B_QEMPTY + st));
      }
      if (ok) tc_commit(bar(B_GFULL));
    }
    __syncwarp();
  } else {
    // ---- epilogue warps: thread = one row of the tile ---------------------------------------------
    const int q = warp & 3;                 // TMEM lane quarter this warp may read
    const int row = q * 32 + lane;          // row inside the tile
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    const __half *rrow = R + (size_t)(ib * BLK + row) * rows_y;
    const uint32_t erow = sm0 + L::OFF_E + row * 128;
    for (int jb = 0; jb < NJ && ok; ++jb) {
      const int b = jb & 1;
      ok = mbar_wait(bar(B_SFULL + b), (jb >> 1) & 1);
      if (ok && jb >= 1) ok = mbar_wait(bar(B_EEMPTY), (jb - 1) & 1);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
#pragma unroll
      for (int c4 = 0; c4 < 4; ++c4) {
        uint32_t sv[32];
        tc_ld32(tmS[b] + lane_off + c4 * 32, sv);
        const uint4 *rp = reinterpret_cast<const uint4 *>(rrow + jb * BLK + c4 * 32);
#pragma unroll
        for (int v = 0; v < 4; ++v) {   // 8 columns per 16-byte vector of R
          const uint4 rv = __ldg(rp + v);
          const uint32_t rw[4] = {rv.x, rv.y, rv.z, rv.w};
          uint32_t ew[4];
#pragma unroll
          for (int p = 0; p < 4; ++p) {
            const uint32_t lo = rw[p] & 0xffffu, hi = rw[p] >> 16;
            const float s0 = __uint_as_float(sv[v * 8 + 2 * p]), s1 = __uint_as_float(sv[v * 8 + 2 * p + 1]);
            const float r0 = __half2float(__ushort_as_half((unsigned short)lo));
            const float r1 = __half2float(__ushort_as_half((unsigned short)hi));
            const float e0 = (lo & 0x7fffu) > 0x7c00u ? 0.f : r0 - s0;
            const float e1 = (hi & 0x7fffu) > 0x7c00u ? 0.f : r1 - s1;
            __nv_bfloat162 pk = __floats2bfloat162_rn(e0, e1);
            ew[p] = *reinterpret_cast<uint32_t *>(&pk);
          }
          const int chunk = (c4 & 1) * 4 + v;   // 16-byte chunk inside the 128-byte swizzled row
          const uint32_t dst = erow + (c4 >> 1) * L::XB + (((uint32_t)chunk ^ (uint32_t)(row & 7)) << 4);
          asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(ew[0]), "r"(ew[1]), "r"(ew[2]), "r"(ew[3])
                       : "memory");
        }
      }
      tc_fence_before();
      mbar_arrive(bar(B_SEMPTY + b));
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_arrive(bar(B_EFULL));
    }
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait(bar(B_GFULL), 0));
    if (ok) {
      tc_fence_after();
      float *grow = G + (size_t)(ib * BLK + row) * K;
#pragma unroll
      for (int c4 = 0; c4 < K / 32; ++c4) {
        uint32_t gv[32];
        tc_ld32(tmG + lane_off + c4 * 32, gv);
#pragma unroll
        for (int v = 0; v < 8; ++v)
          *reinterpret_cast<uint4 *>(grow + c4 * 32 + v * 4) = make_uint4(gv[4 * v], gv[4 * v + 1], gv[4 * v + 2], gv[4 * v + 3]);
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
      const __half h = __float2half_rn(r);
      const int j = col_idx[p];
      R[(size_t)i * n + j] = h;
      RT[(size_t)j * m + i] = h;
    }
  }
}

// out[k][rows] = in[rows][k]   (bf16)
__global__ void transpose_bf16_kernel(const __nv_bfloat16 *__restrict__ in, __nv_bfloat16 *__restrict__ out, int rows,
                                      int k) {
  __shared__ __nv_bfloat16 t[32][33];
  const int r0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
  for (int y = threadIdx.y; y < 32; y += blockDim.y) {
    const int r = r0 + y, c = c0 + threadIdx.x;
    if (r < rows && c < k) t[y][threadIdx.x] = in[(size_t)r * k + c];
  }
  __syncthreads();
  for (int y = threadIdx.y; y < 32; y += blockDim.y) {
    const int c = c0 + y, r = r0 + threadIdx.x;
    if (r < rows && c < k) out[(size_t)c * rows + r] = t[threadIdx.x][y];
  }
}

typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                             const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// bf16 matrix [rows][cols] (cols contiguous), box = box_rows x 64 columns, 128-byte swizzle
cudaError_t make_map(CUtensorMap *tm, void *base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
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
  CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <int K>
cudaError_t launch_dense_pass(cudaStream_t st, const CUtensorMap &tmX, const CUtensorMap &tmY, const CUtensorMap &tmYT,
                              const __half *R, int rows_x, int rows_y, float *G, int32_t *flags) {
  auto kern = dense_pass_kernel<K>;
  CK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<K>::TOTAL));
  kern<<<rows_x / BLK, 192, Smem<K>::TOTAL, st>>>(tmX, tmY, tmYT, R, rows_y, G, flags);
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
  __nv_bfloat16 *PbT = cv.take<__nv_bfloat16>((size_t)c.m * c.k), *QbT = cv.take<__nv_bfloat16>((size_t)c.n * c.k);
  if (d) { d->R = R; d->RT = RT; d->PbT = PbT; d->QbT = QbT; }
}

DenseState *dense_new() { return new (std::nothrow) DenseState; }
void dense_delete(DenseState *d) { delete d; }

// After the layout pass: dense fp16 copies of R and R^T, tensor maps of the four shadow matrices.
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
  CK(make_map(&d->tmP, t->rowside.shadow, c.m, c.k, BLK));
  CK(make_map(&d->tmQ, t->colside.shadow, c.n, c.k, BLK));
  CK(make_map(&d->tmPT, d->PbT, c.k, c.m, c.k));
  CK(make_map(&d->tmQT, d->QbT, c.k, c.n, c.k));
  return cudaSuccess;
}

// G_P and G_Q from the current bf16 shadows (which must be up to date).
cudaError_t dense_grad(tsid_template *t, float *GP, float *GQ) {
  DenseState *d = t->dense;
  const tsid_config_t &c = t->cfg;
  cudaStream_t st = t->stream;
  dim3 tb(32, 8);
  transpose_bf16_kernel<<<dim3((c.m + 31) / 32, (c.k + 31) / 32), tb, 0, st>>>(t->rowside.shadow, d->PbT, c.m, c.k);
  transpose_bf16_kernel<<<dim3((c.n + 31) / 32, (c.k + 31) / 32), tb, 0, st>>>(t->colside.shadow, d->QbT, c.n, c.k);
  CK(cudaGetLastError());
  if (t->prof.on && t->prof.nsteps < kProfSteps) cudaEventRecord(t->prof.ev[t->prof.nsteps * EV_PER_STEP + EV_ROW0], st);
  if (c.k == 128) CK(launch_dense_pass<128>(st, d->tmP, d->tmQ, d->tmQT, d->R, c.m, c.n, GP, t->flags));
  else CK(launch_dense_pass<64>(st, d->tmP, d->tmQ, d->tmQT, d->R, c.m, c.n, GP, t->flags));
  if (t->prof.on && t->prof.nsteps < kProfSteps) {
    cudaEventRecord(t->prof.ev[t->prof.nsteps * EV_PER_STEP + EV_ROW1], st);
    cudaEventRecord(t->prof.ev[t->prof.nsteps * EV_PER_STEP + EV_COL0], st);
  }
  if (c.k == 128) CK(launch_dense_pass<128>(st, d->tmQ, d->tmP, d->tmPT, d->RT, c.n, c.m, GQ, t->flags));
  else CK(launch_dense_pass<64>(st, d->tmQ, d->tmP, d->tmPT, d->RT, c.n, c.m, GQ, t->flags));
  if (t->prof.on && t->prof.nsteps < kProfSteps) cudaEventRecord(t->prof.ev[t->prof.nsteps * EV_PER_STEP + EV_COL1], st);
  return cudaSuccess;
}

}  // namespace tsid
