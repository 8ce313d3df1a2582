// Staged variant of the gradient pass.  Included by sparse.cu inside its namespace, after Geo,
// Raw and the pass_kernel it mirrors.
//
// Same arithmetic as pass_kernel<MODE_GRAD> (the dot products are summed as an even and an odd half
// by packed fp32 FMAs, otherwise in the same order), but the gathered factor rows travel global ->
// shared memory with 16-byte asynchronous copies (cp.async, L2 only), NST chunks of ROWS rows deep.  The bytes in flight then live in
// shared memory instead of registers; the k = 128 passes are bound by exactly that (gathers served
// by L2 / HBM at several hundred ns each, 256 B per entry).  A CTA is ONE warp: segments differ in
// length, and a multi-warp CTA keeps the shared memory of its finished warps idle until its longest
// segment ends.  There is no barrier and no spin-wait: completion is cp.async.wait_group.
#pragma once

template <bool BF16, int VE>
struct SRaw;  // reads a Raw vector from a shared-memory address
template <>
struct SRaw<false, 4> {
  static __device__ __forceinline__ void load(Raw<false, 4> &r, uint32_t a) {
    asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(r.v.x), "=f"(r.v.y), "=f"(r.v.z), "=f"(r.v.w) : "r"(a));
  }
};
template <>
struct SRaw<true, 8> {
  static __device__ __forceinline__ void load(Raw<true, 8> &r, uint32_t a) {
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.v.x), "=r"(r.v.y), "=r"(r.v.z), "=r"(r.v.w) : "r"(a));
  }
};
template <>
struct SRaw<true, 4> {
  static __device__ __forceinline__ void load(Raw<true, 4> &r, uint32_t a) {
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(r.v.x), "=r"(r.v.y) : "r"(a));
  }
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// base + j * rowbytes as one multiply-add with a 64-bit addend
__device__ __forceinline__ const void *row_addr(const unsigned char *base, uint32_t j, uint32_t rowbytes) {
  uint64_t a;
  asm("mad.wide.u32 %0, %1, %2, %3;" : "=l"(a) : "r"(j), "r"(rowbytes), "l"(reinterpret_cast<uint64_t>(base)));
  return reinterpret_cast<const void *>(a);
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// One entry's contribution to one coordinate of the gradient row.  Aggregated modes: e * y.  Entry-wise
// clip (Sec. 5.3 applied to every observed entry): min(2 e y - 2 lambda x, xi), nothing for padding
// lanes of a ragged chunk (for xi > 0 the nested min/max of the paper equals min(d, xi)).
template <bool ENTRY>
__device__ __forceinline__ float entry_acc(float e, float y, float x, float acc, float lam2, float xi, bool valid) {
  if (!ENTRY) return fmaf(e, y, acc);
  const float d = fmaf(-lam2, x, 2.f * e * y);
  return valid ? acc + fminf(d, xi) : acc;
}

// Minimum resident CTAs asked of the compiler: for 256-byte bf16 rows a cap of 96 registers (18 CTAs
// per SM) measured 9 % faster than the unconstrained 101; tighter caps spill and lose.
template <int KP, bool BF16>
struct StagedMinBlocks {
  static constexpr int value = KP <= 64 ? 32 : (KP == 128 ? 18 : 1);
};

// V8: the values come as one byte each (integers 0..255) instead of fp32; the arithmetic is the same.
template <int KP, bool BF16, int NST, int ROWS, bool ENTRY, bool V8>
__global__ void __launch_bounds__(32, StagedMinBlocks<KP, BF16>::value)
pass_staged_kernel(const Segment *__restrict__ segs, int nseg, const int32_t *__restrict__ idx,
                   const void *__restrict__ val_v, const void *__restrict__ stage_v,
                   const void *__restrict__ gather_v, int k, float *__restrict__ G,
                   float *__restrict__ partial, float lam2, float xi) {
  using T = typename std::conditional<BF16, __nv_bfloat16, float>::type;
  constexpr int GROUP = Geo<KP>::GROUP, EPL = Geo<KP>::EPL, EPW = Geo<KP>::EPW;
  constexpr int VE = BF16 ? (EPL >= 8 ? 8 : 4) : 4;
  constexpr int NV = EPL / VE;
  constexpr int SLOT = KP * (int)sizeof(T);  // bytes reserved per gathered row
  constexpr int STAGE = ROWS * SLOT;         // one chunk
  constexpr int PIECES = SLOT / 16;          // 16-byte pieces per row
  constexpr int NCP = ROWS * PIECES / 32;    // cp.async instructions per lane per chunk
  static_assert(ROWS % EPW == 0 && (ROWS / EPW) % 2 == 0, "chunk must hold an even number of warp iterations");
  static_assert(PIECES <= 32 && 32 % PIECES == 0 && ROWS * PIECES % 32 == 0, "piece mapping");
  using R = Raw<BF16, VE>;
  const T *stage = static_cast<const T *>(stage_v);
  const T *gat = static_cast<const T *>(gather_v);

  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int lane = threadIdx.x;
  const uint32_t sbase = smem_u32(smem_raw);
  const int warp = blockIdx.x;
  if (warp >= nseg) return;

  const int g = lane / GROUP, s = lane % GROUP;
  const Segment sg = segs[warp];
  const int pr = lane / PIECES, pp = lane % PIECES;  // this lane's (row within a copy instruction, piece)
  const bool pvalid = pp * 16 < k * (int)sizeof(T);

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

  const int32_t *ip = idx + sg.begin;
  const float *vp = static_cast<const float *>(val_v) + sg.begin;
  const uint8_t *vp8 = static_cast<const uint8_t *>(val_v) + sg.begin;
  const int len = sg.len;
  const int nchunks = (len + ROWS - 1) / ROWS;

  float vring[NST];
#pragma unroll
  for (int u = 0; u < NST; ++u) vring[u] = 0.f;

  // Copies of chunk c (lane l < ROWS holds the index of its l-th entry in j) into the stage at shared address st_addr.
  // Always commits a group, also for chunks past the end, so that wait_group counts stay aligned.
  auto issue = [&](int c, uint32_t st_addr, int32_t j) {
    if (c < nchunks) {
      const int nv = len - c * ROWS < ROWS ? len - c * ROWS : ROWS;
      const uint32_t dst0 = st_addr + pp * 16;
      const unsigned char *src0 = reinterpret_cast<const unsigned char *>(gat) + pp * 16;
      // indices are non-negative: unsigned 32 x 32 + 64 -> 64-bit multiply-add, one instruction per address
      if (k == KP && nv == ROWS) {
#pragma unroll
        for (int q = 0; q < NCP; ++q) {
          const int r = q * (32 / PIECES) + pr;
          const uint32_t jr = (uint32_t)__shfl_sync(0xffffffffu, j, r & 31);
          cp_async16(dst0 + r * SLOT, row_addr(src0, jr, (uint32_t)SLOT));
        }
      } else {
        const uint32_t rowbytes = (uint32_t)k * (uint32_t)sizeof(T);
#pragma unroll
        for (int q = 0; q < NCP; ++q) {
          const int r = q * (32 / PIECES) + pr;
          const uint32_t jr = (uint32_t)__shfl_sync(0xffffffffu, j, r & 31);
          if (r < nv && pvalid) cp_async16(dst0 + r * SLOT, row_addr(src0, jr, rowbytes));
        }
      }
    }
    cp_async_commit();
  };
  auto load_iv = [&](int c, int32_t &j, float &r) {
    j = 0;
    r = 0.f;
    if (lane < ROWS && c * ROWS + lane < len) {
      j = __ldcs(ip + c * ROWS + lane);
      r = V8 ? (float)__ldcs(vp8 + c * ROWS + lane) : __ldcs(vp + c * ROWS + lane);
    }
  };

  // The arithmetic on one landed chunk: stage at shared address sst, values in myr, nv valid entries.
  auto compute = [&](const uint32_t sst, const float myr, const int nv) {
    // One pair of warp iterations (entries sa and sb = sa + EPW of the chunk) on full-width rows.  Two fp32
    // FMAs per instruction (sm_100 packed fp32): the dot products run as an even and an odd partial sum,
    // the accumulation as pairs of coordinates.  FULL: both entries exist.  Otherwise an entry past the
    // end reads the chunk's last valid row (finite values) and gets e = 0, so it adds nothing.
    auto pair = [&](auto full, int sa, int sb) {
      constexpr bool FULL = decltype(full)::value;
      const bool va = FULL || sa < nv, vb = FULL || sb < nv;
      if (!FULL) { sa = va ? sa : nv - 1; sb = vb ? sb : nv - 1; }
      const float ra = __shfl_sync(0xffffffffu, myr, sa);
      const float rb = __shfl_sync(0xffffffffu, myr, sb);
      R ya[NV], yb[NV];
#pragma unroll
      for (int q = 0; q < NV; ++q) {
        SRaw<BF16, VE>::load(ya[q], sst + sa * SLOT + co[q] * (int)sizeof(T));
        SRaw<BF16, VE>::load(yb[q], sst + sb * SLOT + co[q] * (int)sizeof(T));
      }
      float fa[EPL], fb[EPL];
#pragma unroll
      for (int q = 0; q < NV; ++q) { ya[q].unpack(fa + q * VE); yb[q].unpack(fb + q * VE); }
      float2 da2 = __fmul2_rn(make_float2(x[0], x[1]), make_float2(fa[0], fa[1]));
      float2 db2 = __fmul2_rn(make_float2(x[0], x[1]), make_float2(fb[0], fb[1]));
#pragma unroll
      for (int i = 2; i < EPL; i += 2) {
        const float2 x2 = make_float2(x[i], x[i + 1]);
        da2 = __ffma2_rn(x2, make_float2(fa[i], fa[i + 1]), da2);
        db2 = __ffma2_rn(x2, make_float2(fb[i], fb[i + 1]), db2);
      }
      float da = da2.x + da2.y, db = db2.x + db2.y;
#pragma unroll
      for (int o = GROUP / 2; o > 0; o >>= 1) {
        da += __shfl_xor_sync(0xffffffffu, da, o);
        db += __shfl_xor_sync(0xffffffffu, db, o);
      }
      const float ea = va ? ra - da : 0.f, eb = vb ? rb - db : 0.f;
      if (ENTRY) {
#pragma unroll
        for (int i = 0; i < EPL; ++i) acc[i] = entry_acc<ENTRY>(ea, fa[i], x[i], acc[i], lam2, xi, va);
#pragma unroll
        for (int i = 0; i < EPL; ++i) acc[i] = entry_acc<ENTRY>(eb, fb[i], x[i], acc[i], lam2, xi, vb);
      } else {
        const float2 ea2 = make_float2(ea, ea), eb2 = make_float2(eb, eb);
#pragma unroll
        for (int i = 0; i < EPL; i += 2) {
          float2 a2 = make_float2(acc[i], acc[i + 1]);
          a2 = __ffma2_rn(ea2, make_float2(fa[i], fa[i + 1]), a2);
          a2 = __ffma2_rn(eb2, make_float2(fb[i], fb[i + 1]), a2);
          acc[i] = a2.x;
          acc[i + 1] = a2.y;
        }
      }
    };
    if (k == KP && nv == ROWS) {
      // full chunk of full-width rows (the common case): no predicates, fully unrolled
#pragma unroll
      for (int it = 0; it < ROWS / EPW; it += 2) pair(std::true_type{}, it * EPW + g, (it + 1) * EPW + g);
    } else if (k == KP) {
      // ragged last chunk of a segment
      const int iters = (nv + EPW - 1) / EPW;
      for (int it = 0; it < iters; it += 2) pair(std::false_type{}, it * EPW + g, (it + 1) * EPW + g);
    } else {
      const int iters = (nv + EPW - 1) / EPW;
      for (int it = 0; it < iters; it += 2) {
        const int sa = it * EPW + g, sb = sa + EPW;
        const float ra = __shfl_sync(0xffffffffu, myr, sa & 31);
        const float rb = __shfl_sync(0xffffffffu, myr, sb & 31);
        const bool va = sa < nv, vb = sb < nv;
        R ya[NV], yb[NV];
#pragma unroll
        for (int q = 0; q < NV; ++q) {
          ya[q].zero();
          yb[q].zero();
          if (va && cv[q]) SRaw<BF16, VE>::load(ya[q], sst + sa * SLOT + co[q] * (int)sizeof(T));
          if (vb && cv[q]) SRaw<BF16, VE>::load(yb[q], sst + sb * SLOT + co[q] * (int)sizeof(T));
        }
        float fa[EPL], fb[EPL];
#pragma unroll
        for (int q = 0; q < NV; ++q) { ya[q].unpack(fa + q * VE); yb[q].unpack(fb + q * VE); }
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
#pragma unroll
        for (int i = 0; i < EPL; ++i) acc[i] = entry_acc<ENTRY>(ea, fa[i], x[i], acc[i], lam2, xi, va);
#pragma unroll
        for (int i = 0; i < EPL; ++i) acc[i] = entry_acc<ENTRY>(eb, fb[i], x[i], acc[i], lam2, xi, vb);
      }
    }
  };

  if (NST == 2) {
    // two stages: one rolled loop; chunk c is computed while chunk c + 1 lands and the indices and values
    // of chunk c + 2 are fetched
    int32_t nj;
    float nr, rcur;
    load_iv(0, nj, rcur);
    issue(0, sbase, nj);
    load_iv(1, nj, nr);
    uint32_t scur = sbase, snext = sbase + STAGE;
    int rem = len;
    for (int c = 0; c < nchunks; ++c) {
      const float rnext = nr;
      issue(c + 1, snext, nj);
      load_iv(c + 2, nj, nr);
      cp_async_wait<1>();  // all but the newest group are done: chunk c has landed
      __syncwarp();
      compute(scur, rcur, rem < ROWS ? rem : ROWS);
      __syncwarp();  // every lane is done reading this stage before it is refilled
      const uint32_t t = scur;
      scur = snext;
      snext = t;
      rcur = rnext;
      rem -= ROWS;
    }
  } else {
    // prologue: chunks 0 .. NST-2 in flight, indices of chunk NST-1 loaded
    int32_t nj;
    float nr;
  #pragma unroll
    for (int u = 0; u < NST - 1; ++u) {
      int32_t j;
      load_iv(u, j, vring[u]);
      issue(u, sbase + u * STAGE, j);
    }
    load_iv(NST - 1, nj, nr);

    for (int c0 = 0; c0 < nchunks; c0 += NST) {
  #pragma unroll
      for (int u = 0; u < NST; ++u) {
        const int c = c0 + u;
        if (c < nchunks) {
          // keep the pipe full: chunk c+NST-1 goes into the stage that chunk c-1 released
          const int cn = c + NST - 1;
          const int sn = (u + NST - 1) % NST;
          vring[sn] = nr;
          issue(cn, sbase + sn * STAGE, nj);
          load_iv(cn + 1, nj, nr);
          cp_async_wait<NST - 1>();  // all but the newest NST-1 groups are done: chunk c has landed
          __syncwarp();

          compute(sbase + u * STAGE, vring[u], len - c * ROWS < ROWS ? len - c * ROWS : ROWS);
          __syncwarp();  // every lane is done reading this stage before it is refilled
        }
      }
    }
  }
  cp_async_wait<0>();

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
}

template <int KP, bool BF16, int NST, int ROWS, bool ENTRY, bool V8>
cudaError_t launch_staged_t(tsid_template *t, const Side &sd, const void *stage, const void *gather, float *G) {
  using T = typename std::conditional<BF16, __nv_bfloat16, float>::type;
  constexpr int smem = NST * ROWS * KP * (int)sizeof(T);
  auto kern = pass_staged_kernel<KP, BF16, NST, ROWS, ENTRY, V8>;
  CK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  const void *val = V8 ? static_cast<const void *>(sd.val8) : static_cast<const void *>(sd.val);
  kern<<<sd.nseg, 32, smem, t->stream>>>(sd.segs, sd.nseg, sd.idx, val, stage, gather, t->cfg.k, G, t->partial,
                                         2.0f * t->cfg.lambda, t->cfg.xi);
  return cudaGetLastError();
}

// byte values when the side has them
template <int KP, bool BF16, int NST, int ROWS, bool ENTRY>
cudaError_t launch_staged_v(tsid_template *t, const Side &sd, const void *stage, const void *gather, float *G) {
  if (sd.val8) return launch_staged_t<KP, BF16, NST, ROWS, ENTRY, true>(t, sd, stage, gather, G);
  return launch_staged_t<KP, BF16, NST, ROWS, ENTRY, false>(t, sd, stage, gather, G);
}
