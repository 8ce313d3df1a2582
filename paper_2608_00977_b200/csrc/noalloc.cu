// tsid_sse_noalloc: the sum of squared residuals of a template, computed without any device
// allocation and without a workspace.
//
// Who this is for.  tsid_loss needs a template handle, and a handle needs a workspace that
// somebody allocated.  Some callers cannot allocate device memory at the point where they want
// a loss value: a monitoring hook that runs inside a serving process whose framework has already
// claimed the whole GPU for its own pool (cudaMalloc fails there, or steals from the pool);
// latency-critical loops where the implicit device-wide synchronisation of cudaFree is not
// acceptable; plug-ins that are handed raw pointers and a stream and nothing else.  For them the
// scratch that the reduction needs lives in a fixed array inside the library image.
//
// The price: the array has a fixed size (kMaxChunks partial sums, 512 KiB, resident on every GPU
// that loads the library until the process exits), so nnz is limited to kMaxChunks * 1024
// entries; and every call on a device shares the same array, so two calls that overlap on the
// GPU (different streams, or different host threads) race on it and must be serialised by the
// caller.  The array keeps whatever the previous call left in it; this is harmless because each
// call writes every slot it later reads (slots [0, ceil(nnz/1024))) before reading it, so nothing
// has to be cleared.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include <mutex>

#include "../../include/tsid.h"

namespace {

constexpr int kChunk = 1024;          // entries per partial sum (one warp each)
constexpr int kMaxChunks = 1 << 16;   // 65,536 partial sums = 512 KiB of scratch
constexpr int kMaxDevices = 64;

// The scratch.  In host code this name is only a handle for the runtime's symbol table, not a
// device address: the address a kernel can use comes from cudaGetSymbolAddress (below).
static __device__ __align__(256) double g_sse_scratch[kMaxChunks];

std::mutex g_mu;
double *g_scratch_addr[kMaxDevices] = {nullptr};

// One warp per chunk of 1024 consecutive COO entries.  Eight lanes share an entry: lane s of a
// group reads the float4 pieces s, s+8, ... of both factor rows, the partial dots are combined
// with three shuffles, and lane 0 of the group adds e^2 in double.
__global__ void __launch_bounds__(256)
sse_chunks_kernel(const int32_t *__restrict__ rows, const int32_t *__restrict__ cols,
                  const float *__restrict__ vals, int64_t nnz, const float *__restrict__ P,
                  const float *__restrict__ Q, int k, int nchunks, double *__restrict__ partial) {
  const int warp = (int)(((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5);
  if (warp >= nchunks) return;
  const int lane = threadIdx.x & 31, g = lane >> 3, s = lane & 7;
  const int64_t lo = (int64_t)warp * kChunk;
  const int64_t hi = lo + kChunk < nnz ? lo + kChunk : nnz;
  const int k4 = k >> 2;
  double sq = 0.0;
  for (int64_t base = lo; base < hi; base += 4) {   // four entries per warp iteration
    const int64_t t = base + g;
    const bool ok = t < hi;
    float dot = 0.f, r = 0.f;
    if (ok) {
      const float4 *p = reinterpret_cast<const float4 *>(P + (size_t)rows[t] * k);
      const float4 *q = reinterpret_cast<const float4 *>(Q + (size_t)cols[t] * k);
      r = vals[t];
      for (int c = s; c < k4; c += 8) {
        const float4 a = __ldg(p + c), b = __ldg(q + c);
        dot = fmaf(a.x, b.x, dot); dot = fmaf(a.y, b.y, dot);
        dot = fmaf(a.z, b.z, dot); dot = fmaf(a.w, b.w, dot);
      }
    }
    dot += __shfl_xor_sync(0xffffffffu, dot, 4);
    dot += __shfl_xor_sync(0xffffffffu, dot, 2);
    dot += __shfl_xor_sync(0xffffffffu, dot, 1);
    if (ok && s == 0) {
      const double e = (double)(r - dot);
      sq += e * e;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
  if (lane == 0) partial[warp] = sq;
}

// One block adds the partial sums in a fixed order and writes the result.
__global__ void __launch_bounds__(1024) sse_final_kernel(const double *__restrict__ partial, int nchunks,
                                                         double *__restrict__ out) {
  __shared__ double ws[32];
  double v = 0.0;
  for (int i = threadIdx.x; i < nchunks; i += 1024) v += partial[i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((threadIdx.x & 31) == 0) ws[threadIdx.x >> 5] = v;
  __syncthreads();
  if (threadIdx.x < 32) {
    double t = ws[threadIdx.x];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if (threadIdx.x == 0) *out = t;
  }
}

}  // namespace

extern "C" {

tsid_status_t tsid_sse_noalloc(int32_t m, int32_t n, int32_t k, int64_t nnz, const int32_t *d_rows,
                               const int32_t *d_cols, const float *d_vals, const float *d_P,
                               const float *d_Q, void *stream, double *d_sse_out) {
  if (m < 1 || n < 1 || nnz < 0) return TSID_ERR_INVALID_ARG;
  if (k < 4 || k > 256 || (k & 3)) return TSID_ERR_UNSUPPORTED;
  // more entries than the built-in scratch has partial sums for: refuse, the caller needs
  // tsid_loss and a workspace
  if (nnz > (int64_t)kMaxChunks * kChunk) return TSID_ERR_TOO_LARGE;
  if (!d_P || !d_Q || !d_sse_out || (nnz > 0 && (!d_rows || !d_cols || !d_vals))) return TSID_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_P) & 15u) || (reinterpret_cast<uintptr_t>(d_Q) & 15u) ||
      (reinterpret_cast<uintptr_t>(d_sse_out) & 7u))
    return TSID_ERR_INVALID_ARG;

  // Set-up, once per device, with that device current: ask the runtime where this device's copy
  // of the scratch array lives.
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return TSID_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return TSID_ERR_UNSUPPORTED;
  double *scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
      void *p = nullptr;
      e = cudaGetSymbolAddress(&p, g_sse_scratch);
      if (e != cudaSuccess) return TSID_ERR_CUDA;
      g_scratch_addr[dev] = static_cast<double *>(p);
    }
    scratch = g_scratch_addr[dev];
  }

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int nchunks = (int)((nnz + kChunk - 1) / kChunk);
  if (nchunks > 0) {
    const int grid = (nchunks + 7) / 8;
    sse_chunks_kernel<<<grid, 256, 0, st>>>(d_rows, d_cols, d_vals, nnz, d_P, d_Q, k, nchunks, scratch);
  }
  sse_final_kernel<<<1, 1024, 0, st>>>(scratch, nchunks, d_sse_out);
  return cudaGetLastError() == cudaSuccess ? TSID_OK : TSID_ERR_CUDA;
}

}  // extern "C"
