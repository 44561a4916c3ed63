// e3_masked_mean_entropy_static: the masked mean entropy for callers that cannot hand over
// scratch memory.  Same two-stage fixed-order fp64 reduction as e3_masked_mean_entropy, but the
// per-block partial sums live in an array that is part of the library image instead of a
// caller-provided workspace.  The paper has no counterpart for this entry point.
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include <mutex>

#include "e3.h"

namespace {

constexpr int kThreads = 256;
constexpr int kTokensPerBlock = 4096;
constexpr int kMaxBlocks = 1024;  // 1024 partials x 16 bytes = 16 KiB held by every device that loads the library
constexpr int kMaxDevices = 64;

struct Partial {
  double sum;
  double cnt;
};

// The scratch itself.  In host code this name is only a handle for the runtime's symbol
// table, never a device address: the address the kernels get comes from cudaGetSymbolAddress.
static __device__ __align__(256) Partial g_static_partials[kMaxBlocks];

__device__ __forceinline__ void reduce_pair(double &a, double &b, double *sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    a += __shfl_xor_sync(0xffffffffu, a, o);
    b += __shfl_xor_sync(0xffffffffu, b, o);
  }
  if (lane == 0) { sh[2 * warp] = a; sh[2 * warp + 1] = b; }
  __syncthreads();
  if (warp == 0) {
    a = lane < kThreads / 32 ? sh[2 * lane] : 0.0;
    b = lane < kThreads / 32 ? sh[2 * lane + 1] : 0.0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      a += __shfl_xor_sync(0xffffffffu, a, o);
      b += __shfl_xor_sync(0xffffffffu, b, o);
    }
  }
}

// Stage 1: every launched block overwrites its own partial, so nothing left behind by an
// earlier call can leak into this one; stage 2 reads exactly the partials stage 1 wrote.
__global__ void __launch_bounds__(kThreads) static_mean_stage1(const float *__restrict__ ent,
                                                               const uint8_t *__restrict__ mask, int64_t n,
                                                               int64_t chunk, Partial *__restrict__ part) {
  __shared__ double sh[2 * kThreads / 32];
  const int64_t lo = (int64_t)blockIdx.x * chunk;
  const int64_t hi = lo + chunk < n ? lo + chunk : n;
  double s = 0.0, c = 0.0;
  for (int64_t j = lo + threadIdx.x; j < hi; j += kThreads) {
    if (!mask || mask[j] != 0) { s += (double)ent[j]; c += 1.0; }
  }
  reduce_pair(s, c, sh);
  if (threadIdx.x == 0) { part[blockIdx.x].sum = s; part[blockIdx.x].cnt = c; }
}

__global__ void __launch_bounds__(kThreads) static_mean_stage2(const Partial *__restrict__ part, int nparts,
                                                               double *__restrict__ out_mean,
                                                               double *__restrict__ out_count) {
  __shared__ double sh[2 * kThreads / 32];
  double s = 0.0, c = 0.0;
  for (int j = threadIdx.x; j < nparts; j += kThreads) { s += part[j].sum; c += part[j].cnt; }
  reduce_pair(s, c, sh);
  if (threadIdx.x == 0) {
    *out_mean = c > 0.0 ? s / c : CUDART_NAN;
    *out_count = c;
  }
}

std::mutex g_setup_lock;
Partial *g_device_scratch[kMaxDevices] = {};

// Device address of the scratch on the current device, looked up once per device.
cudaError_t scratch_for_current_device(Partial **out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> hold(g_setup_lock);
  if (!g_device_scratch[dev]) {
    Partial *p = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void **>(&p), g_static_partials);
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    g_device_scratch[dev] = p;
  }
  *out = g_device_scratch[dev];
  return cudaSuccess;
}

inline bool off_boundary(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) != 0; }

}  // namespace

extern "C" e3_status e3_masked_mean_entropy_static(const float *ent, const uint8_t *mask, int64_t n,
                                                   double *out_mean, double *out_count, void *stream) {
  if (n < 0 || !out_mean || !out_count || (n > 0 && !ent)) return E3_ERR_INVALID_ARG;
  if (n > E3_STATIC_MEAN_MAX_TOKENS) return E3_ERR_WORKSPACE;  // beyond what the built-in scratch is sized for
  if (off_boundary(ent, 4) || off_boundary(out_mean, 8) || off_boundary(out_count, 8)) return E3_ERR_ALIGNMENT;
  Partial *scratch = nullptr;
  if (scratch_for_current_device(&scratch) != cudaSuccess) {
    (void)cudaGetLastError();
    return E3_ERR_CUDA;
  }
  int64_t blocks = (n + kTokensPerBlock - 1) / kTokensPerBlock;
  if (blocks < 1) blocks = 1;
  if (blocks > kMaxBlocks) blocks = kMaxBlocks;
  const int64_t chunk = (n + blocks - 1) / blocks;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  static_mean_stage1<<<(unsigned)blocks, kThreads, 0, s>>>(ent, mask, n, chunk, scratch);
  static_mean_stage2<<<1, kThreads, 0, s>>>(scratch, (int)blocks, out_mean, out_count);
  return cudaGetLastError() == cudaSuccess ? E3_OK : E3_ERR_CUDA;
}
