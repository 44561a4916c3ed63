// Measurement aid: the practical read-only ceiling of the device.  A grid of one CTA per SM slot reads a buffer
// once with 16-byte loads that bypass L1, adds the words up and stores one number per CTA, so that nothing can be
// elided.  No arithmetic of the method is in here; the benchmark times it over the same logits as the row kernels
// and reports the row kernels against it.
#include <cuda_runtime.h>
#include <stdint.h>

#include "e3.h"

namespace {

constexpr int kProbeThreads = 512;
constexpr int kProbeUnroll = 8;

__global__ void __launch_bounds__(kProbeThreads) read_sum_kernel(const uint4 *__restrict__ src, size_t n_vec,
                                                                 unsigned long long *__restrict__ per_cta) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const size_t stride = (size_t)gridDim.x * kProbeThreads;
  size_t i = (size_t)blockIdx.x * kProbeThreads + threadIdx.x;
  uint32_t acc = 0;
  for (; i + (kProbeUnroll - 1) * stride < n_vec; i += kProbeUnroll * stride) {
    uint4 v[kProbeUnroll];
#pragma unroll
    for (int k = 0; k < kProbeUnroll; ++k)
      asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                   : "=r"(v[k].x), "=r"(v[k].y), "=r"(v[k].z), "=r"(v[k].w)
                   : "l"(src + i + (size_t)k * stride));
#pragma unroll
    for (int k = 0; k < kProbeUnroll; ++k) acc += (v[k].x ^ v[k].y) + (v[k].z ^ v[k].w);
  }
  for (; i < n_vec; i += stride) {
    const uint4 v = __ldg(src + i);
    acc += (v.x ^ v.y) + (v.z ^ v.w);
  }
  acc = __reduce_add_sync(0xffffffffu, acc);
  __shared__ uint32_t part[kProbeThreads / 32];
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long t = 0;
    for (int w = 0; w < kProbeThreads / 32; ++w) t += part[w];
    per_cta[blockIdx.x] = t;
  }
}

}  // namespace

extern "C" e3_status e3_probe_read(const void *buf, size_t bytes, void *scratch, size_t scratch_bytes, void *stream) {
  if (!buf || !scratch || bytes % 16 != 0 || reinterpret_cast<uintptr_t>(buf) % 16 != 0 ||
      reinterpret_cast<uintptr_t>(scratch) % 8 != 0)
    return E3_ERR_INVALID_ARG;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return E3_ERR_CUDA;
  const int grid = sms * 4;
  if (scratch_bytes < (size_t)grid * 8) return E3_ERR_WORKSPACE;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kProbeThreads);
  cfg.stream = static_cast<cudaStream_t>(stream);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, read_sum_kernel, static_cast<const uint4 *>(buf), bytes / 16,
                                     static_cast<unsigned long long *>(scratch));
  return e == cudaSuccess ? E3_OK : E3_ERR_CUDA;
}
