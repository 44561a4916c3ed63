// The two small device steps: masked mean entropy (Sec. 4.2, H_t) and the group-relative
// advantage (Eq. "adv").  Both are latency-bound; they are written for determinism
// (fixed summation order, fp64 accumulation) rather than bandwidth.
#include "e3_small.cuh"

#include <math_constants.h>

namespace e3 {
namespace {

constexpr int kMeanThreads = 256;

struct MeanPartial {
  double sum;
  double cnt;
};

__device__ __forceinline__ void block_reduce_2(double &a, double &b, double *sh /* [2*warps] */) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    a += __shfl_xor_sync(0xffffffffu, a, o);
    b += __shfl_xor_sync(0xffffffffu, b, o);
  }
  if (lane == 0) { sh[2 * warp] = a; sh[2 * warp + 1] = b; }
  __syncthreads();
  if (warp == 0) {
    a = lane < nw ? sh[2 * lane] : 0.0;
    b = lane < nw ? sh[2 * lane + 1] : 0.0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      a += __shfl_xor_sync(0xffffffffu, a, o);
      b += __shfl_xor_sync(0xffffffffu, b, o);
    }
  }
}

// Both stages may be launched with programmatic stream serialization behind the kernel that writes `ent`:
// they wait for it (and for its writes) before they touch memory.  Without that launch attribute the wait
// returns at once.
__device__ __forceinline__ void wait_for_stream_predecessor() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Stage 1: block b sums tokens [b*chunk, (b+1)*chunk) in a fixed order and stores one partial.
__global__ void __launch_bounds__(kMeanThreads) mean_partial_kernel(const float *__restrict__ ent,
                                                                    const uint8_t *__restrict__ mask, int64_t n,
                                                                    int64_t chunk, MeanPartial *__restrict__ part) {
  __shared__ double sh[2 * kMeanThreads / 32];
  wait_for_stream_predecessor();
  const int64_t lo = (int64_t)blockIdx.x * chunk;
  const int64_t hi = lo + chunk < n ? lo + chunk : n;
  double s = 0.0, c = 0.0;
  for (int64_t j = lo + threadIdx.x; j < hi; j += kMeanThreads) {
    const bool on = mask ? mask[j] != 0 : true;
    if (on) { s += (double)ent[j]; c += 1.0; }
  }
  block_reduce_2(s, c, sh);
  if (threadIdx.x == 0) { part[blockIdx.x].sum = s; part[blockIdx.x].cnt = c; }
}

// Stage 2: one block adds the partials in index order and writes mean (or, with want_sum, the sum) and count.
__global__ void __launch_bounds__(kMeanThreads) mean_final_kernel(const MeanPartial *__restrict__ part, int nparts,
                                                                  double *__restrict__ out_mean,
                                                                  double *__restrict__ out_count, int want_sum) {
  __shared__ double sh[2 * kMeanThreads / 32];
  wait_for_stream_predecessor();
  double s = 0.0, c = 0.0;
  for (int j = threadIdx.x; j < nparts; j += kMeanThreads) { s += part[j].sum; c += part[j].cnt; }
  block_reduce_2(s, c, sh);
  if (threadIdx.x == 0) {
    *out_mean = want_sum ? s : (c > 0.0 ? s / c : CUDART_NAN);
    *out_count = c;
  }
}

// Mean of per-sequence means: block s adds the unmasked tokens of sequence s in a fixed order ...
__global__ void __launch_bounds__(kMeanThreads) seq_partial_kernel(const float *__restrict__ ent,
                                                                   const uint8_t *__restrict__ mask, int64_t seq_len,
                                                                   MeanPartial *__restrict__ part) {
  __shared__ double sh[2 * kMeanThreads / 32];
  wait_for_stream_predecessor();
  const int64_t lo = (int64_t)blockIdx.x * seq_len;
  double s = 0.0, c = 0.0;
  for (int64_t j = threadIdx.x; j < seq_len; j += kMeanThreads) {
    const bool on = mask ? mask[lo + j] != 0 : true;
    if (on) { s += (double)ent[lo + j]; c += 1.0; }
  }
  block_reduce_2(s, c, sh);
  if (threadIdx.x == 0) { part[blockIdx.x].sum = s; part[blockIdx.x].cnt = c; }
}

// ... and one block averages the sequences' means in index order (sequences without tokens take no part).
__global__ void __launch_bounds__(kMeanThreads) seq_final_kernel(const MeanPartial *__restrict__ part, int64_t n_seq,
                                                                 double *__restrict__ out_mean,
                                                                 double *__restrict__ out_count) {
  __shared__ double sh[2 * kMeanThreads / 32];
  wait_for_stream_predecessor();
  double m = 0.0, c = 0.0;
  for (int64_t j = threadIdx.x; j < n_seq; j += kMeanThreads)
    if (part[j].cnt > 0.0) { m += part[j].sum / part[j].cnt; c += 1.0; }
  block_reduce_2(m, c, sh);
  if (threadIdx.x == 0) {
    *out_mean = c > 0.0 ? m / c : CUDART_NAN;
    *out_count = c;
  }
}

// One warp per group; a group of any size is walked in strides of 32.
__global__ void __launch_bounds__(256) group_advantage_kernel(const float *__restrict__ rewards,
                                                              const int64_t *__restrict__ off, int64_t n_groups,
                                                              float eps, int unbiased, float *__restrict__ adv,
                                                              uint8_t *__restrict__ flags) {
  const int lane = threadIdx.x & 31;
  const int64_t g = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (g >= n_groups) return;
  const int64_t lo = off[g], hi = off[g + 1], n = hi - lo;
  if (n <= 0) {
    if (flags && lane == 0) flags[g] = 0;
    return;
  }
  const float r0 = rewards[lo];
  double s = 0.0;
  int differs = 0, nonzero = 0;
  for (int64_t i = lo + lane; i < hi; i += 32) {
    const float r = rewards[i];
    s += (double)r;
    differs |= (r != r0);
    nonzero |= (r != 0.f);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  differs = __any_sync(0xffffffffu, differs);
  nonzero = __any_sync(0xffffffffu, nonzero);
  const double mean = s / (double)n;
  double ss = 0.0;
  for (int64_t i = lo + lane; i < hi; i += 32) {
    const double d = (double)rewards[i] - mean;
    ss += d * d;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  const double denom = unbiased ? (double)(n - 1) : (double)n;
  const double sd = n == 1 ? 0.0 : sqrt(ss / denom);
  // std + eps == 0 (eps == 0 and identical rewards): every r_i - mean is 0 and the advantage is 0, not 0/0
  const double inv = sd + (double)eps > 0.0 ? 1.0 / (sd + (double)eps) : 0.0;
  for (int64_t i = lo + lane; i < hi; i += 32)
    adv[i] = n == 1 ? 0.f : (float)(((double)rewards[i] - mean) * inv);
  if (flags && lane == 0) flags[g] = (uint8_t)((differs ? 0 : 1) | (nonzero ? 0 : 2));
}

}  // namespace

int mean_blocks(int64_t n) {
  int64_t b = (n + 4095) / 4096;
  if (b < 1) b = 1;
  if (b > 1024) b = 1024;
  return (int)b;
}

size_t mean_workspace_bytes(int64_t n) { return (size_t)mean_blocks(n) * sizeof(MeanPartial); }

cudaError_t launch_masked_mean(const float *ent, const uint8_t *mask, int64_t n, double *out_mean,
                               double *out_count, void *workspace, bool want_sum, cudaStream_t stream) {
  const int blocks = mean_blocks(n);
  const int64_t chunk = (n + blocks - 1) / blocks;
  MeanPartial *part = static_cast<MeanPartial *>(workspace);
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kMeanThreads);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cfg.gridDim = dim3((unsigned)blocks);
  cudaError_t e = cudaLaunchKernelEx(&cfg, mean_partial_kernel, ent, mask, n, chunk, part);
  if (e != cudaSuccess) return e;
  cfg.gridDim = dim3(1);
  return cudaLaunchKernelEx(&cfg, mean_final_kernel, (const MeanPartial *)part, blocks, out_mean, out_count,
                            want_sum ? 1 : 0);
}

size_t seq_mean_workspace_bytes(int64_t n_seq) { return (size_t)(n_seq < 1 ? 1 : n_seq) * sizeof(MeanPartial); }

cudaError_t launch_sequence_mean(const float *ent, const uint8_t *mask, int64_t n_seq, int64_t seq_len,
                                 double *out_mean, double *out_count, void *workspace, cudaStream_t stream) {
  MeanPartial *part = static_cast<MeanPartial *>(workspace);
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kMeanThreads);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (n_seq > 0) {
    cfg.gridDim = dim3((unsigned)n_seq);
    cudaError_t e = cudaLaunchKernelEx(&cfg, seq_partial_kernel, ent, mask, seq_len, part);
    if (e != cudaSuccess) return e;
  }
  cfg.gridDim = dim3(1);
  return cudaLaunchKernelEx(&cfg, seq_final_kernel, (const MeanPartial *)part, n_seq, out_mean, out_count);
}

cudaError_t launch_group_advantage(const float *rewards, const int64_t *off, int64_t n_groups, float eps,
                                   int unbiased, float *adv, uint8_t *flags, cudaStream_t stream) {
  const int warps_per_block = 8;
  const int64_t blocks = (n_groups + warps_per_block - 1) / warps_per_block;
  group_advantage_kernel<<<(unsigned)blocks, warps_per_block * 32, 0, stream>>>(rewards, off, n_groups, eps,
                                                                               unbiased, adv, flags);
  return cudaGetLastError();
}

}  // namespace e3
