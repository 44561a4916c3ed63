// GRPO objective of Sec. 3.1 without the KL term (the paper drops it), fused over the tokens of a batch:
//   J = mean_q (1/G_q) sum_{i in q} (1/|o_i|) sum_t min( r_{i,t} A_i , clip(r_{i,t}, 1-eps, 1+eps) A_i ),
//   r_{i,t} = exp(logp_{i,t} - logp_old_{i,t}),
// together with dJ/dlogp per token (what the backward of the vocabulary pass takes as g_logp) and the
// fraction of response tokens whose clipped term is the active one.  The data is a few bytes per token
// (nothing of vocabulary size), so the kernels are latency-bound; they are written for determinism:
// all arithmetic in fp64 (the clip decision compares two products and must not depend on fp32 rounding),
// fixed-order reductions, one CTA per response and a single block for the final sum.
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "e3.h"

namespace {

constexpr int kThreads = 256;

struct SeqPartial {
  double J;        // this response's share of the objective, already divided by |o_i| and G_q
  double tokens;   // |o_i|
  double clipped;  // tokens whose clipped term is active
};

__device__ __forceinline__ double block_sum(double v, double *sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();  // sh may still be read from the previous call
  if (lane == 0) sh[warp] = v;
  __syncthreads();
  double t = 0.0;
  for (int w = 0; w < kThreads / 32; ++w) t += sh[w];  // same order in every thread
  return t;
}

__global__ void __launch_bounds__(kThreads) grpo_seq_kernel(const float *__restrict__ logp,
                                                            const float *__restrict__ logp_old,
                                                            const uint8_t *__restrict__ mask, int64_t seq_len,
                                                            const float *__restrict__ adv,
                                                            const int64_t *__restrict__ off, int64_t n_groups,
                                                            double clip_lo, double clip_hi,
                                                            float *__restrict__ g_out, SeqPartial *__restrict__ part) {
  __shared__ double sh[kThreads / 32];
  __shared__ double s_gq;
  // programmatic dependent launch: the final kernel may be set up while this one runs
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int64_t i = blockIdx.x;
  const int64_t base = i * seq_len;
  if (threadIdx.x == 0) {
    // group of this response: the q with off[q] <= i < off[q+1]
    int64_t lo = 0, hi = n_groups;  // invariant: off[lo] <= i, answer in [lo, hi)
    double gq = 0.0;
    if (n_groups > 0 && off[0] <= i && i < off[n_groups]) {
      while (hi - lo > 1) {
        const int64_t mid = (lo + hi) >> 1;
        if (off[mid] <= i) lo = mid; else hi = mid;
      }
      gq = (double)(off[lo + 1] - off[lo]);
    }
    s_gq = gq;
  }
  double cnt = 0.0;
  for (int64_t t = threadIdx.x; t < seq_len; t += kThreads) cnt += (!mask || mask[base + t]) ? 1.0 : 0.0;
  const double len = block_sum(cnt, sh);  // also makes s_gq visible
  const double gq = s_gq;
  const double A = (double)adv[i];
  const double w = (len > 0.0 && gq > 0.0) ? 1.0 / (len * gq * (double)n_groups) : 0.0;
  double J = 0.0, clipped = 0.0;
  for (int64_t t = threadIdx.x; t < seq_len; t += kThreads) {
    const int64_t j = base + t;
    float g = 0.f;
    if ((!mask || mask[j]) && w > 0.0) {
      const double r = exp((double)logp[j] - (double)logp_old[j]);
      const double rc = r < clip_lo ? clip_lo : (r > clip_hi ? clip_hi : r);
      const double s1 = r * A, s2 = rc * A;
      const bool clip_active = s2 < s1;  // the clipped term is the strictly smaller one: no gradient
      J += clip_active ? s2 : s1;
      clipped += clip_active ? 1.0 : 0.0;
      g = clip_active ? 0.f : (float)(s1 * w);
    }
    if (g_out) g_out[j] = g;
  }
  J = block_sum(J, sh);
  clipped = block_sum(clipped, sh);
  if (threadIdx.x == 0) {
    part[i].J = (len > 0.0 && gq > 0.0) ? J / (len * gq) : 0.0;
    part[i].tokens = gq > 0.0 ? len : 0.0;
    part[i].clipped = clipped;
  }
}

__global__ void __launch_bounds__(kThreads) grpo_final_kernel(const SeqPartial *__restrict__ part, int64_t n_seq,
                                                              int64_t n_groups, double *__restrict__ out_J,
                                                              double *__restrict__ out_clip_frac) {
  __shared__ double sh[kThreads / 32];
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the per-response partials are complete and visible
  double J = 0.0, tok = 0.0, cl = 0.0;
  for (int64_t i = threadIdx.x; i < n_seq; i += kThreads) { J += part[i].J; tok += part[i].tokens; cl += part[i].clipped; }
  J = block_sum(J, sh);
  tok = block_sum(tok, sh);
  cl = block_sum(cl, sh);
  if (threadIdx.x == 0) {
    *out_J = n_groups > 0 ? J / (double)n_groups : 0.0;
    if (out_clip_frac) *out_clip_frac = tok > 0.0 ? cl / tok : 0.0;
  }
}

inline bool misaligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) != 0; }

}  // namespace

namespace e3 {
size_t grpo_workspace_bytes(int64_t n_seq) { return (size_t)(n_seq > 0 ? n_seq : 1) * sizeof(SeqPartial); }
}  // namespace e3

extern "C" e3_status e3_grpo_objective(const float *logp, const float *logp_old, const uint8_t *mask, int64_t n_seq,
                                       int64_t seq_len, const float *adv, const int64_t *group_offsets,
                                       int64_t n_groups, float clip_eps, float *out_g_logp, double *out_objective,
                                       double *out_clip_frac, void *workspace, size_t workspace_bytes, void *stream) {
  if (n_seq < 0 || seq_len < 0 || n_groups < 0 || !(clip_eps >= 0.f) || !out_objective) return E3_ERR_INVALID_ARG;
  if (n_seq > 0 && (!adv || (seq_len > 0 && (!logp || !logp_old)))) return E3_ERR_INVALID_ARG;
  if (n_groups > 0 && !group_offsets) return E3_ERR_INVALID_ARG;
  if (n_seq >= (int64_t(1) << 31)) return E3_ERR_INVALID_ARG;
  if (misaligned(logp, 4) || misaligned(logp_old, 4) || misaligned(adv, 4) || misaligned(group_offsets, 8) ||
      misaligned(out_g_logp, 4) || misaligned(out_objective, 8) || misaligned(out_clip_frac, 8) || misaligned(workspace, 8))
    return E3_ERR_ALIGNMENT;
  if (!workspace || workspace_bytes < e3::grpo_workspace_bytes(n_seq)) return E3_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  SeqPartial *part = static_cast<SeqPartial *>(workspace);
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(kThreads);
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (n_seq > 0) {
    cfg.gridDim = dim3((unsigned)n_seq);
    if (cudaLaunchKernelEx(&cfg, grpo_seq_kernel, logp, logp_old, mask, seq_len, adv, group_offsets, n_groups,
                           1.0 - (double)clip_eps, 1.0 + (double)clip_eps, out_g_logp, part) != cudaSuccess)
      return E3_ERR_CUDA;
  }
  cfg.gridDim = dim3(1);
  if (cudaLaunchKernelEx(&cfg, grpo_final_kernel, (const SeqPartial *)part, n_seq, n_groups, out_objective,
                         out_clip_frac) != cudaSuccess)
    return E3_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? E3_OK : E3_ERR_CUDA;
}
