// Backward of the training-side pass: gradient of ln p_tok and of the entropy H with respect to the
// logits (the objective of Sec. 3.1 depends on the logits through ln pi(o_t), the entropy-regularised
// objective discussed in Sec. 4.2 also through H).  With p = softmax(z / tau), beta = 1/tau (App. A):
//   dlogits_i = beta [ g_logp (1[i == tok] - p_i) - g_ent p_i (ln p_i + H) ].
// One more streaming pass: every logit is read once and one gradient entry is written, so the kernel
// is bound by HBM traffic (read + write).  The row's normaliser is not recomputed: the forward pass
// returned ln p_tok, and ln p_i = (z_i - z_tok)/tau + ln p_tok.
//
// Work items are (row, segment of 8,192 entries), one CTA each,
// each thread moving 16-byte vectors (8 bf16 or 4 fp32 logits) with streaming loads and stores.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "e3.h"

namespace {

constexpr int kThreads = 256;
constexpr int kSegE = 8192;  // entries per work item
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct BwdParams {
  const void *logits;
  void *dlogits;
  int64_t rows, V, row_stride, d_stride;
  const int32_t *targets;
  const uint8_t *mask;
  const float *temps;
  float temp_scalar;
  const float *logp, *ent, *g_logp, *g_ent;
  int64_t segs_per_row, items;
};

struct RowCoef {  // everything one entry needs from its row
  float c;       // log2(e) / tau
  float zt;      // logit of the target
  float lp2;     // ln p_tok in log2 units
  float a_lp;    // beta * g_logp
  float a_en;    // beta * g_ent
  float H;
  int tok;
};

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Gradient entry without the 1[i == tok] part: -p_i (beta g_logp + beta g_ent (ln p_i + H)).
// log2 p_i is kept above -16384, so that an entry without weight (-inf logit) gives 0 and not 0 * inf.
__device__ __forceinline__ float grad_entry_no_target(const RowCoef &k, float z) {
  const float t = fmaxf(fmaf(z - k.zt, k.c, k.lp2), -16384.f);
  const float p = ex2f(t);
  return -p * fmaf(k.a_en, fmaf(t, kLn2, k.H), k.a_lp);
}
__device__ __forceinline__ float grad_entry(const RowCoef &k, float z, int i) {
  return grad_entry_no_target(k, z) + (i == k.tok ? k.a_lp : 0.f);
}

template <int DT>
__device__ __forceinline__ float load_logit(const void *base, int64_t idx) {
  if (DT == 0) return __ldg(static_cast<const float *>(base) + idx);
  return __uint_as_float((uint32_t)__ldg(static_cast<const unsigned short *>(base) + idx) << 16);
}
__device__ __forceinline__ unsigned short to_bf16_bits(float f) {  // round to nearest even; NaN stays NaN
  uint32_t u = __float_as_uint(f);
  if (f != f) return 0x7FC0;
  u += 0x7FFFu + ((u >> 16) & 1u);
  return (unsigned short)(u >> 16);
}
template <int DT>
__device__ __forceinline__ void store_grad(void *base, int64_t idx, float v) {
  if (DT == 0) static_cast<float *>(base)[idx] = v;
  else static_cast<unsigned short *>(base)[idx] = to_bf16_bits(v);
}

template <int DT, bool ALIGNED>
__global__ void __launch_bounds__(kThreads) backward_kernel(const BwdParams p) {
  constexpr int kVecE = DT == 0 ? 4 : 8;            // entries per 16-byte vector
  constexpr int kVecPerSeg = kSegE / kVecE;
  constexpr int kPerThread = kVecPerSeg / kThreads;  // 8 fp32 / 4 bf16 vectors per thread and item
  // programmatic dependent launch: nothing in global memory is touched before the wait, which returns once
  // the kernel before this one in the stream has completed
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  for (int64_t item = blockIdx.x; item < p.items; item += gridDim.x) {
    const int64_t row = item / p.segs_per_row;
    const int e0 = (int)((item - row * p.segs_per_row) * kSegE);
    const int e1 = (int64_t)e0 + kSegE < p.V ? e0 + kSegE : (int)p.V;
    const int64_t in0 = row * p.row_stride, out0 = row * p.d_stride;
    // 0: gradient, 1: zeros (masked row), 2: NaN (row or target not usable)
    int kind = 0;
    RowCoef k = {};
    if (p.mask && __ldg(p.mask + row) == 0) {
      kind = 1;
    } else {
      const float tau = p.temps ? __ldg(p.temps + row) : p.temp_scalar;
      k.tok = __ldg(p.targets + row);
      const float lp = __ldg(p.logp + row);
      k.H = __ldg(p.ent + row);
      if (!(tau > 0.f && tau < CUDART_INF_F) || k.tok < 0 || k.tok >= p.V || !(fabsf(lp) < CUDART_INF_F) ||
          !(fabsf(k.H) < CUDART_INF_F)) {
        kind = 2;
      } else {
        const float beta = 1.0f / tau;
        k.c = __fdiv_rn(kLog2e, tau);
        k.zt = load_logit<DT>(p.logits, in0 + k.tok);
        k.lp2 = lp * kLog2e;
        k.a_lp = p.g_logp ? beta * __ldg(p.g_logp + row) : 0.f;
        k.a_en = p.g_ent ? beta * __ldg(p.g_ent + row) : 0.f;
      }
    }
    const float fill = kind == 1 ? 0.f : CUDART_NAN_F;
    if (ALIGNED) {
      const int nvec = (e1 - e0) / kVecE;  // full vectors of this item
      const uint4 *src = reinterpret_cast<const uint4 *>(static_cast<const char *>(p.logits) +
                                                         (in0 + e0) * (DT == 0 ? 4 : 2));
      uint4 *dst = reinterpret_cast<uint4 *>(static_cast<char *>(p.dlogits) + (out0 + e0) * (DT == 0 ? 4 : 2));
      if (kind != 0) {  // nothing to read: zeros or NaN
        const uint32_t f1 = DT == 0 ? __float_as_uint(fill) : (kind == 1 ? 0u : 0x7FC07FC0u);
        const uint4 o = make_uint4(f1, f1, f1, f1);
        for (int vi = threadIdx.x; vi < nvec; vi += kThreads) __stcs(dst + vi, o);
        for (int i = e0 + nvec * kVecE + threadIdx.x; i < e1; i += kThreads) store_grad<DT>(p.dlogits, out0 + i, fill);
        continue;
      }
      uint4 v[kPerThread];
#pragma unroll
      for (int j = 0; j < kPerThread; ++j) {
        const int vi = j * kThreads + threadIdx.x;
        if (vi < nvec) v[j] = __ldcs(src + vi);
      }
#pragma unroll
      for (int j = 0; j < kPerThread; ++j) {
        const int vi = j * kThreads + threadIdx.x;
        if (vi >= nvec) continue;
        const int i0 = e0 + vi * kVecE;
        float g[kVecE];
        {
          const uint32_t w[4] = {v[j].x, v[j].y, v[j].z, v[j].w};
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            if (DT == 0) {
              g[q] = grad_entry_no_target(k, __uint_as_float(w[q]));
            } else {
              g[2 * q] = grad_entry_no_target(k, __uint_as_float(w[q] << 16));
              g[2 * q + 1] = grad_entry_no_target(k, __uint_as_float(w[q] & 0xFFFF0000u));
            }
          }
        }
        if ((unsigned)(k.tok - i0) < (unsigned)kVecE) {  // the vector that holds the target
#pragma unroll
          for (int q = 0; q < kVecE; ++q)
            if (i0 + q == k.tok) g[q] += k.a_lp;
        }
        uint4 o;
        if (DT == 0) {
          o = make_uint4(__float_as_uint(g[0]), __float_as_uint(g[1]), __float_as_uint(g[2]), __float_as_uint(g[3]));
        } else {
          uint32_t r[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(g[2 * q], g[2 * q + 1]);  // round to nearest even
            r[q] = *reinterpret_cast<const uint32_t *>(&h);
          }
          o = make_uint4(r[0], r[1], r[2], r[3]);
        }
        __stcs(dst + vi, o);
      }
      // entries behind the last full vector (the row's length need not be a multiple of the vector)
      for (int i = e0 + nvec * kVecE + threadIdx.x; i < e1; i += kThreads)
        store_grad<DT>(p.dlogits, out0 + i, grad_entry(k, load_logit<DT>(p.logits, in0 + i), i));
    } else {
      for (int i = e0 + threadIdx.x; i < e1; i += kThreads)
        store_grad<DT>(p.dlogits, out0 + i, kind == 0 ? grad_entry(k, load_logit<DT>(p.logits, in0 + i), i) : fill);
    }
  }
}

inline bool misaligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) != 0; }

}  // namespace

extern "C" e3_status e3_token_logp_entropy_backward(const void *logits, e3_dtype dt, int64_t rows, int64_t V,
                                                    int64_t row_stride, const int32_t *targets, const uint8_t *mask,
                                                    const float *temps, float temp_scalar, const float *logp,
                                                    const float *ent, const float *g_logp, const float *g_ent,
                                                    void *dlogits, int64_t dlogits_stride, void *stream) {
  if (dt != E3_F32 && dt != E3_BF16) return E3_ERR_DTYPE;
  if (rows < 0 || V < 1 || V >= (int64_t(1) << 31) || row_stride < V || dlogits_stride < V) return E3_ERR_INVALID_ARG;
  if (rows == 0) return E3_OK;
  if (!logits || !dlogits || !targets || !logp || !ent) return E3_ERR_INVALID_ARG;
  const size_t esize = dt == E3_F32 ? 4 : 2;
  if (misaligned(logits, esize) || misaligned(dlogits, esize) || misaligned(targets, 4) || misaligned(temps, 4) ||
      misaligned(logp, 4) || misaligned(ent, 4) || misaligned(g_logp, 4) || misaligned(g_ent, 4))
    return E3_ERR_ALIGNMENT;
  BwdParams p = {};
  p.logits = logits; p.dlogits = dlogits; p.rows = rows; p.V = V; p.row_stride = row_stride; p.d_stride = dlogits_stride;
  p.targets = targets; p.mask = mask; p.temps = temps; p.temp_scalar = temp_scalar;
  p.logp = logp; p.ent = ent; p.g_logp = g_logp; p.g_ent = g_ent;
  p.segs_per_row = (V + kSegE - 1) / kSegE;
  p.items = rows * p.segs_per_row;
  // One CTA per item (measured faster than a grid of a few CTAs per SM that loops: the hardware hands
  // out CTAs as SMs become free, which evens out the tail); the loop only matters beyond 2^31 - 1 items.
  const int64_t cap = 0x7fffffff;
  const unsigned grid = (unsigned)(p.items < cap ? p.items : cap);
  const bool aligned = !misaligned(logits, 16) && !misaligned(dlogits, 16) && (row_stride * esize) % 16 == 0 &&
                       (dlogits_stride * esize) % 16 == 0;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreads);
  cfg.stream = static_cast<cudaStream_t>(stream);
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e;
  if (dt == E3_F32) e = aligned ? cudaLaunchKernelEx(&cfg, backward_kernel<0, true>, p) : cudaLaunchKernelEx(&cfg, backward_kernel<0, false>, p);
  else e = aligned ? cudaLaunchKernelEx(&cfg, backward_kernel<1, true>, p) : cudaLaunchKernelEx(&cfg, backward_kernel<1, false>, p);
  return e == cudaSuccess ? E3_OK : E3_ERR_CUDA;
}
