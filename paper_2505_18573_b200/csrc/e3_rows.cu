// Row-streaming kernels: one pass over the logits of a row gives the softmax statistics
// (App. A: Z(beta), Eq. "entropy" in its shifted form H = ln Z + beta sum p_i Delta_i), the
// log-probability of one token and, for rollouts, a Gumbel-max sample.
//
// Work split.  A thread-block cluster owns whole rows (cluster c takes rows c, c + n_clusters, ...);
// CTA k of the cluster streams the k-th slice of every row.  Inside a CTA eight warps stream
// 16-entry groups (one coarse Philox call each) and a ninth warp finishes rows: it merges the
// cluster's partial states, which arrive in its shared memory through DSMEM, and writes the
// outputs in fp64.  The owner of a row rotates over the CTAs of the cluster.  Streaming warps
// never wait for the finishing warp: they arrive at the cluster barrier after handing over their
// partial state and only wait for that barrier just before handing over the next one.
//
// Numerics.  Each thread keeps (R, Z, W): R the largest logit it has seen, Z = sum 2^t,
// W = sum 2^t * t with t = z*c - R*c and c = log2(e)/tau.  R only grows, and the sums are
// rescaled when it does.  States merge associatively; the per-row result is formed in fp64:
// H = ln Z - ln2 * W / Z,  ln p_tok = (z_tok*c - M) ln2 - ln Z.
//
// Sampler 0 (one Gumbel per vocabulary entry).  u_i has 8 coarse + 32 fine bits.  An entry can
// only win if its coarse byte is 255 (g_i >= 5.5432) or if z_i/tau exceeds the best score so
// far minus 5.5432, so the fine bits and the logarithms are evaluated for a fraction of a percent
// of the entries.  Those candidates are queued per warp and evaluated in fp64 with all lanes
// busy; every decision that picks the token is taken in fp64 with the same expression order as
// the definition, so the result does not depend on the gating.
#include "e3_rows.cuh"

#include <cooperative_groups.h>
#include <math_constants.h>

namespace cg = cooperative_groups;

namespace e3 {
namespace {

constexpr int kQueueCap = 160;
constexpr int kDrainAt = 32;
constexpr float kLog2e = 1.4426950408889634f;
constexpr double kLn2 = 0.6931471805599453094;
// Largest Gumbel value an entry whose coarse byte is below 255 can reach is -ln(-ln(255/256)) = 5.54322...;
// with all 40 bits set the largest value is -ln(-ln(1 - 2^-41)) = 28.41903...  Both rounded up.
constexpr float kGumbelCapCoarse = 5.5433f;
constexpr float kGumbelCapAll = 28.4192f;

struct Partial {
  double M, Z, W;  // reference (log2 units), sum 2^t, sum 2^t t
  double y;        // best perturbed score (greedy rows: largest logit)
  int idx;         // its vocabulary index, -1 = none
  int err;         // bit 0: NaN or +inf logit seen
};

struct WarpPartial {
  float M, Z, W;
  int idx;
  double y;
  int err;
  int pad;
};

struct Smem {
  Partial part[2][kMaxCluster];         // written by the CTAs of the cluster (DSMEM), read by the finishing warp
  WarpPartial wpart[2][kStreamWarps];
  int queue[kStreamWarps][kQueueCap];
  int qcount[kStreamWarps];
  int best_enc[2];                      // CTA-wide best perturbed score so far (monotone int encoding of a float)
};

struct RowCtx {
  const char *row;   // first element of the row
  float tau;
  float c;           // log2(e) / tau
  uint32_t grow;     // global row index (row_base + row)
};

struct Acc {
  float R, nRc, Z0, Z1, W0, W1;
};

struct Best {
  double y;
  int idx;
  // gate, all conservative (rounded towards "evaluate more")
  int enc;
  float zthr;   // logit above which an entry may win whatever its coarse byte
  float zthr2;  // logit above which an entry with coarse byte 255 may win
};

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void stream_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kStreamThreads) : "memory"); }

__device__ __forceinline__ bool stream_bar_or(bool v) {
  int r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.s32 p, %1, 0;\n\tbar.red.or.pred q, 1, %2, p;\n\tselp.s32 %0, 1, 0, q;\n\t}"
      : "=r"(r)
      : "r"((int)v), "n"(kStreamThreads)
      : "memory");
  return r != 0;
}

__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11) with precomputed round keys.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox(const uint32_t *rk, uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t a = (uint64_t)c0 * 0xD2511F53u;
    const uint64_t b = (uint64_t)c2 * 0xCD9E8D57u;
    const uint32_t y0 = (uint32_t)(b >> 32) ^ c1 ^ rk[2 * r];
    const uint32_t y2 = (uint32_t)(a >> 32) ^ c3 ^ rk[2 * r + 1];
    c1 = (uint32_t)b;
    c3 = (uint32_t)a;
    c0 = y0;
    c2 = y2;
  }
  return make_uint4(c0, c1, c2, c3);
}

__device__ __forceinline__ uint32_t pick_word(const uint4 &w, int k) {
  return k == 0 ? w.x : (k == 1 ? w.y : (k == 2 ? w.z : w.w));
}

// Bit 7 of every byte that equals 0xFF.
__device__ __forceinline__ uint32_t ff_bytes(uint32_t w) { return w & 0x80808080u & ((w & 0x7F7F7F7Fu) + 0x01010101u); }

__device__ __forceinline__ int enc_float(float f) {
  int b = __float_as_int(f);
  return b >= 0 ? b : (b ^ 0x7FFFFFFF);
}
__device__ __forceinline__ float dec_float(int e) { return __int_as_float(e >= 0 ? e : (e ^ 0x7FFFFFFF)); }

// ---------------------------------------------------------------------------------------------
// Loads
// ---------------------------------------------------------------------------------------------
template <int DT>
__device__ __forceinline__ float load_elem(const char *row, int64_t i) {
  if (DT == 0) return __ldg(reinterpret_cast<const float *>(row) + i);
  return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short *>(row) + i) << 16);
}

template <int DT>
__device__ __forceinline__ void load_group_vec(const char *row, int64_t e0, float (&z)[16]) {
  if (DT == 0) {
    const float4 *p = reinterpret_cast<const float4 *>(row + e0 * 4);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      float4 v = __ldg(p + q);
      z[4 * q + 0] = v.x; z[4 * q + 1] = v.y; z[4 * q + 2] = v.z; z[4 * q + 3] = v.w;
    }
  } else {
    const uint4 *p = reinterpret_cast<const uint4 *>(row + e0 * 2);
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      uint4 v = __ldg(p + q);
      uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        z[8 * q + 2 * j + 0] = __uint_as_float(w[j] << 16);
        z[8 * q + 2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
      }
    }
  }
}

template <int DT>
__device__ __forceinline__ void load_group_guarded(const char *row, int64_t e0, int valid, float (&z)[16]) {
#pragma unroll
  for (int k = 0; k < 16; ++k) z[k] = k < valid ? load_elem<DT>(row, e0 + k) : -CUDART_INF_F;
}

// ---------------------------------------------------------------------------------------------
// Online (R, Z, W) accumulation of one group.  Returns the group's largest logit.
// CAREFUL also accepts -inf entries (skipped) and flags NaN; the fast form leaves NaN in the
// sums when it meets either, which sends the slice through the careful form once more.
// ---------------------------------------------------------------------------------------------
template <bool CAREFUL>
__device__ __forceinline__ float accumulate(Acc &a, const float (&z)[16], float c, int &err) {
  float gmax = z[0];
#pragma unroll
  for (int k = 1; k < 16; ++k) gmax = fmaxf(gmax, z[k]);
  if (gmax > a.R) {
    if (gmax == CUDART_INF_F) {
      err |= 1;
      return gmax;
    }
    const float nRc = -gmax * c;
    if (a.R != -CUDART_INF_F) {
      const float d = nRc - a.nRc;
      const float f = ex2f(d);
      if (f == 0.f) {
        a.Z0 = a.Z1 = a.W0 = a.W1 = 0.f;
      } else {
        a.W0 = f * fmaf(d, a.Z0, a.W0);
        a.W1 = f * fmaf(d, a.Z1, a.W1);
        a.Z0 *= f;
        a.Z1 *= f;
      }
    }
    a.R = gmax;
    a.nRc = nRc;
  }
#pragma unroll
  for (int k = 0; k < 16; k += 2) {
    if (CAREFUL) {
      if (z[k] != z[k] || z[k + 1] != z[k + 1]) err |= 1;
      if (z[k] != -CUDART_INF_F && z[k] == z[k]) {
        const float t = fmaf(z[k], c, a.nRc), e = ex2f(t);
        a.Z0 += e;
        a.W0 = fmaf(e, t, a.W0);
      }
      if (z[k + 1] != -CUDART_INF_F && z[k + 1] == z[k + 1]) {
        const float t = fmaf(z[k + 1], c, a.nRc), e = ex2f(t);
        a.Z1 += e;
        a.W1 = fmaf(e, t, a.W1);
      }
    } else {
      const float t0 = fmaf(z[k], c, a.nRc), t1 = fmaf(z[k + 1], c, a.nRc);
      const float e0 = ex2f(t0), e1 = ex2f(t1);
      a.Z0 += e0;
      a.Z1 += e1;
      a.W0 = fmaf(e0, t0, a.W0);
      a.W1 = fmaf(e1, t1, a.W1);
    }
  }
  return gmax;
}

// ---------------------------------------------------------------------------------------------
// Sampler 0: gate, queue and exact evaluation of candidates.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void set_gate(Best &b, int enc, float tau) {
  b.enc = enc;
  const float B = dec_float(enc);
  const float t1 = (B - kGumbelCapCoarse) * tau, t2 = (B - kGumbelCapAll) * tau;
  // two fp32 roundings (<= 1.2e-7 relative) are covered by the 1e-6 relative slack
  b.zthr = t1 - fabsf(t1) * 1e-6f - 1e-30f;
  b.zthr2 = t2 - fabsf(t2) * 1e-6f - 1e-30f;
  if (enc == enc_float(-CUDART_INF_F)) b.zthr = b.zthr2 = -CUDART_INF_F;
}

template <int DT>
__device__ __noinline__ void eval_candidate(const RowsParams &p, const RowCtx &rc, int i, Best &b, int *cta_best) {
  const float zf = load_elem<DT>(rc.row, i);
  if (!(zf > -CUDART_INF_F) || zf == CUDART_INF_F) return;
  const uint4 cw = philox(p.round_key, (uint32_t)i >> 4, rc.grow, p.ctr_lo, p.ctr_hi8 | 0u);
  const uint32_t cbyte = (pick_word(cw, (i & 15) >> 2) >> (8 * (i & 3))) & 0xFFu;
  const uint4 fw = philox(p.round_key, (uint32_t)i >> 2, rc.grow, p.ctr_lo, p.ctr_hi8 | 1u);
  const uint32_t x = pick_word(fw, i & 3);
  // u = (c + (x + 1/2) 2^-32) / 256, exact in fp64; y = z/tau + (-ln(-ln u))
  const double u = ((double)cbyte + ((double)x + 0.5) * 0x1p-32) / 256.0;
  const double s = (double)zf / (double)rc.tau;
  const double y = s + (-log(-log(u)));
  if (y > b.y || (y == b.y && i < b.idx)) {
    b.y = y;
    b.idx = i;
    const int enc = enc_float(__double2float_rd(y));
    if (enc > b.enc) {
      set_gate(b, enc, rc.tau);
      atomicMax(cta_best, enc);
    }
  }
}

template <int DT>
__device__ __forceinline__ void push_candidate(const RowsParams &p, const RowCtx &rc, int i, Best &b, Smem &sm,
                                               int warp, int parity) {
  const int slot = atomicAdd(&sm.qcount[warp], 1);
  if (slot < kQueueCap)
    sm.queue[warp][slot] = i;
  else
    eval_candidate<DT>(p, rc, i, b, &sm.best_enc[parity]);
}

template <int DT>
__device__ __forceinline__ void drain_queue(const RowsParams &p, const RowCtx &rc, Best &b, Smem &sm, int warp,
                                            int lane, int parity, int at_least) {
  __syncwarp();
  int n = *reinterpret_cast<volatile int *>(&sm.qcount[warp]);
  if (n < at_least) return;
  n = n < kQueueCap ? n : kQueueCap;
  for (int e = lane; e < n; e += 32) eval_candidate<DT>(p, rc, sm.queue[warp][e], b, &sm.best_enc[parity]);
  __syncwarp();
  if (lane == 0) sm.qcount[warp] = 0;
  __syncwarp();
}

// ---------------------------------------------------------------------------------------------
// One CTA's slice [e_lo, e_hi) of one row.
// ---------------------------------------------------------------------------------------------
template <int DT, int SAMPLER, bool ALIGNED, bool CAREFUL>
__device__ __forceinline__ void stream_slice(const RowsParams &p, const RowCtx &rc, int64_t e_lo, int64_t e_hi,
                                             Acc &acc, Best &best, int &err, Smem &sm, int warp, int lane,
                                             int parity) {
  if (e_lo >= e_hi) return;  // this CTA has no part of the row (V smaller than the cluster's reach)
  const int64_t g_lo = e_lo >> 4, g_hi = (e_hi + 15) >> 4, g_full = p.V >> 4;
  for (int64_t g0 = g_lo + (int64_t)warp * 32; g0 < g_hi; g0 += kStreamWarps * 32) {
    const int64_t g = g0 + lane;
    if (g < g_hi) {
      float z[16];
      float gmax;
      const int64_t e0 = g << 4;
      if (g < g_full) {
        if (ALIGNED)
          load_group_vec<DT>(rc.row, e0, z);
        else
          load_group_guarded<DT>(rc.row, e0, 16, z);
        gmax = accumulate<CAREFUL>(acc, z, rc.c, err);
      } else {
        load_group_guarded<DT>(rc.row, e0, (int)(p.V - e0), z);
        gmax = accumulate<true>(acc, z, rc.c, err);
      }
      if (SAMPLER == 0) {
        const int enc = *reinterpret_cast<volatile int *>(&sm.best_enc[parity]);
        if (enc > best.enc) set_gate(best, enc, rc.tau);
        const uint4 cb = philox(p.round_key, (uint32_t)g, rc.grow, p.ctr_lo, p.ctr_hi8 | 0u);
        const uint32_t h = ff_bytes(cb.x) | ff_bytes(cb.y) | ff_bytes(cb.z) | ff_bytes(cb.w);
        if (h != 0u || gmax > best.zthr) {
#pragma unroll
          for (int k = 0; k < 16; ++k) {
            const bool ff = (ff_bytes(pick_word(cb, k >> 2)) >> (8 * (k & 3)) & 0x80u) != 0u;
            if ((ff && z[k] > best.zthr2) || z[k] > best.zthr) push_candidate<DT>(p, rc, (int)e0 + k, best, sm, warp, parity);
          }
        }
      }
    }
    if (SAMPLER == 0) drain_queue<DT>(p, rc, best, sm, warp, lane, parity, kDrainAt);
  }
  if (SAMPLER == 0) drain_queue<DT>(p, rc, best, sm, warp, lane, parity, 1);
}

// Greedy rows (tau == 0): largest logit, lowest index.
template <int DT>
__device__ __forceinline__ void greedy_slice(const RowsParams &p, const RowCtx &rc, int64_t e_lo, int64_t e_hi,
                                             Best &best, int &err, int tid) {
  for (int64_t i = e_lo + tid; i < e_hi; i += kStreamThreads) {
    const float z = load_elem<DT>(rc.row, i);
    if (z != z || z == CUDART_INF_F) err |= 1;
    if ((double)z > best.y) {
      best.y = (double)z;
      best.idx = (int)i;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Merging partial states
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void merge_stats_f(float &M, float &Z, float &W, float M2, float Z2, float W2) {
  if (Z2 == 0.f) return;
  if (Z == 0.f) {
    M = M2; Z = Z2; W = W2;
    return;
  }
  const float Mn = fmaxf(M, M2);
  const float d1 = M - Mn, d2 = M2 - Mn;
  const float a = ex2f(d1), b = ex2f(d2);
  W = a * fmaf(d1, Z, W) + b * fmaf(d2, Z2, W2);
  Z = a * Z + b * Z2;
  M = Mn;
}

__device__ __forceinline__ void merge_stats_d(double &M, double &Z, double &W, double M2, double Z2, double W2) {
  if (Z2 == 0.0) return;
  if (Z == 0.0) {
    M = M2; Z = Z2; W = W2;
    return;
  }
  const double Mn = fmax(M, M2);
  const double d1 = M - Mn, d2 = M2 - Mn;
  const double a = exp2(d1), b = exp2(d2);
  W = a * (W + d1 * Z) + b * (W2 + d2 * Z2);
  Z = a * Z + b * Z2;
  M = Mn;
}

__device__ __forceinline__ void merge_best(double &y, int &idx, double y2, int idx2) {
  if (idx2 >= 0 && (idx < 0 || y2 > y || (y2 == y && idx2 < idx))) {
    y = y2;
    idx = idx2;
  }
}

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
template <int DT, int SAMPLER, bool ALIGNED>
__global__ void __launch_bounds__(kThreads, 2) rows_kernel(const __grid_constant__ RowsParams p) {
  __shared__ Smem sm;
  cg::cluster_group cluster = cg::this_cluster();
  const int S = (int)cluster.num_blocks();
  const int rank = (int)cluster.block_rank();
  const int64_t cluster_id = blockIdx.x / S, n_clusters = gridDim.x / S;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool streamer = warp < kStreamWarps;
  const int esize = DT == 0 ? 4 : 2;

  if (tid < kStreamWarps) sm.qcount[tid] = 0;
  if (tid == 0) sm.best_enc[0] = sm.best_enc[1] = enc_float(-CUDART_INF_F);
  __syncthreads();

  int it = 0;  // rows this cluster has put through the cluster barrier
  for (int64_t row = cluster_id; row < p.rows; row += n_clusters) {
    const float tau = p.temps ? __ldg(p.temps + row) : p.temp_scalar;
    const bool sample = p.mode == kModeSample;
    if (!sample && p.mask && __ldg(p.mask + row) == 0) {
      if (rank == 0 && tid == 0) {
        if (p.out_logp) p.out_logp[row] = 0.f;
        if (p.out_ent) p.out_ent[row] = 0.f;
      }
      continue;
    }
    const bool greedy = sample && tau == 0.f;
    if (!greedy && !(tau > 0.f && tau < CUDART_INF_F)) {
      if (rank == 0 && tid == 0) {
        if (sample) p.out_tok[row] = -1;
        if (p.out_logp) p.out_logp[row] = CUDART_NAN_F;
        if (p.out_ent) p.out_ent[row] = CUDART_NAN_F;
      }
      continue;
    }
    RowCtx rc;
    rc.row = reinterpret_cast<const char *>(p.logits) + (size_t)row * (size_t)p.row_stride * esize;
    rc.tau = tau;
    rc.c = greedy ? 0.f : __fdiv_rn(kLog2e, tau);
    rc.grow = p.row_base + (uint32_t)row;
    const int parity = it & 1;
    const int owner = it % S;

    if (streamer) {
      const int64_t e_lo = (int64_t)rank * p.seg < p.V ? (int64_t)rank * p.seg : p.V;
      const int64_t e_hi = e_lo + p.seg < p.V ? e_lo + p.seg : p.V;
      Acc acc;
      Best best;
      int err = 0;
      auto reset = [&]() {
        acc.R = -CUDART_INF_F; acc.nRc = 0.f; acc.Z0 = acc.Z1 = acc.W0 = acc.W1 = 0.f;
        best.y = -CUDART_INF; best.idx = -1;
        set_gate(best, enc_float(-CUDART_INF_F), tau);
        err = 0;
      };
      reset();
      // The CTA-wide best of the row after next shares this row's slot: clear the other slot now;
      // the named barrier below orders the store before anyone reads it.
      if (tid == 0) sm.best_enc[parity ^ 1] = enc_float(-CUDART_INF_F);

      if (greedy) {
        greedy_slice<DT>(p, rc, e_lo, e_hi, best, err, tid);
      } else {
        stream_slice<DT, SAMPLER, ALIGNED, false>(p, rc, e_lo, e_hi, acc, best, err, sm, warp, lane, parity);
        const float zs = acc.Z0 + acc.Z1, ws = acc.W0 + acc.W1;
        const bool bad = !(fabsf(zs) < CUDART_INF_F) || !(fabsf(ws) < CUDART_INF_F);
        if (stream_bar_or(bad)) {
          reset();
          if (tid == 0) sm.best_enc[parity] = enc_float(-CUDART_INF_F);
          stream_bar_sync();
          stream_slice<DT, SAMPLER, ALIGNED, true>(p, rc, e_lo, e_hi, acc, best, err, sm, warp, lane, parity);
        }
      }

      // warp-level merge
      float M = -acc.nRc, Z = acc.Z0 + acc.Z1, W = acc.W0 + acc.W1;
      if (acc.R == -CUDART_INF_F) { M = 0.f; Z = 0.f; W = 0.f; }
      double y = best.y;
      int idx = best.idx;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float M2 = __shfl_xor_sync(0xffffffffu, M, o), Z2 = __shfl_xor_sync(0xffffffffu, Z, o),
                    W2 = __shfl_xor_sync(0xffffffffu, W, o);
        const double y2 = __shfl_xor_sync(0xffffffffu, y, o);
        const int idx2 = __shfl_xor_sync(0xffffffffu, idx, o);
        err |= __shfl_xor_sync(0xffffffffu, err, o);
        merge_stats_f(M, Z, W, M2, Z2, W2);
        merge_best(y, idx, y2, idx2);
      }
      if (lane == 0) {
        WarpPartial &w = sm.wpart[parity][warp];
        w.M = M; w.Z = Z; w.W = W; w.y = y; w.idx = idx; w.err = err;
      }
      stream_bar_sync();
      if (it > 0) cluster_wait();  // the slot written below was read by the owner two rows ago
      if (warp == 0) {
        double Md = 0.0, Zd = 0.0, Wd = 0.0, yd = -CUDART_INF;
        int id = -1, ed = 0;
        if (lane < kStreamWarps) {
          const WarpPartial &w = sm.wpart[parity][lane];
          Md = w.M; Zd = w.Z; Wd = w.W; yd = w.y; id = w.idx; ed = w.err;
        }
#pragma unroll
        for (int o = kStreamWarps / 2; o > 0; o >>= 1) {
          const double M2 = __shfl_xor_sync(0xffffffffu, Md, o), Z2 = __shfl_xor_sync(0xffffffffu, Zd, o),
                       W2 = __shfl_xor_sync(0xffffffffu, Wd, o), y2 = __shfl_xor_sync(0xffffffffu, yd, o);
          const int i2 = __shfl_xor_sync(0xffffffffu, id, o);
          ed |= __shfl_xor_sync(0xffffffffu, ed, o);
          merge_stats_d(Md, Zd, Wd, M2, Z2, W2);
          merge_best(yd, id, y2, i2);
        }
        if (lane == 0) {
          Partial *dst = cluster.map_shared_rank(&sm.part[parity][rank], owner);
          dst->M = Md; dst->Z = Zd; dst->W = Wd; dst->y = yd; dst->idx = id; dst->err = ed;
        }
      }
      cluster_arrive();
    } else {
      // finishing warp
      cluster_arrive();
      cluster_wait();
      if (rank == owner) {
        double Md = 0.0, Zd = 0.0, Wd = 0.0, yd = -CUDART_INF;
        int id = -1, ed = 0;
        if (lane < S) {
          const Partial &q = sm.part[parity][lane];
          Md = q.M; Zd = q.Z; Wd = q.W; yd = q.y; id = q.idx; ed = q.err;
        }
#pragma unroll
        for (int o = kMaxCluster / 2; o > 0; o >>= 1) {
          const double M2 = __shfl_xor_sync(0xffffffffu, Md, o), Z2 = __shfl_xor_sync(0xffffffffu, Zd, o),
                       W2 = __shfl_xor_sync(0xffffffffu, Wd, o), y2 = __shfl_xor_sync(0xffffffffu, yd, o);
          const int i2 = __shfl_xor_sync(0xffffffffu, id, o);
          ed |= __shfl_xor_sync(0xffffffffu, ed, o);
          merge_stats_d(Md, Zd, Wd, M2, Z2, W2);
          merge_best(yd, id, y2, i2);
        }
        if (lane == 0) {
          int tok = -1;
          float logp = CUDART_NAN_F, ent = CUDART_NAN_F;
          if (greedy) {
            if (ed == 0 && id >= 0) { tok = id; logp = 0.f; ent = 0.f; }
          } else if (ed == 0 && Zd > 0.0) {
            const double lnZ = log(Zd);
            ent = (float)(lnZ - kLn2 * (Wd / Zd));
            int t = sample ? id : __ldg(p.targets + row);
            if (sample) tok = t;
            if (t >= 0 && t < p.V) {
              const double zt = (double)load_elem<DT>(rc.row, t);
              logp = (float)((zt * (double)rc.c - Md) * kLn2 - lnZ);
            }
          }
          if (sample) p.out_tok[row] = tok;
          if (p.out_logp) p.out_logp[row] = logp;
          if (p.out_ent) p.out_ent[row] = ent;
        }
      }
    }
    ++it;
  }
  if (streamer && it > 0) cluster_wait();
}

template <int DT, int SAMPLER, bool ALIGNED>
cudaError_t launch_one(const RowsParams &p0, cudaStream_t stream) {
  RowsParams p = p0;
  auto kern = rows_kernel<DT, SAMPLER, ALIGNED>;
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;

  // Pick the cluster size that keeps the most CTAs busy over the whole launch.
  int best_S = 1, best_clusters = 1;
  double best_eff = -1.0;
  for (int S = 1; S <= kMaxCluster; S *= 2) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(S * sms), 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)S; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    int max_clusters = 0;
    e = cudaOccupancyMaxActiveClusters(&max_clusters, kern, &cfg);
    if (e != cudaSuccess || max_clusters < 1) { (void)cudaGetLastError(); continue; }
    const int64_t ncl = p.rows < max_clusters ? p.rows : max_clusters;
    const int64_t waves = (p.rows + ncl - 1) / ncl;
    // busy CTA-slots over the launch, relative to the device's capacity at this cluster size
    const double eff = (double)p.rows * S / ((double)waves * (double)(2 * sms));
    const double eff_c = eff > 1.0 ? 1.0 : eff;
    if (eff_c > best_eff + 0.02) { best_eff = eff_c; best_S = S; best_clusters = (int)ncl; }
  }
  if (best_eff < 0.0) return cudaErrorLaunchFailure;

  const int S = best_S;
  int64_t seg = (p.V + S - 1) / S;
  seg = (seg + kSliceAlign - 1) / kSliceAlign * kSliceAlign;
  p.seg = seg;

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(best_clusters * S), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = (unsigned)S; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, p);
}

}  // namespace

cudaError_t launch_rows(const RowsParams &p, int dtype, int sampler, bool aligned, cudaStream_t stream) {
#define E3_DISPATCH(DT, SM)                                            \
  return aligned ? launch_one<DT, SM, true>(p, stream) : launch_one<DT, SM, false>(p, stream)
  if (dtype == 0) {
    if (sampler < 0) { E3_DISPATCH(0, -1); }
    if (sampler == 0) { E3_DISPATCH(0, 0); }
  } else {
    if (sampler < 0) { E3_DISPATCH(1, -1); }
    if (sampler == 0) { E3_DISPATCH(1, 0); }
  }
#undef E3_DISPATCH
  return cudaErrorInvalidValue;
}

}  // namespace e3
