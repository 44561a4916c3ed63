// Row-streaming kernel: one pass over the logits of a row gives the softmax statistics
// (App. A: Z(beta), Eq. "entropy" in its shifted form H = ln Z + beta sum p_i Delta_i), the
// log-probability of one token and, for rollouts, a Gumbel-max sample.
//
// Work split.  The [rows, V] matrix is cut into tiles of 512 entries and every CTA of a
// persistent grid (two per SM) takes an equal, contiguous run of tiles, so all CTAs stream the
// same number of bytes whatever the number of rows.  A run covers the tail of one row, some
// whole rows and the head of another.  Whole rows are finished by the CTA itself.  For a row
// that is cut, every CTA holding a piece stores its partial state in the caller's workspace and
// announces it with a compare-and-swap on a per-row arrival word tagged with a per-call id; the
// CTA whose announcement completes the row merges the pieces and writes the outputs.  Nobody
// waits for anybody.  (With a response mask, and when no workspace is given, CTAs take whole
// rows round-robin instead.)
//
// Inside a CTA: one warp issues bulk asynchronous copies (cp.async.bulk, no multicast) of 4,096
// entries into a 6-stage shared-memory ring guarded by mbarriers; eight warps consume the ring,
// each thread one 16-entry group per stage (= one coarse Philox call); one warp finishes rows
// (merges the eight warp states, fp64 epilogue, piece protocol) so that the consumers never
// stall on it.  Every mbarrier wait is bounded: when a wait runs out the CTA stops waiting
// altogether, finishes its fixed sequence of steps on whatever data it has and marks its rows
// invalid.
//
// Numerics.  Each thread keeps (R, Z, W): R the largest logit it has seen, Z = sum 2^t,
// W = sum 2^t * t with t = z*c - R*c and c = log2(e)/tau.  R only grows, and the sums are
// rescaled when it does.  States merge associatively; the per-row result is formed in fp64:
// H = ln Z - ln2 * W / Z,  ln p_tok = (z_tok*c - M) ln2 - ln Z.
//
// Sampler 0 (one Gumbel per vocabulary entry).  u_i has 8 coarse + 32 fine bits.  An entry can
// only win if its coarse byte is 255 (g_i >= 5.5432) or if z_i/tau exceeds the best score so
// far minus 5.5432, so the fine bits and the logarithms are evaluated for a fraction of a percent
// of the entries.  Those candidates are queued per warp, screened with an fp32 upper bound and
// the survivors evaluated in fp64 with the same expression order as the definition: the token
// never depends on the gating.
#include "e3_rows.cuh"

#include <math_constants.h>

#include <atomic>
#include <chrono>
#include <mutex>

namespace e3 {
namespace {

constexpr int kQueueCap = 160;
constexpr int kDrainAt = 32;
constexpr int kSlots = 4;  // hand-over slots between the consumer warps and the finishing warp
constexpr uint32_t kSpinLimit = 1u << 21;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2f = 0.6931471805599453f;
constexpr double kLn2 = 0.6931471805599453094;
// Largest Gumbel value an entry whose coarse byte is below 255 can reach is -ln(-ln(255/256)) = 5.54322...;
// with all 40 bits set the largest value is -ln(-ln(1 - 2^-41)) = 28.41903...  Both rounded up.
constexpr float kGumbelCapCoarse = 5.5433f;
constexpr float kGumbelCapAll = 28.4192f;

enum : int { kErrValue = 1, kErrTimeout = 4 };

struct Piece {  // one partial row state in the workspace (kPieceBytes)
  double M, Z, W;  // reference (log2 units), sum 2^t, sum 2^t t
  double y;        // best perturbed score (greedy rows: largest logit)
  int idx;         // its vocabulary index, -1 = none
  int err;
  int pad[6];
};
static_assert(sizeof(Piece) == kPieceBytes, "piece size");

struct WarpPartial {
  float M, Z, W;
  int idx;
  double y;
  int err;
  int pad;
};

struct Smem {
  unsigned long long full[kStages], empty[kStages];  // ring barriers
  unsigned long long wfull[kSlots], wfree[kSlots];   // consumer warps -> finishing warp
  unsigned long long best64;                         // (segment number << 32 | encoded best score) of sampler 0
  WarpPartial wpart[kSlots][kStreamWarps];
  int queue[kStreamWarps][kQueueCap];
  int qcount[kStreamWarps];
  int timeout;                                       // set when a bounded wait ran out
};

struct RowInfo {
  float tau, c;
  bool skip;     // masked out, or invalid temperature: no data is read
  bool invalid;  // temperature not usable
  bool greedy;
};

struct Seg {
  int64_t row;
  int e_lo, e_hi;  // entries [e_lo, e_hi) of the row
  bool whole;      // the CTA holds the whole row
  bool starts;     // holds the row's first tile
  bool first;      // first segment of this CTA
  int k0, k1;      // CTAs holding the first / last tile of the row (cut rows only)
};

struct Acc {
  float R, nRc, Z0, Z1, W0, W1;
};

struct Best {
  double y;
  int idx;
  int enc;      // encoded lower bound of the row's best score known to this thread
  float zthr;   // logit above which an entry may win whatever its coarse byte
  float zthr2;  // logit above which an entry with coarse byte 255 may win
};

// ---------------------------------------------------------------------------------------------
// small helpers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2f(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long *b, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long *b) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(b)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long *b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long *b, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_addr(b)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  After any wait of the CTA has run out, no wait blocks any more.
__device__ __forceinline__ void mbar_wait(unsigned long long *b, uint32_t parity, Smem &sm) {
  if (mbar_try_wait(b, parity)) return;
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (*reinterpret_cast<volatile int *>(&sm.timeout)) return;
    if (mbar_try_wait(b, parity)) return;
    if (it > 32) __nanosleep(it > 4096 ? 256 : 32);
  }
  *reinterpret_cast<volatile int *>(&sm.timeout) = 1;
}
__device__ __forceinline__ void bulk_copy_g2s(void *dst, const void *src, uint32_t bytes, unsigned long long *bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_addr(dst)),
               "l"(src), "r"(bytes), "r"(smem_addr(bar))
               : "memory");
}

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

// Bit 7 of every byte that equals 0xFF (exact).
__device__ __forceinline__ uint32_t ff_bytes(uint32_t w) { return w & 0x80808080u & ((w & 0x7F7F7F7Fu) + 0x01010101u); }
// Non-zero iff some byte equals 0xFF (cheaper; individual bits may over-report).
__device__ __forceinline__ uint32_t any_ff(uint32_t w) { return (~w - 0x01010101u) & w & 0x80808080u; }

__device__ __forceinline__ int enc_float(float f) {
  int b = __float_as_int(f);
  return b >= 0 ? b : (b ^ 0x7FFFFFFF);
}
__device__ __forceinline__ float dec_float(int e) { return __int_as_float(e >= 0 ? e : (e ^ 0x7FFFFFFF)); }
__device__ __forceinline__ int enc_neg_inf() { return enc_float(-CUDART_INF_F); }

// CTA-wide best score of the segment: 64-bit word (segment number, order-preserving code).
__device__ __forceinline__ void post_best(Smem &sm, uint32_t seg, int enc) {
  atomicMax(&sm.best64, ((unsigned long long)seg << 32) | (uint32_t)(enc ^ 0x80000000));
}
__device__ __forceinline__ int read_best(Smem &sm, uint32_t seg) {
  const unsigned long long v = *reinterpret_cast<volatile unsigned long long *>(&sm.best64);
  return (uint32_t)(v >> 32) == seg ? (int)((uint32_t)v ^ 0x80000000u) : enc_neg_inf();
}

// ---------------------------------------------------------------------------------------------
// Loads
// ---------------------------------------------------------------------------------------------
template <int DT>
__device__ __forceinline__ float load_elem(const char *row, int64_t i) {
  if (DT == 0) return __ldg(reinterpret_cast<const float *>(row) + i);
  return __uint_as_float((uint32_t)__ldg(reinterpret_cast<const unsigned short *>(row) + i) << 16);
}

template <int DT>
__device__ __forceinline__ float load_group_guarded(const char *row, int64_t e0, int valid, float (&z)[16]) {
  float gmax = -CUDART_INF_F;
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    z[k] = k < valid ? load_elem<DT>(row, e0 + k) : -CUDART_INF_F;
    gmax = fmaxf(gmax, z[k]);
  }
  return gmax;
}

// One full group from a pipeline stage in shared memory.  Returns the group's largest logit.
template <int DT>
__device__ __forceinline__ float load_group_smem(const unsigned char *stage, int tid, float (&z)[16]) {
  if (DT == 0) {
    const float4 *p = reinterpret_cast<const float4 *>(stage) + tid * 4;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float4 v = p[q];
      z[4 * q + 0] = v.x; z[4 * q + 1] = v.y; z[4 * q + 2] = v.z; z[4 * q + 3] = v.w;
    }
    float m[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) m[q] = fmaxf(fmaxf(z[4 * q], z[4 * q + 1]), fmaxf(z[4 * q + 2], z[4 * q + 3]));
    return fmaxf(fmaxf(m[0], m[1]), fmaxf(m[2], m[3]));
  } else {
    const uint4 *p = reinterpret_cast<const uint4 *>(stage) + tid * 2;
    const uint4 a = p[0], b = p[1];
    const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      z[2 * j + 0] = __uint_as_float(w[j] << 16);
      z[2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
    }
    const uint32_t m = max_bf16x2(max_bf16x2(max_bf16x2(w[0], w[1]), max_bf16x2(w[2], w[3])),
                                  max_bf16x2(max_bf16x2(w[4], w[5]), max_bf16x2(w[6], w[7])));
    return fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u));
  }
}

// ---------------------------------------------------------------------------------------------
// Online (R, Z, W) accumulation of one group whose largest logit is gmax.
// CAREFUL also accepts -inf entries (skipped) and flags NaN; the fast form leaves NaN in the
// sums when it meets either, which sends the thread's groups through the careful form once more.
// ---------------------------------------------------------------------------------------------
template <bool CAREFUL>
__device__ __forceinline__ void accumulate(Acc &a, const float (&z)[16], float c, float gmax, int &err) {
  if (gmax > a.R) {
    if (gmax == CUDART_INF_F) {
      err |= kErrValue;
      return;
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
      if (z[k] != z[k] || z[k + 1] != z[k + 1]) err |= kErrValue;
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
}

// ---------------------------------------------------------------------------------------------
// Sampler 0: gate, queue and evaluation of candidates.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void set_gate(Best &b, int enc, float tau) {
  b.enc = enc;
  const float B = dec_float(enc);
  const float t1 = (B - kGumbelCapCoarse) * tau, t2 = (B - kGumbelCapAll) * tau;
  // two fp32 roundings (<= 1.2e-7 relative) are covered by the 1e-6 relative slack
  b.zthr = t1 - fabsf(t1) * 1e-6f - 1e-30f;
  b.zthr2 = t2 - fabsf(t2) * 1e-6f - 1e-30f;
  if (enc == enc_neg_inf()) b.zthr = b.zthr2 = -CUDART_INF_F;
}

struct EvalCtx {
  const uint32_t *rk;
  const char *row;
  float tau;
  uint32_t grow, ctr_lo, ctr_hi8, seg;
};

template <int DT>
__device__ __noinline__ void eval_candidate(const EvalCtx &x, int i, Best &b, Smem &sm) {
  const float zf = load_elem<DT>(x.row, i);
  if (!(zf > b.zthr2) || zf == CUDART_INF_F) return;  // cannot win even with the largest Gumbel (also NaN, -inf)
  const uint4 cw = philox(x.rk, (uint32_t)i >> 4, x.grow, x.ctr_lo, x.ctr_hi8 | 0u);
  const uint32_t cbyte = (pick_word(cw, (i & 15) >> 2) >> (8 * (i & 3))) & 0xFFu;
  if (cbyte != 255u && !(zf > b.zthr)) return;
  const uint4 fw = philox(x.rk, (uint32_t)i >> 2, x.grow, x.ctr_lo, x.ctr_hi8 | 1u);
  const uint32_t xw = pick_word(fw, i & 3);
  // fp32 upper bound of the score: skip the fp64 evaluation when even that cannot reach the best known score
  {
    float gh;
    if (cbyte == 255u) {
      // 1 - u >= (2^32 - 1 - x) 2^-40 (and >= 2^-41); -ln u >= 1 - u, so g <= -ln(1 - u)
      const float d = fmaxf((float)(~xw), 0.5f) * (0x1p-40f * 0.999999f);
      gh = -lg2f(d) * kLn2f;
    } else {
      const float uh = fminf(((float)cbyte + ((float)xw + 1.0f) * 0x1p-32f) * (0.00390625f * 1.000001f), 0.9999f);
      gh = -lg2f(-lg2f(uh) * kLn2f) * kLn2f;
    }
    const float sf = zf / x.tau;
    const float yh = sf + fabsf(sf) * 2e-6f + gh + 2e-3f;
    if (yh < dec_float(b.enc)) return;
  }
  // u = (c + (x + 1/2) 2^-32) / 256, exact in fp64; y = z/tau + (-ln(-ln u))
  const double u = ((double)cbyte + ((double)xw + 0.5) * 0x1p-32) / 256.0;
  const double s = (double)zf / (double)x.tau;
  const double y = s + (-log(-log(u)));
  if (y > b.y || (y == b.y && i < b.idx)) {
    b.y = y;
    b.idx = i;
    const int enc = enc_float(__double2float_rd(y));
    if (enc > b.enc) {
      set_gate(b, enc, x.tau);
      post_best(sm, x.seg, enc);
    }
  }
}

template <int DT>
__device__ __forceinline__ void push_candidate(const EvalCtx &x, int i, Best &b, Smem &sm, int warp) {
  const int slot = atomicAdd(&sm.qcount[warp], 1);
  if (slot < kQueueCap)
    sm.queue[warp][slot] = i;
  else
    eval_candidate<DT>(x, i, b, sm);
}

template <int DT>
__device__ __forceinline__ void drain_queue(const EvalCtx &x, Best &b, Smem &sm, int warp, int lane, int at_least) {
  __syncwarp();
  int n = *reinterpret_cast<volatile int *>(&sm.qcount[warp]);
  if (n < at_least) return;
  n = n < kQueueCap ? n : kQueueCap;
  for (int e = lane; e < n; e += 32) eval_candidate<DT>(x, sm.queue[warp][e], b, sm);
  __syncwarp();
  if (lane == 0) sm.qcount[warp] = 0;
  __syncwarp();
}

// Gate, seed and queue for one group (sampler 0).  `seed` is warp-uniform: true on the warp's first
// step of a segment, when nothing is known about the row's best score yet.
template <int DT>
__device__ __forceinline__ void sample_group(const EvalCtx &x, const float (&z)[16], float gmax, bool have, int e0,
                                             int valid, Best &b, Smem &sm, int warp, bool seed) {
  uint4 cb = make_uint4(0, 0, 0, 0);
  if (have) cb = philox(x.rk, (uint32_t)e0 >> 4, x.grow, x.ctr_lo, x.ctr_hi8 | 0u);
  if (seed) {
    // A valid lower bound of the row's best score, from the coarse byte of the group's largest entry alone:
    // u >= (c + 2^-33)/256  =>  g >= -ln(ln 256 - ln(c + 2^-33)).
    float ylo = -CUDART_INF_F;
    if (have && gmax > -CUDART_INF_F && gmax < CUDART_INF_F) {
      uint32_t cbyte = 0;
#pragma unroll
      for (int k = 15; k >= 0; --k)
        if (z[k] == gmax) cbyte = (pick_word(cb, k >> 2) >> (8 * (k & 3))) & 0xFFu;
      const float neg_ln_u = (8.0f - lg2f((float)cbyte + 0x1p-33f)) * kLn2f;
      const float glo = -lg2f(neg_ln_u) * kLn2f;
      const float sf = gmax / x.tau;
      ylo = sf - fabsf(sf) * 2e-6f + glo - 2e-3f;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ylo = fmaxf(ylo, __shfl_xor_sync(0xffffffffu, ylo, o));
    int enc = enc_float(ylo);
    if ((threadIdx.x & 31) == 0 && enc > enc_neg_inf()) post_best(sm, x.seg, enc);
    const int cta = read_best(sm, x.seg);
    enc = enc > cta ? enc : cta;
    if (enc > b.enc) set_gate(b, enc, x.tau);
  } else {
    const int enc = read_best(sm, x.seg);
    if (enc > b.enc) set_gate(b, enc, x.tau);
  }
  if (!have) return;
  const uint32_t h = any_ff(cb.x) | any_ff(cb.y) | any_ff(cb.z) | any_ff(cb.w);
  const bool over = gmax > b.zthr;
  if (h != 0u || over) {
    uint32_t bits = 0;  // bit k: entry k is a candidate
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const uint32_t f = ff_bytes(pick_word(cb, w));
      bits |= (((f >> 7) & 1u) | ((f >> 14) & 2u) | ((f >> 21) & 4u) | ((f >> 28) & 8u)) << (4 * w);
    }
    if (over) {
#pragma unroll
      for (int k = 0; k < 16; ++k) bits |= (z[k] > b.zthr ? 1u : 0u) << k;
    }
    bits &= (1u << valid) - 1u;  // the row may end inside the group
    while (bits) {
      const int k = __ffs(bits) - 1;
      bits &= bits - 1;
      push_candidate<DT>(x, e0 + k, b, sm, warp);
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
// Work split
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ int64_t first_tile_of(const RowsParams &p, int64_t b) {
  return b * p.tiles_q + (b < p.tiles_r ? b : p.tiles_r);
}
__device__ __forceinline__ int cta_of_tile(const RowsParams &p, int64_t t) {
  const int64_t big = p.tiles_r * (p.tiles_q + 1);
  return (int)(t < big ? t / (p.tiles_q + 1) : p.tiles_r + (t - big) / p.tiles_q);
}

struct Walker {
  int64_t t, t1, row_i;
  bool first;
  __device__ explicit Walker(const RowsParams &p) {
    first = true;
    row_i = blockIdx.x;
    t = first_tile_of(p, blockIdx.x);
    t1 = first_tile_of(p, (int64_t)blockIdx.x + 1);
  }
  __device__ bool next(const RowsParams &p, Seg &s) {
    if (p.interleaved) {
      if (row_i >= p.rows) return false;
      s.row = row_i; s.e_lo = 0; s.e_hi = (int)p.V; s.whole = true; s.starts = true; s.first = first; s.k0 = s.k1 = 0;
      row_i += gridDim.x;
      first = false;
      return true;
    }
    if (t >= t1) return false;
    const int64_t row = t / p.tiles_per_row, tin = t - row * p.tiles_per_row;
    const int64_t n = p.tiles_per_row - tin < t1 - t ? p.tiles_per_row - tin : t1 - t;
    const int64_t lo = tin * kTile, hi = (tin + n) * kTile;
    s.row = row;
    s.e_lo = (int)(lo < p.V ? lo : p.V);
    s.e_hi = (int)(hi < p.V ? hi : p.V);
    s.starts = tin == 0;
    s.whole = tin == 0 && n == p.tiles_per_row;
    s.first = first;
    s.k0 = s.k1 = 0;
    if (!s.whole) {
      s.k0 = cta_of_tile(p, row * p.tiles_per_row);
      s.k1 = cta_of_tile(p, (row + 1) * p.tiles_per_row - 1);
    }
    first = false;
    t += n;
    return true;
  }
};

__device__ __forceinline__ RowInfo classify(const RowsParams &p, int64_t row) {
  RowInfo r;
  r.tau = p.temps ? __ldg(p.temps + row) : p.temp_scalar;
  const bool sample = p.mode == kModeSample;
  const bool masked = !sample && p.mask && __ldg(p.mask + row) == 0;
  r.greedy = sample && r.tau == 0.f;
  r.invalid = !masked && !r.greedy && !(r.tau > 0.f && r.tau < CUDART_INF_F);
  r.skip = masked || r.invalid;
  r.c = r.greedy || r.skip ? 0.f : __fdiv_rn(kLog2e, r.tau);
  return r;
}

template <int DT>
__device__ __forceinline__ const char *row_ptr(const RowsParams &p, int64_t row) {
  return reinterpret_cast<const char *>(p.logits) + (size_t)row * (size_t)p.row_stride * (DT == 0 ? 4 : 2);
}

// ---------------------------------------------------------------------------------------------
// Row epilogue (one thread, fp64)
// ---------------------------------------------------------------------------------------------
template <int DT>
__device__ __forceinline__ void finish_row(const RowsParams &p, int64_t row, const RowInfo &ri, double M, double Z,
                                           double W, double y, int idx, int err) {
  const bool sample = p.mode == kModeSample;
  int tok = -1;
  float logp = CUDART_NAN_F, ent = CUDART_NAN_F;
  if (ri.greedy) {
    if (err == 0 && idx >= 0) { tok = idx; logp = 0.f; ent = 0.f; }
  } else if (err == 0 && Z > 0.0) {
    const double lnZ = log(Z);
    ent = (float)(lnZ - kLn2 * (W / Z));
    const int t = sample ? idx : __ldg(p.targets + row);
    if (sample) tok = t;
    if (t >= 0 && t < p.V) {
      const double zt = (double)load_elem<DT>(row_ptr<DT>(p, row), t);
      logp = (float)((zt * (double)ri.c - M) * kLn2 - lnZ);
    }
  }
  if (sample) p.out_tok[row] = tok;
  if (p.out_logp) p.out_logp[row] = logp;
  if (p.out_ent) p.out_ent[row] = ent;
}

__device__ __forceinline__ void write_skipped(const RowsParams &p, int64_t row, const RowInfo &ri) {
  const bool sample = p.mode == kModeSample;
  const float v = ri.invalid ? CUDART_NAN_F : 0.f;
  if (sample) p.out_tok[row] = -1;
  if (p.out_logp) p.out_logp[row] = v;
  if (p.out_ent) p.out_ent[row] = v;
}

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
template <int DT, int SAMPLER, bool RING>
__global__ void __launch_bounds__(kThreads, 2) rows_kernel(const __grid_constant__ RowsParams p) {
  extern __shared__ __align__(128) unsigned char ring[];
  __shared__ Smem sm;
  constexpr int kEsize = DT == 0 ? 4 : 2;
  constexpr int kStageBytes = kChunk * kEsize;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&sm.full[s], 1); mbar_init(&sm.empty[s], kStreamWarps); }
    for (int s = 0; s < kSlots; ++s) { mbar_init(&sm.wfull[s], kStreamWarps); mbar_init(&sm.wfree[s], 1); }
    sm.best64 = 0ull;
    sm.timeout = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < kStreamWarps) sm.qcount[tid] = 0;
  __syncthreads();

  const int full_end = (int)(p.V & ~(int64_t)15);  // entries covered by full groups

  if (warp < kStreamWarps) {
    // ------------------------------------------------------------------ consumers
    Walker wk(p);
    Seg s;
    uint32_t cc = 0;   // pipeline chunks consumed so far
    uint32_t n = 0;    // segments handed to the finishing warp so far
    while (wk.next(p, s)) {
      const RowInfo ri = classify(p, s.row);
      if (ri.skip) continue;
      const char *row = row_ptr<DT>(p, s.row);
      EvalCtx ex;
      ex.rk = p.round_key; ex.row = row; ex.tau = ri.tau; ex.grow = p.row_base + (uint32_t)s.row;
      ex.ctr_lo = p.ctr_lo; ex.ctr_hi8 = p.ctr_hi8; ex.seg = n + 1;

      Acc acc;
      acc.R = -CUDART_INF_F; acc.nRc = 0.f; acc.Z0 = acc.Z1 = acc.W0 = acc.W1 = 0.f;
      Best best;
      best.y = -CUDART_INF; best.idx = -1;
      set_gate(best, enc_neg_inf(), ri.tau);
      int err = 0;
      bool seed = SAMPLER == 0 && !ri.greedy;

      const int nchunks = s.e_hi > s.e_lo ? (s.e_hi - s.e_lo + kChunk - 1) / kChunk : 0;
      for (int c = 0; c < nchunks; ++c) {
        const int e0 = s.e_lo + c * kChunk + tid * kGroup;
        const bool have = e0 < s.e_hi;
        const bool full = e0 + kGroup <= full_end;
        float z[16];
        float gmax = -CUDART_INF_F;
        if (RING) {
          const uint32_t stage = cc % kStages, round = cc / kStages;
          mbar_wait(&sm.full[stage], round & 1u, sm);
          if (have && full) gmax = load_group_smem<DT>(ring + (size_t)stage * kStageBytes, tid, z);
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.empty[stage]);
          ++cc;
          if (have && !full) gmax = load_group_guarded<DT>(row, e0, (int)p.V - e0, z);
        } else if (have) {
          gmax = load_group_guarded<DT>(row, e0, full ? 16 : (int)p.V - e0, z);
        }
        if (ri.greedy) {
          if (have) {
            int kk = -1;
#pragma unroll
            for (int k = 15; k >= 0; --k) {
              if (z[k] != z[k] || z[k] == CUDART_INF_F) err |= kErrValue;
              if (z[k] == gmax) kk = k;
            }
            if (kk >= 0 && gmax > -CUDART_INF_F && (double)gmax > best.y) { best.y = (double)gmax; best.idx = e0 + kk; }
          }
          continue;
        }
        if (have) {
          if (full)
            accumulate<false>(acc, z, ri.c, gmax, err);
          else
            accumulate<true>(acc, z, ri.c, gmax, err);
        }
        if (SAMPLER == 0) {
          sample_group<DT>(ex, z, gmax, have, e0, full ? 16 : (int)p.V - e0, best, sm, warp, seed);
          seed = false;
          drain_queue<DT>(ex, best, sm, warp, lane, kDrainAt);
        }
      }
      if (SAMPLER == 0 && !ri.greedy) drain_queue<DT>(ex, best, sm, warp, lane, 1);

      if (!ri.greedy) {
        // -inf or NaN logits poison the fast sums: redo this warp's groups with the careful form
        const float zs = acc.Z0 + acc.Z1, ws = acc.W0 + acc.W1;
        const bool bad = !(fabsf(zs) < CUDART_INF_F) || !(fabsf(ws) < CUDART_INF_F);
        if (__any_sync(0xffffffffu, bad)) {
          acc.R = -CUDART_INF_F; acc.nRc = 0.f; acc.Z0 = acc.Z1 = acc.W0 = acc.W1 = 0.f;
          for (int c = 0; c < nchunks; ++c) {
            const int e0 = s.e_lo + c * kChunk + tid * kGroup;
            if (e0 < s.e_hi) {
              float z[16];
              const float gmax = load_group_guarded<DT>(row, e0, e0 + kGroup <= (int)p.V ? 16 : (int)p.V - e0, z);
              accumulate<true>(acc, z, ri.c, gmax, err);
            }
          }
        }
      }

      // warp-level merge, hand-over to the finishing warp
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
      const uint32_t slot = n % kSlots, use = n / kSlots;
      if (use > 0) mbar_wait(&sm.wfree[slot], (use - 1) & 1u, sm);
      if (lane == 0) {
        WarpPartial &w = sm.wpart[slot][warp];
        w.M = M; w.Z = Z; w.W = W; w.y = y; w.idx = idx; w.err = err;
        mbar_arrive(&sm.wfull[slot]);
      }
      ++n;
    }
  } else if (warp == kStreamWarps) {
    // ------------------------------------------------------------------ producer (one thread)
    if (RING && lane == 0) {
      Walker wk(p);
      Seg s;
      uint32_t cc = 0;
      while (wk.next(p, s)) {
        const RowInfo ri = classify(p, s.row);
        if (ri.skip) continue;
        const char *row = row_ptr<DT>(p, s.row);
        const int nchunks = s.e_hi > s.e_lo ? (s.e_hi - s.e_lo + kChunk - 1) / kChunk : 0;
        const int lim = s.e_hi < full_end ? s.e_hi : full_end;
        for (int c = 0; c < nchunks; ++c) {
          const uint32_t stage = cc % kStages, round = cc / kStages;
          if (round > 0) mbar_wait(&sm.empty[stage], (round - 1) & 1u, sm);
          const int cs = s.e_lo + c * kChunk;
          const int ce = cs + kChunk < lim ? cs + kChunk : lim;
          const uint32_t bytes = ce > cs ? (uint32_t)(ce - cs) * kEsize : 0u;
          const bool dead = *reinterpret_cast<volatile int *>(&sm.timeout) != 0;
          if (bytes > 0 && !dead) {
            mbar_arrive_expect_tx(&sm.full[stage], bytes);
            bulk_copy_g2s(ring + (size_t)stage * kStageBytes, row + (size_t)cs * kEsize, bytes, &sm.full[stage]);
          } else {
            mbar_arrive(&sm.full[stage]);
          }
          ++cc;
        }
      }
      // Before leaving, see every copy still in flight land (bounded).
      const uint32_t back = cc < (uint32_t)kStages ? cc : (uint32_t)kStages;
      for (uint32_t q = cc - back; q < cc; ++q) {
        const uint32_t stage = q % kStages, round = q / kStages;
        for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(&sm.full[stage], round & 1u); ++it) __nanosleep(64);
      }
    }
  } else {
    // ------------------------------------------------------------------ finishing warp
    Walker wk(p);
    Seg s;
    uint32_t n = 0;
    Piece *pieces = reinterpret_cast<Piece *>(p.ws_pieces);
    while (wk.next(p, s)) {
      const RowInfo ri = classify(p, s.row);
      if (ri.skip) {
        if (s.starts && lane == 0) write_skipped(p, s.row, ri);
        continue;
      }
      const uint32_t slot = n % kSlots, use = n / kSlots;
      mbar_wait(&sm.wfull[slot], use & 1u, sm);
      double Md = 0.0, Zd = 0.0, Wd = 0.0, yd = -CUDART_INF;
      int id = -1, ed = 0;
      if (lane < kStreamWarps) {
        const WarpPartial &w = sm.wpart[slot][lane];
        Md = w.M; Zd = w.Z; Wd = w.W; yd = w.y; id = w.idx; ed = w.err;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.wfree[slot]);
      ++n;
#pragma unroll
      for (int o = kStreamWarps / 2; o > 0; o >>= 1) {
        const double M2 = __shfl_xor_sync(0xffffffffu, Md, o), Z2 = __shfl_xor_sync(0xffffffffu, Zd, o),
                     W2 = __shfl_xor_sync(0xffffffffu, Wd, o), y2 = __shfl_xor_sync(0xffffffffu, yd, o);
        const int i2 = __shfl_xor_sync(0xffffffffu, id, o);
        ed |= __shfl_xor_sync(0xffffffffu, ed, o);
        merge_stats_d(Md, Zd, Wd, M2, Z2, W2);
        merge_best(yd, id, y2, i2);
      }
      if (lane != 0) continue;
      if (*reinterpret_cast<volatile int *>(&sm.timeout)) ed |= kErrTimeout;
      if (s.whole) {
        finish_row<DT>(p, s.row, ri, Md, Zd, Wd, yd, id, ed);
        continue;
      }
      // A piece of a cut row: store it, announce it; whoever completes the row finishes it.
      Piece *mine = pieces + (size_t)blockIdx.x * 2 + (s.first ? 0 : 1);
      mine->M = Md; mine->Z = Zd; mine->W = Wd; mine->y = yd; mine->idx = id; mine->err = ed;
      __threadfence();
      const unsigned long long tag = p.call_id << 16;
      unsigned long long *word = p.ws_arrivals + s.k0;
      unsigned long long cur = *reinterpret_cast<volatile unsigned long long *>(word), want = 0;
      bool done = false;
      for (int it = 0; it < 65536 && !done; ++it) {  // lock-free: some contender always gets through
        want = (cur >> 16) == p.call_id ? cur + 1 : (tag | 1ull);
        const unsigned long long prev = atomicCAS(word, cur, want);
        done = prev == cur;
        cur = prev;
      }
      if (!done || (int)(want & 0xFFFFull) != s.k1 - s.k0 + 1) continue;  // not the last piece of the row
      __threadfence();
      double Mt = 0.0, Zt = 0.0, Wt = 0.0, yt = -CUDART_INF;
      int it_ = -1, et = 0;
      for (int k = s.k0; k <= s.k1; ++k) {
        // CTA k keeps this row's piece in slot 0 when the row is the first thing it works on
        const bool is_first_seg = first_tile_of(p, k) / p.tiles_per_row == s.row;
        const volatile Piece *q = pieces + (size_t)k * 2 + (is_first_seg ? 0 : 1);
        const double M2 = q->M, Z2 = q->Z, W2 = q->W, y2 = q->y;
        const int i2 = q->idx;
        et |= q->err;
        merge_stats_d(Mt, Zt, Wt, M2, Z2, W2);
        merge_best(yt, it_, y2, i2);
      }
      finish_row<DT>(p, s.row, ri, Mt, Zt, Wt, yt, it_, et);
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
struct KernelSetup {
  int ctas_per_sm = 0;
  int sms = 0;
};

template <int DT, int SAMPLER, bool RING>
cudaError_t setup_kernel(KernelSetup &out) {
  static std::mutex lock;
  static KernelSetup cache[64];
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> hold(lock);
  if (cache[dev].ctas_per_sm == 0) {
    auto kern = rows_kernel<DT, SAMPLER, RING>;
    const size_t dyn = RING ? (size_t)kStages * kChunk * (DT == 0 ? 4 : 2) : 0;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
    if (e != cudaSuccess) return e;
    KernelSetup ks;
    e = cudaDeviceGetAttribute(&ks.sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&ks.ctas_per_sm, kern, kThreads, dyn);
    if (e != cudaSuccess) return e;
    if (ks.ctas_per_sm < 1) return cudaErrorLaunchOutOfResources;
    if (ks.ctas_per_sm > 2) ks.ctas_per_sm = 2;
    cache[dev] = ks;
  }
  out = cache[dev];
  return cudaSuccess;
}

unsigned long long next_call_id() {
  static std::atomic<unsigned long long> counter{
      (unsigned long long)std::chrono::steady_clock::now().time_since_epoch().count() & ((1ull << 40) - 1)};
  return (counter.fetch_add(1) + 1) & ((1ull << 48) - 1);
}

template <int DT, int SAMPLER, bool RING>
cudaError_t launch_one(RowsParams p, void *workspace, size_t workspace_bytes, cudaStream_t stream) {
  KernelSetup ks;
  cudaError_t e = setup_kernel<DT, SAMPLER, RING>(ks);
  if (e != cudaSuccess) return e;
  int64_t slots = (int64_t)ks.sms * ks.ctas_per_sm;
  if (slots > kMaxGrid) slots = kMaxGrid;
  p.tiles_per_row = (p.V + kTile - 1) / kTile;
  const int64_t tiles = p.rows * p.tiles_per_row;
  const bool can_cut = workspace != nullptr && workspace_bytes >= rows_workspace_bytes();
  // With a response mask the cost of a row is not known on the host: spread whole rows round-robin.
  p.interleaved = (!can_cut || (p.mask != nullptr && p.rows >= 4 * slots)) ? 1 : 0;
  int64_t grid = p.interleaved ? (p.rows < slots ? p.rows : slots) : (tiles < slots ? tiles : slots);
  p.tiles_q = tiles / grid;
  p.tiles_r = tiles % grid;
  p.ws_pieces = nullptr;
  p.ws_arrivals = nullptr;
  if (can_cut) {
    p.ws_pieces = static_cast<unsigned char *>(workspace);
    p.ws_arrivals = reinterpret_cast<unsigned long long *>(p.ws_pieces + (size_t)kMaxGrid * 2 * kPieceBytes);
  }
  p.call_id = next_call_id();
  const size_t dyn = RING ? (size_t)kStages * kChunk * (DT == 0 ? 4 : 2) : 0;
  rows_kernel<DT, SAMPLER, RING><<<(unsigned)grid, kThreads, dyn, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace

size_t rows_workspace_bytes() { return (size_t)kMaxGrid * (2 * kPieceBytes + sizeof(unsigned long long)); }

cudaError_t launch_rows(RowsParams p, int dtype, int sampler, bool aligned, void *workspace, size_t workspace_bytes,
                        cudaStream_t stream) {
#define E3_DISPATCH(DT, SM)                                                                       \
  return aligned ? launch_one<DT, SM, true>(p, workspace, workspace_bytes, stream)                \
                 : launch_one<DT, SM, false>(p, workspace, workspace_bytes, stream)
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
