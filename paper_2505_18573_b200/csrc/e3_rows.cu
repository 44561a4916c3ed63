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
// Inside a CTA: one warp issues bulk asynchronous copies (cp.async.bulk, no multicast) of 16 KiB
// into a 6-stage shared-memory ring guarded by mbarriers; eight warps consume the ring,
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

constexpr int kQueueCap = 192;
constexpr int kDrainEvery = 4;  // chunks between drains (power of two)
constexpr int kSlots = 4;  // hand-over slots between the consumer warps and the finishing warp
constexpr uint32_t kSpinLimit = 1u << 23;  // polls before a wait gives up (seconds)
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
  float ty[3];     // sampler 1: the three best block scores (fp32) ...
  int tb[3];       // ... and their block indices, -1 = none
};
static_assert(sizeof(Piece) == kPieceBytes, "piece size");

struct WarpPartial {
  float M, Z, W;
  int idx;
  double y;
  int err;
  float ty[3];
  int tb[3];
  int pad;
};

struct Smem {
  unsigned long long full[kStages], empty[kStages];  // ring barriers
  unsigned long long wfull[kSlots], wfree[kSlots];   // consumer warps -> finishing warp
  unsigned long long best64;                         // (segment number << 32 | encoded best score) of sampler 0
  WarpPartial wpart[kSlots][kStreamWarps];
  int queue[kStreamWarps][kQueueCap];
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
// One poll (the hardware may park the thread for a short, implementation-defined time).
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
// sleep_ns > 0 parks the thread between polls (roles that mostly wait must not eat issue slots).
__device__ __noinline__ void mbar_wait_slow(unsigned long long *b, uint32_t parity, Smem &sm, unsigned sleep_ns) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(b, parity)) return;
    if (*reinterpret_cast<volatile int *>(&sm.timeout)) return;
    if (sleep_ns) __nanosleep(sleep_ns);
  }
  *reinterpret_cast<volatile int *>(&sm.timeout) = 1;
}
__device__ __forceinline__ void mbar_wait(unsigned long long *b, uint32_t parity, Smem &sm, unsigned sleep_ns = 0) {
  if (!mbar_try_wait(b, parity)) mbar_wait_slow(b, parity, sm, sleep_ns);
}
// Whole-warp wait with a single polling lane (used by the finishing warp, which mostly waits).
__device__ __forceinline__ void mbar_wait_warp(unsigned long long *b, uint32_t parity, Smem &sm, int lane) {
  if (lane == 0) mbar_wait(b, parity, sm, 2000u);
  __syncwarp();
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

// One full group: raw 16-byte words from a pipeline stage, then widening to fp32.
template <int DT>
struct RawGroup {
  uint4 q[DT == 0 ? 4 : 2];
};

template <int DT>
__device__ __forceinline__ void load_raw_smem(const unsigned char *stage, int slot, RawGroup<DT> &r) {
  constexpr int kQ = DT == 0 ? 4 : 2;
  const uint4 *p = reinterpret_cast<const uint4 *>(stage) + slot * kQ;
#pragma unroll
  for (int i = 0; i < kQ; ++i) r.q[i] = p[i];
}

// Returns the group's largest logit.
template <int DT>
__device__ __forceinline__ float unpack_group(const RawGroup<DT> &r, float (&z)[16]) {
  if (DT == 0) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      z[4 * q + 0] = __uint_as_float(r.q[q].x); z[4 * q + 1] = __uint_as_float(r.q[q].y);
      z[4 * q + 2] = __uint_as_float(r.q[q].z); z[4 * q + 3] = __uint_as_float(r.q[q].w);
    }
    float m[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) m[q] = fmaxf(fmaxf(z[4 * q], z[4 * q + 1]), fmaxf(z[4 * q + 2], z[4 * q + 3]));
    return fmaxf(fmaxf(m[0], m[1]), fmaxf(m[2], m[3]));
  } else {
    const uint32_t w[8] = {r.q[0].x, r.q[0].y, r.q[0].z, r.q[0].w, r.q[DT == 0 ? 0 : 1].x, r.q[DT == 0 ? 0 : 1].y,
                           r.q[DT == 0 ? 0 : 1].z, r.q[DT == 0 ? 0 : 1].w};
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
// The reference moves to max(R, gmax) before every group.  The fast form does this without a branch
// (a per-lane branch that is rarely taken is taken by some lane of the warp almost every time):
// the sums are multiplied by f = 2^(nRc_new - nRc_old), which is 1 when the reference stays.
// Acc starts with nRc = kNoRef, a huge finite value, so that the first f is 0 and no inf*0 arises.
constexpr float kNoRef = 1e30f;

template <bool CAREFUL>
__device__ __forceinline__ void accumulate(Acc &a, const float (&z)[16], float c, float gmax, int &err) {
  if (CAREFUL) {
    if (gmax > a.R) {
      if (gmax == CUDART_INF_F) {
        err |= kErrValue;
        return;
      }
      const float nRc = -gmax * c;
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
      a.R = gmax;
      a.nRc = nRc;
    }
  } else {
    const float R = fmaxf(a.R, gmax);  // +inf or NaN logits end up as NaN in the sums and are sorted out later
    const float nRc = -R * c;
    const float d = nRc - a.nRc;       // <= 0
    const float f = ex2f(d);
    a.W0 = f * fmaf(d, a.Z0, a.W0);
    a.W1 = f * fmaf(d, a.Z1, a.W1);
    a.Z0 *= f;
    a.Z1 *= f;
    a.R = R;
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
  int V;
};

// One entry with logit zf and coarse byte cbyte: screen with an fp32 upper bound, then evaluate in fp64.
__device__ __noinline__ void eval_element(const EvalCtx &x, int i, uint32_t cbyte, float zf, Best &b, Smem &sm) {
  if (!(zf > b.zthr2) || zf == CUDART_INF_F) return;  // cannot win even with the largest Gumbel (also NaN, -inf)
  if (cbyte != 255u && !(zf > b.zthr)) return;
  const uint4 fw = philox(x.rk, (uint32_t)i >> 2, x.grow, x.ctr_lo, x.ctr_hi8 | 1u);
  const uint32_t xw = pick_word(fw, i & 3);
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

// A queue entry names one 16-entry group: (group index << 5) | flags.  Flag bits 0-3: the coarse
// bytes of word 0-3 contain 0xFF (may over-report); bit 4: some logit of the group is above the gate.
// Each warp owns a queue; its fill count lives in a warp-uniform register, positions come from a
// ballot, so queueing costs no atomics.  A chunk adds at most 32 entries per group slot, and the
// queue is drained as soon as it holds 32, so kQueueCap >= 31 + 32 * (groups per thread) suffices.
template <int DT>
__device__ __noinline__ void eval_entry(const EvalCtx &x, int entry, Best &b, Smem &sm, bool aligned) {
  const int base = (entry >> 5) << 4;
  // all 16 logits of the group first (independent loads, one memory latency), then the coarse bytes
  float z[16];
  if (aligned && base + 16 <= x.V) {
    if (DT == 0) {
      const float4 *p = reinterpret_cast<const float4 *>(x.row) + (base >> 2);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float4 v = __ldg(p + q);
        z[4 * q] = v.x; z[4 * q + 1] = v.y; z[4 * q + 2] = v.z; z[4 * q + 3] = v.w;
      }
    } else {
      const uint4 *p = reinterpret_cast<const uint4 *>(x.row) + (base >> 3);
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const uint4 v = __ldg(p + q);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          z[8 * q + 2 * j] = __uint_as_float(w[j] << 16);
          z[8 * q + 2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
        }
      }
    }
  } else {
    load_group_guarded<DT>(x.row, base, x.V - base, z);
  }
  const uint4 cw = philox(x.rk, (uint32_t)base >> 4, x.grow, x.ctr_lo, x.ctr_hi8 | 0u);
  const bool over = (entry & 16) != 0;
  // which of the 16 entries need a look (no calls in this loop), then one pass per set bit
  uint32_t todo = 0;
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    const uint32_t cbyte = (pick_word(cw, k >> 2) >> (8 * (k & 3))) & 0xFFu;
    todo |= ((cbyte == 255u || (over && z[k] > b.zthr)) ? 1u : 0u) << k;
  }
  while (todo) {
    const int k = __ffs(todo) - 1;
    todo &= todo - 1;
    const uint32_t cbyte = (pick_word(cw, k >> 2) >> (8 * (k & 3))) & 0xFFu;
    eval_element(x, base + k, cbyte, z[k], b, sm);  // padding beyond the row is -inf and drops out there
  }
}

template <int DT>
__device__ __forceinline__ void drain_queue(const EvalCtx &x, Best &b, Smem &sm, int warp, int lane, int &qn,
                                            bool aligned) {
  __syncwarp();
  for (int e = lane; e < qn; e += 32) eval_entry<DT>(x, sm.queue[warp][e], b, sm, aligned);
  __syncwarp();
  qn = 0;
}

// First step of a segment (warp-uniform): a valid lower bound of the row's best score from the coarse
// byte of each lane's largest entry alone: u >= (c + 2^-33)/256  =>  g >= -ln(ln 256 - ln(c + 2^-33)).
__device__ __forceinline__ void seed_gate(const EvalCtx &x, const float (&z)[16], float gmax, bool have,
                                          const uint4 &cb, Best &b, Smem &sm) {
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
}

// Gate and queue for one group (sampler 0).  qn is the warp's queue fill (warp-uniform).
__device__ __forceinline__ void sample_group(const EvalCtx &x, float gmax, bool have, int e0, const uint4 &cb, Best &b,
                                             Smem &sm, int warp, int lane, int &qn) {
  const uint32_t a0 = any_ff(cb.x), a1 = any_ff(cb.y), a2 = any_ff(cb.z), a3 = any_ff(cb.w);
  const bool over = have && gmax > b.zthr;
  const bool flag = (a0 | a1 | a2 | a3) != 0u || over;
  const uint32_t ballot = __ballot_sync(0xffffffffu, flag);
  if (ballot != 0u) {
    if (flag) {
      const int entry = ((e0 >> 4) << 5) | (over ? 16 : 0) | (a0 ? 1 : 0) | (a1 ? 2 : 0) | (a2 ? 4 : 0) | (a3 ? 8 : 0);
      sm.queue[warp][qn + __popc(ballot & ((1u << lane) - 1u))] = entry;
    }
    qn += __popc(ballot);
  }
}

// A consumer thread's running state for the segment it is working on.
struct LaneState {
  Acc acc;
  Best best;
  int err;
  int qn;  // fill of the warp's candidate queue (warp-uniform)
};

// The common case, kept small so that the streaming loop stays in the instruction cache: a full group
// read from the pipeline stage, finite logits assumed, gate already seeded.
template <int DT, int SAMPLER>
__device__ __forceinline__ void hot_group(const EvalCtx &x, const unsigned char *stage, int slot, int e0, float c,
                                          bool have, Acc &acc, Best &best, int &err, int &qn, Smem &sm, int warp,
                                          int lane) {
  float gmax = -CUDART_INF_F;
  if (have) {
    RawGroup<DT> raw;
    load_raw_smem<DT>(stage, slot, raw);
    float z[16];
    gmax = unpack_group<DT>(raw, z);
    accumulate<false>(acc, z, c, gmax, err);
  }
  if (SAMPLER == 0) {
    uint4 cb = make_uint4(0, 0, 0, 0);
    if (have) cb = philox(x.rk, (uint32_t)e0 >> 4, x.grow, x.ctr_lo, x.ctr_hi8 | 0u);
    sample_group(x, gmax, have, e0, cb, best, sm, warp, lane, qn);
  }
}

// Everything else: the first chunk of a segment (seeds the gate), ragged chunks, rows that do not end on
// a group boundary, greedy rows, rows that cannot use the ring.  One call handles the thread's group
// `slot` of the chunk that starts at entry `cs`.
template <int DT, int SAMPLER>
__device__ __noinline__ void slow_group(const EvalCtx &x, const unsigned char *stage, int slot, int cs, int e_hi,
                                        float c, bool greedy, bool seed, LaneState &st, Smem &sm) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int e0 = cs + slot * kGroup;
  const bool have = e0 < e_hi;
  const bool full = e0 + kGroup <= x.V;
  float z[16];
  float gmax = -CUDART_INF_F;
  if (have && full && stage != nullptr) {
    RawGroup<DT> raw;
    load_raw_smem<DT>(stage, slot, raw);
    gmax = unpack_group<DT>(raw, z);
  } else if (have) {
    gmax = load_group_guarded<DT>(x.row, e0, full ? 16 : x.V - e0, z);
  } else {
#pragma unroll
    for (int k = 0; k < 16; ++k) z[k] = -CUDART_INF_F;
  }
  if (greedy) {
    if (have) {
      int kk = -1;
#pragma unroll
      for (int k = 15; k >= 0; --k) {
        if (z[k] != z[k] || z[k] == CUDART_INF_F) st.err |= kErrValue;
        if (z[k] == gmax) kk = k;
      }
      if (kk >= 0 && gmax > -CUDART_INF_F && (double)gmax > st.best.y) {
        st.best.y = (double)gmax;
        st.best.idx = e0 + kk;
      }
    }
    return;
  }
  if (have) {
    if (full && stage != nullptr)
      accumulate<false>(st.acc, z, c, gmax, st.err);
    else
      accumulate<true>(st.acc, z, c, gmax, st.err);
  }
  if (SAMPLER == 0) {
    uint4 cb = make_uint4(0, 0, 0, 0);
    if (have) cb = philox(x.rk, (uint32_t)e0 >> 4, x.grow, x.ctr_lo, x.ctr_hi8 | 0u);
    if (seed) seed_gate(x, z, gmax, have, cb, st.best, sm);
    sample_group(x, gmax, have, e0, cb, st.best, sm, warp, lane, st.qn);
  }
}

// Seeds the gate of sampler 0 from the thread's first group of a segment (full groups read from the
// stage; other lanes contribute nothing).  Called once per segment, before the streaming loop.
template <int DT>
__device__ __noinline__ void seed_from_stage(const EvalCtx &x, const unsigned char *stage, int slot, int e0,
                                             bool usable, Best &b, Smem &sm) {
  float z[16];
  float gmax = -CUDART_INF_F;
  uint4 cb = make_uint4(0, 0, 0, 0);
  if (usable) {
    RawGroup<DT> raw;
    load_raw_smem<DT>(stage, slot, raw);
    gmax = unpack_group<DT>(raw, z);
    cb = philox(x.rk, (uint32_t)e0 >> 4, x.grow, x.ctr_lo, x.ctr_hi8 | 0u);
  } else {
#pragma unroll
    for (int k = 0; k < 16; ++k) z[k] = -CUDART_INF_F;
  }
  seed_gate(x, z, gmax, usable, cb, b, sm);
}

// ---------------------------------------------------------------------------------------------
// Sampler 1: one Gumbel per block of 256 consecutive entries, applied to the block's log-sum-exp.
// A block is 16 consecutive groups, i.e. one half-warp in one step.  All lanes of a warp keep the
// same reference (the warp-wide largest logit so far), so that the 16 group sums of a block add up
// directly.  Each half-warp parks one block sum per step in one of its lanes; every 16 steps all
// lanes turn their parked block into a score Y_b = L_b + g_b (one Philox call and three MUFU each)
// and keep the three best (fp32).  The finishing warp settles near-ties in fp64 and draws the
// token inside the winning block by inverse CDF.
// ---------------------------------------------------------------------------------------------
struct Top3 {
  float y[3];
  int b[3];
};
__device__ __forceinline__ void top3_reset(Top3 &t) {
  t.y[0] = t.y[1] = t.y[2] = -CUDART_INF_F;
  t.b[0] = t.b[1] = t.b[2] = -1;
}
// order: larger score first, equal scores by lower block index; NaN scores never enter
__device__ __forceinline__ bool top3_before(float y, int b, float y2, int b2) {
  return b2 < 0 || y > y2 || (y == y2 && b < b2);
}
__device__ __forceinline__ void top3_insert(Top3 &t, float y, int b) {
  if (b < 0 || !(y == y)) return;
  if (top3_before(y, b, t.y[0], t.b[0])) {
    t.y[2] = t.y[1]; t.b[2] = t.b[1]; t.y[1] = t.y[0]; t.b[1] = t.b[0]; t.y[0] = y; t.b[0] = b;
  } else if (top3_before(y, b, t.y[1], t.b[1])) {
    t.y[2] = t.y[1]; t.b[2] = t.b[1]; t.y[1] = y; t.b[1] = b;
  } else if (top3_before(y, b, t.y[2], t.b[2])) {
    t.y[2] = y; t.b[2] = b;
  }
}
__device__ __forceinline__ void top3_merge(Top3 &t, const Top3 &o) {
#pragma unroll
  for (int i = 0; i < 3; ++i) top3_insert(t, o.y[i], o.b[i]);
}

struct BlockState {
  Top3 top;
  float S, ref;  // parked block: sum 2^(z c + ref)
  int b;         // its block index
  int it;        // steps taken in this segment (warp-uniform)
};
__device__ __forceinline__ void block_state_reset(BlockState &bs) {
  top3_reset(bs.top);
  bs.S = 0.f; bs.ref = 0.f; bs.b = -1; bs.it = 0;
}

// fp32 Gumbel variate of block b: u = (x + 1/2) 2^-32, g = -ln(-ln u)
__device__ __forceinline__ float block_gumbel_f32(const EvalCtx &x, int b) {
  const uint4 w = philox(x.rk, (uint32_t)b >> 2, x.grow, x.ctr_lo, x.ctr_hi8 | 2u);
  const uint32_t xw = pick_word(w, b & 3);
  float a;  // -ln u
  if (xw >= 0xFE000000u) {
    const float d = ((float)(~xw) + 0.5f) * 0x1p-32f;  // 1 - u < 2^-7: series of -ln(1 - d)
    a = d * fmaf(d, fmaf(d, 0.33333334f, 0.5f), 1.0f);
  } else {
    a = -lg2f(((float)xw + 0.5f) * 0x1p-32f) * kLn2f;
  }
  return -lg2f(a) * kLn2f;
}

__device__ __forceinline__ void block_flush(const EvalCtx &x, BlockState &bs) {
  if (bs.b >= 0 && bs.S > 0.f) {
    const float L = (lg2f(bs.S) - bs.ref) * kLn2f;  // ln sum_i exp(s_i) over the block
    top3_insert(bs.top, L + block_gumbel_f32(x, bs.b), bs.b);
  }
  bs.S = 0.f;
  bs.b = -1;
}

// One step of a warp: every lane brings (at most) one group.  CAREFUL lanes skip -inf / NaN entries.
template <bool CAREFUL>
__device__ __forceinline__ void block_step(const EvalCtx &x, const float (&z)[16], float gmax, bool have, int e0,
                                           float c, Acc &a, BlockState &bs, int &err, int lane) {
  if (CAREFUL && have && gmax == CUDART_INF_F) err |= kErrValue;
  const int mw = __reduce_max_sync(0xffffffffu, enc_float(have ? gmax : -CUDART_INF_F));
  if (mw != enc_neg_inf()) {  // warp-uniform
    const float R = fmaxf(a.R, dec_float(mw));
    const float nRc = -R * c;
    const float d = nRc - a.nRc;
    const float f = ex2f(d);
    a.W0 = f * fmaf(d, a.Z0, a.W0);
    a.W1 = f * fmaf(d, a.Z1, a.W1);
    a.Z0 *= f;
    a.Z1 *= f;
    a.R = R;
    a.nRc = nRc;
    float g0 = 0.f, g1 = 0.f;
    if (have) {
#pragma unroll
      for (int k = 0; k < 16; k += 2) {
        if (CAREFUL) {
          if (z[k] != z[k] || z[k + 1] != z[k + 1]) err |= kErrValue;
          if (z[k] != -CUDART_INF_F && z[k] == z[k]) {
            const float t = fmaf(z[k], c, nRc), e = ex2f(t);
            g0 += e;
            a.W0 = fmaf(e, t, a.W0);
          }
          if (z[k + 1] != -CUDART_INF_F && z[k + 1] == z[k + 1]) {
            const float t = fmaf(z[k + 1], c, nRc), e = ex2f(t);
            g1 += e;
            a.W1 = fmaf(e, t, a.W1);
          }
        } else {
          const float t0 = fmaf(z[k], c, nRc), t1 = fmaf(z[k + 1], c, nRc);
          const float e0_ = ex2f(t0), e1_ = ex2f(t1);
          g0 += e0_;
          g1 += e1_;
          a.W0 = fmaf(e0_, t0, a.W0);
          a.W1 = fmaf(e1_, t1, a.W1);
        }
      }
      a.Z0 += g0;
      a.Z1 += g1;
    }
    float sb = g0 + g1;
#pragma unroll
    for (int o = 1; o < 16; o <<= 1) sb += __shfl_xor_sync(0xffffffffu, sb, o);
    if ((bs.it & 15) == (lane & 15)) {
      bs.S = sb;
      bs.ref = nRc;
      bs.b = e0 >> 8;
    }
  }
  ++bs.it;
  if ((bs.it & 15) == 0) block_flush(x, bs);
}

template <int DT>
__device__ __forceinline__ void hot_group_blocks(const EvalCtx &x, const unsigned char *stage, int slot, int e0,
                                                 float c, Acc &acc, BlockState &bs, int &err, int lane) {
  RawGroup<DT> raw;
  load_raw_smem<DT>(stage, slot, raw);
  float z[16];
  const float gmax = unpack_group<DT>(raw, z);
  block_step<false>(x, z, gmax, true, e0, c, acc, bs, err, lane);
}

struct LaneStateBlocks {
  Acc acc;
  BlockState bs;
  int err;
};

// Out-of-line form: ragged chunks, the row's partial last group, rows that cannot use the ring.
template <int DT>
__device__ __noinline__ void slow_group_blocks(const EvalCtx &x, const unsigned char *stage, int slot, int cs,
                                               int e_hi, float c, LaneStateBlocks &st) {
  const int lane = threadIdx.x & 31;
  const int e0 = cs + slot * kGroup;
  const bool have = e0 < e_hi;
  const bool full = e0 + kGroup <= x.V;
  float z[16];
  float gmax = -CUDART_INF_F;
  if (have && full && stage != nullptr) {
    RawGroup<DT> raw;
    load_raw_smem<DT>(stage, slot, raw);
    gmax = unpack_group<DT>(raw, z);
  } else if (have) {
    gmax = load_group_guarded<DT>(x.row, e0, full ? 16 : x.V - e0, z);
  } else {
#pragma unroll
    for (int k = 0; k < 16; ++k) z[k] = -CUDART_INF_F;
  }
  block_step<true>(x, z, gmax, have, e0, c, st.acc, st.bs, st.err, lane);
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
// Sampler 1, finishing warp: exact (fp64) block scores where fp32 cannot separate the leaders, then the
// in-block inverse-CDF draw.  All 32 lanes take part; a block is 8 consecutive entries per lane.
// ---------------------------------------------------------------------------------------------
struct BlockView {
  double s[8];  // z/tau of the lane's entries (-inf beyond the row)
  double m;     // block maximum
};

template <int DT>
__device__ __forceinline__ void load_block(const char *row, int b, int V, double tau, int lane, BlockView &v) {
  double m = -CUDART_INF;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int i = b * 256 + lane * 8 + k;
    const float z = i < V ? load_elem<DT>(row, i) : -CUDART_INF_F;
    v.s[k] = (double)z / tau;
    m = fmax(m, v.s[k]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
  v.m = m;
}

// Y_b = m_b + ln sum exp(s_i - m_b) + g_b in fp64; -inf for a block without mass.
template <int DT>
__device__ __noinline__ double exact_block_score(const EvalCtx &x, int b, int lane) {
  BlockView v;
  load_block<DT>(x.row, b, x.V, (double)x.tau, lane, v);
  if (v.m == -CUDART_INF) return -CUDART_INF;
  double sum = 0.0;
#pragma unroll
  for (int k = 0; k < 8; ++k)
    if (v.s[k] != -CUDART_INF) sum += exp(v.s[k] - v.m);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  const uint4 w = philox(x.rk, (uint32_t)b >> 2, x.grow, x.ctr_lo, x.ctr_hi8 | 2u);
  const double u = ((double)pick_word(w, b & 3) + 0.5) * 0x1p-32;
  return v.m + log(sum) + (-log(-log(u)));
}

// Token inside block b: first entry whose inclusive prefix sum of exp(s_i - m_b) exceeds v * total.
template <int DT>
__device__ __noinline__ int draw_in_block(const EvalCtx &x, int b, int lane) {
  BlockView v;
  load_block<DT>(x.row, b, x.V, (double)x.tau, lane, v);
  double pre[8];
  double run = 0.0;
  int last_nonzero = -1;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const double w = (v.s[k] != -CUDART_INF) ? exp(v.s[k] - v.m) : 0.0;
    if (w > 0.0) last_nonzero = k;
    run += w;
    pre[k] = run;
  }
  double incl = run;  // inclusive scan of the lane totals
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const double up = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += up;
  }
  const double total = __shfl_sync(0xffffffffu, incl, 31);
  const double before = incl - run;
  const uint4 w3 = philox(x.rk, 0u, x.grow, x.ctr_lo, x.ctr_hi8 | 3u);
  const double t = (((double)w3.x + 0.5) * 0x1p-32) * total;
  int hit = -1;
#pragma unroll
  for (int k = 7; k >= 0; --k)
    if (before + pre[k] > t) hit = k;
  const uint32_t found = __ballot_sync(0xffffffffu, hit >= 0);
  int tok;
  if (found != 0u) {
    const int src = __ffs(found) - 1;
    tok = b * 256 + src * 8 + __shfl_sync(0xffffffffu, hit, src);
  } else {  // rounding left t at or above the total: last entry that carries mass
    const uint32_t any = __ballot_sync(0xffffffffu, last_nonzero >= 0);
    if (any == 0u) return -1;
    const int src = 31 - __clz(any);
    tok = b * 256 + src * 8 + __shfl_sync(0xffffffffu, last_nonzero, src);
  }
  return tok;
}

// Picks the winning block from the three fp32 leaders (exact scores where they are too close) and
// draws the token.  Returns -1 when the row has no block with mass.
template <int DT>
__device__ __noinline__ int sample_in_blocks(const EvalCtx &x, const Top3 &top, int lane) {
  if (top.b[0] < 0) return -1;
  int bstar = top.b[0];
  const float margin = 1e-4f + 2e-5f * fabsf(top.y[0]);
  if (top.b[1] >= 0 && top.y[0] - top.y[1] <= margin) {
    double ybest = -CUDART_INF;
    int bbest = -1;
    if (top.b[2] >= 0 && top.y[0] - top.y[2] <= margin) {
      const int nb = (x.V + 255) / 256;  // more than two contenders: settle all blocks exactly
      for (int b = 0; b < nb; ++b) {
        const double y = exact_block_score<DT>(x, b, lane);
        if (y > ybest) { ybest = y; bbest = b; }
      }
    } else {
      const int lo = top.b[0] < top.b[1] ? top.b[0] : top.b[1], hi = top.b[0] < top.b[1] ? top.b[1] : top.b[0];
      const double y0 = exact_block_score<DT>(x, lo, lane), y1 = exact_block_score<DT>(x, hi, lane);
      bbest = y1 > y0 ? hi : lo;
    }
    if (bbest >= 0) bstar = bbest;
  }
  return draw_in_block<DT>(x, bstar, lane);
}

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
template <int DT, int SAMPLER, bool RING>
__global__ void __launch_bounds__(kThreads, 2) rows_kernel(const __grid_constant__ RowsParams p) {
  extern __shared__ __align__(128) unsigned char ring[];
  __shared__ Smem sm;
  constexpr int kEsize = DT == 0 ? 4 : 2;
  constexpr int kChunkE = kStageBytes / kEsize;                    // entries per stage: 8,192 bf16 / 4,096 fp32
  constexpr int kGPT = kChunkE / (kStreamThreads * kGroup);        // 16-entry groups per consumer thread and stage
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&sm.full[s], 1); mbar_init(&sm.empty[s], kStreamWarps); }
    for (int s = 0; s < kSlots; ++s) { mbar_init(&sm.wfull[s], kStreamWarps); mbar_init(&sm.wfree[s], 1); }
    sm.best64 = 0ull;
    sm.timeout = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  const int full_end = (int)(p.V & ~(int64_t)15);  // entries covered by full groups

  if (warp < kStreamWarps) {
    // ------------------------------------------------------------------ consumers
    Walker wk(p);
    Seg s;
    uint32_t stage = 0, phase = 0;  // ring position
    uint32_t n = 0;                 // segments handed to the finishing warp so far
    while (wk.next(p, s)) {
      const RowInfo ri = classify(p, s.row);
      if (ri.skip) continue;
      const char *row = row_ptr<DT>(p, s.row);
      EvalCtx ex;
      ex.rk = p.round_key; ex.row = row; ex.tau = ri.tau; ex.grow = p.row_base + (uint32_t)s.row;
      ex.ctr_lo = p.ctr_lo; ex.ctr_hi8 = p.ctr_hi8; ex.seg = n + 1; ex.V = (int)p.V;

      Acc acc;
      Best best;
      int err, qn = 0;
      acc.R = -CUDART_INF_F; acc.nRc = kNoRef; acc.Z0 = acc.Z1 = acc.W0 = acc.W1 = 0.f;
      best.y = -CUDART_INF; best.idx = -1;
      set_gate(best, enc_neg_inf(), ri.tau);
      err = 0;
      BlockState bs;
      block_state_reset(bs);

      const int nchunks = s.e_hi > s.e_lo ? (s.e_hi - s.e_lo + kChunkE - 1) / kChunkE : 0;
      const int fast_end = s.e_hi < full_end ? s.e_hi : full_end;  // chunks ending at or before this are full
      if (RING && SAMPLER == 0 && !ri.greedy && nchunks > 0) {
        // seed the gate from the first stage of the segment (the stage is consumed by the loop below)
        mbar_wait(&sm.full[stage], phase, sm);
        const int e0 = s.e_lo + tid * kGroup;
        seed_from_stage<DT>(ex, ring + (size_t)stage * kStageBytes, tid, e0, e0 + kGroup <= fast_end, best, sm);
      }
#pragma unroll 1
      for (int c = 0; c < nchunks; ++c) {
        const int cs = s.e_lo + c * kChunkE;
        const unsigned char *stage_ptr = nullptr;
        if (RING) {
          mbar_wait(&sm.full[stage], phase, sm);
          stage_ptr = ring + (size_t)stage * kStageBytes;
        }
        if (SAMPLER == 0 && !ri.greedy) {
          const int enc = read_best(sm, ex.seg);
          if (enc > best.enc) set_gate(best, enc, ri.tau);
        }
        if (SAMPLER == 1 && !ri.greedy) {
          if (RING && cs + kChunkE <= fast_end) {
#pragma unroll
            for (int j = 0; j < kGPT; ++j) {
              const int slot = j * kStreamThreads + tid;
              hot_group_blocks<DT>(ex, stage_ptr, slot, cs + slot * kGroup, ri.c, acc, bs, err, lane);
            }
          } else {
            LaneStateBlocks st;
            st.acc = acc; st.bs = bs; st.err = err;
#pragma unroll 1
            for (int j = 0; j < kGPT; ++j)
              slow_group_blocks<DT>(ex, stage_ptr, j * kStreamThreads + tid, cs, s.e_hi, ri.c, st);
            acc = st.acc; bs = st.bs; err = st.err;
          }
        } else if (RING && !ri.greedy) {
          const bool all_full = cs + kChunkE <= fast_end;
#pragma unroll
          for (int j = 0; j < kGPT; ++j) {
            const int slot = j * kStreamThreads + tid;
            const int e0 = cs + slot * kGroup;
            hot_group<DT, SAMPLER>(ex, stage_ptr, slot, e0, ri.c, all_full || e0 + kGroup <= fast_end, acc, best, err,
                                   qn, sm, warp, lane);
          }
          // the row's last, partial group (V not a multiple of 16) goes through the out-of-line path
          if (!all_full && fast_end < s.e_hi && fast_end >= cs && fast_end < cs + kChunkE) {
            const int slot = (fast_end - cs) / kGroup;
            if (((slot % kStreamThreads) >> 5) == warp) {
              LaneState st;
              st.acc = acc; st.best = best; st.err = err; st.qn = qn;
              // only the owning lane has the group; the others pass an empty range
              slow_group<DT, SAMPLER>(ex, nullptr, slot, cs, (slot % kStreamThreads) == tid ? s.e_hi : 0, ri.c, false,
                                      false, st, sm);
              acc = st.acc; best = st.best; err = st.err; qn = st.qn;
            }
          }
        } else {
          // the out-of-line path works on a copy, so that the streaming loop keeps its state in registers
          LaneState st;
          st.acc = acc; st.best = best; st.err = err; st.qn = qn;
#pragma unroll 1
          for (int j = 0; j < kGPT; ++j)
            slow_group<DT, SAMPLER>(ex, stage_ptr, j * kStreamThreads + tid, cs, s.e_hi, ri.c, ri.greedy,
                                    !RING && SAMPLER == 0 && !ri.greedy && c == 0 && j == 0, st, sm);
          acc = st.acc; best = st.best; err = st.err; qn = st.qn;
        }
        if (RING) {
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.empty[stage]);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        // All warps of the CTA drain at the same chunks: a drain stalls its warp for microseconds and the
        // ring moves at the pace of the slowest warp, so staggered drains would add up.
        if (SAMPLER == 0 && qn > 0 && ((c & (kDrainEvery - 1)) == kDrainEvery - 1 || qn > kQueueCap - 32 * kGPT))
          drain_queue<DT>(ex, best, sm, warp, lane, qn, RING);
      }
      if (SAMPLER == 0 && qn > 0) drain_queue<DT>(ex, best, sm, warp, lane, qn, RING);
      if (SAMPLER == 1 && !ri.greedy) block_flush(ex, bs);

      if (!ri.greedy) {
        // -inf or NaN logits poison the fast sums: redo this warp's groups with the careful form
        const float zs = acc.Z0 + acc.Z1, ws = acc.W0 + acc.W1;
        const bool bad = !(fabsf(zs) < CUDART_INF_F) || !(fabsf(ws) < CUDART_INF_F);
        if (__any_sync(0xffffffffu, bad)) {
          acc.R = -CUDART_INF_F; acc.nRc = kNoRef; acc.Z0 = acc.Z1 = acc.W0 = acc.W1 = 0.f;
#pragma unroll 1
          for (int c = 0; c < nchunks * kGPT; ++c) {
            const int e0 = s.e_lo + (c * kStreamThreads + tid) * kGroup;
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
        if (SAMPLER == 1) {
          Top3 o2;
#pragma unroll
          for (int i = 0; i < 3; ++i) {
            o2.y[i] = __shfl_xor_sync(0xffffffffu, bs.top.y[i], o);
            o2.b[i] = __shfl_xor_sync(0xffffffffu, bs.top.b[i], o);
          }
          top3_merge(bs.top, o2);
        }
      }
      const uint32_t slot = n % kSlots, use = n / kSlots;
      if (use > 0) mbar_wait(&sm.wfree[slot], (use - 1) & 1u, sm);
      if (lane == 0) {
        WarpPartial &w = sm.wpart[slot][warp];
        w.M = M; w.Z = Z; w.W = W; w.y = y; w.idx = idx; w.err = err;
#pragma unroll
        for (int i = 0; i < 3; ++i) { w.ty[i] = bs.top.y[i]; w.tb[i] = bs.top.b[i]; }
        mbar_arrive(&sm.wfull[slot]);
      }
      ++n;
    }
  } else if (warp == kStreamWarps) {
    // ------------------------------------------------------------------ producer (one thread)
    if (RING && lane == 0) {
      Walker wk(p);
      Seg s;
      uint32_t cc = 0, stage = 0, phase = 1;  // phase: parity of the previous use of the stage
      while (wk.next(p, s)) {
        const RowInfo ri = classify(p, s.row);
        if (ri.skip) continue;
        const char *row = row_ptr<DT>(p, s.row);
        const int nchunks = s.e_hi > s.e_lo ? (s.e_hi - s.e_lo + kChunkE - 1) / kChunkE : 0;
        const int lim = s.e_hi < full_end ? s.e_hi : full_end;
        for (int c = 0; c < nchunks; ++c) {
          if (cc >= (uint32_t)kStages) mbar_wait(&sm.empty[stage], phase, sm, 200u);
          const int cs = s.e_lo + c * kChunkE;
          const int ce = cs + kChunkE < lim ? cs + kChunkE : lim;
          const uint32_t bytes = ce > cs ? (uint32_t)(ce - cs) * kEsize : 0u;
          const bool dead = *reinterpret_cast<volatile int *>(&sm.timeout) != 0;
          if (bytes > 0 && !dead) {
            mbar_arrive_expect_tx(&sm.full[stage], bytes);
            bulk_copy_g2s(ring + (size_t)stage * kStageBytes, row + (size_t)cs * kEsize, bytes, &sm.full[stage]);
          } else {
            mbar_arrive(&sm.full[stage]);
          }
          ++cc;
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
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
      mbar_wait_warp(&sm.wfull[slot], use & 1u, sm, lane);
      double Md = 0.0, Zd = 0.0, Wd = 0.0, yd = -CUDART_INF;
      int id = -1, ed = 0;
      Top3 top;
      top3_reset(top);
      if (lane < kStreamWarps) {
        const WarpPartial &w = sm.wpart[slot][lane];
        Md = w.M; Zd = w.Z; Wd = w.W; yd = w.y; id = w.idx; ed = w.err;
        if (SAMPLER == 1) {
#pragma unroll
          for (int i = 0; i < 3; ++i) { top.y[i] = w.ty[i]; top.b[i] = w.tb[i]; }
        }
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
        if (SAMPLER == 1) {
          Top3 o2;
#pragma unroll
          for (int i = 0; i < 3; ++i) {
            o2.y[i] = __shfl_xor_sync(0xffffffffu, top.y[i], o);
            o2.b[i] = __shfl_xor_sync(0xffffffffu, top.b[i], o);
          }
          top3_merge(top, o2);
        }
      }
      // lane 0 runs the piece protocol and decides whether this CTA finishes the row
      int fin = 0;
      if (lane == 0) {
        if (*reinterpret_cast<volatile int *>(&sm.timeout)) ed |= kErrTimeout;
        if (s.whole) {
          fin = 1;
        } else {
          // A piece of a cut row: store it, announce it; whoever completes the row finishes it.
          Piece *mine = pieces + (size_t)blockIdx.x * 2 + (s.first ? 0 : 1);
          mine->M = Md; mine->Z = Zd; mine->W = Wd; mine->y = yd; mine->idx = id; mine->err = ed;
#pragma unroll
          for (int i = 0; i < 3; ++i) { mine->ty[i] = top.y[i]; mine->tb[i] = top.b[i]; }
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
          if (done && (int)(want & 0xFFFFull) == s.k1 - s.k0 + 1) {  // the last piece of the row
            __threadfence();
            Md = 0.0; Zd = 0.0; Wd = 0.0; yd = -CUDART_INF; id = -1; ed = 0;
            top3_reset(top);
            for (int k = s.k0; k <= s.k1; ++k) {
              // CTA k keeps this row's piece in slot 0 when the row is the first thing it works on
              const bool is_first_seg = first_tile_of(p, k) / p.tiles_per_row == s.row;
              const volatile Piece *q = pieces + (size_t)k * 2 + (is_first_seg ? 0 : 1);
              const double M2 = q->M, Z2 = q->Z, W2 = q->W, y2 = q->y;
              const int i2 = q->idx;
              ed |= q->err;
              merge_stats_d(Md, Zd, Wd, M2, Z2, W2);
              merge_best(yd, id, y2, i2);
              if (SAMPLER == 1) {
#pragma unroll
                for (int i = 0; i < 3; ++i) top3_insert(top, q->ty[i], q->tb[i]);
              }
            }
            fin = 1;
          }
        }
      }
      fin = __shfl_sync(0xffffffffu, fin, 0);
      if (!fin) continue;
      if (SAMPLER == 1 && !ri.greedy) {
        // the whole warp settles the block and draws inside it
#pragma unroll
        for (int i = 0; i < 3; ++i) {
          top.y[i] = __shfl_sync(0xffffffffu, top.y[i], 0);
          top.b[i] = __shfl_sync(0xffffffffu, top.b[i], 0);
        }
        EvalCtx ex;
        ex.rk = p.round_key; ex.row = row_ptr<DT>(p, s.row); ex.tau = ri.tau; ex.grow = p.row_base + (uint32_t)s.row;
        ex.ctr_lo = p.ctr_lo; ex.ctr_hi8 = p.ctr_hi8; ex.seg = 0; ex.V = (int)p.V;
        id = sample_in_blocks<DT>(ex, top, lane);
      }
      if (lane == 0) finish_row<DT>(p, s.row, ri, Md, Zd, Wd, yd, id, ed);
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
    const size_t dyn = RING ? (size_t)kStages * kStageBytes : 0;
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
  const size_t dyn = RING ? (size_t)kStages * kStageBytes : 0;
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
    if (sampler == 1) { E3_DISPATCH(0, 1); }
  } else {
    if (sampler < 0) { E3_DISPATCH(1, -1); }
    if (sampler == 0) { E3_DISPATCH(1, 0); }
    if (sampler == 1) { E3_DISPATCH(1, 1); }
  }
#undef E3_DISPATCH
  return cudaErrorInvalidValue;
}

}  // namespace e3
