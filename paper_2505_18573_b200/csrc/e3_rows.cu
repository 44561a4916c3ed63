// Row-streaming kernel: one pass over the logits of a row gives the softmax statistics
// (App. A: Z(beta), Eq. "entropy" in its shifted form H = ln Z + beta sum p_i Delta_i), the
// log-probability of one token and, for rollouts, a Gumbel-max sample.
//
// Work split.  The [rows, V] matrix is cut into tiles of 512 entries and every CTA of a
// persistent grid (two per SM) takes an equal, contiguous run of tiles, so all CTAs stream the
// same number of bytes whatever the number of rows.  A run covers the tail of one row, some
// whole rows and the head of another.  Whole rows are finished by the CTA itself.  For a row
// that is cut, every CTA holding a piece stores its partial state in the caller's workspace (64-bit
// words tagged with a per-call id), issues a sequentially consistent fence and then looks for the
// row's other pieces: the CTA whose fence comes last finds them all, merges them and writes the
// outputs.  Nobody waits for anybody.  (With a response mask, and when no workspace is given, CTAs
// take whole rows round-robin instead.)
//
// Inside a CTA: one thread issues bulk asynchronous copies (cp.async.bulk, no multicast) of 16 KiB
// into a 4-stage shared-memory ring guarded by mbarriers; eight warps consume the ring, each
// thread 64 contiguous bytes per stage (read in a swizzled vector order that is free of bank
// conflicts); one warp finishes rows (merges the eight warp states, fp64 epilogue, piece protocol)
// so that the consumers never stall on it.  Consumers and the finishing warp look one row ahead for
// the temperature; the copy-issuing thread never needs it.  Every mbarrier wait is bounded: when a
// wait runs out the CTA stops waiting altogether, finishes its fixed sequence of steps on whatever
// data it has and marks its rows invalid.  The kernel is launched with programmatic stream
// serialization: its set-up overlaps the tail of the kernel before it in the stream, and it touches
// global memory only after griddepcontrol.wait.  The finishing warp walks through its own code once
// while the first piece streams (a dry run without side effects), because that code runs last in the
// CTA's life and a first run through cold instructions took several times as long as a warm one.
//
// Numerics.  All lanes of a warp share a reference logit R; each thread keeps the sums Z = sum 2^t,
// W = sum 2^t * t with t = z*c - R*c and c = log2(e)/tau, two entries per instruction (packed fp32).
// The streaming loop never looks for the maximum: R is taken from the first entries of the row piece;
// the sums of a turn stay local until the warp has checked them, and when one leaves the safe range
// (some t above 1..5) the warp moves R up to the largest logit of the current turn, rescales its state
// and repeats the turn.  R therefore stays close to the largest logit seen, which keeps W/Z small and
// the entropy free of cancellation.  A turn is the thread's 64 bytes of a stage in straight-line code
// when the stage lies wholly inside the row and sampler 0's per-group work is not needed, otherwise
// a group of 16 entries.
// -inf logits are clamped to a huge negative finite value on the way in, which gives them weight 0
// without special cases; NaN and +inf end up in a careful out-of-line form that flags the row.
// States merge associatively; the per-row result is formed in fp64:
// H = ln Z - ln2 * W / Z,  ln p_tok = (z_tok*c - M) ln2 - ln Z.
//
// Sampler 0 (one Gumbel per vocabulary entry).  u_i has 8 coarse + 32 fine bits.  An entry can
// only win if its coarse byte is 255 (g_i >= 5.5432) or if z_i/tau exceeds the best score so
// far minus 5.5432; the second condition is tested on the group sum of 2^t, which bounds every
// term from above.  Groups that pass are copied (coarse bytes and logits) into a per-warp queue
// in shared memory with ballot-compacted positions; when 32 are waiting the warp scores them, one
// per lane, in fp32 with a proven error bound, and every thread keeps its three leaders.  The
// finishing warp takes the fp32 leader when it is ahead by more than two error bounds; otherwise
// it evaluates the contenders in fp64 with the expression order of the definition (or looks at the
// whole row again when there are three or more).  The token never depends on the gating or on fp32.
//
// Sampler 1 (one Gumbel per block of 256 entries).  8 (bf16) or 16 (fp32) neighbouring lanes hold
// one block per step; every lane writes its sum to a per-warp scratch in shared memory, and every
// 8 / 16 steps lane j of each group adds up the block of step j and all lanes score their blocks
// together (fp32, three leaders per thread).  The finishing warp settles near-ties of block scores in
// fp64 and draws inside the winning block by inverse CDF (fp32, fp64 near a prefix boundary).
#include "e3_rows.cuh"

#include <limits.h>
#include <math_constants.h>
#include <string.h>

#include <atomic>
#include <chrono>
#include <mutex>

namespace e3 {
namespace {

using u64 = unsigned long long;
using f2 = float2;  // two fp32 values in a register pair

constexpr int kQueueCap = 64;   // candidate groups a warp can hold
constexpr int kDrainAt = 32;    // ... and the fill at which it evaluates them (one per lane)
constexpr int kQueueHdrBytes = kQueueCap * 4;
constexpr int kSlots = 4;  // hand-over slots between the consumer warps and the finishing warp
constexpr uint32_t kSpinLimit = 1u << 23;  // polls before a wait gives up (seconds)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2f = 0.6931471805599453f;
constexpr double kLn2 = 0.6931471805599453094;
// Largest Gumbel value an entry whose coarse byte is below 255 can reach is -ln(-ln(255/256)) = 5.54322...;
// with all 40 bits set the largest value is -ln(-ln(1 - 2^-41)) = 28.41903...  Both rounded up.
constexpr float kGumbelCapCoarse = 5.5433f;
constexpr float kGumbelCapAll = 28.4192f;
// A group of 16 whose sum of 2^t is above this (or NaN) means that the warp's reference logit is stale:
// the warp moves it up to the largest logit of the current turn and repeats the group.  Every entry that
// is added therefore has t <= 5 while the reference is a logit the warp has really seen, so W/Z stays
// small and the entropy ln Z - ln2 W/Z is free of cancellation at the 1e-5 level.
constexpr float kGroupSumMax = 32.f;
// Logits below this (also -inf) enter the streaming form as this value: weight 2^-huge = 0.
constexpr uint32_t kFloorBf16x2 = 0xF180F180u;  // -2^100 twice
constexpr float kFloorF32 = -1.2676506e30f;     // -2^100

enum : int { kErrValue = 1, kErrTimeout = 4 };

template <int DT>
struct Fmt {
  static constexpr int kEsize = DT == 0 ? 4 : 2;
  static constexpr int kLaneE = kLaneBytes / kEsize;          // entries per thread and stage: 16 fp32 / 32 bf16
  static constexpr int kG = kLaneE / kGroup;                  // groups per thread and stage: 1 / 2
  static constexpr int kVG = 4 / kG;                          // 16-byte vectors per group: 4 / 2
  static constexpr int kChunkE = kStageBytes / kEsize;        // entries per stage: 4,096 / 8,192
  static constexpr int kEntryBytes = 16 + kGroup * kEsize;    // queue entry: coarse bytes + logits of one group
  static constexpr int kQueueBytes = kQueueHdrBytes + kQueueCap * kEntryBytes;
  static constexpr int kLB = 256 / kLaneE;                    // lanes that hold one block of sampler 1: 16 / 8
};

// One partial row state.  In the workspace it is kPieceWords 64-bit words, each (tag << 32 | payload):
// the tag depends on the call and on the word, so a reader knows word by word whether what it sees was
// written by this call (64-bit accesses are single-copy atomic); stale or half-written pieces fail the check.
struct Piece {
  float M, Z, W;   // reference (log2 units), sum 2^t, sum 2^t t
  float zf;        // sampler 0: logit of entry tb[0]
  int err;
  int pad;
  float ty[3];     // the three best scores (fp32): sampler 0 entries, sampler 1 blocks; greedy rows: ty[0] = largest logit
  int tb[3];       // ... and their vocabulary / block indices, -1 = none
};
constexpr int kPieceWords = 12;
static_assert(sizeof(Piece) == kPieceWords * 4, "piece payload");
static_assert(kPieceWords * 8 <= kPieceBytes, "piece size");

struct WarpPartial {
  float M, Z, W;
  float zf;
  int err;
  float ty[3];
  int tb[3];
};

struct Smem {
  u64 full[kStages], empty[kStages];  // ring barriers
  u64 wfull[kSlots], wfree[kSlots];   // consumer warps -> finishing warp
  u64 best64;                         // (segment number << 32 | encoded best score) of sampler 0
  WarpPartial wpart[kSlots][kStreamWarps];
  int timeout;                        // set when a bounded wait ran out
};

struct RowInfo {
  float tau, c;
  bool masked;   // masked out: the row's logits are not read and nothing is computed
  bool invalid;  // temperature not usable: the logits still pass through the ring, unused
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

// Running sums of a consumer thread, two fp32 lanes per register pair.
struct Acc {
  float R, nRc;      // reference logit and -R*c; R = -inf, nRc = kNoRef: no reference yet
  f2 Z2, W2;         // Z = sum of both halves of Z2, W likewise
};
// The same state as plain scalars (careful form).
struct AccS {
  float R, nRc, Z, W;
};

// Sampler 0: what a thread knows about the leaders of its row piece.  Scores are fp32 values of
// y_i = z_i/tau + g_i, each within score_slack(y) of the exact value; the three best are kept so that
// the finishing warp can tell whether fp32 separates the winner from the rest.  Greedy rows use
// y[0] / b[0] for the largest logit and its index.
struct Best {
  float y[3];
  int b[3];     // vocabulary indices, -1 = none; order: larger score first, equal scores by lower index
  float zf;     // logit of entry b[0]
  int enc;      // encoded value that is below the row's best score by at least four slacks
  float zthr;   // logit above which an entry may win whatever its coarse byte
  float zthr2;  // logit above which an entry with coarse byte 255 may win
};
// Bound on |fp32 score - exact score|: rounding of 1/tau, of the fused product-sum, of the integer
// conversions and of the two approximate logarithms (worst for coarse byte 254: 1.1e-4).
// k = 1 in normal operation; the audit sampler passes a large k, which sends most rows to the exact path.
__device__ __forceinline__ float score_slack(float y, float k) { return k * (1.7e-4f + 1e-6f * fabsf(y)); }

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
// Packed fp32 arithmetic: both halves of a register pair in one instruction.
__device__ __forceinline__ f2 pack2f(float lo, float hi) { return make_float2(lo, hi); }
__device__ __forceinline__ float sum2(f2 v) { return v.x + v.y; }
__device__ __forceinline__ f2 fma2(f2 a, f2 b, f2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ f2 add2(f2 a, f2 b) { return __fadd2_rn(a, b); }
__device__ __forceinline__ f2 mul2(f2 a, f2 b) { return __fmul2_rn(a, b); }
// max that keeps NaN (a NaN logit must reach the sums)
__device__ __forceinline__ uint32_t floor_bf16x2(uint32_t w) {
  uint32_t d;
  asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(w), "r"(kFloorBf16x2));
  return d;
}
__device__ __forceinline__ uint32_t floor_f32(uint32_t w) {
  float d;
  asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(__uint_as_float(w)), "f"(kFloorF32));
  return __float_as_uint(d);
}
__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(u64 *b, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(u64 *b) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(b)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(u64 *b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(b)), "r"(bytes) : "memory");
}
// One poll (the hardware may park the thread for a short, implementation-defined time).
__device__ __forceinline__ bool mbar_try_wait(u64 *b, uint32_t parity) {
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
__device__ __noinline__ void mbar_wait_slow(u64 *b, uint32_t parity, Smem &sm, unsigned sleep_ns) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(b, parity)) return;
    if (*reinterpret_cast<volatile int *>(&sm.timeout)) return;
    if (sleep_ns) __nanosleep(sleep_ns);
  }
  *reinterpret_cast<volatile int *>(&sm.timeout) = 1;
}
__device__ __forceinline__ void mbar_wait(u64 *b, uint32_t parity, Smem &sm, unsigned sleep_ns = 0) {
  if (!mbar_try_wait(b, parity)) mbar_wait_slow(b, parity, sm, sleep_ns);
}
// Whole-warp wait with a single polling lane (used by the finishing warp, which mostly waits).
__device__ __forceinline__ void mbar_wait_warp(u64 *b, uint32_t parity, Smem &sm, int lane) {
  if (lane == 0) mbar_wait(b, parity, sm, 100u);
  __syncwarp();
}
__device__ __forceinline__ void bulk_copy_g2s(void *dst, const void *src, uint32_t bytes, u64 *bar) {
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
// Non-zero iff some byte of the four words equals 0xFF (a byte is 0xFF iff its complement is zero; the
// borrow of the subtraction can only over-report above a byte that really is 0xFF).
__device__ __forceinline__ uint32_t any_ff4(const uint4 &w) {
  uint32_t r = (0xFEFEFEFEu - w.x) & w.x;
  r |= (0xFEFEFEFEu - w.y) & w.y;
  r |= (0xFEFEFEFEu - w.z) & w.z;
  r |= (0xFEFEFEFEu - w.w) & w.w;
  return r & 0x80808080u;
}

__device__ __forceinline__ int enc_float(float f) {
  int b = __float_as_int(f);
  return b >= 0 ? b : (b ^ 0x7FFFFFFF);
}
__device__ __forceinline__ float dec_float(int e) { return __int_as_float(e >= 0 ? e : (e ^ 0x7FFFFFFF)); }
__device__ __forceinline__ int enc_neg_inf() { return enc_float(-CUDART_INF_F); }

// CTA-wide best score of the segment: 64-bit word (segment number, order-preserving code).
__device__ __forceinline__ void post_best(Smem &sm, uint32_t seg, int enc) {
  atomicMax(&sm.best64, ((u64)seg << 32) | (uint32_t)(enc ^ 0x80000000));
}
__device__ __forceinline__ int read_best(Smem &sm, uint32_t seg) {
  const u64 v = *reinterpret_cast<volatile u64 *>(&sm.best64);
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

// 16 logits from global memory, entries at or beyond `valid` read as -inf.  Returns the largest.
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

// 16 logits that lie contiguously in shared memory (plain order).
template <int DT>
__device__ __forceinline__ void load_group_smem(const unsigned char *src, float (&z)[16]) {
  if (DT == 0) {
    const float4 *p = reinterpret_cast<const float4 *>(src);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float4 v = p[q];
      z[4 * q] = v.x; z[4 * q + 1] = v.y; z[4 * q + 2] = v.z; z[4 * q + 3] = v.w;
    }
  } else {
    const uint4 *p = reinterpret_cast<const uint4 *>(src);
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const uint4 v = p[q];
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        z[8 * q + 2 * j] = __uint_as_float(w[j] << 16);
        z[8 * q + 2 * j + 1] = __uint_as_float(w[j] & 0xFFFF0000u);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Running sums
// ---------------------------------------------------------------------------------------------
constexpr float kNoRef = 1e30f;  // nRc of a state without reference: the first group always overflows into the careful form

__device__ __forceinline__ void acc_reset(Acc &a) {
  a.R = -CUDART_INF_F;
  a.nRc = kNoRef;
  a.Z2 = a.W2 = pack2f(0.f, 0.f);
}
__device__ __forceinline__ AccS to_scalar(const Acc &a) {
  AccS s;
  s.R = a.R;
  s.nRc = a.nRc;
  s.Z = sum2(a.Z2);
  s.W = sum2(a.W2);
  return s;
}
__device__ __forceinline__ void from_scalar(Acc &a, const AccS &s) {
  a.R = s.R;
  a.nRc = s.nRc;
  a.Z2 = pack2f(s.Z, 0.f);
  a.W2 = pack2f(s.W, 0.f);
}

// Careful form for one group: accepts any values.  -inf entries carry no weight, NaN and +inf flag the
// row.  The reference moves up to max(R, ref_floor, largest logit of the group).  Returns the group's
// sum of 2^t under the reference the state has afterwards.
__device__ __forceinline__ float careful_accumulate(AccS &a, const float (&z)[16], float c, float ref_floor, int &err) {
  float gmax = ref_floor;
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    if (z[k] != z[k]) err |= kErrValue;
    gmax = fmaxf(gmax, z[k]);
  }
  if (gmax == CUDART_INF_F) {
    err |= kErrValue;
    return 0.f;
  }
  if (gmax > a.R) {
    const float nRc = -gmax * c;
    if (!(fabsf(nRc) < CUDART_INF_F)) {  // the product left the fp32 range
      err |= kErrValue;
      return 0.f;
    }
    const float d = nRc - a.nRc;
    const float f = a.R == -CUDART_INF_F ? 0.f : ex2f(d);
    if (f == 0.f) {
      a.Z = a.W = 0.f;
    } else {
      a.W = f * fmaf(d, a.Z, a.W);
      a.Z *= f;
    }
    a.R = gmax;
    a.nRc = nRc;
  }
  float g = 0.f;
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    if (z[k] > -CUDART_INF_F) {  // false for NaN as well
      const float t = fmaf(z[k], c, a.nRc), e = ex2f(t);
      g += e;
      a.W = fmaf(e, t, a.W);
    }
  }
  a.Z += g;
  return g;
}

// Largest logit of one group held in raw 16-byte vectors (NaN entries are passed over).
template <int DT>
__device__ __forceinline__ float group_max(const uint4 *v) {
  if (DT == 1) {
    uint32_t m = v[0].x;
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const uint32_t w[4] = {v[q].x, v[q].y, v[q].z, v[q].w};
#pragma unroll
      for (int j = 0; j < 4; ++j) asm("max.bf16x2 %0, %1, %2;" : "=r"(m) : "r"(m), "r"(w[j]));
    }
    return fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u));
  } else {
    float m = -CUDART_INF_F;
#pragma unroll
    for (int q = 0; q < 4; ++q)
      m = fmaxf(fmaxf(m, fmaxf(__uint_as_float(v[q].x), __uint_as_float(v[q].y))),
                fmaxf(__uint_as_float(v[q].z), __uint_as_float(v[q].w)));
    return m;
  }
}

// Streaming form for one group held in raw 16-byte vectors (any order): returns the packed sum of 2^t t in Wg2,
// returns the packed group sum of 2^t in Zg2 and its scalar value.
template <int DT, int NV>
__device__ __forceinline__ float hot_vectors(const uint4 *v, f2 c2, f2 nRc2, f2 &Wg2, f2 &Zg2) {
  f2 Za = pack2f(0.f, 0.f), Zb = pack2f(0.f, 0.f), Wa2 = pack2f(0.f, 0.f), Wb2 = pack2f(0.f, 0.f);
#pragma unroll
  for (int q = 0; q < NV; ++q) {
    const uint32_t w[4] = {v[q].x, v[q].y, v[q].z, v[q].w};
#pragma unroll
    for (int j = 0; j < (DT == 1 ? 4 : 2); ++j) {
      f2 z2;
      if (DT == 1) {
        const uint32_t x = floor_bf16x2(w[j]);
        z2 = pack2f(__uint_as_float(x << 16), __uint_as_float(x & 0xFFFF0000u));
      } else {
        z2 = pack2f(__uint_as_float(floor_f32(w[2 * j])), __uint_as_float(floor_f32(w[2 * j + 1])));
      }
      const f2 t2 = fma2(z2, c2, nRc2);
      const f2 e2 = pack2f(ex2f(t2.x), ex2f(t2.y));
      if (j & 1) {
        Zb = add2(Zb, e2);
        Wb2 = fma2(e2, t2, Wb2);
      } else {
        Za = add2(Za, e2);
        Wa2 = fma2(e2, t2, Wa2);
      }
    }
  }
  Zg2 = add2(Za, Zb);
  Wg2 = add2(Wa2, Wb2);
  return sum2(Zg2);
}

template <int DT>
__device__ __forceinline__ float hot_group(const uint4 *v, f2 c2, f2 nRc2, f2 &Wg2, f2 &Zg2) {
  return hot_vectors<DT, Fmt<DT>::kVG>(v, c2, nRc2, Wg2, Zg2);
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

// The gate of the streaming loop: an entry whose coarse byte is below 255 can only win if
// 2^t_i > 2^((B - 5.5433) log2 e - R c); the group sum of 2^t bounds every term from above.  The slack
// covers the fp32 roundings of t_i, of the threshold and of the approximate 2^x.
__device__ __forceinline__ float gate_threshold(int enc, float nRc) {
  if (enc == enc_neg_inf()) return 0.f;
  const float B = dec_float(enc);
  const float a = (B - kGumbelCapCoarse) * kLog2e;
  const float t = a + nRc - (1e-3f + (fabsf(a) + fabsf(nRc)) * 4e-7f);
  return ex2f(t);  // 0 when far below the range (every group with weight passes), +inf when far above
}

struct EvalCtx {
  const uint32_t *rk;
  const char *row;
  float tau, slack_k;
  uint32_t grow, ctr_lo, ctr_hi8, seg;
  int V;
};

// y_i = z_i/tau + g_i of the definition, in fp64 and in its expression order:
// u = (c + (x + 1/2) 2^-32) / 256 (exact), g = -ln(-ln u).
__device__ __noinline__ double exact_score(float zf, float tau, uint32_t cbyte, uint32_t xw) {
  const double u = ((double)cbyte + ((double)xw + 0.5) * 0x1p-32) / 256.0;
  const double s = (double)zf / (double)tau;
  return s + (-log(-log(u)));
}

// fp32 value of y_i for fine word xw, coarse byte cbyte (within score_slack of the exact value).
__device__ __forceinline__ float score_f32(float zf, float inv_tau, uint32_t cbyte, uint32_t xw) {
  float w;  // -ln u
  if (cbyte == 255u) {
    // 1 - u = (2^32 - x - 1/2) 2^-40 < 2^-8 and -ln u = d + d^2/2 + d^3/3 + ...
    const float d = ((float)(~xw) + 0.5f) * 0x1p-40f;
    w = d * fmaf(d, fmaf(d, 0.33333334f, 0.5f), 1.0f);
  } else {
    const float u = ((float)cbyte + ((float)xw + 0.5f) * 0x1p-32f) * 0.00390625f;
    w = -lg2f(u) * kLn2f;
  }
  return fmaf(zf, inv_tau, -lg2f(w) * kLn2f);
}

__device__ __forceinline__ bool best_before(float y, int i, float y2, int i2) {
  return i2 < 0 || y > y2 || (y == y2 && i < i2);
}
// One entry with logit zf and coarse byte cbyte: cheap bounds first, then its fp32 score.
__device__ __forceinline__ void consider(const uint32_t *rk, uint32_t grow, uint32_t ctr_lo, uint32_t ctr_hi8, float tau,
                                         float inv_tau, float slack_k, uint32_t seg, int i, uint32_t cbyte, float zf,
                                         Best &b, Smem &sm) {
  if (!(zf > b.zthr2) || zf == CUDART_INF_F) return;  // cannot win even with the largest Gumbel (also NaN, -inf)
  if (cbyte != 255u && !(zf > b.zthr)) return;
  const uint4 fw = philox(rk, (uint32_t)i >> 2, grow, ctr_lo, ctr_hi8 | 1u);
  const float y = score_f32(zf, inv_tau, cbyte, pick_word(fw, i & 3));
  if (!(y >= dec_float(b.enc))) return;  // more than two slacks below a score already seen (or NaN)
  if (best_before(y, i, b.y[0], b.b[0])) {
    b.y[2] = b.y[1]; b.b[2] = b.b[1]; b.y[1] = b.y[0]; b.b[1] = b.b[0]; b.y[0] = y; b.b[0] = i;
    b.zf = zf;
    const int enc = enc_float(y - 4.f * score_slack(y, slack_k) - 2e-7f * fabsf(y));
    if (enc > b.enc) {
      set_gate(b, enc, tau);
      post_best(sm, seg, enc);
    }
  } else if (best_before(y, i, b.y[1], b.b[1])) {
    b.y[2] = b.y[1]; b.b[2] = b.b[1]; b.y[1] = y; b.b[1] = i;
  } else if (best_before(y, i, b.y[2], b.b[2])) {
    b.y[2] = y; b.b[2] = i;
  }
}

__device__ __noinline__ void eval_element(const EvalCtx &x, int i, uint32_t cbyte, float zf, Best &b, Smem &sm) {
  consider(x.rk, x.grow, x.ctr_lo, x.ctr_hi8, x.tau, __frcp_rn(x.tau), x.slack_k, x.seg, i, cbyte, zf, b, sm);
}

// A queue entry holds one group: 16 coarse bytes, then its 16 logits in vocabulary order.  Its header
// word is the index of the group's first entry, with bit 0 set when the group passed the sum gate.
template <int DT>
__device__ __forceinline__ float entry_logit(const unsigned char *entry, int k) {
  if (DT == 0) return *reinterpret_cast<const float *>(entry + 16 + 4 * k);
  return __uint_as_float((uint32_t)(*reinterpret_cast<const unsigned short *>(entry + 16 + 2 * k)) << 16);
}

// Evaluates the warp's queued groups, one per lane and round.  Everything it needs comes in registers
// or from the queue in shared memory; only the rare fp64 evaluation is a call.
template <int DT>
__device__ __noinline__ void drain_queue(const uint32_t *rk, uint32_t grow, uint32_t ctr_lo, uint32_t ctr_hi8, float tau,
                                         float slack_k, uint32_t seg, const unsigned char *queue, int qn, Best &best_io,
                                         Smem &sm) {
  const int lane = threadIdx.x & 31;
  Best b = best_io;
  const float inv_tau = __frcp_rn(tau);
  __syncwarp();
  const int *hdrs = reinterpret_cast<const int *>(queue);
#pragma unroll 1
  for (int e = lane; e < qn; e += 32) {
    const unsigned char *entry = queue + kQueueHdrBytes + e * Fmt<DT>::kEntryBytes;
    const int hdr = hdrs[e];
    const uint4 cw = *reinterpret_cast<const uint4 *>(entry);
    // bit k of todo: entry k of the group needs a look (its coarse byte is 255, or its logit is above the gate)
    uint32_t todo = 0;
    {
      const uint32_t w[4] = {cw.x, cw.y, cw.z, cw.w};
#pragma unroll
      for (int q = 0; q < 4; ++q)  // bits 7, 15, 23, 31 -> one nibble
        todo |= (((ff_bytes(w[q]) >> 7) * 0x10204080u) >> 28) << (4 * q);
    }
    if (hdr & 1) {
#pragma unroll 1
      for (int k = 0; k < 16; ++k)
        if (entry_logit<DT>(entry, k) > b.zthr) todo |= 1u << k;
    }
#pragma unroll 1
    while (todo) {
      const int k = __ffs(todo) - 1;
      todo &= todo - 1;
      consider(rk, grow, ctr_lo, ctr_hi8, tau, inv_tau, slack_k, seg, (hdr & ~15) + k, entry[k], entry_logit<DT>(entry, k), b,
               sm);
    }
  }
  __syncwarp();
  best_io = b;
}

// Direct evaluation of one group held as floats (paths that do not stream from the ring).
__device__ __forceinline__ void eval_group_direct(const EvalCtx &x, const float (&z)[16], int e0, int valid, Best &b,
                                                  Smem &sm) {
  if (valid <= 0) return;
  const uint4 cw = philox(x.rk, (uint32_t)e0 >> 4, x.grow, x.ctr_lo, x.ctr_hi8 | 0u);
#pragma unroll 1
  for (int k = 0; k < valid; ++k) {
    const uint32_t cbyte = (pick_word(cw, k >> 2) >> (8 * (k & 3))) & 0xFFu;
    if (cbyte == 255u || z[k] > b.zthr) eval_element(x, e0 + k, cbyte, z[k], b, sm);
  }
}

// ---------------------------------------------------------------------------------------------
// Sampler 1: one Gumbel per block of 256 consecutive entries, applied to the block's log-sum-exp.
// All lanes of a warp keep the same reference, so that the lane sums of a block add up directly.
// kLB neighbouring lanes hold one block per step; every lane parks one block sum per kLB steps and
// then all lanes turn their parked block into a score Y_b = L_b + g_b (one Philox call and three
// MUFU each) and keep the three best (fp32).  The finishing warp settles near-ties in fp64 and
// draws the token inside the winning block by inverse CDF.
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

struct BlockState {
  Top3 top;
  float ref;  // parked block: its lane sums were taken under this reference
  int b;      // its block index, -1: none
};
__device__ __forceinline__ void block_state_reset(BlockState &bs) {
  top3_reset(bs.top);
  bs.ref = 0.f; bs.b = -1;
}

// fp32 Gumbel variate of block b: u = (x + 1/2) 2^-32, g = -ln(-ln u)
__device__ __forceinline__ float block_gumbel_f32(const uint32_t *rk, uint32_t grow, uint32_t ctr_lo, uint32_t ctr_hi8,
                                                  int b) {
  const uint4 w = philox(rk, (uint32_t)b >> 2, grow, ctr_lo, ctr_hi8 | 2u);
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

// fp32 score of a block: ln sum_i exp(s_i) + g_b, from S = sum 2^(z c + ref).  Out of line (scalars in,
// scalar out) so that the streaming loop stays short and its state stays in registers.
__device__ __noinline__ float block_score(const uint32_t *rk, uint32_t grow, uint32_t ctr_lo, uint32_t ctr_hi8, float S,
                                          float ref, int b) {
  return (lg2f(S) - ref) * kLn2f + block_gumbel_f32(rk, grow, ctr_lo, ctr_hi8, b);
}

// Adds up the parked blocks of the warp (lane j of each group of kLB lanes owns the block of step j of
// the current round; its lane sums sit in the warp's scratch) and enters their scores in the lane's list.
template <int DT>
__device__ __forceinline__ void block_flush(const uint32_t *rk, uint32_t grow, uint32_t ctr_lo, uint32_t ctr_hi8,
                                            BlockState &bs, const float *scratch, int lane) {
  constexpr int kLB = Fmt<DT>::kLB;
  __syncwarp();
  // row j of the scratch is rotated by 8 j columns, which spreads the lanes' reads over the banks
  const int j = lane & (kLB - 1), col0 = (lane & ~(kLB - 1)) + 8 * j;
  float S = 0.f;
#pragma unroll
  for (int i = 0; i < kLB / 4; ++i) {
    const float4 v = *reinterpret_cast<const float4 *>(scratch + j * 32 + ((col0 + 4 * i) & 31));
    S += (v.x + v.y) + (v.z + v.w);
  }
  __syncwarp();  // the scratch is written again in the next step
  if (bs.b >= 0 && S > 0.f) top3_insert(bs.top, block_score(rk, grow, ctr_lo, ctr_hi8, S, bs.ref, bs.b), bs.b);
  bs.b = -1;
}

// Step `it` of a warp in its row piece: every lane brings the sum of 2^t over its entries of this step
// (all lanes under the reference nRc), which lie in block `b`; kLB neighbouring lanes share a block.
// The lane sums go to the warp's scratch in shared memory and are added up only every kLB steps: one
// read instead of a chain of shuffles at the end of every step.
template <int DT>
__device__ __forceinline__ void block_step(float zlane, int b, float nRc, const uint32_t *rk, uint32_t grow,
                                           uint32_t ctr_lo, uint32_t ctr_hi8, BlockState &bs, float *scratch,
                                           int lane, int it) {
  constexpr int kLB = Fmt<DT>::kLB;
  const int j = it & (kLB - 1);
  scratch[j * 32 + ((lane + 8 * j) & 31)] = zlane;
  if (j == (lane & (kLB - 1))) {
    bs.ref = nRc;
    bs.b = b;
  }
  if (j == kLB - 1) block_flush<DT>(rk, grow, ctr_lo, ctr_hi8, bs, scratch, lane);
}

// ---------------------------------------------------------------------------------------------
// Out-of-line forms of one consumer step
// ---------------------------------------------------------------------------------------------
struct StepIO {
  Acc acc;
  float Zg[2];   // per group of the thread (vocabulary order): sum of 2^t under the final reference
  float Zextra;  // a sum formed before this call, to be carried to the final reference
  int err;
};

// Redo of the thread's groups of one stage in the careful form (a group sum left the safe range).
// `have` bit g: group g of the thread is part of the row piece.  UNIFORM: all lanes of the warp are
// here and must end with one common reference.
template <int DT, bool UNIFORM>
__device__ __noinline__ void redo_step(StepIO &io, const unsigned char *lane_data, int have, float c) {
  constexpr int kG = Fmt<DT>::kG;
  AccS a = to_scalar(io.acc);
  const float nRc_old = a.nRc;
  float z[kG][16];
  float gm = -CUDART_INF_F;
#pragma unroll
  for (int g = 0; g < kG; ++g) {
    if (have & (1 << g)) {
      load_group_smem<DT>(lane_data + g * kGroup * Fmt<DT>::kEsize, z[g]);
#pragma unroll
      for (int k = 0; k < 16; ++k) gm = fmaxf(gm, z[g][k]);
    } else {
#pragma unroll
      for (int k = 0; k < 16; ++k) z[g][k] = -CUDART_INF_F;
    }
  }
  float ref_floor = -CUDART_INF_F;
  if (UNIFORM) {
    if (gm == CUDART_INF_F) gm = -CUDART_INF_F;  // flagged below; must not become the reference
    ref_floor = dec_float(__reduce_max_sync(0xffffffffu, enc_float(gm)));
  }
  // settle the reference first, so that all group sums of this call refer to the same one
  float top = ref_floor;
#pragma unroll
  for (int g = 0; g < kG; ++g)
#pragma unroll
    for (int k = 0; k < 16; ++k) top = fmaxf(top, z[g][k]);
  if (top == CUDART_INF_F) top = ref_floor;
#pragma unroll
  for (int g = 0; g < kG; ++g) io.Zg[g] = careful_accumulate(a, z[g], c, top, io.err);
  if (a.nRc != nRc_old) io.Zextra = nRc_old == kNoRef ? 0.f : io.Zextra * ex2f(a.nRc - nRc_old);
  from_scalar(io.acc, a);
}

struct SlowIO {
  Acc acc;
  Best best;
  float zsum;  // sum of 2^t over the entries handled by this call, under the final reference
  int err;
};

// Up to kG groups of the thread read from global memory with guards: entries [e0, e_hi) of the row, at
// most kLaneE of them.  Used for the last, partial group of a row, for rows that cannot use the ring
// and for whatever else does not fit the streaming form.  SAMPLER 0 evaluates candidates directly.
template <int DT, int SAMPLER, bool UNIFORM>
__device__ __noinline__ void slow_groups(SlowIO &io, const EvalCtx &x, int e0, int e_hi, float c, Smem &sm) {
  constexpr int kG = Fmt<DT>::kG;
  AccS a = to_scalar(io.acc);
  float z[kG][16];
  int valid[kG];
  float gm = -CUDART_INF_F;
#pragma unroll
  for (int g = 0; g < kG; ++g) {
    const int g0 = e0 + g * kGroup;
    valid[g] = e_hi - g0 < 0 ? 0 : (e_hi - g0 > kGroup ? kGroup : e_hi - g0);
    if (valid[g] > 0) {
      gm = fmaxf(gm, load_group_guarded<DT>(x.row, g0, valid[g], z[g]));
    } else {
#pragma unroll
      for (int k = 0; k < 16; ++k) z[g][k] = -CUDART_INF_F;
    }
  }
  float top = gm;
  if (UNIFORM) {
    if (gm == CUDART_INF_F) gm = -CUDART_INF_F;
    top = dec_float(__reduce_max_sync(0xffffffffu, enc_float(gm)));
  }
  if (top == CUDART_INF_F) top = -CUDART_INF_F;
  float zs = 0.f;
#pragma unroll
  for (int g = 0; g < kG; ++g) {
    if (valid[g] > 0 || UNIFORM) zs += careful_accumulate(a, z[g], c, top, io.err);
    if (SAMPLER == 0) eval_group_direct(x, z[g], e0 + g * kGroup, valid[g], io.best, sm);
  }
  io.zsum = zs;
  from_scalar(io.acc, a);
}

// Greedy rows (tau = 0): largest logit, lowest index; NaN and +inf flag the row.  Full groups below
// `lim` are read from the thread's 64 bytes of the pipeline stage (when there is one), the rest from
// global memory with guards.
template <int DT>
__device__ __noinline__ void greedy_groups(SlowIO &io, const char *row, const unsigned char *lane_data, int e0, int lim,
                                           int e_hi) {
  constexpr int kG = Fmt<DT>::kG;
#pragma unroll 1
  for (int g = 0; g < kG; ++g) {
    const int g0 = e0 + g * kGroup;
    const int valid = e_hi - g0 < 0 ? 0 : (e_hi - g0 > kGroup ? kGroup : e_hi - g0);
    if (valid <= 0) continue;
    float z[16];
    float gmax = -CUDART_INF_F;
    if (lane_data != nullptr && g0 + kGroup <= lim) {
      load_group_smem<DT>(lane_data + g * kGroup * Fmt<DT>::kEsize, z);
#pragma unroll
      for (int k = 0; k < 16; ++k) gmax = fmaxf(gmax, z[k]);
    } else {
      gmax = load_group_guarded<DT>(row, g0, valid, z);
    }
    int kk = -1;
#pragma unroll
    for (int k = 15; k >= 0; --k) {
      if (z[k] != z[k] || z[k] == CUDART_INF_F) io.err |= kErrValue;
      if (z[k] == gmax) kk = k;
    }
    if (kk >= 0 && gmax > -CUDART_INF_F && (io.best.b[0] < 0 || gmax > io.best.y[0])) {
      io.best.y[0] = gmax;
      io.best.b[0] = g0 + kk;
    }
  }
}

// The reference part of seed_piece alone, in line (no per-entry work): the largest finite logit among the
// first groups of the warp's lanes, -inf if there is none.
template <int DT>
__device__ __forceinline__ float seed_reference(const unsigned char *lane_data, int e_lane, int lim) {
  float gmax = -CUDART_INF_F;
  if (e_lane + kGroup <= lim) {
    uint4 v[Fmt<DT>::kVG];
#pragma unroll
    for (int i = 0; i < Fmt<DT>::kVG; ++i) v[i] = reinterpret_cast<const uint4 *>(lane_data)[i];
    gmax = group_max<DT>(v);
  }
  if (!(gmax < CUDART_INF_F)) gmax = -CUDART_INF_F;
  return dec_float(__reduce_max_sync(0xffffffffu, enc_float(gmax)));
}

struct SeedIO {
  float R0;  // warp-wide reference, -inf = none found
  Best best;
};

// First stage of a row piece: a common reference for the warp from each lane's first group, and for
// sampler 0 a valid lower bound of the piece's best score from the coarse byte of each lane's largest
// entry alone: u >= (c + 2^-33)/256  =>  g >= -ln(ln 256 - ln(c + 2^-33)).
template <int DT, int SAMPLER>
__device__ __noinline__ void seed_piece(SeedIO &io, const EvalCtx &x, const unsigned char *lane_data, int e_lane,
                                        int lim, Smem &sm) {
  const bool have = e_lane + kGroup <= lim;
  float z[16];
  float gmax = -CUDART_INF_F;
  if (have) {
    load_group_smem<DT>(lane_data, z);
#pragma unroll
    for (int k = 0; k < 16; ++k) gmax = fmaxf(gmax, z[k]);
  }
  const bool usable = have && gmax > -CUDART_INF_F && gmax < CUDART_INF_F;
  io.R0 = dec_float(__reduce_max_sync(0xffffffffu, enc_float(usable ? gmax : -CUDART_INF_F)));
  if (SAMPLER == 0) {
    float ylo = -CUDART_INF_F;
    if (usable) {
      const uint4 cb = philox(x.rk, (uint32_t)e_lane >> 4, x.grow, x.ctr_lo, x.ctr_hi8 | 0u);
      uint32_t cbyte = 0;
#pragma unroll
      for (int k = 15; k >= 0; --k)
        if (z[k] == gmax) cbyte = (pick_word(cb, k >> 2) >> (8 * (k & 3))) & 0xFFu;
      const float neg_ln_u = (8.0f - lg2f((float)cbyte + 0x1p-33f)) * kLn2f;
      const float glo = -lg2f(neg_ln_u) * kLn2f;
      const float sf = gmax / x.tau;
      ylo = sf - fabsf(sf) * 8e-6f + glo - 4e-3f;  // also five score slacks below the entry's score
    }
    int enc = __reduce_max_sync(0xffffffffu, enc_float(ylo));
    if ((threadIdx.x & 31) == 0 && enc > enc_neg_inf()) post_best(sm, x.seg, enc);
    const int cta = read_best(sm, x.seg);
    enc = enc > cta ? enc : cta;
    if (enc > io.best.enc) set_gate(io.best, enc, x.tau);
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

__device__ __forceinline__ uint32_t piece_tag(u64 call_id, int j) {
  return (uint32_t)((((call_id << 4) | (u64)j) * 0x9E3779B97F4A7C15ull) >> 32);
}
__device__ __forceinline__ void piece_store(u64 *dst, u64 call_id, const Piece &pc) {
  uint32_t w[kPieceWords];
  memcpy(w, &pc, sizeof(Piece));
#pragma unroll
  for (int j = 0; j < kPieceWords; ++j) {
    const u64 v = ((u64)piece_tag(call_id, j) << 32) | w[j];
    asm volatile("st.relaxed.gpu.global.b64 [%0], %1;" ::"l"(dst + j), "l"(v) : "memory");
  }
}
// False when some word does not carry this call's tag.
__device__ __forceinline__ bool piece_load(const u64 *src, u64 call_id, Piece &pc) {
  u64 v[kPieceWords];
#pragma unroll
  for (int j = 0; j < kPieceWords; ++j)
    asm volatile("ld.relaxed.gpu.global.b64 %0, [%1];" : "=l"(v[j]) : "l"(src + j) : "memory");
  uint32_t w[kPieceWords];
  bool ok = true;
#pragma unroll
  for (int j = 0; j < kPieceWords; ++j) {
    ok &= (uint32_t)(v[j] >> 32) == piece_tag(call_id, j);
    w[j] = (uint32_t)v[j];
  }
  memcpy(&pc, w, sizeof(Piece));
  return ok;
}

// Merges the partial states held by the 32 lanes of a warp; every lane ends with the result.  A lane
// without weight (Z = 0) or with an empty list takes no part.  Written with warp-wide reductions so
// that the chain of dependent instructions stays short: this runs at the end of every row piece, when
// nothing else can hide it.  The order of all sums is fixed by lane numbers.  with_top: the lists of
// leaders (sampler 0 entries, sampler 1 blocks, greedy maxima) are merged too; pc.zf follows top.b[0].
__device__ __forceinline__ void warp_merge(Piece &pc, Top3 &top, bool with_top) {
  constexpr unsigned kAll = 0xffffffffu;
  // softmax sums: move every lane to the largest reference, then add
  const bool has = pc.Z > 0.f;
  const int em = __reduce_max_sync(kAll, has ? enc_float(pc.M) : enc_neg_inf());
  float Mw = 0.f, Zs = 0.f, Ws = 0.f;
  if (em != enc_neg_inf()) {
    Mw = dec_float(em);
    if (has) {
      const float d = pc.M - Mw, a = ex2f(d);
      Zs = a * pc.Z;
      Ws = a * fmaf(d, pc.Z, pc.W);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      Zs += __shfl_xor_sync(kAll, Zs, o);
      Ws += __shfl_xor_sync(kAll, Ws, o);
    }
  }
  pc.M = Mw; pc.Z = Zs; pc.W = Ws;
  pc.err = __reduce_or_sync(kAll, pc.err);
  if (with_top) {
    // three rounds of "take the best head": larger score first, equal scores by lower index
    Top3 out;
    top3_reset(out);
    int pos = 0;
#pragma unroll
    for (int r = 0; r < 3; ++r) {
      const float hy = pos == 0 ? top.y[0] : (pos == 1 ? top.y[1] : top.y[2]);
      const int hb = pos >= 3 ? -1 : (pos == 0 ? top.b[0] : (pos == 1 ? top.b[1] : top.b[2]));
      const int e = hb >= 0 ? enc_float(hy) : INT_MIN;
      const int emax = __reduce_max_sync(kAll, e);
      if (emax != INT_MIN) {
        const bool c2 = hb >= 0 && e == emax;
        const int bmin = __reduce_min_sync(kAll, c2 ? hb : INT_MAX);
        out.y[r] = dec_float(emax);
        out.b[r] = bmin;
        const bool mine = c2 && hb == bmin;
        if (r == 0) pc.zf = __shfl_sync(kAll, pc.zf, __ffs(__ballot_sync(kAll, mine)) - 1);
        if (mine) ++pos;
      }
    }
    top = out;
  }
}

// Largest y over the lanes, then lowest index (lanes with idx < 0 take no part); all lanes get the winner.
__device__ __forceinline__ void warp_argmax_double(double &y, int &idx, float &zf) {
  constexpr unsigned kAll = 0xffffffffu;
  const long long bits = __double_as_longlong(y);
  const long long code = bits >= 0 ? bits : (bits ^ 0x7FFFFFFFFFFFFFFFll);  // order-preserving
  bool cand = idx >= 0 && y == y;
  const int hi = cand ? (int)(code >> 32) : INT_MIN;
  const int hmax = __reduce_max_sync(kAll, hi);
  if (hmax == INT_MIN) {
    idx = -1;
    return;
  }
  cand = cand && hi == hmax;
  const unsigned lo = cand ? (unsigned)code : 0u;
  const unsigned lmax = __reduce_max_sync(kAll, lo);
  cand = cand && lo == lmax;
  const int imin = __reduce_min_sync(kAll, cand ? idx : INT_MAX);
  const int src = __ffs(__ballot_sync(kAll, cand && idx == imin)) - 1;
  y = __shfl_sync(kAll, y, src);
  zf = __shfl_sync(kAll, zf, src);
  idx = imin;
}

// ---------------------------------------------------------------------------------------------
// Work split
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ int64_t quot(const RowsParams &p, int64_t a, int64_t b) {
  return p.narrow ? (int64_t)((uint32_t)a / (uint32_t)b) : a / b;
}
__device__ __forceinline__ int64_t first_tile_of(const RowsParams &p, int64_t b) {
  return b * p.tiles_q + (b < p.tiles_r ? b : p.tiles_r);
}
__device__ __forceinline__ int cta_of_tile(const RowsParams &p, int64_t t) {
  const int64_t big = p.tiles_r * (p.tiles_q + 1);
  return (int)(t < big ? quot(p, t, p.tiles_q + 1) : p.tiles_r + quot(p, t - big, p.tiles_q));
}

// Hands out the CTA's row pieces one after the other.  The only state is a count of what has been
// handed out; everything else is recomputed from the launch parameters (registers are scarce here).
struct Walker {
  int rel;  // tiles of the CTA's run handed out so far (interleaved: rows handed out)
  __device__ Walker() : rel(0) {}
  __device__ static int64_t run_length(const RowsParams &p) { return p.tiles_q + ((int64_t)blockIdx.x < p.tiles_r ? 1 : 0); }
  // Row of the first piece, -1 when the CTA has nothing to do.
  __device__ static int64_t first_row(const RowsParams &p) {
    if (p.interleaved) return (int64_t)blockIdx.x < p.rows ? (int64_t)blockIdx.x : -1;
    return run_length(p) > 0 ? quot(p, first_tile_of(p, blockIdx.x), p.tiles_per_row) : -1;
  }
  // Row of the piece after `cur` (the piece handed out last), -1 when there is none.
  __device__ int64_t row_after(const RowsParams &p, const Seg &cur) const {
    if (p.interleaved) return cur.row + gridDim.x < p.rows ? cur.row + gridDim.x : -1;
    return rel < run_length(p) ? cur.row + 1 : -1;
  }
  // with_range: also work out which CTAs hold the row's first and last tile (only the finishing warp asks)
  __device__ bool next(const RowsParams &p, Seg &s, bool with_range) {
    if (p.interleaved) {
      const int64_t row = (int64_t)blockIdx.x + (int64_t)rel * gridDim.x;
      if (row >= p.rows) return false;
      s.row = row; s.e_lo = 0; s.e_hi = (int)p.V; s.whole = true; s.starts = true; s.first = rel == 0; s.k0 = s.k1 = 0;
      ++rel;
      return true;
    }
    const int64_t len = run_length(p);
    if (rel >= len) return false;
    // only the CTA's first piece can start inside a row: every later one starts the row after `s.row`
    // (s still holds the piece handed out before)
    int64_t row, tin;
    if (rel == 0) {
      const int64_t t = first_tile_of(p, blockIdx.x);
      row = quot(p, t, p.tiles_per_row);
      tin = t - row * p.tiles_per_row;
    } else {
      row = s.row + 1;
      tin = 0;
    }
    const int64_t n = p.tiles_per_row - tin < len - rel ? p.tiles_per_row - tin : len - rel;
    const int64_t lo = tin * kTile, hi = (tin + n) * kTile;
    s.row = row;
    s.e_lo = (int)(lo < p.V ? lo : p.V);
    s.e_hi = (int)(hi < p.V ? hi : p.V);
    s.starts = tin == 0;
    s.whole = tin == 0 && n == p.tiles_per_row;
    s.first = rel == 0;
    s.k0 = s.k1 = 0;
    if (!s.whole && with_range) {
      s.k0 = cta_of_tile(p, row * p.tiles_per_row);
      s.k1 = cta_of_tile(p, (row + 1) * p.tiles_per_row - 1);
    }
    rel += (int)n;
    return true;
  }
};

// Walks the CTA's row pieces and loads temperature and mask of the piece after the current one, so
// that nobody waits for them when that piece starts.  The copy-issuing thread passes with_tau = false:
// it only needs the mask, and must not wait for anything before its first copy.
struct SegIter {
  Walker wk;
  float tau_next;
  bool masked_next;
  bool with_tau, with_range;
  __device__ SegIter(const RowsParams &p, bool with_tau_, bool with_range_ = false)
      : with_tau(with_tau_), with_range(with_range_) {
    prefetch(p, Walker::first_row(p));
  }
  __device__ void prefetch(const RowsParams &p, int64_t row) {
    tau_next = p.temp_scalar;
    masked_next = false;
    if (row >= 0) {
      if (with_tau && p.temps) tau_next = __ldg(p.temps + row);
      masked_next = p.mode != kModeSample && p.mask && __ldg(p.mask + row) == 0;
    }
  }
  __device__ bool next(const RowsParams &p, Seg &s, RowInfo &r) {
    if (!wk.next(p, s, with_range)) return false;
    r.tau = tau_next;
    r.masked = masked_next;
    prefetch(p, wk.row_after(p, s));
    r.greedy = p.mode == kModeSample && r.tau == 0.f;
    r.invalid = !r.masked && !r.greedy && !(r.tau > 0.f && r.tau < CUDART_INF_F);
    r.c = r.greedy || r.masked || r.invalid ? 0.f : __fdiv_rn(kLog2e, r.tau);
    return true;
  }
};

template <int DT>
__device__ __forceinline__ const char *row_ptr(const RowsParams &p, int64_t row) {
  return reinterpret_cast<const char *>(p.logits) + (size_t)row * (size_t)p.row_stride * (DT == 0 ? 4 : 2);
}

// ---------------------------------------------------------------------------------------------
// Row epilogue (one thread, fp64).  zt: logit of the token whose log-probability is wanted.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void finish_row(const RowsParams &p, int64_t row, const RowInfo &ri, float Mf, float Zf,
                                           float Wf, int idx, int err, bool have_zt, float zt, bool store) {
  const double M = Mf, Z = Zf, W = Wf;
  const bool sample = p.mode == kModeSample;
  int tok = -1;
  float logp = CUDART_NAN_F, ent = CUDART_NAN_F;
  if (ri.greedy) {
    if (err == 0 && idx >= 0) { tok = idx; logp = 0.f; ent = 0.f; }
  } else if (err == 0 && Z > 0.0) {
    const double lnZ = log(Z);
    ent = (float)(lnZ - kLn2 * (W / Z));
    if (sample) tok = idx;
    if (have_zt) logp = (float)(((double)zt * (double)ri.c - M) * kLn2 - lnZ);
  }
  if (!store) return;
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
// Exact form (fp64, the definition's expression order).
template <int DT>
__device__ __noinline__ int draw_in_block_exact(const EvalCtx &x, int b, int lane) {
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

// The same draw in fp32.  The prefix sums are good to about 3e-6 of the block sum (entries that matter
// have |t| < 25, so the rounding of t costs 2e-6 relative, `ex2` 2e-7, the 13 additions 8e-7); when the
// threshold comes closer than ten times that to a prefix boundary the exact form decides.
// z_tok: logit of the token.
template <int DT>
__device__ __noinline__ int draw_in_block(const EvalCtx &x, int b, int lane, float &z_tok) {
  float z[8];
  float m = -CUDART_INF_F;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int i = b * 256 + lane * 8 + k;
    z[k] = i < x.V ? load_elem<DT>(x.row, i) : -CUDART_INF_F;
    m = fmaxf(m, z[k]);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  int tok = -1;
  bool exact = !(m > -CUDART_INF_F && m < CUDART_INF_F);
  if (!exact) {
    const float c = __fdiv_rn(kLog2e, x.tau);
    float pre[8];
    float run = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      run += z[k] > -CUDART_INF_F ? ex2f((z[k] - m) * c) : 0.f;
      pre[k] = run;
    }
    float incl = run;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const float up = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += up;
    }
    const float total = __shfl_sync(0xffffffffu, incl, 31);
    const float before = incl - run;
    const uint4 w3 = philox(x.rk, 0u, x.grow, x.ctr_lo, x.ctr_hi8 | 3u);
    const float t = (float)((((double)w3.x + 0.5) * 0x1p-32) * (double)total);
    int hit = -1;
    float gap = CUDART_INF_F;
#pragma unroll
    for (int k = 7; k >= 0; --k) {
      const float pk = before + pre[k];
      if (pk > t) hit = k;
      gap = fminf(gap, fabsf(pk - t));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) gap = fminf(gap, __shfl_xor_sync(0xffffffffu, gap, o));
    const uint32_t found = __ballot_sync(0xffffffffu, hit >= 0);
    exact = !(gap > 3e-5f * total) || found == 0u || !(total > 0.f) || !(total < CUDART_INF_F);
    if (!exact) {
      const int src = __ffs(found) - 1;
      const int k = __shfl_sync(0xffffffffu, hit, src);
      tok = b * 256 + src * 8 + k;
      float zk = z[0];
#pragma unroll
      for (int j = 1; j < 8; ++j) zk = k == j ? z[j] : zk;
      z_tok = __shfl_sync(0xffffffffu, zk, src);
    }
  }
  if (exact) {
    tok = draw_in_block_exact<DT>(x, b, lane);
    z_tok = tok >= 0 ? load_elem<DT>(x.row, tok) : 0.f;
  }
  return tok;
}

// Picks the winning block from the three fp32 leaders (exact scores where they are too close) and
// draws the token.  Returns -1 when the row has no block with mass.
template <int DT>
__device__ __noinline__ int sample_in_blocks(const EvalCtx &x, const Top3 &top, int lane, float &z_tok) {
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
  return draw_in_block<DT>(x, bstar, lane, z_tok);
}

// ---------------------------------------------------------------------------------------------
// Sampler 0, finishing warp: the leaders of the row are closer than fp32 can tell apart.  Every entry
// whose fp32 score is within slack2 of the best may be the true winner; they are evaluated in fp64.
// With one or two such entries they are in `top`; with three, others may exist and the whole row is
// looked at again (fp32 scores for all entries, fp64 for those near the top).
// ---------------------------------------------------------------------------------------------
template <int DT>
__device__ __noinline__ int settle_exact(const EvalCtx &x, const Top3 &top, float slack2, int lane, float &z_tok) {
  double ybest = -CUDART_INF;
  int ibest = -1;
  float zbest = 0.f;
  const bool rescan = top.b[2] >= 0 && !(top.y[0] - top.y[2] > slack2);
  if (!rescan) {
    const int i = lane == 0 ? top.b[0] : (lane == 1 ? top.b[1] : -1);
    if (i >= 0) {
      const float z = load_elem<DT>(x.row, i);
      const uint4 cw = philox(x.rk, (uint32_t)i >> 4, x.grow, x.ctr_lo, x.ctr_hi8 | 0u);
      const uint32_t cbyte = (pick_word(cw, (i & 15) >> 2) >> (8 * (i & 3))) & 0xFFu;
      const uint4 fw = philox(x.rk, (uint32_t)i >> 2, x.grow, x.ctr_lo, x.ctr_hi8 | 1u);
      ybest = exact_score(z, x.tau, cbyte, pick_word(fw, i & 3));
      ibest = i;
      zbest = z;
    }
  } else {
    const float inv_tau = __frcp_rn(x.tau);
    const float floor_y = top.y[0] - slack2;
#pragma unroll 1
    for (int q0 = lane * 4; q0 < x.V; q0 += 128) {  // four entries (one fine call) per lane and round
      const uint4 cw = philox(x.rk, (uint32_t)q0 >> 4, x.grow, x.ctr_lo, x.ctr_hi8 | 0u);
      const uint32_t cword = pick_word(cw, (q0 & 15) >> 2);
      const uint4 fw = philox(x.rk, (uint32_t)q0 >> 2, x.grow, x.ctr_lo, x.ctr_hi8 | 1u);
#pragma unroll 1
      for (int k = 0; k < 4 && q0 + k < x.V; ++k) {
        const float z = load_elem<DT>(x.row, q0 + k);
        if (!(z > -CUDART_INF_F && z < CUDART_INF_F)) continue;
        const uint32_t cbyte = (cword >> (8 * k)) & 0xFFu, xw = pick_word(fw, k);
        if (!(score_f32(z, inv_tau, cbyte, xw) >= floor_y)) continue;
        const double y = exact_score(z, x.tau, cbyte, xw);
        if (ibest < 0 || y > ybest) {  // indices ascend within a lane
          ybest = y;
          ibest = q0 + k;
          zbest = z;
        }
      }
    }
  }
  warp_argmax_double(ybest, ibest, zbest);
  z_tok = zbest;
  return ibest;
}

// ---------------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------------
template <int DT, int SAMPLER, bool RING>
__global__ void __launch_bounds__(kThreads, 2) rows_kernel(const __grid_constant__ RowsParams p) {
  extern __shared__ __align__(128) unsigned char dyn[];  // ring, then sampler 0: candidate queues, sampler 1: lane sums
  __shared__ Smem sm;
  using F = Fmt<DT>;
  constexpr int kEsize = F::kEsize;
  constexpr int kChunkE = F::kChunkE;
  constexpr int kLaneE = F::kLaneE;
  constexpr int kG = F::kG;
  constexpr int kVG = F::kVG;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  unsigned char *const ring = dyn;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&sm.full[s], 1); mbar_init(&sm.empty[s], kStreamWarps); }
    for (int s = 0; s < kSlots; ++s) { mbar_init(&sm.wfull[s], kStreamWarps); mbar_init(&sm.wfree[s], 1); }
    sm.best64 = 0ull;
    sm.timeout = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // Programmatic dependent launch: this grid may have been started while the kernel before it in the
  // stream was still finishing (launch latency, block start-up and the set-up above then overlap with that
  // kernel's tail).  Nothing in global memory may be touched before the wait below, which returns once the
  // earlier kernel has completed and its writes are visible; the grid behind this one may start likewise.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const int full_end = (int)(p.V & ~(int64_t)15);  // entries covered by full groups

  if (warp < kStreamWarps) {
    // ------------------------------------------------------------------ consumers
    SegIter it(p, true);
    Seg s;
    RowInfo ri;
    uint32_t stage = 0, phase = 0;  // ring position
    uint32_t n = 0;                 // segments handed to the finishing warp so far
    const uint32_t *const rk = p.round_key;
    unsigned char *const queue = dyn + (RING ? kStages * kStageBytes : 0) + warp * F::kQueueBytes;
    // sampler 1: the warp's lane sums of the last kLB steps
    float *const bscratch = reinterpret_cast<float *>(dyn + (RING ? kStages * kStageBytes : 0)) + warp * (F::kLB * 32);
    // vector order of this lane inside its 64 bytes (the lanes of a quarter warp hit distinct banks)
    const int rot = (lane >> 1) & 3;
    while (it.next(p, s, ri)) {
      if (ri.masked) continue;
      if (ri.invalid) {
        // nothing to compute, but the row's chunks are on their way: let them pass
        if (RING) {
          const int nc = s.e_hi > s.e_lo ? (s.e_hi - s.e_lo + kChunkE - 1) / kChunkE : 0;
          for (int c = 0; c < nc; ++c) {
            mbar_wait(&sm.full[stage], phase, sm);
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.empty[stage]);
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
        continue;
      }
      const char *row = row_ptr<DT>(p, s.row);
      const uint32_t grow = p.row_base + (uint32_t)s.row;
      const uint32_t seg = n + 1;
#define E3_MAKE_CTX(ex)                                                                                  \
  EvalCtx ex;                                                                                            \
  ex.rk = rk; ex.row = row; ex.tau = ri.tau; ex.slack_k = p.slack_scale; ex.grow = grow; ex.ctr_lo = p.ctr_lo; \
  ex.ctr_hi8 = p.ctr_hi8;                                                                                \
  ex.seg = seg; ex.V = (int)p.V

      Acc acc;
      acc_reset(acc);
      Best best;
      best.y[0] = best.y[1] = best.y[2] = -CUDART_INF_F;
      best.b[0] = best.b[1] = best.b[2] = -1;
      best.zf = 0.f;
      set_gate(best, enc_neg_inf(), ri.tau);
      float ethr = 0.f;
      int err = 0, qn = 0;
      BlockState bs;
      block_state_reset(bs);

      const int nchunks = s.e_hi > s.e_lo ? (s.e_hi - s.e_lo + kChunkE - 1) / kChunkE : 0;
      const int fast_end = s.e_hi < full_end ? s.e_hi : full_end;  // full groups of the piece end here
      const bool stream = RING && !ri.greedy;
#pragma unroll 1
      for (int c = 0; c < nchunks; ++c) {
        const int cs = s.e_lo + c * kChunkE;
        const int e_lane = cs + tid * kLaneE;
        const unsigned char *stage_ptr = nullptr;
        if (RING) {
          mbar_wait(&sm.full[stage], phase, sm);
          stage_ptr = ring + (size_t)stage * kStageBytes;
        }
        if (stream) {
          const unsigned char *lane_data = stage_ptr + tid * kLaneBytes;
          const int lim = fast_end < cs + kChunkE ? fast_end : cs + kChunkE;
          if (c == 0) {
            float R0;
            if (SAMPLER == 0) {
              SeedIO sd;
              sd.best = best;
              E3_MAKE_CTX(ex);
              seed_piece<DT, SAMPLER>(sd, ex, lane_data, e_lane, lim, sm);
              best = sd.best;
              R0 = sd.R0;
            } else {
              R0 = seed_reference<DT>(lane_data, e_lane, lim);
            }
            if (R0 > -CUDART_INF_F) {
              const float nRc = -R0 * ri.c;
              if (fabsf(nRc) < CUDART_INF_F) { acc.R = R0; acc.nRc = nRc; }
            }
            if (SAMPLER == 0) ethr = gate_threshold(best.enc, acc.nRc);
          } else if (SAMPLER == 0 && (c & 3) == 0) {
            const int enc = read_best(sm, seg);
            if (enc > best.enc) {
              set_gate(best, enc, ri.tau);
              ethr = gate_threshold(best.enc, acc.nRc);
            }
          }
          // the row's last, partial group (V not a multiple of 16) sits behind the full groups of this chunk
          float zextra = 0.f;
          const bool tail_here = fast_end < s.e_hi && fast_end >= cs && fast_end < cs + kChunkE;
          if (tail_here) {
            const int owner = (fast_end - cs) / kLaneE;  // thread whose 64 bytes would hold it
            if ((owner >> 5) == warp) {
              SlowIO io;
              io.acc = acc; io.err = err; io.zsum = 0.f;
              if (SAMPLER == 0) io.best = best;
              E3_MAKE_CTX(ex);
              slow_groups<DT, SAMPLER, true>(io, ex, owner == tid ? fast_end : s.e_hi, s.e_hi, ri.c, sm);
              acc = io.acc; err = io.err;
              if (SAMPLER == 0) best = io.best;
              zextra = io.zsum;
              if (SAMPLER == 0) ethr = gate_threshold(best.enc, acc.nRc);
            }
          }
          // ---- the streaming form: one group of 16 entries per turn (a single copy of the code, so that
          // the loop stays in the instruction cache).  Turn gi works on group gi ^ ga of the thread's 64
          // bytes and reads its vectors in the order i ^ rot, which keeps the lanes of a quarter warp on
          // distinct banks.  All lanes of the warp share one reference logit.
          const int ga = kG == 2 ? (rot >> 1) : 0;
          float zl = zextra;  // sampler 1: this thread's share of its block
          // Without the per-group work of sampler 0, a stage that lies wholly inside the row is taken in
          // one piece: the thread's 64 bytes in straight-line code and one check for the warp.  If the
          // check fails (stale reference, a value that is not finite) nothing has been added yet and
          // the turns below deal with the stage.
          bool stage_done = false;
          if (SAMPLER != 0 && fast_end >= cs + kChunkE) {
            uint4 raw[4];
            const uint4 *pv = reinterpret_cast<const uint4 *>(lane_data);
#pragma unroll
            for (int i = 0; i < 4; ++i) raw[i] = pv[i ^ rot];
            f2 Zs2, Ws2;
            const float Zs = hot_vectors<DT, 4>(raw, pack2f(ri.c, ri.c), pack2f(acc.nRc, acc.nRc), Ws2, Zs2);
            if (!__any_sync(0xffffffffu, !(Zs <= kGroupSumMax))) {
              acc.Z2 = add2(acc.Z2, Zs2);
              acc.W2 = add2(acc.W2, Ws2);
              zl += Zs;
              stage_done = true;
            }
          }
#pragma unroll 1
          for (int gi = stage_done ? kG : 0; gi < kG; ++gi) {
            const int gn = gi ^ ga;
            const int g0 = e_lane + (gn << 4);
            const bool have = g0 + kGroup <= lim;
            uint4 raw[kVG];
            {
              const uint4 *pv = reinterpret_cast<const uint4 *>(lane_data) + gn * kVG;
#pragma unroll
              for (int i = 0; i < kVG; ++i) raw[i] = pv[(i ^ rot) & (kVG - 1)];
            }
            float Zg = 0.f;
            f2 Zg2 = pack2f(0.f, 0.f), Wg2 = pack2f(0.f, 0.f);  // the group's sums; they join the state once they are known to be sound
#pragma unroll 1
            for (int attempt = 0;; ++attempt) {
              if (have) Zg = hot_group<DT>(raw, pack2f(ri.c, ri.c), pack2f(acc.nRc, acc.nRc), Wg2, Zg2);
              if (!__any_sync(0xffffffffu, have && !(Zg <= kGroupSumMax))) break;
              // the reference is stale for some lane (or a value is not finite)
              const float gm = have ? group_max<DT>(raw) : -CUDART_INF_F;
              const float newR = dec_float(__reduce_max_sync(0xffffffffu, enc_float(gm)));
              const float nRc = -newR * ri.c;
              if (attempt == 0 && newR > acc.R && newR < CUDART_INF_F && fabsf(nRc) < CUDART_INF_F) {
                // move the warp's reference up to the largest logit of this turn and repeat the group
                const float d = nRc - acc.nRc;
                const float f = acc.R == -CUDART_INF_F ? 0.f : ex2f(d);
                const f2 ff = pack2f(f, f);
                acc.W2 = mul2(ff, fma2(pack2f(d, d), acc.Z2, acc.W2));
                acc.Z2 = mul2(ff, acc.Z2);
                if (f == 0.f) acc.Z2 = acc.W2 = pack2f(0.f, 0.f);
                acc.R = newR; acc.nRc = nRc;
                zl *= f;
                if (SAMPLER == 0) ethr = gate_threshold(best.enc, acc.nRc);
                continue;
              }
              // NaN, +inf or numbers outside the fp32 range: the careful form sorts it out
              StepIO io;
              io.acc = acc; io.err = err; io.Zextra = zl;
              io.Zg[0] = 0.f; io.Zg[kG - 1] = 0.f;
              redo_step<DT, true>(io, lane_data, have ? (1 << gn) : 0, ri.c);
              acc = io.acc; err = io.err; zl = io.Zextra;
              Zg = io.Zg[gn];
              Zg2 = Wg2 = pack2f(0.f, 0.f);  // the careful form has added the group already
              if (SAMPLER == 0) ethr = gate_threshold(best.enc, acc.nRc);
              break;
            }
            acc.Z2 = add2(acc.Z2, Zg2);
            acc.W2 = add2(acc.W2, Wg2);
            zl += Zg;
            if (SAMPLER == 0) {
              const uint4 cb = philox(rk, (uint32_t)g0 >> 4, grow, p.ctr_lo, p.ctr_hi8 | 0u);
              const bool over = Zg > ethr;
              const bool flag = have && (any_ff4(cb) != 0u || over);
              const uint32_t ballot = __ballot_sync(0xffffffffu, flag);
              if (ballot != 0u) {
                if (flag) {
                  const int pos = qn + __popc(ballot & ((1u << lane) - 1u));
                  reinterpret_cast<int *>(queue)[pos] = g0 | (over ? 1 : 0);
                  uint4 *ent = reinterpret_cast<uint4 *>(queue + kQueueHdrBytes + pos * F::kEntryBytes);
                  ent[0] = cb;
#pragma unroll
                  for (int i = 0; i < kVG; ++i) ent[1 + ((i ^ rot) & (kVG - 1))] = raw[i];
                }
                qn += __popc(ballot);
                if (qn >= kDrainAt) {
                  Best tb = best;
                  drain_queue<DT>(rk, grow, p.ctr_lo, p.ctr_hi8, ri.tau, p.slack_scale, seg, queue, qn, tb, sm);
                  best = tb;
                  qn = 0;
                  const int enc = read_best(sm, seg);
                  if (enc > best.enc) set_gate(best, enc, ri.tau);
                  ethr = gate_threshold(best.enc, acc.nRc);
                }
              }
            }
          }
          if (SAMPLER == 1) block_step<DT>(zl, e_lane >> 8, acc.nRc, rk, grow, p.ctr_lo, p.ctr_hi8, bs, bscratch, lane, c);
        } else if (ri.greedy) {
          SlowIO io;
          io.acc = acc; io.err = err; io.zsum = 0.f;
          if (SAMPLER != 0) {  // the running maximum lives in the list of blocks, which greedy rows do not use
            io.best.y[0] = bs.top.y[0]; io.best.b[0] = bs.top.b[0];
          } else {
            io.best = best;
          }
          greedy_groups<DT>(io, row, RING ? stage_ptr + tid * kLaneBytes : nullptr, e_lane,
                            fast_end < cs + kChunkE ? fast_end : cs + kChunkE, s.e_hi);
          err = io.err;
          if (SAMPLER != 0) {
            bs.top.y[0] = io.best.y[0]; bs.top.b[0] = io.best.b[0];
          } else {
            best = io.best;
          }
        } else {
          // rows that cannot use the ring: everything through the guarded form
          SlowIO io;
          io.acc = acc; io.err = err; io.zsum = 0.f;
          if (SAMPLER == 0) io.best = best;
          E3_MAKE_CTX(ex);
          slow_groups<DT, SAMPLER, true>(io, ex, e_lane < s.e_hi ? e_lane : s.e_hi, s.e_hi, ri.c, sm);
          acc = io.acc; err = io.err;
          if (SAMPLER == 0) best = io.best;
          if (SAMPLER == 1) block_step<DT>(io.zsum, e_lane >> 8, acc.nRc, rk, grow, p.ctr_lo, p.ctr_hi8, bs, bscratch, lane, c);
        }
        if (RING) {
          __syncwarp();
          if (lane == 0) mbar_arrive(&sm.empty[stage]);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (SAMPLER == 0 && qn > 0) {
        Best tb = best;
        drain_queue<DT>(rk, grow, p.ctr_lo, p.ctr_hi8, ri.tau, p.slack_scale, seg, queue, qn, tb, sm);
        best = tb;
        qn = 0;
      }
      if (SAMPLER == 1 && !ri.greedy) {
        // blocks of the unfinished round: lanes whose step has not come hold no block (b = -1)
        block_flush<DT>(rk, grow, p.ctr_lo, p.ctr_hi8, bs, bscratch, lane);
      }

      AccS fin = to_scalar(acc);
      if (!ri.greedy) {
        // NaN or infinite sums (a NaN or +inf logit, or numbers outside the fp32 range): settle this
        // thread's entries of the piece with the careful form, which also says what was wrong
        const bool odd = !(fabsf(fin.Z) < CUDART_INF_F) || !(fabsf(fin.W) < CUDART_INF_F);
        if (__any_sync(0xffffffffu, odd)) {
          fin.R = -CUDART_INF_F; fin.nRc = kNoRef; fin.Z = fin.W = 0.f;
#pragma unroll 1
          for (int g = 0; g < nchunks * kG; ++g) {
            const int e0 = s.e_lo + (g / kG) * kChunkE + tid * kLaneE + (g % kG) * kGroup;
            if (e0 < s.e_hi) {
              float z[16];
              load_group_guarded<DT>(row, e0, e0 + kGroup <= (int)p.V ? 16 : (int)p.V - e0, z);
              careful_accumulate(fin, z, ri.c, -CUDART_INF_F, err);
            }
          }
        }
      }

      // warp-level merge, hand-over to the finishing warp
      Piece pw;
      pw.M = -fin.nRc; pw.Z = fin.Z; pw.W = fin.W;
      if (fin.R == -CUDART_INF_F) { pw.M = 0.f; pw.Z = 0.f; pw.W = 0.f; }
      pw.zf = SAMPLER == 0 ? best.zf : 0.f; pw.err = err;
      if (SAMPLER == 0) {  // the thread's leaders; sampler 1 has its blocks there (greedy rows: the maximum) already
#pragma unroll
        for (int i = 0; i < 3; ++i) { bs.top.y[i] = best.y[i]; bs.top.b[i] = best.b[i]; }
      }
      warp_merge(pw, bs.top, SAMPLER >= 0);
      const uint32_t slot = n % kSlots, use = n / kSlots;
      if (use > 0) mbar_wait(&sm.wfree[slot], (use - 1) & 1u, sm);
      if (lane == 0) {
        WarpPartial &w = sm.wpart[slot][warp];
        w.M = pw.M; w.Z = pw.Z; w.W = pw.W; w.err = pw.err; w.zf = pw.zf;
#pragma unroll
        for (int i = 0; i < 3; ++i) { w.ty[i] = bs.top.y[i]; w.tb[i] = bs.top.b[i]; }
        mbar_arrive(&sm.wfull[slot]);
      }
      ++n;
    }
#undef E3_MAKE_CTX
  } else if (warp == kStreamWarps) {
    // ------------------------------------------------------------------ producer (one thread)
    if (RING && lane == 0) {
      SegIter it(p, false);
      Seg s;
      RowInfo ri;
      uint32_t cc = 0, stage = 0, phase = 1;  // phase: parity of the previous use of the stage
      while (it.next(p, s, ri)) {
        if (ri.masked) continue;
        const char *row = row_ptr<DT>(p, s.row);
        const int nchunks = s.e_hi > s.e_lo ? (s.e_hi - s.e_lo + kChunkE - 1) / kChunkE : 0;
        const int lim = s.e_hi < full_end ? s.e_hi : full_end;
        for (int c = 0; c < nchunks; ++c) {
          if (cc >= (uint32_t)kStages) mbar_wait(&sm.empty[stage], phase, sm, 32u);
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
        const uint32_t st = q % kStages, round = q / kStages;
        for (uint32_t i = 0; i < kSpinLimit && !mbar_try_wait(&sm.full[st], round & 1u); ++i) __nanosleep(64);
      }
    }
  } else {
    // ------------------------------------------------------------------ finishing warp
    SegIter it(p, true, true);
    Seg s;
    RowInfo ri;
    uint32_t n = 0;
    u64 *const pieces = reinterpret_cast<u64 *>(p.ws_pieces);
    constexpr int kPieceStride = (int)(kPieceBytes / 8);
    const bool sample = p.mode == kModeSample;
    // The code below runs once or twice per CTA, the last time at the very end of the CTA's life, when
    // nothing hides it, and a first run through cold code is dominated by instruction fetches (several
    // times the warm time).  So the warp rehearses it while the consumers work on the first piece: pass
    // number p.rehearse takes the first piece's descriptors and made-up sums through the same
    // instructions with every store, barrier operation and workspace write switched off.  (The pass number
    // is a kernel argument so that the compiler keeps a single copy of the loop body.)
    for (int pass = 0;; ++pass) {
      const bool ghost = pass == p.rehearse;
      if (ghost) {
        SegIter peek = it;
        if (!peek.next(p, s, ri)) continue;
      } else if (!it.next(p, s, ri)) {
        break;
      }
      if (ri.masked || ri.invalid) {
        if (!ghost && s.starts && lane == 0) write_skipped(p, s.row, ri);
        continue;
      }
      // the target's logit is fetched while the consumers work on the piece
      int target = -1;
      float zt = 0.f;
      if (!sample && lane == 0) {
        target = __ldg(p.targets + s.row);
        if (target >= 0 && target < p.V) zt = load_elem<DT>(row_ptr<DT>(p, s.row), target);
      }
      const uint32_t slot = n % kSlots, use = n / kSlots;
      if (!ghost) mbar_wait_warp(&sm.wfull[slot], use & 1u, sm, lane);
      Piece pc;
      pc.M = 0.f; pc.Z = 0.f; pc.W = 0.f; pc.zf = 0.f; pc.err = 0; pc.pad = 0;
      Top3 top;
      top3_reset(top);
      if (!ghost && lane < kStreamWarps) {
        const WarpPartial &w = sm.wpart[slot][lane];
        pc.M = w.M; pc.Z = w.Z; pc.W = w.W; pc.err = w.err; pc.zf = w.zf;
        if (SAMPLER >= 0) {
#pragma unroll
          for (int i = 0; i < 3; ++i) { top.y[i] = w.ty[i]; top.b[i] = w.tb[i]; }
        }
      }
      __syncwarp();
      if (!ghost) {
        if (lane == 0) mbar_arrive(&sm.wfree[slot]);
        ++n;
      }
      // The order of every merge below is fixed by lane and piece numbers alone, so the result does not
      // depend on which CTA ends up finishing the row.
      warp_merge(pc, top, SAMPLER >= 0);
      if (*reinterpret_cast<volatile int *>(&sm.timeout)) pc.err |= kErrTimeout;
      bool fin = s.whole;
      if (!s.whole || (ghost && pieces != nullptr)) {
        // A piece of a cut row.  Store it, then (after a sequentially consistent fence) look for the
        // row's other pieces: of all CTAs that hold a piece, the one whose fence comes last is sure to
        // find them all and finishes the row.  Two CTAs may both find all pieces; they then write the
        // same values.  Nobody waits for anybody.
        if (lane == 0 && !ghost) {
#pragma unroll
          for (int i = 0; i < 3; ++i) { pc.ty[i] = top.y[i]; pc.tb[i] = top.b[i]; }
          piece_store(pieces + ((size_t)blockIdx.x * 2 + (s.first ? 0 : 1)) * kPieceStride, p.call_id, pc);
          asm volatile("fence.sc.gpu;" ::: "memory");
        }
        __syncwarp();
        pc.M = 0.f; pc.Z = 0.f; pc.W = 0.f; pc.zf = 0.f; pc.err = 0;
        top3_reset(top);
        bool ok = true;
        for (int k = s.k0 + lane; k <= s.k1; k += 32) {
          // CTA k keeps this row's piece in slot 0 when the row is the first thing it works on
          const bool is_first_seg = quot(p, first_tile_of(p, k), p.tiles_per_row) == s.row;
          Piece q;
          if (!piece_load(pieces + ((size_t)k * 2 + (is_first_seg ? 0 : 1)) * kPieceStride, p.call_id, q)) {
            ok = false;
            break;
          }
          pc.err |= q.err;
          merge_stats_f(pc.M, pc.Z, pc.W, q.M, q.Z, q.W);
          if (SAMPLER >= 0) {
            if (q.tb[0] >= 0 && best_before(q.ty[0], q.tb[0], top.y[0], top.b[0])) pc.zf = q.zf;
#pragma unroll
            for (int i = 0; i < 3; ++i) top3_insert(top, q.ty[i], q.tb[i]);
          }
        }
        fin = __all_sync(0xffffffffu, ok);
        if (fin || ghost) warp_merge(pc, top, SAMPLER >= 0);
      }
      if (ghost) {  // made-up sums and a leader that exists in every row: entry 0 / block 0
        fin = true;
        pc.M = 0.f; pc.Z = 1.f; pc.W = 0.f; pc.zf = 0.f; pc.err = 0;
        top3_reset(top);
        top.y[0] = 0.f; top.b[0] = 0;
      }
      if (!fin) continue;
      int id = -1;
      bool have_zt = !sample && target >= 0 && target < p.V;
      if (SAMPLER >= 0) {
        id = top.b[0];
        if (!ri.greedy && id >= 0) {
          EvalCtx ex;
          ex.rk = p.round_key; ex.row = row_ptr<DT>(p, s.row); ex.tau = ri.tau; ex.slack_k = p.slack_scale;
          ex.grow = p.row_base + (uint32_t)s.row;
          ex.ctr_lo = p.ctr_lo; ex.ctr_hi8 = p.ctr_hi8; ex.seg = 0; ex.V = (int)p.V;
          if (SAMPLER == 1) {
            // the whole warp settles the block and draws inside it
            id = sample_in_blocks<DT>(ex, top, lane, zt);
          } else {
            // fp32 scores decide unless the runner-up is within two slacks of the leader
            zt = pc.zf;
            const float slack2 = 2.f * fmaxf(score_slack(top.y[0], p.slack_scale), score_slack(top.y[1], p.slack_scale));
            if (top.b[1] >= 0 && !(top.y[0] - top.y[1] > slack2)) id = settle_exact<DT>(ex, top, slack2, lane, zt);
          }
          have_zt = id >= 0;
        }
      }
      if (lane == 0) finish_row(p, s.row, ri, pc.M, pc.Z, pc.W, id, pc.err, have_zt, zt, !ghost);
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
constexpr size_t dyn_smem_bytes() {
  return (RING ? (size_t)kStages * kStageBytes : 0) + (SAMPLER == 0 ? (size_t)kStreamWarps * Fmt<DT>::kQueueBytes : 0) +
         (SAMPLER == 1 ? (size_t)kStreamWarps * Fmt<DT>::kLB * 32 * sizeof(float) : 0);
}

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
    const size_t dyn = dyn_smem_bytes<DT, SAMPLER, RING>();
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
  p.narrow = tiles < (int64_t(1) << 31) ? 1 : 0;
  if (tiles / slots >= (int64_t(1) << 30)) return cudaErrorInvalidValue;  // per-CTA tile counts are kept in 32 bits
  const bool can_cut = workspace != nullptr && workspace_bytes >= rows_workspace_bytes();
  // With a response mask the cost of a row is not known on the host: spread whole rows round-robin.
  p.interleaved = (!can_cut || (p.mask != nullptr && p.rows >= 4 * slots)) ? 1 : 0;
  int64_t grid = p.interleaved ? (p.rows < slots ? p.rows : slots) : (tiles < slots ? tiles : slots);
  p.tiles_q = tiles / grid;
  p.tiles_r = tiles % grid;
  p.ws_pieces = can_cut ? static_cast<unsigned char *>(workspace) : nullptr;
  p.call_id = next_call_id();
  p.rehearse = 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = dyn_smem_bytes<DT, SAMPLER, RING>();
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, rows_kernel<DT, SAMPLER, RING>, p);
}

}  // namespace

size_t rows_workspace_bytes() { return (size_t)kMaxGrid * 2 * kPieceBytes; }

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
