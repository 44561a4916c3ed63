// Row-streaming kernels: one pass over the logits of a row gives the softmax statistics
// (App. A: Z(beta), Eq. "entropy" in its shifted form H = ln Z + beta sum p_i Delta_i), the
// log-probability of one token and, for rollouts, a Gumbel-max sample.
//
// Work split.  A row is cut into tiles of 4 KiB of logits and every CTA of a persistent grid (two per
// SM) takes an equal, contiguous run of tiles, so all CTAs stream the same number of bytes whatever
// the number of rows.  A run covers the tail of one row, some whole rows and the head of another; a
// CTA works on its two cut pieces first and on its whole rows last, so that what is left to do at
// the end of its life is the cheap finish of a row it holds alone.  For a row that is cut, a CTA first
// looks (while its consumers are still streaming, and again when they are done) whether the row's other
// pieces are in the caller's workspace already; if so it is the last to arrive and finishes the row
// without publishing anything.  Otherwise it stores its partial state (64-bit words tagged with a
// per-call id), issues a sequentially consistent fence and looks once more: of all CTAs that hold a
// piece, the one whose fence comes last finds them all.  Whoever finishes a row merges the pieces in
// piece order, writes the outputs and wipes the tags of the pieces it used, so that a replay of the
// same launch (a captured graph) never meets a piece of an earlier run.  Nobody waits for anybody.
// (With a response mask over many rows, and when no workspace is given, CTAs take whole rows
// round-robin instead.)
//
// Inside a CTA.  Each of the eight consumer warps owns a ring of three 4 KiB slots.  One warp feeds
// the rings, lane w feeding consumer warp w: per slot one bulk asynchronous copy (cp.async.bulk with a
// plain, CTA-local shared-memory destination, completion counted in bytes on the slot's mbarrier), a
// 4-byte asynchronous copy of the row's temperature that completes on the same barrier, and a small
// record that says what the slot holds (row, first entry, number of entries, first/last slice of a row
// piece).  The consumers keep no position of their own: every slot describes itself.  Consumer warp w
// takes tiles w, w + 8, ... of a piece.  A consumer thread takes 128 contiguous bytes of a slot, read as
// 16-byte vectors in the order i xor (lane mod 8), which keeps the eight lanes of a quarter warp on
// distinct banks.  One more warp finishes rows (merges the eight warp states, fp64 epilogue, piece
// protocol, sampler 0's settling of near-ties) so that the consumers never stall on it.
// Every wait is bounded in time: when one runs out the CTA stops waiting altogether, marks the rows it
// has not finished as invalid (token -1, NaN), sets the timeout bit of the caller's status word, sees
// its copies in flight land (bounded again) and returns.  The kernels are launched with programmatic
// stream serialization: their set-up overlaps the tail of the kernel before them in the stream, and
// they touch global memory only after griddepcontrol.wait.
//
// Numerics.  All lanes of a warp share a reference logit R; each thread keeps the sums Z = sum 2^t,
// W = sum 2^t * t with t = z*c - R*c and c = log2(e)/tau, two entries per instruction (packed fp32).
// The streaming loop never looks for the maximum: the sums of a turn (the thread's 128 bytes of a
// slot) stay local until the warp has checked them with one vote, and when one leaves the safe range
// (some t above 7, a NaN, an infinity) nothing has been added yet and the turn is taken again by the
// careful form, which moves R up to the largest logit of the slot, rescales the state, skips -inf
// entries and flags NaN and +inf.  R therefore stays close to the largest logit seen, which keeps W/Z
// small and the entropy free of cancellation.  States merge associatively; the per-row result is
// formed in fp64:  H = ln Z - ln2 * W / Z,  ln p_tok = (z_tok*c - M) ln2 - ln Z, and, where the caller
// asks for it, the mean logit gap beta sum p_i Delta_i = (z_max*c - M - W/Z) ln2 of App. A (this variant
// of the kernel also tracks the largest logit, half an instruction per entry more).
//
// Sampler 0 (one Gumbel per vocabulary entry).  u_i has 8 coarse + 32 fine bits.  An entry can
// only win if its coarse byte is 255 (g_i >= 5.5432) or if z_i/tau exceeds the best score so
// far minus 5.5432; the second condition is tested on the sum of 2^t over the entry's group of 16,
// which bounds every term from above.  Groups that pass are copied into a per-warp queue in shared
// memory with ballot-compacted positions; when enough are waiting the warp scores them, one group
// per lane, in fp32 with a proven error bound, and every thread keeps its three leaders.  The
// finishing warp takes the fp32 leader when it is ahead by more than two error bounds; otherwise
// it evaluates the contenders in fp64 with the expression order of the definition (or looks at the
// whole row again when there are three or more).  The token never depends on the gating or on fp32.
//
// Sampler 1 (one Gumbel per block of 256 entries) is two kernels.  The consumers of the streaming kernel
// do nothing for it but one shared-memory store per turn: every lane leaves its sum of 2^t over its 128
// bytes (4 or 8 neighbouring lanes make up a block) and lane 0 the reference the sums refer to in a
// 144-byte record next to the rings; the feeding lane ships the record to the caller's workspace with a
// bulk asynchronous store when it sees the slot freed.  (A global store from a consumer costs the warp
// microseconds while the copies keep the memory system busy, and so does every instruction-cache miss:
// whatever the consumers execute besides their loop is dear.)  block_sample_kernel, launched behind the
// streaming kernel, adds the lanes of every block, turns the sums into scores L_b + g_b (fp32, three
// leaders per thread), settles near-ties of block scores in fp64 and draws inside the winning block by
// inverse CDF (fp32, fp64 near a prefix boundary).  The workspace traffic is 1/28 of the logits.
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

constexpr int kSlots = 4;  // hand-over slots between the consumer warps and the finishing warp
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2f = 0.6931471805599453f;
constexpr double kLn2 = 0.6931471805599453094;
// Largest Gumbel value an entry whose coarse byte is below 255 can reach is -ln(-ln(255/256)) = 5.54322...;
// with all 40 bits set the largest value is -ln(-ln(1 - 2^-41)) = 28.41903...  Both rounded up.
constexpr float kGumbelCapCoarse = 5.5433f;
constexpr float kGumbelCapAll = 28.4192f;
// A turn (up to 64 entries of one thread) whose sum of 2^t is above this (or NaN) means that the warp's
// reference logit is stale: every entry that is added has t <= 7 while the reference is a logit the
// warp has really seen, so W/Z stays small and the entropy ln Z - ln2 W/Z is free of cancellation at the
// 1e-5 level.  (64 entries equal to the reference give 64: a flat row must pass.)
constexpr float kTurnSumMax = 128.f;
constexpr float kTurnWMax = 1e30f;  // |sum 2^t t| of a sound turn stays far below (a -inf logit makes it NaN)
constexpr float kNoRef = 1e30f;     // nRc of a state without reference: the first turn overflows into the careful form

enum : int { kErrValue = 1, kErrTimeout = 4 };
enum : uint32_t { kFlagFirst = 1u, kFlagLast = 2u, kFlagEnd = 8u };

template <int DT>
struct Fmt {
  static constexpr int kEsize = DT == 0 ? 4 : 2;
  static constexpr int kLaneE = kLaneBytes / kEsize;  // entries per thread and stage: 32 fp32 / 64 bf16
  static constexpr int kWarpE = 32 * kLaneE;          // entries per warp and stage = entries per tile: 1,024 / 2,048
  static constexpr int kStageE = kStreamWarps * kWarpE;  // entries per stage: 8,192 / 16,384
  static constexpr int kVG = kEsize;                  // 16-byte vectors per group of 16 entries: 4 / 2
  static constexpr int kG = 8 / kVG;                  // groups per thread and stage: 2 / 4
  static constexpr int kLB = 256 / kLaneE;            // lanes that hold one block of sampler 1: 8 / 4
  static constexpr int kEntryBytes = kGroup * kEsize; // queue entry of sampler 0: the logits of one group
};

// Sampler 0 queues: a push never meets a queue holding kDrainAt or more groups and adds at most 32.
constexpr int kDrainAt = 16;
constexpr int kQueueCap = kDrainAt + 32;
template <int DT>
struct QueueBytes { static constexpr int value = kQueueCap * 4 + kQueueCap * Fmt<DT>::kEntryBytes; };
// fp32 logits with sampler 0 need the larger queue entries: two ring stages there (the variant is bound
// by the per-entry random numbers, not by the copies in flight)
template <int DT, int SAMPLER>
struct RingStages { static constexpr int value = (DT == 0 && SAMPLER == 0) ? 2 : kStages; };
// Sampler 1: per consumer warp two records (144 bytes) per ring slot, used alternately, behind the rings.
constexpr int kRecordBytesPerWarp = 2 * kStages * kRecordFloats * 4;

// One partial row state.  In the workspace it is kPieceWords 64-bit words, each (tag << 32 | payload):
// the tag depends on the call and on the word, so a reader knows word by word whether what it sees was
// written by this call (64-bit accesses are single-copy atomic); stale or half-written pieces fail the check.
struct Piece {
  float M, Z, W;   // reference (log2 units), sum 2^t, sum 2^t t
  float zf;        // sampler 0: logit of entry tb[0]
  int err;
  float zmax;      // largest logit (only where the mean logit gap is asked for)
  float ty[3];     // the three best scores (fp32): sampler 0 entries, sampler 1 blocks; greedy rows: ty[0] = largest logit
  int tb[3];       // ... and their vocabulary / block indices, -1 = none
};
constexpr int kPieceWords = 12;
static_assert(sizeof(Piece) == kPieceWords * 4, "piece payload");
static_assert(kPieceWords * 8 <= kPieceBytes, "piece size");

struct WarpPartial {
  float M, Z, W;
  float zf;
  float zmax;
  int err;
  float ty[3];
  int tb[3];
};

// What a ring slot holds; written by the warp's lane 0 when it starts the copy into the slot (tau arrives with
// the data: a 4-byte asynchronous copy that completes on the slot's barrier).
struct __align__(16) SliceMeta {
  long long row;
  int s_lo;      // first entry of the slice within its row
  int n;         // entries of the slice (0: the warp holds nothing of this row piece, or the closing record)
  uint32_t flags;
  float tau;
  uint32_t pad[2];
};
static_assert(sizeof(SliceMeta) == 32, "slot record");

struct Smem {
  u64 full[kStreamWarps][kStages];    // per warp and ring slot: the slot's data (and its tau) have landed
  u64 empty[kStreamWarps][kStages];   // ... the warp is done with the slot
  u64 wfull[kSlots], wfree[kSlots];   // consumer warps -> finishing warp
  u64 best64;                         // (piece number << 32 | encoded best score) of sampler 0
  SliceMeta meta[kStreamWarps][kStages];
  WarpPartial wpart[kSlots][kStreamWarps];
  int timeout;                        // set when a bounded wait ran out
  unsigned long long deadline_ns;     // a wait that is still unsatisfied this long after it began gives up
  int32_t *status;                    // the caller's status word (may be null)
  uint32_t rk[20];                    // Philox round keys (a copy of the launch parameter: shared memory serves indexed reads best)
};

struct RowInfo {
  float tau, c;
  bool masked;   // masked out: the row's logits are not read and nothing is computed
  bool invalid;  // temperature not usable: the row's logits are not read either
  bool greedy;
};

struct Seg {
  int64_t row;
  int e_lo, e_hi;  // entries [e_lo, e_hi) of the row
  bool whole;      // the CTA holds the whole row
  bool starts;     // holds the row's first tile
  bool slot0;      // cut piece that holds the CTA's first tile (workspace slot 0), else slot 1
  int k0, k1;      // CTAs holding the first / last tile of the row (cut rows only)
};

// Sampler 0: what a thread knows about the leaders of its row piece.  Scores are fp32 values of
// y_i = z_i/tau + g_i, each within score_slack(y) of the exact value; the three best are kept so that
// the finishing warp can tell whether fp32 separates the winner from the rest.
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
__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
template <int DT>
__device__ __forceinline__ float lds_elem(uint32_t addr) {
  if (DT == 0) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
  }
  unsigned short h;
  asm volatile("ld.shared.u16 %0, [%1];" : "=h"(h) : "r"(addr));
  return __uint_as_float((uint32_t)h << 16);
}

__device__ __forceinline__ void mbar_init(u64 *b, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(u64 *b) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(b)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(u64 *b, uint32_t bytes) {
  asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(b)), "r"(bytes) : "memory");
}
// One poll (the hardware may park the thread for a short, implementation-defined time; a loop of these
// needs no sleep of its own, and a warp that has slept with nanosleep runs slowly for a while afterwards).
__device__ __forceinline__ bool mbar_try_wait(u64 *b, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_addr(b)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool timed_out(const Smem &sm) { return *reinterpret_cast<const volatile int *>(&sm.timeout) != 0; }
// A wait has run out: from now on no wait of the CTA blocks, and the caller's status word says so.
__device__ __noinline__ void raise_timeout(Smem &sm) {
  *reinterpret_cast<volatile int *>(&sm.timeout) = 1;
  if (sm.status != nullptr) atomicOr(sm.status, kStatusTimeout);
}
// Bounded wait: true when the barrier phase has completed, false when the wait was given up (it took longer
// than the CTA's limit, or another wait of the CTA has run out before: then no wait blocks any more).
__device__ __noinline__ bool mbar_wait_slow(u64 *b, uint32_t parity, Smem &sm) {
  const unsigned long long t0 = global_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(b, parity)) return true;
    if (timed_out(sm)) return false;
    if ((it & 63u) == 0u && global_ns() - t0 > sm.deadline_ns) break;
  }
  raise_timeout(sm);
  return false;
}
__device__ __forceinline__ bool mbar_wait(u64 *b, uint32_t parity, Smem &sm) {
  return mbar_try_wait(b, parity) ? true : mbar_wait_slow(b, parity, sm);
}
// Whole-warp wait with a single polling lane.
__device__ __forceinline__ bool mbar_wait_warp(u64 *b, uint32_t parity, Smem &sm, int lane) {
  bool ok = true;
  if (lane == 0) ok = mbar_wait(b, parity, sm);
  return __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
}
// Bulk asynchronous copy global -> this CTA's shared memory; completion is counted in bytes on `bar`.
// The logits are read once: their lines are marked evict-first in L2, so that the stream does not push out what
// is used again and again (the kernel's instructions, the workspace, temperatures) -- an L2 miss of any of
// those waits behind the whole queue of the stream.
__device__ __forceinline__ u64 l2_evict_first_policy() {
  u64 pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void *src, uint32_t bytes, u64 *bar, u64 policy) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(smem_addr(bar)), "l"(policy)
               : "memory");
}

// Bulk asynchronous copy this CTA's shared memory -> global, as a bulk group of the issuing thread.
__device__ __forceinline__ void bulk_store_s2g(void *dst, uint32_t src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// Returns when all but the N most recent bulk groups of the thread have read their source.
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// Orders the thread's earlier shared-memory writes before later reads of the asynchronous proxy (bulk copies).
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

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

// The same function as a loop over the rounds: a tenth of the code, for the streaming loop of sampler 0, whose
// speed is set by instruction fetch (four calls per turn would otherwise be 250 instructions each).
__device__ __forceinline__ uint4 philox_rolled(const uint32_t *rk, uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3) {
#pragma unroll 1
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

// CTA-wide best score of the row piece: 64-bit word (piece number, order-preserving code).
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

// 16 consecutive logits of a stage in shared memory (plain order).
template <int DT>
__device__ __forceinline__ void load_group_smem(uint32_t addr, float (&z)[16]) {
  if (DT == 0) {
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const uint4 v = lds128(addr + 16 * q);
      z[4 * q] = __uint_as_float(v.x); z[4 * q + 1] = __uint_as_float(v.y);
      z[4 * q + 2] = __uint_as_float(v.z); z[4 * q + 3] = __uint_as_float(v.w);
    }
  } else {
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const uint4 v = lds128(addr + 16 * q);
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
// Running sums of a consumer thread, two fp32 lanes per register pair.
struct Acc {
  float R, nRc;      // reference logit and -R*c; R = -inf, nRc = kNoRef: no reference yet
  f2 Z2, W2;         // Z = sum of both halves of Z2, W likewise
};
__device__ __forceinline__ void acc_reset(Acc &a) {
  a.R = -CUDART_INF_F;
  a.nRc = kNoRef;
  a.Z2 = a.W2 = pack2f(0.f, 0.f);
}

// A thread's 128 bytes of a stage: B = shared-memory address of the slice with (lane mod 8) << 4 or-ed in;
// v[i] is 16-byte vector number i xor (lane mod 8) of the slice.
__device__ __forceinline__ void load_slice(uint32_t B, uint4 (&v)[8]) {
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = lds128(B ^ (uint32_t)(i << 4));
}

// Entries at or beyond nlane (counted in vocabulary order within the slice) become -inf.
template <int DT>
__device__ __forceinline__ void mask_slice(uint4 (&v)[8], int nlane, int r8) {
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
    if (DT == 1) {
      const int rem = nlane - 8 * (i ^ r8);  // entries of this vector that are valid
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t lo = 2 * j < rem ? (w[j] & 0xFFFFu) : 0xFF80u;
        const uint32_t hi = 2 * j + 1 < rem ? (w[j] & 0xFFFF0000u) : 0xFF800000u;
        w[j] = lo | hi;
      }
    } else {
      const int rem = nlane - 4 * (i ^ r8);
#pragma unroll
      for (int j = 0; j < 4; ++j) w[j] = j < rem ? w[j] : 0xFF800000u;
    }
    v[i] = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// Largest logit of a slice (NaN entries are passed over).
template <int DT>
__device__ __forceinline__ float slice_max(const uint4 (&v)[8]) {
  if (DT == 1) {
    uint32_t m0 = v[0].x, m1 = v[0].y;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      asm("max.bf16x2 %0, %1, %2;" : "=r"(m0) : "r"(m0), "r"(v[i].x));
      asm("max.bf16x2 %0, %1, %2;" : "=r"(m1) : "r"(m1), "r"(v[i].y));
      asm("max.bf16x2 %0, %1, %2;" : "=r"(m0) : "r"(m0), "r"(v[i].z));
      asm("max.bf16x2 %0, %1, %2;" : "=r"(m1) : "r"(m1), "r"(v[i].w));
    }
    asm("max.bf16x2 %0, %1, %2;" : "=r"(m0) : "r"(m0), "r"(m1));
    return fmaxf(__uint_as_float(m0 << 16), __uint_as_float(m0 & 0xFFFF0000u));
  } else {
    float m = -CUDART_INF_F;
#pragma unroll
    for (int i = 0; i < 8; ++i)
      m = fmaxf(fmaxf(m, fmaxf(__uint_as_float(v[i].x), __uint_as_float(v[i].y))),
                fmaxf(__uint_as_float(v[i].z), __uint_as_float(v[i].w)));
    return m;
  }
}

// Streaming form for a slice: the packed sums of 2^t and of 2^t t over its entries, t = z c + nRc; with
// GROUPS also the sum of 2^t of every group of 16 entries: Zg[j] belongs to group j xor ((lane mod 8) /
// vectors per group).  CLAMP: logits below -2^100 (also -inf) enter as -2^100, which gives them weight 0 and
// keeps 2^t t finite; NaN stays NaN.
template <int DT, bool GROUPS, bool CLAMP>
__device__ __forceinline__ void slice_sums(const uint4 (&v)[8], f2 c2, f2 nRc2, f2 &Zt2, f2 &Wt2, float (&Zg)[Fmt<DT>::kG]) {
  constexpr int kVG = Fmt<DT>::kVG;
  f2 Wa = pack2f(0.f, 0.f), Wb = pack2f(0.f, 0.f);
  f2 Zj[Fmt<DT>::kG];
#pragma unroll
  for (int j = 0; j < Fmt<DT>::kG; ++j) Zj[j] = pack2f(0.f, 0.f);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
#pragma unroll
    for (int j = 0; j < (DT == 1 ? 4 : 2); ++j) {
      f2 z2;
      if (DT == 1) {
        uint32_t x = w[j];
        if (CLAMP) asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(x) : "r"(x), "r"(0xF180F180u));
        z2 = pack2f(__uint_as_float(x << 16), __uint_as_float(x & 0xFFFF0000u));
      } else {
        float a = __uint_as_float(w[2 * j]), b = __uint_as_float(w[2 * j + 1]);
        if (CLAMP) {
          asm("max.NaN.f32 %0, %1, %2;" : "=f"(a) : "f"(a), "f"(-1.2676506e30f));
          asm("max.NaN.f32 %0, %1, %2;" : "=f"(b) : "f"(b), "f"(-1.2676506e30f));
        }
        z2 = pack2f(a, b);
      }
      const f2 t2 = fma2(z2, c2, nRc2);
      const f2 e2 = pack2f(ex2f(t2.x), ex2f(t2.y));
      Zj[i / kVG] = add2(Zj[i / kVG], e2);
      if (j & 1) Wb = fma2(e2, t2, Wb); else Wa = fma2(e2, t2, Wa);
    }
  }
  Wt2 = add2(Wa, Wb);
  if (GROUPS) {
#pragma unroll
    for (int j = 0; j < Fmt<DT>::kG; ++j) Zg[j] = sum2(Zj[j]);
  }
  if (Fmt<DT>::kG == 4) {
    Zt2 = add2(add2(Zj[0], Zj[1]), add2(Zj[2], Zj[3]));
  } else {
    Zt2 = add2(Zj[0], Zj[1]);
  }
}

// The streaming form as a loop over the two halves of the slice: the same sums (without group sums) with a
// loop body short enough for the instruction cache.  The thread's slice is read in the order
// i xor (lane mod 8) as everywhere.  GAP: zmax becomes the largest logit of the slice (NaN passed over).
constexpr int kPartVecs = 4;
template <int DT, bool GAP>
__device__ __forceinline__ void slice_sums_rolled(uint32_t B, f2 c2, f2 nRc2, f2 &Zt2, f2 &Wt2, float &zmax) {
  f2 Za = pack2f(0.f, 0.f), Zb = pack2f(0.f, 0.f), Wa = pack2f(0.f, 0.f), Wb = pack2f(0.f, 0.f);
  uint32_t m0 = DT == 1 ? 0xFF80FF80u : 0xFF800000u, m1 = m0;  // -inf
#pragma unroll 1
  for (int h = 0; h < 8 / kPartVecs; ++h) {
    const uint32_t Bh = B ^ (uint32_t)(h * kPartVecs * 16);
    uint4 v[kPartVecs];
#pragma unroll
    for (int i = 0; i < kPartVecs; ++i) v[i] = lds128(Bh ^ (uint32_t)(i << 4));
#pragma unroll
    for (int i = 0; i < kPartVecs; ++i) {
      const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
      if (GAP) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          uint32_t &m = (j & 1) ? m1 : m0;
          if (DT == 1) {
            asm("max.bf16x2 %0, %1, %2;" : "=r"(m) : "r"(m), "r"(w[j]));
          } else {
            m = __float_as_uint(fmaxf(__uint_as_float(m), __uint_as_float(w[j])));
          }
        }
      }
#pragma unroll
      for (int j = 0; j < (DT == 1 ? 4 : 2); ++j) {
        f2 z2;
        if (DT == 1) {
          z2 = pack2f(__uint_as_float(w[j] << 16), __uint_as_float(w[j] & 0xFFFF0000u));
        } else {
          z2 = pack2f(__uint_as_float(w[2 * j]), __uint_as_float(w[2 * j + 1]));
        }
        const f2 t2 = fma2(z2, c2, nRc2);
        const f2 e2 = pack2f(ex2f(t2.x), ex2f(t2.y));
        if (j & 1) { Zb = add2(Zb, e2); Wb = fma2(e2, t2, Wb); } else { Za = add2(Za, e2); Wa = fma2(e2, t2, Wa); }
      }
    }
  }
  Zt2 = add2(Za, Zb);
  Wt2 = add2(Wa, Wb);
  if (GAP) {
    if (DT == 1) {
      asm("max.bf16x2 %0, %1, %2;" : "=r"(m0) : "r"(m0), "r"(m1));
      zmax = fmaxf(__uint_as_float(m0 << 16), __uint_as_float(m0 & 0xFFFF0000u));
    } else {
      zmax = fmaxf(__uint_as_float(m0), __uint_as_float(m1));
    }
  }
}

// The careful form of a turn: for the first turn of a row piece, for a slice that lies only partly inside the
// piece, and when the streaming form's check failed (stale reference, a -inf, a NaN, a +inf).  The warp moves
// its reference up to the largest finite logit of the slice, rescales its state and takes the turn with
// masked and clamped entries.  A NaN or +inf (or numbers outside the fp32 range) flags the row.
template <int DT>
struct CarefulIO {
  Acc acc;
  f2 Zt2, Wt2;
  float Zg[Fmt<DT>::kG];
  float zmax;  // out: the lane's largest finite logit of the slice (-inf when it has none)
  int err;
};
// Inlined: a call would spill the streaming loop's state to local memory around it, and with the memory
// system saturated by the copies every such access takes microseconds.
template <int DT, bool GROUPS>
__device__ __forceinline__ void turn_careful(CarefulIO<DT> &io, uint32_t B, int nlane, int r8, float c) {
  Acc acc = io.acc;
  int err = io.err;
  f2 Zt2, Wt2;
  float Zg[Fmt<DT>::kG];
  uint4 v[8];
  load_slice(B, v);
  if (nlane < Fmt<DT>::kLaneE) mask_slice<DT>(v, nlane, r8);
  float gmax = slice_max<DT>(v);
  if (!(gmax < CUDART_INF_F)) gmax = -CUDART_INF_F;  // +inf is flagged by the sums below
  const float R0 = dec_float(__reduce_max_sync(0xffffffffu, enc_float(gmax)));
  if (R0 > acc.R) {
    const float nRc = -R0 * c;
    if (fabsf(nRc) < CUDART_INF_F) {
      const float d = nRc - acc.nRc;
      const float f = acc.R == -CUDART_INF_F ? 0.f : ex2f(d);
      if (f == 0.f) {
        acc.Z2 = acc.W2 = pack2f(0.f, 0.f);
      } else {
        const f2 ff = pack2f(f, f);
        acc.W2 = __fmul2_rn(ff, fma2(pack2f(d, d), acc.Z2, acc.W2));
        acc.Z2 = __fmul2_rn(ff, acc.Z2);
      }
      acc.R = R0; acc.nRc = nRc;
    } else {
      err |= kErrValue;  // the product left the fp32 range
    }
  }
  // without any reference (nothing finite so far) the sums must come out as zero
  const float nRc_use = acc.R == -CUDART_INF_F ? 0.f : acc.nRc;
  slice_sums<DT, GROUPS, true>(v, pack2f(c, c), pack2f(nRc_use, nRc_use), Zt2, Wt2, Zg);
  const float Zs = sum2(Zt2), Ws = sum2(Wt2);
  const bool bad = !(Zs <= kTurnSumMax) || !(fabsf(Ws) <= kTurnWMax) || (acc.R == -CUDART_INF_F && Zs != 0.f);
  if (__any_sync(0xffffffffu, bad)) {
    err |= kErrValue;
    Zt2 = Wt2 = pack2f(0.f, 0.f);
#pragma unroll
    for (int j = 0; j < Fmt<DT>::kG; ++j) Zg[j] = 0.f;
  }
  io.acc = acc; io.err = err; io.Zt2 = Zt2; io.Wt2 = Wt2; io.zmax = gmax;
#pragma unroll
  for (int j = 0; j < Fmt<DT>::kG; ++j) io.Zg[j] = GROUPS ? Zg[j] : 0.f;
}

// What the bulk copy of a slice did not bring: the last bytes of a row whose length is no multiple of 16 bytes, or
// everything when the rows do not start on 16-byte boundaries.  The warp fetches it entry by entry.
template <int DT>
__device__ __noinline__ void patch_slice(const char *row, int s_lo, int n, bool bulk, uint32_t dst, int lane) {
  constexpr int kEsize = Fmt<DT>::kEsize;
  const int ncopied = bulk ? (int)((((uint32_t)n * kEsize) & ~15u) / kEsize) : 0;
  for (int e = ncopied + lane; e < n; e += 32) {
    if (DT == 0) {
      const float v = __ldg(reinterpret_cast<const float *>(row) + s_lo + e);
      asm volatile("st.shared.f32 [%0], %1;" ::"r"(dst + e * 4), "f"(v) : "memory");
    } else {
      const unsigned short v = __ldg(reinterpret_cast<const unsigned short *>(row) + s_lo + e);
      asm volatile("st.shared.u16 [%0], %1;" ::"r"(dst + e * 2), "h"(v) : "memory");
    }
  }
  fence_async_smem();  // the next bulk copy into the slot comes after these stores
  __syncwarp();
}

// Greedy rows (tau = 0): largest logit, lowest index; NaN and +inf flag the row.
struct GreedyIO {
  float y;
  int i, err;
};
template <int DT>
__device__ __noinline__ void turn_greedy(GreedyIO &io, uint32_t B, int e_lane, int nlane, int r8) {
  float ybest = io.y;
  int ibest = io.i, err = io.err;
  uint4 v[8];
  load_slice(B, v);
  mask_slice<DT>(v, nlane, r8);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
    const int e0 = e_lane + (i ^ r8) * (DT == 1 ? 8 : 4);
#pragma unroll
    for (int k = 0; k < (DT == 1 ? 8 : 4); ++k) {
      const float z = DT == 1 ? __uint_as_float((k & 1) ? (w[k >> 1] & 0xFFFF0000u) : (w[k >> 1] << 16)) : __uint_as_float(w[k]);
      if (z != z || z == CUDART_INF_F) err |= kErrValue;
      if (z > -CUDART_INF_F && (ibest < 0 || z > ybest || (z == ybest && e0 + k < ibest))) {
        ybest = z;
        ibest = e0 + k;
      }
    }
  }
  io.y = ybest; io.i = ibest; io.err = err;
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

// A queue entry holds the 16 logits of one group in vocabulary order.  Its header word is the index
// of the group's first entry, with bit 0 set when the group passed the sum gate.
template <int DT>
__device__ __forceinline__ float entry_logit(const unsigned char *entry, int k) {
  if (DT == 0) return *reinterpret_cast<const float *>(entry + 4 * k);
  return __uint_as_float((uint32_t)(*reinterpret_cast<const unsigned short *>(entry + 2 * k)) << 16);
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
    const unsigned char *entry = queue + kQueueCap * 4 + e * Fmt<DT>::kEntryBytes;
    const int hdr = hdrs[e];
    const int g0 = hdr & ~15;
    const uint4 cw = philox(rk, (uint32_t)g0 >> 4, grow, ctr_lo, ctr_hi8 | 0u);  // the group's coarse bytes
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
      const uint32_t cbyte = (pick_word(cw, k >> 2) >> (8 * (k & 3))) & 0xFFu;
      consider(rk, grow, ctr_lo, ctr_hi8, tau, inv_tau, slack_k, seg, g0 + k, cbyte, entry_logit<DT>(entry, k), b, sm);
    }
  }
  __syncwarp();
  best_io = b;
}

// ---------------------------------------------------------------------------------------------
// Sampler 1: one Gumbel per block of 256 consecutive entries, applied to the block's log-sum-exp.
// All lanes of a warp keep the same reference, so that the lane sums of a block add up directly.
// kLB neighbouring lanes hold one block per stage; lane j of such a group keeps the block of stage j
// of every kLB stages, and then all lanes turn the block they keep into a score Y_b = L_b + g_b (one
// Philox call and three MUFU each) and enter it in their list of three leaders (fp32).  The finishing
// warp settles near-ties in fp64 and draws the token inside the winning block by inverse CDF.
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

// fp32 Gumbel variate from a 32-bit word: u = (x + 1/2) 2^-32, g = -ln(-ln u)
__device__ __forceinline__ float gumbel_from_word(uint32_t xw) {
  float a;  // -ln u
  if (xw >= 0xFE000000u) {
    const float d = ((float)(~xw) + 0.5f) * 0x1p-32f;  // 1 - u < 2^-7: series of -ln(1 - d)
    a = d * fmaf(d, fmaf(d, 0.33333334f, 0.5f), 1.0f);
  } else {
    a = -lg2f(((float)xw + 0.5f) * 0x1p-32f) * kLn2f;
  }
  return -lg2f(a) * kLn2f;
}

// Sampler 0, first stage of a row piece: a valid lower bound of the piece's best score from the coarse byte
// of the largest entry of each lane's first group alone: u >= (c + 2^-33)/256  =>  g >= -ln(ln 256 - ln(c + 2^-33)).
template <int DT>
__device__ __noinline__ void seed_gate(Best &best, const EvalCtx &x, uint32_t lane_addr, int e_lane, Smem &sm) {
  float z[16];
  load_group_smem<DT>(lane_addr, z);
  float gmax = -CUDART_INF_F;
#pragma unroll
  for (int k = 0; k < 16; ++k) gmax = fmaxf(gmax, z[k]);
  const bool usable = gmax > -CUDART_INF_F && gmax < CUDART_INF_F;
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
  if (enc > best.enc) set_gate(best, enc, x.tau);
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
// Makes a piece unreadable for every call id: word j gets the complement of this call's tag.
__device__ __forceinline__ void piece_wipe(u64 *dst, u64 call_id) {
#pragma unroll
  for (int j = 0; j < kPieceWords; ++j) {
    const u64 v = (u64)(~piece_tag(call_id, j)) << 32;
    asm volatile("st.relaxed.gpu.global.b64 [%0], %1;" ::"l"(dst + j), "l"(v) : "memory");
  }
}

// Merges the lists of leaders held by the 32 lanes of a warp (sampler 0 entries, sampler 1 blocks, greedy
// maxima); every lane ends with the result, zf follows top.b[0].  Three rounds of "take the best head":
// larger score first, equal scores by lower index.
__device__ __forceinline__ void warp_merge_top(Top3 &top, float &zf) {
  constexpr unsigned kAll = 0xffffffffu;
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
      if (r == 0) zf = __shfl_sync(kAll, zf, __ffs(__ballot_sync(kAll, mine)) - 1);
      if (mine) ++pos;
    }
  }
  top = out;
}

// Merges the partial states held by the 32 lanes of a warp; every lane ends with the result.  A lane
// without weight (Z = 0) takes no part.  The order of all sums is fixed by lane numbers.
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
  pc.zmax = dec_float(__reduce_max_sync(kAll, enc_float(pc.zmax)));
  if (with_top) warp_merge_top(top, pc.zf);
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

// Hands out the CTA's row pieces: first the piece that starts inside a row (if the run starts so), then
// the piece that ends inside a row, then the whole rows in order.  All divisions happen in the constructor.
struct Walker {
  int64_t row0;     // row of the run's first tile (interleaved: the CTA's first row)
  int n;            // pieces of the run in vocabulary order (interleaved: rows of the CTA)
  int tin0, tend;   // first tile of the run within row0; end tile of the run within its last row (1..tiles_per_row)
  int k;            // pieces handed out so far
  bool first_cut, last_cut;
  __device__ explicit Walker(const RowsParams &p) : row0(0), n(0), tin0(0), tend(0), k(0), first_cut(false), last_cut(false) {
    if (p.interleaved) {
      row0 = blockIdx.x;
      n = (int64_t)blockIdx.x < p.rows ? (int)((p.rows - 1 - blockIdx.x) / gridDim.x) + 1 : 0;
      return;
    }
    const int64_t len = p.tiles_q + ((int64_t)blockIdx.x < p.tiles_r ? 1 : 0);
    if (len <= 0) return;
    const int64_t t0 = first_tile_of(p, blockIdx.x);
    row0 = quot(p, t0, p.tiles_per_row);
    tin0 = (int)(t0 - row0 * p.tiles_per_row);
    const int64_t row_last = quot(p, t0 + len - 1, p.tiles_per_row);
    tend = (int)(t0 + len - row_last * p.tiles_per_row);
    n = (int)(row_last - row0) + 1;
    const int tpr = (int)p.tiles_per_row;
    first_cut = tin0 > 0 || (n == 1 && tend < tpr);
    last_cut = n > 1 && tend < tpr;
  }
  // Row of the piece number q of the hand-out order (q >= 0), -1 when there is none.
  __device__ int64_t row_of(const RowsParams &p, int q) const {
    if (q >= n) return -1;
    if (p.interleaved) return row0 + (int64_t)q * gridDim.x;
    return row0 + index_of(q);
  }
  __device__ int index_of(int q) const {  // hand-out number -> position in vocabulary order
    const int nc = (first_cut ? 1 : 0) + (last_cut ? 1 : 0);
    if (q == 0 && first_cut) return 0;
    if (q == (first_cut ? 1 : 0) && last_cut) return n - 1;
    return q - nc + (first_cut ? 1 : 0);
  }
  // with_range: also work out which CTAs hold the row's first and last tile (only the finishing warp asks)
  template <int DT>
  __device__ bool next(const RowsParams &p, Seg &s, bool with_range) {
    if (k >= n) return false;
    s.k0 = s.k1 = 0;
    if (p.interleaved) {
      s.row = row0 + (int64_t)k * gridDim.x;
      s.e_lo = 0; s.e_hi = (int)p.V; s.whole = true; s.starts = true; s.slot0 = false;
      ++k;
      return true;
    }
    const int j = index_of(k);
    const int tpr = (int)p.tiles_per_row;
    const int lo = j == 0 ? tin0 : 0, hi = j == n - 1 ? tend : tpr;
    const int64_t elo = (int64_t)lo * Fmt<DT>::kWarpE, ehi = (int64_t)hi * Fmt<DT>::kWarpE;
    s.row = row0 + j;
    s.e_lo = (int)elo;
    s.e_hi = (int)(ehi < p.V ? ehi : p.V);
    s.starts = lo == 0;
    s.whole = lo == 0 && hi == tpr;
    s.slot0 = j == 0;
    if (!s.whole && with_range) {
      s.k0 = cta_of_tile(p, s.row * p.tiles_per_row);
      s.k1 = cta_of_tile(p, (s.row + 1) * p.tiles_per_row - 1);
    }
    ++k;
    return true;
  }
};

// Walks the CTA's row pieces and loads temperature and mask of the piece after the current one, so
// that nobody waits for them when that piece starts.
template <int DT>
struct SegIter {
  Walker wk;
  float tau_next;
  bool masked_next;
  bool with_range;
  // The constructor touches no global memory (it may run before the wait for the kernel ahead in the stream);
  // start() loads temperature and mask of the first piece.
  __device__ SegIter(const RowsParams &p, bool with_range_)
      : wk(p), tau_next(0.f), masked_next(false), with_range(with_range_) {}
  __device__ void start(const RowsParams &p) { prefetch(p, wk.row_of(p, 0)); }
  __device__ void prefetch(const RowsParams &p, int64_t row) {
    tau_next = p.temp_scalar;
    masked_next = false;
    if (row >= 0) {
      if (p.temps) tau_next = __ldg(p.temps + row);
      masked_next = p.mode != kModeSample && p.mask && __ldg(p.mask + row) == 0;
    }
  }
  __device__ bool next(const RowsParams &p, Seg &s, RowInfo &r) {
    if (!wk.template next<DT>(p, s, with_range)) return false;
    r.tau = tau_next;
    r.masked = masked_next;
    prefetch(p, wk.row_of(p, wk.k));
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
// defer: the token of this row is drawn by block_sample_kernel, which gets the row's sums through the workspace
// (x: reference in log2 units, y: sum of 2^t, z: non-zero = nothing to do, the row is finished or flagged).
__device__ __forceinline__ void finish_row(const RowsParams &p, int64_t row, const RowInfo &ri, float Mf, float Zf,
                                           float Wf, float zmax, int idx, int err, bool have_zt, float zt, bool defer) {
  const double M = Mf, Z = Zf, W = Wf;
  const bool sample = p.mode == kModeSample;
  int tok = -1;
  float logp = CUDART_NAN_F, ent = CUDART_NAN_F, gap = CUDART_NAN_F;
  bool deferred = false;
  if (ri.greedy) {
    if (err == 0 && idx >= 0) { tok = idx; logp = 0.f; ent = 0.f; gap = 0.f; }
  } else if (err == 0 && Z > 0.0) {
    const double lnZ = log(Z);
    ent = (float)(lnZ - kLn2 * (W / Z));
    // sum p_i (s_max - s_i) with s = z/tau: the mean of s is (M + W/Z) ln2
    gap = (float)(((double)zmax * (double)ri.c - M - W / Z) * kLn2);
    if (sample) tok = idx;
    if (have_zt) logp = (float)(((double)zt * (double)ri.c - M) * kLn2 - lnZ);
    deferred = defer;
  }
  if (defer) p.ws_rowstat[row] = make_float4(Mf, Zf, deferred ? 0.f : 1.f, 0.f);
  if (p.out_ent) p.out_ent[row] = ent;
  if (p.out_gap) p.out_gap[row] = gap;
  if (deferred) return;
  if (sample) p.out_tok[row] = tok;
  if (p.out_logp) p.out_logp[row] = logp;
}

__device__ __forceinline__ void write_skipped(const RowsParams &p, int64_t row, const RowInfo &ri) {
  const bool sample = p.mode == kModeSample;
  const float v = ri.invalid ? CUDART_NAN_F : 0.f;
  if (sample) p.out_tok[row] = -1;
  if (p.out_logp) p.out_logp[row] = v;
  if (p.out_ent) p.out_ent[row] = v;
  if (p.out_gap) p.out_gap[row] = v;
}
// A row the CTA gives up on (a wait ran out).
__device__ __forceinline__ void write_abandoned(const RowsParams &p, int64_t row, bool defer) {
  if (p.mode == kModeSample) p.out_tok[row] = -1;
  if (p.out_logp) p.out_logp[row] = CUDART_NAN_F;
  if (p.out_ent) p.out_ent[row] = CUDART_NAN_F;
  if (p.out_gap) p.out_gap[row] = CUDART_NAN_F;
  if (defer) p.ws_rowstat[row] = make_float4(0.f, 0.f, 1.f, 0.f);
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
// 4-byte asynchronous copy global -> shared and an arrival on `bar` once the thread's earlier copies of this
// kind have landed (the arrival counts as one of the barrier's expected arrivals).
__device__ __forceinline__ void async_copy4(uint32_t dst, const void *src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void async_arrive(u64 *bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_addr(bar)) : "memory");
}

// Keeps the ring of one consumer warp filled: lane w of the feeding warp does this for consumer warp w.  It
// walks the CTA's row pieces; of every piece the consumer warp takes the slices
// [e_lo + q * (entries per stage) + w * (entries per slice), + entries per slice) that start inside the
// piece; a piece of which the warp holds nothing still gives one empty record, so that every warp hands
// exactly one partial state per piece to the finishing warp.  Only whole 16-byte units are copied here (one
// bulk copy per slice); what a row whose length is no multiple of 16 bytes leaves over, and rows that do not
// start on 16-byte boundaries altogether, the consumer warp fetches itself.
template <int DT>
struct Feeder {
  Walker wk;
  int64_t row;
  int s_next, e_hi, q_left;
  bool first, done, stalled, masked_next;
  u64 policy;
  __device__ Feeder(const RowsParams &p) : wk(p), row(0), s_next(0), e_hi(0), q_left(0), first(false), done(false), stalled(false) {
    policy = l2_evict_first_policy();
    masked_next = false;  // the constructor touches no global memory; start() looks at the first row's mask
  }
  __device__ void start(const RowsParams &p) { peek_mask(p, wk.row_of(p, 0)); }
  __device__ void peek_mask(const RowsParams &p, int64_t r) {
    masked_next = r >= 0 && p.mode != kModeSample && p.mask && __ldg(p.mask + r) == 0;
  }
  // Puts the next slice of consumer warp w (or the closing record) into its ring slot `slot`.
  __device__ __forceinline__ void feed(const RowsParams &p, Smem &sm, uint32_t ring, int w, int slot) {
    using F = Fmt<DT>;
    uint32_t flags;
    int n;
    SliceMeta m;
    m.pad[0] = m.pad[1] = 0;
    u64 *const bar = &sm.full[w][slot];
    if (q_left == 0) {
      Seg s;
      bool have;
      for (;;) {
        have = wk.template next<DT>(p, s, false);
        if (!have) break;
        const bool masked = masked_next;
        peek_mask(p, wk.row_of(p, wk.k));
        if (!masked) break;
      }
      if (!have) {
        done = true;
        m.row = 0; m.s_lo = 0; m.n = 0; m.flags = kFlagEnd; m.tau = 0.f;
        sm.meta[w][slot] = m;
        mbar_arrive(bar);
        return;
      }
      row = s.row;
      e_hi = s.e_hi;
      s_next = s.e_lo + w * F::kWarpE;
      q_left = s_next < e_hi ? (e_hi - s_next + F::kStageE - 1) / F::kStageE : 0;
      first = true;
    }
    if (q_left == 0) {  // nothing of this piece lies in the warp's slices
      flags = kFlagFirst | kFlagLast;
      n = 0;
    } else {
      flags = (first ? kFlagFirst : 0u) | (q_left == 1 ? kFlagLast : 0u);
      n = e_hi - s_next < F::kWarpE ? e_hi - s_next : F::kWarpE;
    }
    if (p.stall_tile >= 0 && n > 0 && row * p.tiles_per_row + s_next / F::kWarpE == p.stall_tile) {
      done = stalled = true;  // test hook: this slot is never filled, the consumer's wait for it runs out
      return;
    }
    m.row = row; m.s_lo = s_next; m.n = n; m.flags = flags; m.tau = p.temp_scalar;
    sm.meta[w][slot] = m;
    const uint32_t bytes = p.bulk ? ((uint32_t)n * F::kEsize) & ~15u : 0u;
    if (bytes > 0) {
      mbar_expect_tx(bar, bytes);
      bulk_copy_g2s(ring + (uint32_t)slot * kWarpBytes, row_ptr<DT>(p, row) + (size_t)s_next * F::kEsize, bytes, bar, policy);
    }
    if (p.temps != nullptr) {
      async_copy4(smem_addr(&sm.meta[w][slot].tau), p.temps + row);
      async_arrive(bar);
    } else {
      mbar_arrive(bar);
    }
    if (q_left > 0) {
      s_next += F::kStageE;
      --q_left;
    }
    first = false;
  }
};

// GAP: also track the largest logit of every row (for the mean logit gap).
template <int DT, int SAMPLER, bool GAP>
__global__ void __launch_bounds__(kThreads, 2) rows_kernel(const __grid_constant__ RowsParams p) {
  extern __shared__ __align__(128) unsigned char dyn[];  // the warps' rings, then sampler 0: candidate queues
  __shared__ Smem sm;
  using F = Fmt<DT>;
  constexpr int kEsize = F::kEsize;
  constexpr int kLaneE = F::kLaneE;
  constexpr int kG = F::kG;
  constexpr int kNS = RingStages<DT, SAMPLER>::value;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t ring = smem_addr(dyn);

  if (tid == 0) {
    for (int w = 0; w < kStreamWarps; ++w)
      for (int s = 0; s < kNS; ++s) { mbar_init(&sm.full[w][s], 1); mbar_init(&sm.empty[w][s], 1); }
    for (int s = 0; s < kSlots; ++s) { mbar_init(&sm.wfull[s], kStreamWarps); mbar_init(&sm.wfree[s], 1); }
    sm.best64 = 0ull;
    sm.timeout = 0;
    sm.deadline_ns = p.wait_ns;
    sm.status = p.status;
    for (int i = 0; i < 20; ++i) sm.rk[i] = p.round_key[i];
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  // Programmatic dependent launch: this grid may have been started while the kernel before it in the
  // stream was still finishing (launch latency, block start-up and the set-up above then overlap with that
  // kernel's tail).  Nothing in global memory may be touched before the wait below, which returns once the
  // earlier kernel has completed and its writes are visible; the grid behind this one may start likewise.
  // Every role works out what it can from the launch parameters first and waits right before its first access
  // to global memory.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp < kStreamWarps) {
    // ------------------------------------------------------------------ consumers
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint32_t ring_warp = ring + (uint32_t)warp * (kNS * kWarpBytes);
    uint32_t slot = 0, phase = 0;   // ring position
    uint32_t n = 0;                 // row pieces handed to the finishing warp so far
    const uint32_t *const rk = sm.rk;
    unsigned char *const queue = dyn + kStreamWarps * kNS * kWarpBytes + warp * QueueBytes<DT>::value;
    const uint32_t rec_warp = ring + kStreamWarps * kNS * kWarpBytes + (uint32_t)warp * kRecordBytesPerWarp;  // sampler 1
    const int r8 = lane & 7;        // vector order of this lane inside its 128 bytes
    const int ga = r8 / F::kVG;     // ... and the resulting order of its groups
    Acc acc;
    acc_reset(acc);
    Best best;
    float gy = -CUDART_INF_F;  // greedy rows without sampler 0: the lane's largest logit and its index
    int gi = -1;
    float ethr = 0.f, c = 0.f, tau = 0.f;
    float zmax = -CUDART_INF_F;  // GAP: the lane's largest logit of the row piece
    int err = 0, qn = 0, it = 0;
    bool greedy = false, unusable = false;
    for (;;) {
      // a wait that was given up ends the warp's work: the slot's record cannot be trusted then
      if (__any_sync(0xffffffffu, !mbar_wait(&sm.full[warp][slot], phase, sm))) break;
      const SliceMeta m = sm.meta[warp][slot];
      if (m.flags & kFlagEnd) break;
      const uint32_t seg = n + 1;
      const char *const row = row_ptr<DT>(p, m.row);
      const uint32_t grow = p.row_base + (uint32_t)m.row;
#define E3_MAKE_CTX(ex)                                                                                 \
  EvalCtx ex;                                                                                           \
  ex.rk = rk; ex.row = row; ex.tau = tau; ex.slack_k = p.slack_scale; ex.grow = grow; ex.ctr_lo = p.ctr_lo; \
  ex.ctr_hi8 = p.ctr_hi8;                                                                               \
  ex.seg = seg; ex.V = (int)p.V

      if (m.flags & kFlagFirst) {
        tau = m.tau;
        greedy = p.mode == kModeSample && tau == 0.f;
        unusable = !greedy && !(tau > 0.f && tau < CUDART_INF_F);
        c = greedy || unusable ? 0.f : __fdiv_rn(kLog2e, tau);
        acc_reset(acc);
        gy = -CUDART_INF_F; gi = -1;
        zmax = -CUDART_INF_F;
        if (SAMPLER == 0) {
          best.y[0] = best.y[1] = best.y[2] = -CUDART_INF_F;
          best.b[0] = best.b[1] = best.b[2] = -1;
          best.zf = 0.f;
          set_gate(best, enc_neg_inf(), tau);
          ethr = 0.f;
        }
        err = unusable ? kErrValue : 0;
        qn = 0; it = 0;
      }
      if (m.n > 0 && !unusable) {
        const uint32_t lane_addr = ring_warp + slot * kWarpBytes + (uint32_t)(lane * kLaneBytes);
        if (!p.bulk || (((uint32_t)m.n * kEsize) & 15u) != 0u)
          patch_slice<DT>(row, m.s_lo, m.n, p.bulk != 0, ring_warp + slot * kWarpBytes, lane);
        const int e_lane = m.s_lo + lane * kLaneE;
        const int nlane = m.n - lane * kLaneE < 0 ? 0 : (m.n - lane * kLaneE > kLaneE ? kLaneE : m.n - lane * kLaneE);
        const uint32_t B = lane_addr | (uint32_t)(r8 << 4);
        if (greedy) {
          GreedyIO g;
          g.y = SAMPLER == 0 ? best.y[0] : gy;
          g.i = SAMPLER == 0 ? best.b[0] : gi;
          g.err = err;
          turn_greedy<DT>(g, B, e_lane, nlane, r8);
          if (SAMPLER == 0) { best.y[0] = g.y; best.b[0] = g.i; } else { gy = g.y; gi = g.i; }
          err = g.err;
        } else {
          f2 Zt2, Wt2;
          float Zg[kG];
          float zturn = -CUDART_INF_F;
          bool done = false;
          const bool full = m.n >= F::kWarpE;
          if (full && acc.R > -CUDART_INF_F) {
            if (SAMPLER == 0 && (it & 3) == 0) {
              const int enc = read_best(sm, seg);
              if (enc > best.enc) {
                set_gate(best, enc, tau);
                ethr = gate_threshold(best.enc, acc.nRc);
              }
            }
            if (SAMPLER == 0) {
              uint4 v[8];
              load_slice(B, v);
              slice_sums<DT, true, false>(v, pack2f(c, c), pack2f(acc.nRc, acc.nRc), Zt2, Wt2, Zg);
              if (GAP) zturn = slice_max<DT>(v);
            } else {
              slice_sums_rolled<DT, GAP>(B, pack2f(c, c), pack2f(acc.nRc, acc.nRc), Zt2, Wt2, zturn);
            }
            const float Zs = sum2(Zt2), Ws = sum2(Wt2);
            const bool bad = !(Zs <= kTurnSumMax) || !(fabsf(Ws) <= kTurnWMax);
            done = !__any_sync(0xffffffffu, bad);
          }
          if (!done) {
            const bool fresh = acc.R == -CUDART_INF_F;
            {
              CarefulIO<DT> io;
              io.acc = acc; io.err = err;
              turn_careful<DT, SAMPLER == 0>(io, B, nlane, r8, c);
              acc = io.acc; err = io.err; Zt2 = io.Zt2; Wt2 = io.Wt2; zturn = io.zmax;
              if (SAMPLER == 0) {
#pragma unroll
                for (int j = 0; j < kG; ++j) Zg[j] = io.Zg[j];
              }
            }
            if (SAMPLER == 0) {
              if (fresh && full && acc.R > -CUDART_INF_F) {
                E3_MAKE_CTX(ex);
                Best tb = best;
                seed_gate<DT>(tb, ex, lane_addr, e_lane, sm);
                best = tb;
              }
              ethr = gate_threshold(best.enc, acc.nRc);
            }
          }
          acc.Z2 = add2(acc.Z2, Zt2);
          acc.W2 = add2(acc.W2, Wt2);
          if (GAP) zmax = fmaxf(zmax, zturn);
          if (SAMPLER == 0) {
#pragma unroll 1
            for (int j = 0; j < kG; ++j) {  // a loop on purpose: short code (Zg is picked without indexing)
              const int g0 = e_lane + ((j ^ ga) << 4);
              const uint4 cb = philox_rolled(rk, (uint32_t)g0 >> 4, grow, p.ctr_lo, p.ctr_hi8 | 0u);
              float zg = Zg[0];
#pragma unroll
              for (int q = 1; q < kG; ++q) zg = j == q ? Zg[q] : zg;
              const bool over = zg > ethr;
              const bool flag = g0 < m.s_lo + m.n && (any_ff4(cb) != 0u || over);
              const uint32_t ballot = __ballot_sync(0xffffffffu, flag);
              if (ballot != 0u) {
                if (flag) {
                  const int pos = qn + __popc(ballot & ((1u << lane) - 1u));
                  reinterpret_cast<int *>(queue)[pos] = g0 | (over ? 1 : 0);
                  uint4 *ent = reinterpret_cast<uint4 *>(queue + kQueueCap * 4 + pos * F::kEntryBytes);
                  const uint32_t ga_addr = lane_addr + (uint32_t)((j ^ ga) << 4) * kEsize;
                  const int left = m.s_lo + m.n - g0;  // entries of the group that belong to the row piece
#pragma unroll
                  for (int i = 0; i < F::kVG; ++i) {
                    uint4 q = lds128(ga_addr + 16 * i);
                    if (left < kGroup) {  // the row ends inside the group: what lies behind it counts as -inf
                      uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
                      for (int k = 0; k < 4; ++k) {
                        if (DT == 1) {
                          const int e = 8 * i + 2 * k;
                          w[k] = (e < left ? (w[k] & 0xFFFFu) : 0xFF80u) | (e + 1 < left ? (w[k] & 0xFFFF0000u) : 0xFF800000u);
                        } else {
                          w[k] = 4 * i + k < left ? w[k] : 0xFF800000u;
                        }
                      }
                      q = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                    ent[i] = q;
                  }
                }
                qn += __popc(ballot);
                if (qn >= kDrainAt) {
                  Best tb = best;
                  drain_queue<DT>(rk, grow, p.ctr_lo, p.ctr_hi8, tau, p.slack_scale, seg, queue, qn, tb, sm);
                  best = tb;
                  qn = 0;
                  const int enc = read_best(sm, seg);
                  if (enc > best.enc) set_gate(best, enc, tau);
                  ethr = gate_threshold(best.enc, acc.nRc);
                }
              }
            }
          }
          if (SAMPLER == 1) {
            // The lane's sum and the reference it refers to: into the record of this use of the slot.  The feeding
            // lane ships the record to the workspace when it sees the slot freed (a global store from here would
            // cost the warp microseconds while the copies keep the memory system busy).
            const uint32_t rec = rec_warp + (phase * kNS + slot) * (uint32_t)(kRecordFloats * 4);
            asm volatile("st.shared.f32 [%0], %1;" ::"r"(rec + (uint32_t)lane * 4u), "f"(sum2(Zt2)) : "memory");
            if (lane == 0) asm volatile("st.shared.f32 [%0], %1;" ::"r"(rec + 128u), "f"(acc.nRc) : "memory");
            fence_async_smem();
          }
        }
        ++it;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.empty[warp][slot]);  // the slot is free again
      if (++slot == kNS) { slot = 0; phase ^= 1u; }

      if (m.flags & kFlagLast) {
        if (SAMPLER == 0 && qn > 0) {
          Best tb = best;
          drain_queue<DT>(rk, grow, p.ctr_lo, p.ctr_hi8, tau, p.slack_scale, seg, queue, qn, tb, sm);
          best = tb;
          qn = 0;
        }
        // warp-level merge (all lanes share the reference), hand-over to the finishing warp
        float Zs = sum2(acc.Z2), Ws = sum2(acc.W2);
        if (!(fabsf(Zs) < CUDART_INF_F) || !(fabsf(Ws) < CUDART_INF_F)) err |= kErrValue;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          Zs += __shfl_xor_sync(0xffffffffu, Zs, o);
          Ws += __shfl_xor_sync(0xffffffffu, Ws, o);
        }
        err = __reduce_or_sync(0xffffffffu, err);
        float zf = 0.f;
        Top3 wtop;
        top3_reset(wtop);
        if (SAMPLER == 0) {  // the thread's leaders
#pragma unroll
          for (int i = 0; i < 3; ++i) { wtop.y[i] = best.y[i]; wtop.b[i] = best.b[i]; }
          zf = best.zf;
        } else if (SAMPLER == 1 && greedy) {  // the lane's maximum
          wtop.y[0] = gy; wtop.b[0] = gi;
        }
        if (SAMPLER == 0 || (SAMPLER == 1 && greedy)) warp_merge_top(wtop, zf);
        const float zm = GAP ? dec_float(__reduce_max_sync(0xffffffffu, enc_float(zmax))) : 0.f;
        const uint32_t hslot = n % kSlots, use = n / kSlots;
        if (use > 0 && __any_sync(0xffffffffu, !mbar_wait(&sm.wfree[hslot], (use - 1) & 1u, sm))) break;
        if (lane == 0) {
          WarpPartial &w = sm.wpart[hslot][warp];
          const bool has = acc.R > -CUDART_INF_F;
          w.M = has ? -acc.nRc : 0.f; w.Z = has ? Zs : 0.f; w.W = has ? Ws : 0.f; w.err = err; w.zf = zf;
          w.zmax = zm;
#pragma unroll
          for (int i = 0; i < 3; ++i) { w.ty[i] = wtop.y[i]; w.tb[i] = wtop.b[i]; }
          mbar_arrive(&sm.wfull[hslot]);
        }
        ++n;
      }
    }
#undef E3_MAKE_CTX
  } else if (warp == kStreamWarps) {
    // ------------------------------------------------------------------ feeding warp: lane w feeds consumer warp w
    if (lane < kStreamWarps) {
      constexpr unsigned kLanes = (1u << kStreamWarps) - 1u;
      const uint32_t ring_w = ring + (uint32_t)lane * (kNS * kWarpBytes);
      Feeder<DT> feeder(p);
      asm volatile("griddepcontrol.wait;" ::: "memory");
      feeder.start(p);
      uint32_t issued = 0, slot = 0, phase = 1;  // phase: parity of the previous use of the slot
      // Sampler 1: ships the record the consumer warp left for the use `par` of slot `st` (the slot's record still
      // describes that use).  A record's buffer comes round again six uses later; by then its bulk store has read it
      // (all but the two most recent stores of this thread have, before a new one is issued).
      const uint32_t rec_lane = ring + kStreamWarps * kNS * kWarpBytes + (uint32_t)lane * kRecordBytesPerWarp;
      auto ship_tile = [&](int64_t ti, uint32_t st, uint32_t par) {
        bulk_wait_read<2>();
        bulk_store_s2g(p.ws_records + ti * kRecordFloats, rec_lane + (par * kNS + st) * (uint32_t)(kRecordFloats * 4),
                       kRecordFloats * 4);
      };
      // tile number of the slice the slot's record describes, -1 when it holds no entries (or closes the ring)
      auto tile_of = [&](uint32_t st) -> int64_t {
        const SliceMeta &pm = sm.meta[lane][st];
        return (pm.n > 0 && !(pm.flags & kFlagEnd)) ? pm.row * p.tiles_per_row + pm.s_lo / F::kWarpE : (int64_t)-1;
      };
      auto ship = [&](uint32_t st, uint32_t par) {
        const int64_t ti = tile_of(st);
        if (ti >= 0) ship_tile(ti, st, par);
      };
      unsigned long long idle_since = 0;         // 0: the last pass over the lanes fed something
      uint32_t idle_passes = 0;
      while (__any_sync(kLanes, !feeder.done)) {
        if (timed_out(sm)) break;  // somebody gave up: nothing more is fed, the consumers run out on their next wait
        bool ready = false;
        if (!feeder.done) {
          ready = issued < (uint32_t)kNS;
          if (!ready) {
            uint32_t ok;
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(ok) : "r"(smem_addr(&sm.empty[lane][slot])), "r"(phase) : "memory");
            ready = ok != 0;
          }
          if (ready) {
            // sampler 1: the record of the slot's previous use goes out AFTER the refill has been issued (the refill
            // is what the consumer warp waits for); its slice is read from the slot's record before that is rewritten
            const int64_t prev_tile = (SAMPLER == 1 && issued >= (uint32_t)kNS) ? tile_of(slot) : (int64_t)-1;
            feeder.feed(p, sm, ring_w, lane, (int)slot);
            if (SAMPLER == 1 && prev_tile >= 0) ship_tile(prev_tile, slot, phase);
            if (!feeder.stalled) {
              ++issued;
              if (++slot == kNS) { slot = 0; phase ^= 1u; }
            }
          }
        }
        if (__any_sync(kLanes, ready)) {
          idle_since = 0;
          idle_passes = 0;
        } else if ((++idle_passes & 255u) == 0u) {  // no consumer has freed a slot for a while: look at the clock
          const unsigned long long now = global_ns();
          if (idle_since == 0) idle_since = now;
          if (now - idle_since > p.wait_ns) raise_timeout(sm);
        }
      }
      // Before leaving, see every copy still in flight land (bounded): the slots handed out last.
      {
        const uint32_t back = issued < (uint32_t)kNS ? issued : (uint32_t)kNS;
        const unsigned long long t0 = global_ns();
        for (uint32_t q = issued - back; q < issued; ++q) {
          const uint32_t st = q % kNS, round = q / kNS;
          for (uint32_t i = 1; !mbar_try_wait(&sm.full[lane][st], round & 1u); ++i)
            if ((i & 63u) == 0u && global_ns() - t0 > p.wait_ns) break;
        }
        if (SAMPLER == 1) {  // ... and the records of those slots, once the consumer warp is done with them
          for (uint32_t q = issued - back; q < issued; ++q) {
            const uint32_t st = q % kNS, round = q / kNS;
            if (sm.meta[lane][st].flags & kFlagEnd) continue;
            bool ok = true;
            for (uint32_t i = 1; !mbar_try_wait(&sm.empty[lane][st], round & 1u); ++i)
              if (timed_out(sm) || ((i & 63u) == 0u && global_ns() - t0 > p.wait_ns)) { ok = false; break; }
            if (ok) ship(st, round & 1u);
          }
          bulk_wait_all();
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ finishing warp
    SegIter<DT> sit(p, true);
    asm volatile("griddepcontrol.wait;" ::: "memory");
    sit.start(p);
    Seg s;
    RowInfo ri;
    uint32_t n = 0;
    u64 *const pieces = reinterpret_cast<u64 *>(p.ws_pieces);
    constexpr int kPieceStride = (int)(kPieceBytes / 8);
    const bool sample = p.mode == kModeSample;
    while (sit.next(p, s, ri)) {
      if (ri.masked) {
        if (s.starts && lane == 0) write_skipped(p, s.row, ri);
        continue;
      }
      // the target's logit is fetched while the consumers work on the piece
      int target = -1;
      float zt = 0.f;
      if (!sample && lane == 0) {
        target = __ldg(p.targets + s.row);
        if (target >= 0 && target < p.V) zt = load_elem<DT>(row_ptr<DT>(p, s.row), target);
      }
      // A piece of a cut row: while the consumers still work on it, look for the row's other pieces.  When all
      // of them are there already, this CTA is the last one to arrive and finishes the row as soon as its own
      // piece is complete, without publishing it: the others have looked for it in vain and have given up.
      const int span = s.whole ? 0 : s.k1 - s.k0 + 1;
      const int kmine = s.k0 + lane;  // the CTA whose piece this lane looks after (rows held by up to 32 CTAs)
      Piece early;
      bool early_ok = false;
      if (!s.whole && span <= 32) {
        bool ok = true;
        if (lane < span && kmine != (int)blockIdx.x) {
          const bool is_first_seg = quot(p, first_tile_of(p, kmine), p.tiles_per_row) == s.row;
          ok = piece_load(pieces + ((size_t)kmine * 2 + (is_first_seg ? 0 : 1)) * kPieceStride, p.call_id, early);
        }
        early_ok = __all_sync(0xffffffffu, ok);
      }
      const uint32_t slot = n % kSlots, use = n / kSlots;
      if (!mbar_wait_warp(&sm.wfull[slot], use & 1u, sm, lane)) {
        // A wait of this CTA ran out: it gives up on this piece and on all that follow.  Nobody else can finish
        // these rows (a cut row needs this CTA's piece, which is never published), so they are marked here.
        do {
          if (lane == 0) {
            if (!ri.masked) write_abandoned(p, s.row, SAMPLER == 1);
            else if (s.starts) write_skipped(p, s.row, ri);
          }
        } while (sit.next(p, s, ri));
        break;
      }
      if (!s.whole && span <= 32 && !early_ok) {  // a second look, now that the own piece is complete
        bool ok = true;
        if (lane < span && kmine != (int)blockIdx.x) {
          const bool is_first_seg = quot(p, first_tile_of(p, kmine), p.tiles_per_row) == s.row;
          ok = piece_load(pieces + ((size_t)kmine * 2 + (is_first_seg ? 0 : 1)) * kPieceStride, p.call_id, early);
        }
        early_ok = __all_sync(0xffffffffu, ok);
      }
      Piece pc;
      pc.M = 0.f; pc.Z = 0.f; pc.W = 0.f; pc.zf = 0.f; pc.err = 0; pc.zmax = -CUDART_INF_F;
      Top3 top;
      top3_reset(top);
      if (lane < kStreamWarps) {
        const WarpPartial &w = sm.wpart[slot][lane];
        pc.M = w.M; pc.Z = w.Z; pc.W = w.W; pc.err = w.err; pc.zf = w.zf; pc.zmax = w.zmax;
        if (SAMPLER >= 0) {
#pragma unroll
          for (int i = 0; i < 3; ++i) { top.y[i] = w.ty[i]; top.b[i] = w.tb[i]; }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm.wfree[slot]);
      ++n;
      // The order of every merge below is fixed by lane and piece numbers alone, so the result does not
      // depend on which CTA ends up finishing the row, nor on the way it got hold of the pieces.
      warp_merge(pc, top, false);
      if (SAMPLER == 0 || (SAMPLER == 1 && ri.greedy)) warp_merge_top(top, pc.zf);
      if (timed_out(sm)) pc.err |= kErrTimeout;
      bool fin = s.whole;
      if (!s.whole) {
#pragma unroll
        for (int i = 0; i < 3; ++i) { pc.ty[i] = top.y[i]; pc.tb[i] = top.b[i]; }
        const Piece own = pc;
        if (!early_ok) {
          // Store the piece, then (after a sequentially consistent fence) look for the row's other pieces: of
          // all CTAs that hold a piece, the one whose fence comes last is sure to find them all and finishes
          // the row.  Two CTAs may both find all pieces; they then write the same values.  Nobody waits for
          // anybody.
          if (lane == 0) {
            piece_store(pieces + ((size_t)blockIdx.x * 2 + (s.slot0 ? 0 : 1)) * kPieceStride, p.call_id, own);
            asm volatile("fence.sc.gpu;" ::: "memory");
          }
          __syncwarp();
        }
        pc.M = 0.f; pc.Z = 0.f; pc.W = 0.f; pc.zf = 0.f; pc.err = 0; pc.zmax = -CUDART_INF_F;
        top3_reset(top);
        bool ok = true;
        for (int k = s.k0 + lane; k <= s.k1; k += 32) {
          Piece q;
          if (k == (int)blockIdx.x) {
            q = own;
          } else if (early_ok) {
            q = early;
          } else {
            // CTA k keeps this row's piece in slot 0 when the row is the first thing in its run
            const bool is_first_seg = quot(p, first_tile_of(p, k), p.tiles_per_row) == s.row;
            if (!piece_load(pieces + ((size_t)k * 2 + (is_first_seg ? 0 : 1)) * kPieceStride, p.call_id, q)) {
              ok = false;
              break;
            }
          }
          pc.err |= q.err;
          pc.zmax = fmaxf(pc.zmax, q.zmax);
          merge_stats_f(pc.M, pc.Z, pc.W, q.M, q.Z, q.W);
          if (SAMPLER >= 0) {
            if (q.tb[0] >= 0 && best_before(q.ty[0], q.tb[0], top.y[0], top.b[0])) pc.zf = q.zf;
#pragma unroll
            for (int i = 0; i < 3; ++i) top3_insert(top, q.ty[i], q.tb[i]);
          }
        }
        fin = __all_sync(0xffffffffu, ok);
        if (fin) warp_merge(pc, top, SAMPLER >= 0);
      }
      if (!fin) continue;
      int id = -1;
      bool have_zt = !sample && target >= 0 && target < p.V;
      if (SAMPLER >= 0) {
        id = top.b[0];
        if (!ri.greedy && id >= 0) {
          EvalCtx ex;
          ex.rk = sm.rk; ex.row = row_ptr<DT>(p, s.row); ex.tau = ri.tau; ex.slack_k = p.slack_scale;
          ex.grow = p.row_base + (uint32_t)s.row;
          ex.ctr_lo = p.ctr_lo; ex.ctr_hi8 = p.ctr_hi8; ex.seg = 0; ex.V = (int)p.V;
          if (SAMPLER == 1) {
            // the token comes from block_sample_kernel
          } else {
            // fp32 scores decide unless the runner-up is within two slacks of the leader
            zt = pc.zf;
            const float slack2 = 2.f * fmaxf(score_slack(top.y[0], p.slack_scale), score_slack(top.y[1], p.slack_scale));
            if (top.b[1] >= 0 && !(top.y[0] - top.y[1] > slack2)) {
              Top3 tcall = top;
              float zcall = zt;
              id = settle_exact<DT>(ex, tcall, slack2, lane, zcall);
              zt = zcall;
            }
          }
          have_zt = id >= 0;
        }
      }
      if (lane == 0) finish_row(p, s.row, ri, pc.M, pc.Z, pc.W, pc.zmax, id, pc.err, have_zt, zt, SAMPLER == 1);
      if (!s.whole) {
        // the row is done: nobody needs its pieces any more (a later run of this very launch must not find them)
        for (int k = s.k0 + lane; k <= s.k1; k += 32) {
          const bool is_first_seg = quot(p, first_tile_of(p, k), p.tiles_per_row) == s.row;
          piece_wipe(pieces + ((size_t)k * 2 + (is_first_seg ? 0 : 1)) * kPieceStride, p.call_id);
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Sampler 1, second kernel: one CTA of four warps per row.  It adds up the lanes of every block (the sums the
// streaming kernel left in the workspace), turns the blocks into fp32 scores Y_b = L_b + g_b (one Philox call per
// thread and round for four neighbouring blocks), keeps three leaders per thread, merges them, settles near-ties in
// fp64 and draws the token inside the winning block by inverse CDF.  Rows the streaming kernel has finished itself
// (greedy, flagged) are passed over.  It is launched behind the streaming kernel with programmatic stream
// serialization, so its start-up overlaps that kernel's tail.
// ---------------------------------------------------------------------------------------------
constexpr int kSampleWarps = 4;
template <int DT>
__global__ void __launch_bounds__(kSampleWarps * 32) block_sample_kernel(const __grid_constant__ RowsParams p) {
  using F = Fmt<DT>;
  constexpr int kBS = F::kWarpE / 256;  // blocks per tile
  constexpr int kLB = F::kLB;           // lanes per block
  __shared__ uint32_t rk[20];
  __shared__ float cand_y[kSampleWarps * 3];
  __shared__ int cand_b[kSampleWarps * 3];
  if (threadIdx.x < 20) rk[threadIdx.x] = p.round_key[threadIdx.x];
  __syncthreads();
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t row = blockIdx.x;
  const float4 st = p.ws_rowstat[row];
  if (st.z != 0.f) return;  // the whole block leaves: the record is the same for all its threads
  const float tau = __ldg(p.temps + row);
  const uint32_t grow = p.row_base + (uint32_t)row;
  const int nblocks = (int)((p.V + 255) / 256);
  const int ncalls = (nblocks + 3) / 4;
  const float *const recs = p.ws_records + row * p.tiles_per_row * kRecordFloats;
  Top3 top;
  top3_reset(top);
#pragma unroll 1
  for (int q = threadIdx.x; q < ncalls; q += kSampleWarps * 32) {
    const int b0 = 4 * q, tile = b0 / kBS, j0 = b0 % kBS;
    const float ref = __ldg(recs + tile * kRecordFloats + 32);
    const float4 *pp = reinterpret_cast<const float4 *>(recs + tile * kRecordFloats + j0 * kLB);
    float4 v[kLB];
#pragma unroll
    for (int i = 0; i < kLB; ++i) v[i] = __ldg(pp + i);
    const uint4 w = philox(rk, (uint32_t)q, grow, p.ctr_lo, p.ctr_hi8 | 2u);
    const uint32_t xw[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      float S = 0.f;
#pragma unroll
      for (int i = 0; i < kLB / 4; ++i) {
        const float4 u = v[k * (kLB / 4) + i];
        S += (u.x + u.y) + (u.z + u.w);
      }
      // ln sum_i exp(s_i) + g_b, from S = sum 2^(z c + ref); a block without mass (or beyond the row) takes no part
      if (b0 + k < nblocks && S > 0.f) top3_insert(top, (lg2f(S) - ref) * kLn2f + gumbel_from_word(xw[k]), b0 + k);
    }
  }
  float zf = 0.f;
  warp_merge_top(top, zf);
  if (lane < 3) { cand_y[warp * 3 + lane] = lane == 0 ? top.y[0] : (lane == 1 ? top.y[1] : top.y[2]);
                  cand_b[warp * 3 + lane] = lane == 0 ? top.b[0] : (lane == 1 ? top.b[1] : top.b[2]); }
  __syncthreads();
  if (warp != 0) return;
  top3_reset(top);
  if (lane < kSampleWarps * 3) top3_insert(top, cand_y[lane], cand_b[lane]);
  warp_merge_top(top, zf);
  EvalCtx ex;
  ex.rk = rk; ex.row = row_ptr<DT>(p, row); ex.tau = tau; ex.slack_k = p.slack_scale; ex.grow = grow;
  ex.ctr_lo = p.ctr_lo; ex.ctr_hi8 = p.ctr_hi8; ex.seg = 0; ex.V = (int)p.V;
  float zt = 0.f;
  const int id = sample_in_blocks<DT>(ex, top, lane, zt);
  if (lane == 0) {
    float logp = CUDART_NAN_F;
    if (id >= 0) {
      const double c = (double)__fdiv_rn(kLog2e, tau);
      logp = (float)(((double)zt * c - (double)st.x) * kLn2 - log((double)st.y));
    }
    p.out_tok[row] = id;
    if (p.out_logp) p.out_logp[row] = logp;
  }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
struct KernelSetup {
  int ctas_per_sm = 0;
  int sms = 0;
};

template <int DT, int SAMPLER>
constexpr size_t dyn_smem_bytes() {
  return (size_t)kStreamWarps * RingStages<DT, SAMPLER>::value * kWarpBytes +
         (SAMPLER == 0 ? (size_t)kStreamWarps * QueueBytes<DT>::value : 0) +
         (SAMPLER == 1 ? (size_t)kStreamWarps * kRecordBytesPerWarp : 0);
}

// Per device and kernel variant, once: opt in to the dynamic shared memory and ask how many CTAs fit an SM.
template <int DT, int SAMPLER, bool GAP>
cudaError_t setup_kernel(KernelSetup &out) {
  static std::mutex lock;
  static KernelSetup cache[64];
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> hold(lock);
  if (cache[dev].ctas_per_sm == 0) {
    auto kern = rows_kernel<DT, SAMPLER, GAP>;
    const size_t dyn = dyn_smem_bytes<DT, SAMPLER>();
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

// Test hook state (see arm_stall).
std::atomic<long long> g_stall_tile{-1};
std::atomic<unsigned long long> g_stall_wait_ns{0};

constexpr unsigned long long kDefaultWaitNs = 2000000000ull;  // two seconds

// Workspace: the pieces of cut rows first, then (sampler 1) per row a record for block_sample_kernel and per
// tile the lanes' sums with their reference.
size_t pieces_bytes() { return (size_t)kMaxGrid * 2 * kPieceBytes; }
template <int DT>
size_t partials_bytes(int64_t rows, int64_t V) {
  const int64_t tiles = (V + Fmt<DT>::kWarpE - 1) / Fmt<DT>::kWarpE;
  return (size_t)rows * 16 + (size_t)rows * tiles * (kRecordFloats * 4);
}

template <int DT, int SAMPLER, bool GAP>
cudaError_t launch_one(RowsParams p, void *workspace, size_t workspace_bytes, cudaStream_t stream) {
  KernelSetup ks;
  cudaError_t e = setup_kernel<DT, SAMPLER, GAP>(ks);
  if (e != cudaSuccess) return e;
  int64_t slots = (int64_t)ks.sms * ks.ctas_per_sm;
  if (slots > kMaxGrid) slots = kMaxGrid;
  p.tiles_per_row = (p.V + Fmt<DT>::kWarpE - 1) / Fmt<DT>::kWarpE;
  const int64_t tiles = p.rows * p.tiles_per_row;
  p.narrow = tiles < (int64_t(1) << 31) ? 1 : 0;
  if (tiles / slots >= (int64_t(1) << 30)) return cudaErrorInvalidValue;  // per-CTA tile counts are kept in 32 bits
  const bool can_cut = workspace != nullptr && workspace_bytes >= pieces_bytes();
  if (SAMPLER == 1) {
    if (!can_cut || workspace_bytes < pieces_bytes() + partials_bytes<DT>(p.rows, p.V)) return cudaErrorInvalidValue;
    unsigned char *w = static_cast<unsigned char *>(workspace) + pieces_bytes();
    p.ws_rowstat = reinterpret_cast<float4 *>(w);
    w += (size_t)p.rows * 16;
    p.ws_records = reinterpret_cast<float *>(w);
  }
  // With a response mask the cost of a row is not known on the host: with many rows, spread whole rows round-robin.
  p.interleaved = (!can_cut || (p.mask != nullptr && p.rows >= 4 * slots)) ? 1 : 0;
  int64_t grid = p.interleaved ? (p.rows < slots ? p.rows : slots) : (tiles < slots ? tiles : slots);
  p.tiles_q = tiles / grid;
  p.tiles_r = tiles % grid;
  p.ws_pieces = can_cut ? static_cast<unsigned char *>(workspace) : nullptr;
  p.call_id = next_call_id();
  p.wait_ns = kDefaultWaitNs;
  p.stall_tile = g_stall_tile.exchange(-1);
  if (p.stall_tile >= 0) p.wait_ns = g_stall_wait_ns.load();
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = dyn_smem_bytes<DT, SAMPLER>();
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  e = cudaLaunchKernelEx(&cfg, rows_kernel<DT, SAMPLER, GAP>, p);
  if (e != cudaSuccess || SAMPLER != 1) return e;
  cfg.gridDim = dim3((unsigned)p.rows);
  cfg.blockDim = dim3(kSampleWarps * 32);
  cfg.dynamicSmemBytes = 0;
  return cudaLaunchKernelEx(&cfg, block_sample_kernel<DT>, p);
}

template <int DT, int SAMPLER>
cudaError_t launch_gap(const RowsParams &p, void *workspace, size_t workspace_bytes, cudaStream_t stream) {
  return p.out_gap ? launch_one<DT, SAMPLER, true>(p, workspace, workspace_bytes, stream)
                   : launch_one<DT, SAMPLER, false>(p, workspace, workspace_bytes, stream);
}

}  // namespace

size_t rows_workspace_bytes() { return pieces_bytes(); }
size_t sample_workspace_bytes(int dtype, int64_t rows, int64_t V) {
  if (rows < 0 || V < 1) return pieces_bytes();
  return pieces_bytes() + (dtype == 0 ? partials_bytes<0>(rows, V) : partials_bytes<1>(rows, V));
}

void arm_stall(int64_t stall_tile, unsigned long long wait_ns) {
  g_stall_wait_ns.store(wait_ns);
  g_stall_tile.store(stall_tile);
}

cudaError_t launch_rows(RowsParams p, int dtype, int sampler, bool aligned, void *workspace, size_t workspace_bytes,
                        cudaStream_t stream) {
  p.bulk = aligned ? 1 : 0;
  if (dtype == 0) {
    if (sampler < 0) return launch_gap<0, -1>(p, workspace, workspace_bytes, stream);
    if (sampler == 0) return launch_gap<0, 0>(p, workspace, workspace_bytes, stream);
    if (sampler == 1) return launch_gap<0, 1>(p, workspace, workspace_bytes, stream);
  } else if (dtype == 1) {
    if (sampler < 0) return launch_gap<1, -1>(p, workspace, workspace_bytes, stream);
    if (sampler == 0) return launch_gap<1, 0>(p, workspace, workspace_bytes, stream);
    if (sampler == 1) return launch_gap<1, 1>(p, workspace, workspace_bytes, stream);
  }
  return cudaErrorInvalidValue;
}

}  // namespace e3
