// Shared declarations of the row-streaming kernels (host side of the launch and device parameters).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace e3 {

constexpr int kStreamWarps = 8;                     // warps that consume logits
constexpr int kStreamThreads = kStreamWarps * 32;   // 256
constexpr int kThreads = kStreamThreads + 64;       // + one warp that feeds the rings + one that finishes rows
constexpr int kGroup = 16;                          // vocabulary entries per coarse Philox call
constexpr int kLaneBytes = 128;                     // bytes a consumer thread takes from one ring slot
constexpr int kWarpBytes = 32 * kLaneBytes;         // 4 KiB: one ring slot (a "tile"), and the unit of the work split
constexpr int kStages = 3;                          // ring slots per consumer warp
constexpr int kMaxGrid = 1024;                      // CTAs the piece workspace is sized for
constexpr size_t kPieceBytes = 128;                 // one partial row state in the workspace
constexpr int kRecordFloats = 36;                   // blocked sampler: per tile 32 lane sums + reference, padded to 144 bytes

enum RowsMode : int { kModeSample = 0, kModeTargets = 1 };

// Bits of the optional device status word.
enum : int { kStatusTimeout = 1 };

struct RowsParams {
  const void *logits;
  int64_t rows, V, row_stride;
  const float *temps;       // per-row temperature, or nullptr -> temp_scalar
  float temp_scalar;
  const int32_t *targets;   // kModeTargets
  const uint8_t *mask;      // kModeTargets, may be nullptr
  int32_t *out_tok;         // kModeSample
  float *out_logp;
  float *out_ent;
  float *out_gap;           // may be nullptr
  int32_t *status;          // may be nullptr: kStatusTimeout is OR-ed in when a bounded wait ran out
  uint32_t round_key[20];   // Philox round keys: key_lo + r*W0, key_hi + r*W1, r = 0..9
  uint32_t ctr_lo;          // low word of the step counter
  uint32_t ctr_hi8;         // (high bits of the step counter) << 8; the stream tag is OR-ed in
  uint32_t row_base;
  int mode;
  float slack_scale;        // 1; the audit sampler widens the fp32 score slack so that rows are settled in fp64
  int bulk;                 // 1: rows start on 16-byte boundaries (bulk asynchronous copies), 0: element-wise copies
  // work split
  int interleaved;          // 1: CTA b takes whole rows b, b + grid, ...; 0: contiguous tile ranges (rows may be cut)
  int narrow;               // 1: every tile number fits in 31 bits (32-bit index arithmetic on the device)
  int64_t tiles_per_row;    // ceil(V / entries per tile); a tile is kWarpBytes of logits
  int64_t tiles_q, tiles_r; // total tiles = grid * tiles_q + tiles_r: CTA b starts at tile b*tiles_q + min(b, tiles_r)
  // cut rows: partial states in the caller's workspace
  unsigned char *ws_pieces;          // [grid][2] pieces of kPieceBytes, every word tagged with the call id
  // blocked sampler: what the streaming kernel leaves for block_sample_kernel
  float4 *ws_rowstat;                // [rows] reference, sum of 2^t, non-zero = row finished or flagged
  float *ws_records;                 // [rows][tiles_per_row][kRecordFloats]: every lane's sum of 2^t over its 128 bytes
                                     // of the tile (32 floats), then the reference the sums refer to, then padding
  unsigned long long call_id;        // unique per call within the process (48 bits)
  unsigned long long wait_ns;        // time after which a wait inside the kernel gives up
  int64_t stall_tile;                // test hook: the copy of this tile (row * tiles_per_row + tile in row) is never issued; -1 = none
};

size_t rows_workspace_bytes();                                      // cut rows only
size_t sample_workspace_bytes(int dtype, int64_t rows, int64_t V);  // e3_sample (covers the blocked sampler)

// Test hook: the next launch_rows of this process gives up waiting after wait_ns and never issues the copy of
// tile stall_tile.  One shot.
void arm_stall(int64_t stall_tile, unsigned long long wait_ns);

// Launches the streaming kernel (and, for the blocked sampler, block_sample_kernel behind it).
// sampler: -1 = none (targets given), 0 = per-token Gumbel-max, 1 = blocked Gumbel-max (the caller sets slack_scale).
// workspace may be nullptr unless sampler == 1: rows are then never cut (whole rows per CTA).
cudaError_t launch_rows(RowsParams p, int dtype, int sampler, bool aligned, void *workspace, size_t workspace_bytes,
                        cudaStream_t stream);

}  // namespace e3
