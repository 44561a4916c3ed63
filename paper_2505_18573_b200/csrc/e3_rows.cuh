// Shared declarations of the row-streaming kernel (host side of the launch and device parameters).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace e3 {

constexpr int kStreamWarps = 8;                     // warps that consume logits
constexpr int kStreamThreads = kStreamWarps * 32;   // 256
constexpr int kThreads = kStreamThreads + 64;       // + one warp that issues bulk copies + one that finishes rows
constexpr int kGroup = 16;                          // vocabulary entries per coarse Philox call
constexpr int kTile = 512;                          // unit of the work split (entries); CTA ranges start on tile bounds
constexpr int kLaneBytes = 64;                      // bytes a consumer thread takes from one pipeline stage
constexpr int kStageBytes = kStreamThreads * kLaneBytes;  // 16 KiB per pipeline stage (one bulk copy)
constexpr int kStages = 4;
constexpr int kMaxGrid = 1024;                      // CTAs the piece workspace is sized for
constexpr size_t kPieceBytes = 128;                 // one partial row state in the workspace

enum RowsMode : int { kModeSample = 0, kModeTargets = 1 };

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
  uint32_t round_key[20];   // Philox round keys: key_lo + r*W0, key_hi + r*W1, r = 0..9
  uint32_t ctr_lo;          // low word of the step counter
  uint32_t ctr_hi8;         // (high bits of the step counter) << 8; the stream tag is OR-ed in
  uint32_t row_base;
  int mode;
  float slack_scale;        // 1; the audit sampler widens the fp32 score slack so that rows are settled in fp64
  // work split
  int interleaved;          // 1: CTA b takes whole rows b, b + grid, ...; 0: contiguous tile ranges (rows may be cut)
  int narrow;               // 1: every tile number fits in 31 bits (32-bit index arithmetic on the device)
  int64_t tiles_per_row;    // ceil(V / kTile)
  int64_t tiles_q, tiles_r; // total tiles = grid * tiles_q + tiles_r: CTA b starts at tile b*tiles_q + min(b, tiles_r)
  // cut rows: partial states in the caller's workspace
  unsigned char *ws_pieces;          // [grid][2] pieces of kPieceBytes, every word tagged with the call id
  unsigned long long call_id;        // unique per call within the process (48 bits)
  int rehearse;                      // pass of the finishing warp that is a dry run (0), -1: none
};

size_t rows_workspace_bytes();

// Launches the streaming kernel.  sampler: -1 = none (targets given), 0 = per-token Gumbel-max,
// 1 = blocked Gumbel-max (the caller sets slack_scale).  workspace may be nullptr: rows are then never cut (whole rows per CTA).
cudaError_t launch_rows(RowsParams p, int dtype, int sampler, bool aligned, void *workspace, size_t workspace_bytes,
                        cudaStream_t stream);

}  // namespace e3
