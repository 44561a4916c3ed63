// Shared declarations of the row-streaming kernels (host side of the launch and device parameters).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace e3 {

constexpr int kStreamWarps = 8;                     // warps that stream logits
constexpr int kStreamThreads = kStreamWarps * 32;   // 256
constexpr int kThreads = kStreamThreads + 32;       // + one warp that finishes rows
constexpr int kGroup = 16;                          // vocabulary entries per coarse Philox call
constexpr int kSliceAlign = 512;                    // a CTA's slice of a row starts on a multiple of this
constexpr int kMaxCluster = 8;

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
  int64_t seg;              // vocabulary entries per CTA of a cluster (multiple of kSliceAlign)
  int mode;
};

// Launches the streaming kernel for the given element type / sampler.  sampler: -1 = none (targets given).
cudaError_t launch_rows(const RowsParams &p, int dtype, int sampler, bool aligned, cudaStream_t stream);

}  // namespace e3
