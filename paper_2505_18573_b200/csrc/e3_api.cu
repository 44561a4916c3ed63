// C ABI of the device calls: argument checks, parameter marshalling, launches.
#include <cuda_runtime.h>
#include <stdint.h>

#include "e3.h"
#include "e3_rows.cuh"
#include "e3_small.cuh"

namespace e3 {
size_t grpo_workspace_bytes(int64_t n_seq);
}

namespace {

inline bool misaligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) != 0; }

e3_status check_logits(const void *logits, e3_dtype dt, int64_t rows, int64_t V, int64_t row_stride) {
  if (dt != E3_F32 && dt != E3_BF16) return E3_ERR_DTYPE;
  if (rows < 0 || V < 1 || V >= (int64_t(1) << 31) || row_stride < V) return E3_ERR_INVALID_ARG;
  if (rows > 0 && !logits) return E3_ERR_INVALID_ARG;
  if (misaligned(logits, dt == E3_F32 ? 4 : 2)) return E3_ERR_ALIGNMENT;
  return E3_OK;
}

bool rows_are_16B_aligned(const void *logits, e3_dtype dt, int64_t row_stride) {
  const int64_t esize = dt == E3_F32 ? 4 : 2;
  return !misaligned(logits, 16) && (row_stride * esize) % 16 == 0;
}

void philox_round_keys(uint64_t seed, uint32_t rk[20]) {
  uint32_t k0 = static_cast<uint32_t>(seed), k1 = static_cast<uint32_t>(seed >> 32);
  for (int r = 0; r < 10; ++r) {
    rk[2 * r] = k0;
    rk[2 * r + 1] = k1;
    k0 += 0x9E3779B9u;  // Weyl increments of the Philox key schedule
    k1 += 0xBB67AE85u;
  }
}

// e3_token_logp_entropy: the pieces of cut rows, then the partial sums of the fused mean entropy.
size_t token_mean_offset() { return e3::rows_workspace_bytes(); }

}  // namespace

extern "C" size_t e3_workspace_bytes(e3_call which, int64_t rows, int64_t V, e3_dtype dt) {
  switch (which) {
    case E3_CALL_SAMPLE: return e3::sample_workspace_bytes(static_cast<int>(dt), rows, V);
    case E3_CALL_TOKEN_LOGP_ENTROPY: return token_mean_offset() + e3::mean_workspace_bytes(rows < 0 ? 0 : rows);
    case E3_CALL_MASKED_MEAN_ENTROPY: return e3::mean_workspace_bytes(rows < 0 ? 0 : rows);
    case E3_CALL_GRPO_OBJECTIVE: return e3::grpo_workspace_bytes(rows);
    case E3_CALL_SEQUENCE_MEAN_ENTROPY: return e3::seq_mean_workspace_bytes(rows);
  }
  return 0;
}

extern "C" e3_status e3_sample(const void *logits, e3_dtype dt, int64_t rows, int64_t V, int64_t row_stride,
                               const float *temps, uint64_t seed, uint64_t counter, int64_t row_base,
                               e3_sampler sampler, int32_t *out_tok, float *out_logp, float *out_ent, float *out_gap,
                               int32_t *out_status, void *workspace, size_t workspace_bytes, void *stream) {
  e3_status st = check_logits(logits, dt, rows, V, row_stride);
  if (st != E3_OK) return st;
  if (misaligned(workspace, 16)) return E3_ERR_ALIGNMENT;
  if (sampler != E3_SAMPLER_TOKEN && sampler != E3_SAMPLER_BLOCK && sampler != E3_SAMPLER_TOKEN_AUDIT)
    return E3_ERR_INVALID_ARG;
  // the row number that enters the random stream is a 32-bit counter word
  if (row_base < 0 || row_base + rows > (int64_t(1) << 32) || counter >= (uint64_t(1) << 56)) return E3_ERR_INVALID_ARG;
  if (rows == 0) return E3_OK;
  if (!temps || !out_tok) return E3_ERR_INVALID_ARG;
  if (misaligned(temps, 4) || misaligned(out_tok, 4) || misaligned(out_logp, 4) || misaligned(out_ent, 4) ||
      misaligned(out_gap, 4) || misaligned(out_status, 4))
    return E3_ERR_ALIGNMENT;
  if (sampler == E3_SAMPLER_BLOCK &&
      (!workspace || workspace_bytes < e3::sample_workspace_bytes(static_cast<int>(dt), rows, V)))
    return E3_ERR_WORKSPACE;

  e3::RowsParams p = {};
  p.logits = logits; p.rows = rows; p.V = V; p.row_stride = row_stride;
  p.temps = temps; p.temp_scalar = 1.f;
  p.out_tok = out_tok; p.out_logp = out_logp; p.out_ent = out_ent; p.out_gap = out_gap; p.status = out_status;
  philox_round_keys(seed, p.round_key);
  p.ctr_lo = static_cast<uint32_t>(counter);
  p.ctr_hi8 = static_cast<uint32_t>(counter >> 32) << 8;
  p.row_base = static_cast<uint32_t>(row_base);
  p.mode = e3::kModeSample;
  p.slack_scale = sampler == E3_SAMPLER_TOKEN_AUDIT ? 1000.f : 1.f;
  cudaError_t e = e3::launch_rows(p, static_cast<int>(dt), sampler == E3_SAMPLER_BLOCK ? 1 : 0,
                                  rows_are_16B_aligned(logits, dt, row_stride), workspace, workspace_bytes,
                                  static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? E3_OK : E3_ERR_CUDA;
}

extern "C" e3_status e3_token_logp_entropy(const void *logits, e3_dtype dt, int64_t rows, int64_t V,
                                           int64_t row_stride, const int32_t *targets, const uint8_t *mask,
                                           const float *temps, float temp_scalar, float *out_logp, float *out_ent,
                                           float *out_gap, double *out_ent_sum, double *out_count,
                                           int32_t *out_status, void *workspace, size_t workspace_bytes,
                                           void *stream) {
  e3_status st = check_logits(logits, dt, rows, V, row_stride);
  if (st != E3_OK) return st;
  if (misaligned(workspace, 16)) return E3_ERR_ALIGNMENT;
  const bool fused_mean = out_ent_sum != nullptr || out_count != nullptr;
  if (fused_mean && (!out_ent_sum || !out_count || (rows > 0 && !out_ent))) return E3_ERR_INVALID_ARG;
  if (misaligned(out_ent_sum, 8) || misaligned(out_count, 8)) return E3_ERR_ALIGNMENT;
  if (fused_mean && (!workspace || workspace_bytes < token_mean_offset() + e3::mean_workspace_bytes(rows)))
    return E3_ERR_WORKSPACE;
  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  if (rows == 0) {
    if (!fused_mean) return E3_OK;
    cudaError_t e0 = e3::launch_masked_mean(nullptr, nullptr, 0, out_ent_sum, out_count,
                                            static_cast<unsigned char *>(workspace) + token_mean_offset(), true, cs);
    return e0 == cudaSuccess ? E3_OK : E3_ERR_CUDA;
  }
  if (!targets) return E3_ERR_INVALID_ARG;
  if (misaligned(targets, 4) || misaligned(temps, 4) || misaligned(out_logp, 4) || misaligned(out_ent, 4) ||
      misaligned(out_gap, 4) || misaligned(out_status, 4))
    return E3_ERR_ALIGNMENT;

  e3::RowsParams p = {};
  p.logits = logits; p.rows = rows; p.V = V; p.row_stride = row_stride;
  p.temps = temps; p.temp_scalar = temp_scalar;
  p.targets = targets; p.mask = mask;
  p.out_logp = out_logp; p.out_ent = out_ent; p.out_gap = out_gap; p.status = out_status;
  p.mode = e3::kModeTargets;
  p.slack_scale = 1.f;
  cudaError_t e = e3::launch_rows(p, static_cast<int>(dt), -1, rows_are_16B_aligned(logits, dt, row_stride),
                                  workspace, workspace_bytes < token_mean_offset() ? workspace_bytes : token_mean_offset(),
                                  cs);
  // The fused mean entropy: the two reduction kernels of e3_masked_mean_entropy behind the row kernel, chained by
  // programmatic dependent launch; the same blocks add the same values in the same order.
  if (e == cudaSuccess && fused_mean)
    e = e3::launch_masked_mean(out_ent, mask, rows, out_ent_sum, out_count,
                               static_cast<unsigned char *>(workspace) + token_mean_offset(), true, cs);
  return e == cudaSuccess ? E3_OK : E3_ERR_CUDA;
}

extern "C" e3_status e3_masked_mean_entropy(const float *ent, const uint8_t *mask, int64_t n, double *out_mean,
                                            double *out_count, void *workspace, size_t workspace_bytes,
                                            void *stream) {
  if (n < 0 || !out_mean || !out_count || (n > 0 && !ent)) return E3_ERR_INVALID_ARG;
  if (misaligned(ent, 4) || misaligned(out_mean, 8) || misaligned(out_count, 8) || misaligned(workspace, 8))
    return E3_ERR_ALIGNMENT;
  if (!workspace || workspace_bytes < e3::mean_workspace_bytes(n)) return E3_ERR_WORKSPACE;
  cudaError_t e = e3::launch_masked_mean(ent, mask, n, out_mean, out_count, workspace, false,
                                         static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? E3_OK : E3_ERR_CUDA;
}

extern "C" e3_status e3_sequence_mean_entropy(const float *ent, const uint8_t *mask, int64_t n_seq, int64_t seq_len,
                                              double *out_mean, double *out_count, void *workspace,
                                              size_t workspace_bytes, void *stream) {
  if (n_seq < 0 || seq_len < 0 || n_seq >= (int64_t(1) << 31) || !out_mean || !out_count ||
      (n_seq > 0 && seq_len > 0 && !ent))
    return E3_ERR_INVALID_ARG;
  if (misaligned(ent, 4) || misaligned(out_mean, 8) || misaligned(out_count, 8) || misaligned(workspace, 8))
    return E3_ERR_ALIGNMENT;
  if (!workspace || workspace_bytes < e3::seq_mean_workspace_bytes(n_seq)) return E3_ERR_WORKSPACE;
  cudaError_t e = e3::launch_sequence_mean(ent, mask, n_seq, seq_len, out_mean, out_count, workspace,
                                           static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? E3_OK : E3_ERR_CUDA;
}

extern "C" e3_status e3_group_advantage(const float *rewards, const int64_t *group_offsets, int64_t n_groups,
                                        float eps, int unbiased, float *out_adv, uint8_t *out_group_flags,
                                        void *stream) {
  if (n_groups < 0 || !(eps >= 0.f) || !(eps < 3.0e38f)) return E3_ERR_INVALID_ARG;
  if (n_groups == 0) return E3_OK;
  if (!rewards || !group_offsets || !out_adv) return E3_ERR_INVALID_ARG;
  if (misaligned(rewards, 4) || misaligned(group_offsets, 8) || misaligned(out_adv, 4)) return E3_ERR_ALIGNMENT;
  cudaError_t e = e3::launch_group_advantage(rewards, group_offsets, n_groups, eps, unbiased, out_adv,
                                             out_group_flags, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? E3_OK : E3_ERR_CUDA;
}

extern "C" void e3_test_arm_stall(int64_t tile, uint64_t wait_ns) { e3::arm_stall(tile, wait_ns); }
