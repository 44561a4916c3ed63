// Host-side launchers of the small device steps (masked mean entropy, group advantage).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace e3 {

size_t mean_workspace_bytes(int64_t n);
cudaError_t launch_masked_mean(const float *ent, const uint8_t *mask, int64_t n, double *out_mean,
                               double *out_count, void *workspace, bool want_sum, cudaStream_t stream);
size_t seq_mean_workspace_bytes(int64_t n_seq);
cudaError_t launch_sequence_mean(const float *ent, const uint8_t *mask, int64_t n_seq, int64_t seq_len,
                                 double *out_mean, double *out_count, void *workspace, cudaStream_t stream);
cudaError_t launch_group_advantage(const float *rewards, const int64_t *off, int64_t n_groups, float eps,
                                   int unbiased, float *adv, uint8_t *flags, cudaStream_t stream);

}  // namespace e3
