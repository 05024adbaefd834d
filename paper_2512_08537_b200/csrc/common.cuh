// Small host-side helpers shared by the translation units of libardiff.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/ardiff.h"

namespace ardiff {

// launches enqueued by the last gate / head call on this host thread
void set_launch_count(int n);
int get_launch_count();

// cta_stats / stats_out3: both NULL, or scratch for 3 doubles per block and the device address of
// {mean, std, 0.3 mean - 0.1 std} of the entropies
int gate_launch(const void* feat, int64_t n, int32_t d, float tau, uint8_t* mask, int32_t* idx,
                int32_t* count, float* entropy, int32_t* block_counts, double* cta_stats, double* stats_out3,
                int max_blocks, int n_sm, cudaStream_t st);
int gate_blocks_fused_launch(const void* feat, int64_t n, int32_t r, int32_t d, int32_t gamma, float tau,
                             float* row_entropy, float* token_entropy, uint8_t* mask, int32_t* idx, int32_t* count,
                             int32_t* block_len, int32_t* cta_counts, int max_blocks, int n_sm, cudaStream_t st);

int entropy_rows_launch(const void* feat, int64_t rows, int32_t d, float* entropy, int n_sm, cudaStream_t st);
int compact_launch(const uint8_t* mask, int64_t n, const int32_t* block_counts, int64_t tokens_per_block, int grid,
                   int32_t* idx, int32_t* count, cudaStream_t st);
// per-block count scratch of the allocating gate calls: a slice private to `st` on the current device
int gate_scratch_get(cudaStream_t st, int32_t** counts, int* max_blocks, int* sms);
int write_zero_count(int32_t* count, cudaStream_t st);

// shape of a head (for callers that must match their buffers to it)
const ardiff_head_desc* head_desc(const ardiff_head* head);

}  // namespace ardiff
