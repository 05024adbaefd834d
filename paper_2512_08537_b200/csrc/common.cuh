// Small host-side helpers shared by the translation units of libardiff.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace ardiff {

// launches enqueued by the last gate / head call on this host thread
void set_launch_count(int n);
int get_launch_count();

int gate_launch(const void* feat, int64_t n, int32_t d, float tau, uint8_t* mask, int32_t* idx,
                int32_t* count, float* entropy, int32_t* block_counts, int max_blocks, int n_sm,
                cudaStream_t st);

}  // namespace ardiff
