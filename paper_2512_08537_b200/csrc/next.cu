// Later stages of the entropy-gated pipeline, built on the row-entropy kernel of gate.cu:
//   ardiff_entropy_gate_blocks  the early stop of Algorithm 1, Step 1 as written: per draft block, the
//                               first token whose indicator falls below tau drops itself and the rest
//                               of the block; the indicator is the mean of the token's row entropies
//                               (the entropy-loss equation's mean over rows and heads);
//   ardiff_tau_calibrate        the threshold equation tau = 0.3 mean(H) - 0.1 std(H);
//   ardiff_accept_prefix        Algorithm 1, Step 4: accepted draft length per block.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "../../include/ardiff.h"
#include "common.cuh"

namespace {

constexpr int kThreads = 256;

// One thread per draft block: token indicators (mean over rows_per_token row entropies, summed in row
// order), prefix test, mask, kept length. A CTA covers blocks_per_cta consecutive blocks and leaves
// its kept-token count for the compaction pass.
__global__ void __launch_bounds__(kThreads)
block_prefix_kernel(const float* __restrict__ row_entropy, int64_t n, int32_t r, int32_t gamma, float tau,
                    float* __restrict__ token_entropy, uint8_t* __restrict__ mask, int32_t* __restrict__ block_len,
                    int32_t* __restrict__ cta_counts, int64_t blocks_per_cta, int64_t n_blocks) {
    __shared__ int s_cnt[kThreads / 32];
    int kept_total = 0;
    const int64_t b_begin = (int64_t)blockIdx.x * blocks_per_cta;
    const int64_t b_end = min(n_blocks, b_begin + blocks_per_cta);
    for (int64_t b = b_begin + threadIdx.x; b < b_end; b += kThreads) {
        const int64_t t0 = b * gamma;
        const int64_t t1 = min(n, t0 + gamma);
        bool speculate = true;
        int kept = 0;
        const float inv = 1.0f / (float)r;
        for (int64_t t = t0; t < t1; ++t) {
            const float* src = row_entropy + t * r;
            float acc = 0.f;
            for (int j = 0; j < r; ++j) acc += src[j];
            const float hs = acc * inv;
            if (token_entropy) token_entropy[t] = hs;
            if (speculate && !(hs >= tau)) speculate = false;   // H < tau, or NaN
            mask[t] = speculate ? 1 : 0;
            kept += speculate ? 1 : 0;
        }
        if (block_len) block_len[b] = kept;
        kept_total += kept;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) kept_total += __shfl_xor_sync(0xffffffffu, kept_total, o);
    if ((threadIdx.x & 31) == 0) s_cnt[threadIdx.x >> 5] = kept_total;
    __syncthreads();
    if (threadIdx.x == 0) {
        int tot = 0;
        for (int w = 0; w < kThreads / 32; ++w) tot += s_cnt[w];
        cta_counts[blockIdx.x] = tot;
    }
}

// mean, standard deviation (divisor n) and tau of n entropies; one CTA, fp64, fixed summation order
// (thread-strided partial sums, then a tree), two passes so that the deviations are taken from the mean.
__global__ void __launch_bounds__(1024) tau_kernel(const float* __restrict__ H, int64_t n, double* __restrict__ out) {
    __shared__ double s[1024];
    __shared__ double s_mean;
    double acc = 0.0;
    for (int64_t i = threadIdx.x; i < n; i += 1024) acc += (double)H[i];
    s[threadIdx.x] = acc;
    __syncthreads();
    for (int o = 512; o > 0; o >>= 1) {
        if (threadIdx.x < o) s[threadIdx.x] += s[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) s_mean = s[0] / (double)n;
    __syncthreads();
    const double mean = s_mean;
    acc = 0.0;
    for (int64_t i = threadIdx.x; i < n; i += 1024) {
        const double dlt = (double)H[i] - mean;
        acc += dlt * dlt;
    }
    s[threadIdx.x] = acc;
    __syncthreads();
    for (int o = 512; o > 0; o >>= 1) {
        if (threadIdx.x < o) s[threadIdx.x] += s[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const double sd = sqrt(s[0] / (double)n);
        out[0] = mean;
        out[1] = sd;
        out[2] = 0.3 * mean - 0.1 * sd;
    }
}

__global__ void __launch_bounds__(kThreads)
accept_prefix_kernel(const float* __restrict__ r, const float* __restrict__ ratio, int64_t n, int32_t gamma,
                     int64_t n_blocks, const int32_t* __restrict__ block_len, int32_t* __restrict__ accepted) {
    const int64_t b = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (b >= n_blocks) return;
    const int64_t t0 = b * gamma;
    int64_t t1 = min(n, t0 + gamma);
    // the draft that reaches Step 4 is what Step 1 left of the block
    if (block_len) t1 = min(t1, t0 + (int64_t)max(block_len[b], 0));
    int acc = (int)(t1 - t0);
    for (int64_t t = t0; t < t1; ++t) {
        if (r[t] > ratio[t]) {
            acc = (int)(t - t0);
            break;
        }
    }
    accepted[b] = acc;
}

}  // namespace

extern "C" int ardiff_entropy_gate_blocks(const void* feat, int64_t n, int32_t rows_per_token, int32_t d,
                                          int32_t gamma, float tau, float* row_entropy, float* token_entropy,
                                          uint8_t* mask, int32_t* idx, int32_t* count, int32_t* block_len,
                                          void* stream) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!count) return ARDIFF_ERR_NULL;
    if (n < 0 || rows_per_token < 1 || gamma < 1 || d < 1 || d > 65536) return ARDIFF_ERR_SHAPE;
    if (n >= (int64_t)1 << 31 || n * (int64_t)rows_per_token >= (int64_t)1 << 31) return ARDIFF_ERR_SHAPE;
    if (n == 0) {
        ardiff::set_launch_count(1);
        return ardiff::write_zero_count(count, st);
    }
    if (!feat || !mask || !idx) return ARDIFF_ERR_NULL;
    int32_t* counts = nullptr;
    int max_blocks = 0, sms = 0;
    int rc = ardiff::gate_scratch_get(st, &counts, &max_blocks, &sms);
    if (rc != ARDIFF_OK) return rc;
    // one pass over the features when the shape allows it; else row entropies through global memory
    rc = ardiff::gate_blocks_fused_launch(feat, n, rows_per_token, d, gamma, tau, row_entropy, token_entropy, mask,
                                          idx, count, block_len, counts, max_blocks, sms, st);
    if (rc != ARDIFF_ERR_UNSUPPORTED) return rc;
    if (!row_entropy) return ARDIFF_ERR_NULL;      // this path needs it as scratch
    rc = ardiff::entropy_rows_launch(feat, n * rows_per_token, d, row_entropy, sms, st);
    if (rc != ARDIFF_OK) return rc;
    // CTAs own whole draft blocks, so a block never straddles two compaction ranges
    const int64_t n_blocks = (n + gamma - 1) / gamma;
    int64_t want = (int64_t)sms * 4;
    if (want > max_blocks) want = max_blocks;
    int64_t bpc = (n_blocks + want - 1) / want;
    if (bpc < 1) bpc = 1;
    const int grid = (int)((n_blocks + bpc - 1) / bpc);
    block_prefix_kernel<<<grid, kThreads, 0, st>>>(row_entropy, n, rows_per_token, gamma, tau, token_entropy, mask,
                                                   block_len, counts, bpc, n_blocks);
    if (cudaGetLastError() != cudaSuccess) return ARDIFF_ERR_CUDA;
    rc = ardiff::compact_launch(mask, n, counts, bpc * gamma, grid, idx, count, st);
    ardiff::set_launch_count(3);
    return rc;
}

extern "C" int ardiff_tau_calibrate(const float* entropy, int64_t n, double* out3, void* stream) {
    if (!entropy || !out3) return ARDIFF_ERR_NULL;
    if (n < 1) return ARDIFF_ERR_SHAPE;
    tau_kernel<<<1, 1024, 0, static_cast<cudaStream_t>(stream)>>>(entropy, n, out3);
    ardiff::set_launch_count(1);
    return cudaGetLastError() == cudaSuccess ? ARDIFF_OK : ARDIFF_ERR_CUDA;
}

extern "C" int ardiff_accept_prefix(const float* r, const float* ratio, int64_t n, int32_t gamma,
                                    const int32_t* block_len, int32_t* accepted, void* stream) {
    if (n < 0 || gamma < 1) return ARDIFF_ERR_SHAPE;
    if (n == 0) return ARDIFF_OK;
    if (!r || !ratio || !accepted) return ARDIFF_ERR_NULL;
    const int64_t n_blocks = (n + gamma - 1) / gamma;
    const int grid = (int)((n_blocks + kThreads - 1) / kThreads);
    accept_prefix_kernel<<<grid, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(r, ratio, n, gamma, n_blocks,
                                                                                 block_len, accepted);
    ardiff::set_launch_count(1);
    return cudaGetLastError() == cudaSuccess ? ARDIFF_OK : ARDIFF_ERR_CUDA;
}
