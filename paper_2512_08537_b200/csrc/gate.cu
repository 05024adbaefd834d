// Entropy gate + stream compaction for sm_100a.
//
// Kernel 1 (gate_rows_kernel): one warp per token. The whole bf16 row is fetched with
// 128-bit streaming loads into registers (one HBM pass), the row maximum is taken with packed
// bf16x2 max, then S = sum 2^t and T = sum t 2^t with t = (x - m) log2(e) are accumulated in
// fp32, and H = ln S - ln2 * T / S. The warp writes the mask byte (and the entropy, if asked)
// and each block leaves its number of kept tokens in a small scratch array.
// Kernel 2 (compact_kernel): every block sums the counts of the blocks before it and writes the
// ascending token ids of its own contiguous token range (ballot + prefix), the last block
// writes the total.
//
// Definition being computed: the softmax-row entropy indicator of the paper's entropy-informed
// speculative decoding (H = -L_entropy of one row, natural log) and Algorithm 1's threshold test
// (a token is dropped iff H < tau).
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <string.h>
#include <math_constants.h>
#include <stdint.h>

#include <mutex>
#include <type_traits>

#include "../../include/ardiff.h"
#include "common.cuh"

namespace {

constexpr int kGateThreads = 256;
constexpr int kGateWarps = kGateThreads / 32;
constexpr int kMaxGateBlocks = 4096;  // capacity of the per-device block-count scratch
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ uint4 ld_stream_v4(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// NaN-propagating packed max of two bf16 pairs held in 32-bit words
__device__ __forceinline__ uint32_t max_bf16x2_nan(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ float warp_max_nan(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        float other = __shfl_xor_sync(0xffffffffu, v, o);
        // NaN-propagating max
        v = (v != v || other != other) ? CUDART_NAN_F : fmaxf(v, other);
    }
    return v;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// accumulate one 32-bit word (two bf16 values) into S and T; mneg = -m*log2e
__device__ __forceinline__ void acc_word(uint32_t w, float mneg, float& S, float& T) {
    float t0 = fmaf(bf16_lo(w), kLog2e, mneg);
    float t1 = fmaf(bf16_hi(w), kLog2e, mneg);
    float e0 = ex2_approx(t0);
    float e1 = ex2_approx(t1);
    S += e0;
    S += e1;
    T = fmaf(t0, e0, T);
    T = fmaf(t1, e1, T);
}

// Slow exact-semantics path for one row: used when the fast path meets a non-finite
// intermediate (a -inf channel makes t*e = -inf*0). Re-reads the row from memory (rare), so the
// register-resident copy of the fast path never needs an address. Terms with e == 0 contribute 0.
__device__ __noinline__ float row_entropy_careful(const uint4* row, int nchunks, int lane, float m) {
    float S = 0.f, T = 0.f;
    const float mneg = -m * kLog2e;
    for (int c = lane; c < nchunks; c += 32) {
        const uint4 v = ld_stream_v4(row + c);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float t0 = fmaf(bf16_lo(w[q]), kLog2e, mneg), t1 = fmaf(bf16_hi(w[q]), kLog2e, mneg);
            float e0 = ex2_approx(t0), e1 = ex2_approx(t1);
            S += e0 + e1;
            if (e0 > 0.f || e0 != e0) T = fmaf(t0, e0, T);
            if (e1 > 0.f || e1 != e1) T = fmaf(t1, e1, T);
        }
    }
    S = warp_sum(S);
    T = warp_sum(T);
    return logf(S) - kLn2 * (T / S);
}

// Entropy of the row held in v (NCH 16-byte chunks per lane). Each chunk is refilled with the warp's NEXT row
// as soon as the exponentials of the current row have consumed it, so a warp always has loads in flight while
// it computes (with 128 registers per thread only 16 warps fit an SM: they cannot hide HBM latency by
// switching alone).
template <int NCH>
__device__ __forceinline__ float resident_row_entropy(uint4 (&v)[NCH], const uint4* row, const uint4* next_row,
                                                      bool has_next, int32_t nchunks, int lane) {
    // row maximum (packed, exact in bf16)
    uint32_t mx = 0xff80ff80u;
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
        mx = max_bf16x2_nan(mx, max_bf16x2_nan(max_bf16x2_nan(v[j].x, v[j].y), max_bf16x2_nan(v[j].z, v[j].w)));
    }
    float ml = bf16_lo(mx), mh = bf16_hi(mx);
    float m = (ml != ml || mh != mh) ? CUDART_NAN_F : fmaxf(ml, mh);
    m = warp_max_nan(m);
    const float mneg = -m * kLog2e;
    float S = 0.f, T = 0.f;
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
        const int c = lane + 32 * j;
        if (c < nchunks) {
            acc_word(v[j].x, mneg, S, T);
            acc_word(v[j].y, mneg, S, T);
            acc_word(v[j].z, mneg, S, T);
            acc_word(v[j].w, mneg, S, T);
            if (has_next) v[j] = ld_stream_v4(next_row + c);
        }
    }
    S = warp_sum(S);
    T = warp_sum(T);
    float H = logf(S) - kLn2 * (T / S);
    if (H != H) {
        // a -inf channel (t*e = -inf*0) lands here, as do genuinely undefined rows
        H = row_entropy_careful(row, nchunks, lane, m);
    }
    return H;
}

template <int NCH>
__device__ __forceinline__ void load_resident_row(uint4 (&v)[NCH], const uint4* row, int32_t nchunks, int lane) {
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
        const int c = lane + 32 * j;
        v[j] = c < nchunks ? ld_stream_v4(row + c) : make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
    }
}

// Count, sum and sum of squares (fp64) of the entropies a CTA has seen, one slot per warp, merged in warp order.
struct WarpStats { double n, s, q; };
__device__ __forceinline__ void cta_merge_stats(const WarpStats& mine, int warp, int lane, double* out3) {
    __shared__ double s_st[kGateWarps][3];
    if (lane == 0) { s_st[warp][0] = mine.n; s_st[warp][1] = mine.s; s_st[warp][2] = mine.q; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double n = 0, sm = 0, q = 0;
        for (int w = 0; w < kGateWarps; ++w) { n += s_st[w][0]; sm += s_st[w][1]; q += s_st[w][2]; }
        out3[0] = n; out3[1] = sm; out3[2] = q;
    }
}

// One warp per token, row resident in registers: NCH 16-byte chunks per lane.
template <int NCH>
__global__ void __launch_bounds__(kGateThreads)
gate_rows_kernel(const uint4* __restrict__ feat, int64_t n, int32_t nchunks, float tau,
                 uint8_t* __restrict__ mask, float* __restrict__ entropy,
                 int32_t* __restrict__ block_counts, double* __restrict__ cta_stats, int64_t tokens_per_block) {
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    // the compaction kernel may be launched as soon as every block of this grid has started: its launch
    // latency then hides under this kernel's tail (it waits for this grid's completion before reading)
    asm volatile("griddepcontrol.launch_dependents;");
    const int64_t t_begin = (int64_t)blockIdx.x * tokens_per_block;
    const int64_t t_end = min(n, t_begin + tokens_per_block);
    int kept = 0;
    WarpStats st{0.0, 0.0, 0.0};
    uint4 v[NCH];
    if (t_begin + warp < t_end) load_resident_row(v, feat + (t_begin + warp) * (int64_t)nchunks, nchunks, lane);
    for (int64_t tok = t_begin + warp; tok < t_end; tok += kGateWarps) {
        const uint4* row = feat + tok * (int64_t)nchunks;
        const float H = resident_row_entropy(v, row, row + (int64_t)kGateWarps * nchunks, tok + kGateWarps < t_end,
                                             nchunks, lane);
        const bool keep = (H >= tau);  // false for NaN
        if (lane == 0) {
            if (mask) mask[tok] = keep ? 1 : 0;
            if (entropy) entropy[tok] = H;
        }
        kept += keep ? 1 : 0;
        st.n += 1.0; st.s += (double)H; st.q += (double)H * (double)H;
    }
    // block count (every lane of a warp holds the same `kept`)
    __shared__ int s_cnt[kGateWarps];
    if (lane == 0) s_cnt[warp] = kept;
    __syncthreads();
    if (threadIdx.x == 0) {
        int tot = 0;
#pragma unroll
        for (int w = 0; w < kGateWarps; ++w) tot += s_cnt[w];
        if (block_counts) block_counts[blockIdx.x] = tot;
    }
    if (cta_stats) cta_merge_stats(st, warp, lane, cta_stats + 3 * (size_t)blockIdx.x);
}

// Block-prefix form (Algorithm 1, Step 1, in one pass over the features): a CTA owns whole draft blocks. Its
// warps leave the row entropies in shared memory; then one thread per draft block forms the token indicators
// (mean of the token's r row entropies, summed in row order), runs the prefix test, and writes mask, kept
// length and, if asked, the indicators. No row entropy goes through global memory unless the caller wants it.
template <int NCH>
__global__ void __launch_bounds__(kGateThreads)
gate_blocks_kernel(const uint4* __restrict__ feat, int64_t n_tokens, int32_t r, int32_t gamma, int32_t nchunks,
                   float tau, float* __restrict__ row_entropy, float* __restrict__ token_entropy,
                   uint8_t* __restrict__ mask, int32_t* __restrict__ block_len, int32_t* __restrict__ cta_counts,
                   int64_t blocks_per_cta, int64_t n_blocks) {
    extern __shared__ float s_H[];      // row entropies of this CTA's draft blocks
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    asm volatile("griddepcontrol.launch_dependents;");
    const int64_t b_begin = (int64_t)blockIdx.x * blocks_per_cta;
    const int64_t b_end = min(n_blocks, b_begin + blocks_per_cta);
    const int64_t t_begin = b_begin * gamma;
    const int64_t t_end = min(n_tokens, b_end * gamma);
    const int64_t r_begin = t_begin * r, r_end = t_end * r;
    uint4 v[NCH];
    if (r_begin + warp < r_end) load_resident_row(v, feat + (r_begin + warp) * (int64_t)nchunks, nchunks, lane);
    for (int64_t row_i = r_begin + warp; row_i < r_end; row_i += kGateWarps) {
        const uint4* row = feat + row_i * (int64_t)nchunks;
        const float H = resident_row_entropy(v, row, row + (int64_t)kGateWarps * nchunks, row_i + kGateWarps < r_end,
                                             nchunks, lane);
        if (lane == 0) {
            s_H[row_i - r_begin] = H;
            if (row_entropy) row_entropy[row_i] = H;
        }
    }
    __syncthreads();
    int kept_total = 0;
    const float inv = 1.0f / (float)r;
    for (int64_t b = b_begin + threadIdx.x; b < b_end; b += kGateThreads) {
        const int64_t t0 = b * gamma;
        const int64_t t1 = min(n_tokens, t0 + gamma);
        bool speculate = true;
        int kept = 0;
        for (int64_t t = t0; t < t1; ++t) {
            const float* src = s_H + (t - t_begin) * r;
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
    __shared__ int s_cnt[kGateWarps];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) kept_total += __shfl_xor_sync(0xffffffffu, kept_total, o);
    if (lane == 0) s_cnt[warp] = kept_total;
    __syncthreads();
    if (threadIdx.x == 0) {
        int tot = 0;
        for (int w = 0; w < kGateWarps; ++w) tot += s_cnt[w];
        cta_counts[blockIdx.x] = tot;
    }
}

// Rows longer than the registers hold (d > 8192, d % 8 == 0): still one pass with 128-bit loads. Every lane
// keeps a running maximum of its own share of the row and rescales its partial sums when the maximum grows
// (S <- S 2^D, T <- (T + D S) 2^D with D = (m_old - m_new) log2 e <= 0); the lanes' partials are merged the
// same way at the end.
__global__ void __launch_bounds__(kGateThreads)
gate_rows_long_kernel(const uint4* __restrict__ feat, int64_t n, int32_t nchunks, float tau,
                      uint8_t* __restrict__ mask, float* __restrict__ entropy,
                      int32_t* __restrict__ block_counts, double* __restrict__ cta_stats, int64_t tokens_per_block) {
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    asm volatile("griddepcontrol.launch_dependents;");
    const int64_t t_begin = (int64_t)blockIdx.x * tokens_per_block;
    const int64_t t_end = min(n, t_begin + tokens_per_block);
    int kept = 0;
    WarpStats st{0.0, 0.0, 0.0};
    for (int64_t tok = t_begin + warp; tok < t_end; tok += kGateWarps) {
        const uint4* row = feat + tok * (int64_t)nchunks;
        float ml = -CUDART_INF_F, S = 0.f, T = 0.f;
        for (int c0 = lane; c0 < nchunks; c0 += 32 * 4) {
            uint4 v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j)
                v[j] = c0 + 32 * j < nchunks ? ld_stream_v4(row + c0 + 32 * j)
                                             : make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
            uint32_t mx = 0xff80ff80u;
#pragma unroll
            for (int j = 0; j < 4; ++j)
                mx = max_bf16x2_nan(mx, max_bf16x2_nan(max_bf16x2_nan(v[j].x, v[j].y), max_bf16x2_nan(v[j].z, v[j].w)));
            const float a = bf16_lo(mx), b = bf16_hi(mx);
            const float mc = (a != a || b != b) ? CUDART_NAN_F : fmaxf(a, b);
            if (mc != mc) ml = CUDART_NAN_F;
            else if (mc > ml) {
                if (S > 0.f) {
                    const float D = (ml - mc) * kLog2e;
                    const float f = ex2_approx(D);
                    T = (T + D * S) * f;
                    S = S * f;
                }
                ml = mc;
            }
            const float mneg = -ml * kLog2e;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (c0 + 32 * j < nchunks) {
                    acc_word(v[j].x, mneg, S, T);
                    acc_word(v[j].y, mneg, S, T);
                    acc_word(v[j].z, mneg, S, T);
                    acc_word(v[j].w, mneg, S, T);
                }
            }
        }
        const float m = warp_max_nan(ml);
        if (S > 0.f && ml < m) {               // bring this lane's partials to the row maximum
            const float D = (ml - m) * kLog2e;
            const float f = ex2_approx(D);
            T = (T + D * S) * f;
            S = S * f;
        }
        S = warp_sum(S);
        T = warp_sum(T);
        float H = logf(S) - kLn2 * (T / S);
        if (H != H) H = row_entropy_careful(row, nchunks, lane, m);
        const bool keep = (H >= tau);
        if (lane == 0) {
            if (mask) mask[tok] = keep ? 1 : 0;
            if (entropy) entropy[tok] = H;
        }
        kept += keep ? 1 : 0;
        st.n += 1.0; st.s += (double)H; st.q += (double)H * (double)H;
    }
    __shared__ int s_cnt[kGateWarps];
    if (lane == 0) s_cnt[warp] = kept;
    __syncthreads();
    if (threadIdx.x == 0) {
        int tot = 0;
        for (int w = 0; w < kGateWarps; ++w) tot += s_cnt[w];
        if (block_counts) block_counts[blockIdx.x] = tot;
    }
    if (cta_stats) cta_merge_stats(st, warp, lane, cta_stats + 3 * (size_t)blockIdx.x);
}

// Any d (no alignment assumption, any length): two passes over the row with scalar loads.
__global__ void __launch_bounds__(kGateThreads)
gate_rows_generic_kernel(const uint16_t* __restrict__ feat, int64_t n, int32_t d, float tau,
                         uint8_t* __restrict__ mask, float* __restrict__ entropy,
                         int32_t* __restrict__ block_counts, double* __restrict__ cta_stats,
                         int64_t tokens_per_block) {
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int64_t t_begin = (int64_t)blockIdx.x * tokens_per_block;
    const int64_t t_end = min(n, t_begin + tokens_per_block);
    int kept = 0;
    WarpStats st{0.0, 0.0, 0.0};
    for (int64_t tok = t_begin + warp; tok < t_end; tok += kGateWarps) {
        const uint16_t* row = feat + tok * (int64_t)d;
        float m = -CUDART_INF_F;
        bool nan = false;
        for (int c = lane; c < d; c += 32) {
            float x = __uint_as_float((uint32_t)row[c] << 16);
            nan |= (x != x);
            m = fmaxf(m, x);
        }
        if (nan) m = CUDART_NAN_F;
        m = warp_max_nan(m);
        const float mneg = -m * kLog2e;
        float S = 0.f, T = 0.f;
        for (int c = lane; c < d; c += 32) {
            float x = __uint_as_float((uint32_t)row[c] << 16);
            float t = fmaf(x, kLog2e, mneg);
            float e = ex2_approx(t);
            S += e;
            if (e > 0.f || e != e) T = fmaf(t, e, T);
        }
        S = warp_sum(S);
        T = warp_sum(T);
        const float H = logf(S) - kLn2 * (T / S);
        const bool keep = (H >= tau);
        if (lane == 0) {
            if (mask) mask[tok] = keep ? 1 : 0;
            if (entropy) entropy[tok] = H;
        }
        kept += keep ? 1 : 0;
        st.n += 1.0; st.s += (double)H; st.q += (double)H * (double)H;
    }
    __shared__ int s_cnt[kGateWarps];
    if (lane == 0) s_cnt[warp] = kept;
    __syncthreads();
    if (threadIdx.x == 0) {
        int tot = 0;
        for (int w = 0; w < kGateWarps; ++w) tot += s_cnt[w];
        if (block_counts) block_counts[blockIdx.x] = tot;
    }
    if (cta_stats) cta_merge_stats(st, warp, lane, cta_stats + 3 * (size_t)blockIdx.x);
}

// Stable compaction: block b writes the ids of kept tokens of its own range at the offset given
// by the counts of blocks 0..b-1.
__global__ void __launch_bounds__(kGateThreads)
compact_kernel(const uint8_t* __restrict__ mask, int64_t n, const int32_t* __restrict__ block_counts,
               int64_t tokens_per_block, int32_t* __restrict__ idx, int32_t* __restrict__ count,
               const double* __restrict__ cta_stats, double* __restrict__ stats_out3) {
    __shared__ int s_warp[kGateWarps];
    __shared__ int s_base;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    // launched with programmatic stream serialization: its blocks may be resident before the kernel that
    // writes mask and block_counts has finished; nothing of that kernel's output is read before this wait
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // Threshold statistics of the entropies (the tau equation): the per-CTA partial sums of the row kernel,
    // merged in a fixed order (lane-strided, then a fixed tree) so that the result is reproducible run to run.
    if (cta_stats && blockIdx.x == 0 && warp == 0) {
        double cn = 0, cs = 0, cq = 0;
        for (int b = lane; b < (int)gridDim.x; b += 32) {
            cn += cta_stats[3 * b]; cs += cta_stats[3 * b + 1]; cq += cta_stats[3 * b + 2];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            cn += __shfl_xor_sync(0xffffffffu, cn, o);
            cs += __shfl_xor_sync(0xffffffffu, cs, o);
            cq += __shfl_xor_sync(0xffffffffu, cq, o);
        }
        if (lane == 0) {
            const double mean = cs / cn;
            const double var = fmax(cq / cn - mean * mean, 0.0);
            stats_out3[0] = mean;
            stats_out3[1] = sqrt(var);
            stats_out3[2] = 0.3 * mean - 0.1 * sqrt(var);
        }
    }
    // offset = sum of counts of the blocks before this one
    int part = 0;
    for (int b = threadIdx.x; b < (int)blockIdx.x; b += kGateThreads) part += block_counts[b];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    if (lane == 0) s_warp[warp] = part;
    __syncthreads();
    if (threadIdx.x == 0) {
        int tot = 0;
        for (int w = 0; w < kGateWarps; ++w) tot += s_warp[w];
        s_base = tot;
        if (blockIdx.x == gridDim.x - 1) *count = tot + block_counts[blockIdx.x];
    }
    __syncthreads();
    int base = s_base;
    const int64_t t_begin = (int64_t)blockIdx.x * tokens_per_block;
    const int64_t t_end = min(n, t_begin + tokens_per_block);
    for (int64_t t0 = t_begin; t0 < t_end; t0 += kGateThreads) {
        const int64_t tok = t0 + threadIdx.x;
        const bool keep = (tok < t_end) && (mask[tok] != 0);
        const unsigned bal = __ballot_sync(0xffffffffu, keep);
        const int rank = __popc(bal & ((1u << lane) - 1u));
        __syncthreads();  // s_warp reuse
        if (lane == 0) s_warp[warp] = __popc(bal);
        __syncthreads();
        int woff = 0, tot = 0;
#pragma unroll
        for (int w = 0; w < kGateWarps; ++w) {
            const int cw = s_warp[w];
            woff += (w < warp) ? cw : 0;
            tot += cw;
        }
        if (keep) idx[base + woff + rank] = (int32_t)tok;
        base += tot;
    }
}

__global__ void write_zero_count_kernel(int32_t* count) { *count = 0; }

// ---- per-device scratch: one slice per stream ---------------------------------------------------
// A slice holds what the two kernels of a call hand to each other: per-block kept counts and, for the calls
// that ask for the threshold statistics, per-block partial sums. Two gate calls may run on the GPU at the same
// time only when they were enqueued on different streams, so every stream gets a slice of its own (calls on
// one stream are ordered and share theirs). The table holds kGateSlices - 1 streams per device; any further
// stream shares the last slice.
constexpr int kMaxDevices = 64;
constexpr int kGateSlices = 32;
constexpr size_t kSliceBytes = (size_t)kMaxGateBlocks * (sizeof(int32_t) + 3 * sizeof(double));
struct GateScratch {
    char* base = nullptr;
    int n_sm = 0;
    int used = 0;
    cudaStream_t key[kGateSlices];
};
GateScratch g_scratch[kMaxDevices];
std::mutex g_scratch_mutex;

int gate_scratch(cudaStream_t st, int32_t** counts, double** stats, int* sms) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ARDIFF_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return ARDIFF_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    GateScratch& g = g_scratch[dev];
    if (!g.base) {
        int n_sm = 0;
        if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            return ARDIFF_ERR_CUDA;
        void* p = nullptr;
        if (cudaMalloc(&p, kSliceBytes * kGateSlices) != cudaSuccess) {
            (void)cudaGetLastError();
            return ARDIFF_ERR_NOMEM;
        }
        g.n_sm = n_sm;
        g.base = static_cast<char*>(p);
    }
    int slice = -1;
    for (int i = 0; i < g.used; ++i)
        if (g.key[i] == st) { slice = i; break; }
    if (slice < 0) {
        if (g.used < kGateSlices - 1) {
            g.key[g.used] = st;
            slice = g.used++;
        } else {
            slice = kGateSlices - 1;
        }
    }
    char* sl = g.base + (size_t)slice * kSliceBytes;
    *stats = reinterpret_cast<double*>(sl);                                        // 8-byte aligned part first
    *counts = reinterpret_cast<int32_t*>(sl + (size_t)kMaxGateBlocks * 3 * sizeof(double));
    *sms = g.n_sm;
    return ARDIFF_OK;
}

// compact_kernel behind programmatic stream serialization (see the wait at its top)
cudaError_t launch_compact(int grid, cudaStream_t st, const uint8_t* mask, int64_t n, const int32_t* block_counts,
                           int64_t tpb, int32_t* idx, int32_t* count, const double* cta_stats, double* out3) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kGateThreads); cfg.dynamicSmemBytes = 0; cfg.stream = st;
    cfg.attrs = at; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, compact_kernel, mask, n, block_counts, tpb, idx, count, cta_stats, out3);
}

// the row kernel that holds a row of `need` x 32 sixteen-byte chunks in registers: f(integral_constant<NCH>)
template <typename F>
void dispatch_nch(int need, F&& f) {
    if (need <= 1) f(std::integral_constant<int, 1>());
    else if (need <= 2) f(std::integral_constant<int, 2>());
    else if (need <= 4) f(std::integral_constant<int, 4>());
    else if (need <= 8) f(std::integral_constant<int, 8>());
    else if (need <= 12) f(std::integral_constant<int, 12>());
    else if (need <= 16) f(std::integral_constant<int, 16>());
    else if (need <= 20) f(std::integral_constant<int, 20>());
    else if (need <= 24) f(std::integral_constant<int, 24>());
    else f(std::integral_constant<int, 32>());
}

// Launches the row kernel for any d (vector path when the row fits the registers, else the generic one).
void launch_rows(int grid, cudaStream_t st, const void* feat, int64_t n, int32_t d, float tau, uint8_t* mask,
                 float* entropy, int32_t* counts, double* cta_stats, int64_t tpb) {
    const bool vec = (d % 8 == 0) && (d <= 8192);
    if (vec) {
        dispatch_nch((d / 8 + 31) / 32, [&](auto nch) {
            gate_rows_kernel<decltype(nch)::value><<<grid, kGateThreads, 0, st>>>(
                reinterpret_cast<const uint4*>(feat), n, d / 8, tau, mask, entropy, counts, cta_stats, tpb);
        });
    } else if (d % 8 == 0) {
        gate_rows_long_kernel<<<grid, kGateThreads, 0, st>>>(reinterpret_cast<const uint4*>(feat), n, d / 8, tau, mask,
                                                            entropy, counts, cta_stats, tpb);
    } else {
        gate_rows_generic_kernel<<<grid, kGateThreads, 0, st>>>(reinterpret_cast<const uint16_t*>(feat), n, d, tau,
                                                               mask, entropy, counts, cta_stats, tpb);
    }
}

// Resident blocks per SM of the row kernel that serves rows of `need` x 32 chunks (0: the generic kernel).
// One block per resident slot, i.e. a grid of exactly one wave, measured best: with more blocks the later
// waves start against a full memory system and the kernel grows a tail (32768 x 5120: 74.8 -> 68.6 us).
int rows_blocks_per_sm(int need) {
    static int cache[10] = {0};
    int slot = need <= 0 ? 0 : need <= 1 ? 1 : need <= 2 ? 2 : need <= 4 ? 3 : need <= 8 ? 4 : need <= 12 ? 5
               : need <= 16 ? 6 : need <= 20 ? 7 : need <= 24 ? 8 : 9;
    if (cache[slot] > 0) return cache[slot];
    int occ = 0;
    cudaError_t e = cudaSuccess;
    if (slot == 0) {
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, gate_rows_generic_kernel, kGateThreads, 0);
    } else {
        dispatch_nch(need, [&](auto nch) {
            e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, gate_rows_kernel<decltype(nch)::value>,
                                                              kGateThreads, 0);
        });
    }
    if (e != cudaSuccess || occ < 1) {
        (void)cudaGetLastError();
        occ = 2;
    }
    if (occ > 8) occ = 8;
    cache[slot] = occ;
    return occ;
}

// Waves of blocks: one while a block's share of the input stays small (then ramp and tail dominate and a
// single wave is fastest), up to four once a block would stream more than 4 MB (then finer blocks even out
// the finish: 2^19 x 5120 is 1 % faster with four waves than with one).
int grid_waves(int64_t rows, int32_t d, int64_t resident_blocks) {
    const int64_t per_block = rows * (int64_t)d * 2 / (resident_blocks > 0 ? resident_blocks : 1);
    const int64_t w = per_block / (4ll << 20);
    return w < 1 ? 1 : (w > 4 ? 4 : (int)w);
}

int check_feat(const void* feat, int32_t d) {
    const bool vec = (d % 8 == 0);
    if (vec && (reinterpret_cast<uintptr_t>(feat) & 15u)) return ARDIFF_ERR_ALIGN;
    if (!vec && (reinterpret_cast<uintptr_t>(feat) & 1u)) return ARDIFF_ERR_ALIGN;
    return ARDIFF_OK;
}

}  // namespace

namespace ardiff {

// Shared by the allocating entry points and by variants that bring their own block-count
// scratch: validates, picks the row kernel, launches gate + compaction on `st`. With cta_stats and
// stats_out3 the entropies' mean, standard deviation and threshold are produced on the way.
int gate_launch(const void* feat, int64_t n, int32_t d, float tau, uint8_t* mask, int32_t* idx,
                int32_t* count, float* entropy, int32_t* block_counts, double* cta_stats, double* stats_out3,
                int max_blocks, int n_sm, cudaStream_t st) {
    if (!count) return ARDIFF_ERR_NULL;
    if (n < 0 || n >= (int64_t)1 << 31 || d < 1 || d > 65536) return ARDIFF_ERR_SHAPE;
    if (n == 0) {
        write_zero_count_kernel<<<1, 1, 0, st>>>(count);
        set_launch_count(1);
        return cudaGetLastError() == cudaSuccess ? ARDIFF_OK : ARDIFF_ERR_CUDA;
    }
    if (!feat || !mask || !idx || !block_counts) return ARDIFF_ERR_NULL;
    const int rc = check_feat(feat, d);
    if (rc != ARDIFF_OK) return rc;
    const bool vec = (d % 8 == 0) && (d <= 8192);

    // contiguous token range per block; one block per resident slot of the GPU, each with >= 1 token per warp
    int64_t want = (int64_t)n_sm * rows_blocks_per_sm(vec ? (d / 8 + 31) / 32 : 0);
    want *= grid_waves(n, d, want);
    if (want > max_blocks) want = max_blocks;
    int64_t tpb = (n + want - 1) / want;
    if (tpb < kGateWarps) tpb = kGateWarps;
    const int grid = (int)((n + tpb - 1) / tpb);

    launch_rows(grid, st, feat, n, d, tau, mask, entropy, block_counts, stats_out3 ? cta_stats : nullptr, tpb);
    (void)launch_compact(grid, st, mask, n, block_counts, tpb, idx, count, stats_out3 ? cta_stats : nullptr,
                         stats_out3);
    set_launch_count(2);
    return cudaGetLastError() == cudaSuccess ? ARDIFF_OK : ARDIFF_ERR_CUDA;
}

// Row entropies only (no threshold, no compaction): entropy[i] = H of row i.
int entropy_rows_launch(const void* feat, int64_t rows, int32_t d, float* entropy, int n_sm, cudaStream_t st) {
    if (rows < 0 || rows >= (int64_t)1 << 31 || d < 1 || d > 65536) return ARDIFF_ERR_SHAPE;
    if (rows == 0) return ARDIFF_OK;
    if (!feat || !entropy) return ARDIFF_ERR_NULL;
    const int rc = check_feat(feat, d);
    if (rc != ARDIFF_OK) return rc;
    const bool vec = (d % 8 == 0) && (d <= 8192);
    int64_t want = (int64_t)n_sm * rows_blocks_per_sm(vec ? (d / 8 + 31) / 32 : 0);
    want *= grid_waves(rows, d, want);
    int64_t tpb = (rows + want - 1) / want;
    if (tpb < kGateWarps) tpb = kGateWarps;
    const int grid = (int)((rows + tpb - 1) / tpb);
    launch_rows(grid, st, feat, rows, d, 0.f, nullptr, entropy, nullptr, nullptr, tpb);
    return cudaGetLastError() == cudaSuccess ? ARDIFF_OK : ARDIFF_ERR_CUDA;
}

// The block-prefix gate in one pass over the features (gate_blocks_kernel + compaction). Returns
// ARDIFF_ERR_UNSUPPORTED, with nothing launched, when the shape does not fit it: rows that do not fit the
// registers, or a draft block whose row entropies exceed a CTA's shared memory.
int gate_blocks_fused_launch(const void* feat, int64_t n, int32_t r, int32_t d, int32_t gamma, float tau,
                             float* row_entropy, float* token_entropy, uint8_t* mask, int32_t* idx, int32_t* count,
                             int32_t* block_len, int32_t* cta_counts, int max_blocks, int n_sm, cudaStream_t st) {
    const bool vec = (d % 8 == 0) && (d <= 8192);
    constexpr int64_t kMaxRowsPerCta = 24576;     // 96 KB of row entropies
    if (!vec || (int64_t)gamma * r > kMaxRowsPerCta) return ARDIFF_ERR_UNSUPPORTED;
    const int rc = check_feat(feat, d);
    if (rc != ARDIFF_OK) return rc;
    const int need = (d / 8 + 31) / 32;
    const int64_t n_blocks = (n + gamma - 1) / gamma;
    const int64_t rows = n * r;
    int64_t want = (int64_t)n_sm * rows_blocks_per_sm(need);
    want *= grid_waves(rows, d, want);
    if (want > max_blocks) want = max_blocks;
    int64_t bpc = (n_blocks + want - 1) / want;                        // draft blocks per CTA
    const int64_t rows_per_block = (int64_t)gamma * r;
    if (bpc * rows_per_block > kMaxRowsPerCta) bpc = kMaxRowsPerCta / rows_per_block;
    if (bpc < 1) bpc = 1;
    const int64_t grid64 = (n_blocks + bpc - 1) / bpc;
    if (grid64 > max_blocks) return ARDIFF_ERR_UNSUPPORTED;          // too many CTAs for the count scratch
    const int grid = (int)grid64;
    const size_t smem = (size_t)(bpc * rows_per_block) * sizeof(float);
    cudaError_t e = cudaSuccess;
    dispatch_nch(need, [&](auto nch) {
        auto kern = gate_blocks_kernel<decltype(nch)::value>;
        if (smem > 48 * 1024) e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
        if (e == cudaSuccess)
            kern<<<grid, kGateThreads, smem, st>>>(reinterpret_cast<const uint4*>(feat), n, r, gamma, d / 8, tau,
                                                  row_entropy, token_entropy, mask, block_len, cta_counts, bpc,
                                                  n_blocks);
    });
    if (e != cudaSuccess) return ARDIFF_ERR_CUDA;
    (void)launch_compact(grid, st, mask, n, cta_counts, bpc * gamma, idx, count, nullptr, nullptr);
    set_launch_count(2);
    return cudaGetLastError() == cudaSuccess ? ARDIFF_OK : ARDIFF_ERR_CUDA;
}

// Stable compaction of a mask whose per-block kept counts (blocks of tokens_per_block tokens) are known.
int compact_launch(const uint8_t* mask, int64_t n, const int32_t* block_counts, int64_t tokens_per_block, int grid,
                   int32_t* idx, int32_t* count, cudaStream_t st) {
    (void)launch_compact(grid, st, mask, n, block_counts, tokens_per_block, idx, count, nullptr, nullptr);
    return cudaGetLastError() == cudaSuccess ? ARDIFF_OK : ARDIFF_ERR_CUDA;
}

int gate_scratch_get(cudaStream_t st, int32_t** counts, int* max_blocks, int* sms) {
    *max_blocks = kMaxGateBlocks;
    double* stats = nullptr;
    return gate_scratch(st, counts, &stats, sms);
}

int write_zero_count(int32_t* count, cudaStream_t st) {
    write_zero_count_kernel<<<1, 1, 0, st>>>(count);
    return cudaGetLastError() == cudaSuccess ? ARDIFF_OK : ARDIFF_ERR_CUDA;
}

}  // namespace ardiff

namespace {
int gate_entry(const void* feat, int64_t n, int32_t d, float tau, uint8_t* mask, int32_t* idx, int32_t* count,
               float* entropy, double* stats_out3, void* stream) {
    int32_t* counts = nullptr;
    double* stats = nullptr;
    int sms = 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int rc = gate_scratch(st, &counts, &stats, &sms);
    if (rc != ARDIFF_OK) return rc;
    return ardiff::gate_launch(feat, n, d, tau, mask, idx, count, entropy, counts, stats, stats_out3,
                               kMaxGateBlocks, sms, st);
}
}  // namespace

extern "C" int ardiff_entropy_gate_ex(const void* feat, int64_t n, int32_t d, float tau,
                                      uint8_t* mask, int32_t* idx, int32_t* count, float* entropy,
                                      void* stream) {
    return gate_entry(feat, n, d, tau, mask, idx, count, entropy, nullptr, stream);
}

extern "C" int ardiff_entropy_gate(const void* feat, int64_t n, int32_t d, float tau, uint8_t* mask,
                                   int32_t* idx, int32_t* count, void* stream) {
    return gate_entry(feat, n, d, tau, mask, idx, count, nullptr, nullptr, stream);
}

extern "C" int ardiff_entropy_gate_stats(const void* feat, int64_t n, int32_t d, float tau, uint8_t* mask,
                                         int32_t* idx, int32_t* count, float* entropy, double* out3,
                                         void* stream) {
    if (!out3) return ARDIFF_ERR_NULL;
    if (n < 1) return ARDIFF_ERR_SHAPE;
    return gate_entry(feat, n, d, tau, mask, idx, count, entropy, out3, stream);
}
