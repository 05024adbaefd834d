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

// One warp per token, row resident in registers: NCH 16-byte chunks per lane.
template <int NCH>
__global__ void __launch_bounds__(kGateThreads)
gate_rows_kernel(const uint4* __restrict__ feat, int64_t n, int32_t nchunks, float tau,
                 uint8_t* __restrict__ mask, float* __restrict__ entropy,
                 int32_t* __restrict__ block_counts, int64_t tokens_per_block) {
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    // the compaction kernel may be launched as soon as every block of this grid has started: its launch
    // latency then hides under this kernel's tail (it waits for this grid's completion before reading)
    asm volatile("griddepcontrol.launch_dependents;");
    const int64_t t_begin = (int64_t)blockIdx.x * tokens_per_block;
    const int64_t t_end = min(n, t_begin + tokens_per_block);
    int kept = 0;
    for (int64_t tok = t_begin + warp; tok < t_end; tok += kGateWarps) {
        const uint4* row = feat + tok * (int64_t)nchunks;
        uint4 v[NCH];
#pragma unroll
        for (int j = 0; j < NCH; ++j) {
            const int c = lane + 32 * j;
            if (c < nchunks) v[j] = ld_stream_v4(row + c);
            else v[j] = make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);  // -inf
        }
        // row maximum (packed, exact in bf16)
        uint32_t mx = 0xff80ff80u;
#pragma unroll
        for (int j = 0; j < NCH; ++j) {
            mx = max_bf16x2_nan(mx, max_bf16x2_nan(max_bf16x2_nan(v[j].x, v[j].y),
                                                   max_bf16x2_nan(v[j].z, v[j].w)));
        }
        float ml = bf16_lo(mx), mh = bf16_hi(mx);
        float m = (ml != ml || mh != mh) ? CUDART_NAN_F : fmaxf(ml, mh);
        m = warp_max_nan(m);
        const float mneg = -m * kLog2e;
        float S = 0.f, T = 0.f;
#pragma unroll
        for (int j = 0; j < NCH; ++j) {
            if (lane + 32 * j < nchunks) {
                acc_word(v[j].x, mneg, S, T);
                acc_word(v[j].y, mneg, S, T);
                acc_word(v[j].z, mneg, S, T);
                acc_word(v[j].w, mneg, S, T);
            }
        }
        S = warp_sum(S);
        T = warp_sum(T);
        float H = logf(S) - kLn2 * (T / S);
        if (H != H) {
            // a -inf channel (t*e = -inf*0) lands here, as do genuinely undefined rows
            H = row_entropy_careful(row, nchunks, lane, m);
        }
        const bool keep = (H >= tau);  // false for NaN
        if (lane == 0) {
            if (mask) mask[tok] = keep ? 1 : 0;
            if (entropy) entropy[tok] = H;
        }
        kept += keep ? 1 : 0;
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
}

// Any d (no alignment assumption, any length): two passes over the row with scalar loads.
__global__ void __launch_bounds__(kGateThreads)
gate_rows_generic_kernel(const uint16_t* __restrict__ feat, int64_t n, int32_t d, float tau,
                         uint8_t* __restrict__ mask, float* __restrict__ entropy,
                         int32_t* __restrict__ block_counts, int64_t tokens_per_block) {
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int64_t t_begin = (int64_t)blockIdx.x * tokens_per_block;
    const int64_t t_end = min(n, t_begin + tokens_per_block);
    int kept = 0;
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
    }
    __shared__ int s_cnt[kGateWarps];
    if (lane == 0) s_cnt[warp] = kept;
    __syncthreads();
    if (threadIdx.x == 0) {
        int tot = 0;
        for (int w = 0; w < kGateWarps; ++w) tot += s_cnt[w];
        if (block_counts) block_counts[blockIdx.x] = tot;
    }
}

// Stable compaction: block b writes the ids of kept tokens of its own range at the offset given
// by the counts of blocks 0..b-1.
__global__ void __launch_bounds__(kGateThreads)
compact_kernel(const uint8_t* __restrict__ mask, int64_t n, const int32_t* __restrict__ block_counts,
               int64_t tokens_per_block, int32_t* __restrict__ idx, int32_t* __restrict__ count) {
    __shared__ int s_warp[kGateWarps];
    __shared__ int s_base;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    // launched with programmatic stream serialization: its blocks may be resident before the kernel that
    // writes mask and block_counts has finished; nothing of that kernel's output is read before this wait
    asm volatile("griddepcontrol.wait;" ::: "memory");
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

// ---- per-device scratch for the block counts: one slice per stream -----------------------------
// Two gate calls may run on the GPU at the same time only when they were enqueued on different streams,
// so every stream gets a slice of its own (calls on one stream are ordered and share theirs). The table
// holds kGateSlices - 1 streams per device; any further stream shares the last slice.
constexpr int kMaxDevices = 64;
constexpr int kGateSlices = 32;
struct GateScratch {
    int32_t* base = nullptr;
    int n_sm = 0;
    int used = 0;
    cudaStream_t key[kGateSlices];
};
GateScratch g_scratch[kMaxDevices];
std::mutex g_scratch_mutex;

int gate_scratch(cudaStream_t st, int32_t** out, int* sms) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ARDIFF_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return ARDIFF_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    GateScratch& g = g_scratch[dev];
    if (!g.base) {
        int n_sm = 0;
        if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            return ARDIFF_ERR_CUDA;
        int32_t* p = nullptr;
        if (cudaMalloc(&p, sizeof(int32_t) * kMaxGateBlocks * kGateSlices) != cudaSuccess) {
            (void)cudaGetLastError();
            return ARDIFF_ERR_NOMEM;
        }
        g.n_sm = n_sm;
        g.base = p;
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
    *out = g.base + (size_t)slice * kMaxGateBlocks;
    *sms = g.n_sm;
    return ARDIFF_OK;
}

// compact_kernel behind programmatic stream serialization (see the wait at its top)
cudaError_t launch_compact(int grid, cudaStream_t st, const uint8_t* mask, int64_t n, const int32_t* block_counts,
                           int64_t tpb, int32_t* idx, int32_t* count) {
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kGateThreads); cfg.dynamicSmemBytes = 0; cfg.stream = st;
    cfg.attrs = at; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, compact_kernel, mask, n, block_counts, tpb, idx, count);
}

template <int NCH>
void launch_rows(int grid, cudaStream_t st, const void* feat, int64_t n, int32_t d, float tau,
                 uint8_t* mask, float* entropy, int32_t* counts, int64_t tpb) {
    gate_rows_kernel<NCH><<<grid, kGateThreads, 0, st>>>(
        reinterpret_cast<const uint4*>(feat), n, d / 8, tau, mask, entropy, counts, tpb);
}

// Resident blocks per SM of the row kernel that serves rows of `nchunks` 16-byte chunks (0: the generic kernel).
// One block per resident slot, i.e. a grid of exactly one wave, measured best: with more blocks the later
// waves start against a full memory system and the kernel grows a tail (32768 x 5120: 74.8 -> 68.6 us).
int rows_blocks_per_sm(int need) {
    static int cache[10] = {0};
    int slot = need <= 0 ? 0 : need <= 1 ? 1 : need <= 2 ? 2 : need <= 4 ? 3 : need <= 8 ? 4 : need <= 12 ? 5
               : need <= 16 ? 6 : need <= 20 ? 7 : need <= 24 ? 8 : 9;
    if (cache[slot] > 0) return cache[slot];
    int occ = 0;
    cudaError_t e;
    switch (slot) {
        case 0: e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, gate_rows_generic_kernel, kGateThreads, 0); break;
        case 1: e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, gate_rows_kernel<1>, kGateThreads, 0); break;
        case 2: e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, gate_rows_kernel<2>, kGateThreads, 0); break;
        case 3: e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, gate_rows_kernel<4>, kGateThreads, 0); break;
        case 4: e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, gate_rows_kernel<8>, kGateThreads, 0); break;
        case 5: e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, gate_rows_kernel<12>, kGateThreads, 0); break;
        case 6: e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, gate_rows_kernel<16>, kGateThreads, 0); break;
        case 7: e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, gate_rows_kernel<20>, kGateThreads, 0); break;
        case 8: e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, gate_rows_kernel<24>, kGateThreads, 0); break;
        default: e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, gate_rows_kernel<32>, kGateThreads, 0); break;
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

}  // namespace

namespace ardiff {

// Shared by the allocating entry points and by variants that bring their own block-count
// scratch: validates, picks the row kernel, launches gate + compaction on `st`.
int gate_launch(const void* feat, int64_t n, int32_t d, float tau, uint8_t* mask, int32_t* idx,
                int32_t* count, float* entropy, int32_t* block_counts, int max_blocks, int n_sm,
                cudaStream_t st) {
    if (!count) return ARDIFF_ERR_NULL;
    if (n < 0 || n >= (int64_t)1 << 31 || d < 1 || d > 65536) return ARDIFF_ERR_SHAPE;
    if (n == 0) {
        write_zero_count_kernel<<<1, 1, 0, st>>>(count);
        set_launch_count(1);
        return cudaGetLastError() == cudaSuccess ? ARDIFF_OK : ARDIFF_ERR_CUDA;
    }
    if (!feat || !mask || !idx || !block_counts) return ARDIFF_ERR_NULL;
    const bool vec = (d % 8 == 0) && (d <= 8192);
    if (vec && (reinterpret_cast<uintptr_t>(feat) & 15u)) return ARDIFF_ERR_ALIGN;
    if (!vec && (reinterpret_cast<uintptr_t>(feat) & 1u)) return ARDIFF_ERR_ALIGN;

    // contiguous token range per block; one block per resident slot of the GPU, each with >= 1 token per warp
    int64_t want = (int64_t)n_sm * rows_blocks_per_sm(vec ? (d / 8 + 31) / 32 : 0);
    want *= grid_waves(n, d, want);
    if (want > max_blocks) want = max_blocks;
    int64_t tpb = (n + want - 1) / want;
    if (tpb < kGateWarps) tpb = kGateWarps;
    const int grid = (int)((n + tpb - 1) / tpb);

    if (vec) {
        const int need = (d / 8 + 31) / 32;
        if (need <= 1) launch_rows<1>(grid, st, feat, n, d, tau, mask, entropy, block_counts, tpb);
        else if (need <= 2) launch_rows<2>(grid, st, feat, n, d, tau, mask, entropy, block_counts, tpb);
        else if (need <= 4) launch_rows<4>(grid, st, feat, n, d, tau, mask, entropy, block_counts, tpb);
        else if (need <= 8) launch_rows<8>(grid, st, feat, n, d, tau, mask, entropy, block_counts, tpb);
        else if (need <= 12) launch_rows<12>(grid, st, feat, n, d, tau, mask, entropy, block_counts, tpb);
        else if (need <= 16) launch_rows<16>(grid, st, feat, n, d, tau, mask, entropy, block_counts, tpb);
        else if (need <= 20) launch_rows<20>(grid, st, feat, n, d, tau, mask, entropy, block_counts, tpb);
        else if (need <= 24) launch_rows<24>(grid, st, feat, n, d, tau, mask, entropy, block_counts, tpb);
        else launch_rows<32>(grid, st, feat, n, d, tau, mask, entropy, block_counts, tpb);
    } else {
        gate_rows_generic_kernel<<<grid, kGateThreads, 0, st>>>(
            reinterpret_cast<const uint16_t*>(feat), n, d, tau, mask, entropy, block_counts, tpb);
    }
    (void)launch_compact(grid, st, mask, n, block_counts, tpb, idx, count);
    set_launch_count(2);
    return cudaGetLastError() == cudaSuccess ? ARDIFF_OK : ARDIFF_ERR_CUDA;
}

// Row entropies only (no threshold, no compaction): entropy[i] = H of row i.
int entropy_rows_launch(const void* feat, int64_t rows, int32_t d, float* entropy, int n_sm, cudaStream_t st) {
    if (rows < 0 || rows >= (int64_t)1 << 31 || d < 1 || d > 65536) return ARDIFF_ERR_SHAPE;
    if (rows == 0) return ARDIFF_OK;
    if (!feat || !entropy) return ARDIFF_ERR_NULL;
    const bool vec = (d % 8 == 0) && (d <= 8192);
    if (vec && (reinterpret_cast<uintptr_t>(feat) & 15u)) return ARDIFF_ERR_ALIGN;
    if (!vec && (reinterpret_cast<uintptr_t>(feat) & 1u)) return ARDIFF_ERR_ALIGN;
    int64_t want = (int64_t)n_sm * rows_blocks_per_sm(vec ? (d / 8 + 31) / 32 : 0);
    want *= grid_waves(rows, d, want);
    int64_t tpb = (rows + want - 1) / want;
    if (tpb < kGateWarps) tpb = kGateWarps;
    const int grid = (int)((rows + tpb - 1) / tpb);
    const float tau = 0.f;
    if (vec) {
        const int need = (d / 8 + 31) / 32;
        if (need <= 1) launch_rows<1>(grid, st, feat, rows, d, tau, nullptr, entropy, nullptr, tpb);
        else if (need <= 2) launch_rows<2>(grid, st, feat, rows, d, tau, nullptr, entropy, nullptr, tpb);
        else if (need <= 4) launch_rows<4>(grid, st, feat, rows, d, tau, nullptr, entropy, nullptr, tpb);
        else if (need <= 8) launch_rows<8>(grid, st, feat, rows, d, tau, nullptr, entropy, nullptr, tpb);
        else if (need <= 12) launch_rows<12>(grid, st, feat, rows, d, tau, nullptr, entropy, nullptr, tpb);
        else if (need <= 16) launch_rows<16>(grid, st, feat, rows, d, tau, nullptr, entropy, nullptr, tpb);
        else if (need <= 20) launch_rows<20>(grid, st, feat, rows, d, tau, nullptr, entropy, nullptr, tpb);
        else if (need <= 24) launch_rows<24>(grid, st, feat, rows, d, tau, nullptr, entropy, nullptr, tpb);
        else launch_rows<32>(grid, st, feat, rows, d, tau, nullptr, entropy, nullptr, tpb);
    } else {
        gate_rows_generic_kernel<<<grid, kGateThreads, 0, st>>>(reinterpret_cast<const uint16_t*>(feat), rows, d, tau,
                                                               nullptr, entropy, nullptr, tpb);
    }
    return cudaGetLastError() == cudaSuccess ? ARDIFF_OK : ARDIFF_ERR_CUDA;
}

// Stable compaction of a mask whose per-block kept counts (blocks of tokens_per_block tokens) are known.
int compact_launch(const uint8_t* mask, int64_t n, const int32_t* block_counts, int64_t tokens_per_block, int grid,
                   int32_t* idx, int32_t* count, cudaStream_t st) {
    (void)launch_compact(grid, st, mask, n, block_counts, tokens_per_block, idx, count);
    return cudaGetLastError() == cudaSuccess ? ARDIFF_OK : ARDIFF_ERR_CUDA;
}

int gate_scratch_get(cudaStream_t st, int32_t** counts, int* max_blocks, int* sms) {
    *max_blocks = kMaxGateBlocks;
    return gate_scratch(st, counts, sms);
}

int write_zero_count(int32_t* count, cudaStream_t st) {
    write_zero_count_kernel<<<1, 1, 0, st>>>(count);
    return cudaGetLastError() == cudaSuccess ? ARDIFF_OK : ARDIFF_ERR_CUDA;
}

}  // namespace ardiff

extern "C" int ardiff_entropy_gate_ex(const void* feat, int64_t n, int32_t d, float tau,
                                      uint8_t* mask, int32_t* idx, int32_t* count, float* entropy,
                                      void* stream) {
    int32_t* counts = nullptr;
    int sms = 0;
    int rc = gate_scratch(static_cast<cudaStream_t>(stream), &counts, &sms);
    if (rc != ARDIFF_OK) return rc;
    return ardiff::gate_launch(feat, n, d, tau, mask, idx, count, entropy, counts, kMaxGateBlocks,
                               sms, static_cast<cudaStream_t>(stream));
}

extern "C" int ardiff_entropy_gate(const void* feat, int64_t n, int32_t d, float tau, uint8_t* mask,
                                   int32_t* idx, int32_t* count, void* stream) {
    return ardiff_entropy_gate_ex(feat, n, d, tau, mask, idx, count, nullptr, stream);
}
