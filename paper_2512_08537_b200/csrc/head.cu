// K-step AdaLN residual-MLP flow head for sm_100a: one persistent kernel of CTA pairs.
//
// What it computes (per surviving token; see include/ardiff.h for the formulas): the head call
// x = Diff_theta(x_t | t, z) of the AR+Diffusion hybrid, conditioned on the token's AR hidden
// state z and on t, sampled with K Euler flow steps from caller-supplied noise.
//
// How: every matrix product of the head is cut into items of 128 tokens x 256 output columns. The two
// CTAs of a cluster form a unit: each owns one token tile, stages its own A tile (activations) and
// half of the B tile (weights) per 64-wide K slice by TMA into a 6-stage shared-memory ring, and the
// even CTA issues tcgen05.mma.cta_group::2 (256 x 256 x 16, bf16 -> fp32) into one of two TMEM
// accumulators. Eight epilogue warps per CTA read the accumulator back with tcgen05.ld and apply the
// fused tail of the layer (bias, SiLU, LayerNorm statistics, LayerNorm + modulation, gated residual,
// Euler update, scatter) while the next item's MMAs run. Results that a later GEMM reads as an operand
// (s, u, a) leave as swizzled bf16 slabs by TMA stores; the residual stream h and the gate values, which
// only epilogues touch, move between registers and global memory directly in a layout made for that.
// All items of a call form one static list (a per-step "program" of phases, repeated for every step
// and every group of token tiles); unit u takes items u, u + units, ... . The modulation GEMM of a
// block is split: its gate third does not depend on the residual stream, so gate items of block b+1
// are placed between the dependent phases of block b, where they cover the latency of the chain.
// Dependencies between items are tracked per token tile by three counters (chain, gates of even
// blocks, gates of odd blocks) with release/acquire at gpu scope; every wait is bounded.
// What binds it: the producer and the MMA issuer each walk a chain of dependent instructions per K slice
// (poll, vote, descriptors, two copies or four MMAs, commit) that takes most of the 512 cycles a slice lasts,
// and they share their schedulers with two epilogue warps each (the TMEM lane quarter a warp may read is its
// id modulo 4, so every scheduler hosts the epilogue of one quarter). Every slot an epilogue warp takes there
// lengthens the chain, and the epilogue's own loads and stores compete with the copies; the ring drains and
// the tensor pipe waits. Measured on copies of this kernel that skip work: without any epilogue work a slice
// is consumed every 545 cycles and the launch takes 21 % fewer cycles (8 points of that are the epilogue's
// memory operations); with a sixteenth of the operand bytes it takes 4 % fewer. So the kernel keeps the two chains and the
// epilogue short: biases travel in registers (one column per lane, handed round by shuffle), c never leaves
// the accumulator, epilogue inputs are plain loads issued three units ahead, h and the gate values stay off
// shared memory, and proxy fences sit only where a proxy is really crossed.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <vector>

#include "../../include/ardiff.h"
#include "common.cuh"
#include "ptx.cuh"

namespace {

using bf16 = __nv_bfloat16;

constexpr int BM = 128;           // tokens per tile (one CTA)
constexpr int BN = 256;           // output columns per item (UMMA N)
constexpr int BK = 64;            // K slice per pipeline stage (128 bytes of bf16: one swizzle row)
constexpr int A_BYTES = BM * BK * 2;
constexpr int B_ROWS = BN / 2;    // rows of the weight tile that one CTA of the pair stages
constexpr int STAGES = 6;
constexpr int STAGE_BYTES = A_BYTES + B_ROWS * BK * 2;   // 32 KB
// epilogue staging: every epilogue warp owns EPI_NB bf16 slabs (32 rows x 64 B, 64-byte swizzle) for the
// results that later GEMMs read as operands (s, u, a): written by the lanes, drained by TMA stores.
// Everything else an epilogue reads or writes (h, gate values, x) moves between registers and global memory
// directly, so that shared memory belongs to the operand ring: its depth, not its bandwidth, sets the pace.
constexpr int EPI_WARPS = 8;
constexpr int EPI_NB = 2;
constexpr int SLAB_H = 32 * 64;
constexpr int EPI_BYTES = EPI_WARPS * EPI_NB * SLAB_H;
constexpr int DEP_BARS = 8;       // the producer runs at most 6 items ahead of the epilogue
constexpr int NUM_BARS = 2 * STAGES + 5 + DEP_BARS;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + 1024 /*align slack*/ + 8 * NUM_BARS + 16;
constexpr int NUM_THREADS = 64 + 32 * EPI_WARPS;  // warp 0: TMA producer, warp 1: MMA issuer, warps 2-9: epilogue
constexpr int XB_COLS = 64;       // x is fed to the in-projection as bf16, K padded to one slice
constexpr int KMAX = 64;
constexpr int CTRS = 4;           // counters per token tile: chain, gates of even blocks, gates of odd blocks, pad
constexpr uint64_t kWaitLimitNs = 4000000000ull;   // default: a bounded wait gives up after 4 s
constexpr uint64_t kDrainLimitNs = 20000000ull;    // waits for own copies in flight at exit (ignore the abort flag)

// Optional per-item time stamps of CTA 0 (compile with -DARDIFF_HEAD_PROFILE):
// trace[(local item number * 3 + role) * 4 + slot] = clock64(); slot 3 = type * 1000 + column tile.
#ifdef ARDIFF_HEAD_PROFILE
constexpr int TRACE_ITEMS = 4096;
#define TRACE(role, slot) do { if (blockIdx.x == 0 && lane == 0 && P.trace && trace_n < TRACE_ITEMS) P.trace[((size_t)trace_n * 3 + (role)) * 4 + (slot)] = clock64(); } while (0)
#define TRACE_TYPE(role) do { if (blockIdx.x == 0 && lane == 0 && P.trace && trace_n < TRACE_ITEMS) P.trace[((size_t)trace_n * 3 + (role)) * 4 + 3] = it.type * 1000 + it.nt; } while (0)
#define TRACE_DECL int trace_n = 0;
#define TRACE_NEXT() ++trace_n
// per pipeline stage of the first 16 K slices of an item: role 0 = load issued, role 1 = MMA saw the stage full
// (bit 0 of the stamp: it had to wait for it)
#define TRACE_STAGE(role, kb) do { if (blockIdx.x == 0 && lane == 0 && P.trace && trace_n < TRACE_ITEMS / 2 && (kb) < 16) P.trace[(size_t)TRACE_ITEMS * 12 + ((size_t)trace_n * 16 + (kb)) * 2 + (role)] = clock64(); } while (0)
#else
#define TRACE_STAGE(role, kb)
#define TRACE(role, slot)
#define TRACE_TYPE(role)
#define TRACE_DECL
#define TRACE_NEXT()
#endif

enum OpType : int { OP_GATHER = 0, OP_COND, OP_IN, OP_SS, OP_GATE, OP_G1, OP_G2, OP_FSS, OP_OUT, OP_NOP, OP_END = 15 };
enum MapId : int {
    MAP_Z = 0, MAP_XB, MAP_S, MAP_U, MAP_A, MAP_WC, MAP_WIN, MAP_WCAT, MAP_WOUT,   // GEMM operands
    EMAP_S, EMAP_U, EMAP_A,                                                 // epilogue output slabs
    MAP_COUNT
};

// One phase of the per-step program: `ntiles` column tiles (tile0 ..) of one layer for every token
// tile of the group.
struct Phase {
    int type;      // OpType
    int block;     // residual block index (or -1)
    int tile0;     // first column tile of the layer this phase covers
    int ntiles;    // column tiles in this phase
    int cum;       // column tiles per token tile in the phases before it within one step
    int b_row0;    // first row of the layer's weights in the B matrix
    int offA;      // chain items of this step that must be complete (per token tile)
    int kplus;     // OP_GATE: 1 when the gate belongs to block `block` of the NEXT step
};

struct HeadParams {
    int C, Dc, W, L, K, NT, TGu, slots;     // NT = W/256, TGu = largest group in units, slots = scratch tiles
    int T_pro, T_step, T_chain;             // items per unit: prologue, one step, whole call
    int C_pro, C_step, C_total;             // chain-counter items per token tile: prologue, one step, whole call
    int R;                                  // rows of the scratch arrays (slots * 128)
    int max_tokens;
    const Phase* phases;
    const uint16_t* cum2phase;              // [T_step]: phase that holds the c-th column tile of a step
    const CUtensorMap* maps;
    const bf16* cond;
    const float* noise;
    const int* idx;
    const int* count;
    float* out;
    bf16 *z, *xb, *s, *u, *a, *g0, *g1;
    float *x, *h;
    float2* stats;
    const float *bias_cat, *bc, *bin, *temb;
    int* counters;
    int* status;
    int* abort_flag;
    long long* trace;
    const float* step_noise;                // [K][n][C] fresh noise of the sampler steps, or nullptr
    long long step_stride;                  // n * C
    float ax[KMAX], av[KMAX], an[KMAX];     // sampler step k: x <- ax x + av v + an z_k
    unsigned long long wait_limit_ns;       // bound of every dependency wait
    int stall_tile;                         // self-test: conditioning items of this token tile wait for one
                                            // predecessor more than exists (-1: none)
    long long* clock_probe;                 // [4]: clock64 and globaltimer of CTA 0 at start and end
};

struct Packed { uint32_t w0, w1, w2, w3, w4; };

struct Item {
    int type, abs_m, slot_row0, a_row0, nt, k, block, gsel;   // a_row0: first row of the A operand in its tensor
    int needA, needB;
    int map_a, map_b, b_row, kblocks, umma_n;
};

// ------------------------------------------------------------------------------------------
// device helpers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void raise_timeout(const HeadParams& P) {
    atomicExch(P.abort_flag, 1);
    atomicCAS(P.status, 0, ARDIFF_ERR_TIMEOUT);
}

// bounded wait on an mbarrier phase; false = gave up (abort raised or seen)
__device__ __forceinline__ bool wait_mbar(uint32_t bar, uint32_t parity, const HeadParams& P) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    uint64_t t0 = 0;
    for (uint32_t it = 1;; ++it) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if ((it & 127u) == 0) {
            if (ptx::ld_relaxed_gpu(P.abort_flag) != 0) return false;
            const uint64_t now = ptx::globaltimer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > P.wait_limit_ns) {
                raise_timeout(P);
                return false;
            }
        }
    }
}

// Wait at exit for this CTA's own asynchronous work (copies landing in its shared memory, MMAs writing
// its tensor memory). Bounded by time alone: after an abort the barrier may never complete (the partner's
// share of the bytes is missing), and the limit covers any latency of the work itself.
__device__ __forceinline__ void drain_mbar(uint32_t bar, uint32_t parity) {
    if (ptx::mbar_try_wait(bar, parity)) return;
    const uint64_t t0 = ptx::globaltimer_ns();
    for (uint32_t it = 1;; ++it) {
        if (ptx::mbar_try_wait(bar, parity)) return;
        if ((it & 63u) == 0 && ptx::globaltimer_ns() - t0 > kDrainLimitNs) return;
    }
}

// bounded wait until *c1 >= n1 and (c2 == nullptr or *c2 >= n2) (acquire); one thread calls it
__device__ __forceinline__ bool wait_counters(const int* c1, int n1, const int* c2, int n2, const HeadParams& P) {
    uint64_t t0 = 0;
    for (uint32_t it = 0;; ++it) {
        const int v1 = ptx::ld_acquire_gpu(c1);
        const int v2 = c2 ? ptx::ld_acquire_gpu(c2) : n2;
        if (v1 >= n1 && v2 >= n2) return true;
        if (it > 8) __nanosleep(64);
        if ((it & 63u) == 63u) {
            if (ptx::ld_relaxed_gpu(P.abort_flag) != 0) return false;
            const uint64_t now = ptx::globaltimer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > P.wait_limit_ns) {
                raise_timeout(P);
                return false;
            }
        }
    }
}

// SiLU(a) = a * sigmoid(a) = h + h * tanh(h) with h = a / 2: one special-function instruction per element
// instead of two (exp and reciprocal); the epilogues that apply it are bound by that unit. tanh.approx is
// accurate to about 2^-11, an order of magnitude below the bf16 rounding of the value that is stored.
__device__ __forceinline__ float silu_f(float a) {
    const float h = 0.5f * a;
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(h));
    return fmaf(h, t, h);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Item `item` of the static list, for the CTA of rank `rank` within its unit. MTu = units (pairs of
// token tiles) of this call, tgu = units per group (balanced over the groups).
__device__ __forceinline__ Packed decode_packed(const HeadParams& P, int MTu, int tgu, int rank, long long item,
                                                long long total) {
    Packed pk{(uint32_t)OP_END << 24, 0u, 0u, 0u, 0u};
    if (item >= total) return pk;
    const long long per_group = (long long)tgu * P.T_chain;
    const int grp = (int)(item / per_group);
    int r = (int)(item - (long long)grp * per_group);
    const int m0 = grp * tgu;
    const int mtg = min(tgu, MTu - m0);
    const int pro = mtg * P.T_pro;
    int m, type, nt = 0, k = 0, block = 0, gsel = 0;
    int needA = 0, needB = 0, b_row = 0;
    if (r < pro) {
        if (r < mtg) {
            type = OP_GATHER; m = r;
        } else if (r < mtg + mtg * P.NT) {
            r -= mtg;
            m = r / P.NT;
            nt = r - m * P.NT;
            type = OP_COND;
            needA = EPI_WARPS;            // the gather of this token tile
            b_row = nt * BN;
        } else {
            // the gate of step 0, block 0 (gate number 0): needs s_0, i.e. the conditioning items
            r -= mtg + mtg * P.NT;
            m = r / P.NT;
            nt = r - m * P.NT;
            type = OP_GATE; gsel = 1;
            needA = EPI_WARPS * P.C_pro;
            b_row = 2 * P.W + nt * BN;
        }
    } else {
        r -= pro;
        const int per_step = mtg * P.T_step;
        k = r / per_step;
        r -= k * per_step;
        const int c = r / mtg;
        const Phase p = P.phases[__ldg(P.cum2phase + c)];
        const int q = r - p.cum * mtg;
        m = q / p.ntiles;
        nt = p.tile0 + (q - m * p.ntiles);
        type = p.type; block = p.block;
        needA = EPI_WARPS * (P.C_pro + k * P.C_step + p.offA);
        b_row = p.b_row0 + nt * BN;
        // gates are numbered q = step * L + block over the whole call; gate q lives in buffer q & 1 and
        // ticks counter 1 + (q & 1), so the (q >> 1) + 1 -th gate of that parity is complete at NT * that many ticks
        if (type == OP_GATE) {
            k += p.kplus;                         // the step whose s it reads
            if (k >= P.K) type = OP_NOP;          // beyond the last step: nothing to do
            else gsel = 1 + ((k * P.L + block) & 1);
        } else if (type == OP_G2) {
            const int q = k * P.L + block;
            gsel = 1 + (q & 1);
            needB = EPI_WARPS * P.NT * ((q >> 1) + 1);
        }
    }
    const int abs_m = (m0 + m) * 2 + rank;
    if (type == OP_COND && abs_m == P.stall_tile) needA += 1;   // self-test: never satisfied
    pk.w0 = (uint32_t)abs_m | ((uint32_t)type << 24);
    pk.w1 = (uint32_t)nt | ((uint32_t)k << 8) | ((uint32_t)(block & 0xff) << 16) | ((uint32_t)gsel << 24);
    pk.w2 = (uint32_t)needA; pk.w3 = (uint32_t)needB; pk.w4 = (uint32_t)b_row;
    return pk;
}

__device__ __forceinline__ void unpack_item(const HeadParams& P, const Packed& pk, Item& it) {
    it.type = (int)(pk.w0 >> 24);
    it.abs_m = (int)(pk.w0 & 0xffffffu);
    it.slot_row0 = (it.abs_m % P.slots) * BM;
    it.nt = (int)(pk.w1 & 0xffu);
    it.k = (int)((pk.w1 >> 8) & 0xffu);
    it.block = (int)((pk.w1 >> 16) & 0xffu);
    it.gsel = (int)(pk.w1 >> 24);
    it.needA = (int)pk.w2; it.needB = (int)pk.w3; it.b_row = (int)pk.w4;
    it.kblocks = P.W / BK; it.umma_n = BN; it.map_b = MAP_WCAT; it.map_a = MAP_S;
    it.a_row0 = it.slot_row0;
    switch (it.type) {
        case OP_SS:
        case OP_GATE:
        case OP_FSS: it.a_row0 = it.k * P.R + it.slot_row0; break;     // s of step k
        case OP_COND: it.map_a = MAP_Z; it.map_b = MAP_WC; it.kblocks = P.Dc / BK; break;
        case OP_IN: it.map_a = MAP_XB; it.map_b = MAP_WIN; it.kblocks = 1; break;
        case OP_G1: it.map_a = MAP_U; break;
        case OP_G2: it.map_a = MAP_A; break;
        case OP_OUT: it.map_a = MAP_U; it.map_b = MAP_WOUT; it.umma_n = P.C; break;
        default: break;
    }
}

// The items of one CTA, decoded 32 at a time (lane l decodes the l-th of the next 32) and handed
// out by shuffle. Every lane of the warp calls next() together.
struct ItemStream {
    Packed mine;
    int n = 0;
    __device__ __forceinline__ bool next(const HeadParams& P, int MTu, int tgu, int rank, int unit_id, int n_units,
                                         long long total, int lane, Item& it) {
        if ((n & 31) == 0)
            mine = decode_packed(P, MTu, tgu, rank, (long long)unit_id + (long long)(n + lane) * n_units, total);
        Packed cur;
        const int src = n & 31;
        cur.w0 = __shfl_sync(0xffffffffu, mine.w0, src);
        cur.w1 = __shfl_sync(0xffffffffu, mine.w1, src);
        cur.w2 = __shfl_sync(0xffffffffu, mine.w2, src);
        cur.w3 = __shfl_sync(0xffffffffu, mine.w3, src);
        cur.w4 = __shfl_sync(0xffffffffu, mine.w4, src);
        ++n;
        if ((cur.w0 >> 24) == (uint32_t)OP_END) return false;
        unpack_item(P, cur, it);
        return true;
    }
};

// ------------------------------------------------------------------------------------------
// epilogues. Two epilogue warps share each 32-row quarter of the tile (TMEM lane quarter*32 + lane);
// warp half h of the pair takes accumulator columns [128 h, 128 h + 128). A thread owns one row and
// works through it in units of 16 accumulator columns.
//   h (fp32 residual stream) and the gate values (bf16) are read and written only by epilogue threads.
//   They live in a layout of their own: chunks of 32 rows x 32 columns in which the 16-byte pieces of
//   the 32 rows lie side by side, so that every 128-bit access of a warp is one contiguous 512 bytes.
//   Loads go straight to registers (L2 only: other CTAs rewrite the data) and are issued three units
//   ahead, the first ones before the accumulator is even complete.
//   s, u, a are operands of later GEMMs (read by TMA): bf16 slabs in shared memory, drained by TMA stores.
// ------------------------------------------------------------------------------------------
struct Stats {
    float p, sd, sq;
    __device__ __forceinline__ void init(float first) { p = first; sd = 0.f; sq = 0.f; }
    __device__ __forceinline__ void add(float v) { const float e = v - p; sd += e; sq = fmaf(e, e, sq); }
    __device__ __forceinline__ float2 finish(int n) const {
        const float inv = 1.0f / (float)n;
        const float mean = p + sd * inv;
        const float m2 = fmaxf(sq - sd * sd * inv, 0.f);
        return make_float2(mean, m2);
    }
};

__device__ __forceinline__ uint32_t slabH_addr(uint32_t base, int r, int c16) {
    return base + r * 64 + ((c16 ^ ((r >> 1) & 3)) << 4);
}

__device__ __forceinline__ void load_acc16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    ptx::tmem_ld_32x32b_x16(taddr, r);
    ptx::tmem_ld_wait();
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// The 32 bias values of a 32-column chunk sit one per lane (fetched at the start of the item, while the
// accumulator is still being produced) and are handed round by shuffle: no global load on the critical path.
__device__ __forceinline__ void add_bias16(float (&v)[16], float b_lane, int lane0) {
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] += __shfl_sync(0xffffffffu, b_lane, lane0 + i);
}

// 16 columns of this lane's row as bf16 into a slab (pieces 2 hu and 2 hu + 1 of the row's four)
__device__ __forceinline__ void slabH_write16(uint32_t base, int r, int hu, const float (&v)[16]) {
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        uint4 w;
        w.x = pack_bf16x2(v[8 * c], v[8 * c + 1]);
        w.y = pack_bf16x2(v[8 * c + 2], v[8 * c + 3]);
        w.z = pack_bf16x2(v[8 * c + 4], v[8 * c + 5]);
        w.w = pack_bf16x2(v[8 * c + 6], v[8 * c + 7]);
        ptx::sts_u4(slabH_addr(base, r, 2 * hu + c), w);
    }
}

// Chunked layout of h (fp32) and of the gate values (bf16): element (row, col) of a [rows][W] array lives
// in chunk (row / 32, col / 32); inside the chunk the 16-byte piece p of the row's 32 columns of lane
// row % 32 sits at 16-byte index p * 32 + lane. A 16-column unit u of a warp's span is pieces
// 4 (u & 1) .. + 3 (fp32) or 2 (u & 1), + 1 (bf16) of chunk (first chunk + u / 2).
// h is the one array that every residual block reads twice and writes once (three bytes of DRAM traffic per
// byte held and block when it misses), and one group's h fits the part of L2 that a context may set aside for
// persisting accesses: its loads and stores carry the evict_last policy, which keeps it there while the
// bf16 operands stream past (ardiff_head_create sets that part aside).
__device__ __forceinline__ size_t chunk_of(const HeadParams& P, int row0, int col0) {
    return (size_t)(row0 >> 5) * (size_t)(P.W >> 5) + (size_t)(col0 >> 5);
}
struct UnitH { float4 p[4]; };      // 16 fp32 of one row
struct UnitG { uint4 p[2]; };       // 16 bf16 of one row
__device__ __forceinline__ void load_unit_h(const float* h, size_t chunk, int u, int lane, UnitH& d) {
    const float* src = h + (chunk + (size_t)(u >> 1)) * 1024 + (size_t)((u & 1) * 4) * 128 + lane * 4;
    const uint64_t pol = ptx::l2_evict_last_policy();
#pragma unroll
    for (int q = 0; q < 4; ++q) d.p[q] = ptx::ldcg_f4_hint(src + q * 128, pol);
}
__device__ __forceinline__ void store_unit_h(float* h, size_t chunk, int u, int lane, const float (&v)[16]) {
    float* dst = h + (chunk + (size_t)(u >> 1)) * 1024 + (size_t)((u & 1) * 4) * 128 + lane * 4;
    const uint64_t pol = ptx::l2_evict_last_policy();
#pragma unroll
    for (int q = 0; q < 4; ++q)
        ptx::st_f4_hint(dst + q * 128, make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]), pol);
}
__device__ __forceinline__ void load_unit_g(const bf16* g, size_t chunk, int u, int lane, UnitG& d) {
    const bf16* src = g + (chunk + (size_t)(u >> 1)) * 1024 + (size_t)((u & 1) * 2) * 256 + lane * 8;
#pragma unroll
    for (int q = 0; q < 2; ++q) d.p[q] = ptx::ldcg_u4(src + q * 256);
}
__device__ __forceinline__ void store_unit_g(bf16* g, size_t chunk, int u, int lane, const float (&v)[16]) {
    bf16* dst = g + (chunk + (size_t)(u >> 1)) * 1024 + (size_t)((u & 1) * 2) * 256 + lane * 8;
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        uint4 w;
        w.x = pack_bf16x2(v[8 * q], v[8 * q + 1]);
        w.y = pack_bf16x2(v[8 * q + 2], v[8 * q + 3]);
        w.z = pack_bf16x2(v[8 * q + 4], v[8 * q + 5]);
        w.w = pack_bf16x2(v[8 * q + 6], v[8 * q + 7]);
        ptx::st_u4(dst + q * 256, w);
    }
}
__device__ __forceinline__ void unit_h_values(const UnitH& d, float (&v)[16]) {
#pragma unroll
    for (int q = 0; q < 4; ++q) { v[4 * q] = d.p[q].x; v[4 * q + 1] = d.p[q].y; v[4 * q + 2] = d.p[q].z; v[4 * q + 3] = d.p[q].w; }
}
__device__ __forceinline__ void unit_g_values(const UnitG& d, float (&v)[16]) {
#pragma unroll
    for (int q = 0; q < 2; ++q) {
        const uint4 w = d.p[q];
        v[8 * q] = bf16lo(w.x); v[8 * q + 1] = bf16hi(w.x); v[8 * q + 2] = bf16lo(w.y); v[8 * q + 3] = bf16hi(w.y);
        v[8 * q + 4] = bf16lo(w.z); v[8 * q + 5] = bf16hi(w.z); v[8 * q + 6] = bf16lo(w.w); v[8 * q + 7] = bf16hi(w.w);
    }
}

// LayerNorm statistics of one row from its 2*NT partials (mean, M2 over 128 columns each). One pass:
// the first partial's mean serves as pivot, so nothing cancels.
__device__ __forceinline__ void row_mean_rstd(const HeadParams& P, int grow, float& mean, float& rstd) {
    const int np = 2 * P.NT;
    const float2* sp = P.stats + (size_t)grow * np;
    const float2 v0 = ptx::ldcg_f2(sp);
    float sd = 0.f, m2 = v0.y;
#pragma unroll 4
    for (int t = 1; t < np; ++t) {
        const float2 v = ptx::ldcg_f2(sp + t);
        const float dm = v.x - v0.x;
        sd += dm;
        m2 += fmaf(128.0f * dm, dm, v.y);
    }
    const float dmean = sd / (float)np;                       // mean - pivot
    mean = v0.x + dmean;
    m2 = fmaxf(m2 - (float)P.W * dmean * dmean, 0.f);
    rstd = rsqrtf(m2 / (float)P.W + 1e-6f);
}

// v = acc + bout ; x <- ax_k x + av_k v + an_k z_k ; bf16 copy for the next in-projection ; last step: out[idx[j]] = x
__device__ __forceinline__ void epi_out(const HeadParams& P, const Item& it, uint32_t tacc, int grow,
                                        int j, int count) {
    const float ax = P.ax[it.k], av = P.av[it.k], an = P.an[it.k];
    float* xrow = P.x + (size_t)grow * P.C;
    bf16* xbrow = P.xb + (size_t)grow * XB_COLS;
    const float* bias = P.bias_cat + it.b_row;
    const bool last = (it.k == P.K - 1);
    float* orow = nullptr;
    const float* zrow = nullptr;
    if (j < count && (last || P.step_noise)) {
        const size_t tok = (size_t)__ldg(P.idx + j);
        if (last) orow = P.out + tok * P.C;
        if (P.step_noise) zrow = P.step_noise + (size_t)it.k * (size_t)P.step_stride + tok * P.C;
    }
    for (int cc = 0; cc < P.C / 16; ++cc) {
        uint32_t r[16];
        ptx::tmem_ld_32x32b_x16(tacc + cc * 16, r);
        ptx::tmem_ld_wait();
        float xn[16];
#pragma unroll
        for (int i = 0; i < 16; i += 4) {
            const float4 b = __ldg(reinterpret_cast<const float4*>(bias + cc * 16 + i));
            const float4 xo = ptx::ldcg_f4(xrow + cc * 16 + i);
            float4 base = make_float4(ax * xo.x, ax * xo.y, ax * xo.z, ax * xo.w);   // ax = 1: exactly x
            if (zrow) {
                const float4 z = __ldg(reinterpret_cast<const float4*>(zrow + cc * 16 + i));
                base.x = fmaf(an, z.x, base.x); base.y = fmaf(an, z.y, base.y);
                base.z = fmaf(an, z.z, base.z); base.w = fmaf(an, z.w, base.w);
            }
            xn[i] = fmaf(av, __uint_as_float(r[i]) + b.x, base.x);
            xn[i + 1] = fmaf(av, __uint_as_float(r[i + 1]) + b.y, base.y);
            xn[i + 2] = fmaf(av, __uint_as_float(r[i + 2]) + b.z, base.z);
            xn[i + 3] = fmaf(av, __uint_as_float(r[i + 3]) + b.w, base.w);
        }
#pragma unroll
        for (int i = 0; i < 16; i += 4) {
            const float4 v4 = make_float4(xn[i], xn[i + 1], xn[i + 2], xn[i + 3]);
            ptx::st_f4(xrow + cc * 16 + i, v4);
            if (orow) ptx::st_f4(orow + cc * 16 + i, v4);
        }
#pragma unroll
        for (int i = 0; i < 16; i += 8) {
            uint4 w;
            w.x = pack_bf16x2(xn[i], xn[i + 1]);
            w.y = pack_bf16x2(xn[i + 2], xn[i + 3]);
            w.z = pack_bf16x2(xn[i + 4], xn[i + 5]);
            w.w = pack_bf16x2(xn[i + 6], xn[i + 7]);
            ptx::st_u4(xbrow + cc * 16 + i, w);
        }
    }
}

// 16 rows of this token tile per epilogue warp: z = cond[idx[j]], x = noise[idx[j]], xb = bf16(x);
// rows past count: 0. The 16 token ids are fetched with one load and the rows are copied four at a
// time, so that many independent loads are in flight (the rows sit in HBM).
__device__ __forceinline__ void gather_rows(const HeadParams& P, const Item& it, int ew, int lane, int count) {
    const int chunks = P.Dc / 8;  // 16-byte chunks per cond row
    constexpr int RPW = BM / EPI_WARPS;
    const int r0 = ew * RPW;
    const int j0 = it.abs_m * BM + r0;
    int my_tok = -1;
    if (lane < RPW && j0 + lane < count) my_tok = __ldg(P.idx + j0 + lane);
#pragma unroll 1
    for (int rr = 0; rr < RPW; rr += 4) {
        int tok[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) tok[q] = __shfl_sync(0xffffffffu, my_tok, rr + q);
        for (int c = lane; c < chunks; c += 32) {
            uint4 v[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                v[q] = make_uint4(0, 0, 0, 0);
                if (tok[q] >= 0) v[q] = __ldg(reinterpret_cast<const uint4*>(P.cond + (size_t)tok[q] * P.Dc) + c);
            }
#pragma unroll
            for (int q = 0; q < 4; ++q)
                reinterpret_cast<uint4*>(P.z + (size_t)(it.slot_row0 + r0 + rr + q) * P.Dc)[c] = v[q];
        }
        for (int c = lane; c < P.C; c += 32) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int grow = it.slot_row0 + r0 + rr + q;
                const float xv = tok[q] >= 0 ? __ldg(P.noise + (size_t)tok[q] * P.C + c) : 0.f;
                P.x[(size_t)grow * P.C + c] = xv;
                P.xb[(size_t)grow * XB_COLS + c] = __float2bfloat16_rn(xv);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// the persistent kernel: clusters of two CTAs. Both load their own token tile (A) and half of the
// weight tile (B); the even CTA issues cta_group::2 MMAs that read both CTAs' shared memory and
// write 128 accumulator rows into each CTA's TMEM; every CTA runs the epilogue of its own token tile.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(NUM_THREADS, 1) head_kernel(const __grid_constant__ HeadParams P) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t smem_base = ptx::smem_u32(smem);
    const uint32_t epi_base = smem_base + STAGES * STAGE_BYTES;      // 1024-aligned
    const uint32_t bars = epi_base + EPI_BYTES;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
    auto tfull_bar = [&](int b) { return bars + 8u * (2 * STAGES + b); };
    auto tempty_bar = [&](int b) { return bars + 8u * (2 * STAGES + 2 + b); };
    const uint32_t drain_bar = bars + 8u * (2 * STAGES + 4);
    auto dep_bar = [&](uint32_t i) { return bars + 8u * (2 * STAGES + 5 + (i % DEP_BARS)); };
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + STAGES * STAGE_BYTES + EPI_BYTES + 8 * NUM_BARS);
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int rank = (int)ptx::cluster_ctarank();                  // token tile of the unit this CTA owns
    const int unit_id = (int)blockIdx.x / 2;
    const int n_units = (int)gridDim.x / 2;

    int count = __ldg(P.count);
    if (count > P.max_tokens) {
        count = P.max_tokens;
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicCAS(P.status, 0, ARDIFF_ERR_SHAPE);
    }
    if (count < 0) count = 0;
    const int MT = (count + BM - 1) / BM;
    const int MTu = (MT + 1) / 2;                  // an odd last tile gets an all-padding partner
    const int n_groups = (MTu + P.TGu - 1) / P.TGu;
    const int tgu = n_groups > 0 ? (MTu + n_groups - 1) / n_groups : 1;   // balanced group size
    const long long total = (long long)MTu * P.T_chain;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(full_bar(s), 1);
            ptx::mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            ptx::mbar_init(tfull_bar(b), 1);
            ptx::mbar_init(tempty_bar(b), 2 * EPI_WARPS);   // epilogue warps of both CTAs of the unit
        }
        ptx::mbar_init(drain_bar, 1);
        for (int i = 0; i < DEP_BARS; ++i) ptx::mbar_init(dep_bar(i), 1);
        ptx::fence_mbar_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(ptx::smem_u32(tmem_slot), 512);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before();
    ptx::cluster_sync_all();
    ptx::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    long long probe_c0 = 0;
    unsigned long long probe_g0 = 0;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        probe_c0 = clock64();
        probe_g0 = ptx::globaltimer_ns();
    }

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        int stage = 0;
        uint32_t phase = 0;
        uint32_t issued = 0, issued_parity = 0;
        uint32_t seq = 0;
        bool aborted = false;
        ItemStream ist;
        Item it, nx;
        TRACE_DECL
        // next item with operands to load (gather items have none)
        auto next_item = [&](Item& dst) {
            bool have;
            do have = ist.next(P, MTu, tgu, rank, unit_id, n_units, total, lane, dst);
            while (have && (dst.type == OP_GATHER || dst.type == OP_NOP));
            return have;
        };
        bool have = next_item(it);
        bool pre_ok = false;    // the dependencies of `it` were already seen complete while the item before it streamed
        while (have) {
            const bool have_nx = next_item(nx);
            bool ok = true;
            if (lane == 0 && !pre_ok) {
                const int* ctr = P.counters + (size_t)it.abs_m * CTRS;
                ok = wait_counters(ctr, it.needA, it.needB ? ctr + it.gsel : nullptr, it.needB, P);
            }
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) { aborted = true; break; }
            TRACE(0, 0);
            if (lane == 0) ptx::mbar_arrive(dep_bar(seq));      // the epilogue may now load this item's inputs
            ++seq;
            // operands that other CTAs wrote with plain stores (z, xb) cross from the generic to the async proxy;
            // everything else was written by TMA stores and is read by TMA loads
            if (it.type == OP_COND || it.type == OP_IN) ptx::fence_proxy_async();
            const void* map_a = P.maps + it.map_a;
            const void* map_b = P.maps + it.map_b;
            const int b_rows = it.umma_n / 2;                         // rows of B this CTA stages
            const uint32_t tx = 2u * (A_BYTES + (uint32_t)b_rows * BK * 2);
            const int peek_kb = it.kblocks > 3 ? it.kblocks - 3 : 0;
            int pv1 = 0, pv2 = 0;      // the next item's counters, read while this item still streams
            for (int kb = 0; kb < it.kblocks; ++kb) {
                ok = wait_mbar(empty_bar(stage), phase ^ 1u, P);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (kb == 0) TRACE(0, 1);
                TRACE_STAGE(0, kb);
                if (lane == 0) {
                    const uint32_t sa = smem_base + stage * STAGE_BYTES;
                    // the even CTA arms its barrier for the bytes of both CTAs
                    if (rank == 0) ptx::mbar_arrive_expect_tx(full_bar(stage), tx);
                    ptx::tma_load_2d_pair(sa, map_a, full_bar(stage), kb * BK, it.a_row0);
                    ptx::tma_load_2d_pair(sa + A_BYTES, map_b, full_bar(stage), kb * BK, it.b_row + rank * b_rows);
                    if (kb == peek_kb && have_nx) {
                        // issued here, looked at only after the last slice went out
                        const int* ctr = P.counters + (size_t)nx.abs_m * CTRS;
                        pv1 = ptx::ld_acquire_gpu(ctr);
                        pv2 = nx.needB ? ptx::ld_acquire_gpu(ctr + nx.gsel) : 0;
                    }
                }
                issued |= 1u << stage;
                issued_parity = (issued_parity & ~(1u << stage)) | (phase << stage);
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
            TRACE(0, 2); TRACE_TYPE(0); TRACE_NEXT();
            if (!ok) { aborted = true; break; }
            const int pre = (have_nx && pv1 >= nx.needA && pv2 >= nx.needB) ? 1 : 0;
            pre_ok = __shfl_sync(0xffffffffu, pre, 0) != 0;
            it = nx;
            have = have_nx;
        }
        // own copies in flight must have landed before the CTA exits. In the even CTA the full
        // barriers are local: wait for every stage's last issue. The odd CTA's loads are counted on
        // the even CTA's barriers; after a normal run they were all consumed, after an abort it
        // simply waits out a bounded time that covers any TMA latency.
        if (rank == 0) {
            for (int s = 0; s < STAGES; ++s)
                if (issued & (1u << s)) drain_mbar(full_bar(s), (issued_parity >> s) & 1u);
        } else if (aborted) {
            const uint64_t t0 = ptx::globaltimer_ns();
            while (ptx::globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (the even CTA issues for the pair) ----------------
        if (rank == 0) {
            int stage = 0;
            uint32_t phase = 0;
            uint32_t acc_iter = 0;
            ItemStream ist;
            Item it;
            TRACE_DECL
            while (ist.next(P, MTu, tgu, rank, unit_id, n_units, total, lane, it)) {
                if (it.type == OP_GATHER || it.type == OP_NOP) continue;
                const uint32_t buf = acc_iter & 1u;
                const uint32_t acc_phase = (acc_iter >> 1) & 1u;
                bool ok = wait_mbar(tempty_bar(buf), acc_phase ^ 1u, P);
                ok = __all_sync(0xffffffffu, ok);
                TRACE(1, 0);
                if (!ok) break;
                ptx::tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                const uint32_t idesc = ptx::idesc_bf16_f32(2 * BM, (uint32_t)it.umma_n);
                for (int kb = 0; kb < it.kblocks; ++kb) {
                    ok = wait_mbar(full_bar(stage), phase, P);
                    ok = __all_sync(0xffffffffu, ok);
                    if (kb == 0) TRACE(1, 1);
                    TRACE_STAGE(1, kb);
                    if (!ok) break;
                    ptx::tc_fence_after();
                    if (lane == 0) {
                        const uint32_t sa = smem_base + stage * STAGE_BYTES;
                        const uint64_t da = ptx::smem_desc_sw128(sa);
                        const uint64_t db = ptx::smem_desc_sw128(sa + A_BYTES);
#pragma unroll
                        for (int k = 0; k < BK / 16; ++k)
                            ptx::mma_f16_ss_pair(d_tmem, da + (uint64_t)(k * 2), db + (uint64_t)(k * 2), idesc,
                                                 (kb | k) != 0 ? 1u : 0u);
                        ptx::mma_commit_pair_mc(empty_bar(stage), 3);   // frees the stage in both CTAs
                    }
                    __syncwarp();
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                if (lane == 0) ptx::mma_commit_pair_mc(tfull_bar(buf), 3);
                __syncwarp();
                ++acc_iter;
                TRACE(1, 2); TRACE_TYPE(1); TRACE_NEXT();
            }
            // all MMAs this thread issued must be done before TMEM is freed
            if (lane == 0) ptx::mma_commit_pair(drain_bar);
            __syncwarp();
            drain_mbar(drain_bar, 0);
        }
    } else {
        // ---------------- epilogue warps ----------------
        const int ew = warp - 2;              // 0..7
        const int quarter = warp & 3;         // TMEM lane quarter this warp may read
        const int half = ew >> 2;             // column half of the accumulator this warp takes
        const int row = quarter * 32 + lane;  // row of the tile owned by this thread
        const uint32_t my_buf = epi_base + (uint32_t)ew * EPI_NB * SLAB_H;
        uint32_t acc_iter = 0;
        uint32_t seq = 0;
        ItemStream ist;
        Item it;
        TRACE_DECL
        while (ist.next(P, MTu, tgu, rank, unit_id, n_units, total, lane, it)) {
            bool fail = false;
            if (it.type == OP_NOP) continue;
            if (it.type == OP_GATHER) {
                bool ok = true;
                // the scratch slot is free once the token tile that used it before has run its whole chain
                if (lane == 0 && it.abs_m >= P.slots)
                    ok = wait_counters(P.counters + (size_t)(it.abs_m - P.slots) * CTRS, EPI_WARPS * P.C_total,
                                       nullptr, 0, P);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                gather_rows(P, it, ew, lane, count);
            } else {
                // the producer has seen this item's dependencies complete
                bool ok = wait_mbar(dep_bar(seq), (seq / DEP_BARS) & 1u, P);
                ok = __all_sync(0xffffffffu, ok);
                ++seq;
                if (!ok) break;
                if (ew == 0) TRACE(2, 0);
                const bool mod = (it.type == OP_SS || it.type == OP_FSS);
                // this warp's span: 128 accumulator columns (64 of shift and 64 of scale for a modulation item)
                const int acc0 = mod ? half * 64 : half * 128;
                const int col0 = mod ? it.nt * 128 + half * 64 : it.nt * BN + half * 128;   // column of the layer's output
                const int row0 = it.slot_row0 + quarter * 32;
                const int grow = it.slot_row0 + row;
                const size_t chunk0 = chunk_of(P, row0, col0);
                // inputs that do not come from the accumulator are asked for now, three units deep, while the
                // MMAs of this item still run
                UnitH hin[4];
                UnitG gin[4];
                const bf16* gsrc = it.gsel == 2 ? P.g1 : P.g0;
                if (it.type == OP_G2) {
#pragma unroll
                    for (int u = 0; u < 3; ++u) {
                        load_unit_h(P.h, chunk0, u, lane, hin[u]);
                        load_unit_g(gsrc, chunk0, u, lane, gin[u]);
                    }
                } else if (mod) {
#pragma unroll
                    for (int u = 0; u < 3; ++u) load_unit_h(P.h, chunk0, u, lane, hin[u]);
                }
                // bias values of the warp's chunks, one column per lane (modulation items: shift in bq[0..1], scale in bq[2..3])
                float bq[4] = {0.f, 0.f, 0.f, 0.f};
                {
                    const float* bb = it.type == OP_IN     ? P.bin + col0
                                      : it.type == OP_COND ? P.bc + col0
                                                           : P.bias_cat + it.b_row + acc0;
                    if (it.type != OP_OUT) {
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            bq[q] = __ldg(bb + (mod ? (q & 1) * 32 + (q >> 1) * 128 : q * 32) + lane);
                    }
                }
                float mean = 0.f, rstd = 0.f;
                if (mod) row_mean_rstd(P, grow, mean, rstd);
                const uint32_t buf = acc_iter & 1u;
                const uint32_t acc_phase = (acc_iter >> 1) & 1u;
                ok = wait_mbar(tfull_bar(buf), acc_phase, P);
                ok = __all_sync(0xffffffffu, ok);
                fail = !ok;
                if (ew == 0) TRACE(2, 1);
                ptx::tc_fence_after();
                const uint32_t tacc = tmem_base + buf * BN + ((uint32_t)(quarter * 32) << 16);
                // a slab may be rewritten once the TMA store that read it last (two stores back) is done reading
                auto slab_ready = [&]() {
                    if (lane == 0) ptx::bulk_wait_read<EPI_NB - 1>();
                    __syncwarp();
                };
                auto slab_store = [&](int map, uint32_t slab, int col, int grow0) {
                    ptx::fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        ptx::tma_store_2d(P.maps + map, slab, col, grow0);
                        ptx::bulk_commit();
                    }
                };
                if (fail) {
                    // aborted: nothing valid to work on
                } else if (it.type == OP_OUT) {
                    if (half == 0) epi_out(P, it, tacc, grow, it.abs_m * BM + row, count);
                } else if (it.type == OP_COND) {
                    // c = acc + bc stays in registers; s_k = SiLU(c + temb_k) leaves as one bf16 slab per step
                    int n_st = 0;
#pragma unroll 1
                    for (int j = 0; j < 4; ++j) {
                        float cv[32];
                        {
                            float lo[16], hi[16];
                            load_acc16(tacc + acc0 + 32 * j, lo);
                            load_acc16(tacc + acc0 + 32 * j + 16, hi);
                            const float bj = j == 0 ? bq[0] : j == 1 ? bq[1] : j == 2 ? bq[2] : bq[3];
                            add_bias16(lo, bj, 0);
                            add_bias16(hi, bj, 16);
#pragma unroll
                            for (int i = 0; i < 16; ++i) { cv[i] = lo[i]; cv[16 + i] = hi[i]; }
                        }
                        float tk = __ldg(P.temb + col0 + 32 * j + lane);          // temb_k of this lane's column
#pragma unroll 1
                        for (int k = 0; k < P.K; ++k, ++n_st) {
                            const float tcur = tk;
                            if (k + 1 < P.K) tk = __ldg(P.temb + (size_t)(k + 1) * P.W + col0 + 32 * j + lane);
                            const uint32_t sl = my_buf + (uint32_t)(n_st & 1) * SLAB_H;
                            slab_ready();
                            float sv[16];
#pragma unroll
                            for (int hu = 0; hu < 2; ++hu) {
#pragma unroll
                                for (int i = 0; i < 16; ++i)
                                    sv[i] = silu_f(cv[16 * hu + i] + __shfl_sync(0xffffffffu, tcur, 16 * hu + i));
                                slabH_write16(sl, lane, hu, sv);
                            }
                            slab_store(EMAP_S, sl, col0 + 32 * j, k * P.R + row0);
                        }
                    }
                } else if (it.type == OP_IN) {
                    // h = acc + bin, straight to global memory; LayerNorm partials of the 128 columns
                    Stats st;
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        float v[16];
                        load_acc16(tacc + acc0 + 16 * u, v);
                        add_bias16(v, (u >> 1) == 0 ? bq[0] : (u >> 1) == 1 ? bq[1] : (u >> 1) == 2 ? bq[2] : bq[3], 16 * (u & 1));
                        if (u == 0) st.init(v[0]);
#pragma unroll
                        for (int i = 0; i < 16; ++i) st.add(v[i]);
                        store_unit_h(P.h, chunk0, u, lane, v);
                    }
                    P.stats[(size_t)grow * (2 * P.NT) + it.nt * 2 + half] = st.finish(128);
                } else if (it.type == OP_GATE) {
                    // g = acc + bias, as bf16 straight to global memory
                    bf16* gdst = it.gsel == 2 ? P.g1 : P.g0;
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        float v[16];
                        load_acc16(tacc + acc0 + 16 * u, v);
                        add_bias16(v, (u >> 1) == 0 ? bq[0] : (u >> 1) == 1 ? bq[1] : (u >> 1) == 2 ? bq[2] : bq[3], 16 * (u & 1));
                        store_unit_g(gdst, chunk0, u, lane, v);
                    }
                } else if (it.type == OP_G1) {
                    // a = SiLU(acc + b1): operand of the next GEMM, leaves as bf16 slabs
#pragma unroll 1
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t sl = my_buf + (uint32_t)(j & 1) * SLAB_H;
                        const float bj = j == 0 ? bq[0] : j == 1 ? bq[1] : j == 2 ? bq[2] : bq[3];
                        slab_ready();
#pragma unroll
                        for (int hu = 0; hu < 2; ++hu) {
                            float v[16];
                            load_acc16(tacc + acc0 + 32 * j + 16 * hu, v);
                            add_bias16(v, bj, 16 * hu);
#pragma unroll
                            for (int i = 0; i < 16; ++i) v[i] = silu_f(v[i]);
                            slabH_write16(sl, lane, hu, v);
                        }
                        slab_store(EMAP_A, sl, col0 + 32 * j, row0);
                    }
                } else if (mod) {
                    // u = LN(h) * (1 + scale) + shift: operand of the next GEMM, leaves as bf16 slabs
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const uint32_t sl = my_buf + (uint32_t)((u >> 1) & 1) * SLAB_H;
                        if (u + 3 < 4) load_unit_h(P.h, chunk0, u + 3, lane, hin[(u + 3) & 3]);
                        if ((u & 1) == 0) slab_ready();
                        float sh[16], sc[16], hv[16];
                        load_acc16(tacc + acc0 + 16 * u, sh);
                        load_acc16(tacc + acc0 + 128 + 16 * u, sc);
                        add_bias16(sh, (u >> 1) == 0 ? bq[0] : bq[1], 16 * (u & 1));
                        add_bias16(sc, (u >> 1) == 0 ? bq[2] : bq[3], 16 * (u & 1));
                        unit_h_values(hin[u & 3], hv);
#pragma unroll
                        for (int i = 0; i < 16; ++i) hv[i] = fmaf((hv[i] - mean) * rstd, 1.0f + sc[i], sh[i]);
                        slabH_write16(sl, lane, u & 1, hv);
                        if (u & 1) slab_store(EMAP_U, sl, col0 + 32 * (u >> 1), row0);
                    }
                } else {
                    // OP_G2: h += g * (acc + b2), read and written in place; LayerNorm partials of the 128 columns
                    Stats st;
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        if (u + 3 < 8) {
                            load_unit_h(P.h, chunk0, u + 3, lane, hin[(u + 3) & 3]);
                            load_unit_g(gsrc, chunk0, u + 3, lane, gin[(u + 3) & 3]);
                        }
                        float v[16], gv[16], hv[16];
                        load_acc16(tacc + acc0 + 16 * u, v);
                        add_bias16(v, (u >> 1) == 0 ? bq[0] : (u >> 1) == 1 ? bq[1] : (u >> 1) == 2 ? bq[2] : bq[3], 16 * (u & 1));
                        unit_g_values(gin[u & 3], gv);
                        unit_h_values(hin[u & 3], hv);
#pragma unroll
                        for (int i = 0; i < 16; ++i) hv[i] = fmaf(gv[i], v[i], hv[i]);
                        if (u == 0) st.init(hv[0]);
#pragma unroll
                        for (int i = 0; i < 16; ++i) st.add(hv[i]);
                        store_unit_h(P.h, chunk0, u, lane, hv);
                    }
                    P.stats[(size_t)grow * (2 * P.NT) + it.nt * 2 + half] = st.finish(128);
                }
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive_even_cta(tempty_bar(buf));
                ++acc_iter;
                if (lane == 0) ptx::bulk_wait<0>();   // this warp's TMA stores are performed
                __syncwarp();
            }
            if (fail) break;
            // publish: this warp's global writes, then one tick of the token tile's counter
            // The release below is cumulative: it covers this lane's completed TMA stores and, through the
            // warp barrier, the other lanes' plain stores. Rows written with plain stores that other CTAs
            // read by TMA (z, xb) additionally need the generic -> async proxy fence on the writer's side.
            if (it.type == OP_GATHER || it.type == OP_OUT) ptx::fence_proxy_async();
            __syncwarp();
            if (lane == 0)
                ptx::red_release_gpu_add(P.counters + (size_t)it.abs_m * CTRS + (it.type == OP_GATE ? it.gsel : 0), 1);
            if (it.type != OP_GATHER) {
                if (ew == 0) { TRACE(2, 2); TRACE_TYPE(2); }
                TRACE_NEXT();
            }
        }
        // own copies in flight: stores not yet done
        if (lane == 0) ptx::bulk_wait<0>();
        __syncwarp();
    }

    ptx::tc_fence_before();
    // nobody leaves while its partner may still signal its barriers or read its shared memory
    ptx::cluster_sync_all();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc_pair(tmem_base, 512);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0 && P.clock_probe) {
        // SM cycles and wall time of this launch as seen by CTA 0: their ratio is the clock the SM really ran at
        P.clock_probe[0] = clock64() - probe_c0;
        P.clock_probe[1] = (long long)(ptx::globaltimer_ns() - probe_g0);
    }
}

// ------------------------------------------------------------------------------------------
// small kernels: time embedding MLP, K = 0 copy
// ------------------------------------------------------------------------------------------
struct TimeArgs {
    float t[KMAX];
};

// hidden[k][o] = SiLU(Wt1[o] . e(t_k) + bt1[o]); one warp per output
__global__ void __launch_bounds__(256) temb_hidden_kernel(const bf16* __restrict__ Wt1,
                                                         const float* __restrict__ bt1, int W, int F,
                                                         TimeArgs ta, float* __restrict__ hidden) {
    extern __shared__ float e_s[];
    const int k = blockIdx.y;
    const int half = F / 2;
    for (int f = threadIdx.x; f < half; f += blockDim.x) {
        const double w = exp(-log(10000.0) * (double)f / (double)half);
        const double arg = 1000.0 * (double)ta.t[k] * w;
        double sn, cs;
        sincos(arg, &sn, &cs);
        e_s[f] = (float)cs;
        e_s[half + f] = (float)sn;
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int o = blockIdx.x * 8 + warp;
    if (o >= W) return;
    const bf16* wr = Wt1 + (size_t)o * F;
    float acc = 0.f;
    for (int i = lane; i < F; i += 32) acc = fmaf(__bfloat162float(wr[i]), e_s[i], acc);
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, d);
    if (lane == 0) {
        const float a = acc + bt1[o];
        hidden[(size_t)k * W + o] = a / (1.0f + expf(-a));
    }
}

// temb[k][o] = Wt2[o] . hidden[k] + bt2[o]
__global__ void __launch_bounds__(256) temb_out_kernel(const bf16* __restrict__ Wt2,
                                                      const float* __restrict__ bt2, int W,
                                                      const float* __restrict__ hidden,
                                                      float* __restrict__ temb) {
    const int k = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int o = blockIdx.x * 8 + warp;
    if (o >= W) return;
    const bf16* wr = Wt2 + (size_t)o * W;
    const float* hk = hidden + (size_t)k * W;
    float acc = 0.f;
    for (int i = lane * 2; i < W; i += 64) {
        const __nv_bfloat162 w2 = *reinterpret_cast<const __nv_bfloat162*>(wr + i);
        acc = fmaf(__low2float(w2), hk[i], acc);
        acc = fmaf(__high2float(w2), hk[i + 1], acc);
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, d);
    if (lane == 0) temb[(size_t)k * W + o] = acc + bt2[o];
}

__global__ void copy_noise_rows_kernel(const float* __restrict__ noise, const int* __restrict__ idx,
                                       const int* __restrict__ count, int max_tokens, int C,
                                       float* __restrict__ out) {
    int cnt = min(*count, max_tokens);
    const long long total = (long long)cnt * C;
    for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < total;
         e += (long long)gridDim.x * blockDim.x) {
        const int j = (int)(e / C), c = (int)(e % C);
        const size_t tok = (size_t)idx[j];
        out[tok * C + c] = noise[tok * C + c];
    }
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// 2-D bf16 row-major [rows][cols] tensor, box = [box_rows][64 cols], 128-byte swizzle
bool make_map(CUtensorMap* m, void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {BK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// epilogue output slabs: bf16, box = [32 rows][32 columns], 64-byte rows, 64-byte swizzle
bool make_slab_map(CUtensorMap* m, void* base, uint64_t rows, uint64_t cols) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {32, 32};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline float bf16_bits_to_float(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

}  // namespace

struct ardiff_head {
    ardiff_head_desc d;
    int device, n_sm, grid, coop;
    int NT, TGu, slots, T_pro, T_step, C_pro, C_step, n_phases;
    int64_t max_tiles;
    std::vector<void*> allocs;
    // device
    bf16 *Wcat, *Wc, *Win, *Wt1, *Wt2;
    float *bias_cat, *bc, *bin, *bt1, *bt2, *temb, *temb_hidden;
    bf16 *z, *xb, *s, *u, *a, *g0, *g1;
    float *x, *h;
    float2* stats;
    int *counters, *status;  // status[0] = status word, status[1] = abort flag
    long long* trace;        // per-item time stamps (only with ARDIFF_HEAD_PROFILE)
    Phase* phases;
    uint16_t* cum2phase;
    CUtensorMap* maps;
    long long* clock_probe;  // [2]: SM cycles and nanoseconds of the last launch, stamped by CTA 0
    // optional timing of the persistent kernel (state of the last call, not of the head: mutable)
    int timing;
    mutable int timed;
    cudaEvent_t ev0, ev1;
    // self-test of the bounded waits, armed for the next sample call only
    mutable int stall_tile;
    mutable unsigned int stall_limit_us;
};

namespace {

template <typename T>
int dev_alloc(ardiff_head* H, T** p, size_t count, bool zero) {
    void* q = nullptr;
    if (cudaMalloc(&q, count * sizeof(T) + 256) != cudaSuccess) {
        (void)cudaGetLastError();
        return ARDIFF_ERR_NOMEM;
    }
    H->allocs.push_back(q);
    if (zero && cudaMemset(q, 0, count * sizeof(T) + 256) != cudaSuccess) return ARDIFF_ERR_CUDA;
    *p = reinterpret_cast<T*>(q);
    return ARDIFF_OK;
}

int upload(void* dst, const void* src, size_t bytes) {
    return cudaMemcpy(dst, src, bytes, cudaMemcpyHostToDevice) == cudaSuccess ? ARDIFF_OK : ARDIFF_ERR_CUDA;
}

int upload_bias(float* dst, const uint16_t* src, size_t n) {
    std::vector<float> tmp(n);
    for (size_t i = 0; i < n; ++i) tmp[i] = bf16_bits_to_float(src[i]);
    return upload(dst, tmp.data(), n * sizeof(float));
}

void free_all(ardiff_head* H) {
    for (void* p : H->allocs) cudaFree(p);
    H->allocs.clear();
}

#ifdef ARDIFF_TUNING
int env_int(const char* name, int dflt) {
    const char* v = getenv(name);
    if (!v || !*v) return dflt;
    return atoi(v);
}
#endif

}  // namespace

#define TRY(expr)                   \
    do {                            \
        int _rc = (expr);           \
        if (_rc != ARDIFF_OK) {     \
            free_all(H);            \
            delete H;               \
            return _rc;             \
        }                           \
    } while (0)

namespace {
// The persisting part of L2 (a limit of the CUDA context, per device): raised while heads exist on the device
// to what one token group's h needs, put back when the last of them is destroyed. A device or context that
// refuses (no such part, MIG) leaves the kernel's evict_last hints without effect and nothing else changes.
std::mutex g_l2_mu;
struct L2SetAside { int users = 0; size_t before = 0, set = 0; };
L2SetAside g_l2[64];

void l2_set_aside_acquire(int dev, const cudaDeviceProp& prop, size_t want) {
    if (dev < 0 || dev >= 64 || prop.persistingL2CacheMaxSize <= 0) return;
    if (want > (size_t)prop.persistingL2CacheMaxSize) want = (size_t)prop.persistingL2CacheMaxSize;
    std::lock_guard<std::mutex> lk(g_l2_mu);
    L2SetAside& a = g_l2[dev];
    size_t now = 0;
    if (cudaDeviceGetLimit(&now, cudaLimitPersistingL2CacheSize) != cudaSuccess) { cudaGetLastError(); return; }
    if (a.users == 0) { a.before = now; a.set = 0; }
    ++a.users;
    if (now < want) {
        if (cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, want) != cudaSuccess) { cudaGetLastError(); return; }
        cudaDeviceGetLimit(&a.set, cudaLimitPersistingL2CacheSize);
    }
}
void l2_set_aside_release(int dev) {
    if (dev < 0 || dev >= 64) return;
    std::lock_guard<std::mutex> lk(g_l2_mu);
    L2SetAside& a = g_l2[dev];
    if (a.users == 0 || --a.users > 0 || a.set == 0) return;
    size_t now = 0;
    // only if nobody else has changed it since
    if (cudaDeviceGetLimit(&now, cudaLimitPersistingL2CacheSize) == cudaSuccess && now == a.set)
        cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, a.before);
    cudaGetLastError();
    a.set = 0;
}
}  // namespace

extern "C" int ardiff_head_create(const ardiff_head_desc* desc, const ardiff_head_host_weights* w,
                                  ardiff_head** head_out) {
    if (!desc || !w || !head_out) return ARDIFF_ERR_NULL;
    *head_out = nullptr;
    const ardiff_head_desc d = *desc;
    if (d.C < 16 || d.C > 64 || d.Dc < 64 || d.W < 256 || d.W > 4096 || d.L < 1 || d.L > 64 || d.F < 2 ||
        d.F > 1024 || d.K_max < 0 || d.K_max > KMAX || d.max_tokens < 0 || d.max_tokens >= ((int64_t)1 << 31) - 256)
        return ARDIFF_ERR_SHAPE;
    if (d.C % 16 || d.Dc % 64 || d.W % 256 || d.F % 2) return ARDIFF_ERR_UNSUPPORTED;
    const void* ptrs[] = {w->Wc, w->bc, w->Wt1, w->bt1, w->Wt2, w->bt2, w->Win, w->bin, w->Wmod, w->bmod,
                          w->W1, w->b1, w->W2, w->b2, w->Wfm, w->bfm, w->Wout, w->bout};
    for (const void* p : ptrs)
        if (!p) return ARDIFF_ERR_NULL;

    int dev = 0;
    cudaDeviceProp prop;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess)
        return ARDIFF_ERR_CUDA;
    if (prop.major != 10) return ARDIFF_ERR_CUDA;
    if (!get_encode_fn()) return ARDIFF_ERR_CUDA;

    ardiff_head* H = new ardiff_head();
    H->d = d;
    H->device = dev;
    H->n_sm = prop.multiProcessorCount;
    const int W = d.W, C = d.C, Dc = d.Dc, L = d.L;
    const int NT = W / BN;
    H->NT = NT;
    H->T_pro = 1 + 2 * NT;     // gather, conditioning items, the gate of step 0 / block 0
    H->T_step = NT * (3 + 5 * L) + 1;
    H->C_pro = 1 + NT;
    H->C_step = NT * (3 + 4 * L) + 1;
    H->max_tiles = (d.max_tokens + BM - 1) / BM;
    if (H->max_tiles < 1) H->max_tiles = 1;

    // grid: one CTA per SM in clusters of two, all co-resident. The cooperative attribute makes the
    // launch fail instead of start when the grid cannot be co-resident (ardiff_head_set_cooperative
    // drops it for profilers that cannot replay such launches).
    H->coop = 1;
    H->stall_tile = -1;
    H->grid = H->n_sm;
#ifdef ARDIFF_TUNING
    H->grid = env_int("ARDIFF_HEAD_GRID", H->n_sm);
    if (H->grid < 2 || H->grid > H->n_sm) H->grid = H->n_sm;
#endif
    H->grid &= ~1;
    {
        bool ok = cudaFuncSetAttribute(head_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) ==
                  cudaSuccess;
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof(cfg));
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.gridDim = dim3(H->grid); cfg.blockDim = dim3(NUM_THREADS);
        cfg.dynamicSmemBytes = SMEM_BYTES; cfg.attrs = at; cfg.numAttrs = 1;
        int max_clusters = 0;
        ok = ok && cudaOccupancyMaxActiveClusters(&max_clusters, head_kernel, &cfg) == cudaSuccess && max_clusters >= 1;
        if (!ok) {
            (void)cudaGetLastError();
            delete H;
            return ARDIFF_ERR_CUDA;
        }
        if (H->grid > 2 * max_clusters) H->grid = 2 * max_clusters;
    }
    const int units = H->grid / 2;

    // largest group, in units (pairs of token tiles): a phase of NT column tiles per token tile should
    // span about 2.5 grids of items so that a dependent phase finds its producers long finished
    int tgu = (5 * units / 2 + NT - 1) / NT;
#ifdef ARDIFF_TUNING
    {
        const int tg_env = env_int("ARDIFF_HEAD_TGU", 0);
        if (tg_env > 0) tgu = tg_env;
    }
#endif
    // A unit gets r = ceil(tgu * NT / units) in-projection items in a row, each a single K slice: the producer can
    // then be r + 1 items ahead of the MMA issuer, which with its two accumulators is up to 2 ahead of the
    // epilogue; the dependency barriers are a ring of DEP_BARS phases, so r + 3 must stay below DEP_BARS
    // (r = 3 with the group size chosen above).
    while (tgu > 1 && ((int64_t)tgu * NT + units - 1) / units > DEP_BARS - 4) --tgu;
    if (tgu < 1) tgu = 1;
    if ((int64_t)tgu * 2 > H->max_tiles + 1) tgu = (int)((H->max_tiles + 1) / 2);
    H->TGu = tgu;
    H->slots = 4 * tgu;   // two groups of token tiles
    const size_t R = (size_t)H->slots * BM;

    // ---- pack the weights: one K-major matrix [rows][W] for every W-input layer ----
    const size_t blk_rows = (size_t)5 * W;
    const size_t fm_row0 = blk_rows * L, out_row0 = fm_row0 + 2 * (size_t)W;
    const size_t cat_rows = out_row0 + C;
    {
        std::vector<uint16_t> cat(cat_rows * W);
        std::vector<float> bias(cat_rows);
        auto put = [&](size_t dst_row, const uint16_t* Wsrc, const uint16_t* bsrc, size_t src_row, size_t nrows) {
            memcpy(&cat[dst_row * W], Wsrc + src_row * W, nrows * W * 2);
            for (size_t i = 0; i < nrows; ++i) bias[dst_row + i] = bf16_bits_to_float(bsrc[src_row + i]);
        };
        auto put_shift_scale = [&](size_t dst_row, const uint16_t* Wsrc, const uint16_t* bsrc) {
            for (int t = 0; t < W / 128; ++t) {
                put(dst_row + (size_t)t * 256, Wsrc, bsrc, (size_t)t * 128, 128);            // shift rows
                put(dst_row + (size_t)t * 256 + 128, Wsrc, bsrc, (size_t)W + t * 128, 128);  // scale rows
            }
        };
        for (int b = 0; b < L; ++b) {
            const uint16_t* Wm = w->Wmod + (size_t)b * 3 * W * W;
            const uint16_t* bm = w->bmod + (size_t)b * 3 * W;
            put_shift_scale(b * blk_rows, Wm, bm);
            put(b * blk_rows + 2 * (size_t)W, Wm, bm, 2 * (size_t)W, W);  // gate rows
            put(b * blk_rows + 3 * (size_t)W, w->W1 + (size_t)b * W * W, w->b1 + (size_t)b * W, 0, W);
            put(b * blk_rows + 4 * (size_t)W, w->W2 + (size_t)b * W * W, w->b2 + (size_t)b * W, 0, W);
        }
        put_shift_scale(fm_row0, w->Wfm, w->bfm);
        put(out_row0, w->Wout, w->bout, 0, C);
        TRY(dev_alloc(H, &H->Wcat, cat_rows * W, false));
        TRY(dev_alloc(H, &H->bias_cat, cat_rows, false));
        TRY(upload(H->Wcat, cat.data(), cat.size() * 2));
        TRY(upload(H->bias_cat, bias.data(), bias.size() * 4));
    }
    {
        std::vector<uint16_t> win((size_t)W * XB_COLS, 0);
        for (int o = 0; o < W; ++o) memcpy(&win[(size_t)o * XB_COLS], w->Win + (size_t)o * C, (size_t)C * 2);
        TRY(dev_alloc(H, &H->Win, win.size(), false));
        TRY(upload(H->Win, win.data(), win.size() * 2));
    }
    TRY(dev_alloc(H, &H->Wc, (size_t)W * Dc, false));
    TRY(upload(H->Wc, w->Wc, (size_t)W * Dc * 2));
    TRY(dev_alloc(H, &H->Wt1, (size_t)W * d.F, false));
    TRY(upload(H->Wt1, w->Wt1, (size_t)W * d.F * 2));
    TRY(dev_alloc(H, &H->Wt2, (size_t)W * W, false));
    TRY(upload(H->Wt2, w->Wt2, (size_t)W * W * 2));
    TRY(dev_alloc(H, &H->bc, W, false));
    TRY(upload_bias(H->bc, w->bc, W));
    TRY(dev_alloc(H, &H->bin, W, false));
    TRY(upload_bias(H->bin, w->bin, W));
    TRY(dev_alloc(H, &H->bt1, W, false));
    TRY(upload_bias(H->bt1, w->bt1, W));
    TRY(dev_alloc(H, &H->bt2, W, false));
    TRY(upload_bias(H->bt2, w->bt2, W));
    const int kmax = d.K_max > 0 ? d.K_max : 1;
    TRY(dev_alloc(H, &H->temb, (size_t)kmax * W, true));
    TRY(dev_alloc(H, &H->temb_hidden, (size_t)kmax * W, true));

    // ---- scratch ----
    TRY(dev_alloc(H, &H->z, R * Dc, true));
    TRY(dev_alloc(H, &H->xb, R * XB_COLS, true));  // columns >= C stay zero for ever
    TRY(dev_alloc(H, &H->s, (size_t)kmax * R * W, true));   // s_k for every step, [k][row][W]
    TRY(dev_alloc(H, &H->u, R * W, true));
    TRY(dev_alloc(H, &H->a, R * W, true));
    TRY(dev_alloc(H, &H->g0, R * W, true));
    TRY(dev_alloc(H, &H->g1, R * W, true));
    TRY(dev_alloc(H, &H->x, R * C, true));
    TRY(dev_alloc(H, &H->h, R * W, true));
    TRY(dev_alloc(H, &H->stats, R * 2 * NT, true));
    TRY(dev_alloc(H, &H->counters, ((size_t)H->max_tiles + 2) * CTRS, true));
    TRY(dev_alloc(H, &H->status, 2, true));
    TRY(dev_alloc(H, &H->clock_probe, 2, true));
#ifdef ARDIFF_HEAD_PROFILE
    TRY(dev_alloc(H, &H->trace, (size_t)TRACE_ITEMS * 12 + (size_t)TRACE_ITEMS * 16, true));
#endif

    // ---- the program of one step: phases in list order ----
    {
        std::vector<Phase> ph;
        int cum = 0;
        auto add = [&](int type, int block, int tile0, int ntiles, size_t b_row0, int offA, int kplus) {
            if (ntiles <= 0) return;
            ph.push_back(Phase{type, block, tile0, ntiles, cum, (int)b_row0, offA, kplus});
            cum += ntiles;
        };
        // A gate only needs s (known from the start of the call) and its buffer, last read by the block two
        // gates earlier: chain items of the blocks before `host` must be complete.
        auto gate = [&](int b, int kplus, int host, int tile0, int ntiles) {
            add(OP_GATE, b, tile0, ntiles, b * blk_rows + 2 * (size_t)W, NT + 4 * NT * host, kplus);
        };
        const int na = NT / 2;
        add(OP_IN, -1, 0, NT, 0, 0, 0);
        for (int b = 0; b < L; ++b) {
            const int base = NT + 4 * NT * b;
            add(OP_SS, b, 0, 2 * NT, b * blk_rows, base, 0);
            add(OP_G1, b, 0, NT, b * blk_rows + 3 * (size_t)W, base + 2 * NT, 0);
            // block b hosts the gate of the next block: half between its two dependent GEMMs, half after
            if (b + 1 < L) gate(b + 1, 0, b, 0, na);
            add(OP_G2, b, 0, NT, b * blk_rows + 4 * (size_t)W, base + 3 * NT, 0);
            if (b + 1 < L) gate(b + 1, 0, b, na, NT - na);
        }
        // the last block hosts the first gate of the NEXT step, spread over the step boundary where the chain
        // (final modulation -> out-projection -> in-projection) has little else to overlap with
        add(OP_FSS, -1, 0, 2 * NT, fm_row0, NT + 4 * NT * L, 0);
        gate(0, 1, L - 1, 0, na);
        add(OP_OUT, -1, 0, 1, out_row0, NT + 4 * NT * L + 2 * NT, 0);
        gate(0, 1, L - 1, na, NT - na);
        if (cum != H->T_step) {
            free_all(H);
            delete H;
            return ARDIFF_ERR_UNSUPPORTED;
        }
        std::vector<uint16_t> c2p(cum);
        for (size_t i = 0; i < ph.size(); ++i)
            for (int t = 0; t < ph[i].ntiles; ++t) c2p[ph[i].cum + t] = (uint16_t)i;
        H->n_phases = (int)ph.size();
        TRY(dev_alloc(H, &H->phases, ph.size(), false));
        TRY(upload(H->phases, ph.data(), ph.size() * sizeof(Phase)));
        TRY(dev_alloc(H, &H->cum2phase, c2p.size(), false));
        TRY(upload(H->cum2phase, c2p.data(), c2p.size() * sizeof(uint16_t)));
    }

    // ---- tensor maps ----
    {
        CUtensorMap maps[MAP_COUNT];
        bool ok = true;
        ok &= make_map(&maps[MAP_Z], H->z, R, Dc, BM);
        ok &= make_map(&maps[MAP_XB], H->xb, R, XB_COLS, BM);
        ok &= make_map(&maps[MAP_S], H->s, (uint64_t)kmax * R, W, BM);
        ok &= make_map(&maps[MAP_U], H->u, R, W, BM);
        ok &= make_map(&maps[MAP_A], H->a, R, W, BM);
        // a CTA of a pair stages half of the weight tile's rows
        ok &= make_map(&maps[MAP_WC], H->Wc, W, Dc, B_ROWS);
        ok &= make_map(&maps[MAP_WIN], H->Win, W, XB_COLS, B_ROWS);
        ok &= make_map(&maps[MAP_WCAT], H->Wcat, cat_rows, W, B_ROWS);
        ok &= make_map(&maps[MAP_WOUT], H->Wcat, cat_rows, W, (uint32_t)C / 2);
        ok &= make_slab_map(&maps[EMAP_S], H->s, (uint64_t)kmax * R, W);
        ok &= make_slab_map(&maps[EMAP_U], H->u, R, W);
        ok &= make_slab_map(&maps[EMAP_A], H->a, R, W);
        if (!ok) {
            free_all(H);
            delete H;
            return ARDIFF_ERR_CUDA;
        }
        TRY(dev_alloc(H, &H->maps, MAP_COUNT, false));
        TRY(upload(H->maps, maps, sizeof(maps)));
    }
    if (cudaDeviceSynchronize() != cudaSuccess) {
        free_all(H);
        delete H;
        return ARDIFF_ERR_CUDA;
    }
    // one token group's residual stream (half of the scratch rows, fp32)
    l2_set_aside_acquire(dev, prop, (size_t)(H->slots / 2) * BM * (size_t)W * sizeof(float));
    *head_out = H;
    return ARDIFF_OK;
}

extern "C" int ardiff_head_destroy(ardiff_head* H) {
    if (!H) return ARDIFF_OK;
    cudaSetDevice(H->device);
    cudaDeviceSynchronize();
    l2_set_aside_release(H->device);
    if (H->ev0) cudaEventDestroy(H->ev0);
    if (H->ev1) cudaEventDestroy(H->ev1);
    free_all(H);
    delete H;
    return ARDIFF_OK;
}

namespace {
// t_in [K]: the times fed to the head; coef [3K]: (ax, av, an) of every step
int head_sample_impl(const ardiff_head* H, const void* cond, const float* noise, const float* t_sched, int32_t K,
                     const float* coef, const float* step_noise, int64_t n_rows, const int32_t* idx,
                     const int32_t* count, float* out, void* stream) {
    if (!H || !idx || !count) return ARDIFF_ERR_NULL;
    if (K < 0 || K > H->d.K_max) return ARDIFF_ERR_SHAPE;
    if (H->d.max_tokens > 0 && (!cond || !noise || !out || !t_sched || !coef)) return ARDIFF_ERR_NULL;
    if (step_noise && (n_rows < 1 || (reinterpret_cast<uintptr_t>(step_noise) & 15u))) return ARDIFF_ERR_ALIGN;
    if (reinterpret_cast<uintptr_t>(cond) & 15u) return ARDIFF_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(noise) & 15u) || (reinterpret_cast<uintptr_t>(out) & 15u))
        return ARDIFF_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != H->device) return ARDIFF_ERR_CUDA;
    const int W = H->d.W, C = H->d.C;
    int launches = 0;

    if (K == 0) {
        copy_noise_rows_kernel<<<H->n_sm * 4, 256, 0, st>>>(noise, idx, count, (int)H->d.max_tokens, C, out);
        ardiff::set_launch_count(1);
        return cudaGetLastError() == cudaSuccess ? ARDIFF_OK : ARDIFF_ERR_CUDA;
    }

    TimeArgs ta;
    for (int k = 0; k < K; ++k) ta.t[k] = t_sched[k];
    temb_hidden_kernel<<<dim3((W + 7) / 8, K), 256, H->d.F * sizeof(float), st>>>(H->Wt1, H->bt1, W, H->d.F, ta,
                                                                                  H->temb_hidden);
    temb_out_kernel<<<dim3((W + 7) / 8, K), 256, 0, st>>>(H->Wt2, H->bt2, W, H->temb_hidden, H->temb);
    launches += 2;
    if (cudaMemsetAsync(H->counters, 0, sizeof(int) * ((size_t)H->max_tiles + 2) * CTRS, st) != cudaSuccess)
        return ARDIFF_ERR_CUDA;
    if (cudaMemsetAsync(H->status + 1, 0, sizeof(int), st) != cudaSuccess) return ARDIFF_ERR_CUDA;

    HeadParams P;
    memset(&P, 0, sizeof(P));
    P.C = C; P.Dc = H->d.Dc; P.W = W; P.L = H->d.L; P.K = K; P.NT = H->NT; P.TGu = H->TGu; P.slots = H->slots;
    P.T_pro = H->T_pro; P.T_step = H->T_step; P.T_chain = H->T_pro + K * H->T_step;
    P.C_pro = H->C_pro; P.C_step = H->C_step; P.C_total = H->C_pro + K * H->C_step;
    P.R = H->slots * BM;
    P.max_tokens = (int)H->d.max_tokens;
    P.phases = H->phases; P.cum2phase = H->cum2phase; P.maps = H->maps;
    P.cond = reinterpret_cast<const bf16*>(cond); P.noise = noise; P.idx = idx; P.count = count; P.out = out;
    P.z = H->z; P.xb = H->xb; P.s = H->s; P.u = H->u; P.a = H->a; P.g0 = H->g0; P.g1 = H->g1;
    P.x = H->x; P.h = H->h; P.stats = H->stats;
    P.bias_cat = H->bias_cat; P.bc = H->bc; P.bin = H->bin; P.temb = H->temb;
    P.counters = H->counters; P.status = H->status; P.abort_flag = H->status + 1;
    P.trace = H->trace;
    for (int k = 0; k < K; ++k) {
        P.ax[k] = coef[3 * k]; P.av[k] = coef[3 * k + 1]; P.an[k] = coef[3 * k + 2];
    }
    P.step_noise = step_noise;
    P.step_stride = (long long)n_rows * C;
    P.clock_probe = H->clock_probe;
    P.wait_limit_ns = kWaitLimitNs;
    P.stall_tile = -1;
    if (H->stall_tile >= 0) {             // armed self-test: this call only
        P.stall_tile = H->stall_tile;
        P.wait_limit_ns = (unsigned long long)H->stall_limit_us * 1000ull;
        H->stall_tile = -1;
    }

    if (H->timing) cudaEventRecord(H->ev0, st);
    {
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof(cfg));
        cudaLaunchAttribute at[2];
        int na = 0;
        if (H->coop) {
            at[na].id = cudaLaunchAttributeCooperative;
            at[na].val.cooperative = 1;
            ++na;
        }
        at[na].id = cudaLaunchAttributeClusterDimension;
        at[na].val.clusterDim.x = 2; at[na].val.clusterDim.y = 1; at[na].val.clusterDim.z = 1;
        ++na;
        cfg.gridDim = dim3(H->grid); cfg.blockDim = dim3(NUM_THREADS);
        cfg.dynamicSmemBytes = SMEM_BYTES;
        cfg.stream = st; cfg.attrs = at; cfg.numAttrs = na;
        if (cudaLaunchKernelEx(&cfg, head_kernel, P) != cudaSuccess) {
            (void)cudaGetLastError();
            return ARDIFF_ERR_CUDA;
        }
    }
    if (H->timing) {
        cudaEventRecord(H->ev1, st);
        H->timed = 1;
    }
    launches += 1;
    ardiff::set_launch_count(launches);
    return ARDIFF_OK;
}
}  // namespace

extern "C" int ardiff_head_sample(const ardiff_head* H, const void* cond, const float* noise,
                                  const float* t_sched, int32_t K, const int32_t* idx, const int32_t* count,
                                  float* out, void* stream) {
    if (K < 0 || K > KMAX) return ARDIFF_ERR_SHAPE;
    if (K > 0 && !t_sched) return ARDIFF_ERR_NULL;
    float coef[3 * KMAX + 3];
    for (int k = 0; k < K; ++k) {      // Euler flow step: x <- x + (t_{k+1} - t_k) v
        coef[3 * k] = 1.0f;
        coef[3 * k + 1] = (float)((double)t_sched[k + 1] - (double)t_sched[k]);
        coef[3 * k + 2] = 0.0f;
    }
    return head_sample_impl(H, cond, noise, t_sched, K, coef, nullptr, 0, idx, count, out, stream);
}

extern "C" int ardiff_head_sample_coef(const ardiff_head* H, const void* cond, const float* noise,
                                       const float* t_in, int32_t K, const float* coef, const float* step_noise,
                                       int64_t n, const int32_t* idx, const int32_t* count, float* out,
                                       void* stream) {
    return head_sample_impl(H, cond, noise, t_in, K, coef, step_noise, n, idx, count, out, stream);
}

extern "C" int ardiff_head_set_timing(ardiff_head* H, int on) {
    if (!H) return ARDIFF_ERR_NULL;
    if (on && !H->ev0) {
        if (cudaEventCreate(&H->ev0) != cudaSuccess || cudaEventCreate(&H->ev1) != cudaSuccess) return ARDIFF_ERR_CUDA;
    }
    H->timing = on ? 1 : 0;
    H->timed = 0;
    return ARDIFF_OK;
}

extern "C" int ardiff_head_last_kernel_ms(ardiff_head* H, float* ms) {
    if (!H || !ms) return ARDIFF_ERR_NULL;
    if (!H->timed) return ARDIFF_ERR_SHAPE;
    if (cudaEventSynchronize(H->ev1) != cudaSuccess) return ARDIFF_ERR_CUDA;
    return cudaEventElapsedTime(ms, H->ev0, H->ev1) == cudaSuccess ? ARDIFF_OK : ARDIFF_ERR_CUDA;
}

extern "C" int ardiff_head_status(ardiff_head* H, void* stream) {
    if (!H) return ARDIFF_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaStreamSynchronize(st) != cudaSuccess) return ARDIFF_ERR_CUDA;
    int v[2] = {0, 0};
    if (cudaMemcpy(v, H->status, sizeof(v), cudaMemcpyDeviceToHost) != cudaSuccess) return ARDIFF_ERR_CUDA;
    if (v[0] != 0 && cudaMemset(H->status, 0, sizeof(int)) != cudaSuccess) return ARDIFF_ERR_CUDA;
    return v[0];
}

extern "C" int ardiff_head_last_kernel_clock(ardiff_head* H, void* stream, double* sm_mhz) {
    if (!H || !sm_mhz) return ARDIFF_ERR_NULL;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return ARDIFF_ERR_CUDA;
    long long v[2] = {0, 0};
    if (cudaMemcpy(v, H->clock_probe, sizeof(v), cudaMemcpyDeviceToHost) != cudaSuccess) return ARDIFF_ERR_CUDA;
    if (v[1] <= 0) return ARDIFF_ERR_SHAPE;
    *sm_mhz = 1e3 * (double)v[0] / (double)v[1];
    return ARDIFF_OK;
}

extern "C" int ardiff_head_set_cooperative(ardiff_head* H, int on) {
    if (!H) return ARDIFF_ERR_NULL;
    H->coop = on ? 1 : 0;
    return ARDIFF_OK;
}

extern "C" int ardiff_head_inject_stall(ardiff_head* H, int32_t token_tile, uint32_t wait_limit_us) {
    if (!H) return ARDIFF_ERR_NULL;
    if (token_tile < 0 || wait_limit_us < 100 || wait_limit_us > 4000000u) return ARDIFF_ERR_SHAPE;
    H->stall_tile = token_tile;
    H->stall_limit_us = wait_limit_us;
    return ARDIFF_OK;
}

namespace ardiff {
const ardiff_head_desc* head_desc(const ardiff_head* H) { return H ? &H->d : nullptr; }
}  // namespace ardiff

#ifdef ARDIFF_HEAD_PROFILE
// Only in profiling builds: the per-item time stamps of CTA 0, copied to the host.
extern "C" int ardiff_head_copy_trace(ardiff_head* H, long long* dst, size_t count) {
    if (!H || !dst || !H->trace) return ARDIFF_ERR_NULL;
    if (cudaDeviceSynchronize() != cudaSuccess) return ARDIFF_ERR_CUDA;
    if (count > (size_t)TRACE_ITEMS * 28) count = (size_t)TRACE_ITEMS * 28;
    return cudaMemcpy(dst, H->trace, count * sizeof(long long), cudaMemcpyDeviceToHost) == cudaSuccess ? ARDIFF_OK
                                                                                                   : ARDIFF_ERR_CUDA;
}
#endif
