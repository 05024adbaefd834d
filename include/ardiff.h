/*
 * ardiff.h -- C ABI of the entropy-gated few-step diffusion-head hot path (B200, sm_100a).
 *
 * Two calls make the path:
 *   ardiff_entropy_gate  per-token entropy of the softmax-normalised shallow-feature row,
 *                        threshold, stream-compacted ascending list of surviving token ids;
 *   ardiff_head_sample   K Euler flow steps of the AdaLN residual-MLP head, conditioned on
 *                        each surviving token's AR hidden state, from caller-supplied noise.
 *
 * Conventions for every call
 *   - "dev" pointers are CUDA device pointers on the current device, "host" pointers are
 *     ordinary host memory. The caller owns every buffer it passes.
 *   - bf16 data is passed as raw 16-bit patterns (uint16_t / void*).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream). All
 *     device work is enqueued on it; calls return without waiting unless stated otherwise.
 *   - return value: 0 on success, a negative ARDIFF_ERR_* otherwise. Nothing throws,
 *     aborts or traps the device. Invalid arguments are rejected before any launch.
 */
#ifndef ARDIFF_H
#define ARDIFF_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ARDIFF_OK 0
#define ARDIFF_ERR_NULL (-1)        /* a required pointer is NULL                           */
#define ARDIFF_ERR_SHAPE (-2)       /* a size is negative, zero where it may not be, or too big */
#define ARDIFF_ERR_ALIGN (-3)       /* a pointer or row pitch misses its alignment rule      */
#define ARDIFF_ERR_UNSUPPORTED (-4) /* a shape the kernels do not cover (see each call)      */
#define ARDIFF_ERR_CUDA (-5)        /* a CUDA runtime/driver call failed                     */
#define ARDIFF_ERR_TIMEOUT (-6)     /* a bounded device-side wait ran out (results invalid)  */
#define ARDIFF_ERR_NOMEM (-7)       /* an allocation inside a create call failed             */

const char* ardiff_strerror(int code);
/* major*10000 + minor*100 + patch */
int ardiff_version(void);

/* ---------------------------------------------------------------------------------------
 * Entropy gate + stream compaction.
 *
 * Operation (the paper's entropy indicator: "Entropy-Informed Speculative Decoding",
 * equation for L_entropy, and the supplementary "Entropy Calculation Logic"; the test is
 * Algorithm 1's "if H^s < tau_ent"): for every token i, Omega = softmax(feat[i, :]) over
 * the d channels, H_i = -sum_c Omega_c ln Omega_c (natural log, zero-probability terms
 * contribute 0), keep_i = (H_i >= tau). A row that holds NaN, +inf or only -inf gives
 * H_i = NaN and is dropped.
 *
 *   feat   dev  bf16 [n][d] row-major (pre-softmax values), 16-byte aligned when d % 8 == 0
 *   n      tokens, 0 <= n < 2^31;  d channels per token, 1 <= d <= 65536
 *   tau    threshold (compared in fp32)
 *   mask   dev  uint8 [n]  out: 1 = keep, 0 = dropped
 *   idx    dev  int32 [n]  out: the first *count entries are the kept token ids, ascending
 *   count  dev  int32 [1]  out: number of kept tokens (stays on the device)
 *   entropy (the _ex form) dev float [n] out, or NULL: H_i as computed
 *
 * Rows are read once from HBM when d % 8 == 0 (d <= 8192: registers hold the row; longer rows:
 * a running maximum per lane with rescaled partial sums); other d take a slower two-pass kernel
 * with scalar loads. n == 0 is valid (writes *count = 0).
 *
 * Scratch and concurrency. The two kernels of a call hand per-block counts to each other
 * through a small per-device scratch (512 KB) that the library allocates on the first call on
 * each device: make that first call outside any stream capture. Every stream gets a slice of
 * its own, so calls on different streams may overlap on the GPU and calls on one stream are
 * ordered anyway. The table holds 31 streams per device; calls on any further stream share one
 * slice and must not overlap each other on the GPU. A call captured into a graph keeps the slice
 * of the stream it was captured on, whatever stream the graph is later launched on.
 * ardiff_entropy_gate_ex and ardiff_entropy_gate_blocks use the same scratch under the same rule.
 * ------------------------------------------------------------------------------------- */
int ardiff_entropy_gate(const void* feat, int64_t n, int32_t d, float tau, uint8_t* mask,
                        int32_t* idx, int32_t* count, void* stream);

int ardiff_entropy_gate_ex(const void* feat, int64_t n, int32_t d, float tau, uint8_t* mask,
                           int32_t* idx, int32_t* count, float* entropy, void* stream);

/* The gate together with the statistics that the paper's threshold equation needs ("Entropy-Based
 * Early Stopping in Inference Phase": tau_ent = 0.3 E[H] - 0.1 std(H)), in the same pass over the
 * features: the row kernel leaves per-block partial sums (fp64) beside its counts and the compaction
 * kernel merges them in a fixed order. Run it on a calibration batch with any tau (e.g. -1: keep all)
 * and use out3[2] as the threshold of the following calls.
 *   out3  dev double [3]  out: { mean(H), std(H) with divisor n, 0.3 mean - 0.1 std } over the n rows
 *         (a row with NaN entropy makes all three NaN). Reproducible run to run for a given n and d.
 *   entropy  as in the _ex form, may be NULL.  n >= 1.  Everything else as ardiff_entropy_gate. */
int ardiff_entropy_gate_stats(const void* feat, int64_t n, int32_t d, float tau, uint8_t* mask,
                              int32_t* idx, int32_t* count, float* entropy, double* out3, void* stream);

/* ---------------------------------------------------------------------------------------
 * Block-prefix gate: the early stop as the paper's Algorithm 1, Step 1 writes it ("if H^s <
 * tau_ent: draft_tokens <- draft_tokens[1 : i-1]; break"). Tokens come in draft blocks of
 * `gamma` consecutive tokens (the last block may be shorter). Token i owns the
 * rows_per_token consecutive rows i*rows_per_token .. of feat, and its indicator is the mean
 * of their row entropies (H^s = -L_entropy: the entropy-loss equation averages over the R
 * rows, the supplementary form over rows and heads). Scanning a block in order, the first
 * token with indicator < tau (or NaN) drops itself and every later token of the block.
 *
 *   feat           dev bf16 [n * rows_per_token][d], alignment as for ardiff_entropy_gate
 *   row_entropy    dev float [n * rows_per_token]  out, or NULL. One pass over the features does all of it
 *                  (row entropies stay in shared memory) when d % 8 == 0, d <= 8192 and
 *                  gamma * rows_per_token <= 24576; other shapes go through row_entropy as scratch and
 *                  return ARDIFF_ERR_NULL without it
 *   token_entropy  dev float [n]  out, or NULL
 *   mask, idx, count   as for ardiff_entropy_gate (idx ascending)
 *   block_len      dev int32 [ceil(n / gamma)]  out, or NULL: tokens kept in each block
 * gamma == 1 and rows_per_token == 1 give exactly ardiff_entropy_gate's results.
 * n * rows_per_token < 2^31. Allocates and uses the same per-device, per-stream scratch as
 * ardiff_entropy_gate.
 * ------------------------------------------------------------------------------------- */
int ardiff_entropy_gate_blocks(const void* feat, int64_t n, int32_t rows_per_token, int32_t d,
                               int32_t gamma, float tau, float* row_entropy, float* token_entropy,
                               uint8_t* mask, int32_t* idx, int32_t* count, int32_t* block_len,
                               void* stream);

/* Threshold from entropy statistics (the tau equation of "Entropy-Based Early Stopping in Inference
 * Phase"): out3 = { mean(H), std(H), 0.3 * mean - 0.1 * std }, std with divisor n, all in fp64
 * with a fixed summation order (results are reproducible run to run).
 *   entropy dev float [n], n >= 1;  out3 dev double [3]. One CTA: meant for calibration, not the hot path. */
int ardiff_tau_calibrate(const float* entropy, int64_t n, double* out3, void* stream);

/* Accepted draft length per block (Algorithm 1, Step 4):
 * accepted[b] = min({ i-1 : r_i > ratio_i } U { len_b }), i counted from 1 inside block b, where len_b
 * is the length of the draft that reaches Step 4, i.e. what Step 1's early stop left of the block.
 *   r, ratio   dev float [n] (the uniform draws and the density ratios p_i/q_i, both supplied by
 *              the caller; positions are those of the untruncated blocks of gamma tokens)
 *   block_len  dev int32 [ceil(n / gamma)], or NULL: tokens of each block that survived Step 1, as
 *              ardiff_entropy_gate_blocks writes them (NULL: every block is whole)
 *   accepted   dev int32 [ceil(n / gamma)] */
int ardiff_accept_prefix(const float* r, const float* ratio, int64_t n, int32_t gamma,
                         const int32_t* block_len, int32_t* accepted, void* stream);

/* ---------------------------------------------------------------------------------------
 * Entropy gate for callers that cannot allocate device memory. (The paper has no counterpart:
 * this is a packaging variant of ardiff_entropy_gate, same operation, same results.)
 *
 * Who needs it: a process whose own pool owns all device memory and forbids a library to
 * call cudaMalloc behind its back; a caller between cudaStreamBeginCapture and EndCapture,
 * where allocating is an error; a latency-critical loop that must not meet the allocator's
 * lock or the device-wide synchronisation an allocation may imply. ardiff_entropy_gate
 * allocates its per-block count array on its first call on a device; this entry point never
 * calls cudaMalloc, cudaFree or any allocating routine. Its scratch is a fixed array of
 * ARDIFF_GATE_NOALLOC_MAX_BLOCKS int32 (4 KB) compiled into the library as a __device__
 * variable, so every GPU that loads the library holds it until the process exits.
 *
 * Arguments, layouts, alignment rules and error codes are those of ardiff_entropy_gate, with
 * one more limit: n <= ARDIFF_GATE_NOALLOC_MAX_TOKENS, else ARDIFF_ERR_SHAPE and nothing is
 * launched (the fixed number of blocks would otherwise each walk an ever longer token range).
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress,
 * with that device current), and the first call for each feature-width class (d / 256 rounded up
 * to 1, 2, 4, 8, 12, 16, 20, 24, 32, or the generic path) loads that kernel and queries its
 * occupancy: make those first calls before any stream capture starts.
 * All calls on one device share the one array. Every call overwrites the entries it uses
 * before it reads them, so nothing needs clearing between calls and back-to-back calls on one
 * stream are safe; two calls that can run on the GPU at the same time (different streams
 * with no event between them, or mixed host threads) race on it and give undefined idx/count.
 * ------------------------------------------------------------------------------------- */
#define ARDIFF_GATE_NOALLOC_MAX_BLOCKS 1024
#define ARDIFF_GATE_NOALLOC_MAX_TOKENS (1 << 24)
int ardiff_entropy_gate_noalloc(const void* feat, int64_t n, int32_t d, float tau, uint8_t* mask,
                                int32_t* idx, int32_t* count, void* stream);

/* ---------------------------------------------------------------------------------------
 * Diffusion / flow head.
 *
 * Operation (the head call "x = Diff_theta(x_t | t, z)" of the AR+Diffusion hybrid
 * paradigm, sampled in "extremely few steps" from noise fixed up front as in Algorithm 1's
 * "Initialize"): for every survivor j < *count, with i = idx[j], z = cond[i], x = noise[i]:
 *   c = Wc z + bc
 *   for k in 0..K-1:
 *     s = SiLU(c + temb(t_k)),   temb(t) = Wt2 SiLU(Wt1 e(t) + bt1) + bt2,
 *         e(t) = [cos(1000 t w_f) | sin(1000 t w_f)], w_f = 10000^(-f/(F/2)), f < F/2
 *     h = Win x + bin
 *     for b in 0..L-1:  (shift, scale, gate) = Wmod[b] s + bmod[b]
 *                       u = LN(h) * (1 + scale) + shift          LN: eps 1e-6, no affine
 *                       h = h + gate * (W2[b] SiLU(W1[b] u + b1[b]) + b2[b])
 *     (shift, scale) = Wfm s + bfm ;  v = Wout (LN(h) * (1 + scale) + shift) + bout
 *     x = x + (t_{k+1} - t_k) v
 *   out[i] = x
 * Matrix products take bf16 operands with fp32 accumulation on the tensor cores; the
 * residual stream h, the state x, LayerNorm statistics and SiLU are fp32.
 * ------------------------------------------------------------------------------------- */
typedef struct ardiff_head ardiff_head; /* opaque; owns device copies of the weights + scratch */

typedef struct {
    int32_t C;      /* token (latent) dim: multiple of 16, 16 <= C <= 64                   */
    int32_t Dc;     /* conditioning dim: multiple of 64                                    */
    int32_t W;      /* head width: multiple of 256, <= 4096                                */
    int32_t L;      /* residual blocks, 1 <= L <= 64                                       */
    int32_t F;      /* time-embedding size (even), <= 1024                                 */
    int32_t K_max;  /* largest K a later ardiff_head_sample may ask for, <= 64             */
    int64_t max_tokens; /* largest *count a later ardiff_head_sample may meet              */
} ardiff_head_desc;

/* HOST pointers, bf16 bit patterns, Linear layout [out][in] row-major, biases [out]. */
typedef struct {
    const uint16_t *Wc, *bc;     /* [W][Dc], [W]                                          */
    const uint16_t *Wt1, *bt1;   /* [W][F],  [W]                                          */
    const uint16_t *Wt2, *bt2;   /* [W][W],  [W]                                          */
    const uint16_t *Win, *bin;   /* [W][C],  [W]                                          */
    const uint16_t *Wmod, *bmod; /* [L][3W][W], [L][3W]   rows: shift | scale | gate      */
    const uint16_t *W1, *b1;     /* [L][W][W], [L][W]                                     */
    const uint16_t *W2, *b2;     /* [L][W][W], [L][W]                                     */
    const uint16_t *Wfm, *bfm;   /* [2W][W], [2W]         rows: shift | scale             */
    const uint16_t *Wout, *bout; /* [C][W],  [C]                                          */
} ardiff_head_host_weights;

/*
 * Packs the weights into the kernels' tile layout on the current device and allocates
 * the head's scratch (a fixed-size activation workspace for two groups of token tiles plus
 * max_tokens/128 progress counters). Synchronous; the only head call that allocates.
 * Side effect on the CUDA context: while at least one head exists on a device, the context's
 * cudaLimitPersistingL2CacheSize is at least the size of one token group's fp32 residual
 * stream (about 49 MB, capped at the device's maximum); the kernel keeps that array in the
 * persisting part of L2. The value found before the first head is put back when the last
 * head of the device is destroyed, unless the caller changed the limit meanwhile. A device
 * that refuses the limit runs the same kernel without that residency.
 * Errors: ERR_NULL, ERR_SHAPE / ERR_UNSUPPORTED for dims outside the ranges above,
 * ERR_NOMEM, ERR_CUDA (also when the device is not compute capability 10.x).
 */
int ardiff_head_create(const ardiff_head_desc* desc, const ardiff_head_host_weights* weights,
                       ardiff_head** head_out);

/* Frees everything create allocated. Waits for the device first. NULL is accepted. */
int ardiff_head_destroy(ardiff_head* head);

/*
 *   head     from ardiff_head_create (same device)
 *   cond     dev  bf16 [n][Dc] row-major, 16-byte aligned
 *   noise    dev  float [n][C]
 *   t_sched  HOST float [K+1]: t_0 .. t_K (read before the call returns)
 *   K        steps, 0 <= K <= K_max (K == 0 copies noise rows to out rows)
 *   idx      dev  int32: token ids of the survivors (as written by the gate; any order,
 *                 each a valid row of cond / noise / out, no duplicates)
 *   count    dev  int32 [1]: number of survivors; read on the device, never on the host;
 *                 values above max_tokens are clamped to max_tokens (and flagged in the
 *                 status word as ARDIFF_ERR_SHAPE)
 *   out      dev  float [n][C]: rows idx[j] are written, all other rows are left untouched
 * One persistent cooperative kernel walks a static schedule of GEMM tiles; tiles wait for
 * their producers on device-side counters with bounded spins. If a wait runs out the
 * kernel finishes early, the results are invalid and ardiff_head_status reports
 * ARDIFF_ERR_TIMEOUT. Calls on one head must not overlap on the device (they share its
 * scratch): enqueue them on one stream or order them with events.
 */
int ardiff_head_sample(const ardiff_head* head, const void* cond, const float* noise,
                       const float* t_sched, int32_t K, const int32_t* idx, const int32_t* count,
                       float* out, void* stream);

/*
 * The same head under another sampler. The paper's heads are also run as eps-prediction DDPM
 * heads ("x_t = sqrt(abar_t) x + sqrt(1 - abar_t) eps", AR+Diffusion Hybrid Paradigm) and, after
 * consistency distillation, as x_0-predicting students ("x_0 = Diff_theta(x_t | t, z)"); every such
 * sampler step is linear in the state, the head output v and fresh noise, so the caller passes
 * three coefficients per step:  x <- ax_k x + av_k v + an_k z_k.
 *   t_in        HOST float [K]: the time fed to the head at step k
 *   coef        HOST float [3K]: ax_0, av_0, an_0, ax_1, ...   (Euler flow: 1, t_{k+1} - t_k, 0;
 *               deterministic eps-prediction step from abar to abar': ax = sqrt(abar'/abar),
 *               av = sqrt(1 - abar') - ax sqrt(1 - abar), an = 0; x_0-prediction with re-noising:
 *               ax = 0, av = sqrt(abar'), an = sqrt(1 - abar'))
 *   step_noise  dev float [K][n][C], 16-byte aligned, or NULL (then an_k is ignored); row i of
 *               slice k is the fresh noise of token i at step k;  n = rows of noise / out
 * Everything else as ardiff_head_sample (which is this call with the Euler coefficients).
 */
int ardiff_head_sample_coef(const ardiff_head* head, const void* cond, const float* noise,
                            const float* t_in, int32_t K, const float* coef, const float* step_noise,
                            int64_t n, const int32_t* idx, const int32_t* count, float* out, void* stream);

/* Waits for `stream`, then returns the head's device status word: ARDIFF_OK, or
 * ARDIFF_ERR_TIMEOUT if any bounded wait of an earlier sample call ran out, or
 * ARDIFF_ERR_SHAPE if *count exceeded max_tokens. Clears it. (The status word belongs to the
 * head, not to a stream: this is the call that reports what the device saw.) */
int ardiff_head_status(ardiff_head* head, void* stream);

/* Profiling aids. With on != 0, every later ardiff_head_sample on this head records CUDA events
 * on its stream directly around the persistent head kernel. ardiff_head_last_kernel_ms waits
 * for that kernel and writes its device time in milliseconds (ERR_SHAPE if nothing was timed).
 * ardiff_head_last_kernel_clock waits for `stream` and writes the SM clock the last head kernel
 * really ran at, in MHz: SM cycles divided by wall time, both stamped by one CTA at the start and
 * the end of the launch (ERR_SHAPE before the first launch).
 * ardiff_head_set_cooperative(head, 0) launches the head kernel without the cooperative attribute,
 * for profilers that cannot replay cooperative launches; the kernel and its grid are unchanged, but
 * the launch no longer fails when the GPU cannot hold the whole grid at once (then waits run into
 * their bound and ARDIFF_ERR_TIMEOUT is reported). Default: on. */
int ardiff_head_set_timing(ardiff_head* head, int on);
int ardiff_head_last_kernel_ms(ardiff_head* head, float* ms);
int ardiff_head_last_kernel_clock(ardiff_head* head, void* stream, double* sm_mhz);
int ardiff_head_set_cooperative(ardiff_head* head, int on);

/* Self-test of the bounded device-side waits. Arms the NEXT ardiff_head_sample call on this head:
 * its dependency waits give up after wait_limit_us microseconds (100 .. 4 000 000) instead of the
 * default 4 s, and the conditioning tiles of token tile `token_tile` (survivors 128 token_tile ..)
 * wait for one predecessor more than exists, so that wait runs out. The kernel then raises its
 * abort flag, every CTA leaves its loops, waits for its own copies in flight, frees its tensor
 * memory and returns; ardiff_head_status reports ARDIFF_ERR_TIMEOUT and the call's results are
 * invalid. Nothing faults or traps, and the call after it runs normally. A token_tile beyond the
 * tiles of that call has no effect. */
int ardiff_head_inject_stall(ardiff_head* head, int32_t token_tile, uint32_t wait_limit_us);

/* ---------------------------------------------------------------------------------------
 * Host-buffer front end: one call takes a batch that lives in HOST memory through the whole
 * path (copy in, gate, head, copy out). The pipeline object owns device staging buffers for
 * up to max_n tokens of feature width d, conditioning width Dc and token dim C (Dc and C must
 * equal the head's and max_n may not exceed its max_tokens, else ARDIFF_ERR_SHAPE). Pinned host
 * buffers make the copies asynchronous; pageable ones work too.
 *
 *   feat   host bf16 [n][d],  cond host bf16 [n][Dc],  noise host float [n][C]
 *   out    host float [n][C]: rows of kept tokens hold the sample, dropped rows are 0
 *   mask   host uint8 [n],    count host int32 [1]
 * With n == 0 the five batch pointers may be NULL (count is still written).
 * The call waits for `stream` before it returns, so the host outputs are valid on return.
 * ------------------------------------------------------------------------------------- */
typedef struct ardiff_pipeline ardiff_pipeline;
int ardiff_pipeline_create(ardiff_head* head, int64_t max_n, int32_t d, int32_t Dc, int32_t C,
                           ardiff_pipeline** pipeline_out);
int ardiff_pipeline_destroy(ardiff_pipeline* pipeline);
int ardiff_pipeline_run_host(ardiff_pipeline* pipeline, const void* feat, const void* cond,
                             const float* noise, int64_t n, float tau, const float* t_sched, int32_t K,
                             float* out, uint8_t* mask, int32_t* count, void* stream);

/* Overlapped form of the same path, for a stream of batches. A pipeline created with
 * ardiff_pipeline_create_slots(..., n_slots >= 2, ...) owns n_slots sets of device staging
 * buffers and three streams (copy-in, compute, copy-out), so the host->device copy of one batch
 * and the device->host copy of another run under the kernels of a third. (The paper describes
 * no host interface; this is packaging around the path of Sec. 3.2-3.3.)
 *
 *   ardiff_pipeline_submit  enqueues copy-in, gate, head and copy-out of one batch on `slot`
 *                           (0 <= slot < n_slots) and returns without waiting. Arguments as for
 *                           ardiff_pipeline_run_host; t_sched is read before the call returns,
 *                           every other host buffer must stay valid (and, for the copies to be
 *                           asynchronous, pinned) until ardiff_pipeline_wait(slot) has returned.
 *                           The batch starts after the work `stream` holds at the time of the
 *                           call; nothing else is enqueued on `stream`. Re-using a slot is ordered
 *                           on the device after the slot's previous batch; the HOST buffers of that
 *                           previous batch are the caller's to keep apart (wait first, or use others).
 *   ardiff_pipeline_wait    blocks the host until the batch last submitted on `slot` has been
 *                           copied out, stores its number of kept tokens in that submission's
 *                           `count` (only this call writes it: the pipeline stages the value in
 *                           pinned memory of its own so that a pageable `count` cannot stall the
 *                           submitting thread) and returns what that submission returned. A slot never
 *                           submitted to returns ARDIFF_OK at once.
 *   ardiff_pipeline_join    makes `stream` wait (on the device) for every batch submitted so far;
 *                           the host does not block.
 *
 * Batches run through the head in submission order. Calls on one pipeline must come from one
 * host thread at a time. ardiff_pipeline_create gives a one-slot pipeline, on which these three
 * calls return ARDIFF_ERR_UNSUPPORTED; ardiff_pipeline_run_host works on any pipeline and uses
 * slot 0: it first waits for a batch still in flight there (delivering its count as
 * ardiff_pipeline_wait would) and orders its own work on the device after every batch submitted
 * on the other slots. Errors: ARDIFF_ERR_NULL,
 * ARDIFF_ERR_SHAPE (slot or n out of range), ARDIFF_ERR_CUDA, and whatever the gate or the head
 * return; after a failed submit the slot's events are still recorded, so wait never hangs. */
#define ARDIFF_PIPELINE_MAX_SLOTS 4
int ardiff_pipeline_create_slots(ardiff_head* head, int64_t max_n, int32_t d, int32_t Dc, int32_t C,
                                 int32_t n_slots, ardiff_pipeline** pipeline_out);
int ardiff_pipeline_submit(ardiff_pipeline* pipeline, int32_t slot, const void* feat, const void* cond,
                           const float* noise, int64_t n, float tau, const float* t_sched, int32_t K,
                           float* out, uint8_t* mask, int32_t* count, void* stream);
int ardiff_pipeline_wait(ardiff_pipeline* pipeline, int32_t slot);
int ardiff_pipeline_join(ardiff_pipeline* pipeline, void* stream);

/* Number of kernel launches the last ardiff_head_sample / ardiff_entropy_gate call on this
 * thread enqueued (for launch accounting by benchmarks). */
int ardiff_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* ARDIFF_H */
