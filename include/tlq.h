/*
 * tlq.h - C ABI of libtlq: the hot path of TLQ's layer-wise calibration on one B200 (sm_100a).
 *
 * For one linear layer Y = X W^T + b (X: N tokens x C1 input channels, W: C2 x C1), every candidate
 * r_k = k/K of the ratio grid gives a per-input-channel scale = x_stat^r_k (paper Sec. 3.1.2, first
 * equation; Sec. 3.2.1, first equation).  The scaled weights are fake-quantized (Sec. 2.2 quantizer),
 * the quantized layer f_q = Q_w(W*scale) Q_a(x/scale) + b is applied to the calibration tokens and
 * the squared output error against f_fp = W x + b (Sec. 3.2.1, objective) is reduced per token with
 * the token-importance weights (Sec. 3.1: gradient-derived importance; a 0/1 weight vector is the
 * paper's top-50% token selection, a constant vector its plain expectation).  The argmin is kept.
 *
 * Conventions
 *  - Every pointer is a DEVICE pointer unless its comment says "host".  The caller owns all buffers;
 *    the library allocates and frees no device memory.  bf16 tensors are raw uint16 bit patterns,
 *    row-major, innermost dimension contiguous.  X, W and the workspace must be 16-byte aligned
 *    (TMA base-address rule) and C1 must be a multiple of 8 (16-byte row pitch), of 16 in the
 *    symmetric mode (16-byte rows of int8 codes) and of the group size in the group mode.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls validate
 *    their arguments on the host, enqueue kernels on `stream` and return without synchronising.
 *  - Return value: TLQ_OK or a negative TLQ_ERR_* for errors found on the host.  Errors found on
 *    the device (a bounded wait that ran out, a grid whose losses are all non-finite) are written
 *    to the int32 status word at byte 0 of the workspace; tlq_read_status() synchronises the stream
 *    and returns it.
 *  - There is no CPU fallback: without a CUDA device every compute call returns TLQ_ERR_CUDA.
 *  - Every call acts on the device that is current when it is made; the few pieces of host-side state the library
 *    keeps (kernel attributes, SM counts, addresses of its built-in device arrays) are kept per device, so one process
 *    may drive several GPUs.  Calls are not synchronised against each other: host threads that share a device, or a
 *    workspace, must take turns.
 */
#ifndef TLQ_H_
#define TLQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TLQ_OK 0
#define TLQ_ERR_INVALID_ARG (-1) /* NULL pointer, bad enum, bad struct_size */
#define TLQ_ERR_SHAPE (-2)       /* N<1, C1%8, C1%group, K outside [1,64], ... */
#define TLQ_ERR_ALIGN (-3)       /* a pointer that must be 16-byte aligned is not */
#define TLQ_ERR_UNSUPPORTED (-4) /* bit width / mode combination not built */
#define TLQ_ERR_WORKSPACE (-5)   /* workspace_bytes smaller than tlq_*_workspace_bytes() */
#define TLQ_ERR_CUDA (-6)        /* a CUDA runtime / driver call failed (no device, launch error) */
#define TLQ_ERR_TIMEOUT (-7)     /* device: a bounded barrier wait expired; results are invalid */
#define TLQ_ERR_NONFINITE (-8)   /* device: every candidate's loss was non-finite */
#define TLQ_ERR_OVERRUN (-9)     /* device: a guard word between workspace regions changed (TLQ_FLAG_DEBUG_CANARIES) */

/* tlq_config.mode */
#define TLQ_W4A16_ASYM_GROUP 0 /* weights: w_bits (2..8) asymmetric, one step + integer zero-point per
                                  `group_size` consecutive input channels of an output row; activations
                                  stay bf16 (Q_a = identity) */
#define TLQ_W8A8_SYM 1         /* weights: w_bits (2..8) symmetric per output row; activations: a_bits (2..8)
                                  symmetric per token; step max|.|/(2^(bits-1)-1), integers in
                                  [-2^(bits-1), 2^(bits-1)-1] held in int8 containers (Sec. 2.2, first two
                                  equations).  w_bits = a_bits = 8 is W8A8; the paper's main settings are
                                  w_bits = 4 with a_bits = 8 or 6 (Experiments, quantization settings) */
#define TLQ_WA_SYM_CHANNEL TLQ_W8A8_SYM /* the same mode under the name of what it does */

/* tlq_config.stat_mode: x_stat over the calibration tokens */
#define TLQ_STAT_MEAN_ABS 0   /* mean_n |X_nc| (x_mean row of the paper's ablation table) */
#define TLQ_STAT_MAX_ABS 1    /* max_n |X_nc| (x_max row) */
#define TLQ_STAT_MASKED_MAX 2 /* max over the selected tokens I (Sec. 3.1.2, second equation) */

/* tlq_token_importance: norm_kind, g_dtype */
#define TLQ_NORM_MEAN_ABS 0 /* mean over channels of |g| (the text of Sec. 3.1.2) */
#define TLQ_NORM_L2 1       /* ||g||_2 (the equation of Sec. 3.1.2 read as a Euclidean norm) */
#define TLQ_DTYPE_BF16 0
#define TLQ_DTYPE_F32 1

/* tlq_config.flags */
#define TLQ_FLAG_SKIP_ZERO_WEIGHT_TOKENS 1u /* tlq_scale_search_layer: tokens whose importance weight is not > 0 add
                                               nothing to any loss, so the quantized layer is applied only to the
                                               others (packed on the device, order kept).  With the paper's Top-50%
                                               token set as a 0/1 weight vector (Sec. 3.1.2) this halves the tensor
                                               work.  x_stat still sees every token (or those of `mask`).  Needs
                                               w_imp; per_token_err must be NULL.  Losses equal the unflagged call's
                                               up to the order of the fp32 partial sums. */

#define TLQ_FLAG_GEMM_CTA_PAIRS 2u          /* tlq_scale_search_layer, group mode: run the fused GEMM on pairs of CTAs
                                               (one 256 x 256 MMA per two SMs, the weight tile split between them)
                                               instead of one CTA per tile.  Same results layout and tolerances.
                                               Off by default: equal speed in isolation, slower under the power cap
                                               of a long run on the parts measured. */

#define TLQ_FLAG_GEMM_NARROW_TILES 4u       /* tlq_scale_search_layer, group mode: one CTA per 128-token x 256-channel
                                               tile, as used for N <= 128, instead of the default 256-token tile that
                                               stages the weight tile once for two 128-token halves (measured 8 %
                                               faster inside a benchmark step). */

#define TLQ_FLAG_NO_REFINE 8u                /* tlq_scale_search_layer, group mode: skip the refine pass.  By default,
                                               when other candidates' losses come within 1e-4 (relative; wider
                                               below 1024 output channels: 3.2e-3 / sqrt(C2)) of the smallest, those candidates (if there are no more than four, and no
                                               more than K/2, of them: a flatter loss curve keeps its first result)
                                               are evaluated a second time with delta weights split into two bf16
                                               parts and short tensor-core accumulation chunks summed in registers
                                               and fp64, which brings their losses from about 6e-5 to about 1e-6 of
                                               the exact value; losses[] of those candidates, best_idx and s_best
                                               come from the second evaluation.  per_token_err keeps the first
                                               evaluation's values.  The pass costs a few idle launches when no
                                               candidate is that close, and about four screening-candidates' time per
                                               re-evaluated candidate when some are.  Not run by the two-stream call
                                               nor in the symmetric modes (whose integer accumulation is exact). */

#define TLQ_FLAG_DEBUG_CANARIES 16u          /* tlq_scale_search_layer (both forms), tlq_apply_layer: a debugging aid.
                                               Every region of the workspace is followed by 256 bytes of guard words,
                                               written when the call starts and compared when it ends; a guard that
                                               changed sets the status word to TLQ_ERR_OVERRUN (and the header's second
                                               int32 to 100 + the index of the guard), which shows a kernel writing
                                               past the end of its region.  The flag is part of the configuration, so
                                               the *_workspace_bytes() calls account for the guards.  Two tiny extra
                                               launches per call; results are unchanged. */

#define TLQ_MAX_GRID 64

typedef struct {
  uint32_t struct_size; /* sizeof(tlq_config); checked */
  int32_t mode;         /* TLQ_W4A16_ASYM_GROUP | TLQ_W8A8_SYM */
  int32_t w_bits;       /* 2..8 (codes are one per byte in both modes) */
  int32_t a_bits;       /* 16 for the group mode; 2..8 for the symmetric mode */
  int32_t group_size;   /* 32, 64, 128 or 256 for the group mode (must divide C1); ignored for W8A8 */
  int32_t n_grid;       /* K >= 1; candidate k uses r_k = k / K, so candidate 0 is scale = 1 */
  int32_t stat_mode;    /* TLQ_STAT_* */
  uint32_t flags;       /* TLQ_FLAG_* bits, 0 by default */
} tlq_config;

/* Stages of tlq_scale_search_layer, for tlq_stage_timing_drain(). */
#define TLQ_STAGE_STATS 0     /* x_stat and the K x C1 scale table */
#define TLQ_STAGE_FAKEQUANT 1 /* operands of all K candidates (delta weights, or int8 weights + activations) */
#define TLQ_STAGE_GEMM 2      /* fused tensor-core GEMM + per-token weighted error epilogue */
#define TLQ_STAGE_REDUCE 3    /* losses, argmin, s_best, optional per-token table */
#define TLQ_N_STAGES 4

const char* tlq_status_string(int status);

/* Version of this ABI (major*1000 + minor). */
int tlq_version(void);

/*
 * Token importance (Sec. 3.1.2, third equation and the Top-50% selection):
 *   imp[n] = sum_{b<B} norm(G[b,n,:]),  norm = mean_c |g| (TLQ_NORM_MEAN_ABS) or sqrt(sum_c g^2).
 * If mask_out != NULL and top_frac > 0: mask_out[n] = 1 for the max(1, floor(top_frac*N)) positions
 * with the largest imp (equal values: lower index first), else 0.
 *   G        [B,N,C] bf16 bits or fp32 (g_dtype), C a multiple of 8
 *   imp_out  [N] fp32            mask_out [N] uint8 or NULL
 * Uses no scratch memory.
 */
int tlq_token_importance(const void* G, int g_dtype, int64_t B, int64_t N, int64_t C, int norm_kind,
                         float top_frac, float* imp_out, uint8_t* mask_out, void* stream);

/*
 * Scale candidates (Sec. 3.1.2 first two equations; Table 2 variants):
 *   x_stat[c] per cfg->stat_mode (mask [N] uint8 is read only for TLQ_STAT_MASKED_MAX),
 *   m = max(x_stat, 2^-20),  s[k,c] = bf16(m^(k/K)).
 *   X [N,C1] bf16; x_stat_out [C1] fp64 or NULL; s_out [K,C1] bf16
 *   workspace: at least tlq_scale_candidates_workspace_bytes(N, C1) bytes (partial sums).
 */
size_t tlq_scale_candidates_workspace_bytes(int64_t N, int64_t C1);
int tlq_scale_candidates(const void* X, int64_t N, int64_t C1, const uint8_t* mask, const tlq_config* cfg,
                         void* workspace, size_t workspace_bytes, double* x_stat_out, void* s_out,
                         void* stream);

/*
 * tlq_scale_candidates for callers that may not allocate device memory.  (The paper has no counterpart;
 * this is a packaging variant of the call above and computes the same x_stat and scale table.)
 *
 * Some hosts of this library cannot hand it a workspace: code that runs where cudaMalloc is off limits
 * (inside a framework's allocator callback, in a process whose memory pool is fixed at start-up, in a
 * plug-in that is only given its input and output tensors).  For them the partial sums live in a 4 MiB
 * device array that is part of the library image, so the call needs nothing but X and the outputs.
 *  - Limit: C1 <= 32768 (TLQ_ERR_SHAPE beyond that); N is unlimited, large N simply uses fewer, taller
 *    row chunks than the workspace version.  Every GPU that loads the library holds the 4 MiB until exit.
 *  - The first call on each device looks up the array's device address (with that device current) and
 *    keeps it; make that first call outside of any stream capture.  No call allocates or frees memory.
 *  - All calls share the one array.  Each call overwrites every partial it later reads, so nothing is
 *    carried over from the previous call, but two calls whose kernels overlap on the GPU (different
 *    streams, or different threads on one device) race on it: serialise them.
 */
int tlq_scale_candidates_noalloc(const void* X, int64_t N, int64_t C1, const uint8_t* mask, const tlq_config* cfg,
                                 double* x_stat_out, void* s_out, void* stream);

/*
 * Fake-quantize the scaled weights for ONE scale vector: Q_w(W * scale) (Sec. 3.2.1, f_q; quantizer Sec. 2.2).
 *   W [C2,C1] bf16;  s [C1] bf16 or NULL (= all ones, plain round-to-nearest)
 * Group mode: codes [C2,C1] uint8 in [0,2^w_bits-1]; steps [C2,C1/G] fp32; zeros [C2,C1/G] int32;
 *             dW_out [C2,C1] bf16 or NULL: W - dequant/scale (the tensor-core operand of the search).
 * Symmetric mode: codes [C2,C1] int8 (w_bits wide); steps [C2] fp32; zeros ignored (may be NULL); dW_out must be NULL.
 * Any of codes/steps/zeros may be NULL when not wanted.
 */
int tlq_quantize_weights(const void* W, const void* s, int64_t C2, int64_t C1, const tlq_config* cfg,
                         uint8_t* codes, float* steps, int32_t* zeros, void* dW_out, void* stream);

/*
 * Storage format for 4-bit weights (Sec. 2.2, integer range for n = 4: sixteen levels, half a byte per weight):
 * packs the one-code-per-byte output of tlq_quantize_weights / tlq_apply_layer two per byte,
 *   packed[r, j] = (codes[r, 2j] & 15) | (codes[r, 2j+1] & 15) << 4,
 * for the group mode's unsigned codes (0..15) as well as the symmetric mode's integers (-8..7, which stay
 * two's-complement nibbles).  codes [rows, cols] one per byte, cols a multiple of 32; packed [rows, cols/2].
 * Only the low four bits of every code are kept: the caller quantized with w_bits <= 4.
 */
int tlq_pack_codes4(const uint8_t* codes, int64_t rows, int64_t cols, uint8_t* packed, void* stream);

/*
 * Quantize the smoothed activations for ONE scale vector: Q_a(x / scale), per-token symmetric, a_bits wide
 * (Sec. 2.2 first two equations; Sec. 3.2.1 f_q).  Symmetric mode only.
 *   X [N,C1] bf16; s [C1] bf16 or NULL (= ones); codes [N,C1] int8; steps [N] fp32.
 */
int tlq_quantize_activations(const void* X, const void* s, int64_t N, int64_t C1, const tlq_config* cfg,
                             int8_t* codes, float* steps, void* stream);

/*
 * The layer-wise search (Sec. 3.2.1): for k in [0,K): loss[k] = sum_n w_n e_{k,n} / (C2 * sum_n w_n),
 * e_{k,n} = || f_fp(x_n) - f_q(x_n; scale_k) ||_2^2; best_idx = argmin (lowest index on ties).
 *   X [N,C1] bf16, W [C2,C1] bf16, w_imp [N] fp32 >= 0 or NULL (uniform),
 *   mask [N] uint8 or NULL (token selection for TLQ_STAT_MASKED_MAX only),
 *   best_idx [1] int32, losses [K] fp64, s_best [C1] bf16 (the winning scale),
 *   per_token_err [K,N] fp32 or NULL (e_{k,n}).
 * The workspace holds the operands of all K candidates; its status word is reset by this call.
 * Group mode: the first call on a device whose K x C2 x C1 delta-weight region is at least 35 MB also enqueues, once,
 * a measurement of about a millisecond (which half of the L2 each SM sits next to; it uses that region before
 * anything else is written there) and looks up a device symbol's address; make that first call outside of any
 * stream capture.  Results do not depend on it, only the order in which tiles are visited.
 */
size_t tlq_scale_search_workspace_bytes(int64_t N, int64_t C1, int64_t C2, const tlq_config* cfg);
int tlq_scale_search_layer(const void* X, int64_t N, int64_t C1, const void* W, int64_t C2,
                           const float* w_imp, const uint8_t* mask, const tlq_config* cfg, void* workspace,
                           size_t workspace_bytes, int32_t* best_idx, double* losses, void* s_best,
                           float* per_token_err, void* stream);

/*
 * The same search under the paper's first propagation strategy (Sec. 3.2.1, PassAct1): two activation streams.
 * X_fp [N,C1] bf16 is the layer's input as the full-precision layers before it produce it, X_q [N,C1] bf16 its input
 * as the already quantized layers produce it; e_{k,n} = || f_fp(x_fp,n) - f_q(x_q,n; scale_k) ||_2^2.  The scale
 * statistic, the smoothing and the activation quantizer all act on X_q.  Everything else as in
 * tlq_scale_search_layer (same workspace size); the flags TLQ_FLAG_SKIP_ZERO_WEIGHT_TOKENS and
 * TLQ_FLAG_GEMM_CTA_PAIRS are not accepted here.
 */
int tlq_scale_search_layer_two_stream(const void* X_q, const void* X_fp, int64_t N, int64_t C1, const void* W,
                                      int64_t C2, const float* w_imp, const uint8_t* mask, const tlq_config* cfg,
                                      void* workspace, size_t workspace_bytes, int32_t* best_idx, double* losses,
                                      void* s_best, float* per_token_err, void* stream);

/*
 * Apply the quantized layer with a chosen scale: Y_q = f_q(X; s) (+ bias), the activation the next
 * layer calibrates on under the paper's adopted propagation strategy (Sec. 3.2.1, PassAct2).
 *   s [C1] bf16 or NULL; bias [C2] bf16 or NULL; Yq [N,C2] bf16 (C2 a multiple of 8);
 *   codes/steps/zeros as in tlq_quantize_weights (NULL = not wanted).
 */
size_t tlq_apply_layer_workspace_bytes(int64_t N, int64_t C1, int64_t C2, const tlq_config* cfg);
int tlq_apply_layer(const void* X, int64_t N, int64_t C1, const void* W, int64_t C2, const void* s,
                    const void* bias, const tlq_config* cfg, void* workspace, size_t workspace_bytes,
                    uint8_t* codes, float* steps, int32_t* zeros, void* Yq, void* stream);

/* Synchronise `stream` and return the device status word of `workspace` (TLQ_OK, TLQ_ERR_TIMEOUT,
 * TLQ_ERR_NONFINITE) or TLQ_ERR_CUDA if the stream reports an error. */
int tlq_read_status(const void* workspace, void* stream);

/*
 * Diagnostic of the device-side error path (the paper has no counterpart).  Every barrier wait inside the fused
 * tensor-core kernels is bounded; when a bound expires the kernel writes TLQ_ERR_TIMEOUT to the status word and
 * returns instead of hanging.  A correct run never gets there, so this call takes that path on purpose and
 * harmlessly: one warp waits `limit_cycles` SM clock cycles (1 .. 2e9, i.e. at most about a second) on a barrier
 * that nothing arrives on, then reports through the status word of `workspace` (at least 256 bytes, 16-byte
 * aligned, zeroed by this call).  Afterwards tlq_read_status(workspace, stream) returns TLQ_ERR_TIMEOUT and the
 * device context is as usable as before: no fault, no trap, no unbounded loop.
 */
int tlq_selftest_bounded_wait(void* workspace, size_t workspace_bytes, int64_t limit_cycles, void* stream);

/*
 * Diagnostics for TLQ_FLAG_DEBUG_CANARIES (the paper has no counterpart).  kind: 0 = the workspace of
 * tlq_scale_search_layer, 1 = of tlq_apply_layer; cfg must carry the flag.
 * tlq_debug_canary_offsets (host only, no device is touched): writes the byte offset of each guard (256 bytes each)
 * into offsets[0 .. max_offsets) (host; may be NULL) and returns how many guards the layout has, or a negative
 * TLQ_ERR_*.
 * tlq_debug_check_canaries: compares the guards of a workspace that a flagged call has left behind once more (for
 * instance after other work that might have scribbled on it); the outcome goes to the status word like the call's own
 * check.  It does not clear the status word first.
 */
int tlq_debug_canary_offsets(int kind, int64_t N, int64_t C1, int64_t C2, const tlq_config* cfg,
                             uint64_t* offsets /* host */, int max_offsets);
int tlq_debug_check_canaries(int kind, int64_t N, int64_t C1, int64_t C2, const tlq_config* cfg, void* workspace,
                             size_t workspace_bytes, void* stream);

/*
 * Diagnostic (the paper has no counterpart): what the library measured about the current device's L2.  The L2 of this
 * GPU is two partitions; the first large group-mode search on a device measures which partition each SM sits next to,
 * and the fused bf16 GEMM then keeps each partition's CTAs to their own token tiles.  This call synchronises the device
 * and copies the table to the HOST: info[0] = 1 if a usable table exists (0: not measured yet, or the measurement did
 * not split the SMs into two clear groups, in which case the GEMM uses its plain tile order), info[1] = SMs measured,
 * info[2], info[3] = SMs per partition; part (256 bytes, or NULL) = partition of each SM id.
 */
int tlq_l2_partition_info(int32_t* info /* host [4] */, uint8_t* part /* host [256] or NULL */);

/*
 * Diagnostic, host only (the paper has no counterpart; no device is touched): the order in which the persistent CTAs
 * of the fused bf16 GEMM visit the (candidate, output tile, token tile) space, replayed on the host.  With n1 = 0
 * it is the walk of a grid of n0 CTAs (blocked != 0: by blocks of block_a token tiles); with n1 > 0 the walk of
 * n0 + n1 CTAs split over the two L2 partitions (n0 and n1 SMs; token tiles cut between them, blocked must be 0,
 * mtiles >= 4).  Every visit adds one to visits[(k * otiles + ot) * mtiles + mt] (HOST array of K * otiles * mtiles
 * int32, zeroed by the caller): a correct walk leaves every entry at exactly 1.
 */
int tlq_debug_tile_walk(int64_t mtiles, int64_t otiles, int32_t K, int32_t n0, int32_t n1, int32_t blocked,
                        int32_t block_a, int32_t* visits /* host */);

/* The same replay for the tile-resident kernels (symmetric modes, two-stream search): `grid` persistent CTAs, each
 * keeping an output tile for all K candidates, the tiles of the last partial wave split by candidates over the idle
 * CTAs; blocked != 0 walks the tiles in blocks of 16 token tiles.  Same `visits` layout and meaning. */
int tlq_debug_resident_walk(int64_t mtiles, int64_t otiles, int32_t K, int32_t grid, int32_t blocked,
                            int32_t* visits /* host */);

/*
 * Per-stage device timing of tlq_scale_search_layer, for benchmarks.  While enabled, every search call
 * records CUDA events on its stream between its stages (event sets come from a pool of 512 created on
 * first use; further calls are not recorded).  _drain() synchronises on the recorded events, writes
 * TLQ_N_STAGES durations in milliseconds per recorded call, oldest first, to the HOST array ms_out
 * (room for max_calls calls), forgets them and returns how many calls it wrote (or a negative
 * TLQ_ERR_*).  _enable() also forgets what was recorded.  Off by default; not thread-safe.
 */
int tlq_stage_timing_enable(int on);
int tlq_stage_timing_drain(float* ms_out /* host [max_calls][TLQ_N_STAGES] */, int max_calls);

/* Number of kernels launched by this library since load (host counter; benchmarks report it). */
int64_t tlq_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* TLQ_H_ */
