/*
 * gptaq.h -- C ABI of the B200 (sm_100a) GPTAQ per-layer solve.
 *
 * GPTAQ quantizes one linear layer W (m x n, rows = output channels) so that
 * the quantized layer fed with the quantized model's input X reproduces the
 * full-precision layer fed with the full-precision input X~ (the paper's
 * asymmetric calibration objective, Eq. "asym obj", Section 4).  The calls
 * map to the steps of Algorithm 1 of the paper:
 *
 *   gptaq_accumulate   the statistics          H += X X^T,  dXX^T += (X~ - X) X^T
 *   gptaq_factor       the inverse Cholesky    L = Inverse_Cholesky(H + lambda_1 I), kept as U = L^T
 *   gptaq_build_P      the correction matrix   P = ((dXX^T L) .* M_U) L^T          (Theorem 4.2)
 *   gptaq_quantize     the blocked loop        column loop + lazy-batch trailing update
 *
 * Conventions
 *  - Every pointer named d_* is DEVICE memory, every pointer named h_* is
 *    HOST memory.  All device memory is allocated and owned by the caller;
 *    the library allocates no device memory.  The handle itself is a small
 *    host object owned by the library between gptaq_create / gptaq_destroy.
 *  - Matrices are row-major float32 unless stated.  Activations are
 *    token-major: X is passed as X^T, [tokens x n] with leading dimension ld.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *    Calls only enqueue work and return; host-side argument and call-order
 *    errors are returned at once, conditions found on the device (a
 *    non-positive pivot, a non-finite value, a bounded wait that ran out) are
 *    recorded in a device status word that gptaq_sync_status() reads.  Nothing
 *    traps or asserts on the device.  The calls on one handle are one sequence of
 *    work: give them one stream, or order the streams yourself (an event between
 *    calls); the handle keeps host-side counters that mirror device-side ones in
 *    the order of the calls, and one call's kernels read what the previous call's wrote.
 *  - Call order: create -> accumulate* -> factor -> build_P -> quantize*.
 *    Anything else returns GPTAQ_ERR_BAD_STATE.  gptaq_reset() returns a
 *    handle to the state right after create.  quantize may be called many
 *    times on one state (layers that share an input share H, U and P).
 *  - A handle is not thread-safe; distinct handles are independent.
 */
#ifndef GPTAQ_H_
#define GPTAQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gptaq_ctx *gptaq_handle_t;
typedef void *gptaq_stream_t; /* a cudaStream_t */

typedef enum {
    GPTAQ_OK = 0,
    GPTAQ_ERR_INVALID_ARG = 1,  /* null pointer, negative size, misaligned buffer */
    GPTAQ_ERR_BAD_STATE = 2,    /* call out of order */
    GPTAQ_ERR_WORKSPACE = 3,    /* state / workspace / staging buffer too small */
    GPTAQ_ERR_NOT_SPD = 4,      /* device: a pivot of the damped H was <= 0; info = its index */
    GPTAQ_ERR_NONFINITE = 5,    /* device: NaN/Inf met in H or W; info = row or column index */
    GPTAQ_ERR_TIMEOUT = 6,      /* device: a bounded wait ran out; info = where */
    GPTAQ_ERR_UNSUPPORTED = 7,  /* argument combination outside the supported set */
    GPTAQ_ERR_CUDA = 8          /* a CUDA runtime call failed; see gptaq_last_cuda_error */
} gptaq_status_t;

enum { GPTAQ_W_FP32 = 0, GPTAQ_W_BF16 = 1 };

/* Arithmetic of the statistics (Algorithm 1, first step).  In the two tensor-core modes X and
 * X~ - X (the difference taken in float32 first) are rounded to fp16, scaled by a power of two
 * if the batch would leave the fp16 range, and multiplied by tcgen05 MMAs with float32
 * accumulation; they apply for n >= 256 and for n = 128, other small layers always take the float32 path.
 * GPTAQ_STATS_FP16_SPLIT_TENSOR (default): H additionally carries the rounding remainder of X
 *   as a second fp16 term (H = hi hi^T + hi lo^T + lo hi^T, about 22 significant bits), so that
 *   the factor U keeps its accuracy even with few tokens per input channel.
 * GPTAQ_STATS_FP16_TENSOR: single fp16 term (11 significant bits), 40 % fewer MMAs; accurate
 *   enough for U once total tokens >= 16 n (see gptaq_recommended_stats_precision).
 * GPTAQ_STATS_FP16_SPLIT_FULL_TENSOR: both sums carry the remainders (dXX^T = dh xh^T + dh xl^T +
 *   dl xh^T as well): float32-grade statistics at three times the MMAs of the single-term mode.
 *   The entries of dXX^T are themselves sums of randomly signed products, so the fp16 rounding of
 *   single terms stays visible in them (about 3e-4 relative, and as much in P); that is far inside the
 *   tolerances at alpha = 0.25 and 2-4 bits, but shows as rounding-tie flips at 8 bits and in the
 *   objective once alpha approaches 1 with weak damping: use this mode (or GPTAQ_STATS_FP32) there.
 * GPTAQ_STATS_FP32: float32 products and sums on the plain FMA pipes (exact inputs). */
enum { GPTAQ_STATS_FP16_TENSOR = 0, GPTAQ_STATS_FP32 = 1, GPTAQ_STATS_FP16_SPLIT_TENSOR = 2,
       GPTAQ_STATS_FP16_SPLIT_FULL_TENSOR = 3 };

/* Bytes of the caller-owned device state for layer width n: a header (status
 * word, pivot index), H (n x n), dXX^T (n x n) and the dead-input flags.
 * After gptaq_factor, U overwrites H; after gptaq_build_P, P overwrites dXX^T. */
size_t gptaq_state_bytes(int64_t n);

/* Bytes of caller-owned device scratch that accumulate / factor / build_P / quantize need
 * for width n, at most m_max weight rows and the given lazy-batch block size
 * (Algorithm 1, input B).  max_batch_tokens is the largest `tokens` that
 * gptaq_accumulate will be given in one call (larger batches still work: they
 * are processed in chunks that fit).  For n >= 512 the scratch holds split (high part / low part)
 * operand copies of U^T and P^T for the tensor cores: about 4 n^2 floats in all where n is a multiple
 * of 8 (fp16 parts), about 7 n^2 where it is a multiple of 4 only (TF32 parts).  The library reads them
 * in every gptaq_quantize, so the workspace must be left untouched from gptaq_factor until the last
 * gptaq_quantize on this state. */
size_t gptaq_workspace_bytes(int64_t n, int64_t m_max, int64_t max_batch_tokens, int blocksize);

/* Creates a handle over caller-owned device buffers (both 256-byte aligned)
 * on the current CUDA device and enqueues the zeroing of H and dXX^T
 * (the statistics of Algorithm 1 start from empty sums). */
gptaq_status_t gptaq_create(gptaq_handle_t *out, int64_t n, void *d_state, size_t state_bytes,
                            void *d_workspace, size_t workspace_bytes, gptaq_stream_t stream);

/* Back to the state right after gptaq_create (sums zeroed, token count 0). */
gptaq_status_t gptaq_reset(gptaq_handle_t h, gptaq_stream_t stream);

gptaq_status_t gptaq_destroy(gptaq_handle_t h);

/* Algorithm 1, the statistics, one token batch:  H += X X^T,  dXX^T += (X~ - X) X^T.
 * d_X, d_Xfp: [tokens x n] float32, leading dimension ld >= n, read only.
 * The difference X~ - X is formed in float32 before any product.
 * tokens == 0 is a no-op.  Only the upper triangle of H is maintained (H is symmetric).  Of dXX^T only the
 * part above the diagonal is guaranteed: Theorem 4.2 masks (dXX^T U^T) with the strictly upper triangular
 * M_U and row j of U starts at column j, so entry (i, k) of dXX^T reaches P only where k > i; the entries on
 * and below the diagonal are accumulated where that is free (the simple FMA path; inside the diagonal
 * tiles of the tensor-core path) and otherwise left as they were -- a third of the products saved.  With
 * act_order enabled the whole of dXX^T is accumulated, because the permutation mixes the two triangles:
 * enable it before the first token batch (see gptaq_set_act_order). */
gptaq_status_t gptaq_accumulate(gptaq_handle_t h, const float *d_X, const float *d_Xfp,
                                int64_t tokens, int64_t ld, gptaq_stream_t stream);

/* gptaq_accumulate converts the batch on `stream` and may run the product itself on a stream
 * of the handle's own, so that the conversion of the next batch overlaps it.  Every other call
 * that takes the handle and a stream (reset, factor, sync_status) first orders its stream after
 * that work.  A caller that wants to read the sums through gptaq_H / gptaq_D on `stream` right
 * after gptaq_accumulate, or to time the accumulation with events on `stream`, calls
 * gptaq_flush: it makes `stream` wait (on the device, not on the host) for the pending
 * products. */
gptaq_status_t gptaq_flush(gptaq_handle_t h, gptaq_stream_t stream);

/* Same with HOST inputs (pinned memory for asynchronous copies): copies the
 * batch into d_stage (device, >= 2 * tokens * n * 4 bytes) on `stream`, then
 * accumulates from there. */
gptaq_status_t gptaq_accumulate_host(gptaq_handle_t h, const float *h_X, const float *h_Xfp,
                                     int64_t tokens, int64_t ld, void *d_stage, size_t stage_bytes,
                                     gptaq_stream_t stream);

/* Algorithm 1, the inverse-Cholesky step, with the customary GPTQ preprocessing that Section 4 refers to:
 * H <- H / tokens; inputs with H_qq == 0 get H_qq = 1 (their weight columns
 * are zeroed by gptaq_quantize); H_d = H + damp * mean(diag H) * I; then the
 * upper factor U of H_d^-1 = U^T U (U = L^T of the paper) overwrites H
 * (strict lower triangle zeroed).  Needs at least one accumulated token. */
gptaq_status_t gptaq_factor(gptaq_handle_t h, float damp, gptaq_stream_t stream);

/* Algorithm 1, the step that forms P / Theorem 4.2:  P = alpha * ((dXX^T U^T) .* M_U) U with
 * dXX^T normalised by the token count like H, M_U the strictly-upper mask.
 * alpha = 1 is the paper's P; alpha = 0 reduces the solve to GPTQ.
 * P overwrites dXX^T (lower triangle and diagonal zero). */
gptaq_status_t gptaq_build_P(gptaq_handle_t h, float alpha, gptaq_stream_t stream);

/* The same P computed row by row, Eq. "unparallel" (Section 4, Step 3):
 *   P[q, q+1:] = alpha * dXX^T[q, q+1:] L[q+1:, q+1:] L[q+1:, q+1:]^T,   L = U^T,
 * i.e. two passes over the trailing triangle of U for every row q: the form that Theorem 4.2 replaces by
 * two matrix products.  It exists as the slow side of the latency comparison of Section 5 ("Efficiency")
 * and gives the same P up to rounding; the solve itself uses gptaq_build_P.  Same call order and effects
 * as gptaq_build_P; n <= 16384 (GPTAQ_ERR_UNSUPPORTED beyond). */
gptaq_status_t gptaq_build_P_rowwise(gptaq_handle_t h, float alpha, gptaq_stream_t stream);

/* Algorithm 1, the blocked loop, for one weight matrix sharing this state.
 *   d_W      [m x ldw], float32 or bf16 (w_dtype).  If d_Wq is given, d_W is read
 *            only and the float32 working copy lives in d_Wq (required for bf16
 *            weights).  If d_Wq is NULL (or equal to d_W), float32 weights are
 *            updated in place and hold the dequantized result on return
 *            (column j becomes Q[:, j] at step j).
 *   bits     2..8;  group: 0 = one grid per output channel taken from the
 *            original row, else a grid per `group` consecutive columns taken
 *            from the current (already updated) weights at the group's first
 *            column; requires blocksize % group == 0.
 *   sym      0: asymmetric min/max grid containing zero, zero point = rint(-lo/scale);
 *            1: symmetric grid, scale = max|w| / (2^(bits-1) - 1), stored code
 *            = s + 2^(bits-1).  Rounding is round-half-to-even.
 *   blocksize  lazy-batch block B in {32, 64, 128}.
 *   d_codes  [m x n] uint8 out;  d_scales, d_zeros [m x G] float32 out,
 *            G = 1 (group == 0) or ceil(n / group).
 *   d_Wq     [m x n] float32 out, dequantized weights (ld n); may be NULL for
 *            float32 weights.
 * m == 0 is a no-op. */
gptaq_status_t gptaq_quantize(gptaq_handle_t h, void *d_W, int w_dtype, int64_t m, int64_t ldw,
                              int bits, int group, int sym, int blocksize,
                              uint8_t *d_codes, float *d_scales, float *d_zeros, float *d_Wq,
                              gptaq_stream_t stream);

/* Same with HOST weights in and HOST codes / scales / zeros out: copies W into
 * d_stage (device, >= gptaq_quantize_stage_bytes(m, n, group)), quantizes there and copies
 * the three results back; all on `stream`, asynchronous if the host memory is
 * pinned.  h_Wq (dequantized float32, [m x n]) may be NULL. */
size_t gptaq_quantize_stage_bytes(int64_t m, int64_t n, int group);
gptaq_status_t gptaq_quantize_host(gptaq_handle_t h, const float *h_W, int64_t m, int64_t ldw,
                                   int bits, int group, int sym, int blocksize,
                                   uint8_t *h_codes, float *h_scales, float *h_zeros, float *h_Wq,
                                   void *d_stage, size_t stage_bytes, gptaq_stream_t stream);

/* (No counterpart in the paper.)  gptaq_quantize for callers that cannot hand the library a
 * scratch buffer of their own -- code that runs where device allocation is off limits (inside a
 * real-time loop, under a memory pool whose budget is already spent, in a plug-in that is not
 * allowed to call the CUDA allocator) and that therefore cannot size a workspace per layer.
 * It needs no handle and no workspace: the factor and the correction matrix are plain inputs,
 * and the m x 2B scratch of the lazy-batch update ([-Err | Wpre]: the error matrix E of Algorithm 1 and the block's columns) lives in
 * an array built into the library.  The function allocates nothing, on the device or through
 * any library.
 *   d_U, d_P   [n x n] float32, leading dimension n: U (upper, H_d^-1 = U^T U) and P (strictly
 *              upper), e.g. gptaq_H / gptaq_D of a handle after gptaq_build_P, or restored
 *              copies of them.  All n inputs are taken as live: there are no dead-input flags
 *              here, so a caller whose layer has inputs that never fired (H_qq = 0) zeroes those
 *              columns of W itself before the call, as gptaq_quantize would.  U and P of a
 *              handle with act_order enabled are in SORTED column order: such a caller passes W
 *              with its columns gathered by gptaq_perm and scatters the codes and dequantized
 *              weights back; this entry point does not permute.
 *   d_status   device int64[2] or NULL: receives the status a handle would record
 *              (GPTAQ_OK or GPTAQ_ERR_NONFINITE) and the row index that goes with it.
 *   All other arguments as in gptaq_quantize.
 * Limits: n <= GPTAQ_STATIC_MAX_N and m * 2 * blocksize <= GPTAQ_STATIC_SCRATCH_FLOATS (4 MiB
 * of scratch: m <= 4096 at blocksize 128); beyond them GPTAQ_ERR_WORKSPACE is returned before
 * any work is enqueued.  Every GPU that loads the library holds the array (about 4 MiB) until
 * the process exits.
 * The first call on each device looks up the array's device address and configures the
 * kernels (with that device current); make that first call outside any stream capture.
 * All calls on a device share the one array, which still holds the previous call's contents;
 * the function clears what has to start from zero, but two calls whose work overlaps on the
 * GPU (different streams, no dependency between them) race on it: order them. */
#define GPTAQ_STATIC_MAX_N 16384
#define GPTAQ_STATIC_SCRATCH_FLOATS (1 << 20)
gptaq_status_t gptaq_quantize_static(const float *d_U, const float *d_P, int64_t n, void *d_W, int w_dtype,
                                     int64_t m, int64_t ldw, int bits, int group, int sym, int blocksize,
                                     uint8_t *d_codes, float *d_scales, float *d_zeros, float *d_Wq,
                                     int64_t *d_status, gptaq_stream_t stream);

/* Synchronises `stream`, then returns the device status word (GPTAQ_OK, or the
 * first device-side condition recorded since create/reset) and, in *info, the
 * index that goes with it (may be NULL). */
gptaq_status_t gptaq_sync_status(gptaq_handle_t h, int64_t *info, gptaq_stream_t stream);

/* Device views into the state (n x n, leading dimension n), for tests and for
 * callers that checkpoint the sums: H / U and dXX^T / P share storage.  What is defined of the sums:
 * the upper triangle of H; of dXX^T the part above the diagonal, all of it under act_order. */
float *gptaq_H(gptaq_handle_t h);
float *gptaq_D(gptaq_handle_t h);
/* The same storage under the names of what it holds later: U (the inverse-Cholesky factor of Algorithm 1; NULL
 * before gptaq_factor) and P (Theorem 4.2; NULL before gptaq_build_P). */
const float *gptaq_U(gptaq_handle_t h);
const float *gptaq_P(gptaq_handle_t h);
int64_t gptaq_tokens(gptaq_handle_t h);
/* Sets the token count (for callers that restore checkpointed sums). */
gptaq_status_t gptaq_set_tokens(gptaq_handle_t h, int64_t tokens);

/* Chooses the arithmetic of gptaq_accumulate (see GPTAQ_STATS_*); allowed before gptaq_factor. */
gptaq_status_t gptaq_set_stats_precision(gptaq_handle_t h, int precision);
/* The cheapest tensor-core mode whose rounding keeps the relative error of U below 1e-4 for a
 * layer of width n calibrated on total_tokens tokens. */
int gptaq_recommended_stats_precision(int64_t n, int64_t total_tokens);

/* act_order (Section 5, experimental setup: columns processed in the order of the Hessian's diagonal):
 * when enabled (before gptaq_factor), gptaq_factor orders the inputs by decreasing diag(H) (dead inputs
 * count as 1; ties keep the lower index first), permutes H and dXX^T accordingly, and gptaq_quantize
 * processes the weight columns in that order.  Outputs: d_codes and d_Wq in the CALLER's column order;
 * group grids (d_scales / d_zeros, group > 0) belong to groups of `group` consecutive columns of the
 * SORTED order, i.e. caller column c uses group rank(c) / group, rank being the inverse of gptaq_perm.
 * gptaq_quantize then needs d_Wq as a second buffer (non-NULL, different from d_W).
 * gptaq_H / gptaq_D show U and P in sorted order.  Supported for n <= 57344.
 * Enabling it after a token batch has gone in without the lower triangle of dXX^T (see gptaq_accumulate)
 * returns GPTAQ_ERR_BAD_STATE; gptaq_reset clears that.
 * gptaq_perm: device array of n int32, sorted position -> caller column; NULL unless enabled and factored. */
gptaq_status_t gptaq_set_act_order(gptaq_handle_t h, int enable);
const int32_t *gptaq_perm(gptaq_handle_t h);

/* Static groups (Section 5, setup of the per-group results with act_order): when enabled, later gptaq_quantize
 * calls with group > 0 take every group grid BEFORE the loop, from the original weights, for groups of
 * `group` consecutive columns of the CALLER's column order; a column keeps the grid of its own group wherever
 * act_order moves it in the processing order.  d_scales / d_zeros [m x G] then index caller column c by
 * c / group, with or without act_order -- no index table is needed to dequantize.  Without act_order the
 * only difference from the default is that grids come from the original instead of the updated weights.
 * Such calls take the general column kernel (one warp per row), not the 32-columns-per-thread one. */
gptaq_status_t gptaq_set_static_groups(gptaq_handle_t h, int enable);

/* Clipping-range search of the quantization grids by least squared rounding error (experimental
 * setup of Section 5; the paper gives no further detail).  With steps > 0 every
 * grid -- per output channel, or per group at the group's first column -- is chosen among `steps`
 * candidates that shrink the min/max range by p_k = 1 - k (1 - min_ratio) / steps, k = 0 .. steps - 1:
 * the candidate with the smallest sum of squared rounding errors over the grid's weights, the widest one
 * on ties.  steps = 0 (default) is the plain min/max grid; 0 < min_ratio < 1. */
gptaq_status_t gptaq_set_clip_search(gptaq_handle_t h, int steps, float min_ratio);

/* Ablation switches of the weight update (Section 5.3, Table "ablation"): which of the two terms of
 * Eq. "divided update" later gptaq_quantize calls on this handle apply.
 *   GPTAQ_TERM_ERR    the quantization-error term  -(w_q - q_q)/U_qq * U[q, :]   (GPTQ's update)
 *   GPTAQ_TERM_ASYM   the asymmetry term           w_q * P[q, :]
 * Both (default) = GPTAQ; ERR alone = GPTQ; ASYM alone = the paper's GPTAQ'; none = round to
 * nearest on the same grids. */
enum { GPTAQ_TERM_ERR = 1, GPTAQ_TERM_ASYM = 2 };
gptaq_status_t gptaq_set_update_terms(gptaq_handle_t h, int terms);

/* Number of kernels this handle has launched since create (bookkeeping for benchmarks). */
int64_t gptaq_launch_count(gptaq_handle_t h);

/* Timing of the dominant kernel by itself (bookkeeping for benchmarks).  While enabled, every launch of the
 * tensor-core statistics kernel (the statistics of Algorithm 1) is bracketed by a pair of CUDA events on the stream it
 * runs on -- the handle's own stream, which events of the caller cannot reach.  gptaq_stats_kernel_time waits
 * (on the host) for the recorded launches, returns the sum of their durations in milliseconds and their number,
 * and starts a new record.  The conversion prologue and the fix-up of K-split tiles are not included. */
gptaq_status_t gptaq_set_kernel_timing(gptaq_handle_t h, int enable);
gptaq_status_t gptaq_stats_kernel_time(gptaq_handle_t h, double *ms_total, int64_t *launches);

/* Failure-path self-test: enqueues one warp that waits, with the bounded wait of the tensor-core
 * kernels, for a barrier that nothing completes; after `seconds` (0 < seconds <= 2, in SM clock
 * cycles at the nominal clock) it gives up and records GPTAQ_ERR_TIMEOUT (info 2000000) for
 * gptaq_sync_status.  Nothing traps and the context stays usable; gptaq_reset clears the status. */
gptaq_status_t gptaq_selftest_bounded_wait(gptaq_handle_t h, double seconds, gptaq_stream_t stream);

const char *gptaq_status_string(gptaq_status_t s);
/* Text of the last CUDA runtime error seen by this handle ("" if none). */
const char *gptaq_last_cuda_error(gptaq_handle_t h);

#ifdef __cplusplus
}
#endif
#endif /* GPTAQ_H_ */
