/*
 * obc.h -- C ABI of the B200 (sm_100a) ExactOBS / OBQ layer solver ("Optimal Brain Compression").
 *
 * One layer is a weight matrix W (d_row x d_col) and calibration inputs X (d_col x N), as in the paper's
 * layer-wise compression problem (Section 2, Eq. 2).  The calls below are the stages of the method:
 *
 *   obc_hessian            H = 2 X X^T, accumulated over chunks of N          (Section 3, "ExactOBS")
 *   obc_hessian_inverse    Hinv = inv(H + damp I)                             (Section 3, "Implementation Details")
 *   obc_prune_trace        Algorithm 1 on every row: order P, loss trace L    (Section 3, Steps 1-2)
 *   obc_select_global_mask Algorithm 2: global mask with k pruned weights     (appendix, global step)
 *   obc_prune_apply        remaining weights for the chosen per-row counts    (Section 3, Figure 1)
 *   obc_minmax_grid        per-row uniform grid over the kept weights
 *   obc_quantize           Algorithm 3 (OBQ), optionally after a pruning replay (Section 4; Section 6 setup)
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer owned by the caller unless the comment says "host".  The library
 *     allocates nothing, frees nothing and keeps no state between calls (the kernel-launch counter of
 *     obc_kernel_launches is a diagnostic only).  Scratch memory comes from the caller's workspace `ws` of at
 *     least obc_workspace_bytes(...) bytes (256-byte aligned).
 *   - Matrices are row-major FP32 with a leading dimension in elements.  Base pointers of FP32 matrices
 *     are 16-byte aligned and leading dimensions are multiples of 4.
 *   - Calls enqueue work on `stream` and return without synchronising.  Argument errors are found on the
 *     host and returned before anything is launched or written.  Data-dependent failures never trap: they
 *     are written to `info` / `row_status` in device memory.
 *   - row_begin / row_count select a row range; outputs of other rows are not touched, so a layer can be
 *     split across calls (or devices) and resumed by range.
 *   - Original column indices are 0-based.  mask: 1 = kept, 0 = pruned.
 */
#ifndef OBC_H_
#define OBC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    OBC_OK = 0,
    OBC_ERR_INVALID_ARG = 1,   /* NULL pointer, negative or inconsistent size, unknown enum              */
    OBC_ERR_ALIGNMENT = 2,     /* pointer not 16-byte aligned or leading dimension not a multiple of 4   */
    OBC_ERR_WORKSPACE = 3,     /* ws is NULL, misaligned or smaller than obc_workspace_bytes(...)        */
    OBC_ERR_NOT_POSDEF = 4,    /* (reported through info[]) Cholesky met a non-positive pivot            */
    OBC_ERR_NONFINITE = 5,     /* (reported through row_status[]) non-positive / non-finite [Hinv]_pp    */
    OBC_ERR_TIMEOUT = 6,       /* (reported through info[]) a bounded device-side wait expired           */
    OBC_ERR_CUDA = 7,          /* a CUDA runtime call failed (launch configuration, missing device ...)  */
    OBC_ERR_UNSUPPORTED = 8,   /* size outside what the kernels support (d_col > OBC_MAX_DCOL)           */
    OBC_ERR_STATIC_SCRATCH = 9 /* problem larger than the built-in scratch area of a *_static entry point */
} obc_status;

typedef enum { OBC_PREC_FP32 = 0, OBC_PREC_TF32 = 1, OBC_PREC_BF16X3 = 2 } obc_prec;

enum {
    OBC_FLAG_OUTLIERS = 1      /* obc_quantize: quantise weights whose error exceeds Delta/2 first
                                  (Section 4, "Quantization Outliers"); off = plain argmin of Eq. 7      */
};

typedef enum {
    OBC_OP_HESSIAN = 0, OBC_OP_INVERSE = 1, OBC_OP_PRUNE_TRACE = 2, OBC_OP_SELECT = 3,
    OBC_OP_PRUNE_APPLY = 4, OBC_OP_QUANTIZE = 5, OBC_OP_PRUNE_BLOCKS = 6, OBC_OP_CROSS_GRAM = 7, OBC_OP_REFIT = 8
} obc_op;

/* Which row elimination engine obc_prune_trace / obc_prune_apply / obc_quantize run (all compute Algorithm 1 /
 * Algorithm 3; they differ in how the Lemma-1 updates reach the row's private inverse Hessian):
 *   STREAMING  one pass over the row's active triangle per step (rank-1 update, bound by memory bandwidth);
 *   BLOCKED    the updates are held back as vectors and applied several at a time, so the triangle is read and
 *              written once per block of steps; the pivot column of a step is corrected by the pending vectors;
 *   AUTO       = BLOCKED. */
typedef enum { OBC_ENGINE_AUTO = 0, OBC_ENGINE_STREAMING = 1, OBC_ENGINE_BLOCKED = 2 } obc_engine;

#define OBC_MAX_DCOL 5120      /* per-row state of the elimination engine lives in one CTA's shared memory */

typedef void *obc_stream;      /* a cudaStream_t (NULL = default stream) */

const char *obc_status_string(obc_status s);

/* Diagnostic (host function): number of kernels this library has launched in the calling process so far. */
unsigned long long obc_kernel_launches(void);

/* Per-call choice of how the row elimination engine runs (HOST struct, read before the call returns).  Every
 * row-engine entry point takes a pointer to one; NULL means all defaults.  Nothing here changes results beyond the
 * order of FP32 roundings: every choice computes Algorithm 1 / Algorithm 3.
 *   engine      : a value of the obc_engine enum, AUTO = BLOCKED.  obc_prune_nm / obc_prune_blocks always run BLOCKED and ignore it.
 *   threads     : BLOCKED engine, threads per row: 128, 256, 512, or 0 = chosen from d_col and row_count.
 *   max_pending : BLOCKED engine, upper limit on the number of deferred updates, 1..64, or 0 = as many as the
 *                 shared memory holds.
 *   flags       : OBC_ENGINE_WHOLE_WAVES or 0.  By default, when a call has more rows than the GPU holds at once (with
 *                 several rows per SM: up to three times as many) and they do not divide evenly, the BLOCKED engine
 *                 gives every thread block the same amount of work, so a row may be started by one block and finished
 *                 by another; with OBC_ENGINE_WHOLE_WAVES every row stays on one block and the last wave runs partly
 *                 empty.
 * Values outside these sets make the call return OBC_ERR_INVALID_ARG.  Workspace sizes reported by
 * obc_workspace_bytes are valid for every choice. */
typedef struct {
    int32_t engine;
    int32_t threads;
    int32_t max_pending;
    int32_t flags;
} obc_engine_opts;
enum { OBC_ENGINE_WHOLE_WAVES = 1 };

/* How the row engines would run row_count rows (0 = many) of length d_col on the CURRENT device with the options
 * `opts` (host function, no launch).  with_trace != 0: as for obc_prune_trace with a weight trace.
 * plan (host int32[8]): [0] engine (OBC_ENGINE_STREAMING or OBC_ENGINE_BLOCKED), [1] threads per row,
 * [2] rows resident per SM, [3] active size at which a row moves into shared memory, [4] floats of shared memory
 * for deferred update vectors (BLOCKED), [5] limit on deferred updates (BLOCKED), [6] SM count, [7] further
 * deferred update vectors kept in global memory (BLOCKED, long rows; sized to stay in L2).
 * A BLOCKED row of current size m defers min(plan[5], plan[4] / stride(m) + plan[7]) updates between two passes
 * over its matrix, stride(m) = round_up(m + 8, 32) + 8 floats per deferred vector.  Used by the benchmark to state
 * the bytes a launch has to move. */
obc_status obc_engine_plan(int d_col, int with_trace, int row_count, const obc_engine_opts *opts, int32_t *plan);

/* Bytes of workspace the given call needs for these sizes on the CURRENT device (host function, no launch).
 * n is only used by OBC_OP_HESSIAN; row_count (the rows one call processes) by the three row-engine ops,
 * where 0 means "size for any row_count".  Returns 0 on invalid arguments. */
size_t obc_workspace_bytes(obc_op op, int row_count, int d_col, int64_t n);

/* Section 3 ("ExactOBS"): the Hessian of every row's least-squares problem is H = 2 X X^T.
 * X: d_col x n, row-major, ldx >= n (one chunk of the calibration axis).  H: d_col x d_col, ldh >= d_col.
 * accumulate = 0 overwrites H, 1 adds to it (Section 3, "Implementation Details": further samples are
 * accumulated into the Hessian once).  H is written in full (both triangles, exactly symmetric).
 * prec picks the tensor-core input precision of the contraction; accumulation is FP32.
 * The tensor-core kernels synchronise their copy / multiply pipeline through device-side waits, all of them bounded:
 *   wait_limit : 0 = the built-in bound (about a second per wait); > 0 = that many polls per wait; < 0 = the
 *                pipeline's waits expire at once (a test hook: it exercises the time-out path without waiting).
 *   info       : nullable device int32; receives 0, or OBC_ERR_TIMEOUT when a wait expired.  In that case the
 *                kernel has abandoned its tile cleanly (its copies in flight and issued products are waited for with
 *                the built-in bound, tensor memory is released), the call has still returned OBC_OK, and H is
 *                filled with NaN -- also when info is NULL -- so the failure cannot pass unnoticed.
 * OBC_PREC_FP32 has no waits: wait_limit is ignored and info[0] = 0. */
obc_status obc_hessian(const float *X, int d_col, int64_t n, int64_t ldx,
                       float *H, int ldh, int accumulate, obc_prec prec, int32_t *info, int wait_limit,
                       void *ws, size_t ws_bytes, obc_stream stream);

/* Appendix "Sequential Quantization with OBQ": when the layer inputs X come from the already compressed model, the
 * dense weights are first re-fitted in closed form, W^T = (X X^T)^-1 X Y^T (Y = the dense model's outputs, d_row x n),
 * so that they minimise the layer objective again.  X Y^T is accumulated over batches like the Hessian:
 *   obc_cross_gram : G (+)= Y X^T   (G: d_row x d_col, ldg >= d_col; Y: d_row x n, ldy >= n; X: d_col x n, ldx >= n;
 *                    prec, info, wait_limit as in obc_hessian (G = NaN after a time-out);
 *                    workspace obc_workspace_bytes(OBC_OP_CROSS_GRAM, d_row, d_col, n))
 *   obc_refit      : W = 2 G Hinv with Hinv = inv(2 X X^T + lambda I) from obc_hessian / obc_hessian_inverse on the
 *                    same X, i.e. the least-squares weights with the solver's dampening lambda/2 on X X^T.  A dense
 *                    d_row x d_col x d_col contraction: prec = OBC_PREC_FP32 runs it on the CUDA cores (no workspace),
 *                    TF32 / BF16X3 on the tensor cores with the kernel of obc_cross_gram (workspace
 *                    obc_workspace_bytes(OBC_OP_REFIT, d_row, d_col, 0); a time-out of its bounded waits leaves NaN). */
obc_status obc_cross_gram(const float *Y, int64_t ldy, const float *X, int64_t ldx, int d_row, int d_col, int64_t n,
                          float *G, int ldg, int accumulate, obc_prec prec, int32_t *info, int wait_limit,
                          void *ws, size_t ws_bytes, obc_stream stream);
obc_status obc_refit(const float *G, int ldg, const float *Hinv, int ldhi, int d_row, int d_col,
                     float *W_out, int ldwo, obc_prec prec, void *ws, size_t ws_bytes, obc_stream stream);

/* Section 3 ("Implementation Details"): Hinv = inv(H + damp_rel * mean(diag H) * I) through a Cholesky
 * factorisation carried in FP64, written as an exactly symmetric FP32 matrix (ldhi >= d_col).
 * info[0] (device int32) = 0, or 1 + index of the first non-positive pivot (Hinv is then undefined). */
obc_status obc_hessian_inverse(const float *H, int d_col, int ldh, float damp_rel,
                               float *Hinv, int ldhi, int32_t *info,
                               void *ws, size_t ws_bytes, obc_stream stream);

/* Algorithm 1 for rows [row_begin, row_begin+row_count) of W (d_row x d_col, ldw >= d_col), each on its
 * own FP32 copy of Hinv: `steps` (1..d_col) greedy eliminations; step t removes
 * p = argmin_{p in M} w_p^2 / [Hinv]_pp (ties: lowest index), compensates the remaining weights (Eq. 3)
 * and eliminates p from the row's inverse Hessian (Lemma 1).
 *   order  : d_row x d_col int32, order[r][t] = column removed at step t        (entries t >= steps untouched)
 *   loss   : d_row x d_col FP32,  loss[r][t] = w_p^2/[Hinv]_pp at that moment   (Section 3, Step 2)
 *   w_trace: NULL, or d_row x (steps+1) x d_col FP32: the whole row after t = 0..steps eliminations
 *            (Figure 1, the "more memory" option)
 *   row_status: d_row int32, 0 or 1+t if [Hinv]_pp was non-positive / non-finite at step t (the row stops:
 *            its later order entries are -1 and loss entries +inf). */
obc_status obc_prune_trace(const float *W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                           const float *Hinv, int ldhi, int steps,
                           int32_t *order, float *loss, float *w_trace, int32_t *row_status,
                           void *ws, size_t ws_bytes, const obc_engine_opts *opts, obc_stream stream);

/* Section 3, "N:M Sparsity": Algorithm 1 with the argmin restricted to weights whose block of m_block consecutive
 * columns has lost fewer than m_block - n_keep weights so far; after d_col * (m_block - n_keep) / m_block
 * eliminations every block keeps exactly n_keep non-zeros, and no global step is needed (all rows have the same
 * sparsity).  (The paper's sentence counts "< N pruned weights", which equals m_block - n_keep for its 2:4 and 4:8
 * patterns; the count used here is the general one.)
 *   m_block in {2, 4, 8, 16, 32}, 0 < n_keep < m_block, d_col a multiple of m_block.
 *   order, loss: d_row x d_col as in obc_prune_trace, the first d_col*(m_block-n_keep)/m_block entries of a row
 *                are written; nullable.
 *   W_out : d_row x d_col FP32 (ldwo): the compensated weights, 0 at pruned positions.
 *   mask  : nullable d_row x d_col uint8, 1 = kept.
 * Always runs on the BLOCKED engine.  Workspace: obc_workspace_bytes(OBC_OP_PRUNE_TRACE, row_count, d_col, 0). */
obc_status obc_prune_nm(const float *W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                        const float *Hinv, int ldhi, int n_keep, int m_block,
                        int32_t *order, float *loss, float *W_out, int ldwo, uint8_t *mask, int32_t *row_status,
                        void *ws, size_t ws_bytes, const obc_engine_opts *opts, obc_stream stream);

/* Section 3, "Block-Sparsity" (Eq. 5): Algorithm 1 on blocks of `block` consecutive columns.  Each step removes the
 * remaining block P with the smallest w_P^T ((Hinv)_P)^-1 w_P (ties: lowest block), compensates the other weights by
 * -Hinv[:,P] ((Hinv)_P)^-1 w_P and eliminates the members of P from the row's inverse Hessian one after the other
 * (Lemma 1) -- which is the same as eliminating the members singly in ascending order, and that is how it runs.
 *   block = c = 4 or 8 (the sizes the section names; others: OBC_ERR_UNSUPPORTED); d_col a multiple of c.  Full trace
 *           (all d_col / c blocks).
 *   order : d_row x d_col, the members of the t-th block at [ct, ct+c), ascending.
 *   loss  : d_row x d_col, loss[r][ct] = the block's score, loss[r][ct+1..ct+c-1] = 0, so that
 *           obc_select_global_mask with k a multiple of c takes whole blocks, and obc_prune_apply works unchanged.
 *   w_trace: as in obc_prune_trace (one row per single elimination), nullable.
 * Always runs on the BLOCKED engine.  Workspace: obc_workspace_bytes(OBC_OP_PRUNE_BLOCKS, row_count, d_col, 0). */
obc_status obc_prune_blocks(const float *W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                            const float *Hinv, int ldhi, int block,
                            int32_t *order, float *loss, float *w_trace, int32_t *row_status,
                            void *ws, size_t ws_bytes, const obc_engine_opts *opts, obc_stream stream);

/* Algorithm 2 (appendix, "ExactOBS Global Step"): repeatedly prune, across all rows, the weight whose
 * next recorded loss is smallest (ties: lowest row), k times.  k is a count, 0 <= k <= d_row*d_col.
 *   counts: d_row int32, weights pruned per row;  mask: d_row x d_col uint8, 0 at order[r][t], t < counts[r].
 * The result is exactly the sequential procedure's (computed as a selection over prefix-maximum keys). */
obc_status obc_select_global_mask(const float *loss, const int32_t *order, int d_row, int d_col, int64_t k,
                                  int32_t *counts, uint8_t *mask,
                                  void *ws, size_t ws_bytes, obc_stream stream);

/* Allocation-free variant of obc_select_global_mask.  The paper has no counterpart: this exists for callers
 * that cannot provide a workspace because they are not allowed to allocate device memory at this point --
 * for example a plug-in running inside a host application that handed the whole GPU to its own memory pool at
 * start-up, or a service loop where a cudaMalloc (which may synchronise the device and can fail under
 * fragmentation) is not acceptable once it is running.  Inputs and outputs are still the caller's; the scratch
 * memory is a fixed array inside the library's device image, so every GPU that loads the library carries it
 * (about 16.2 MiB) until the process exits.
 *   Limits: d_row <= OBC_SELECT_STATIC_MAX_ROWS and d_row*d_col <= OBC_SELECT_STATIC_MAX_KEYS; anything larger
 *   returns OBC_ERR_STATIC_SCRATCH and launches nothing.
 *   The first call on each device looks up the array's device address (a host-side runtime call).  With CUDA's
 *   lazy module loading that first call may also be the moment the driver loads this library's device image and
 *   sets the array aside, which can fail once a host application owns all remaining memory: make the first call at
 *   start-up, before the memory is handed out and outside any stream capture (or run with CUDA_MODULE_LOADING=EAGER,
 *   which ties the reservation to library load).  After it, no call allocates or frees memory.
 *   All calls on a device share the one array: the call rewrites everything it later reads, so back-to-back calls
 *   on one stream are fine, but two calls that can overlap on the GPU (different streams or threads) race.
 * Results are identical to obc_select_global_mask. */
#define OBC_SELECT_STATIC_MAX_KEYS (4 * 1024 * 1024)
#define OBC_SELECT_STATIC_MAX_ROWS 16384
obc_status obc_select_global_mask_static(const float *loss, const int32_t *order, int d_row, int d_col, int64_t k,
                                         int32_t *counts, uint8_t *mask, obc_stream stream);

/* Section 3 / Figure 1: the weights of each row after its first counts[r] eliminations.
 * w_trace != NULL (layout of obc_prune_trace with this `trace_steps`): rows are gathered from the trace.
 * w_trace == NULL: the eliminations order[r][0..counts[r]) are replayed on W (no argmin). */
obc_status obc_prune_apply(const float *W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                           const float *Hinv, int ldhi, const int32_t *order, const int32_t *counts,
                           const float *w_trace, int trace_steps,
                           float *W_out, int ldwo, int32_t *row_status,
                           void *ws, size_t ws_bytes, const obc_engine_opts *opts, obc_stream stream);

/* Per-row uniform grid over the kept entries (mask NULL = all kept); the range always contains 0.
 *   asymmetric: maxq = 2^bits-1, scale = (hi-lo)/maxq, zero = rne(-lo/scale)
 *   symmetric : Q = 2^(bits-1)-1, scale = max|w|/Q, zero = Q, maxq = 2Q
 * A row without spread gets scale = 1.  bits in 2..16.  *maxq_host (host pointer, nullable) receives maxq.
 * The paper fixes only "symmetric / asymmetric per-channel grids" (Section 6); this min-max rule is the
 * benchmark configurations' choice, and any other grid can be passed to obc_quantize instead. */
obc_status obc_minmax_grid(const float *W, int ldw, int d_row, int d_col, const uint8_t *mask,
                           int bits, int symmetric, float *scale, float *zero, int *maxq_host,
                           obc_stream stream);

/* Algorithm 3 (OBQ) for a row range: like Algorithm 1 with the target q(w_p) instead of 0 (Eq. 7), where
 * q(x) = scale * (clamp(rne(x/scale) + zero, 0, maxq) - zero) and maxq follows from bits/symmetric as above.
 *   prune_order / prune_counts == NULL: scale, zero (d_row FP32) are INPUTS; all d_col weights are quantised.
 *   otherwise (compound, Section 6 "Experimental Setup": sparsify first, then quantise the rest): the first
 *     prune_counts[r] eliminations of prune_order[r] are replayed, the row's min-max grid is built from the
 *     compensated survivors and written to scale/zero (OUTPUTS), and only the survivors are quantised.
 *   W_out  : d_row x d_col FP32 (ldwo), quantised weights (pruned entries 0)
 *   codes  : d_row x d_col int32 in [0, maxq] (pruned entries -1)
 *   loss, qorder: nullable d_row x d_col; step t of the quantisation loop (same meaning as in obc_prune_trace)
 *   flags  : OBC_FLAG_OUTLIERS or 0 */
obc_status obc_quantize(const float *W, int ldw, int d_row, int d_col, int row_begin, int row_count,
                        const float *Hinv, int ldhi, float *scale, float *zero, int bits, int symmetric,
                        const int32_t *prune_order, const int32_t *prune_counts, int flags,
                        float *W_out, int ldwo, int32_t *codes, float *loss, int32_t *qorder,
                        int32_t *row_status, void *ws, size_t ws_bytes, const obc_engine_opts *opts, obc_stream stream);

#ifdef __cplusplus
}
#endif
#endif /* OBC_H_ */
