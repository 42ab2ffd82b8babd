/*
 * algproj.h -- C ABI of the row-typed associative-algebra projection  Y = X *_q W  for
 * NVIDIA B200 (sm_100a).
 *
 * The operation (paper, Section "Transformer Projections", Eqs. typed-diag / typed-off, and
 * Section "Training and Inference", Eq. recursive-row-action, Algorithm 1):
 *   X is M x K, W is the ordinary K x N weight bank.  Input features are split into q groups
 *   of widths s[0..q-1] (sum K), output features into q groups of widths r[0..q-1] (sum N);
 *   W_{kj} = W[S_k, R_j] is the s[k] x r[j] sub-block.  Row b carries a type t_b in [0,q)
 *   (0-based; the paper counts types from 1).  Its output group j is
 *        y_j = bias_j + sum_{k in B(t_b, j)} x_k W_{kj},
 *   where for the paper's complete-graph law Q_q the support set is B(i,j) = {i,j} as a set:
 *        y_i = x_i W_ii,      y_j = x_i W_ij + x_j W_jj   (j != i).
 *   For q = 2 this is the six-product rule (Eq. six-product): type-0 rows give
 *   [A Wa, A Wu + U Wd], type-1 rows give [V Wa + D Wv, D Wd].
 *
 * Conventions
 *   - All matrices are row-major; leading dimensions are in ELEMENTS.
 *   - Every pointer named X, W, bias, Y, types, workspace is a DEVICE pointer unless the
 *     function name ends in _host; the caller owns all of them and the stream.
 *   - W is the canonical bank: no packing or transposition is required.
 *   - Y is overwritten, never accumulated into (Algorithm 1 starts from Y <- 0).
 *   - forward calls enqueue work on `stream` and return; they never synchronise with the
 *     host and never allocate, so they can be captured into a CUDA graph (the captured graph
 *     bakes in the addresses and M it was captured with).
 *   - Two forward calls that share a workspace must be ordered on the GPU (same stream or an
 *     event between them).
 *   - Nothing aborts, traps or throws across this boundary; every function returns a status.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 */
#ifndef ALGPROJ_H_
#define ALGPROJ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct alg_proj_s *alg_proj_t;
typedef struct alg_ffn_s *alg_ffn_t;
typedef struct alg_proj_grad_s *alg_proj_grad_t;

typedef enum {
  ALG_OK = 0,
  ALG_ERR_INVALID_ARG = 1,         /* NULL pointer, q out of range, non-positive width, ...   */
  ALG_ERR_UNSUPPORTED_SHAPE = 2,   /* legal problem this build has no kernel for              */
  ALG_ERR_WORKSPACE_TOO_SMALL = 3, /* workspace_bytes below alg_*_workspace_bytes(M)          */
  ALG_ERR_CUDA = 4,                /* a CUDA runtime/driver call failed                       */
  ALG_ERR_BAD_TYPE = 5,            /* device saw types[b] outside [0,q); that row of Y is 0   */
  ALG_ERR_DEVICE_TIMEOUT = 6       /* a bounded device-side wait expired; output is invalid   */
} alg_status_t;

typedef enum { ALG_F32 = 0, ALG_BF16 = 1 } alg_dtype_t;

/* Which (type i, output group j, input group k) products are kept.
 * QQ     : the paper's complete-graph law, k in {i,j}  (2q^2-q block GEMMs, Eq. q-rank).
 * DENSE  : all k -- the ordinary product X W (q^3 block GEMMs); the same-library control.
 * CUSTOM : caller-supplied keep[(i*q+j)*q+k] bytes (non-zero = kept).
 * Q2POW  : the tensor power Q_2^{(x)L}, q = 2^L (appendix "The Tensor-Square Candidate", the law
 *          of the paper's pretraining pilot with L = 2): types and groups are L-bit strings and
 *          k is kept for (i,j) iff every bit of k equals the matching bit of i or of j
 *          (6^L block GEMMs; 36 for q = 4; arithmetic fraction (3/4)^L with equal groups). */
typedef enum { ALG_TABLE_QQ = 0, ALG_TABLE_DENSE = 1, ALG_TABLE_CUSTOM = 2, ALG_TABLE_Q2POW = 3 } alg_table_t;

/* Activation applied to (acc + bias) before the store. GELU_ERF is z/2 (1 + erf(z/sqrt 2)). */
typedef enum { ALG_ACT_NONE = 0, ALG_ACT_GELU_ERF = 1, ALG_ACT_GELU_TANH = 2 } alg_act_t;

/* EXPLICIT: the caller passes types[M] with every forward call.
 * CYCLIC  : type of row b is b mod q (the paper's example schedule tau(p) = p mod q for a
 *           batch whose sequence length is a multiple of q); `types` may be NULL.
 *           With q | M the tensor-core path needs no permutation, and the tile sequences of its
 *           persistent CTAs depend only on (handle, M): they are planned on the host at the
 *           first forward call with a given M, uploaded asynchronously on `stream` (no host
 *           wait) into device memory the handle owns (sized at create; forward allocates
 *           nothing) and kept for the last few M.  A call made while `stream` is being captured
 *           lets the kernels plan for themselves instead (same result), so a captured graph
 *           never depends on the handle's plan cache.  Forward calls on one handle must be
 *           ordered on the GPU (one stream, or events between streams).
 * INTERVAL: type of row b is b / (M/q), q | M: the rows of a type are contiguous -- the typing of
 *           the square product A * B of two algebra elements (Eqs. q-product-diag/off), where
 *           the rows of block row i of A carry type i; `types` may be NULL.  No permutation and
 *           no copy of X.  Handles that fit the large-algebra path (see alg_proj_create) take it;
 *           other bf16 handles with tensor-core widths read X in 64-row boxes inside the runs of
 *           a type (M / q a multiple of 64) and may repeat the typing with a period
 *           (ALG_OPT_INTERVAL_PERIOD); FFN handles of that kind accept INTERVAL too. */
typedef enum { ALG_SCHED_EXPLICIT = 0, ALG_SCHED_CYCLIC = 1, ALG_SCHED_INTERVAL = 2 } alg_schedule_t;

/* Kernel families, reported by alg_proj_kernel_path(). */
typedef enum {
  ALG_PATH_SIMT = 0,    /* fp32-FMA tiles, any widths                                    */
  ALG_PATH_TCGEN05 = 1, /* bf16 grouped tcgen05 GEMM, TMA-fed, TMEM accumulators         */
  ALG_PATH_DECODE = 2   /* small-M kernels (one row: plain FMAs; up to 64 rows: weight streaming) */
} alg_path_t;

#define ALG_MAX_Q 32        /* general interaction tables (32-bit keep masks) */
#define ALG_MAX_Q_LARGE 256 /* complete-graph law Q_q with equal group widths: the large-algebra path */

/* Per-handle options (alg_proj_set_option / alg_ffn_set_option).  They replace process-wide
 * switches: nothing in the library reads the environment.  Set them between forward calls,
 * not concurrently with one; a value the handle's shape cannot honour is refused with
 * ALG_ERR_UNSUPPORTED_SHAPE and changes nothing.
 *   GEMM_KERNEL       which prefill tensor-core kernel runs: 0 = the library's choice (default),
 *                     1 = one-CTA 128-row tiles (tcgen05 cta_group::1), 2 = CTA pairs
 *                     (cta_group::2), 3 = one-CTA 256-row x 128-column tiles (two accumulators
 *                     per tile, each B block feeds two MMAs).  2 and 3 need every output group
 *                     width to be a multiple of 128.  4 = the large-algebra kernel (see
 *                     alg_proj_create) for a projection handle whose law, dtype and widths fit it.
 *   TILE_N            tile width of the one-CTA kernel: 0 = automatic, or 128 / 192 / 256 when
 *                     that divides every output group width.
 *   STAGE_K           reduction depth of one pipeline stage of the one-CTA GEMM kernel: 0 =
 *                     automatic, 32 (eight stages of 24 KB) or 64 (four stages of 48 KB).  Results
 *                     are identical; only the operand pipeline differs.  A table-driven INTERVAL
 *                     handle reads its runs with 64-deep stages only: 32 is ALG_ERR_UNSUPPORTED_SHAPE there.
 *   ROW_GATHER        explicit row types on the one-CTA GEMM kernel: how the rows of a type reach the kernel.
 *                     1 = a copy pass writes the type-bucketed copy of X into the workspace; 2 = the kernel's
 *                     producer warps fetch the rows through the permutation themselves (four rows per copy
 *                     instruction, X read in place, one launch fewer); 0 (default) = 1, which measures faster or
 *                     equal on every benchmark step.  Results are identical.  Ignored by the other kernels.
 *   WEIGHT_PACKED     1: the W given to alg_proj_forward is the padded bank alg_proj_pack_weight wrote (ldw is
 *                     ignored); 0 (default): the caller's K x N bank.  Only handles whose
 *                     alg_proj_packed_weight_bytes is not 0 take 1 (else ALG_ERR_UNSUPPORTED_SHAPE).
 *   INTERVAL_PERIOD   INTERVAL schedule of a table-driven handle: the typing repeats every P rows, type of
 *                     row b = (b mod P) / (P / q) -- the pilot model's schedule
 *                     floor((p mod 768) / 192) over a batch of sequences.  0 (default) = one period,
 *                     P = M.  q must divide P, P must divide M, and P / q must be a multiple of 64.
 *   SMALL_M_KERNEL    1 (default): small batches run the small-M kernels where the library expects them to
 *                     be faster; 0: the prefill kernels take every M; 2: only the weight-streaming /
 *                     staged kernels (M <= 64 / M <= 16) besides the prefill kernels; 3: the row kernel
 *                     (plain FMAs, M <= 8) wherever it fits.
 *   HOST_PLAN         1 (default): cyclic-schedule tile sequences are planned on the host;
 *                     0: every CTA plans for itself.
 *   WAIT_LIMIT_CYCLES bound of every device-side wait (mbarrier, counter), in SM clock cycles;
 *                     default 4e9 (about 2 s).  A wait that runs out sets
 *                     ALG_ERR_DEVICE_TIMEOUT in the status word and the kernel returns.
 *   TEST_STALL_BYTES  test aid, default 0: the small-M kernels add this many bytes to what they
 *                     expect on their weight barrier.  The bytes never arrive, every issued
 *                     copy still lands, the bounded wait runs out and the call reports
 *                     ALG_ERR_DEVICE_TIMEOUT -- the way to exercise that path without a fault. */
typedef enum {
  ALG_OPT_GEMM_KERNEL = 1,
  ALG_OPT_TILE_N = 2,
  ALG_OPT_SMALL_M_KERNEL = 3,
  ALG_OPT_HOST_PLAN = 4,
  ALG_OPT_WAIT_LIMIT_CYCLES = 5,
  ALG_OPT_TEST_STALL_BYTES = 6,
  ALG_OPT_STAGE_K = 7,
  ALG_OPT_INTERVAL_PERIOD = 8,
  ALG_OPT_ROW_GATHER = 9,
  ALG_OPT_WEIGHT_PACKED = 10
} alg_option_t;

/* ---- projection handle ---------------------------------------------------------------------
 * alg_proj_create: build the interaction table for q groups (Eqs. q-product-diag/off, or the
 * DENSE / CUSTOM variants), pick kernels, allocate a few hundred bytes of device metadata on
 * the CURRENT device.  in_widths = s[q], out_widths = r[q] (host arrays, copied).  dtype is
 * the element type of X and W (ALG_F32: true fp32 FMAs; ALG_BF16: bf16 operands, fp32
 * accumulation).  custom_keep is read only for ALG_TABLE_CUSTOM, else pass NULL; every
 * (i,j) of a custom table must keep at least one k.  1 <= q <= ALG_MAX_Q.
 * The tensor-core path needs every s[k] to be a multiple of 64 and every r[j] a multiple of
 * 128 (or of 192); other bf16/fp32 shapes run on the SIMT path, except:
 *
 * Large-algebra path (the fixed-block regime of Section "Kernel Benchmarks" and of the appendix
 * "Large Projections and Square Products": q = n / b grows with the matrix, blocks such as
 * 160 x 800 or 40 x 200 that are no multiple of the GPU tile).  Taken for ALG_TABLE_QQ with
 * bf16 operands and EQUAL group widths s, r that are multiples of 4, when q > ALG_MAX_Q (up to
 * ALG_MAX_Q_LARGE), when the widths do not fit the ordinary tensor-core path, or when the
 * schedule is INTERVAL.  Same tcgen05 pipeline; tiles are enumerated by arithmetic (type-major,
 * so a row panel W[S_i, :] is streamed once), the operands are fetched through per-group tensor
 * maps whose out-of-range elements read as zero (a group narrower than the 32- or 64-deep
 * pipeline stage, or a last column tile narrower than the tile, costs arithmetic on zeros but
 * no extra bytes), and stores are masked at 8-column granularity.  Widths that are multiples of
 * 4 but not of 8 (20 x 100) cannot be addressed by tensor maps: every call first repacks X and W
 * into the workspace with each group widened to the next multiple of 8 (zeros), and stores Y in
 * 4-column pieces; alg_proj_workspace_bytes accounts for the two repacked operands.  All three schedules work
 * (EXPLICIT and CYCLIC with q not dividing M go through bucketing and a row gather first;
 * INTERVAL needs q | M); fp32 operands, other tables, unequal or odd widths with q > ALG_MAX_Q
 * are refused with ALG_ERR_UNSUPPORTED_SHAPE.  The FFN and gradient
 * handles do not take this path.  */
alg_status_t alg_proj_create(alg_proj_t *out, int q, const int32_t *in_widths,
                             const int32_t *out_widths, alg_dtype_t dtype, alg_table_t table,
                             const uint8_t *custom_keep, alg_schedule_t schedule);
alg_status_t alg_proj_destroy(alg_proj_t h);
alg_status_t alg_proj_set_option(alg_proj_t h, alg_option_t option, int64_t value);

/* Bytes of device scratch a forward call with at most max_M rows needs (row permutation,
 * bucket offsets, and -- on the tensor-core path -- the type-bucketed copy of X).  The contents
 * need no initialisation. */
alg_status_t alg_proj_workspace_bytes(alg_proj_t h, int64_t max_M, size_t *bytes);

/* Y[M x N] = act( X[M x K] *_q W[K x N] + bias ).
 * X: dtype of the handle, ldx >= K.  types: int32[M] device (ignored for CYCLIC).
 * W: dtype of the handle, ldw >= N.  bias: N values of the handle's dtype, or NULL.
 * Y: y_dtype (ALG_F32 or ALG_BF16, round-to-nearest-even), ldy >= N.
 * workspace: >= alg_proj_workspace_bytes(h, M), 256-byte aligned.
 * bf16 pointers and leading dimensions must keep rows 16-byte aligned (multiples of 8
 * elements).  M = 0 is a successful no-op; a type with no rows is legal.
 * Small M with bf16: up to 8 rows under ALG_TABLE_QQ with equal widths in multiples of 8 are one launch
 * of plain FMAs over the 2 / q of the bank each row's type needs (any q up to ALG_MAX_Q_LARGE), taken
 * while the rows' weight segments stay below a measured break-even (always for one row); M <= 64
 * runs the weight-streaming decode kernel when its per-CTA weight slice fits shared memory and the
 * handle has at most 8 groups or a bank of at most 4 Mi elements; everything else the prefill
 * kernels.  (The FFN calls: a few rows likewise one launch -- both projections around a bounded
 * wait -- and M <= 16 for shapes whose weight slices fit shared memory.)
 * Kernels are launched with programmatic stream serialization: they may start while the
 * kernel before them on `stream` is finishing, and wait for it before they touch X, bias, Y or
 * the workspace.  The decode kernel requests W before that wait (weights do not change during
 * a step): W must not be written by the kernel that immediately precedes the call on `stream`.
 * `types` may be: it is read once early to choose the weight blocks to request and again after
 * the wait; if the two readings differ the blocks are requested again. */
alg_status_t alg_proj_forward(alg_proj_t h, const void *X, int64_t ldx, const int32_t *types,
                              int64_t M, const void *W, int64_t ldw, const void *bias,
                              alg_act_t act, void *Y, int64_t ldy, alg_dtype_t y_dtype,
                              void *workspace, size_t workspace_bytes, void *stream);

/* alg_proj_forward without a workspace argument and without any allocation.  (The paper has
 * no counterpart to this call; it exists for integration reasons only.)
 *
 * Who needs it: code that runs where device memory cannot be requested -- a serving loop whose
 * memory was handed out once at start-up to a pool it may not grow, a plug-in called from a
 * host framework that forbids cudaMalloc / cudaFree on its hot path because they synchronise
 * the whole device, or a caller that simply has no allocator to hand.  Such callers still pass
 * their own X, types, W, bias and Y; only the scratch (row permutation, bucket offsets,
 * type-bucketed copy of X) comes from the library, from a fixed array of
 * ALG_STATIC_SCRATCH_BYTES that is part of the loaded library image on every GPU and stays
 * there until the process exits.
 *
 * Limits and rules
 *   - The handle must exist already: create it once at start-up (creation does allocate a few
 *     hundred bytes).  This call itself performs no cudaMalloc, cudaFree or other allocation.
 *   - Problems whose scratch need, alg_proj_workspace_bytes(h, M), exceeds
 *     ALG_STATIC_SCRATCH_BYTES are refused with ALG_ERR_WORKSPACE_TOO_SMALL and nothing is
 *     launched; use alg_proj_forward with your own workspace for those.
 *   - The first call on each device looks up the device address of the array (with that device
 *     current); with lazy module loading that is also when the driver places the array, so
 *     the device's free memory drops by its size once, during that call and never after.
 *     Make that first call at start-up, outside any stream capture.
 *   - All calls on one device share the one array.  It keeps whatever the previous call left;
 *     nothing in it has to start at zero, every call rewrites what it reads.  Two calls that
 *     overlap on the GPU (different streams without an event between them) race on it and
 *     give undefined results: order them.
 * Arguments, layouts and results are otherwise exactly those of alg_proj_forward. */
#define ALG_STATIC_SCRATCH_BYTES (8u << 20)
alg_status_t alg_proj_forward_static(alg_proj_t h, const void *X, int64_t ldx,
                                     const int32_t *types, int64_t M, const void *W, int64_t ldw,
                                     const void *bias, alg_act_t act, void *Y, int64_t ldy,
                                     alg_dtype_t y_dtype, void *stream);

/* Number of kept block GEMMs (2q^2-q for QQ, Eq. q-rank). */
alg_status_t alg_proj_gemm_count(alg_proj_t h, int64_t *n);
/* Multiply-accumulates of one forward pass with rows_per_type[i] rows of type i
 * (Eq. rectangular-batch-cost: M D_diag + sum_i M_i s_i (N - r_i) for QQ). Host array in. */
alg_status_t alg_proj_macs(alg_proj_t h, const int64_t *rows_per_type, int64_t *macs);
/* Kernel family a forward call with M rows would use. */
alg_status_t alg_proj_kernel_path(alg_proj_t h, int64_t M, alg_path_t *path);
/* Read and clear the handle's device status word (ALG_OK, ALG_ERR_BAD_TYPE or
 * ALG_ERR_DEVICE_TIMEOUT).  Synchronises `stream` first.  After ALG_ERR_DEVICE_TIMEOUT the
 * handle's internal counters are reset, so the next forward call starts clean. */
alg_status_t alg_proj_last_status(alg_proj_t h, void *stream, alg_status_t *status);

/* ---- weights packed once (large-algebra handles with group widths that are multiples of 4 only) ---
 * Such a handle copies X and W with every group widened to a multiple of 8 by zeros on each forward
 * call (tiled copies start on 16 bytes).  W does not change between calls: alg_proj_pack_weight
 * writes the padded bank once -- (q * ceil8(s)) x (q * ceil8(r)) elements of the handle's dtype,
 * row-major, device memory, 16-byte aligned -- and with option WEIGHT_PACKED = 1 alg_proj_forward
 * reads it in place, so that only X is copied per call.  alg_proj_packed_weight_bytes: size of that
 * buffer; 0 when the handle pads nothing (then there is nothing to pack: ALG_ERR_UNSUPPORTED_SHAPE
 * from alg_proj_pack_weight).  The pack runs on `stream`; W: K x N, ldw >= N, as in
 * alg_proj_forward. */
alg_status_t alg_proj_packed_weight_bytes(alg_proj_t h, size_t *bytes);
alg_status_t alg_proj_pack_weight(alg_proj_t h, const void *W, int64_t ldw, void *W_packed,
                                  size_t packed_bytes, void *stream);

/* ---- FFN handle: Y = act(X *_q W_up + b_up) *_q W_down + b_down  ---------------------------
 * The two-map MLP (g = 1 in Eq. icml-decode-total) with both projections under the same law
 * and the same row types (the projection is row-local).  d_widths: q groups of d_model,
 * f_widths: q groups of d_ff.  X: M x D packed (ld = D), W_up: D x F packed, W_down: F x D
 * packed, Y: M x D packed.  The hidden state H = act(.) is kept in the workspace in the
 * handle's dtype (bf16: rounded to nearest even), rows in type-bucketed order.
 * 1 <= q <= ALG_MAX_Q, schedule EXPLICIT or CYCLIC (larger algebras and the INTERVAL schedule
 * exist for single projections only: ALG_ERR_UNSUPPORTED_SHAPE).  Which GEMM kernel runs the two
 * projections is the library's choice per call (alg_ffn_set_option(GEMM_KERNEL) overrides it);
 * kernels differ in the order of their fp32 sums, so results agree to rounding between them. */
alg_status_t alg_ffn_create(alg_ffn_t *out, int q, const int32_t *d_widths,
                            const int32_t *f_widths, alg_dtype_t dtype, alg_table_t table,
                            const uint8_t *custom_keep, alg_schedule_t schedule);
alg_status_t alg_ffn_destroy(alg_ffn_t h);
alg_status_t alg_ffn_set_option(alg_ffn_t h, alg_option_t option, int64_t value);  /* both projections */
alg_status_t alg_ffn_workspace_bytes(alg_ffn_t h, int64_t max_M, size_t *bytes);
alg_status_t alg_ffn_forward(alg_ffn_t h, const void *X, const int32_t *types, int64_t M,
                             const void *W_up, const void *b_up, const void *W_down,
                             const void *b_down, alg_act_t act, void *Y, alg_dtype_t y_dtype,
                             void *workspace, size_t workspace_bytes, void *stream);
/* ---- gated FFN (SwiGLU): Y = (silu(X *_q W_gate) .* (X *_q W_up)) *_q W_down  -----------------
 * The FFN of the paper's pretraining pilot (Section "Projection Shapes": a gated FFN uses two
 * D x F weights and one F x D weight, the same row law on each; appendix "Experimental Details":
 * bias-free SwiGLU; appendix "Kernel Benchmark Details", Table kernel-ffn: gate and up merged).
 * silu(g) = g / (1 + exp(-g)).  No biases.
 * W_gate_up is the merged bank, D x 2F packed: columns [0, F) are W_gate, columns [F, 2F) are W_up,
 * each split into the q hidden groups f_widths; one kernel accumulates the gate and the up columns
 * of a tile side by side and stores silu(gate) * up, so the two pre-activations never reach memory.
 * W_down is F x D packed.  Create with alg_ffn_gated_create (bf16 only).  Shapes: every d width a
 * multiple of 64 and every f width a multiple of 128 (any table); or, under ALG_TABLE_QQ, equal d
 * widths and equal f widths that are multiples of 8 (the large-algebra kernel: e.g. 2048 -> 6144 or
 * 2048 -> 768 split 32 ways); anything else is ALG_ERR_UNSUPPORTED_SHAPE.  Workspace size, options,
 * MAC count (three projections), status and destruction through the alg_ffn_* calls.
 * A few rows (always M = 1) under ALG_TABLE_QQ with equal widths are ONE launch (two matrix-vector
 * phases on plain FMAs around a bounded wait; option SMALL_M_KERNEL = 0 sends them through the prefill
 * kernels instead); every other M runs the prefill kernels.  With the CYCLIC schedule and q | M the rows are read and
 * written in place (two launches); otherwise bucketing and the row gather run first. */
alg_status_t alg_ffn_gated_create(alg_ffn_t *out, int q, const int32_t *d_widths,
                                  const int32_t *f_widths, alg_dtype_t dtype, alg_table_t table,
                                  const uint8_t *custom_keep, alg_schedule_t schedule);
alg_status_t alg_ffn_gated_forward(alg_ffn_t h, const void *X, const int32_t *types, int64_t M,
                                   const void *W_gate_up, const void *W_down, void *Y,
                                   alg_dtype_t y_dtype, void *workspace, size_t workspace_bytes,
                                   void *stream);

/* ---- gradient maps of the projection (training) ------------------------------------------------
 * Appendix "Vector-Jacobian Products", Eqs. vjp-xi ... vjp-wjj: with G the gradient with respect to
 * Y = X *_q W,
 *     dX[b, S_k]   = sum_{j : k in B(t_b, j)} G[b, R_j] W[S_k, R_j]^T
 *     dW[S_k, R_j] = sum_{b : k in B(t_b, j)} X[b, S_k]^T G[b, R_j].
 * Both keep exactly the block support of the forward table, so each costs the forward MACs
 * (Section "Scaling and Practical Implementation"); every output element has one owner (no atomics,
 * bitwise repeatable).  bf16 operands, fp32 accumulation; dX / dW in x_dtype / w_dtype.
 * A gradient handle is created with the parameters of the forward projection it belongs to
 * (in_widths = s[q] of X, out_widths = r[q] of Y).  dW runs on the tensor-core path only: every r
 * must be a multiple of 128 (or of 192), else ALG_ERR_UNSUPPORTED_SHAPE; dX needs every r to be a
 * multiple of 64 and every s a multiple of 128 (or 192) for that path and otherwise runs on the
 * SIMT kernel.  A custom table must give every weight block at least one row type that uses it.
 *   grad_input : W is the forward bank (K x N, ldw >= N), used transposed in place.
 *   grad_weight: dW (K x N, lddw >= N) is overwritten, never accumulated into; blocks whose row
 *                types are absent from the batch come out zero.  Internally the rows are bucketed
 *                by type, X is copied transposed and G bucketed (both padded per bucket to a
 *                multiple of 64 rows with zeros), and one grouped GEMM reduces over the buckets.
 * Workspace: alg_proj_grad_workspace_bytes(h, M), 256-byte aligned, no initialisation needed. */
alg_status_t alg_proj_grad_create(alg_proj_grad_t *out, int q, const int32_t *in_widths,
                                  const int32_t *out_widths, alg_table_t table,
                                  const uint8_t *custom_keep, alg_schedule_t schedule);
alg_status_t alg_proj_grad_destroy(alg_proj_grad_t h);
alg_status_t alg_proj_grad_workspace_bytes(alg_proj_grad_t h, int64_t max_M, size_t *bytes);
alg_status_t alg_proj_grad_input(alg_proj_grad_t h, const void *G, int64_t ldg, const int32_t *types,
                                 int64_t M, const void *W, int64_t ldw, void *dX, int64_t lddx,
                                 alg_dtype_t x_dtype, void *workspace, size_t workspace_bytes,
                                 void *stream);
alg_status_t alg_proj_grad_weight(alg_proj_grad_t h, const void *X, int64_t ldx, const void *G,
                                  int64_t ldg, const int32_t *types, int64_t M, void *dW,
                                  int64_t lddw, alg_dtype_t w_dtype, void *workspace,
                                  size_t workspace_bytes, void *stream);
alg_status_t alg_proj_grad_last_status(alg_proj_grad_t h, void *stream, alg_status_t *status);

/* alg_proj_forward with X, types and Y in HOST memory (packed rows: ldx = K, ldy = N; pinned
 * memory makes the copies asynchronous): copies X and types to device staging inside the
 * workspace, runs the projection, copies Y back, all on `stream`; returns without
 * synchronising.  W and bias stay device pointers.  Workspace size:
 * alg_proj_host_workspace_bytes (device memory, 256-byte aligned). */
alg_status_t alg_proj_host_workspace_bytes(alg_proj_t h, int64_t max_M, alg_dtype_t y_dtype,
                                           size_t *bytes);
alg_status_t alg_proj_forward_host(alg_proj_t h, const void *X_host, const int32_t *types_host,
                                   int64_t M, const void *W, int64_t ldw, const void *bias,
                                   alg_act_t act, void *Y_host, alg_dtype_t y_dtype,
                                   void *workspace, size_t workspace_bytes, void *stream);

/* Same computation with X, types and Y in HOST memory (pinned memory makes the copies
 * asynchronous).  Copies X and types to device staging inside the workspace, runs the
 * forward pass, copies Y back, all on `stream`; returns without synchronising.  Weights and
 * biases stay device pointers.  Workspace size: alg_ffn_host_workspace_bytes. */
alg_status_t alg_ffn_host_workspace_bytes(alg_ffn_t h, int64_t max_M, alg_dtype_t y_dtype,
                                          size_t *bytes);
alg_status_t alg_ffn_forward_host(alg_ffn_t h, const void *X_host, const int32_t *types_host,
                                  int64_t M, const void *W_up, const void *b_up,
                                  const void *W_down, const void *b_down, alg_act_t act,
                                  void *Y_host, alg_dtype_t y_dtype, void *workspace,
                                  size_t workspace_bytes, void *stream);
/* Benchmark aid: when enabled, every alg_ffn_forward on this handle records CUDA events on the
 * call's stream between its kernels (do not enable while capturing a graph).
 * alg_ffn_get_timing waits for the most recent call and returns four durations in
 * milliseconds: [0] row-type bucketing, [1] row gather, [2] up projection (with activation),
 * [3] down projection. */
alg_status_t alg_ffn_set_timing(alg_ffn_t h, int enable);
alg_status_t alg_ffn_get_timing(alg_ffn_t h, float *ms);
alg_status_t alg_ffn_macs(alg_ffn_t h, const int64_t *rows_per_type, int64_t *macs);
alg_status_t alg_ffn_last_status(alg_ffn_t h, void *stream, alg_status_t *status);

const char *alg_status_string(alg_status_t s);
/* Number of kernels the library has launched in this process (all handles, all streams). */
int64_t alg_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* ALGPROJ_H_ */
