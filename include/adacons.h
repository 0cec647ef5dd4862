/*
 * adacons.h -- C ABI of the AdaCons gradient-aggregation library for NVIDIA B200 (sm_100a).
 *
 * AdaCons (arXiv 2411.03742, Section 3) aggregates the gradients g_1..g_N of N data-parallel
 * workers into one direction psi_t = sum_i gamma_i g_i (Eq. 4, Eq. 12).  The weights come from
 * a first-order step on the subspace spanned by the gradients (Eq. 5-7), smoothed over time by
 * a momentum on the *sorted* coefficients (Eq. 11) and rescaled to sum to one (Eq. 12-13).
 *
 * One call of adacons_aggregate runs, entirely on the device and asynchronously on the
 * caller's stream:
 *   pass 1   one streaming read of the N x d matrix: column sums, p_i = <g_i, gbar>,
 *            q_i = ||g_i||^2                                              (Eq. 7)
 *   finish   fixed-order reduction of the per-block partial sums, a_i = p_i/sqrt(q_i),
 *            sorted momentum, gamma_i                                     (Eq. 11, Eq. 12-13;
 *                                                                          Algorithm 1, steps 2-3)
 *   pass 2   a second streaming read: out_k = cast(sum_i gamma_i g_ik)   (Eq. 12; Algorithm 1, step 4)
 *
 * Conventions
 *   - All functions return an adacons_error code (0 = success); none throws or aborts.
 *   - "device pointer" = memory of the CUDA device that was current when the context was
 *     created; "host pointer" = ordinary host memory.  `cuda_stream` is a cudaStream_t passed
 *     as void* (NULL = the legacy default stream).
 *   - Results are deterministic: the same inputs, state and options give the same bytes on the
 *     same GPU model (no floating-point atomics, fixed reduction order).
 *   - A context is not thread-safe; distinct contexts are independent.
 *   - Numerical degeneracies (a zero gradient, a vanishing or negative normaliser, Inf/NaN in
 *     the input) are not errors: the call completes with the documented fallback and raises a
 *     flag that adacons_get_status returns.
 *   - Magnitudes.  Products g*g and g*s (s = the column sum) are accumulated in fp32, block
 *     totals in fp64.  The result is scale-equivariant (exactly so for powers of two) while
 *     those products stay normal fp32 numbers and a block's share of a row's sum does not
 *     overflow: roughly 1e-15 <= |g| <= 1e15 for every element that matters to a norm.
 *     Smaller elements lose relative accuracy in q_i (a row made only of such elements is
 *     reported as a zero row); larger ones overflow to Inf and raise ADACONS_FLAG_NONFINITE.
 */
#ifndef ADACONS_H_
#define ADACONS_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct adacons_ctx adacons_ctx; /* opaque, owned by the library */

/* Storage type of BOTH the gradient matrix and the result.  Accumulation is always fp32 inside
 * a thread block and fp64 across blocks and in the coefficient step. */
enum adacons_dtype { ADACONS_F32 = 0, ADACONS_BF16 = 1 };

enum adacons_error {
  ADACONS_OK = 0,
  ADACONS_EINVAL = 1, /* bad argument (NULL, N < 1, d < 1, unknown enum, bad offsets, overlap) */
  ADACONS_EALIGN = 2, /* per-segment mode only: it needs 16-byte aligned buffers and row pitch
                         and N <= 64 (model-wise mode serves anything through a slower path)   */
  ADACONS_ENOMEM = 3, /* device or host allocation failed                                       */
  ADACONS_ECUDA = 4,  /* a CUDA runtime/driver call failed, or no CUDA device                   */
  ADACONS_EARCH = 5,  /* the current device is not compute capability 10.x                      */
  ADACONS_ETIMEOUT = 6, /* reserved; an expired on-device wait is reported through the flag
                           ADACONS_FLAG_TIMEOUT of adacons_get_status, not as a return code    */
  ADACONS_ELIMIT = 7   /* problem larger than the fixed scratch of adacons_stats_noalloc         */
};

/* Flags returned by adacons_get_status (OR over all segments since the last reset). */
enum adacons_flag {
  ADACONS_FLAG_ZERO_ROW = 1u,     /* some ||g_i|| = 0: that worker got weight 0.  (A segment with
                                     no columns at all is not data and raises neither this flag
                                     nor the next; its weights read 1/N.)                        */
  ADACONS_FLAG_DEGENERATE_Z = 2u, /* sum_i u_i = 0 (|Z| <= 1e-12 sum|u_i|) or not finite:
                                     gamma_i = 1/N (plain mean) was used                         */
  ADACONS_FLAG_NONFINITE = 4u,    /* Inf/NaN statistic: gamma_i = 1/N, momentum state unchanged  */
  ADACONS_FLAG_NEG_Z = 8u,        /* sum_i u_i < 0: computed as defined                          */
  ADACONS_FLAG_TIMEOUT = 0x100u   /* a bounded wait inside a kernel expired; the result of that
                                     call is invalid.  Call adacons_reset before the next
                                     aggregation: it also re-arms the single-pass kernel's grid
                                     barrier, which a call that gave up leaves out of step.       */
};

/* Options (adacons_set_option / adacons_get_option).  Variants follow the ablation in Table 2. */
enum adacons_option {
  ADACONS_OPT_BETA = 0,        /* momentum factor of Eq. 11, in [0,1); default 0.99 (Table 2)    */
  ADACONS_OPT_MOMENTUM = 1,    /* 1 (default): apply Eq. 11; 0: a~ = a, state untouched          */
  ADACONS_OPT_SORTED = 2,      /* 1 (default): sorted momentum, Eq. 11; 0: index EMA, Eq. 10     */
  ADACONS_OPT_NORMALIZE = 3,   /* 1 (default): weights sum to one, Eq. 12-13;
                                  0: lambda = 1 and the 1/N of Eq. 8, gamma_i = u_i / N          */
  ADACONS_OPT_PER_SEGMENT = 4, /* 0 (default): one set of coefficients for the whole vector
                                  ("model-wise"); 1: an independent set, with its own momentum
                                  state, for each segment given to adacons_create ("layer-wise",
                                  Section 4).  Changing it synchronises the device, allocates
                                  the per-segment plan and state, and resets the state.
                                  Errors: EALIGN (see above), ENOMEM.                            */
  ADACONS_OPT_PROFILE = 5,     /* 0 (default) / 1: record CUDA events around each of the three
                                  kernels of every aggregate call (see adacons_get_profile).
                                  Setting it (to either value) clears the recorded samples.      */
  ADACONS_OPT_OVERLAP_LAUNCH = 6, /* 1 (default): the one-block coefficient kernel is launched with
                                  programmatic stream serialisation, so its launch latency hides
                                  behind pass 1 (it waits for pass 1 on the device); 0: plain
                                  stream order.  Pass 2 is always launched in plain stream order
                                  (letting its blocks become resident early measured slower).
                                  No effect on results.                                          */
  ADACONS_OPT_FUSED_SMALL = 7, /* 1 (default): when the whole matrix fits in the shared memory of
                                  the grid (about 148 x 160 KB) and the buffers are 16-byte
                                  aligned, one cooperative kernel reads it from HBM once and does
                                  all three steps; 0: always the three-kernel path.              */
  ADACONS_OPT_ROW_PITCH = 8,   /* elements between the starts of two consecutive rows of the
                                  gradient matrix, >= d; default d (contiguous rows).  Applies to
                                  adacons_aggregate and adacons_aggregate_host.  A gradient length
                                  that is not a multiple of 16 bytes runs on the fast path when the
                                  rows are padded to a pitch that is; the padding is never read
                                  as data and nothing is written past out[d-1], but the vector
                                  loads may touch it: with a pitch > d the whole N * pitch
                                  elements must be readable (and out must not overlap them).
                                  The same serves a column range of a wider matrix (base pointer
                                  at the range's first column, pitch = the matrix's): the
                                  kernels then read at most 31 bytes past the range in every
                                  row, other columns of the matrix except after the last row
                                  of a range that ends the matrix, where those bytes must be
                                  readable too.
                                  Setting it synchronises the device and may re-allocate scratch. */
  ADACONS_OPT_ONE_LAUNCH = 9,  /* 1 (default): a matrix of up to 1 GiB that does not fit in shared
                                  memory, on 16-byte aligned buffers and pitch with N <= 64, is
                                  aggregated by ONE cooperative kernel (pass 1, the coefficient
                                  step of Algorithm 1 steps 2-3 by the block that finishes pass 1
                                  last, pass 2) instead of three launches: two reads of the
                                  matrix as before, no kernel boundaries.  2: whenever the
                                  buffers allow it, whatever the size.  0: never.  Same
                                  coefficients, state and output bytes as the three-kernel path
                                  (the block partials are added in the same fixed order).         */
  ADACONS_OPT_ALIGNED_BODY = 12, /* 1 (default): when the row pitch is a multiple of 16 bytes but the
                                  matrix starts off a 16-byte boundary (a slice of a larger
                                  buffer), every row is misaligned by the same amount; with
                                  N <= 64 pass 1 then runs its TMA-staged kernel on the aligned
                                  body (from each row's first 16-byte boundary on) and a one-block
                                  kernel adds the up to 7 columns before it, and if `out` is off
                                  by the same amount pass 2 does likewise (whole 16-byte groups
                                  vectorised, head and ragged tail element by element).  0: such
                                  buffers take the generic path, as a pitch that is not a
                                  multiple of 16 bytes always does.  Same results either way to
                                  fp32 accumulation order.                                       */
  ADACONS_OPT_SHIFTED_LOADS = 14, /* 1 (default): a matrix whose rows start at arbitrary element
                                  offsets (a row pitch that is not a multiple of 16 bytes, e.g.
                                  contiguous rows of an odd length) or a result buffer off the
                                  rows' alignment is still moved 16 bytes at a time (pass 1,
                                  N <= 64: the staged kernel with one tensor map per class of
                                  rows that share an offset, taken for bf16 always and for fp32
                                  when a class has 4 rows or more; pass 2: 16-byte loads), each
                                  row's bytes shifted into place in registers; the first and
                                  last 16 to 31 bytes of the vector are done element by element.  0: such buffers take the scalar
                                  kernels.  Same results to fp32 accumulation order (pass 2
                                  given the same weights: the same bytes).                      */
  ADACONS_OPT_GRAM_PASS1 = 13,  /* bf16, N <= 64, aligned buffers, d <= 2^30.  n >= 1: pass 1 takes
                                  the statistics from the Gram matrix of every column tile,
                                  computed on the tensor cores (Eq. 7, third line: N p_i is the
                                  i-th row sum of G G^T, q_i its diagonal), with n tiles of 256
                                  columns per first-level accumulation (integer, 1..32).  The
                                  tensor cores round their running sums toward zero: a sum of
                                  squares comes out low by about 4e-8 relative per chained
                                  product (four per tile), hence the bound on n (n = 16: q_i
                                  low by 2e-6 to 3e-6).  0 (default):
                                  column sums and dot products on the fp32 pipes, which is both
                                  more accurate and, as measured, faster; the option exists
                                  for comparison.                                                */
  ADACONS_OPT_TALL_TILES = 11, /* 1 (default): with 64 < N <= 256 on aligned buffers pass 1 reads the
                                  matrix ONCE, as for N <= 64, from taller and narrower tiles:
                                  128 rows x 256 bytes (half a warp per row) up to N = 128,
                                  256 rows x 256 bytes on 512 threads beyond.  2: beyond N = 128
                                  tiles of 256 rows x 128 bytes on 256 threads (a quarter-warp
                                  per row) instead; slower, because box rows of 128 bytes hold
                                  the copy engine below the memory's rate, kept for comparison.
                                  0: the two-read form (column sums first, then dot products per
                                  64 rows), which N > 256 always takes unless
                                  ADACONS_OPT_CLUSTER_PASS1 says otherwise.  The forms agree to
                                  fp32 rounding of the column sums.  Errors: EINVAL (other
                                  values), ENOMEM (the other tile shape needs more partial
                                  records than the context holds; the setting is left as it was). */
  ADACONS_OPT_CLUSTER_PASS1 = 10 /* 0 (default) / 1: with 64 < N <= 512 on aligned buffers pass 1
                                  reads the matrix ONCE through thread-block clusters of 2, 4 or 8
                                  blocks that share each column tile (64 rows per block) and
                                  exchange partial column sums through distributed shared memory,
                                  one cluster barrier per tile.  Takes precedence over
                                  ADACONS_OPT_TALL_TILES.  Off by default: the barrier per tile
                                  makes it slower than the alternatives (tall tiles up to
                                  N = 256, the two-read form beyond).  The forms agree to
                                  fp32 rounding of the column sums.                              */
};

/* Which N-vector adacons_get_coeffs returns (values of the most recent aggregate call). */
enum adacons_coeff {
  ADACONS_COEFF_A = 0,       /* a_i  = <g_i,gbar>/||g_i||            (Eq. 7)                      */
  ADACONS_COEFF_A_TILDE = 1, /* a~_i after the momentum of Eq. 11                                */
  ADACONS_COEFF_GAMMA = 2,   /* gamma_i, the weights applied in pass 2 (Eq. 12)                  */
  ADACONS_COEFF_P = 3,       /* p_i  = <g_i,gbar>                                                 */
  ADACONS_COEFF_Q = 4        /* q_i  = ||g_i||^2                                                  */
};

/* Read-only facts about a context (adacons_get_info). */
enum adacons_info {
  ADACONS_INFO_NUM_SEGMENTS = 0,     /* S given to create (1 if none)                            */
  ADACONS_INFO_COEFF_SETS = 1,       /* 1 in model-wise mode, S in layer-wise mode               */
  ADACONS_INFO_PASS1_BLOCKS = 2,     /* thread blocks of the pass-1 kernel (= partial-sum rows)  */
  ADACONS_INFO_SCRATCH_BYTES = 3,    /* device bytes owned by the context                        */
  ADACONS_INFO_LAUNCHES_PER_CALL = 4,/* kernels launched by the most recent adacons_aggregate    */
  ADACONS_INFO_LAST_PATH = 5,        /* 0 = none yet, 1 = TMA-staged fast path, 2 = generic path,
                                        3 = single-pass kernel (matrix held in shared memory),
                                        4 = N > 64: column sums, then dot products per 64 rows,
                                        5 = one launch, two reads (see ADACONS_OPT_ONE_LAUNCH),
                                        6 = N > 64: clusters, one read in pass 1
                                            (see ADACONS_OPT_CLUSTER_PASS1),
                                        7 = 64 < N <= 256: tiles of 128 or 256 rows, one read in pass 1
                                            (see ADACONS_OPT_TALL_TILES),
                                        8 = misaligned base, aligned body: TMA-staged pass 1 plus
                                            the head columns (see ADACONS_OPT_ALIGNED_BODY),
                                        9 = pass 1 from the Gram matrix on the tensor cores
                                            (see ADACONS_OPT_GRAM_PASS1),
                                        10 = rows at arbitrary element offsets: staged pass 1 with
                                            a tensor map per class of equally offset rows
                                            (see ADACONS_OPT_SHIFTED_LOADS)                       */
  ADACONS_INFO_TOTAL_LAUNCHES = 6,   /* kernels launched by this context so far                  */
  ADACONS_INFO_LAST_PASS2 = 7,       /* pass-2 kernel of the most recent aggregate call: 0 = none
                                        (no call yet, or the single-pass kernel), 1 = generic,
                                        2 = 16-byte vectors, 3 = 32-byte vectors (grads, out and
                                        the row pitch 32-byte aligned), 4 = the second phase of
                                        the one-launch kernel (TMA-staged chunks of 8 rows),
                                        5 = vector kernel on the aligned body plus element-wise
                                        edges (grads and out off a 16-byte boundary alike),
                                        6 = 16-byte loads shifted into place per row
                                        (see ADACONS_OPT_SHIFTED_LOADS)                          */
  ADACONS_INFO_STATS_DOUBLES = 8     /* doubles in one shard's statistics (adacons_pass1):
                                        sets * (2 N + 1)                                         */
};

/*
 * Create a context for N workers and gradients of d elements of type `dtype`
 * (problem statement: Eq. 4, psi_t : {g_i}_{i=1..N} -> R^d, stateful in t).
 *   out          receives the context (host pointer, must not be NULL).
 *   N            1 <= N <= 1024.
 *   d            1 <= d < 2^40 (per-segment mode and the N > 64 fast path: d <= 2^30).
 *   seg_offsets  host pointer to num_segments+1 ascending offsets with seg_offsets[0] = 0 and
 *                seg_offsets[num_segments] = d (segments may be empty and need no alignment);
 *                NULL / num_segments = 0 means one segment [0, d).  Copied; the caller keeps
 *                ownership.  The segments matter only with ADACONS_OPT_PER_SEGMENT = 1.
 * Allocates all device memory the context will ever need on the current device (state,
 * coefficients, per-block partial sums) and zeroes the momentum state (alpha^m_0 = 0, t = 0).
 * Errors: EINVAL, ENOMEM, ECUDA (no device / CUDA failure), EARCH (device is not sm_100).
 */
int adacons_create(adacons_ctx **out, int N, int64_t d, int dtype,
                   const int64_t *seg_offsets, int num_segments);

/*
 * Aggregate one set of gradients (Eq. 12; Algorithm 1 on a single device).
 *   grads  device pointer, read-only: N rows of d elements, row-major and contiguous
 *          (row i = g_i starts at element i*pitch; pitch = d unless ADACONS_OPT_ROW_PITCH is set).
 *   out    device pointer, d elements of the same type; must not overlap grads.
 *   Fast path: grads and out 16-byte aligned, the row pitch in bytes (d*sizeof(element) unless
 *   ADACONS_OPT_ROW_PITCH says otherwise) a multiple of 16; with all three multiples of 32 pass 2
 *   moves 32 bytes per instruction and is about 2 % faster still.  With N <= 64 the matrix is read
 *   twice, and so it is with 64 < N <= 256 (taller tiles, see ADACONS_OPT_TALL_TILES); with
 *   N > 256 three times (column sums first, then dot products per 64 rows; needs d floats of
 *   scratch, allocated in adacons_create; see ADACONS_OPT_CLUSTER_PASS1).  A matrix that merely starts off a 16-byte
 *   boundary keeps the fast pass 1 (ADACONS_OPT_ALIGNED_BODY); a pitch that is not a multiple of
 *   16 bytes (contiguous rows of an odd length) is still moved 16 bytes at a time, at about
 *   two thirds of the aligned speed (ADACONS_OPT_SHIFTED_LOADS); scalar kernels serve what is
 *   left (such a pitch with N > 64, vectors of a few elements) with the same results.
 * Enqueues its kernels on `cuda_stream` and returns; performs no host synchronisation and no
 * allocation.  Advances the momentum state by one step.  Owner of every buffer: the caller.
 * Errors: EINVAL (NULL pointers, overlap), ECUDA (launch failure), EALIGN (per-segment mode with
 * misaligned buffers), ENOMEM (an earlier adacons_set_option ran out of memory and left the
 * context without its buffers; destroy it).
 */
int adacons_aggregate(adacons_ctx *ctx, const void *grads, void *out, void *cuda_stream);

/*
 * The step in two halves, for a matrix whose COLUMNS are spread over several devices (device r
 * holds columns [c_r, c_{r+1}) of all N rows, one context per device created with the shard's own
 * d).  The statistics of Eq. 7 are sums over columns, so the shards' sums add up to the whole
 * matrix's: every device computes its own, the caller exchanges them (an all-gather of a few
 * KB; nothing else of the step crosses devices), and every device finishes with the same
 * coefficients, each on its own columns.  The paper spreads the WORKERS over devices instead and
 * needs two all-reduces of d elements (Algorithm 1, steps 1 and 4); this form is its single-
 * device arithmetic (Eq. 7, Eq. 11, Eq. 12-13) on another layout, not a step the paper prints.
 *
 * adacons_pass1: pass 1 on this shard.
 *   stats  device pointer, 8-byte aligned, receives ADACONS_INFO_STATS_DOUBLES doubles: per
 *          coefficient set the N sums sum_k g_ik s_k (N p_i of Eq. 7 before the division by N),
 *          the N squared norms q_i, and the set's number of columns on this shard.
 *   Changes neither the momentum state nor the step counter.
 * adacons_finish: coefficients from all shards' statistics, then pass 2 on this shard.
 *   stats  device pointer: `shards` records of ADACONS_INFO_STATS_DOUBLES doubles each, in the
 *          same shard order on every device; they are added in that order in fp64, so all
 *          devices get the same bits (coefficients, weights, state).
 *   grads, out  as for adacons_aggregate (the same matrix that adacons_pass1 was given).
 *   Advances the momentum state by one step.  With one shard, adacons_pass1 followed by
 *   adacons_finish gives the bits of adacons_aggregate's three-kernel path.
 * Per-segment mode: give every shard's context ALL the segments, clipped to the shard's column
 * range (segments that lie elsewhere become empty); the sets then line up across shards.  A set is
 * "without columns" (no flags, see adacons_flag) only if it is empty on every shard.
 * Both calls are asynchronous on `cuda_stream`, allocate nothing and never take the one-launch
 * or single-pass paths.  Errors: as adacons_aggregate; EINVAL also for a NULL or misaligned
 * `stats` and shards < 1.
 */
int adacons_pass1(adacons_ctx *ctx, const void *grads, double *stats, void *cuda_stream);
int adacons_finish(adacons_ctx *ctx, const void *grads, void *out, const double *stats, int shards,
                   void *cuda_stream);

/*
 * The same aggregation for callers whose gradients live in HOST memory.
 *   host_grads  host pointer, N x d row-major (pinned memory gives asynchronous copies).
 *   host_out    host pointer, d elements.
 * Copies the matrix to a device staging buffer owned by the context (allocated on first use,
 * N*d elements + d elements), runs adacons_aggregate on it and copies the result back, all on
 * `cuda_stream`; returns after synchronising that stream.  Errors: EINVAL, ENOMEM, ECUDA.
 */
int adacons_aggregate_host(adacons_ctx *ctx, const void *host_grads, void *host_out,
                           void *cuda_stream);

/* Forget the history of Eq. 11: the momentum state alpha^m := 0 (so that the next call is the
 * momentum-free rule of Eq. 7 and Eq. 12-13), t := 0, status flags cleared, the single-pass
 * kernel's grid barrier re-armed.  Asynchronous on the stream.  Errors: EINVAL, ENOMEM, ECUDA. */
int adacons_reset(adacons_ctx *ctx, void *cuda_stream);

/* Free the context and everything it owns.  The caller must make sure no work of this context
 * is still running.  NULL is accepted. */
int adacons_destroy(adacons_ctx *ctx);

/* Options; see enum adacons_option.  Takes effect from the next aggregate call.
 * Errors: EINVAL (unknown key, beta outside [0,1), per-segment requested without segments). */
int adacons_set_option(adacons_ctx *ctx, int key, double value);
int adacons_get_option(adacons_ctx *ctx, int key, double *value);

/*
 * Copy one coefficient vector of the most recent aggregate call to the host.
 *   host   receives sets*N doubles, set-major (sets = ADACONS_INFO_COEFF_SETS).
 * Synchronises `cuda_stream`.
 */
int adacons_get_coeffs(adacons_ctx *ctx, int which, double *host, void *cuda_stream);

/*
 * The normaliser Z = sum_i u_i of Eq. 13 (u_i = a~_i / ||g_i||) of the most recent aggregate call,
 * one double per coefficient set.  |Z| small against sum_i |u_i| means weights of both signs with
 * large magnitude (an ill-conditioned step).  NaN after a non-finite input.  Synchronises
 * `cuda_stream`.
 */
int adacons_get_normaliser(adacons_ctx *ctx, double *host_z, void *cuda_stream);

/*
 * Momentum state for checkpoint / resume (Eq. 11): host_m receives / provides sets*N doubles,
 * slot k of a set = EMA of the k-th smallest coefficient; *step = number of aggregations since
 * the last reset.  Either pointer of get may be NULL.  Both synchronise `cuda_stream`.
 */
int adacons_get_state(adacons_ctx *ctx, double *host_m, int64_t *step, void *cuda_stream);
int adacons_set_state(adacons_ctx *ctx, const double *host_m, int64_t step, void *cuda_stream);

/* OR of the adacons_flag bits raised since the last reset.  Synchronises `cuda_stream`. */
int adacons_get_status(adacons_ctx *ctx, uint32_t *flags, void *cuda_stream);

/*
 * Per-kernel device time, for roofline reporting.  With ADACONS_OPT_PROFILE = 1 every aggregate
 * call records four CUDA events on its stream (before pass 1, after pass 1, after the
 * coefficient step, after pass 2) into a ring of 64 slots.  This call synchronises
 * `cuda_stream` and returns the mean duration in milliseconds of {pass 1, coefficient step,
 * pass 2} over the recorded calls (at most the last 64) and their number.  No paper counterpart.
 * Errors: EINVAL (NULL, profiling off or nothing recorded), ECUDA.
 */
int adacons_get_profile(adacons_ctx *ctx, double ms[3], int64_t *calls, void *cuda_stream);

/*
 * Consensus statistics without any allocation.  (The paper has no counterpart: this entry point
 * exists for integration, not for the method.)
 *
 * Who needs it: a gradient hook that runs inside a training framework usually finds the device's
 * memory already handed to that framework's caching allocator, so a raw cudaMalloc -- which
 * adacons_create performs -- may fail there, and it synchronises the whole device in the middle
 * of the backward pass.  Such a caller, or one that only wants to log p_i and q_i, can call this
 * function instead: it creates no context and calls no cudaMalloc, cudaFree or other allocating
 * routine.  The per-block partial sums of pass 1 live in a fixed array inside the library's
 * device image (ADACONS_NOALLOC_SCRATCH_BYTES, held by every GPU that loads the library until the
 * process exits).
 *
 *   grads   device pointer, N x d row-major, as for adacons_aggregate (read-only).
 *   N, d    1 <= N <= ADACONS_NOALLOC_MAX_N, 1 <= d < 2^31; larger N returns ADACONS_ELIMIT.
 *   dtype   enum adacons_dtype.
 *   pq_out  device pointer to 2N doubles owned by the caller: p_0..p_{N-1} = <g_i, gbar>, then
 *           q_0..q_{N-1} = ||g_i||^2 (Eq. 7) -- the values adacons_get_coeffs returns as
 *           ADACONS_COEFF_P / ADACONS_COEFF_Q after adacons_aggregate on the same input.
 * Runs pass 1 and a small reduction kernel on `cuda_stream`; no host synchronisation.
 * The first call on each device also looks up the device address of the scratch array and the
 * driver's tensor-map encoder; make that first call before any stream capture begins.
 * All calls share the one scratch array, which keeps the previous call's contents: every word a
 * call reads it has written itself first (the status word is cleared on the stream), but two
 * calls that overlap on the GPU (different streams, or threads) race on it -- serialise them.
 * If a bounded wait inside pass 1 expires, pq_out is filled with NaN.
 * Errors: EINVAL (NULL, bad N/d/dtype), ELIMIT, EARCH, ECUDA.
 */
#define ADACONS_NOALLOC_MAX_N 64
#define ADACONS_NOALLOC_MAX_BLOCKS 1024
#define ADACONS_NOALLOC_SCRATCH_BYTES (ADACONS_NOALLOC_MAX_BLOCKS * 2 * ADACONS_NOALLOC_MAX_N * 4 + 256)
int adacons_stats_noalloc(const void *grads, int N, int64_t d, int dtype, double *pq_out,
                          void *cuda_stream);

/*
 * Self-test of the hang protection (no paper counterpart).  Every wait inside the library's
 * kernels -- on a TMA completion barrier, on the grid barrier of the single-pass kernel, on the
 * published weights in the one-launch kernel -- gives
 * up after 2 s, raises ADACONS_FLAG_TIMEOUT and lets the kernel return.  This call launches a tiny
 * kernel whose wait can never be satisfied (which = 0: an mbarrier nobody arrives on; which = 1: a
 * grid barrier that expects one more block than was launched; which = 2: the one-launch kernel's
 * wait for weights that nobody publishes) so that the give-up path can be
 * exercised without faulting or hanging the device: about 2 s later adacons_get_status reports
 * ADACONS_FLAG_TIMEOUT.  Call adacons_reset afterwards (it clears the flag and the barrier
 * counter that which = 1 leaves odd).  Errors: EINVAL, ECUDA.
 */
int adacons_selftest_bounded_wait(adacons_ctx *ctx, int which, void *cuda_stream);

/* Facts about the context; see enum adacons_info.  No device work. */
int adacons_get_info(adacons_ctx *ctx, int key, int64_t *value);

/* Static, human-readable text for an adacons_error code. */
const char *adacons_strerror(int code);

/* Library version as major*10000 + minor*100 + patch. */
int adacons_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ADACONS_H_ */
