/*
 * cdq.h -- C ABI of the B200 (sm_100a) CDQuant hot path.
 *
 * Post-training weight quantization by greedy coordinate descent on the
 * layer-wise reconstruction loss ||X (W - W_hat)||_F^2 (paper, Section 3,
 * Eq. 1).  Every output column of W is an independent descent problem; all of
 * them share one Hessian H = X^T X.
 *
 * Notation (paper, Section 3 "Notation"):
 *   X      [n, d_in]      calibration inputs, row-major
 *   W      [d_in, d_out]  layer weights, row-major with leading dimension ldw
 *   H      [d_in, d_in]   X^T X, fp32, both triangles stored
 *   c      bits; levels are 0 .. 2^c - 1
 *   Q      [d_in, d_out]  codes, one byte each, row-major, dense
 *   a, b   scale and zero, [d_in/g, d_out] fp32 row-major (one row when
 *          per-channel); W_hat[i,j] = a[i/g,j] * Q[i,j] + b[i/g,j]
 *
 * General rules
 *   - Every data pointer is a DEVICE pointer owned by the caller unless the
 *     argument is marked "host".  The library allocates no device memory:
 *     scratch comes from the caller's workspace `ws` (size from
 *     cdq_workspace_bytes, 256-byte aligned).  A too-small workspace gives
 *     CDQ_ERR_WORKSPACE before anything is launched.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls only enqueue work, except where a host result is returned
 *     (cdq_cd_solve with stats != NULL, cdq_layer_loss with loss != NULL):
 *     those synchronise `stream` before returning.  cdq_init_rtn with a clipping
 *     search of four or more strengths in the production mode synchronises `stream`
 *     once in the middle (it reads back how many columns each strength is still a
 *     candidate for, see there).
 *   - Errors are returned as status codes; nothing aborts or throws.
 *     Arguments are validated before any launch.  A device-side wait that
 *     exceeds its bound is reported as CDQ_ERR_TIMEOUT by the next call that
 *     synchronises (cdq_last_device_status reads it explicitly).
 *   - Two arithmetic modes.  CDQ_MODE_FAST is the production path: fp32 H, tensor cores for
 *     the Hessian (bf16) and for the products H (W_hat - W) (exact int8 slices, summed in fp64),
 *     the gradient of the descent kept in fp64 and the candidate scores in fp32.  Grouped grids
 *     whose group size is not a multiple of 4, and layers longer than 18432 inputs, run their
 *     descent with the fp64 kernel of the other mode.  CDQ_MODE_FP64_VERIFY runs plain fp64
 *     kernels that follow a fixed summation order (ascending index, no fused multiply-add) so
 *     that codes can be compared bit for bit with a CPU implementation of the same steps; it is
 *     meant for small layers.
 *   - H must be finite; the descent multiplies rows of H by a zero step in its first sweep.
 *   - H must be 16-byte aligned wherever it is passed (it is read with 16-byte vector loads and
 *     bulk copies); a misaligned H is CDQ_ERR_INVALID_ARG before anything is launched.
 *   - Environment (read once per process, for debugging only): CDQ_DEBUG_SYNC=1 synchronises the
 *     device after every step of a call, so that an asynchronous kernel failure is attributed to
 *     the step that caused it; CDQ_BCD_G=global keeps the gradient of cdq_bcd_solve in global
 *     memory at every size (the path that only layers of more than ~25 K inputs take otherwise).
 */
#ifndef CDQ_H_
#define CDQ_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  CDQ_OK = 0,
  CDQ_ERR_INVALID_ARG = 1, /* null pointer, bad enum, bits outside 1..8, ...    */
  CDQ_ERR_SHAPE = 2,       /* non-positive size, d_in % group_size != 0, ld too small */
  CDQ_ERR_UNSUPPORTED = 3, /* valid request this build has no kernel for       */
  CDQ_ERR_WORKSPACE = 4,   /* ws NULL / misaligned / smaller than required      */
  CDQ_ERR_CUDA = 5,        /* a CUDA runtime call failed                        */
  CDQ_ERR_TIMEOUT = 6      /* a bounded device-side wait ran out                */
} cdq_status;

typedef enum { CDQ_F32 = 0, CDQ_BF16 = 1 } cdq_dtype;
typedef enum { CDQ_MODE_FAST = 0, CDQ_MODE_FP64_VERIFY = 1 } cdq_mode;

/* Which entry point a workspace size is asked for. */
typedef enum {
  CDQ_CALL_HESSIAN = 0,
  CDQ_CALL_INIT_RTN = 1,
  CDQ_CALL_CD_SOLVE = 2,
  CDQ_CALL_LAYER_LOSS = 3,
  CDQ_CALL_INIT_OWC_CD = 4,
  CDQ_CALL_BCD_SOLVE = 5,  /* n: steps per column */
  CDQ_CALL_CD_SOLVE_ROWS16 = 6
} cdq_call;

/* Quantization grid (paper: c in "Notation"; group size g in the sub-channel
 * section; clipping grid Gamma in the OWC paragraph after Eq. 2). */
typedef struct {
  int bits;       /* c, 1..8 */
  int group_size; /* g along d_in; 0 => per-channel (g = d_in); d_in % g == 0 */
  int n_clip;     /* |Gamma|; <= 1 => MinMax (gamma = 1) */
  float clip_lo;  /* Gamma = { lo + (hi-lo)*k/(n_clip-1), k = 0..n_clip-1 } */
  float clip_hi;
} cdq_grid_desc;

typedef struct {
  unsigned long long steps;             /* step budget: passes * d_in * d_out            */
  unsigned long long committed;         /* moves actually made                           */
  unsigned long long columns_converged; /* columns that ran out of improving moves       */
  double loss_before;                   /* sum_j e_j^T H e_j at entry (from G0)          */
  double loss_after;                    /* loss_before + sum of committed decreases (FAST:
                                           the fp32 scores of the moves, ~1e-7 relative)  */
  double kernel_ms;                     /* device time of the descent kernel alone (CUDA
                                           events on `stream`), for roofline accounting   */
} cdq_cd_stats;

/*
 * H = X^T X  (paper: Section 3 "Notation"; Algorithm 1), plus the
 * optional regulariser of Section 4: H_ii += lambda_rel * mean(diag H).
 *   X          [n, d_in] of type xt, leading dimension ldx (elements, >= d_in).
 *              BF16 input additionally needs X 16-byte aligned and ldx % 8 == 0.
 *   accumulate 0: H is overwritten.  1: H += X^T X (calibration rows arriving
 *              in chunks); lambda_rel must then be 0 except on the last chunk.
 *   H          [d_in, d_in] fp32 out (in/out when accumulating).
 * FAST: bf16 inputs run on the tensor cores (fp32 accumulation); fp32 inputs
 * use an fp64-accumulating SIMT kernel.  VERIFY: every entry is the ascending-k
 * fp64 sum, rounded once to fp32; accumulate is not supported there.
 */
cdq_status cdq_hessian(const void* X, cdq_dtype xt, long long n, long long d_in, long long ldx,
                       float lambda_rel, int accumulate, float* H, cdq_mode mode, void* ws,
                       size_t ws_bytes, void* stream);

/*
 * The regulariser alone: H_ii += lambda_rel * mean(diag H) (paper: Section 4, the lambda I added to
 * the Hessian as for GPTQ).  For a Hessian that is summed from several parts first (row
 * chunks, or the row shards of several GPUs after their all-reduce): the parts are formed with
 * lambda_rel = 0 and the sum is regularised once.
 *   H  [d_in, d_in] fp32 device, in/out, owned by the caller.  lambda_rel >= 0 (0: nothing is launched).
 * Errors: CDQ_ERR_INVALID_ARG (NULL H, negative or NaN lambda_rel), CDQ_ERR_SHAPE (d_in < 1),
 * CDQ_ERR_UNSUPPORTED (d_in > 65535), CDQ_ERR_CUDA.  No workspace; asynchronous on `stream`.
 */
cdq_status cdq_hessian_add_lambda(float* H, long long d_in, float lambda_rel, void* stream);

/*
 * Grid and round-to-nearest codes (paper: Eq. 2; gamma = 1 is MinMax), with
 * the Optimal Weight Clipping search when grid->n_clip > 1 (paper: the
 * minimisation over gamma stated after Eq. 2, solved by grid search).
 * Per column j and group t: b = min(w), a = gamma * (max(w) - min(w)) / (2^c - 1),
 * q = clamp(round_half_even((w - b) / a), 0, 2^c - 1); a constant group gets
 * a = 0 and all-zero codes.  With n_clip > 1, one gamma per output column is
 * applied to every group of the column and is the grid point with the
 * smallest column loss e^T H e (lowest index on ties).
 *   W          [d_in, d_out] of type wt, leading dimension ldw.
 *   H          [d_in, d_in] fp32; may be NULL iff n_clip <= 1.
 *   scale,zero [d_in/g, d_out] fp32 out.
 *   Q          [d_in, d_out] u8 out.
 *   gamma_out  [d_out] fp32 out, chosen clipping strength; may be NULL.
 * FAST, layers of at least 256 x 128: the column losses are products on the int8 tensor cores.  All
 * strengths are first screened with three slice-pair products (six on grids of more than 4 bits); a strength
 * within 1 % of a column's smallest screened loss stays a candidate and gets the thirteen-pair loss (~1e-8
 * relative); the argmin is taken over the candidates.  The candidate counts go through the host: one synchronisation of `stream`.
 * The rounding decision is taken in fp64 in both modes.
 */
cdq_status cdq_init_rtn(const void* W, cdq_dtype wt, long long d_in, long long d_out, long long ldw,
                        const float* H, const cdq_grid_desc* grid, float* scale, float* zero,
                        unsigned char* Q, float* gamma_out, cdq_mode mode, void* ws,
                        size_t ws_bytes, void* stream);

typedef struct {
  unsigned long long moves; /* changes of a group's clipping strength, over all columns */
  double loss_before;       /* sum_j e_j^T H e_j with every group at the last grid point  */
  double loss_after;        /* the same at the chosen strengths (start + changes made)    */
} cdq_owc_cd_stats;

/*
 * Grid and round-to-nearest codes with one clipping strength per GROUP, chosen by greedy
 * coordinate descent over the groups (paper: Algorithm 3, "Coordinate Descent for Optimal
 * Weight Clipping"; Eq. 2 per group).  Every group of a column starts at the last point of
 * the grid Gamma (its largest strength; MinMax when clip_hi = 1).  A step evaluates, for every
 * group t and grid point k, the change of the column loss
 *     delta^T H_tt delta + delta^T (2 H e)_t,   delta = residual(t, k) - residual(t, current),
 * makes the change that lowers the loss most (ties: lowest group, then lowest grid index), and
 * stops when no change lowers it or after `steps` changes (steps <= 0: d_in / g, the paper's
 * setting).  The sign of the linear term follows the algebra of the quadratic loss; the
 * algorithm box of the paper prints it with the opposite sign of its own definitions.
 *   grid       n_clip >= 2; group_size 0 means one group per column, which makes one step the
 *              plain OWC grid search.
 *   scale,zero [d_in/g, d_out] fp32 out.    Q [d_in, d_out] u8 out.
 *   gamma_out  [d_in/g, d_out] fp32 out, chosen strengths; may be NULL.
 *   stats      host pointer, may be NULL (then the call does not synchronise).
 * fp64 in both modes; VERIFY sums in ascending order without fused multiply-add
 * (bit-reproducible against a CPU statement of the steps), FAST tabulates H_tt r per grid point
 * once per column so that a step costs dot products of length g.
 */
cdq_status cdq_init_owc_cd(const void* W, cdq_dtype wt, long long d_in, long long d_out, long long ldw,
                           const float* H, const cdq_grid_desc* grid, long long steps, float* scale,
                           float* zero, unsigned char* Q, float* gamma_out, cdq_owc_cd_stats* stats,
                           cdq_mode mode, void* ws, size_t ws_bytes, void* stream);

/*
 * Greedy coordinate descent on every column (paper: Algorithm 1; Algorithm 4
 * for sub-channel grids), T = passes * d_in steps per column at most.
 * Weight-unit form of the iteration: G = 2 H (W_hat - W); a move of
 * coordinate i to level r changes the loss by d^2 H_ii + d G_i with
 * d = a_i (r - q_i); the move with the most negative change is made (ties:
 * lowest i, then lowest r); G += 2 d H[i,:].  A column stops early when no
 * move lowers its loss.
 *   Q      in: initial codes q0 (e.g. from cdq_init_rtn); out: result.
 *   stats  host pointer, may be NULL (then the call does not synchronise).
 * FAST: scoring in fp32 from an fp64 gradient; VERIFY: fp64 level scan in the
 * fixed order, bit-reproducible.
 */
cdq_status cdq_cd_solve(const float* H, const void* W, cdq_dtype wt, long long d_in, long long d_out,
                        long long ldw, const cdq_grid_desc* grid, const float* scale,
                        const float* zero, unsigned char* Q, int passes, cdq_mode mode,
                        cdq_cd_stats* stats, void* ws, size_t ws_bytes, void* stream);

/*
 * The same descent with the budget given in steps per column instead of passes: T = steps_per_col
 * (paper: the study of fewer iterations, T = d_in / 2, d_in / 4, d_in / 8, in the appendix on
 * speeding up CD; Algorithm 1 takes T as its input).  cdq_cd_solve(passes) is
 * cdq_cd_solve_steps(passes * d_in).
 */
cdq_status cdq_cd_solve_steps(const float* H, const void* W, cdq_dtype wt, long long d_in, long long d_out,
                              long long ldw, const cdq_grid_desc* grid, const float* scale,
                              const float* zero, unsigned char* Q, long long steps_per_col, cdq_mode mode,
                              cdq_cd_stats* stats, void* ws, size_t ws_bytes, void* stream);

/*
 * cdq_cd_solve_steps followed by the loss of its result (paper: Eq. 1 with H = X^T X, the quantity
 * Algorithm 1 descends on), sum_j e_j^T H e_j with e_j = W_hat[:, j] - W[:, j].  The descent keeps the
 * gradient g_j = 2 H e_j of every column up to date, so the loss of the result is 1/2 sum_i e_ij g_ij:
 * one dot product per column instead of the product H E.  FAST takes it that way on the shapes its
 * register-resident kernels cover and agrees with cdq_layer_loss to ~1e-12 relative; VERIFY, and the
 * remaining shapes, run cdq_layer_loss on the result.
 *   loss     host pointer, may be NULL; the call synchronises when it is given.
 *   per_col  [d_out] device doubles, may be NULL; not both NULL.
 * Workspace: cdq_workspace_bytes(CDQ_CALL_CD_SOLVE, ...).
 */
cdq_status cdq_cd_solve_with_loss(const float* H, const void* W, cdq_dtype wt, long long d_in, long long d_out,
                                  long long ldw, const cdq_grid_desc* grid, const float* scale,
                                  const float* zero, unsigned char* Q, long long steps_per_col, cdq_mode mode,
                                  cdq_cd_stats* stats, double* loss, double* per_col, void* ws, size_t ws_bytes,
                                  void* stream);

/*
 * Block coordinate descent with random blocks (paper: Algorithm 2; Algorithm 5 for sub-channel
 * grids), weight-unit form as above.  Step t cuts the d_in coordinates into d_in / block blocks
 * by a pseudo-random permutation pi (block u holds pi(block u), ..., pi(block u + block - 1)),
 * drawn once per step for all columns; every block b and every assignment r of levels to its coordinates is
 * scored, with d = a (r - q) on b,
 *     change = d^T H_bb d + d^T G_b,
 * the most negative change is applied (ties: the block whose lowest coordinate is lowest, then
 * the lowest levels in ascending order of the block's coordinates) and G += 2 sum_i d_i H[i,:].
 * A step whose partition holds no improving block changes nothing; the descent runs all
 * steps_per_col steps.
 *   block  1: the greedy descent of cdq_cd_solve_steps (seed unused); 2: pairs.  Other sizes
 *          return CDQ_ERR_UNSUPPORTED; d_in % block != 0 returns CDQ_ERR_SHAPE; pairs need
 *          d_in <= 32768.
 *   seed   pi is a counter-based bijection of {0..d_in-1}: with b = ceil(log2 d_in) bits, three
 *          rounds  x <- (x (2 K_r + 1) + (K_r >> 33)) mod 2^b;  x <- x xor (x >> max(1, b / 2)),
 *          repeated while x >= d_in, with K_r = splitmix64(splitmix64(seed) xor (4 t + r)).
 *          The same (seed, t) gives the same partition on every run and on every
 *          implementation of this definition.
 *   stats  as for cdq_cd_solve; columns_converged is 0 for block > 1 (no early stop).
 * Workspace: cdq_workspace_bytes(CDQ_CALL_BCD_SOLVE, steps_per_col, ...); with block == 2 the
 * production mode lists the pairs of all steps there (8 d_in bytes per step), so
 * steps_per_col <= 65535.
 * FAST: fp32 scoring from an fp64 gradient, one pass over the levels of the block's lower
 * coordinate with the other level in closed form; VERIFY: fp64 scan of all (L+1)^2 assignments
 * in the fixed order, bit-reproducible.
 */
cdq_status cdq_bcd_solve(const float* H, const void* W, cdq_dtype wt, long long d_in, long long d_out,
                         long long ldw, const cdq_grid_desc* grid, const float* scale,
                         const float* zero, unsigned char* Q, int block, long long steps_per_col,
                         unsigned long long seed, cdq_mode mode, cdq_cd_stats* stats, void* ws,
                         size_t ws_bytes, void* stream);

/*
 * The greedy descent with 2-byte rows (paper: the appendix on run time puts the cost of a step in the
 * gather of the Hessian row and its scatter into the gradient, and speeds the method up by taking fewer
 * steps; this variant halves the bytes of each step instead, at a stated cost in the loss).
 * The update g += 2 d H[i*, :] reads row i* from a bf16 copy of H that the call builds in its workspace
 * (round to nearest even); H_ii stays fp32 everywhere (the scores, and the moved coordinate's own entry of
 * the row).  The call is therefore exactly cdq_cd_solve_steps on the matrix H' with H'_ij = bf16(H_ij) for
 * i != j and H'_ii = H_ii: the starting gradient, the tracked loss in `stats` and the picks all refer to
 * H'.  What that costs on the true objective is for the caller to measure with cdq_layer_loss on H.
 *   Arguments as for cdq_cd_solve_steps; production arithmetic only.
 *   Workspace: cdq_workspace_bytes(CDQ_CALL_CD_SOLVE_ROWS16, ...) = that of cdq_cd_solve plus 6 d_in^2 bytes.
 *   CDQ_ERR_UNSUPPORTED unless d_in > 2048, d_in % 8 == 0 and the group size is a multiple of 4 (shorter rows
 *   are served from L2 and gain nothing from fewer bytes).
 */
cdq_status cdq_cd_solve_rows16(const float* H, const void* W, cdq_dtype wt, long long d_in, long long d_out,
                               long long ldw, const cdq_grid_desc* grid, const float* scale, const float* zero,
                               unsigned char* Q, long long steps_per_col, cdq_cd_stats* stats, void* ws,
                               size_t ws_bytes, void* stream);

/*
 * Layer loss sum_j e_j^T H e_j with e = W_hat - W (paper: Eq. 1 written with
 * H = X^T X; the objective value the paper reports for a solution).
 *   loss     host pointer to one double, may be NULL.
 *   per_col  [d_out] fp64 device out, may be NULL.
 */
cdq_status cdq_layer_loss(const float* H, const void* W, cdq_dtype wt, long long d_in, long long d_out,
                          long long ldw, const cdq_grid_desc* grid, const float* scale,
                          const float* zero, const unsigned char* Q, double* loss, double* per_col,
                          cdq_mode mode, void* ws, size_t ws_bytes, void* stream);

/*
 * The layer loss for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a deployment variant of cdq_layer_loss, same result.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a region whose memory
 * was handed out up front and is now frozen (a serving process after start-up, a plugin
 * inside another framework's memory pool that does not lend scratch), or a latency-critical
 * path where an allocation could block on the driver.  Such a caller cannot provide the
 * workspace that cdq_layer_loss asks for, so this entry point brings its own: a fixed array
 * of CDQ_STATIC_SCRATCH_BYTES that is part of the library image.  Every GPU on which the
 * library is used holds that much memory from the first use until the process exits.
 *
 *   Arguments as for cdq_layer_loss, FAST arithmetic, no workspace.  Inputs and outputs are
 *   still the caller's: H, W, scale, zero, Q and per_col are device pointers, loss is a host
 *   pointer (the call synchronises `stream` when loss != NULL).
 *   Limit: 8 * d_in * d_out bytes for the residual plus about 8 * d_out * (d_in / 128 + 2)
 *   must fit in the array (e.g. 2048 x 1024 or 1024 x 2048); a larger layer is rejected with
 *   CDQ_ERR_WORKSPACE before anything is launched, and cdq_last_error_detail() says how
 *   much was needed.
 *   The call itself allocates and frees nothing, on the host side of the runtime included
 *   (no cudaMalloc / cudaFree, no allocating library routine).
 *   First call on a device: it looks up the device address of the array (the device must be
 *   current).  Make that first call during set-up, before any stream capture is begun.
 *   All calls on one GPU share the one array, and it keeps the previous call's contents.
 *   Nothing in it has to start at zero -- each call overwrites every region before reading
 *   it -- but two calls that overlap on the GPU (different streams, or different host threads
 *   on different streams) race on it: serialise them.
 */
#define CDQ_STATIC_SCRATCH_BYTES (20u * 1024u * 1024u)
cdq_status cdq_layer_loss_static(const float* H, const void* W, cdq_dtype wt, long long d_in,
                                 long long d_out, long long ldw, const cdq_grid_desc* grid,
                                 const float* scale, const float* zero, const unsigned char* Q,
                                 double* loss, double* per_col, void* stream);

/* Bytes of workspace `which` needs for these sizes (n is used by the Hessian only). */
size_t cdq_workspace_bytes(cdq_call which, long long n, long long d_in, long long d_out,
                           const cdq_grid_desc* grid, cdq_mode mode);

/* Reads and clears the device-side status word (synchronises the device): CDQ_OK,
 * CDQ_ERR_TIMEOUT (a bounded wait on a copy barrier ran out) or CDQ_ERR_CUDA (a kernel stopped on
 * an internal consistency check; cdq_last_error_detail() names it). */
cdq_status cdq_last_device_status(void);

/* Kernels this library has launched in this process so far (all entry points, all streams).
 * Host-side count, no synchronisation.  (No counterpart in the paper: bookkeeping for benchmarks.) */
unsigned long long cdq_kernel_launches(void);

/*
 * Diagnostics for the failure path (no counterpart in the paper).  Neither faults nor hangs the GPU.
 * cdq_debug_expire_wait: launches one small CTA on `stream` that arms a copy barrier for bytes that
 *   nothing will ever send and waits on it with the library's bounded wait (limit_cycles clock
 *   cycles, 1 .. 2^31); the wait runs out, the kernel records that in the device status word
 *   and returns.  The next cdq_last_device_status() (or synchronising call) reports CDQ_ERR_TIMEOUT.
 * cdq_debug_set_device_status: writes `flag` (0 ok, 1 wait ran out, 2 consistency check) into the
 *   status word from the host, synchronously.
 * Errors: CDQ_ERR_INVALID_ARG (limit or flag out of range), CDQ_ERR_CUDA.
 */
cdq_status cdq_debug_expire_wait(long long limit_cycles, void* stream);
cdq_status cdq_debug_set_device_status(int flag);

/* Text of the most recent CDQ_ERR_CUDA in this process (CUDA error name, the failing step),
 * or of a size rejection by cdq_layer_loss_static; an empty string if there was none.  The pointer stays valid; the text is overwritten by
 * the next such error. */
const char* cdq_last_error_detail(void);

const char* cdq_status_string(cdq_status s);
int cdq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* CDQ_H_ */
