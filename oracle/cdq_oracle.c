/*
 * cdq_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, fp64 CPU statement of the CDQuant per-layer pipeline, written
 * from the paper so that the CUDA library can be checked against it.  Only the
 * tests, the smoke check and the benchmark's CPU-baseline leg may use it; the
 * CUDA library shares no code with it and never calls it.
 *
 * What it computes (paper, Section 3):
 *   - H = X^T X                                   (Notation; Algorithm 1)
 *   - MinMax / OWC grid and round-to-nearest codes (Eq. 2 and the grid search
 *     over the clipping strength gamma that follows it; per-group form of the
 *     "Initialization" paragraph of the sub-channel section)
 *   - gradient of the layer loss                   (Algorithm 1)
 *   - greedy coordinate descent                    (the loop of Algorithm 1;
 *     Algorithm 4 for sub-channel grids)
 *   - the layer loss  sum_j e_j^T H e_j            (Eq. 1 written with H)
 *   - OWC-CD: greedy descent over per-group clipping strengths (Algorithm 3;
 *     its readings are listed above cdqo_owc_cd)
 *   - BCD with random blocks (Algorithm 2 / Algorithm 5; readings above
 *     cdqo_bcd_solve, including the counter-based partition)
 *
 * Formulation.  Algorithm 1 works in code units (g = 2H(q - (w-b)/a), the
 * printed decrease (r-q_i)^2 H_ii + (r-q_i) g_i is the loss change divided by
 * a^2).  Algorithm 4 rescales X by the per-coordinate scales, which gives a
 * different matrix for every output column.  Both are the same iteration as
 * the weight-unit form used here,
 *        G = 2 H (w_hat - w),   d = a_i (r - q_i),
 *        Delta(i, r) = d^2 H_ii + d G_i      (the true change of the loss),
 *        G <- G + 2 d H[i*, :]
 * because g_tilde = D_a G and H_tilde_ii = a_i^2 H_ii.  cdqo_cd_code_units()
 * below is the literal code-unit iteration of Algorithm 1 / Algorithm 4 and
 * the tests check that both pick the same moves.
 *
 * Fixed readings where the paper is silent:
 *   - ties: lowest coordinate i, then lowest level r; a move is taken only if
 *     it strictly lowers the loss (the no-op r = q_i has Delta = 0), otherwise
 *     the column is finished;
 *   - rounding in Eq. 2 is round-half-to-even;
 *   - OWC keeps b = min(w) and shrinks only a (Eq. 2 taken literally); with
 *     groups, one gamma per output column is applied to every group of it and
 *     is chosen on the full column loss;
 *   - scale a and zero b are stored as fp32 (what a dequantiser would hold);
 *   - H handed from one stage to the next is fp32 (the library's H is fp32).
 *
 * Arithmetic: fp64 everywhere, sums in ascending index order, no fused
 * multiply-add (build with -ffp-contract=off) so that an fp64 device kernel
 * that follows the same order can match bit for bit.
 *
 * Pins (tests/test_oracle_*.py): brute force over all codes on tiny layers;
 * Delta against the loss recomputed from X; incremental G against a fresh
 * 2H(w_hat-w); monotone loss; closed-form coordinate optimum against the level
 * scan; diagonal H => no move; gamma = 1 => MinMax; code-unit Algorithm 4 ==
 * weight-unit picks; local optimality at convergence; d_in = 1.  OWC-CD:
 * tracked loss against the loss recomputed from X; one group == the OWC grid
 * search; brute force over all assignments of grid points to groups; first
 * change == best single-group change; convergence == no improving change.
 * BCD: the partition is a permutation that varies with step and seed
 * and reaches every pair; block size 1 == the greedy descent; one step == the
 * brute-force best block move with the loss from the definition; prefixes of
 * a run are monotone.
 * Parity unpinned: anything that depends on the paper's (unstated) lambda.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef long long i64;

int cdqo_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ------------------------------------------------------------------------ */
/* H = X^T X  (Notation paragraph of Section 3; Algorithm 1).                */
/* X: [n, d_in] row-major, already widened exactly to fp64.                  */
/* H64: [d_in, d_in] fp64 result; H32 (may be NULL): the same rounded to     */
/* fp32, which is what every later stage consumes.                           */
/* lambda_rel > 0 adds lambda_rel * mean(diag H) to the diagonal (the        */
/* "lambda I" regulariser of Section 4; the paper does not give its value).  */
/* ------------------------------------------------------------------------ */
int cdqo_hessian(const double* X, i64 n, i64 d_in, double lambda_rel,
                 double* H64, float* H32) {
  if (!X || !H64 || n < 0 || d_in <= 0) return 1;
#pragma omp parallel for schedule(dynamic, 1)
  for (i64 p = 0; p < d_in; ++p) {
    double* row = H64 + p * d_in;
    for (i64 r = 0; r < d_in; ++r) row[r] = 0.0;
    for (i64 k = 0; k < n; ++k) {
      const double xp = X[k * d_in + p];
      const double* xr = X + k * d_in;
      for (i64 r = 0; r < d_in; ++r) row[r] = row[r] + xp * xr[r];
    }
  }
  if (lambda_rel > 0.0) {
    double tr = 0.0;
    for (i64 p = 0; p < d_in; ++p) tr = tr + H64[p * d_in + p];
    const double add = lambda_rel * (tr / (double)d_in);
    for (i64 p = 0; p < d_in; ++p) H64[p * d_in + p] = H64[p * d_in + p] + add;
  }
  if (H32)
    for (i64 e = 0; e < d_in * d_in; ++e) H32[e] = (float)H64[e];
  return 0;
}

/* Selected entries of H = X^T X: out[s] = sum_k X[k,rows[s]] X[k,cols[s]].  */
int cdqo_hessian_entries(const double* X, i64 n, i64 d_in, const i64* rows,
                         const i64* cols, i64 n_entries, double* out) {
  if (!X || !rows || !cols || !out) return 1;
#pragma omp parallel for schedule(static)
  for (i64 s = 0; s < n_entries; ++s) {
    double acc = 0.0;
    for (i64 k = 0; k < n; ++k)
      acc = acc + X[k * d_in + rows[s]] * X[k * d_in + cols[s]];
    out[s] = acc;
  }
  return 0;
}

/* gamma_k of the clipping grid: lo + (hi-lo)*k/(n_clip-1); a one-point grid */
/* is MinMax (gamma = 1).                                                    */
double cdqo_gamma(int k, int n_clip, double lo, double hi) {
  if (n_clip <= 1) return 1.0;
  return lo + ((hi - lo) * (double)k) / (double)(n_clip - 1);
}

/* Eq. 2 for one group of one column: w[0..len) with stride 1.               */
static void grid_rtn_group(const double* w, i64 len, int L, double gamma,
                           float* a_out, float* b_out, uint8_t* q) {
  double mn = w[0], mx = w[0];
  for (i64 i = 1; i < len; ++i) {
    if (w[i] < mn) mn = w[i];
    if (w[i] > mx) mx = w[i];
  }
  const float b32 = (float)mn;
  const float a32 = (float)((gamma * (mx - mn)) / (double)L);
  *a_out = a32;
  *b_out = b32;
  if (!(a32 > 0.0f)) { /* constant group: every code 0, nothing to move */
    for (i64 i = 0; i < len; ++i) q[i] = 0;
    return;
  }
  const double a = (double)a32, b = (double)b32;
  for (i64 i = 0; i < len; ++i) {
    double r = rint((w[i] - b) / a); /* round half to even */
    if (r < 0.0) r = 0.0;
    if (r > (double)L) r = (double)L;
    q[i] = (uint8_t)r;
  }
}

/* e = (a*q + b) - w for one column. */
static void residual(const double* w, const uint8_t* q, const float* a,
                     const float* b, i64 d_in, i64 g, double* e) {
  for (i64 i = 0; i < d_in; ++i) {
    const double ai = (double)a[i / g], bi = (double)b[i / g];
    e[i] = (ai * (double)q[i] + bi) - w[i];
  }
}

/* e^T H e, sums ascending. he (scratch, d_in) receives H e. */
static double quad_form(const float* H, const double* e, i64 d_in, double* he) {
  double loss = 0.0;
  for (i64 p = 0; p < d_in; ++p) {
    const float* row = H + p * d_in;
    double acc = 0.0;
    for (i64 k = 0; k < d_in; ++k) acc = acc + (double)row[k] * e[k];
    he[p] = acc;
  }
  for (i64 p = 0; p < d_in; ++p) loss = loss + e[p] * he[p];
  return loss;
}

/* ------------------------------------------------------------------------ */
/* Grid + round-to-nearest, with the OWC grid search when n_clip > 1         */
/* (Eq. 2 and the minimisation over gamma stated right after it).            */
/* W: [d_in, d_out] row-major fp64 (widened).  group_size 0 => per-channel.  */
/* scale, zero: [d_in/g, d_out] fp32.  Q: [d_in, d_out] u8.                  */
/* gamma_idx (may be NULL): [d_out] chosen grid index.                       */
/* loss_table (may be NULL): [n_clip, d_out] loss of every gamma.            */
/* H (fp32, [d_in,d_in]) is needed only when n_clip > 1.                     */
/* ------------------------------------------------------------------------ */
int cdqo_init_rtn(const double* W, i64 d_in, i64 d_out, const float* H,
                  int bits, i64 group_size, int n_clip, double clip_lo,
                  double clip_hi, float* scale, float* zero, uint8_t* Q,
                  int* gamma_idx, double* loss_table) {
  if (!W || !scale || !zero || !Q || bits < 1 || bits > 8 || d_in <= 0 || d_out <= 0)
    return 1;
  const i64 g = group_size > 0 ? group_size : d_in;
  if (d_in % g) return 2;
  if (n_clip > 1 && !H) return 1;
  const i64 ng = d_in / g;
  const int L = (1 << bits) - 1;
  const int nk = n_clip > 1 ? n_clip : 1;
#pragma omp parallel
  {
    double* w = (double*)malloc(sizeof(double) * d_in);
    double* e = (double*)malloc(sizeof(double) * d_in);
    double* he = (double*)malloc(sizeof(double) * d_in);
    uint8_t* q = (uint8_t*)malloc(d_in);
    float* a = (float*)malloc(sizeof(float) * ng);
    float* b = (float*)malloc(sizeof(float) * ng);
#pragma omp for schedule(dynamic, 1)
    for (i64 j = 0; j < d_out; ++j) {
      for (i64 i = 0; i < d_in; ++i) w[i] = W[i * d_out + j];
      int best_k = 0;
      if (nk > 1) {
        double best = 0.0;
        for (int k = 0; k < nk; ++k) {
          const double gamma = cdqo_gamma(k, nk, clip_lo, clip_hi);
          for (i64 t = 0; t < ng; ++t)
            grid_rtn_group(w + t * g, g, L, gamma, a + t, b + t, q + t * g);
          residual(w, q, a, b, d_in, g, e);
          const double loss = quad_form(H, e, d_in, he);
          if (loss_table) loss_table[(i64)k * d_out + j] = loss;
          if (k == 0 || loss < best) { best = loss; best_k = k; }
        }
      }
      const double gamma = cdqo_gamma(best_k, nk, clip_lo, clip_hi);
      for (i64 t = 0; t < ng; ++t)
        grid_rtn_group(w + t * g, g, L, gamma, a + t, b + t, q + t * g);
      for (i64 t = 0; t < ng; ++t) {
        scale[t * d_out + j] = a[t];
        zero[t * d_out + j] = b[t];
      }
      for (i64 i = 0; i < d_in; ++i) Q[i * d_out + j] = q[i];
      if (gamma_idx) gamma_idx[j] = best_k;
    }
    free(w); free(e); free(he); free(q); free(a); free(b);
  }
  return 0;
}

/* ------------------------------------------------------------------------ */
/* Gradient G = 2 H (w_hat - w) for every column (Algorithm 1, in             */
/* weight units).  G: [d_out, d_in] fp64, one column of the layer per row.   */
/* ------------------------------------------------------------------------ */
int cdqo_gradient(const float* H, const double* W, i64 d_in, i64 d_out,
                  i64 group_size, const float* scale, const float* zero,
                  const uint8_t* Q, double* G) {
  if (!H || !W || !scale || !zero || !Q || !G) return 1;
  const i64 g = group_size > 0 ? group_size : d_in;
  if (d_in % g) return 2;
  const i64 ng = d_in / g;
#pragma omp parallel
  {
    double* w = (double*)malloc(sizeof(double) * d_in);
    double* e = (double*)malloc(sizeof(double) * d_in);
    uint8_t* q = (uint8_t*)malloc(d_in);
    float* a = (float*)malloc(sizeof(float) * ng);
    float* b = (float*)malloc(sizeof(float) * ng);
#pragma omp for schedule(dynamic, 1)
    for (i64 j = 0; j < d_out; ++j) {
      for (i64 i = 0; i < d_in; ++i) { w[i] = W[i * d_out + j]; q[i] = Q[i * d_out + j]; }
      for (i64 t = 0; t < ng; ++t) { a[t] = scale[t * d_out + j]; b[t] = zero[t * d_out + j]; }
      residual(w, q, a, b, d_in, g, e);
      for (i64 p = 0; p < d_in; ++p) {
        const float* row = H + p * d_in;
        double acc = 0.0;
        for (i64 k = 0; k < d_in; ++k) acc = acc + (double)row[k] * e[k];
        G[j * d_in + p] = 2.0 * acc;
      }
    }
    free(w); free(e); free(q); free(a); free(b);
  }
  return 0;
}

/* ------------------------------------------------------------------------ */
/* Greedy coordinate descent, weight-unit form (the loop of Algorithm 1; the */
/* sub-channel Algorithm 4 is the same iteration, see the header).           */
/* Q is updated in place.  T = passes * d_in steps per column at most.       */
/* stats_u64[3] = {steps budget (T*d_out), committed moves, columns that ran */
/* out of improving moves}; loss_ba[2] = {loss before, loss after}, both     */
/* recomputed from scratch as sum_j e_j^T H e_j.                             */
/* trace_* (may be NULL): for column trace_col, the move of every committed  */
/* step (capacity T): coordinate, new level, Delta.                          */
/* moves_per_col (may be NULL): [d_out] committed moves of each column.      */
/* G_final (may be NULL): [d_out, d_in] the incrementally kept gradient.     */
/* ------------------------------------------------------------------------ */
int cdqo_cd_solve(const float* H, const double* W, i64 d_in, i64 d_out, int bits,
                  i64 group_size, const float* scale, const float* zero,
                  uint8_t* Q, i64 steps_per_col, unsigned long long* stats_u64,
                  double* loss_ba, i64 trace_col, int* trace_i, int* trace_r,
                  double* trace_delta, i64* moves_per_col, double* G_final) {
  if (!H || !W || !scale || !zero || !Q || bits < 1 || bits > 8) return 1;
  const i64 g = group_size > 0 ? group_size : d_in;
  if (d_in % g) return 2;
  const i64 ng = d_in / g;
  const int L = (1 << bits) - 1;
  const i64 T = steps_per_col;
  unsigned long long committed = 0, converged = 0;
  double* lb = (double*)malloc(sizeof(double) * d_out);
  double* la = (double*)malloc(sizeof(double) * d_out);
#pragma omp parallel reduction(+ : committed, converged)
  {
    double* w = (double*)malloc(sizeof(double) * d_in);
    double* e = (double*)malloc(sizeof(double) * d_in);
    double* G = (double*)malloc(sizeof(double) * d_in);
    double* he = (double*)malloc(sizeof(double) * d_in);
    uint8_t* q = (uint8_t*)malloc(d_in);
    float* a = (float*)malloc(sizeof(float) * ng);
    float* b = (float*)malloc(sizeof(float) * ng);
#pragma omp for schedule(dynamic, 1)
    for (i64 j = 0; j < d_out; ++j) {
      for (i64 i = 0; i < d_in; ++i) { w[i] = W[i * d_out + j]; q[i] = Q[i * d_out + j]; }
      for (i64 t = 0; t < ng; ++t) { a[t] = scale[t * d_out + j]; b[t] = zero[t * d_out + j]; }
      residual(w, q, a, b, d_in, g, e);
      lb[j] = quad_form(H, e, d_in, he);
      for (i64 p = 0; p < d_in; ++p) G[p] = 2.0 * he[p];
      i64 moves = 0;
      int done = 0;
      for (i64 t = 0; t < T; ++t) {
        double best = 0.0; /* the no-op */
        i64 bi = -1;
        int br = 0;
        double bd = 0.0;
        for (i64 i = 0; i < d_in; ++i) {
          const double ai = (double)a[i / g];
          const double hii = (double)H[i * d_in + i];
          const int qi = (int)q[i];
          for (int r = 0; r <= L; ++r) {
            if (r == qi) continue;
            const double d = ai * (double)(r - qi);
            const double delta = (d * d) * hii + d * G[i];
            if (delta < best) { best = delta; bi = i; br = r; bd = d; }
          }
        }
        if (bi < 0) { done = 1; break; }
        if (j == trace_col && trace_i) {
          trace_i[moves] = (int)bi; trace_r[moves] = br; trace_delta[moves] = best;
        }
        q[bi] = (uint8_t)br;
        const float* row = H + bi * d_in; /* H symmetric: column i* = row i* */
        const double two_d = 2.0 * bd;
        for (i64 p = 0; p < d_in; ++p) G[p] = G[p] + two_d * (double)row[p];
        ++moves;
      }
      committed += (unsigned long long)moves;
      converged += (unsigned long long)done;
      if (moves_per_col) moves_per_col[j] = moves;
      if (G_final) for (i64 p = 0; p < d_in; ++p) G_final[j * d_in + p] = G[p];
      for (i64 i = 0; i < d_in; ++i) Q[i * d_out + j] = q[i];
      residual(w, q, a, b, d_in, g, e);
      la[j] = quad_form(H, e, d_in, he);
    }
    free(w); free(e); free(G); free(he); free(q); free(a); free(b);
  }
  double loss_before = 0.0, loss_after = 0.0;
  for (i64 j = 0; j < d_out; ++j) { /* ascending j */
    loss_before = loss_before + lb[j];
    loss_after = loss_after + la[j];
  }
  free(lb); free(la);
  if (stats_u64) {
    stats_u64[0] = (unsigned long long)T * (unsigned long long)d_out;
    stats_u64[1] = committed;
    stats_u64[2] = converged;
  }
  if (loss_ba) { loss_ba[0] = loss_before; loss_ba[1] = loss_after; }
  return 0;
}

/* ------------------------------------------------------------------------ */
/* The literal code-unit iteration for ONE column: Algorithm 4 (which is     */
/* Algorithm 1 when the scale is one constant): H_t = D_a H D_a,             */
/* g = 2 H_t (q0 - (w - b)/a), decrease (r-q_i)^2 H_t,ii + (r-q_i) g_i.      */
/* Records the committed moves; used only to check the weight-unit form.     */
/* a_full, b_full: per-coordinate scale and zero, all a_full > 0.            */
/* Returns the number of moves.                                              */
/* ------------------------------------------------------------------------ */
i64 cdqo_cd_code_units(const float* H, const double* w, const double* a_full,
                       const double* b_full, i64 d_in, int bits, uint8_t* q,
                       i64 T, int* trace_i, int* trace_r) {
  const int L = (1 << bits) - 1;
  double* Ht = (double*)malloc(sizeof(double) * d_in * d_in);
  double* gt = (double*)malloc(sizeof(double) * d_in);
  double* z = (double*)malloc(sizeof(double) * d_in);
  for (i64 p = 0; p < d_in; ++p)
    for (i64 k = 0; k < d_in; ++k)
      Ht[p * d_in + k] = a_full[p] * (double)H[p * d_in + k] * a_full[k];
  for (i64 i = 0; i < d_in; ++i) z[i] = (double)q[i] - (w[i] - b_full[i]) / a_full[i];
  for (i64 p = 0; p < d_in; ++p) {
    double acc = 0.0;
    for (i64 k = 0; k < d_in; ++k) acc = acc + Ht[p * d_in + k] * z[k];
    gt[p] = 2.0 * acc;
  }
  i64 moves = 0;
  for (i64 t = 0; t < T; ++t) {
    double best = 0.0;
    i64 bi = -1;
    int br = 0;
    for (i64 i = 0; i < d_in; ++i)
      for (int r = 0; r <= L; ++r) {
        const double dr = (double)(r - (int)q[i]);
        if (dr == 0.0) continue;
        const double delta = dr * dr * Ht[i * d_in + i] + dr * gt[i];
        if (delta < best) { best = delta; bi = i; br = r; }
      }
    if (bi < 0) break;
    const double dr = (double)(br - (int)q[bi]);
    for (i64 p = 0; p < d_in; ++p) gt[p] = gt[p] + 2.0 * dr * Ht[bi * d_in + p];
    q[bi] = (uint8_t)br;
    if (trace_i) { trace_i[moves] = (int)bi; trace_r[moves] = br; }
    ++moves;
  }
  free(Ht); free(gt); free(z);
  return moves;
}

/* ------------------------------------------------------------------------ */
/* Layer loss sum_j e_j^T H e_j (Eq. 1 expanded with H = X^T X).             */
/* per_col (may be NULL): [d_out].  Returns the total through *total.        */
/* ------------------------------------------------------------------------ */
int cdqo_layer_loss(const float* H, const double* W, i64 d_in, i64 d_out,
                    i64 group_size, const float* scale, const float* zero,
                    const uint8_t* Q, double* per_col, double* total) {
  if (!H || !W || !scale || !zero || !Q || !total) return 1;
  const i64 g = group_size > 0 ? group_size : d_in;
  if (d_in % g) return 2;
  const i64 ng = d_in / g;
  double* col_loss = (double*)malloc(sizeof(double) * d_out);
#pragma omp parallel
  {
    double* w = (double*)malloc(sizeof(double) * d_in);
    double* e = (double*)malloc(sizeof(double) * d_in);
    double* he = (double*)malloc(sizeof(double) * d_in);
    uint8_t* q = (uint8_t*)malloc(d_in);
    float* a = (float*)malloc(sizeof(float) * ng);
    float* b = (float*)malloc(sizeof(float) * ng);
#pragma omp for schedule(dynamic, 1)
    for (i64 j = 0; j < d_out; ++j) {
      for (i64 i = 0; i < d_in; ++i) { w[i] = W[i * d_out + j]; q[i] = Q[i * d_out + j]; }
      for (i64 t = 0; t < ng; ++t) { a[t] = scale[t * d_out + j]; b[t] = zero[t * d_out + j]; }
      residual(w, q, a, b, d_in, g, e);
      col_loss[j] = quad_form(H, e, d_in, he);
    }
    free(w); free(e); free(he); free(q); free(a); free(b);
  }
  double sum = 0.0;
  for (i64 j = 0; j < d_out; ++j) sum = sum + col_loss[j]; /* ascending j */
  if (per_col) memcpy(per_col, col_loss, sizeof(double) * d_out);
  *total = sum;
  free(col_loss);
  return 0;
}

/* ------------------------------------------------------------------------ */
/* OWC-CD: greedy coordinate descent over the clipping strengths of the      */
/* groups of a column (Algorithm 3, "Coordinate Descent for Optimal Weight   */
/* Clipping", sub-channel section).                                          */
/*                                                                           */
/* State per column: one grid index per group, and G = 2 H e with            */
/* e = w_hat - w (the vector the algorithm calls v; see the sign note).      */
/* Table: for every group t and grid point k the residual of that group      */
/* under Eq. 2 with gamma_k (the table that Algorithm 3 builds first).       */
/* Step: for every group t and every k other than its current index, with    */
/* delta = residual(t, k) - residual(t, current) (a vector over the group),  */
/*     change(t, k) = delta^T H_tt delta + delta^T G_t                       */
/* take the most negative one, then G <- G + 2 H[:, t] delta                 */
/* and set the group's index to k.                                           */
/*                                                                           */
/* Readings:                                                                 */
/*  - sign: the paper defines the table entry as w - w_hat and v as          */
/*    -2 H (w_hat - w) but adds v^T (Delta_old - Delta_new); with those      */
/*    signs the linear term would be minus the true one.  The change of the  */
/*    quadratic loss for e -> e + delta is delta^T H delta + 2 e^T H delta,  */
/*    which is what is computed here, and the algorithm's update of v is     */
/*    consistent with it;                                                    */
/*  - start (the algorithm does not say from where): every group starts at   */
/*    the last                                                               */
/*    grid point (the largest gamma; MinMax when clip_hi = 1);               */
/*  - ties: lowest group, then lowest grid index; a change is made only if   */
/*    it strictly lowers the loss, otherwise the column is finished;         */
/*  - T: `steps` per column (the paper's experiments use d_in / g).          */
/* Sums run in ascending index order, no fused multiply-add.                 */
/*                                                                           */
/* W: [d_in, d_out] fp64 (widened), H fp32.  Outputs: scale, zero            */
/* [d_in/g, d_out] fp32, Q [d_in, d_out] u8, gamma_idx [d_in/g, d_out],      */
/* moves / loss_before / loss_after [d_out] (each may be NULL).              */
/* ------------------------------------------------------------------------ */
int cdqo_owc_cd(const double* W, i64 d_in, i64 d_out, const float* H, int bits,
                i64 group_size, int n_clip, double clip_lo, double clip_hi,
                i64 steps, float* scale, float* zero, uint8_t* Q, int* gamma_idx,
                i64* moves, double* loss_before, double* loss_after) {
  if (!W || !H || !scale || !zero || !Q || bits < 1 || bits > 8 || d_in <= 0 || d_out <= 0 || n_clip < 1)
    return 1;
  const i64 g = group_size > 0 ? group_size : d_in;
  if (d_in % g) return 2;
  const i64 ng = d_in / g;
  const int L = (1 << bits) - 1;
  const int nk = n_clip;
#pragma omp parallel
  {
    double* w = (double*)malloc(sizeof(double) * d_in);
    double* tab = (double*)malloc(sizeof(double) * (size_t)nk * d_in); /* [k][i]: residual of coordinate i under gamma_k */
    double* G = (double*)malloc(sizeof(double) * d_in);
    double* e = (double*)malloc(sizeof(double) * d_in);
    double* he = (double*)malloc(sizeof(double) * d_in);
    double* delta = (double*)malloc(sizeof(double) * g);
    uint8_t* q = (uint8_t*)malloc(d_in);
    float* a = (float*)malloc(sizeof(float) * ng);
    float* b = (float*)malloc(sizeof(float) * ng);
    int* cur = (int*)malloc(sizeof(int) * ng);
#pragma omp for schedule(dynamic, 1)
    for (i64 j = 0; j < d_out; ++j) {
      for (i64 i = 0; i < d_in; ++i) w[i] = W[i * d_out + j];
      /* residual table */
      for (int k = 0; k < nk; ++k) {
        const double gamma = cdqo_gamma(k, nk, clip_lo, clip_hi);
        for (i64 t = 0; t < ng; ++t)
          grid_rtn_group(w + t * g, g, L, gamma, a + t, b + t, q + t * g);
        residual(w, q, a, b, d_in, g, tab + (size_t)k * d_in);
      }
      /* start and G = 2 H e */
      for (i64 t = 0; t < ng; ++t) cur[t] = nk - 1;
      for (i64 i = 0; i < d_in; ++i) e[i] = tab[(size_t)(nk - 1) * d_in + i];
      double loss = quad_form(H, e, d_in, he);
      for (i64 i = 0; i < d_in; ++i) G[i] = 2.0 * he[i];
      if (loss_before) loss_before[j] = loss;
      i64 nmoves = 0;
      for (i64 step = 0; step < steps; ++step) {
        double best = 0.0;
        i64 bt = -1;
        int bk = 0;
        for (i64 t = 0; t < ng; ++t) {
          const double* old = tab + (size_t)cur[t] * d_in + t * g;
          for (int k = 0; k < nk; ++k) {
            if (k == cur[t]) continue;
            const double* cand = tab + (size_t)k * d_in + t * g;
            for (i64 p = 0; p < g; ++p) delta[p] = cand[p] - old[p];
            double quad = 0.0, lin = 0.0;
            for (i64 p = 0; p < g; ++p) {
              const float* row = H + (t * g + p) * d_in + t * g;
              double acc = 0.0;
              for (i64 r = 0; r < g; ++r) acc = acc + (double)row[r] * delta[r];
              quad = quad + delta[p] * acc;
              lin = lin + delta[p] * G[t * g + p];
            }
            const double change = quad + lin;
            if (change < best) { best = change; bt = t; bk = k; }
          }
        }
        if (bt < 0) break;
        const double* old = tab + (size_t)cur[bt] * d_in + bt * g;
        const double* cand = tab + (size_t)bk * d_in + bt * g;
        for (i64 p = 0; p < g; ++p) delta[p] = cand[p] - old[p];
        for (i64 i = 0; i < d_in; ++i) {
          const float* row = H + i * d_in + bt * g;
          double acc = 0.0;
          for (i64 r = 0; r < g; ++r) acc = acc + (double)row[r] * delta[r];
          G[i] = G[i] + 2.0 * acc;
        }
        cur[bt] = bk;
        loss = loss + best;
        ++nmoves;
      }
      /* emit the grid and the codes of the chosen strengths */
      for (i64 t = 0; t < ng; ++t) {
        const double gamma = cdqo_gamma(cur[t], nk, clip_lo, clip_hi);
        grid_rtn_group(w + t * g, g, L, gamma, a + t, b + t, q + t * g);
        scale[t * d_out + j] = a[t];
        zero[t * d_out + j] = b[t];
        if (gamma_idx) gamma_idx[t * d_out + j] = cur[t];
      }
      for (i64 i = 0; i < d_in; ++i) Q[i * d_out + j] = q[i];
      if (moves) moves[j] = nmoves;
      if (loss_after) loss_after[j] = loss;
    }
    free(w); free(tab); free(G); free(e); free(he); free(delta); free(q); free(a); free(b); free(cur);
  }
  return 0;
}

/* ------------------------------------------------------------------------ */
/* BCD with random blocks (Algorithm 2; Algorithm 5 for sub-channel grids),  */
/* block size k, weight-unit form as for the greedy descent above.           */
/*                                                                           */
/* Step t: the coordinates are cut into d_in / k blocks by a pseudo-random   */
/* permutation pi (block u = {pi(k u), ..., pi(k u + k - 1)}), drawn once    */
/* per step for the whole layer (all columns see the same partition);        */
/* for every block and every assignment r of levels to its coordinates, with */
/* d_i = a_i (r_i - q_i),                                                    */
/*     change = sum_i d_i^2 H_ii + 2 sum_{i<m} d_i d_m H_im + sum_i d_i G_i  */
/* (the algorithm's (r-q)^T H_bb (r-q) + (r-q)^T g_b in weight units); the   */
/* most                                                                      */
/* negative change is applied: q_b <- r, G <- G + 2 sum_i d_i H[i, :].       */
/*                                                                           */
/* Readings:                                                                 */
/*  - the partition (the algorithm gives no rule for the random draw): pi is */
/*    a                                                                      */
/*    counter-based bijection of {0..d_in-1}, the same on every              */
/*    implementation: with b = bits of d_in - 1 and mask = 2^b - 1, three    */
/*    rounds  x <- (x * (2 K_r + 1) + (K_r >> 33)) & mask;  x <- x ^ (x >> s) */
/*    with                                                                   */
/*    s = max(1, b / 2) and K_r = splitmix64(seed, t, r) (each round is a    */
/*    bijection of b-bit words), repeated while x >= d_in (cycle walking).   */
/*    The column is not part of the key: the algorithm is stated for one     */
/*    vector and applied to a layer as a batch, one draw per step;           */
/*    splitmix64 is the published finaliser  z += 0x9E3779B97F4A7C15;        */
/*    z = (z ^ z >> 30) * 0xBF58476D1CE4E5B9; z = (z ^ z >> 27) *            */
/*    0x94D049BB133111EB; z ^ z >> 31  applied to                            */
/*    splitmix64(seed) ^ (4 t + r);                                          */
/*  - a step whose partition holds no improving block changes nothing and    */
/*    the next step draws the next partition (the loop does not stop);       */
/*  - ties: the block whose smallest coordinate is lowest, then the          */
/*    assignment that is lowest in the order of the block's coordinates      */
/*    sorted ascending; for k = 1 this is the rule of the greedy descent,    */
/*    which BCD then reproduces exactly.                                     */
/* ------------------------------------------------------------------------ */
static unsigned long long cdqo_splitmix64(unsigned long long z) {
  z += 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
/* keys of the three rounds for (seed, step) */
static void bcd_round_keys(unsigned long long seed, i64 t, unsigned long long key[3]) {
  const unsigned long long base = cdqo_splitmix64(seed);
  for (int r = 0; r < 3; ++r) key[r] = cdqo_splitmix64(base ^ (((unsigned long long)t << 2) | (unsigned long long)r));
}
/* pi(x) for the partition of step t; exported for the tests */
i64 cdqo_bcd_perm(i64 x, i64 d_in, unsigned long long seed, i64 t) {
  int b = 0;
  while (((i64)1 << b) < d_in) ++b;
  if (b == 0) return 0;
  const unsigned long long mask = (b >= 64) ? ~0ull : (((unsigned long long)1 << b) - 1);
  const int s = b / 2 > 1 ? b / 2 : 1;
  unsigned long long key[3];
  bcd_round_keys(seed, t, key);
  unsigned long long v = (unsigned long long)x;
  do {
    for (int r = 0; r < 3; ++r) {
      v = (v * (2ull * key[r] + 1ull) + (key[r] >> 33)) & mask;
      v ^= v >> s;
    }
  } while (v >= (unsigned long long)d_in);
  return (i64)v;
}

/* Q in/out.  k: block size (d_in % k == 0, k <= 4).  steps_per_col: T.      */
/* moves_per_col, loss_before, loss_after: [d_out] (may be NULL); the losses */
/* are recomputed from scratch as e^T H e.                                   */
int cdqo_bcd_solve(const float* H, const double* W, i64 d_in, i64 d_out, int bits, i64 group_size,
                   const float* scale, const float* zero, uint8_t* Q, int k, i64 steps_per_col,
                   unsigned long long seed, i64* moves_per_col, double* loss_before, double* loss_after) {
  if (!H || !W || !scale || !zero || !Q || bits < 1 || bits > 8 || k < 1 || k > 4) return 1;
  const i64 g = group_size > 0 ? group_size : d_in;
  if (d_in % g || d_in % k) return 2;
  const i64 ng = d_in / g, nb = d_in / k;
  const int L = (1 << bits) - 1;
  i64 ncomb = 1;
  for (int c = 0; c < k; ++c) ncomb *= (L + 1);
#pragma omp parallel
  {
    double* w = (double*)malloc(sizeof(double) * d_in);
    double* e = (double*)malloc(sizeof(double) * d_in);
    double* G = (double*)malloc(sizeof(double) * d_in);
    double* he = (double*)malloc(sizeof(double) * d_in);
    uint8_t* q = (uint8_t*)malloc(d_in);
    float* a = (float*)malloc(sizeof(float) * ng);
    float* b = (float*)malloc(sizeof(float) * ng);
#pragma omp for schedule(dynamic, 1)
    for (i64 j = 0; j < d_out; ++j) {
      for (i64 i = 0; i < d_in; ++i) { w[i] = W[i * d_out + j]; q[i] = Q[i * d_out + j]; }
      for (i64 t = 0; t < ng; ++t) { a[t] = scale[t * d_out + j]; b[t] = zero[t * d_out + j]; }
      residual(w, q, a, b, d_in, g, e);
      const double l0 = quad_form(H, e, d_in, he);
      if (loss_before) loss_before[j] = l0;
      for (i64 p = 0; p < d_in; ++p) G[p] = 2.0 * he[p];
      i64 moves = 0;
      for (i64 t = 0; t < steps_per_col; ++t) {
        double best = 0.0;
        i64 best_min = -1;
        i64 bm[4] = {0, 0, 0, 0};
        int br[4] = {0, 0, 0, 0};
        for (i64 u = 0; u < nb; ++u) {
          i64 m[4];
          for (int c = 0; c < k; ++c) m[c] = cdqo_bcd_perm(u * k + c, d_in, seed, t);
          for (int c = 1; c < k; ++c) /* ascending coordinates */
            for (int z = c; z > 0 && m[z] < m[z - 1]; --z) { const i64 tmp = m[z]; m[z] = m[z - 1]; m[z - 1] = tmp; }
          for (i64 comb = 0; comb < ncomb; ++comb) {
            int r[4];
            i64 rest = comb;
            for (int c = k - 1; c >= 0; --c) { r[c] = (int)(rest % (L + 1)); rest /= (L + 1); } /* first coordinate most significant */
            double d[4];
            int same = 1;
            for (int c = 0; c < k; ++c) {
              d[c] = (double)a[m[c] / g] * (double)(r[c] - (int)q[m[c]]);
              if (r[c] != (int)q[m[c]]) same = 0;
            }
            if (same) continue;
            double quad = 0.0, lin = 0.0;
            for (int c = 0; c < k; ++c) {
              for (int z = 0; z < k; ++z) quad = quad + (d[c] * d[z]) * (double)H[m[c] * d_in + m[z]];
              lin = lin + d[c] * G[m[c]];
            }
            const double change = quad + lin;
            if (change < best || (change == best && best_min >= 0 && m[0] < best_min && change < 0.0)) {
              best = change; best_min = m[0];
              for (int c = 0; c < k; ++c) { bm[c] = m[c]; br[c] = r[c]; }
            }
          }
        }
        if (best_min < 0) continue; /* this partition has no improving block */
        for (int c = 0; c < k; ++c) {
          const double dc = (double)a[bm[c] / g] * (double)(br[c] - (int)q[bm[c]]);
          q[bm[c]] = (uint8_t)br[c];
          if (dc == 0.0) continue;
          const float* row = H + bm[c] * d_in;
          const double two_d = 2.0 * dc;
          for (i64 p = 0; p < d_in; ++p) G[p] = G[p] + two_d * (double)row[p];
        }
        ++moves;
      }
      if (moves_per_col) moves_per_col[j] = moves;
      for (i64 i = 0; i < d_in; ++i) Q[i * d_out + j] = q[i];
      residual(w, q, a, b, d_in, g, e);
      if (loss_after) loss_after[j] = quad_form(H, e, d_in, he);
    }
    free(w); free(e); free(G); free(he); free(q); free(a); free(b);
  }
  return 0;
}
