// Shared declarations of the CUDA library behind include/cdq.h.
// Everything here is internal; the only exported symbols are the extern "C"
// entry points in api.cu.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/cdq.h"

namespace cdq {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }

// Device status word: kernels with bounded waits record a failure here.
enum DeviceFlag : int { kFlagOk = 0, kFlagWaitTimeout = 1, kFlagBadIndex = 2 };
int* device_status_word();  // device address of the status word (per process)

// Text returned by cdq_last_error_detail().
void set_error_detail(const char* text);

// Every kernel launch of the library goes through this count (cdq_kernel_launches()).
void count_launch();
// H is read with 16-byte vector loads and bulk copies by every consumer after cdq_hessian.
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Resolved problem description shared by the launchers.
struct Layer {
  const float* H;
  const void* W;
  cdq_dtype wt;
  long long d_in, d_out, ldw;
  int bits, L;
  long long g;   // group size actually used (d_in when per-channel)
  long long ng;  // d_in / g
  const float* scale;
  const float* zero;
};

// Load one weight as double (exact widening).
__device__ __forceinline__ double load_w(const void* W, cdq_dtype wt, long long idx) {
  if (wt == CDQ_BF16) return (double)__bfloat162float(((const __nv_bfloat16*)W)[idx]);
  return (double)((const float*)W)[idx];
}

// ---- launchers (one per .cu file) -----------------------------------------
// hessian_simt.cu
cudaError_t launch_hessian_verify(const void* X, cdq_dtype xt, long long n, long long d_in, long long ldx,
                                  double lambda_rel, float* H, double* H64, cudaStream_t st);
cudaError_t launch_hessian_simt(const void* X, cdq_dtype xt, long long n, long long d_in, long long ldx,
                                int accumulate, float* H, cudaStream_t st);
cudaError_t launch_hessian_lambda(float* H, long long d_in, double lambda_rel, double* scratch, cudaStream_t st);

// hessian_tc.cu (tcgen05 / TMEM / TMA path for bf16 inputs)
bool hessian_tc_supported(long long n, long long d_in, long long ldx, const void* X);
size_t hessian_tc_workspace(long long n, long long d_in);
cudaError_t launch_hessian_tc(const void* X, long long n, long long d_in, long long ldx, int accumulate,
                              float* H, void* ws, cudaStream_t st);

// init_rtn.cu
size_t init_rtn_workspace(long long d_in, long long d_out, long long g, int n_clip, cdq_mode mode);
cudaError_t launch_init_rtn(const Layer& ly, const cdq_grid_desc& grid, float* scale, float* zero,
                            unsigned char* Q, float* gamma_out, cdq_mode mode, void* ws, cudaStream_t st);

cudaError_t launch_group_minmax(const Layer& ly, float* pmn, float* pmx, float* mn, float* mx, cudaStream_t st);

// owc_cd.cu : greedy descent over per-group clipping strengths (paper: Algorithm 3)
size_t owc_cd_workspace(long long d_in, long long d_out, long long g, int n_clip, cdq_mode mode);
cudaError_t launch_owc_cd(const Layer& ly, const cdq_grid_desc& grid, long long steps, float* scale, float* zero,
                          unsigned char* Q, float* gamma_out, cdq_mode mode, void* ws, unsigned long long* host_moves,
                          double* host_before, double* host_after, cudaStream_t st);

// Residual E = W_hat - W in fp64, [d_in, d_out] row-major, either from stored codes or, for
// the OWC search, from per-group min/max and one clipping strength (codes formed on the fly).
struct ResidualSrc {
  const void* W; cdq_dtype wt; long long ldw;
  const float* scale; const float* zero; const unsigned char* Q;  // codes path
  const float* mn; const float* mx; double gamma; int L; int use_gamma;  // OWC path
  long long g, d_out;      // d_out: columns of the layer (the width of W's companions scale, zero, Q, mn, mx)
  const int* col_idx;      // NULL: E has a column for every layer column; else E column c is layer column col_idx[c] ...
  long long n_cols;        // ... and E is [d_in, n_cols]
  const int* col_gamma;    // OWC path, with col_idx: E column c takes the clipping strength gammas[col_gamma[c]] ...
  const double* gammas;    // ... instead of `gamma` (NULL: `gamma` for every column)
};
cudaError_t launch_residual_f64(const ResidualSrc& src, long long d_in, double* E, cudaStream_t st);

// gemm_f64.cu : C = H * E in fp64.
// G (may be NULL): [d_out, ldg] doubles, G[j][p] = 2 * C[p][j].
// col_loss (may be NULL): [d_out] doubles, e_j^T H e_j = sum_p E[p][j] C[p][j]; needs the
// scratch `part` of gemm_partials_elems(d_in, d_out) doubles.
size_t gemm_partials_elems(long long d_in, long long d_out);
cudaError_t launch_gemm_he(const float* H, long long d_in, long long d_out, const double* E,
                           double* G, long long ldg, double* col_loss, double* part, cudaStream_t st);
// fixed-order version (ascending k, no fused multiply-add)
// C: scratch of d_in * d_out doubles.
cudaError_t launch_gemm_he_verify(const float* H, long long d_in, long long d_out, const double* E, double* C,
                                  double* G, long long ldg, double* col_loss, cudaStream_t st);

// gemm_i8.cu : C[j, p] = scale * sum_k E[k, j] H[p, k] on the int8 tensor cores from 7-bit slices of
// both operands (nh slices of H, ne of E, slice pairs up to i + j = smax); C is [d_out, ldc].
// col_loss (may be NULL): [d_out], e_j^T H e_j.
bool gemm_tc_supported(long long d_in, long long d_out);
size_t gemm_tc_h_bytes(long long d_in, int nh);
size_t gemm_tc_e_bytes(long long d_in, long long d_out, int ne);
cudaError_t gemm_tc_prepare_h(const float* H, long long d_in, int nh, void* hbuf, cudaStream_t st);
cudaError_t gemm_tc_run(const void* hbuf, int nh, const double* E, long long d_in, long long d_out, int ne, int smax,
                        double scale, double* C, long long ldc, double* col_loss, void* ebuf, cudaStream_t st);
// Slice counts: the gradient and the loss of a descended solution need ~1e-9 of a_j H_pp (see
// gemm_i8.cu); the losses of the OWC search (round-to-nearest residuals) need ~1e-7 relative.
constexpr int kTcGradNH = 6, kTcGradNE = 5, kTcGradSmax = 9;
constexpr int kTcLossNH = 4, kTcLossNE = 4, kTcLossSmax = 6;

// cd_kernel.cu
struct CdCounters {            // lives in the workspace, zeroed by the launcher
  unsigned long long committed;
  unsigned long long converged;
  double delta_sum;
  int next_col;
  int pad;
};
cudaError_t launch_transpose_u8(const unsigned char* src, long long rows, long long cols, long long ld_src,
                                unsigned char* dst, long long ld_dst, cudaStream_t st);  // dst[c][r] = src[r][c]
long long cd_fast_pad(long long d_in);      // padded length of hdiag / hs
bool cd_fast_supported(long long d_in, long long g);
// hdiag = H_ii, hs = 0.5 / H_ii
cudaError_t launch_diag(const float* H, long long d_in, long long d_pad, float* hdiag, float* hs, cudaStream_t st);
// col_loss[j] = 1/2 sum_i E[i][j] G[j][i] (E [d_in, d_out], G [d_out, ldg]): e^T H e from the gradient g = 2 H e.
cudaError_t launch_loss_from_gradient(const double* E, const double* G, long long ldg, long long d_in, long long d_out,
                                      double* col_loss, cudaStream_t st);
// H16 (may be NULL): bf16 copy of H for the rows of the update; cudaErrorNotSupported if the shape has no such kernel
cudaError_t launch_cd_fast(const Layer& ly, const __nv_bfloat16* H16, double* G, long long ldg, unsigned char* Qt,
                           long long ldq, const float* hdiag, const float* hs, long long steps_per_col,
                           CdCounters* ctr, cudaStream_t st);
bool cd_rows16_supported(long long d_in, long long g);   // shapes whose descent can read bf16 rows
// H16 = bf16(H) and Hr = the fp32 matrix the bf16-row descent works on: off-diagonal entries rounded to bf16
// (round to nearest even), diagonal exact
cudaError_t launch_round_rows_bf16(const float* H, long long d_in, __nv_bfloat16* H16, float* Hr, cudaStream_t st);
cudaError_t launch_cd_verify(const Layer& ly, double* G, long long ldg, unsigned char* Qt, long long ldq,
                             long long steps_per_col, CdCounters* ctr, cudaStream_t st);
// bcd_kernel.cu: random blocks of two coordinates (Algorithm 2 / 5)
bool bcd_supported(long long d_in, int block);
cudaError_t launch_bcd(const Layer& ly, double* G, long long ldg, unsigned char* Qt, long long ldq, const float* hdiag,
                       const float* hs, long long steps_per_col, unsigned long long seed, bool fast, void* table,
                       CdCounters* ctr, cudaStream_t st);
size_t bcd_table_bytes(long long d_in, long long steps_per_col);  // the production kernel's list of pairs
cudaError_t launch_sum_f64(const double* v, long long n, double* out, cudaStream_t st);  // ascending order
cudaError_t launch_sum_f64_tree(const double* v, long long n, double* out, cudaStream_t st);  // fixed tree order

}  // namespace cdq
