// extern "C" entry points declared in include/cdq.h: argument validation, workspace
// carving and kernel sequencing.  No device memory is allocated here.
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <mutex>

#include "async_copy.cuh"
#include "common.cuh"

namespace cdq {

// One CTA: a copy barrier armed for bytes that never come, waited on with the bounded wait.
__global__ void expire_wait_kernel(long long limit_cycles, int* status) {
  __shared__ __align__(8) unsigned long long bar;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    mbar_fence_init();
    mbar_expect_tx(smem_u32(&bar), 16);
  }
  __syncthreads();
  if (!mbar_wait_cycles(smem_u32(&bar), 0, limit_cycles) && threadIdx.x == 0)
    atomicCAS(status, (int)kFlagOk, (int)kFlagWaitTimeout);
}

__device__ int g_device_status = 0;

int* device_status_word() {
  int* p = nullptr;
  if (cudaGetSymbolAddress((void**)&p, g_device_status) != cudaSuccess) return nullptr;
  return p;
}

static std::atomic<unsigned long long> g_launches{0};
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

static char g_error_detail[256] = "";
void set_error_detail(const char* text) { snprintf(g_error_detail, sizeof(g_error_detail), "%s", text); }

namespace {

bool valid_dtype(cdq_dtype t) { return t == CDQ_F32 || t == CDQ_BF16; }
bool valid_mode(cdq_mode m) { return m == CDQ_MODE_FAST || m == CDQ_MODE_FP64_VERIFY; }

cdq_status check_grid(const cdq_grid_desc* g, long long d_in) {
  if (!g) return CDQ_ERR_INVALID_ARG;
  if (g->bits < 1 || g->bits > 8) return CDQ_ERR_INVALID_ARG;
  if (g->group_size < 0) return CDQ_ERR_INVALID_ARG;
  if (g->n_clip > 256) return CDQ_ERR_INVALID_ARG;
  if (g->n_clip > 1 && !(g->clip_lo > 0.f && g->clip_hi >= g->clip_lo)) return CDQ_ERR_INVALID_ARG;
  if (g->group_size > 0 && d_in % g->group_size) return CDQ_ERR_SHAPE;
  return CDQ_OK;
}

cdq_status check_ws(const void* ws, size_t have, size_t need) {
  if (need == 0) return CDQ_OK;
  if (!ws || ((uintptr_t)ws % kAlign) || have < need) return CDQ_ERR_WORKSPACE;
  return CDQ_OK;
}

cdq_status check_layer_shape(long long d_in, long long d_out, long long ldw) {
  if (d_in < 1 || d_out < 1 || ldw < d_out) return CDQ_ERR_SHAPE;
  if (d_in > 65535) return CDQ_ERR_UNSUPPORTED;  // rows index a grid dimension
  if (d_out > 2147483647LL / 2) return CDQ_ERR_UNSUPPORTED;
  return CDQ_OK;
}

Layer make_layer(const float* H, const void* W, cdq_dtype wt, long long d_in, long long d_out, long long ldw,
                 const cdq_grid_desc* grid, const float* scale, const float* zero) {
  Layer ly{};
  ly.H = H; ly.W = W; ly.wt = wt; ly.d_in = d_in; ly.d_out = d_out; ly.ldw = ldw;
  ly.bits = grid->bits; ly.L = (1 << grid->bits) - 1;
  ly.g = grid->group_size > 0 ? grid->group_size : d_in;
  ly.ng = d_in / ly.g;
  ly.scale = scale; ly.zero = zero;
  return ly;
}

// Workspace of cdq_cd_solve / cdq_layer_loss.
struct SolveWs {
  size_t E, G, Qt, hdiag, half_inv, part, col_loss, scalars, hbuf, ebuf, bcd_tab, h16, hr, total;
  long long ldg, d_pad;
  bool tc;        // H E on the int8 tensor cores
  int nh, ne, smax;
};
SolveWs solve_ws_layout(long long d_in, long long d_out, cdq_mode mode, bool with_cd, long long bcd_steps = 0,
                        bool rows16 = false) {
  SolveWs w{};
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes); return o; };
  w.ldg = (d_in + 3) / 4 * 4;
  w.d_pad = cd_fast_pad(d_in);
  w.tc = mode == CDQ_MODE_FAST && gemm_tc_supported(d_in, d_out);
  // the loss of a descended solution is a sum with heavy cancellation (the descent tunes e against the
  // large entries of H): it takes the same slice depth as the gradient; the shallower setting serves
  // the OWC search, whose residuals are plain rounding errors
  w.nh = kTcGradNH; w.ne = kTcGradNE; w.smax = kTcGradSmax;
  w.E = take(sizeof(double) * d_in * d_out);
  if (with_cd || w.tc) w.G = take(sizeof(double) * d_out * w.ldg);
  if (w.tc) {
    w.hbuf = take(gemm_tc_h_bytes(d_in, w.nh));
    w.ebuf = take(gemm_tc_e_bytes(d_in, d_out, w.ne));
  }
  if (with_cd) {
    w.Qt = take((size_t)d_out * w.ldg);  // transposed codes, same leading dimension as G
    w.hdiag = take(sizeof(float) * w.d_pad);
    w.half_inv = take(sizeof(float) * w.d_pad);
  }
  w.part = take(sizeof(double) * (mode == CDQ_MODE_FAST ? gemm_partials_elems(d_in, d_out) : (size_t)d_in * d_out));
  w.col_loss = take(sizeof(double) * d_out);
  w.scalars = take(256);  // [0]: loss sum; [64..): CdCounters
  if (bcd_steps > 0 && mode == CDQ_MODE_FAST) w.bcd_tab = take(bcd_table_bytes(d_in, bcd_steps));
  if (rows16) {
    w.h16 = take(sizeof(__nv_bfloat16) * (size_t)d_in * d_in);
    w.hr = take(sizeof(float) * (size_t)d_in * d_in);
  }
  w.total = off;
  return w;
}

ResidualSrc codes_src(const Layer& ly, const unsigned char* Q) {
  ResidualSrc s{};
  s.W = ly.W; s.wt = ly.wt; s.ldw = ly.ldw; s.scale = ly.scale; s.zero = ly.zero; s.Q = Q;
  s.use_gamma = 0; s.L = ly.L; s.g = ly.g; s.d_out = ly.d_out;
  return s;
}

void note_cuda_error(cudaError_t e, const char* what, int line) {
  snprintf(g_error_detail, sizeof(g_error_detail), "%s (%s) at api.cu:%d: %s", cudaGetErrorName(e),
           cudaGetErrorString(e), line, what);
}

// CDQ_DEBUG_SYNC=1 in the environment synchronises the device after every step, so that an
// asynchronous kernel failure is attributed to the step that caused it.

bool debug_sync() {
  static int v = -1;
  if (v < 0) {
    const char* e = getenv("CDQ_DEBUG_SYNC");
    v = (e && e[0] == '1') ? 1 : 0;
  }
  return v == 1;
}

#define CDQ_CUDA(expr)                                  \
  do {                                                  \
    cudaError_t _e = (expr);                            \
    if (_e == cudaSuccess && debug_sync()) _e = cudaDeviceSynchronize(); \
    if (_e != cudaSuccess) {                            \
      note_cuda_error(_e, #expr, __LINE__);             \
      return CDQ_ERR_CUDA;                              \
    }                                                   \
  } while (0)

// Two events per device, made on first use and kept: cdq_cd_solve times its descent kernel with them.
cudaError_t timing_events(cudaEvent_t* ev0, cudaEvent_t* ev1) {
  constexpr int kMaxDevices = 64;
  static std::mutex mu;
  static cudaEvent_t evs[kMaxDevices][2] = {};
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(mu);
  for (int i = 0; i < 2; ++i)
    if (!evs[dev][i]) {
      e = cudaEventCreate(&evs[dev][i]);
      if (e != cudaSuccess) { evs[dev][i] = nullptr; return e; }
    }
  *ev0 = evs[dev][0]; *ev1 = evs[dev][1];
  return cudaSuccess;
}

cdq_status read_device_status_after_sync() {
  int flag = 0;
  if (cudaMemcpyFromSymbol(&flag, g_device_status, sizeof(int)) != cudaSuccess) return CDQ_ERR_CUDA;
  if (flag == kFlagOk) return CDQ_OK;
  int zero = 0;
  cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int));
  if (flag == kFlagBadIndex) {
    set_error_detail("the descent kernel produced an out-of-range coordinate and stopped");
    return CDQ_ERR_CUDA;
  }
  return CDQ_ERR_TIMEOUT;
}

}  // namespace
}  // namespace cdq

using namespace cdq;

extern "C" {

int cdq_version(void) { return 200; }

unsigned long long cdq_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

const char* cdq_status_string(cdq_status s) {
  switch (s) {
    case CDQ_OK: return "ok";
    case CDQ_ERR_INVALID_ARG: return "invalid argument";
    case CDQ_ERR_SHAPE: return "bad shape";
    case CDQ_ERR_UNSUPPORTED: return "unsupported";
    case CDQ_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case CDQ_ERR_CUDA: return "CUDA runtime error";
    case CDQ_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

const char* cdq_last_error_detail(void) { return g_error_detail; }

cdq_status cdq_last_device_status(void) {
  if (cudaDeviceSynchronize() != cudaSuccess) return CDQ_ERR_CUDA;
  return read_device_status_after_sync();
}

cdq_status cdq_debug_expire_wait(long long limit_cycles, void* stream) {
  if (limit_cycles < 1 || limit_cycles > (1ll << 31)) return CDQ_ERR_INVALID_ARG;
  int* status = device_status_word();
  if (!status) return CDQ_ERR_CUDA;
  { expire_wait_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(limit_cycles, status); count_launch(); }
  CDQ_CUDA(cudaGetLastError());
  return CDQ_OK;
}

cdq_status cdq_debug_set_device_status(int flag) {
  if (flag < (int)kFlagOk || flag > (int)kFlagBadIndex) return CDQ_ERR_INVALID_ARG;
  CDQ_CUDA(cudaDeviceSynchronize());
  CDQ_CUDA(cudaMemcpyToSymbol(g_device_status, &flag, sizeof(int)));
  return CDQ_OK;
}

size_t cdq_workspace_bytes(cdq_call which, long long n, long long d_in, long long d_out, const cdq_grid_desc* grid,
                           cdq_mode mode) {
  if (d_in < 1) return 0;
  switch (which) {
    case CDQ_CALL_HESSIAN:
      if (mode == CDQ_MODE_FP64_VERIFY) return align_up(sizeof(double) * d_in * d_in);
      return hessian_tc_workspace(n, d_in);
    case CDQ_CALL_INIT_RTN: {
      if (!grid || d_out < 1) return 0;
      const long long g = grid->group_size > 0 ? grid->group_size : d_in;
      if (g < 1 || d_in % g) return 0;
      return init_rtn_workspace(d_in, d_out, g, grid->n_clip, mode);
    }
    case CDQ_CALL_INIT_OWC_CD: {
      if (!grid || d_out < 1 || grid->n_clip < 2 || grid->n_clip > 256) return 0;
      const long long g = grid->group_size > 0 ? grid->group_size : d_in;
      if (g < 1 || d_in % g) return 0;
      return owc_cd_workspace(d_in, d_out, g, grid->n_clip, mode);
    }
    case CDQ_CALL_CD_SOLVE:
      if (d_out < 1) return 0;
      return solve_ws_layout(d_in, d_out, mode, true).total;
    case CDQ_CALL_BCD_SOLVE:  // n: steps per column
      if (d_out < 1 || n < 0) return 0;
      return solve_ws_layout(d_in, d_out, mode, true, n).total;
    case CDQ_CALL_LAYER_LOSS:
      if (d_out < 1) return 0;
      return solve_ws_layout(d_in, d_out, mode, false).total;
    case CDQ_CALL_CD_SOLVE_ROWS16:
      if (d_out < 1) return 0;
      return solve_ws_layout(d_in, d_out, mode, true, 0, true).total;
  }
  return 0;
}

cdq_status cdq_hessian(const void* X, cdq_dtype xt, long long n, long long d_in, long long ldx, float lambda_rel,
                       int accumulate, float* H, cdq_mode mode, void* ws, size_t ws_bytes, void* stream) {
  if (!X || !H || !valid_dtype(xt) || !valid_mode(mode) || !(lambda_rel >= 0.f)) return CDQ_ERR_INVALID_ARG;
  if (!aligned16(H)) return CDQ_ERR_INVALID_ARG;
  if (n < 1 || d_in < 1 || ldx < d_in) return CDQ_ERR_SHAPE;
  if (d_in > 65535) return CDQ_ERR_UNSUPPORTED;
  cudaStream_t st = (cudaStream_t)stream;
  if (mode == CDQ_MODE_FP64_VERIFY) {
    if (accumulate) return CDQ_ERR_UNSUPPORTED;
    cdq_status s = check_ws(ws, ws_bytes, align_up(sizeof(double) * d_in * d_in));
    if (s != CDQ_OK) return s;
    CDQ_CUDA(launch_hessian_verify(X, xt, n, d_in, ldx, (double)lambda_rel, H, (double*)ws, st));
    return CDQ_OK;
  }
  if (xt == CDQ_BF16 && hessian_tc_supported(n, d_in, ldx, X)) {
    cdq_status s = check_ws(ws, ws_bytes, hessian_tc_workspace(n, d_in));
    if (s != CDQ_OK) return s;
    CDQ_CUDA(launch_hessian_tc(X, n, d_in, ldx, accumulate, H, ws, st));
  } else {
    CDQ_CUDA(launch_hessian_simt(X, xt, n, d_in, ldx, accumulate, H, st));
  }
  if (lambda_rel > 0.f) CDQ_CUDA(launch_hessian_lambda(H, d_in, (double)lambda_rel, nullptr, st));
  return CDQ_OK;
}

cdq_status cdq_hessian_add_lambda(float* H, long long d_in, float lambda_rel, void* stream) {
  if (!H || !(lambda_rel >= 0.f)) return CDQ_ERR_INVALID_ARG;
  if (d_in < 1) return CDQ_ERR_SHAPE;
  if (d_in > 65535) return CDQ_ERR_UNSUPPORTED;
  if (lambda_rel > 0.f) CDQ_CUDA(launch_hessian_lambda(H, d_in, (double)lambda_rel, nullptr, (cudaStream_t)stream));
  return CDQ_OK;
}

cdq_status cdq_init_rtn(const void* W, cdq_dtype wt, long long d_in, long long d_out, long long ldw, const float* H,
                        const cdq_grid_desc* grid, float* scale, float* zero, unsigned char* Q, float* gamma_out,
                        cdq_mode mode, void* ws, size_t ws_bytes, void* stream) {
  if (!W || !scale || !zero || !Q || !valid_dtype(wt) || !valid_mode(mode)) return CDQ_ERR_INVALID_ARG;
  cdq_status s = check_layer_shape(d_in, d_out, ldw);
  if (s != CDQ_OK) return s;
  s = check_grid(grid, d_in);
  if (s != CDQ_OK) return s;
  if (grid->n_clip > 1 && (!H || !aligned16(H))) return CDQ_ERR_INVALID_ARG;
  Layer ly = make_layer(H, W, wt, d_in, d_out, ldw, grid, nullptr, nullptr);
  if (ly.ng > 65535) return CDQ_ERR_UNSUPPORTED;
  s = check_ws(ws, ws_bytes, init_rtn_workspace(d_in, d_out, ly.g, grid->n_clip, mode));
  if (s != CDQ_OK) return s;
  CDQ_CUDA(launch_init_rtn(ly, *grid, scale, zero, Q, gamma_out, mode, ws, (cudaStream_t)stream));
  return CDQ_OK;
}

cdq_status cdq_init_owc_cd(const void* W, cdq_dtype wt, long long d_in, long long d_out, long long ldw, const float* H,
                           const cdq_grid_desc* grid, long long steps, float* scale, float* zero, unsigned char* Q,
                           float* gamma_out, cdq_owc_cd_stats* stats, cdq_mode mode, void* ws, size_t ws_bytes,
                           void* stream) {
  if (!W || !H || !scale || !zero || !Q || !valid_dtype(wt) || !valid_mode(mode)) return CDQ_ERR_INVALID_ARG;
  if (!aligned16(H)) return CDQ_ERR_INVALID_ARG;
  cdq_status s = check_layer_shape(d_in, d_out, ldw);
  if (s != CDQ_OK) return s;
  s = check_grid(grid, d_in);
  if (s != CDQ_OK) return s;
  if (grid->n_clip < 2) return CDQ_ERR_INVALID_ARG;
  Layer ly = make_layer(H, W, wt, d_in, d_out, ldw, grid, nullptr, nullptr);
  if (ly.ng > 65535) return CDQ_ERR_UNSUPPORTED;
  s = check_ws(ws, ws_bytes, owc_cd_workspace(d_in, d_out, ly.g, grid->n_clip, mode));
  if (s != CDQ_OK) return s;
  if (steps <= 0) steps = ly.ng;
  unsigned long long moves = 0;
  double lb = 0.0, la = 0.0;
  CDQ_CUDA(launch_owc_cd(ly, *grid, steps, scale, zero, Q, gamma_out, mode, ws, stats ? &moves : nullptr,
                         stats ? &lb : nullptr, stats ? &la : nullptr, (cudaStream_t)stream));
  if (stats) { stats->moves = moves; stats->loss_before = lb; stats->loss_after = la; }
  return CDQ_OK;
}

static cdq_status cd_solve_impl(const float* H, const void* W, cdq_dtype wt, long long d_in, long long d_out, long long ldw,
                                const cdq_grid_desc* grid, const float* scale, const float* zero, unsigned char* Q,
                                long long steps_per_col, int block, unsigned long long seed, cdq_mode mode,
                                cdq_cd_stats* stats, void* ws, size_t ws_bytes, void* stream, bool rows16 = false,
                                double* loss_out = nullptr, double* per_col_out = nullptr) {
  if (!H || !W || !scale || !zero || !Q || !valid_dtype(wt) || !valid_mode(mode) || steps_per_col < 0)
    return CDQ_ERR_INVALID_ARG;
  if (!aligned16(H)) return CDQ_ERR_INVALID_ARG;
  if (block < 1) return CDQ_ERR_INVALID_ARG;
  if (block > 1 && d_in % block) return CDQ_ERR_SHAPE;
  if (block > 1 && !bcd_supported(d_in, block)) return CDQ_ERR_UNSUPPORTED;
  cdq_status s = check_layer_shape(d_in, d_out, ldw);
  if (s != CDQ_OK) return s;
  s = check_grid(grid, d_in);
  if (s != CDQ_OK) return s;
  if (block > 1 && steps_per_col > 65535) return CDQ_ERR_UNSUPPORTED;
  if (rows16) {
    const long long g = grid->group_size > 0 ? grid->group_size : d_in;
    if (mode != CDQ_MODE_FAST || block != 1 || !cd_rows16_supported(d_in, g)) return CDQ_ERR_UNSUPPORTED;
  }
  const SolveWs L = solve_ws_layout(d_in, d_out, mode, true, block > 1 ? steps_per_col : 0, rows16);
  s = check_ws(ws, ws_bytes, L.total);
  if (s != CDQ_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  char* base = (char*)ws;
  const __nv_bfloat16* H16 = nullptr;
  if (rows16) {   // everything below works on H with its off-diagonal entries rounded to bf16
    CDQ_CUDA(launch_round_rows_bf16(H, d_in, (__nv_bfloat16*)(base + L.h16), (float*)(base + L.hr), st));
    H16 = (const __nv_bfloat16*)(base + L.h16);
    H = (const float*)(base + L.hr);
  }
  Layer ly = make_layer(H, W, wt, d_in, d_out, ldw, grid, scale, zero);
  double* E = (double*)(base + L.E);
  double* G = (double*)(base + L.G);
  unsigned char* Qt = (unsigned char*)(base + L.Qt);
  float* hdiag = (float*)(base + L.hdiag);
  float* half_inv = (float*)(base + L.half_inv);
  double* part = (double*)(base + L.part);
  double* col_loss = (double*)(base + L.col_loss);
  double* loss_sum = (double*)(base + L.scalars);
  CdCounters* ctr = (CdCounters*)(base + L.scalars + 64);

  // G0 = 2 H (W_hat - W) and the loss at entry
  CDQ_CUDA(launch_residual_f64(codes_src(ly, Q), d_in, E, st));
  if (L.tc) {
    CDQ_CUDA(gemm_tc_prepare_h(H, d_in, L.nh, base + L.hbuf, st));
    CDQ_CUDA(gemm_tc_run(base + L.hbuf, L.nh, E, d_in, d_out, L.ne, L.smax, 2.0, G, L.ldg, col_loss, base + L.ebuf, st));
  } else if (mode == CDQ_MODE_FAST) {
    CDQ_CUDA(launch_gemm_he(H, d_in, d_out, E, G, L.ldg, col_loss, part, st));
  } else {
    CDQ_CUDA(launch_gemm_he_verify(H, d_in, d_out, E, part, G, L.ldg, col_loss, st));
  }
  if (mode == CDQ_MODE_FAST) CDQ_CUDA(launch_sum_f64_tree(col_loss, d_out, loss_sum, st));
  else CDQ_CUDA(launch_sum_f64(col_loss, d_out, loss_sum, st));
  CDQ_CUDA(launch_transpose_u8(Q, d_in, d_out, d_out, Qt, L.ldg, st));
  CDQ_CUDA(cudaMemsetAsync(ctr, 0, sizeof(CdCounters), st));
  cudaEvent_t ev0 = nullptr, ev1 = nullptr;
  if (stats) CDQ_CUDA(timing_events(&ev0, &ev1));
  // shapes the fast kernels do not cover (a group size that is not a multiple of 4, very long
  // columns) take the fixed-order fp64 kernel: slower, same result
  const bool fast_cd = mode == CDQ_MODE_FAST && cd_fast_supported(d_in, ly.g);
  if (block > 1) {
    const bool fast = mode == CDQ_MODE_FAST;
    if (fast) CDQ_CUDA(launch_diag(H, d_in, L.d_pad, hdiag, half_inv, st));
    if (stats) CDQ_CUDA(cudaEventRecord(ev0, st));
    CDQ_CUDA(launch_bcd(ly, G, L.ldg, Qt, L.ldg, hdiag, half_inv, steps_per_col, seed, fast, base + L.bcd_tab, ctr,
                        st));
  } else if (fast_cd) {
    CDQ_CUDA(launch_diag(H, d_in, L.d_pad, hdiag, half_inv, st));
    if (stats) CDQ_CUDA(cudaEventRecord(ev0, st));
    CDQ_CUDA(launch_cd_fast(ly, H16, G, L.ldg, Qt, L.ldg, hdiag, half_inv, steps_per_col, ctr, st));
  } else {
    if (stats) CDQ_CUDA(cudaEventRecord(ev0, st));
    CDQ_CUDA(launch_cd_verify(ly, G, L.ldg, Qt, L.ldg, steps_per_col, ctr, st));
  }
  if (stats) CDQ_CUDA(cudaEventRecord(ev1, st));
  CDQ_CUDA(launch_transpose_u8(Qt, d_out, d_in, L.ldg, Q, d_out, st));
  const bool want_loss = loss_out || per_col_out;
  // The register-resident kernels leave the gradient of their result in G: the loss is then a dot product
  // per column.  The other kernels' results get the loss from its definition.
  const bool loss_from_g = want_loss && fast_cd && block == 1 && !rows16;
  if (loss_from_g) {
    double* col_after = per_col_out ? per_col_out : col_loss;   // col_loss has been summed into loss_sum[0] by now
    CDQ_CUDA(launch_residual_f64(codes_src(ly, Q), d_in, E, st));
    CDQ_CUDA(launch_loss_from_gradient(E, G, L.ldg, d_in, d_out, col_after, st));
    if (loss_out) {
      CDQ_CUDA(launch_sum_f64_tree(col_after, d_out, loss_sum + 1, st));
      CDQ_CUDA(cudaMemcpyAsync(loss_out, loss_sum + 1, sizeof(double), cudaMemcpyDeviceToHost, st));
      if (!stats) CDQ_CUDA(cudaStreamSynchronize(st));
    }
  }
  if (stats) {
    CdCounters hc;
    double lb = 0.0;
    CDQ_CUDA(cudaMemcpyAsync(&hc, ctr, sizeof(CdCounters), cudaMemcpyDeviceToHost, st));
    CDQ_CUDA(cudaMemcpyAsync(&lb, loss_sum, sizeof(double), cudaMemcpyDeviceToHost, st));
    CDQ_CUDA(cudaStreamSynchronize(st));
    stats->steps = (unsigned long long)steps_per_col * (unsigned long long)d_out;
    stats->committed = hc.committed;
    stats->columns_converged = hc.converged;
    stats->loss_before = lb;
    stats->loss_after = lb + hc.delta_sum;
    float ms = 0.f;
    CDQ_CUDA(cudaEventElapsedTime(&ms, ev0, ev1));
    stats->kernel_ms = (double)ms;
    const cdq_status ds = read_device_status_after_sync();
    if (ds != CDQ_OK) return ds;
  }
  if (want_loss && !loss_from_g)
    return cdq_layer_loss(H, W, wt, d_in, d_out, ldw, grid, scale, zero, Q, loss_out, per_col_out, mode, ws, ws_bytes, stream);
  return CDQ_OK;
}

cdq_status cdq_cd_solve(const float* H, const void* W, cdq_dtype wt, long long d_in, long long d_out, long long ldw,
                        const cdq_grid_desc* grid, const float* scale, const float* zero, unsigned char* Q,
                        int passes, cdq_mode mode, cdq_cd_stats* stats, void* ws, size_t ws_bytes, void* stream) {
  if (passes < 0) return CDQ_ERR_INVALID_ARG;
  return cd_solve_impl(H, W, wt, d_in, d_out, ldw, grid, scale, zero, Q, (long long)passes * d_in, 1, 0ull, mode, stats,
                       ws, ws_bytes, stream);
}

cdq_status cdq_cd_solve_steps(const float* H, const void* W, cdq_dtype wt, long long d_in, long long d_out,
                              long long ldw, const cdq_grid_desc* grid, const float* scale, const float* zero,
                              unsigned char* Q, long long steps_per_col, cdq_mode mode, cdq_cd_stats* stats, void* ws,
                              size_t ws_bytes, void* stream) {
  return cd_solve_impl(H, W, wt, d_in, d_out, ldw, grid, scale, zero, Q, steps_per_col, 1, 0ull, mode, stats, ws,
                       ws_bytes, stream);
}

cdq_status cdq_cd_solve_with_loss(const float* H, const void* W, cdq_dtype wt, long long d_in, long long d_out,
                                  long long ldw, const cdq_grid_desc* grid, const float* scale, const float* zero,
                                  unsigned char* Q, long long steps_per_col, cdq_mode mode, cdq_cd_stats* stats,
                                  double* loss, double* per_col, void* ws, size_t ws_bytes, void* stream) {
  if (!loss && !per_col) return CDQ_ERR_INVALID_ARG;
  return cd_solve_impl(H, W, wt, d_in, d_out, ldw, grid, scale, zero, Q, steps_per_col, 1, 0ull, mode, stats, ws,
                       ws_bytes, stream, false, loss, per_col);
}

cdq_status cdq_cd_solve_rows16(const float* H, const void* W, cdq_dtype wt, long long d_in, long long d_out,
                               long long ldw, const cdq_grid_desc* grid, const float* scale, const float* zero,
                               unsigned char* Q, long long steps_per_col, cdq_cd_stats* stats, void* ws,
                               size_t ws_bytes, void* stream) {
  return cd_solve_impl(H, W, wt, d_in, d_out, ldw, grid, scale, zero, Q, steps_per_col, 1, 0ull, CDQ_MODE_FAST, stats, ws,
                       ws_bytes, stream, true);
}

cdq_status cdq_bcd_solve(const float* H, const void* W, cdq_dtype wt, long long d_in, long long d_out, long long ldw,
                         const cdq_grid_desc* grid, const float* scale, const float* zero, unsigned char* Q, int block,
                         long long steps_per_col, unsigned long long seed, cdq_mode mode, cdq_cd_stats* stats, void* ws,
                         size_t ws_bytes, void* stream) {
  return cd_solve_impl(H, W, wt, d_in, d_out, ldw, grid, scale, zero, Q, steps_per_col, block, seed, mode, stats, ws,
                       ws_bytes, stream);
}

cdq_status cdq_layer_loss(const float* H, const void* W, cdq_dtype wt, long long d_in, long long d_out, long long ldw,
                          const cdq_grid_desc* grid, const float* scale, const float* zero, const unsigned char* Q,
                          double* loss, double* per_col, cdq_mode mode, void* ws, size_t ws_bytes, void* stream) {
  if (!H || !W || !scale || !zero || !Q || !valid_dtype(wt) || !valid_mode(mode)) return CDQ_ERR_INVALID_ARG;
  if (!aligned16(H)) return CDQ_ERR_INVALID_ARG;
  cdq_status s = check_layer_shape(d_in, d_out, ldw);
  if (s != CDQ_OK) return s;
  s = check_grid(grid, d_in);
  if (s != CDQ_OK) return s;
  const SolveWs L = solve_ws_layout(d_in, d_out, mode, false);
  s = check_ws(ws, ws_bytes, L.total);
  if (s != CDQ_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  Layer ly = make_layer(H, W, wt, d_in, d_out, ldw, grid, scale, zero);
  char* base = (char*)ws;
  double* E = (double*)(base + L.E);
  double* part = (double*)(base + L.part);
  double* col_loss = per_col ? per_col : (double*)(base + L.col_loss);
  double* loss_sum = (double*)(base + L.scalars);
  CDQ_CUDA(launch_residual_f64(codes_src(ly, Q), d_in, E, st));
  if (L.tc) {
    CDQ_CUDA(gemm_tc_prepare_h(H, d_in, L.nh, base + L.hbuf, st));
    CDQ_CUDA(gemm_tc_run(base + L.hbuf, L.nh, E, d_in, d_out, L.ne, L.smax, 1.0, (double*)(base + L.G), L.ldg, col_loss,
                         base + L.ebuf, st));
  } else if (mode == CDQ_MODE_FAST) {
    CDQ_CUDA(launch_gemm_he(H, d_in, d_out, E, nullptr, 0, col_loss, part, st));
  } else {
    CDQ_CUDA(launch_gemm_he_verify(H, d_in, d_out, E, part, nullptr, 0, col_loss, st));
  }
  if (loss) {
    if (mode == CDQ_MODE_FAST) CDQ_CUDA(launch_sum_f64_tree(col_loss, d_out, loss_sum, st));
    else CDQ_CUDA(launch_sum_f64(col_loss, d_out, loss_sum, st));
    CDQ_CUDA(cudaMemcpyAsync(loss, loss_sum, sizeof(double), cudaMemcpyDeviceToHost, st));
    CDQ_CUDA(cudaStreamSynchronize(st));
  }
  return CDQ_OK;
}

}  // extern "C"
