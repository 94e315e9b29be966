// Grid and round-to-nearest codes (paper: Eq. 2), with the OWC grid search over the
// clipping strength gamma (the minimisation stated after Eq. 2).
//
//   min/max per (group, column)  ->  b = min, a = fp32(gamma (max-min) / L)
//   q = clamp(round_half_even((w - b) / a), 0, L)      (decided in fp64)
//   OWC: loss_k[j] = e_k^T H e_k for every gamma_k, argmin over k per column.
#include "common.cuh"

namespace cdq {

constexpr int kChunkRows = 256;  // rows of one min/max partial

__global__ void minmax_partial_kernel(const void* __restrict__ W, cdq_dtype wt, long long d_in, long long d_out,
                                      long long ldw, long long g, long long cpg, float* __restrict__ pmn,
                                      float* __restrict__ pmx) {
  const long long j = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  const long long chunk = blockIdx.y;  // global chunk id = t * cpg + c
  if (j >= d_out) return;
  const long long t = chunk / cpg, c = chunk % cpg;
  const long long i0 = t * g + c * kChunkRows;
  long long i1 = i0 + kChunkRows;
  if (i1 > (t + 1) * g) i1 = (t + 1) * g;
  float mn = 0.f, mx = 0.f;
  bool first = true;
  for (long long i = i0; i < i1; ++i) {
    float w;
    if (wt == CDQ_BF16) w = __bfloat162float(((const __nv_bfloat16*)W)[i * ldw + j]);
    else w = ((const float*)W)[i * ldw + j];
    if (first) { mn = mx = w; first = false; }
    else { mn = fminf(mn, w); mx = fmaxf(mx, w); }
  }
  pmn[chunk * d_out + j] = mn;
  pmx[chunk * d_out + j] = mx;
}

__global__ void minmax_final_kernel(const float* __restrict__ pmn, const float* __restrict__ pmx, long long ng,
                                    long long d_out, long long cpg, float* __restrict__ mn_out,
                                    float* __restrict__ mx_out) {
  const long long j = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  const long long t = blockIdx.y;
  if (j >= d_out) return;
  float mn = pmn[(t * cpg) * d_out + j], mx = pmx[(t * cpg) * d_out + j];
  for (long long c = 1; c < cpg; ++c) {
    mn = fminf(mn, pmn[(t * cpg + c) * d_out + j]);
    mx = fmaxf(mx, pmx[(t * cpg + c) * d_out + j]);
  }
  mn_out[t * d_out + j] = mn;
  mx_out[t * d_out + j] = mx;
}

// a = fp32((gamma * (max - min)) / L) in fp64, b = min.  gamma per column (gam != NULL) or 1.
__global__ void scale_zero_kernel(const float* __restrict__ mn, const float* __restrict__ mx, long long ng,
                                  long long d_out, int L, const double* __restrict__ gam,
                                  float* __restrict__ scale, float* __restrict__ zero) {
  const long long j = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  const long long t = blockIdx.y;
  if (j >= d_out) return;
  const double lo = (double)mn[t * d_out + j], hi = (double)mx[t * d_out + j];
  const double gamma = gam ? gam[j] : 1.0;
  const double a = __ddiv_rn(__dmul_rn(gamma, __dadd_rn(hi, -lo)), (double)L);
  scale[t * d_out + j] = (float)a;
  zero[t * d_out + j] = (float)lo;
}

__global__ void rtn_codes_kernel(const void* __restrict__ W, cdq_dtype wt, long long d_in, long long d_out,
                                 long long ldw, long long g, int L, const float* __restrict__ scale,
                                 const float* __restrict__ zero, unsigned char* __restrict__ Q) {
  const long long j = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  const long long i = blockIdx.y;
  if (j >= d_out) return;
  const float a32 = scale[(i / g) * d_out + j];
  unsigned char q = 0;
  if (a32 > 0.f) {
    const double a = (double)a32, b = (double)zero[(i / g) * d_out + j];
    const double w = load_w(W, wt, i * ldw + j);
    double r = rint(__ddiv_rn(__dadd_rn(w, -b), a));
    r = r < 0.0 ? 0.0 : r;
    r = r > (double)L ? (double)L : r;
    q = (unsigned char)r;
  }
  Q[i * d_out + j] = q;
}

// Residual E[i][j] = (a q + b) - w in fp64, either from stored codes or, for the OWC search,
// from min/max and a clipping strength (codes formed on the fly, never stored).
__global__ void residual_kernel(ResidualSrc s, long long d_in, double* __restrict__ E) {
  const long long j = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  const long long i = blockIdx.y;
  if (j >= s.d_out) return;
  const long long t = i / s.g;
  const double w = load_w(s.W, s.wt, i * s.ldw + j);
  double a, b, q;
  if (s.use_gamma) {
    const double lo = (double)s.mn[t * s.d_out + j], hi = (double)s.mx[t * s.d_out + j];
    const float a32 = (float)__ddiv_rn(__dmul_rn(s.gamma, __dadd_rn(hi, -lo)), (double)s.L);
    a = (double)a32;
    b = lo;
    q = 0.0;
    if (a32 > 0.f) {
      q = rint(__ddiv_rn(__dadd_rn(w, -b), a));
      q = q < 0.0 ? 0.0 : q;
      q = q > (double)s.L ? (double)s.L : q;
    }
  } else {
    a = (double)s.scale[t * s.d_out + j];
    b = (double)s.zero[t * s.d_out + j];
    q = (double)s.Q[i * s.d_out + j];
  }
  E[i * s.d_out + j] = __dadd_rn(__dadd_rn(__dmul_rn(a, q), b), -w);
}

cudaError_t launch_residual_f64(const ResidualSrc& src, long long d_in, double* E, cudaStream_t st) {
  dim3 block(128), grid((unsigned)((src.d_out + 127) / 128), (unsigned)d_in);
  { residual_kernel<<<grid, block, 0, st>>>(src, d_in, E); count_launch(); }
  return cudaGetLastError();
}

// Per column: index of the smallest loss (lowest index on ties) and its gamma.
__global__ void owc_argmin_kernel(const double* __restrict__ table, int n_clip, long long d_out,
                                  const double* __restrict__ gammas, double* __restrict__ gam_col,
                                  float* __restrict__ gamma_out) {
  const long long j = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (j >= d_out) return;
  double best = table[j];
  int bk = 0;
  for (int k = 1; k < n_clip; ++k) {
    const double v = table[(long long)k * d_out + j];
    if (v < best) { best = v; bk = k; }
  }
  gam_col[j] = gammas[bk];
  if (gamma_out) gamma_out[j] = (float)gammas[bk];
}

__global__ void fill_gamma_kernel(float* gamma_out, long long d_out) {
  const long long j = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (j < d_out) gamma_out[j] = 1.0f;
}

// Group minima and maxima of every column: mn, mx [ng, d_out]; pmn, pmx [ng * ceil(g / 256), d_out] scratch.
cudaError_t launch_group_minmax(const Layer& ly, float* pmn, float* pmx, float* mn, float* mx, cudaStream_t st) {
  const long long cpg = (ly.g + kChunkRows - 1) / kChunkRows;
  const unsigned bx = (unsigned)((ly.d_out + 127) / 128);
  { minmax_partial_kernel<<<dim3(bx, (unsigned)(ly.ng * cpg)), 128, 0, st>>>(ly.W, ly.wt, ly.d_in, ly.d_out, ly.ldw, ly.g,
                                                                            cpg, pmn, pmx); count_launch(); }
  { minmax_final_kernel<<<dim3(bx, (unsigned)ly.ng), 128, 0, st>>>(pmn, pmx, ly.ng, ly.d_out, cpg, mn, mx); count_launch(); }
  return cudaGetLastError();
}

// Workspace layout (all blocks 256-byte aligned):
//   pmn, pmx : [ng*cpg, d_out] f32     mn, mx : [ng, d_out] f32
//   OWC only : gammas [n_clip] f64, gam_col [d_out] f64, table [n_clip, d_out] f64,
//              E [d_in, d_out] f64, loss partials (FAST) or the product H E (VERIFY)
struct InitWs {
  size_t pmn, pmx, mn, mx, gammas, gam_col, table, E, part, C, hbuf, ebuf, total;
  bool tc;          // losses on the int8 tensor cores
  long long ldc;
};
static InitWs init_ws_layout(long long d_in, long long d_out, long long g, int n_clip, cdq_mode mode) {
  InitWs w{};
  const long long ng = d_in / g;
  const long long cpg = (g + kChunkRows - 1) / kChunkRows;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes); return o; };
  w.pmn = take(sizeof(float) * ng * cpg * d_out);
  w.pmx = take(sizeof(float) * ng * cpg * d_out);
  w.mn = take(sizeof(float) * ng * d_out);
  w.mx = take(sizeof(float) * ng * d_out);
  if (n_clip > 1) {
    w.gammas = take(sizeof(double) * n_clip);
    w.gam_col = take(sizeof(double) * d_out);
    w.table = take(sizeof(double) * n_clip * d_out);
    w.E = take(sizeof(double) * d_in * d_out);
    w.part = take(sizeof(double) * (mode == CDQ_MODE_FAST ? gemm_partials_elems(d_in, d_out) : (size_t)d_in * d_out));
    w.tc = mode == CDQ_MODE_FAST && gemm_tc_supported(d_in, d_out);
    w.ldc = (d_in + 3) / 4 * 4;
    if (w.tc) {
      w.C = take(sizeof(double) * d_out * w.ldc);
      w.hbuf = take(gemm_tc_h_bytes(d_in, kTcLossNH));
      w.ebuf = take(gemm_tc_e_bytes(d_in, d_out, kTcLossNE));
    }
  }
  w.total = off;
  return w;
}

size_t init_rtn_workspace(long long d_in, long long d_out, long long g, int n_clip, cdq_mode mode) {
  return init_ws_layout(d_in, d_out, g, n_clip, mode).total;
}

cudaError_t launch_init_rtn(const Layer& ly, const cdq_grid_desc& grid, float* scale, float* zero,
                            unsigned char* Q, float* gamma_out, cdq_mode mode, void* ws, cudaStream_t st) {
  const long long d_in = ly.d_in, d_out = ly.d_out, g = ly.g, ng = ly.ng;
  const long long cpg = (g + kChunkRows - 1) / kChunkRows;
  const int n_clip = grid.n_clip > 1 ? grid.n_clip : 1;
  const InitWs L = init_ws_layout(d_in, d_out, g, n_clip, mode);
  char* base = (char*)ws;
  float* pmn = (float*)(base + L.pmn);
  float* pmx = (float*)(base + L.pmx);
  float* mn = (float*)(base + L.mn);
  float* mx = (float*)(base + L.mx);
  const unsigned bx = (unsigned)((d_out + 127) / 128);

  { minmax_partial_kernel<<<dim3(bx, (unsigned)(ng * cpg)), 128, 0, st>>>(ly.W, ly.wt, d_in, d_out, ly.ldw, g, cpg,
                                                                         pmn, pmx); count_launch(); }
  { minmax_final_kernel<<<dim3(bx, (unsigned)ng), 128, 0, st>>>(pmn, pmx, ng, d_out, cpg, mn, mx); count_launch(); }

  const double* gam_col = nullptr;
  if (n_clip > 1) {
    double* gammas = (double*)(base + L.gammas);
    double* gcol = (double*)(base + L.gam_col);
    double* table = (double*)(base + L.table);
    double* E = (double*)(base + L.E);
    double* part = (double*)(base + L.part);
    double hg[256];
    const double lo = (double)grid.clip_lo, hi = (double)grid.clip_hi;
    for (int k = 0; k < n_clip; ++k) hg[k] = lo + ((hi - lo) * (double)k) / (double)(n_clip - 1);
    cudaError_t e = cudaMemcpyAsync(gammas, hg, sizeof(double) * n_clip, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return e;
    // the host array must outlive the copy: pageable memcpy is staged before return
    if (L.tc) {   // the slices of H serve every clipping strength
      e = gemm_tc_prepare_h(ly.H, d_in, kTcLossNH, base + L.hbuf, st);
      if (e != cudaSuccess) return e;
    }
    for (int k = 0; k < n_clip; ++k) {
      ResidualSrc src{};
      src.W = ly.W; src.wt = ly.wt; src.ldw = ly.ldw;
      src.mn = mn; src.mx = mx; src.gamma = hg[k]; src.L = ly.L; src.use_gamma = 1;
      src.g = g; src.d_out = d_out;
      e = launch_residual_f64(src, d_in, E, st);
      if (e != cudaSuccess) return e;
      if (L.tc)
        e = gemm_tc_run(base + L.hbuf, kTcLossNH, E, d_in, d_out, kTcLossNE, kTcLossSmax, 1.0, (double*)(base + L.C), L.ldc,
                        table + (long long)k * d_out, base + L.ebuf, st);
      else if (mode == CDQ_MODE_FAST)
        e = launch_gemm_he(ly.H, d_in, d_out, E, nullptr, 0, table + (long long)k * d_out, part, st);
      else
        e = launch_gemm_he_verify(ly.H, d_in, d_out, E, part, nullptr, 0, table + (long long)k * d_out, st);
      if (e != cudaSuccess) return e;
    }
    { owc_argmin_kernel<<<bx, 128, 0, st>>>(table, n_clip, d_out, gammas, gcol, gamma_out); count_launch(); }
    gam_col = gcol;
  } else if (gamma_out) {
    { fill_gamma_kernel<<<bx, 128, 0, st>>>(gamma_out, d_out); count_launch(); }
  }
  { scale_zero_kernel<<<dim3(bx, (unsigned)ng), 128, 0, st>>>(mn, mx, ng, d_out, ly.L, gam_col, scale, zero); count_launch(); }
  { rtn_codes_kernel<<<dim3(bx, (unsigned)d_in), 128, 0, st>>>(ly.W, ly.wt, d_in, d_out, ly.ldw, g, ly.L, scale, zero, Q); count_launch(); }
  return cudaGetLastError();
}

}  // namespace cdq
