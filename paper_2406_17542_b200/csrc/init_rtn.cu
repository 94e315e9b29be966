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
  const long long c = blockIdx.x * (long long)blockDim.x + threadIdx.x;   // column of E
  const long long i = blockIdx.y;
  const long long width = s.col_idx ? s.n_cols : s.d_out;
  if (c >= width) return;
  const long long j = s.col_idx ? (long long)s.col_idx[c] : c;            // column of the layer
  const long long t = i / s.g;
  const double w = load_w(s.W, s.wt, i * s.ldw + j);
  double a, b, q;
  if (s.use_gamma) {
    const double lo = (double)s.mn[t * s.d_out + j], hi = (double)s.mx[t * s.d_out + j];
    const double gamma = s.col_gamma ? s.gammas[s.col_gamma[c]] : s.gamma;
    const float a32 = (float)__ddiv_rn(__dmul_rn(gamma, __dadd_rn(hi, -lo)), (double)s.L);
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
  E[i * width + c] = __dadd_rn(__dadd_rn(__dmul_rn(a, q), b), -w);
}

cudaError_t launch_residual_f64(const ResidualSrc& src, long long d_in, double* E, cudaStream_t st) {
  const long long width = src.col_idx ? src.n_cols : src.d_out;
  dim3 block(128), grid((unsigned)((width + 127) / 128), (unsigned)d_in);
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

// ---- screening of the clipping search (production mode, tensor-core losses) ----
// The losses of all clipping strengths are first formed cheaply (three slice-pair products instead of thirteen);
// a strength stays a candidate of a column if its screened loss is within kScreenBand of the column's smallest.
// Only candidates get the thirteen-pair loss, and the argmin is taken over those: the same result as the full
// table as long as the screening error stays inside the band.  The loss as a function of the strength is smooth
// with one minimum, and the second-best strength of a column is typically percents away (median 2.5 % on 2-bit,
// 5 % on 3-bit grouped layers), so a band of 1 % keeps 1.1 to 1.3 candidates per column.  The screen keeps two
// 7-bit slices of the residual and of H on grids of up to 4 bits: the slicing truncates below 2^-14 of the column's
// largest residual, and a clipped weight leaves a residual up to (1 - gamma) L times the typical rounding error
// (7.5 times at 4 bits), which put the screened loss off by up to 6e-4 on a 3-bit layer -- a factor of 8 inside half
// the band.  Finer grids (L up to 255) keep three slices and six products.
constexpr double kScreenBand = 1e-2;
__host__ __device__ constexpr int screen_slices(int bits) { return bits <= 4 ? 2 : 3; }   // pairs up to i + j = slices + 1

// mask[k][j] = 1 for candidates; the table starts at +inf everywhere.
__global__ void owc_candidates_kernel(const double* __restrict__ screen, int n_clip, long long d_out,
                                      unsigned char* __restrict__ mask, double* __restrict__ table) {
  const long long j = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (j >= d_out) return;
  double best = screen[j];
  for (int k = 1; k < n_clip; ++k) best = fmin(best, screen[(long long)k * d_out + j]);
  const double lim = best + kScreenBand * fabs(best);
  for (int k = 0; k < n_clip; ++k) {
    mask[(long long)k * d_out + j] = screen[(long long)k * d_out + j] <= lim ? 1 : 0;
    table[(long long)k * d_out + j] = __longlong_as_double(0x7FF0000000000000ll);
  }
}

// One CTA per clipping strength: its candidate columns in ascending order; cnt[k] = their number.
__global__ void __launch_bounds__(1024) owc_compact_kernel(const unsigned char* __restrict__ mask, long long d_out,
                                                           int* __restrict__ idx, int* __restrict__ cnt) {
  __shared__ int s_scan[1024];
  __shared__ int s_base;
  const int k = blockIdx.x, tid = threadIdx.x;
  const unsigned char* m = mask + (long long)k * d_out;
  int* out = idx + (long long)k * (d_out + 128);
  if (tid == 0) s_base = 0;
  __syncthreads();
  for (long long j0 = 0; j0 < d_out; j0 += 1024) {
    const long long j = j0 + tid;
    const int f = (j < d_out && m[j]) ? 1 : 0;
    s_scan[tid] = f;
    __syncthreads();
    for (int o = 1; o < 1024; o <<= 1) {
      const int v = tid >= o ? s_scan[tid - o] : 0;
      __syncthreads();
      s_scan[tid] += v;
      __syncthreads();
    }
    if (f) out[s_base + s_scan[tid] - 1] = (int)j;
    __syncthreads();
    if (tid == 0) s_base += s_scan[1023];
    __syncthreads();
  }
  if (tid == 0) cnt[k] = s_base;
}

// The candidates of all strengths as one list of (column, strength) in the order of the strengths, so that the
// exact losses take a few wide products instead of one narrow product per strength.  off[k]: where strength k's
// candidates start (off[n_clip] = their total); entries from the total up to `padded` (a multiple of 128, the
// granularity of the tensor-core product) repeat the last candidate.
struct OwcOffsets { int off[257]; };
__global__ void owc_concat_kernel(const int* __restrict__ idx, long long d_out, OwcOffsets offs, int n_clip, int padded,
                                  int* __restrict__ cj, int* __restrict__ ck) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= padded) return;
  const int total = offs.off[n_clip];
  const int cc = c < total ? c : total - 1;
  int k = 0;
  while (k + 1 < n_clip && offs.off[k + 1] <= cc) ++k;
  cj[c] = idx[(long long)k * (d_out + 128) + (cc - offs.off[k])];
  ck[c] = k;
}

// Columns of a screening product over several strengths at once: column c is layer column c % d_out under strength
// k0 + c / d_out.
__global__ void owc_iota_kernel(long long d_out, int k0, long long width, int* __restrict__ cj, int* __restrict__ ck) {
  const long long c = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (c >= width) return;
  cj[c] = (int)(c % d_out);
  ck[c] = k0 + (int)(c / d_out);
}

__global__ void owc_scatter_kernel(const double* __restrict__ loss_c, const int* __restrict__ cj, const int* __restrict__ ck,
                                   int n, long long d_out, double* __restrict__ table) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c < n) table[(long long)ck[c] * d_out + cj[c]] = loss_c[c];   // padding repeats a candidate with its own value
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
  size_t pmn, pmx, mn, mx, gammas, gam_col, table, E, part, C, hbuf, ebuf, screen, mask, idx, cnt, loss_c, cj, ck, total;
  bool screened;    // cheap losses first, exact ones for the near-tied strengths only
  int sbatch;       // strengths per screening product (several on small layers, where a product per strength is launch-bound)
  long long wcap;   // columns that E, C and the slice buffers hold
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
    w.tc = mode == CDQ_MODE_FAST && gemm_tc_supported(d_in, d_out);
    w.screened = w.tc && n_clip >= 4;
    w.sbatch = 1;
    if (w.screened) {   // up to 1 GiB of residuals per product
      const long long fit = (1ll << 30) / (8 * d_in * d_out);
      w.sbatch = (int)(fit < 1 ? 1 : (fit > n_clip ? n_clip : fit));
    }
    w.wcap = d_out + 128 > (long long)w.sbatch * d_out ? d_out + 128 : (long long)w.sbatch * d_out;
    w.E = take(sizeof(double) * d_in * w.wcap);
    w.part = take(sizeof(double) * (mode == CDQ_MODE_FAST ? gemm_partials_elems(d_in, d_out) : (size_t)d_in * d_out));
    w.ldc = (d_in + 3) / 4 * 4;
    if (w.tc) {
      w.C = take(sizeof(double) * w.wcap * w.ldc);
      w.hbuf = take(gemm_tc_h_bytes(d_in, kTcLossNH));
      w.ebuf = take(gemm_tc_e_bytes(d_in, w.wcap, kTcLossNE));
      if (w.screened) {
        w.screen = take(sizeof(double) * n_clip * d_out);
        w.mask = take((size_t)n_clip * d_out);
        w.idx = take(sizeof(int) * (size_t)n_clip * (d_out + 128));
        w.cnt = take(sizeof(int) * n_clip);
        w.loss_c = take(sizeof(double) * w.wcap);
        w.cj = take(sizeof(int) * ((size_t)n_clip * d_out + 128));
        w.ck = take(sizeof(int) * ((size_t)n_clip * d_out + 128));
      }
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
    if (L.screened) {
      double* screen = (double*)(base + L.screen);
      unsigned char* mask = (unsigned char*)(base + L.mask);
      int* idx = (int*)(base + L.idx);
      int* cnt = (int*)(base + L.cnt);
      double* loss_c = (double*)(base + L.loss_c);
      int* cj = (int*)(base + L.cj);
      int* ck = (int*)(base + L.ck);
      for (int k0 = 0; k0 < n_clip; k0 += L.sbatch) {   // screening, L.sbatch strengths per product
        const int gb = n_clip - k0 < L.sbatch ? n_clip - k0 : L.sbatch;
        const long long width = (long long)gb * d_out;
        ResidualSrc src{};
        src.W = ly.W; src.wt = ly.wt; src.ldw = ly.ldw;
        src.mn = mn; src.mx = mx; src.gamma = hg[k0]; src.L = ly.L; src.use_gamma = 1;
        src.g = g; src.d_out = d_out;
        if (gb > 1) {
          { owc_iota_kernel<<<(unsigned)((width + 255) / 256), 256, 0, st>>>(d_out, k0, width, cj, ck); count_launch(); }
          src.col_idx = cj; src.n_cols = width; src.col_gamma = ck; src.gammas = gammas;
        }
        e = launch_residual_f64(src, d_in, E, st);
        if (e != cudaSuccess) return e;
        e = gemm_tc_run(base + L.hbuf, kTcLossNH, E, d_in, width, screen_slices(ly.bits), screen_slices(ly.bits) + 1, 1.0,
                        (double*)(base + L.C), L.ldc, screen + (long long)k0 * d_out, base + L.ebuf, st);
        if (e != cudaSuccess) return e;
      }
      { owc_candidates_kernel<<<bx, 128, 0, st>>>(screen, n_clip, d_out, mask, table); count_launch(); }
      { owc_compact_kernel<<<(unsigned)n_clip, 1024, 0, st>>>(mask, d_out, idx, cnt); count_launch(); }
      int hcnt[256];
      e = cudaMemcpyAsync(hcnt, cnt, sizeof(int) * n_clip, cudaMemcpyDeviceToHost, st);
      if (e != cudaSuccess) return e;
      e = cudaStreamSynchronize(st);   // the sizes of the exact products are decided on the host
      if (e != cudaSuccess) return e;
      OwcOffsets offs{};
      for (int k = 0; k < n_clip; ++k) offs.off[k + 1] = offs.off[k] + hcnt[k];
      const int total = offs.off[n_clip], padded = (total + 127) / 128 * 128;
      if (total <= 0) return cudaErrorUnknown;   // every column has at least its best strength as a candidate
      { owc_concat_kernel<<<(unsigned)((padded + 255) / 256), 256, 0, st>>>(idx, d_out, offs, n_clip, padded, cj, ck); count_launch(); }
      const int cap = (int)(L.wcap / 128 * 128);   // columns per product: what E, C and the slice buffers hold
      for (int b0 = 0; b0 < padded; b0 += cap) {
        const int width = padded - b0 < cap ? padded - b0 : cap;
        ResidualSrc src{};
        src.W = ly.W; src.wt = ly.wt; src.ldw = ly.ldw;
        src.mn = mn; src.mx = mx; src.L = ly.L; src.use_gamma = 1;
        src.g = g; src.d_out = d_out; src.col_idx = cj + b0; src.n_cols = width;
        src.col_gamma = ck + b0; src.gammas = gammas;
        e = launch_residual_f64(src, d_in, E, st);
        if (e != cudaSuccess) return e;
        e = gemm_tc_run(base + L.hbuf, kTcLossNH, E, d_in, width, kTcLossNE, kTcLossSmax, 1.0, (double*)(base + L.C), L.ldc,
                        loss_c, base + L.ebuf, st);
        if (e != cudaSuccess) return e;
        { owc_scatter_kernel<<<(unsigned)((width + 255) / 256), 256, 0, st>>>(loss_c, cj + b0, ck + b0, width, d_out, table); count_launch(); }
      }
    } else
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
