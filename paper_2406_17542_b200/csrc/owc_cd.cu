// OWC-CD: greedy coordinate descent over the clipping strengths of a column's groups (paper:
// Algorithm 3, "Coordinate Descent for Optimal Weight Clipping").
//
// Per column j: every group t holds a grid index cur[t] (start: the last grid point), the state is
// G = 2 H e with e = w_hat - w, and one step changes the strength of the one group whose change
// lowers the loss most:
//     delta = r(t, k) - r(t, cur[t])           r(t, k): residual of group t under gamma_k (Eq. 2)
//     change(t, k) = delta^T H_tt delta + delta^T G_t
//     G <- G + 2 H[:, t] delta
// (the sign convention is the one under which the change is the true change of the quadratic
// loss; the paper's box has the linear term with the opposite sign of its own definitions).
// Ties go to the lowest group, then the lowest grid index; a change must strictly lower the loss.
//
// One CTA per column at a time (columns handed out by an atomic counter), fp64 throughout.  The
// residual table r(., k) of the column is built once in a per-CTA scratch area.
//   VERIFY: every sum in ascending index order without fused multiply-add, one thread per output,
//           so that indices and codes can be compared bit for bit with a CPU statement of the steps.
//   FAST:   M(k) = H_tt r(t, k) is tabulated once per column, after which a step needs only
//           dot products of length g:  delta^T H_tt delta = r_k.M_k - 2 r_k.M_c + r_c.M_c;
//           one warp per dot product, lanes across the group.
#include "common.cuh"

namespace cdq {
namespace owc {

constexpr int NT = 512;
constexpr int KC = 8;     // grid points per pass of the M table (accumulators per thread)

struct Counters {
  int next_col;
  int pad;
  unsigned long long moves;
};

struct Params {
  const float* H;
  const void* W;
  cdq_dtype wt;
  long long d_in, d_out, ldw, g, ng;
  int L, nk;
  const double* gammas;   // [nk]
  const float* mn;        // [ng, d_out] group minima
  const float* mx;        // [ng, d_out] group maxima
  long long steps;
  float* scale;           // [ng, d_out]
  float* zero;            // [ng, d_out]
  unsigned char* Q;       // [d_in, d_out]
  float* gamma_out;       // [ng, d_out] or NULL
  double* scratch;        // per CTA: R [nk, d_in], M [nk, d_in], G [d_in], S [max(ng * nk, g)]
  size_t scratch_per_cta; // doubles
  int* cur;               // per CTA: [ng]
  double* col_before;     // [d_out]
  double* col_after;      // [d_out]
  double* Gext;           // FAST, optional: [d_out, ldg] G = 2 H e at the start, made by the tensor-core GEMM
  long long ldg;          //   (then col_before is already filled and the kernel skips that product)
  Counters* ctr;
};

// Residual a q + b - w of one weight under clipping strength gamma (Eq. 2; the arithmetic of
// residual_kernel in init_rtn.cu).  Also returns the code and the grid through the pointers.
__device__ __forceinline__ double resid(double w, double lo, double hi, double gamma, int L, float* a_out,
                                        unsigned char* q_out) {
  const float a32 = (float)__ddiv_rn(__dmul_rn(gamma, __dadd_rn(hi, -lo)), (double)L);
  const double a = (double)a32;
  double q = 0.0;
  if (a32 > 0.f) {
    q = rint(__ddiv_rn(__dadd_rn(w, -lo), a));
    q = q < 0.0 ? 0.0 : q;
    q = q > (double)L ? (double)L : q;
  }
  if (a_out) *a_out = a32;
  if (q_out) *q_out = (unsigned char)q;
  return __dadd_rn(__dadd_rn(__dmul_rn(a, q), lo), -w);
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}

template <bool VERIFY>
__global__ void __launch_bounds__(NT, 2) owc_cd_kernel(Params p) {
  __shared__ int s_col;
  __shared__ double s_val[NT];
  __shared__ int s_idx[NT];
  extern __shared__ double dyn[];   // FAST: quad [ng * nk] (delta^T H_tt delta per candidate), rg [ng * nk] (r_k . G_t)
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = NT >> 5;
  const long long d_in = p.d_in, g = p.g, ng = p.ng;
  const int nk = p.nk;
  double* R = p.scratch + (size_t)blockIdx.x * p.scratch_per_cta;   // [nk, d_in] residuals
  double* M = R + (size_t)nk * d_in;                                 // [nk, d_in] H_tt r (FAST), H e (VERIFY, row 0)
  double* Gown = M + (size_t)nk * d_in;                              // [d_in]
  double* S = Gown + d_in;                                            // [max(ng * nk, g)] scores / delta
  int* cur = p.cur + (size_t)blockIdx.x * ng;
  unsigned long long my_moves = 0;

  for (;;) {
    __syncthreads();
    if (tid == 0) s_col = atomicAdd(&p.ctr->next_col, 1);
    __syncthreads();
    const long long j = s_col;
    if (j >= p.d_out) break;

    // ---- residual table per clipping strength and start (Algorithm 3) ----
    for (long long idx = tid; idx < (long long)nk * d_in; idx += NT) {
      const int k = (int)(idx / d_in);
      const long long i = idx - (long long)k * d_in, t = i / g;
      R[idx] = resid(load_w(p.W, p.wt, i * p.ldw + j), (double)p.mn[t * p.d_out + j], (double)p.mx[t * p.d_out + j],
                     p.gammas[k], p.L, nullptr, nullptr);
    }
    for (long long t = tid; t < ng; t += NT) cur[t] = nk - 1;
    __syncthreads();

    // ---- G = 2 H e and the starting loss ----
    double* G = (!VERIFY && p.Gext) ? p.Gext + j * p.ldg : Gown;
    const double* e0 = R + (size_t)(nk - 1) * d_in;
    double loss = 0.0;
    if (VERIFY) {
      for (long long pp = tid; pp < d_in; pp += NT) {
        const float* row = p.H + pp * d_in;
        double acc = 0.0;
        for (long long k = 0; k < d_in; ++k) acc = __dadd_rn(acc, __dmul_rn((double)row[k], e0[k]));
        M[pp] = acc;
        G[pp] = __dmul_rn(2.0, acc);
      }
      __syncthreads();
      if (tid == 0) {
        double l = 0.0;
        for (long long pp = 0; pp < d_in; ++pp) l = __dadd_rn(l, __dmul_rn(e0[pp], M[pp]));
        s_val[0] = l;
      }
      __syncthreads();
      loss = s_val[0];
      __syncthreads();
    } else {
      if (p.Gext) {
        loss = p.col_before[j];
      } else {
        double part = 0.0;
        for (long long pp = warp; pp < d_in; pp += nwarps) {
          const float* row = p.H + pp * d_in;
          double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
          long long k = lane;
          for (; k + 96 < d_in; k += 128) {
            a0 = fma((double)row[k], e0[k], a0);
            a1 = fma((double)row[k + 32], e0[k + 32], a1);
            a2 = fma((double)row[k + 64], e0[k + 64], a2);
            a3 = fma((double)row[k + 96], e0[k + 96], a3);
          }
          for (; k < d_in; k += 32) a0 = fma((double)row[k], e0[k], a0);
          const double acc = warp_sum((a0 + a1) + (a2 + a3));
          if (lane == 0) { G[pp] = 2.0 * acc; part = fma(e0[pp], acc, part); }
        }
        s_val[tid] = part;
        __syncthreads();
        for (int w = NT / 2; w > 0; w >>= 1) {
          if (tid < w) s_val[tid] += s_val[tid + w];
          __syncthreads();
        }
        loss = s_val[0];
        __syncthreads();
      }
      // M(k) = H_tt r(t, k): one thread per coordinate i and pass of KC grid points, so that a
      // value of H feeds KC independent accumulators.  H is symmetric, so M(k)[i] is summed down
      // column i of the block, H[t0 + q][i]: neighbouring threads read neighbouring addresses.
      const int npass = (nk + KC - 1) / KC;
      for (long long idx = tid; idx < (long long)npass * d_in; idx += NT) {
        const int ps = (int)(idx / d_in);
        const long long i = idx - (long long)ps * d_in, t0 = (i / g) * g;
        const float* col = p.H + t0 * d_in + i;
        double acc[KC];
#pragma unroll
        for (int c = 0; c < KC; ++c) acc[c] = 0.0;
#pragma unroll 4
        for (long long q = 0; q < g; ++q) {
          const double h = (double)col[q * d_in];
#pragma unroll
          for (int c = 0; c < KC; ++c) {
            const int k = ps * KC + c;
            if (k < nk) acc[c] = fma(h, R[(size_t)k * d_in + t0 + q], acc[c]);
          }
        }
#pragma unroll
        for (int c = 0; c < KC; ++c) {
          const int k = ps * KC + c;
          if (k < nk) M[(size_t)k * d_in + i] = acc[c];
        }
      }
      __syncthreads();
    }
    if (tid == 0 && (VERIFY || !p.Gext)) p.col_before[j] = loss;

    // ---- descent over the strengths (the loop of Algorithm 3) ----
    const long long ntask = ng * nk;
    long long nmoves = 0;
    double* quad_s = dyn;
    double* rg_s = dyn + ntask;
    // delta^T H_tt delta = r_k.M_k - 2 r_k.M_c + r_c.M_c for every candidate of the groups [t_lo, t_hi)
    auto refresh_quad = [&](long long t_lo, long long t_hi) {
      for (long long task = t_lo * nk + warp; task < t_hi * nk; task += nwarps) {
        const long long t = task / nk;
        const int k = (int)(task - t * nk), c = cur[t];
        const double* rk = R + (size_t)k * d_in + t * g;
        const double* rc = R + (size_t)c * d_in + t * g;
        const double* mk = M + (size_t)k * d_in + t * g;
        const double* mc = M + (size_t)c * d_in + t * g;
        double v = 0.0;
#pragma unroll 4
        for (long long pp = lane; pp < g; pp += 32) {
          const double a = rk[pp], b = rc[pp], m = mc[pp];
          v += a * mk[pp] - 2.0 * a * m + b * m;
        }
        v = warp_sum(v);
        if (lane == 0) quad_s[task] = v;
      }
    };
    if (!VERIFY) { refresh_quad(0, ng); __syncthreads(); }
    for (long long step = 0; step < p.steps; ++step) {
      // score of every (group, grid point); the current point scores +0 and is never taken
      if (VERIFY) {
        for (long long task = tid; task < ntask; task += NT) {
          const long long t = task / nk;
          const int k = (int)(task - t * nk), c = cur[t];
          double change = 0.0;
          if (k != c) {
            const double* cand = R + (size_t)k * d_in + t * g;
            const double* old = R + (size_t)c * d_in + t * g;
            double quad = 0.0, lin = 0.0;
            for (long long pp = 0; pp < g; ++pp) {
              const float* row = p.H + (t * g + pp) * d_in + t * g;
              double acc = 0.0;
              for (long long r = 0; r < g; ++r)
                acc = __dadd_rn(acc, __dmul_rn((double)row[r], __dadd_rn(cand[r], -old[r])));
              const double dp = __dadd_rn(cand[pp], -old[pp]);
              quad = __dadd_rn(quad, __dmul_rn(dp, acc));
              lin = __dadd_rn(lin, __dmul_rn(dp, G[t * g + pp]));
            }
            change = __dadd_rn(quad, lin);
          }
          S[task] = change;
        }
      } else {
        // r_k . G_t for every candidate: one warp per group and four grid points, so that 16 loads are in flight
        const int kq = (nk + 3) / 4;
        for (long long wt = warp; wt < ng * kq; wt += nwarps) {
          const long long t = wt / kq;
          const int k0 = (int)(wt - t * kq) * 4;
          double acc[4] = {0.0, 0.0, 0.0, 0.0};
          for (long long pp = lane; pp < g; pp += 32) {
            const double gv = G[t * g + pp];
#pragma unroll
            for (int u = 0; u < 4; ++u)
              if (k0 + u < nk) acc[u] = fma(R[(size_t)(k0 + u) * d_in + t * g + pp], gv, acc[u]);
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const double a = warp_sum(acc[u]);
            if (lane == 0 && k0 + u < nk) rg_s[t * nk + k0 + u] = a;
          }
        }
        __syncthreads();
        for (long long task = tid; task < ntask; task += NT) {
          const long long t = task / nk;
          const int k = (int)(task - t * nk), c = cur[t];
          S[task] = k == c ? 0.0 : quad_s[task] + (rg_s[task] - rg_s[t * nk + c]);
        }
      }
      __syncthreads();
      // argmin: lowest (group, grid index) among equal scores
      double bv = 0.0;
      int bi = -1;
      for (long long task = tid; task < ntask; task += NT) {
        const double v = S[task];
        if (v < bv) { bv = v; bi = (int)task; }
      }
      s_val[tid] = bv; s_idx[tid] = bi;
      __syncthreads();
      for (int w = NT / 2; w > 0; w >>= 1) {
        if (tid < w) {
          const double ov = s_val[tid + w];
          const int oi = s_idx[tid + w];
          const bool take = oi >= 0 && (s_idx[tid] < 0 || ov < s_val[tid] || (ov == s_val[tid] && oi < s_idx[tid]));
          if (take) { s_val[tid] = ov; s_idx[tid] = oi; }
        }
        __syncthreads();
      }
      const int best = s_idx[0];
      const double bchange = s_val[0];
      __syncthreads();
      if (best < 0) break;
      const long long ts = best / nk;
      const int ks = best - (int)ts * nk, cs = cur[ts];
      // delta of the winning group, then G <- G + 2 H[:, group] delta
      for (long long r = tid; r < g; r += NT) S[r] = __dadd_rn(R[(size_t)ks * d_in + ts * g + r], -R[(size_t)cs * d_in + ts * g + r]);
      __syncthreads();
      if (VERIFY) {
        for (long long i = tid; i < d_in; i += NT) {
          const float* row = p.H + i * d_in + ts * g;
          double acc = 0.0;
          for (long long r = 0; r < g; ++r) acc = __dadd_rn(acc, __dmul_rn((double)row[r], S[r]));
          G[i] = __dadd_rn(G[i], __dmul_rn(2.0, acc));
        }
      } else {
        // G[i] += 2 sum_r H[ts g + r][i] delta_r: H is symmetric, so the g rows of the group are read
        // along i, four coordinates per thread and 16 bytes per load, as the descent kernels read
        // their rows; the sum over r runs in ascending order
        const float* rows = p.H + ts * g * d_in;
        if ((d_in & 3) == 0 && (reinterpret_cast<uintptr_t>(p.H) & 15) == 0) {
          for (long long i = 4ll * tid; i < d_in; i += 4ll * NT) {
            double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
#pragma unroll 8
            for (long long r = 0; r < g; ++r) {
              const float4 h = __ldg(reinterpret_cast<const float4*>(rows + r * d_in + i));
              const double dl = S[r];
              a0 = fma((double)h.x, dl, a0);
              a1 = fma((double)h.y, dl, a1);
              a2 = fma((double)h.z, dl, a2);
              a3 = fma((double)h.w, dl, a3);
            }
            G[i] += 2.0 * a0; G[i + 1] += 2.0 * a1; G[i + 2] += 2.0 * a2; G[i + 3] += 2.0 * a3;
          }
        } else {
          for (long long i = tid; i < d_in; i += NT) {
            double a0 = 0.0;
            for (long long r = 0; r < g; ++r) a0 = fma((double)rows[r * d_in + i], S[r], a0);
            G[i] += 2.0 * a0;
          }
        }
      }
      __syncthreads();
      if (tid == 0) cur[ts] = ks;
      loss = __dadd_rn(loss, bchange);
      ++nmoves;
      __syncthreads();
      if (!VERIFY) { refresh_quad(ts, ts + 1); __syncthreads(); }
    }
    if (tid == 0) { p.col_after[j] = loss; my_moves += (unsigned long long)nmoves; }

    // ---- emit grid, codes and strengths of the chosen points ----
    for (long long t = tid; t < ng; t += NT) {
      float a32;
      resid(0.0, (double)p.mn[t * p.d_out + j], (double)p.mx[t * p.d_out + j], p.gammas[cur[t]], p.L, &a32, nullptr);
      p.scale[t * p.d_out + j] = a32;
      p.zero[t * p.d_out + j] = p.mn[t * p.d_out + j];
      if (p.gamma_out) p.gamma_out[t * p.d_out + j] = (float)p.gammas[cur[t]];
    }
    for (long long i = tid; i < d_in; i += NT) {
      const long long t = i / g;
      unsigned char q;
      resid(load_w(p.W, p.wt, i * p.ldw + j), (double)p.mn[t * p.d_out + j], (double)p.mx[t * p.d_out + j],
            p.gammas[cur[t]], p.L, nullptr, &q);
      p.Q[i * p.d_out + j] = q;
    }
  }
  if (tid == 0 && my_moves) atomicAdd(&p.ctr->moves, my_moves);
}

}  // namespace owc

// ---------------------------------------------------------------------------------------------
constexpr int kOwcMaxCtas = 296;

struct OwcWs {
  size_t pmn, pmx, mn, mx, gammas, scratch, cur, col_before, col_after, sums, ctr, E, G, hbuf, ebuf, total;
  bool tc;            // starting gradient by the int8 tensor-core GEMM (production mode, large enough layers)
  long long ldg;
  size_t scratch_per_cta;   // doubles
  long long cpg;
};
static OwcWs owc_ws_layout(long long d_in, long long d_out, long long g, int nk, cdq_mode mode) {
  OwcWs w{};
  const long long ng = d_in / g;
  w.cpg = (g + 255) / 256;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes); return o; };
  w.pmn = take(sizeof(float) * ng * w.cpg * d_out);
  w.pmx = take(sizeof(float) * ng * w.cpg * d_out);
  w.mn = take(sizeof(float) * ng * d_out);
  w.mx = take(sizeof(float) * ng * d_out);
  w.gammas = take(sizeof(double) * nk);
  const size_t tail = (size_t)(ng * nk > g ? ng * nk : g);
  w.scratch_per_cta = (2 * (size_t)nk * d_in + (size_t)d_in + tail + 31) / 32 * 32;
  const long long ctas = d_out < kOwcMaxCtas ? d_out : kOwcMaxCtas;
  w.scratch = take(sizeof(double) * w.scratch_per_cta * ctas);
  w.cur = take(sizeof(int) * ng * ctas);
  w.col_before = take(sizeof(double) * d_out);
  w.col_after = take(sizeof(double) * d_out);
  w.sums = take(sizeof(double) * 2);
  w.ctr = take(sizeof(owc::Counters));
  w.tc = mode == CDQ_MODE_FAST && gemm_tc_supported(d_in, d_out);
  w.ldg = (d_in + 3) / 4 * 4;
  if (w.tc) {
    w.E = take(sizeof(double) * d_in * d_out);
    w.G = take(sizeof(double) * d_out * w.ldg);
    w.hbuf = take(gemm_tc_h_bytes(d_in, kTcGradNH));
    w.ebuf = take(gemm_tc_e_bytes(d_in, d_out, kTcGradNE));
  }
  w.total = off;
  return w;
}

size_t owc_cd_workspace(long long d_in, long long d_out, long long g, int n_clip, cdq_mode mode) {
  return owc_ws_layout(d_in, d_out, g, n_clip, mode).total;
}

// Enqueues the whole OWC-CD on `st`.  host_moves / host_before / host_after (all NULL or all
// non-NULL) are filled after a stream synchronisation.
cudaError_t launch_owc_cd(const Layer& ly, const cdq_grid_desc& grid, long long steps, float* scale, float* zero,
                          unsigned char* Q, float* gamma_out, cdq_mode mode, void* ws, unsigned long long* host_moves,
                          double* host_before, double* host_after, cudaStream_t st) {
  const long long d_in = ly.d_in, d_out = ly.d_out, g = ly.g, ng = ly.ng;
  const int nk = grid.n_clip;
  const OwcWs L = owc_ws_layout(d_in, d_out, g, nk, mode);
  char* base = (char*)ws;
  float* mn = (float*)(base + L.mn);
  float* mx = (float*)(base + L.mx);
  cudaError_t e = launch_group_minmax(ly, (float*)(base + L.pmn), (float*)(base + L.pmx), mn, mx, st);
  if (e != cudaSuccess) return e;
  double hg[256];
  const double lo = (double)grid.clip_lo, hi = (double)grid.clip_hi;
  for (int k = 0; k < nk; ++k) hg[k] = nk > 1 ? lo + ((hi - lo) * (double)k) / (double)(nk - 1) : 1.0;
  e = cudaMemcpyAsync(base + L.gammas, hg, sizeof(double) * nk, cudaMemcpyHostToDevice, st);  // pageable: staged before return
  if (e != cudaSuccess) return e;
  e = cudaMemsetAsync(base + L.ctr, 0, sizeof(owc::Counters), st);
  if (e != cudaSuccess) return e;

  owc::Params p{};
  p.H = ly.H; p.W = ly.W; p.wt = ly.wt; p.d_in = d_in; p.d_out = d_out; p.ldw = ly.ldw; p.g = g; p.ng = ng;
  p.L = ly.L; p.nk = nk; p.gammas = (const double*)(base + L.gammas); p.mn = mn; p.mx = mx; p.steps = steps;
  p.scale = scale; p.zero = zero; p.Q = Q; p.gamma_out = gamma_out;
  p.scratch = (double*)(base + L.scratch); p.scratch_per_cta = L.scratch_per_cta; p.cur = (int*)(base + L.cur);
  p.col_before = (double*)(base + L.col_before); p.col_after = (double*)(base + L.col_after);
  p.ctr = (owc::Counters*)(base + L.ctr);
  if (L.tc) {   // G = 2 H e and the column losses at the starting strengths
    ResidualSrc src{};
    src.W = ly.W; src.wt = ly.wt; src.ldw = ly.ldw; src.mn = mn; src.mx = mx; src.gamma = hg[nk - 1]; src.L = ly.L;
    src.use_gamma = 1; src.g = g; src.d_out = d_out;
    double* E = (double*)(base + L.E);
    e = launch_residual_f64(src, d_in, E, st);
    if (e != cudaSuccess) return e;
    e = gemm_tc_prepare_h(ly.H, d_in, kTcGradNH, base + L.hbuf, st);
    if (e != cudaSuccess) return e;
    p.Gext = (double*)(base + L.G); p.ldg = L.ldg;
    e = gemm_tc_run(base + L.hbuf, kTcGradNH, E, d_in, d_out, kTcGradNE, kTcGradSmax, 2.0, p.Gext, p.ldg, p.col_before,
                    base + L.ebuf, st);
    if (e != cudaSuccess) return e;
  }
  const unsigned ctas = (unsigned)(d_out < kOwcMaxCtas ? d_out : kOwcMaxCtas);
  // the production kernel keeps two tables of ng * n_clip doubles in shared memory; grids too fine for
  // that run the fixed-order kernel (slower, same result)
  const size_t smem = 2 * sizeof(double) * (size_t)ng * nk;
  if (mode == CDQ_MODE_FP64_VERIFY || smem > 160 * 1024) {
    p.Gext = nullptr;
    { owc::owc_cd_kernel<true><<<ctas, owc::NT, 0, st>>>(p); count_launch(); }
  } else {
    if (smem > 40 * 1024) {
      e = cudaFuncSetAttribute(owc::owc_cd_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
    }
    { owc::owc_cd_kernel<false><<<ctas, owc::NT, smem, st>>>(p); count_launch(); }
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (host_moves) {
    double* sums = (double*)(base + L.sums);
    e = launch_sum_f64(p.col_before, d_out, sums, st);
    if (e != cudaSuccess) return e;
    e = launch_sum_f64(p.col_after, d_out, sums + 1, st);
    if (e != cudaSuccess) return e;
    owc::Counters hc;
    double hs[2];
    e = cudaMemcpyAsync(&hc, p.ctr, sizeof(hc), cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return e;
    e = cudaMemcpyAsync(hs, sums, sizeof(hs), cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return e;
    e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return e;
    *host_moves = hc.moves; *host_before = hs[0]; *host_after = hs[1];
  }
  return cudaSuccess;
}

}  // namespace cdq
