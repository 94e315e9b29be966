// Greedy coordinate descent, batched over all output columns (paper: Algorithm 1 lines
// 4-8; Algorithm 4 for sub-channel grids; weight-unit form, see include/cdq.h).
//
// One CTA owns one column at a time (columns are handed out through an atomic counter).
// The column's whole state stays on chip for its T steps: the gradient g (fp64) and the
// codes q (packed bytes) live in registers, EPT coordinates per thread.  One step is
//   1. every thread holds the best move among its coordinates (scored in fp32);
//   2. warp argmin with two redux.sync, then one shared-memory exchange per CTA;
//   3. the winning row H[i*, :] is read once, contiguously (H is symmetric, so the
//      "column i*" of Algorithm 1 line 6 is row i*), 16 bytes per thread per load;
//   4. g += 2 d H[i*, :] in fp64, and each coordinate is re-scored in the same sweep.
// The best level of a coordinate is the clamped rounding of the vertex of its parabola
//   r = clamp(rint(q_i - g_i / (2 a_i H_ii)), 0, L),
// so the level scan of Algorithm 1 line 5 costs O(1) per coordinate.
#include <cstdio>
#include <cstdlib>

#include "common.cuh"
#include "cd_params.cuh"

namespace cdq {


// ---------------------------------------------------------------------------
__global__ void diag_kernel(const float* __restrict__ H, long long d_in, long long d_pad,
                            float* __restrict__ hdiag, float* __restrict__ half_inv) {
  const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (i >= d_pad) return;
  float h = 0.f, hi = 0.f;
  if (i < d_in) {
    h = H[i * d_in + i];
    hi = h > 0.f ? 0.5f / h : 0.f;
  }
  hdiag[i] = h;
  half_inv[i] = hi;
}

cudaError_t launch_diag(const float* H, long long d_in, long long d_pad, float* hdiag, float* half_inv,
                        cudaStream_t st) {
  diag_kernel<<<(unsigned)((d_pad + 255) / 256), 256, 0, st>>>(H, d_in, d_pad, hdiag, half_inv);
  return cudaGetLastError();
}

// dst[c][r] = src[r][c] for byte matrices with leading dimensions, 32x32 tiles through shared memory.
__global__ void transpose_u8_kernel(const unsigned char* __restrict__ src, long long rows, long long cols,
                                    long long ld_src, unsigned char* __restrict__ dst, long long ld_dst) {
  __shared__ unsigned char tile[32][33];
  const long long c0 = (long long)blockIdx.x * 32, r0 = (long long)blockIdx.y * 32;
  for (int rr = threadIdx.y; rr < 32; rr += blockDim.y) {
    const long long r = r0 + rr, c = c0 + threadIdx.x;
    tile[rr][threadIdx.x] = (r < rows && c < cols) ? src[r * ld_src + c] : 0;
  }
  __syncthreads();
  for (int cc = threadIdx.y; cc < 32; cc += blockDim.y) {
    const long long c = c0 + cc, r = r0 + threadIdx.x;
    if (c < cols && r < rows) dst[c * ld_dst + r] = tile[threadIdx.x][cc];
  }
}

cudaError_t launch_transpose_u8(const unsigned char* src, long long rows, long long cols, long long ld_src,
                                unsigned char* dst, long long ld_dst, cudaStream_t st) {
  dim3 grid((unsigned)((cols + 31) / 32), (unsigned)((rows + 31) / 32)), block(32, 8);
  transpose_u8_kernel<<<grid, block, 0, st>>>(src, rows, cols, ld_src, dst, ld_dst);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
__device__ __forceinline__ float4 ld_row4(const float* p) {
  float4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
               : "l"(p));
  return v;
}

// One CTA ("team") owns one column at a time.  Thread t holds chunks t, t + NT, t + 2 NT, ...
// of 4 consecutive coordinates; the gradient of the first RCH chunks lives in registers, that
// of the other NCH - RCH chunks in shared memory (two planes of double2, conflict-free).
// EXACT: d_in == 4 * NT * NCH, so no chunk needs a bounds test.
template <int NCH, int RCH, int MAXNT, int MINB, int SMODE, bool EXACT>
__global__ void __launch_bounds__(MAXNT, MINB) cd_fast_kernel(CdParams p) {
  constexpr int SCH = NCH - RCH;
  extern __shared__ __align__(16) unsigned char dyn_smem[];
  __shared__ unsigned s_key[2][32];
  __shared__ unsigned s_pk[2][32];
  __shared__ int s_col;

  const int tid = threadIdx.x, NT = blockDim.x;
  const int lane = tid & 31, warp = tid >> 5, nwarps = NT >> 5;
  const long long d_in = p.d_in;
  const int nchunks = (int)((d_in + 3) >> 2);
  const bool vec = EXACT || (d_in & 3) == 0;
  const float topf = kMagic + (float)p.L;

  auto group_of = [&](unsigned i) -> unsigned { return p.g == 1 ? i : __umulhi(i, p.gmagic); };
  double2* gs0 = reinterpret_cast<double2*>(dyn_smem);           // [SCH][NT] coordinates 0,1 of a chunk
  double2* gs1 = gs0 + (size_t)SCH * NT;                          // [SCH][NT] coordinates 2,3
  float2* ag_s = reinterpret_cast<float2*>(gs1 + (size_t)SCH * NT);  // [ng] (a, 1/a), grouped modes
  // kGroupFast: byte offset of this thread's first group entry and the stride between chunks
  const int g4 = SMODE == kGroupFast ? (int)(p.g >> 2) : 1;
  const float2* ag_mine = ag_s + (SMODE == kGroupFast ? tid / g4 : 0);
  const int ag_stride = SMODE == kGroupFast ? NT / g4 : 0;

  unsigned long long my_committed = 0, my_converged = 0;
  double my_dsum = 0.0;
  int buf = 0;

  for (;;) {
    __syncthreads();  // the previous column's use of shared memory is over
    if (tid == 0) s_col = atomicAdd(&p.ctr->next_col, 1);
    __syncthreads();
    const long long j = s_col;
    if (j >= p.d_out) break;

    // ---- column state ----
    float a_col = 1.f;
    double inv_a = 1.0;
    if (SMODE == kPerChannel) {
      a_col = p.scale[j];
      if (!(a_col > 0.f)) {  // constant column: its grid has one point, nothing can move
        ++my_converged;
        continue;
      }
      inv_a = 1.0 / (double)a_col;
    } else {
      // groups past the last real one (chunk slots beyond d_in) get a zero scale
      for (int t = tid; t < p.ag_count; t += NT) {
        const float a = t < p.ng ? p.scale[(long long)t * p.d_out + j] : 0.f;
        ag_s[t] = make_float2(a, a > 0.f ? 1.0f / a : 0.f);
      }
      __syncthreads();
    }
    double g[RCH > 0 ? 4 * RCH : 1];
    unsigned qp[NCH];
    {
      const double* gcol = p.G + j * p.ldg;
      const unsigned char* qcol = p.Qt + j * p.ldq;
#pragma unroll
      for (int k = 0; k < NCH; ++k) {
        const int chunk = tid + NT * k;
        double2 g0 = make_double2(0.0, 0.0), g1 = g0;
        qp[k] = 0;
        if (EXACT || chunk < nchunks) {
          g0 = *reinterpret_cast<const double2*>(gcol + (long long)chunk * 4);
          g1 = *reinterpret_cast<const double2*>(gcol + (long long)chunk * 4 + 2);
          qp[k] = *reinterpret_cast<const unsigned*>(qcol + (long long)chunk * 4);
        }
        if (!EXACT) {  // coordinates past d_in inside the last chunk: padding of the rows of G and Qt
          const long long i0 = (long long)chunk * 4;
          if (i0 + 1 >= d_in) { g0.y = 0.0; qp[k] &= 0x000000FFu; }
          if (i0 + 2 >= d_in) { g1.x = 0.0; qp[k] &= 0x0000FFFFu; }
          if (i0 + 3 >= d_in) { g1.y = 0.0; qp[k] &= 0x00FFFFFFu; }
        }
        g0.x *= inv_a; g0.y *= inv_a; g1.x *= inv_a; g1.y *= inv_a;
        if (k < RCH) {
          g[4 * k] = g0.x; g[4 * k + 1] = g0.y; g[4 * k + 2] = g1.x; g[4 * k + 3] = g1.y;
        } else {
          gs0[(k - RCH) * NT + tid] = g0;
          gs1[(k - RCH) * NT + tid] = g1;
        }
      }
    }

    // ---- descent ----
    // The first sweep only scores: it "applies" a step of size zero along row 0.
    long long step = 0;
    const float* rp = p.H;
    double c2 = 0.0;       // twice the step being applied (code units when per-channel)
    double col_dsum = 0.0;
    bool done = false;
    for (;;) {
      float4 row[NCH];
#pragma unroll
      for (int k = 0; k < NCH; ++k) {
        const int chunk = tid + NT * k;
        if (EXACT) row[k] = ld_row4(rp + (long long)chunk * 4);
        else {
          row[k] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (chunk < nchunks) {
            if (vec) row[k] = ld_row4(rp + (long long)chunk * 4);
            else {
              const long long i0 = (long long)chunk * 4;
              row[k].x = rp[i0];
              if (i0 + 1 < d_in) row[k].y = rp[i0 + 1];
              if (i0 + 2 < d_in) row[k].z = rp[i0 + 2];
              if (i0 + 3 < d_in) row[k].w = rp[i0 + 3];
            }
          }
        }
      }
      float best = 0.f, bpk = 0.f;
#pragma unroll
      for (int k = 0; k < NCH; ++k) {
        const int chunk = tid + NT * k;
        const float4 hd = __ldg(reinterpret_cast<const float4*>(p.hdiag) + chunk);
        const float4 hi = __ldg(reinterpret_cast<const float4*>(p.half_inv) + chunk);
        float a = 1.f, ia = 1.f;
        if (SMODE == kGroupFast) {
          const float2 ag = ag_mine[k * ag_stride];
          a = ag.x; ia = ag.y;
        }
        double gk[4];
        if (k < RCH) {
#pragma unroll
          for (int v = 0; v < 4; ++v) gk[v] = g[4 * (k < RCH ? k : 0) + v];
        } else {
          const double2 g0 = gs0[(k - RCH) * NT + tid], g1 = gs1[(k - RCH) * NT + tid];
          gk[0] = g0.x; gk[1] = g0.y; gk[2] = g1.x; gk[3] = g1.y;
        }
        const float hv[4] = {row[k].x, row[k].y, row[k].z, row[k].w};
        const float hdv[4] = {hd.x, hd.y, hd.z, hd.w};
        const float hiv[4] = {hi.x, hi.y, hi.z, hi.w};
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          const int e = 4 * k + v;
          if (SMODE == kGroupAny) {
            const unsigned i = (unsigned)chunk * 4u + v;
            const float2 ag = i < (unsigned)d_in ? ag_s[group_of(i)] : make_float2(0.f, 0.f);
            a = ag.x; ia = ag.y;
          }
          gk[v] = fma(c2, (double)hv[v], gk[v]);
          const float gf = (float)gk[v];
          const float qmf = __uint_as_float(__byte_perm(qp[k], kMagicBits, 0x7650 | v));  // kMagic + q
          // kMagic + rint(vertex of the coordinate's parabola), clamped to the grid
          float t = SMODE == kPerChannel ? fmaf(-gf, hiv[v], qmf) : fmaf(-gf, ia * hiv[v], qmf);
          t = fminf(fmaxf(t, kMagic), topf);
          const float dr = t - qmf;
          const float d = SMODE == kPerChannel ? dr : a * dr;
          const float dl = fmaf(d, hdv[v], gf) * d;
          if (dl < best) { best = dl; bpk = dr + (float)(e * 1024); }
        }
        if (k < RCH) {
#pragma unroll
          for (int v = 0; v < 4; ++v) g[4 * (k < RCH ? k : 0) + v] = gk[v];
        } else {
          gs0[(k - RCH) * NT + tid] = make_double2(gk[0], gk[1]);
          gs1[(k - RCH) * NT + tid] = make_double2(gk[2], gk[3]);
        }
      }
      if (step >= p.T) break;

      // team-wide argmin: (decrease, lowest coordinate, lowest level).  `best` is negative or
      // +0, so the complement of its bits orders the candidates; +0 becomes kNoMove.
      unsigned packed = kNoMove;
      if (best < 0.f) {
        const int ipk = (int)bpk;
        const int e = (ipk + 512) >> 10;
        const int drq = ipk - (e << 10);
        // (chunk slot, thread, coordinate in chunk) orders like the coordinate index
        packed = ((unsigned)(e >> 2) << 21) | ((unsigned)tid << 11) | ((unsigned)(e & 3) << 9) | (unsigned)(drq + 256);
      }
      // (a zero step scores -0 and the compiler may keep it as the running minimum: test the sign)
      unsigned key = best < 0.f ? ~__float_as_uint(best) : kNoMove;
      unsigned m = __reduce_min_sync(0xFFFFFFFFu, key);
      unsigned w = __reduce_min_sync(0xFFFFFFFFu, key == m ? packed : kNoMove);
      if (nwarps > 1) {
        if (lane == 0) { s_key[buf][warp] = m; s_pk[buf][warp] = w; }
        __syncthreads();
        key = lane < nwarps ? s_key[buf][lane] : kNoMove;
        packed = lane < nwarps ? s_pk[buf][lane] : kNoMove;
        m = __reduce_min_sync(0xFFFFFFFFu, key);
        w = __reduce_min_sync(0xFFFFFFFFu, key == m ? packed : kNoMove);
        buf ^= 1;
      }
      if (m == kNoMove) { done = true; break; }  // no move lowers the loss
      const int kstar = (int)(w >> 21), tstar = (int)((w >> 11) & 1023u), vstar = (int)((w >> 9) & 3u);
      const int dri = (int)(w & 511u) - 256;
      const int istar = 4 * (tstar + NT * kstar) + vstar;
      if ((unsigned)istar >= (unsigned)d_in) {  // cannot happen; never follow a bad row index
        if (tid == 0) atomicExch(p.status, (int)kFlagBadIndex);
        break;
      }
      if (tid == tstar) {
        const unsigned dq = (unsigned)dri << (8 * vstar);
#pragma unroll
        for (int k = 0; k < NCH; ++k)
          if (k == kstar) qp[k] += dq;
      }
      float astar = 1.f;
      if (SMODE != kPerChannel) astar = ag_s[group_of((unsigned)istar)].x;
      c2 = 2.0 * ((double)astar * (double)dri);
      rp = p.H + (long long)istar * d_in;
      if (tid == 0) col_dsum += (double)__uint_as_float(~m);
      ++step;
    }
    if (done) ++my_converged;
    my_committed += (unsigned long long)step;
    my_dsum += SMODE == kPerChannel ? col_dsum * ((double)a_col * (double)a_col) : col_dsum;

    // ---- write the codes back ----
    {
      unsigned char* qcol = p.Qt + j * p.ldq;
#pragma unroll
      for (int k = 0; k < NCH; ++k) {
        const int chunk = tid + NT * k;
        if (EXACT || chunk < nchunks) *reinterpret_cast<unsigned*>(qcol + (long long)chunk * 4) = qp[k];
      }
    }
  }

  // ---- statistics ----
  if (tid == 0) {
    if (my_dsum != 0.0) atomicAdd(&p.ctr->delta_sum, my_dsum);
    if (my_committed) atomicAdd(&p.ctr->committed, my_committed);
    if (my_converged) atomicAdd(&p.ctr->converged, my_converged);
  }
}

template <int NCH, int RCH, int MAXNT, int MINB, int SMODE, bool EXACT>
static cudaError_t launch_cd_cfg(CdParams p, int nt, cudaStream_t st) {
  p.ag_count = (int)p.ng;
  if (SMODE == kGroupFast) {
    const int g4 = (int)(p.g >> 2), slots = (nt * NCH + g4 - 1) / g4;
    if (slots > p.ag_count) p.ag_count = slots;
  }
  auto kern = cd_fast_kernel<NCH, RCH, MAXNT, MINB, SMODE, EXACT>;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const size_t smem = (size_t)(NCH - RCH) * nt * 2 * sizeof(double2) + (SMODE == kPerChannel ? 0 : sizeof(float2) * (size_t)p.ag_count);
  cudaError_t e;
  if (smem > 48 * 1024) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  int per_sm = 1;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, nt, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorInvalidConfiguration;
  long long blocks = (long long)sms * per_sm;
  if (blocks > p.d_out) blocks = p.d_out;
  kern<<<(unsigned)blocks, nt, smem, st>>>(p);
  return cudaGetLastError();
}

// Picks the scale mode and whether the team covers d_in exactly.
template <int NCH, int RCH, int MAXNT, int MINB>
static cudaError_t launch_cd_shape(const CdParams& p, int nt, cudaStream_t st) {
  const bool exact = p.d_in == 4ll * nt * NCH;
  int smode = kPerChannel;
  if (p.ng > 1) smode = ((p.g & 3) == 0 && nt % (int)(p.g >> 2) == 0) ? kGroupFast : kGroupAny;
  if (smode == kPerChannel)
    return exact ? launch_cd_cfg<NCH, RCH, MAXNT, MINB, kPerChannel, true>(p, nt, st)
                 : launch_cd_cfg<NCH, RCH, MAXNT, MINB, kPerChannel, false>(p, nt, st);
  if (smode == kGroupFast)
    return exact ? launch_cd_cfg<NCH, RCH, MAXNT, MINB, kGroupFast, true>(p, nt, st)
                 : launch_cd_cfg<NCH, RCH, MAXNT, MINB, kGroupFast, false>(p, nt, st);
  return launch_cd_cfg<NCH, RCH, MAXNT, MINB, kGroupAny, false>(p, nt, st);
}

long long cd_fast_pad(long long d_in) {
  // hdiag / half_inv are read in 16-byte pieces by every chunk slot of a team, so they are
  // padded to beyond the largest team footprint (at most 32 extra threads of 32 coordinates).
  return (d_in + 2048 + 255) / 256 * 256;
}

bool cd_fast_supported(long long d_in) { return d_in >= 1 && d_in <= 18432; }

cudaError_t launch_cd_fast(const Layer& ly, double* G, long long ldg, unsigned char* Qt, long long ldq,
                           const float* hdiag, const float* half_inv, long long steps_per_col, CdCounters* ctr,
                           cudaStream_t st) {
  CdParams p{};
  p.H = ly.H; p.d_in = ly.d_in; p.d_out = ly.d_out; p.G = G; p.ldg = ldg; p.Qt = Qt; p.ldq = ldq; p.scale = ly.scale;
  p.hdiag = hdiag; p.half_inv = half_inv; p.g = ly.g; p.ng = ly.ng; p.L = ly.L; p.T = steps_per_col; p.ctr = ctr;
  p.status = device_status_word();
  if (!p.status) return cudaErrorInvalidSymbol;
  p.gmagic = ly.g > 1 ? (unsigned)(((1ull << 32) + (unsigned long long)ly.g - 1) / (unsigned long long)ly.g) : 0u;
  // CDQ_CD_KERNEL=plain in the environment keeps the rows in registers (no bulk copies, no clusters)
  static const bool force_plain = [] { const char* e = getenv("CDQ_CD_KERNEL"); return e && e[0] == 'p'; }();
  if (!force_plain) {
    const cudaError_t e = launch_cd_tma(p, st);
    if (e != cudaErrorNotSupported) return e;
  }
  const long long d = ly.d_in;
  auto team = [&](int ept) { return (int)(((d + ept - 1) / ept + 31) / 32 * 32); };
  if (d <= 512) return launch_cd_shape<2, 2, 64, 8>(p, team(8), st);
  if (d <= 4096) return launch_cd_shape<4, 4, 256, 3>(p, team(16), st);
  if (d <= 8192) return launch_cd_shape<8, 8, 256, 2>(p, team(32), st);
  if (d <= 14336) return launch_cd_shape<8, 8, 448, 1>(p, team(32), st);
  return launch_cd_shape<8, 6, 576, 1>(p, team(32), st);
}

// ---------------------------------------------------------------------------
// Fixed-order fp64 version: the level scan of Algorithm 1 line 5 as written, no fused
// multiply-add, ties to the lowest coordinate then the lowest level.  One CTA per column,
// gradient in global memory.  Small layers only.
__global__ void __launch_bounds__(128) cd_verify_kernel(CdParams p) {
  __shared__ double s_delta[128];
  __shared__ int s_i[128];
  __shared__ int s_r[128];
  const long long j = blockIdx.x;
  const int tid = threadIdx.x;
  const long long d_in = p.d_in;
  double* g = p.G + j * p.ldg;
  unsigned char* q = p.Qt + j * p.ldq;
  unsigned long long moves = 0;
  double dsum = 0.0;
  bool done = false;
  for (long long step = 0; step < p.T; ++step) {
    double best = 0.0;
    int bi = -1, br = 0;
    for (long long i = tid; i < d_in; i += 128) {
      const double ai = (double)p.scale[(i / p.g) * p.d_out + j];
      const double hii = (double)p.H[i * d_in + i];
      const double gi = g[i];
      const int qi = q[i];
      for (int r = 0; r <= p.L; ++r) {
        if (r == qi) continue;
        const double d = __dmul_rn(ai, (double)(r - qi));
        const double delta = __dadd_rn(__dmul_rn(__dmul_rn(d, d), hii), __dmul_rn(d, gi));
        if (delta < best) { best = delta; bi = (int)i; br = r; }
      }
    }
    s_delta[tid] = best; s_i[tid] = bi; s_r[tid] = br;
    __syncthreads();
    for (int w = 64; w > 0; w >>= 1) {
      if (tid < w) {
        const double od = s_delta[tid + w];
        const int oi = s_i[tid + w];
        const bool take = oi >= 0 && (s_i[tid] < 0 || od < s_delta[tid] || (od == s_delta[tid] && oi < s_i[tid]));
        if (take) { s_delta[tid] = od; s_i[tid] = oi; s_r[tid] = s_r[tid + w]; }
      }
      __syncthreads();
    }
    const int istar = s_i[0], rstar = s_r[0];
    const double dstar = s_delta[0];
    __syncthreads();
    if (istar < 0) { done = true; break; }
    const double ai = (double)p.scale[(istar / p.g) * p.d_out + j];
    const double d = __dmul_rn(ai, (double)(rstar - (int)q[istar]));
    const double two_d = __dmul_rn(2.0, d);
    __syncthreads();
    if (tid == 0) q[istar] = (unsigned char)rstar;
    const float* row = p.H + (long long)istar * d_in;
    for (long long i = tid; i < d_in; i += 128) g[i] = __dadd_rn(g[i], __dmul_rn(two_d, (double)row[i]));
    ++moves;
    dsum += dstar;
    __syncthreads();
  }
  if (tid == 0) {
    atomicAdd(&p.ctr->committed, moves);
    if (done) atomicAdd(&p.ctr->converged, 1ull);
    atomicAdd(&p.ctr->delta_sum, dsum);
  }
}

cudaError_t launch_cd_verify(const Layer& ly, double* G, long long ldg, unsigned char* Qt, long long ldq,
                             long long steps_per_col, CdCounters* ctr, cudaStream_t st) {
  CdParams p{};
  p.H = ly.H; p.d_in = ly.d_in; p.d_out = ly.d_out; p.G = G; p.ldg = ldg; p.Qt = Qt; p.ldq = ldq; p.scale = ly.scale;
  p.g = ly.g; p.ng = ly.ng; p.L = ly.L; p.T = steps_per_col; p.ctr = ctr;
  cd_verify_kernel<<<(unsigned)ly.d_out, 128, 0, st>>>(p);
  return cudaGetLastError();
}

}  // namespace cdq
