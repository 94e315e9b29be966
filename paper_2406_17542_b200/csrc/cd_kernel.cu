// Greedy coordinate descent, batched over all output columns (paper: the loop of Algorithm 1;
// Algorithm 4 for sub-channel grids; weight-unit form, see include/cdq.h).
//
// One CTA owns one column at a time (columns are handed out through an atomic counter).
// The column's whole state stays on chip for its T steps: the gradient g (fp64) and the
// codes q (packed bytes) live in registers, EPT coordinates per thread.  One step is
//   1. every thread holds the best move among its coordinates (scored in fp32);
//   2. warp argmin with two redux.sync, then one shared-memory exchange per CTA;
//   3. the winning row H[i*, :] is read once, contiguously (H is symmetric, so the
//      "column i*" in the update of Algorithm 1 is row i*), 16 bytes per thread per load;
//   4. g += 2 d H[i*, :] in fp64, and each coordinate is re-scored in the same sweep.
// The best level of a coordinate is the clamped rounding of the vertex of its parabola
//   r = clamp(rint(q_i - g_i / (2 a_i H_ii)), 0, L),
// so the scan over the levels in Algorithm 1 costs O(1) per coordinate.
#include "common.cuh"
#include "cd_params.cuh"
#include "cd_sweep.cuh"

namespace cdq {


// ---------------------------------------------------------------------------
// Diagonal of H for the scoring arithmetic: hdiag = H_ii, hs = 0.5 / H_ii (0 for a dead feature
// and in the padding beyond d_in).
__global__ void diag_kernel(const float* __restrict__ H, long long d_in, long long d_pad,
                            float* __restrict__ hdiag, float* __restrict__ hs) {
  const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (i >= d_pad) return;
  float h = 0.f, w = 0.f;
  if (i < d_in) {
    h = H[i * d_in + i];
    if (!(h > 0.f)) h = 0.f;
    w = h > 0.f ? 0.5f / h : 0.f;
  }
  hdiag[i] = h;
  hs[i] = w;
}

cudaError_t launch_diag(const float* H, long long d_in, long long d_pad, float* hdiag, float* hs, cudaStream_t st) {
  { diag_kernel<<<(unsigned)((d_pad + 255) / 256), 256, 0, st>>>(H, d_in, d_pad, hdiag, hs); count_launch(); }
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
  { transpose_u8_kernel<<<grid, block, 0, st>>>(src, rows, cols, ld_src, dst, ld_dst); count_launch(); }
  return cudaGetLastError();
}

// col_loss[j] = 1/2 sum_i E[i][j] G[j][i]: with g = 2 H e the loss e^T H e (Eq. 1) of a column is half the dot
// product of its residual and its gradient.  One CTA per 32 columns, rows in ascending tiles of 32, every column's
// sum kept by one warp: the result does not depend on the launch shape.
__global__ void __launch_bounds__(256) loss_from_gradient_kernel(const double* __restrict__ E, const double* __restrict__ G,
                                                                 long long ldg, long long d_in, long long d_out,
                                                                 double* __restrict__ col_loss) {
  __shared__ double tile[32][33];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const long long j0 = (long long)blockIdx.x * 32;
  double acc[4] = {0.0, 0.0, 0.0, 0.0};
  for (long long i0 = 0; i0 < d_in; i0 += 32) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {   // E[i0 + ty + 8 r][j0 + tx], contiguous along the columns
      const long long i = i0 + ty + 8 * r, j = j0 + tx;
      tile[ty + 8 * r][tx] = (i < d_in && j < d_out) ? E[i * d_out + j] : 0.0;
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 4; ++r) {   // G[j0 + ty + 8 r][i0 + tx], contiguous along the rows
      const long long i = i0 + tx, j = j0 + ty + 8 * r;
      if (i < d_in && j < d_out) acc[r] += tile[tx][ty + 8 * r] * G[j * ldg + i];
    }
    __syncthreads();
  }
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    double v = acc[r];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    const long long j = j0 + ty + 8 * r;
    if (tx == 0 && j < d_out) col_loss[j] = 0.5 * v;
  }
}

cudaError_t launch_loss_from_gradient(const double* E, const double* G, long long ldg, long long d_in, long long d_out,
                                      double* col_loss, cudaStream_t st) {
  { loss_from_gradient_kernel<<<(unsigned)((d_out + 31) / 32), 256, 0, st>>>(E, G, ldg, d_in, d_out, col_loss); count_launch(); }
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
// of 4 consecutive coordinates: gradient (fp64) and codes (packed bytes) in registers.
// EXACT: d_in == 4 * NT * NCH, so no chunk needs a bounds test.
template <int NCH, int MAXNT, int MINB, int SMODE, bool EXACT>
__global__ void __launch_bounds__(MAXNT, MINB) cd_fast_kernel(CdParams p) {
  extern __shared__ __align__(16) unsigned char dyn_smem[];
  __shared__ __align__(8) uint2 s_exch[2][32];
  __shared__ int s_col;

  const int tid = threadIdx.x, NT = blockDim.x;
  const int lane = tid & 31, warp = tid >> 5, nwarps = NT >> 5;
  const long long d_in = p.d_in;
  const int nchunks = (int)((d_in + 3) >> 2);
  const bool vec = EXACT || (d_in & 3) == 0;
  const float top = kMagic + (float)p.L;

  auto group_of = [&](unsigned i) -> unsigned { return p.g == 1 ? i : __umulhi(i, p.gmagic); };
  float2* ag_s = reinterpret_cast<float2*>(dyn_smem);  // [ag_count] (a, 1/a), grouped modes
  const int g4 = SMODE == kGroupFast ? (int)(p.g >> 2) : 1;
  const float2* ag_mine = ag_s + (SMODE == kGroupFast ? tid / g4 : 0);
  const int ag_stride = SMODE == kGroupFast ? NT / g4 : 0;
  // scale (a, 1/a) of chunk slot k of this thread; kGroupAny keeps one scale per chunk only when
  // the group size is a multiple of 4, otherwise the launcher does not pick this kernel
  auto chunk_scale = [&](int k, float& a, float& ia) {
    a = 1.f; ia = 1.f;
    if (SMODE == kGroupFast) { const float2 ag = ag_mine[k * ag_stride]; a = ag.x; ia = ag.y; }
    if (SMODE == kGroupAny) {
      const unsigned i = (unsigned)(tid + NT * k) * 4u;
      const float2 ag = i < (unsigned)d_in ? ag_s[group_of(i)] : make_float2(0.f, 0.f);
      a = ag.x; ia = ag.y;
    }
  };

  unsigned long long my_committed = 0, my_converged = 0;
  double my_dsum = 0.0;
  int xbuf = 0;

  for (;;) {
    __syncthreads();  // the previous column's use of shared memory is over
    if (tid == 0) s_col = atomicAdd(&p.ctr->next_col, 1);
    __syncthreads();
    const long long j = s_col;
    if (j >= p.d_out) break;

    // ---- column state ----
    float a_col = 1.f;
    double gscale = 1.0;   // what the stored gradient is multiplied by on load
    if (SMODE == kPerChannel) {
      a_col = p.scale[j];
      if (!(a_col > 0.f)) {  // constant column: its grid has one point, nothing can move
        if (tid == 0) ++my_converged;
        continue;
      }
      gscale = 1.0 / (double)a_col;
    } else {
      // groups past the last real one (chunk slots beyond d_in) get a zero scale
      for (int t = tid; t < p.ag_count; t += NT) {
        const float a = t < p.ng ? p.scale[(long long)t * p.d_out + j] : 0.f;
        ag_s[t] = make_float2(a, a > 0.f ? 1.0f / a : 0.f);
      }
      __syncthreads();
    }
    double g[4 * NCH];
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
        g[4 * k] = g0.x * gscale; g[4 * k + 1] = g0.y * gscale; g[4 * k + 2] = g1.x * gscale; g[4 * k + 3] = g1.y * gscale;
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
      SweepBest sb;
      sb.init();
#pragma unroll
      for (int k = 0; k < NCH; ++k) {
        const int chunk = tid + NT * k;
        const float4 hd = __ldg(reinterpret_cast<const float4*>(p.hdiag) + chunk);
        const float4 hs = __ldg(reinterpret_cast<const float4*>(p.hs) + chunk);
        float a, ia;
        chunk_scale(k, a, ia);
        double gk[4] = {g[4 * k], g[4 * k + 1], g[4 * k + 2], g[4 * k + 3]};
        sweep_chunk<SMODE>(gk, row[k], hd, hs, qp[k], c2, a, ia, top, k, sb);
        g[4 * k] = gk[0]; g[4 * k + 1] = gk[1]; g[4 * k + 2] = gk[2]; g[4 * k + 3] = gk[3];
      }

      if (step >= p.T) break;

      // ---- team-wide argmin: (decrease, lowest coordinate, lowest level) ----
      unsigned key, packed;
      sweep_candidate(sb, tid, key, packed);
      unsigned m = __reduce_min_sync(0xFFFFFFFFu, key);
      unsigned w = __reduce_min_sync(0xFFFFFFFFu, key == m ? packed : kNoMove);
      if (nwarps > 1) {
        if (lane == 0) s_exch[xbuf][warp] = make_uint2(m, w);
        __syncthreads();
        const uint2 x = lane < nwarps ? s_exch[xbuf][lane] : make_uint2(kNoMove, kNoMove);
        m = __reduce_min_sync(0xFFFFFFFFu, x.x);
        w = __reduce_min_sync(0xFFFFFFFFu, x.x == m ? x.y : kNoMove);
        xbuf ^= 1;
      } else {
        __syncwarp();
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
    if (tid == 0) {
      if (done) ++my_converged;
      my_committed += (unsigned long long)step;
      my_dsum += SMODE == kPerChannel ? col_dsum * ((double)a_col * (double)a_col) : col_dsum;
    }

    // ---- write the codes back, and the gradient of the result (weight units) ----
    {
      unsigned char* qcol = p.Qt + j * p.ldq;
      double* gcol = p.G + j * p.ldg;
      const double ga = SMODE == kPerChannel ? (double)a_col : 1.0;
#pragma unroll
      for (int k = 0; k < NCH; ++k) {
        const int chunk = tid + NT * k;
        if (EXACT || chunk < nchunks) {
          *reinterpret_cast<unsigned*>(qcol + (long long)chunk * 4) = qp[k];
          *reinterpret_cast<double2*>(gcol + (long long)chunk * 4) = make_double2(g[4 * k] * ga, g[4 * k + 1] * ga);
          *reinterpret_cast<double2*>(gcol + (long long)chunk * 4 + 2) = make_double2(g[4 * k + 2] * ga, g[4 * k + 3] * ga);
        }
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

template <int NCH, int MAXNT, int MINB, int SMODE, bool EXACT>
static cudaError_t launch_cd_cfg(CdParams p, int nt, cudaStream_t st) {
  p.ag_count = (int)p.ng;
  if (SMODE == kGroupFast) {
    const int g4 = (int)(p.g >> 2), slots = (nt * NCH + g4 - 1) / g4;
    if (slots > p.ag_count) p.ag_count = slots;
  }
  auto kern = cd_fast_kernel<NCH, MAXNT, MINB, SMODE, EXACT>;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const size_t smem = SMODE == kPerChannel ? 0 : sizeof(float2) * (size_t)p.ag_count;
  cudaError_t e;
  if (smem > 32 * 1024) {   // the 48 KB that need no opt-in include the kernel's static shared memory
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  int per_sm = 1;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, nt, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorInvalidConfiguration;
  long long blocks = (long long)sms * per_sm;
  if (blocks > p.d_out) blocks = p.d_out;
  { kern<<<(unsigned)blocks, nt, smem, st>>>(p); count_launch(); }
  return cudaGetLastError();
}

// Picks the scale mode and whether the team covers d_in exactly.
template <int NCH, int MAXNT, int MINB>
static cudaError_t launch_cd_shape(const CdParams& p, int nt, cudaStream_t st) {
  const bool exact = p.d_in == 4ll * nt * NCH;
  const int smode = cd_scale_mode(p, nt);
  if (smode < 0) return cudaErrorNotSupported;
  if (smode == kPerChannel)
    return exact ? launch_cd_cfg<NCH, MAXNT, MINB, kPerChannel, true>(p, nt, st)
                 : launch_cd_cfg<NCH, MAXNT, MINB, kPerChannel, false>(p, nt, st);
  if (smode == kGroupFast)
    return exact ? launch_cd_cfg<NCH, MAXNT, MINB, kGroupFast, true>(p, nt, st)
                 : launch_cd_cfg<NCH, MAXNT, MINB, kGroupFast, false>(p, nt, st);
  return launch_cd_cfg<NCH, MAXNT, MINB, kGroupAny, false>(p, nt, st);
}

long long cd_fast_pad(long long d_in) {
  // hdiag / half_inv are read in 16-byte pieces by every chunk slot of a team, so they are
  // padded to beyond the largest team footprint (at most 32 extra threads of 32 coordinates).
  return (d_in + 2048 + 255) / 256 * 256;
}

// The fast kernels keep one scale per chunk of 4 coordinates, so grouped grids need a group
// size that is a multiple of 4 (any group size runs in the verification mode).
bool cd_fast_supported(long long d_in, long long g) {
  return d_in >= 1 && d_in <= 18432 && (g == d_in || (g & 3) == 0);
}

// The bf16-row descent runs in the kernel that stages its rows through shared memory: d_in > 2048 (shorter rows
// are L2-served and gain nothing), rows 16-byte aligned as bf16.
bool cd_rows16_supported(long long d_in, long long g) {
  return cd_fast_supported(d_in, g) && d_in > 2048 && (d_in & 7) == 0;
}

__global__ void round_rows_bf16_kernel(const float* __restrict__ H, long long d_in, __nv_bfloat16* __restrict__ H16,
                                       float* __restrict__ Hr) {
  const long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (idx >= d_in * d_in) return;
  const float h = H[idx];
  const __nv_bfloat16 b = __float2bfloat16_rn(h);
  H16[idx] = b;
  Hr[idx] = (idx / d_in == idx % d_in) ? h : __bfloat162float(b);
}

cudaError_t launch_round_rows_bf16(const float* H, long long d_in, __nv_bfloat16* H16, float* Hr, cudaStream_t st) {
  const long long total = d_in * d_in;
  { round_rows_bf16_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(H, d_in, H16, Hr); count_launch(); }
  return cudaGetLastError();
}

cudaError_t launch_cd_fast(const Layer& ly, const __nv_bfloat16* H16, double* G, long long ldg, unsigned char* Qt,
                           long long ldq, const float* hdiag, const float* hs, long long steps_per_col,
                           CdCounters* ctr, cudaStream_t st) {
  CdParams p{};
  p.H = ly.H; p.H16 = H16; p.d_in = ly.d_in; p.d_out = ly.d_out; p.G = G; p.ldg = ldg; p.Qt = Qt; p.ldq = ldq; p.scale = ly.scale;
  p.hdiag = hdiag; p.hs = hs; p.g = ly.g; p.ng = ly.ng; p.L = ly.L; p.T = steps_per_col; p.ctr = ctr;
  p.status = device_status_word();
  if (!p.status) return cudaErrorInvalidSymbol;
  p.gmagic = ly.g > 1 ? (unsigned)(((1ull << 32) + (unsigned long long)ly.g - 1) / (unsigned long long)ly.g) : 0u;
  const long long d = ly.d_in;
  if (steps_per_col <= 0) return cudaSuccess;   // nothing to do: the counters stay zero, the codes untouched
  // short rows are quickest as plain loads into registers, longer ones as bulk copies into shared memory
  // (measured crossover: 1536 entries 2.0 against 2.5 ms, 1792 entries 11.5 against 10.8, 2048 entries 52.0 against 45.3)
  if (d > 1536) {
    const cudaError_t e = launch_cd_tma(p, st);
    if (e != cudaErrorNotSupported) return e;
  }
  if (H16) return cudaErrorNotSupported;
  auto team = [&](int ept) { return (int)(((d + ept - 1) / ept + 31) / 32 * 32); };
  if (d <= 512) return launch_cd_shape<2, 64, 8>(p, team(8), st);
  if (d <= 4096) return launch_cd_shape<4, 256, 3>(p, team(16), st);
  if (d <= 8192) return launch_cd_shape<8, 256, 2>(p, team(32), st);
  if (d <= 14336) return launch_cd_shape<8, 448, 1>(p, team(32), st);
  return launch_cd_shape<8, 576, 1>(p, team(32), st);
}

// ---------------------------------------------------------------------------
// Fixed-order fp64 version: the scan over the levels of Algorithm 1 as written, no fused
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
  { cd_verify_kernel<<<(unsigned)ly.d_out, 128, 0, st>>>(p); count_launch(); }
  return cudaGetLastError();
}

}  // namespace cdq
