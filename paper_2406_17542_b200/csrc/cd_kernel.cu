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

#include "common.cuh"

namespace cdq {

struct CdParams {
  const float* H;
  long long d_in, d_out;
  double* G;            // [d_out, ldg]
  long long ldg;
  unsigned char* Qt;    // [d_out, d_in] (transposed codes)
  const float* scale;   // [ng, d_out]
  const float* hdiag;   // [d_in_pad] H_ii (0 beyond d_in)
  const float* half_inv;  // [d_in_pad] 0.5 / H_ii (0 where H_ii <= 0 and beyond d_in)
  long long g, ng;
  int L;
  long long T;
  CdCounters* ctr;
};

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

// dst[c][r] = src[r][c] for byte matrices, 32x32 tiles through shared memory.
__global__ void transpose_u8_kernel(const unsigned char* __restrict__ src, long long rows, long long cols,
                                    unsigned char* __restrict__ dst) {
  __shared__ unsigned char tile[32][33];
  const long long c0 = (long long)blockIdx.x * 32, r0 = (long long)blockIdx.y * 32;
  for (int rr = threadIdx.y; rr < 32; rr += blockDim.y) {
    const long long r = r0 + rr, c = c0 + threadIdx.x;
    tile[rr][threadIdx.x] = (r < rows && c < cols) ? src[r * cols + c] : 0;
  }
  __syncthreads();
  for (int cc = threadIdx.y; cc < 32; cc += blockDim.y) {
    const long long c = c0 + cc, r = r0 + threadIdx.x;
    if (c < cols && r < rows) dst[c * rows + r] = tile[threadIdx.x][cc];
  }
}

cudaError_t launch_transpose_u8(const unsigned char* src, long long rows, long long cols, unsigned char* dst,
                                cudaStream_t st) {
  dim3 grid((unsigned)((cols + 31) / 32), (unsigned)((rows + 31) / 32)), block(32, 8);
  transpose_u8_kernel<<<grid, block, 0, st>>>(src, rows, cols, dst);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
__device__ __forceinline__ unsigned order_key(float x) {
  const unsigned u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
constexpr unsigned kKeyZero = 0x80000000u;  // order_key(+0.0f)
constexpr float kMagic = 12582912.0f;       // 1.5 * 2^23: adding it rounds to an integer
constexpr unsigned kMagicBits = 0x4B400000u;

__device__ __forceinline__ float4 ld_row4(const float* p) {
  float4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
               : "l"(p));
  return v;
}

template <int EPT, int MAXNT, bool GROUPED>
__global__ void __launch_bounds__(MAXNT) cd_fast_kernel(CdParams p) {
  constexpr int NCH = EPT / 4;
  extern __shared__ float a_s[];  // [ng] scales of the current column (GROUPED only)
  __shared__ unsigned s_key[2][32];
  __shared__ unsigned s_pk[2][32];
  __shared__ int s_col;

  const int tid = threadIdx.x, NT = blockDim.x;
  const int lane = tid & 31, warp = tid >> 5, nwarps = NT >> 5;
  const long long d_in = p.d_in;
  const int nchunks = (int)((d_in + 3) >> 2);
  const bool vec = (d_in & 3) == 0;
  // a 4-coordinate chunk lies inside one group unless the group size is not a multiple of 4
  const bool chunk_scale = !GROUPED || (p.g & 3) == 0;
  const float topf = kMagic + (float)p.L;

  unsigned long long my_committed = 0, my_converged = 0;
  double my_dsum = 0.0;
  int buf = 0;

  for (;;) {
    __syncthreads();  // previous column's use of shared memory is over
    if (tid == 0) s_col = atomicAdd(&p.ctr->next_col, 1);
    __syncthreads();
    const long long j = s_col;
    if (j >= p.d_out) break;
#ifdef CDQ_CD_CHECKED
    if (j < 0) { if (tid == 0) printf("cd_fast: bad column %lld\n", j); break; }
#endif

    // ---- column state ----
    double g[EPT];
    unsigned qp[NCH];
    float ak[GROUPED ? NCH : 1], iak[GROUPED ? NCH : 1];
    if (GROUPED) {
      for (long long t = tid; t < p.ng; t += NT) a_s[t] = p.scale[t * p.d_out + j];
      __syncthreads();
    }
    const float a_col = GROUPED ? 0.f : p.scale[j];
    const float ia_col = (!GROUPED && a_col > 0.f) ? 1.0f / a_col : 0.f;
#pragma unroll
    for (int k = 0; k < NCH; ++k) {
      const int chunk = tid + NT * k;
      const long long i0 = (long long)chunk * 4;
      qp[k] = 0;
#pragma unroll
      for (int v = 0; v < 4; ++v) g[4 * k + v] = 0.0;
      if (chunk < nchunks) {
        if (vec) {
          const double2 g0 = *reinterpret_cast<const double2*>(p.G + j * p.ldg + i0);
          const double2 g1 = *reinterpret_cast<const double2*>(p.G + j * p.ldg + i0 + 2);
          g[4 * k] = g0.x; g[4 * k + 1] = g0.y; g[4 * k + 2] = g1.x; g[4 * k + 3] = g1.y;
          qp[k] = *reinterpret_cast<const unsigned*>(p.Qt + j * d_in + i0);
        } else {
#pragma unroll
          for (int v = 0; v < 4; ++v)
            if (i0 + v < d_in) {
              g[4 * k + v] = p.G[j * p.ldg + i0 + v];
              qp[k] |= (unsigned)p.Qt[j * d_in + i0 + v] << (8 * v);
            }
        }
      }
      if (GROUPED) {
        const long long gi = i0 < d_in ? i0 / p.g : 0;
        ak[k] = a_s[gi];
        iak[k] = ak[k] > 0.f ? 1.0f / ak[k] : 0.f;
      }
    }

    // ---- descent ----
    long long step = 0;
    int istar = 0, dri = 0;
    double c2 = 0.0, dd = 0.0;  // 2 d and d of the move being applied
    bool have_move = false;
    bool done = false;
    for (;;) {
      // sweep: apply the pending move (if any) and re-score every coordinate
      float4 row[NCH];
      const int cstar = istar >> 2, vstar = istar & 3;
      if (have_move) {
        const float* rp = p.H + (long long)istar * d_in;
#pragma unroll
        for (int k = 0; k < NCH; ++k) {
          const int chunk = tid + NT * k;
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
        float a = GROUPED ? ak[k] : a_col;
        float ia = GROUPED ? iak[k] : ia_col;
        const float hv[4] = {have_move ? row[k].x : 0.f, have_move ? row[k].y : 0.f,
                             have_move ? row[k].z : 0.f, have_move ? row[k].w : 0.f};
        const float hdv[4] = {hd.x, hd.y, hd.z, hd.w};
        const float hiv[4] = {hi.x, hi.y, hi.z, hi.w};
        if (have_move && chunk == cstar) {
          // this thread owns the moved coordinate: exact decrease, then the new code
#pragma unroll
          for (int v = 0; v < 4; ++v)
            if (v == vstar) my_dsum += dd * (dd * (double)hv[v] + g[4 * k + v]);
          qp[k] += (unsigned)dri << (8 * vstar);
        }
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          const int e = 4 * k + v;
          if (GROUPED && !chunk_scale) {  // rare layout: look the scale up per coordinate
            const long long i = (long long)chunk * 4 + v;
            a = i < d_in ? a_s[i / p.g] : 0.f;
            ia = a > 0.f ? 1.0f / a : 0.f;
          }
          if (have_move) g[e] = fma(c2, (double)hv[v], g[e]);
          const float gf = (float)g[e];
          const float qmf = __uint_as_float(__byte_perm(qp[k], kMagicBits, 0x7650 | v));  // kMagic + q
          float t = fmaf(-gf, ia * hiv[v], qmf);   // kMagic + rint(vertex)
          t = fminf(fmaxf(t, kMagic), topf);
          const float dr = t - qmf;
          const float d = a * dr;
          const float dl = fmaf(d, hdv[v], gf) * d;
          if (dl < best) { best = dl; bpk = dr + (float)(e * 1024); }
        }
      }
      if (have_move) { ++step; ++my_committed; }
      if (step >= p.T) break;

      // CTA-wide argmin: (decrease, lowest coordinate, lowest level)
      unsigned packed = 0xFFFFFFFFu;
      if (best < 0.f) {
        const int ipk = (int)bpk;
        const int e = (ipk + 512) >> 10;
        const int drq = ipk - (e << 10);
        const int i = 4 * (tid + NT * (e >> 2)) + (e & 3);
        packed = ((unsigned)i << 9) | (unsigned)(drq + 256);
      }
      // a thread without an improving move reports exactly +0 (the compiler may have turned the
      // running minimum into a min instruction, which can leave -0 behind)
      unsigned key = best < 0.f ? order_key(best) : kKeyZero;
      unsigned m = __reduce_min_sync(0xFFFFFFFFu, key);
      unsigned w = __reduce_min_sync(0xFFFFFFFFu, key == m ? packed : 0xFFFFFFFFu);
      if (nwarps > 1) {
        if (lane == 0) { s_key[buf][warp] = m; s_pk[buf][warp] = w; }
        __syncthreads();
        key = lane < nwarps ? s_key[buf][lane] : 0xFFFFFFFFu;
        packed = lane < nwarps ? s_pk[buf][lane] : 0xFFFFFFFFu;
        m = __reduce_min_sync(0xFFFFFFFFu, key);
        w = __reduce_min_sync(0xFFFFFFFFu, key == m ? packed : 0xFFFFFFFFu);
        buf ^= 1;
      }
      if (m >= kKeyZero) { done = true; break; }  // no move lowers the loss
      istar = (int)(w >> 9);
      dri = (int)(w & 511u) - 256;
#ifdef CDQ_CD_CHECKED
      if (istar < 0 || istar >= d_in || dri == 0 || dri > p.L || dri < -p.L) {
        if (tid == 0) printf("cd_fast: bad winner col %lld step %lld m %08x w %08x istar %d dri %d\n", j, step, m, w,
                             istar, dri);
        break;
      }
#endif
      const float astar = GROUPED ? a_s[istar / p.g] : a_col;
      dd = (double)astar * (double)dri;
      c2 = 2.0 * dd;
      have_move = true;
    }
    if (done) ++my_converged;

    // ---- write the codes back ----
#pragma unroll
    for (int k = 0; k < NCH; ++k) {
      const int chunk = tid + NT * k;
      const long long i0 = (long long)chunk * 4;
      if (chunk < nchunks) {
        if (vec) *reinterpret_cast<unsigned*>(p.Qt + j * d_in + i0) = qp[k];
        else {
#pragma unroll
          for (int v = 0; v < 4; ++v)
            if (i0 + v < d_in) p.Qt[j * d_in + i0 + v] = (unsigned char)(qp[k] >> (8 * v));
        }
      }
    }
  }

  // ---- statistics ----
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) my_dsum += __shfl_xor_sync(0xFFFFFFFFu, my_dsum, o);
  if (lane == 0 && my_dsum != 0.0) atomicAdd(&p.ctr->delta_sum, my_dsum);
  if (tid == 0) {
    if (my_committed) atomicAdd(&p.ctr->committed, my_committed);
    if (my_converged) atomicAdd(&p.ctr->converged, my_converged);
  }
}

template <int EPT, int MAXNT>
static cudaError_t launch_cd_fast_t(const CdParams& p, int nt, bool grouped, cudaStream_t st) {
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const size_t smem = grouped ? sizeof(float) * (size_t)p.ng : 0;
  int per_sm = 1;
  cudaError_t e;
  if (grouped) {
    if (smem > 48 * 1024) {
      e = cudaFuncSetAttribute(cd_fast_kernel<EPT, MAXNT, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
    }
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, cd_fast_kernel<EPT, MAXNT, true>, nt, smem);
  } else {
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, cd_fast_kernel<EPT, MAXNT, false>, nt, smem);
  }
  if (e != cudaSuccess) return e;
  if (per_sm < 1) per_sm = 1;
  long long blocks = (long long)sms * per_sm;
  if (blocks > p.d_out) blocks = p.d_out;
  if (grouped) cd_fast_kernel<EPT, MAXNT, true><<<(unsigned)blocks, nt, smem, st>>>(p);
  else cd_fast_kernel<EPT, MAXNT, false><<<(unsigned)blocks, nt, smem, st>>>(p);
  return cudaGetLastError();
}

long long cd_fast_pad(long long d_in) {
  // hdiag / half_inv are read in 16-byte pieces by every thread slot of a team, so they are
  // padded to beyond the largest team footprint (threads are a multiple of 32, 32 slots each).
  return (d_in + 2048 + 255) / 256 * 256;
}

bool cd_fast_supported(long long d_in) { return d_in >= 1 && d_in <= 18432; }

cudaError_t launch_cd_fast(const Layer& ly, double* G, long long ldg, unsigned char* Qt, const float* hdiag,
                           const float* half_inv, long long steps_per_col, CdCounters* ctr, cudaStream_t st) {
  CdParams p{};
  p.H = ly.H; p.d_in = ly.d_in; p.d_out = ly.d_out; p.G = G; p.ldg = ldg; p.Qt = Qt; p.scale = ly.scale;
  p.hdiag = hdiag; p.half_inv = half_inv; p.g = ly.g; p.ng = ly.ng; p.L = ly.L; p.T = steps_per_col; p.ctr = ctr;
  const bool grouped = ly.ng > 1;
  const long long d = ly.d_in;
  auto team = [&](int ept) { return (int)(((d + ept - 1) / ept + 31) / 32 * 32); };
  if (d <= 512) return launch_cd_fast_t<8, 64>(p, team(8), grouped, st);
  if (d <= 4096) return launch_cd_fast_t<16, 256>(p, team(16), grouped, st);
  if (d <= 8192) return launch_cd_fast_t<32, 256>(p, team(32), grouped, st);
  if (d <= 14336) return launch_cd_fast_t<32, 448>(p, team(32), grouped, st);
  return launch_cd_fast_t<32, 576>(p, team(32), grouped, st);
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
  unsigned char* q = p.Qt + j * d_in;
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

cudaError_t launch_cd_verify(const Layer& ly, double* G, long long ldg, unsigned char* Qt, long long steps_per_col,
                             CdCounters* ctr, cudaStream_t st) {
  CdParams p{};
  p.H = ly.H; p.d_in = ly.d_in; p.d_out = ly.d_out; p.G = G; p.ldg = ldg; p.Qt = Qt; p.scale = ly.scale;
  p.g = ly.g; p.ng = ly.ng; p.L = ly.L; p.T = steps_per_col; p.ctr = ctr;
  cd_verify_kernel<<<(unsigned)ly.d_out, 128, 0, st>>>(p);
  return cudaGetLastError();
}

}  // namespace cdq
