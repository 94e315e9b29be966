// Block coordinate descent with random blocks of two coordinates, batched over all output
// columns (paper: Algorithm 2; Algorithm 5 for sub-channel grids; weight-unit form).
//
// Step t of column j cuts the coordinates into d_in / 2 pairs by a counter-based bijection
// of {0..d_in-1} keyed by (seed, j, t); every pair (i, m) is scored over all (L+1)^2
// assignments of levels,
//   change = d_i^2 H_ii + 2 d_i d_m H_im + d_m^2 H_mm + d_i g_i + d_m g_m,  d = a (r - q),
// the most negative change of the step is applied and g += 2 d_i H[i, :] + 2 d_m H[m, :].
//
// One CTA owns one column at a time.  Pairs touch the gradient and the codes at random, so
// both live in shared memory (gradient fp64, 8 bytes per coordinate; codes 1 byte); the rows
// of H stream through registers, and the off-diagonal entry H_im of every pair of step t + 1
// is gathered while step t is applied (the partition does not depend on the state).
// The scan over the (L+1)^2 assignments takes one pass over the levels of the lower
// coordinate; for each, the best level of the other is the clamped rounding of the vertex of
// its parabola, as in the greedy descent.
#include <cstdio>
#include <cstdlib>

#include "common.cuh"
#include "cd_params.cuh"

namespace cdq {

// ---------------------------------------------------------------------------
// The partition: x -> pi(x), three rounds of (odd multiply + add) mod 2^b and xor-shift on
// b = ceil(log2 d_in) bits, keyed per (seed, column, step); values >= d_in walk the cycle
// until they fall below d_in (a bijection maps the cycle back to its start, so this ends).
__host__ __device__ __forceinline__ unsigned long long splitmix64(unsigned long long z) {
  z += 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

struct BcdKeys {
  unsigned mul[3], add[3];  // the low 32 bits decide a result of at most 16 bits
};

__device__ __forceinline__ BcdKeys bcd_keys(unsigned long long base, long long t) {
  BcdKeys k;
#pragma unroll
  for (int r = 0; r < 3; ++r) {
    const unsigned long long key = splitmix64(base ^ (((unsigned long long)t << 2) | (unsigned long long)r));
    k.mul[r] = (unsigned)(2ull * key + 1ull);
    k.add[r] = (unsigned)(key >> 33);
  }
  return k;
}

__device__ __forceinline__ unsigned bcd_perm(unsigned x, unsigned d_in, unsigned mask, int s, const BcdKeys& k) {
  unsigned v = x;
  do {
#pragma unroll
    for (int r = 0; r < 3; ++r) {
      v = (v * k.mul[r] + k.add[r]) & mask;
      v ^= v >> s;
    }
  } while (v >= d_in);
  return v;
}

struct BcdShape {
  unsigned mask;
  int shift;
};
static BcdShape bcd_shape(long long d_in) {
  int b = 0;
  while ((1ll << b) < d_in) ++b;
  BcdShape s;
  s.mask = (unsigned)((1ull << b) - 1);
  s.shift = b / 2 > 1 ? b / 2 : 1;
  return s;
}

__device__ __forceinline__ float ld_nc_f32(const float* p) {
  float v;
  asm volatile("ld.global.nc.L1::no_allocate.f32 %0, [%1];" : "=f"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ float2 ld_row2(const float* p) {
  float2 v;
  asm volatile("ld.global.nc.L1::no_allocate.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "l"(p));
  return v;
}

// ---------------------------------------------------------------------------
// PPT: pairs per thread (pair u = tid + NT * slot).  g_in_smem == 0: the gradient stays in
// its global-memory column (layers whose column does not fit in shared memory).
// a_in_smem == 0: the group scales are read from global memory.
template <int PPT, int MAXNT, int MINB>
__global__ void __launch_bounds__(MAXNT, MINB)
bcd2_kernel(CdParams p, unsigned long long seed, BcdShape shape, int g_in_smem, int a_in_smem) {
  extern __shared__ __align__(16) unsigned char dyn_smem[];
  __shared__ __align__(16) uint4 s_exch[2][32];
  __shared__ int s_col;

  const int tid = threadIdx.x, NT = blockDim.x;
  const int lane = tid & 31, warp = tid >> 5, nwarps = NT >> 5;
  const unsigned d_in = (unsigned)p.d_in;
  const unsigned nb = d_in >> 1;
  const float Lf = (float)p.L;

  // shared memory: [gradient, 8 ldg bytes][codes, ldg bytes rounded to 16][scales, 4 ng bytes]
  double* g_smem = reinterpret_cast<double*>(dyn_smem);
  unsigned char* q_s = dyn_smem + (g_in_smem ? sizeof(double) * (size_t)p.ldg : 0);
  float* a_smem = reinterpret_cast<float*>(q_s + ((p.ldg + 15) / 16) * 16);
  auto group_of = [&](unsigned i) -> unsigned { return p.g == 1 ? i : __umulhi(i, p.gmagic); };

  unsigned long long my_moves = 0;
  double my_dsum = 0.0;
  int xbuf = 0;

  for (;;) {
    __syncthreads();  // the previous column's use of shared memory is over
    if (tid == 0) s_col = atomicAdd(&p.ctr->next_col, 1);
    __syncthreads();
    const long long j = s_col;
    if (j >= p.d_out) break;

    // ---- column state ----
    double* g_s = g_in_smem ? g_smem : p.G + j * p.ldg;
    const float* a_ptr = a_in_smem ? a_smem : p.scale + j;
    const long long a_stride = a_in_smem ? 1 : p.d_out;
    if (g_in_smem) {
      const double* gcol = p.G + j * p.ldg;
      for (unsigned i = tid; i < d_in; i += NT) g_s[i] = gcol[i];
    }
    {
      const unsigned char* qcol = p.Qt + j * p.ldq;
      for (unsigned i = tid; i < d_in; i += NT) q_s[i] = qcol[i];
    }
    if (a_in_smem)
      for (int t = tid; t < (int)p.ng; t += NT) a_smem[t] = p.scale[(long long)t * p.d_out + j];
    __syncthreads();
    auto scale_of = [&](unsigned i) -> float { return a_ptr[(long long)group_of(i) * a_stride]; };

    const unsigned long long base = splitmix64(seed ^ splitmix64((unsigned long long)j));
    unsigned idx[PPT];   // m0 | m1 << 16, m0 < m1
    float h01[PPT];
    auto draw = [&](long long t) {
      const BcdKeys keys = bcd_keys(base, t);
#pragma unroll
      for (int s = 0; s < PPT; ++s) {
        const unsigned u = (unsigned)tid + (unsigned)NT * s;
        idx[s] = 0; h01[s] = 0.f;
        if (u < nb) {
          unsigned m0 = bcd_perm(2 * u, d_in, shape.mask, shape.shift, keys);
          unsigned m1 = bcd_perm(2 * u + 1, d_in, shape.mask, shape.shift, keys);
          if (m1 < m0) { const unsigned x = m0; m0 = m1; m1 = x; }
          idx[s] = m0 | (m1 << 16);
          h01[s] = ld_nc_f32(p.H + (size_t)m0 * d_in + m1);
        }
      }
    };

    double col_dsum = 0.0;
    long long moves = 0;
    bool bad = false;
    if (p.T > 0) draw(0);
    for (long long t = 0; t < p.T; ++t) {
      // ---- best move of every pair of this thread ----
      float best = 0.f;
      unsigned bpk = kNoMove, bextra = 0;
#pragma unroll
      for (int s = 0; s < PPT; ++s) {
        const unsigned u = (unsigned)tid + (unsigned)NT * s;
        if (u >= nb) continue;
        const unsigned m0 = idx[s] & 0xFFFFu, m1 = idx[s] >> 16;
        const float g0 = (float)g_s[m0], g1 = (float)g_s[m1];
        const int q0 = q_s[m0], q1 = q_s[m1];
        const float a0 = scale_of(m0), a1 = scale_of(m1);
        const float H00 = __ldg(p.hdiag + m0), H11 = __ldg(p.hdiag + m1);
        const float w1 = a1 > 0.f ? __ldg(p.hs + m1) / a1 : 0.f;   // 1 / (2 a H_mm)
        const float h2 = 2.f * h01[s];
        const float q1f = (float)q1;
        float pbest = 0.f;
        int pr0 = 0, pr1 = 0;
        for (int r0 = 0; r0 <= p.L; ++r0) {
          const float d0 = a0 * (float)(r0 - q0);
          const float fixed = d0 * fmaf(d0, H00, g0);
          const float g1p = fmaf(d0, h2, g1);            // gradient of the second coordinate once the first has moved
          const float r1f = fminf(fmaxf(rintf(fmaf(-g1p, w1, q1f)), 0.f), Lf);
          const float d1 = a1 * (r1f - q1f);
          const float val = fmaf(d1, fmaf(d1, H11, g1p), fixed);
          if (val < pbest) { pbest = val; pr0 = r0; pr1 = (int)r1f; }
        }
        if (pbest < best || (pbest == best && pbest < 0.f && ((m0 << 16) < (bpk & 0xFFFF0000u)))) {
          best = pbest;
          bpk = (m0 << 16) | ((unsigned)pr0 << 8) | (unsigned)pr1;
          bextra = m1 | ((unsigned)q0 << 16) | ((unsigned)q1 << 24);
        }
      }

      // ---- team-wide argmin: (change, lowest first coordinate, lowest levels) ----
      const unsigned key = best < 0.f ? ~__float_as_uint(best) : kNoMove;
      const unsigned packed = best < 0.f ? bpk : kNoMove;
      unsigned m = __reduce_min_sync(0xFFFFFFFFu, key);
      unsigned w = __reduce_min_sync(0xFFFFFFFFu, key == m ? packed : kNoMove);
      unsigned src = __ffs(__ballot_sync(0xFFFFFFFFu, key == m && packed == w)) - 1;
      unsigned extra = __shfl_sync(0xFFFFFFFFu, bextra, src & 31);
      if (nwarps > 1) {
        if (lane == 0) s_exch[xbuf][warp] = make_uint4(m, w, extra, 0u);
        __syncthreads();
        const uint4 x = lane < nwarps ? s_exch[xbuf][lane] : make_uint4(kNoMove, kNoMove, 0u, 0u);
        m = __reduce_min_sync(0xFFFFFFFFu, x.x);
        w = __reduce_min_sync(0xFFFFFFFFu, x.x == m ? x.y : kNoMove);
        src = __ffs(__ballot_sync(0xFFFFFFFFu, x.x == m && x.y == w)) - 1;
        extra = __shfl_sync(0xFFFFFFFFu, x.z, src & 31);
        xbuf ^= 1;
      } else {
        __syncwarp();
      }
      if (t + 1 < p.T) draw(t + 1);
      if (m == kNoMove) continue;  // this partition holds no improving pair

      const unsigned m0 = w >> 16, m1 = extra & 0xFFFFu;
      const int r0 = (int)((w >> 8) & 255u), r1 = (int)(w & 255u);
      const int q0 = (int)((extra >> 16) & 255u), q1 = (int)(extra >> 24);
      if (m0 >= d_in || m1 >= d_in) {  // cannot happen; never follow a bad row index
        if (tid == 0) atomicExch(p.status, (int)kFlagBadIndex);
        bad = true;
        break;
      }
      const double c0 = 2.0 * ((double)scale_of(m0) * (double)(r0 - q0));
      const double c1 = 2.0 * ((double)scale_of(m1) * (double)(r1 - q1));
      const float* row0 = p.H + (size_t)m0 * d_in;
      const float* row1 = p.H + (size_t)m1 * d_in;
      const unsigned nch = d_in >> 1;
      if (c0 != 0.0 && c1 != 0.0) {
#pragma unroll 4
        for (unsigned c = tid; c < nch; c += NT) {
          const float2 ha = ld_row2(row0 + 2 * c), hb = ld_row2(row1 + 2 * c);
          double2 gv = *reinterpret_cast<double2*>(g_s + 2 * c);
          gv.x = fma(c1, (double)hb.x, fma(c0, (double)ha.x, gv.x));
          gv.y = fma(c1, (double)hb.y, fma(c0, (double)ha.y, gv.y));
          *reinterpret_cast<double2*>(g_s + 2 * c) = gv;
        }
      } else {
        const float* row = c0 != 0.0 ? row0 : row1;
        const double cc = c0 != 0.0 ? c0 : c1;
#pragma unroll 4
        for (unsigned c = tid; c < nch; c += NT) {
          const float2 ha = ld_row2(row + 2 * c);
          double2 gv = *reinterpret_cast<double2*>(g_s + 2 * c);
          gv.x = fma(cc, (double)ha.x, gv.x);
          gv.y = fma(cc, (double)ha.y, gv.y);
          *reinterpret_cast<double2*>(g_s + 2 * c) = gv;
        }
      }
      if (tid == 0) {
        q_s[m0] = (unsigned char)r0;
        q_s[m1] = (unsigned char)r1;
        col_dsum += (double)__uint_as_float(~m);
        ++moves;
      }
      __syncthreads();
    }
    if (tid == 0) { my_moves += (unsigned long long)moves; my_dsum += col_dsum; }
    __syncthreads();
    if (bad) break;

    // ---- write the codes back ----
    {
      unsigned char* qcol = p.Qt + j * p.ldq;
      for (unsigned i = tid; i < d_in; i += NT) qcol[i] = q_s[i];
    }
  }

  if (tid == 0) {
    if (my_dsum != 0.0) atomicAdd(&p.ctr->delta_sum, my_dsum);
    if (my_moves) atomicAdd(&p.ctr->committed, my_moves);
  }
}

// ---------------------------------------------------------------------------
// Fixed-order fp64 version: every assignment of levels is scored as written in Algorithm 2
// (no fused multiply-add, the sums in the order of the definition), ties to the pair whose
// lower coordinate is lowest, then to the lowest levels.  One CTA per column, gradient and
// codes in global memory.  Small layers only.
__global__ void __launch_bounds__(128) bcd2_verify_kernel(CdParams p, unsigned long long seed, BcdShape shape) {
  __shared__ double s_change[128];
  __shared__ int s_m0[128], s_m1[128], s_lv[128];
  const long long j = blockIdx.x;
  const int tid = threadIdx.x;
  const unsigned d_in = (unsigned)p.d_in, nb = d_in >> 1;
  const int nlev = p.L + 1;
  double* g = p.G + j * p.ldg;
  unsigned char* q = p.Qt + j * p.ldq;
  const unsigned long long base = splitmix64(seed ^ splitmix64((unsigned long long)j));
  unsigned long long moves = 0;
  double dsum = 0.0;
  for (long long t = 0; t < p.T; ++t) {
    const BcdKeys keys = bcd_keys(base, t);
    double best = 0.0;
    int bm0 = -1, bm1 = 0, blv = 0;
    for (unsigned u = tid; u < nb; u += 128) {
      unsigned m0 = bcd_perm(2 * u, d_in, shape.mask, shape.shift, keys);
      unsigned m1 = bcd_perm(2 * u + 1, d_in, shape.mask, shape.shift, keys);
      if (m1 < m0) { const unsigned x = m0; m0 = m1; m1 = x; }
      const double a0 = (double)p.scale[(m0 / p.g) * p.d_out + j], a1 = (double)p.scale[(m1 / p.g) * p.d_out + j];
      const double H00 = (double)p.H[(size_t)m0 * d_in + m0], H01 = (double)p.H[(size_t)m0 * d_in + m1];
      const double H10 = (double)p.H[(size_t)m1 * d_in + m0], H11 = (double)p.H[(size_t)m1 * d_in + m1];
      const double g0 = g[m0], g1 = g[m1];
      const int q0 = q[m0], q1 = q[m1];
      for (int r0 = 0; r0 < nlev; ++r0) {
        const double d0 = __dmul_rn(a0, (double)(r0 - q0));
        for (int r1 = 0; r1 < nlev; ++r1) {
          if (r0 == q0 && r1 == q1) continue;
          const double d1 = __dmul_rn(a1, (double)(r1 - q1));
          double quad = __dmul_rn(__dmul_rn(d0, d0), H00);
          quad = __dadd_rn(quad, __dmul_rn(__dmul_rn(d0, d1), H01));
          double lin = __dmul_rn(d0, g0);
          quad = __dadd_rn(quad, __dmul_rn(__dmul_rn(d1, d0), H10));
          quad = __dadd_rn(quad, __dmul_rn(__dmul_rn(d1, d1), H11));
          lin = __dadd_rn(lin, __dmul_rn(d1, g1));
          const double change = __dadd_rn(quad, lin);
          const int lv = r0 * 256 + r1;
          if (change < best || (change == best && bm0 >= 0 && ((int)m0 < bm0 || ((int)m0 == bm0 && lv < blv)))) {
            best = change; bm0 = (int)m0; bm1 = (int)m1; blv = lv;
          }
        }
      }
    }
    s_change[tid] = best; s_m0[tid] = bm0; s_m1[tid] = bm1; s_lv[tid] = blv;
    __syncthreads();
    for (int w = 64; w > 0; w >>= 1) {
      if (tid < w) {
        const double oc = s_change[tid + w];
        const int om0 = s_m0[tid + w];
        const bool take = om0 >= 0 && (s_m0[tid] < 0 || oc < s_change[tid] ||
                                       (oc == s_change[tid] && (om0 < s_m0[tid] || (om0 == s_m0[tid] && s_lv[tid + w] < s_lv[tid]))));
        if (take) { s_change[tid] = oc; s_m0[tid] = om0; s_m1[tid] = s_m1[tid + w]; s_lv[tid] = s_lv[tid + w]; }
      }
      __syncthreads();
    }
    const int m0 = s_m0[0], m1 = s_m1[0], lv = s_lv[0];
    const double change = s_change[0];
    __syncthreads();
    if (m0 < 0) continue;  // this partition holds no improving pair
    const int mm[2] = {m0, m1}, rr[2] = {lv >> 8, lv & 255};
    const int qq[2] = {q[m0], q[m1]};
    __syncthreads();
    if (tid == 0) { q[m0] = (unsigned char)rr[0]; q[m1] = (unsigned char)rr[1]; }
    for (int c = 0; c < 2; ++c) {
      const double a = (double)p.scale[(mm[c] / p.g) * p.d_out + j];
      const double d = __dmul_rn(a, (double)(rr[c] - qq[c]));
      if (d == 0.0) continue;
      const double two_d = __dmul_rn(2.0, d);
      const float* row = p.H + (size_t)mm[c] * d_in;
      for (unsigned i = tid; i < d_in; i += 128) g[i] = __dadd_rn(g[i], __dmul_rn(two_d, (double)row[i]));
    }
    ++moves;
    dsum += change;
    __syncthreads();
  }
  if (tid == 0) {
    atomicAdd(&p.ctr->committed, moves);
    atomicAdd(&p.ctr->delta_sum, dsum);
  }
}

// ---------------------------------------------------------------------------
bool bcd_supported(long long d_in, int block) {
  return block == 2 && d_in >= 2 && (d_in & 1) == 0 && d_in <= 32768;
}

template <int PPT, int MAXNT, int MINB>
static cudaError_t launch_bcd_cfg(const CdParams& p, unsigned long long seed, int nt, cudaStream_t st) {
  auto kern = bcd2_kernel<PPT, MAXNT, MINB>;
  int dev = 0, sms = 0, smem_max = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  const size_t q_bytes = (size_t)((p.ldg + 15) / 16 * 16), a_bytes = sizeof(float) * (size_t)p.ng;
  const size_t budget = (size_t)smem_max - 2048;  // the kernel's static shared memory and the runtime's share
  const int a_in_smem = q_bytes + a_bytes <= budget / 2 ? 1 : 0;
  size_t smem = q_bytes + (a_in_smem ? a_bytes : 0);
  if (smem > budget) return cudaErrorNotSupported;
  // CDQ_BCD_G=global in the environment keeps the gradient in global memory at every size
  static const bool force_global = [] { const char* e = getenv("CDQ_BCD_G"); return e && e[0] == 'g'; }();
  const int g_in_smem = !force_global && smem + sizeof(double) * (size_t)p.ldg <= budget ? 1 : 0;
  if (g_in_smem) smem += sizeof(double) * (size_t)p.ldg;
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
  kern<<<(unsigned)blocks, nt, smem, st>>>(p, seed, bcd_shape(p.d_in), g_in_smem, a_in_smem);
  return cudaGetLastError();
}

cudaError_t launch_bcd(const Layer& ly, double* G, long long ldg, unsigned char* Qt, long long ldq, const float* hdiag,
                       const float* hs, long long steps_per_col, unsigned long long seed, bool fast, CdCounters* ctr,
                       cudaStream_t st) {
  CdParams p{};
  p.H = ly.H; p.d_in = ly.d_in; p.d_out = ly.d_out; p.G = G; p.ldg = ldg; p.Qt = Qt; p.ldq = ldq; p.scale = ly.scale;
  p.hdiag = hdiag; p.hs = hs; p.g = ly.g; p.ng = ly.ng; p.L = ly.L; p.T = steps_per_col; p.ctr = ctr;
  p.status = device_status_word();
  if (!p.status) return cudaErrorInvalidSymbol;
  p.gmagic = ly.g > 1 ? (unsigned)(((1ull << 32) + (unsigned long long)ly.g - 1) / (unsigned long long)ly.g) : 0u;
  if (!fast) {
    bcd2_verify_kernel<<<(unsigned)ly.d_out, 128, 0, st>>>(p, seed, bcd_shape(ly.d_in));
    return cudaGetLastError();
  }
  const long long nb = ly.d_in / 2;
  auto team = [&](int ppt) { return (int)(((nb + ppt - 1) / ppt + 31) / 32 * 32); };
  if (nb <= 256) return launch_bcd_cfg<1, 256, 4>(p, seed, team(1), st);
  if (nb <= 2048) return launch_bcd_cfg<4, 512, 2>(p, seed, team(4), st);
  if (nb <= 8192) return launch_bcd_cfg<8, 1024, 1>(p, seed, team(8), st);
  return launch_bcd_cfg<16, 1024, 1>(p, seed, team(16), st);
}

}  // namespace cdq
