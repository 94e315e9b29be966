// Block coordinate descent with random blocks of two coordinates, batched over all output
// columns (paper: Algorithm 2; Algorithm 5 for sub-channel grids; weight-unit form).
//
// Step t cuts the coordinates into d_in / 2 pairs by a counter-based bijection of
// {0..d_in-1} keyed by (seed, t), the same for every column; every pair (i, m) is scored over
// all (L+1)^2 assignments of levels,
//   change = d_i^2 H_ii + 2 d_i d_m H_im + d_m^2 H_mm + d_i g_i + d_m g_m,  d = a (r - q),
// the most negative change of the step is applied and g += 2 d_i H[i, :] + 2 d_m H[m, :].
//
// One CTA owns one column at a time.  Pairs touch the gradient and the codes at random, so
// both live in shared memory (gradient fp64, 8 bytes per coordinate; codes 1 byte); the rows
// of H stream through registers.  The partition does not depend on the state or the column,
// so a kernel of its own lists, once per call, the pairs of every step with their
// off-diagonal entry H_im (d_in / 2 scattered reads per step, which would otherwise be paid
// per column and bound the descent by the rate of random DRAM reads) and with the two
// diagonal entries; the descent reads that table in order (16 bytes per pair and pass).
// The scan over the (L+1)^2 assignments fixes a level of the lower coordinate and takes the
// best level of the other in closed form (the clamped rounding of the vertex of its parabola,
// as in the greedy descent); convexity of the change in the pair bounds which levels of the
// lower coordinate can still win, so only a few of them are visited.
#include <cstdio>
#include <cstdlib>

#include "common.cuh"
#include "cd_params.cuh"

namespace cdq {

// ---------------------------------------------------------------------------
// The partition: x -> pi(x), three rounds of (odd multiply + add) mod 2^b and xor-shift on
// b = ceil(log2 d_in) bits, keyed per (seed, step); values >= d_in walk the cycle
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
// tab[t * nb + u] = (m0 | m1 << 16, bits of H[m0, m1], H[m0, m0], H[m1, m1]) with m0 < m1 the pair u
// of step t (the diagonal with negative entries set to 0).
__global__ void bcd2_table_kernel(const float* __restrict__ H, const float* __restrict__ hdiag, unsigned d_in,
                                  unsigned long long seed, BcdShape shape, uint4* __restrict__ tab) {
  const unsigned nb = d_in >> 1;
  const unsigned u = blockIdx.x * blockDim.x + threadIdx.x;
  const long long t = blockIdx.y;
  if (u >= nb) return;
  const BcdKeys keys = bcd_keys(splitmix64(seed), t);
  unsigned m0 = bcd_perm(2 * u, d_in, shape.mask, shape.shift, keys);
  unsigned m1 = bcd_perm(2 * u + 1, d_in, shape.mask, shape.shift, keys);
  if (m1 < m0) { const unsigned x = m0; m0 = m1; m1 = x; }
  tab[(size_t)t * nb + u] = make_uint4(m0 | (m1 << 16), __float_as_uint(ld_nc_f32(H + (size_t)m0 * d_in + m1)),
                                       __float_as_uint(hdiag[m0]), __float_as_uint(hdiag[m1]));
}

// ---------------------------------------------------------------------------
// PPT: pairs per thread (pair u = tid + NT * slot).  g_in_smem == 0: the gradient stays in
// its global-memory column (layers whose column does not fit in shared memory).
// a_in_smem == 0: the group scales are read from global memory.
template <int PPT, int MAXNT, int MINB>
__global__ void __launch_bounds__(MAXNT, MINB)
bcd2_kernel(CdParams p, const uint4* __restrict__ tab, int g_in_smem, int a_in_smem) {
  extern __shared__ __align__(16) unsigned char dyn_smem[];
  __shared__ __align__(16) uint4 s_exch[2][32];
  __shared__ unsigned s_bound[2][32];
  __shared__ int s_col;

  const int tid = threadIdx.x, NT = blockDim.x;
  const int lane = tid & 31, warp = tid >> 5, nwarps = NT >> 5;
  const unsigned d_in = (unsigned)p.d_in;
  const unsigned nb = d_in >> 1;
  const float Lf = (float)p.L;

  // shared memory: [gradient, 8 ldg bytes][codes, ldg bytes rounded to 16][scales, 4 ng bytes]
  double* g_smem = reinterpret_cast<double*>(dyn_smem);
  unsigned char* q_s = dyn_smem + (g_in_smem ? sizeof(double) * (size_t)p.ldg : 0);
  float2* a_smem = reinterpret_cast<float2*>(q_s + ((p.ldg + 15) / 16) * 16);   // (a, 1 / a) per group
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
    if (g_in_smem) {
      const double* gcol = p.G + j * p.ldg;
      for (unsigned i = tid; i < d_in; i += NT) g_s[i] = gcol[i];
    }
    {
      const unsigned char* qcol = p.Qt + j * p.ldq;
      for (unsigned i = tid; i < d_in; i += NT) q_s[i] = qcol[i];
    }
    if (a_in_smem)
      for (int t = tid; t < (int)p.ng; t += NT) {
        const float a = p.scale[(long long)t * p.d_out + j];
        a_smem[t] = make_float2(a, a > 0.f ? 1.0f / a : 0.f);
      }
    __syncthreads();
    auto scale_of = [&](unsigned i) -> float2 {
      if (a_in_smem) return a_smem[group_of(i)];
      const float a = p.scale[(long long)group_of(i) * p.d_out + j];
      return make_float2(a, a > 0.f ? 1.0f / a : 0.f);
    };

    double col_dsum = 0.0;
    long long moves = 0;
    bool bad = false;
    for (long long t = 0; t < p.T; ++t) {
      // ---- pass 1: the best move of each coordinate alone (the pair with the other level kept) ----
      const uint4* trow = tab + (size_t)t * nb;
      float best = 0.f;
      unsigned bpk = kNoMove, bextra = 0;
#pragma unroll
      for (int s = 0; s < PPT; ++s) {
        const unsigned u = (unsigned)tid + (unsigned)NT * s;
        if (u >= nb) continue;
        const uint4 e = __ldg(trow + u);
        const unsigned m0 = e.x & 0xFFFFu, m1 = e.x >> 16;
        const unsigned q0 = q_s[m0], q1 = q_s[m1];
        const unsigned extra_s = m1 | (q0 << 16) | (q1 << 24);
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const unsigned mc = c ? m1 : m0;
          const float gc = (float)g_s[mc], qf = (float)(c ? q1 : q0);
          const float2 ac = scale_of(mc);
          const float Hcc = __uint_as_float(c ? e.w : e.z);
          const float hsc = Hcc > 0.f ? 0.5f / Hcc : 0.f;
          const float rf = fminf(fmaxf(rintf(fmaf(-gc, hsc * ac.y, qf)), 0.f), Lf);
          const float d = ac.x * (rf - qf);
          const float val = d * fmaf(d, Hcc, gc);
          const unsigned pk = (m0 << 16) | (c ? (q0 << 8) | (unsigned)rf : ((unsigned)rf << 8) | q1);
          if (val < best || (val == best && val < 0.f && pk < bpk)) { best = val; bpk = pk; bextra = extra_s; }
        }
      }
      // the best of them over the team bounds what a pair has to beat
      float bound;
      {
        unsigned k1 = __reduce_min_sync(0xFFFFFFFFu, best < 0.f ? ~__float_as_uint(best) : kNoMove);
        if (nwarps > 1) {
          if (lane == 0) s_bound[xbuf][warp] = k1;
          __syncthreads();
          k1 = __reduce_min_sync(0xFFFFFFFFu, lane < nwarps ? s_bound[xbuf][lane] : kNoMove);
        }
        bound = k1 == kNoMove ? 0.f : __uint_as_float(~k1);
      }

      // ---- pass 2: pairs that can beat the bound ----
#pragma unroll
      for (int s = 0; s < PPT; ++s) {
        const unsigned u = (unsigned)tid + (unsigned)NT * s;
        if (u >= nb) continue;
        const uint4 e = __ldg(trow + u);
        const unsigned m0 = e.x & 0xFFFFu, m1 = e.x >> 16;
        const float g0 = (float)g_s[m0], g1 = (float)g_s[m1];
        const float H00 = __uint_as_float(e.z), H11 = __uint_as_float(e.w), h01 = __uint_as_float(e.y);
        const float h2 = 2.f * h01;
        // The change is convex in the pair (H is positive semi-definite): no assignment does
        // better than the free minimum -N / (4 det), N = g0^2 H11 - 2 g0 g1 H01 + g1^2 H00.
        // A pair whose 2 x 2 block of H is close to singular in fp32 is never skipped and is
        // scanned in full.
        const float det = fmaf(H00, H11, -h01 * h01);
        const bool full = !(det > 1e-4f * H00 * H11);
        const float N = fmaf(g1 * g1, H00, fmaf(g0 * g0, H11, -g0 * g1 * h2));
        if (!full && 1.001f * N < -4.f * bound * det) continue;
        const int q0 = q_s[m0], q1 = q_s[m1];
        const float2 a0 = scale_of(m0), a1 = scale_of(m1);
        const unsigned extra_s = m1 | ((unsigned)q0 << 16) | ((unsigned)q1 << 24);
        // S: the coordinate whose levels are scanned (the one with the larger a^2 H_ii, so that
        // few of its levels can win); F: the other, whose level follows in closed form
        const bool swap = !full && a1.x * a1.x * H11 > a0.x * a0.x * H00;
        const float gS = swap ? g1 : g0, gF = swap ? g0 : g1;
        const int qS = swap ? q1 : q0, qF = swap ? q0 : q1;
        const float aS = swap ? a1.x : a0.x, aF = swap ? a0.x : a1.x;
        const float HSS = swap ? H11 : H00, HFF = swap ? H00 : H11;
        const float wF = HFF > 0.f ? 0.5f / HFF * (swap ? a0.y : a1.y) : 0.f;   // 1 / (2 a H_ii)
        const float qFf = (float)qF;
        // phi(rS): the change with F free in [0, L] (not rounded): convex in rS and a lower
        // bound of the rounded change, so the scan walks outwards from qS and stops on a side
        // once phi has passed the bound and no longer falls.
        auto eval = [&](int rS) -> float {
          const float dS = aS * (float)(rS - qS);
          const float fixed = dS * fmaf(dS, HSS, gS);
          const float gFp = fmaf(dS, h2, gF);            // gradient of F once S has moved
          const float x = fminf(fmaxf(fmaf(-gFp, wF, qFf), 0.f), Lf);
          const float dc = aF * (x - qFf);
          const float phi = fmaf(dc, fmaf(dc, HFF, gFp), fixed);
          if (phi <= bound) {
            const float rFf = rintf(x);
            const float dF = aF * (rFf - qFf);
            const float val = fmaf(dF, fmaf(dF, HFF, gFp), fixed);
            const unsigned r0 = swap ? (unsigned)rFf : (unsigned)rS, r1 = swap ? (unsigned)rS : (unsigned)rFf;
            const unsigned pk = (m0 << 16) | (r0 << 8) | r1;
            if (val < best || (val == best && val < 0.f && pk < bpk)) {
              best = val; bpk = pk; bextra = extra_s;
              bound = fminf(bound, best);
            }
          }
          return phi;
        };
        const float phi_q = eval(qS);
        float prev = phi_q;
        for (int rS = qS + 1; rS <= p.L; ++rS) {
          const float phi = eval(rS);
          if (!full && phi > bound && phi >= prev) break;
          prev = phi;
        }
        prev = phi_q;
        for (int rS = qS - 1; rS >= 0; --rS) {
          const float phi = eval(rS);
          if (!full && phi > bound && phi >= prev) break;
          prev = phi;
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
      if (m == kNoMove) continue;  // this partition holds no improving pair

      const unsigned m0 = w >> 16, m1 = extra & 0xFFFFu;
      const int r0 = (int)((w >> 8) & 255u), r1 = (int)(w & 255u);
      const int q0 = (int)((extra >> 16) & 255u), q1 = (int)(extra >> 24);
      if (m0 >= d_in || m1 >= d_in) {  // cannot happen; never follow a bad row index
        if (tid == 0) atomicExch(p.status, (int)kFlagBadIndex);
        bad = true;
        break;
      }
      const double c0 = 2.0 * ((double)scale_of(m0).x * (double)(r0 - q0));
      const double c1 = 2.0 * ((double)scale_of(m1).x * (double)(r1 - q1));
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
  const unsigned long long base = splitmix64(seed);
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
static cudaError_t launch_bcd_cfg(const CdParams& p, const uint4* tab, int nt, cudaStream_t st) {
  auto kern = bcd2_kernel<PPT, MAXNT, MINB>;
  int dev = 0, sms = 0, smem_max = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  const size_t q_bytes = (size_t)((p.ldg + 15) / 16 * 16), a_bytes = sizeof(float2) * (size_t)p.ng;
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
  kern<<<(unsigned)blocks, nt, smem, st>>>(p, tab, g_in_smem, a_in_smem);
  return cudaGetLastError();
}

size_t bcd_table_bytes(long long d_in, long long steps_per_col) {
  return sizeof(uint4) * (size_t)(d_in / 2) * (size_t)(steps_per_col > 0 ? steps_per_col : 0);
}

cudaError_t launch_bcd(const Layer& ly, double* G, long long ldg, unsigned char* Qt, long long ldq, const float* hdiag,
                       const float* hs, long long steps_per_col, unsigned long long seed, bool fast, void* table,
                       CdCounters* ctr, cudaStream_t st) {
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
  uint4* tab = (uint4*)table;
  if (steps_per_col > 0) {
    if (steps_per_col > 65535) return cudaErrorNotSupported;  // steps index a grid dimension
    dim3 grid((unsigned)((nb + 255) / 256), (unsigned)steps_per_col);
    bcd2_table_kernel<<<grid, 256, 0, st>>>(ly.H, hdiag, (unsigned)ly.d_in, seed, bcd_shape(ly.d_in), tab);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  auto team = [&](int ppt) { return (int)(((nb + ppt - 1) / ppt + 31) / 32 * 32); };
  if (nb <= 256) return launch_bcd_cfg<1, 256, 4>(p, tab, team(1), st);
  if (nb <= 2048) return launch_bcd_cfg<4, 512, 2>(p, tab, team(4), st);
  if (nb <= 8192) return launch_bcd_cfg<8, 1024, 1>(p, tab, team(8), st);
  return launch_bcd_cfg<16, 1024, 1>(p, tab, team(16), st);
}

}  // namespace cdq
