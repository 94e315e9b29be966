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
// The scan over the (L+1)^2 assignments fixes a level of one coordinate and takes the best
// level of the other in closed form (the clamped rounding of the vertex of its parabola, as
// in the greedy descent); convexity of the change in the pair tells which pairs, and which
// levels, can still win, so only a few are visited (see the kernel's header).
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
//
// One step:
//   1. (with the update of the previous step) every thread sweeps its own coordinates, two
//      per chunk: g += 2 d_i H[i, :] + 2 d_m H[m, :], and the best move of each coordinate
//      alone is scored as in the greedy descent; its minimum over the team, `bound`, is a
//      change that some pair reaches (a pair may keep one of its levels);
//   2. every pair is tested against the bound with the free minimum of its 2 x 2 quadratic,
//      -N / (4 det), N = g_i^2 H_mm - 2 g_i g_m H_im + g_m^2 H_ii (H is positive
//      semi-definite, so no assignment of levels does better); most pairs stop here.  When the
//      bound is 0 (no single move lowers the loss: the state the greedy descent leaves) that test
//      passes every pair, and a sharper one takes its place: a lower bound of the change over
//      the moves of both coordinates by at least one level each;
//   3. the pairs that are left are scanned, after the test loop so that a warp scans only as
//      many rounds as its busiest lane has such pairs: the levels of one coordinate S are
//      walked outwards from its current level, the level of the other, F, follows in closed
//      form; phi(r_S), the change with F free in [0, L], is convex in r_S and bounds the
//      rounded change from below, so a side ends once phi has passed the best change known
//      and no longer falls.  S is the coordinate with the larger a^2 H_ii (few of its levels
//      can win).  A pair whose 2 x 2 block is close to singular in fp32 is always scanned, in
//      full;
//   4. team-wide argmin (change, lowest first coordinate, lowest levels), as in the greedy
//      descent, carrying the pair's other coordinate and old levels.
template <int PPT, int MAXNT, int MINB>
__global__ void __launch_bounds__(MAXNT, MINB)
bcd2_kernel(CdParams p, const uint4* __restrict__ tab, int g_in_smem, int a_in_smem) {
  extern __shared__ __align__(16) unsigned char dyn_smem[];
  __shared__ __align__(16) uint4 s_exch[2][32];
  __shared__ unsigned s_bound[32];
  __shared__ int s_col;

  const int tid = threadIdx.x, NT = blockDim.x;
  const int lane = tid & 31, warp = tid >> 5, nwarps = NT >> 5;
  const unsigned d_in = (unsigned)p.d_in;
  const unsigned nb = d_in >> 1;   // pairs, and chunks of two coordinates
  const float Lf = (float)p.L;

  // shared memory: [gradient, 8 ldg bytes][codes, ldg bytes rounded to 16][(a, 1 / a) per group]
  double* g_smem = reinterpret_cast<double*>(dyn_smem);
  unsigned char* q_s = dyn_smem + (g_in_smem ? sizeof(double) * (size_t)p.ldg : 0);
  float2* a_smem = reinterpret_cast<float2*>(q_s + ((p.ldg + 15) / 16) * 16);
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
    const bool one_scale = p.ng == 1;   // per-channel grid: one (a, 1 / a) for the column
    float2 a_col = make_float2(0.f, 0.f);
    if (one_scale) {
      const float a = p.scale[j];
      a_col = make_float2(a, a > 0.f ? 1.0f / a : 0.f);
    }
    auto scale_of = [&](unsigned i) -> float2 {
      if (one_scale) return a_col;
      if (a_in_smem) return a_smem[group_of(i)];
      const float a = p.scale[(long long)group_of(i) * p.d_out + j];
      return make_float2(a, a > 0.f ? 1.0f / a : 0.f);
    };

    // Applies g += c0 row0 + c1 row1 (nrows of them) to the thread's chunks and returns the best
    // change of a single coordinate among them (0 if none lowers the loss).  A thread owns the
    // chunks tid + NT * s, s < PPT, as it owns the pairs; the loads of SB chunks are issued
    // together so that a sweep waits for memory PPT / SB times, not once per chunk.
    auto sweep = [&](int nrows, double c0, double c1, const float* row0, const float* row1) -> float {
      constexpr int SB = PPT < 4 ? PPT : 4;
      float ub = 0.f;
#pragma unroll
      for (int s0 = 0; s0 < PPT; s0 += SB) {
        float2 ha[SB], hb[SB], hd[SB], hs[SB];
#pragma unroll
        for (int k = 0; k < SB; ++k) {
          const unsigned c = (unsigned)tid + (unsigned)NT * (s0 + k);
          ha[k] = hb[k] = hd[k] = hs[k] = make_float2(0.f, 0.f);
          if (c < nb) {
            if (nrows >= 1) ha[k] = ld_row2(row0 + 2 * c);
            if (nrows == 2) hb[k] = ld_row2(row1 + 2 * c);
            hd[k] = __ldg(reinterpret_cast<const float2*>(p.hdiag) + c);
            hs[k] = __ldg(reinterpret_cast<const float2*>(p.hs) + c);
          }
        }
#pragma unroll
        for (int k = 0; k < SB; ++k) {
          const unsigned c = (unsigned)tid + (unsigned)NT * (s0 + k);
          if (c >= nb) continue;
          double2 gv = *reinterpret_cast<double2*>(g_s + 2 * c);
          if (nrows >= 1) {
            gv.x = fma(c0, (double)ha[k].x, gv.x);
            gv.y = fma(c0, (double)ha[k].y, gv.y);
          }
          if (nrows == 2) {
            gv.x = fma(c1, (double)hb[k].x, gv.x);
            gv.y = fma(c1, (double)hb[k].y, gv.y);
          }
          if (nrows >= 1) *reinterpret_cast<double2*>(g_s + 2 * c) = gv;
          const unsigned qq = *reinterpret_cast<const unsigned short*>(q_s + 2 * c);
          const float2 ax = scale_of(2 * c), ay = scale_of(2 * c + 1);
          {
            const float gf = (float)gv.x, qf = (float)(qq & 255u);
            const float rf = fminf(fmaxf(rintf(fmaf(-gf, hs[k].x * ax.y, qf)), 0.f), Lf);
            const float d = ax.x * (rf - qf);
            ub = fminf(ub, d * fmaf(d, hd[k].x, gf));
          }
          {
            const float gf = (float)gv.y, qf = (float)(qq >> 8);
            const float rf = fminf(fmaxf(rintf(fmaf(-gf, hs[k].y * ay.y, qf)), 0.f), Lf);
            const float d = ay.x * (rf - qf);
            ub = fminf(ub, d * fmaf(d, hd[k].y, gf));
          }
        }
      }
      return ub;
    };
    // Team-wide minimum of the sweeps' results; ends with every thread past the barrier.
    auto team_bound = [&](float ub) -> float {
      unsigned k = __reduce_min_sync(0xFFFFFFFFu, ub < 0.f ? ~__float_as_uint(ub) : kNoMove);
      if (nwarps > 1) {
        if (lane == 0) s_bound[warp] = k;
        __syncthreads();
        k = __reduce_min_sync(0xFFFFFFFFu, lane < nwarps ? s_bound[lane] : kNoMove);
      } else {
        __syncwarp();
      }
      return k == kNoMove ? 0.f : __uint_as_float(~k);
    };

    double col_dsum = 0.0;
    long long moves = 0;
    bool bad = false;
    float bound = p.T > 0 ? team_bound(sweep(0, 0.0, 0.0, p.H, p.H)) : 0.f;
    for (long long t = 0; t < p.T; ++t) {
      const uint4* trow = tab + (size_t)t * nb;
      // what a pair has to reach: the bound, eased by a few ulps so that the single move that
      // set it is found again by the scan of its pair
      float lim = bound * 0.99999f;
      float best = 0.f;
      unsigned bpk = kNoMove, bextra = 0;

      // Scan of one pair: the levels of S outwards from its current level, the level of F in
      // closed form (see the header of the kernel).
      auto scan_pair = [&](const uint4 e, const float g0, const float g1) {
        const unsigned m0 = e.x & 0xFFFFu, m1 = e.x >> 16;
        const float H00 = __uint_as_float(e.z), H11 = __uint_as_float(e.w), h01 = __uint_as_float(e.y);
        const float h2 = 2.f * h01;
        const bool full = !(fmaf(H00, H11, -h01 * h01) > 1e-4f * H00 * H11);
        const int q0 = q_s[m0], q1 = q_s[m1];
        const float2 a0 = scale_of(m0), a1 = scale_of(m1);
        const unsigned extra_s = m1 | ((unsigned)q0 << 16) | ((unsigned)q1 << 24);
        const bool swap = !full && a1.x * a1.x * H11 > a0.x * a0.x * H00;
        const float gS = swap ? g1 : g0, gF = swap ? g0 : g1;
        const int qS = swap ? q1 : q0, qF = swap ? q0 : q1;
        const float aS = swap ? a1.x : a0.x, aF = swap ? a0.x : a1.x;
        const float HSS = swap ? H11 : H00, HFF = swap ? H00 : H11;
        const float wF = HFF > 0.f ? __fdividef(0.5f, HFF) * (swap ? a0.y : a1.y) : 0.f;   // 1 / (2 a H_ii), 2 ulp
        const float qFf = (float)qF;
        auto eval = [&](int rS) -> float {
          const float dS = aS * (float)(rS - qS);
          const float fixed = dS * fmaf(dS, HSS, gS);
          const float gFp = fmaf(dS, h2, gF);            // gradient of F once S has moved
          const float x = fminf(fmaxf(fmaf(-gFp, wF, qFf), 0.f), Lf);
          const float dc = aF * (x - qFf);
          const float phi = fmaf(dc, fmaf(dc, HFF, gFp), fixed);
          if (phi <= lim) {
            const float rFf = rintf(x);
            const float dF = aF * (rFf - qFf);
            const float val = fmaf(dF, fmaf(dF, HFF, gFp), fixed);
            const unsigned r0 = swap ? (unsigned)rFf : (unsigned)rS, r1 = swap ? (unsigned)rS : (unsigned)rFf;
            const unsigned pk = (m0 << 16) | (r0 << 8) | r1;
            if (val < best || (val == best && val < 0.f && pk < bpk)) {
              best = val; bpk = pk; bextra = extra_s;
              lim = fminf(lim, best * 0.99999f);
            }
          }
          return phi;
        };
        const float phi_q = eval(qS);
        float prev = phi_q;
        for (int rS = qS + 1; rS <= p.L; ++rS) {
          const float phi = eval(rS);
          if (!full && phi > lim && phi >= prev) break;
          prev = phi;
        }
        prev = phi_q;
        for (int rS = qS - 1; rS >= 0; --rS) {
          const float phi = eval(rS);
          if (!full && phi > lim && phi >= prev) break;
          prev = phi;
        }
      };

      // ---- test every pair of this thread against the bound ----
      // The table entries of up to 8 pairs are requested together, so that a step waits for the
      // table once or twice, not once per pair; the pairs that are left wait for the loop below,
      // where a warp scans only as many rounds as its busiest lane has pairs.
      unsigned todo = 0;
      constexpr int TB = PPT < 8 ? PPT : 8;
#pragma unroll
      for (int s0 = 0; s0 < PPT; s0 += TB) {
        uint4 ev[TB];
#pragma unroll
        for (int k = 0; k < TB; ++k) {
          const unsigned u = (unsigned)tid + (unsigned)NT * (s0 + k);
          ev[k] = u < nb ? __ldg(trow + u) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int k = 0; k < TB; ++k) {
          const unsigned u = (unsigned)tid + (unsigned)NT * (s0 + k);
          if (u >= nb) continue;
          const uint4 e = ev[k];
          const unsigned m0 = e.x & 0xFFFFu, m1 = e.x >> 16;
          const float g0 = (float)g_s[m0], g1 = (float)g_s[m1];
          const float H00 = __uint_as_float(e.z), H11 = __uint_as_float(e.w), h01 = __uint_as_float(e.y);
          const float det = fmaf(H00, H11, -h01 * h01);
          const bool full = !(det > 1e-4f * H00 * H11);
          bool need;
          if (lim == 0.f) {
            // No single move lowers the loss, so a pair can only win by moving both coordinates.
            // In level units, with u, v >= 1 the sizes of the two steps, A = a0^2 H00, B = a1^2 H11,
            // C = a0 a1 H01, rho = |C| / sqrt(A B):
            //   change >= (1 - rho)(A u^2 + B v^2) - |a0 g0| u - |a1 g1| v     (2 |C| u v <= rho (A u^2 + B v^2))
            // which splits into one parabola per coordinate; each is bounded below over u >= 1 by its
            // value at 1 when its vertex is at or left of 1, and by its free minimum otherwise.
            const float a0 = scale_of(m0).x, a1 = scale_of(m1).x;
            const float A = a0 * a0 * H00, Bq = a1 * a1 * H11;
            const float kap = 1.f - fabsf(a0 * a1 * h01) * rsqrtf(A * Bq);
            const float kA = kap * A, kB = kap * Bq;
            const float al = fabsf(a0 * g0), be = fabsf(a1 * g1);
            const float mS = al <= 2.f * kA ? kA - al : -__fdividef(al * al, 4.f * kA);
            const float mF = be <= 2.f * kB ? kB - be : -__fdividef(be * be, 4.f * kB);
            need = full || !(mS + mF >= 2e-6f * (A + Bq));   // margin: fp32 rounding of the bound; a NaN (dead coordinate) keeps the pair
          } else {
            const float N = fmaf(g1 * g1, H00, fmaf(g0 * g0, H11, -2.f * g0 * g1 * h01));
            need = full || !(1.01f * N < -4.f * lim * det);   // 1 % for the rounding of N and det
          }
          if (need) todo |= 1u << (s0 + k);
        }
      }

      // ---- scan the pairs that are left ----
      while (todo) {
        const int s = __ffs(todo) - 1;
        todo &= todo - 1;
        const uint4 e = __ldg(trow + (unsigned)tid + (unsigned)NT * s);
        scan_pair(e, (float)g_s[e.x & 0xFFFFu], (float)g_s[e.x >> 16]);
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
      if (m == kNoMove) continue;  // this partition holds no improving pair; the state and the bound stand

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
      // the new codes are written by the threads that own these coordinates in the sweep, the
      // only readers of a code until the barrier that ends it
      if ((unsigned)tid == (m0 >> 1) % (unsigned)NT) q_s[m0] = (unsigned char)r0;
      if ((unsigned)tid == (m1 >> 1) % (unsigned)NT) q_s[m1] = (unsigned char)r1;
      float ub;
      if (c0 != 0.0 && c1 != 0.0) ub = sweep(2, c0, c1, row0, row1);
      else if (c0 != 0.0) ub = sweep(1, c0, 0.0, row0, row0);
      else ub = sweep(1, c1, 0.0, row1, row1);
      if (tid == 0) {
        col_dsum += (double)__uint_as_float(~m);
        ++moves;
      }
      bound = team_bound(ub);
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
  { kern<<<(unsigned)blocks, nt, smem, st>>>(p, tab, g_in_smem, a_in_smem); count_launch(); }
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
    { bcd2_verify_kernel<<<(unsigned)ly.d_out, 128, 0, st>>>(p, seed, bcd_shape(ly.d_in)); count_launch(); }
    return cudaGetLastError();
  }
  const long long nb = ly.d_in / 2;
  uint4* tab = (uint4*)table;
  if (steps_per_col > 0) {
    if (steps_per_col > 65535) return cudaErrorNotSupported;  // steps index a grid dimension
    dim3 grid((unsigned)((nb + 255) / 256), (unsigned)steps_per_col);
    { bcd2_table_kernel<<<grid, 256, 0, st>>>(ly.H, hdiag, (unsigned)ly.d_in, seed, bcd_shape(ly.d_in), tab); count_launch(); }
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  auto team = [&](int ppt) { return (int)(((nb + ppt - 1) / ppt + 31) / 32 * 32); };
  if (nb <= 256) return launch_bcd_cfg<1, 256, 2>(p, tab, team(1), st);
  if (nb <= 2048) return launch_bcd_cfg<4, 512, 2>(p, tab, team(4), st);
  if (nb <= 7168) return launch_bcd_cfg<8, 896, 1>(p, tab, team(8), st);
  if (nb <= 8192) return launch_bcd_cfg<8, 1024, 1>(p, tab, team(8), st);
  if (nb <= 9216) return launch_bcd_cfg<12, 768, 1>(p, tab, team(12), st);
  return launch_bcd_cfg<16, 1024, 1>(p, tab, team(16), st);
}

}  // namespace cdq
