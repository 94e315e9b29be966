// Greedy coordinate descent (paper: the loop of Algorithm 1; Algorithm 4 for sub-channel grids)
// for layers whose rows of H stream from HBM (d_in > 4096, d_in % 4 == 0).
//
// A step of one column is a chain: sweep (apply the last move to the gradient, score every
// coordinate) -> team argmin -> fetch of the winner's row H[i*, :] -> next sweep.  Nothing in the
// chain can start early, so a CTA that owns one column leaves HBM idle while it sweeps and the
// arithmetic idle while the row is in flight.  This kernel keeps TWO columns per CTA and
// alternates between them: while the team sweeps column A, the row that column B asked for is
// landing, and the other way round.
//
// Where the state lives (one CTA per SM, NT threads, thread t owns chunk slots t + NT*k, k < NCH,
// of 4 consecutive coordinates, the same slots in both columns):
//   registers      : the gradient's leading fp32 part and the packed codes of both columns
//   shared memory  : one row buffer ("ring") that both columns' rows pass through, H_ii, and the
//                    trailing fp32 part of both gradients (bf16 when fp32 does not fit: LO16)
// The ring is refilled piece by piece behind the sweep that is reading it: the last warp to finish
// chunk slot k of the current row requests piece k of the other column's row (cp.async.bulk, no
// multicast, one mbarrier per piece), so that row has a whole sweep and an argmin to arrive in.
//
// Gradient arithmetic.  g is held as an unevaluated sum hi + lo of two floats (about 48 bits).
// g += c h is an error-free product (c h = p + e with one fused multiply-add) followed by an
// error-free sum of hi and p; all rounding errors go to lo; the score reads fl(hi + lo).  That
// keeps the fp64-grade accumulation the picks need (a rounded gradient drifts by sqrt(T) ulps over T
// steps and forks near-tied columns) without fp64 <-> fp32 conversions, which run at 16 lanes per
// clock per SM on this GPU and bounded the sweep of the fp64 version.
// The vertex of a coordinate's parabola uses an approximate reciprocal of H_ii (1 ulp): it only
// decides the rounding to a level, and a vertex that close to a half-way point scores the two levels
// the same to fp32 resolution; the score itself uses the exact H_ii.
//
// Waits on the copy barriers are bounded by a cycle count; a thread whose wait runs out enters the
// argmin with a key that no real move can have, the whole team sees it after the exchange, waits
// (bounded) for the copies still in flight, records kFlagWaitTimeout and returns.
#include <type_traits>

#include "async_copy.cuh"
#include "cd_params.cuh"
#include "cd_sweep.cuh"

namespace cdq {
namespace {

constexpr long long kWaitCycles = 400ll * 1000 * 1000;   // about 0.2 s
constexpr float kDeadDiag = 1e30f;    // H_ii of a dead or padded coordinate: its vertex never leaves the code
constexpr unsigned kAbortKey = 0u;    // below the key of every real move (a move's key is at most 0x7FFFFFFF)

__device__ __forceinline__ float rcp_approx(float x) {
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ unsigned atom_add_acq_rel(unsigned* smem_word, unsigned v) {
  unsigned old;
  asm volatile("atom.acq_rel.cta.shared::cta.add.u32 %0, [%1], %2;" : "=r"(old) : "r"(smem_u32(smem_word)), "r"(v) : "memory");
  return old;
}
// a - b on both lanes, correctly rounded (a fused multiply-add with -1 is exact in the product).
__device__ __forceinline__ float2 sub2(float2 a, float2 b) { return __ffma2_rn(b, make_float2(-1.f, -1.f), a); }

// One chunk of 4 coordinates: (hi, lo) += c h with c = c_hi + c_lo, then the best move of each
// coordinate folded into the thread's running best.  a: scale of the chunk (1 when per-channel, which
// runs in code units); nkk = -0.5 / a.
template <int SMODE>
__device__ __forceinline__ void pair_sweep_chunk(float (&hi)[4], float (&lo)[4], const float4 rv, const float4 hd4,
                                                 unsigned qpk, float c_hi, float c_lo, float a, float nkk, float top,
                                                 int k, SweepBest& sb) {
  const float hv[4] = {rv.x, rv.y, rv.z, rv.w};
  const float hdv[4] = {hd4.x, hd4.y, hd4.z, hd4.w};
  const float2 c2 = make_float2(c_hi, c_hi), nc2 = make_float2(-c_hi, -c_hi), ncl2 = make_float2(-c_lo, -c_lo);
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    const float2 h = make_float2(hv[2 * u], hv[2 * u + 1]);
    const float2 g = make_float2(hi[2 * u], hi[2 * u + 1]);
    const float2 l = make_float2(lo[2 * u], lo[2 * u + 1]);
    const float2 hd = make_float2(hdv[2 * u], hdv[2 * u + 1]);
    // c h = p - en exactly (en = p - c_hi h, minus the part of the step below c_hi)
    const float2 p = __fmul2_rn(c2, h);
    float2 en = __ffma2_rn(nc2, h, p);
    if (SMODE != kPerChannel) en = __ffma2_rn(ncl2, h, en);
    // hi + p = s + err exactly
    const float2 s = __fadd2_rn(g, p);
    const float2 z = sub2(s, g);
    const float2 t1 = sub2(s, z);
    const float2 t2 = sub2(g, t1);
    const float2 t3 = sub2(p, z);
    const float2 err = __fadd2_rn(t2, t3);
    const float2 l1 = __fadd2_rn(l, sub2(err, en));
    const float2 gf = __fadd2_rn(s, l1);          // the gradient, rounded once
    hi[2 * u] = s.x; hi[2 * u + 1] = s.y;
    lo[2 * u] = l1.x; lo[2 * u + 1] = l1.y;
    // level of the vertex: q - g / (2 a H_ii), rounded by the addition to 1.5 * 2^23 + q and clamped to the grid
    const float2 nihs = __fmul2_rn(make_float2(nkk, nkk), make_float2(rcp_approx(hd.x), rcp_approx(hd.y)));
    const float2 qmf = make_float2(__uint_as_float(__byte_perm(qpk, kMagicBits, 0x7650 | (2 * u))),
                                   __uint_as_float(__byte_perm(qpk, kMagicBits, 0x7650 | (2 * u + 1))));
    float2 t = __ffma2_rn(gf, nihs, qmf);
    t.x = fminf(fmaxf(t.x, kMagic), top);
    t.y = fminf(fmaxf(t.y, kMagic), top);
    const float2 dr = sub2(t, qmf);
    const float2 d = SMODE == kPerChannel ? dr : __fmul2_rn(make_float2(a, a), dr);
    const float2 dl = __fmul2_rn(__ffma2_rn(d, hd, gf), d);   // change of the loss
    if (dl.x < sb.best) { sb.best = dl.x; sb.bpk = dr.x + (float)((4 * k + 2 * u) * 1024); }
    if (dl.y < sb.best) { sb.best = dl.y; sb.bpk = dr.y + (float)((4 * k + 2 * u + 1) * 1024); }
  }
}

// NTS: stride between chunk slots in shared memory (the largest team of the configuration), so that
// every shared-memory access of a thread is one base address plus a compile-time offset.
template <int NCH, int NTS, int SMODE, bool LO16>
__global__ void __launch_bounds__(NTS, 1) cd_pair_kernel(CdParams p) {
  extern __shared__ __align__(128) unsigned char dyn_smem[];
  __shared__ __align__(8) unsigned long long s_full[NCH];   // piece k of the ring has landed
  __shared__ unsigned s_cnt[NCH];                           // warps done with piece k of the row in the ring
  __shared__ __align__(8) uint2 s_exch[2][32];
  __shared__ int s_col;
  __shared__ int s_jcol[2];                                 // layer column held by each slot
  // private to thread 0 (kept out of everyone's registers)
  __shared__ double s_col_dsum[2], s_my_dsum;
  __shared__ unsigned long long s_committed, s_converged;
  __shared__ float s_a_col[2];

  const int tid = threadIdx.x, NT = blockDim.x;
  const int lane = tid & 31, warp = tid >> 5, nwarps = NT >> 5;
  const int d_in = (int)p.d_in;
  const int nchs = d_in >> 2;                   // chunks of a row
  const float top = kMagic + (float)p.L;
  const float* const Hbase = p.H;
  constexpr int SLOTS = NCH * NTS;
  constexpr int LOB = LO16 ? 8 : 16;            // bytes of the gradient's trailing part per chunk

  // shared memory: ring [NCH][NTS] float4 | H_ii [NCH][NTS] float4 | trailing parts [2][NCH][NTS] | scales [2][ag_count]
  float4* const ring = reinterpret_cast<float4*>(dyn_smem);
  const float4* const ring_t = ring + tid;
  float4* const hd_t = ring + SLOTS + tid;
  unsigned char* const lo_t = dyn_smem + (size_t)2 * SLOTS * 16 + (size_t)tid * LOB;
  float2* const ag_base = reinterpret_cast<float2*>(dyn_smem + (size_t)2 * SLOTS * 16 + (size_t)2 * SLOTS * LOB);
  auto group_of = [&](unsigned i) -> unsigned { return p.g == 1 ? i : __umulhi(i, p.gmagic); };
  const int g4 = SMODE == kGroupFast ? (int)(p.g >> 2) : 1;
  const int ag_first = SMODE == kGroupFast ? tid / g4 : 0;
  const int ag_stride = SMODE == kGroupFast ? NT / g4 : 0;

  auto load_lo = [&](int s, int k, float (&lo)[4]) {
    const unsigned char* a = lo_t + ((size_t)s * SLOTS + (size_t)k * NTS) * LOB;
    if (LO16) {
      const uint2 v = *reinterpret_cast<const uint2*>(a);
      lo[0] = __uint_as_float(v.x << 16); lo[1] = __uint_as_float(v.x & 0xFFFF0000u);
      lo[2] = __uint_as_float(v.y << 16); lo[3] = __uint_as_float(v.y & 0xFFFF0000u);
    } else {
      const float4 v = *reinterpret_cast<const float4*>(a);
      lo[0] = v.x; lo[1] = v.y; lo[2] = v.z; lo[3] = v.w;
    }
  };
  auto store_lo = [&](int s, int k, const float (&lo)[4]) {
    unsigned char* a = lo_t + ((size_t)s * SLOTS + (size_t)k * NTS) * LOB;
    if (LO16) {
      const __nv_bfloat162 b0 = __floats2bfloat162_rn(lo[0], lo[1]), b1 = __floats2bfloat162_rn(lo[2], lo[3]);
      uint2 v;
      v.x = *reinterpret_cast<const unsigned*>(&b0); v.y = *reinterpret_cast<const unsigned*>(&b1);
      *reinterpret_cast<uint2*>(a) = v;
    } else {
      *reinterpret_cast<float4*>(a) = make_float4(lo[0], lo[1], lo[2], lo[3]);
    }
  };

  // slots past the end of the row stay zero in the ring: no copy ever writes there
#pragma unroll
  for (int k = 0; k < NCH; ++k) {
    ring[k * NTS + tid] = make_float4(0.f, 0.f, 0.f, 0.f);
    float4 d = __ldg(reinterpret_cast<const float4*>(p.hdiag) + tid + NT * k);
    d.x = d.x > 0.f ? d.x : kDeadDiag; d.y = d.y > 0.f ? d.y : kDeadDiag;
    d.z = d.z > 0.f ? d.z : kDeadDiag; d.w = d.w > 0.f ? d.w : kDeadDiag;
    hd_t[k * NTS] = d;
  }
  if (tid == 0) {
#pragma unroll
    for (int k = 0; k < NCH; ++k) { mbar_init(smem_u32(&s_full[k]), 1); s_cnt[k] = 0; }
    mbar_fence_init();
  }
  __syncthreads();
  fence_proxy_async_smem();   // the zero fill is in place before the first copy lands

  // bytes of the row piece behind chunk slot k (0 when the slot lies past the row)
  auto piece_bytes = [&](int k) -> uint32_t {
    const int lo = NT * k, hi = min(NT * (k + 1), nchs);
    return hi > lo ? (uint32_t)(hi - lo) * 16u : 0u;
  };
  auto issue_piece = [&](int k, int row) {   // one thread
    const uint32_t bytes = piece_bytes(k);
    if (bytes) {
      const uint32_t bar = smem_u32(&s_full[k]);
      mbar_expect_tx(bar, bytes);
      bulk_load(smem_u32(ring + k * NTS), Hbase + (size_t)row * (size_t)d_in + (size_t)NT * k * 4, bytes, bar);
    }
  };

  // ---- state of the two column slots (uniform over the team unless noted; never indexed at run time) ----
  float hi[2][4 * NCH];        // per thread: leading part of the gradient
  unsigned qp[2][NCH];         // per thread: packed codes
  bool active[2] = {false, false};
  bool has_row[2] = {false, false};   // the slot's next sweep applies a move (needs its row in the ring)
  int irow[2] = {0, 0};               // row of H the slot's next sweep applies
  float c_hi[2] = {0.f, 0.f}, c_lo[2] = {0.f, 0.f};   // twice the step being applied (code units when per-channel)
  int step[2] = {0, 0};
  int ring_owner = -1;         // slot whose row is in the ring or on its way there
  uint32_t ph = 0;             // parity of the copy barriers for the next row
  int xbuf = 0;
  bool aborted = false;
  const int budget = (int)(p.T < 2147483647ll ? p.T : 2147483647ll);
  if (tid == 0) { s_my_dsum = 0.0; s_committed = 0; s_converged = 0; }
  const bool two = p.d_out >= 2ll * gridDim.x;   // too few columns: one per CTA reaches more SMs

  // Takes the next column of the layer into slot S (or leaves the slot inactive).
  auto next_column = [&](auto S) {
    constexpr int s = decltype(S)::value;
    active[s] = false;
    for (;;) {
      __syncthreads();
      if (tid == 0) s_col = atomicAdd(&p.ctr->next_col, 1);
      __syncthreads();
      const long long j = s_col;
      if (j >= p.d_out) return;
      double gscale = 1.0;
      if (SMODE == kPerChannel) {
        const float a = p.scale[j];
        if (!(a > 0.f)) {   // constant column: its grid has one point, nothing can move
          if (tid == 0) ++s_converged;
          continue;
        }
        if (tid == 0) s_a_col[s] = a;
        gscale = 1.0 / (double)a;
      } else {
        float2* ag = ag_base + (size_t)s * p.ag_count;
        for (int t = tid; t < p.ag_count; t += NT) {
          const float a = t < p.ng ? p.scale[(long long)t * p.d_out + j] : 0.f;
          ag[t] = make_float2(a, a > 0.f ? 1.0f / a : 0.f);
        }
      }
      const double* gcol = p.G + j * p.ldg;
      const unsigned char* qcol = p.Qt + j * p.ldq;
#pragma unroll
      for (int k = 0; k < NCH; ++k) {
        const int cs = tid + NT * k;
        double gd[4] = {0.0, 0.0, 0.0, 0.0};
        qp[s][k] = 0;
        if (cs < nchs) {
          const double2 g0 = *reinterpret_cast<const double2*>(gcol + (long long)cs * 4);
          const double2 g1 = *reinterpret_cast<const double2*>(gcol + (long long)cs * 4 + 2);
          gd[0] = g0.x * gscale; gd[1] = g0.y * gscale; gd[2] = g1.x * gscale; gd[3] = g1.y * gscale;
          qp[s][k] = *reinterpret_cast<const unsigned*>(qcol + (long long)cs * 4);
        }
        float lo[4];
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          hi[s][4 * k + v] = (float)gd[v];
          lo[v] = (float)(gd[v] - (double)hi[s][4 * k + v]);
        }
        store_lo(s, k, lo);
      }
      active[s] = true; has_row[s] = false; c_hi[s] = 0.f; c_lo[s] = 0.f; step[s] = 0;
      if (tid == 0) { s_jcol[s] = (int)j; s_col_dsum[s] = 0.0; }
      __syncthreads();   // the scale table is complete
      return;
    }
  };

  if (budget > 0) {
    next_column(std::integral_constant<int, 0>{});
    if (two) next_column(std::integral_constant<int, 1>{});
  }

  while ((active[0] || active[1]) && !aborted) {
#pragma unroll
    for (int s = 0; s < 2; ++s) {
      if (!active[s] || aborted) continue;
      const int o = s ^ 1;
      // ---- sweep of slot s ----
      const bool rowsweep = has_row[s];
      // the next sweep that needs a row is the other slot's, and its row is known: refill behind this sweep
      const bool early = rowsweep && active[o] && has_row[o];
      const int row_o = irow[o];
      const float ch = c_hi[s], cl = c_lo[s];
      bool timed_out = false;
      if (rowsweep && ring_owner != s) {   // cannot happen: the row of this sweep was never requested
        if (tid == 0) atomicExch(p.status, (int)kFlagBadIndex);
        timed_out = true;
      }
      const float2* ag = ag_base + (size_t)s * p.ag_count;
      SweepBest sb;
      sb.init();
      // operands of chunk slot k: the row piece (after its copy has landed), H_ii and the trailing part
      auto fetch = [&](int k, float4& rv, float4& hd, float (&lo)[4]) {
        hd = hd_t[k * NTS];
        load_lo(s, k, lo);
        rv = make_float4(0.f, 0.f, 0.f, 0.f);
        if (rowsweep) {
          if (NT * k < nchs && !mbar_wait_cycles(smem_u32(&s_full[k]), ph, kWaitCycles)) timed_out = true;
          rv = ring_t[k * NTS];
        }
      };
      float4 rv, hd, rv_n, hd_n;
      float lo[4], lo_n[4];
      fetch(0, rv, hd, lo);
#pragma unroll
      for (int k = 0; k < NCH; ++k) {
        if (k + 1 < NCH) fetch(k + 1, rv_n, hd_n, lo_n);   // in flight while chunk k is worked on
        float a = 1.f, nkk = -0.5f;
        if (SMODE == kGroupFast) { const float2 x = ag[ag_first + k * ag_stride]; a = x.x; nkk = -0.5f * x.y; }
        if (SMODE == kGroupAny) {
          const unsigned i = (unsigned)(tid + NT * k) * 4u;
          const float2 x = i < (unsigned)d_in ? ag[group_of(i)] : make_float2(0.f, 0.f);
          a = x.x; nkk = -0.5f * x.y;
        }
        float hk[4] = {hi[s][4 * k], hi[s][4 * k + 1], hi[s][4 * k + 2], hi[s][4 * k + 3]};
        pair_sweep_chunk<SMODE>(hk, lo, rv, hd, qp[s][k], ch, cl, a, nkk, top, k, sb);
        hi[s][4 * k] = hk[0]; hi[s][4 * k + 1] = hk[1]; hi[s][4 * k + 2] = hk[2]; hi[s][4 * k + 3] = hk[3];
        store_lo(s, k, lo);
        if (early) {
          // the last warp to leave piece k hands it to the copy engine for the other column's row
          __syncwarp();
          if (lane == 0) {
            const unsigned before = atom_add_acq_rel(&s_cnt[k], 1u);
            if (before == (unsigned)nwarps - 1u) {
              s_cnt[k] = 0;
              issue_piece(k, row_o);
            }
          }
        }
        if (k + 1 < NCH) {
          rv = rv_n; hd = hd_n;
          lo[0] = lo_n[0]; lo[1] = lo_n[1]; lo[2] = lo_n[2]; lo[3] = lo_n[3];
        }
      }
      if (rowsweep) { ph ^= 1u; ring_owner = early ? o : -1; }

      // ---- team-wide argmin: (decrease, lowest coordinate, lowest level) ----
      unsigned key, packed;
      sweep_candidate(sb, tid, key, packed);
      if (timed_out) { key = kAbortKey; packed = 0u; }
      unsigned m = __reduce_min_sync(0xFFFFFFFFu, key);
      unsigned w = __reduce_min_sync(0xFFFFFFFFu, key == m ? packed : kNoMove);
      if (lane == 0) s_exch[xbuf][warp] = make_uint2(m, w);
      __syncthreads();
      {
        const uint2 x = lane < nwarps ? s_exch[xbuf][lane] : make_uint2(kNoMove, kNoMove);
        m = __reduce_min_sync(0xFFFFFFFFu, x.x);
        w = __reduce_min_sync(0xFFFFFFFFu, x.x == m ? x.y : kNoMove);
        xbuf ^= 1;
      }
      if (m == kAbortKey) { aborted = true; continue; }
      bool col_done = false, converged = false;
      if (m == kNoMove) {          // no move lowers the loss
        col_done = true; converged = true;
      } else {
        const int kstar = (int)(w >> 21), tstar = (int)((w >> 11) & 1023u), vstar = (int)((w >> 9) & 3u);
        const int dri = (int)(w & 511u) - 256;
        const int istar = 4 * (tstar + NT * kstar) + vstar;
        if ((unsigned)istar >= (unsigned)d_in) {  // cannot happen; never follow a bad row index
          if (tid == 0) atomicExch(p.status, (int)kFlagBadIndex);
          col_done = true;
        } else {
          if (tid == tstar) {
            const unsigned dq = (unsigned)dri << (8 * vstar);
#pragma unroll
            for (int k = 0; k < NCH; ++k)
              if (k == kstar) qp[s][k] += dq;
          }
          if (SMODE == kPerChannel) {
            c_hi[s] = (float)(2 * dri); c_lo[s] = 0.f;
          } else {
            const double c = 2.0 * ((double)ag[group_of((unsigned)istar)].x * (double)dri);
            c_hi[s] = (float)c; c_lo[s] = (float)(c - (double)c_hi[s]);
          }
          irow[s] = istar;
          has_row[s] = true;
          if (tid == 0) s_col_dsum[s] += (double)__uint_as_float(~m);
          // budget used up: the gradient after the last move is never read, so no sweep follows it
          if (++step[s] >= budget) col_done = true;
        }
      }
      if (col_done) {
        if (tid == 0) {
          if (converged) ++s_converged;
          s_committed += (unsigned long long)step[s];
          s_my_dsum += SMODE == kPerChannel ? s_col_dsum[s] * ((double)s_a_col[s] * (double)s_a_col[s]) : s_col_dsum[s];
        }
        unsigned char* qcol = p.Qt + (long long)s_jcol[s] * p.ldq;
#pragma unroll
        for (int k = 0; k < NCH; ++k) {
          const int cs = tid + NT * k;
          if (cs < nchs) *reinterpret_cast<unsigned*>(qcol + (long long)cs * 4) = qp[s][k];
        }
        has_row[s] = false;
        if (s == 0) next_column(std::integral_constant<int, 0>{});
        else next_column(std::integral_constant<int, 1>{});
      }
      // ---- the ring is idle: request the row of the next sweep that needs one, if it is known ----
      // (every thread is past its reads of the previous row: the barrier of the argmin lies between)
      if (ring_owner < 0) {
        // the other slot sweeps next when it is active; if that sweep starts a column (no row), this
        // slot's row can land meanwhile
        const bool use_o = active[o] && has_row[o];
        const bool use_s = !use_o && active[s] && has_row[s];
        if (use_o || use_s) {
          const int row = use_o ? irow[o] : irow[s];
          if (nwarps >= NCH) {
            if (lane == 0 && warp < NCH) issue_piece(warp, row);
          } else if (tid == 0) {
#pragma unroll
            for (int k = 0; k < NCH; ++k) issue_piece(k, row);
          }
          ring_owner = use_o ? o : s;
        }
      }
    }
  }

  if (aborted) {
    // let the copies in flight finish before the CTA gives its shared memory back: the row of the sweep
    // that gave up (the barriers' previous phase) and, if it was requested, the row behind it
    if (tid == 0) {
#pragma unroll
      for (int k = 0; k < NCH; ++k) {
        if (!piece_bytes(k)) continue;
        mbar_wait_cycles(smem_u32(&s_full[k]), ph ^ 1u, kWaitCycles);
        if (ring_owner >= 0) mbar_wait_cycles(smem_u32(&s_full[k]), ph, kWaitCycles);
      }
      atomicCAS(p.status, (int)kFlagOk, (int)kFlagWaitTimeout);
    }
    __syncthreads();
  }
  if (tid == 0) {
    if (s_my_dsum != 0.0) atomicAdd(&p.ctr->delta_sum, s_my_dsum);
    if (s_committed) atomicAdd(&p.ctr->committed, s_committed);
    if (s_converged) atomicAdd(&p.ctr->converged, s_converged);
  }
}

template <int NCH, int MAXNT, int SMODE, bool LO16>
cudaError_t launch_cfg(CdParams p, int nt, cudaStream_t st) {
  p.ag_count = SMODE == kPerChannel ? 0 : (int)p.ng;
  if (SMODE == kGroupFast) {
    const int g4 = (int)(p.g >> 2), slots = (nt * NCH + g4 - 1) / g4;
    if (slots > p.ag_count) p.ag_count = slots;
  }
  auto kern = cd_pair_kernel<NCH, MAXNT, SMODE, LO16>;
  int dev = 0, sms = 0, smem_max = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaDeviceGetAttribute(&smem_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  const size_t slots = (size_t)NCH * MAXNT;
  const size_t smem = slots * (16 + 16 + 2 * (LO16 ? 8 : 16)) + 2 * sizeof(float2) * (size_t)p.ag_count;
  cudaFuncAttributes fa;
  cudaError_t e = cudaFuncGetAttributes(&fa, kern);
  if (e != cudaSuccess) return e;
  if (smem + fa.sharedSizeBytes > (size_t)smem_max) return cudaErrorNotSupported;
  e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  long long blocks = sms;
  if (blocks > p.d_out) blocks = p.d_out;
  kern<<<(unsigned)blocks, nt, smem, st>>>(p);
  return cudaGetLastError();
}

template <int NCH, int MAXNT>
cudaError_t launch_mode(const CdParams& p, int nt, cudaStream_t st) {
  const int smode = cd_scale_mode(p, nt);
  // the trailing part of the gradient stays fp32 when that fits beside the ring and H_ii
  const size_t slots = (size_t)NCH * MAXNT;
  const size_t ag = smode == kPerChannel ? 0 : 2 * sizeof(float2) * (size_t)(p.ng + slots / 4 + 1);
  const bool lo16 = slots * 64 + ag + 2048 > 227 * 1024;
  if (smode == kPerChannel)
    return lo16 ? launch_cfg<NCH, MAXNT, kPerChannel, true>(p, nt, st) : launch_cfg<NCH, MAXNT, kPerChannel, false>(p, nt, st);
  if (smode == kGroupFast)
    return lo16 ? launch_cfg<NCH, MAXNT, kGroupFast, true>(p, nt, st) : launch_cfg<NCH, MAXNT, kGroupFast, false>(p, nt, st);
  if (smode == kGroupAny)
    return lo16 ? launch_cfg<NCH, MAXNT, kGroupAny, true>(p, nt, st) : launch_cfg<NCH, MAXNT, kGroupAny, false>(p, nt, st);
  return cudaErrorNotSupported;
}

}  // namespace

// Two columns in flight per SM.  Returns cudaErrorNotSupported when the shape has no such
// configuration (rows not 16-byte aligned, or too long for the state of two columns to fit on an SM).
cudaError_t launch_cd_pair(const CdParams& p, cudaStream_t st) {
  if (p.d_in & 3) return cudaErrorNotSupported;
  if ((reinterpret_cast<uintptr_t>(p.H) & 15) != 0) return cudaErrorNotSupported;
  const long long ch = p.d_in >> 2;
  auto team = [&](long long chunks, int nch) { return (int)((chunks + nch - 1) / nch + 31) / 32 * 32; };
  if (ch <= 2048) return launch_mode<4, 512>(p, team(ch, 4), st);
  if (ch <= 3584) return launch_mode<7, 512>(p, team(ch, 7), st);
  if (ch <= 4608) return launch_mode<9, 512>(p, team(ch, 9), st);
  return cudaErrorNotSupported;
}

}  // namespace cdq
