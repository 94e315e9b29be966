// Greedy coordinate descent (paper: Algorithm 1 lines 4-8; Algorithm 4 for sub-channel
// grids), the variant for layers whose rows of H are 16-byte aligned (d_in % 4 == 0).
//
// Same step as cd_kernel.cu -- score, argmin, read row i*, update the gradient -- with two
// changes that matter once a row of H no longer comes out of L2 in a microsecond:
//
//   * The row H[i*, :] is fetched by bulk asynchronous copies (cp.async.bulk, no multicast)
//     into shared memory, one copy and one mbarrier per chunk slot of the team, issued by a
//     single thread.  The copy engine keeps the whole row in flight at once; loads issued by
//     the threads themselves did not (the SM tracks only so many outstanding misses), and the
//     row no longer occupies 32 registers per thread.
//
//   * A column can be split over a thread-block cluster of S CTAs (S SMs): CTA r owns the
//     coordinates [r d_in/S, (r+1) d_in/S).  An SM then hosts slices of S different columns
//     whose steps are out of phase, so one slice's row fetch overlaps another slice's sweep;
//     the on-chip state per SM is the same as with one whole column.  The argmin crosses the
//     cluster once per step: every warp writes its candidate into every CTA's exchange
//     table (st.shared::cluster), one cluster barrier, and every CTA reduces the same table.
//
// Waits on the copy barriers are bounded; when one runs out the kernel records
// kFlagWaitTimeout in the device status word and carries on (its results are then void) so
// that no CTA of a cluster is left waiting at a barrier for one that has gone.
#include "cd_params.cuh"

namespace cdq {
namespace {

constexpr uint32_t kSpinLimit = 1u << 24;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait; false if it ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t it = 0; it < kSpinLimit; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
// 1-D bulk copy global -> this CTA's shared memory; bytes % 16 == 0, both addresses 16-byte aligned.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_cluster_v2(uint32_t addr, unsigned a, unsigned b) {
  asm volatile("st.shared::cluster.v2.u32 [%0], {%1, %2};" ::"r"(addr), "r"(a), "r"(b) : "memory");
}
__device__ __forceinline__ void st_cluster_u32(uint32_t addr, unsigned a) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(a) : "memory");
}
template <int S>
__device__ __forceinline__ void team_sync() {
  if (S == 1) __syncthreads();
  else {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  }
}

// NCH chunk slots per thread, S CTAs per column.  S > 1 needs d_in == S * 4 * NT * NCH.
template <int NCH, int MAXNT, int MINB, int SMODE, int S>
__global__ void __launch_bounds__(MAXNT, MINB) cd_tma_kernel(CdParams p) {
  extern __shared__ __align__(128) unsigned char dyn_smem[];
  __shared__ __align__(8) unsigned long long s_bar[NCH];
  __shared__ __align__(8) uint2 s_exch[2][32];
  __shared__ int s_col;

  const int tid = threadIdx.x, NT = blockDim.x;
  const int lane = tid & 31, warp = tid >> 5, nwarps = NT >> 5;
  const unsigned rank = S > 1 ? cluster_ctarank() : 0u;
  const int dsl = (int)(p.d_in / S);          // coordinates of this CTA's slice
  const int nchs = dsl >> 2;                   // chunks of the slice
  const int c0 = (int)rank * dsl;              // first coordinate of the slice
  const bool exact = nchs == NT * NCH;
  const float topf = kMagic + (float)p.L;

  float4* row_s = reinterpret_cast<float4*>(dyn_smem);                  // [NCH * NT]
  float2* ag_s = reinterpret_cast<float2*>(row_s + (size_t)NCH * NT);  // [ag_count] (a, 1/a), grouped modes
  auto group_of = [&](unsigned i) -> unsigned { return p.g == 1 ? i : __umulhi(i, p.gmagic); };
  const int g4 = SMODE == kGroupFast ? (int)(p.g >> 2) : 1;
  const float2* ag_mine = ag_s + (SMODE == kGroupFast ? ((c0 >> 2) + tid) / g4 : 0);
  const int ag_stride = SMODE == kGroupFast ? NT / g4 : 0;

  for (int t = tid; t < NCH * NT; t += NT) row_s[t] = make_float4(0.f, 0.f, 0.f, 0.f);
  if (tid == 0) {
#pragma unroll
    for (int k = 0; k < NCH; ++k) mbar_init(smem_u32(&s_bar[k]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // bytes of the row piece behind chunk slot k (0 when the slot lies past the slice)
  auto piece_bytes = [&](int k) -> uint32_t {
    const int lo = NT * k, hi = min(NT * (k + 1), nchs);
    return hi > lo ? (uint32_t)(hi - lo) * 16u : 0u;
  };
  __syncthreads();
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // zero fill before the first copy lands

  unsigned long long my_committed = 0, my_converged = 0;
  double my_dsum = 0.0;
  uint32_t phase = 0;   // parity of the copy barriers for the next sweep
  int xbuf = 0;
  bool timed_out = false;

  for (;;) {
    team_sync<S>();  // everyone is done with the previous column (s_col, exchange table)
    if (rank == 0 && tid == 0) {
      const int jn = atomicAdd(&p.ctr->next_col, 1);
      if (S == 1) s_col = jn;
      else {
#pragma unroll
        for (int r = 0; r < S; ++r) st_cluster_u32(map_to_cta(smem_u32(&s_col), r), (unsigned)jn);
      }
    }
    team_sync<S>();
    const long long j = s_col;
    if (j >= p.d_out) break;

    // ---- column state ----
    float a_col = 1.f;
    double inv_a = 1.0;
    bool frozen = false;
    if (SMODE == kPerChannel) {
      a_col = p.scale[j];
      frozen = !(a_col > 0.f);   // constant column: its grid has one point, nothing can move
      inv_a = frozen ? 0.0 : 1.0 / (double)a_col;
    } else {
      for (int t = tid; t < p.ag_count; t += NT) {
        const float a = t < p.ng ? p.scale[(long long)t * p.d_out + j] : 0.f;
        ag_s[t] = make_float2(a, a > 0.f ? 1.0f / a : 0.f);
      }
      __syncthreads();
    }
    double g[4 * NCH];
    unsigned qp[NCH];
    {
      const double* gcol = p.G + j * p.ldg + c0;
      const unsigned char* qcol = p.Qt + j * p.ldq + c0;
#pragma unroll
      for (int k = 0; k < NCH; ++k) {
        const int cs = tid + NT * k;
        double2 g0 = make_double2(0.0, 0.0), g1 = g0;
        qp[k] = 0;
        if (exact || cs < nchs) {
          g0 = *reinterpret_cast<const double2*>(gcol + (long long)cs * 4);
          g1 = *reinterpret_cast<const double2*>(gcol + (long long)cs * 4 + 2);
          qp[k] = *reinterpret_cast<const unsigned*>(qcol + (long long)cs * 4);
        }
        g[4 * k] = g0.x * inv_a; g[4 * k + 1] = g0.y * inv_a; g[4 * k + 2] = g1.x * inv_a; g[4 * k + 3] = g1.y * inv_a;
      }
    }

    // ---- descent ----
    // The first sweep only scores: it "applies" a step of size zero along row 0.
    long long step = 0;
    long long rowoff = 0;
    double c2 = 0.0;       // twice the step being applied (code units when per-channel)
    double col_dsum = 0.0;
    bool done = frozen;
    while (!done) {
      // all threads of the CTA are past their reads of the previous row (team barrier in the
      // argmin, or the barriers of the column prologue): the copies may overwrite it
      if (tid == 0) {
        const float* src = p.H + rowoff + c0;
#pragma unroll
        for (int k = 0; k < NCH; ++k) {
          const uint32_t bytes = piece_bytes(k);
          if (bytes) {
            const uint32_t bar = smem_u32(&s_bar[k]);
            mbar_expect_tx(bar, bytes);
            bulk_load(smem_u32(row_s + (size_t)NT * k), src + (size_t)NT * k * 4, bytes, bar);
          }
        }
      }
      float best = 0.f, bpk = 0.f;
#pragma unroll
      for (int k = 0; k < NCH; ++k) {
        const int cs = tid + NT * k;
        const float4 hd = __ldg(reinterpret_cast<const float4*>(p.hdiag + c0) + cs);
        const float4 hi = __ldg(reinterpret_cast<const float4*>(p.half_inv + c0) + cs);
        float a = 1.f, ia = 1.f;
        if (SMODE == kGroupFast) {
          const float2 ag = ag_mine[k * ag_stride];
          a = ag.x; ia = ag.y;
        }
        if (exact || NT * k < nchs) {
          if (!mbar_wait(smem_u32(&s_bar[k]), phase)) timed_out = true;
        }
        const float4 rv = row_s[cs];
        const float hv[4] = {rv.x, rv.y, rv.z, rv.w};
        const float hdv[4] = {hd.x, hd.y, hd.z, hd.w};
        const float hiv[4] = {hi.x, hi.y, hi.z, hi.w};
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          const int e = 4 * k + v;
          if (SMODE == kGroupAny) {
            const unsigned i = (unsigned)c0 + (unsigned)cs * 4u + v;
            const float2 ag = i < (unsigned)p.d_in ? ag_s[group_of(i)] : make_float2(0.f, 0.f);
            a = ag.x; ia = ag.y;
          }
          g[e] = fma(c2, (double)hv[v], g[e]);
          const float gf = (float)g[e];
          const float qmf = __uint_as_float(__byte_perm(qp[k], kMagicBits, 0x7650 | v));  // kMagic + q
          // kMagic + rint(vertex of the coordinate's parabola), clamped to the grid
          float t = SMODE == kPerChannel ? fmaf(-gf, hiv[v], qmf) : fmaf(-gf, ia * hiv[v], qmf);
          t = fminf(fmaxf(t, kMagic), topf);
          const float dr = t - qmf;
          const float d = SMODE == kPerChannel ? dr : a * dr;
          const float dl = fmaf(d, hdv[v], gf) * d;
          if (dl < best) { best = dl; bpk = dr + (float)(e * 1024); }
        }
      }
      phase ^= 1u;
      if (step >= p.T) break;

      // team-wide argmin: (decrease, lowest coordinate, lowest level).  `best` is negative or
      // zero; the complement of a negative float's bits orders the candidates.
      unsigned packed = kNoMove;
      if (best < 0.f) {
        const int ipk = (int)bpk;
        const int e = (ipk + 512) >> 10;
        const int drq = ipk - (e << 10);
        // (slice, chunk slot, thread, coordinate in chunk) orders like the coordinate index
        packed = (rank << 26) | ((unsigned)(e >> 2) << 21) | ((unsigned)tid << 11) | ((unsigned)(e & 3) << 9) |
                 (unsigned)(drq + 256);
      }
      unsigned key = best < 0.f ? ~__float_as_uint(best) : kNoMove;
      unsigned m = __reduce_min_sync(0xFFFFFFFFu, key);
      unsigned w = __reduce_min_sync(0xFFFFFFFFu, key == m ? packed : kNoMove);
      if (S == 1 && nwarps == 1) {
        __syncwarp();
      } else {
        const int nslots = S * nwarps;
        if (lane == 0) {
          if (S == 1) s_exch[xbuf][warp] = make_uint2(m, w);
          else {
            const uint32_t slot = smem_u32(&s_exch[xbuf][rank * nwarps + warp]);
#pragma unroll
            for (int r = 0; r < S; ++r) st_cluster_v2(map_to_cta(slot, r), m, w);
          }
        }
        team_sync<S>();
        const uint2 x = lane < nslots ? s_exch[xbuf][lane] : make_uint2(kNoMove, kNoMove);
        m = __reduce_min_sync(0xFFFFFFFFu, x.x);
        w = __reduce_min_sync(0xFFFFFFFFu, x.x == m ? x.y : kNoMove);
        xbuf ^= 1;
      }
      if (m == kNoMove) { done = true; break; }  // no move lowers the loss
      const unsigned rstar = w >> 26;
      const int kstar = (int)((w >> 21) & 31u), tstar = (int)((w >> 11) & 1023u), vstar = (int)((w >> 9) & 3u);
      const int dri = (int)(w & 511u) - 256;
      int istar = (int)rstar * dsl + 4 * (tstar + NT * kstar) + vstar;
      if ((unsigned)istar >= (unsigned)p.d_in) {  // cannot happen; never follow a bad row index
        if (tid == 0) atomicExch(p.status, (int)kFlagBadIndex);
        istar = 0;
      }
      if (rank == rstar && tid == tstar) {
        const unsigned dq = (unsigned)dri << (8 * vstar);
#pragma unroll
        for (int k = 0; k < NCH; ++k)
          if (k == kstar) qp[k] += dq;
      }
      float astar = 1.f;
      if (SMODE != kPerChannel) astar = ag_s[group_of((unsigned)istar)].x;
      c2 = 2.0 * ((double)astar * (double)dri);
      rowoff = (long long)istar * p.d_in;
      if (tid == 0) col_dsum += (double)__uint_as_float(~m);
      ++step;
    }
    if (rank == 0 && tid == 0) {
      if (done) ++my_converged;
      my_committed += (unsigned long long)step;
      my_dsum += SMODE == kPerChannel ? col_dsum * ((double)a_col * (double)a_col) : col_dsum;
    }

    // ---- write the codes back ----
    if (!frozen) {
      unsigned char* qcol = p.Qt + j * p.ldq + c0;
#pragma unroll
      for (int k = 0; k < NCH; ++k) {
        const int cs = tid + NT * k;
        if (exact || cs < nchs) *reinterpret_cast<unsigned*>(qcol + (long long)cs * 4) = qp[k];
      }
    }
  }

  if (timed_out) atomicExch(p.status, (int)kFlagWaitTimeout);
  if (rank == 0 && tid == 0) {
    if (my_dsum != 0.0) atomicAdd(&p.ctr->delta_sum, my_dsum);
    if (my_committed) atomicAdd(&p.ctr->committed, my_committed);
    if (my_converged) atomicAdd(&p.ctr->converged, my_converged);
  }
  if (S > 1) team_sync<S>();  // no CTA leaves while a peer may still write into its shared memory
}

template <int NCH, int MAXNT, int MINB, int SMODE, int S>
cudaError_t launch_cfg(CdParams p, int nt, cudaStream_t st) {
  p.ag_count = (int)p.ng;
  if (SMODE == kGroupFast) {
    const int g4 = (int)(p.g >> 2), slots = (int)((p.d_in / 4 + (long long)nt * NCH + g4 - 1) / g4);
    if (slots > p.ag_count) p.ag_count = slots;
  }
  auto kern = cd_tma_kernel<NCH, MAXNT, MINB, SMODE, S>;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const size_t smem = (size_t)NCH * nt * sizeof(float4) + (SMODE == kPerChannel ? 0 : sizeof(float2) * (size_t)p.ag_count);
  cudaError_t e;
  if (smem > 48 * 1024) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg{};
  cfg.blockDim = dim3((unsigned)nt);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = S; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  long long teams;
  if (S == 1) {
    int per_sm = 1;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, nt, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) return cudaErrorInvalidConfiguration;
    teams = (long long)sms * per_sm;
  } else {
    cfg.gridDim = dim3((unsigned)(S * sms));
    int clusters = 0;
    e = cudaOccupancyMaxActiveClusters(&clusters, kern, &cfg);
    if (e != cudaSuccess) return e;
    if (clusters < 1) return cudaErrorInvalidConfiguration;
    teams = clusters;
  }
  if (teams > p.d_out) teams = p.d_out;
  cfg.gridDim = dim3((unsigned)(teams * S));
  return cudaLaunchKernelEx(&cfg, kern, p);
}

template <int NCH, int MAXNT, int MINB, int S>
cudaError_t launch_mode(const CdParams& p, int nt, cudaStream_t st) {
  int smode = kPerChannel;
  if (p.ng > 1) {
    // kGroupFast: a thread's chunk slots stride through the scale table, and a slice starts on a group boundary
    const bool fast = (p.g & 3) == 0 && nt % (int)(p.g >> 2) == 0 && (p.d_in / S) % p.g == 0;
    smode = fast ? kGroupFast : kGroupAny;
  }
  if (smode == kPerChannel) return launch_cfg<NCH, MAXNT, MINB, kPerChannel, S>(p, nt, st);
  if (smode == kGroupFast) return launch_cfg<NCH, MAXNT, MINB, kGroupFast, S>(p, nt, st);
  if (S == 1) return launch_cfg<NCH, MAXNT, MINB, kGroupAny, 1>(p, nt, st);
  return cudaErrorNotSupported;
}

}  // namespace

// Team shapes.  A slice of ch = d_in / (4 S) chunks needs ch <= NT * NCH, and for S > 1 equality.
cudaError_t launch_cd_tma(const CdParams& p, cudaStream_t st) {
  if (p.d_in & 3) return cudaErrorNotSupported;
  if ((reinterpret_cast<uintptr_t>(p.H) & 15) != 0) return cudaErrorNotSupported;
  const long long ch = p.d_in >> 2;
  auto team = [&](long long chunks, int nch) { return (int)((chunks + nch - 1) / nch + 31) / 32 * 32; };
  if (ch <= 128) return launch_mode<2, 64, 8, 1>(p, team(ch, 2), st);
  if (ch <= 1024) return launch_mode<4, 256, 3, 1>(p, team(ch, 4), st);
  if (ch <= 2048) return launch_mode<8, 256, 2, 1>(p, team(ch, 8), st);
  // large rows (HBM-served): split over a cluster of 4 when the shape divides, else one CTA
  if (ch % 4 == 0) {
    const long long c4 = ch / 4;
    if (c4 % 7 == 0 && (c4 / 7) % 32 == 0 && c4 / 7 <= 256) return launch_mode<7, 256, 2, 4>(p, (int)(c4 / 7), st);
    if (c4 % 8 == 0 && (c4 / 8) % 32 == 0 && c4 / 8 <= 256) return launch_mode<8, 256, 2, 4>(p, (int)(c4 / 8), st);
    if (c4 % 9 == 0 && (c4 / 9) % 32 == 0 && c4 / 9 <= 256) return launch_mode<9, 256, 2, 4>(p, (int)(c4 / 9), st);
  }
  if (ch <= 3584) return launch_mode<8, 448, 1, 1>(p, team(ch, 8), st);
  if (ch <= 4608) return launch_mode<8, 576, 1, 1>(p, team(ch, 8), st);
  return cudaErrorNotSupported;
}

}  // namespace cdq
