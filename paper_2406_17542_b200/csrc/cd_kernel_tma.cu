// Greedy coordinate descent (paper: the loop of Algorithm 1; Algorithm 4 for sub-channel
// grids), the variant for rows of H that have to come from HBM (large d_in) and are 16-byte
// aligned (d_in % 4 == 0).
//
// Same step as cd_kernel.cu -- score, argmin, read row i*, update the gradient -- but the row
// H[i*, :] is fetched by one bulk asynchronous copy (cp.async.bulk, no multicast) into shared
// memory, issued by a single thread and completed on one mbarrier.
// The copy engine keeps the whole row in flight at once (loads issued by the threads themselves
// did not: the SM tracks only so many outstanding misses), and the row no longer occupies
// registers.
//
// Waits on the copy barriers are bounded by a cycle count.  A thread whose wait runs out enters the
// argmin with a key that no real move can have; the whole team sees it after the exchange, starts no
// further step or column, waits (bounded) for the copies still in flight, records kFlagWaitTimeout
// in the device status word and returns.
#include "async_copy.cuh"
#include "cd_params.cuh"
#include "cd_sweep.cuh"

namespace cdq {
namespace {

constexpr unsigned kWaitCycles = 400u * 1000u * 1000u;   // about 0.2 s
constexpr unsigned kAbortKey = 0u;    // below the key of every real move (a move's key is at most 0x7FFFFFFF)

// NCH chunk slots per thread; the team covers ceil(d_in / 4) <= NT * NCH chunks.
// ROW16: the rows come from a bf16 copy of H (half the bytes per move); the row's own diagonal element is
// replaced by the exact H_ii, so the iteration is the descent on H with its off-diagonal entries rounded to bf16.
template <int NCH, int MAXNT, int MINB, int SMODE, bool ROW16>
__global__ void __launch_bounds__(MAXNT, MINB) cd_tma_kernel(CdParams p) {
  extern __shared__ __align__(128) unsigned char dyn_smem[];
  __shared__ __align__(8) unsigned long long s_bar;   // completion of the row's copy
  __shared__ __align__(8) uint2 s_exch[2][32];
  __shared__ int s_col;

  const int tid = threadIdx.x, NT = blockDim.x;
  const int lane = tid & 31, warp = tid >> 5, nwarps = NT >> 5;
  const int nchs = (int)(p.d_in >> 2);         // chunks of a row
  const bool exact = nchs == NT * NCH;
  const float top = kMagic + (float)p.L;

  constexpr int CHB = ROW16 ? 8 : 16;                                   // bytes of a chunk of 4 row entries
  // H_ii and 0.5 / H_ii of the team's chunk slots sit in shared memory too: they are the same for every column and
  // every sweep reads them (8 d_in bytes); from L1 they cost more latency, and beside the row buffer of the longest
  // rows the L1 does not hold them.  (148 to 1184 columns, before -> after: 2048 entries 12.4 -> 10.6 ms, 6144
  // 23.4 -> 19.4, 8192 42.1 -> 36.8, 14336 163.7 -> 160.1, 18432 67.5 -> 60.4.)
  unsigned char* row_s = dyn_smem;                                      // [NCH * NT] chunks
  float4* hd_s = reinterpret_cast<float4*>(row_s + (size_t)NCH * NT * CHB);   // [NCH * NT] H_ii
  float4* hs_s = hd_s + NCH * NT;                                             // [NCH * NT] 0.5 / H_ii
  float2* ag_s = reinterpret_cast<float2*>(hs_s + NCH * NT);                  // [ag_count] (a, 1/a), grouped modes
  auto group_of = [&](unsigned i) -> unsigned { return p.g == 1 ? i : __umulhi(i, p.gmagic); };
  const int g4 = SMODE == kGroupFast ? (int)(p.g >> 2) : 1;
  const float2* ag_mine = ag_s + (SMODE == kGroupFast ? tid / g4 : 0);
  const int ag_stride = SMODE == kGroupFast ? NT / g4 : 0;
  auto chunk_scale = [&](int k, float& a, float& ia) {
    a = 1.f; ia = 1.f;
    if (SMODE == kGroupFast) { const float2 ag = ag_mine[k * ag_stride]; a = ag.x; ia = ag.y; }
    if (SMODE == kGroupAny) {
      const unsigned i = (unsigned)(tid + NT * k) * 4u;
      const float2 ag = i < (unsigned)p.d_in ? ag_s[group_of(i)] : make_float2(0.f, 0.f);
      a = ag.x; ia = ag.y;
    }
  };

  // slots past the end of the row stay zero: no copy ever writes there
  for (int t = tid; t < NCH * NT * CHB / 8; t += NT) reinterpret_cast<uint2*>(row_s)[t] = make_uint2(0u, 0u);
  for (int t = tid; t < NCH * NT; t += NT) {   // (the arrays are padded past every team's footprint)
    hd_s[t] = __ldg(reinterpret_cast<const float4*>(p.hdiag) + t);
    hs_s[t] = __ldg(reinterpret_cast<const float4*>(p.hs) + t);
  }
  if (tid == 0) {
    mbar_init(smem_u32(&s_bar), 1);
    mbar_fence_init();
  }
  const uint32_t row_bytes = (uint32_t)nchs * (uint32_t)CHB;
  __syncthreads();
  fence_proxy_async_smem();  // zero fill before the first copy lands

  unsigned long long my_committed = 0, my_converged = 0;
  double my_dsum = 0.0;
  uint32_t phase = 0;   // parity of the copy barriers for the next sweep
  int xbuf = 0;
  bool aborted = false;

  while (!aborted) {
    __syncthreads();  // everyone is done with the previous column
    if (tid == 0) s_col = atomicAdd(&p.ctr->next_col, 1);
    __syncthreads();
    const long long j = s_col;
    if (j >= p.d_out) break;

    // ---- column state ----
    float a_col = 1.f;
    double gscale = 1.0;
    bool frozen = false;
    if (SMODE == kPerChannel) {
      a_col = p.scale[j];
      frozen = !(a_col > 0.f);   // constant column: its grid has one point, nothing can move
      gscale = frozen ? 0.0 : 1.0 / (double)a_col;
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
      const double* gcol = p.G + j * p.ldg;
      const unsigned char* qcol = p.Qt + j * p.ldq;
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
        g[4 * k] = g0.x * gscale; g[4 * k + 1] = g0.y * gscale; g[4 * k + 2] = g1.x * gscale; g[4 * k + 3] = g1.y * gscale;
      }
    }

    // ---- descent ----
    // The first sweep only scores: it "applies" a step of size zero along row 0.
    long long step = 0;
    [[maybe_unused]] bool fix_diag = false;   // ROW16: this thread owns the coordinate of the move being applied ...
    [[maybe_unused]] int kprev = 0, vprev = 0;   // ... in chunk slot kprev, position vprev
    double c2 = 0.0;       // twice the step being applied (code units when per-channel)
    double col_dsum = 0.0;
    bool done = frozen;
    // Requests row `off / d_in` of H.  Called when every thread is past its reads of the previous row (behind the
    // barrier of the argmin, or of the column prologue), and as early as the row is known: what follows the argmin
    // overlaps with the copy.
    auto request_row = [&](long long off) {
      if (tid == 0) {
        const unsigned char* src = ROW16 ? reinterpret_cast<const unsigned char*>(p.H16 + off)
                                         : reinterpret_cast<const unsigned char*>(p.H + off);
        mbar_expect_tx(smem_u32(&s_bar), row_bytes);
        bulk_load(smem_u32(row_s), src, row_bytes, smem_u32(&s_bar));
      }
    };
    if (!done) request_row(0);
    while (!done) {
      SweepBest sb;
      sb.init();
      bool timed_out = false;
#pragma unroll
      for (int k = 0; k < NCH; ++k) {
        const int cs = tid + NT * k;
        const float4 hd = hd_s[cs];
        const float4 hs = hs_s[cs];
        float a, ia;
        chunk_scale(k, a, ia);
        if (k == 0 && !mbar_wait_clock32(smem_u32(&s_bar), phase, kWaitCycles)) timed_out = true;
        float4 rv;
        if constexpr (ROW16) {
          const uint2 rr = reinterpret_cast<const uint2*>(row_s)[cs];
          rv = make_float4(__uint_as_float(rr.x << 16), __uint_as_float(rr.x & 0xFFFF0000u),
                           __uint_as_float(rr.y << 16), __uint_as_float(rr.y & 0xFFFF0000u));
          if (fix_diag && k == kprev) {   // this thread holds the coordinate that moved: its own entry of the row is H_ii
            rv.x = vprev == 0 ? hd.x : rv.x; rv.y = vprev == 1 ? hd.y : rv.y;
            rv.z = vprev == 2 ? hd.z : rv.z; rv.w = vprev == 3 ? hd.w : rv.w;
          }
        } else {
          rv = reinterpret_cast<const float4*>(row_s)[cs];
        }
        double gk[4] = {g[4 * k], g[4 * k + 1], g[4 * k + 2], g[4 * k + 3]};
        sweep_chunk<SMODE>(gk, rv, hd, hs, qp[k], c2, a, ia, top, k, sb);
        g[4 * k] = gk[0]; g[4 * k + 1] = gk[1]; g[4 * k + 2] = gk[2]; g[4 * k + 3] = gk[3];
      }
      phase ^= 1u;
      if (step >= p.T) {   // budget used up (this sweep only brought the gradient up to date)
        if (timed_out) atomicCAS(p.status, (int)kFlagOk, (int)kFlagWaitTimeout);
        break;
      }

      // ---- team-wide argmin: (decrease, lowest coordinate, lowest level) ----
      unsigned key, packed;
      sweep_candidate(sb, tid, key, packed);
      if (timed_out) { key = kAbortKey; packed = 0u; }
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
      if (m == kAbortKey) {   // a copy never landed: wait (bounded) for the pieces of this row, then give up
        if (tid == 0) {
          mbar_wait_clock32(smem_u32(&s_bar), phase ^ 1u, kWaitCycles);
          atomicCAS(p.status, (int)kFlagOk, (int)kFlagWaitTimeout);
        }
        aborted = true;
        break;
      }
      if (m == kNoMove) { done = true; break; }  // no move lowers the loss
      const int kstar = (int)(w >> 21), tstar = (int)((w >> 11) & 1023u), vstar = (int)((w >> 9) & 3u);
      const int dri = (int)(w & 511u) - 256;
      int istar = 4 * (tstar + NT * kstar) + vstar;
      if ((unsigned)istar >= (unsigned)p.d_in) {  // cannot happen; never follow a bad row index
        if (tid == 0) atomicExch(p.status, (int)kFlagBadIndex);
        istar = 0;
      }
      request_row((long long)istar * p.d_in);
      if constexpr (ROW16) { fix_diag = tid == tstar; kprev = kstar; vprev = vstar; }
      if (tid == tstar) {
        const unsigned dq = (unsigned)dri << (8 * vstar);
#pragma unroll
        for (int k = 0; k < NCH; ++k)
          if (k == kstar) qp[k] += dq;
      }
      float astar = 1.f;
      if (SMODE != kPerChannel) astar = ag_s[group_of((unsigned)istar)].x;
      c2 = 2.0 * ((double)astar * (double)dri);
      if (tid == 0) col_dsum += (double)__uint_as_float(~m);
      ++step;
    }
    if (aborted) break;
    if (tid == 0) {
      if (done) ++my_converged;
      my_committed += (unsigned long long)step;
      my_dsum += SMODE == kPerChannel ? col_dsum * ((double)a_col * (double)a_col) : col_dsum;
    }

    // ---- write the codes back, and the gradient of the result (weight units) ----
    if (!frozen) {
      unsigned char* qcol = p.Qt + j * p.ldq;
      double* gcol = p.G + j * p.ldg;
      const double ga = SMODE == kPerChannel ? (double)a_col : 1.0;
#pragma unroll
      for (int k = 0; k < NCH; ++k) {
        const int cs = tid + NT * k;
        if (exact || cs < nchs) {
          *reinterpret_cast<unsigned*>(qcol + (long long)cs * 4) = qp[k];
          *reinterpret_cast<double2*>(gcol + (long long)cs * 4) = make_double2(g[4 * k] * ga, g[4 * k + 1] * ga);
          *reinterpret_cast<double2*>(gcol + (long long)cs * 4 + 2) = make_double2(g[4 * k + 2] * ga, g[4 * k + 3] * ga);
        }
      }
    }
  }

  if (tid == 0) {
    if (my_dsum != 0.0) atomicAdd(&p.ctr->delta_sum, my_dsum);
    if (my_committed) atomicAdd(&p.ctr->committed, my_committed);
    if (my_converged) atomicAdd(&p.ctr->converged, my_converged);
  }
}

template <int NCH, int MAXNT, int MINB, int SMODE, bool ROW16>
cudaError_t launch_cfg(CdParams p, int nt, cudaStream_t st) {
  p.ag_count = (int)p.ng;
  if (SMODE == kGroupFast) {
    const int g4 = (int)(p.g >> 2), slots = (nt * NCH + g4 - 1) / g4;
    if (slots > p.ag_count) p.ag_count = slots;
  }
  auto kern = cd_tma_kernel<NCH, MAXNT, MINB, SMODE, ROW16>;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const size_t smem = (size_t)NCH * nt * (ROW16 ? 8 : 16) + (size_t)NCH * nt * 32 +
                      (SMODE == kPerChannel ? 0 : sizeof(float2) * (size_t)p.ag_count);
  cudaError_t e;
  {   // rows, tables and a long list of group scales together can exceed what a block may have (18432 entries in
      // groups of 16, say): the caller then takes the kernel that reads its rows and tables through the caches
    cudaFuncAttributes fa{};
    int optin = 0;
    e = cudaFuncGetAttributes(&fa, kern);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e != cudaSuccess) return e;
    if (smem + fa.sharedSizeBytes > (size_t)optin) return cudaErrorNotSupported;
  }
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

template <int NCH, int MAXNT, int MINB>
cudaError_t launch_mode(const CdParams& p, int nt, cudaStream_t st) {
  const int smode = cd_scale_mode(p, nt);
  if (p.H16) {
    if (smode == kPerChannel) return launch_cfg<NCH, MAXNT, MINB, kPerChannel, true>(p, nt, st);
    if (smode == kGroupFast) return launch_cfg<NCH, MAXNT, MINB, kGroupFast, true>(p, nt, st);
    if (smode == kGroupAny) return launch_cfg<NCH, MAXNT, MINB, kGroupAny, true>(p, nt, st);
    return cudaErrorNotSupported;
  }
  if (smode == kPerChannel) return launch_cfg<NCH, MAXNT, MINB, kPerChannel, false>(p, nt, st);
  if (smode == kGroupFast) return launch_cfg<NCH, MAXNT, MINB, kGroupFast, false>(p, nt, st);
  if (smode == kGroupAny) return launch_cfg<NCH, MAXNT, MINB, kGroupAny, false>(p, nt, st);
  return cudaErrorNotSupported;
}

}  // namespace

cudaError_t launch_cd_tma(const CdParams& p, cudaStream_t st) {
  if (p.d_in & 3) return cudaErrorNotSupported;
  if ((reinterpret_cast<uintptr_t>(p.H) & 15) != 0) return cudaErrorNotSupported;
  if (p.H16 && ((p.d_in & 7) != 0 || (reinterpret_cast<uintptr_t>(p.H16) & 15) != 0)) return cudaErrorNotSupported;
  const long long ch = p.d_in >> 2;
  auto team = [&](long long chunks, int nch) { return (int)((chunks + nch - 1) / nch + 31) / 32 * 32; };
  // (called for rows of more than 1536 entries)  Rows up to 8192 entries: several teams per SM.
  if (ch <= 1024) return launch_mode<8, 128, 4>(p, team(ch, 8), st);
  if (ch <= 2048) return launch_mode<8, 256, 2>(p, team(ch, 8), st);
  // Longer rows: one team per SM.  Few threads with many chunks each beat many threads with few (no spills, a
  // cheaper argmin exchange, fixed costs per thread spread over more state), and a team of full warps in equal
  // numbers per scheduler beats a ragged one.  With H_ii and 0.5 / H_ii in shared memory eight warps hide the
  // latencies that are left, so rows up to 14336 entries take 256 threads with 9 to 14 chunks each; beyond that the
  // registers of a 256-thread team run out (15 and 16 chunks measured 3 % slower, 18 chunks 15 %) and the team is the
  // smallest of 10..12 x 384 and 8 x 512 chunk slots that holds the row.  Cycles per move and SM against the
  // 4 x 896 / 6 x 768 teams of an earlier version, which also read the tables through L1: d_in 10240 4049 (4813),
  // 11008 4038 (5079), 14336 4892 (5903), 15360 5531 (7482), 16384 5879 (8022), 18432 6416 (8418).
  if (ch <= 2304) return launch_mode<9, 256, 1>(p, team(ch, 9), st);
  if (ch <= 2560) return launch_mode<10, 256, 1>(p, team(ch, 10), st);
  if (ch <= 2816) return launch_mode<11, 256, 1>(p, team(ch, 11), st);
  if (ch <= 3072) return launch_mode<12, 256, 1>(p, team(ch, 12), st);
  if (ch <= 3328) return launch_mode<13, 256, 1>(p, team(ch, 13), st);
  if (ch <= 3584) return launch_mode<14, 256, 1>(p, team(ch, 14), st);
  if (ch <= 3840) return launch_mode<10, 384, 1>(p, team(ch, 10), st);
  if (ch <= 4096) return launch_mode<8, 512, 1>(p, team(ch, 8), st);
  if (ch <= 4224) return launch_mode<11, 384, 1>(p, team(ch, 11), st);
  if (ch <= 4608) return launch_mode<12, 384, 1>(p, team(ch, 12), st);
  return cudaErrorNotSupported;
}

}  // namespace cdq
