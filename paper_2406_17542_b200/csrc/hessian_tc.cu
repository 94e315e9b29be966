// H = X^T X on the 5th-generation tensor cores (paper: Section 3 "Notation"; Algorithm 1).
// X is [n, d_in] bf16 row-major, H is [d_in, d_in] fp32.
//
// The contraction runs over the calibration rows: D[M,N] += A[M,K] B[K,N] with A = X^T,
// B = X, K = n.  Both operands are slices of the same matrix and are "MN-major" for the
// tensor core (d_in is the contiguous dimension), so one TMA tensor map serves both.
//
//   * tile 128 x 256 per CTA, one tcgen05.mma (kind::f16, bf16 in, fp32 accumulate in TMEM)
//     per 16 rows of X; only tiles that touch the lower triangle are computed (SYRK), the
//     mirror image is written by the reduction kernel;
//   * TMA boxes of 64 columns x 64 rows with the 128-byte swizzle land in shared memory in
//     exactly the canonical MN-major layout: 64-column blocks LBO = 8 KB apart, groups of
//     8 rows SBO = 1 KB apart;
//   * 4-stage TMA ring (full/empty mbarriers), two 256-column TMEM accumulators so that the
//     epilogue of one tile overlaps the MMAs of the next, persistent CTAs over a static
//     round-robin list of (K-split, tile) units;
//   * warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner, warps 2-5 = epilogue;
//   * split-K partial tiles go to the caller's workspace and are summed in a fixed order, so
//     the result does not depend on scheduling.
// Every mbarrier wait is bounded: on expiry the kernel records kFlagWaitTimeout in the
// device status word, lets the other roles drain, frees its TMEM and returns.
#include <cuda.h>

#include "async_copy.cuh"
#include "common.cuh"

namespace cdq {
namespace tc {

constexpr int BM = 128, BN = 256, BK = 64, STAGES = 4;
constexpr int BOX_COLS = 64;                       // 64 bf16 = 128 bytes = one swizzle row
constexpr int BOX_BYTES = BOX_COLS * BK * 2;       // 8192
constexpr int A_BYTES = BM * BK * 2;               // 2 boxes
constexpr int B_BYTES = BN * BK * 2;               // 4 boxes
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;     // 49152
constexpr int TILE_ELEMS = BM * BN;
// K blocks (of BK rows) that one TMEM accumulator takes before the epilogue drains it.  The tensor core's
// fp32 accumulation truncates, so the error of an entry grows with the number of accumulation steps behind
// it: with all 131072 rows of a layer in one accumulator the entries came out up to 7e-4 (of sqrt(H_ii H_jj))
// low, with 262144 rows past the 1e-3 the Hessian is allowed.  256 blocks = 16384 rows per accumulator bound
// that near 6e-5; the chunks of a tile are added up by the epilogue with round-to-nearest fp32 adds.
constexpr int KCHUNK = 256;
constexpr int NUM_THREADS = 192;
constexpr int TMEM_COLS = 512;
constexpr uint32_t SPIN_LIMIT = 1u << 22;
constexpr size_t SMEM_BYTES = 1024 /*alignment slack*/ + (size_t)STAGES * STAGE_BYTES + 256;

struct Params {
  long long n, d_in;
  int tiles_m, ntiles, splits, kblocks;
  float* partials;   // [splits][ntiles][BM*BN]
  const int2* tiles; // [ntiles] (tm, tn) in the order the tiles are handed out
  int* status;
};

// Bounded wait of this pipeline's roles (see async_copy.cuh).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  return mbar_wait_or_abort(bar, parity, abort_flag, SPIN_LIMIT);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar)
      : "memory");
}

// Shared-memory matrix descriptor, MN-major, 128-byte swizzle:
// bits [0,14) start >> 4, [16,30) LBO >> 4, [32,46) SBO >> 4, [46,48) version 1, [61,64) layout 2.
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr) {
  constexpr uint64_t LBO = (uint64_t)(BOX_BYTES >> 4);   // between 64-column blocks
  constexpr uint64_t SBO = (uint64_t)(1024 >> 4);        // between groups of 8 rows
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (LBO << 16) | (SBO << 32) | (1ull << 46) | (2ull << 61);
}

// Instruction descriptor: fp32 accumulate, bf16 A and B, both MN-major, N = 256, M = 128.
constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) |
                           ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

__device__ __forceinline__ void mma_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(IDESC), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}

// Order in which the lower-triangle tiles (tn <= tm / 2) are handed out: bands of BAND tile
// rows, and inside a band column by column.  Consecutive tiles -- the ones the persistent CTAs
// work on at the same time -- then form a compact block of about BAND x (SMs / BAND) tiles that
// shares its operand panels in L2, instead of a strip that spans every column of X.
constexpr int BAND = 16;
__global__ void hessian_tile_order_kernel(int tiles_m, int2* __restrict__ tiles) {
  if (blockIdx.x != 0 || threadIdx.x != 0) return;
  int t = 0;
  for (int r0 = 0; r0 < tiles_m; r0 += BAND) {
    const int r1 = min(tiles_m, r0 + BAND);
    for (int tn = 0; tn <= (r1 - 1) / 2; ++tn)
      for (int tm = max(r0, 2 * tn); tm < r1; ++tm) tiles[t++] = make_int2(tm, tn);
  }
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
hessian_tc_kernel(const __grid_constant__ CUtensorMap tmap, Params p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t tiles = (raw + 1023u) & ~1023u;           // stage buffers, 1 KB aligned
  unsigned char* ctrl = smem_raw + (tiles - raw) + (size_t)STAGES * STAGE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(ctrl);      // full[4] empty[4] tfull[2] tempty[2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(ctrl + 128);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl + 136);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto tfull_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + b); };
  auto tempty_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + 2 + b); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"((uint32_t)TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  const int units = p.ntiles * p.splits;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int issued = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
        const int s = u / p.ntiles, t = u - s * p.ntiles;
        const int2 tc = p.tiles[t];
        const int tm = tc.x, tn = tc.y;
        const int kb0 = (int)((long long)s * p.kblocks / p.splits), kb1 = (int)((long long)(s + 1) * p.kblocks / p.splits);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          mbar_expect_tx(full_bar(stage), STAGE_BYTES);
          const uint32_t a_dst = tiles + (uint32_t)stage * STAGE_BYTES;
          const uint32_t b_dst = a_dst + A_BYTES;
#pragma unroll
          for (int b = 0; b < BM / BOX_COLS; ++b)
            tma_load_2d(a_dst + b * BOX_BYTES, &tmap, tm * BM + b * BOX_COLS, kb * BK, full_bar(stage));
#pragma unroll
          for (int b = 0; b < BN / BOX_COLS; ++b)
            tma_load_2d(b_dst + b * BOX_BYTES, &tmap, tn * BN + b * BOX_COLS, kb * BK, full_bar(stage));
          ++issued;
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // let copies already in flight land before the CTA goes away (bounded)
        const int pending = issued < STAGES ? issued : STAGES;
        for (int q = 0; q < pending; ++q) {
          int s2 = stage - 1 - q;
          uint32_t ph2 = phase;
          if (s2 < 0) { s2 += STAGES; ph2 ^= 1u; }
          for (uint32_t it = 0; it < SPIN_LIMIT; ++it)
            if (mbar_try_wait(full_bar(s2), ph2)) break;
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int buf = 0;
      uint32_t tphase = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
        const int s = u / p.ntiles;
        const int kb0 = (int)((long long)s * p.kblocks / p.splits), kb1 = (int)((long long)(s + 1) * p.kblocks / p.splits);
        // one accumulator takes at most KCHUNK K blocks (see KCHUNK); the epilogue adds the chunks up
        for (int kc0 = kb0; kc0 < kb1 && ok; kc0 += KCHUNK) {
          const int kc1 = min(kb1, kc0 + KCHUNK);
          if (!mbar_wait(tempty_bar(buf), tphase ^ 1u, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t tmem_d = tmem_base + (uint32_t)buf * BN;
          for (int kb = kc0; kb < kc1; ++kb) {
            if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a_src = tiles + (uint32_t)stage * STAGE_BYTES;
            const uint32_t b_src = a_src + A_BYTES;
#pragma unroll
            for (int kk = 0; kk < BK / 16; ++kk) {
              // 16 rows of X = two 8-row swizzle groups = 2 KB further into every 64-column block
              const uint64_t adesc = make_desc(a_src + kk * 2048);
              const uint64_t bdesc = make_desc(b_src + kk * 2048);
              mma_f16(tmem_d, adesc, bdesc, (kb > kc0 || kk > 0) ? 1u : 0u);
            }
            mma_commit(empty_bar(stage));   // frees the stage once these MMAs have read it
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          mma_commit(tfull_bar(buf));       // accumulator complete
          if (++buf == 2) { buf = 0; tphase ^= 1u; }
        }
      }
    }
  } else {
    // ---------------- epilogue: TMEM -> registers -> partial tile in global memory ----------------
    const int q = warp & 3;                 // TMEM lane quarter this warp may read
    const int row = q * 32 + lane;          // row of the tile
    int buf = 0;
    uint32_t tphase = 0;
    bool ok = true;
    for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
      const int s = u / p.ntiles;
      const int kb0 = (int)((long long)s * p.kblocks / p.splits), kb1 = (int)((long long)(s + 1) * p.kblocks / p.splits);
      float* out = p.partials + (size_t)u * TILE_ELEMS + (size_t)row * BN;
      for (int kc0 = kb0; kc0 < kb1 && ok; kc0 += KCHUNK) {
        if (!mbar_wait(tfull_bar(buf), tphase, abort_flag)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const bool first = kc0 == kb0;   // later chunks add to what this thread stored before (round-to-nearest adds)
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
          uint32_t r[32];
          tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + c * 32), r);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
          for (int v = 0; v < 8; ++v) {
            float4 x = make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]), __uint_as_float(r[4 * v + 2]),
                                   __uint_as_float(r[4 * v + 3]));
            float4* dst = reinterpret_cast<float4*>(out + c * 32 + v * 4);
            if (!first) {
              const float4 y = *dst;
              x.x += y.x; x.y += y.y; x.z += y.z; x.w += y.w;
            }
            *dst = x;
          }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar(buf));
        if (++buf == 2) { buf = 0; tphase ^= 1u; }
      }
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(p.status, (int)kFlagWaitTimeout);
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS)
                 : "memory");
  }
}

// Sum the K-split partials of every tile in ascending split order, add the previous H when
// accumulating, and write the lower-triangle entry together with its mirror image.
__global__ void __launch_bounds__(256) hessian_reduce_kernel(Params p, int accumulate, float* __restrict__ H) {
  const int t = blockIdx.x;
  const int tm = p.tiles[t].x, tn = p.tiles[t].y;
  const long long d = p.d_in;
  for (int idx = threadIdx.x; idx < TILE_ELEMS; idx += blockDim.x) {
    const long long r = (long long)tm * BM + idx / BN, c = (long long)tn * BN + idx % BN;
    if (r >= d || c > r) continue;
    float v = 0.f;
    for (int s = 0; s < p.splits; ++s) v += p.partials[((size_t)s * p.ntiles + t) * TILE_ELEMS + idx];
    if (accumulate) v += H[r * d + c];
    H[r * d + c] = v;
    if (c != r) H[c * d + r] = v;
  }
}

struct Plan {
  int tiles_m, ntiles, splits, kblocks;
};
static Plan make_plan(long long n, long long d_in) {
  Plan pl{};
  pl.tiles_m = (int)((d_in + BM - 1) / BM);
  int nt = 0;
  for (int tm = 0; tm < pl.tiles_m; ++tm) nt += tm / 2 + 1;
  pl.ntiles = nt;
  pl.kblocks = (int)((n + BK - 1) / BK);
  // K-splits: the units (tile x split) run in waves of one per SM; pick the split count whose waves cost
  // least -- ceil(units / SMs) waves of kblocks / splits K blocks each, plus a fixed cost per unit
  // (pipeline fill, the epilogue that nothing overlaps) of about 16 K blocks
  int splits = 1;
  long long best = -1;
  for (int s = 1; s <= 16 && s <= pl.kblocks; ++s) {
    const long long waves = ((long long)nt * s + 147) / 148;
    const long long cost = waves * ((pl.kblocks + s - 1) / s + 16);
    if (best < 0 || cost * 100 < best * 97) { best = cost; splits = s; }   // more partial tiles only for a real gain
  }
  pl.splits = splits;
  return pl;
}

}  // namespace tc

bool hessian_tc_supported(long long n, long long d_in, long long ldx, const void* X) {
  return n >= 256 && d_in >= 256 && d_in <= 65535 && (ldx % 8) == 0 && ((uintptr_t)X % 16) == 0 &&
         n < (1ll << 31) && ldx * 2 < (1ll << 40);
}

size_t hessian_tc_workspace(long long n, long long d_in) {
  if (d_in < 256 || n < 256) return 0;
  const tc::Plan pl = tc::make_plan(n, d_in);
  return align_up((size_t)pl.splits * pl.ntiles * tc::TILE_ELEMS * sizeof(float)) + align_up((size_t)pl.ntiles * sizeof(int2));
}

cudaError_t launch_hessian_tc(const void* X, long long n, long long d_in, long long ldx, int accumulate, float* H,
                              void* ws, cudaStream_t st) {
  using namespace tc;
  CUtensorMap tmap;
  const cuuint64_t gdim[2] = {(cuuint64_t)d_in, (cuuint64_t)n};
  const cuuint64_t gstride[1] = {(cuuint64_t)ldx * 2};
  const cuuint32_t box[2] = {(cuuint32_t)BOX_COLS, (cuuint32_t)BK};
  const cuuint32_t estr[2] = {1, 1};
  // the driver entry point is looked up through the runtime, so the library has no link-time
  // dependency on libcuda (it must load on machines without a driver)
  typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                               const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                               CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static EncodeFn encode = nullptr;
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t ge = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (ge != cudaSuccess) return ge;
    if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
    encode = (EncodeFn)fn;
  }
  const CUresult cr = encode(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(X), gdim,
                                             gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (cr != CUDA_SUCCESS) return cudaErrorInvalidValue;
  const Plan pl = make_plan(n, d_in);
  Params p{};
  p.n = n; p.d_in = d_in; p.tiles_m = pl.tiles_m; p.ntiles = pl.ntiles; p.splits = pl.splits; p.kblocks = pl.kblocks;
  p.partials = (float*)ws;
  int2* tiles = (int2*)((char*)ws + align_up((size_t)pl.splits * pl.ntiles * TILE_ELEMS * sizeof(float)));
  p.tiles = tiles;
  { hessian_tile_order_kernel<<<1, 32, 0, st>>>(pl.tiles_m, tiles); count_launch(); }
  p.status = device_status_word();
  if (!p.status) return cudaErrorInvalidSymbol;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaError_t e = cudaFuncSetAttribute(hessian_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
  if (e != cudaSuccess) return e;
  const int units = pl.ntiles * pl.splits;
  const int grid = units < sms ? units : sms;
  { hessian_tc_kernel<<<grid, NUM_THREADS, SMEM_BYTES, st>>>(tmap, p); count_launch(); }
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  { hessian_reduce_kernel<<<pl.ntiles, 256, 0, st>>>(p, accumulate, H); count_launch(); }
  return cudaGetLastError();
}

}  // namespace cdq
