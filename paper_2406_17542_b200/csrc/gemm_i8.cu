// C = E^T H on the integer tensor cores, exact to a chosen number of bits: the contraction
// behind the gradient G = 2 H (W_hat - W) (paper: Algorithm 1, the gradient step), the column losses
// e_j^T H e_j (paper: Eq. 1 with H = X^T X) and the loss per clipping strength of the OWC
// search (the minimisation stated after Eq. 2).
//
// Why integers.  The descent compares scores whose gradient term must be right to ~1e-9 of
// a_j H_pp, while a row of H mixes entries that differ by many powers of two (feature scales),
// so the products need about 40 bits.  The fp64 pipe of B200 gives ~15 TFLOP/s to a SIMT GEMM;
// the int8 tensor cores give two orders of magnitude more, and integer accumulation is exact.
// So both operands are cut into 7-bit signed slices (error-free splitting):
//     H[p,k]   = 2^hexp[p] * sum_i hs_i[p,k] 128^-i,     i = 1..NH   (row p scaled by its max)
//     E[k,j]   = 2^eexp[j] * sum_i es_i[j,k] 128^-i,     i = 1..NE   (column j scaled by its max)
// with hs_i, es_i in [-127, 127].  Every slice pair is an int8 x int8 -> int32 GEMM without
// rounding; pairs with the same i + j = s share one accumulator (up to 5 pairs x K x 127^2 fits
// in 31 bits for K <= 26 000) and the result is sum_s 128^-s acc_s, summed in fp64 from the
// smallest term up.  Pairs beyond i + j = smax are dropped: that is the only approximation, and
// it is bounded by K * (#dropped) * 128^-(smax+1) relative to (row max) x (column max).
//
// Kernel: M = 128 columns j of the layer (rows of E^T), N = 256 coordinates p (rows of H),
// K-major operands in 128-byte swizzled tiles loaded by TMA, tcgen05.mma kind::i8 with the
// int32 accumulators in TMEM (two of them, so the epilogue of one group overlaps the MMAs of
// the next), the same warp roles as the Hessian kernel.  Every mbarrier wait is bounded.
#include <cuda.h>

#include "async_copy.cuh"
#include "common.cuh"

namespace cdq {
namespace i8 {

constexpr int BM = 128, BN = 256, BKB = 128;       // tile; BKB = bytes (= int8 elements) of K per stage
constexpr int STAGES = 4;
constexpr int A_BYTES = BM * BKB, B_BYTES = BN * BKB, STAGE_BYTES = A_BYTES + B_BYTES;  // 16 + 32 KB
constexpr int NUM_THREADS = 320;     // producer, MMA issuer, 8 epilogue warps (two per TMEM lane quarter)
constexpr int EPI_WARPS = 8;
constexpr int TMEM_COLS = 512;
constexpr uint32_t SPIN_LIMIT = 1u << 24;
constexpr size_t SMEM_BYTES = 1024 + (size_t)STAGES * STAGE_BYTES + 256;
constexpr int MAX_SLICES = 6;
constexpr int MAX_GROUPS = 12;

// ---------------------------------------------------------------------------------------------
// Slicing.  exps[r] = e with max_k |x[r,k]| 2^-e in [0.5, 1) (0 for an all-zero row).

// Row maxima of a row-major fp32 matrix [rows, cols] -> exponent per row.
__global__ void row_exp_f32_kernel(const float* __restrict__ x, long long rows, long long cols, int* __restrict__ exps) {
  const long long r = blockIdx.x;
  float m = 0.f;
  for (long long k = threadIdx.x; k < cols; k += blockDim.x) m = fmaxf(m, fabsf(x[r * cols + k]));
  __shared__ float red[32];
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x < 32) {
    m = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0.f;
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    if (threadIdx.x == 0) {
      int e = 0;
      if (m > 0.f && m < __int_as_float(0x7f800000)) frexpf(m, &e);
      exps[r] = e;
    }
  }
}

// Column maxima of a row-major fp64 matrix [rows, cols] -> exponent per column (two steps:
// partial maxima over row blocks as ordered bit patterns, then the exponent).
__global__ void col_max_f64_kernel(const double* __restrict__ x, long long rows, long long cols,
                                   unsigned long long* __restrict__ colmax_bits) {
  const long long c = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (c >= cols) return;
  const long long r0 = (long long)blockIdx.y * 256, r1 = min(rows, r0 + 256);
  double m = 0.0;
  for (long long r = r0; r < r1; ++r) m = fmax(m, fabs(x[r * cols + c]));
  if (isfinite(m)) atomicMax(&colmax_bits[c], (unsigned long long)__double_as_longlong(m));  // m >= 0: bits order like values
}
__global__ void col_exp_kernel(const unsigned long long* __restrict__ colmax_bits, long long cols, int* __restrict__ exps) {
  const long long c = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (c >= cols) return;
  const double m = __longlong_as_double((long long)colmax_bits[c]);
  int e = 0;
  if (m > 0.0) frexp(m, &e);
  exps[c] = e;
}

// The ns slices of one value already scaled into (-1, 1).
__device__ __forceinline__ void slice_value(double r, int ns, signed char (&out)[MAX_SLICES]) {
#pragma unroll
  for (int i = 0; i < MAX_SLICES; ++i) {
    if (i < ns) {
      r *= 128.0;
      const double s = trunc(r);
      r -= s;
      out[i] = (signed char)(int)s;
    }
  }
}

// H [d, d] fp32 -> slices [ns][d][kp] int8 (row p scaled by 2^-exps[p]; columns >= d zero).
__global__ void slice_h_kernel(const float* __restrict__ H, long long d, long long kp, const int* __restrict__ exps,
                               int ns, signed char* __restrict__ out) {
  const long long p = blockIdx.y;
  const long long k = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (k >= kp) return;
  signed char s[MAX_SLICES] = {0, 0, 0, 0, 0, 0};
  if (k < d) slice_value(ldexp((double)H[p * d + k], -exps[p]), ns, s);
  for (int i = 0; i < ns; ++i) out[((size_t)i * d + p) * kp + k] = s[i];
}

// E [d_in, d_out] fp64 -> slices of E^T [ns][d_out][kp] int8 (column j scaled by 2^-exps[j]),
// 32 x 32 tiles through shared memory so that both the reads and the writes are contiguous.
__global__ void slice_et_kernel(const double* __restrict__ E, long long d_in, long long d_out, long long kp,
                                const int* __restrict__ exps, int ns, signed char* __restrict__ out) {
  __shared__ double tile[32][33];
  const long long k0 = (long long)blockIdx.x * 32, j0 = (long long)blockIdx.y * 32;
  for (int rr = threadIdx.y; rr < 32; rr += blockDim.y) {
    const long long k = k0 + rr, j = j0 + threadIdx.x;
    tile[rr][threadIdx.x] = (k < d_in && j < d_out) ? E[k * d_out + j] : 0.0;
  }
  __syncthreads();
  for (int jj = threadIdx.y; jj < 32; jj += blockDim.y) {
    const long long j = j0 + jj, k = k0 + threadIdx.x;
    if (j < d_out && k < kp) {
      signed char s[MAX_SLICES] = {0, 0, 0, 0, 0, 0};
      slice_value(ldexp(tile[threadIdx.x][jj], -exps[j]), ns, s);
      for (int i = 0; i < ns; ++i) out[((size_t)i * d_out + j) * kp + k] = s[i];
    }
  }
}

// ---------------------------------------------------------------------------------------------
// The int8 GEMM.

struct Params {
  int M, N;                 // rows of E^T (layer columns j), rows of H (coordinates p)
  int kblocks;              // K blocks of BKB bytes
  int tiles_m, tiles_n;
  int ngroups;              // groups in the order they are processed: descending i + j
  int group_first[MAX_GROUPS + 1];    // pairs [first, next first) of each group
  int group_s[MAX_GROUPS];            // i + j of the group (slices numbered from 1)
  signed char pair_e[MAX_SLICES * MAX_SLICES], pair_h[MAX_SLICES * MAX_SLICES];  // slice indices (from 0)
  double* C;                // [M, ldc] fp64
  long long ldc;
  const int* eexp;          // [M]
  const int* hexp;          // [N]
  double final_scale;       // applied with the exponents after the last group
  const double* E;          // optional, [N, lde]: with dot_part, the epilogue also sums E[p, j] C[j, p] over its columns
  long long lde;
  double* dot_part;         // [2 * tiles_n, M] partial column dots, one row per (tile column, epilogue half)
  int* status;
};

// Bounded wait of this pipeline's roles (see async_copy.cuh).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  return mbar_wait_or_abort(bar, parity, abort_flag, SPIN_LIMIT);
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}
// Shared-memory matrix descriptor, K-major, 128-byte swizzle: rows of 128 bytes, groups of 8
// rows 1024 bytes apart (SBO); the leading-dimension offset is not used by swizzled K-major
// layouts.  Bits [0,14) start >> 4, [16,30) LBO >> 4, [32,46) SBO >> 4, [46,48) version 1,
// [61,64) layout 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: int32 accumulate, signed 8-bit A and B, both K-major, N = 256, M = 128.
constexpr uint32_t IDESC = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

__device__ __forceinline__ void mma_i8(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(IDESC), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}

// Tiles are handed out in bands of 8 tile rows, column by column inside a band, so that the
// tiles in flight at one time share their operand panels in L2.
__device__ __forceinline__ void tile_coords(int t, int tiles_m, int tiles_n, int& tm, int& tn) {
  const int band = t / (8 * tiles_n);
  const int rows = min(8, tiles_m - band * 8);
  const int tl = t - band * 8 * tiles_n;
  tn = tl / rows;
  tm = band * 8 + tl - tn * rows;
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_i8_kernel(const __grid_constant__ CUtensorMap map_e, const __grid_constant__ CUtensorMap map_h, const Params p) {
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
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), EPI_WARPS); }
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

  const int ntiles = p.tiles_m * p.tiles_n;

  if (warp == 0) {
    // ---------------- TMA producer: one stage per (pair, K block) ----------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int issued = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x) {
        int tm, tn;
        tile_coords(t, p.tiles_m, p.tiles_n, tm, tn);
        for (int g = 0; g < p.ngroups && ok; ++g) {
          for (int pr = p.group_first[g]; pr < p.group_first[g + 1] && ok; ++pr) {
            const int se = p.pair_e[pr], sh = p.pair_h[pr];
            for (int kb = 0; kb < p.kblocks; ++kb) {
              if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
              mbar_expect_tx(full_bar(stage), STAGE_BYTES);
              const uint32_t a_dst = tiles + (uint32_t)stage * STAGE_BYTES;
              tma_load_3d(a_dst, &map_e, kb * BKB, tm * BM, se, full_bar(stage));
              tma_load_3d(a_dst + A_BYTES, &map_h, kb * BKB, tn * BN, sh, full_bar(stage));
              ++issued;
              if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
          }
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
    // ---------------- MMA issuer: one accumulator per (tile, group) ----------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int buf = 0;
      uint32_t tphase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x) {
        for (int g = 0; g < p.ngroups && ok; ++g) {
          if (!mbar_wait(tempty_bar(buf), tphase ^ 1u, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t tmem_d = tmem_base + (uint32_t)buf * BN;
          const int nsteps = (p.group_first[g + 1] - p.group_first[g]) * p.kblocks;
          for (int it = 0; it < nsteps; ++it) {
            if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a_src = tiles + (uint32_t)stage * STAGE_BYTES;
            const uint32_t b_src = a_src + A_BYTES;
#pragma unroll
            for (int kk = 0; kk < BKB / 32; ++kk)   // 32 bytes of K per MMA, inside the 128-byte swizzled row
              mma_i8(tmem_d, make_desc(a_src + kk * 32), make_desc(b_src + kk * 32), (it > 0 || kk > 0) ? 1u : 0u);
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
    // ---------------- epilogue: TMEM -> fp64 running sum in C ----------------
    // Two warps per TMEM lane quarter; they take the 16-column chunks of the tile in turn.
    const int q = warp & 3;                 // TMEM lane quarter this warp may read
    const int half = (warp - 2) >> 2;       // which of the two warps of the quarter
    const int row = q * 32 + lane;          // row of the tile
    int buf = 0;
    uint32_t tphase = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < ntiles && ok; t += gridDim.x) {
      int tm, tn;
      tile_coords(t, p.tiles_m, p.tiles_n, tm, tn);
      const long long j = (long long)tm * BM + row;
      const long long p0 = (long long)tn * BN;
      const bool row_ok = j < p.M;
      double* crow = p.C + (row_ok ? j : 0) * p.ldc;
      const int ej = row_ok ? p.eexp[j] : 0;
      double dot = 0.0;
      for (int g = 0; g < p.ngroups && ok; ++g) {
        if (!mbar_wait(tfull_bar(buf), tphase, abort_flag)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const double w = ldexp(1.0, -7 * p.group_s[g]);
        const bool first = g == 0, last = g == p.ngroups - 1;
#pragma unroll 1
        for (int c = half; c < BN / 16; c += 2) {
          uint32_t r[16];
          tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + c * 16), r);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
          if (row_ok) {
            const long long pc0 = p0 + c * 16;
            if (pc0 + 16 <= p.N) {
              // whole chunk inside the matrix: 16-byte accesses (ldc is a multiple of 4, pc0 of 16)
              double2* cp = reinterpret_cast<double2*>(crow + pc0);
              double2 old[8];
              if (!first) {
#pragma unroll
                for (int v = 0; v < 8; ++v) old[v] = cp[v];
              }
#pragma unroll
              for (int v = 0; v < 8; ++v) {
                double x0 = w * (double)(int)r[2 * v], x1 = w * (double)(int)r[2 * v + 1];
                if (!first) { x0 += old[v].x; x1 += old[v].y; }
                if (last) {
                  x0 = ldexp(x0 * p.final_scale, ej + p.hexp[pc0 + 2 * v]);
                  x1 = ldexp(x1 * p.final_scale, ej + p.hexp[pc0 + 2 * v + 1]);
                  if (p.dot_part) {
                    dot = fma(p.E[(pc0 + 2 * v) * p.lde + j], x0, dot);
                    dot = fma(p.E[(pc0 + 2 * v + 1) * p.lde + j], x1, dot);
                  }
                }
                cp[v] = make_double2(x0, x1);
              }
            } else {
#pragma unroll
              for (int v = 0; v < 16; ++v) {
                const long long pc = pc0 + v;
                if (pc < p.N) {
                  double x = w * (double)(int)r[v];
                  if (!first) x += crow[pc];
                  if (last) {
                    x = ldexp(x * p.final_scale, ej + p.hexp[pc]);
                    if (p.dot_part) dot = fma(p.E[pc * p.lde + j], x, dot);
                  }
                  crow[pc] = x;
                }
              }
            }
          }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty_bar(buf));
        if (++buf == 2) { buf = 0; tphase ^= 1u; }
      }
      if (p.dot_part && row_ok && ok) p.dot_part[(size_t)(2 * tn + half) * p.M + j] = dot;
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

// col_loss[j] = inv_scale * sum_b part[b, j], b ascending: the partial column dots
// sum_p E[p, j] C[j, p] that the GEMM's epilogue leaves per (tile column, epilogue half).  The
// order of the sum is fixed, so the result does not depend on the schedule.
__global__ void __launch_bounds__(256) dot_reduce_kernel(const double* __restrict__ part, int nparts, long long m,
                                                         double inv_scale, double* __restrict__ col_loss) {
  const long long j = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= m) return;
  double v = 0.0;
  for (int b = 0; b < nparts; ++b) v += part[(size_t)b * m + j];
  col_loss[j] = v * inv_scale;
}

}  // namespace i8

// ---------------------------------------------------------------------------------------------
// Host side.

static long long tc_kpad(long long d_in) { return (d_in + 127) / 128 * 128; }

bool gemm_tc_supported(long long d_in, long long d_out) {
  // 5 slice pairs of one accumulator must stay below 2^31: 5 * K * 127^2
  return d_in >= 256 && d_out >= 128 && d_in <= 26000 && d_out < (1ll << 30);
}

size_t gemm_tc_h_bytes(long long d_in, int nh) {
  return align_up((size_t)nh * d_in * tc_kpad(d_in)) + align_up(sizeof(int) * (size_t)d_in);
}
size_t gemm_tc_e_bytes(long long d_in, long long d_out, int ne) {
  return align_up(sizeof(double) * 2 * (size_t)((d_in + i8::BN - 1) / i8::BN) * (size_t)d_out) +   // partial column dots
         align_up((size_t)ne * d_out * tc_kpad(d_in)) + align_up(sizeof(int) * (size_t)d_out) +
         align_up(sizeof(unsigned long long) * (size_t)d_out);
}

// Slices of H (done once per call of the library; the OWC search reuses them for every gamma).
cudaError_t gemm_tc_prepare_h(const float* H, long long d_in, int nh, void* hbuf, cudaStream_t st) {
  const long long kp = tc_kpad(d_in);
  signed char* slices = (signed char*)hbuf;
  int* hexp = (int*)((char*)hbuf + align_up((size_t)nh * d_in * kp));
  { i8::row_exp_f32_kernel<<<(unsigned)d_in, 256, 0, st>>>(H, d_in, d_in, hexp); count_launch(); }
  dim3 grid((unsigned)((kp + 255) / 256), (unsigned)d_in);
  { i8::slice_h_kernel<<<grid, 256, 0, st>>>(H, d_in, kp, hexp, nh, slices); count_launch(); }
  return cudaGetLastError();
}

static cudaError_t encode_map3(CUtensorMap* map, const void* base, long long kp, long long rows, int ns, int box_rows) {
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
  const cuuint64_t gdim[3] = {(cuuint64_t)kp, (cuuint64_t)rows, (cuuint64_t)ns};
  const cuuint64_t gstride[2] = {(cuuint64_t)kp, (cuuint64_t)kp * (cuuint64_t)rows};
  const cuuint32_t box[3] = {(cuuint32_t)i8::BKB, (cuuint32_t)box_rows, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult cr = encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(base), gdim, gstride, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return cr == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// C[j, p] = scale * sum_k E[k, j] H[p, k]  for j < d_out, p < d_in, to the precision of
// (ne, nh, smax); optionally col_loss[j] = sum_p E[p, j] C[j, p] / scale.
// hbuf: from gemm_tc_prepare_h with the same nh.  ebuf: gemm_tc_e_bytes of scratch.
cudaError_t gemm_tc_run(const void* hbuf, int nh, const double* E, long long d_in, long long d_out, int ne, int smax,
                        double scale, double* C, long long ldc, double* col_loss, void* ebuf, cudaStream_t st) {
  using namespace i8;
  if (nh < 1 || nh > MAX_SLICES || ne < 1 || ne > MAX_SLICES || smax < 2) return cudaErrorInvalidValue;
  const long long kp = tc_kpad(d_in);
  const signed char* hsl = (const signed char*)hbuf;
  const int* hexp = (const int*)((const char*)hbuf + align_up((size_t)nh * d_in * kp));
  signed char* esl = (signed char*)ebuf;
  int* eexp = (int*)((char*)ebuf + align_up((size_t)ne * d_out * kp));
  unsigned long long* colmax = (unsigned long long*)((char*)eexp + align_up(sizeof(int) * (size_t)d_out));
  double* dot_part = (double*)((char*)colmax + align_up(sizeof(unsigned long long) * (size_t)d_out));

  cudaError_t e = cudaMemsetAsync(colmax, 0, sizeof(unsigned long long) * (size_t)d_out, st);
  if (e != cudaSuccess) return e;
  {
    dim3 grid((unsigned)((d_out + 255) / 256), (unsigned)((d_in + 255) / 256));
    { col_max_f64_kernel<<<grid, 256, 0, st>>>(E, d_in, d_out, colmax); count_launch(); }
    { col_exp_kernel<<<(unsigned)((d_out + 255) / 256), 256, 0, st>>>(colmax, d_out, eexp); count_launch(); }
    dim3 g2((unsigned)((kp + 31) / 32), (unsigned)((d_out + 31) / 32)), b2(32, 8);
    { slice_et_kernel<<<g2, b2, 0, st>>>(E, d_in, d_out, kp, eexp, ne, esl); count_launch(); }
  }
  Params p{};
  p.M = (int)d_out; p.N = (int)d_in; p.kblocks = (int)(kp / BKB);
  p.tiles_m = (int)((d_out + BM - 1) / BM); p.tiles_n = (int)((d_in + BN - 1) / BN);
  int npairs = 0, ng = 0;
  for (int s = smax; s >= 2; --s) {
    const int first = npairs;
    for (int i = 1; i <= ne; ++i) {
      const int j = s - i;
      if (j >= 1 && j <= nh) { p.pair_e[npairs] = (signed char)(i - 1); p.pair_h[npairs] = (signed char)(j - 1); ++npairs; }
    }
    if (npairs > first) {
      if (ng >= MAX_GROUPS) return cudaErrorInvalidValue;
      if ((long long)(npairs - first) * kp * 16129ll >= (1ll << 31)) return cudaErrorInvalidValue;
      p.group_first[ng] = first; p.group_s[ng] = s; ++ng;
    }
  }
  if (ng == 0) return cudaErrorInvalidValue;
  p.group_first[ng] = npairs;
  p.ngroups = ng;
  p.C = C; p.ldc = ldc; p.eexp = eexp; p.hexp = hexp; p.final_scale = scale;
  p.E = E; p.lde = d_out; p.dot_part = col_loss ? dot_part : nullptr;
  p.status = device_status_word();
  if (!p.status) return cudaErrorInvalidSymbol;

  CUtensorMap map_e, map_h;
  e = encode_map3(&map_e, esl, kp, d_out, ne, BM);
  if (e != cudaSuccess) return e;
  e = encode_map3(&map_h, hsl, kp, d_in, nh, BN);
  if (e != cudaSuccess) return e;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  e = cudaFuncSetAttribute(gemm_i8_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
  if (e != cudaSuccess) return e;
  const int ntiles = p.tiles_m * p.tiles_n;
  { gemm_i8_kernel<<<ntiles < sms ? ntiles : sms, NUM_THREADS, SMEM_BYTES, st>>>(map_e, map_h, p); count_launch(); }
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (col_loss) {
    { dot_reduce_kernel<<<(unsigned)((d_out + 255) / 256), 256, 0, st>>>(dot_part, 2 * p.tiles_n, d_out, 1.0 / scale, col_loss); count_launch(); }
    e = cudaGetLastError();
  }
  return e;
}

}  // namespace cdq
