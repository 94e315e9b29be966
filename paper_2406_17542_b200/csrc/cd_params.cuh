// Arguments shared by the descent kernels (cd_kernel.cu, cd_kernel_tma.cu).
#pragma once

#include "common.cuh"

namespace cdq {

struct CdParams {
  const float* H;
  const __nv_bfloat16* H16;   // bf16 copy of H for the rows of the update (NULL: fp32 rows)
  long long d_in, d_out;
  double* G;            // [d_out, ldg]
  long long ldg;
  unsigned char* Qt;    // [d_out, ldq] (transposed codes, ldq a multiple of 4)
  long long ldq;
  const float* scale;   // [ng, d_out]
  const float* hdiag;   // [d_in_pad] H_ii (0 beyond d_in)
  const float* hs;      // [d_in_pad] 0.5 / H_ii (0 where H_ii <= 0 and beyond d_in)
  long long g, ng;
  int ag_count;         // entries of the shared-memory scale table (>= ng)
  unsigned gmagic;      // ceil(2^32 / g): i / g == umulhi(i, gmagic) for i, g < 2^16 (unused when g == 1)
  int L;
  long long T;
  CdCounters* ctr;
  int* status;          // device status word
};

constexpr float kMagic = 12582912.0f;       // 1.5 * 2^23: adding it rounds to an integer
constexpr unsigned kMagicBits = 0x4B400000u;
constexpr unsigned kNoMove = 0xFFFFFFFFu;

// How the scale of a coordinate is found.
//   kPerChannel : one scale per column.  The descent runs in code units (g / a, the form of
//                 Algorithm 1): the step 2 (r - q) is an exact small integer and the scale
//                 drops out of every score, which saves two multiplies per coordinate.
//   kGroupFast  : group size a multiple of 4 whose quarter divides the team size, so a thread's
//                 chunks sit at a fixed stride in the table of group scales (shared memory).
//   kGroupAny   : any other group size; the group of every coordinate is looked up.
enum ScaleMode : int { kPerChannel = 0, kGroupFast = 1, kGroupAny = 2 };

// Scale mode of a layer for a team of nt threads (-1: no fast kernel handles it).
inline int cd_scale_mode(const CdParams& p, int nt) {
  if (p.ng <= 1) return kPerChannel;
  if (p.g & 3) return -1;
  return nt % (int)(p.g >> 2) == 0 ? kGroupFast : kGroupAny;
}

// cd_kernel_tma.cu: rows staged through shared memory by bulk copies.  Returns
// cudaErrorNotSupported when the shape has no such configuration (the caller then uses the
// plain kernel).
cudaError_t launch_cd_tma(const CdParams& p, cudaStream_t st);

}  // namespace cdq
