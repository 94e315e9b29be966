// The arithmetic of one descent sweep, shared by the two descent kernels (cd_kernel.cu keeps
// the row of H in registers, cd_kernel_tma.cu stages it through shared memory).
//
// For a chunk of 4 consecutive coordinates the sweep applies the pending step to the gradient
// (fp64) and scores the best move of every coordinate (fp32) -- the body of the loop of
// Algorithm 1 of the paper, with its scan over the levels replaced by the clamped rounding of the parabola's vertex
//   r = clamp(rint(q - g / (2 a H_ii)), 0, L).
#pragma once

#include "cd_params.cuh"

namespace cdq {

// A thread's running best move: the score and, packed into one float, the step in levels plus
// 1024 times the thread-local coordinate slot (both small integers, exact in fp32).
struct SweepBest {
  float best, bpk;
  __device__ __forceinline__ void init() { best = 0.f; bpk = 0.f; }
  __device__ __forceinline__ int slot() const { return ((int)bpk + 512) >> 10; }
  __device__ __forceinline__ int dr() const { const int ipk = (int)bpk; return ipk - (((ipk + 512) >> 10) << 10); }
};

// Applies g += c2 * h to the 4 coordinates of chunk slot k and folds their best moves into the
// thread's running best.  qpk: the 4 codes, packed; hd4: H_ii; hs4: 0.5 / H_ii; a, ia: scale of
// the chunk and its reciprocal (grouped modes; per-channel columns run in code units, a == 1);
// top = kMagic + L.
template <int SMODE>
__device__ __forceinline__ void sweep_chunk(double (&gk)[4], const float4 rv, const float4 hd4, const float4 hs4,
                                            unsigned qpk, double c2, float a, float ia, float top, int k,
                                            SweepBest& sb) {
  const float hv[4] = {rv.x, rv.y, rv.z, rv.w};
  const float hdv[4] = {hd4.x, hd4.y, hd4.z, hd4.w};
  const float hsv[4] = {hs4.x, hs4.y, hs4.z, hs4.w};
#pragma unroll
  for (int v = 0; v < 4; ++v) {
    gk[v] = fma(c2, (double)hv[v], gk[v]);
    const float gf = (float)gk[v];
    // kMagic + q: a float whose unit in the last place is 1, so the fused multiply-add below
    // rounds the vertex to a level
    const float qmf = __uint_as_float(__byte_perm(qpk, kMagicBits, 0x7650 | v));
    float t = fmaf(-gf, SMODE == kPerChannel ? hsv[v] : ia * hsv[v], qmf);
    t = fminf(fmaxf(t, kMagic), top);                    // clamped to the grid
    const float dr = t - qmf;
    const float d = SMODE == kPerChannel ? dr : a * dr;
    const float dl = fmaf(d, hdv[v], gf) * d;            // change of the loss
    if (dl < sb.best) { sb.best = dl; sb.bpk = dr + (float)((4 * k + v) * 1024); }
  }
}

// The thread's candidate for the team-wide argmin: key orders by decrease (the complement of a
// negative float's bits; a zero step scores -0, so the sign is tested), packed orders equal
// decreases by (chunk slot, thread, coordinate in chunk) -- the order of the coordinate index --
// and then by level.
__device__ __forceinline__ void sweep_candidate(const SweepBest& sb, int tid, unsigned& key, unsigned& packed) {
  key = kNoMove; packed = kNoMove;
  if (sb.best < 0.f) {
    const int e = sb.slot();
    key = ~__float_as_uint(sb.best);
    packed = ((unsigned)(e >> 2) << 21) | ((unsigned)tid << 11) | ((unsigned)(e & 3) << 9) | (unsigned)(sb.dr() + 256);
  }
}

}  // namespace cdq
