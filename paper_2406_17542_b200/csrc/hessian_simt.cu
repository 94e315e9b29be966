// H = X^T X on the CUDA cores (paper: Section 3 "Notation"; Algorithm 1).
//  - verify kernels: every entry is the ascending-k fp64 sum without fused
//    multiply-add, rounded once to fp32 (bit-reproducible on a CPU);
//  - SIMT kernel: tiled, fp64 accumulation, any shape and input type; used for
//    fp32 inputs and for shapes the tensor-core kernel does not take.
#include "common.cuh"

namespace cdq {

template <typename T> __device__ __forceinline__ double ld_as_double(const T* p, long long i);
template <> __device__ __forceinline__ double ld_as_double<float>(const float* p, long long i) { return (double)p[i]; }
template <> __device__ __forceinline__ double ld_as_double<__nv_bfloat16>(const __nv_bfloat16* p, long long i) {
  return (double)__bfloat162float(p[i]);
}

template <typename T>
__global__ void hessian_verify_kernel(const T* __restrict__ X, long long n, long long d_in, long long ldx,
                                      double* __restrict__ H64) {
  const long long r = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  const long long p = blockIdx.y;
  if (r >= d_in) return;
  double acc = 0.0;
  for (long long k = 0; k < n; ++k) {
    const double xp = ld_as_double(X, k * ldx + p);
    const double xr = ld_as_double(X, k * ldx + r);
    acc = __dadd_rn(acc, __dmul_rn(xp, xr));
  }
  H64[p * d_in + r] = acc;
}

// One thread: trace in ascending order, then the regulariser on the diagonal.
__global__ void lambda_verify_kernel(double* H64, long long d_in, double lambda_rel) {
  if (blockIdx.x || threadIdx.x) return;
  double tr = 0.0;
  for (long long p = 0; p < d_in; ++p) tr = __dadd_rn(tr, H64[p * d_in + p]);
  const double add = __dmul_rn(lambda_rel, __ddiv_rn(tr, (double)d_in));
  for (long long p = 0; p < d_in; ++p) H64[p * d_in + p] = __dadd_rn(H64[p * d_in + p], add);
}

__global__ void round_to_f32_kernel(const double* __restrict__ src, float* __restrict__ dst, long long count) {
  const long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (i < count) dst[i] = (float)src[i];
}

cudaError_t launch_hessian_verify(const void* X, cdq_dtype xt, long long n, long long d_in, long long ldx,
                                  double lambda_rel, float* H, double* H64, cudaStream_t st) {
  dim3 block(128), grid((unsigned)((d_in + 127) / 128), (unsigned)d_in);
  if (xt == CDQ_BF16)
    { hessian_verify_kernel<__nv_bfloat16><<<grid, block, 0, st>>>((const __nv_bfloat16*)X, n, d_in, ldx, H64); count_launch(); }
  else
    { hessian_verify_kernel<float><<<grid, block, 0, st>>>((const float*)X, n, d_in, ldx, H64); count_launch(); }
  if (lambda_rel > 0.0) { lambda_verify_kernel<<<1, 32, 0, st>>>(H64, d_in, lambda_rel); count_launch(); }
  const long long count = d_in * d_in;
  { round_to_f32_kernel<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(H64, H, count); count_launch(); }
  return cudaGetLastError();
}

// ---- tiled SIMT kernel -----------------------------------------------------
constexpr int HT = 64;   // output tile edge
constexpr int HK = 16;   // rows of X per stage

template <typename T>
__global__ void __launch_bounds__(256) hessian_simt_kernel(const T* __restrict__ X, long long n, long long d_in,
                                                           long long ldx, int accumulate, float* __restrict__ H) {
  // Only tiles on or below the diagonal are computed; the mirror image is written too.
  const int tp = blockIdx.y, tr = blockIdx.x;
  if (tr > tp) return;
  __shared__ float sa[HK][HT + 4];
  __shared__ float sb[HK][HT + 4];
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  const long long p0 = (long long)tp * HT, r0 = (long long)tr * HT;
  double acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.0;
  for (long long k0 = 0; k0 < n; k0 += HK) {
    for (int e = threadIdx.x; e < HK * HT; e += 256) {
      const int kk = e / HT, cc = e % HT;
      const long long k = k0 + kk;
      float va = 0.f, vb = 0.f;
      if (k < n) {
        if (p0 + cc < d_in) va = (float)ld_as_double(X, k * ldx + p0 + cc);
        if (r0 + cc < d_in) vb = (float)ld_as_double(X, k * ldx + r0 + cc);
      }
      sa[kk][cc] = va;
      sb[kk][cc] = vb;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < HK; ++kk) {
      double a[4], b[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) { a[u] = (double)sa[kk][ty * 4 + u]; b[u] = (double)sb[kk][tx * 4 + u]; }
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[u][v] = fma(a[u], b[v], acc[u][v]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int u = 0; u < 4; ++u)
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      const long long p = p0 + ty * 4 + u, r = r0 + tx * 4 + v;
      if (p < d_in && r < d_in) {
        if (tp == tr) {
          // diagonal tile: every entry is computed directly, no mirroring
          const float prev = accumulate ? H[p * d_in + r] : 0.f;
          H[p * d_in + r] = (float)((double)prev + acc[u][v]);
        } else {
          const float prev = accumulate ? H[p * d_in + r] : 0.f;
          const float val = (float)((double)prev + acc[u][v]);
          H[p * d_in + r] = val;
          H[r * d_in + p] = val;
        }
      }
    }
}

cudaError_t launch_hessian_simt(const void* X, cdq_dtype xt, long long n, long long d_in, long long ldx,
                                int accumulate, float* H, cudaStream_t st) {
  const unsigned t = (unsigned)((d_in + HT - 1) / HT);
  dim3 grid(t, t), block(256);
  if (xt == CDQ_BF16)
    { hessian_simt_kernel<__nv_bfloat16><<<grid, block, 0, st>>>((const __nv_bfloat16*)X, n, d_in, ldx, accumulate, H); count_launch(); }
  else
    { hessian_simt_kernel<float><<<grid, block, 0, st>>>((const float*)X, n, d_in, ldx, accumulate, H); count_launch(); }
  return cudaGetLastError();
}

// H_ii += lambda_rel * mean(diag H), trace reduced in fp64 by one block.
__global__ void lambda_kernel(float* H, long long d_in, double lambda_rel) {
  __shared__ double red[256];
  double s = 0.0;
  for (long long p = threadIdx.x; p < d_in; p += blockDim.x) s += (double)H[p * d_in + p];
  red[threadIdx.x] = s;
  __syncthreads();
  for (int w = 128; w > 0; w >>= 1) {
    if ((int)threadIdx.x < w) red[threadIdx.x] += red[threadIdx.x + w];
    __syncthreads();
  }
  const double add = lambda_rel * (red[0] / (double)d_in);
  for (long long p = threadIdx.x; p < d_in; p += blockDim.x) H[p * d_in + p] = (float)((double)H[p * d_in + p] + add);
}

cudaError_t launch_hessian_lambda(float* H, long long d_in, double lambda_rel, double*, cudaStream_t st) {
  { lambda_kernel<<<1, 256, 0, st>>>(H, d_in, lambda_rel); count_launch(); }
  return cudaGetLastError();
}

}  // namespace cdq
