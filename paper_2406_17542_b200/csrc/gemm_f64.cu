// C = H E in fp64, where E = W_hat - W is the residual of every column.
// Used for the gradient G = 2 H E (paper: Algorithm 1, the gradient step, in weight units), for the
// layer loss sum_j e_j^T H e_j (Eq. 1 written with H) and for the OWC loss of each
// clipping strength (the objective minimised after Eq. 2).
//
// H is fp32 [d_in, d_in]; E is fp64 [d_in, d_out] row-major.  The contraction runs on the
// fp64 pipe: the gradient feeds discrete decisions of the descent, so it is kept far more
// accurate than the fp32 candidate scores that consume it.
#include "common.cuh"

namespace cdq {

constexpr int GM = 128;  // tile of p (rows of H)
constexpr int GN = 64;   // tile of j (columns of the layer)
constexpr int GK = 16;

size_t gemm_partials_elems(long long d_in, long long d_out) {
  return (size_t)((d_in + GM - 1) / GM) * (size_t)d_out;
}

__global__ void __launch_bounds__(256) gemm_he_kernel(const float* __restrict__ H, long long d_in, long long d_out,
                                                      const double* __restrict__ E, double* __restrict__ G,
                                                      long long ldg, double* __restrict__ part) {
  __shared__ double sA[GK][GM];      // sA[k][p]
  __shared__ double sB[GK][GN];      // sB[k][j]
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const long long p0 = (long long)blockIdx.y * GM, j0 = (long long)blockIdx.x * GN;
  const bool vecA = (d_in % 4 == 0);
  const bool vecB = (d_out % 2 == 0);

  double acc[8][4];
#pragma unroll
  for (int u = 0; u < 8; ++u)
#pragma unroll
    for (int v = 0; v < 4; ++v) acc[u][v] = 0.0;

  const int a_p = tid >> 1, a_k = (tid & 1) * 8;       // A: row a_p, k offsets a_k..a_k+7
  const int b_k = tid >> 4, b_j = (tid & 15) * 4;      // B: row b_k, columns b_j..b_j+3

  for (long long k0 = 0; k0 < d_in; k0 += GK) {
    {  // A tile, transposed into sA[k][p]
      float a[8];
      const long long p = p0 + a_p;
      if (p < d_in && vecA && k0 + a_k + 8 <= d_in) {
        const float4 v0 = *reinterpret_cast<const float4*>(H + p * d_in + k0 + a_k);
        const float4 v1 = *reinterpret_cast<const float4*>(H + p * d_in + k0 + a_k + 4);
        a[0] = v0.x; a[1] = v0.y; a[2] = v0.z; a[3] = v0.w;
        a[4] = v1.x; a[5] = v1.y; a[6] = v1.z; a[7] = v1.w;
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const long long k = k0 + a_k + e;
          a[e] = (p < d_in && k < d_in) ? H[p * d_in + k] : 0.f;
        }
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) sA[a_k + e][a_p] = (double)a[e];
    }
    {  // B tile
      const long long k = k0 + b_k;
      double b[4];
      if (k < d_in && vecB && j0 + b_j + 4 <= d_out) {
        const double2 v0 = *reinterpret_cast<const double2*>(E + k * d_out + j0 + b_j);
        const double2 v1 = *reinterpret_cast<const double2*>(E + k * d_out + j0 + b_j + 2);
        b[0] = v0.x; b[1] = v0.y; b[2] = v1.x; b[3] = v1.y;
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const long long j = j0 + b_j + e;
          b[e] = (k < d_in && j < d_out) ? E[k * d_out + j] : 0.0;
        }
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) sB[b_k][b_j + e] = b[e];
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < GK; ++kk) {
      double a[8], b[4];
#pragma unroll
      for (int u = 0; u < 8; u += 2) {
        const double2 t = *reinterpret_cast<const double2*>(&sA[kk][ty * 8 + u]);
        a[u] = t.x; a[u + 1] = t.y;
      }
#pragma unroll
      for (int v = 0; v < 4; v += 2) {
        const double2 t = *reinterpret_cast<const double2*>(&sB[kk][tx * 4 + v]);
        b[v] = t.x; b[v + 1] = t.y;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[u][v] = fma(a[u], b[v], acc[u][v]);
    }
    __syncthreads();
  }

  if (G) {
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      const long long j = j0 + tx * 4 + v;
      if (j >= d_out) continue;
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const long long p = p0 + ty * 8 + u;
        if (p < d_in) G[j * ldg + p] = 2.0 * acc[u][v];
      }
    }
  }
  if (part) {
    // sum_p E[p][j] C[p][j] over this tile's rows: per-thread 8 rows, then 16 row groups
    double* red = &sA[0][0];  // reuse: 16 x 64 doubles
    double s[4];
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      const long long j = j0 + tx * 4 + v;
      double t = 0.0;
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const long long p = p0 + ty * 8 + u;
        if (p < d_in && j < d_out) t = fma(E[p * d_out + j], acc[u][v], t);
      }
      s[v] = t;
    }
#pragma unroll
    for (int v = 0; v < 4; ++v) red[ty * GN + tx * 4 + v] = s[v];
    __syncthreads();
    if (tid < GN) {
      double t = 0.0;
#pragma unroll
      for (int r = 0; r < 16; ++r) t += red[r * GN + tid];
      const long long j = j0 + tid;
      if (j < d_out) part[(long long)blockIdx.y * d_out + j] = t;
    }
  }
}

__global__ void partials_reduce_kernel(const double* __restrict__ part, long long tiles, long long d_out,
                                       double* __restrict__ col_loss) {
  const long long j = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (j >= d_out) return;
  double t = 0.0;
  for (long long r = 0; r < tiles; ++r) t += part[r * d_out + j];
  col_loss[j] = t;
}

cudaError_t launch_gemm_he(const float* H, long long d_in, long long d_out, const double* E, double* G,
                           long long ldg, double* col_loss, double* part, cudaStream_t st) {
  dim3 grid((unsigned)((d_out + GN - 1) / GN), (unsigned)((d_in + GM - 1) / GM));
  { gemm_he_kernel<<<grid, 256, 0, st>>>(H, d_in, d_out, E, G, ldg, col_loss ? part : nullptr); count_launch(); }
  if (col_loss)
    { partials_reduce_kernel<<<(unsigned)((d_out + 127) / 128), 128, 0, st>>>(part, (d_in + GM - 1) / GM, d_out, col_loss); count_launch(); }
  return cudaGetLastError();
}

// ---- fixed-order kernels ---------------------------------------------------
__global__ void gemm_he_verify_kernel(const float* __restrict__ H, long long d_in, long long d_out,
                                      const double* __restrict__ E, double* __restrict__ C) {
  const long long j = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  const long long p = blockIdx.y;
  if (j >= d_out) return;
  double acc = 0.0;
  for (long long k = 0; k < d_in; ++k) acc = __dadd_rn(acc, __dmul_rn((double)H[p * d_in + k], E[k * d_out + j]));
  C[p * d_out + j] = acc;
}

__global__ void verify_epilogue_kernel(const double* __restrict__ C, const double* __restrict__ E, long long d_in,
                                       long long d_out, double* __restrict__ G, long long ldg,
                                       double* __restrict__ col_loss) {
  const long long j = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (j >= d_out) return;
  double loss = 0.0;
  for (long long p = 0; p < d_in; ++p) {
    const double c = C[p * d_out + j];
    if (G) G[j * ldg + p] = __dmul_rn(2.0, c);
    loss = __dadd_rn(loss, __dmul_rn(E[p * d_out + j], c));
  }
  if (col_loss) col_loss[j] = loss;
}

cudaError_t launch_gemm_he_verify(const float* H, long long d_in, long long d_out, const double* E, double* C,
                                  double* G, long long ldg, double* col_loss, cudaStream_t st) {
  dim3 grid((unsigned)((d_out + 127) / 128), (unsigned)d_in);
  { gemm_he_verify_kernel<<<grid, 128, 0, st>>>(H, d_in, d_out, E, C); count_launch(); }
  { verify_epilogue_kernel<<<(unsigned)((d_out + 127) / 128), 128, 0, st>>>(C, E, d_in, d_out, G, ldg, col_loss); count_launch(); }
  return cudaGetLastError();
}

// Ascending-order sum of a vector by one thread (d_out values: cheap, and reproducible).
__global__ void sum_f64_kernel(const double* __restrict__ v, long long n, double* __restrict__ out) {
  if (blockIdx.x || threadIdx.x) return;
  double s = 0.0;
  for (long long i = 0; i < n; ++i) s = __dadd_rn(s, v[i]);
  *out = s;
}

cudaError_t launch_sum_f64(const double* v, long long n, double* out, cudaStream_t st) {
  { sum_f64_kernel<<<1, 32, 0, st>>>(v, n, out); count_launch(); }
  return cudaGetLastError();
}

// The same sum by one block in a fixed tree order (reproducible from run to run, not the
// ascending order): for the production mode, where d_out can be tens of thousands.
__global__ void __launch_bounds__(1024) sum_f64_tree_kernel(const double* __restrict__ v, long long n,
                                                            double* __restrict__ out) {
  __shared__ double red[1024];
  double s = 0.0;
  for (long long i = threadIdx.x; i < n; i += 1024) s += v[i];
  red[threadIdx.x] = s;
  __syncthreads();
  for (int w = 512; w > 0; w >>= 1) {
    if ((int)threadIdx.x < w) red[threadIdx.x] += red[threadIdx.x + w];
    __syncthreads();
  }
  if (threadIdx.x == 0) *out = red[0];
}

cudaError_t launch_sum_f64_tree(const double* v, long long n, double* out, cudaStream_t st) {
  { sum_f64_tree_kernel<<<1, 1024, 0, st>>>(v, n, out); count_launch(); }
  return cudaGetLastError();
}

}  // namespace cdq
