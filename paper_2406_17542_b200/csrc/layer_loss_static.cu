// cdq_layer_loss_static: the layer loss with its scratch in a fixed device array that is part
// of the library image, for callers that must not allocate device memory.
//
// The scratch array is a file-scope __device__ object: every GPU that loads the library holds
// kStaticScratchBytes of it until the process exits.  In host code the array's name is only a
// host-side handle, so its device address is looked up once per device with
// cudaGetSymbolAddress (with that device current) and that address is what the kernels get.
#include <cstdio>
#include <mutex>

#include "common.cuh"

namespace cdq {

constexpr size_t kStaticScratchBytes = CDQ_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
unsigned char* g_scratch_addr[kMaxDevices] = {};

// Device address of the scratch array on the current device (set-up on first use).
cudaError_t static_scratch(unsigned char** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_addr[dev]) {
    unsigned char* ptr = nullptr;
    e = cudaGetSymbolAddress((void**)&ptr, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_addr[dev] = ptr;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}
}  // namespace
}  // namespace cdq

using namespace cdq;

extern "C" cdq_status cdq_layer_loss_static(const float* H, const void* W, cdq_dtype wt, long long d_in,
                                            long long d_out, long long ldw, const cdq_grid_desc* grid,
                                            const float* scale, const float* zero, const unsigned char* Q,
                                            double* loss, double* per_col, void* stream) {
  if (!H || !W || !scale || !zero || !Q || !grid || (wt != CDQ_F32 && wt != CDQ_BF16)) return CDQ_ERR_INVALID_ARG;
  if (!aligned16(H)) return CDQ_ERR_INVALID_ARG;
  if (grid->bits < 1 || grid->bits > 8 || grid->group_size < 0) return CDQ_ERR_INVALID_ARG;
  if (d_in < 1 || d_out < 1 || ldw < d_out) return CDQ_ERR_SHAPE;
  if (grid->group_size > 0 && d_in % grid->group_size) return CDQ_ERR_SHAPE;
  if (d_in > 65535) return CDQ_ERR_UNSUPPORTED;

  // carve the fixed array: residual E, per-tile loss partials, per-column losses, the total
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes); return o; };
  const size_t oE = take(sizeof(double) * (size_t)d_in * (size_t)d_out);
  const size_t oPart = take(sizeof(double) * gemm_partials_elems(d_in, d_out));
  const size_t oCol = take(sizeof(double) * (size_t)d_out);
  const size_t oSum = take(sizeof(double));
  if (off > kStaticScratchBytes) {
    char msg[200];
    snprintf(msg, sizeof(msg), "cdq_layer_loss_static: a %lld x %lld layer needs %zu bytes of scratch, the fixed "
             "array holds %zu", d_in, d_out, off, kStaticScratchBytes);
    set_error_detail(msg);
    return CDQ_ERR_WORKSPACE;
  }

  unsigned char* base = nullptr;
  cudaError_t e = static_scratch(&base);
  if (e != cudaSuccess) {
    set_error_detail("cdq_layer_loss_static: cudaGetSymbolAddress of the scratch array failed");
    return CDQ_ERR_CUDA;
  }
  cudaStream_t st = (cudaStream_t)stream;
  double* E = (double*)(base + oE);
  double* part = (double*)(base + oPart);
  double* col_loss = per_col ? per_col : (double*)(base + oCol);
  double* sum = (double*)(base + oSum);

  ResidualSrc src{};
  src.W = W; src.wt = wt; src.ldw = ldw; src.scale = scale; src.zero = zero; src.Q = Q;
  src.use_gamma = 0; src.L = (1 << grid->bits) - 1;
  src.g = grid->group_size > 0 ? grid->group_size : d_in;
  src.d_out = d_out;
  // every scratch region is fully overwritten before it is read, so nothing needs clearing
  if ((e = launch_residual_f64(src, d_in, E, st)) != cudaSuccess ||
      (e = launch_gemm_he(H, d_in, d_out, E, nullptr, 0, col_loss, part, st)) != cudaSuccess) {
    set_error_detail(cudaGetErrorString(e));
    return CDQ_ERR_CUDA;
  }
  if (loss) {
    if ((e = launch_sum_f64(col_loss, d_out, sum, st)) != cudaSuccess ||
        (e = cudaMemcpyAsync(loss, sum, sizeof(double), cudaMemcpyDeviceToHost, st)) != cudaSuccess ||
        (e = cudaStreamSynchronize(st)) != cudaSuccess) {
      set_error_detail(cudaGetErrorString(e));
      return CDQ_ERR_CUDA;
    }
  }
  return CDQ_OK;
}
