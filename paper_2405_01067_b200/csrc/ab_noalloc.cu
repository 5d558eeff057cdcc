// ab_layer_forward_static: the forward of the factorised layer for callers that cannot hand
// the library a workspace because they cannot allocate device memory at the point of the
// call -- code running inside another framework's allocator-free region, a plug-in loaded
// into a process whose memory pool is owned and fully reserved by the host application, a
// real-time loop where cudaMalloc's implicit synchronisation is not acceptable.  The rank-r
// intermediate T = x B^T lives in a fixed array that is part of the library image instead.
#include <mutex>

#include "ab_common.cuh"

namespace ab {
namespace {

// 4 MiB of fp32: room for N*r <= 1,048,576 (e.g. 4096 rows at rank 256, 16384 rows at rank 64).
// Every GPU that loads the library carries this array until the process exits.
constexpr size_t kStaticScratchElems = (size_t)1 << 20;
static __device__ __align__(256) float g_static_scratch[kStaticScratchElems];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
float* g_scratch_ptr[kMaxDevices] = {nullptr};

// The array's name is only a host-side handle; the device address has to be asked for, once
// per device, with that device current.
int scratch_for_current_device(float** out) {
  int dev = -1;
  AB_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return AB_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p) { cudaGetLastError(); return AB_ERR_CUDA; }
    g_scratch_ptr[dev] = static_cast<float*>(p);
  }
  *out = g_scratch_ptr[dev];
  return AB_OK;
}

}  // namespace
}  // namespace ab

using namespace ab;

extern "C" {

size_t ab_static_scratch_elems(void) { return kStaticScratchElems; }

int ab_layer_forward_static(const void* x, const void* A, const void* B, void* y,
                            int64_t N, int m, int n, int r, int ldA, int ldB, int dt, void* cuda_stream) {
  if (!dtype_ok(dt)) return AB_ERR_INVALID_ARG;
  if (N < 0 || m <= 0 || n <= 0 || r <= 0 || r > m || r > n || ldA < r || ldB < n) return AB_ERR_INVALID_ARG;
  if (!A || !B || (N > 0 && (!x || !y))) return AB_ERR_INVALID_ARG;
  // N*r beyond the built-in scratch (by division: the product of two unchecked arguments could wrap)
  if ((uint64_t)N > kStaticScratchElems / (uint64_t)r) return AB_ERR_UNSUPPORTED;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev <= 0) return AB_ERR_CUDA;
  if (N == 0) return AB_OK;
  float* T = nullptr;
  AB_TRY(scratch_for_current_device(&T));
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // T is written in full (all N*r entries) before it is read: nothing needs clearing.
  AB_TRY(gemm_simt(x, dt, n, 1, B, dt, 1, ldB, T, AB_F32, r, N, r, n, st));   // T = x B^T
  AB_TRY(gemm_simt(T, AB_F32, r, 1, A, dt, 1, ldA, y, dt, m, N, m, r, st));   // y = T A^T
  return AB_OK;
}

}  // extern "C"
