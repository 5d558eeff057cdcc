// Dense layer of the full-rank phases of the training cycle (Algorithm 1: the warm-up before the first
// decomposition and the rebound steps after "W <- AB"): y = x W^T, dX = dY W, dW = dY^T x.
// bf16 storage with sizes the tensor-core GEMM takes goes to ab_gemm_tc.cu (one bf16 term, fp32 accumulation;
// dW is a reduction over the rows, cut into slices whose partial sums are added in ascending order);
// everything else goes to the general fp32-pipe GEMM.
#include "ab_common.cuh"

namespace ab {
namespace {

bool have_device() {
  int n = 0;
  return cudaGetDeviceCount(&n) == cudaSuccess && n > 0;
}

bool tc_shape_ok(int64_t N, int m, int n, int dt, const void* a, const void* b, const void* c) {
  return dt == AB_BF16 && m % 8 == 0 && n % 8 == 0 && N < ((int64_t)1 << 30) && aligned(a, 16) && aligned(b, 16) &&
         aligned(c, 16) && gemm_tc_available();
}

struct DenseWs { int* status; void* table; float* partial; int ksplit; size_t bytes; };

// slices of the rows for dW: enough CTAs to fill the device, at least 2048 rows a slice
int dw_ksplit(int64_t N, int m, int n) {
  const int tiles = ((m + 127) / 128) * ((n + 255) / 256);
  int sms = sm_count();
  if (sms <= 0) sms = 148;
  int ks = (2 * sms + tiles - 1) / tiles;
  const int64_t cap = (N + 2047) / 2048;
  if (ks > cap) ks = (int)cap;
  if (ks > 32) ks = 32;
  return ks < 1 ? 1 : ks;
}

DenseWs dense_ws(void* ws, int64_t N, int m, int n, bool backward) {
  Arena ar(ws, 0);
  DenseWs w;
  w.status = ar.take_n<int>(64);
  w.table = ar.take(gemm_tc_table_bytes(2));
  w.ksplit = backward ? dw_ksplit(N, m, n) : 1;
  w.partial = backward && w.ksplit > 1 ? ar.take_n<float>((size_t)w.ksplit * ((m + 127) / 128 * 128) * n) : nullptr;
  w.bytes = align_up(ar.used, 256);
  return w;
}

TcOperand op1(const void* p, int64_t ld, bool mn) {
  TcOperand o;
  o.p[0] = p; o.p[1] = o.p[2] = nullptr; o.pieces = 1; o.ld = ld; o.mn = mn;
  return o;
}

}  // namespace

size_t dense_forward_ws(int64_t N, int m, int n) { return dense_ws(nullptr, N, m, n, false).bytes; }
size_t dense_backward_ws(int64_t N, int m, int n) { return dense_ws(nullptr, N, m, n, true).bytes; }

}  // namespace ab

using namespace ab;

extern "C" {

int ab_dense_forward(const void* x, const void* W, void* y, int64_t N, int m, int n, int dt,
                     void* ws, size_t ws_bytes, void* cuda_stream) {
  if (!dtype_ok(dt) || N < 0 || m <= 0 || n <= 0) return AB_ERR_INVALID_ARG;
  if (!W || (N > 0 && (!x || !y))) return AB_ERR_INVALID_ARG;
  if (!have_device()) return AB_ERR_CUDA;
  if (N == 0) return AB_OK;
  if (!ws || !aligned(ws, 256)) return AB_ERR_WORKSPACE;
  DenseWs w = dense_ws(ws, N, m, n, false);
  if (w.bytes > ws_bytes) return AB_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  AB_CUDA_OK(cudaMemsetAsync(w.status, 0, sizeof(int), st));
  if (tc_shape_ok(N, m, n, dt, x, W, y)) {
    TcProblem q;
    q.A = op1(x, n, false);      // x: N x n, the reduction index n is the fast one
    q.B = op1(W, n, false);      // W: m x n
    q.C = y; q.ldc = m; q.M = (int)N; q.N = m; q.K = n; q.c_f32 = false; q.ksplit = 1;
    q.live_rows = q.live_cols = nullptr;
    return gemm_tc_batched(&q, 1, w.table, w.status, st);
  }
  return gemm_simt(x, dt, n, 1, W, dt, 1, n, y, dt, m, N, m, n, st);
}

int ab_dense_backward(const void* x, const void* dY, const void* W, void* dX, float* dW,
                      int64_t N, int m, int n, int dt, void* ws, size_t ws_bytes, void* cuda_stream) {
  if (!dtype_ok(dt) || N < 0 || m <= 0 || n <= 0) return AB_ERR_INVALID_ARG;
  if (!W || (N > 0 && (!x || !dY))) return AB_ERR_INVALID_ARG;
  if (!have_device()) return AB_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (N == 0) {
    if (dW) AB_CUDA_OK(cudaMemsetAsync(dW, 0, (size_t)m * n * sizeof(float), st));
    return AB_OK;
  }
  if (!ws || !aligned(ws, 256)) return AB_ERR_WORKSPACE;
  DenseWs w = dense_ws(ws, N, m, n, true);
  if (w.bytes > ws_bytes) return AB_ERR_WORKSPACE;
  AB_CUDA_OK(cudaMemsetAsync(w.status, 0, sizeof(int), st));
  const bool tc = tc_shape_ok(N, m, n, dt, x, dY, W) && (!dX || aligned(dX, 16)) && (!dW || aligned(dW, 16)) && n % 4 == 0;
  if (!tc) {
    if (dX) AB_TRY(gemm_simt(dY, dt, m, 1, W, dt, n, 1, dX, dt, n, N, n, m, st));          // dX = dY W
    if (dW) AB_TRY(gemm_simt(dY, dt, 1, m, x, dt, n, 1, dW, AB_F32, n, m, n, N, st));      // dW = dY^T x
    return AB_OK;
  }
  TcProblem q[2];
  int nq = 0;
  if (dX) {     // dX = dY W: W is stored m x n, i.e. (reduction index) x (output column)
    q[nq].A = op1(dY, m, false);
    q[nq].B = op1(W, n, true);
    q[nq].C = dX; q[nq].ldc = n; q[nq].M = (int)N; q[nq].N = n; q[nq].K = m; q[nq].c_f32 = false; q[nq].ksplit = 1;
    q[nq].live_rows = q[nq].live_cols = nullptr;
    ++nq;
  }
  if (dW) {     // dW = dY^T x: both operands stored (reduction index) x (output index)
    q[nq].A = op1(dY, m, true);
    q[nq].B = op1(x, n, true);
    q[nq].C = w.ksplit > 1 ? static_cast<void*>(w.partial) : static_cast<void*>(dW);
    q[nq].ldc = n; q[nq].M = m; q[nq].N = n; q[nq].K = (int)N; q[nq].c_f32 = true; q[nq].ksplit = w.ksplit;
    q[nq].live_rows = q[nq].live_cols = nullptr;
    ++nq;
  }
  if (nq == 0) return AB_OK;
  AB_TRY(gemm_tc_batched(q, nq, w.table, w.status, st));
  if (dW && w.ksplit > 1)
    AB_TRY(sum_slices(w.partial, dW, (int64_t)m * n, (int64_t)((m + 127) / 128 * 128) * n, w.ksplit, st));
  return AB_OK;
}

}  // extern "C"
