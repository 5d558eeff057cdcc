// C-ABI entry points: argument checks, workspace carving, dispatch.  See include/ab.h.
#include <vector>
#include <string.h>

#include "ab_common.cuh"

#include <atomic>

namespace ab {
static std::atomic<long long> g_launches{0};
void count_launches(long long n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

int sm_count() {
  static std::atomic<int> cache[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (dev >= 0 && dev < 64) {
    const int c = cache[dev].load(std::memory_order_relaxed);
    if (c > 0) return c;
  }
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  if (dev >= 0 && dev < 64) cache[dev].store(sms, std::memory_order_relaxed);
  return sms;
}

namespace {

template <typename TI, typename TO>
__global__ void cast_kernel(const TI* __restrict__ in, TO* __restrict__ out, int64_t count) {
  const int64_t step = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += step) from_f32(out[i], to_f32(in[i]));
}

int cast_f32_to(const float* in, void* out, int dt, int64_t count, cudaStream_t st) {
  if (count == 0) return AB_OK;
  const int64_t cap = (int64_t)(sm_count() > 0 ? sm_count() : 1) * 8;
  unsigned grid = (unsigned)((count + 255) / 256 < cap ? (count + 255) / 256 : cap);
  if (dt == AB_F32) cast_kernel<float, float><<<grid, 256, 0, st>>>(in, static_cast<float*>(out), count);
  else cast_kernel<float, bf16><<<grid, 256, 0, st>>>(in, static_cast<bf16*>(out), count);
  AB_LAUNCH_OK();
  return AB_OK;
}

bool have_device() {
  int n = 0;
  return cudaGetDeviceCount(&n) == cudaSuccess && n > 0;
}

int check_layer_args(const void* x, const void* A, const void* B, int64_t N, int m, int n, int r,
                     int ldA, int ldB, int dt) {
  if (!dtype_ok(dt)) return AB_ERR_INVALID_ARG;
  if (N < 0 || m <= 0 || n <= 0 || r <= 0) return AB_ERR_INVALID_ARG;
  if (r > m || r > n) return AB_ERR_INVALID_ARG;
  if (ldA < r || ldB < n) return AB_ERR_INVALID_ARG;
  if (!A || !B || (N > 0 && !x)) return AB_ERR_INVALID_ARG;
  return AB_OK;
}

// general path: every product is one strided GEMM on the fp32 pipes, T and dT live in the workspace
// (the first 256 bytes of every layer workspace hold the device status word)
size_t general_forward_ws(int64_t N, int r) { return 256 + align_up((size_t)N * r * sizeof(float), 256); }
size_t general_backward_ws(int64_t N, int r) { return 256 + 2 * align_up((size_t)N * r * sizeof(float), 256); }

// Workspace of the tensor-core route of ab_recombine: status word, problem table, two split jobs and the three
// bf16 pieces of each factor.
struct RecombWs { int* status; void* table; SplitJob* jobs; bf16 *Asp, *Bsp; size_t ea, eb; int r8, n8; size_t bytes; };
RecombWs recombine_ws(void* ws, int m, int n, int r) {
  Arena ar(ws, 0);
  RecombWs w;
  w.r8 = (r + 7) & ~7; w.n8 = (n + 7) & ~7;
  w.ea = (size_t)m * w.r8; w.eb = (size_t)r * w.n8;
  w.status = ar.take_n<int>(64);
  w.table = ar.take(gemm_tc_table_bytes(1));
  w.jobs = ar.take_n<SplitJob>(2);
  w.Asp = ar.take_n<bf16>(3 * w.ea);
  w.Bsp = ar.take_n<bf16>(3 * w.eb);
  w.bytes = align_up(ar.used, 256);
  return w;
}

int general_forward(const void* x, const void* A, const void* B, void* y, void* T_save,
                    int64_t N, int m, int n, int r, int ldA, int ldB, int dt, void* ws, size_t ws_bytes,
                    cudaStream_t st) {
  Arena ar(ws, ws_bytes);
  int* status = ar.take_n<int>(64);
  float* T = ar.take_n<float>((size_t)N * r);
  if (!ws || !ar.fits()) return AB_ERR_WORKSPACE;
  AB_CUDA_OK(cudaMemsetAsync(status, 0, sizeof(int), st));
  AB_TRY(gemm_simt(x, dt, n, 1, B, dt, 1, ldB, T, AB_F32, r, N, r, n, st));        // T = x B^T
  if (T_save) AB_TRY(cast_f32_to(T, T_save, dt, N * r, st));
  AB_TRY(gemm_simt(T, AB_F32, r, 1, A, dt, 1, ldA, y, dt, m, N, m, r, st));         // y = T A^T
  return AB_OK;
}

int general_backward(const void* x, const void* dY, const void* A, const void* B, const void* T_saved,
                     void* dX, float* dA, float* dB, int64_t N, int m, int n, int r, int ldA, int ldB, int dt,
                     void* ws, size_t ws_bytes, cudaStream_t st) {
  Arena ar(ws, ws_bytes);
  int* status = ar.take_n<int>(64);
  float* T = ar.take_n<float>((size_t)N * r);
  float* dT = ar.take_n<float>((size_t)N * r);
  if (!ws || !ar.fits()) return AB_ERR_WORKSPACE;
  AB_CUDA_OK(cudaMemsetAsync(status, 0, sizeof(int), st));
  AB_TRY(gemm_simt(dY, dt, m, 1, A, dt, ldA, 1, dT, AB_F32, r, N, r, m, st));      // dT = dY A
  if (dX) AB_TRY(gemm_simt(dT, AB_F32, r, 1, B, dt, ldB, 1, dX, dt, n, N, n, r, st));   // dX = dT B
  if (dA) {
    const void* Tsrc = T_saved;
    int t_dt = dt;
    if (!Tsrc) {
      AB_TRY(gemm_simt(x, dt, n, 1, B, dt, 1, ldB, T, AB_F32, r, N, r, n, st));
      Tsrc = T;
      t_dt = AB_F32;
    }
    AB_TRY(gemm_simt(dY, dt, 1, m, Tsrc, t_dt, r, 1, dA, AB_F32, r, m, r, N, st));  // dA = dY^T T
  }
  if (dB) AB_TRY(gemm_simt(dT, AB_F32, 1, r, x, dt, n, 1, dB, AB_F32, n, r, n, N, st));  // dB = dT^T x
  return AB_OK;
}

}  // namespace
}  // namespace ab

using namespace ab;

extern "C" {

const char* ab_status_string(int s) {
  switch (s) {
    case AB_OK: return "ok";
    case AB_ERR_INVALID_ARG: return "invalid argument";
    case AB_ERR_UNSUPPORTED: return "unsupported size";
    case AB_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case AB_ERR_NOT_CONVERGED: return "iteration did not converge";
    case AB_ERR_TIMEOUT: return "bounded device wait expired";
    case AB_ERR_CUDA: return "CUDA runtime error";
    case AB_ERR_ACCURACY: return "kept singular values below the accuracy domain";
    default: return "unknown status";
  }
}

const char* ab_version(void) { return "0.1"; }

long long ab_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

size_t ab_workspace_bytes(int op, int64_t N, int m, int n, int r, int K, int dt) {
  (void)K;
  if (m <= 0 || n <= 0 || N < 0) return 0;
  if (r <= 0 && op != AB_OP_DENSE_FORWARD && op != AB_OP_DENSE_BACKWARD) return 0;
  switch (op) {
    case AB_OP_LAYER_FORWARD: {
      size_t g = general_forward_ws(N, r), t = chain_tc_forward_ws(N, m, n, r);
      return (g > t ? g : t) + 256;
    }
    case AB_OP_LAYER_BACKWARD: {
      size_t g = general_backward_ws(N, r), t = chain_tc_backward_ws(N, m, n, r);
      return (g > t ? g : t) + 256;
    }
    case AB_OP_RECOMBINE: return recombine_ws(nullptr, m, n, r).bytes + 256;
    case AB_OP_DENSE_FORWARD: return dense_forward_ws(N, m, n) + 256;
    case AB_OP_DENSE_BACKWARD: return dense_backward_ws(N, m, n) + 256;
    case AB_OP_SVD_SPLIT: {
      SvdItem it;
      memset(&it, 0, sizeof(it));
      it.m = m; it.n = n; it.r_max = r; it.w_dt = dt; it.out_dt = dt;
      return svd_batch_ws(&it, 1) + 256;
    }
    default: return 0;
  }
}

int ab_selftest_bounded_wait(int* dev_status, unsigned limit_us, void* cuda_stream) {
  if (!dev_status || limit_us == 0 || limit_us > 1000000u) return AB_ERR_INVALID_ARG;
  if (!have_device()) return AB_ERR_CUDA;
  return bounded_wait_selftest(dev_status, limit_us, static_cast<cudaStream_t>(cuda_stream));
}

size_t ab_selftest_chain_stall_workspace_bytes(void) { return chain_stall_selftest_ws(); }

int ab_selftest_chain_stall(void* ws, size_t ws_bytes, unsigned limit_us, void* cuda_stream) {
  if (limit_us == 0 || limit_us > 1000000u) return AB_ERR_INVALID_ARG;
  if (!have_device()) return AB_ERR_CUDA;
  return chain_stall_selftest(ws, ws_bytes, limit_us, static_cast<cudaStream_t>(cuda_stream));
}

int ab_layer_forward(const void* x, const void* A, const void* B, void* y, void* T_save,
                     int64_t N, int m, int n, int r, int ldA, int ldB, int dt,
                     void* ws, size_t ws_bytes, void* cuda_stream) {
  AB_TRY(check_layer_args(x, A, B, N, m, n, r, ldA, ldB, dt));
  if (N > 0 && !y) return AB_ERR_INVALID_ARG;
  if (!have_device()) return AB_ERR_CUDA;
  if (N == 0) return AB_OK;
  if (ws && !aligned(ws, 256)) return AB_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (chain_tc_supported(N, m, n, r, ldA, ldB, dt, x, A, B, y))
    return chain_tc_forward(x, A, B, y, T_save, N, m, n, r, ldA, ldB, ws, ws_bytes, st);
  return general_forward(x, A, B, y, T_save, N, m, n, r, ldA, ldB, dt, ws, ws_bytes, st);
}

int ab_layer_backward(const void* x, const void* dY, const void* A, const void* B,
                      const void* T_saved, void* dX, float* dA, float* dB,
                      int64_t N, int m, int n, int r, int ldA, int ldB, int dt,
                      void* ws, size_t ws_bytes, void* cuda_stream) {
  AB_TRY(check_layer_args(x, A, B, N, m, n, r, ldA, ldB, dt));
  if (N > 0 && !dY) return AB_ERR_INVALID_ARG;
  if (!have_device()) return AB_ERR_CUDA;
  if (ws && !aligned(ws, 256)) return AB_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (N == 0) {   // empty batch: the sums over N are empty
    if (dA) AB_CUDA_OK(cudaMemsetAsync(dA, 0, (size_t)m * r * sizeof(float), st));
    if (dB) AB_CUDA_OK(cudaMemsetAsync(dB, 0, (size_t)r * n * sizeof(float), st));
    return AB_OK;
  }
  if (chain_tc_supported(N, m, n, r, ldA, ldB, dt, x, A, B, dY))
    return chain_tc_backward(x, dY, A, B, T_saved, dX, dA, dB, N, m, n, r, ldA, ldB, ws, ws_bytes, st);
  return general_backward(x, dY, A, B, T_saved, dX, dA, dB, N, m, n, r, ldA, ldB, dt, ws, ws_bytes, st);
}

size_t ab_conv3x3_workspace_bytes(int batch, int H, int W, int C, int m, int r) {
  if (batch <= 0 || H <= 0 || W <= 0 || C <= 0 || m <= 0 || r <= 0) return 0;
  return conv_tc_ws(batch, H, W, C, m, r) + 256;
}

static int check_conv_args(const void* x, const void* A, const void* B, int batch, int H, int W, int C, int m, int r,
                           int ldA, int ldB, int dt) {
  if (!dtype_ok(dt)) return AB_ERR_INVALID_ARG;
  if (batch < 0 || H <= 0 || W <= 0 || C <= 0 || m <= 0 || r <= 0) return AB_ERR_INVALID_ARG;
  if (r > m || r > 9 * C || ldA < r || ldB < 9 * C) return AB_ERR_INVALID_ARG;
  if (!A || !B || (batch > 0 && !x)) return AB_ERR_INVALID_ARG;
  return AB_OK;
}

int ab_conv3x3_forward(const void* x, const void* A, const void* B, void* y, void* T_save,
                       int batch, int H, int W, int C, int m, int r, int ldA, int ldB, int dt,
                       void* ws, size_t ws_bytes, void* cuda_stream) {
  AB_TRY(check_conv_args(x, A, B, batch, H, W, C, m, r, ldA, ldB, dt));
  if (batch > 0 && !y) return AB_ERR_INVALID_ARG;
  if (!have_device()) return AB_ERR_CUDA;
  if (batch == 0) return AB_OK;
  if (!ws || !aligned(ws, 256)) return AB_ERR_WORKSPACE;
  if (!conv_tc_supported(batch, H, W, C, m, r, ldA, ldB, dt, x, A, B)) return AB_ERR_UNSUPPORTED;
  return conv_tc_forward(x, A, B, y, T_save, batch, H, W, C, m, r, ldA, ldB, ws, ws_bytes, static_cast<cudaStream_t>(cuda_stream));
}

int ab_conv3x3_backward(const void* x, const void* dY, const void* A, const void* B, const void* T_saved,
                        void* dX, float* dA, float* dB, int batch, int H, int W, int C, int m, int r,
                        int ldA, int ldB, int dt, void* ws, size_t ws_bytes, void* cuda_stream) {
  AB_TRY(check_conv_args(x, A, B, batch, H, W, C, m, r, ldA, ldB, dt));
  if (batch > 0 && !dY) return AB_ERR_INVALID_ARG;
  if (!have_device()) return AB_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (batch == 0) {
    if (dA) AB_CUDA_OK(cudaMemsetAsync(dA, 0, (size_t)m * r * sizeof(float), st));
    if (dB) AB_CUDA_OK(cudaMemsetAsync(dB, 0, (size_t)r * 9 * C * sizeof(float), st));
    return AB_OK;
  }
  if (!ws || !aligned(ws, 256)) return AB_ERR_WORKSPACE;
  if (!conv_tc_supported(batch, H, W, C, m, r, ldA, ldB, dt, x, A, B) || !aligned(dY, 16)) return AB_ERR_UNSUPPORTED;
  return conv_tc_backward(x, dY, A, B, T_saved, dX, dA, dB, batch, H, W, C, m, r, ldA, ldB, ws, ws_bytes, st);
}

int ab_adamw_step(float* param, const float* grad, float* m, float* v, void* param_bf16, int64_t count,
                  float lr, float beta1, float beta2, float eps, float weight_decay, int step,
                  void* cuda_stream) {
  if (count < 0 || step < 1) return AB_ERR_INVALID_ARG;
  if (count == 0) return AB_OK;
  if (!param || !grad || !m || !v) return AB_ERR_INVALID_ARG;
  if (!(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(eps > 0.f)) return AB_ERR_INVALID_ARG;
  if (!have_device()) return AB_ERR_CUDA;
  return adamw_step(param, grad, m, v, static_cast<bf16*>(param_bf16), count, lr, beta1, beta2, eps, weight_decay,
                    step, static_cast<cudaStream_t>(cuda_stream));
}

float ab_lr_rebound_factor(int steps_since_change, int rebound_steps, float floor) {
  if (rebound_steps <= 0 || steps_since_change >= rebound_steps) return 1.f;
  if (steps_since_change < 0) steps_since_change = 0;
  return floor + (1.f - floor) * ((float)steps_since_change / (float)rebound_steps);
}

int ab_group_average(const void* base, int64_t stride_elems, int K, int64_t count,
                     int in_dt, int out_dt, void* out, void* cuda_stream) {
  if (!dtype_ok(in_dt) || !dtype_ok(out_dt)) return AB_ERR_INVALID_ARG;
  if (K < 1 || count < 0) return AB_ERR_INVALID_ARG;
  if (K > 64) return AB_ERR_UNSUPPORTED;
  if (count > 0 && (!base || !out)) return AB_ERR_INVALID_ARG;
  if (K > 1 && stride_elems < count) return AB_ERR_INVALID_ARG;   // copies would overlap
  if (!aligned(base, dtype_size(in_dt)) || !aligned(out, dtype_size(out_dt))) return AB_ERR_INVALID_ARG;
  if (!have_device()) return AB_ERR_CUDA;
  return group_average(base, stride_elems, K, count, in_dt, out_dt, out, static_cast<cudaStream_t>(cuda_stream));
}

int ab_recombine(const void* Abar, const void* Bbar, float* W, int m, int n, int r,
                 int ldA, int ldB, int dt, void* ws, size_t ws_bytes, void* cuda_stream) {
  if (!dtype_ok(dt) || m <= 0 || n <= 0 || r <= 0 || ldA < r || ldB < n) return AB_ERR_INVALID_ARG;
  if (!Abar || !Bbar || !W) return AB_ERR_INVALID_ARG;
  if (!have_device()) return AB_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // Tensor-core route: bf16 factors multiply exactly in fp32 (one term); fp32 factors are cut into three bf16
  // pieces and multiplied as six terms.  It needs the workspace and 16-byte rows; without them the product
  // runs on the fp32 pipes.
  RecombWs w = recombine_ws(ws, m, n, r);
  const bool tc = ws && aligned(ws, 256) && ws_bytes >= w.bytes && gemm_tc_available() && n % 4 == 0 && aligned(W, 16) &&
                  (dt == AB_F32 || (ldA % 8 == 0 && ldB % 8 == 0 && aligned(Abar, 16) && aligned(Bbar, 16)));
  if (!tc) return gemm_simt(Abar, dt, ldA, 1, Bbar, dt, ldB, 1, W, AB_F32, n, m, n, r, st);
  AB_CUDA_OK(cudaMemsetAsync(w.status, 0, sizeof(int), st));
  TcProblem q;
  q.C = W; q.ldc = n; q.M = m; q.N = n; q.K = r; q.c_f32 = true; q.ksplit = 1; q.live_rows = q.live_cols = nullptr;
  if (dt == AB_BF16) {
    q.A.p[0] = Abar; q.A.p[1] = q.A.p[2] = nullptr; q.A.pieces = 1; q.A.ld = ldA; q.A.mn = false;
    q.B.p[0] = Bbar; q.B.p[1] = q.B.p[2] = nullptr; q.B.pieces = 1; q.B.ld = ldB; q.B.mn = true;
  } else {
    SplitJob jobs[2];
    jobs[0] = SplitJob{static_cast<const float*>(Abar), ldA, m, r, w.Asp, w.Asp + w.ea, w.Asp + 2 * w.ea, w.r8, 0};
    jobs[1] = SplitJob{static_cast<const float*>(Bbar), ldB, r, n, w.Bsp, w.Bsp + w.eb, w.Bsp + 2 * w.eb, w.n8,
                       split_job_blocks(m, r)};
    AB_CUDA_OK(cudaMemcpyAsync(w.jobs, jobs, sizeof(jobs), cudaMemcpyHostToDevice, st));
    AB_TRY(split3_batched(w.jobs, 2, split_job_blocks(m, r) + split_job_blocks(r, n), st));
    for (int k = 0; k < 3; ++k) { q.A.p[k] = w.Asp + k * w.ea; q.B.p[k] = w.Bsp + k * w.eb; }
    q.A.pieces = q.B.pieces = 3; q.A.ld = w.r8; q.B.ld = w.n8; q.A.mn = false; q.B.mn = true;
  }
  return gemm_tc_batched(&q, 1, w.table, w.status, st);
}

int ab_recombine_mean(const void* A_copies, int64_t strideA, const void* B_copies, int64_t strideB, int K,
                      float* W, float* Abar, float* Bbar, int m, int n, int r, int dt, void* cuda_stream) {
  if (!dtype_ok(dt) || m <= 0 || n <= 0 || r <= 0 || K < 1) return AB_ERR_INVALID_ARG;
  if (!A_copies || !B_copies || !W) return AB_ERR_INVALID_ARG;
  if (K > 1 && (strideA < (int64_t)m * r || strideB < (int64_t)r * n)) return AB_ERR_INVALID_ARG;
  if (K > 64 || dt != AB_F32) return AB_ERR_UNSUPPORTED;
  if (!have_device()) return AB_ERR_CUDA;
  return recombine_mean_simt(static_cast<const float*>(A_copies), strideA, static_cast<const float*>(B_copies), strideB, K,
                             W, Abar, Bbar, m, n, r, static_cast<cudaStream_t>(cuda_stream));
}

int ab_svd_split(const void* W, int m, int n, int r_max, float sigma_cutoff,
                 void* A, void* B, float* sigma, int* r_out, int* dev_status,
                 int w_dt, int out_dt, void* ws, size_t ws_bytes, void* cuda_stream) {
  if (!dtype_ok(w_dt) || !dtype_ok(out_dt)) return AB_ERR_INVALID_ARG;
  if (m <= 0 || n <= 0 || r_max <= 0 || !(sigma_cutoff >= 0.f)) return AB_ERR_INVALID_ARG;
  if (!W || !A || !B || !sigma || !r_out) return AB_ERR_INVALID_ARG;
  if ((m < n ? m : n) > 3072) return AB_ERR_UNSUPPORTED;
  if (!ws || !aligned(ws, 256)) return AB_ERR_WORKSPACE;
  if (!have_device()) return AB_ERR_CUDA;
  SvdItem it;
  it.W = W; it.w_dt = w_dt; it.m = m; it.n = n; it.r_max = r_max; it.A = A; it.B = B; it.out_dt = out_dt;
  it.sigma = sigma; it.r_out = r_out; it.dev_status = dev_status;
  return svd_batch(&it, 1, sigma_cutoff, ws, ws_bytes, static_cast<cudaStream_t>(cuda_stream));
}

// Workspace of ab_group_sync: per matrix Abar, Bbar (fp32) and W (fp32), then the SVD batch.
static size_t sync_layout(const ab_sync_desc* d, int L, int dt, void* ws, std::vector<float*>* Ab,
                          std::vector<float*>* Bb, std::vector<float*>* Wd, std::vector<SvdItem>* items, void** svd_ws) {
  Arena ar(ws, 0);
  std::vector<SvdItem> loc(L);
  for (int i = 0; i < L; ++i) {
    float* a = ar.take_n<float>((size_t)d[i].m * d[i].r);
    float* b = ar.take_n<float>((size_t)d[i].r * d[i].n);
    float* w = ar.take_n<float>((size_t)d[i].m * d[i].n);
    if (Ab) { (*Ab)[i] = a; (*Bb)[i] = b; (*Wd)[i] = w; }
    SvdItem& it = loc[i];
    it.W = w; it.w_dt = AB_F32; it.m = d[i].m; it.n = d[i].n; it.r_max = d[i].r;
    it.A = d[i].A_out; it.B = d[i].B_out; it.out_dt = dt; it.sigma = d[i].sigma; it.r_out = d[i].r_out;
    it.dev_status = nullptr;
  }
  void* sw = ar.take(0);
  size_t svd_bytes = svd_batch_ws(loc.data(), L);
  if (svd_ws) *svd_ws = sw;
  if (items) *items = loc;
  return align_up(ar.used, 256) + svd_bytes;
}

size_t ab_sync_workspace_bytes(const ab_sync_desc* descs, int L, int K, int dt) {
  (void)K;
  if (!descs || L <= 0) return 0;
  size_t dense = sync_layout(descs, L, dt, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr);
  size_t fact = sync_factored_supported(descs, L) ? sync_factored_ws(descs, L) : 0;
  return (dense > fact ? dense : fact) + 256;
}

int ab_group_sync(const ab_sync_desc* descs, int L, int K, float sigma_cutoff, int dt,
                  int* dev_status, void* ws, size_t ws_bytes, void* cuda_stream, int path) {
  if (!descs || L <= 0 || K < 1 || !dtype_ok(dt) || !(sigma_cutoff >= 0.f)) return AB_ERR_INVALID_ARG;
  if (path != AB_SYNC_AUTO && path != AB_SYNC_DENSE && path != AB_SYNC_FACTORED) return AB_ERR_INVALID_ARG;
  if (K > 64) return AB_ERR_UNSUPPORTED;
  for (int i = 0; i < L; ++i) {
    const ab_sync_desc& d = descs[i];
    if (d.m <= 0 || d.n <= 0 || d.r <= 0 || d.r > d.m || d.r > d.n) return AB_ERR_INVALID_ARG;
    if (!d.A_copies || !d.B_copies || !d.A_out || !d.B_out || !d.sigma || !d.r_out) return AB_ERR_INVALID_ARG;
    if (K > 1 && (d.strideA < (int64_t)d.m * d.r || d.strideB < (int64_t)d.r * d.n)) return AB_ERR_INVALID_ARG;
    if ((d.m < d.n ? d.m : d.n) > 3072) return AB_ERR_UNSUPPORTED;
  }
  if (!ws || !aligned(ws, 256)) return AB_ERR_WORKSPACE;
  if (!have_device()) return AB_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const bool can_factor = sync_factored_supported(descs, L);
  if (path == AB_SYNC_FACTORED && !can_factor) return AB_ERR_UNSUPPORTED;
  if (path != AB_SYNC_DENSE && can_factor)
    return sync_factored(descs, L, K, sigma_cutoff, dt, dev_status, ws, ws_bytes, st);
  std::vector<float*> Ab(L), Bb(L), Wd(L);
  std::vector<SvdItem> items;
  void* svd_ws = nullptr;
  size_t need = sync_layout(descs, L, dt, ws, &Ab, &Bb, &Wd, &items, &svd_ws);
  if (need > ws_bytes) return AB_ERR_WORKSPACE;
  for (int i = 0; i < L; ++i) {
    const ab_sync_desc& d = descs[i];
    AB_TRY(group_average(d.A_copies, d.strideA, K, (int64_t)d.m * d.r, dt, AB_F32, Ab[i], st));
    AB_TRY(group_average(d.B_copies, d.strideB, K, (int64_t)d.r * d.n, dt, AB_F32, Bb[i], st));
    AB_TRY(gemm_simt(Ab[i], AB_F32, d.r, 1, Bb[i], AB_F32, d.n, 1, Wd[i], AB_F32, d.n, d.m, d.n, d.r, st));
    if (d.W_out)
      AB_CUDA_OK(cudaMemcpyAsync(d.W_out, Wd[i], (size_t)d.m * d.n * sizeof(float), cudaMemcpyDeviceToDevice, st));
    items[i].dev_status = dev_status ? dev_status + i : nullptr;
  }
  size_t used = static_cast<char*>(svd_ws) - static_cast<char*>(ws);
  return svd_batch(items.data(), L, sigma_cutoff, svd_ws, ws_bytes - used, st);
}

}  // extern "C"
