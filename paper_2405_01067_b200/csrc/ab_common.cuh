// Shared declarations of the library's translation units (internal; the public surface is include/ab.h).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "ab.h"

namespace ab {

typedef __nv_bfloat16 bf16;

#define AB_CUDA_OK(expr)                                   \
  do {                                                     \
    cudaError_t _e = (expr);                               \
    if (_e != cudaSuccess) return AB_ERR_CUDA;             \
  } while (0)

// Every kernel launch site is followed by AB_LAUNCH_OK(), which also counts the launch.
void count_launches(long long n);

#define AB_LAUNCH_OK()                                     \
  do {                                                     \
    ::ab::count_launches(1);                               \
    if (cudaPeekAtLastError() != cudaSuccess) {            \
      cudaGetLastError();                                  \
      return AB_ERR_CUDA;                                  \
    }                                                      \
  } while (0)

#define AB_TRY(expr)                                       \
  do {                                                     \
    int _s = (expr);                                       \
    if (_s != AB_OK) return _s;                            \
  } while (0)

// Multiprocessors of the current device (cached per device; 0 if the query fails).  Grid sizes that are
// meant to fill the GPU are derived from it.
int sm_count();

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }
static inline size_t dtype_size(int dt) { return dt == AB_BF16 ? 2 : 4; }
static inline bool dtype_ok(int dt) { return dt == AB_F32 || dt == AB_BF16; }
static inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Carves 256-byte aligned pieces out of the caller's workspace.
struct Arena {
  char* base;
  size_t used;
  size_t cap;
  Arena(void* p, size_t bytes) : base(static_cast<char*>(p)), used(0), cap(bytes) {}
  void* take(size_t bytes) {
    size_t off = align_up(used, 256);
    used = off + bytes;
    return base ? base + off : nullptr;
  }
  template <typename T> T* take_n(size_t n) { return static_cast<T*>(take(n * sizeof(T))); }
  bool fits() const { return used <= cap; }
};

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(bf16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void from_f32(float& d, float v) { d = v; }
__device__ __forceinline__ void from_f32(bf16& d, float v) { d = __float2bfloat16_rn(v); }

// ---- general strided GEMM on the plain fp32 pipes (ab_gemm_simt.cu) ----------------------------
// C[i,j] = sum_k A(i,k) * B(k,j), A(i,k) at A + i*sAm + k*sAk, B(k,j) at B + k*sBk + j*sBn,
// C row-major with row stride ldc.  fp32 accumulation, k ascending inside a thread: results
// do not depend on the launch.  a_dt/b_dt/c_dt are ab_dtype values.
int gemm_simt(const void* A, int a_dt, int64_t sAm, int64_t sAk,
              const void* B, int b_dt, int64_t sBk, int64_t sBn,
              void* C, int c_dt, int64_t ldc,
              int64_t M, int64_t N, int64_t K, cudaStream_t st);

// Batched form for the small products of the factored group sync: problem z of the batch is
// described by one GemmDesc in device memory.  fp32 operands; optional diagonal scalings
//   C[i,j] = rs(i) * cs(j) * sum_k A(i,k) * ks(k) * B(k,j)
// where each of rs/cs/ks is derived from a vector v sorted in descending order:
//   mode 0: 1,  mode 1: sqrt(v),  mode 2: 1/sqrt(v);  entries with v <= thr * v[0] count as 0.
// Rows >= *live_rows and columns >= *live_cols (device ints, optional) are written as zero.
struct GemmDesc {
  const float* A; const float* B; void* C;
  int64_t sAm, sAk, sBk, sBn, ldc;
  int M, N, K;
  int c_bf16;
  const float* row_vec; const float* col_vec; const float* k_vec;
  int row_mode, col_mode, k_mode;
  float thr;
  const int* live_rows; const int* live_cols;
  int upper_only;   // 1: tiles entirely below the diagonal are skipped (symmetric result, upper part used)
  // Operand prologue that averages group copies (0 / 1 copies: plain operand).  Copy c of A starts a_cstride
  // elements after copy c - 1; the loader adds the copies in ascending c in fp32 and scales by copy_inv, the
  // arithmetic of the group mean.  The CTAs of the first tile column / row also write the averaged operand out.
  int a_copies, b_copies;
  int64_t a_cstride, b_cstride;
  float copy_inv;
  float* a_mean_out;   // optional, M x K row-major
  float* b_mean_out;   // optional, K x N row-major
};
int gemm_simt_batched(const GemmDesc* d_descs, int count, int max_M, int max_N, cudaStream_t st);
// W = mean_k(A_k) mean_k(B_k) in one kernel (the mean as the product's operand prologue); Abar, Bbar optional outputs.
int recombine_mean_simt(const float* A_copies, int64_t strideA, const float* B_copies, int64_t strideB, int K,
                        float* W, float* Abar, float* Bbar, int m, int n, int r, cudaStream_t st);

// ---- general tensor-core GEMM (ab_gemm_tc.cu) --------------------------------------------------
// C[M x N] = sum over terms of A_t B_t^T on the tensor cores; see the head of ab_gemm_tc.cu.
struct TcOperand {
  const void* p[3];   // bf16 pieces: one (plain product) or three (hi, mid, lo of an fp32 matrix)
  int pieces;
  int64_t ld;         // row stride in elements, a multiple of 8
  bool mn;            // false: stored M x K (resp. N x K); true: stored K x M (resp. K x N)
};
struct TcProblem {
  TcOperand A, B;
  void* C;            // fp32 or bf16, row stride ldc; with ksplit > 1: ksplit partial results, each
  int64_t ldc;        //   round_up(M, 128) rows, one after the other (fp32 only)
  int M, N, K;
  bool c_f32;
  int ksplit;
  const int* live_rows;   // optional device ints: rows / columns at or beyond them are written as zero
  const int* live_cols;
};
bool gemm_tc_available();
bool gemm_tc_problem_ok(const TcProblem& q);
size_t gemm_tc_table_bytes(int count);
// table_dev: device memory of gemm_tc_table_bytes(count); status: device int that receives AB_ERR_TIMEOUT
// if a bounded wait ran out (never cleared here).
int gemm_tc_batched(const TcProblem* probs, int count, void* table_dev, int* status, cudaStream_t st);
struct SplitJob { const float* src; int64_t ld_src; int rows, cols; bf16 *hi, *mid, *lo; int64_t ld_dst; int64_t first_block; };
int64_t split_job_blocks(int rows, int cols);
int split3_batched(const SplitJob* d_jobs, int njobs, int64_t total_blocks, cudaStream_t st);
int sum_slices(const float* part, float* out, int64_t count, int64_t slice_stride, int slices, cudaStream_t st);

// ---- dense layer of the full-rank phases (ab_dense.cu) ------------------------------------------
size_t dense_forward_ws(int64_t N, int m, int n);
size_t dense_backward_ws(int64_t N, int m, int n);

// ---- fused tensor-core chain (ab_chain_tc.cu) --------------------------------------------------
bool chain_tc_supported(int64_t N, int m, int n, int r, int ldA, int ldB, int dt,
                        const void* x, const void* A, const void* B, const void* y);
size_t chain_tc_forward_ws(int64_t N, int m, int n, int r);
size_t chain_tc_backward_ws(int64_t N, int m, int n, int r);
int chain_tc_forward(const void* x, const void* A, const void* B, void* y, void* T_save,
                     int64_t N, int m, int n, int r, int ldA, int ldB,
                     void* ws, size_t ws_bytes, cudaStream_t st);
int chain_tc_backward(const void* x, const void* dY, const void* A, const void* B,
                      const void* T_saved, void* dX, float* dA, float* dB,
                      int64_t N, int m, int n, int r, int ldA, int ldB,
                      void* ws, size_t ws_bytes, cudaStream_t st);

// 3 x 3 convolution with the factorised weight on NHWC activations, im2col rows never formed (ab_chain_tc.cu)
bool conv_tc_supported(int B, int H, int W, int C, int m, int r, int ldA, int ldB, int dt,
                       const void* x, const void* A, const void* Bf);
size_t conv_tc_ws(int B, int H, int W, int C, int m, int r);
int conv_tc_forward(const void* x, const void* A, const void* Bf, void* y, void* T_save, int B, int H, int W, int C,
                    int m, int r, int ldA, int ldB, void* ws, size_t ws_bytes, cudaStream_t st);
int conv_tc_backward(const void* x, const void* dY, const void* A, const void* Bf, const void* T_saved, void* dX,
                     float* dA, float* dB, int B, int H, int W, int C, int m, int r, int ldA, int ldB,
                     void* ws, size_t ws_bytes, cudaStream_t st);

int bounded_wait_selftest(int* dev_status, unsigned limit_us, cudaStream_t st);
size_t chain_stall_selftest_ws();
int chain_stall_selftest(void* ws, size_t ws_bytes, unsigned limit_us, cudaStream_t st);

// ---- SVD pipeline (ab_svd.cu) ------------------------------------------------------------------
struct SvdItem {
  const void* W;     // dense m x n
  int w_dt;
  int m, n, r_max;
  void* A;           // m x r_max
  void* B;           // r_max x n
  int out_dt;
  float* sigma;
  int* r_out;
  int* dev_status;
};
size_t svd_batch_ws(const SvdItem* items, int L);
int svd_batch(const SvdItem* items, int L, float sigma_cutoff, void* ws, size_t ws_bytes, cudaStream_t st);

// ---- factored group sync (ab_sync_fast.cu) ------------------------------------------------------
// One-sided Jacobi on the rows of `count` s x s matrices (s <= 256) kept in shared memory, one CTA or
// one cluster of CTAs per matrix (ab_sync_fast.cu).  X: count matrices, s * s apart.  rows: the
// orthogonalised rows scaled to unit length, sorted by descending norm; norms: those norms.  status:
// one int per matrix, status_stride_bytes apart (AB_OK / AB_ERR_NOT_CONVERGED).  scratch: device memory
// of rows_jacobi_scratch_bytes(count).
bool rows_jacobi_fits(int count, int s);
size_t rows_jacobi_scratch_bytes(int count);
int rows_jacobi(const float* X, float* rows, float* norms, int* status, size_t status_stride_bytes, int count, int s,
                void* scratch, cudaStream_t st);
bool sync_factored_supported(const ab_sync_desc* d, int L);
size_t sync_factored_ws(const ab_sync_desc* d, int L);
int sync_factored(const ab_sync_desc* d, int L, int K, float sigma_cutoff, int dt, int* dev_status,
                  void* ws, size_t ws_bytes, cudaStream_t st);

// ---- group mean (ab_average.cu) ----------------------------------------------------------------
// AdamW step on fp32 master values (ab_optim.cu); p_lp: optional bf16 copy of the result.
int adamw_step(float* p, const float* g, float* m, float* v, bf16* p_lp, int64_t count, float lr, float beta1,
               float beta2, float eps, float weight_decay, int step, cudaStream_t st);

// One mean per job in a single launch; results are fp32.  d_jobs is device memory.
// One mean of a batched launch.  first_block: the job's first block in the flat grid (running sum of
// average_job_blocks over the jobs before it); the launch gets the sum over all jobs.
struct AvgJob { const void* base; int64_t stride; int64_t count; float* out; int64_t first_block; };
int64_t average_job_blocks(int64_t count, int in_dt);
int group_average_batched(const AvgJob* d_jobs, int njobs, int K, int in_dt, int64_t total_blocks, cudaStream_t st);
int group_average(const void* base, int64_t stride_elems, int K, int64_t count,
                  int in_dt, int out_dt, void* out, cudaStream_t st);

}  // namespace ab
