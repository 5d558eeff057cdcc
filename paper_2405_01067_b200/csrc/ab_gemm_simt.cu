// Strided GEMMs on the fp32 pipes: the path for fp32 storage (where a reduced-precision
// tensor-core pass would miss the 1e-4 bound) and for shapes the fused tensor-core chain does
// not take.  Two kernels:
//  - gemm_simt_kernel: any mix of fp32 / bf16 operands (all-fp32 problems go to the second kernel).  64x64 output tile per CTA, 16-deep k
//    slabs staged in shared memory, 4x4 accumulators per thread.  Each 16-term partial dot
//    product is formed in fp32 and added to a running fp64 sum, so long reductions keep ~1e-7
//    relative accuracy; the order of additions is fixed by the shape alone.
//  - gemm_simt_batched_kernel: many fp32 GEMMs per launch with diagonal scalings and live-rank
//    masks (the group synchronisation's products), register-tiled 8x8 and double-buffered.
#include "ab_common.cuh"

namespace ab {
namespace {

constexpr int BM = 64, BN = 64, BK = 16, PAD = 4;

template <typename T>
__device__ __forceinline__ float load_elem(const T* p, int64_t off) { return to_f32(p[off]); }

template <typename TA, typename TB, typename TC>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const TA* __restrict__ A, int64_t sAm, int64_t sAk,
                 const TB* __restrict__ B, int64_t sBk, int64_t sBn,
                 TC* __restrict__ C, int64_t ldc, int64_t M, int64_t N, int64_t K) {
  __shared__ float As[BK][BM + PAD];
  __shared__ float Bs[BK][BN + PAD];
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const int64_t m0 = (int64_t)blockIdx.y * BM, n0 = (int64_t)blockIdx.x * BN;
  const bool a_kfast = (sAk == 1);   // consecutive threads walk the contiguous direction
  const bool b_nfast = (sBn == 1);

  double acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0;

  for (int64_t k0 = 0; k0 < K; k0 += BK) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      int idx = tid + e * 256;
      int kk, mm;
      if (a_kfast) { kk = idx % BK; mm = idx / BK; } else { mm = idx % BM; kk = idx / BM; }
      int64_t gm = m0 + mm, gk = k0 + kk;
      As[kk][mm] = (gm < M && gk < K) ? load_elem(A, gm * sAm + gk * sAk) : 0.f;
      int nn;
      if (b_nfast) { nn = idx % BN; kk = idx / BN; } else { kk = idx % BK; nn = idx / BK; }
      int64_t gn = n0 + nn;
      gk = k0 + kk;
      Bs[kk][nn] = (gn < N && gk < K) ? load_elem(B, gk * sBk + gn * sBn) : 0.f;
    }
    __syncthreads();
    float part[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) part[i][j] = 0.f;
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float4 a = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
      float4 b = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
      float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) part[i][j] = fmaf(av[i], bv[j], part[i][j]);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] += (double)part[i][j];
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int64_t gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int64_t gn = n0 + tx * 4 + j;
      if (gn < N) from_f32(C[gm * ldc + gn], (float)acc[i][j]);
    }
  }
}

template <typename TA, typename TB, typename TC>
int launch(const void* A, int64_t sAm, int64_t sAk, const void* B, int64_t sBk, int64_t sBn,
           void* C, int64_t ldc, int64_t M, int64_t N, int64_t K, cudaStream_t st) {
  dim3 grid((unsigned)((N + BN - 1) / BN), (unsigned)((M + BM - 1) / BM));
  if (grid.y > 65535u) return AB_ERR_UNSUPPORTED;
  gemm_simt_kernel<TA, TB, TC><<<grid, 256, 0, st>>>(
      static_cast<const TA*>(A), sAm, sAk, static_cast<const TB*>(B), sBk, sBn,
      static_cast<TC*>(C), ldc, M, N, K);
  AB_LAUNCH_OK();
  return AB_OK;
}

__device__ __forceinline__ float diag_scale(const float* v, int idx, int mode, float thr) {
  if (mode == 0 || v == nullptr) return 1.f;
  const float x = v[idx];
  if (!(x > thr * v[0]) || !(x > 0.f)) return 0.f;
  return mode == 1 ? sqrtf(x) : 1.f / sqrtf(x);
}

// ---- batched fp32 GEMM with diagonal scalings ---------------------------------------------------
// One descriptor per blockIdx.z.  BM_ x BN_ output tile, 8 x 8 accumulators per thread (two 4-wide
// groups half a tile apart, so the float4 operand reads from shared memory are conflict-free and an
// 8 x 8 update needs four of them: the FMA pipe, not the shared-memory port, is the limit), 16-deep k
// slabs double-buffered: the next slab's global loads are issued before the current slab's FMAs and
// stored after them.  An operand whose unit stride is along k is fetched with float4 loads along k
// and scattered into the k-major tile; one whose unit stride is along m/n is fetched and stored as
// float4.  Anything unaligned or ragged falls back to guarded scalar loads of the same elements.
// Sums are fp32 in a fixed order (k ascending); the caller's tolerances allow for K up to a few
// thousand.
template <int R_, int NT>
struct TileIo {
  static constexpr int F = R_ * 16 / 4 / NT;     // float4 groups per thread
  const float* P;
  int64_t s_r, s_k;
  bool along_k, vec;
  int copies; int64_t cstride; float cinv;      // group copies averaged on the way in (see GemmDesc)
  __device__ __forceinline__ void add_copies(float (&t)[4], const float* p, bool as_vec, int64_t step, int valid) const {
    for (int c = 1; c < copies; ++c) {
      const float* q = p + c * cstride;
      if (as_vec) {
        const float4 v = *reinterpret_cast<const float4*>(q);
        t[0] = __fadd_rn(t[0], v.x); t[1] = __fadd_rn(t[1], v.y); t[2] = __fadd_rn(t[2], v.z); t[3] = __fadd_rn(t[3], v.w);
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) if (j < valid) t[j] = __fadd_rn(t[j], q[j * step]);
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) t[j] = __fmul_rn(t[j], cinv);
  }
  __device__ __forceinline__ void init(const float* p, int64_t sr, int64_t sk) {
    P = p; s_r = sr; s_k = sk; copies = 1; cstride = 0; cinv = 1.f;
    along_k = (sk == 1) || (sk < sr && sr != 1);
    const bool al = (reinterpret_cast<uintptr_t>(p) & 15u) == 0;
    vec = al && (along_k ? (sk == 1 && (sr & 3) == 0) : (sr == 1 && (sk & 3) == 0));
  }
  __device__ __forceinline__ void fetch(float4 (&v)[F], int64_t r0, int R, int64_t k0, int K, const float* kvec,
                                        int kmode, float thr, int tid) const {
#pragma unroll
    for (int e = 0; e < F; ++e) {
      const int f = tid + e * NT;
      float t[4];
      if (along_k) {
        const int k4 = f & 3, row = f >> 2;
        const int64_t gr = r0 + row, gk = k0 + 4 * k4;
        const float* p = P + gr * s_r + gk * s_k;
        if (vec && gr < R && gk + 3 < K) {
          const float4 q = *reinterpret_cast<const float4*>(p);
          t[0] = q.x; t[1] = q.y; t[2] = q.z; t[3] = q.w;
          if (copies > 1) add_copies(t, p, true, 0, 4);
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j) t[j] = (gr < R && gk + j < K) ? p[j * s_k] : 0.f;
          if (copies > 1 && gr < R) add_copies(t, p, false, s_k, (int)(K - gk < 4 ? (K - gk < 0 ? 0 : K - gk) : 4));
        }
        if (kvec) {
#pragma unroll
          for (int j = 0; j < 4; ++j) if (gk + j < K) t[j] *= diag_scale(kvec, (int)(gk + j), kmode, thr);
        }
      } else {
        const int r4 = f % (R_ / 4), kk = f / (R_ / 4);
        const int64_t gr = r0 + 4 * r4, gk = k0 + kk;
        const float* p = P + gr * s_r + gk * s_k;
        if (vec && gr + 3 < R && gk < K) {
          const float4 q = *reinterpret_cast<const float4*>(p);
          t[0] = q.x; t[1] = q.y; t[2] = q.z; t[3] = q.w;
          if (copies > 1) add_copies(t, p, true, 0, 4);
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j) t[j] = (gr + j < R && gk < K) ? p[j * s_r] : 0.f;
          if (copies > 1 && gk < K) add_copies(t, p, false, s_r, (int)(R - gr < 4 ? (R - gr < 0 ? 0 : R - gr) : 4));
        }
        if (kvec && gk < K) {
          const float sc = diag_scale(kvec, (int)gk, kmode, thr);
#pragma unroll
          for (int j = 0; j < 4; ++j) t[j] *= sc;
        }
      }
      v[e] = make_float4(t[0], t[1], t[2], t[3]);
    }
  }
  // writes the fetched values to a dense copy of the operand: element (r, k) at out[r * o_r + k * o_k]
  __device__ __forceinline__ void emit(float* out, int64_t o_r, int64_t o_k, const float4 (&v)[F], int64_t r0, int R,
                                       int64_t k0, int K, int tid) const {
#pragma unroll
    for (int e = 0; e < F; ++e) {
      const int f = tid + e * NT;
      const float t[4] = {v[e].x, v[e].y, v[e].z, v[e].w};
      if (along_k) {
        const int k4 = f & 3, row = f >> 2;
        const int64_t gr = r0 + row, gk = k0 + 4 * k4;
#pragma unroll
        for (int j = 0; j < 4; ++j) if (gr < R && gk + j < K) out[gr * o_r + (gk + j) * o_k] = t[j];
      } else {
        const int r4 = f % (R_ / 4), kk = f / (R_ / 4);
        const int64_t gr = r0 + 4 * r4, gk = k0 + kk;
#pragma unroll
        for (int j = 0; j < 4; ++j) if (gr + j < R && gk < K) out[(gr + j) * o_r + gk * o_k] = t[j];
      }
    }
  }
  __device__ __forceinline__ void stash(float (*S)[R_ + 4], const float4 (&v)[F], int tid) const {
#pragma unroll
    for (int e = 0; e < F; ++e) {
      const int f = tid + e * NT;
      if (along_k) {
        const int k4 = f & 3, row = f >> 2;
        S[4 * k4 + 0][row] = v[e].x; S[4 * k4 + 1][row] = v[e].y;
        S[4 * k4 + 2][row] = v[e].z; S[4 * k4 + 3][row] = v[e].w;
      } else {
        const int r4 = f % (R_ / 4), kk = f / (R_ / 4);
        *reinterpret_cast<float4*>(&S[kk][4 * r4]) = v[e];
      }
    }
  }
};

template <int BM_, int BN_>
__device__ __forceinline__ void gemm_tile_8x8(const GemmDesc& d) {
  constexpr int NT = (BM_ / 8) * (BN_ / 8);
  const int64_t m0 = (int64_t)blockIdx.y * BM_, n0 = (int64_t)blockIdx.x * BN_;
  if (m0 >= d.M || n0 >= d.N) return;
  if (d.upper_only && n0 + BN_ <= m0) return;
  __shared__ __align__(16) float As[2][BK][BM_ + 4];
  __shared__ __align__(16) float Bs[2][BK][BN_ + 4];
  const int tid = threadIdx.x;
  const int tx = tid % (BN_ / 8), ty = tid / (BN_ / 8);
  TileIo<BM_, NT> ioA;
  TileIo<BN_, NT> ioB;
  ioA.init(d.A, d.sAm, d.sAk);
  ioB.init(d.B, d.sBn, d.sBk);
  if (d.a_copies > 1) { ioA.copies = d.a_copies; ioA.cstride = d.a_cstride; ioA.cinv = d.copy_inv; }
  if (d.b_copies > 1) { ioB.copies = d.b_copies; ioB.cstride = d.b_cstride; ioB.cinv = d.copy_inv; }
  const bool emit_a = d.a_mean_out != nullptr && blockIdx.x == 0;     // first tile column writes Abar
  const bool emit_b = d.b_mean_out != nullptr && blockIdx.y == 0;     // first tile row writes Bbar
  float4 va[TileIo<BM_, NT>::F], vb[TileIo<BN_, NT>::F];
  float acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

  const int nk = (d.K + BK - 1) / BK;
  ioA.fetch(va, m0, d.M, 0, d.K, d.k_vec, d.k_mode, d.thr, tid);
  ioB.fetch(vb, n0, d.N, 0, d.K, nullptr, 0, 0.f, tid);
  if (emit_a) ioA.emit(d.a_mean_out, d.K, 1, va, m0, d.M, 0, d.K, tid);
  if (emit_b) ioB.emit(d.b_mean_out, 1, d.N, vb, n0, d.N, 0, d.K, tid);
  ioA.stash(As[0], va, tid);
  ioB.stash(Bs[0], vb, tid);
  __syncthreads();
  for (int kt = 0; kt < nk; ++kt) {
    const int cur = kt & 1;
    const bool more = kt + 1 < nk;
    if (more) {
      ioA.fetch(va, m0, d.M, (int64_t)(kt + 1) * BK, d.K, d.k_vec, d.k_mode, d.thr, tid);
      ioB.fetch(vb, n0, d.N, (int64_t)(kt + 1) * BK, d.K, nullptr, 0, 0.f, tid);
      if (emit_a) ioA.emit(d.a_mean_out, d.K, 1, va, m0, d.M, (int64_t)(kt + 1) * BK, d.K, tid);
      if (emit_b) ioB.emit(d.b_mean_out, 1, d.N, vb, n0, d.N, (int64_t)(kt + 1) * BK, d.K, tid);
    }
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      const float4 a0 = *reinterpret_cast<const float4*>(&As[cur][kk][ty * 4]);
      const float4 a1 = *reinterpret_cast<const float4*>(&As[cur][kk][BM_ / 2 + ty * 4]);
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[cur][kk][tx * 4]);
      const float4 b1 = *reinterpret_cast<const float4*>(&Bs[cur][kk][BN_ / 2 + tx * 4]);
      const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    if (more) {
      ioA.stash(As[cur ^ 1], va, tid);
      ioB.stash(Bs[cur ^ 1], vb, tid);
    }
    __syncthreads();
  }

  const int live_r = d.live_rows ? *d.live_rows : d.M;
  const int live_c = d.live_cols ? *d.live_cols : d.N;
  const bool c_vec = (d.ldc & 3) == 0 && (reinterpret_cast<uintptr_t>(d.C) & 15u) == 0;
  float cs[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const int64_t gn = n0 + (j < 4 ? tx * 4 + j : BN_ / 2 + tx * 4 + (j - 4));
    cs[j] = (gn < d.N && gn < live_c) ? diag_scale(d.col_vec, (int)gn, d.col_mode, d.thr) : 0.f;
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int64_t gm = m0 + (i < 4 ? ty * 4 + i : BM_ / 2 + ty * 4 + (i - 4));
    if (gm >= d.M) continue;
    const float rs = gm < live_r ? diag_scale(d.row_vec, (int)gm, d.row_mode, d.thr) : 0.f;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int64_t gn = n0 + (h == 0 ? tx * 4 : BN_ / 2 + tx * 4);
      float v[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) v[j] = acc[i][4 * h + j] * rs * cs[4 * h + j];
      if (c_vec && gn + 3 < d.N) {
        if (d.c_bf16) {
          __nv_bfloat162 lo = __floats2bfloat162_rn(v[0], v[1]), hi = __floats2bfloat162_rn(v[2], v[3]);
          uint2 pk;
          pk.x = *reinterpret_cast<uint32_t*>(&lo);
          pk.y = *reinterpret_cast<uint32_t*>(&hi);
          *reinterpret_cast<uint2*>(static_cast<bf16*>(d.C) + gm * d.ldc + gn) = pk;
        } else {
          *reinterpret_cast<float4*>(static_cast<float*>(d.C) + gm * d.ldc + gn) = make_float4(v[0], v[1], v[2], v[3]);
        }
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (gn + j >= d.N) continue;
          if (d.c_bf16) static_cast<bf16*>(d.C)[gm * d.ldc + gn + j] = __float2bfloat16_rn(v[j]);
          else static_cast<float*>(d.C)[gm * d.ldc + gn + j] = v[j];
        }
      }
    }
  }
}

template <int BM_, int BN_>
__global__ void __launch_bounds__((BM_ / 8) * (BN_ / 8), 512 / ((BM_ / 8) * (BN_ / 8)))
gemm_simt_batched_kernel(const GemmDesc* __restrict__ descs) {
  const GemmDesc d = descs[blockIdx.z];
  gemm_tile_8x8<BM_, BN_>(d);
}

// The same tile code for one problem whose descriptor travels as a kernel argument.
template <int BM_, int BN_>
__global__ void __launch_bounds__((BM_ / 8) * (BN_ / 8), 512 / ((BM_ / 8) * (BN_ / 8)))
gemm_simt_one_kernel(const __grid_constant__ GemmDesc d) {
  gemm_tile_8x8<BM_, BN_>(d);
}

template <int BM_, int BN_>
int launch_one(const GemmDesc& d, cudaStream_t st) {
  dim3 grid((unsigned)((d.N + BN_ - 1) / BN_), (unsigned)((d.M + BM_ - 1) / BM_), 1u);
  if (grid.y > 65535u) return AB_ERR_UNSUPPORTED;
  gemm_simt_one_kernel<BM_, BN_><<<grid, (BM_ / 8) * (BN_ / 8), 0, st>>>(d);
  AB_LAUNCH_OK();
  return AB_OK;
}

template <int BM_, int BN_>
int launch_batched(const GemmDesc* d_descs, int count, int max_M, int max_N, cudaStream_t st) {
  dim3 grid((unsigned)((max_N + BN_ - 1) / BN_), (unsigned)((max_M + BM_ - 1) / BM_), (unsigned)count);
  if (grid.y > 65535u || grid.z > 65535u) return AB_ERR_UNSUPPORTED;
  gemm_simt_batched_kernel<BM_, BN_><<<grid, (BM_ / 8) * (BN_ / 8), 0, st>>>(d_descs);
  AB_LAUNCH_OK();
  return AB_OK;
}

}  // namespace

// Tile edges of 128 for the long dimensions (m, n), 64 for the rank-sized ones.
int gemm_simt_batched(const GemmDesc* d_descs, int count, int max_M, int max_N, cudaStream_t st) {
  if (count <= 0 || max_M <= 0 || max_N <= 0) return AB_OK;
  const bool bigM = max_M >= 512, bigN = max_N >= 512;
  if (bigM && bigN) return launch_batched<128, 128>(d_descs, count, max_M, max_N, st);
  if (bigM) return launch_batched<128, 64>(d_descs, count, max_M, max_N, st);
  if (bigN) return launch_batched<64, 128>(d_descs, count, max_M, max_N, st);
  return launch_batched<64, 64>(d_descs, count, max_M, max_N, st);
}

int recombine_mean_simt(const float* A_copies, int64_t strideA, const float* B_copies, int64_t strideB, int K,
                        float* W, float* Abar, float* Bbar, int m, int n, int r, cudaStream_t st) {
  GemmDesc d;
  d.A = A_copies; d.B = B_copies; d.C = W;
  d.sAm = r; d.sAk = 1; d.sBk = n; d.sBn = 1; d.ldc = n;
  d.M = m; d.N = n; d.K = r; d.c_bf16 = 0;
  d.row_vec = d.col_vec = d.k_vec = nullptr;
  d.row_mode = d.col_mode = d.k_mode = 0;
  d.thr = 0.f;
  d.live_rows = d.live_cols = nullptr;
  d.upper_only = 0;
  d.a_copies = d.b_copies = K; d.a_cstride = strideA; d.b_cstride = strideB; d.copy_inv = 1.0f / (float)K;
  d.a_mean_out = Abar; d.b_mean_out = Bbar;
  const bool bigM = m >= 512, bigN = n >= 512;
  if (bigM && bigN) return launch_one<128, 128>(d, st);
  if (bigM) return launch_one<128, 64>(d, st);
  if (bigN) return launch_one<64, 128>(d, st);
  return launch_one<64, 64>(d, st);
}

int gemm_simt(const void* A, int a_dt, int64_t sAm, int64_t sAk,
              const void* B, int b_dt, int64_t sBk, int64_t sBn,
              void* C, int c_dt, int64_t ldc,
              int64_t M, int64_t N, int64_t K, cudaStream_t st) {
  if (M <= 0 || N <= 0) return AB_OK;
  const int64_t tiles64 = ((M + 63) / 64) * ((N + 63) / 64);
  if (a_dt == AB_F32 && b_dt == AB_F32 && c_dt == AB_F32 && M < ((int64_t)1 << 22) && N < ((int64_t)1 << 31) &&
      K < ((int64_t)1 << 31) && tiles64 >= 296) {
    // all-fp32 problems with enough tiles to fill the SMs twice take the register-tiled kernel (fp32
    // sums in ascending k); smaller ones are latency-bound and do better with 256 threads per tile
    GemmDesc d;
    d.A = static_cast<const float*>(A); d.B = static_cast<const float*>(B); d.C = C;
    d.sAm = sAm; d.sAk = sAk; d.sBk = sBk; d.sBn = sBn; d.ldc = ldc;
    d.M = (int)M; d.N = (int)N; d.K = (int)K; d.c_bf16 = 0;
    d.row_vec = d.col_vec = d.k_vec = nullptr;
    d.row_mode = d.col_mode = d.k_mode = 0;
    d.thr = 0.f;
    d.live_rows = d.live_cols = nullptr;
    d.upper_only = 0;
    d.a_copies = d.b_copies = 1; d.a_cstride = d.b_cstride = 0; d.copy_inv = 1.f; d.a_mean_out = d.b_mean_out = nullptr;
    const bool bigM = M >= 512, bigN = N >= 512;
    if (bigM && bigN) return launch_one<128, 128>(d, st);
    if (bigM) return launch_one<128, 64>(d, st);
    if (bigN) return launch_one<64, 128>(d, st);
    return launch_one<64, 64>(d, st);
  }
  // rows beyond 65535 tiles are covered by splitting M into bands
  const int64_t band = (int64_t)65535 * BM;
  for (int64_t mo = 0; mo < M; mo += band) {
    int64_t mb = (M - mo < band) ? (M - mo) : band;
    const char* Ap = static_cast<const char*>(A) + mo * sAm * (int64_t)dtype_size(a_dt);
    char* Cp = static_cast<char*>(C) + mo * ldc * (int64_t)dtype_size(c_dt);
    int s;
#define AB_GEMM_CASE(TA, TB, TC) s = launch<TA, TB, TC>(Ap, sAm, sAk, B, sBk, sBn, Cp, ldc, mb, N, K, st)
    int key = (a_dt << 2) | (b_dt << 1) | c_dt;
    switch (key) {
      case 0: AB_GEMM_CASE(float, float, float); break;
      case 1: AB_GEMM_CASE(float, float, bf16); break;
      case 2: AB_GEMM_CASE(float, bf16, float); break;
      case 3: AB_GEMM_CASE(float, bf16, bf16); break;
      case 4: AB_GEMM_CASE(bf16, float, float); break;
      case 5: AB_GEMM_CASE(bf16, float, bf16); break;
      case 6: AB_GEMM_CASE(bf16, bf16, float); break;
      default: AB_GEMM_CASE(bf16, bf16, bf16); break;
    }
#undef AB_GEMM_CASE
    if (s != AB_OK) return s;
  }
  return AB_OK;
}

}  // namespace ab
