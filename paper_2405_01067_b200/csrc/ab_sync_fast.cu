// Factored group synchronisation: the split of W = Abar Bbar (Algorithm 1, the decomposition that
// follows the all-reduces and "W <- AB") without ever forming the m x n matrix.  W has rank <= r,
// so everything reduces to r x r problems:
//   G_A = Abar^T Abar = R_A^T R_A,   G_B = Bbar Bbar^T = R_B^T R_B      (Cholesky, r x r, upper R)
//   Abar = Q_A R_A,  Bbar^T = Q_B R_B   with Q_A = Abar R_A^-1, Q_B = Bbar^T R_B^-1 orthonormal
//   W = Q_A M Q_B^T,  M = R_A R_B^T  (r x r),   M = U_M S V_M^T         (SVD, r x r)
//   A' = Abar Z_A,  Z_A = R_A^-1 (M V_M) S^(-1/2);   B' = Z_B Bbar,  Z_B = S^(1/2) V_M^T R_B^-T
// One CTA per Gram matrix factors it in shared memory and inverts the triangle in place; one CTA
// per M keeps it in shared memory and orthogonalises its ROWS with one-sided Jacobi rotations
// (the rows of the result are sigma_i v_i^T), so no kernel boundary and no global traffic sits
// between rotations.  Cholesky pivots below 1e-6 of the largest diagonal entry of G are treated
// as zero: the row of R and the row and column of its inverse are dropped, which is exactly right
// for factors truncated by the rank rule (zero columns of A, zero rows of B).  Otherwise the
// factors need a condition number below about 300 -- all workloads here are far inside.
#include <algorithm>
#include <cstring>
#include <mutex>
#include <type_traits>
#include <vector>

#include <cooperative_groups.h>

#include "ab_common.cuh"

namespace ab {
namespace {

namespace cg = cooperative_groups;

constexpr int kJMaxSweeps = 40;
constexpr float kJDead2 = 1e-12f;    // rows below 1e-6 of the largest norm are zero rows
constexpr float kJCount2 = 1e-8f;    // rows below 1e-4 of the largest norm do not hold up convergence
constexpr float kJEarly2 = 4e-6f;    // a sweep whose largest rotated cosine was below 2e-3 is the last one: one-sided
                                     // Jacobi converges quadratically, so what it leaves is of the order 4e-6 <= tol
constexpr float kEigThr = 1e-6f;     // relative pivot cut of G_A, G_B (and of sigma in the scalings)
// Accuracy domain of the factored route: the relative error of a singular value grows as it falls below the
// largest and the worse conditioned the factors are (measured: at most 7e-5 down to 1 % of the largest for
// factors of condition number up to 1e4; 1e-4 to 5e-3 below that); a kept value between
// kFZeroRel and kFDomainRel of the largest, or a Cholesky pivot that was dropped although it was not exactly
// zero, is reported through the status word.
constexpr float kFDomainRel = 1e-2f, kFZeroRel = 1e-6f;
constexpr int kCThreads = 512;

struct JacobiJob {
  const float* X;   // k x r input (row stride r)
  float* rows;      // k x r output: unit rows, sorted by descending norm (zero rows stay zero)
  float* norms;     // k
  int* status;      // AB_OK / AB_ERR_NOT_CONVERGED (may be null)
  int k, r;
};

__device__ __forceinline__ void rr_pair2(int ne, int t, int idx, int& p, int& q) {
  // t < ne - 1 and idx < ne / 2: one conditional subtraction replaces each modulo
  const int n1 = ne - 1;
  if (idx == 0) { p = n1; q = t; }
  else {
    p = t + idx; if (p >= n1) p -= n1;
    q = t - idx + n1; if (q >= n1) q -= n1;
  }
  if (p > q) { int tmp = p; p = q; q = tmp; }
}

// One matrix per cluster of kC CTAs.  Rows are grouped in blocks of 4; block b lives in the shared
// memory of CTA b % kC, and every CTA reads and writes any row through distributed shared memory.
// Each row carries its squared norm in the padding element behind it.  In each round a warp takes
// one pair of blocks, pulls its 8 rows into registers (r/32 elements per lane and row), rotates the
// 16 cross pairs (4 steps of 4 disjoint pairs worked on side by side; in the first round of a
// sweep also the pairs inside each block) and writes the rows back: shared memory is touched once
// per 16 rotations.  Rounds end with a cluster barrier (a hardware barrier: every CTA of the
// cluster runs the same number of them, since sweep and round counts depend only on values all
// CTAs agree on).
template <int kEL, int kC>      // kEL elements per lane and row in registers: r <= 32 kEL
__global__ void __launch_bounds__((kC == 1 && kEL == 6) ? 768 : 512, 1)
jacobi_rows_cluster_kernel(const JacobiJob* __restrict__ jobs, float tol) {
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ __align__(16) float sm[];
  const int crank = (kC == 1) ? 0 : (int)cluster.block_rank();
  const JacobiJob job = jobs[blockIdx.x / kC];
  const int k = job.k, r = job.r, ld = r + 1;
  const int nb = (k + 3) / 4;                  // blocks of 4 rows
  const int nbl = (nb + kC - 1) / kC;          // blocks held by each CTA (same layout in all)
  float* X = sm;                               // 4 nbl x ld; X[i * ld + r] = squared norm of local row i
  float* zrow = X + (size_t)4 * nbl * ld;      // ld zeros: stands in for rows beyond k (rotations leave it zero)
  float* lmax = zrow + ld;                     // kC: largest squared norm seen by each CTA
  int* lflag = reinterpret_cast<int*>(lmax + kC);   // kC: per CTA, the largest squared cosine it rotated (float bits)
  int* rank = lflag + kC;                      // 4 nbl
  __shared__ int wflag;
  __shared__ float wmax;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nthreads = blockDim.x, nwarps = nthreads >> 5;
  auto csync = [&]() {                         // all CTAs that hold a part of this matrix
    if constexpr (kC == 1) __syncthreads(); else cluster.sync();
  };

  auto row_ptr = [&](int row) -> float* {      // any row of the matrix, wherever it lives
    const int b = row >> 2;
    float* p = X + (size_t)(((b / kC) << 2) + (row & 3)) * ld;
    if (kC == 1) return p;
    return cluster.map_shared_rank(p, b % kC);
  };
  auto global_row = [&](int lr) { return (((lr >> 2) * kC + crank) << 2) + (lr & 3); };
  const int nlocal = 4 * nbl;

  for (int lr = warp; lr < nlocal; lr += nwarps) {
    const int g = global_row(lr);
    for (int t = lane; t < r; t += 32) X[lr * ld + t] = (g < k) ? job.X[(size_t)g * r + t] : 0.f;
  }
  for (int t = tid; t < ld; t += nthreads) zrow[t] = 0.f;
  csync();                              // every CTA of the cluster is running and loaded

  // exact squared norms of the local rows into their padding element; the cluster-wide maximum
  auto refresh_norms = [&]() -> float {
    if (tid == 0) { wmax = 0.f; wflag = 0; }
    __syncthreads();
    for (int lr = warp; lr < nlocal; lr += nwarps) {
      float a = 0.f;
      for (int t = lane; t < r; t += 32) { const float v = X[lr * ld + t]; a = fmaf(v, v, a); }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
      if (lane == 0) { X[lr * ld + r] = a; atomicMax(reinterpret_cast<int*>(&wmax), __float_as_int(a)); }
    }
    __syncthreads();
    if (tid < kC) {
      float* dst = (kC == 1) ? lmax : cluster.map_shared_rank(lmax, tid);
      dst[crank] = wmax;
    }
    csync();
    float m = 0.f;
#pragma unroll
    for (int c = 0; c < kC; ++c) m = fmaxf(m, lmax[c]);
    return m;
  };

  const int nbe = nb + (nb & 1);
  const int brounds = nbe > 2 ? nbe - 1 : 1;
  int sweeps = 0;
  bool converged = (k < 2);
  for (; sweeps < kJMaxSweeps && !converged; ++sweeps) {
    const float max_n2 = refresh_norms();      // the running updates drift: exact norms every sweep
    const float dead2 = kJDead2 * max_n2, count2 = kJCount2 * max_n2;
    for (int round = 0; round < brounds; ++round) {
      for (int task = crank + kC * warp; task < nbe / 2; task += kC * nwarps) {
        int bi, bj;
        rr_pair2(nbe, round, task, bi, bj);
        const bool has_j = bj < nb;
        if (bi >= nb) continue;
        if (!has_j && round != 0) continue;
        float x[8][kEL];
        float nn[8];
        // where each of the 8 rows lives: an offset into X for a single CTA (fewer registers and
        // plain shared-memory addressing), a pointer that may lead to a peer's shared memory otherwise
        typename std::conditional<kC == 1, int, float*>::type ref[8];
        auto at = [&](int a) -> float* {
          if constexpr (kC == 1) return X + ref[a]; else return ref[a];
        };
#pragma unroll
        for (int a = 0; a < 8; ++a) {
          const int row = (a < 4 ? bi * 4 + a : bj * 4 + (a - 4));
          const bool in = row < k && (a < 4 || has_j);
          if constexpr (kC == 1) ref[a] = in ? row * ld : 4 * nbl * ld;
          else ref[a] = in ? row_ptr(row) : zrow;
        }
        const bool full = (r == 32 * kEL);       // every lane element exists: no per-element checks
#pragma unroll
        for (int a = 0; a < 8; ++a) {
          const float* rp = at(a);
          nn[a] = rp[r];
          if (full) {
#pragma unroll
            for (int e = 0; e < kEL; ++e) x[a][e] = rp[lane + 32 * e];
          } else {
#pragma unroll
            for (int e = 0; e < kEL; ++e) {
              const int t = lane + 32 * e;
              x[a][e] = (t < r) ? rp[t] : 0.f;
            }
          }
        }
        unsigned counted = 0u;                  // largest squared cosine among the pairs rotated here (float bits)
#pragma unroll
        for (int stp = 0; stp < 7; ++stp) {     // fully unrolled: every register index below is a constant
          if (stp >= 4 && round != 0) break;
          // pairs of this step: cross steps pair row a with row 4 + (a + stp) % 4; the three extra
          // steps of round 0 are the rest of an 8-player tournament (pairs inside the blocks)
          float g[4], c[4], sn[4];
          int pa[4], pb[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            if (stp < 4) { pa[u] = u; pb[u] = 4 + ((u + stp) & 3); }
            else if (stp == 4) { pa[u] = (u < 2) ? 0 + 2 * u : 4 + 2 * (u - 2); pb[u] = pa[u] + 1; }          // (0,1)(2,3)(4,5)(6,7)
            else if (stp == 5) { pa[u] = (u < 2) ? u : 4 + (u - 2); pb[u] = pa[u] + 2; }                         // (0,2)(1,3)(4,6)(5,7)
            else { pa[u] = (u < 2) ? u : 4 + (u - 2); pb[u] = (u < 2) ? 3 - u : 7 - (u - 2); }                  // (0,3)(1,2)(4,7)(5,6)
            g[u] = 0.f;
          }
          // dot products (register indices are resolved by full unrolling over the 8 x 8 choices)
#pragma unroll
          for (int u = 0; u < 4; ++u) {
#pragma unroll
            for (int a = 0; a < 8; ++a)
#pragma unroll
              for (int bb = 0; bb < 8; ++bb)
                if (a == pa[u] && bb == pb[u]) {
#pragma unroll
                  for (int e = 0; e < kEL; ++e) g[u] = fmaf(x[a][e], x[bb][e], g[u]);
                }
          }
          // four sums across the warp in 6 shuffles: each exchange halves what a lane still carries
          // (two of the four values after the first, one after the second); the lanes of octet u
          // (lanes 8u .. 8u+7) end up with the whole of g[u]
          float gsum;
          {
            const bool h16 = (lane & 16) != 0, h8 = (lane & 8) != 0;
            float k0 = h16 ? g[2] : g[0], k1 = h16 ? g[3] : g[1];
            const float s0 = h16 ? g[0] : g[2], s1 = h16 ? g[1] : g[3];
            k0 += __shfl_xor_sync(0xffffffffu, s0, 16);
            k1 += __shfl_xor_sync(0xffffffffu, s1, 16);
            gsum = h8 ? k1 : k0;
            const float sd = h8 ? k0 : k1;
            gsum += __shfl_xor_sync(0xffffffffu, sd, 8);
            gsum += __shfl_xor_sync(0xffffffffu, gsum, 4);
            gsum += __shfl_xor_sync(0xffffffffu, gsum, 2);
            gsum += __shfl_xor_sync(0xffffffffu, gsum, 1);
          }
          // rotation parameters: the lanes of octet u work out pair u, then the results are broadcast
          float appv[4], aqqv[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            appv[u] = 0.f; aqqv[u] = 0.f;
#pragma unroll
            for (int a = 0; a < 8; ++a) { if (a == pa[u]) appv[u] = nn[a]; if (a == pb[u]) aqqv[u] = nn[a]; }
          }
          const int lu = lane >> 3;
          const float my_g = gsum;
          const float my_app = lu == 0 ? appv[0] : lu == 1 ? appv[1] : lu == 2 ? appv[2] : appv[3];
          const float my_aqq = lu == 0 ? aqqv[0] : lu == 1 ? aqqv[1] : lu == 2 ? aqqv[2] : aqqv[3];
          const bool my_act = my_app > dead2 && my_aqq > dead2 && my_app > 0.f && my_aqq > 0.f &&
                              my_g * my_g > tol * tol * my_app * my_aqq;
          float my_c = 1.f, my_s = 0.f, my_dn = 0.f;
          if (my_act) {
            float zeta = __fdividef(my_aqq - my_app, 2.f * my_g);
            zeta = fminf(fmaxf(zeta, -1e15f), 1e15f);
            const float h = fmaf(zeta, zeta, 1.f);
            const float t1 = __fdividef(copysignf(1.f, zeta), fabsf(zeta) + h * rsqrtf(h));
            my_c = rsqrtf(fmaf(t1, t1, 1.f));
            my_s = my_c * t1;
            my_dn = t1 * my_g;
          }
          const bool my_counted = my_act && my_app > count2 && my_aqq > count2;
          const float my_cos2 = my_counted ? __fdividef(my_g * my_g, my_app * my_aqq) : 0.f;
          counted = max(counted, __reduce_max_sync(0xffffffffu, __float_as_uint(my_cos2)));
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            c[u] = __shfl_sync(0xffffffffu, my_c, 8 * u);
            sn[u] = __shfl_sync(0xffffffffu, my_s, 8 * u);
            const float dn = __shfl_sync(0xffffffffu, my_dn, 8 * u);
#pragma unroll
            for (int a = 0; a < 8; ++a) { if (a == pa[u]) nn[a] = appv[u] - dn; if (a == pb[u]) nn[a] = aqqv[u] + dn; }
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
#pragma unroll
            for (int a = 0; a < 8; ++a)
#pragma unroll
              for (int bb = 0; bb < 8; ++bb)
                if (a == pa[u] && bb == pb[u]) {
#pragma unroll
                  for (int e = 0; e < kEL; ++e) {
                    const float xp = x[a][e], xq = x[bb][e];
                    x[a][e] = c[u] * xp - sn[u] * xq;
                    x[bb][e] = sn[u] * xp + c[u] * xq;
                  }
                }
          }
        }
#pragma unroll
        for (int a = 0; a < 8; ++a) {
          float* rp = at(a);
          if (full) {
#pragma unroll
            for (int e = 0; e < kEL; ++e) rp[lane + 32 * e] = x[a][e];
          } else {
#pragma unroll
            for (int e = 0; e < kEL; ++e) {
              const int t = lane + 32 * e;
              if (t < r) rp[t] = x[a][e];
            }
          }
          if (lane == 0) rp[r] = nn[a];
        }
        if (lane == 0 && counted) atomicMax(&wflag, (int)counted);
      }
      csync();                          // all rows of this round are back in place
    }
    if (tid < kC) {
      int* dst = (kC == 1) ? lflag : cluster.map_shared_rank(lflag, tid);
      dst[crank] = wflag;
    }
    csync();
    int any = 0;
#pragma unroll
    for (int c = 0; c < kC; ++c) any = max(any, lflag[c]);
    converged = (__int_as_float(any) <= kJEarly2);     // nothing rotated, or only by angles whose square is noise
  }

  // norms, descending order, unit rows: each CTA finishes the rows it holds
  const float max_n2 = refresh_norms();
  for (int lr = tid; lr < nlocal; lr += nthreads) {
    const int gi = global_row(lr);
    if (gi >= k) continue;
    const float li = X[lr * ld + r];
    int rk = 0;
    for (int j = 0; j < k; ++j) { const float lj = row_ptr(j)[r]; rk += (lj > li) || (lj == li && j < gi); }
    rank[lr] = rk;
  }
  __syncthreads();
  const float dead2 = kJDead2 * max_n2;
  for (int lr = warp; lr < nlocal; lr += nwarps) {
    if (global_row(lr) >= k) continue;
    const float a = X[lr * ld + r];
    const bool live = a > dead2 && a > 0.f;
    const float nrm = live ? sqrtf(a) : 0.f, inv = live ? 1.f / nrm : 0.f;
    float* dst = job.rows + (size_t)rank[lr] * r;
    for (int t = lane; t < r; t += 32) dst[t] = X[lr * ld + t] * inv;
    if (lane == 0) job.norms[rank[lr]] = nrm;
  }
  if (crank == 0 && tid == 0 && job.status) *job.status = converged ? AB_OK : AB_ERR_NOT_CONVERGED;
  csync();                              // nobody leaves while a peer may still read its rows
}

size_t jacobi_smem_bytes(int k, int r, int C) {
  const int nbl = ((k + 3) / 4 + C - 1) / C;
  return sizeof(float) * ((size_t)(4 * nbl + 1) * (r + 1) + C) + sizeof(int) * ((size_t)C + 4 * nbl) + 64;
}

template <int EL, int C>
cudaLaunchConfig_t jacobi_config(int count, int rmax, cudaStream_t st, cudaLaunchAttribute* attr) {
  const int tasks = ((rmax + 3) / 4 + 1) / 2;                         // block pairs per round
  const int max_warps = (C == 1 && EL == 6) ? 24 : 16;              // matches the kernel's launch bounds
  const int warps = std::max(1, std::min(max_warps, (tasks + C - 1) / C));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(count * C));
  cfg.blockDim = dim3((unsigned)(32 * warps));
  cfg.dynamicSmemBytes = jacobi_smem_bytes(rmax, rmax, C);
  cfg.stream = st;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cfg;
}
// Launches with clusters of C CTAs if `count` such clusters can be resident at once (or if C == 1).
// Returns 1 when it declined, so that the caller tries a narrower cluster.
template <int EL, int C>
int try_launch_jacobi(const JacobiJob* jobs, int count, int rmax, float tol, cudaStream_t st) {
  cudaLaunchAttribute attr[1];
  cudaLaunchConfig_t cfg = jacobi_config<EL, C>(count, rmax, st, attr);
  if (cfg.dynamicSmemBytes > 227u * 1024u) return C == 1 ? AB_ERR_UNSUPPORTED : 1;
  AB_CUDA_OK(cudaFuncSetAttribute(jacobi_rows_cluster_kernel<EL, C>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  (int)cfg.dynamicSmemBytes));
  if (C > 1) {
    // one CTA per SM: CTAs that share an SM would only take turns on its issue slots
    int resident = 0;
    const int sms = sm_count();
    if (sms <= 0) return AB_ERR_CUDA;
    if (rmax < 16 * C || (long long)count * C > sms) return 1;
    if (cudaOccupancyMaxActiveClusters(&resident, jacobi_rows_cluster_kernel<EL, C>, &cfg) != cudaSuccess) {
      (void)cudaGetLastError();
      return 1;
    }
    if (resident < count) return 1;
  }
  AB_CUDA_OK(cudaLaunchKernelEx(&cfg, jacobi_rows_cluster_kernel<EL, C>, jobs, tol));
  AB_LAUNCH_OK();
  return AB_OK;
}
// Clusters of 8 or 4 CTAs per matrix when that many SMs are free for every matrix, else one CTA each
// (measured: a pair of CTAs gains nothing over one CTA with twice the warps; the round time is then
// set by the latency of one warp's 16 rotations, not by issue slots).
template <int EL>
int launch_jacobi_el(const JacobiJob* jobs, int count, int rmax, float tol, cudaStream_t st) {
  int s = try_launch_jacobi<EL, 8>(jobs, count, rmax, tol, st);
  if (s == 1) s = try_launch_jacobi<EL, 4>(jobs, count, rmax, tol, st);
  if (s == 1) s = try_launch_jacobi<EL, 1>(jobs, count, rmax, tol, st);
  if (s == AB_ERR_UNSUPPORTED) {            // too large for one CTA's shared memory: two CTAs hold half each
    s = try_launch_jacobi<EL, 2>(jobs, count, rmax, tol, st);
    if (s == 1) s = AB_ERR_UNSUPPORTED;
  }
  return s;
}
int launch_jacobi(const JacobiJob* jobs, int count, int rmax, float tol, cudaStream_t st) {
  if (rmax <= 64) return launch_jacobi_el<2>(jobs, count, rmax, tol, st);
  if (rmax <= 128) return launch_jacobi_el<4>(jobs, count, rmax, tol, st);
  if (rmax <= 192) return launch_jacobi_el<6>(jobs, count, rmax, tol, st);
  return launch_jacobi_el<8>(jobs, count, rmax, tol, st);
}

constexpr int kCPanel = 8;       // rows per panel of the Cholesky elimination (kCThreads / 64)

struct CholJob {
  const float* G;   // nparts partial sums of an r x r symmetric positive semi-definite matrix (row stride r,
                    // r * r apart); only the upper triangle is read
  int nparts;
  float* R;         // r x r upper triangular, G = R^T R; zeros below the diagonal, dropped rows zero
  float* Rinv;      // r x r upper triangular inverse of the kept part; dropped rows and columns zero
  int* status;      // receives AB_OK (may be null)
  int r;
};

// Right-looking Cholesky of one Gram matrix in shared memory (r <= 256), then the inverse of the
// triangle by back substitution, one warp per column.  R lives in the upper triangle; column j of
// the inverse is parked in the strict lower triangle of row j (contiguous), its diagonal in dinv[].
__global__ void __launch_bounds__(kCThreads, 1) chol_inv_kernel(const CholJob* __restrict__ jobs) {
  extern __shared__ __align__(16) float sm[];
  const CholJob job = jobs[blockIdx.x];
  const int r = job.r, ld = r + 1;
  float* S = sm;                       // r x ld
  float* dinv = S + (size_t)r * ld;    // r
  __shared__ float maxdiag;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nwarps = kCThreads / 32;

  __shared__ int dropped_live;          // pivots taken as zero although they were not exactly zero
  if (tid == 0) { maxdiag = 0.f; dropped_live = 0; }
  {
    const float* __restrict__ G = job.G;
    const size_t part = (size_t)r * r;
    for (int i = warp; i < r; i += nwarps) {           // one row per warp; the loads of a row are all in flight
      const float* g = G + (size_t)i * r;
#pragma unroll 8
      for (int k = lane; k < r; k += 32) {
        float v = g[k];
        for (int q = 1; q < job.nparts; ++q) v += g[q * part + k];                 // ascending part order
        S[i * ld + k] = v;
      }
    }
  }
  __syncthreads();
  for (int i = tid; i < r; i += kCThreads)
    atomicMax(reinterpret_cast<int*>(&maxdiag), __float_as_int(fmaxf(S[i * ld + i], 0.f)));
  __syncthreads();
  const float cut = kEigThr * maxdiag;

  // Panels of kCPanel rows: inside a panel the rows are finished one after the other (scale row j,
  // subtract it from the few panel rows below it), then all rows below the panel take the panel's
  // kCPanel rank-one terms in one pass, in ascending j -- the same sums per entry as a column-by-column
  // elimination, with one long step per panel instead of one per column.
  for (int j0 = 0; j0 < r; j0 += kCPanel) {
    const int jend = (j0 + kCPanel < r) ? j0 + kCPanel : r;
    for (int j = j0; j < jend; ++j) {
      const float dj = S[j * ld + j];
      const bool live = dj > cut && dj > 0.f;
      const float inv = live ? 1.f / sqrtf(dj) : 0.f;
      for (int k = j + 1 + tid; k < r; k += kCThreads) S[j * ld + k] *= inv;   // a dropped row becomes zero
      __syncthreads();
      if (tid == 0) {
        S[j * ld + j] = dj * inv; dinv[j] = inv;                                // nobody reads the pivot below
        if (!live && dj != 0.f) dropped_live = 1;
      }
      {                                              // panel rows still open: 64 threads per row
        const int i = j + 1 + (tid >> 6);
        if (i < jend) {
          const float f = S[j * ld + i];
          for (int k = i + (tid & 63); k < r; k += 64) S[i * ld + k] = fmaf(-f, S[j * ld + k], S[i * ld + k]);
        }
      }
      __syncthreads();
    }
    const int np = jend - j0;
    for (int i = jend + warp; i < r; i += nwarps) {
      float f[kCPanel];
#pragma unroll
      for (int q = 0; q < kCPanel; ++q) f[q] = (q < np) ? S[(j0 + q) * ld + i] : 0.f;
      for (int k = i + lane; k < r; k += 32) {
        float acc = S[i * ld + k];
#pragma unroll
        for (int q = 0; q < kCPanel; ++q)
          if (q < np) acc = fmaf(-f[q], S[(j0 + q) * ld + k], acc);
        S[i * ld + k] = acc;
      }
    }
    __syncthreads();
  }

  // X = R^-1 restricted to the kept rows, one warp per column j, by back substitution in update
  // form: lane l owns rows l, l + 32, ... of the column.  b starts as e_j; going down from k = j,
  // x_k = b_k / R_kk is final (one shuffle hands it to all lanes) and every row i < k takes
  // b_i -= R_ik x_k -- no reduction across lanes, and only the upper triangle (R) is read.
  for (int j = warp; j < r; j += nwarps) {
    float b[8], dk[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int i = 32 * e + lane;
      b[e] = (i == j) ? 1.f : 0.f;
      dk[e] = (i < r) ? dinv[i] : 0.f;
    }
#pragma unroll
    for (int e = 7; e >= 0; --e) {
      if (32 * e > j) continue;                  // uniform over the warp
      const int ltop = (j - 32 * e < 31) ? j - 32 * e : 31;
      for (int l = ltop; l >= 0; --l) {
        const int k = 32 * e + l;
        const float xk = __shfl_sync(0xffffffffu, b[e] * dk[e], l);
        if (lane == l) b[e] = xk;
#pragma unroll
        for (int e2 = 0; e2 <= e; ++e2) {
          const int i = 32 * e2 + lane;
          if (i < k) b[e2] = fmaf(-S[i * ld + k], xk, b[e2]);
        }
      }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int i = 32 * e + lane;
      if (i < j) S[j * ld + i] = b[e];           // column j of X, parked in row j below the diagonal
    }
  }
  __syncthreads();
  for (int idx = tid; idx < r * r; idx += kCThreads) {
    const int i = idx / r, k = idx % r;
    job.R[idx] = (k >= i) ? S[i * ld + k] : 0.f;
    job.Rinv[idx] = (k > i) ? S[k * ld + i] : (k == i ? dinv[i] : 0.f);
  }
  if (tid == 0 && job.status) *job.status = dropped_live ? (int)AB_ERR_ACCURACY : (int)AB_OK;
}

size_t chol_smem_bytes(int r) { return sizeof(float) * ((size_t)r * (r + 1) + r) + 64; }

// r' = #{ i < r : sigma_i >= cutoff * sigma_0 } (at least 1); folds the three solver statuses.
__global__ void fast_rank_rule_kernel(const float* const* __restrict__ sigma, const int* __restrict__ rs,
                                      float cutoff, int* const* __restrict__ r_out,
                                      const int* __restrict__ jstatus, int* __restrict__ dev_status, int L) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= L) return;
  const float* sg = sigma[i];
  const int r = rs[i];
  float top = 0.f;
  for (int k = 0; k < r; ++k) top = fmaxf(top, sg[k]);
  int keep = 0;
  for (int k = 0; k < r; ++k) keep += (sg[k] >= cutoff * top) ? 1 : 0;
  if (keep < 1) keep = 1;
  *r_out[i] = keep;
  if (dev_status) {
    int st = AB_OK;
    for (int k = 0; k < keep; ++k)
      if (sg[k] < kFDomainRel * top && sg[k] > kFZeroRel * top) st = AB_ERR_ACCURACY;
    for (int j = 0; j < 3; ++j) if (jstatus[3 * i + j] == AB_ERR_ACCURACY) st = AB_ERR_ACCURACY;
    for (int j = 0; j < 3; ++j)          // a solver that did not converge outranks the accuracy note
      if (jstatus[3 * i + j] != AB_OK && jstatus[3 * i + j] != AB_ERR_ACCURACY) st = jstatus[3 * i + j];
    dev_status[i] = st;
  }
}

// A bounded wait that ran out inside one of the tensor-core launches of the call reaches every matrix's status.
__global__ void fold_tc_status_kernel(const int* __restrict__ tc_status, int* __restrict__ dev_status, int L) {
  const int bad = (tc_status[0] != AB_OK) ? tc_status[0] : (tc_status[1] != AB_OK) ? tc_status[1] : tc_status[2];
  if (bad == AB_OK) return;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < L; i += gridDim.x * blockDim.x) dev_status[i] = bad;
}

// The long index of a Gram product is cut into slices of about kGramSlice (at most kGramMaxParts).
constexpr int kGramSlice = 768, kGramMaxParts = 8;
int gram_parts(int len) { return std::max(1, std::min(kGramMaxParts, (len + kGramSlice - 1) / kGramSlice)); }
int gram_k0(int len, int parts, int q) {      // start of slice q (a multiple of 16), len for q == parts
  if (q >= parts) return len;
  const int per = (((len + parts - 1) / parts) + 15) / 16 * 16;
  return std::min(len, q * per);
}

struct FastWs {
  std::vector<float*> Abar, Bbar, GA, GB, RA, RB, IA, IB, M, Vs, Y1, ZA, ZB;
  GemmDesc* descs;      // 9 L
  GemmDesc* gram_descs; // up to 2 kGramMaxParts L
  CholJob* cjobs;       // 2 L
  AvgJob* ajobs;        // 2 L
  JacobiJob* jobs;      // L
  int* jstatus;         // 3 L
  const float** sig_ptrs;
  int** rout_ptrs;
  int* rs;
  // tensor-core route of the long products: bf16 pieces (hi, mid, lo) of Abar, Bbar, Z_A, Z_B
  SplitJob* sjobs;      // 4 L
  std::vector<bf16*> Asp, Bsp, ZAsp, ZBsp;    // each: three pieces one after the other
  void* tc_table[3];    // problem tables of the three tensor-core launches
  int* tc_status;
  size_t bytes;
};

int r8(int v) { return (v + 7) & ~7; }

FastWs fast_layout(const ab_sync_desc* d, int L, void* ws) {
  FastWs w;
  Arena ar(ws, 0);
  auto each = [&](std::vector<float*>& v, auto count) {
    v.resize(L);
    for (int i = 0; i < L; ++i) v[i] = ar.take_n<float>(count(d[i]));
  };
  each(w.Abar, [](const ab_sync_desc& x) { return (size_t)x.m * x.r; });
  each(w.Bbar, [](const ab_sync_desc& x) { return (size_t)x.r * x.n; });
  auto rr = [](const ab_sync_desc& x) { return (size_t)x.r * x.r; };
  each(w.GA, [](const ab_sync_desc& x) { return (size_t)gram_parts(x.m) * x.r * x.r; });
  each(w.GB, [](const ab_sync_desc& x) { return (size_t)gram_parts(x.n) * x.r * x.r; });
  each(w.RA, rr); each(w.RB, rr); each(w.IA, rr); each(w.IB, rr);
  each(w.M, rr); each(w.Vs, rr); each(w.Y1, rr); each(w.ZA, rr); each(w.ZB, rr);
  w.descs = ar.take_n<GemmDesc>((size_t)9 * L);
  w.gram_descs = ar.take_n<GemmDesc>((size_t)2 * kGramMaxParts * L);
  w.cjobs = ar.take_n<CholJob>((size_t)2 * L);
  w.ajobs = ar.take_n<AvgJob>((size_t)2 * L);
  w.jobs = ar.take_n<JacobiJob>((size_t)L);
  w.jstatus = ar.take_n<int>((size_t)3 * L);
  w.sig_ptrs = ar.take_n<const float*>(L);
  w.rout_ptrs = ar.take_n<int*>(L);
  w.rs = ar.take_n<int>(L);
  w.sjobs = ar.take_n<SplitJob>((size_t)4 * L);
  auto each_bf = [&](std::vector<bf16*>& v, auto count) {
    v.resize(L);
    for (int i = 0; i < L; ++i) v[i] = ar.take_n<bf16>(3 * count(d[i]));
  };
  each_bf(w.Asp, [](const ab_sync_desc& x) { return (size_t)x.m * r8(x.r); });
  each_bf(w.Bsp, [](const ab_sync_desc& x) { return (size_t)x.r * r8(x.n); });
  each_bf(w.ZAsp, [](const ab_sync_desc& x) { return (size_t)x.r * r8(x.r); });
  each_bf(w.ZBsp, [](const ab_sync_desc& x) { return (size_t)x.r * r8(x.r); });
  w.tc_table[0] = ar.take(gemm_tc_table_bytes(2 * L));
  w.tc_table[1] = ar.take(gemm_tc_table_bytes(2 * L));
  w.tc_table[2] = ar.take(gemm_tc_table_bytes(L));
  w.tc_status = ar.take_n<int>(64);
  w.bytes = align_up(ar.used, 256);
  return w;
}

TcOperand pieces3(const bf16* base, size_t piece_elems, int64_t ld, bool mn) {
  TcOperand o;
  for (int k = 0; k < 3; ++k) o.p[k] = base + k * piece_elems;
  o.pieces = 3; o.ld = ld; o.mn = mn;
  return o;
}

GemmDesc mk(const float* A, int64_t sAm, int64_t sAk, const float* B, int64_t sBk, int64_t sBn, void* C, int64_t ldc,
            int M, int N, int K) {
  GemmDesc g;
  g.A = A; g.B = B; g.C = C; g.sAm = sAm; g.sAk = sAk; g.sBk = sBk; g.sBn = sBn; g.ldc = ldc;
  g.M = M; g.N = N; g.K = K; g.c_bf16 = 0;
  g.row_vec = g.col_vec = g.k_vec = nullptr;
  g.row_mode = g.col_mode = g.k_mode = 0;
  g.thr = kEigThr;
  g.live_rows = g.live_cols = nullptr;
  g.upper_only = 0;
  g.a_copies = g.b_copies = 1; g.a_cstride = g.b_cstride = 0; g.copy_inv = 1.f; g.a_mean_out = g.b_mean_out = nullptr;
  return g;
}

}  // namespace

// One helper stream per device (lowest priority, created on first use, kept for the life of the
// process): the optional product W = Abar Bbar depends only on the means, so it runs there beside the
// Cholesky and Jacobi kernels, which leave half of the SMs idle.
cudaStream_t side_stream() {
  static std::mutex mu;
  static cudaStream_t streams[64] = {};
  static bool tried[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (!tried[dev]) {
    tried[dev] = true;
    int lo = 0, hi = 0;
    if (cudaDeviceGetStreamPriorityRange(&lo, &hi) != cudaSuccess ||
        cudaStreamCreateWithPriority(&streams[dev], cudaStreamNonBlocking, lo) != cudaSuccess) {
      (void)cudaGetLastError();
      streams[dev] = nullptr;
    }
  }
  return streams[dev];
}

float rows_jacobi_tol(int s) { return 5e-7f * sqrtf((float)s) < 4e-6f ? 4e-6f : 5e-7f * sqrtf((float)s); }

bool rows_jacobi_fits(int count, int s) {
  if (s < 1 || s > 256 || count < 1) return false;
  if (jacobi_smem_bytes(s, s, 1) <= 227 * 1024 - 256) return true;
  const int sms = sm_count();
  return sms > 0 && (long long)count * 2 <= sms && s >= 32;
}

size_t rows_jacobi_scratch_bytes(int count) { return align_up((size_t)count * sizeof(JacobiJob), 256); }

int rows_jacobi(const float* X, float* rows, float* norms, int* status, size_t status_stride_bytes, int count, int s,
                void* scratch, cudaStream_t st) {
  std::vector<JacobiJob> jb((size_t)count);
  for (int j = 0; j < count; ++j) {
    int* stj = reinterpret_cast<int*>(reinterpret_cast<char*>(status) + (size_t)j * status_stride_bytes);
    jb[j] = JacobiJob{X + (size_t)j * s * s, rows + (size_t)j * s * s, norms + (size_t)j * s, stj, s, s};
  }
  AB_CUDA_OK(cudaMemcpyAsync(scratch, jb.data(), jb.size() * sizeof(JacobiJob), cudaMemcpyHostToDevice, st));
  return launch_jacobi(static_cast<const JacobiJob*>(scratch), count, s, rows_jacobi_tol(s), st);
}

bool sync_factored_supported(const ab_sync_desc* d, int L) {
  // dynamic shared memory of the two single-CTA kernels, with room for their few static words
  const size_t cap = 227 * 1024 - 256;
  for (int i = 0; i < L; ++i)
    if (chol_smem_bytes(d[i].r) > cap || jacobi_smem_bytes(d[i].r, d[i].r, 1) > cap) return false;
  return true;
}

size_t sync_factored_ws(const ab_sync_desc* d, int L) { return fast_layout(d, L, nullptr).bytes; }

int sync_factored(const ab_sync_desc* d, int L, int K, float sigma_cutoff, int dt, int* dev_status,
                  void* ws, size_t ws_bytes, cudaStream_t st) {
  FastWs w = fast_layout(d, L, ws);
  if (w.bytes > ws_bytes) return AB_ERR_WORKSPACE;
  const int out_bf16 = (dt == AB_BF16) ? 1 : 0;
  int rmax = 0, mmax = 0, nmax = 0;
  for (int i = 0; i < L; ++i) {
    rmax = std::max(rmax, d[i].r); mmax = std::max(mmax, d[i].m); nmax = std::max(nmax, d[i].n);
  }
  // The long products (Gram matrices, A', B', W) run on the tensor cores as six-term bf16 products when
  // every output can be stored by 16-byte rows; otherwise on the fp32 pipes.
  bool use_tc = gemm_tc_available();
  for (int i = 0; i < L && use_tc; ++i) {
    const int q = out_bf16 ? 8 : 4;
    use_tc = d[i].r % 4 == 0 && d[i].r % q == 0 && d[i].n % q == 0 && aligned(d[i].A_out, 16) && aligned(d[i].B_out, 16) &&
             (!d[i].W_out || (d[i].n % 4 == 0 && aligned(d[i].W_out, 16)));
  }
  std::vector<SplitJob> sj((size_t)4 * L);
  std::vector<TcProblem> tp_gram, tp_out, tp_w;
  int64_t split_blocks[2] = {0, 0};
  // ---- host-built tables: 9 GEMM descriptors, 2 Cholesky jobs and 1 Jacobi job per matrix, copied in one go each
  std::vector<GemmDesc> g((size_t)9 * L);
  std::vector<CholJob> cj((size_t)2 * L);
  std::vector<GemmDesc> gg;
  gg.reserve((size_t)2 * kGramMaxParts * L);
  std::vector<JacobiJob> jb((size_t)L);
  std::vector<const float*> sigp(L);
  std::vector<int*> routp(L);
  std::vector<int> rs(L);
  for (int i = 0; i < L; ++i) {
    const int m = d[i].m, n = d[i].n, r = d[i].r;
    float *Ab = w.Abar[i], *Bb = w.Bbar[i];
    // (slots 0 .. 2L of this table are unused: the Gram products G_A = Abar^T Abar and
    // G_B = Bbar Bbar^T have a table of their own, one entry per slice of the long index)
    g[0 * L + i] = mk(nullptr, 0, 0, nullptr, 0, 0, nullptr, 0, 0, 0, 0);
    g[1 * L + i] = g[0 * L + i];
    // batch 1 (L): M = R_A R_B^T
    g[2 * L + i] = mk(w.RA[i], r, 1, w.RB[i], 1, r, w.M[i], r, r, r, r);
    // batch 2 (2L): Y1 = M Vs^T ;  Z_B = diag(sqrt sig) Vs R_B^-T
    g[3 * L + i] = mk(w.M[i], r, 1, w.Vs[i], 1, r, w.Y1[i], r, r, r, r);
    GemmDesc& gzb = g[4 * L + i];
    gzb = mk(w.Vs[i], r, 1, w.IB[i], 1, r, w.ZB[i], r, r, r, r);
    gzb.row_vec = d[i].sigma; gzb.row_mode = 1;
    // batch 3 (L): Z_A = R_A^-1 Y1 diag(sig^-1/2)
    GemmDesc& gza = g[5 * L + i];
    gza = mk(w.IA[i], r, 1, w.Y1[i], r, 1, w.ZA[i], r, r, r, r);
    gza.col_vec = d[i].sigma; gza.col_mode = 2;
    // batch 4 (L): A' = Abar Z_A (columns >= r' zero);  batch 5 (L): B' = Z_B Bbar (rows >= r' zero)
    GemmDesc& ga = g[6 * L + i];
    ga = mk(Ab, r, 1, w.ZA[i], r, 1, d[i].A_out, r, m, r, r);
    ga.c_bf16 = out_bf16; ga.live_cols = d[i].r_out;
    GemmDesc& gb = g[7 * L + i];
    gb = mk(w.ZB[i], r, 1, Bb, n, 1, d[i].B_out, n, r, n, r);
    gb.c_bf16 = out_bf16; gb.live_rows = d[i].r_out;
    // batch 6 (L, optional): W = Abar Bbar
    g[8 * L + i] = mk(Ab, r, 1, Bb, n, 1, d[i].W_out, n, d[i].W_out ? m : 0, d[i].W_out ? n : 0, r);
    const int pa = use_tc ? 1 : gram_parts(m), pb = use_tc ? 1 : gram_parts(n);
    if (use_tc) {
      const int rr8 = r8(r), n8 = r8(n);
      const size_t ea = (size_t)m * rr8, eb = (size_t)r * n8, ez = (size_t)r * rr8;
      sj[2 * i] = SplitJob{Ab, r, m, r, w.Asp[i], w.Asp[i] + ea, w.Asp[i] + 2 * ea, rr8, 0};
      sj[2 * i + 1] = SplitJob{Bb, n, r, n, w.Bsp[i], w.Bsp[i] + eb, w.Bsp[i] + 2 * eb, n8, 0};
      sj[2 * L + 2 * i] = SplitJob{w.ZA[i], r, r, r, w.ZAsp[i], w.ZAsp[i] + ez, w.ZAsp[i] + 2 * ez, rr8, 0};
      sj[2 * L + 2 * i + 1] = SplitJob{w.ZB[i], r, r, r, w.ZBsp[i], w.ZBsp[i] + ez, w.ZBsp[i] + 2 * ez, rr8, 0};
      for (int h = 0; h < 2; ++h) {
        sj[2 * i + h].first_block = split_blocks[0];
        split_blocks[0] += split_job_blocks(sj[2 * i + h].rows, sj[2 * i + h].cols);
        sj[2 * L + 2 * i + h].first_block = split_blocks[1];
        split_blocks[1] += split_job_blocks(r, r);
      }
      const TcOperand A_k = pieces3(w.Asp[i], ea, rr8, false), A_t = pieces3(w.Asp[i], ea, rr8, true);
      const TcOperand B_k = pieces3(w.Bsp[i], eb, n8, false), B_t = pieces3(w.Bsp[i], eb, n8, true);
      TcProblem q;
      q.ksplit = 1; q.live_rows = q.live_cols = nullptr; q.c_f32 = true;
      // G_A = Abar^T Abar: both operands are Abar as it lies, (reduction index m) x r
      q.A = A_t; q.B = A_t; q.C = w.GA[i]; q.ldc = r; q.M = r; q.N = r; q.K = m;
      tp_gram.push_back(q);
      // G_B = Bbar Bbar^T: both operands Bbar, r x (reduction index n)
      q.A = B_k; q.B = B_k; q.C = w.GB[i]; q.ldc = r; q.M = r; q.N = r; q.K = n;
      tp_gram.push_back(q);
      // A' = Abar Z_A (columns at or beyond r' zero), B' = Z_B Bbar (rows at or beyond r' zero)
      q.c_f32 = !out_bf16;
      q.A = A_k; q.B = pieces3(w.ZAsp[i], ez, rr8, true); q.C = d[i].A_out; q.ldc = r; q.M = m; q.N = r; q.K = r;
      q.live_cols = d[i].r_out;
      tp_out.push_back(q);
      q.A = pieces3(w.ZBsp[i], ez, rr8, false); q.B = B_t; q.C = d[i].B_out; q.ldc = n; q.M = r; q.N = n; q.K = r;
      q.live_cols = nullptr; q.live_rows = d[i].r_out;
      tp_out.push_back(q);
      if (d[i].W_out) {     // W = Abar Bbar
        q.c_f32 = true; q.live_rows = nullptr;
        q.A = A_k; q.B = B_t; q.C = d[i].W_out; q.ldc = n; q.M = m; q.N = n; q.K = r;
        tp_w.push_back(q);
      }
    }
    cj[i] = CholJob{w.GA[i], pa, w.RA[i], w.IA[i], w.jstatus + 3 * i, r};
    cj[L + i] = CholJob{w.GB[i], pb, w.RB[i], w.IB[i], w.jstatus + 3 * i + 1, r};
    // Gram matrices in slices of the long index (equal work per CTA, partial sums added by the
    // Cholesky kernel in ascending slice order), upper tiles only
    for (int q = 0; q < pa && !use_tc; ++q) {
      const int k0 = gram_k0(m, pa, q), k1 = gram_k0(m, pa, q + 1);
      GemmDesc x = mk(Ab + (size_t)k0 * r, 1, r, Ab + (size_t)k0 * r, r, 1, w.GA[i] + (size_t)q * r * r, r, r, r, k1 - k0);
      x.upper_only = 1;
      gg.push_back(x);
    }
    for (int q = 0; q < pb && !use_tc; ++q) {
      const int k0 = gram_k0(n, pb, q), k1 = gram_k0(n, pb, q + 1);
      GemmDesc x = mk(Bb + k0, n, 1, Bb + k0, 1, n, w.GB[i] + (size_t)q * r * r, r, r, r, k1 - k0);
      x.upper_only = 1;
      gg.push_back(x);
    }
    jb[i] = JacobiJob{w.M[i], w.Vs[i], d[i].sigma, w.jstatus + 3 * i + 2, r, r};
    sigp[i] = d[i].sigma; routp[i] = d[i].r_out; rs[i] = r;
  }
  // All tables sit back to back in the workspace (descs ... rs): one host image, one copy.
  std::vector<AvgJob> aj((size_t)2 * L);
  int64_t avg_blocks = 0;            // flat grid of the batched mean: one 16-byte group per thread
  for (int i = 0; i < L; ++i) {
    aj[2 * i] = AvgJob{d[i].A_copies, d[i].strideA, (int64_t)d[i].m * d[i].r, w.Abar[i], 0};
    aj[2 * i + 1] = AvgJob{d[i].B_copies, d[i].strideB, (int64_t)d[i].r * d[i].n, w.Bbar[i], 0};
    for (int h = 0; h < 2; ++h) {
      aj[2 * i + h].first_block = avg_blocks;
      avg_blocks += average_job_blocks(aj[2 * i + h].count, dt);
    }
  }
  {
    char* base = reinterpret_cast<char*>(w.descs);
    const size_t span = (size_t)(reinterpret_cast<char*>(w.sjobs + 4 * L) - base);
    std::vector<char> img(span, 0);
    auto put = [&](const void* dev_ptr, const void* src, size_t bytes) {
      std::memcpy(img.data() + (reinterpret_cast<const char*>(dev_ptr) - base), src, bytes);
    };
    put(w.descs, g.data(), g.size() * sizeof(GemmDesc));
    put(w.gram_descs, gg.data(), gg.size() * sizeof(GemmDesc));
    put(w.cjobs, cj.data(), cj.size() * sizeof(CholJob));
    put(w.ajobs, aj.data(), aj.size() * sizeof(AvgJob));
    put(w.jobs, jb.data(), jb.size() * sizeof(JacobiJob));
    put(w.sig_ptrs, sigp.data(), L * sizeof(float*));
    put(w.rout_ptrs, routp.data(), L * sizeof(int*));
    put(w.rs, rs.data(), L * sizeof(int));
    put(w.sjobs, sj.data(), sj.size() * sizeof(SplitJob));
    AB_CUDA_OK(cudaMemcpyAsync(base, img.data(), span, cudaMemcpyHostToDevice, st));
  }

  // ---- a7: means of the K copies (fp32), all matrices in one launch
  AB_TRY(group_average_batched(w.ajobs, 2 * L, K, dt, avg_blocks, st));
  const float tol = rows_jacobi_tol(rmax);
  bool any_w = false;
  for (int i = 0; i < L; ++i) any_w = any_w || d[i].W_out != nullptr;
  // a8 (optional): forked off where the Jacobi kernel starts (the kernels before it fill every SM
  // themselves), joined at the end
  cudaStream_t side = any_w ? side_stream() : nullptr;
  // the two events live for this call only; every return below destroys them (destroying an event that
  // has been recorded releases it once the recorded work is done)
  struct EventPair {
    cudaEvent_t fork = nullptr, join = nullptr;
    bool create() {
      if (cudaEventCreateWithFlags(&fork, cudaEventDisableTiming) == cudaSuccess &&
          cudaEventCreateWithFlags(&join, cudaEventDisableTiming) == cudaSuccess)
        return true;
      (void)cudaGetLastError();
      return false;
    }
    ~EventPair() {
      if (fork) cudaEventDestroy(fork);
      if (join) cudaEventDestroy(join);
    }
  } evs;
  if (side && !evs.create()) side = nullptr;
  cudaEvent_t fork = evs.fork, join = evs.join;
  auto product_w = [&](cudaStream_t s2) -> int {
    if (use_tc) return gemm_tc_batched(tp_w.data(), (int)tp_w.size(), w.tc_table[2], w.tc_status + 2, s2);
    return gemm_simt_batched(w.descs + 8 * L, L, mmax, nmax, s2);
  };
  if (use_tc) {
    AB_CUDA_OK(cudaMemsetAsync(w.tc_status, 0, 4 * sizeof(int), st));
    AB_TRY(split3_batched(w.sjobs, 2 * L, split_blocks[0], st));                            // pieces of Abar, Bbar
  }
  if (any_w && !side) AB_TRY(product_w(st));
  if (use_tc) AB_TRY(gemm_tc_batched(tp_gram.data(), (int)tp_gram.size(), w.tc_table[0], w.tc_status, st));
  else AB_TRY(gemm_simt_batched(w.gram_descs, (int)gg.size(), rmax, rmax, st));             // Gram slices
  const size_t csm = chol_smem_bytes(rmax);
  AB_CUDA_OK(cudaFuncSetAttribute(chol_inv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)csm));
  chol_inv_kernel<<<2 * L, kCThreads, csm, st>>>(w.cjobs);                                  // R_A, R_B and inverses
  AB_LAUNCH_OK();
  AB_TRY(gemm_simt_batched(w.descs + 2 * L, L, rmax, rmax, st));                            // M
  int side_rc = AB_OK;
  if (side && cudaEventRecord(fork, st) != cudaSuccess) side_rc = AB_ERR_CUDA;
  AB_TRY(launch_jacobi(w.jobs, L, rmax, tol, st));                                    // SVD of M
  if (side) {
    if (side_rc == AB_OK && cudaStreamWaitEvent(side, fork, 0) != cudaSuccess) side_rc = AB_ERR_CUDA;
    if (side_rc == AB_OK) side_rc = product_w(side);
    if (side_rc == AB_OK && cudaEventRecord(join, side) != cudaSuccess) side_rc = AB_ERR_CUDA;
  }
  fast_rank_rule_kernel<<<(L + 127) / 128, 128, 0, st>>>(w.sig_ptrs, w.rs, sigma_cutoff, w.rout_ptrs, w.jstatus,
                                                         dev_status, L);
  AB_LAUNCH_OK();
  AB_TRY(gemm_simt_batched(w.descs + 3 * L, 2 * L, rmax, rmax, st));                        // Y1, Z_B
  AB_TRY(gemm_simt_batched(w.descs + 5 * L, L, rmax, rmax, st));                            // Z_A
  if (use_tc) {
    AB_TRY(split3_batched(w.sjobs + 2 * L, 2 * L, split_blocks[1], st));                    // pieces of Z_A, Z_B
    AB_TRY(gemm_tc_batched(tp_out.data(), (int)tp_out.size(), w.tc_table[1], w.tc_status + 1, st));   // A', B'
  } else {
    AB_TRY(gemm_simt_batched(w.descs + 6 * L, L, mmax, rmax, st));                          // A'
    AB_TRY(gemm_simt_batched(w.descs + 7 * L, L, rmax, nmax, st));                          // B'
  }
  if (side) {
    if (side_rc == AB_OK && cudaStreamWaitEvent(st, join, 0) != cudaSuccess) side_rc = AB_ERR_CUDA;
    if (side_rc != AB_OK) { (void)cudaGetLastError(); return side_rc; }
  }
  if (use_tc && dev_status) {
    fold_tc_status_kernel<<<1, 128, 0, st>>>(w.tc_status, dev_status, L);
    AB_LAUNCH_OK();
  }
  return AB_OK;
}
}  // namespace ab
