// Truncated SVD and sqrt-sigma split (Eq. 3 with the rank rule), batched over matrices.
//
// Route: Gram matrix of the shorter side, G = W^T W (m >= n) or W W^T (m < n) -- the paper's
// "transpose when n > m" is this choice of side -- then a block one-sided Jacobi eigensolve on
// X = G with the rotations accumulated in V^T, all in fp32:
//   * vectors are stored as ROWS (X is s x s, V^T is s x s), split into blocks of b rows;
//   * a sweep is nb-1 rounds of disjoint block pairs (round-robin); one CTA per pair keeps the
//     2b x s panel in shared memory (b = 16), forms its 32 x 32 Gram matrix M, runs a few
//     sweeps of a two-sided cyclic Jacobi on M in shared memory (accumulating Q),
//     applies Q^T to the panel and to the matching panel of V^T;
//   * sweeps repeat until no pair of rows has |x_i.x_j| > tol |x_i||x_j| (a device flag; the
//     host enqueues a fixed number of sweeps and converged matrices return at once).
// At convergence the rows of V^T are eigenvectors of G (singular vectors of the short side)
// and |x_i| = sigma_i^2.  The long-side factor is W V_r (or V_r^T W) by a GEMM; sigma_i is
// re-measured as the norm of that product, which makes A^T A = B B^T = diag(sigma) hold by
// construction.  No wait in these kernels can spin: every loop has a fixed trip count.
#include <vector>
#include <algorithm>
#include <map>

#include <cooperative_groups.h>

#include "ab_common.cuh"

namespace ab {
namespace {

struct JState {
  int done;            // 1 once converged (or sweep cap reached)
  unsigned off_bits;   // max relative off-orthogonality seen in the running sweep (float bits)
  int sweeps;
  unsigned maxn2_bits;      // largest squared row norm of the previous sweep (float bits)
  unsigned next_maxn2_bits; // the same, being collected in the running sweep
  int status;
  float off_hist[26];       // off-orthogonality after each sweep (diagnostics)
};

constexpr int kMaxSweeps = 30;
constexpr int kInnerSweeps = 1;
constexpr float kCountRel2 = 1e-8f;  // rows below 1e-4 of the largest norm do not hold up convergence
constexpr float kDeadRel2 = 1e-12f;   // rows below 1e-6 of the largest norm count as zero
// Accuracy domain of this route: a kept singular value between kZeroRel and kDomainRel of the largest has lost
// relative accuracy to the squaring in the Gram matrix (measured: 2e-7 above 2 %, up to 1.3e-4 at 1-2 %, 5e-3 at
// 0.5-1 %); the status word then says so.  Below kZeroRel a value is zero to working precision (a W of lower rank than asked for).
constexpr float kDomainRel = 2e-2f, kZeroRel = 1e-5f;

// Rows count as orthogonal when |x_i.x_j| <= tol |x_i||x_j|.  An fp32 dot product of length s
// carries rounding noise of about 6e-8 sqrt(s) relative to |x_i||x_j|; the maximum over all
// pairs sits a few times above that, so tol is placed at eight times the noise.
__host__ __device__ inline float jacobi_tol(int s) {
  float t = 5e-7f * sqrtf((float)s);
  return t < 4e-6f ? 4e-6f : t;
}

__global__ void init_state_kernel(float* __restrict__ Vt, JState* __restrict__ st, int s, int count) {
  const int mat = blockIdx.y;
  float* V = Vt + (size_t)mat * s * s;
  const size_t total = (size_t)s * s;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x)
    V[i] = (i / s == i % s) ? 1.f : 0.f;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    JState z;
    z.done = 0; z.off_bits = 0; z.sweeps = 0; z.maxn2_bits = 0; z.next_maxn2_bits = 0; z.status = AB_OK;
    for (int i = 0; i < 26; ++i) z.off_hist[i] = 0.f;
    st[mat] = z;
  }
}

__global__ void sweep_end_kernel(JState* __restrict__ st, int count, float tol) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  JState z = st[i];
  if (z.done) return;
  if (z.sweeps < 26) z.off_hist[z.sweeps] = __uint_as_float(z.off_bits);
  z.sweeps += 1;
  if (__uint_as_float(z.off_bits) <= tol) z.done = 1;
  else if (z.sweeps >= kMaxSweeps) { z.done = 1; z.status = AB_ERR_NOT_CONVERGED; }
  z.off_bits = 0;
  if (z.next_maxn2_bits) z.maxn2_bits = z.next_maxn2_bits;
  z.next_maxn2_bits = 0;
  st[i] = z;
}

// Index pair k of round t in a round-robin over an even number `ne` of players.
__device__ __forceinline__ void rr_pair(int ne, int t, int k, int& p, int& q) {
  const int n1 = ne - 1;
  if (k == 0) { p = n1; q = t % n1; }
  else { p = (t + k) % n1; q = (t - k + n1) % n1; }
  if (p > q) { int tmp = p; p = q; q = tmp; }
}

// ---- 32 x 32 symmetric eigenproblem of a panel ---------------------------------------------------
// Two-sided cyclic Jacobi: 31 steps of 16 disjoint pairs (round-robin tournament) cover every pair once.
// Solved by the whole CTA (256 threads) in shared memory, two barriers and a few dozen instructions per thread
// and step; an earlier version that kept the matrix
// in one warp's registers and moved columns by shuffles took a few hundred dependent shuffles per step
// (measured on the 3072 x 768 split: 118 us per round of the block Jacobi with it).
// Ms: the symmetric matrix (leading dimension ldm), Qs: receives Q (identity on entry is set here).
// Rotation that annihilates M[p][q].  Approximate reciprocal and square-root units are enough here: an error in
// c scales both rotated vectors alike (their orthogonality is untouched, and the singular vectors are
// normalised at the end), an error in t leaves a residue of second order that the next sweep removes.
__device__ __forceinline__ void jacobi_rotation(const float* Ms, int ldm, int pp, int qq, float thr, float dead2,
                                                float& c, float& sn) {
  const float app = Ms[pp * ldm + pp], aqq = Ms[qq * ldm + qq], g = Ms[pp * ldm + qq];
  c = 1.f; sn = 0.f;
  if (app > dead2 && aqq > dead2 && app > 0.f && aqq > 0.f && g * g > thr * thr * app * aqq) {
    float zeta = __fdividef(aqq - app, 2.f * g);
    zeta = fminf(fmaxf(zeta, -1e15f), 1e15f);
    const float h = fmaf(zeta, zeta, 1.f);
    const float t = __fdividef(copysignf(1.f, zeta), fabsf(zeta) + h * rsqrtf(h));
    c = rsqrtf(fmaf(t, t, 1.f));
    sn = c * t;
  }
}

// Thread (k, k2) of the 16 x 16 grid owns the 2 x 2 block of M at the rows of pair k and the columns of pair k2.
// Per step: 16 threads work out the 16 rotations (the pairs of all 31 steps come from a table built once); after
// a barrier every thread reads its block, applies J_k^T B J_k2 and writes it back (the blocks of a step are
// disjoint), and carries two rows of Q through the column rotation of pair k2; a second barrier ends the step.
struct EigScratch {
  unsigned char pp[31 * 16], qq[31 * 16];
  float c[16], s[16];
  int flag;
};
__device__ __forceinline__ void cta_eig32(float* Ms, float* Qs, int ldm, float thr, float dead2, int max_sweeps, EigScratch* es) {
  const int tid = threadIdx.x;
  const int k = tid >> 4, k2 = tid & 15;
  for (int idx = tid; idx < 32 * 32; idx += 256) Qs[(idx >> 5) * ldm + (idx & 31)] = ((idx >> 5) == (idx & 31)) ? 1.f : 0.f;
  for (int idx = tid; idx < 31 * 16; idx += 256) {
    int a, b;
    rr_pair(32, idx >> 4, idx & 15, a, b);
    es->pp[idx] = (unsigned char)a; es->qq[idx] = (unsigned char)b;
  }
  __syncthreads();
  for (int sweep = 0; sweep < max_sweeps; ++sweep) {
    if (tid == 0) es->flag = 0;
    __syncthreads();
    for (int step = 0; step < 31; ++step) {
      if (tid < 16) {
        float c, sn;
        jacobi_rotation(Ms, ldm, es->pp[step * 16 + tid], es->qq[step * 16 + tid], thr, dead2, c, sn);
        es->c[tid] = c; es->s[tid] = sn;
        if (sn != 0.f) es->flag = 1;
      }
      __syncthreads();
      const float c1 = es->c[k], s1 = es->s[k], c2 = es->c[k2], s2 = es->s[k2];
      const int p1 = es->pp[step * 16 + k], q1 = es->qq[step * 16 + k], p2 = es->pp[step * 16 + k2], q2 = es->qq[step * 16 + k2];
      if (s1 != 0.f || s2 != 0.f) {
        const float b00 = Ms[p1 * ldm + p2], b01 = Ms[p1 * ldm + q2], b10 = Ms[q1 * ldm + p2], b11 = Ms[q1 * ldm + q2];
        // rows (pair k), then columns (pair k2)
        const float r00 = c1 * b00 - s1 * b10, r10 = s1 * b00 + c1 * b10;
        const float r01 = c1 * b01 - s1 * b11, r11 = s1 * b01 + c1 * b11;
        Ms[p1 * ldm + p2] = c2 * r00 - s2 * r01; Ms[p1 * ldm + q2] = s2 * r00 + c2 * r01;
        Ms[q1 * ldm + p2] = c2 * r10 - s2 * r11; Ms[q1 * ldm + q2] = s2 * r10 + c2 * r11;
      }
      if (s2 != 0.f) {
        const int i0 = k, i1 = k + 16;                // the two rows of Q this thread rotates (columns p2, q2)
        const float qa0 = Qs[i0 * ldm + p2], qb0 = Qs[i0 * ldm + q2], qa1 = Qs[i1 * ldm + p2], qb1 = Qs[i1 * ldm + q2];
        Qs[i0 * ldm + p2] = c2 * qa0 - s2 * qb0; Qs[i0 * ldm + q2] = s2 * qa0 + c2 * qb0;
        Qs[i1 * ldm + p2] = c2 * qa1 - s2 * qb1; Qs[i1 * ldm + q2] = s2 * qa1 + c2 * qb1;
      }
      __syncthreads();
    }
    if (!es->flag) break;
  }
}

// One cluster of kCl CTAs (8, or 1 when a batch already fills the device) per block pair: PB = 32 rows (16 + 16)
// or PB = 16 (8 + 8).  A panel is only PB rows, so
// one CTA per pair would leave most of the device idle (24 CTAs for a 768 x 768 matrix: 116 us per round); the
// columns of the panel are cut into kCl slices instead, one per CTA of the cluster.  Each CTA forms the Gram matrix
// of its slice; the partial matrices are added through distributed shared memory in ascending CTA order, so every
// CTA of the cluster holds the same M to the bit, solves the same small eigenproblem and rotates its own slice of
// the X panel and of the V^T panel.  No wait spins: the only waits are cluster barriers that every CTA of the
// cluster reaches (all early exits depend on values the whole cluster agrees on).
template <int PB, int kCl>
__global__ void __launch_bounds__(256, 2)
jacobi_pair_kernel(float* __restrict__ Xall, float* __restrict__ Vall, int s, int nb, int round,
                   float tol, JState* __restrict__ states) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  constexpr int HB = PB / 2;          // rows per block
  constexpr int LDM = 33;
  constexpr int LDQ = PB + 4;
  extern __shared__ __align__(16) float smem[];
  const int mat = blockIdx.y;
  const int pair = blockIdx.x / kCl, crank = blockIdx.x % kCl;
  JState* st = states + mat;
  if (st->done) return;               // the same for the whole cluster
  const int nbe = nb + (nb & 1);
  int bi, bj;
  rr_pair(nbe, round, pair, bi, bj);
  if (bj >= nb && nb > 1) return;     // this block sits the round out (whole cluster)
  // this CTA's slice of the columns: multiples of 4, as equal as they come
  const int s4 = (s + 3) >> 2;
  const int c_lo = (int)((long long)crank * s4 / kCl) * 4;
  int c_hi = (int)((long long)(crank + 1) * s4 / kCl) * 4;
  if (c_hi > s) c_hi = s;
  const int w = c_hi > c_lo ? c_hi - c_lo : 0;     // width of the slice
  const int ldp = (((s4 + kCl - 1) / kCl) * 4) + 4;  // the same in every CTA
  float* P = smem;                    // PB x ldp
  float* Mp = P + (size_t)PB * ldp;   // 32 x LDM: this CTA's partial Gram matrix (zero beyond PB)
  float* Ms = Mp + 32 * LDM;          // 32 x LDM: the sum
  float* Qs = Ms + 32 * LDM;          // 32 x LDM
  float* Qt = Qs + 32 * LDM + 1;      // PB x LDQ, Qt[c][i] = Q[i][c]; realigned below
  Qt = reinterpret_cast<float*>((reinterpret_cast<uintptr_t>(Qt) + 15) & ~(uintptr_t)15);
  __shared__ int any_rot;
  __shared__ EigScratch eig_scratch;
  const int tid = threadIdx.x;
  float* X = Xall + (size_t)mat * s * s;
  float* V = Vall + (size_t)mat * s * s;
  const float maxn2 = __uint_as_float(st->maxn2_bits);
  const float dead2 = kDeadRel2 * maxn2;
  const float count2 = kCountRel2 * maxn2;

  auto grow = [&](int lr) -> int {    // local panel row -> global row (or -1)
    int g = (lr < HB) ? bi * HB + lr : bj * HB + (lr - HB);
    if (lr >= HB && bj >= nb) return -1;
    return g < s ? g : -1;
  };
  auto load_panel = [&](const float* src) {
    for (int lr = tid >> 5; lr < PB; lr += 8) {      // a warp per row: coalesced
      const int g = grow(lr);
      for (int k = tid & 31; k < ldp - 4; k += 32)
        P[(size_t)lr * ldp + k] = (g >= 0 && k < w) ? src[(size_t)g * s + c_lo + k] : 0.f;
    }
  };
  auto store_panel = [&](float* dst) {
    for (int lr = tid >> 5; lr < PB; lr += 8) {
      const int g = grow(lr);
      if (g < 0) continue;
      for (int k = tid & 31; k < w; k += 32) dst[(size_t)g * s + c_lo + k] = P[(size_t)lr * ldp + k];
    }
  };
  auto apply_q = [&]() {              // P <- Q^T P, one panel column per thread at a time
    for (int k = tid; k < w; k += 256) {
      float col[PB];
#pragma unroll
      for (int j = 0; j < PB; ++j) col[j] = P[(size_t)j * ldp + k];
#pragma unroll 4
      for (int i = 0; i < PB; ++i) {
        const float4* qrow = reinterpret_cast<const float4*>(Qt + i * LDQ);
        float acc = 0.f;
#pragma unroll
        for (int j4 = 0; j4 < PB / 4; ++j4) {
          float4 q4 = qrow[j4];
          acc = fmaf(q4.x, col[4 * j4], acc);
          acc = fmaf(q4.y, col[4 * j4 + 1], acc);
          acc = fmaf(q4.z, col[4 * j4 + 2], acc);
          acc = fmaf(q4.w, col[4 * j4 + 3], acc);
        }
        P[(size_t)i * ldp + k] = acc;
      }
    }
  };

  load_panel(X);
  for (int idx = tid; idx < 32 * LDM; idx += 256) Mp[idx] = 0.f;
  if (tid == 0) any_rot = 0;
  __syncthreads();

  // ---- partial Gram matrix of this slice: entry (i, j) by thread i * PB + j (and + 256 ...), k ascending
  for (int e = tid; e < PB * PB; e += 256) {
    const int i = e / PB, jj = e - i * PB;
    if (jj < i) continue;             // symmetric: the upper triangle is computed, the lower mirrored
    const float4* a = reinterpret_cast<const float4*>(P + (size_t)i * ldp);
    const float4* b = reinterpret_cast<const float4*>(P + (size_t)jj * ldp);
    float acc = 0.f;
    for (int k = 0; k < (ldp - 4) / 4; ++k) {
      const float4 x = a[k], y = b[k];
      acc = fmaf(x.x, y.x, acc); acc = fmaf(x.y, y.y, acc); acc = fmaf(x.z, y.z, acc); acc = fmaf(x.w, y.w, acc);
    }
    Mp[i * LDM + jj] = acc;
    Mp[jj * LDM + i] = acc;
  }
  if constexpr (kCl > 1) cluster.sync(); else __syncthreads();     // every CTA's partial matrix is complete
  for (int idx = tid; idx < 32 * LDM; idx += 256) {
    float acc = 0.f;
    if constexpr (kCl > 1) {
#pragma unroll
      for (int c = 0; c < kCl; ++c) acc += cluster.map_shared_rank(Mp, c)[idx];   // ascending CTA order in every CTA
    } else {
      acc = Mp[idx];
    }
    Ms[idx] = acc;
  }
  if constexpr (kCl > 1) cluster.sync(); else __syncthreads();     // nobody reads a peer's partial matrix after this

  // ---- how far from orthogonal is this panel?  (also collects the largest squared norm)
  {
    float worst = 0.f, big = 0.f;
    int rot = 0;
    for (int idx = tid; idx < PB * PB; idx += 256) {
      int i = idx / PB, jj = idx - i * PB;
      float mii = Ms[i * LDM + i], mjj = Ms[jj * LDM + jj];
      if (i == jj) { big = fmaxf(big, mii); continue; }
      if (i < jj && mii > dead2 && mjj > dead2 && mii > 0.f && mjj > 0.f) {
        float rel = fabsf(Ms[i * LDM + jj]) / (sqrtf(mii) * sqrtf(mjj));
        if (rel > tol) rot = 1;
        // rows far below the largest norm are rounding noise of the large ones: they are still
        // rotated, but the sweep counts as converged without them
        if (mii > count2 && mjj > count2) worst = fmaxf(worst, rel);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      worst = fmaxf(worst, __shfl_xor_sync(0xffffffffu, worst, o));
      big = fmaxf(big, __shfl_xor_sync(0xffffffffu, big, o));
    }
    if ((tid & 31) == 0 && crank == 0) {
      atomicMax(&st->off_bits, __float_as_uint(worst));
      atomicMax(&st->next_maxn2_bits, __float_as_uint(big));
    }
    if (rot) atomicExch(&any_rot, 1);
  }
  __syncthreads();
  if (!any_rot) return;               // panel already orthogonal: nothing to write (the same M in every CTA)

  // ---- diagonalise M (all threads; the same arithmetic in every CTA of the cluster), then Qt[c][i] = Q[i][c]
  cta_eig32(Ms, Qs, LDM, 0.25f * tol, dead2, kInnerSweeps, &eig_scratch);
  for (int idx = tid; idx < PB * PB; idx += 256) {
    const int c = idx / PB, i = idx - c * PB;
    Qt[c * LDQ + i] = Qs[i * LDM + c];
  }
  __syncthreads();

  // ---- rotate this slice of the panel of X, then of the same rows of V^T
  apply_q();
  __syncthreads();
  store_panel(X);
  __syncthreads();
  load_panel(V);
  __syncthreads();
  apply_q();
  __syncthreads();
  store_panel(V);
}

template <int PB, int kCl>
size_t jacobi_smem_bytes(int s) {
  const int s4 = (s + 3) >> 2;
  const int ldp = (((s4 + kCl - 1) / kCl) * 4) + 4;
  return sizeof(float) * ((size_t)PB * ldp + 3 * 32 * 33 + 8 + (size_t)PB * (PB + 4));
}

// lam[i] = |row i of X|, perm = indices by descending lam (ties by index).  One CTA per matrix.
__global__ void __launch_bounds__(256)
norms_sort_kernel(const float* __restrict__ Xall, int s, float* __restrict__ lam_all, int* __restrict__ perm_all) {
  extern __shared__ float lam_s[];
  const int mat = blockIdx.x;
  const float* X = Xall + (size_t)mat * s * s;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i = warp; i < s; i += 8) {
    double acc = 0.0;
    for (int k = lane; k < s; k += 32) { float v = X[(size_t)i * s + k]; acc += (double)v * v; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) lam_s[i] = (float)sqrt(acc);
  }
  __syncthreads();
  for (int i = threadIdx.x; i < s; i += 256) {
    float li = lam_s[i];
    int rank = 0;
    for (int j = 0; j < s; ++j) {
      float lj = lam_s[j];
      rank += (lj > li) || (lj == li && j < i);
    }
    perm_all[(size_t)mat * s + rank] = i;
    lam_all[(size_t)mat * s + i] = li;
  }
}

// After the in-shared-memory solver: rows (unit length, sorted by descending lam) whose lam is below
// 1e-4 of the largest carry directions of rounding noise, not eigenvectors.  Each of them is made
// orthogonal to every row before it (Gram-Schmidt, two passes) and rescaled, so that the rows stay an
// orthonormal set and W v picks up nothing of the resolved directions; a row that does not survive the
// projection becomes zero (it then contributes nothing to either factor).  Only the first r_need rows
// are ever used.  One CTA per matrix.
__global__ void __launch_bounds__(256)
complete_basis_kernel(float* __restrict__ rows_all, const float* __restrict__ lam_all, int s, int r_need) {
  extern __shared__ float cb_sm[];
  float* v = cb_sm;            // s
  float* coef = cb_sm + s;     // s
  __shared__ float red[8];
  __shared__ int k_first;
  float* rows = rows_all + (size_t)blockIdx.x * s * s;
  const float* lam = lam_all + (size_t)blockIdx.x * s;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    int k = 0;
    const float thr = 1e-4f * lam[0];
    while (k < s && lam[k] >= thr && lam[k] > 0.f) ++k;
    k_first = k;
  }
  __syncthreads();
  const int k_end = r_need < s ? r_need : s;
  for (int k = k_first; k < k_end; ++k) {
    for (int u = tid; u < s; u += 256) v[u] = rows[(size_t)k * s + u];
    __syncthreads();
    for (int pass = 0; pass < 2; ++pass) {
      for (int j = warp; j < k; j += 8) {
        float a = 0.f;
        for (int u = lane; u < s; u += 32) a = fmaf(rows[(size_t)j * s + u], v[u], a);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        if (lane == 0) coef[j] = a;
      }
      __syncthreads();
      for (int u = tid; u < s; u += 256) {
        float a = v[u];
        for (int j = 0; j < k; ++j) a = fmaf(-coef[j], rows[(size_t)j * s + u], a);
        v[u] = a;
      }
      __syncthreads();
    }
    float a = 0.f;
    for (int u = tid; u < s; u += 256) a = fmaf(v[u], v[u], a);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
    if (lane == 0) red[warp] = a;
    __syncthreads();
    float n2 = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) n2 += red[i];
    const float inv = n2 > 1e-6f ? rsqrtf(n2) : 0.f;       // the row started at unit length (or zero)
    for (int u = tid; u < s; u += 256) rows[(size_t)k * s + u] = v[u] * inv;
    __syncthreads();                                         // the next row reads this one from global memory
  }
}

__global__ void identity_perm_kernel(int* __restrict__ perm, int s, int total) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < total) perm[i] = i % s;
}

// Vr[k][:] = Vt[perm[k]][:] scaled to unit length, k < r_cap (thousands of fp32 rotations leave
// the rows orthogonal but let their norms wander by ~1e-6)
__global__ void __launch_bounds__(256)
gather_rows_kernel(const float* __restrict__ Vt, const int* __restrict__ perm, int s, int r_cap,
                   float* __restrict__ Vr) {
  __shared__ double red[8];
  const int k = blockIdx.x;
  if (k >= r_cap) return;
  const float* src = Vt + (size_t)perm[k] * s;
  double acc = 0.0;
  for (int u = threadIdx.x; u < s; u += 256) { float v = src[u]; acc += (double)v * v; }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
  __syncthreads();
  double tot = 0.0;
#pragma unroll
  for (int i = 0; i < 8; ++i) tot += red[i];
  const float inv = tot > 0.0 ? (float)(1.0 / sqrt(tot)) : 0.f;
  for (int u = threadIdx.x; u < s; u += 256) Vr[(size_t)k * s + u] = src[u] * inv;
}

// sigma[k] = norm over t of Ylong(k,t), Ylong(k,t) = Y[t*st_ + k*sk].  32 values of k per CTA.
__global__ void __launch_bounds__(256)
long_norms_kernel(const float* __restrict__ Y, int64_t st_, int64_t sk, int L, int r_cap, float* __restrict__ sigma) {
  __shared__ double red[8][33];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (sk == 1) {                      // neighbouring k adjacent in memory: lane = k, warps stride over t
    const int k = blockIdx.x * 32 + lane;
    double acc = 0.0;
    if (k < r_cap)
      for (int t = warp; t < L; t += 8) { float v = Y[(int64_t)t * st_ + k]; acc += (double)v * v; }
    red[warp][lane] = acc;
    __syncthreads();
    if (warp == 0 && k < r_cap) {
      double t = 0.0;
#pragma unroll
      for (int i = 0; i < 8; ++i) t += red[i][lane];
      sigma[k] = (float)sqrt(t);
    }
  } else {                            // neighbouring t adjacent: one warp walks one k
    for (int kk = warp; kk < 32; kk += 8) {
      const int k = blockIdx.x * 32 + kk;
      if (k >= r_cap) continue;
      double acc = 0.0;
      for (int t = lane; t < L; t += 32) { float v = Y[(int64_t)t * st_ + (int64_t)k * sk]; acc += (double)v * v; }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
      if (lane == 0) sigma[k] = (float)sqrt(acc);
    }
  }
}

__global__ void rank_rule_kernel(const float* __restrict__ sigma, int r_cap, float cutoff, int* __restrict__ r_out,
                                 const JState* __restrict__ st, int* __restrict__ dev_status) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  float top = 0.f;
  for (int k = 0; k < r_cap; ++k) top = fmaxf(top, sigma[k]);
  const float thr = cutoff * top;
  int keep = 0;
  for (int k = 0; k < r_cap; ++k) keep += (sigma[k] >= thr) ? 1 : 0;
  if (keep < 1) keep = 1;
  *r_out = keep;
  if (dev_status) {
    int code = st->status;
    if (code == AB_OK)
      for (int k = 0; k < keep; ++k)
        if (sigma[k] < kDomainRel * top && sigma[k] > kZeroRel * top) code = AB_ERR_ACCURACY;
    *dev_status = code;
  }
}

// long factor: F(t,k) = Ylong(k,t) / sqrt(sigma_k); short factor: F(k,u) = sqrt(sigma_k) Vr[k][u].
// Columns/rows k >= r' (and k >= r_cap) are written as zero.
template <typename TO>
__global__ void write_factors_kernel(const float* __restrict__ Y, int64_t yt, int64_t yk,
                                     const float* __restrict__ Vr, const float* __restrict__ sigma,
                                     const int* __restrict__ r_out, int L, int s, int r_cap, int r_max,
                                     TO* __restrict__ Flong, int64_t lt, int64_t lk,
                                     TO* __restrict__ Fshort, int64_t sk_, int64_t su) {
  const int rk = *r_out;
  const int64_t nlong = (int64_t)L * r_max, nshort = (int64_t)s * r_max;
  const int64_t step = (int64_t)gridDim.x * blockDim.x;
  for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < nlong + nshort; idx += step) {
    if (idx < nlong) {
      // walk the long factor in its own memory order
      int64_t t, k;
      if (lk == 1) { t = idx / r_max; k = idx - t * r_max; } else { k = idx / L; t = idx - k * L; }
      float v = 0.f;
      if (k < rk && k < r_cap) {
        float sg = sigma[k];
        v = sg > 0.f ? Y[t * yt + k * yk] * rsqrtf(sg) : 0.f;
      }
      from_f32(Flong[t * lt + k * lk], v);
    } else {
      int64_t j = idx - nlong, k, u;
      if (su == 1) { k = j / s; u = j - k * s; } else { u = j / r_max; k = j - u * r_max; }
      float v = 0.f;
      if (k < rk && k < r_cap) v = sqrtf(sigma[k]) * Vr[k * (int64_t)s + u];
      from_f32(Fshort[k * sk_ + u * su], v);
    }
  }
}

struct Plan {
  int s, L, r_cap, pb, nb;
  bool tall;           // m >= n
};

Plan make_plan(const SvdItem& it) {
  Plan p;
  p.tall = it.m >= it.n;
  p.s = p.tall ? it.n : it.m;
  p.L = p.tall ? it.m : it.n;
  p.r_cap = std::min(it.r_max, p.s);
  p.pb = p.s <= 1536 ? 32 : 16;
  int hb = p.pb / 2;
  p.nb = (p.s + hb - 1) / hb;
  return p;
}

struct ItemWs {
  float *lam, *Vr, *Y, *Wf;
  int* perm;
};

// Lays out the workspace: per group (equal s) X, Vt and states; per item the rest.
struct Layout {
  std::map<int, std::vector<int>> groups;     // s -> item indices
  std::map<int, float*> X, Vt;
  std::map<int, JState*> st;
  std::map<int, void*> jobs;                  // scratch of the in-shared-memory solver
  std::vector<ItemWs> item;
  size_t bytes;
};

Layout make_layout(const SvdItem* items, int L, void* ws) {
  Layout lo;
  Arena ar(ws, 0);
  for (int i = 0; i < L; ++i) lo.groups[make_plan(items[i]).s].push_back(i);
  for (auto& g : lo.groups) {
    size_t s = (size_t)g.first, cnt = g.second.size();
    lo.X[g.first] = ar.take_n<float>(cnt * s * s);
    lo.Vt[g.first] = ar.take_n<float>(cnt * s * s);
    lo.st[g.first] = ar.take_n<JState>(cnt);
    lo.jobs[g.first] = ar.take_n<char>(rows_jacobi_scratch_bytes((int)cnt));
  }
  lo.item.resize(L);
  for (int i = 0; i < L; ++i) {
    Plan p = make_plan(items[i]);
    lo.item[i].lam = nullptr;
    lo.item[i].perm = nullptr;
    lo.item[i].Vr = ar.take_n<float>((size_t)p.r_cap * p.s);
    lo.item[i].Y = ar.take_n<float>((size_t)p.L * p.r_cap);
    lo.item[i].Wf = nullptr;
  }
  for (auto& g : lo.groups) {   // lam/perm are group-contiguous (one sort launch per group)
    size_t s = (size_t)g.first, cnt = g.second.size();
    float* lam = ar.take_n<float>(cnt * s);
    int* perm = ar.take_n<int>(cnt * s);
    for (size_t j = 0; j < cnt; ++j) {
      lo.item[g.second[j]].lam = lam ? lam + j * s : nullptr;
      lo.item[g.second[j]].perm = perm ? perm + j * s : nullptr;
    }
  }
  lo.bytes = align_up(ar.used, 256);
  return lo;
}

template <int PB, int CL>
int run_jacobi_cl(float* X, float* Vt, JState* st, int s, int nb, int count, cudaStream_t stream) {
  const size_t smem = jacobi_smem_bytes<PB, CL>(s);
  if (smem > 227 * 1024) return AB_ERR_UNSUPPORTED;
  AB_CUDA_OK(cudaFuncSetAttribute(jacobi_pair_kernel<PB, CL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  const int nbe = nb + (nb & 1);
  const int rounds = nbe > 2 ? nbe - 1 : 1;
  const float tol = jacobi_tol(s);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(nbe / 2) * CL, (unsigned)count);
  cfg.blockDim = dim3(256);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CL; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  for (int sw = 0; sw < kMaxSweeps; ++sw) {
    for (int r = 0; r < rounds; ++r) {
      AB_CUDA_OK(cudaLaunchKernelEx(&cfg, jacobi_pair_kernel<PB, CL>, X, Vt, s, nb, r, tol, st));
    }
    sweep_end_kernel<<<(count + 127) / 128, 128, 0, stream>>>(st, count, tol);
  }
  count_launches((long long)kMaxSweeps * (rounds + 1) - 1);
  AB_LAUNCH_OK();
  return AB_OK;
}

// Clusters of 8 CTAs per block pair while that leaves the device room for every pair of a round (a lone matrix);
// one CTA per pair for batches, whose pairs fill the device by themselves.
template <int PB>
int run_jacobi(float* X, float* Vt, JState* st, int s, int nb, int count, cudaStream_t stream) {
  const int nbe = nb + (nb & 1);
  const long long pairs = (long long)(nbe / 2) * count;
  int sms = sm_count();
  if (sms <= 0) sms = 1;
  if (pairs * 8 <= 2LL * sms + 8) return run_jacobi_cl<PB, 8>(X, Vt, st, s, nb, count, stream);
  return run_jacobi_cl<PB, 1>(X, Vt, st, s, nb, count, stream);
}

}  // namespace

size_t svd_batch_ws(const SvdItem* items, int L) {
  return make_layout(items, L, nullptr).bytes;
}

int svd_batch(const SvdItem* items, int L, float sigma_cutoff, void* ws, size_t ws_bytes, cudaStream_t stream) {
  Layout lo = make_layout(items, L, ws);
  if (lo.bytes > ws_bytes) return AB_ERR_WORKSPACE;
  // 1. Gram matrices into X
  for (auto& g : lo.groups) {
    const int s = g.first;
    for (size_t j = 0; j < g.second.size(); ++j) {
      const SvdItem& it = items[g.second[j]];
      float* G = lo.X[s] + j * (size_t)s * s;
      if (it.m >= it.n)   // G = W^T W
        AB_TRY(gemm_simt(it.W, it.w_dt, 1, it.n, it.W, it.w_dt, it.n, 1, G, AB_F32, s, s, s, it.m, stream));
      else                // G = W W^T
        AB_TRY(gemm_simt(it.W, it.w_dt, it.n, 1, it.W, it.w_dt, 1, it.n, G, AB_F32, s, s, s, it.n, stream));
    }
  }
  // 2. eigen-decomposition of every group
  for (auto& g : lo.groups) {
    const int s = g.first, count = (int)g.second.size();
    Plan p = make_plan(items[g.second[0]]);
    if (rows_jacobi_fits(count, s)) {
      // small enough to stay in shared memory for the whole iteration: the rows of G rotated until
      // orthogonal are lambda_i v_i^T, so the unit rows are the eigenvectors, already sorted
      AB_CUDA_OK(cudaMemsetAsync(lo.st[s], 0, sizeof(JState) * count, stream));
      AB_TRY(rows_jacobi(lo.X[s], lo.Vt[s], lo.item[g.second[0]].lam, &lo.st[s]->status, sizeof(JState), count, s,
                         lo.jobs[s], stream));
      int r_need = 0;
      for (int idx : g.second) r_need = std::max(r_need, make_plan(items[idx]).r_cap);
      complete_basis_kernel<<<count, 256, 2 * (size_t)s * sizeof(float), stream>>>(lo.Vt[s], lo.item[g.second[0]].lam, s,
                                                                                  r_need);
      AB_LAUNCH_OK();
      identity_perm_kernel<<<(count * s + 255) / 256, 256, 0, stream>>>(lo.item[g.second[0]].perm, s, count * s);
      AB_LAUNCH_OK();
      continue;
    }
    dim3 ig(64, (unsigned)count);
    init_state_kernel<<<ig, 256, 0, stream>>>(lo.Vt[s], lo.st[s], s, count);
    AB_LAUNCH_OK();
    int rc;
    if (p.pb == 32) rc = run_jacobi<32>(lo.X[s], lo.Vt[s], lo.st[s], s, p.nb, count, stream);
    else rc = run_jacobi<16>(lo.X[s], lo.Vt[s], lo.st[s], s, p.nb, count, stream);
    AB_TRY(rc);
    norms_sort_kernel<<<count, 256, (size_t)s * sizeof(float), stream>>>(
        lo.X[s], s, lo.item[g.second[0]].lam, lo.item[g.second[0]].perm);
    AB_LAUNCH_OK();
  }
  // 3. per matrix: leading vectors, long-side product, sigma, rank rule, factors
  for (auto& g : lo.groups) {
    const int s = g.first;
    for (size_t j = 0; j < g.second.size(); ++j) {
      const int i = g.second[j];
      const SvdItem& it = items[i];
      Plan p = make_plan(it);
      const ItemWs& w = lo.item[i];
      const float* Vt = lo.Vt[s] + j * (size_t)s * s;
      gather_rows_kernel<<<p.r_cap, 256, 0, stream>>>(Vt, w.perm, s, p.r_cap, w.Vr);
      AB_LAUNCH_OK();
      int64_t yt, yk;   // Ylong(k,t) = Y[t*yt + k*yk]
      if (p.tall) {     // Y (m x r_cap) = W Vr^T
        AB_TRY(gemm_simt(it.W, it.w_dt, it.n, 1, w.Vr, AB_F32, 1, s, w.Y, AB_F32, p.r_cap, it.m, p.r_cap, it.n, stream));
        yt = p.r_cap; yk = 1;
      } else {          // Y (r_cap x n) = Vr W
        AB_TRY(gemm_simt(w.Vr, AB_F32, s, 1, it.W, it.w_dt, it.n, 1, w.Y, AB_F32, it.n, p.r_cap, it.n, it.m, stream));
        yt = 1; yk = it.n;
      }
      long_norms_kernel<<<(p.r_cap + 31) / 32, 256, 0, stream>>>(w.Y, yt, yk, p.L, p.r_cap, it.sigma);
      AB_LAUNCH_OK();
      rank_rule_kernel<<<1, 32, 0, stream>>>(it.sigma, p.r_cap, sigma_cutoff, it.r_out, lo.st[s] + j, it.dev_status);
      AB_LAUNCH_OK();
      // tall: A is the long factor (A[t][k], strides r_max, 1), B the short one (B[k][u], strides n, 1)
      // wide: B is the long factor (B[k][t], strides 1, n),     A the short one (A[u][k]: k stride 1, u stride r_max)
      void* Fl = p.tall ? it.A : it.B;
      void* Fs = p.tall ? it.B : it.A;
      int64_t lt = p.tall ? it.r_max : 1, lk = p.tall ? 1 : it.n;
      int64_t sk = p.tall ? it.n : 1, su = p.tall ? 1 : it.r_max;
      int64_t total = (int64_t)(p.L + s) * it.r_max;
      unsigned grid = (unsigned)std::min<int64_t>((total + 255) / 256, (int64_t)std::max(sm_count(), 1) * 8);
      if (it.out_dt == AB_F32)
        write_factors_kernel<float><<<grid, 256, 0, stream>>>(w.Y, yt, yk, w.Vr, it.sigma, it.r_out, p.L, s, p.r_cap,
                                                             it.r_max, (float*)Fl, lt, lk, (float*)Fs, sk, su);
      else
        write_factors_kernel<bf16><<<grid, 256, 0, stream>>>(w.Y, yt, yk, w.Vr, it.sigma, it.r_out, p.L, s, p.r_cap,
                                                            it.r_max, (bf16*)Fl, lt, lk, (bf16*)Fs, sk, su);
      AB_LAUNCH_OK();
    }
  }
  return AB_OK;
}

}  // namespace ab
