// General tensor-core GEMM on sm_100a: the products of the path that are plain contractions.
//
//   C[M x N] = sum over terms t of  A_t[M x K] * B_t[N x K]^T        (bf16 operands, fp32 accumulation in TMEM)
//
// One term is the ordinary bf16 product (the dense layer of the full-rank phases: y = x W^T, dX = dY W,
// dW = dY^T x).  Six terms are the fp32-accurate product of two fp32 matrices that were cut into three bf16
// pieces each (hi + mid + lo carries 24 bits): hi*hi, hi*mid, mid*hi, hi*lo, lo*hi, mid*mid, the small terms
// first.  bf16 products are exact in fp32, so what is lost is the three products of order 2^-24 and the
// rounding of the fp32 sums.  This carries W = Abar Bbar, the Gram matrices and the long products of the
// group synchronisation, which need the 1e-6 / 1e-4 bounds of the fp32 path.
//
// Either operand may lie K-major (M x K resp. N x K, row-major) or MN-major (stored K x M resp. K x N,
// row-major); the shared-memory descriptors of the MMAs express the difference, nothing is transposed.
// Many problems run in one launch: a table of problem records (tensor maps included) sits in device memory
// and a CTA finds its problem and its 128 x 256 tile from its block index.  K may be cut into slices, each
// writing its own partial result (summed afterwards in ascending order: fixed bits).
//
// Warps (192 threads): 0 = TMA producer, 1 = MMA issuer and TMEM owner, 2..5 = epilogue (TMEM -> registers
// -> a staging tile of the warp's own -> TMA store of 32 rows).  Every wait is bounded (see ab_tc_ptx.cuh).
#include <vector>
#include <cstring>

#include "ab_common.cuh"
#include "ab_tc_ptx.cuh"

namespace ab {
namespace {

using namespace tc;

constexpr int kBM = 128, kBN = 256, kBK = 64;
constexpr int kAStage = kBM * 128;        // 16 KB: 128 x 64 bf16
constexpr int kBStage = kBN * 128;        // 32 KB
constexpr int kStage = kAStage + kBStage;
constexpr int kStages = 4;
constexpr int kStgBytes = 4096;           // 32 rows x 128 bytes
constexpr int kTcThreads = 192;
constexpr int kMaxTerms = 6;

struct TcBars {
  uint64_t full[kStages], empty[kStages];
  uint64_t acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  int abort_any;
};

// One problem of a batch, as the kernel reads it from device memory.
struct alignas(64) TcProblemDev {
  CUtensorMap a[3], b[3];   // the pieces of A and of B (one piece for a plain bf16 product)
  CUtensorMap c;            // output, boxes of 32 rows x 128 bytes
  int M, N, K;
  int nterms;
  int term_a[kMaxTerms], term_b[kMaxTerms];
  int a_mn, b_mn;           // 1: stored K x M / K x N
  int c_f32;                // 1: fp32 output (32 columns per box), 0: bf16 (64 columns per box)
  int tiles_n;              // column tiles
  int ksplit;               // slices of K
  int kslice;               // K per slice, a multiple of 64
  int c_rows;               // rows of one partial result in the output map (M when ksplit == 1)
  int first_tile;           // index of this problem's first tile among all tiles of the batch
  const int* live_rows;     // optional device ints: rows / columns at or beyond them are written as zero
  const int* live_cols;
};

__device__ __forceinline__ void tc_raise(TcBars* b, int* status) {
  *reinterpret_cast<volatile int*>(&b->abort_any) = 1;
  atomicExch(status, (int)AB_ERR_TIMEOUT);
}

// What one tile of the batch is: its problem, its corner, its slice of K.
struct TileInfo {
  const TcProblemDev* P;
  int m0, n0, slice, k_begin, k_end, nslab, ncols, nmma;
};
__device__ __forceinline__ TileInfo decode_tile(const TcProblemDev* __restrict__ probs, int nprobs, int tile) {
  int lo = 0, hi = nprobs - 1;
  while (lo < hi) {                       // the last problem whose first tile is <= tile
    const int mid = (lo + hi + 1) >> 1;
    if (probs[mid].first_tile <= tile) lo = mid; else hi = mid - 1;
  }
  TileInfo ti;
  ti.P = probs + lo;
  int t = tile - ti.P->first_tile;
  ti.slice = t % ti.P->ksplit;
  t /= ti.P->ksplit;
  ti.n0 = (t % ti.P->tiles_n) * kBN;
  ti.m0 = (t / ti.P->tiles_n) * kBM;
  ti.k_begin = ti.slice * ti.P->kslice;
  ti.k_end = ti.k_begin + ti.P->kslice;
  if (ti.k_end > ti.P->K) ti.k_end = ti.P->K;
  ti.nslab = ti.k_end > ti.k_begin ? (ti.k_end - ti.k_begin + kBK - 1) / kBK : 0;
  ti.ncols = ti.P->N - ti.n0;
  if (ti.ncols > kBN) ti.ncols = kBN;
  ti.nmma = (ti.ncols + 15) & ~15;
  return ti;
}

// Persistent CTAs: CTA b takes the tiles b, b + gridDim.x, ... of the batch.  Two 256-column accumulators in
// TMEM alternate between a CTA's tiles, so the epilogue of one tile (TMEM -> staging -> TMA stores) runs
// beside the loads and MMAs of the next.
__global__ void __launch_bounds__(kTcThreads, 1)
gemm_tc_kernel(const TcProblemDev* __restrict__ probs, int nprobs, int ntiles, int* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* ring = smem;
  uint8_t* stg = smem + kStages * kStage;
  TcBars* bars = reinterpret_cast<TcBars*>(stg + 4 * 2 * kStgBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) { mbar_init(&bars->full[i], 1); mbar_init(&bars->empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&bars->acc_full[i], 1); mbar_init(&bars->acc_empty[i], 4); }
    bars->abort_any = 0;
    fence_barrier_init();
  }
  if (warp == 1) tmem_alloc(&bars->tmem_base, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&bars->tmem_base);

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int i = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x) {
        const TileInfo ti = decode_tile(probs, nprobs, tile);
        const TcProblemDev* P = ti.P;
        const int a_mn = P->a_mn, b_mn = P->b_mn;
        for (int tix = 0; tix < P->nterms && ok; ++tix) {
          const CUtensorMap* ma = &P->a[P->term_a[tix]];
          const CUtensorMap* mb = &P->b[P->term_b[tix]];
          for (int ks = 0; ks < ti.nslab; ++ks, ++i) {
            const int slot = i % kStages, ph = (i / kStages) & 1;
            if (!mbar_wait(&bars->empty[slot], ph ^ 1)) { tc_raise(bars, status); ok = false; break; }
            uint8_t* da = ring + (size_t)slot * kStage;
            uint8_t* db = da + kAStage;
            const int k0 = ti.k_begin + ks * kBK;
            mbar_arrive_expect_tx(&bars->full[slot], kStage);
            if (a_mn) { for (int h = 0; h < 2; ++h) tma_load_2d(da + h * 8192, ma, &bars->full[slot], ti.m0 + 64 * h, k0); }
            else tma_load_2d(da, ma, &bars->full[slot], k0, ti.m0);
            if (b_mn) { for (int h = 0; h < 4; ++h) tma_load_2d(db + h * 8192, mb, &bars->full[slot], ti.n0 + 64 * h, k0); }
            else tma_load_2d(db, mb, &bars->full[slot], k0, ti.n0);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int i = 0, it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++it) {
        const TileInfo ti = decode_tile(probs, nprobs, tile);
        const TcProblemDev* P = ti.P;
        const int a_mn = P->a_mn, b_mn = P->b_mn;
        const uint32_t idesc = instr_desc_bf16(kBM, ti.nmma, a_mn, b_mn);
        const int b = it & 1;
        if (!mbar_wait(&bars->acc_empty[b], ((it >> 1) & 1) ^ 1)) { tc_raise(bars, status); ok = false; break; }
        tc_fence_after();
        const uint32_t tacc = tmem_base + 256 * b;
        int first = 1;
        for (int tix = 0; tix < P->nterms && ok; ++tix) {
          for (int ks = 0; ks < ti.nslab; ++ks, ++i) {
            const int slot = i % kStages, ph = (i / kStages) & 1;
            if (!mbar_wait(&bars->full[slot], ph)) { tc_raise(bars, status); ok = false; break; }
            tc_fence_after();
            const uint32_t sa = smem_u32(ring + (size_t)slot * kStage), sb = sa + kAStage;
            int ksteps = (ti.k_end - (ti.k_begin + ks * kBK) + 15) >> 4;
            if (ksteps > 4) ksteps = 4;
            for (int kk = 0; kk < ksteps; ++kk) {
              const uint64_t da = a_mn ? smem_desc_sw128(sa + kk * 2048, 8192) : smem_desc_sw128(sa, 16) + 2 * kk;
              const uint64_t db = b_mn ? smem_desc_sw128(sb + kk * 2048, 8192) : smem_desc_sw128(sb, 16) + 2 * kk;
              tc_mma_bf16(tacc, da, db, idesc, first ? 0u : 1u);
              first = 0;
            }
            tc_commit(&bars->empty[slot]);
          }
        }
        if (ok) tc_commit(&bars->acc_full[b]);
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int qw = warp & 3;
    const uint32_t lane_base = (uint32_t)(qw * 32) << 16;
    uint8_t* mystg = stg + (size_t)(warp - 2) * 2 * kStgBytes;
    int nst = 0, it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < ntiles && ok; tile += gridDim.x, ++it) {
      const TileInfo ti = decode_tile(probs, nprobs, tile);
      const TcProblemDev* P = ti.P;
      const int b = it & 1;
      const bool have_acc = ti.nslab > 0 && P->nterms > 0;      // an empty reduction leaves zeros
      {
        int w = 1;
        if (lane == 0) { w = mbar_wait(&bars->acc_full[b], (it >> 1) & 1) ? 1 : 0; if (!w) tc_raise(bars, status); }
        ok = __shfl_sync(0xffffffffu, w, 0) != 0;
      }
      if (!ok) break;
      tc_fence_after();
      const int grow = ti.m0 + qw * 32 + lane;           // row of C this thread holds
      const int live_r = P->live_rows ? *P->live_rows : P->M;
      const int live_c = P->live_cols ? *P->live_cols : P->N;
      const bool rows_in = ti.m0 + qw * 32 < P->M;
      const int c_f32 = P->c_f32;
      const int pcols = c_f32 ? 32 : 64;                 // columns of one 128-byte piece
      const int crow = ti.slice * P->c_rows + ti.m0 + qw * 32;
      const uint32_t tacc = tmem_base + 256 * b + lane_base;
      for (int c0 = 0; c0 < ti.ncols; c0 += pcols) {
        uint32_t v[4][16];
        if (have_acc && rows_in) {
#pragma unroll
          for (int gq = 0; gq < 4; ++gq)
            if (gq * 16 < pcols) tmem_ld16_nowait(tacc + c0 + gq * 16, v[gq]);
          tmem_wait_ld();
        } else {
#pragma unroll
          for (int gq = 0; gq < 4; ++gq)
#pragma unroll
            for (int e = 0; e < 16; ++e) v[gq][e] = 0u;
        }
        if (c0 + pcols >= ti.ncols) {                    // the last piece is in registers: hand the accumulator back
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&bars->acc_empty[b]);
        }
        if (!rows_in) continue;
        const bool row_dead = grow >= live_r;
#pragma unroll
        for (int gq = 0; gq < 4; ++gq)
#pragma unroll
          for (int e = 0; e < 16; ++e)
            if (row_dead || ti.n0 + c0 + gq * 16 + e >= live_c) v[gq][e] = 0u;
        uint8_t* buf = mystg + (nst & 1) * kStgBytes;
        ++nst;
        if (lane == 0) tma_store_wait_read<1>();
        __syncwarp();
        uint8_t* rowp = buf + lane * 128;
        if (c_f32) {
#pragma unroll
          for (int ch = 0; ch < 8; ++ch)
            *reinterpret_cast<uint4*>(rowp + ((ch ^ (lane & 7)) << 4)) =
                make_uint4(v[ch >> 2][(ch & 3) * 4], v[ch >> 2][(ch & 3) * 4 + 1], v[ch >> 2][(ch & 3) * 4 + 2],
                           v[ch >> 2][(ch & 3) * 4 + 3]);
        } else {
#pragma unroll
          for (int ch = 0; ch < 8; ++ch) {
            uint32_t w4[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int idx = ch * 8 + 2 * e;          // column within the 64-column piece
              __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(v[idx >> 4][idx & 15]),
                                                        __uint_as_float(v[(idx + 1) >> 4][(idx + 1) & 15]));
              w4[e] = *reinterpret_cast<uint32_t*>(&h2);
            }
            *reinterpret_cast<uint4*>(rowp + ((ch ^ (lane & 7)) << 4)) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_2d(&P->c, buf, ti.n0 + c0, crow);
          tma_store_commit();
        }
      }
    }
    if (lane == 0) tma_store_wait_all();
  }

  tc_fence_before();
  __syncthreads();
  if (*reinterpret_cast<volatile int*>(&bars->abort_any)) {
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) { }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// ---------------------------------------------------------------------------------------------
// fp32 -> three bf16 pieces: hi = bf16(x), mid = bf16(x - hi), lo = bf16(x - hi - mid); hi + mid + lo = x to
// 2^-24 (the subtractions are exact).  One job per matrix, all jobs in one launch.
__global__ void __launch_bounds__(256)
split3_kernel(const SplitJob* __restrict__ jobs, int njobs) {
  int lo = 0, hi = njobs - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (jobs[mid].first_block <= (int64_t)blockIdx.x) lo = mid; else hi = mid - 1;
  }
  const SplitJob j = jobs[lo];
  // four consecutive elements of a row per thread when the rows allow 16-byte loads and 8-byte stores
  const bool vec = (j.cols & 3) == 0 && (j.ld_src & 3) == 0 && (j.ld_dst & 3) == 0 &&
                   ((reinterpret_cast<uintptr_t>(j.src) & 15u) == 0) && ((reinterpret_cast<uintptr_t>(j.hi) & 7u) == 0) &&
                   ((reinterpret_cast<uintptr_t>(j.mid) & 7u) == 0) && ((reinterpret_cast<uintptr_t>(j.lo) & 7u) == 0);
  const unsigned cols4 = (unsigned)(j.cols + 3) >> 2;
  const unsigned total4 = (unsigned)j.rows * cols4;
  const unsigned i = (unsigned)((int64_t)blockIdx.x - j.first_block) * 256u + threadIdx.x;
  if (i >= total4) return;
  const unsigned r = i / cols4, c = (i - r * cols4) * 4u;
  float x[4];
  const float* src = j.src + (int64_t)r * j.ld_src + c;
  if (vec) {
    const float4 q = *reinterpret_cast<const float4*>(src);
    x[0] = q.x; x[1] = q.y; x[2] = q.z; x[3] = q.w;
  } else {
#pragma unroll
    for (int e = 0; e < 4; ++e) x[e] = (c + e < (unsigned)j.cols) ? src[e] : 0.f;
  }
  bf16 h[4], m[4], l[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    h[e] = __float2bfloat16_rn(x[e]);
    const float r1 = x[e] - __bfloat162float(h[e]);
    m[e] = __float2bfloat16_rn(r1);
    l[e] = __float2bfloat16_rn(r1 - __bfloat162float(m[e]));
  }
  const int64_t o = (int64_t)r * j.ld_dst + c;
  if (vec) {
    *reinterpret_cast<uint2*>(j.hi + o) = *reinterpret_cast<const uint2*>(h);
    *reinterpret_cast<uint2*>(j.mid + o) = *reinterpret_cast<const uint2*>(m);
    *reinterpret_cast<uint2*>(j.lo + o) = *reinterpret_cast<const uint2*>(l);
  } else {
#pragma unroll
    for (int e = 0; e < 4; ++e)
      if (c + e < (unsigned)j.cols) { j.hi[o + e] = h[e]; j.mid[o + e] = m[e]; j.lo[o + e] = l[e]; }
  }
}

// out[i] = sum over slices of part[s][i], ascending s (fixed order); partials are rows_pad x ld, out is rows x ld
__global__ void __launch_bounds__(256)
sum_slices_kernel(const float* __restrict__ part, float* __restrict__ out, int64_t count, int64_t slice_stride, int slices) {
  const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (i >= count) return;
  float acc = part[i];
  for (int s = 1; s < slices; ++s) acc += part[i + s * slice_stride];
  out[i] = acc;
}

}  // namespace

int64_t split_job_blocks(int rows, int cols) { return ((int64_t)rows * ((cols + 3) / 4) + 255) / 256; }

int split3_batched(const SplitJob* d_jobs, int njobs, int64_t total_blocks, cudaStream_t st) {
  if (njobs <= 0 || total_blocks <= 0) return AB_OK;
  if (total_blocks > ((int64_t)1 << 30)) return AB_ERR_UNSUPPORTED;
  split3_kernel<<<(unsigned)total_blocks, 256, 0, st>>>(d_jobs, njobs);
  AB_LAUNCH_OK();
  return AB_OK;
}

int sum_slices(const float* part, float* out, int64_t count, int64_t slice_stride, int slices, cudaStream_t st) {
  if (count <= 0) return AB_OK;
  sum_slices_kernel<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(part, out, count, slice_stride, slices);
  AB_LAUNCH_OK();
  return AB_OK;
}

bool gemm_tc_available() { return tc_device_ok(); }

size_t gemm_tc_table_bytes(int count) { return align_up((size_t)count * sizeof(TcProblemDev), 256); }

bool gemm_tc_problem_ok(const TcProblem& q) {
  if (q.M <= 0 || q.N <= 0 || q.K <= 0) return false;
  if (q.A.pieces != q.B.pieces || (q.A.pieces != 1 && q.A.pieces != 3)) return false;
  if (q.A.ld % 8 != 0 || q.B.ld % 8 != 0) return false;
  for (int i = 0; i < q.A.pieces; ++i)
    if (!aligned(q.A.p[i], 16) || !aligned(q.B.p[i], 16)) return false;
  if (!aligned(q.C, 16) || (q.ldc * (q.c_f32 ? 4 : 2)) % 16 != 0) return false;
  if (q.ksplit < 1 || (q.ksplit > 1 && !q.c_f32)) return false;
  return true;
}

int gemm_tc_batched(const TcProblem* probs, int count, void* table_dev, int* status, cudaStream_t st) {
  if (count <= 0) return AB_OK;
  if (!tc_device_ok()) return AB_ERR_UNSUPPORTED;
  std::vector<TcProblemDev> tab((size_t)count);
  int tiles = 0;
  for (int i = 0; i < count; ++i) {
    const TcProblem& q = probs[i];
    if (!gemm_tc_problem_ok(q)) return AB_ERR_UNSUPPORTED;
    TcProblemDev& d = tab[i];
    std::memset(&d, 0, sizeof(d));
    for (int pc = 0; pc < q.A.pieces; ++pc) {
      if (q.A.mn) AB_TRY(make_tensor_map_2d(&d.a[pc], q.A.p[pc], false, q.K, q.M, q.A.ld, 64, 64));
      else AB_TRY(make_tensor_map_2d(&d.a[pc], q.A.p[pc], false, q.M, q.K, q.A.ld, 64, kBM));
      if (q.B.mn) AB_TRY(make_tensor_map_2d(&d.b[pc], q.B.p[pc], false, q.K, q.N, q.B.ld, 64, 64));
      else AB_TRY(make_tensor_map_2d(&d.b[pc], q.B.p[pc], false, q.N, q.K, q.B.ld, 64, kBN));
    }
    d.M = q.M; d.N = q.N; d.K = q.K;
    if (q.A.pieces == 1) { d.nterms = 1; d.term_a[0] = 0; d.term_b[0] = 0; }
    else {   // small terms first: mid*mid, lo*hi, hi*lo, mid*hi, hi*mid, hi*hi
      const int ta[6] = {1, 2, 0, 1, 0, 0}, tb[6] = {1, 0, 2, 0, 1, 0};
      d.nterms = 6;
      for (int k = 0; k < 6; ++k) { d.term_a[k] = ta[k]; d.term_b[k] = tb[k]; }
    }
    d.a_mn = q.A.mn ? 1 : 0; d.b_mn = q.B.mn ? 1 : 0; d.c_f32 = q.c_f32 ? 1 : 0;
    d.tiles_n = (q.N + kBN - 1) / kBN;
    d.ksplit = q.ksplit;
    const int slabs = (q.K + kBK - 1) / kBK;
    d.kslice = ((slabs + q.ksplit - 1) / q.ksplit) * kBK;
    d.c_rows = q.ksplit > 1 ? (q.M + kBM - 1) / kBM * kBM : q.M;
    AB_TRY(make_tensor_map_2d(&d.c, q.C, q.c_f32, (uint64_t)d.c_rows * q.ksplit - (q.ksplit > 1 ? 0 : 0), q.N, q.ldc,
                              q.c_f32 ? 32 : 64, 32));
    d.first_tile = tiles;
    d.live_rows = q.live_rows; d.live_cols = q.live_cols;
    tiles += ((q.M + kBM - 1) / kBM) * d.tiles_n * q.ksplit;
  }
  AB_CUDA_OK(cudaMemcpyAsync(table_dev, tab.data(), tab.size() * sizeof(TcProblemDev), cudaMemcpyHostToDevice, st));
  const size_t smem = (size_t)kStages * kStage + 4 * 2 * kStgBytes + sizeof(TcBars) + 1024;
  AB_CUDA_OK(cudaFuncSetAttribute(gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  int sms = sm_count();
  if (sms <= 0) return AB_ERR_CUDA;
  const int grid = tiles < sms ? tiles : sms;
  gemm_tc_kernel<<<(unsigned)grid, kTcThreads, smem, st>>>(static_cast<const TcProblemDev*>(table_dev), count, tiles, status);
  AB_LAUNCH_OK();
  return AB_OK;
}

}  // namespace ab
