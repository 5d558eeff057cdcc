// Fused tensor-core chain for bf16 storage (fp32 accumulation) on sm_100a.
//
// row_chain_kernel: one CTA per block of 128 rows computes  S = In F1^T  (128 x r, K-loop over
// the input width, accumulator in TMEM), rounds S to bf16 into shared memory, and multiplies
// on:  Out = S F2^T  in 128-column chunks (two TMEM accumulators so the epilogue of one chunk
// overlaps the MMAs of the next).  The rank-r intermediate never goes to HBM unless the
// caller asks for a copy.
//   forward : In = x,  F1 = B  (r x n), F2 = A   (m x r), Out = y,  S = T
//   backward: In = dY, F1 = A^T (r x m), F2 = B^T (n x r), Out = dX, S = dT
// grad_kernel: dA = dY^T T and dB^T = x^T dT are reductions over the rows; a CTA owns 128
// output rows (a slice of m or of n) and one slice of the N rows, streams 64-row slabs of
// both operands (both "MN-major": the reduction index is the slow one in memory) and leaves
// an fp32 partial; reduce_kernel adds the partials in ascending slice order.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer (and TMEM owner),
// warps 2-5 = epilogue (TMEM -> registers -> shared/global).  All operand tiles are TMA
// boxes of 64 bf16 (128 bytes) x rows with 128-byte swizzle.  Every mbarrier wait gives up
// after about a second, raises AB_ERR_TIMEOUT in the status word and unwinds to the common
// exit, where TMEM is released.
#include <mutex>

#include "ab_common.cuh"
#include "ab_tc_ptx.cuh"

namespace ab {
namespace {

using namespace tc;

constexpr int kAtomBytes = 16384;      // 128 rows x 128 bytes
constexpr int kMaxStages = 6;
constexpr int kMaxStages2 = 6;         // 32 KB slots of the second product, carved from the same ring memory
constexpr int kChunk = 256;            // output columns per accumulator of the second product
constexpr int kAtom2Bytes = kChunk * 128;   // one 256 x 64 tile of F2
constexpr int kSmemLimit = 227 * 1024;
constexpr int kTmemCols = 512;
constexpr int kEpiThreads = 128;

struct RowChainParams {
  int K1;        // width of In (reduction length of the first product)
  int P;         // width of Out (0: first product only)
  int r;
  int nk1;       // ceil(K1 / 64)
  int nchunks;   // ceil(P / 256)
  int natoms;    // ceil(r / 64)
  int ns;        // ring stages
  int slot_bytes;
  int ns2;       // stages of the second product's ring (one 128 x 64 atom of F2 each)
  int save_s;    // 1: copy S to global through tmS
  int clear_status;   // 1: this is the first kernel of a call and zeroes the status word (see clear_status_word)
  int* status;
};

struct Bars {
  uint64_t full[kMaxStages], empty[kMaxStages];
  uint64_t full2[kMaxStages2], empty2[kMaxStages2];
  uint64_t t_full, s_ready, unit_done;
  uint64_t acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  int abort_any;   // set by any role that gave up
  int epi_abort;   // written and read by the epilogue warps only, around their own barrier
};

__device__ __forceinline__ void raise_timeout(Bars* b, int* status) {
  *reinterpret_cast<volatile int*>(&b->abort_any) = 1;
  atomicExch(status, (int)AB_ERR_TIMEOUT);
}

// The status word of a call starts at zero.  The first kernel of the call clears it itself (block 0,
// right after dep_wait) instead of a memset in the stream, which would sit between this kernel and the
// one before it and undo the overlap of dep_wait.  Block 0 runs in the first wave and gets here within
// microseconds of the launch; a kernel raises AB_ERR_TIMEOUT only after a wait of about a second, so
// the clear cannot wipe a raised error.
__device__ __forceinline__ void clear_status_word(int enabled, int* status) {
  if (enabled && blockIdx.x == 0 && threadIdx.x == 0) atomicExch(status, 0);
}

// epilogue-wide wait: every epilogue thread calls it; the verdict is uniform
__device__ __forceinline__ bool epi_wait(Bars* b, uint64_t* bar, uint32_t parity, int* status) {
  if (!mbar_wait(bar, parity)) {
    *reinterpret_cast<volatile int*>(&b->epi_abort) = 1;
    raise_timeout(b, status);
  }
  named_bar_sync(1, kEpiThreads);
  return *reinterpret_cast<volatile int*>(&b->epi_abort) == 0;
}

__device__ __forceinline__ void store_bf16x16_swizzled(uint8_t* row_base, int row, int c0, const uint32_t (&v)[16]) {
  // 16 consecutive columns c0..c0+15 (c0 % 16 == 0) of a 128-byte row inside a swizzled atom
  uint32_t w[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
    w[i] = *reinterpret_cast<uint32_t*>(&h);
  }
  const int ch = (c0 & 63) >> 3;
  uint4* p0 = reinterpret_cast<uint4*>(row_base + (((ch) ^ (row & 7)) << 4));
  uint4* p1 = reinterpret_cast<uint4*>(row_base + (((ch + 1) ^ (row & 7)) << 4));
  *p0 = make_uint4(w[0], w[1], w[2], w[3]);
  *p1 = make_uint4(w[4], w[5], w[6], w[7]);
}

__global__ void __launch_bounds__(192, 1)
row_chain_kernel(const __grid_constant__ CUtensorMap tmIn, const __grid_constant__ CUtensorMap tmF1,
                 const __grid_constant__ CUtensorMap tmF2, const __grid_constant__ CUtensorMap tmOut,
                 const __grid_constant__ CUtensorMap tmS, const RowChainParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* S = smem;
  uint8_t* stg = S + p.natoms * kAtomBytes;
  uint8_t* ring = stg + 2 * kAtomBytes;
  Bars* bars = reinterpret_cast<Bars*>(ring + (size_t)p.ns * p.slot_bytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row0 = blockIdx.x * 128;
  // All CTAs walk the same factor tiles.  Started together they would all ask L2 for the same
  // few lines at the same moment (measured: 29 GB/s per SM); each CTA therefore starts its walk
  // at a different slab / chunk and wraps round.  The order is a function of blockIdx only.
  const int rot1 = blockIdx.x % p.nk1;
  const int rot2 = p.nchunks > 0 ? (blockIdx.x * 5) % p.nchunks : 0;

  if (threadIdx.x == 0) {
    for (int i = 0; i < p.ns; ++i) { mbar_init(&bars->full[i], 1); mbar_init(&bars->empty[i], 1); }
    for (int i = 0; i < p.ns2; ++i) { mbar_init(&bars->full2[i], 1); mbar_init(&bars->empty2[i], 1); }
    mbar_init(&bars->t_full, 1);
    mbar_init(&bars->s_ready, kEpiThreads);
    for (int i = 0; i < 2; ++i) { mbar_init(&bars->acc_full[i], 1); mbar_init(&bars->acc_empty[i], 4); }
    bars->abort_any = 0;
    bars->epi_abort = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tmIn); tma_prefetch_desc(&tmF1); tma_prefetch_desc(&tmF2);
    tma_prefetch_desc(&tmOut); tma_prefetch_desc(&tmS);
  }
  if (warp == 1) tmem_alloc(&bars->tmem_base, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&bars->tmem_base);
  dep_wait();            // nothing above touches global memory
  dep_launch();
  clear_status_word(p.clear_status, p.status);
  // T (r <= 256 columns) is read out into S before the second product starts, so the two
  // 256-column accumulators of the second product reuse its columns.
  const uint32_t tT = tmem_base;
  const uint32_t tAcc0 = tmem_base;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int i = 0;
      bool ok = true;
      for (int ks = 0; ks < p.nk1 && ok; ++ks, ++i) {
        const int slot = i % p.ns, ph = (i / p.ns) & 1;
        if (!mbar_wait(&bars->empty[slot], ph ^ 1)) { raise_timeout(bars, p.status); ok = false; break; }
        uint8_t* dst = ring + (size_t)slot * p.slot_bytes;
        mbar_arrive_expect_tx(&bars->full[slot], kAtomBytes + p.r * 128);
        const int kr = (ks + rot1) % p.nk1;   // every CTA starts on a different slab: see rot1
        tma_load_2d(dst, &tmIn, &bars->full[slot], kr * 64, row0);
        tma_load_2d(dst + kAtomBytes, &tmF1, &bars->full[slot], kr * 64, 0);
      }
      // The second product re-cuts the ring memory into 16 KB slots, so that many atoms of F2
      // are in flight at once (L2 latency x the rate the MMAs need is > 100 KB); it may only be
      // refilled once every MMA of the first product has read its slabs.
      if (ok && p.nchunks > 0 && !mbar_wait(&bars->t_full, 0)) { raise_timeout(bars, p.status); ok = false; }
      i = 0;
      for (int c = 0; c < p.nchunks && ok; ++c) {
        for (int j = 0; j < p.natoms; ++j, ++i) {
          const int slot = i % p.ns2, ph = (i / p.ns2) & 1;
          if (!mbar_wait(&bars->empty2[slot], ph ^ 1)) { raise_timeout(bars, p.status); ok = false; break; }
          mbar_arrive_expect_tx(&bars->full2[slot], kAtom2Bytes);
          tma_load_2d(ring + (size_t)slot * kAtom2Bytes, &tmF2, &bars->full2[slot], j * 64, ((c + rot2) % p.nchunks) * kChunk);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc1 = instr_desc_bf16(128, p.r, 0, 0);
      const uint32_t idesc2 = instr_desc_bf16(128, kChunk, 0, 0);
      int i = 0;
      bool ok = true;
      for (int ks = 0; ks < p.nk1; ++ks, ++i) {
        const int slot = i % p.ns, ph = (i / p.ns) & 1;
        if (!mbar_wait(&bars->full[slot], ph)) { raise_timeout(bars, p.status); ok = false; break; }
        tc_fence_after();
        const uint32_t sa = smem_u32(ring + (size_t)slot * p.slot_bytes);
        const uint64_t da = smem_desc_sw128(sa, 16), db = smem_desc_sw128(sa + kAtomBytes, 16);
        int ksteps = (p.K1 - ((ks + rot1) % p.nk1) * 64 + 15) >> 4;
        if (ksteps > 4) ksteps = 4;
        for (int kk = 0; kk < ksteps; ++kk) tc_mma_bf16(tT, da + 2 * kk, db + 2 * kk, idesc1, (ks | kk) != 0);
        tc_commit(&bars->empty[slot]);
      }
      if (ok) {
        tc_commit(&bars->t_full);
        if (p.nchunks > 0) {
          if (!mbar_wait(&bars->s_ready, 0)) { raise_timeout(bars, p.status); ok = false; }
          tc_fence_after();
        }
      }
      i = 0;
      for (int c = 0; c < p.nchunks && ok; ++c) {
        const int b = c & 1;
        if (!mbar_wait(&bars->acc_empty[b], ((c >> 1) & 1) ^ 1)) { raise_timeout(bars, p.status); ok = false; break; }
        tc_fence_after();
        const uint32_t tacc = tAcc0 + kChunk * b;
        for (int j = 0; j < p.natoms; ++j, ++i) {
          const int slot = i % p.ns2, ph = (i / p.ns2) & 1;
          if (!mbar_wait(&bars->full2[slot], ph)) { raise_timeout(bars, p.status); ok = false; break; }
          tc_fence_after();
          const uint64_t da = smem_desc_sw128(smem_u32(S + j * kAtomBytes), 16);
          const uint64_t db = smem_desc_sw128(smem_u32(ring + (size_t)slot * kAtom2Bytes), 16);
          int ksteps = (p.r - j * 64) >> 4;
          if (ksteps > 4) ksteps = 4;
          for (int kk = 0; kk < ksteps; ++kk) tc_mma_bf16(tacc, da + 2 * kk, db + 2 * kk, idesc2, (j | kk) != 0);
          tc_commit(&bars->empty2[slot]);
        }
        if (ok) tc_commit(&bars->acc_full[b]);
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int q = warp & 3;                 // TMEM lane quarter this warp may read
    const int row = q * 32 + lane;          // row of the 128-row block
    const uint32_t lane_base = (uint32_t)(q * 32) << 16;
    const bool issuer = (threadIdx.x == 64);
    bool ok = epi_wait(bars, &bars->t_full, 0, p.status);
    if (ok) {
      tc_fence_after();
      for (int c0 = 0; c0 < p.r; c0 += 64) {       // up to four 16-column loads in flight per wait
        uint32_t v[4][16];
#pragma unroll
        for (int g = 0; g < 4; ++g)
          if (c0 + g * 16 < p.r) tmem_ld16_nowait(tT + lane_base + c0 + g * 16, v[g]);
        tmem_wait_ld();
#pragma unroll
        for (int g = 0; g < 4; ++g)
          if (c0 + g * 16 < p.r) store_bf16x16_swizzled(S + (c0 >> 6) * kAtomBytes + row * 128, row, c0 + g * 16, v[g]);
      }
      tc_fence_before();
      fence_proxy_async_smem();
      mbar_arrive(&bars->s_ready);
      if (p.save_s) {
        named_bar_sync(1, kEpiThreads);
        if (issuer) {
          for (int j = 0; j < p.natoms; ++j) tma_store_2d(&tmS, S + j * kAtomBytes, j * 64, row0);
          tma_store_commit();
        }
      }
    }
    int nstores = 0;
    for (int c = 0; c < p.nchunks && ok; ++c) {
      const int b = c & 1;
      ok = epi_wait(bars, &bars->acc_full[b], (c >> 1) & 1, p.status);
      if (!ok) break;
      tc_fence_after();
      const uint32_t tacc = tAcc0 + kChunk * b + lane_base;
      for (int h = 0; h < kChunk / 64; ++h) {
        const int col = ((c + rot2) % p.nchunks) * kChunk + h * 64;
        const bool live = col < p.P;                 // columns beyond the output are not staged at all
        uint32_t v[4][16];
        if (live) {
#pragma unroll
          for (int g = 0; g < 4; ++g) tmem_ld16_nowait(tacc + h * 64 + g * 16, v[g]);
          tmem_wait_ld();
        }
        if (h == kChunk / 64 - 1) {                  // the last columns are in registers: release the accumulator
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&bars->acc_empty[b]);
        }
        if (!live) continue;
        // staging tiles alternate with every store issued, so "at most one store still reading"
        // always means the other tile
        uint8_t* buf = stg + (nstores & 1) * kAtomBytes;
        ++nstores;
        if (issuer) tma_store_wait_read<1>();
        named_bar_sync(1, kEpiThreads);
#pragma unroll
        for (int g = 0; g < 4; ++g) store_bf16x16_swizzled(buf + row * 128, row, g * 16, v[g]);
        fence_proxy_async_smem();
        named_bar_sync(1, kEpiThreads);
        if (issuer) {
          tma_store_2d(&tmOut, buf, col, row0);
          tma_store_commit();
        }
      }
    }
    if (issuer) tma_store_wait_all();
  }

  // ------------------------------------------------------------ common exit
  tc_fence_before();
  __syncthreads();
  if (*reinterpret_cast<volatile int*>(&bars->abort_any)) {
    // give loads that are still in flight time to land before the shared memory is released
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) { }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---------------------------------------------------------------------------------------------
// row_chain_units_kernel: the same chain for many row blocks per CTA.  A persistent CTA owns a
// contiguous range of 128-row blocks and works through it in units of two blocks (one block when
// the range is odd).  Both blocks of a unit share every factor tile that is loaded -- each slab of
// F1 feeds two first-product MMAs, each tile of F2 two second-product MMAs -- so a row costs half
// the factor bytes; what paces the single-block kernel is exactly those bytes (1.5 MB of factors
// against 0.2 MB of activations per block at the ViT shapes).  In a two-block unit the two
// accumulators belong to the two blocks (the epilogue of one overlaps the MMAs of the other); in a
// one-block unit they alternate between chunks as in row_chain_kernel.
struct UnitParams {
  int K1, P, r, nk1, nchunks, natoms;
  int ns, slot_bytes;      // first product: slots of two 128-row In tiles + one F1 slab
  int ns2, ring2_bytes;    // second product: 32 KB slots at the start of shared memory
  int save_s;
  int tiles;               // 128-row blocks in all
  int clear_status;
  int* status;
};

__global__ void __launch_bounds__(192, 1)
row_chain_units_kernel(const __grid_constant__ CUtensorMap tmIn, const __grid_constant__ CUtensorMap tmF1,
                       const __grid_constant__ CUtensorMap tmF2, const __grid_constant__ CUtensorMap tmOut,
                       const __grid_constant__ CUtensorMap tmS, const UnitParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  // [ second-product ring | S of block 0 | S of block 1 | two staging tiles | barriers ]; the first
  // product's ring lies over the first three regions, which it has to itself while it runs
  uint8_t* ring = smem;
  uint8_t* S0 = smem + p.ring2_bytes;
  uint8_t* stg = S0 + 2 * p.natoms * kAtomBytes;
  Bars* bars = reinterpret_cast<Bars*>(stg + 2 * kAtomBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t_begin = (int)((int64_t)blockIdx.x * p.tiles / gridDim.x);
  const int t_end = (int)((int64_t)(blockIdx.x + 1) * p.tiles / gridDim.x);
  const int rot1 = blockIdx.x % p.nk1;
  const int rot2 = p.nchunks > 0 ? (blockIdx.x * 5) % p.nchunks : 0;

  if (threadIdx.x == 0) {
    for (int i = 0; i < p.ns; ++i) { mbar_init(&bars->full[i], 1); mbar_init(&bars->empty[i], 1); }
    for (int i = 0; i < p.ns2; ++i) { mbar_init(&bars->full2[i], 1); mbar_init(&bars->empty2[i], 1); }
    mbar_init(&bars->t_full, 1);
    mbar_init(&bars->s_ready, kEpiThreads);
    mbar_init(&bars->unit_done, 2);             // the MMA issuer's commit and the epilogue's store issuer
    for (int i = 0; i < 2; ++i) { mbar_init(&bars->acc_full[i], 1); mbar_init(&bars->acc_empty[i], 4); }
    bars->abort_any = 0;
    bars->epi_abort = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tmIn); tma_prefetch_desc(&tmF1); tma_prefetch_desc(&tmF2);
    tma_prefetch_desc(&tmOut); tma_prefetch_desc(&tmS);
  }
  if (warp == 1) tmem_alloc(&bars->tmem_base, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&bars->tmem_base);
  dep_wait();            // nothing above touches global memory
  dep_launch();
  clear_status_word(p.clear_status, p.status);
  // TMEM: block b of a unit keeps its S accumulator at column 256 b while the first product runs;
  // accumulator b of the second product takes the same 256 columns afterwards.

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int i1 = 0, i2 = 0, u = 0;
      bool ok = true;
      for (int t = t_begin; t < t_end && ok; ++u) {
        const int nt = (t_end - t >= 2) ? 2 : 1;
        const int row0 = t * 128;
        // the shared memory of the last unit is free once its MMAs are done and its stores have been read
        if (u > 0 && !mbar_wait(&bars->unit_done, (u - 1) & 1)) { raise_timeout(bars, p.status); ok = false; break; }
        for (int ks = 0; ks < p.nk1 && ok; ++ks, ++i1) {
          const int slot = i1 % p.ns, ph = (i1 / p.ns) & 1;
          if (!mbar_wait(&bars->empty[slot], ph ^ 1)) { raise_timeout(bars, p.status); ok = false; break; }
          uint8_t* dst = smem + (size_t)slot * p.slot_bytes;
          mbar_arrive_expect_tx(&bars->full[slot], nt * kAtomBytes + p.r * 128);
          const int kr = (ks + rot1) % p.nk1;
          tma_load_2d(dst, &tmIn, &bars->full[slot], kr * 64, row0);
          if (nt == 2) tma_load_2d(dst + kAtomBytes, &tmIn, &bars->full[slot], kr * 64, row0 + 128);
          tma_load_2d(dst + 2 * kAtomBytes, &tmF1, &bars->full[slot], kr * 64, 0);
        }
        // the second product's slots lie over the first product's: wait until its MMAs have read them
        if (ok && !mbar_wait(&bars->t_full, u & 1)) { raise_timeout(bars, p.status); ok = false; }
        for (int c = 0; c < p.nchunks && ok; ++c) {
          for (int j = 0; j < p.natoms; ++j, ++i2) {
            const int slot = i2 % p.ns2, ph = (i2 / p.ns2) & 1;
            if (!mbar_wait(&bars->empty2[slot], ph ^ 1)) { raise_timeout(bars, p.status); ok = false; break; }
            mbar_arrive_expect_tx(&bars->full2[slot], kAtom2Bytes);
            tma_load_2d(ring + (size_t)slot * kAtom2Bytes, &tmF2, &bars->full2[slot], j * 64,
                        ((c + rot2) % p.nchunks) * kChunk);
          }
        }
        t += nt;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc1 = instr_desc_bf16(128, p.r, 0, 0);
      const uint32_t idesc2 = instr_desc_bf16(128, kChunk, 0, 0);
      int i1 = 0, i2 = 0, u = 0;
      int q[2] = {0, 0};                       // uses of each accumulator so far
      bool ok = true;
      for (int t = t_begin; t < t_end && ok; ++u) {
        const int nt = (t_end - t >= 2) ? 2 : 1;
        for (int ks = 0; ks < p.nk1; ++ks, ++i1) {
          const int slot = i1 % p.ns, ph = (i1 / p.ns) & 1;
          if (!mbar_wait(&bars->full[slot], ph)) { raise_timeout(bars, p.status); ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + (size_t)slot * p.slot_bytes);
          const uint64_t da0 = smem_desc_sw128(sa, 16), da1 = smem_desc_sw128(sa + kAtomBytes, 16);
          const uint64_t db = smem_desc_sw128(sa + 2 * kAtomBytes, 16);
          int ksteps = (p.K1 - ((ks + rot1) % p.nk1) * 64 + 15) >> 4;
          if (ksteps > 4) ksteps = 4;
          for (int kk = 0; kk < ksteps; ++kk) {
            tc_mma_bf16(tmem_base, da0 + 2 * kk, db + 2 * kk, idesc1, (ks | kk) != 0);
            if (nt == 2) tc_mma_bf16(tmem_base + 256, da1 + 2 * kk, db + 2 * kk, idesc1, (ks | kk) != 0);
          }
          tc_commit(&bars->empty[slot]);
        }
        if (!ok) break;
        tc_commit(&bars->t_full);
        if (p.nchunks > 0) {
          if (!mbar_wait(&bars->s_ready, u & 1)) { raise_timeout(bars, p.status); ok = false; break; }
          tc_fence_after();
        }
        for (int c = 0; c < p.nchunks && ok; ++c) {
          for (int tt = 0; tt < nt && ok; ++tt) {
            const int b = (nt == 2) ? tt : (c & 1);
            if (!mbar_wait(&bars->acc_empty[b], (q[b] & 1) ^ 1)) { raise_timeout(bars, p.status); ok = false; break; }
            tc_fence_after();
            const uint32_t tacc = tmem_base + kChunk * b;
            const uint8_t* Sb = S0 + (size_t)tt * p.natoms * kAtomBytes;
            for (int j = 0; j < p.natoms; ++j) {
              const int idx = i2 + j, slot = idx % p.ns2, ph = (idx / p.ns2) & 1;
              if (!mbar_wait(&bars->full2[slot], ph)) { raise_timeout(bars, p.status); ok = false; break; }
              tc_fence_after();
              const uint64_t da = smem_desc_sw128(smem_u32(Sb + j * kAtomBytes), 16);
              const uint64_t db = smem_desc_sw128(smem_u32(ring + (size_t)slot * kAtom2Bytes), 16);
              int ksteps = (p.r - j * 64) >> 4;
              if (ksteps > 4) ksteps = 4;
              for (int kk = 0; kk < ksteps; ++kk) tc_mma_bf16(tacc, da + 2 * kk, db + 2 * kk, idesc2, (j | kk) != 0);
              if (tt == nt - 1) tc_commit(&bars->empty2[slot]);     // the last block of the unit is done with this tile
            }
            if (ok) { tc_commit(&bars->acc_full[b]); ++q[b]; }
          }
          i2 += p.natoms;
        }
        if (ok) tc_commit(&bars->unit_done);
        t += nt;
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int qw = warp & 3;                // TMEM lane quarter this warp may read
    const int row = qw * 32 + lane;
    const uint32_t lane_base = (uint32_t)(qw * 32) << 16;
    const bool issuer = (threadIdx.x == 64);
    int q[2] = {0, 0};
    int nstores = 0, u = 0;
    bool ok = true;
    for (int t = t_begin; t < t_end && ok; ++u) {
      const int nt = (t_end - t >= 2) ? 2 : 1;
      const int row0 = t * 128;
      ok = epi_wait(bars, &bars->t_full, u & 1, p.status);
      if (!ok) break;
      tc_fence_after();
      for (int tt = 0; tt < nt; ++tt) {
        uint8_t* Sb = S0 + (size_t)tt * p.natoms * kAtomBytes;
        for (int c0 = 0; c0 < p.r; c0 += 64) {
          uint32_t v[4][16];
#pragma unroll
          for (int g = 0; g < 4; ++g)
            if (c0 + g * 16 < p.r) tmem_ld16_nowait(tmem_base + 256 * tt + lane_base + c0 + g * 16, v[g]);
          tmem_wait_ld();
#pragma unroll
          for (int g = 0; g < 4; ++g)
            if (c0 + g * 16 < p.r) store_bf16x16_swizzled(Sb + (c0 >> 6) * kAtomBytes + row * 128, row, c0 + g * 16, v[g]);
        }
      }
      tc_fence_before();
      fence_proxy_async_smem();
      mbar_arrive(&bars->s_ready);
      if (p.save_s) {
        named_bar_sync(1, kEpiThreads);
        if (issuer) {
          for (int tt = 0; tt < nt; ++tt)
            for (int j = 0; j < p.natoms; ++j)
              tma_store_2d(&tmS, S0 + ((size_t)tt * p.natoms + j) * kAtomBytes, j * 64, row0 + tt * 128);
          tma_store_commit();
        }
      }
      for (int c = 0; c < p.nchunks && ok; ++c) {
        for (int tt = 0; tt < nt && ok; ++tt) {
          const int b = (nt == 2) ? tt : (c & 1);
          ok = epi_wait(bars, &bars->acc_full[b], q[b] & 1, p.status);
          if (!ok) break;
          ++q[b];
          tc_fence_after();
          const uint32_t tacc = tmem_base + kChunk * b + lane_base;
          for (int h = 0; h < kChunk / 64; ++h) {
            const int col = ((c + rot2) % p.nchunks) * kChunk + h * 64;
            const bool live = col < p.P;
            uint32_t v[4][16];
            if (live) {
#pragma unroll
              for (int g = 0; g < 4; ++g) tmem_ld16_nowait(tacc + h * 64 + g * 16, v[g]);
              tmem_wait_ld();
            }
            if (h == kChunk / 64 - 1) {
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(&bars->acc_empty[b]);
            }
            if (!live) continue;
            uint8_t* buf = stg + (nstores & 1) * kAtomBytes;
            ++nstores;
            if (issuer) tma_store_wait_read<1>();
            named_bar_sync(1, kEpiThreads);
#pragma unroll
            for (int g = 0; g < 4; ++g) store_bf16x16_swizzled(buf + row * 128, row, g * 16, v[g]);
            fence_proxy_async_smem();
            named_bar_sync(1, kEpiThreads);
            if (issuer) {
              tma_store_2d(&tmOut, buf, col, row0 + tt * 128);
              tma_store_commit();
            }
          }
        }
      }
      // every epilogue thread has passed the last barrier, so all TMEM reads of the unit are done; once
      // the stores issued so far have read their shared memory the next unit may overwrite S
      if (issuer && ok) {
        tma_store_wait_read<0>();
        mbar_arrive(&bars->unit_done);
      }
      t += nt;
    }
    if (issuer) tma_store_wait_all();
  }

  // ------------------------------------------------------------ common exit
  tc_fence_before();
  __syncthreads();
  if (*reinterpret_cast<volatile int*>(&bars->abort_any)) {
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) { }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---------------------------------------------------------------------------------------------
// grad kernel: partial[slice][p][j] = sum_{k in slice} act[k][p] * small[k][j]
struct GradJob {
  int P;          // columns of act = rows of the output
  int chunks;     // ceil(P / 256)
  float* partial; // [slices][P][r]
};
struct GradParams {
  GradJob job[2];
  int njobs;
  int r, natoms, ns, slot_bytes;
  int slices, rows_per_slice;   // rows_per_slice is a multiple of 64
  int N;
  int clear_status;
  int job0_independent;   // 1: job 0 reads nothing the kernel before this one in the stream writes (see grad_kernel)
  int* status;
};

__global__ void __launch_bounds__(192, 1)
grad_kernel(const __grid_constant__ CUtensorMap tmAct0, const __grid_constant__ CUtensorMap tmSmall0,
            const __grid_constant__ CUtensorMap tmAct1, const __grid_constant__ CUtensorMap tmSmall1,
            const GradParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* ring = smem;
  Bars* bars = reinterpret_cast<Bars*>(ring + (size_t)p.ns * p.slot_bytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // which job, which 128-row chunk of its output, which slice of the N rows
  int tile = blockIdx.x;
  const int slice = tile % p.slices;
  tile /= p.slices;
  int jb = 0;
  if (tile >= p.job[0].chunks) { jb = 1; tile -= p.job[0].chunks; }
  const int chunk = tile;
  const CUtensorMap* tmAct = jb ? &tmAct1 : &tmAct0;
  const CUtensorMap* tmSmall = jb ? &tmSmall1 : &tmSmall0;
  const int k_begin = slice * p.rows_per_slice;
  int k_end = k_begin + p.rows_per_slice;
  if (k_end > p.N) k_end = p.N;
  const int nk = k_end > k_begin ? (k_end - k_begin + 63) / 64 : 0;

  if (threadIdx.x == 0) {
    for (int i = 0; i < p.ns; ++i) { mbar_init(&bars->full[i], 1); mbar_init(&bars->empty[i], 1); }
    mbar_init(&bars->t_full, 1);
    bars->abort_any = 0;
    bars->epi_abort = 0;
    fence_barrier_init();
    tma_prefetch_desc(tmAct); tma_prefetch_desc(tmSmall);
  }
  if (warp == 1) tmem_alloc(&bars->tmem_base, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&bars->tmem_base);
  // In a full backward the kernel before this one is the dT/dX chain, which writes dT and dX: the dB
  // job reads dT and has to wait for it, the dA job reads only dY and T.  This kernel becomes resident
  // only after every CTA of the chain kernel has passed its own dep_wait, i.e. after everything
  // earlier in the stream (T included) is complete, so the dA CTAs start at once on the SMs that the
  // chain kernel's short CTAs have already left (its last third runs on two thirds of the SMs).
  if (!(p.job0_independent && jb == 0)) dep_wait();
  dep_launch();
  clear_status_word(p.clear_status, p.status);

  if (warp == 0) {
    if (lane == 0) {
      for (int i = 0; i < nk; ++i) {
        const int slot = i % p.ns, ph = (i / p.ns) & 1;
        if (!mbar_wait(&bars->empty[slot], ph ^ 1)) { raise_timeout(bars, p.status); break; }
        uint8_t* dst = ring + (size_t)slot * p.slot_bytes;
        const int k0 = k_begin + i * 64;
        // two 128-row accumulators share every slab of `small`: four 64-wide boxes of act, then small
        mbar_arrive_expect_tx(&bars->full[slot], (4 + p.natoms) * 8192);
        for (int a = 0; a < 4; ++a) tma_load_2d(dst + a * 8192, tmAct, &bars->full[slot], chunk * 256 + a * 64, k0);
        for (int a = 0; a < p.natoms; ++a)
          tma_load_2d(dst + 32768 + a * 8192, tmSmall, &bars->full[slot], a * 64, k0);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = instr_desc_bf16(128, p.r, 1, 1);
      bool ok = true;
      for (int i = 0; i < nk; ++i) {
        const int slot = i % p.ns, ph = (i / p.ns) & 1;
        if (!mbar_wait(&bars->full[slot], ph)) { raise_timeout(bars, p.status); ok = false; break; }
        tc_fence_after();
        const uint32_t sa = smem_u32(ring + (size_t)slot * p.slot_bytes);
        for (int kk = 0; kk < 4; ++kk) {
          const uint64_t db = smem_desc_sw128(sa + 32768 + kk * 2048, 8192);
          tc_mma_bf16(tmem_base, smem_desc_sw128(sa + kk * 2048, 8192), db, idesc, (i | kk) != 0);
          tc_mma_bf16(tmem_base + 256, smem_desc_sw128(sa + 16384 + kk * 2048, 8192), db, idesc, (i | kk) != 0);
        }
        tc_commit(&bars->empty[slot]);
      }
      if (ok) tc_commit(&bars->t_full);
    }
  } else {
    const int q = warp & 3;
    const int row = q * 32 + lane;
    const uint32_t lane_base = (uint32_t)(q * 32) << 16;
    const GradJob& job = p.job[jb];
    bool ok = true;
    if (nk > 0) ok = epi_wait(bars, &bars->t_full, 0, p.status);
    if (ok) {
      tc_fence_after();
      for (int mt = 0; mt < 2; ++mt) {
        const int prow = chunk * 256 + mt * 128 + row;
        float* out = job.partial + ((size_t)slice * job.P + prow) * p.r;
        for (int c0 = 0; c0 < p.r; c0 += 16) {
          float v[16];
          if (nk > 0) tmem_ld16(tmem_base + mt * 256 + lane_base + c0, v);
          else {
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = 0.f;
          }
          if (prow < job.P) {
            float4* o = reinterpret_cast<float4*>(out + c0);
            o[0] = make_float4(v[0], v[1], v[2], v[3]);
            o[1] = make_float4(v[4], v[5], v[6], v[7]);
            o[2] = make_float4(v[8], v[9], v[10], v[11]);
            o[3] = make_float4(v[12], v[13], v[14], v[15]);
          }
        }
      }
    }
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
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// Sums the per-slice partials in ascending slice order (fixed order: identical bits every run).
//   blocks [0, nA):  dA[p][j]  = sum_s pA[s][p][j]            (float4 per thread)
//   blocks [nA, ..): dB[j][q]  = sum_s pB[s][q][j]            (32 x 32 tiles transposed through shared memory)
__global__ void __launch_bounds__(256)
reduce_partials_kernel(const float* __restrict__ pA, float* __restrict__ dA, int PA, int nA,
                       const float* __restrict__ pB, float* __restrict__ dB, int PB, int slices, int r, int rp) {
  // r: columns of the results; rp: row length of the partials (r rounded up to 16)
  dep_wait();
  dep_launch();
  if ((int)blockIdx.x < nA) {
    const int64_t total4 = (int64_t)PA * r / 4;
    const int64_t i4 = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (i4 >= total4) return;
    const int64_t prow = (i4 * 4) / r;
    const int col = (int)((i4 * 4) % r);
    const float* src = pA + prow * rp + col;
    const int64_t slice_stride = (int64_t)PA * rp;
    float4 acc = *reinterpret_cast<const float4*>(src);
#pragma unroll 4
    for (int s = 1; s < slices; ++s) {
      const float4 v = *reinterpret_cast<const float4*>(src + s * slice_stride);
      acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    reinterpret_cast<float4*>(dA)[i4] = acc;
    return;
  }
  __shared__ float tile[32][33];
  const int t = blockIdx.x - nA;
  const int tiles_j = (r + 31) / 32;
  const int q0 = (t / tiles_j) * 32, j0 = (t % tiles_j) * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int i = ty; i < 32; i += 8) {
    const int q = q0 + i, j = j0 + tx;
    float acc = 0.f;
    if (q < PB && j < r)
#pragma unroll 4
      for (int s = 0; s < slices; ++s) acc += pB[((int64_t)s * PB + q) * rp + j];
    tile[i][tx] = acc;
  }
  __syncthreads();
  for (int i = ty; i < 32; i += 8) {
    const int j = j0 + i, q = q0 + tx;
    if (j < r && q < PB) dB[(int64_t)j * PB + q] = tile[tx][i];
  }
}

// Both factor transposes of a backward call in one launch: At[j][i] = A[i][j] (A is m x r, row stride
// ldA) for blocks [0, nA), Bt[j][i] = B[i][j] (B is r x n, row stride ldB) after that.
__global__ void transpose_factors_kernel(const bf16* __restrict__ A, int m, int r, int ldA, bf16* __restrict__ At, int nA,
                                         const bf16* __restrict__ B, int n, int ldB, bf16* __restrict__ Bt,
                                         int* status_to_clear) {
  __shared__ bf16 tile[32][33];
  dep_wait();
  dep_launch();
  clear_status_word(status_to_clear != nullptr, status_to_clear);
  const bool first = (int)blockIdx.x < nA;
  const bf16* src = first ? A : B;
  bf16* dst = first ? At : Bt;
  const int rows = first ? m : r, cols = first ? r : n, ld = first ? ldA : ldB;
  const int t = first ? blockIdx.x : blockIdx.x - nA;
  const int tiles_c = (cols + 31) / 32;
  const int by = (t / tiles_c) * 32, bx = (t % tiles_c) * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int i = ty; i < 32; i += 8) {
    const int rr = by + i, cc = bx + tx;
    tile[i][tx] = (rr < rows && cc < cols) ? src[(size_t)rr * ld + cc] : __float2bfloat16(0.f);
  }
  __syncthreads();
  for (int i = ty; i < 32; i += 8) {
    const int cc = bx + i, rr = by + tx;
    if (cc < cols && rr < rows) dst[(size_t)cc * rows + rr] = tile[tx][i];
  }
}

// Self-test of the bounded wait every pipeline stage of the kernels above relies on: one thread waits on
// an mbarrier that nobody ever arrives at.  The wait gives up after limit_ns and the kernel reports
// AB_ERR_TIMEOUT through the status word, exactly as the chain kernels do; nothing spins for ever and the
// context stays usable.
__global__ void bounded_wait_selftest_kernel(int* status, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    fence_barrier_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) *status = mbar_wait(&bar, 0, limit_ns) ? (int)AB_OK : (int)AB_ERR_TIMEOUT;
}

// ---------------------------------------------------------------------------------------------
// host side
// Launch with programmatic stream serialisation (see dep_wait): only for kernels that call dep_wait()
// before their first access to global memory.
template <typename... KArgs, typename... Args>
cudaError_t launch_dep(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
#define AB_LAUNCH_DEP(...)                         \
  do {                                             \
    if (launch_dep(__VA_ARGS__) != cudaSuccess) {  \
      cudaGetLastError();                          \
      return AB_ERR_CUDA;                          \
    }                                              \
  } while (0)

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

bool device_is_sm100() {
  static std::mutex mu;
  static int cache[64];
  static bool init = false;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
  std::lock_guard<std::mutex> lock(mu);
  if (!init) { for (int i = 0; i < 64; ++i) cache[i] = -1; init = true; }
  if (cache[dev] < 0) {
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return false;
    cache[dev] = (major == 10) ? 1 : 0;
  }
  return cache[dev] == 1;
}

// bf16 matrix [rows x cols], row stride ld elements, box of box_cols x box_rows, 128-byte swizzle
int make_map(CUtensorMap* m, const void* ptr, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_cols,
             uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return AB_ERR_CUDA;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {ld * 2};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult rc = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? AB_OK : AB_ERR_CUDA;
}

struct RowPlan { int natoms, ns, slot_bytes, ns2; size_t smem; };
// Ranks that are multiples of 8 but not of 16 run as the next multiple of 16: the tensor maps keep the
// true extents, so the extra rows / columns of every factor tile arrive as zeros.
int pad16(int r) { return (r + 15) & ~15; }

RowPlan row_plan(int r) {      // r: padded rank
  RowPlan pl;
  pl.natoms = (r + 63) / 64;
  pl.slot_bytes = kAtomBytes + r * 128;
  const int fixed = pl.natoms * kAtomBytes + 2 * kAtomBytes + (int)sizeof(Bars) + 1024;
  pl.ns = (kSmemLimit - fixed) / pl.slot_bytes;
  if (pl.ns > kMaxStages) pl.ns = kMaxStages;
  pl.smem = (size_t)fixed + (size_t)pl.ns * pl.slot_bytes;
  pl.ns2 = pl.ns * pl.slot_bytes / kAtom2Bytes;
  if (pl.ns2 > kMaxStages2) pl.ns2 = kMaxStages2;
  return pl;
}

struct UnitPlan { int natoms, ns, slot_bytes, ns2, ring2_bytes; size_t smem; bool ok; };
UnitPlan unit_plan(int r) {    // r: padded rank
  UnitPlan pl;
  pl.natoms = (r + 63) / 64;
  pl.slot_bytes = 2 * kAtomBytes + r * 128;
  const int fixed = 2 * pl.natoms * kAtomBytes + 2 * kAtomBytes + (int)sizeof(Bars) + 1024;
  pl.ns2 = (kSmemLimit - fixed) / kAtom2Bytes;
  if (pl.ns2 > kMaxStages2) pl.ns2 = kMaxStages2;
  pl.ring2_bytes = pl.ns2 > 0 ? pl.ns2 * kAtom2Bytes : 0;
  pl.ns = (pl.ring2_bytes + 2 * pl.natoms * kAtomBytes) / pl.slot_bytes;
  if (pl.ns > kMaxStages) pl.ns = kMaxStages;
  pl.smem = (size_t)fixed + (size_t)pl.ring2_bytes;
  pl.ok = pl.ns2 >= pl.natoms && pl.ns2 >= 2 && pl.ns >= 2;
  return pl;
}

struct GradPlan { int natoms, ns, slot_bytes, slices, rows_per_slice; size_t smem; };
GradPlan grad_plan(int64_t N, int m, int n, int r) {
  GradPlan pl;
  pl.natoms = (r + 63) / 64;
  pl.slot_bytes = 32768 + pl.natoms * 8192;
  const int fixed = (int)sizeof(Bars) + 1024;
  pl.ns = (kSmemLimit - fixed) / pl.slot_bytes;
  if (pl.ns > kMaxStages) pl.ns = kMaxStages;
  pl.smem = (size_t)fixed + (size_t)pl.ns * pl.slot_bytes;
  const int tiles = (m + 255) / 256 + (n + 255) / 256;
  int slices = (sm_count() > 0 ? sm_count() : 1) / tiles;   // one wave of CTAs
  if (slices < 1) slices = 1;
  const int64_t slabs = (N + 63) / 64;
  if (slices > slabs) slices = (int)slabs;
  int64_t per = (slabs + slices - 1) / slices;
  pl.rows_per_slice = (int)(per * 64);
  pl.slices = (int)((slabs + per - 1) / per);
  return pl;
}

struct BwdWs { int* status; bf16 *At, *Bt, *T, *dT; float *pA, *pB; size_t bytes; };
BwdWs bwd_ws(void* ws, int64_t N, int m, int n, int r) {
  GradPlan gp = grad_plan(N, m, n, r);
  Arena ar(ws, 0);
  BwdWs w;
  w.status = ar.take_n<int>(64);
  w.At = ar.take_n<bf16>((size_t)r * m);
  w.Bt = ar.take_n<bf16>((size_t)n * r);
  w.T = ar.take_n<bf16>((size_t)N * r);
  w.dT = ar.take_n<bf16>((size_t)N * r);
  w.pA = ar.take_n<float>((size_t)gp.slices * m * pad16(r));
  w.pB = ar.take_n<float>((size_t)gp.slices * n * pad16(r));
  w.bytes = align_up(ar.used, 256);
  return w;
}

// S = In F1^T (saved to Sg if not null), Out = S F2^T (skipped if Out is null)
int launch_row_chain(const void* In, int64_t N, int K1, const void* F1, int ldF1, const void* F2, int ldF2, int P,
                     void* Out, void* Sg, int r, int* status, bool clear_status, cudaStream_t st) {
  const int rp = pad16(r);
  RowPlan pl = row_plan(rp);
  if (pl.ns < 2 || pl.ns2 < 2) return AB_ERR_UNSUPPORTED;
  CUtensorMap tmIn, tmF1, tmF2, tmOut, tmS;
  AB_TRY(make_map(&tmIn, In, (uint64_t)N, K1, K1, 64, 128));
  AB_TRY(make_map(&tmF1, F1, r, K1, ldF1, 64, rp));
  const bool second = Out != nullptr && P > 0;
  // unused maps still have to be valid objects: alias them to the first operand
  if (second) {
    AB_TRY(make_map(&tmF2, F2, P, r, ldF2, 64, kChunk));
    AB_TRY(make_map(&tmOut, Out, (uint64_t)N, P, P, 64, 128));
  } else {
    tmF2 = tmIn;
    tmOut = tmIn;
  }
  if (Sg) AB_TRY(make_map(&tmS, Sg, (uint64_t)N, r, r, 64, 128));
  else tmS = tmIn;
  // More row blocks than SMs: persistent CTAs that take two blocks at a time and load each factor
  // tile once for both.
  {
    const int64_t tiles = (N + 127) / 128;
    const int sms = sm_count();
    const UnitPlan up = unit_plan(rp);
    if (second && sms > 0 && tiles > sms && up.ok) {
      UnitParams q;
      q.K1 = K1; q.P = P; q.r = rp; q.nk1 = (K1 + 63) / 64; q.nchunks = (P + kChunk - 1) / kChunk; q.natoms = up.natoms;
      q.ns = up.ns; q.slot_bytes = up.slot_bytes; q.ns2 = up.ns2; q.ring2_bytes = up.ring2_bytes;
      q.save_s = Sg ? 1 : 0; q.tiles = (int)tiles; q.clear_status = clear_status ? 1 : 0; q.status = status;
      AB_CUDA_OK(cudaFuncSetAttribute(row_chain_units_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)up.smem));
      AB_LAUNCH_DEP(row_chain_units_kernel, dim3((unsigned)sms), dim3(192), up.smem, st, tmIn, tmF1, tmF2, tmOut, tmS, q);
      AB_LAUNCH_OK();
      return AB_OK;
    }
  }
  RowChainParams p;
  p.K1 = K1; p.P = second ? P : 0; p.r = rp; p.nk1 = (K1 + 63) / 64; p.nchunks = second ? (P + kChunk - 1) / kChunk : 0;
  p.natoms = pl.natoms; p.ns = pl.ns; p.slot_bytes = pl.slot_bytes; p.ns2 = pl.ns2; p.save_s = Sg ? 1 : 0;
  p.clear_status = clear_status ? 1 : 0;
  p.status = status;
  AB_CUDA_OK(cudaFuncSetAttribute(row_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem));
  const unsigned grid = (unsigned)((N + 127) / 128);
  AB_LAUNCH_DEP(row_chain_kernel, dim3(grid), dim3(192), pl.smem, st, tmIn, tmF1, tmF2, tmOut, tmS, p);
  AB_LAUNCH_OK();
  return AB_OK;
}

}  // namespace

int bounded_wait_selftest(int* dev_status, unsigned limit_us, cudaStream_t st) {
  bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(dev_status, (unsigned long long)limit_us * 1000ull);
  AB_LAUNCH_OK();
  return AB_OK;
}

bool chain_tc_supported(int64_t N, int m, int n, int r, int ldA, int ldB, int dt,
                        const void* x, const void* A, const void* B, const void* y) {
  if (dt != AB_BF16) return false;
  if (r % 8 != 0 || r < 8 || r > 256) return false;
  if (m % 8 != 0 || n % 8 != 0 || ldA % 8 != 0 || ldB % 8 != 0) return false;
  if (N > (int64_t)1 << 30) return false;
  if (!aligned(x, 16) || !aligned(A, 16) || !aligned(B, 16) || !aligned(y, 16)) return false;
  if (!device_is_sm100() || !encode_fn()) return false;
  return row_plan(pad16(r)).ns >= 2 && row_plan(pad16(r)).ns2 >= 2;
}

size_t chain_tc_forward_ws(int64_t, int, int, int) { return 256; }
size_t chain_tc_backward_ws(int64_t N, int m, int n, int r) {
  if (r % 8 != 0 || r < 8 || r > 256) return 0;
  return bwd_ws(nullptr, N, m, n, r).bytes;
}

int chain_tc_forward(const void* x, const void* A, const void* B, void* y, void* T_save,
                     int64_t N, int m, int n, int r, int ldA, int ldB,
                     void* ws, size_t ws_bytes, cudaStream_t st) {
  if (!ws || ws_bytes < 256) return AB_ERR_WORKSPACE;
  if (T_save && !aligned(T_save, 16)) return AB_ERR_INVALID_ARG;
  int* status = static_cast<int*>(ws);
  return launch_row_chain(x, N, n, B, ldB, A, ldA, m, y, T_save, r, status, true, st);
}

int chain_tc_backward(const void* x, const void* dY, const void* A, const void* B,
                      const void* T_saved, void* dX, float* dA, float* dB,
                      int64_t N, int m, int n, int r, int ldA, int ldB,
                      void* ws, size_t ws_bytes, cudaStream_t st) {
  if (!ws) return AB_ERR_WORKSPACE;
  BwdWs w = bwd_ws(ws, N, m, n, r);
  if (w.bytes > ws_bytes) return AB_ERR_WORKSPACE;
  if ((dX && !aligned(dX, 16)) || (T_saved && !aligned(T_saved, 16)) || (dA && !aligned(dA, 16)) ||
      (dB && !aligned(dB, 16)))
    return AB_ERR_INVALID_ARG;
  bool first = true;     // the first kernel of the call zeroes the status word
  bool after_chain = false;   // the dT/dX chain kernel is the launch right before the gradient kernel
  const bf16* T = static_cast<const bf16*>(T_saved);
  if (dA && !T) {   // recompute T = x B^T (first product only)
    AB_TRY(launch_row_chain(x, N, n, B, ldB, nullptr, 0, 0, nullptr, w.T, r, w.status, first, st));
    first = false;
    T = w.T;
  }
  if (dX || dB) {
    {
      const int nA = ((m + 31) / 32) * ((r + 31) / 32);
      const int nB = dX ? ((r + 31) / 32) * ((n + 31) / 32) : 0;
      AB_LAUNCH_DEP(transpose_factors_kernel, dim3(nA + nB), dim3(256), 0, st, static_cast<const bf16*>(A), m, r, ldA, w.At,
                 nA, static_cast<const bf16*>(B), n, ldB, w.Bt, first ? w.status : static_cast<int*>(nullptr));
      AB_LAUNCH_OK();
      first = false;
    }
    // dT = dY A (kept for dB), dX = dT B
    AB_TRY(launch_row_chain(dY, N, m, w.At, m, w.Bt, r, n, dX, dB ? w.dT : nullptr, r, w.status, false, st));
    after_chain = true;
  }
  if (dA || dB) {
    GradPlan gp = grad_plan(N, m, n, r);
    const int rp = pad16(r);
    GradParams p;
    CUtensorMap tmAct[2], tmSmall[2];
    int nj = 0;
    if (dA) {
      AB_TRY(make_map(&tmAct[nj], dY, (uint64_t)N, m, m, 64, 64));
      AB_TRY(make_map(&tmSmall[nj], T, (uint64_t)N, r, r, 64, 64));
      p.job[nj].P = m; p.job[nj].chunks = (m + 255) / 256; p.job[nj].partial = w.pA;
      ++nj;
    }
    if (dB) {
      AB_TRY(make_map(&tmAct[nj], x, (uint64_t)N, n, n, 64, 64));
      AB_TRY(make_map(&tmSmall[nj], w.dT, (uint64_t)N, r, r, 64, 64));
      p.job[nj].P = n; p.job[nj].chunks = (n + 255) / 256; p.job[nj].partial = w.pB;
      ++nj;
    }
    if (nj == 1) { tmAct[1] = tmAct[0]; tmSmall[1] = tmSmall[0]; p.job[1] = p.job[0]; p.job[1].chunks = 0; }
    p.njobs = nj; p.r = rp; p.natoms = gp.natoms; p.ns = gp.ns; p.slot_bytes = gp.slot_bytes;
    p.slices = gp.slices; p.rows_per_slice = gp.rows_per_slice; p.N = (int)N; p.clear_status = first ? 1 : 0; p.status = w.status;
    p.job0_independent = (after_chain && dA) ? 1 : 0;   // job 0 is the dA job whenever dA is asked for
    AB_CUDA_OK(cudaFuncSetAttribute(grad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gp.smem));
    const unsigned grid = (unsigned)((p.job[0].chunks + p.job[1].chunks) * gp.slices);
    AB_LAUNCH_DEP(grad_kernel, dim3(grid), dim3(192), gp.smem, st, tmAct[0], tmSmall[0], tmAct[1], tmSmall[1], p);
    AB_LAUNCH_OK();
    {
      const int nA = dA ? (int)(((int64_t)m * r / 4 + 255) / 256) : 0;
      const int nB = dB ? ((n + 31) / 32) * ((r + 31) / 32) : 0;
      AB_LAUNCH_DEP(reduce_partials_kernel, dim3(nA + nB), dim3(256), 0, st, static_cast<const float*>(w.pA), dA, m, nA,
                 static_cast<const float*>(w.pB), dB, n, gp.slices, r, rp);
      AB_LAUNCH_OK();
    }
    first = false;
  }
  if (first) AB_CUDA_OK(cudaMemsetAsync(w.status, 0, sizeof(int), st));   // nothing was asked for
  return AB_OK;
}

}  // namespace ab
