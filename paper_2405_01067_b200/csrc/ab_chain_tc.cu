// Fused tensor-core chain for bf16 storage (fp32 accumulation) on sm_100a.
//
// chain_kernel: persistent CTAs; for a block of 128 rows  S = In F1^T  (128 x r, K-loop over the input
// width, accumulator in TMEM), S rounded to bf16 into shared memory, multiplied on:  Out = S F2^T  in
// 256-column chunks.  The rank-r intermediate never goes to HBM unless the caller asks for a copy.
//   forward : In = x,  F1 = B   (r x n), F2 = A   (m x r), Out = y,  S = T
//   backward: In = dY, F1 = A^T (r x m), F2 = B^T (n x r), Out = dX, S = dT   (A and B read as they lie)
// grad_kernel: dA = dY^T T and dB^T = x^T dT are reductions over the rows; a CTA owns 256 output rows (a
// slice of m or of n) and one slice of the N rows, streams 64-row slabs of both operands (both
// "MN-major": the reduction index is the slow one in memory) and leaves an fp32 partial;
// reduce_partials_kernel adds the partials in ascending slice order.
//
// All operand tiles are TMA boxes of 64 bf16 (128 bytes) x rows with 128-byte swizzle.  Every mbarrier
// wait gives up after about a second, raises AB_ERR_TIMEOUT in the status word and unwinds to the common
// exit, where TMEM is released.
#include <cstring>
#include <mutex>

#include "ab_common.cuh"
#include "ab_tc_ptx.cuh"

namespace ab {
namespace {

using namespace tc;

constexpr int kAtomBytes = 16384;      // 128 rows x 128 bytes
constexpr int kMaxStages = 10;
constexpr int kMaxStages2 = 6;         // 32 KB slots of the second product, carved from the same ring memory
constexpr int kChunk = 256;            // output columns per accumulator of the second product
constexpr int kAtom2Bytes = kChunk * 128;   // one 256 x 64 tile of F2
constexpr int kSmemLimit = 227 * 1024;
constexpr int kTmemCols = 512;
constexpr int kEpiThreads = 128;

constexpr int kEpiWarps = 4;                         // 4 or 8: one or two warps per quarter of the TMEM lanes
constexpr int kWarpsPerQuarter = kEpiWarps / 4;
constexpr int kPiecesPerWarp = 4 / kWarpsPerQuarter;  // 64-column pieces of a 256-column chunk per warp
constexpr int kStgTiles = 2;                         // staging tiles per epilogue warp
constexpr int kChainThreads = 32 * (2 + kEpiWarps);
constexpr int kGroupRows = 32;                   // rows are dealt to CTAs, loaded and stored in groups of 32
constexpr int kGroupBytes = kGroupRows * 128;    // one group of one 64-column tile
constexpr int kF1AtomBytes = 8192;               // 64 x 64 box of an MN-major factor

// Convolution mode (3 x 3, stride 1, padding 1, activations NHWC): the rows of In are never materialised.  A
// block is a tile of whole image rows (bh rows of one image, or bb whole images when an image has at most 128
// pixels), i.e. a run of consecutive pixels; slab kr of the reduction is tap kr / cslabs and 64 channels, and the
// block's In tile for it is the 4-D box of the activation shifted by the tap (what falls outside an image
// arrives as zeros: the padding).  The factor's slab is found at column tap * tap_stride (+ f1_col_off).
struct ConvGeom {
  int on;
  int B, H, W;
  int in_ch;       // channels of the In tensor
  int cslabs;      // ceil(in_ch / 64)
  int bh, bb;      // tile: bh image rows (bb == 1) or bb whole images (bh == H)
  int tpi;         // tiles per image (bb == 1) or 1
  int box_rows;    // W * bh * bb: rows one In box delivers
  int sign;        // +1: In pixel = out pixel + (tap - 1); -1: In pixel = out pixel - (tap - 1)
  int tap_stride;  // columns of the factor between taps
  int f1_col_off;  // first column of this launch's factor window inside a tap
  int s_col_off;   // first column of S in the output it is stored to
};

struct ChainParams {
  int K1;        // width of In (reduction length of the first product)
  int P;         // width of Out (0: first product only)
  int r;         // rank, padded to a multiple of 16
  int nk1;       // ceil(K1 / 64)
  int nchunks;   // ceil(P / 256)
  int natoms;    // ceil(r / 64)
  int max_blocks;          // 128-row blocks per unit: 1 or 2
  int ns, slot_bytes;      // first product: slots of max_blocks In tiles + one slab of F1
  int ns2;                 // second product: 32 KB slots at the start of shared memory
  int f1_bytes;            // bytes of one F1 slab as the loads deliver it
  int f1_mn, f2_mn;        // 1: the factor is held with the reduction index as the slow one (MN-major operand)
  int save_s;              // 1: copy S to global through tmS
  int groups;              // work items in all: 32-row groups, or tiles of a convolution (see ConvGeom)
  int deal;                // items are dealt to the CTAs in runs of this many
  ConvGeom cv;
  bf16* out_ptr;           // convolution mode: Out and S as plain pointers for the rows of a tile's last, partial
  bf16* s_ptr;             //   group of 32 (row strides P and s_ld)
  int s_ld, s_cols;        // s_cols: true width of S
  int clear_status;        // 1: this is the first kernel of a call and zeroes the status word (see clear_status_word)
  int stall_selftest;      // 1: the producer loads nothing, so every wait of the kernel runs out (failure-path self-test)
  unsigned long long wait_ns;   // limit of every on-chip wait
  int* status;
};

struct Bars {
  uint64_t full[kMaxStages], empty[kMaxStages];
  uint64_t full2[kMaxStages2], empty2[kMaxStages2];
  uint64_t t_full, s_ready, unit_done;
  uint64_t acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  int abort_any;   // set by any role that gave up
  int epi_abort;   // used by the gradient kernel's epilogue warps around their own barrier
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

// epilogue-wide wait of the gradient kernel: every epilogue thread calls it; the verdict is uniform
__device__ __forceinline__ bool epi_wait(Bars* b, uint64_t* bar, uint32_t parity, int* status) {
  if (!mbar_wait(bar, parity)) {
    *reinterpret_cast<volatile int*>(&b->epi_abort) = 1;
    raise_timeout(b, status);
  }
  named_bar_sync(1, kEpiThreads);
  return *reinterpret_cast<volatile int*>(&b->epi_abort) == 0;
}

// one warp waits; the verdict is uniform over the warp
__device__ __forceinline__ bool warp_wait(Bars* b, uint64_t* bar, uint32_t parity, unsigned long long limit, int* status) {
  int ok = 1;
  if ((threadIdx.x & 31) == 0) {          // one lane polls; the others rest at the shuffle
    ok = mbar_wait(bar, parity, limit) ? 1 : 0;
    if (!ok) raise_timeout(b, status);
  }
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

__device__ __forceinline__ void store_bf16x16_swizzled(uint8_t* row_base, int row, int c0, const uint32_t* v) {
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

// One unit of a CTA's run: up to two blocks, each with its first row, its count of valid rows and (convolution
// mode) the image and image row its tile starts at.
struct Unit { int nt, adv; int row0[2], nrows[2], b0[2], y0[2]; };
__device__ __forceinline__ Unit make_unit(const ChainParams& p, int it, int it_end) {
  Unit u;
  if (!p.cv.on) {
    const int cap = 4 * p.max_blocks;
    const int ng = (it_end - it < cap) ? it_end - it : cap;
    u.nt = ng > 4 ? 2 : 1;
    u.adv = ng;
    u.row0[0] = it * kGroupRows; u.row0[1] = u.row0[0] + 128;
    u.nrows[0] = (ng < 4 ? ng : 4) * kGroupRows; u.nrows[1] = (ng - 4) * kGroupRows;
    u.b0[0] = u.b0[1] = u.y0[0] = u.y0[1] = 0;
  } else {
    u.nt = (it_end - it < p.max_blocks) ? it_end - it : p.max_blocks;
    u.adv = u.nt;
    for (int tt = 0; tt < 2; ++tt) {
      const int t = it + tt;
      const int grp = t / p.cv.tpi, ty = t - grp * p.cv.tpi;
      u.b0[tt] = grp * p.cv.bb;
      u.y0[tt] = ty * p.cv.bh;
      u.row0[tt] = (u.b0[tt] * p.cv.H + u.y0[tt]) * p.cv.W;
      int nb = p.cv.B - u.b0[tt]; if (nb > p.cv.bb) nb = p.cv.bb;
      int nh = p.cv.H - u.y0[tt]; if (nh > p.cv.bh) nh = p.cv.bh;
      u.nrows[tt] = nb * nh * p.cv.W;
    }
  }
  return u;
}

// The rows of a partial group (fewer than 32) of a staged 32 x 64 tile go out with plain 16-byte stores.
__device__ __forceinline__ void store_partial_group(const uint8_t* buf, bf16* dst, int64_t ld, int rows, int cols_left) {
  const int lane = threadIdx.x & 31;
  for (int idx = lane; idx < rows * 8; idx += 32) {
    const int rr = idx >> 3, ch = idx & 7;
    if (ch * 8 >= cols_left) continue;
    const uint4 v = *reinterpret_cast<const uint4*>(buf + rr * 128 + ((ch ^ (rr & 7)) << 4));
    *reinterpret_cast<uint4*>(dst + (int64_t)rr * ld + ch * 8) = v;
  }
}

// ---------------------------------------------------------------------------------------------
// chain_kernel:  S = In F1^T (rows x r, accumulated in TMEM over the width of In), S rounded to bf16 into
// shared memory, Out = S F2^T in 256-column chunks, stored as bf16.  One persistent CTA per SM.
//
// Rows.  The rows are cut into groups of 32 and every CTA owns a contiguous run of groups, as equal as the
// group count allows, so the CTAs finish together whatever the row count is.  A CTA works through its run
// in units of up to two blocks of 128 rows (one block when max_blocks == 1).  Both blocks of a unit share
// every factor tile that is loaded -- each slab of F1 feeds two first-product MMAs, each tile of F2 two
// second-product MMAs -- so a row costs half the factor bytes from L2.  A block at the end of a run may
// hold fewer than four groups: only its groups are stored; the block is loaded and multiplied whole (rows are
// independent in every product, and the rows past the run are never stored).
//
// Warps (192 threads): 0 = TMA producer, 1 = MMA issuer and TMEM owner, 2..5 = epilogue.  An epilogue
// warp may read the quarter of the TMEM lanes given by its index modulo 4, i.e. the 32 rows of one group.
// Each warp converts its 32 x 64 pieces into staging tiles of its own (two, used in turn) and stores them
// with TMA stores of its own: no barrier spans the epilogue warps.  (Measured: two warps per quarter with
// one staging tile each are slower, 129 against 110 us for a ViT forward; more pollers, no more overlap.)
//
// TMEM: block b of a unit keeps its S accumulator at column 256 b while the first product runs; the
// accumulators of the second product take the same columns afterwards (in a two-block unit accumulator b
// belongs to block b; in a one-block unit the two alternate between chunks).
//
// Factors.  F1 is r x K1 and F2 is P x r as operands.  Either may be given as it lies in memory (K-major:
// the reduction index is the fast one -- B and A in the forward pass) or transposed (MN-major: the
// reduction index is the slow one -- A and B in the backward pass, where F1 = A^T and F2 = B^T), which the
// shared-memory descriptors of the MMAs express directly; nothing is transposed in memory.
__global__ void __launch_bounds__(kChainThreads, 1)
chain_kernel(const __grid_constant__ CUtensorMap tmIn, const __grid_constant__ CUtensorMap tmIn4,
             const __grid_constant__ CUtensorMap tmF1, const __grid_constant__ CUtensorMap tmF2,
             const __grid_constant__ CUtensorMap tmOut, const __grid_constant__ CUtensorMap tmS, const ChainParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  // [ second-product ring | S of block 0 | S of block 1 | staging tiles of the epilogue warps | barriers ]; the
  // first product's ring lies over all of the first four regions, which it has to itself while it runs (the
  // staging tiles are written only after the unit's first product is complete, and a unit ends only when the
  // stores that read them are done)
  uint8_t* ring = smem;
  uint8_t* S0 = smem + (size_t)p.ns2 * kAtom2Bytes;
  uint8_t* stg = S0 + (size_t)p.max_blocks * p.natoms * kAtomBytes;
  Bars* bars = reinterpret_cast<Bars*>(stg + kEpiWarps * kStgTiles * kGroupBytes);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // items are dealt in runs of p.deal (1, or 4 = whole 128-row blocks when every CTA gets at least two blocks:
  // a block costs the same whether full or not, so whole blocks waste none, and the CTAs with one block fewer
  // leave their SMs to the kernel that follows)
  const int nruns = (p.groups + p.deal - 1) / p.deal;
  const int g_begin = (int)((int64_t)blockIdx.x * nruns / gridDim.x) * p.deal;
  int g_end = (int)((int64_t)(blockIdx.x + 1) * nruns / gridDim.x) * p.deal;
  if (g_end > p.groups) g_end = p.groups;
  // All CTAs walk the same factor tiles.  Started together they would all ask L2 for the same few lines at
  // the same moment; each CTA therefore starts its walk at a different slab / chunk and wraps round.
  const int rot1 = blockIdx.x % p.nk1;
  const int rot2 = p.nchunks > 0 ? (blockIdx.x * 5) % p.nchunks : 0;

  if (threadIdx.x == 0) {
    for (int i = 0; i < p.ns; ++i) { mbar_init(&bars->full[i], 1); mbar_init(&bars->empty[i], 1); }
    for (int i = 0; i < p.ns2; ++i) { mbar_init(&bars->full2[i], 1); mbar_init(&bars->empty2[i], 1); }
    mbar_init(&bars->t_full, 1);
    mbar_init(&bars->s_ready, kEpiWarps);
    mbar_init(&bars->unit_done, 1 + kEpiWarps);   // the MMA issuer's commit and every epilogue warp
    for (int i = 0; i < 2; ++i) { mbar_init(&bars->acc_full[i], 1); mbar_init(&bars->acc_empty[i], kEpiWarps); }
    bars->abort_any = 0;
    bars->epi_abort = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tmIn); tma_prefetch_desc(&tmIn4); tma_prefetch_desc(&tmF1); tma_prefetch_desc(&tmF2);
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
  const unsigned long long lim = p.wait_ns;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0 && !p.stall_selftest) {
      int i1 = 0, i2 = 0, u = 0;
      bool ok = true;
      for (int g = g_begin; g < g_end && ok; ++u) {
        const Unit un = make_unit(p, g, g_end);
        const int nt = un.nt;
        // the shared memory of the last unit is free once its MMAs are done and its stores have been read
        if (u > 0 && !mbar_wait(&bars->unit_done, (u - 1) & 1, lim)) { raise_timeout(bars, p.status); ok = false; break; }
        for (int ks = 0; ks < p.nk1 && ok; ++ks, ++i1) {
          const int slot = i1 % p.ns, ph = (i1 / p.ns) & 1;
          if (!mbar_wait(&bars->empty[slot], ph ^ 1, lim)) { raise_timeout(bars, p.status); ok = false; break; }
          uint8_t* dst = smem + (size_t)slot * p.slot_bytes;
          const int kr = (ks + rot1) % p.nk1;
          uint8_t* f1 = dst + p.max_blocks * kAtomBytes;
          if (!p.cv.on) {
            mbar_arrive_expect_tx(&bars->full[slot], nt * kAtomBytes + p.f1_bytes);
            // a block at the end of the run is loaded whole as well: the rows past the run are a neighbour's
            // (or zeros past the last row) and cost less than four separate 32-row loads
            for (int tt = 0; tt < nt; ++tt)
              tma_load_2d(dst + tt * kAtomBytes, &tmIn, &bars->full[slot], kr * 64, un.row0[tt]);
            if (p.f1_mn)
              for (int a = 0; a < p.natoms; ++a) tma_load_2d(f1 + a * kF1AtomBytes, &tmF1, &bars->full[slot], a * 64, kr * 64);
            else
              tma_load_2d(f1, &tmF1, &bars->full[slot], kr * 64, 0);
          } else {
            // slab kr = (tap, 64 channels): the tile's box of the activation, shifted by the tap
            const int tap = kr / p.cv.cslabs, cs = kr - tap * p.cv.cslabs;
            const int dy = (tap / 3 - 1) * p.cv.sign, dx = (tap % 3 - 1) * p.cv.sign;
            mbar_arrive_expect_tx(&bars->full[slot], nt * p.cv.box_rows * 128 + p.f1_bytes);
            for (int tt = 0; tt < nt; ++tt)
              tma_load_4d(dst + tt * kAtomBytes, &tmIn4, &bars->full[slot], cs * 64, dx, un.y0[tt] + dy, un.b0[tt]);
            const int fcol = tap * p.cv.tap_stride + p.cv.f1_col_off;
            if (p.f1_mn)
              for (int a = 0; a < p.natoms; ++a)
                tma_load_2d(f1 + a * kF1AtomBytes, &tmF1, &bars->full[slot], fcol + a * 64, cs * 64);
            else
              tma_load_2d(f1, &tmF1, &bars->full[slot], fcol + cs * 64, 0);
          }
        }
        // the second product's slots lie over the first product's: wait until its MMAs have read them
        if (ok && !mbar_wait(&bars->t_full, u & 1, lim)) { raise_timeout(bars, p.status); ok = false; }
        for (int c = 0; c < p.nchunks && ok; ++c) {
          const int col0 = ((c + rot2) % p.nchunks) * kChunk;
          for (int j = 0; j < p.natoms; ++j, ++i2) {
            const int slot = i2 % p.ns2, ph = (i2 / p.ns2) & 1;
            if (!mbar_wait(&bars->empty2[slot], ph ^ 1, lim)) { raise_timeout(bars, p.status); ok = false; break; }
            uint8_t* d = ring + (size_t)slot * kAtom2Bytes;
            mbar_arrive_expect_tx(&bars->full2[slot], kAtom2Bytes);
            if (p.f2_mn)
              for (int b = 0; b < 4; ++b) tma_load_2d(d + b * kF1AtomBytes, &tmF2, &bars->full2[slot], col0 + 64 * b, j * 64);
            else
              tma_load_2d(d, &tmF2, &bars->full2[slot], j * 64, col0);
          }
        }
        g += un.adv;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    // One thread feeds the tensor pipe; its own instruction count per MMA is kept small: the descriptors of
    // slot 0 are built once, a slot is an addition, a K step is an addition (32 bytes along a K-major row,
    // 2048 bytes -- 16 rows -- down an MN-major tile), and the four K steps are unrolled.  (Measured: a second
    // issuing thread, one per block of a unit, changes nothing -- 100.7 against 102.2 us for a ViT forward:
    // the pipe itself takes about 200 cycles per 128 x 256 x 16 MMA here.)
    if (lane == 0) {
      const uint32_t idesc1 = instr_desc_bf16(128, p.r, 0, p.f1_mn);
      const uint32_t idesc2 = instr_desc_bf16(128, kChunk, 0, p.f2_mn);
      const uint32_t s_base = smem_u32(smem);
      const uint64_t dA1 = smem_desc_sw128(s_base, 16);                          // In tile of block 0, slot 0
      const uint64_t dF1 = p.f1_mn ? smem_desc_sw128(s_base + p.max_blocks * kAtomBytes, kF1AtomBytes)
                                   : smem_desc_sw128(s_base + p.max_blocks * kAtomBytes, 16);
      const uint64_t f1_step = p.f1_mn ? (2048u >> 4) : 2u;
      const uint64_t slot_step = (uint64_t)(p.slot_bytes >> 4);
      const uint64_t dS = smem_desc_sw128(smem_u32(S0), 16);                     // S tile 0 of block 0
      const uint64_t dF2 = p.f2_mn ? smem_desc_sw128(s_base, kF1AtomBytes) : smem_desc_sw128(s_base, 16);
      const uint64_t f2_step = p.f2_mn ? (2048u >> 4) : 2u;
      const uint64_t blk_step = (uint64_t)(kAtomBytes >> 4);
      int i2 = 0, u = 0;
      int slot1 = 0, ph1 = 0;                  // first-product ring position
      int q0 = 0, q1 = 0;                      // uses of each accumulator so far
      bool ok = true;
      for (int g = g_begin; g < g_end && ok; ++u) {
        const Unit un = make_unit(p, g, g_end);
        const int nt = un.nt;
        int kr = rot1;
        for (int ks = 0; ks < p.nk1; ++ks) {
          if (!mbar_wait(&bars->full[slot1], ph1, lim)) { raise_timeout(bars, p.status); ok = false; break; }
          tc_fence_after();
          const uint64_t da0 = dA1 + slot_step * slot1, db0 = dF1 + slot_step * slot1;
          const int ksteps = p.cv.on ? (p.cv.in_ch - (kr % p.cv.cslabs) * 64 + 15) >> 4 : (p.K1 - kr * 64 + 15) >> 4;
          const uint32_t acc0 = ks != 0;
          if (nt == 2) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
              if (kk < ksteps) {
                tc_mma_bf16(tmem_base, da0 + 2 * kk, db0 + f1_step * kk, idesc1, kk ? 1u : acc0);
                tc_mma_bf16(tmem_base + 256, da0 + blk_step + 2 * kk, db0 + f1_step * kk, idesc1, kk ? 1u : acc0);
              }
            }
          } else {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
              if (kk < ksteps) tc_mma_bf16(tmem_base, da0 + 2 * kk, db0 + f1_step * kk, idesc1, kk ? 1u : acc0);
          }
          tc_commit(&bars->empty[slot1]);
          if (++slot1 == p.ns) { slot1 = 0; ph1 ^= 1; }
          if (++kr == p.nk1) kr = 0;
        }
        if (!ok) break;
        tc_commit(&bars->t_full);
        if (p.nchunks > 0) {
          if (!mbar_wait(&bars->s_ready, u & 1, lim)) { raise_timeout(bars, p.status); ok = false; break; }
          tc_fence_after();
        }
        for (int c = 0; c < p.nchunks && ok; ++c) {
          for (int tt = 0; tt < nt && ok; ++tt) {
            const int b = (nt == 2) ? tt : (c & 1);
            if (!mbar_wait(&bars->acc_empty[b], ((b ? q1 : q0) & 1) ^ 1, lim)) { raise_timeout(bars, p.status); ok = false; break; }
            tc_fence_after();
            const uint32_t tacc = tmem_base + kChunk * b;
            const uint64_t dSb = dS + blk_step * (uint64_t)(tt * p.natoms);
            for (int j = 0; j < p.natoms; ++j) {
              const int idx = i2 + j, slot = idx % p.ns2, ph = (idx / p.ns2) & 1;
              if (!mbar_wait(&bars->full2[slot], ph, lim)) { raise_timeout(bars, p.status); ok = false; break; }
              tc_fence_after();
              const uint64_t da = dSb + blk_step * j;
              const uint64_t db = dF2 + (uint64_t)(kAtom2Bytes >> 4) * slot;
              const int ksteps = (p.r - j * 64) >> 4;
              const uint32_t acc0 = j != 0;
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)
                if (kk < ksteps) tc_mma_bf16(tacc, da + 2 * kk, db + f2_step * kk, idesc2, kk ? 1u : acc0);
              if (tt == nt - 1) tc_commit(&bars->empty2[slot]);     // the last block of the unit is done with this tile
            }
            if (ok) { tc_commit(&bars->acc_full[b]); if (b) ++q1; else ++q0; }
          }
          i2 += p.natoms;
        }
        if (ok) tc_commit(&bars->unit_done);
        g += un.adv;
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..9)
    const int qw = warp & 3;                // TMEM lane quarter this warp may read = the 32-row group it serves
    const int hw = (warp - 2) >> 2;         // which of the warps of that quarter
    const int row = qw * 32 + lane;         // row of the 128-row block
    const uint32_t lane_base = (uint32_t)(qw * 32) << 16;
    uint8_t* mystg = stg + (size_t)(warp - 2) * kStgTiles * kGroupBytes;
    int nst = 0;                            // stores issued from this warp's staging tiles
    int q0 = 0, q1 = 0;
    int u = 0;
    bool ok = true;
    for (int g = g_begin; g < g_end && ok; ++u) {
      const Unit un = make_unit(p, g, g_end);
      const int nt = un.nt;
      ok = warp_wait(bars, &bars->t_full, u & 1, lim, p.status);
      if (!ok) break;
      tc_fence_after();
      // S of every block of the unit: the two warps of a quarter take alternate 64-column tiles
      for (int tt = 0; tt < nt; ++tt) {
        uint8_t* Sb = S0 + (size_t)tt * p.natoms * kAtomBytes;
        for (int j = 0; j < p.natoms; ++j) {
          if (((tt * p.natoms + j) % kWarpsPerQuarter) != hw) continue;
          const int c0 = j * 64;
          uint32_t v[4][16];
#pragma unroll
          for (int gq = 0; gq < 4; ++gq)
            if (c0 + gq * 16 < p.r) tmem_ld16_nowait(tmem_base + 256 * tt + lane_base + c0 + gq * 16, v[gq]);
          tmem_wait_ld();
#pragma unroll
          for (int gq = 0; gq < 4; ++gq)
            if (c0 + gq * 16 < p.r) store_bf16x16_swizzled(Sb + j * kAtomBytes + row * 128, row, c0 + gq * 16, v[gq]);
        }
      }
      tc_fence_before();
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->s_ready);
      if (p.save_s) {                        // this warp's tiles, this warp's 32 rows, if the block has them
        for (int tt = 0; tt < nt; ++tt) {
          const int grows = un.nrows[tt] - qw * kGroupRows;      // rows of this warp's group in the block
          if (grows <= 0) continue;
          const int grow0 = un.row0[tt] + qw * kGroupRows;
          for (int j = 0; j < p.natoms; ++j) {
            if (((tt * p.natoms + j) % kWarpsPerQuarter) != hw) continue;
            const uint8_t* src = S0 + ((size_t)tt * p.natoms + j) * kAtomBytes + qw * kGroupBytes;
            if (grows >= kGroupRows) {
              if (lane == 0) tma_store_2d(&tmS, src, j * 64 + p.cv.s_col_off, grow0);
            } else {
              store_partial_group(src, p.s_ptr + (int64_t)grow0 * p.s_ld + p.cv.s_col_off + j * 64, p.s_ld, grows,
                                  p.s_cols - j * 64);
            }
          }
        }
        if (lane == 0) tma_store_commit();
      }
      for (int c = 0; c < p.nchunks && ok; ++c) {
        const int col0 = ((c + rot2) % p.nchunks) * kChunk + hw * (64 * kPiecesPerWarp);
        for (int tt = 0; tt < nt && ok; ++tt) {
          const int b = (nt == 2) ? tt : (c & 1);
          ok = warp_wait(bars, &bars->acc_full[b], (b ? q1 : q0) & 1, lim, p.status);
          if (!ok) break;
          if (b) ++q1; else ++q0;
          tc_fence_after();
          const int grows = un.nrows[tt] - qw * kGroupRows;   // rows of this warp's group in the block
          const bool rows_live = grows > 0;
          const int grow0 = un.row0[tt] + qw * kGroupRows;
          const uint32_t tacc = tmem_base + kChunk * b + lane_base + hw * (64 * kPiecesPerWarp);
          // the warp's 64-column pieces: each is read from TMEM and rounded to bf16 pairs at once (32
          // registers a piece); they are staged and stored after the accumulator has been handed back
          uint32_t w[kPiecesPerWarp][32];
#pragma unroll
          for (int pc = 0; pc < kPiecesPerWarp; ++pc) {
            if (rows_live && col0 + pc * 64 < p.P) {
              uint32_t v[4][16];
#pragma unroll
              for (int gq = 0; gq < 4; ++gq) tmem_ld16_nowait(tacc + pc * 64 + gq * 16, v[gq]);
              tmem_wait_ld();
#pragma unroll
              for (int gq = 0; gq < 4; ++gq)
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                  __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(v[gq][2 * i]), __uint_as_float(v[gq][2 * i + 1]));
                  w[pc][gq * 8 + i] = *reinterpret_cast<uint32_t*>(&h2);
                }
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&bars->acc_empty[b]);
#pragma unroll
          for (int pc = 0; pc < kPiecesPerWarp; ++pc) {
            if (!(rows_live && col0 + pc * 64 < p.P)) continue;
            uint8_t* buf = mystg + (nst % kStgTiles) * kGroupBytes;
            ++nst;
            if (lane == 0) tma_store_wait_read<kStgTiles - 1>();   // the store that last read this staging tile
            __syncwarp();
            uint8_t* rowp = buf + lane * 128;
#pragma unroll
            for (int ch = 0; ch < 8; ++ch)                 // 16-byte chunk ch of the row goes to slot ch ^ (row & 7)
              *reinterpret_cast<uint4*>(rowp + ((ch ^ (lane & 7)) << 4)) =
                  make_uint4(w[pc][4 * ch], w[pc][4 * ch + 1], w[pc][4 * ch + 2], w[pc][4 * ch + 3]);
            fence_proxy_async_smem();
            __syncwarp();
            if (grows >= kGroupRows) {
              if (lane == 0) {
                tma_store_2d(&tmOut, buf, col0 + pc * 64, grow0);
                tma_store_commit();
              }
            } else {        // the last rows of a convolution tile: fewer than 32
              store_partial_group(buf, p.out_ptr + (int64_t)grow0 * p.P + col0 + pc * 64, p.P, grows, p.P - (col0 + pc * 64));
              __syncwarp();
            }
          }
        }
      }
      // this warp has read all it will of the unit's accumulators; once its stores have read their
      // shared memory (S tiles and staging) the next unit may overwrite both
      if (ok) {
        if (lane == 0) { tma_store_wait_read<0>(); mbar_arrive(&bars->unit_done); }
        __syncwarp();
      }
      g += un.adv;
    }
    if (lane == 0) tma_store_wait_all();
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

// ---------------------------------------------------------------------------------------------
// conv_grad_kernel: dB of a 3 x 3 convolution without materialised im2col rows,
//   dB[j][tap * C + c] = sum over pixels of dT[pixel][j] * x[pixel shifted by the tap][c].
// Same shape as grad_kernel (two 128-row accumulators per CTA, a slice of the reduction each, fp32 partials),
// but the reduction runs over boxes of whole image rows (at most 64 pixels: bhk rows of one image, or kb whole
// images), loaded with 4-D boxes: x shifted by the tap (zeros outside an image: the padding), dT unshifted.
// A box may hold fewer than 64 pixels; the ring is zeroed once, so the rows no box ever writes stay zero in
// both operands and add nothing.
struct ConvGradParams {
  int B, H, W, C;
  int r, natoms, ns, slot_bytes;
  int spi, kb, bhk, box_rows;    // slabs per image (kb == 1) or 1; images per slab; image rows per slab; pixels per box
  int cpt;                       // 256-channel windows per tap
  int slices, slabs_per_slice, nslabs;
  float* partial;                // [slices][9 C][r]
  int* status;
};

__global__ void __launch_bounds__(192, 1)
conv_grad_kernel(const __grid_constant__ CUtensorMap tmX4, const __grid_constant__ CUtensorMap tmT4,
                 const ConvGradParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* ring = smem;
  Bars* bars = reinterpret_cast<Bars*>(ring + (size_t)p.ns * p.slot_bytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int tile = blockIdx.x;
  const int slice = tile % p.slices;
  const int chunk = tile / p.slices;
  const int tap = chunk / p.cpt, cwin = (chunk - tap * p.cpt) * 256;
  const int s_begin = slice * p.slabs_per_slice;
  int s_end = s_begin + p.slabs_per_slice;
  if (s_end > p.nslabs) s_end = p.nslabs;
  const int nk = s_end > s_begin ? s_end - s_begin : 0;

  if (threadIdx.x == 0) {
    for (int i = 0; i < p.ns; ++i) { mbar_init(&bars->full[i], 1); mbar_init(&bars->empty[i], 1); }
    mbar_init(&bars->t_full, 1);
    bars->abort_any = 0;
    bars->epi_abort = 0;
    fence_barrier_init();
    tma_prefetch_desc(&tmX4); tma_prefetch_desc(&tmT4);
  }
  {
    uint4* z = reinterpret_cast<uint4*>(ring);
    const int n16 = p.ns * p.slot_bytes / 16;
    for (int i = threadIdx.x; i < n16; i += blockDim.x) z[i] = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async_smem();
  }
  if (warp == 1) tmem_alloc(&bars->tmem_base, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&bars->tmem_base);
  dep_wait();
  dep_launch();

  if (warp == 0) {
    if (lane == 0) {
      const int dy = tap / 3 - 1, dx = tap % 3 - 1;
      for (int i = 0; i < nk; ++i) {
        const int slot = i % p.ns, ph = (i / p.ns) & 1;
        if (!mbar_wait(&bars->empty[slot], ph ^ 1)) { raise_timeout(bars, p.status); break; }
        uint8_t* dst = ring + (size_t)slot * p.slot_bytes;
        const int sl = s_begin + i;
        const int grp = sl / p.spi, ty = sl - grp * p.spi;
        const int b0 = grp * p.kb, y0 = ty * p.bhk;
        mbar_arrive_expect_tx(&bars->full[slot], (4 + p.natoms) * p.box_rows * 128);
        for (int a = 0; a < 4; ++a) tma_load_4d(dst + a * 8192, &tmX4, &bars->full[slot], cwin + a * 64, dx, y0 + dy, b0);
        for (int a = 0; a < p.natoms; ++a) tma_load_4d(dst + 32768 + a * 8192, &tmT4, &bars->full[slot], a * 64, 0, y0, b0);
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
    bool ok = true;
    if (nk > 0) ok = epi_wait(bars, &bars->t_full, 0, p.status);
    if (ok) {
      tc_fence_after();
      for (int mt = 0; mt < 2; ++mt) {
        const int ch = cwin + mt * 128 + row;             // channel within the tap
        float* out = p.partial + ((size_t)slice * 9 * p.C + (size_t)tap * p.C + ch) * p.r;
        for (int c0 = 0; c0 < p.r; c0 += 16) {
          float v[16];
          if (nk > 0) tmem_ld16(tmem_base + mt * 256 + lane_base + c0, v);
          else {
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = 0.f;
          }
          if (ch < p.C) {
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

// Ranks that are multiples of 8 but not of 16 run as the next multiple of 16: the tensor maps keep the
// true extents, so the extra rows / columns of every factor tile arrive as zeros.
int pad16(int r) { return (r + 15) & ~15; }

// Shared-memory plan of chain_kernel for a (padded) rank and a number of blocks per unit.
struct ChainPlan { int natoms, max_blocks, ns, slot_bytes, ns2, f1_bytes; size_t smem; bool ok; };
ChainPlan chain_plan(int rp, int max_blocks, bool f1_mn) {
  ChainPlan pl;
  pl.natoms = (rp + 63) / 64;
  pl.max_blocks = max_blocks;
  pl.f1_bytes = f1_mn ? pl.natoms * kF1AtomBytes : rp * 128;
  pl.slot_bytes = max_blocks * kAtomBytes + pl.f1_bytes;
  const int s_bytes = max_blocks * pl.natoms * kAtomBytes;
  const int fixed = s_bytes + kEpiWarps * kStgTiles * kGroupBytes + (int)sizeof(Bars) + 1024;
  pl.ns2 = (kSmemLimit - fixed) / kAtom2Bytes;
  if (pl.ns2 > kMaxStages2) pl.ns2 = kMaxStages2;
  if (pl.ns2 < 0) pl.ns2 = 0;
  // the first product's ring lies over the second product's ring, S and the staging tiles (all idle while it runs)
  pl.ns = (pl.ns2 * kAtom2Bytes + s_bytes + kEpiWarps * kStgTiles * kGroupBytes) / pl.slot_bytes;
  if (pl.ns > kMaxStages) pl.ns = kMaxStages;
  pl.smem = (size_t)fixed + (size_t)pl.ns2 * kAtom2Bytes;
  // a two-block unit keeps every tile of a chunk of F2 until its second block has used it
  pl.ok = pl.ns >= 2 && pl.ns2 >= 2 && (max_blocks == 1 || pl.ns2 >= pl.natoms);
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

struct BwdWs { int* status; bf16 *T, *dT; float *pA, *pB; size_t bytes; };
BwdWs bwd_ws(void* ws, int64_t N, int m, int n, int r) {
  GradPlan gp = grad_plan(N, m, n, r);
  Arena ar(ws, 0);
  BwdWs w;
  w.status = ar.take_n<int>(64);
  w.T = ar.take_n<bf16>((size_t)N * r);
  w.dT = ar.take_n<bf16>((size_t)N * r);
  w.pA = ar.take_n<float>((size_t)gp.slices * m * pad16(r));
  w.pB = ar.take_n<float>((size_t)gp.slices * n * pad16(r));
  w.bytes = align_up(ar.used, 256);
  return w;
}

// Everything one launch of chain_kernel needs.  Regular mode: In is N x K1.  Convolution mode (cv != null): In is
// the NHWC activation cv describes, N = B H W pixels, K1 is not used; F1 is the factor that holds the nine taps
// side by side (r x 9 C as an operand, or, MN-major, stored (reduction index) x (9 C)).
struct ChainLaunch {
  const void* In; int64_t N; int K1;
  const void* F1; int ldF1; int f1_rows, f1_cols;   // extents of F1 as it lies in memory
  const void* F2; int ldF2; int P;
  bool f_mn;
  void* Out; void* Sg; int s_ld, s_cols;   // S is stored to Sg (row stride s_ld) at column cv->s_col_off
  int r;                                   // width of S
  const ConvGeom* cv;
  int* status; bool clear_status;
  bool stall_selftest; unsigned long long wait_ns;
};

int launch_chain_ex(const ChainLaunch& L, cudaStream_t st) {
  const int rp = pad16(L.r);
  const bool second = L.Out != nullptr && L.P > 0;
  const int sms = sm_count();
  if (sms <= 0) return AB_ERR_CUDA;
  const bool conv = L.cv != nullptr;
  int64_t items, per_unit;
  if (conv) {
    const int groups_of_images = (L.cv->B + L.cv->bb - 1) / L.cv->bb;
    items = (int64_t)groups_of_images * L.cv->tpi;
    per_unit = 1;
  } else {
    items = (L.N + kGroupRows - 1) / kGroupRows;
    per_unit = 4;
  }
  const int grid = (int)(items < sms ? items : sms);
  const int64_t per_cta = (items + grid - 1) / grid;
  ChainPlan pl = chain_plan(rp, per_cta > per_unit ? 2 : 1, L.f_mn);
  if (!pl.ok && pl.max_blocks == 2) pl = chain_plan(rp, 1, L.f_mn);
  if (!pl.ok) return AB_ERR_UNSUPPORTED;
  CUtensorMap tmIn, tmIn4, tmF1, tmF2, tmOut, tmS;
  if (conv) {
    AB_TRY(make_tensor_map_nhwc(&tmIn4, L.In, L.cv->B, L.cv->H, L.cv->W, L.cv->in_ch, L.cv->W, L.cv->bh, L.cv->bb));
    AB_TRY(make_map(&tmF1, L.F1, L.f1_rows, L.f1_cols, L.ldF1, 64, L.f_mn ? 64 : rp));
    tmIn = tmF1;
  } else {
    AB_TRY(make_map(&tmIn, L.In, (uint64_t)L.N, L.K1, L.K1, 64, 128));
    tmIn4 = tmIn;
    if (L.f_mn) AB_TRY(make_map(&tmF1, L.F1, L.K1, L.r, L.ldF1, 64, 64));
    else AB_TRY(make_map(&tmF1, L.F1, L.r, L.K1, L.ldF1, 64, rp));
  }
  // unused maps still have to be valid objects: alias them to another operand
  if (second) {
    if (L.f_mn) AB_TRY(make_map(&tmF2, L.F2, L.r, L.P, L.ldF2, 64, 64));
    else AB_TRY(make_map(&tmF2, L.F2, L.P, L.r, L.ldF2, 64, kChunk));
    AB_TRY(make_map(&tmOut, L.Out, (uint64_t)L.N, L.P, L.P, 64, kGroupRows));
  } else {
    tmF2 = tmF1;
    tmOut = tmF1;
  }
  if (L.Sg) AB_TRY(make_map(&tmS, L.Sg, (uint64_t)L.N, conv ? L.cv->s_col_off + L.s_cols : L.s_cols, L.s_ld, 64, kGroupRows));
  else tmS = tmF1;
  ChainParams q;
  std::memset(&q, 0, sizeof(q));
  q.K1 = L.K1; q.P = second ? L.P : 0; q.r = rp;
  q.nk1 = conv ? 9 * L.cv->cslabs : (L.K1 + 63) / 64;
  q.nchunks = second ? (L.P + kChunk - 1) / kChunk : 0;
  q.natoms = pl.natoms; q.max_blocks = pl.max_blocks; q.ns = pl.ns; q.slot_bytes = pl.slot_bytes; q.ns2 = pl.ns2;
  q.f1_bytes = pl.f1_bytes; q.f1_mn = L.f_mn ? 1 : 0; q.f2_mn = L.f_mn ? 1 : 0; q.save_s = L.Sg ? 1 : 0;
  q.groups = (int)items;
  q.deal = (!conv && items >= (int64_t)8 * grid) ? 4 : 1;
  q.clear_status = L.clear_status ? 1 : 0; q.stall_selftest = L.stall_selftest ? 1 : 0;
  q.wait_ns = L.wait_ns; q.status = L.status;
  if (conv) q.cv = *L.cv;
  q.out_ptr = static_cast<bf16*>(L.Out); q.s_ptr = static_cast<bf16*>(L.Sg); q.s_ld = L.s_ld; q.s_cols = L.s_cols;
  AB_CUDA_OK(cudaFuncSetAttribute(chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem));
  AB_LAUNCH_DEP(chain_kernel, dim3((unsigned)grid), dim3(kChainThreads), pl.smem, st, tmIn, tmIn4, tmF1, tmF2, tmOut,
                tmS, q);
  AB_LAUNCH_OK();
  return AB_OK;
}

// S = In F1^T (saved to Sg if not null), Out = S F2^T (skipped if Out is null).
// f_mn = false: F1 is given as r x K1 (row stride ldF1) and F2 as P x r (row stride ldF2);
// f_mn = true : F1 is given transposed, K1 x r, and F2 transposed, r x P (the factors A and B as they lie in
//               memory when the chain runs backwards).
int launch_chain(const void* In, int64_t N, int K1, const void* F1, int ldF1, const void* F2, int ldF2, int P,
                 bool f_mn, void* Out, void* Sg, int r, int* status, bool clear_status, cudaStream_t st,
                 bool stall_selftest = false, unsigned long long wait_ns = kWaitLimitNs) {
  ChainLaunch L;
  L.In = In; L.N = N; L.K1 = K1; L.F1 = F1; L.ldF1 = ldF1; L.f1_rows = 0; L.f1_cols = 0; L.F2 = F2; L.ldF2 = ldF2; L.P = P;
  L.f_mn = f_mn; L.Out = Out; L.Sg = Sg; L.s_ld = r; L.s_cols = r; L.r = r; L.cv = nullptr; L.status = status;
  L.clear_status = clear_status; L.stall_selftest = stall_selftest; L.wait_ns = wait_ns;
  return launch_chain_ex(L, st);
}

}  // namespace

int bounded_wait_selftest(int* dev_status, unsigned limit_us, cudaStream_t st) {
  bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(dev_status, (unsigned long long)limit_us * 1000ull);
  AB_LAUNCH_OK();
  return AB_OK;
}

// The chain kernel itself with a producer that loads nothing: the MMA issuer's and the epilogue warps'
// waits run out after limit_us, every role unwinds to the common exit, TMEM is released and the status
// word (first int of ws) holds AB_ERR_TIMEOUT.  The operands are carved from ws; their contents do not
// matter, since nothing is ever loaded.
size_t chain_stall_selftest_ws() { return 256 + 4 * 65536; }
int chain_stall_selftest(void* ws, size_t ws_bytes, unsigned limit_us, cudaStream_t st) {
  if (!ws || !aligned(ws, 256) || ws_bytes < chain_stall_selftest_ws()) return AB_ERR_WORKSPACE;
  if (!device_is_sm100() || !encode_fn()) return AB_ERR_UNSUPPORTED;
  char* base = static_cast<char*>(ws);
  int* status = reinterpret_cast<int*>(base);
  void* In = base + 256;                 // 256 x 64 bf16
  void* F1 = base + 256 + 65536;         // 16 x 64
  void* F2 = base + 256 + 2 * 65536;     // 64 x 16
  void* Out = base + 256 + 3 * 65536;    // 256 x 64
  return launch_chain(In, 256, 64, F1, 64, F2, 16, 64, false, Out, nullptr, 16, status, true, st, true,
                      (unsigned long long)limit_us * 1000ull);
}

int make_tensor_map_2d(CUtensorMap* m, const void* ptr, bool f32, uint64_t rows, uint64_t cols, uint64_t ld,
                       uint32_t box_cols, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return AB_ERR_CUDA;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {ld * (f32 ? 4 : 2)};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult rc = fn(m, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr),
                   dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? AB_OK : AB_ERR_CUDA;
}

int make_tensor_map_nhwc(CUtensorMap* m, const void* ptr, uint64_t B, uint64_t H, uint64_t W, uint64_t C,
                         uint32_t bw, uint32_t bh, uint32_t bb) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return AB_ERR_CUDA;
  cuuint64_t dims[4] = {C, W, H, B};
  cuuint64_t strides[3] = {C * 2, W * C * 2, H * W * C * 2};
  cuuint32_t box[4] = {64, bw, bh, bb};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult rc = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? AB_OK : AB_ERR_CUDA;
}

bool tc_device_ok() { return device_is_sm100() && encode_fn() != nullptr; }

bool chain_tc_supported(int64_t N, int m, int n, int r, int ldA, int ldB, int dt,
                        const void* x, const void* A, const void* B, const void* y) {
  if (dt != AB_BF16) return false;
  if (r % 8 != 0 || r < 8 || r > 256) return false;
  if (m % 8 != 0 || n % 8 != 0 || ldA % 8 != 0 || ldB % 8 != 0) return false;
  if (N > (int64_t)1 << 30) return false;
  if (!aligned(x, 16) || !aligned(A, 16) || !aligned(B, 16) || !aligned(y, 16)) return false;
  if (!device_is_sm100() || !encode_fn()) return false;
  return chain_plan(pad16(r), 1, false).ok && chain_plan(pad16(r), 1, true).ok;
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
  return launch_chain(x, N, n, B, ldB, A, ldA, m, false, y, T_save, r, status, true, st);
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
    AB_TRY(launch_chain(x, N, n, B, ldB, nullptr, 0, 0, false, nullptr, w.T, r, w.status, first, st));
    first = false;
    T = w.T;
  }
  if (dX || dB) {
    // dT = dY A (kept for dB), dX = dT B: the chain with F1 = A^T and F2 = B^T, i.e. A and B as they lie
    AB_TRY(launch_chain(dY, N, m, A, ldA, B, ldB, n, true, dX, dB ? w.dT : nullptr, r, w.status, first, st));
    first = false;
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

// ---------------------------------------------------------------------------------------------
// 3 x 3 convolution (stride 1, padding 1, NHWC) with the factorised weight, im2col rows never materialised.
namespace {

ConvGeom conv_geom(int B, int H, int W, int in_ch, int sign, int tap_stride, int f1_col_off, int s_col_off) {
  ConvGeom g;
  g.on = 1; g.B = B; g.H = H; g.W = W; g.in_ch = in_ch; g.cslabs = (in_ch + 63) / 64;
  if (H * W <= 128) { g.bb = 128 / (H * W); g.bh = H; g.tpi = 1; }
  else {
    const int bhmax = 128 / W;
    g.bb = 1; g.tpi = (H + bhmax - 1) / bhmax; g.bh = (H + g.tpi - 1) / g.tpi;
  }
  g.box_rows = W * g.bh * g.bb;
  g.sign = sign; g.tap_stride = tap_stride; g.f1_col_off = f1_col_off; g.s_col_off = s_col_off;
  return g;
}

struct ConvGradPlan { int natoms, ns, slot_bytes, spi, kb, bhk, box_rows, cpt, slices, slabs_per_slice, nslabs; size_t smem; bool ok; };
ConvGradPlan conv_grad_plan(int B, int H, int W, int C, int rp) {
  ConvGradPlan pl;
  pl.natoms = (rp + 63) / 64;
  pl.slot_bytes = 32768 + pl.natoms * 8192;
  const int fixed = (int)sizeof(Bars) + 1024;
  pl.ns = (kSmemLimit - fixed) / pl.slot_bytes;
  if (pl.ns > kMaxStages) pl.ns = kMaxStages;
  pl.smem = (size_t)fixed + (size_t)pl.ns * pl.slot_bytes;
  pl.ok = W <= 64 && pl.ns >= 2;
  if (H * W <= 64) { pl.kb = 64 / (H * W); pl.bhk = H; pl.spi = 1; pl.nslabs = (B + pl.kb - 1) / pl.kb; }
  else { pl.kb = 1; pl.bhk = W <= 64 ? 64 / W : 1; pl.spi = (H + pl.bhk - 1) / pl.bhk; pl.nslabs = B * pl.spi; }
  pl.box_rows = W * pl.bhk * pl.kb;
  pl.cpt = (C + 255) / 256;
  const int chunks = 9 * pl.cpt;
  int sms = sm_count();
  if (sms <= 0) sms = 1;
  int slices = sms / chunks;
  if (slices < 1) slices = 1;
  if (slices > pl.nslabs) slices = pl.nslabs;
  pl.slabs_per_slice = (pl.nslabs + slices - 1) / slices;
  pl.slices = (pl.nslabs + pl.slabs_per_slice - 1) / pl.slabs_per_slice;
  return pl;
}

struct ConvWs { int* status; bf16 *T, *dT; float *pA, *pB; size_t bytes; };
ConvWs conv_ws(void* ws, int B, int H, int W, int C, int m, int r) {
  const int64_t N = (int64_t)B * H * W;
  const int rp = pad16(r);
  GradPlan ga = grad_plan(N, m, 0, r);
  ConvGradPlan gb = conv_grad_plan(B, H, W, C, rp);
  Arena ar(ws, 0);
  ConvWs w;
  w.status = ar.take_n<int>(64);
  w.T = ar.take_n<bf16>((size_t)N * r);
  w.dT = ar.take_n<bf16>((size_t)N * r);
  w.pA = ar.take_n<float>((size_t)ga.slices * m * rp);
  w.pB = ar.take_n<float>((size_t)gb.slices * 9 * C * rp);
  w.bytes = align_up(ar.used, 256);
  return w;
}

}  // namespace

bool conv_tc_supported(int B, int H, int W, int C, int m, int r, int ldA, int ldB, int dt,
                       const void* x, const void* A, const void* Bf) {
  if (dt != AB_BF16) return false;
  if (r % 8 != 0 || r < 8 || r > 256 || C % 8 != 0 || m % 8 != 0 || ldA % 8 != 0 || ldB % 8 != 0) return false;
  if (B < 1 || H < 1 || W < 1 || W > 64 || H > 256 || (int64_t)B * H * W > ((int64_t)1 << 30)) return false;
  if (!aligned(x, 16) || !aligned(A, 16) || !aligned(Bf, 16)) return false;
  if (!device_is_sm100() || !encode_fn()) return false;
  const int cw = C < 256 ? C : 256;
  return chain_plan(pad16(r), 1, false).ok && chain_plan(pad16(r), 1, true).ok && chain_plan(pad16(cw), 1, true).ok &&
         conv_grad_plan(B, H, W, C, pad16(r)).ok;
}

size_t conv_tc_ws(int B, int H, int W, int C, int m, int r) { return conv_ws(nullptr, B, H, W, C, m, r).bytes; }

// y[pixel][:] = (sum over taps of x[pixel + tap][:] B_tap^T) A^T, B_tap = columns tap C .. tap C + C of B
int conv_tc_forward(const void* x, const void* A, const void* Bf, void* y, void* T_save, int B, int H, int W, int C,
                    int m, int r, int ldA, int ldB, void* ws, size_t ws_bytes, cudaStream_t st) {
  if (!ws || ws_bytes < 256) return AB_ERR_WORKSPACE;
  if ((T_save && !aligned(T_save, 16)) || !aligned(y, 16)) return AB_ERR_INVALID_ARG;
  const ConvGeom g = conv_geom(B, H, W, C, +1, C, 0, 0);
  ChainLaunch L;
  L.In = x; L.N = (int64_t)B * H * W; L.K1 = 0; L.F1 = Bf; L.ldF1 = ldB; L.f1_rows = r; L.f1_cols = 9 * C;
  L.F2 = A; L.ldF2 = ldA; L.P = m; L.f_mn = false; L.Out = y; L.Sg = T_save; L.s_ld = r; L.s_cols = r; L.r = r; L.cv = &g;
  L.status = static_cast<int*>(ws); L.clear_status = true; L.stall_selftest = false; L.wait_ns = kWaitLimitNs;
  return launch_chain_ex(L, st);
}

// dT = dY A; dX[pixel][c] = sum over taps of dT[pixel - tap][:] B[:, tap C + c] (the col2im sum, folded into the
// reduction); dA = dY^T T; dB[j][tap C + c] = sum over pixels of dT[pixel][j] x[pixel + tap][c].
int conv_tc_backward(const void* x, const void* dY, const void* A, const void* Bf, const void* T_saved, void* dX,
                     float* dA, float* dB, int B, int H, int W, int C, int m, int r, int ldA, int ldB,
                     void* ws, size_t ws_bytes, cudaStream_t st) {
  if (!ws) return AB_ERR_WORKSPACE;
  ConvWs w = conv_ws(ws, B, H, W, C, m, r);
  if (w.bytes > ws_bytes) return AB_ERR_WORKSPACE;
  if ((dX && !aligned(dX, 16)) || (T_saved && !aligned(T_saved, 16)) || (dA && !aligned(dA, 16)) || (dB && !aligned(dB, 16)))
    return AB_ERR_INVALID_ARG;
  const int64_t N = (int64_t)B * H * W;
  const int rp = pad16(r);
  bool first = true;
  const bf16* T = static_cast<const bf16*>(T_saved);
  if (dA && !T) {      // T rebuilt from x (first product of the forward pass only)
    const ConvGeom g = conv_geom(B, H, W, C, +1, C, 0, 0);
    ChainLaunch L;
    L.In = x; L.N = N; L.K1 = 0; L.F1 = Bf; L.ldF1 = ldB; L.f1_rows = r; L.f1_cols = 9 * C; L.F2 = nullptr; L.ldF2 = 0; L.P = 0;
    L.f_mn = false; L.Out = nullptr; L.Sg = w.T; L.s_ld = r; L.s_cols = r; L.r = r; L.cv = &g; L.status = w.status;
    L.clear_status = first; L.stall_selftest = false; L.wait_ns = kWaitLimitNs;
    AB_TRY(launch_chain_ex(L, st));
    first = false;
    T = w.T;
  }
  if (dX || dB) {
    AB_TRY(launch_chain(dY, N, m, A, ldA, nullptr, 0, 0, true, nullptr, w.dT, r, w.status, first, st));   // dT = dY A
    first = false;
  }
  if (dX) {
    for (int c0 = 0; c0 < C; c0 += 256) {      // 256 channels of dX per launch: the width of one accumulator
      const int cw = C - c0 < 256 ? C - c0 : 256;
      const ConvGeom g = conv_geom(B, H, W, r, -1, C, c0, c0);
      ChainLaunch L;
      L.In = w.dT; L.N = N; L.K1 = 0; L.F1 = Bf; L.ldF1 = ldB; L.f1_rows = r; L.f1_cols = 9 * C; L.F2 = nullptr; L.ldF2 = 0;
      L.P = 0; L.f_mn = true; L.Out = nullptr; L.Sg = dX; L.s_ld = C; L.s_cols = cw; L.r = cw; L.cv = &g; L.status = w.status;
      L.clear_status = false; L.stall_selftest = false; L.wait_ns = kWaitLimitNs;
      AB_TRY(launch_chain_ex(L, st));
    }
  }
  if (dA) {
    GradPlan gp = grad_plan(N, m, 0, r);
    GradParams p;
    std::memset(&p, 0, sizeof(p));
    CUtensorMap tmAct, tmSmall;
    AB_TRY(make_map(&tmAct, dY, (uint64_t)N, m, m, 64, 64));
    AB_TRY(make_map(&tmSmall, T, (uint64_t)N, r, r, 64, 64));
    p.job[0].P = m; p.job[0].chunks = (m + 255) / 256; p.job[0].partial = w.pA;
    p.job[1] = p.job[0]; p.job[1].chunks = 0;
    p.njobs = 1; p.r = rp; p.natoms = gp.natoms; p.ns = gp.ns; p.slot_bytes = gp.slot_bytes;
    p.slices = gp.slices; p.rows_per_slice = gp.rows_per_slice; p.N = (int)N; p.clear_status = first ? 1 : 0;
    p.status = w.status; p.job0_independent = 0;
    AB_CUDA_OK(cudaFuncSetAttribute(grad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gp.smem));
    AB_LAUNCH_DEP(grad_kernel, dim3((unsigned)(p.job[0].chunks * gp.slices)), dim3(192), gp.smem, st, tmAct, tmSmall, tmAct,
                  tmSmall, p);
    AB_LAUNCH_OK();
    first = false;
    const int nA = (int)(((int64_t)m * r / 4 + 255) / 256);
    AB_LAUNCH_DEP(reduce_partials_kernel, dim3(nA), dim3(256), 0, st, static_cast<const float*>(w.pA), dA, m, nA,
                  static_cast<const float*>(w.pA), static_cast<float*>(nullptr), 0, gp.slices, r, rp);
    AB_LAUNCH_OK();
  }
  if (dB) {
    ConvGradPlan gp = conv_grad_plan(B, H, W, C, rp);
    ConvGradParams p;
    std::memset(&p, 0, sizeof(p));
    CUtensorMap tmX4, tmT4;
    AB_TRY(make_tensor_map_nhwc(&tmX4, x, B, H, W, C, W, gp.bhk, gp.kb));
    AB_TRY(make_tensor_map_nhwc(&tmT4, w.dT, B, H, W, r, W, gp.bhk, gp.kb));
    p.B = B; p.H = H; p.W = W; p.C = C; p.r = rp; p.natoms = gp.natoms; p.ns = gp.ns; p.slot_bytes = gp.slot_bytes;
    p.spi = gp.spi; p.kb = gp.kb; p.bhk = gp.bhk; p.box_rows = gp.box_rows; p.cpt = gp.cpt; p.slices = gp.slices;
    p.slabs_per_slice = gp.slabs_per_slice; p.nslabs = gp.nslabs; p.partial = w.pB; p.status = w.status;
    AB_CUDA_OK(cudaFuncSetAttribute(conv_grad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gp.smem));
    AB_LAUNCH_DEP(conv_grad_kernel, dim3((unsigned)(9 * gp.cpt * gp.slices)), dim3(192), gp.smem, st, tmX4, tmT4, p);
    AB_LAUNCH_OK();
    const int nB = ((9 * C + 31) / 32) * ((r + 31) / 32);
    AB_LAUNCH_DEP(reduce_partials_kernel, dim3(nB), dim3(256), 0, st, static_cast<const float*>(w.pB), static_cast<float*>(nullptr),
                  0, 0, static_cast<const float*>(w.pB), dB, 9 * C, gp.slices, r, rp);
    AB_LAUNCH_OK();
  }
  if (first) AB_CUDA_OK(cudaMemsetAsync(w.status, 0, sizeof(int), st));
  return AB_OK;
}

}  // namespace ab
