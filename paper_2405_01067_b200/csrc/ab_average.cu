// Group mean of K factor copies held in one device's memory: a pure HBM stream.
// Each thread owns 16 input bytes per copy (4 fp32 or 8 bf16 values), keeps up to four copies'
// loads in flight, adds them in fp32 in ascending k and scales by fl(1/K).  The sum order is
// part of the contract (results are compared bit for bit).
// Launch shape: one 16-byte group per thread, i.e. as many 256-thread blocks as the data has
// groups.  On a 1.15 GB stream (8 copies of 31.85 M fp32 values) that draws 6.9-7.0 TB/s, against
// 6.0 TB/s for a grid of 8 blocks per SM walking the data with a grid-sized stride and 6.7 TB/s
// for 16 or 32 blocks per SM; all K loads in flight at once, two groups per thread, 256-bit
// loads and other cache hints measured the same or worse.
#include <algorithm>

#include "ab_common.cuh"

namespace ab {
namespace {

template <typename T> struct Vec;
template <> struct Vec<float> {
  static constexpr int N = 4;
  __device__ static void load(const float* p, float (&v)[4]) {
    float4 t = __ldcs(reinterpret_cast<const float4*>(p));
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
  }
};
template <> struct Vec<bf16> {
  static constexpr int N = 8;
  __device__ static void load(const bf16* p, float (&v)[8]) {
    uint4 t = __ldcs(reinterpret_cast<const uint4*>(p));
    uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {   // a bf16 is the high half of the fp32 with the same value
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
};

template <int N>
__device__ __forceinline__ void store_vec(float* p, const float (&v)[N]) {
#pragma unroll
  for (int i = 0; i < N; i += 4) __stcs(reinterpret_cast<float4*>(p + i), make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]));
}
template <int N>
__device__ __forceinline__ void store_vec(bf16* p, const float (&v)[N]) {
  uint32_t w[N / 2];
#pragma unroll
  for (int i = 0; i < N / 2; ++i) {
    __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
    w[i] = *reinterpret_cast<uint32_t*>(&h);
  }
  if constexpr (N == 8) __stcs(reinterpret_cast<uint4*>(p), make_uint4(w[0], w[1], w[2], w[3]));
  else __stcs(reinterpret_cast<uint2*>(p), make_uint2(w[0], w[1]));
}

// Mean of element group i (V values) of K copies: the one place that fixes the order of the sums.
template <typename TIn, typename TOut>
__device__ __forceinline__ void mean_vec_at(const TIn* __restrict__ base, int64_t stride, int K, float inv,
                                            TOut* __restrict__ out, int64_t i) {
  constexpr int V = Vec<TIn>::N;
  const TIn* p = base + i * V;
  float s[V];
  Vec<TIn>::load(p, s);
  int k = 1;
  for (; k + 3 <= K; k += 3) {       // three more copies in flight, added in ascending k
    float a[V], b[V], c[V];
    Vec<TIn>::load(p + (int64_t)k * stride, a);
    Vec<TIn>::load(p + (int64_t)(k + 1) * stride, b);
    Vec<TIn>::load(p + (int64_t)(k + 2) * stride, c);
#pragma unroll
    for (int j = 0; j < V; ++j) s[j] = __fadd_rn(__fadd_rn(__fadd_rn(s[j], a[j]), b[j]), c[j]);
  }
  for (; k < K; ++k) {
    float a[V];
    Vec<TIn>::load(p + (int64_t)k * stride, a);
#pragma unroll
    for (int j = 0; j < V; ++j) s[j] = __fadd_rn(s[j], a[j]);
  }
#pragma unroll
  for (int j = 0; j < V; ++j) s[j] = __fmul_rn(s[j], inv);
  store_vec<V>(out + i * V, s);
}

template <typename TIn, typename TOut>
__global__ void __launch_bounds__(256)
average_vec_kernel(const TIn* __restrict__ base, int64_t stride, int K, int64_t nvec, float inv,
                   TOut* __restrict__ out) {
  const int64_t step = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += step)
    mean_vec_at<TIn, TOut>(base, stride, K, inv, out, i);
}

// Many means in one launch, fp32 results.  The grid is flat: job j owns the blocks
// [first_block_j, first_block_{j+1}), one 16-byte group per thread, and a block finds its job by
// bisection over the table.  The vector body runs where the job's pointers and stride allow it,
// single elements cover the rest.  Same sums as the kernels above.
template <typename TIn>
__global__ void __launch_bounds__(256)
average_batched_kernel(const AvgJob* __restrict__ jobs, int njobs, int K, float inv) {
  constexpr int V = Vec<TIn>::N;
  int lo = 0, hi = njobs - 1;
  while (lo < hi) {                         // last job whose first block is <= blockIdx.x
    const int mid = (lo + hi + 1) >> 1;
    if (jobs[mid].first_block <= (int64_t)blockIdx.x) lo = mid; else hi = mid - 1;
  }
  const AvgJob j = jobs[lo];
  const int64_t nblocks = (lo + 1 < njobs ? jobs[lo + 1].first_block : (int64_t)gridDim.x) - j.first_block;
  const TIn* base = static_cast<const TIn*>(j.base);
  const bool vec_ok = ((reinterpret_cast<uintptr_t>(j.base) | reinterpret_cast<uintptr_t>(j.out)) & 15u) == 0 &&
                      (j.stride % V == 0);
  const int64_t nvec = vec_ok ? j.count / V : 0;
  const int64_t step = nblocks * blockDim.x;
  const int64_t t0 = ((int64_t)blockIdx.x - j.first_block) * blockDim.x + threadIdx.x;
  for (int64_t i = t0; i < nvec; i += step) mean_vec_at<TIn, float>(base, j.stride, K, inv, j.out, i);
  for (int64_t i = nvec * V + t0; i < j.count; i += step) {
    float s = to_f32(base[i]);
    for (int k = 1; k < K; ++k) s = __fadd_rn(s, to_f32(base[i + (int64_t)k * j.stride]));
    j.out[i] = __fmul_rn(s, inv);
  }
}

// Any alignment, any count: one element per thread (also handles the ragged tail).
template <typename TIn, typename TOut>
__global__ void __launch_bounds__(256)
average_scalar_kernel(const TIn* __restrict__ base, int64_t stride, int K, int64_t first, int64_t count,
                      float inv, TOut* __restrict__ out) {
  const int64_t step = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = first + (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += step) {
    float s = to_f32(base[i]);
    for (int k = 1; k < K; ++k) s = __fadd_rn(s, to_f32(base[i + (int64_t)k * stride]));
    from_f32(out[i], __fmul_rn(s, inv));
  }
}

template <typename TIn, typename TOut>
int run(const void* base_, int64_t stride, int K, int64_t count, void* out_, cudaStream_t st) {
  const TIn* base = static_cast<const TIn*>(base_);
  TOut* out = static_cast<TOut*>(out_);
  constexpr int V = Vec<TIn>::N;
  const float inv = 1.0f / (float)K;
  const bool vec_ok = aligned(base, 16) && aligned(out, 16) && (stride % V == 0);
  int64_t nvec = vec_ok ? count / V : 0;
  const int sms = sm_count() > 0 ? sm_count() : 1;
  if (nvec > 0) {
    int64_t blocks = (nvec + 255) / 256;
    int64_t cap = (int64_t)1 << 30;          // beyond that the kernel's stride loop takes over
    unsigned grid = (unsigned)(blocks < cap ? blocks : cap);
    average_vec_kernel<TIn, TOut><<<grid, 256, 0, st>>>(base, stride, K, nvec, inv, out);
    AB_LAUNCH_OK();
  }
  int64_t first = nvec * V;
  if (first < count) {
    int64_t rest = count - first;
    int64_t blocks = (rest + 255) / 256;
    int64_t cap = (int64_t)sms * 8;
    unsigned grid = (unsigned)(blocks < cap ? blocks : cap);
    average_scalar_kernel<TIn, TOut><<<grid, 256, 0, st>>>(base, stride, K, first, count, inv, out);
    AB_LAUNCH_OK();
  }
  return AB_OK;
}

}  // namespace

int group_average(const void* base, int64_t stride_elems, int K, int64_t count,
                  int in_dt, int out_dt, void* out, cudaStream_t st) {
  if (count == 0) return AB_OK;
  if (in_dt == AB_F32 && out_dt == AB_F32) return run<float, float>(base, stride_elems, K, count, out, st);
  if (in_dt == AB_F32 && out_dt == AB_BF16) return run<float, bf16>(base, stride_elems, K, count, out, st);
  if (in_dt == AB_BF16 && out_dt == AB_F32) return run<bf16, float>(base, stride_elems, K, count, out, st);
  return run<bf16, bf16>(base, stride_elems, K, count, out, st);
}

int64_t average_job_blocks(int64_t count, int in_dt) {
  const int64_t v = in_dt == AB_F32 ? 4 : 8;
  const int64_t groups = (count + v - 1) / v;
  return std::max<int64_t>(1, (groups + 255) / 256);
}

int group_average_batched(const AvgJob* d_jobs, int njobs, int K, int in_dt, int64_t total_blocks, cudaStream_t st) {
  if (njobs <= 0 || total_blocks <= 0) return AB_OK;
  if (total_blocks > ((int64_t)1 << 30)) return AB_ERR_UNSUPPORTED;
  const float inv = 1.0f / (float)K;
  if (in_dt == AB_F32) average_batched_kernel<float><<<(unsigned)total_blocks, 256, 0, st>>>(d_jobs, njobs, K, inv);
  else average_batched_kernel<bf16><<<(unsigned)total_blocks, 256, 0, st>>>(d_jobs, njobs, K, inv);
  AB_LAUNCH_OK();
  return AB_OK;
}

}  // namespace ab
