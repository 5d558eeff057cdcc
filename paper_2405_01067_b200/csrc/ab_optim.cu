// Optimizer glue next to the layer step: one AdamW update (decoupled weight decay) of a factor from the
// gradient ab_layer_backward left, as a single HBM stream.  fp32 master values, moments in fp32, an
// optional bf16 copy of the updated values for the tensor-core chain.  The learning-rate rebound of the
// method (the rate drops to a floor whenever the parameters change shape and climbs back over a given
// number of steps) is a scalar the caller multiplies into lr.
#include "ab_common.cuh"

namespace ab {
namespace {

struct AdamArgs {
  float b1, b2, one_minus_b1, one_minus_b2, eps, lr, decay, c1, c2;   // decay = 1 - lr * weight_decay; c = 1 / (1 - beta^t)
};

__device__ __forceinline__ float adam_one(float p, float g, float& m, float& v, const AdamArgs& a) {
  m = fmaf(a.b1, m, a.one_minus_b1 * g);
  v = fmaf(a.b2, v, a.one_minus_b2 * g * g);
  const float mhat = m * a.c1, vhat = v * a.c2;
  return fmaf(-a.lr, mhat / (sqrtf(vhat) + a.eps), p * a.decay);
}

__global__ void __launch_bounds__(256)
adamw_kernel(float* __restrict__ p, const float* __restrict__ g, float* __restrict__ m, float* __restrict__ v,
             bf16* __restrict__ p_lp, int64_t count, int vec_ok, AdamArgs a) {
  const int64_t step = (int64_t)gridDim.x * blockDim.x;
  const int64_t t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t nvec = vec_ok ? count / 4 : 0;
  for (int64_t i = t0; i < nvec; i += step) {
    float4 pp = reinterpret_cast<float4*>(p)[i];
    const float4 gg = __ldcs(reinterpret_cast<const float4*>(g) + i);
    float4 mm = reinterpret_cast<float4*>(m)[i], vv = reinterpret_cast<float4*>(v)[i];
    pp.x = adam_one(pp.x, gg.x, mm.x, vv.x, a);
    pp.y = adam_one(pp.y, gg.y, mm.y, vv.y, a);
    pp.z = adam_one(pp.z, gg.z, mm.z, vv.z, a);
    pp.w = adam_one(pp.w, gg.w, mm.w, vv.w, a);
    reinterpret_cast<float4*>(p)[i] = pp;
    reinterpret_cast<float4*>(m)[i] = mm;
    reinterpret_cast<float4*>(v)[i] = vv;
    if (p_lp) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(pp.x, pp.y), hi = __floats2bfloat162_rn(pp.z, pp.w);
      uint2 pk;
      pk.x = *reinterpret_cast<uint32_t*>(&lo);
      pk.y = *reinterpret_cast<uint32_t*>(&hi);
      reinterpret_cast<uint2*>(p_lp)[i] = pk;
    }
  }
  for (int64_t i = nvec * 4 + t0; i < count; i += step) {
    float mm = m[i], vv = v[i];
    const float pn = adam_one(p[i], g[i], mm, vv, a);
    p[i] = pn; m[i] = mm; v[i] = vv;
    if (p_lp) p_lp[i] = __float2bfloat16_rn(pn);
  }
}

}  // namespace

int adamw_step(float* p, const float* g, float* m, float* v, bf16* p_lp, int64_t count, float lr, float beta1,
               float beta2, float eps, float weight_decay, int step, cudaStream_t st) {
  if (count == 0) return AB_OK;
  AdamArgs a;
  a.b1 = beta1; a.b2 = beta2; a.one_minus_b1 = 1.f - beta1; a.one_minus_b2 = 1.f - beta2;
  a.eps = eps; a.lr = lr; a.decay = 1.f - lr * weight_decay;
  a.c1 = (float)(1.0 / (1.0 - pow((double)beta1, (double)step)));
  a.c2 = (float)(1.0 / (1.0 - pow((double)beta2, (double)step)));
  const int vec_ok = aligned(p, 16) && aligned(g, 16) && aligned(m, 16) && aligned(v, 16) && (!p_lp || aligned(p_lp, 8));
  // one float4 per thread: a grid as long as the data streams faster than a few blocks per SM striding over it
  const int64_t blocks = ((vec_ok ? count / 4 : count) + 255) / 256 + 1;
  const int64_t cap = (int64_t)1 << 30;
  const unsigned grid = (unsigned)(blocks < cap ? blocks : cap);
  adamw_kernel<<<grid, 256, 0, st>>>(p, g, m, v, p_lp, count, vec_ok, a);
  AB_LAUNCH_OK();
  return AB_OK;
}

}  // namespace ab
