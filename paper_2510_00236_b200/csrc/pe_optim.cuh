// Fused elementwise parameter updates that consume the per-example statistics.  Pure streaming
// kernels: every operand is read once and every result written once with 128-bit accesses, so the
// bound is HBM bandwidth (MicroAdam 32 B/parameter, MicroSignSGD 20 B/parameter, +2 B with the
// bf16 weight copy).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

namespace pe {

struct AdamParams {
  float mu_scale;    // s / B
  float nu_scale;    // s^2 / B
  float beta1, beta2;
  float inv_c1, inv_c2;   // 1/(1-beta1^t), 1/(1-beta2^t)
  float eps, lr, wd;
  int eps_inside;
  float inv_B;       // 1 / B
  float bessel;      // 1 / (1 - 1/B): the factor of the unbiased estimators of Eq. (6)
};

// Members of the extended Adam family (Section 3.2.3): what the second-moment EMA is fed.
enum : int { ADAM_ORIGINAL = 0, ADAM_MICRO = 1, ADAM_MICRO_VAR = 2, ADAM_MICRO_MSQ = 3 };

// Algorithm 1 for one parameter.  VARIANT picks the preconditioner: mu^2 (Adam), the average of the
// per-example squares (MicroAdam), or the unbiased estimators of Eq. (6) built from the two
// (MicroAdamVar: the variance; MicroAdamMSQ: the squared mean, clamped at zero only where it is used).
template <int VARIANT>
__device__ __forceinline__ void adam_one(float& th, float& m, float& v, float sg, float sg2, const AdamParams& p) {
  float mu = sg * p.mu_scale;
  float nu_micro = sg2 * p.nu_scale;
  float nu;
  if (VARIANT == ADAM_ORIGINAL) nu = mu * mu;
  else if (VARIANT == ADAM_MICRO) nu = nu_micro;
  else if (VARIANT == ADAM_MICRO_VAR) nu = p.bessel * (nu_micro - mu * mu);
  else nu = p.bessel * (mu * mu - nu_micro * p.inv_B);
  m = fmaf(p.beta1, m, (1.f - p.beta1) * mu);
  v = fmaf(p.beta2, v, (1.f - p.beta2) * nu);
  float mh = m * p.inv_c1;
  float vh = v * p.inv_c2;
  if (VARIANT == ADAM_MICRO_MSQ) vh = fmaxf(vh, 0.f);
  float u = p.eps_inside ? mh / sqrtf(p.eps + vh) : mh / (sqrtf(vh) + p.eps);
  th = th - p.lr * u - p.wd * th;
}

// The same with the member of the family chosen at run time (the update fused into the statistics kernels).
__device__ __forceinline__ void adam_one_rt(int variant, float& th, float& m, float& v, float sg, float sg2, const AdamParams& p) {
  switch (variant) {
    case ADAM_ORIGINAL: adam_one<ADAM_ORIGINAL>(th, m, v, sg, sg2, p); break;
    case ADAM_MICRO: adam_one<ADAM_MICRO>(th, m, v, sg, sg2, p); break;
    case ADAM_MICRO_VAR: adam_one<ADAM_MICRO_VAR>(th, m, v, sg, sg2, p); break;
    default: adam_one<ADAM_MICRO_MSQ>(th, m, v, sg, sg2, p); break;
  }
}

__device__ __forceinline__ float4 ld_stream(const float4* p) { return __ldcs(p); }

constexpr int OPT_THREADS = 256;

template <int VARIANT>
__global__ void __launch_bounds__(OPT_THREADS)
microadam_kernel(float* __restrict__ theta, __nv_bfloat16* __restrict__ theta_lp, float* __restrict__ m,
                 float* __restrict__ v, const float* __restrict__ sum_g, const float* __restrict__ sum_g2,
                 long long n, AdamParams p, const unsigned int* __restrict__ skip_if_set = nullptr) {
  // when this step follows a statistics kernel in the same call: leave the parameters alone if that kernel gave up
  if (skip_if_set && *reinterpret_cast<const volatile unsigned int*>(skip_if_set) != 0u) return;
  const long long n4 = n >> 2;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long k = (long long)blockIdx.x * blockDim.x + threadIdx.x; k < n4; k += stride) {
    float4 th = reinterpret_cast<float4*>(theta)[k];
    float4 mm = reinterpret_cast<float4*>(m)[k];
    float4 vv = reinterpret_cast<float4*>(v)[k];
    float4 g = ld_stream(reinterpret_cast<const float4*>(sum_g) + k);
    float4 g2 = ld_stream(reinterpret_cast<const float4*>(sum_g2) + k);
    adam_one<VARIANT>(th.x, mm.x, vv.x, g.x, g2.x, p);
    adam_one<VARIANT>(th.y, mm.y, vv.y, g.y, g2.y, p);
    adam_one<VARIANT>(th.z, mm.z, vv.z, g.z, g2.z, p);
    adam_one<VARIANT>(th.w, mm.w, vv.w, g.w, g2.w, p);
    reinterpret_cast<float4*>(theta)[k] = th;
    reinterpret_cast<float4*>(m)[k] = mm;
    reinterpret_cast<float4*>(v)[k] = vv;
    if (theta_lp) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(th.x, th.y);
      __nv_bfloat162 hi = __floats2bfloat162_rn(th.z, th.w);
      uint2 pk;
      pk.x = *reinterpret_cast<unsigned int*>(&lo);
      pk.y = *reinterpret_cast<unsigned int*>(&hi);
      reinterpret_cast<uint2*>(theta_lp)[k] = pk;
    }
  }
  // ragged tail (n % 4 elements)
  long long k = (n4 << 2) + (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (k < n) {
    float th = theta[k], mm = m[k], vv = v[k];
    adam_one<VARIANT>(th, mm, vv, sum_g[k], sum_g2[k], p);
    theta[k] = th; m[k] = mm; v[k] = vv;
    if (theta_lp) theta_lp[k] = __float2bfloat16_rn(th);
  }
}

struct SignParams {
  float inv_B, beta, lr, wd;
};

// Section 3.1, MicroSignSGD = EMA o avg o sign, for one parameter.
__device__ __forceinline__ void sign_one(float& th, float& m, float ss, const SignParams& p) {
  float sbar = ss * p.inv_B;
  m = fmaf(p.beta, m, (1.f - p.beta) * sbar);
  th = th - p.lr * m - p.wd * th;
}

__global__ void __launch_bounds__(OPT_THREADS)
microsignsgd_kernel(float* __restrict__ theta, __nv_bfloat16* __restrict__ theta_lp, float* __restrict__ m,
                    const float* __restrict__ sum_sign, long long n, SignParams p,
                    const unsigned int* __restrict__ skip_if_set = nullptr) {
  if (skip_if_set && *reinterpret_cast<const volatile unsigned int*>(skip_if_set) != 0u) return;
  const long long n4 = n >> 2;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long k = (long long)blockIdx.x * blockDim.x + threadIdx.x; k < n4; k += stride) {
    float4 th = reinterpret_cast<float4*>(theta)[k];
    float4 mm = reinterpret_cast<float4*>(m)[k];
    float4 s = ld_stream(reinterpret_cast<const float4*>(sum_sign) + k);
    sign_one(th.x, mm.x, s.x, p);
    sign_one(th.y, mm.y, s.y, p);
    sign_one(th.z, mm.z, s.z, p);
    sign_one(th.w, mm.w, s.w, p);
    reinterpret_cast<float4*>(theta)[k] = th;
    reinterpret_cast<float4*>(m)[k] = mm;
    if (theta_lp) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(th.x, th.y);
      __nv_bfloat162 hi = __floats2bfloat162_rn(th.z, th.w);
      uint2 pk;
      pk.x = *reinterpret_cast<unsigned int*>(&lo);
      pk.y = *reinterpret_cast<unsigned int*>(&hi);
      reinterpret_cast<uint2*>(theta_lp)[k] = pk;
    }
  }
  long long k = (n4 << 2) + (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (k < n) {
    float th = theta[k], mm = m[k];
    sign_one(th, mm, sum_sign[k], p);
    theta[k] = th; m[k] = mm;
    if (theta_lp) theta_lp[k] = __float2bfloat16_rn(th);
  }
}

// The parameter update a statistics kernel applies itself once a tile's sums over the whole batch are
// known (Algorithm 1 / Section 3.1 applied where the sums already are, instead of in a second kernel).
// kind: 0 none, 1 a member of the Adam family (needs sum_b G_b and sum_b G_b^2), 2 MicroSignSGD (needs
// sum_b sign(G_b)).  theta, m, v: [d_out, d_in] fp32, updated in place; theta_lp: optional bf16 copy.
// tile_counters: one word per thread block of the grid's x dimension, zero on entry, used when the
// batch is split across blocks: the block that adds the last partial sum of a tile applies the update.
enum : int { OPT_NONE = 0, OPT_ADAM = 1, OPT_SIGN = 2 };
struct FusedOpt {
  int kind, variant;
  AdamParams adam;
  SignParams sign;
  float* theta;
  __nv_bfloat16* theta_lp;
  float* m;
  float* v;
  unsigned int* tile_counters;
};

// One parameter of the fused update; s1 = sum_b G_b (Adam) or sum_b sign(G_b) (MicroSignSGD), s2 = sum_b G_b^2.
template <int OPT>
__device__ __forceinline__ void fused_update_one(const FusedOpt& o, long long idx, float s1, float s2) {
  float th = o.theta[idx], mm = o.m[idx];
  if constexpr (OPT == OPT_ADAM) {
    float vv = o.v[idx];
    adam_one_rt(o.variant, th, mm, vv, s1, s2, o.adam);
    o.v[idx] = vv;
  } else {
    sign_one(th, mm, s1, o.sign);
  }
  o.theta[idx] = th;
  o.m[idx] = mm;
  if (o.theta_lp) o.theta_lp[idx] = __float2bfloat16_rn(th);
}

}  // namespace pe
