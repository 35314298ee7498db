// AdamW step with global-norm gradient clipping for the LM-head weight: the update that
// follows the loss gradient in a trainer step (optimizer tables of the paper's
// "Experimental Details": AdamW, gradient clipping by norm).  Two HBM-bound kernels:
//   1. per-CTA partial sums of dW^2 (double, fixed order);
//   2. every CTA adds the partials in the same order (so all agree on the clip factor), then
//      updates m, v, the fp32 master weight and the bf16 weight element-wise, 16 bytes per
//      thread per array.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace oapl {

constexpr int kAdamMaxPartials = 2048;  // doubles of scratch the caller provides
constexpr int kAdamThreads = 256;

__global__ void sqnorm_partial_kernel(const float* __restrict__ g, size_t n, double* __restrict__ partial) {
  __shared__ double sh[kAdamThreads / 32];
  const size_t n4 = n >> 2;
  const float4* g4 = reinterpret_cast<const float4*>(g);
  double acc = 0.0;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    const float4 x = __ldg(g4 + i);
    acc += ((double)x.x * x.x + (double)x.y * x.y) + ((double)x.z * x.z + (double)x.w * x.w);
  }
  if (blockIdx.x == 0)
    for (size_t i = (n4 << 2) + threadIdx.x; i < n; i += blockDim.x) acc += (double)g[i] * g[i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_down_sync(0xffffffffu, acc, o);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) sh[warp] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int w = 0; w < kAdamThreads / 32; ++w) t += sh[w];
    partial[blockIdx.x] = t;
  }
}

struct AdamParams {
  float lr, beta1, beta2, eps, weight_decay, clip_norm;
  float bias1, bias2;  // 1 - beta1^t, 1 - beta2^t
};

__device__ __forceinline__ void adam_one(float g, float& m, float& v, float& th, const AdamParams& a,
                                         float clip) {
  g *= clip;
  m = a.beta1 * m + (1.f - a.beta1) * g;
  v = a.beta2 * v + (1.f - a.beta2) * g * g;
  const float mhat = m / a.bias1, vhat = v / a.bias2;
  th = th * (1.f - a.lr * a.weight_decay) - a.lr * mhat / (sqrtf(vhat) + a.eps);
}

// master == nullptr: the bf16 weight itself is the parameter (read, updated in fp32, rounded back).
__global__ void adamw_kernel(const float* __restrict__ g, float* __restrict__ m, float* __restrict__ v,
                             float* __restrict__ master, __nv_bfloat16* __restrict__ W, size_t n,
                             const double* __restrict__ partial, int n_partial,
                             const float* __restrict__ other_sq_norm, AdamParams a,
                             float* __restrict__ grad_norm_out) {
  __shared__ float clip_sh;
  if (threadIdx.x == 0) {
    double t = other_sq_norm ? (double)*other_sq_norm : 0.0;
    for (int i = 0; i < n_partial; ++i) t += partial[i];
    const double norm = sqrt(t);
    // clip factor min(1, c / (norm + 1e-6)); clip_norm <= 0 disables clipping
    double cf = 1.0;
    if (a.clip_norm > 0.f) cf = fmin(1.0, (double)a.clip_norm / (norm + 1e-6));
    clip_sh = (float)cf;
    if (blockIdx.x == 0 && grad_norm_out) *grad_norm_out = (float)norm;
  }
  __syncthreads();
  const float clip = clip_sh;
  const size_t n4 = n >> 2;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
    const float4 gg = __ldg(reinterpret_cast<const float4*>(g) + i);
    float4 mm = reinterpret_cast<float4*>(m)[i], vv = reinterpret_cast<float4*>(v)[i];
    float4 th;
    uint2* wp = reinterpret_cast<uint2*>(W) + i;
    if (master) {
      th = reinterpret_cast<float4*>(master)[i];
    } else {
      const uint2 wb = *wp;
      const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162*>(&wb.x);
      const __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162*>(&wb.y);
      const float2 a0 = __bfloat1622float2(lo), a1 = __bfloat1622float2(hi);
      th = make_float4(a0.x, a0.y, a1.x, a1.y);
    }
    adam_one(gg.x, mm.x, vv.x, th.x, a, clip);
    adam_one(gg.y, mm.y, vv.y, th.y, a, clip);
    adam_one(gg.z, mm.z, vv.z, th.z, a, clip);
    adam_one(gg.w, mm.w, vv.w, th.w, a, clip);
    reinterpret_cast<float4*>(m)[i] = mm;
    reinterpret_cast<float4*>(v)[i] = vv;
    if (master) reinterpret_cast<float4*>(master)[i] = th;
    const __nv_bfloat162 lo = __floats2bfloat162_rn(th.x, th.y), hi = __floats2bfloat162_rn(th.z, th.w);
    uint2 wb;
    wb.x = *reinterpret_cast<const uint32_t*>(&lo);
    wb.y = *reinterpret_cast<const uint32_t*>(&hi);
    *wp = wb;
  }
  if (blockIdx.x == 0) {
    for (size_t i = (n4 << 2) + threadIdx.x; i < n; i += blockDim.x) {
      float th = master ? master[i] : __bfloat162float(W[i]);
      adam_one(g[i], m[i], v[i], th, a, clip);
      if (master) master[i] = th;
      W[i] = __float2bfloat16_rn(th);
    }
  }
}

}  // namespace oapl
