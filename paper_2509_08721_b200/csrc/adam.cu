// sapo_adam_step: the optimiser step that follows the policy gradient on the LM head
// (paper Section 4.2: Adam with default hyper-parameters, learning rate 0.001).  One pass over
// the weight: fp32 master weight and moments are updated in place from the fp32 gradient that
// sapo_policy_loss_bwd produced, and the bf16 copy the next forward reads is rewritten.
// HBM-bound: 30 bytes per weight (16 read, 14 written), vectorised by four.
#include <cuda_bf16.h>

#include "common.cuh"

namespace sapo {

struct AdamArgs {
  float* master; float* m; float* v; const float* grad; __nv_bfloat16* w_bf16;
  int64_t rows; int32_t cols; int64_t ld_w;   // bf16 copy may be padded: ld_w elements per row
  float lr, beta1, beta2, eps, inv_bias1, inv_bias2_sqrt, one_minus_b1, one_minus_b2;
};

__device__ __forceinline__ float adam_one(float& theta, float& m, float& v, float g, const AdamArgs& a) {
  m = a.beta1 * m + a.one_minus_b1 * g;
  v = a.beta2 * v + a.one_minus_b2 * g * g;
  // m_hat / (sqrt(v_hat) + eps) with the bias corrections folded into two constants
  theta -= a.lr * (m * a.inv_bias1) / (sqrtf(v) * a.inv_bias2_sqrt + a.eps);
  return theta;
}

__global__ void __launch_bounds__(256) adam_kernel(AdamArgs a) {
  const int64_t n4 = a.rows * (int64_t)(a.cols / 4);
  const int c4 = a.cols / 4;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / c4; const int c = (int)(i - r * c4) * 4;
    const int64_t at = r * a.cols + c;
    float4 th = *reinterpret_cast<float4*>(a.master + at);
    float4 m = *reinterpret_cast<float4*>(a.m + at);
    float4 v = *reinterpret_cast<float4*>(a.v + at);
    const float4 g = *reinterpret_cast<const float4*>(a.grad + at);
    adam_one(th.x, m.x, v.x, g.x, a); adam_one(th.y, m.y, v.y, g.y, a);
    adam_one(th.z, m.z, v.z, g.z, a); adam_one(th.w, m.w, v.w, g.w, a);
    *reinterpret_cast<float4*>(a.master + at) = th;
    *reinterpret_cast<float4*>(a.m + at) = m;
    *reinterpret_cast<float4*>(a.v + at) = v;
    if (a.w_bf16 != nullptr) {
      __nv_bfloat162 lo = __floats2bfloat162_rn(th.x, th.y), hi = __floats2bfloat162_rn(th.z, th.w);
      uint2 packed = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
      *reinterpret_cast<uint2*>(a.w_bf16 + r * a.ld_w + c) = packed;
    }
  }
}

}  // namespace sapo

extern "C" int sapo_adam_step(float* master, float* m, float* v, const float* grad, void* w_bf16,
                              int64_t rows, int32_t cols, int64_t ld_w, int32_t step,
                              float lr, float beta1, float beta2, float eps, void* stream) {
  using namespace sapo;
  if (!master || !m || !v || !grad || rows < 0 || cols < 4 || (cols % 4) != 0 || step < 1) return SAPO_ERR_INVALID_ARG;
  if (!(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(eps >= 0.f)) return SAPO_ERR_INVALID_ARG;
  if (!aligned16(master) || !aligned16(m) || !aligned16(v) || !aligned16(grad)) return SAPO_ERR_INVALID_ARG;
  if (w_bf16 && (ld_w < cols || (ld_w % 4) != 0 || (reinterpret_cast<uintptr_t>(w_bf16) & 7u))) return SAPO_ERR_INVALID_ARG;
  if (rows == 0) return SAPO_OK;
  AdamArgs a{master, m, v, grad, static_cast<__nv_bfloat16*>(w_bf16), rows, cols, ld_w, lr, beta1, beta2, eps,
             0.f, 0.f, (float)(1.0 - (double)beta1), (float)(1.0 - (double)beta2)};
  // bias corrections in double on the host: 1/(1-b1^t) and 1/sqrt(1-b2^t)
  double p1 = 1.0, p2 = 1.0;
  for (int i = 0; i < step && (p1 > 1e-300 || p2 > 1e-300); ++i) { p1 *= (double)beta1; p2 *= (double)beta2; }
  a.inv_bias1 = (float)(1.0 / (1.0 - p1));
  a.inv_bias2_sqrt = (float)(1.0 / sqrt(1.0 - p2));
  const int sms = sm_count();
  if (sms <= 0) return SAPO_ERR_CUDA;
  const int64_t n4 = rows * (int64_t)(cols / 4);
  int64_t blocks = ceil_div<int64_t>(n4, 256);
  // (a grid of only the resident blocks was measured slower here, 0.89 against 0.96 of copy bandwidth:
  //  seven streams per thread, and short-lived blocks keep them closer together in memory)
  if (blocks > (int64_t)sms * 16) blocks = (int64_t)sms * 16;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  {
    KernelScope scope(SAPO_K_ADAM, st);
    adam_kernel<<<(int)blocks, 256, 0, st>>>(a);
  }
  return check_launch();
}
