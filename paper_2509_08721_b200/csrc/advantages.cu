// sapo_group_advantages: GRPO group-relative advantages (paper Section 4.2 names GRPO as
// the update rule): A_s = (r_s - mean_g) / (std_g + eps) over all completions of a question.
// One warp per question; sums in fp64 (two passes: mean, then squared deviations) combined
// with shuffles in a fixed order, so results do not depend on the launch shape.
#include "common.cuh"

namespace sapo {

__device__ __forceinline__ double warp_sum(double x) {
  #pragma unroll
  for (int d = 16; d > 0; d >>= 1) x += __shfl_xor_sync(0xffffffffu, x, d);
  return x;
}

__global__ void __launch_bounds__(256)
group_adv_kernel(const float* __restrict__ rewards, const int32_t* __restrict__ group_offsets,
                 int32_t Q, double adv_eps, int32_t ddof, float* __restrict__ adv,
                 float* __restrict__ mean, float* __restrict__ stdv, int32_t* status) {
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t g = warp0; g < Q; g += n_warps) {
    const int32_t a = group_offsets[g], b = group_offsets[g + 1];
    const int32_t G = b - a;
    if (G <= 0) {
      if (lane == 0) { if (mean) mean[g] = 0.f; if (stdv) stdv[g] = 0.f; }
      continue;
    }
    double sum = 0.0;
    bool bad = false;
    for (int32_t i = a + lane; i < b; i += 32) {
      const float r = rewards[i];
      bad |= !isfinite(r);
      sum += (double)r;
    }
    if (__any_sync(0xffffffffu, bad) && lane == 0) raise_status(status, SAPO_ST_NONFINITE_REWARD);
    const double mu = warp_sum(sum) / (double)G;
    double ss = 0.0;
    for (int32_t i = a + lane; i < b; i += 32) {
      const double d = (double)rewards[i] - mu;
      ss += d * d;
    }
    const int32_t denom = G - ddof;
    const double sd = denom > 0 ? sqrt(warp_sum(ss) / (double)denom) : 0.0;
    const double inv = 1.0 / (sd + adv_eps);
    for (int32_t i = a + lane; i < b; i += 32) adv[i] = (float)(((double)rewards[i] - mu) * inv);
    if (lane == 0) { if (mean) mean[g] = (float)mu; if (stdv) stdv[g] = (float)sd; }
  }
}

}  // namespace sapo

extern "C" int sapo_group_advantages(const float* rewards, const int32_t* group_offsets, int32_t Q,
                                     float adv_eps, int32_t ddof, float* adv, float* mean,
                                     float* std, int32_t* status, void* stream) {
  using namespace sapo;
  if (Q < 0 || !group_offsets || !status || ddof < 0 || !(adv_eps >= 0.f)) return SAPO_ERR_INVALID_ARG;
  if (Q == 0) return SAPO_OK;
  if (!rewards || !adv) return SAPO_ERR_INVALID_ARG;
  const int sms = sm_count();
  if (sms <= 0) return SAPO_ERR_CUDA;
  int64_t blocks = ((int64_t)Q + 7) / 8;
  if (blocks > (int64_t)sms * 8) blocks = (int64_t)sms * 8;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  {
    KernelScope scope(SAPO_K_GROUP_ADV, st);
    group_adv_kernel<<<(int)blocks, 256, 0, st>>>(rewards, group_offsets, Q, (double)adv_eps, ddof, adv,
                                                  mean, std, status);
  }
  return check_launch();
}
