// sapo_group_advantages: GRPO group-relative advantages (paper Section 4.2 names GRPO as
// the update rule): A_s = (r_s - mean_g) / (std_g + eps) over all completions of a question.
// One warp (or eight lanes of it) per question; sums in fp64 (two passes: mean, then squared deviations) combined
// with shuffles in a fixed order, so results do not depend on the launch shape.
#include "common.cuh"

namespace sapo {

// sum over the LANES consecutive lanes this lane belongs to (LANES a power of two)
template <int LANES>
__device__ __forceinline__ double lane_group_sum(double x) {
  #pragma unroll
  for (int d = LANES / 2; d > 0; d >>= 1) x += __shfl_xor_sync(0xffffffffu, x, d);
  return x;
}

// LANES lanes per question (32 in use; batches of thousands of questions take the
// thread-per-question kernel below instead).
template <int LANES>
__global__ void __launch_bounds__(256)
group_adv_kernel(const float* __restrict__ rewards, const int32_t* __restrict__ group_offsets,
                 int32_t Q, double adv_eps, int32_t ddof, float* __restrict__ adv,
                 float* __restrict__ mean, float* __restrict__ stdv, int32_t* status) {
  constexpr int PER_WARP = 32 / LANES;
  const int lane = threadIdx.x & 31;
  const int sub = lane / LANES, l = lane % LANES;
  const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t g0 = warp0 * PER_WARP; g0 < Q; g0 += n_warps * PER_WARP) {
    const int64_t g = g0 + sub;
    const bool live = g < Q;                 // every lane still takes part in the shuffles
    const int32_t a = live ? group_offsets[g] : 0, b = live ? group_offsets[g + 1] : 0;
    const int32_t G = b - a;
    double sum = 0.0;
    bool bad = false;
    for (int32_t i = a + l; i < b; i += LANES) {
      const float r = rewards[i];
      bad |= !isfinite(r);
      sum += (double)r;
    }
    if (__any_sync(0xffffffffu, bad) && lane == 0) raise_status(status, SAPO_ST_NONFINITE_REWARD);
    const double mu = G > 0 ? lane_group_sum<LANES>(sum) / (double)G : lane_group_sum<LANES>(sum);
    double ss = 0.0;
    for (int32_t i = a + l; i < b; i += LANES) {
      const double d = (double)rewards[i] - mu;
      ss += d * d;
    }
    ss = lane_group_sum<LANES>(ss);
    const int32_t denom = G - ddof;
    const double sd = denom > 0 ? sqrt(ss / (double)denom) : 0.0;
    const double inv = 1.0 / (sd + adv_eps);
    for (int32_t i = a + l; i < b; i += LANES) adv[i] = (float)(((double)rewards[i] - mu) * inv);
    if (live && l == 0) {
      if (mean) mean[g] = G > 0 ? (float)mu : 0.f;
      if (stdv) stdv[g] = G > 0 ? (float)sd : 0.f;
    }
  }
}

// 1/n for the small integers a group size (or size minus ddof) can be on the register path
__constant__ double c_inv_small[17] = {0.0, 1.0, 1.0 / 2, 1.0 / 3, 1.0 / 4, 1.0 / 5, 1.0 / 6, 1.0 / 7, 1.0 / 8, 1.0 / 9,
                                       1.0 / 10, 1.0 / 11, 1.0 / 12, 1.0 / 13, 1.0 / 14, 1.0 / 15, 1.0 / 16};

// sqrt and reciprocal in fp64 from an fp32 estimate and one Newton step (relative error about
// 1e-14, far below the fp32 rounding of the results); arguments outside the comfortable fp32
// range take the library routine.  The library's fp64 division and square root cost several
// times more fp64 instructions, and this kernel is bound by them.
__device__ __forceinline__ double sqrt_newton(double v) {
  if (!(v > 1e-30 && v < 1e30)) return v > 0.0 ? sqrt(v) : 0.0;
  double r = (double)rsqrtf((float)v);
  r = r * (1.5 - 0.5 * v * r * r);
  return v * r;
}
__device__ __forceinline__ double rcp_newton(double x) {
  if (!(x > 1e-30 && x < 1e30)) return 1.0 / x;
  double r = (double)(1.f / (float)x);
  return r * (2.0 - x * r);
}

// One thread per question, for batches of very many small groups: no shuffles, and the three
// passes over a group hit L1 after the first.  Groups whose start and size are multiples of
// four move as float4.
__global__ void __launch_bounds__(256)
group_adv_thread_kernel(const float* __restrict__ rewards, const int32_t* __restrict__ group_offsets,
                        int32_t Q, double adv_eps, int32_t ddof, float* __restrict__ adv,
                        float* __restrict__ mean, float* __restrict__ stdv, int32_t* status) {
  for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < Q; g += (int64_t)gridDim.x * blockDim.x) {
    const int32_t a = group_offsets[g], b = group_offsets[g + 1];
    const int32_t G = b - a;
    if (G <= 0) { if (mean) mean[g] = 0.f; if (stdv) stdv[g] = 0.f; continue; }
    const bool vec = ((a | G) & 3) == 0;
    if (vec && G <= 16) {
      // the usual case (8 or 16 completions per question): the group lives in registers
      const float4* r4 = reinterpret_cast<const float4*>(rewards + a);
      float4 buf[4];
      const int n4 = G >> 2;
      #pragma unroll
      for (int i = 0; i < 4; ++i) buf[i] = i < n4 ? r4[i] : make_float4(0.f, 0.f, 0.f, 0.f);
      double sum = 0.0;
      bool bad = false;
      #pragma unroll
      for (int i = 0; i < 4; ++i) {
        bad |= !isfinite(buf[i].x) | !isfinite(buf[i].y) | !isfinite(buf[i].z) | !isfinite(buf[i].w);
        sum += (double)buf[i].x; sum += (double)buf[i].y; sum += (double)buf[i].z; sum += (double)buf[i].w;
      }
      if (bad) raise_status(status, SAPO_ST_NONFINITE_REWARD);
      const double mu = sum * c_inv_small[G];
      double ss = 0.0;
      #pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (i < n4) {
          double d;
          d = (double)buf[i].x - mu; ss += d * d;  d = (double)buf[i].y - mu; ss += d * d;
          d = (double)buf[i].z - mu; ss += d * d;  d = (double)buf[i].w - mu; ss += d * d;
        }
      }
      const int32_t denom = G - ddof;
      const double sd = denom > 0 ? sqrt_newton(ss * c_inv_small[denom]) : 0.0;
      const double inv = rcp_newton(sd + adv_eps);
      float4* a4 = reinterpret_cast<float4*>(adv + a);
      #pragma unroll
      for (int i = 0; i < 4; ++i)
        if (i < n4)
          a4[i] = make_float4((float)(((double)buf[i].x - mu) * inv), (float)(((double)buf[i].y - mu) * inv),
                              (float)(((double)buf[i].z - mu) * inv), (float)(((double)buf[i].w - mu) * inv));
      if (mean) mean[g] = (float)mu;
      if (stdv) stdv[g] = (float)sd;
      continue;
    }
    double sum = 0.0;
    bool bad = false;
    if (vec) {
      const float4* r4 = reinterpret_cast<const float4*>(rewards + a);
      for (int32_t i = 0; i < G / 4; ++i) {
        const float4 r = r4[i];
        bad |= !isfinite(r.x) | !isfinite(r.y) | !isfinite(r.z) | !isfinite(r.w);
        sum += (double)r.x; sum += (double)r.y; sum += (double)r.z; sum += (double)r.w;
      }
    } else {
      for (int32_t i = a; i < b; ++i) { const float r = rewards[i]; bad |= !isfinite(r); sum += (double)r; }
    }
    if (bad) raise_status(status, SAPO_ST_NONFINITE_REWARD);
    const double mu = sum / (double)G;
    double ss = 0.0;
    for (int32_t i = a; i < b; ++i) { const double d = (double)rewards[i] - mu; ss += d * d; }
    const int32_t denom = G - ddof;
    const double sd = denom > 0 ? sqrt(ss / (double)denom) : 0.0;
    const double inv = 1.0 / (sd + adv_eps);
    if (vec) {
      const float4* r4 = reinterpret_cast<const float4*>(rewards + a);
      float4* a4 = reinterpret_cast<float4*>(adv + a);
      for (int32_t i = 0; i < G / 4; ++i) {
        const float4 r = r4[i];
        a4[i] = make_float4((float)(((double)r.x - mu) * inv), (float)(((double)r.y - mu) * inv),
                            (float)(((double)r.z - mu) * inv), (float)(((double)r.w - mu) * inv));
      }
    } else {
      for (int32_t i = a; i < b; ++i) adv[i] = (float)(((double)rewards[i] - mu) * inv);
    }
    if (mean) mean[g] = (float)mu;
    if (stdv) stdv[g] = (float)sd;
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
  const bool many = Q >= 4096;        // then: one thread per question
  int64_t blocks = ((int64_t)Q + (many ? 255 : 7)) / (many ? 256 : 8);
  if (blocks > (int64_t)sms * 8) blocks = (int64_t)sms * 8;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  {
    KernelScope scope(SAPO_K_GROUP_ADV, st);
    if (many)
      group_adv_thread_kernel<<<(int)blocks, 256, 0, st>>>(rewards, group_offsets, Q, (double)adv_eps, ddof,
                                                           adv, mean, std, status);
    else
      group_adv_kernel<32><<<(int)blocks, 256, 0, st>>>(rewards, group_offsets, Q, (double)adv_eps, ddof, adv,
                                                        mean, std, status);
  }
  return check_launch();
}
