// sapo_group_advantages: GRPO group-relative advantages (paper Section 4.2 names GRPO as
// the update rule): A_s = (r_s - mean_g) / (std_g + eps) over all completions of a question.
//
// Arithmetic.  Rewards and results are fp32 and these kernels are bound by device memory, so the
// sums are kept in fp32 with their rounding errors carried along (error-free transformations)
// instead of in fp64, whose conversions and slower pipe made an earlier version of this kernel
// ALU-bound at 0.70 of the copy bandwidth:
//   - sum of the group: every addition is a two_sum, the rounding errors are added up beside it,
//     so mean = (s + c) / G is known as an unevaluated pair mu_hi + mu_lo to about 2^-46;
//   - d_i = (r_i - mu_hi) - mu_lo: at most one ulp off, however large the common offset of the
//     rewards is (an all-equal group gives exactly 0);
//   - sum of d_i^2 by fused multiply-adds on interleaved accumulators, combined pairwise;
//   - correctly rounded division, square root and reciprocal for the scalars.
// Worst-case error of an advantage against the exact value for groups of up to 16: 1 ulp (d)
// + 2.5 (std: half of the 4-5 ulp of the sum of squares) + 1.5 (division by G - ddof, root,
// adding eps) + 1 (reciprocal, product) = 6 ulp; typical 1-2 ulp.  Groups that are longer than
// 16 or not aligned for vector loads take plain fp64 loops.
// Reductions have a fixed order, so results do not depend on the launch shape.
#include "common.cuh"

namespace sapo {

// a + b = s + e exactly (Knuth)
__device__ __forceinline__ void two_sum(float a, float b, float& s, float& e) {
  s = __fadd_rn(a, b);
  const float bb = __fsub_rn(s, a);
  e = __fadd_rn(__fsub_rn(a, __fsub_rn(s, bb)), __fsub_rn(b, bb));
}
// (s, c) += x with the rounding error of the addition collected in c
__device__ __forceinline__ void comp_add(float& s, float& c, float x) {
  float t, e;
  two_sum(s, x, t, e);
  s = t; c = __fadd_rn(c, e);
}
// mean of a compensated sum as an unevaluated pair: (s + c) / G = hi + lo
__device__ __forceinline__ void comp_mean(float s, float c, int32_t G, float& hi, float& lo) {
  const float Gf = (float)G;
  if ((G & (G - 1)) == 0) {                         // a power of two: both words scale exactly
    const float inv = __frcp_rn(Gf);
    hi = s * inv; lo = c * inv;
    return;
  }
  hi = __fdiv_rn(s, Gf);
  const float rem = __fmaf_rn(-hi, Gf, s);          // exact: s - hi * G
  lo = __fdiv_rn(__fadd_rn(rem, c), Gf);
}
// std from the sum of squared deviations, and 1 / (std + eps)
__device__ __forceinline__ void std_and_inverse(float ss, int32_t G, int32_t ddof, float eps, float& sd, float& inv) {
  const int32_t denom = G - ddof;
  // (the reciprocal of a power of two is exact, so the product is the correctly rounded quotient)
  const float var = denom <= 0 ? 0.f : ((denom & (denom - 1)) == 0 ? ss * __frcp_rn((float)denom)
                                                                    : __fdiv_rn(ss, (float)denom));
  sd = __fsqrt_rn(var);
  inv = __frcp_rn(__fadd_rn(sd, eps));
}

// The warp-level kernel: LANES lanes per question, 32 / LANES questions per warp, segmented
// shuffles.  A lane takes every LANES-th 16-byte vector of its question's rewards (groups whose
// start and size are multiples of four: with two lanes a group of eight is one vector per lane and
// a warp's loads cover 16 neighbouring questions, 512 contiguous bytes), or every LANES-th reward
// otherwise.  The offsets of the next question are loaded a turn ahead, as in the thread kernel.
// Serves batches of any size; the thread-per-question kernel below takes over for very many
// questions because it spends fewer instructions on each.
template <int LANES>
__global__ void __launch_bounds__(256)
group_adv_kernel(const float* __restrict__ rewards, const int32_t* __restrict__ group_offsets,
                 int32_t Q, float adv_eps, int32_t ddof, float* __restrict__ adv,
                 float* __restrict__ mean, float* __restrict__ stdv, int32_t* status) {
  constexpr int PER_WARP = 32 / LANES;
  const int lane = threadIdx.x & 31;
  const int sub = lane / LANES, l = lane % LANES;
  const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  const int64_t stride = n_warps * PER_WARP;
  int64_t g = warp0 * PER_WARP + sub;
  int32_t a_next = 0, b_next = 0;
  if (g < Q) { a_next = group_offsets[g]; b_next = group_offsets[g + 1]; }
  // the loop bound is the same for all lanes of a warp: every lane takes part in the shuffles
  for (int64_t g0 = warp0 * PER_WARP; g0 < Q; g0 += stride, g += stride) {
    const bool live = g < Q;
    const int32_t a = live ? a_next : 0, b = live ? b_next : 0;
    if (g + stride < Q) { a_next = group_offsets[g + stride]; b_next = group_offsets[g + stride + 1]; }
    const int32_t G = b - a;
    const bool vec = ((a | G) & 3) == 0;
    const int32_t n4 = G >> 2;
    // this lane's rewards, compensated; its first vector (or reward) is kept for the later passes
    float s = 0.f, c = 0.f;
    float4 first = make_float4(0.f, 0.f, 0.f, 0.f);
    bool bad = false;
    if (vec) {
      const float4* r4 = reinterpret_cast<const float4*>(rewards + a);
      for (int32_t v = l; v < n4; v += LANES) {
        const float4 r = __ldg(r4 + v);
        if (v == l) first = r;
        bad |= !isfinite(r.x) | !isfinite(r.y) | !isfinite(r.z) | !isfinite(r.w);
        comp_add(s, c, r.x); comp_add(s, c, r.y); comp_add(s, c, r.z); comp_add(s, c, r.w);
      }
    } else {
      for (int32_t i = a + l; i < b; i += LANES) {
        const float r = rewards[i];
        if (i == a + l) first.x = r;
        bad |= !isfinite(r);
        comp_add(s, c, r);
      }
    }
    if (__any_sync(0xffffffffu, bad) && lane == 0) raise_status(status, SAPO_ST_NONFINITE_REWARD);
    #pragma unroll
    for (int d = 1; d < LANES; d <<= 1) {    // fixed pairing: lane ^ 1, ^ 2, ...
      const float so = __shfl_xor_sync(0xffffffffu, s, d), co = __shfl_xor_sync(0xffffffffu, c, d);
      float t, e;
      // both partners must get the same bits: add in the order (lower lane, upper lane)
      const bool lower = (lane & d) == 0;
      two_sum(lower ? s : so, lower ? so : s, t, e);
      s = t; c = __fadd_rn(__fadd_rn(lower ? c : co, lower ? co : c), e);
    }
    float mu_hi = 0.f, mu_lo = 0.f;
    if (G > 0) comp_mean(s, c, G, mu_hi, mu_lo);
    auto dev = [&](float r) { return __fsub_rn(__fsub_rn(r, mu_hi), mu_lo); };
    float ss = 0.f;
    if (vec) {
      const float4* r4 = reinterpret_cast<const float4*>(rewards + a);
      for (int32_t v = l; v < n4; v += LANES) {
        const float4 r = v == l ? first : __ldg(r4 + v);
        const float dx = dev(r.x), dy = dev(r.y), dz = dev(r.z), dw = dev(r.w);
        ss = __fadd_rn(ss, __fadd_rn(__fmaf_rn(dy, dy, __fmul_rn(dx, dx)), __fmaf_rn(dw, dw, __fmul_rn(dz, dz))));
      }
    } else {
      for (int32_t i = a + l; i < b; i += LANES) {
        const float dv = dev(i == a + l ? first.x : rewards[i]);
        ss = __fmaf_rn(dv, dv, ss);
      }
    }
    #pragma unroll
    for (int d = 1; d < LANES; d <<= 1) ss = __fadd_rn(ss, __shfl_xor_sync(0xffffffffu, ss, d));
    float sd, inv;
    std_and_inverse(ss, G, ddof, adv_eps, sd, inv);
    if (vec) {
      const float4* r4 = reinterpret_cast<const float4*>(rewards + a);
      float4* a4 = reinterpret_cast<float4*>(adv + a);
      for (int32_t v = l; v < n4; v += LANES) {
        const float4 r = v == l ? first : __ldg(r4 + v);
        a4[v] = make_float4(__fmul_rn(dev(r.x), inv), __fmul_rn(dev(r.y), inv), __fmul_rn(dev(r.z), inv),
                            __fmul_rn(dev(r.w), inv));
      }
    } else {
      for (int32_t i = a + l; i < b; i += LANES)
        adv[i] = __fmul_rn(dev(i == a + l ? first.x : rewards[i]), inv);
    }
    if (live && l == 0) {
      if (mean) mean[g] = G > 0 ? mu_hi : 0.f;
      if (stdv) stdv[g] = G > 0 ? sd : 0.f;
    }
  }
}

// A group of 4 * N4 rewards (N4 = 2 or 4; shorter groups are padded with zeros that do not count)
// held in registers by one thread.  Loads and stores are 32 bytes wide, so a thread touches whole
// sectors and a warp's accesses to neighbouring groups of eight are contiguous.
template <int N4>
__device__ __forceinline__ void group_finish(float (&r)[4 * N4], float* __restrict__ adv, int32_t a, int32_t G,
                                             float adv_eps, int32_t ddof, float& mu_out, float& sd_out, bool& bad);

// eight rewards of a group that starts on a 32-byte boundary
__device__ __forceinline__ void load_eight(const float* __restrict__ p, float (&r)[8]) {
  asm volatile("ld.global.nc.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=f"(r[0]), "=f"(r[1]), "=f"(r[2]), "=f"(r[3]), "=f"(r[4]), "=f"(r[5]), "=f"(r[6]), "=f"(r[7])
               : "l"(p));
}

template <int N4>
__device__ __forceinline__ void group_in_registers(const float* __restrict__ rewards, float* __restrict__ adv,
                                                   int32_t a, int32_t G, float adv_eps, int32_t ddof,
                                                   float& mu_out, float& sd_out, bool& bad) {
  constexpr int N = 4 * N4;
  float r[N];
  #pragma unroll
  for (int i = 0; i < N4; i += 2) {
    if (4 * i < G) {     // 32 bytes at once where the group has them (G is a multiple of 4, a of 4: 16-byte aligned;
                         // the 32-byte form needs a multiple of 8)
      if (((a + 4 * i) & 7) == 0 && 4 * i + 8 <= G) {
        asm volatile("ld.global.nc.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                     : "=f"(r[4 * i]), "=f"(r[4 * i + 1]), "=f"(r[4 * i + 2]), "=f"(r[4 * i + 3]),
                       "=f"(r[4 * i + 4]), "=f"(r[4 * i + 5]), "=f"(r[4 * i + 6]), "=f"(r[4 * i + 7])
                     : "l"(rewards + a + 4 * i));
      } else {
        const float4 v = __ldg(reinterpret_cast<const float4*>(rewards + a + 4 * i));
        r[4 * i] = v.x; r[4 * i + 1] = v.y; r[4 * i + 2] = v.z; r[4 * i + 3] = v.w;
        if (4 * i + 4 < G) {
          const float4 w = __ldg(reinterpret_cast<const float4*>(rewards + a + 4 * i + 4));
          r[4 * i + 4] = w.x; r[4 * i + 5] = w.y; r[4 * i + 6] = w.z; r[4 * i + 7] = w.w;
        } else {
          r[4 * i + 4] = r[4 * i + 5] = r[4 * i + 6] = r[4 * i + 7] = 0.f;
        }
      }
    } else {
      #pragma unroll
      for (int j = 0; j < 8; ++j) r[4 * i + j] = 0.f;
    }
  }
  group_finish<N4>(r, adv, a, G, adv_eps, ddof, mu_out, sd_out, bad);
}

// the arithmetic and the stores of a group whose rewards are in r (padding zeros past G)
template <int N4>
__device__ __forceinline__ void group_finish(float (&r)[4 * N4], float* __restrict__ adv, int32_t a, int32_t G,
                                             float adv_eps, int32_t ddof, float& mu_out, float& sd_out, bool& bad) {
  constexpr int N = 4 * N4;
  float s = r[0], c = 0.f;
  bad = !isfinite(r[0]);
  #pragma unroll
  for (int i = 1; i < N; ++i) { bad |= !isfinite(r[i]); comp_add(s, c, r[i]); }    // padding adds exact zeros
  float mu_hi, mu_lo;
  comp_mean(s, c, G, mu_hi, mu_lo);
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  #pragma unroll
  for (int i = 0; i < N; ++i) {
    r[i] = i < G ? __fsub_rn(__fsub_rn(r[i], mu_hi), mu_lo) : 0.f;        // the deviation replaces the reward
    acc[i & 3] = __fmaf_rn(r[i], r[i], acc[i & 3]);
  }
  const float ss = __fadd_rn(__fadd_rn(acc[0], acc[1]), __fadd_rn(acc[2], acc[3]));
  float inv;
  std_and_inverse(ss, G, ddof, adv_eps, sd_out, inv);
  mu_out = mu_hi;
  #pragma unroll
  for (int i = 0; i < N4; i += 2) {
    if (4 * i < G) {
      if (((a + 4 * i) & 7) == 0 && 4 * i + 8 <= G) {
        asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                     ::"l"(adv + a + 4 * i), "f"(r[4 * i] * inv), "f"(r[4 * i + 1] * inv), "f"(r[4 * i + 2] * inv),
                       "f"(r[4 * i + 3] * inv), "f"(r[4 * i + 4] * inv), "f"(r[4 * i + 5] * inv),
                       "f"(r[4 * i + 6] * inv), "f"(r[4 * i + 7] * inv)
                     : "memory");
      } else {
        *reinterpret_cast<float4*>(adv + a + 4 * i) =
            make_float4(r[4 * i] * inv, r[4 * i + 1] * inv, r[4 * i + 2] * inv, r[4 * i + 3] * inv);
        if (4 * i + 4 < G)
          *reinterpret_cast<float4*>(adv + a + 4 * i + 4) =
              make_float4(r[4 * i + 4] * inv, r[4 * i + 5] * inv, r[4 * i + 6] * inv, r[4 * i + 7] * inv);
      }
    }
  }
}

// One thread per question, for batches of very many small groups: no shuffles and no idle lanes.
// A group of up to 16 whose start and size are multiples of four lives in registers; other groups
// take plain loops in fp64.
__global__ void __launch_bounds__(256, 3)
group_adv_thread_kernel(const float* __restrict__ rewards, const int32_t* __restrict__ group_offsets,
                        int32_t Q, float adv_eps, int32_t ddof, float* __restrict__ adv,
                        float* __restrict__ mean, float* __restrict__ stdv, int32_t* status) {
  // The kernel is bound by how many loads it keeps in flight: a question's rewards can only be
  // fetched once its offsets are known.  So a thread runs two turns ahead with the offsets and one
  // turn ahead with the rewards of a group of eight on a 32-byte boundary (the usual case): every
  // turn has a 32-byte reward load and an offset load in flight while it computes and stores.
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int32_t a1 = 0, b1 = 0, a2 = 0, b2 = 0;
  if (g < Q) { a1 = group_offsets[g]; b1 = group_offsets[g + 1]; }
  if (g + stride < Q) { a2 = group_offsets[g + stride]; b2 = group_offsets[g + stride + 1]; }
  float ahead[8];
  bool have = g < Q && (a1 & 7) == 0 && b1 - a1 == 8;
  if (have) load_eight(rewards + a1, ahead);
  for (; g < Q; g += stride) {
    const int32_t a = a1, b = b1;
    a1 = a2; b1 = b2;
    if (g + 2 * stride < Q) { a2 = group_offsets[g + 2 * stride]; b2 = group_offsets[g + 2 * stride + 1]; }
    const bool had = have;
    float r8[8];
    #pragma unroll
    for (int i = 0; i < 8; ++i) r8[i] = ahead[i];
    have = g + stride < Q && (a1 & 7) == 0 && b1 - a1 == 8;
    if (have) load_eight(rewards + a1, ahead);
    const int32_t G = b - a;
    if (had) {
      float mu, sd; bool bad;
      group_finish<2>(r8, adv, a, 8, adv_eps, ddof, mu, sd, bad);
      if (bad) raise_status(status, SAPO_ST_NONFINITE_REWARD);
      if (mean) mean[g] = mu;
      if (stdv) stdv[g] = sd;
      continue;
    }
    if (G <= 0) { if (mean) mean[g] = 0.f; if (stdv) stdv[g] = 0.f; continue; }
    const bool vec = ((a | G) & 3) == 0;
    if (vec && G <= 16) {
      // 4, 12 or 16 completions, or eight off the 32-byte boundary
      float mu, sd; bool bad;
      if (G <= 8) group_in_registers<2>(rewards, adv, a, G, adv_eps, ddof, mu, sd, bad);
      else        group_in_registers<4>(rewards, adv, a, G, adv_eps, ddof, mu, sd, bad);
      if (bad) raise_status(status, SAPO_ST_NONFINITE_REWARD);
      if (mean) mean[g] = mu;
      if (stdv) stdv[g] = sd;
      continue;
    }
    double sum = 0.0;
    bool bad = false;
    for (int32_t i = a; i < b; ++i) { const float r = rewards[i]; bad |= !isfinite(r); sum += (double)r; }
    if (bad) raise_status(status, SAPO_ST_NONFINITE_REWARD);
    const double mu = sum / (double)G;
    double ss = 0.0;
    for (int32_t i = a; i < b; ++i) { const double d = (double)rewards[i] - mu; ss += d * d; }
    const int32_t denom = G - ddof;
    const double sd = denom > 0 ? sqrt(ss / (double)denom) : 0.0;
    const double inv = 1.0 / (sd + (double)adv_eps);
    for (int32_t i = a; i < b; ++i) adv[i] = (float)(((double)rewards[i] - mu) * inv);
    if (mean) mean[g] = (float)mu;
    if (stdv) stdv[g] = (float)sd;
  }
}

static int launch_group_adv(const float* rewards, const int32_t* group_offsets, int32_t Q, float adv_eps,
                            int32_t ddof, float* adv, float* mean, float* std, int32_t* status, void* stream,
                            int which /* 0: by size, 1: warp-level, 2: thread per question */) {
  if (Q < 0 || !group_offsets || !status || ddof < 0 || !(adv_eps >= 0.f)) return SAPO_ERR_INVALID_ARG;
  if (Q == 0) return SAPO_OK;
  if (!rewards || !adv) return SAPO_ERR_INVALID_ARG;
  const int sms = sm_count();
  if (sms <= 0) return SAPO_ERR_CUDA;
  const bool many = which == 2 || (which == 0 && Q >= 4096);        // then: one thread per question
  int64_t blocks = ((int64_t)Q + (many ? 255 : 127)) / (many ? 256 : 128);   // warp-level: 16 questions per warp
  // at most the blocks the device holds at once (three per SM for the thread-per-question kernel)
  const int64_t cap = (int64_t)sms * (many ? resident_blocks_per_sm(group_adv_thread_kernel, 256)
                                           : resident_blocks_per_sm(group_adv_kernel<2>, 256));
  if (blocks > cap) blocks = cap;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  {
    KernelScope scope(SAPO_K_GROUP_ADV, st);
    if (many)
      group_adv_thread_kernel<<<(int)blocks, 256, 0, st>>>(rewards, group_offsets, Q, adv_eps, ddof,
                                                           adv, mean, std, status);
    else
      group_adv_kernel<2><<<(int)blocks, 256, 0, st>>>(rewards, group_offsets, Q, adv_eps, ddof, adv,
                                                       mean, std, status);
  }
  return check_launch();
}

}  // namespace sapo

extern "C" int sapo_group_advantages(const float* rewards, const int32_t* group_offsets, int32_t Q,
                                     float adv_eps, int32_t ddof, float* adv, float* mean,
                                     float* std, int32_t* status, void* stream) {
  return sapo::launch_group_adv(rewards, group_offsets, Q, adv_eps, ddof, adv, mean, std, status, stream, 0);
}

extern "C" int sapo_group_advantages_warp(const float* rewards, const int32_t* group_offsets, int32_t Q,
                                          float adv_eps, int32_t ddof, float* adv, float* mean,
                                          float* std, int32_t* status, void* stream) {
  return sapo::launch_group_adv(rewards, group_offsets, Q, adv_eps, ddof, adv, mean, std, status, stream, 1);
}
