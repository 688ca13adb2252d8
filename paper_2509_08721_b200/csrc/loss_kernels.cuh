// The per-token and per-sequence kernels around the GEMMs: bf16 splitting of fp32 operands, the
// loss tail of the separate forward, and the small kernels of the single-pass call.
#pragma once

#include "gemm_sched.cuh"

namespace sapo {
using namespace umma;

// ---------------------------------------------------------------------------- small kernels
// fp32 -> bf16 operands.  mode 0: [hi | hi | lo] (A side), mode 1: [hi | lo | hi] (B side),
// so that sum_k A'[k] B'[k] = hi.hi + hi.lo + lo.hi; mode 2: hi only.
__global__ void __launch_bounds__(256)
split_bf16_kernel(const float* __restrict__ X, int64_t ld, int64_t R, int32_t H,
                  __nv_bfloat16* __restrict__ out, int mode) {
  const int64_t n = R * (int64_t)H;
  const int64_t ldo = mode == 2 ? H : 3 * (int64_t)H;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
       i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t r = i / H; const int32_t c = (int32_t)(i - r * H);
    const float x = X[r * ld + c];
    const __nv_bfloat16 hi = __float2bfloat16_rn(x);
    __nv_bfloat16* o = out + r * ldo;
    o[c] = hi;
    if (mode != 2) {
      const __nv_bfloat16 lo = __float2bfloat16_rn(x - __bfloat162float(hi));
      o[H + c] = mode == 0 ? hi : lo;
      o[2 * H + c] = mode == 0 ? lo : hi;
    }
  }
}

struct TailArgs {
  const float* pm; const float* ps; const float* pz; int32_t n_splits; int64_t T;
  int64_t part_stride;                 // elements from one partial of a token to the next (T when packed)
  const float* pe; float* entropy;     // optional: partial sums of 2^(x - m) z, and the per-token entropy
  const int32_t* ids; int32_t V; const float* old_logp; const float* adv; const int32_t* cu; int32_t S;
  float lo_edge, hi_edge, grad_scale;
  int32_t loss_agg; float kl_beta; const float* ref_logp;   // variants: token-level mean, KL penalty
  float* logp; float* lse; float* ratio; float* surr; float* gscale; float* seq_surr;
  int32_t* status;
};

__device__ __forceinline__ double block_sum_256(double x, double* sh) {
  #pragma unroll
  for (int d = 16; d > 0; d >>= 1) x += __shfl_xor_sync(0xffffffffu, x, d);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  __syncthreads();
  if (lane == 0) sh[warp] = x;
  __syncthreads();
  double t = 0.0;
  if (threadIdx.x == 0) for (int i = 0; i < 8; ++i) t += sh[i];
  return t;   // valid in thread 0
}

// Token range of sequence s as the kernels may use it: cu_seqlens must be a non-decreasing
// sequence inside [0, T].  An entry outside that range, or below its predecessor, is clamped and
// reported (SAPO_ST_BAD_INDEX), so that no kernel indexes a per-token array out of bounds.
__device__ __forceinline__ void seq_range(const int32_t* cu, int32_t s, int64_t T, int32_t& t0, int32_t& t1,
                                          int32_t* status) {
  const int32_t c0 = cu[s], c1 = cu[s + 1];
  const int32_t Tc = (int32_t)T;
  t0 = c0 < 0 ? 0 : (c0 > Tc ? Tc : c0);
  t1 = c1 < 0 ? 0 : (c1 > Tc ? Tc : c1);
  if (t1 < t0) t1 = t0;
  if ((t0 != c0 || t1 != c1) && threadIdx.x == 0) raise_status(status, SAPO_ST_BAD_INDEX);
}
// first and one-past-last token that belongs to a sequence, clamped the same way
__device__ __forceinline__ void scored_range(const int32_t* cu, int32_t S, int64_t T, int32_t& lo, int32_t& hi) {
  const int32_t Tc = (int32_t)T;
  const int32_t c0 = cu[0], c1 = cu[S];
  lo = c0 < 0 ? 0 : (c0 > Tc ? Tc : c0);
  hi = c1 < 0 ? 0 : (c1 > Tc ? Tc : c1);
  if (hi < lo) hi = lo;
}

// One block per sequence: merge the vocab-split partials, then the clipped surrogate.  Blocks
// past the last sequence only help with the tokens of [0, T) that belong to no sequence (a
// caller that passes its buffer capacity as T): those are scored as masked, all outputs zero.
__global__ void __launch_bounds__(256) loss_tail_kernel(TailArgs a) {
  __shared__ double sh[8];
  int32_t lo, hi;                      // the tokens that belong to some sequence
  scored_range(a.cu, a.S, a.T, lo, hi);
  const float n_scored = (float)(hi - lo);
  for (int32_t s = blockIdx.x; s < a.S; s += gridDim.x) {
    int32_t t0, t1;
    seq_range(a.cu, s, a.T, t0, t1, a.status);
    const int32_t Ts = t1 - t0;
    const float A = a.adv[s];
    const bool bad_adv = !isfinite(A);
    if (bad_adv && Ts > 0 && threadIdx.x == 0) raise_status(a.status, SAPO_ST_NONFINITE_INPUT);
    // weight of a token of this sequence: 1/(S T_s) (mean of token means) or 1/T (token mean)
    const float w = Ts <= 0 ? 0.f : (a.loss_agg == 0 ? 1.f / ((float)a.S * (float)Ts) : 1.f / n_scored);
    double acc = 0.0;
    for (int32_t t = t0 + threadIdx.x; t < t1; t += 256) {
      float M = -INFINITY;
      for (int i = 0; i < a.n_splits; ++i) M = fmaxf(M, a.pm[(int64_t)i * a.part_stride + t]);
      float sum = 0.f, zy = 0.f, sz = 0.f;
      for (int i = 0; i < a.n_splits; ++i) {
        const int64_t o = (int64_t)i * a.part_stride + t;
        const float scale = exp2f(a.pm[o] - M);
        sum += a.ps[o] * scale;
        zy += a.pz[o];
        if (a.entropy != nullptr) sz += a.pe[o] * scale;
      }
      const float lse = (M + log2f(sum)) * LN2;
      // entropy of the row's distribution: - sum_v p log p = lse - sum_v p z
      if (a.entropy != nullptr) a.entropy[t] = lse - sz / sum;
      const int32_t y = a.ids[t];
      const bool bad_id = y < 0 || y >= a.V;
      if (bad_id) raise_status(a.status, SAPO_ST_BAD_TOKEN_ID);
      const float old = a.old_logp[t];
      const bool bad_in = !isfinite(old);
      if (bad_in) raise_status(a.status, SAPO_ST_NONFINITE_INPUT);
      const bool bad = bad_id || bad_in || bad_adv;
      const float lp = bad_id ? 0.f : zy - lse;
      const float rho = bad ? 0.f : expf(lp - old);
      const float un = rho * A;
      const float cl = fminf(fmaxf(rho, a.lo_edge), a.hi_edge) * A;
      const float u = bad ? 0.f : fminf(un, cl);
      float g = (!bad && un <= cl) ? -a.grad_scale * A * rho * w : 0.f;
      float obj = u;
      if (a.kl_beta != 0.f && !bad) {
        // penalty towards a reference policy: kl = e^d - d - 1, d = ref - logp; d kl / d logp = 1 - e^d
        const float d = a.ref_logp[t] - lp;
        const float ed = expf(d);
        obj -= a.kl_beta * (ed - d - 1.f);
        g += a.grad_scale * w * a.kl_beta * (1.f - ed);
      }
      a.lse[t] = lse; a.logp[t] = lp; a.ratio[t] = rho; a.surr[t] = u; a.gscale[t] = g;
      acc += (double)obj;
    }
    const double tot = block_sum_256(acc, sh);
    if (threadIdx.x == 0) a.seq_surr[s] = Ts > 0 ? (float)(tot / (double)Ts) : 0.f;
  }
  // tokens before the first or after the last sequence
  const int64_t n_out = (int64_t)lo + (a.T - hi);
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n_out; i += (int64_t)gridDim.x * 256) {
    const int64_t t = i < lo ? i : hi + (i - lo);
    a.lse[t] = 0.f; a.logp[t] = 0.f; a.ratio[t] = 0.f; a.surr[t] = 0.f; a.gscale[t] = 0.f;
    if (a.entropy != nullptr) a.entropy[t] = 0.f;
  }
}

// The vocab-split partials of every token merged into one (max, sum, target logit) triple:
// what a rank that holds one vocabulary shard hands to the others.  out is [3][T].
__global__ void __launch_bounds__(256)
merge_partials_kernel(const float* __restrict__ pm, const float* __restrict__ ps, const float* __restrict__ pz,
                      int32_t n_splits, int64_t T, float* __restrict__ out) {
  for (int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x; t < T; t += (int64_t)gridDim.x * 256) {
    float M = -INFINITY;
    for (int i = 0; i < n_splits; ++i) M = fmaxf(M, pm[(int64_t)i * T + t]);
    float sum = 0.f, zy = 0.f;
    for (int i = 0; i < n_splits; ++i) {
      const int64_t o = (int64_t)i * T + t;
      sum += ps[o] * exp2f(pm[o] - M);
      zy += pz[o];
    }
    out[t] = M; out[T + t] = sum; out[2 * T + t] = zy;
  }
}

// loss = -(1/S) sum_s seq_surr[s], or with token-level aggregation -(1/T) sum_s T_s seq_surr[s]
__global__ void __launch_bounds__(256)
loss_final_kernel(const float* seq_surr, const int32_t* cu, int32_t S, int64_t T, int32_t loss_agg, float* loss) {
  __shared__ double sh[8];
  double acc = 0.0;
  for (int32_t s = threadIdx.x; s < S; s += 256) {
    if (loss_agg == 0) { acc += (double)seq_surr[s]; continue; }
    int32_t t0, t1;
    seq_range(cu, s, T, t0, t1, nullptr);
    acc += (double)seq_surr[s] * (double)(t1 - t0);
  }
  const double tot = block_sum_256(acc, sh);
  int32_t lo, hi;
  scored_range(cu, S, T, lo, hi);
  const double n = loss_agg == 0 ? (double)S : (double)(hi - lo);
  if (threadIdx.x == 0) *loss = n > 0 ? (float)(-tot / n) : 0.f;
}

// ---------------------------------------------------------------------------- hidden rows in place
// Where token t's hidden row is: row t of one matrix, or (tok_src given) a row of one of the two
// rollout stores: tok_src[t] = source row, plus 2^62 for the external store, or -1 for no row.
struct RowSource {
  const __nv_bfloat16* base0; const __nv_bfloat16* base1; int64_t ld; const int64_t* tok_src;
  int64_t n_rows0, n_rows1;     // rows of the two stores (tok_src given): a row outside them is not read
  __device__ __forceinline__ const __nv_bfloat16* row(int64_t t) const {
    if (tok_src == nullptr) return base0 + t * ld;
    const int64_t s = tok_src[t];
    if (s < 0) return nullptr;
    const bool ext = (s >> 62) & 1;
    const int64_t r = s & ((1ll << 62) - 1);
    if (r >= (ext ? n_rows1 : n_rows0)) return nullptr;      // gather_boxes_kernel reports it
    return (ext ? base1 : base0) + r * ld;
  }
};

// The box list of every 128-token block for the GEMM that fetches its A rows in place (see
// GatherArgs): maximal runs of tokens whose source rows are consecutive in one store, each run
// cut into boxes of 2^k rows, largest first (every box is one copy instruction per 64 columns, and
// the copy unit's instruction rate is what bounds a block with many runs: coarser sets of box
// heights were measured 25 % to 6 times slower).  One thread per block; at most 128 boxes.
// n_boxes[b] = number of boxes | rows they cover << 16.
// A source row outside its store is reported (SAPO_ST_BAD_INDEX) and not fetched.
__global__ void __launch_bounds__(128)
gather_boxes_kernel(const int64_t* __restrict__ tok_src, int64_t T, int64_t n_rows0, int64_t n_rows1,
                    uint64_t* __restrict__ boxes, int32_t* __restrict__ n_boxes, int32_t* status) {
  const int64_t blk = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t t_begin = blk * BM;
  if (t_begin >= T) return;
  const int64_t t_end = t_begin + BM < T ? t_begin + BM : T;
  uint64_t* out = boxes + blk * 128;
  int n = 0, rows = 0;
  int64_t t = t_begin;
  while (t < t_end) {
    const int64_t s = tok_src[t];
    if (s < 0) { ++t; continue; }                       // a slot without a token: nothing to fetch
    const int side = (int)((s >> 62) & 1);
    const int64_t row = s & ((1ll << 62) - 1);
    int64_t len = 1;
    while (t + len < t_end && tok_src[t + len] == s + len) ++len;
    if (row + len > (side ? n_rows1 : n_rows0)) {        // would read past the store
      raise_status(status, SAPO_ST_BAD_INDEX);
      t += len;
      continue;
    }
    int64_t done = 0;
    while (done < len) {
      int lg = 7;
      while ((1ll << lg) > len - done) --lg;
      if (!SAPO_IN_BOUNDS(n < 128)) break;
      out[n++] = (uint64_t)(t - t_begin + done) | ((uint64_t)lg << 7) | ((uint64_t)side << 10) |
                 ((uint64_t)(row + done) << 16);
      done += 1ll << lg;
    }
    rows += (int)len;
    t += len;
  }
  n_boxes[blk] = n | (rows << 16);      // boxes, and the rows they bring (what the copy barrier must count)
}

// ---------------------------------------------------------------------------- fused call: small kernels
// Before the forward pass of the fused call: the logit of the chosen token, z_y[t] = <h_t, W_y>,
// as a plain fp32 dot product (one warp per token), and the reference of the exponentials
//   c_t = z_y[t] - old_logp[t],
// which equals lse_t when the policy has not moved since old_logp was taken and is off by
// log(ratio_t) otherwise: exp(z - c_t) then stays within a few powers of e of a probability.
// c2 is c_t * log2(e).  A token id outside [0, V) gets z_y = c = 0 (the tail reports it).
// need (optional, zeroed by the caller): one bit per 128-token block, set when a token of the
// block belongs to a sequence whose advantage is not zero.  Without a KL term every other token
// has g_t = 0 whatever the pass finds, so the forward need not keep the block's exponentials.
__global__ void __launch_bounds__(256)
target_logit_kernel(const RowSource rows, const __nv_bfloat16* __restrict__ W,
                    int64_t ldw, const int32_t* __restrict__ ids, const float* __restrict__ old_logp,
                    int64_t T, int32_t H, int32_t V, float* __restrict__ zy, float* __restrict__ c2,
                    const float* __restrict__ adv, const int32_t* __restrict__ cu, int32_t S,
                    uint32_t* __restrict__ need) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int64_t n_warps = (int64_t)gridDim.x * 8;
  for (int64_t t = warp; t < T; t += n_warps) {
    const int32_t y = ids[t];
    float acc = 0.f;
    const __nv_bfloat16* hrow = rows.row(t);
    if (y >= 0 && y < V && hrow != nullptr) {
      const uint4* a = reinterpret_cast<const uint4*>(hrow);
      const uint4* b = reinterpret_cast<const uint4*>(W + (int64_t)y * ldw);
      for (int i = lane; i < H / 8; i += 32) {
        const uint4 ua = a[i], ub = b[i];
        const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&ua);
        const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&ub);
        #pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float2 fa = __bfloat1622float2(pa[j]), fb = __bfloat1622float2(pb[j]);
          acc = fmaf(fa.x, fb.x, acc); acc = fmaf(fa.y, fb.y, acc);
        }
      }
      #pragma unroll
      for (int d = 16; d > 0; d >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, d);
    }
    if (lane == 0) {
      const bool ok = y >= 0 && y < V;
      const float old = old_logp[t];
      zy[t] = ok ? acc : 0.f;
      // a non-finite old log-prob (the tail reports it and masks the token) must not reach the panel
      c2[t] = ok ? (isfinite(old) ? acc - old : acc) * LOG2E : 0.f;
      if (need != nullptr) {
        // the token's sequence (last s with cu[s] <= t) and whether its advantage can give a gradient
        int lo = 0, hi = S - 1;
        while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if ((int64_t)cu[mid] <= t) lo = mid; else hi = mid - 1; }
        const uint32_t bit = 1u << ((t >> 7) & 31);
        if (adv[lo] != 0.f && (need[t >> 12] & bit) == 0u) atomicOr(&need[t >> 12], bit);
      }
    }
  }
}

struct FusedTailArgs {
  const float* ps; int32_t n_parts; int64_t t0, tc;        // partial sums [n_parts][tc] of this token chunk
  const float* pe; float* entropy;                         // optional: partial sums of e z [n_parts][tc]; entropy [T]
  const float* zy; const float* c2;                        // [T]
  const int32_t* ids; int32_t V; const float* old_logp; const float* adv; const int32_t* cu; int32_t S;
  int64_t T; float lo_edge, hi_edge, grad_scale; int32_t loss_agg; float kl_beta; const float* ref_logp;
  float* logp; float* lse; float* ratio; float* surr; float* gscale; float* obj;   // [T]
  float* row_scale;                                        // [tc]
  __nv_bfloat16* panel; int32_t nvt;                       // exponentials of the chunk
  int64_t panel_rows;                                      // 128-byte rows it holds (checked builds)
  RowSource rows; int32_t H; __nv_bfloat16* hs;            // hs [tc, H] = row_scale * hidden row
  uint32_t* active_mask;   // one bit per 128-token block of the chunk (zeroed by the caller), or nullptr
  int32_t* status;
};

// After the forward pass of a token chunk of the fused call, one warp per token:
//   sum_t = sum_v exp(z - c_t);  lse = c_t + log sum_t;  logp = z_y - lse;  ratio, surrogate and
//   g_t = dloss/dlogp as in loss_tail_kernel;
// then what turns the stored exponentials e into dz = g ([v = y] - e / sum_t) = a_t e' with
//   a_t = -g_t / sum_t,   e'[t,v] = e[t,v] - [v = y_t] sum_t :
// the panel entry of the chosen token is replaced by e_y - sum_t, a_t becomes the row scale of
// the dhidden contraction, and hs = a_t * hidden (bf16) the operand of the dW_head contraction.
__global__ void __launch_bounds__(256) fused_tail_kernel(FusedTailArgs a) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int64_t n_warps = (int64_t)gridDim.x * 8;
  int32_t first_scored, end_scored;
  scored_range(a.cu, a.S, a.T, first_scored, end_scored);
  const float n_scored = (float)(end_scored - first_scored);
  for (int64_t lr = warp; lr < a.tc; lr += n_warps) {
    const int64_t t = a.t0 + lr;
    float part = 0.f, part_z = 0.f;
    for (int i = lane; i < a.n_parts; i += 32) {
      part += a.ps[(int64_t)i * a.tc + lr];
      if (a.entropy != nullptr) part_z += a.pe[(int64_t)i * a.tc + lr];
    }
    #pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      part += __shfl_xor_sync(0xffffffffu, part, d);
      part_z += __shfl_xor_sync(0xffffffffu, part_z, d);
    }
    const float sum = part;
    // the sequence of this token: last s with cu[s] <= t; a token before the first or after the
    // last sequence (the caller passed its buffer capacity as T) is scored as masked
    int lo = 0, hi = a.S - 1;
    while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if ((int64_t)a.cu[mid] <= t) lo = mid; else hi = mid - 1; }
    int32_t s0, s1;
    seq_range(a.cu, lo, a.T, s0, s1, nullptr);       // seq_mean_kernel reports a bad cu_seqlens
    const bool in_seq = t >= s0 && t < s1;
    const int32_t Ts = s1 - s0;
    const float A = a.adv[lo];
    const float w = Ts <= 0 ? 0.f : (a.loss_agg == 0 ? 1.f / ((float)a.S * (float)Ts) : 1.f / n_scored);
    const int32_t y = a.ids[t];
    const bool bad_id = in_seq && (y < 0 || y >= a.V);
    // a sum of exponentials that left the safe range (or is not a number): the reference was too far off
    const bool bad_range = !(sum < EXP_CAP) || !(sum > 1.f / EXP_CAP);
    const float old = a.old_logp[t];
    const bool bad_in = in_seq && (!isfinite(old) || !isfinite(A));
    const bool bad = !in_seq || bad_id || bad_range || bad_in;
    const float c2 = a.c2[t], zy = a.zy[t];
    const float lse = (bad_range || !in_seq) ? 0.f : (c2 + log2f(sum)) * LN2;
    const float lp = (bad_id || bad_range || !in_seq) ? 0.f : zy - lse;
    const float rho = bad ? 0.f : expf(lp - old);
    const float un = rho * A;
    const float cl = fminf(fmaxf(rho, a.lo_edge), a.hi_edge) * A;
    const float u = bad ? 0.f : fminf(un, cl);
    float g = (!bad && un <= cl) ? -a.grad_scale * A * rho * w : 0.f;
    float obj = u;
    if (a.kl_beta != 0.f && !bad) {
      const float d = a.ref_logp[t] - lp;
      const float ed = expf(d);
      obj -= a.kl_beta * (ed - d - 1.f);
      g += a.grad_scale * w * a.kl_beta * (1.f - ed);
    }
    const float scale = (bad || g == 0.f) ? 0.f : -g / sum;
    if (lane == 0) {
      if (bad_id) raise_status(a.status, SAPO_ST_BAD_TOKEN_ID);
      if (bad_range && in_seq) raise_status(a.status, SAPO_ST_EXP_RANGE);
      if (bad_in) raise_status(a.status, SAPO_ST_NONFINITE_INPUT);
      a.lse[t] = lse; a.logp[t] = lp; a.ratio[t] = rho; a.surr[t] = u; a.gscale[t] = g; a.obj[t] = obj;
      if (a.entropy != nullptr) a.entropy[t] = (bad_range || !in_seq) ? 0.f : lse - part_z / sum;
      a.row_scale[lr] = scale;
      if (scale != 0.f && a.active_mask != nullptr)
        atomicOr(&a.active_mask[lr >> 12], 1u << ((lr >> 7) & 31));
      if (!bad_id && !bad_range && in_seq) {
        const float ey = ex2(fmaf(zy, LOG2E, -c2));
        const int64_t tile = (lr >> 7) * a.nvt + (y >> 6);
        if (SAPO_IN_BOUNDS(tile * BM + (lr & 127) < a.panel_rows))
          a.panel[(tile * BM + (lr & 127)) * 64 + (y & 63)] = __float2bfloat16_rn(ey - sum);
      }
    }
    if (!(sum < EXP_CAP)) {
      // huge, infinite or NaN exponentials in this row: clear it (the row scale is zero, but
      // zero times a non-finite entry would still poison dW_head); rare, so one warp does it
      uint32_t* row32 = reinterpret_cast<uint32_t*>(a.panel);
      for (int vt = 0; vt < a.nvt; ++vt)
        row32[((((lr >> 7) * (int64_t)a.nvt + vt) * BM + (lr & 127)) * 64 >> 1) + lane] = 0u;
    }
    const __nv_bfloat16* hrow = a.rows.row(t);
    const uint4* src = reinterpret_cast<const uint4*>(hrow);
    uint4* dst = reinterpret_cast<uint4*>(a.hs + lr * (int64_t)a.H);
    for (int i = lane; i < a.H / 8; i += 32) {
      uint4 x = (hrow != nullptr && scale != 0.f) ? src[i] : make_uint4(0u, 0u, 0u, 0u);
      __nv_bfloat162* px = reinterpret_cast<__nv_bfloat162*>(&x);
      #pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 f = __bfloat1622float2(px[j]);
        px[j] = __floats2bfloat162_rn(scale * f.x, scale * f.y);
      }
      if (scale == 0.f) x = make_uint4(0u, 0u, 0u, 0u);    // also when the hidden row is not finite
      dst[i] = x;
    }
  }
}

// seq_surr[s] = mean over the tokens of s of obj[t] (same summation order as loss_tail_kernel)
__global__ void __launch_bounds__(256)
seq_mean_kernel(const float* __restrict__ obj, const int32_t* __restrict__ cu, int32_t S, int64_t T,
                float* seq_surr, int32_t* status) {
  __shared__ double sh[8];
  for (int32_t s = blockIdx.x; s < S; s += gridDim.x) {
    int32_t t0, t1;
    seq_range(cu, s, T, t0, t1, status);
    double acc = 0.0;
    for (int32_t t = t0 + threadIdx.x; t < t1; t += 256) acc += (double)obj[t];
    const double tot = block_sum_256(acc, sh);
    if (threadIdx.x == 0) seq_surr[s] = t1 > t0 ? (float)(tot / (double)(t1 - t0)) : 0.f;
  }
}

}  // namespace sapo
