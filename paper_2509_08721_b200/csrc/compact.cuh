// Row compaction for the backward pass: tokens whose gradient factor g_t is zero (sequences
// of a zero-advantage group, tokens clipped on the binding side) contribute nothing to dhidden
// or dW_head, so only the others are contracted.  The paper calls rollouts with zero advantage
// uninformative (Section 5, first paragraph of the experiments); skipping them here changes no
// result.  Order is preserved (a two-level exclusive scan), so sums keep a fixed order.
#pragma once

#include <cuda_bf16.h>

#include "common.cuh"

namespace sapo {

constexpr int COMPACT_BLOCK = 1024;   // tokens per block of the scan

// counts[b] = active tokens among tokens [1024 b, 1024 b + 1024)
__global__ void __launch_bounds__(COMPACT_BLOCK)
active_count_kernel(const float* __restrict__ gscale, int64_t T, int32_t* __restrict__ counts) {
  __shared__ int32_t warp_n[COMPACT_BLOCK / 32];
  const int64_t t = (int64_t)blockIdx.x * COMPACT_BLOCK + threadIdx.x;
  const bool act = t < T && gscale[t] != 0.f;
  const unsigned m = __ballot_sync(0xffffffffu, act);
  if ((threadIdx.x & 31) == 0) warp_n[threadIdx.x >> 5] = __popc(m);
  __syncthreads();
  if (threadIdx.x < 32) {
    int32_t v = warp_n[threadIdx.x];
    #pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    if (threadIdx.x == 0) counts[blockIdx.x] = v;
  }
}

// In place: counts[b] -> number of active tokens before block b; *n_active = their total.
__global__ void __launch_bounds__(1024)
active_scan_kernel(int32_t* __restrict__ counts, int32_t n_blocks, int32_t* __restrict__ n_active) {
  __shared__ int32_t warp_sums[32];
  __shared__ int32_t running;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) running = 0;
  __syncthreads();
  for (int32_t base = 0; base < n_blocks; base += 1024) {
    const int32_t i = base + tid;
    const int32_t mine = i < n_blocks ? counts[i] : 0;
    int32_t x = mine;
    #pragma unroll
    for (int d = 1; d < 32; d <<= 1) { const int32_t y = __shfl_up_sync(0xffffffffu, x, d); if (lane >= d) x += y; }
    if (lane == 31) warp_sums[warp] = x;
    __syncthreads();
    if (warp == 0) {
      int32_t w = warp_sums[lane];
      #pragma unroll
      for (int d = 1; d < 32; d <<= 1) { const int32_t y = __shfl_up_sync(0xffffffffu, w, d); if (lane >= d) w += y; }
      warp_sums[lane] = w;
    }
    __syncthreads();
    const int32_t incl = running + (warp > 0 ? warp_sums[warp - 1] : 0) + x;
    if (i < n_blocks) counts[i] = incl - mine;
    __syncthreads();
    if (tid == 1023) running = incl;
    __syncthreads();
  }
  if (tid == 0) *n_active = running;
}

// Position of every token among the active ones (or -1), the inverse list, and the compacted
// per-token vectors.  Also zeroes the dhidden rows of inactive tokens.
__global__ void __launch_bounds__(COMPACT_BLOCK)
active_assign_kernel(const float* __restrict__ gscale, const float* __restrict__ lse,
                     const int32_t* __restrict__ ids, int64_t T, const int32_t* __restrict__ block_base,
                     int32_t* __restrict__ act_idx, int32_t* __restrict__ ids_act,
                     float* __restrict__ lse_act, float* __restrict__ g_act,
                     void* __restrict__ dhidden, int64_t row_bytes) {
  __shared__ int32_t warp_n[COMPACT_BLOCK / 32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t t = (int64_t)blockIdx.x * COMPACT_BLOCK + threadIdx.x;
  const float g = t < T ? gscale[t] : 0.f;
  const bool act = t < T && g != 0.f;
  const unsigned m = __ballot_sync(0xffffffffu, act);
  if (lane == 0) warp_n[warp] = __popc(m);
  __syncthreads();
  int32_t before = block_base[blockIdx.x];
  for (int w = 0; w < warp; ++w) before += warp_n[w];
  const int32_t pos = before + __popc(m & ((1u << lane) - 1u));
  if (act) {
    act_idx[pos] = (int32_t)t;
    ids_act[pos] = ids[t];
    lse_act[pos] = lse[t];
    g_act[pos] = g;
  }
  // rows of inactive tokens get no store from the GEMM: clear them, one warp per row
  for (int i = 0; i < 32; ++i) {
    const int64_t tt = (int64_t)blockIdx.x * COMPACT_BLOCK + warp * 32 + i;
    if (tt >= T) break;
    if ((m >> i) & 1u) continue;
    uint4* row = reinterpret_cast<uint4*>(static_cast<uint8_t*>(dhidden) + tt * row_bytes);    // a multiple of 16 bytes
    for (int j = lane; j < (int)(row_bytes >> 4); j += 32) row[j] = make_uint4(0u, 0u, 0u, 0u);
  }
}

// hidden_act[p, :] = hidden[act_idx[p], :] for p < n_active; rows up to the next multiple of 128
// are zero (the contraction over tokens reads whole 128-row blocks).
__global__ void __launch_bounds__(256)
active_gather_kernel(const __nv_bfloat16* __restrict__ hidden, int64_t ld, int32_t H,
                     const int32_t* __restrict__ act_idx, const int32_t* __restrict__ n_active,
                     __nv_bfloat16* __restrict__ hidden_act) {
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  const int32_t n = *n_active;
  const int32_t n_pad = (n + 127) & ~127;
  const int n4 = H / 8;                               // 16-byte vectors per row (H % 8 == 0)
  for (int64_t p = warp0; p < n_pad; p += n_warps) {
    uint4* to = reinterpret_cast<uint4*>(hidden_act + p * (int64_t)H);
    if (p < n) {
      const uint4* from = reinterpret_cast<const uint4*>(hidden + (int64_t)act_idx[p] * ld);
      for (int j = lane; j < n4; j += 32) to[j] = __ldg(from + j);
    } else {
      for (int j = lane; j < n4; j += 32) to[j] = make_uint4(0u, 0u, 0u, 0u);
    }
  }
}

}  // namespace sapo
