// sapo_select_external: filter the shared pool and draw the external rollouts
// (paper Section 3.2, last paragraph before Algorithm 1, and Section 5: nodes first discard
// rollouts with zero advantage, then sample uniformly from the rest).  A pool entry is one
// question's rollout (its group of completions); all its advantages are zero exactly when all
// its rewards are equal.  Sampling without replacement = the J smallest of per-entry random
// keys; the keys come from the counter-based Philox-4x32-10 generator (Salmon et al., SC'11),
// so the draw depends only on (seed, entry index).  One block: key generation, an 8-pass radix
// select of the J-th smallest 64-bit key, and an ordered compaction.  All integer work.
#include "common.cuh"

namespace sapo {

__device__ __forceinline__ uint32_t philox4x32_10_first(uint32_t c0, uint32_t k0, uint32_t k1) {
  uint32_t c1 = 0, c2 = 0, c3 = 0;
  #pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  return c0;
}

constexpr int SEL_THREADS = 1024;
constexpr uint64_t NOT_A_CANDIDATE = ~0ull;

// exclusive scan of one value per thread over the block; returns the block total in `total`
__device__ __forceinline__ int32_t block_exclusive_scan(int32_t x, int32_t* warp_sums, int32_t& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int32_t incl = x;
  #pragma unroll
  for (int d = 1; d < 32; d <<= 1) { const int32_t y = __shfl_up_sync(0xffffffffu, incl, d); if (lane >= d) incl += y; }
  __syncthreads();
  if (lane == 31) warp_sums[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int32_t w = warp_sums[lane];
    #pragma unroll
    for (int d = 1; d < 32; d <<= 1) { const int32_t y = __shfl_up_sync(0xffffffffu, w, d); if (lane >= d) w += y; }
    warp_sums[lane] = w;
  }
  __syncthreads();
  total = warp_sums[31];
  return incl - x + (warp > 0 ? warp_sums[warp - 1] : 0);
}

__global__ void __launch_bounds__(SEL_THREADS)
select_external_kernel(const float* __restrict__ rewards, const int32_t* __restrict__ group_offsets,
                       int32_t n, int32_t J, uint32_t seed_lo, uint32_t seed_hi,
                       uint64_t* __restrict__ keys, int32_t* __restrict__ selected,
                       int32_t* __restrict__ n_selected, int32_t* __restrict__ n_candidates) {
  __shared__ int32_t hist[256];
  __shared__ int32_t warp_sums[32];
  __shared__ int32_t sh_count;
  __shared__ uint64_t sh_prefix;
  __shared__ int32_t sh_rank;
  const int tid = threadIdx.x;

  // 1. candidates and their keys
  int32_t mine = 0;
  for (int32_t g = tid; g < n; g += SEL_THREADS) {
    const int32_t a = group_offsets[g], b = group_offsets[g + 1];
    bool informative = false;
    if (b > a) {
      const float r0 = rewards[a];
      for (int32_t i = a + 1; i < b; ++i) informative |= rewards[i] != r0;
    }
    keys[g] = informative ? ((uint64_t)philox4x32_10_first((uint32_t)g, seed_lo, seed_hi) << 32) | (uint32_t)g
                          : NOT_A_CANDIDATE;
    mine += informative ? 1 : 0;
  }
  int32_t n_cand;
  block_exclusive_scan(mine, warp_sums, n_cand);
  const int32_t want = J < n_cand ? (J < 0 ? 0 : J) : n_cand;
  if (tid == 0) { *n_candidates = n_cand; *n_selected = want; sh_prefix = 0; sh_rank = want; }
  __syncthreads();
  if (want == 0) return;

  // 2. the want-th smallest key, one byte at a time from the top
  for (int pass = 0; pass < 8; ++pass) {
    const int shift = 56 - 8 * pass;
    for (int i = tid; i < 256; i += SEL_THREADS) hist[i] = 0;
    __syncthreads();
    const uint64_t prefix = sh_prefix;
    const uint64_t mask = pass == 0 ? 0ull : (~0ull << (shift + 8));
    for (int32_t g = tid; g < n; g += SEL_THREADS) {
      const uint64_t k = keys[g];
      if (k != NOT_A_CANDIDATE && (k & mask) == prefix) atomicAdd(&hist[(k >> shift) & 0xFF], 1);
    }
    __syncthreads();
    if (tid == 0) {
      int32_t rank = sh_rank, b = 0;           // rank: how many keys with this prefix are still wanted
      while (hist[b] < rank) { rank -= hist[b]; ++b; }
      sh_rank = rank;
      sh_prefix = prefix | ((uint64_t)b << shift);
    }
    __syncthreads();
  }
  const uint64_t kth = sh_prefix;              // keys are distinct: exactly `want` keys are <= kth

  // 3. the chosen entries, in pool order
  if (tid == 0) sh_count = 0;
  __syncthreads();
  for (int32_t base = 0; base < n; base += SEL_THREADS) {
    const int32_t g = base + tid;
    const int32_t take = (g < n && keys[g] <= kth) ? 1 : 0;
    int32_t total;
    const int32_t pos = block_exclusive_scan(take, warp_sums, total);
    if (take) selected[sh_count + pos] = g;
    __syncthreads();
    if (tid == 0) sh_count += total;
    __syncthreads();
  }
}

}  // namespace sapo

extern "C" size_t sapo_select_workspace_bytes(int32_t n_entries) {
  return n_entries < 0 ? 0 : (size_t)n_entries * sizeof(uint64_t) + 256;
}

extern "C" int sapo_select_external(const float* rewards, const int32_t* group_offsets, int32_t n_entries,
                                    int32_t J, uint64_t seed, int32_t* selected, int32_t* n_selected,
                                    int32_t* n_candidates, void* workspace, size_t workspace_bytes,
                                    void* stream) {
  using namespace sapo;
  if (n_entries < 0 || J < 0 || !group_offsets || !selected || !n_selected || !n_candidates || !workspace)
    return SAPO_ERR_INVALID_ARG;
  if (n_entries > 0 && !rewards) return SAPO_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 7u) != 0) return SAPO_ERR_INVALID_ARG;
  if (workspace_bytes < sapo_select_workspace_bytes(n_entries)) return SAPO_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  {
    KernelScope scope(SAPO_K_SELECT, st);
    select_external_kernel<<<1, SEL_THREADS, 0, st>>>(rewards, group_offsets, n_entries, J,
                                                      (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32),
                                                      static_cast<uint64_t*>(workspace), selected, n_selected,
                                                      n_candidates);
  }
  return check_launch();
}
