// The two persistent, warp-specialised tcgen05 GEMM kernels (CTA pairs, operands staged by TMA,
// accumulators in tensor memory): the general one with double-buffered accumulators, and the
// wide-tile one for the long-K contractions of the backward pass.
#pragma once

#include <type_traits>

#include "gemm_epilogues.cuh"

namespace sapo {
using namespace umma;

// ---------------------------------------------------------------------------- the GEMM kernel
// D[m, n] = sum_k A[m, k] * B[n, k], one 256 x tile_n tile per CTA pair and step.
// A stage holds a K depth of 128.  All boxes are 64 elements (128 bytes) wide.
//   A_KIND 0: A is stored [M, K] with K contiguous; two boxes {64 k, 128 m} per stage
//   A_KIND 1: A is stored [K, M] with M contiguous; two boxes {64 m, 128 k} per stage
//   A_KIND 2: A is the tiled dz panel read K-major  (M = tokens, K = vocab): one 256-row box
//             (two consecutive vocab tiles of the CTA's token block)
//   A_KIND 3: A is the tiled dz panel read MN-major (M = vocab, K = tokens): two whole tiles
//   B_MN false: B is stored [N, K]; two boxes {64 k, 128 n}.  true: [K, N]; boxes {64 n, 128 k}.
// CTA `rank` of the pair owns rows [256 mb + 128 rank, +128) of the tile and stages columns
// [n0 + rank * n_eff / 2, + n_eff / 2) of B.  All TMA completions of a stage are counted on the
// even CTA's barrier; the even CTA's MMA thread frees stages and publishes accumulators on
// both CTAs' barriers.
//   GATHER (A_KIND 0 only): the rows of A come from two source buffers through a per-block box
//             list (GatherArgs) instead of from one matrix; map_a is unused.
template <int A_KIND, bool B_MN, class Epi, int BKT = BK, int NSTAGE = STAGES, class Gather = NoGather>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const Sched sched_arg, const typename Epi::Params ep_arg, int32_t* status,
                 const __grid_constant__ Gather ga) {
  constexpr bool GATHER = !std::is_same<Gather, NoGather>::value;
  static_assert(!GATHER || (A_KIND == 0 && !B_MN), "gathered rows: K-major A only");
  SAPO_CLOCK_BEGIN
  // a stage holds a K depth of BKT (128: two 64-element boxes per K-major operand; 64: one)
  static_assert(BKT == 128 || (BKT == 64 && A_KIND == 0 && !B_MN), "64-deep stages: K-major operands only");
  constexpr int KBOX = BKT / 64;
  constexpr uint32_t A_ST = BM * BKT * 2, B_ST = (BN / 2) * BKT * 2;
  Sched sched = sched_arg;
  typename Epi::Params ep = ep_arg;
  finalize_sched(sched, (int)(gridDim.x >> 1));
  Epi::set_dynamic(ep, sched);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + NSTAGE * A_ST;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + NSTAGE * (A_ST + B_ST));
  uint64_t* full = bars;                 // [NSTAGE] TMA -> MMA          (even CTA's are used)
  uint64_t* empty = bars + NSTAGE;       // [NSTAGE] MMA -> TMA          (each CTA waits on its own)
  uint64_t* acc_full = bars + 2 * NSTAGE;      // [2] MMA -> epilogue    (each CTA waits on its own)
  uint64_t* acc_empty = bars + 2 * NSTAGE + 2; // [2] epilogue -> MMA    (even CTA's are used)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * NSTAGE + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  uint64_t* drain = bars + 2 * NSTAGE + 5;   // MMA thread only: "all my MMAs have retired" after a wait ran out
  uint64_t* box_s = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(bars) + 256);   // GATHER: this block's box list

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr bool A_MN = (A_KIND & 1) != 0;
  const uint32_t rank = cluster_cta_rank();
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int i = 0; i < NSTAGE; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], 16); }
    mbar_init(drain, 1);
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tensormap(&map_a);
    prefetch_tensormap(&map_b);
  }
  if (warp == 1) { tmem_alloc_pair(tmem_slot, TMEM_COLS); tmem_relinquish_pair(); }
  fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // cluster addresses of barriers the other CTA signals or that live in the even CTA
  const uint32_t full0_addr = map_to_cta(smem_u32(full), 0);
  const uint32_t empty_addr[2] = {map_to_cta(smem_u32(empty), 0), map_to_cta(smem_u32(empty), 1)};
  const uint32_t acc_full_addr[2] = {map_to_cta(smem_u32(acc_full), 0), map_to_cta(smem_u32(acc_full), 1)};
  const uint32_t acc_empty0_addr = map_to_cta(smem_u32(acc_empty), 0);

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    // The whole warp walks the schedule; lane i issues box i of this CTA's share of the
    // stage; lane 0 of the even CTA posts the byte count of both CTAs' shares.
    SAPO_STATS_DECL
    int stage = 0; uint32_t phase = 0;
    uint32_t in_flight = 0;   // bit i: stage i was filled in the current ring pass
    bool ok = true;
    constexpr int A_BOXES = A_KIND == 2 ? 1 : KBOX;
    WorkList work(sched, pair, num_pairs);
    int pmb, un, n_begin, n_end, kb0, kb1, slot;
    while (ok && work.next(pmb, un, n_begin, n_end, kb0, kb1, slot)) {
      const int mb = 2 * pmb + (int)rank;                 // this CTA's 128-row block
      int n_box = 0;
      uint32_t gather_tx = 0;      // bytes of A rows per stage, both CTAs (rows past the end are not fetched)
      if constexpr (GATHER) {
        __syncwarp();
        auto word_of = [&](int b) -> uint32_t { return (int64_t)b * BM < ga.rows ? (uint32_t)ga.n_boxes[b] : 0u; };
        n_box = (int)(word_of(mb) & 0xffffu);
        for (int i = lane; i < n_box; i += 32) box_s[i] = ga.boxes[(size_t)mb * 128 + i];
        __syncwarp();
        gather_tx = ((word_of(2 * pmb) >> 16) + (word_of(2 * pmb + 1) >> 16)) * 128u * KBOX;
      }
      for (int nb = n_begin; ok && nb < n_end; ++nb) {
        const int half = tile_n_eff(sched, nb) >> 1;       // B columns this CTA stages
        const int b_boxes = B_MN ? ((half + 63) >> 6) : KBOX;
        const uint32_t tx = GATHER ? gather_tx + 2 * b_boxes * BOX_BYTES : 2 * (A_ST + b_boxes * BOX_BYTES);
        const bool mine = lane < A_BOXES + b_boxes;
        const bool is_a = lane < A_BOXES;
        const int bi = is_a ? lane : lane - A_BOXES;
        const CUtensorMap* map = is_a ? &map_a : &map_b;
        const uint32_t dst_off = is_a ? bi * BOX_BYTES : NSTAGE * A_ST + bi * BOX_BYTES;
        const bool mn = is_a ? A_MN : B_MN;
        // m or n coordinate of the box (an MN-major box covers 64 of them, a K-major one 128)
        const int row0 = is_a ? mb * BM + (mn ? 64 * bi : 0)
                              : nb * sched.tile_n + (int)rank * half + (mn ? 64 * bi : 0);
        const int k_off = mn ? 0 : 64 * bi;                // K-major boxes split the stage's K depth
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!SAPO_TIMED(0, mbar_wait(&empty[stage], phase ^ 1, abort_flag, sched.wait_limit))) { ok = false; break; }
          if (rank == 0 && lane == 0) mbar_arrive_expect_tx(&full[stage], tx);
          if constexpr (GATHER) {
            // the A rows of this block, box by box (a lane takes every 32nd box, both k boxes of it)
            const uint32_t bar = full0_addr + stage * 8;
            for (int i = lane; i < n_box; i += 32) {
              const uint64_t e = box_s[i];
              const int dst_row = (int)(e & 127u), lg = (int)((e >> 7) & 7u), side = (int)((e >> 10) & 1u);
              const int32_t src_row = (int32_t)(e >> 16);
              #pragma unroll
              for (int kx = 0; kx < KBOX; ++kx)
                tma_load_2d_pair(smem_a + stage * A_ST + kx * BOX_BYTES + dst_row * 128, &ga.maps[side][lg], bar,
                                 kb * BKT + 64 * kx, src_row);
            }
          }
          if (mine && !(GATHER && is_a)) {
            uint8_t* dst = smem + dst_off + stage * (is_a ? A_ST : B_ST);
            const uint32_t bar = full0_addr + stage * 8;
            if (is_a && A_KIND == 2)        // vocab tiles 2 kb and 2 kb + 1 of token block mb: 256 rows
              tma_load_2d_pair(dst, map, bar, 0, (mb * sched.panel_nvt + 2 * kb) * BM);
            else if (is_a && A_KIND == 3)   // token block kb, vocab tile 2 mb + bi: all 128 rows
              tma_load_2d_pair(dst, map, bar, 0, (kb * sched.panel_nvt + 2 * mb + bi) * BM);
            else if (mn) tma_load_2d_pair(dst, map, bar, row0, kb * BKT);
            else         tma_load_2d_pair(dst, map, bar, kb * BKT + k_off, row0);
          }
          in_flight |= 1u << stage;
          if (++stage == NSTAGE) { stage = 0; phase ^= 1; }
        }
      }
    }
    if (lane == 0) SAPO_STATS_FLUSH(4);
    if (!ok && rank == 0 && lane == 0) {
      // give copies already issued a bounded chance to land before the pair leaves
      for (int i = 0; i < NSTAGE; ++i) {
        if (!(in_flight & (1u << i))) continue;
        const uint32_t ph = (i < stage) ? phase : (phase ^ 1);
        for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(&full[i], ph); ++spin) {}
      }
    }
  } else if (warp == 1 && lane == 0 && rank == 0) {
    // ------------------------------------------------------------ MMA issuer (even CTA only)
    SAPO_STATS_DECL
    int stage = 0; uint32_t phase = 0;
    int acc = 0; uint32_t acc_phase = 0;
    bool ok = true;
    WorkList work(sched, pair, num_pairs);
    int pmb, un, n_begin, n_end, kb0, kb1, slot;
    while (ok && work.next(pmb, un, n_begin, n_end, kb0, kb1, slot)) {
      for (int nb = n_begin; ok && nb < n_end; ++nb) {
        const uint32_t idesc = make_idesc_bf16(PAIR_M, tile_n_eff(sched, nb), A_MN, B_MN);
        if (!SAPO_TIMED(2, mbar_wait(&acc_empty[acc], acc_phase ^ 1, abort_flag, sched.wait_limit))) { ok = false; break; }
        fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!SAPO_TIMED(1, mbar_wait(&full[stage], phase, abort_flag, sched.wait_limit))) { ok = false; break; }
          fence_after_sync();
          const uint32_t a_addr = smem_u32(smem_a + stage * A_ST);
          const uint32_t b_addr = smem_u32(smem_b + stage * B_ST);
          #pragma unroll
          for (int k = 0; k < BKT / UMMA_K; ++k) {
            // K-major: 16 elements = 32 bytes along the row, the second half of the depth in
            // the next box; MN-major: 16 rows = 2048 bytes, 64-column chunks one box apart
            const uint32_t k_major_off = (k >> 2) * BOX_BYTES + (k & 3) * 32;
            const uint64_t a_desc = A_MN ? make_smem_desc(a_addr + k * 2048, BOX_BYTES, 1024)
                                         : make_smem_desc(a_addr + k_major_off, 16, 1024);
            const uint64_t b_desc = B_MN ? make_smem_desc(b_addr + k * 2048, BOX_BYTES, 1024)
                                         : make_smem_desc(b_addr + k_major_off, 16, 1024);
            mma_bf16_pair(d_tmem, a_desc, b_desc, idesc, (kb > kb0 || k != 0) ? 1u : 0u);
          }
          // free the stage in both CTAs once these MMAs retire
          mma_commit_pair(empty_addr[0] + stage * 8);
          mma_commit_pair(empty_addr[1] + stage * 8);
          if (++stage == NSTAGE) { stage = 0; phase ^= 1; }
        }
        if (ok) {                                  // accumulator complete, in both CTAs
          mma_commit_pair(acc_full_addr[0] + acc * 8);
          mma_commit_pair(acc_full_addr[1] + acc * 8);
        }
        if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      }
    }
    if (!ok) {
      // a wait ran out: no MMA of this pair may still be running when tensor memory is freed
      mma_commit_pair(map_to_cta(smem_u32(drain), 0));
      for (int spin = 0; spin < (1 << 22) && !mbar_try_wait(drain, 0); ++spin) {}
    }
#ifdef SAPO_WAIT_STATS
    atomicMax(&g_wait_stats[sched.stats_id & 3][7], (unsigned long long)(clock64() - role_t0));
#endif
    SAPO_STATS_FLUSH(5);
  } else if (warp >= 2) {
    // ------------------------------------------------------------ epilogue (8 warps, both CTAs)
    // Warps 2-5 drain the first four 32-column chunks of a tile, warps 6-9 the rest; a warp
    // may only read the TMEM lane quadrant warp_id % 4, so each quadrant has one warp of each set.
    const int quad = warp & 3;
    const int col_half = (warp - 2) >> 2;
    const int r = quad * 32 + lane;
    SAPO_STATS_DECL
    int acc = 0; uint32_t acc_phase = 0;
    bool ok = true;
    Epi epi;
    WorkList work(sched, pair, num_pairs);
    int pmb, un, n_begin, n_end, kb0, kb1, slot;
    while (ok && work.next(pmb, un, n_begin, n_end, kb0, kb1, slot)) {
      epi.begin_unit(ep, 2 * pmb + (int)rank, r);
      if constexpr (Epi::STREAMK) epi.set_dest(ep, slot, (int)rank, r, n_begin * sched.tile_n, sched.part_ld);
      for (int nb = n_begin; ok && nb < n_end; ++nb) {
        if (!SAPO_TIMED(3, mbar_wait(&acc_full[acc], acc_phase, abort_flag, sched.wait_limit))) { ok = false; break; }
        fence_after_sync();
        const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + acc * BN;
        const int n0 = nb * sched.tile_n;
        // the last tile also visits the padding columns up to n_cover (they hold no accumulator)
        const int n_visit = nb == sched.num_n_blocks - 1 ? sched.n_cover - n0 : sched.tile_n;
        const int chunks = (n_visit + 31) >> 5;
        const int c_begin = col_half ? 4 : 0;
        const int c_end = col_half ? chunks : min(chunks, 4);
        const int c_tmem = (sched.tile_n + 31) >> 5;      // chunks that exist in tensor memory
        // two buffers: the load of the next chunk is in flight while this one is processed
        float va[32], vb[32];
        if (c_begin < c_end && c_begin < c_tmem) tmem_ld32(t_addr + c_begin * 32, va);
        for (int c = c_begin; c < c_end; c += 2) {      // one 64-column group per turn
          tmem_ld_wait();
          if (c + 1 < c_end && c + 1 < c_tmem) tmem_ld32(t_addr + (c + 1) * 32, vb);
          if (c >= c_tmem || kb1 == kb0) {       // padding columns, or an empty contraction
            #pragma unroll
            for (int j = 0; j < 32; ++j) va[j] = 0.f;
          }
          epi.template chunk<0>(ep, va, n0 + c * 32);
          if (c + 1 < c_end) {
            tmem_ld_wait();
            if (c + 2 < c_end && c + 2 < c_tmem) tmem_ld32(t_addr + (c + 2) * 32, va);
            if (c + 1 >= c_tmem || kb1 == kb0) {
              #pragma unroll
              for (int j = 0; j < 32; ++j) vb[j] = 0.f;
            }
            epi.template chunk<1>(ep, vb, n0 + (c + 1) * 32);
          }
          if constexpr (Epi::PANEL) epi.group_end(ep, n0 + c * 32);
        }
        fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(acc_empty0_addr + acc * 8);
        if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      }
      if (ok) epi.end_unit(ep, un, col_half);
    }
    if (threadIdx.x == 64) SAPO_STATS_FLUSH(6);
  }

  // neither CTA may leave while the other can still touch its shared or tensor memory
  fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) { fence_after_sync(); tmem_dealloc_pair(tmem_base, TMEM_COLS); }
  if (threadIdx.x == 0 && *abort_flag) raise_status(status, SAPO_ST_WAIT_TIMEOUT);
  SAPO_CLOCK_END(sched.stats_id);
}

// ---------------------------------------------------------------------------- the wide-tile GEMM kernel
// The two long-K contractions of the backward pass (dhidden: K = vocabulary, dW_head: K = tokens)
// read the panel as A and an [K, N] matrix (W_head or hidden rows) as B, and store fp32.  Their
// tiles are long enough that the epilogue need not overlap the next tile's MMAs, so both
// accumulators of tensor memory can serve one tile: a pair works on a 256 x (2 tn) tile
// (tn <= 256) whose two halves share every A stage.  Per flop that is a quarter fewer operand
// bytes into shared memory than 256 x 256 tiles, which is what bounds these contractions.
//   A_KIND 2: A = panel read K-major  (M = tokens, K = vocab): one [128 token x 64 vocab] tile per stage
//   A_KIND 3: A = panel read MN-major (M = vocab, K = tokens): 64-token halves of two tiles per stage
//   B is stored [K, N], N contiguous: per accumulator, this CTA's tn/2 columns as 64-column boxes.
// A stage holds a K depth of 64; four stages.  Work units, K-split parts and barriers as in
// umma_gemm_kernel, with one accumulator barrier pair instead of two.
constexpr int BK2 = 64;
constexpr int STAGES2 = 4;
constexpr uint32_t A2_STAGE_BYTES = BM * BK2 * 2;          // 16 KB
constexpr uint32_t BOX2_BYTES = 64 * 128;                  // a 64-row box of 128-byte rows
constexpr uint32_t B2_ACC_BYTES = 2 * BOX2_BYTES;          // up to 128 columns per accumulator and CTA
constexpr uint32_t B2_STAGE_BYTES = 2 * B2_ACC_BYTES;      // 32 KB
// after the stages: 256 bytes of barriers, the active-block bits, then (1024-byte aligned) one
// fp32 staging tile of 128 rows x 32 columns per accumulator for the TMA stores of the epilogue
constexpr int MASK_WORDS_MAX = 448;                        // active-block bits kept in shared memory
constexpr uint32_t GEMM2_TAIL_BYTES = 2048;                // barriers + mask
constexpr uint32_t OUT_STAGING_BYTES = 128 * 128;          // per accumulator
constexpr size_t GEMM2_SMEM_BYTES =
    1024 + STAGES2 * (A2_STAGE_BYTES + B2_STAGE_BYTES) + GEMM2_TAIL_BYTES + 2 * OUT_STAGING_BYTES;
static_assert(256 + 4 * MASK_WORDS_MAX <= GEMM2_TAIL_BYTES, "barriers and mask overflow their region");
static_assert(GEMM2_SMEM_BYTES <= 232448, "more shared memory than a CTA can have");

template <int A_KIND>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
umma_gemm2_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                  const __grid_constant__ CUtensorMap map_c,   // the output (fp32 or bf16), boxes of 32 columns x 128 rows
                  const Sched sched_arg, const StoreEpi::Params ep_arg, int32_t* status) {
  static_assert(A_KIND == 2 || A_KIND == 3, "panel operands only");
  SAPO_CLOCK_BEGIN
  Sched sched = sched_arg;
  StoreEpi::Params ep = ep_arg;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + STAGES2 * A2_STAGE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES2 * (A2_STAGE_BYTES + B2_STAGE_BYTES));
  uint64_t* full = bars;                  // [STAGES2] TMA -> MMA          (even CTA's are used)
  uint64_t* empty = bars + STAGES2;       // [STAGES2] MMA -> TMA          (each CTA waits on its own)
  uint64_t* acc_full = bars + 2 * STAGES2;      // MMA -> epilogue         (each CTA waits on its own)
  uint64_t* acc_empty = bars + 2 * STAGES2 + 1; // epilogue -> MMA         (even CTA's is used)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES2 + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  uint64_t* drain = bars + 2 * STAGES2 + 3;   // MMA thread only, after a wait ran out (see umma_gemm_kernel)
  uint32_t* mask_s = reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(bars) + 256);
  uint8_t* out_staging = reinterpret_cast<uint8_t*>(bars) + GEMM2_TAIL_BYTES;
  // the mask only matters if some block of the chunk is clear: decided once, by every thread alike
  bool has_mask = false;
  if (sched.active_mask != nullptr) {
    const int n_blocks = sched.mask_dim == 1 ? (int)((ep.M + BM - 1) / BM) : (sched.num_k_blocks + 1) >> 1;
    for (int w = 0; w < sched.mask_words && !has_mask; ++w) {
      const int left = n_blocks - 32 * w;
      const uint32_t want = left >= 32 ? 0xffffffffu : (left > 0 ? (1u << left) - 1u : 0u);
      has_mask = (sched.active_mask[w] & want) != want;
    }
  }
  for (int i = threadIdx.x; has_mask && i < sched.mask_words; i += blockDim.x) mask_s[i] = sched.active_mask[i];
  // bit of 128-token block b (blocks past the mask count as clear)
  auto blk_active = [&](int b) -> bool {
    return !has_mask || (b < 32 * sched.mask_words && ((mask_s[b >> 5] >> (b & 31)) & 1u));
  };
  // A_KIND 2: an output tile none of whose rows is active needs no contraction at all
  auto rows_active = [&](int pmb) -> bool { return blk_active(2 * pmb) || blk_active(2 * pmb + 1); };
  // A_KIND 3: stage kb holds tokens [64 kb, 64 kb + 64) of block kb / 2.  The loops over stages
  // keep the mask word of the current 32 blocks in a register (`word`, reloaded every 64 stages).
  const bool skip_stages = A_KIND == 3 && has_mask;
  auto stage_active = [&](int kb, int kb_first, uint32_t& word) -> bool {
    if (!skip_stages) return true;
    if (kb == kb_first || (kb & 63) == 0) word = (kb >> 6) < sched.mask_words ? mask_s[kb >> 6] : 0u;
    return (word >> ((kb >> 1) & 31)) & 1u;
  };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr bool A_MN = A_KIND == 3;
  const uint32_t rank = cluster_cta_rank();
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
  const int tn = sched.tile_n >> 1;       // columns per accumulator
  const int half = tn >> 1;               // B columns per accumulator this CTA stages
  const int b_boxes = (half + 63) >> 6;   // 64-column boxes per accumulator (1 or 2)

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES2; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    mbar_init(acc_full, 1); mbar_init(acc_empty, 16);
    mbar_init(drain, 1);
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tensormap(&map_a);
    prefetch_tensormap(&map_b);
  }
  if (warp == 1) { tmem_alloc_pair(tmem_slot, TMEM_COLS); tmem_relinquish_pair(); }
  fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t full0_addr = map_to_cta(smem_u32(full), 0);
  const uint32_t empty_addr[2] = {map_to_cta(smem_u32(empty), 0), map_to_cta(smem_u32(empty), 1)};
  const uint32_t acc_full_addr[2] = {map_to_cta(smem_u32(acc_full), 0), map_to_cta(smem_u32(acc_full), 1)};
  const uint32_t acc_empty0_addr = map_to_cta(smem_u32(acc_empty), 0);

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (both CTAs)
    int stage = 0; uint32_t phase = 0;
    uint32_t in_flight = 0;
    bool ok = true;
    constexpr int A_BOXES = A_KIND == 2 ? 1 : 2;
    const uint32_t tx = 2 * (A2_STAGE_BYTES + 2 * b_boxes * BOX2_BYTES);
    const bool is_a = lane < A_BOXES;
    const int bidx = lane - A_BOXES;                  // B box: accumulator bidx / b_boxes, box bidx % b_boxes
    const bool mine = lane < A_BOXES + 2 * b_boxes;
    const int bj = is_a ? 0 : bidx / b_boxes, bb = is_a ? 0 : bidx - bj * b_boxes;
    WorkList work(sched, pair, num_pairs);
    int pmb, un, n_begin, n_end, kb0, kb1, slot;
    while (ok && work.next(pmb, un, n_begin, n_end, kb0, kb1, slot)) {
      const int mb = 2 * pmb + (int)rank;
      const int n0 = n_begin * sched.tile_n;
      const int bcol = n0 + bj * tn + (int)rank * half + 64 * bb;      // first column of this lane's B box
      if (A_KIND == 2 && !rows_active(pmb)) kb1 = kb0;
      uint32_t word = 0;
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!stage_active(kb, kb0, word)) continue;
        if (!mbar_wait(&empty[stage], phase ^ 1, abort_flag, sched.wait_limit)) { ok = false; break; }
        if (rank == 0 && lane == 0) mbar_arrive_expect_tx(&full[stage], tx);
        if (mine) {
          const uint32_t bar = full0_addr + stage * 8;
          if (is_a) {
            uint8_t* dst = smem_a + stage * A2_STAGE_BYTES + lane * BOX2_BYTES;
            if (A_KIND == 2)      // vocab tile kb of token block mb
              tma_load_2d_pair(dst, &map_a, bar, 0, (mb * sched.panel_nvt + kb) * BM);
            else                  // tokens [64 kb, +64): half of token block kb / 2, vocab tile 2 mb + lane
              tma_load_2d_pair(dst, &map_a, bar, 0,
                               ((kb >> 1) * sched.panel_nvt + 2 * mb + lane) * BM + (kb & 1) * 64);
          } else {
            uint8_t* dst = smem_b + stage * B2_STAGE_BYTES + bj * B2_ACC_BYTES + bb * BOX2_BYTES;
            tma_load_2d_pair(dst, &map_b, bar, bcol, kb * BK2);
          }
        }
        in_flight |= 1u << stage;
        if (++stage == STAGES2) { stage = 0; phase ^= 1; }
      }
    }
    if (!ok && rank == 0 && lane == 0) {
      for (int i = 0; i < STAGES2; ++i) {
        if (!(in_flight & (1u << i))) continue;
        const uint32_t ph = (i < stage) ? phase : (phase ^ 1);
        for (int spin = 0; spin < (1 << 20) && !mbar_try_wait(&full[i], ph); ++spin) {}
      }
    }
  } else if (warp == 1 && lane == 0 && rank == 0) {
    // ------------------------------------------------------------ MMA issuer (even CTA only)
    int stage = 0; uint32_t phase = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    const uint32_t idesc = make_idesc_bf16(PAIR_M, tn, A_MN, true);
    WorkList work(sched, pair, num_pairs);
    int pmb, un, n_begin, n_end, kb0, kb1, slot;
    while (ok && work.next(pmb, un, n_begin, n_end, kb0, kb1, slot)) {
      if (!mbar_wait(acc_empty, acc_phase ^ 1, abort_flag, sched.wait_limit)) { ok = false; break; }
      fence_after_sync();
      if (A_KIND == 2 && !rows_active(pmb)) kb1 = kb0;
      bool first = true;                       // the first stage that runs overwrites the accumulators
      uint32_t word = 0;
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!stage_active(kb, kb0, word)) continue;
        if (!mbar_wait(&full[stage], phase, abort_flag, sched.wait_limit)) { ok = false; break; }
        fence_after_sync();
        const uint32_t a_addr = smem_u32(smem_a + stage * A2_STAGE_BYTES);
        const uint32_t b_addr = smem_u32(smem_b + stage * B2_STAGE_BYTES);
        #pragma unroll
        for (int k = 0; k < BK2 / UMMA_K; ++k) {
          const uint64_t a_desc = A_MN ? make_smem_desc(a_addr + k * 2048, BOX2_BYTES, 1024)
                                       : make_smem_desc(a_addr + k * 32, 16, 1024);
          const uint32_t acc_on = (!first || k != 0) ? 1u : 0u;
          mma_bf16_pair(tmem_base, a_desc, make_smem_desc(b_addr + k * 2048, BOX2_BYTES, 1024), idesc, acc_on);
          mma_bf16_pair(tmem_base + BN, a_desc,
                        make_smem_desc(b_addr + B2_ACC_BYTES + k * 2048, BOX2_BYTES, 1024), idesc, acc_on);
        }
        first = false;
        mma_commit_pair(empty_addr[0] + stage * 8);
        mma_commit_pair(empty_addr[1] + stage * 8);
        if (++stage == STAGES2) { stage = 0; phase ^= 1; }
      }
      if (ok) {
        mma_commit_pair(acc_full_addr[0]);
        mma_commit_pair(acc_full_addr[1]);
      }
      acc_phase ^= 1;
    }
    if (!ok) {
      mma_commit_pair(map_to_cta(smem_u32(drain), 0));
      for (int spin = 0; spin < (1 << 22) && !mbar_try_wait(drain, 0); ++spin) {}
    }
  } else if (warp >= 2) {
    // ------------------------------------------------------------ epilogue (8 warps, both CTAs)
    // warps 2-5 drain the first accumulator, warps 6-9 the second; one TMEM lane quadrant each
    const int quad = warp & 3;
    const int j = (warp - 2) >> 2;
    const int r = quad * 32 + lane;
    uint32_t acc_phase = 0;
    bool ok = true;
    StoreEpi epi;
    const uint32_t buf = smem_u32(out_staging) + j * OUT_STAGING_BYTES;
    const bool elected = quad == 0 && lane == 0;     // issues and tracks this accumulator's TMA stores
    WorkList work(sched, pair, num_pairs);
    int pmb, un, n_begin, n_end, kb0, kb1, slot;
    while (ok && work.next(pmb, un, n_begin, n_end, kb0, kb1, slot)) {
      const int n0 = n_begin * sched.tile_n;
      epi.begin_unit(ep, 2 * pmb + (int)rank, r);
      epi.set_dest(ep, slot, (int)rank, r, n0, sched.part_ld);
      // did any stage run?  if not the accumulators hold nothing of this tile: store zeros
      bool any = kb1 > kb0;
      if (A_KIND == 2 && !rows_active(pmb)) any = false;
      if (A_KIND == 3 && has_mask && any) {
        any = false;
        for (int b = kb0 >> 1; b <= (kb1 - 1) >> 1 && !any; ++b) any = blk_active(b);
      }
      if (!mbar_wait(acc_full, acc_phase, abort_flag, sched.wait_limit)) { ok = false; break; }
      fence_after_sync();
      const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + j * BN;
      const int chunks = (tn + 31) >> 5;
      const int row0 = (2 * pmb + (int)rank) * BM;      // first output row of this CTA's half of the tile
      // One 32-column chunk of this thread's row.  A K-split part goes to scratch with plain
      // stores.  A whole tile goes through the staging tile of this accumulator (128-byte rows,
      // 128-byte swizzle) and leaves as one TMA store, or TMA add when accumulating, of
      // 128 rows x 32 columns: full lines, and rows / columns outside the output are clipped.
      auto emit = [&](float (&v)[32], int col0) {
        if (!any || epi.scale == 0.f) {    // (a row without a gradient gives exact zeros: its panel
          #pragma unroll                   //  block may never have been written)
          for (int q = 0; q < 32; ++q) v[q] = 0.f;
        }
        if (epi.part != nullptr) { epi.template chunk<0>(ep, v, col0); return; }
        if (col0 >= ep.N || row0 >= ep.M) return;      // nothing of this box lies inside the output
        if (elected) bulk_wait_read_all();
        named_barrier_sync(1 + j, 128);
        if (ep.out_bf16) {
          // bf16 output: rows of 64 bytes in the 64-byte swizzle (16-byte unit q of row r sits at
          // unit q ^ ((r >> 1) & 3)), as the tensor map of a bf16 output expects
          uint32_t w[16];
          pack_bf16_32(v, epi.scale, w);
          #pragma unroll
          for (int q = 0; q < 4; ++q)
            st_shared_v4(buf + r * 64 + ((q ^ ((r >> 1) & 3)) << 4), w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
        } else {
          #pragma unroll
          for (int q = 0; q < 8; ++q)
            st_shared_v4(buf + r * 128 + ((q ^ (r & 7)) << 4),
                         __float_as_uint(epi.scale * v[4 * q]), __float_as_uint(epi.scale * v[4 * q + 1]),
                         __float_as_uint(epi.scale * v[4 * q + 2]), __float_as_uint(epi.scale * v[4 * q + 3]));
        }
        fence_proxy_async_smem();
        named_barrier_sync(1 + j, 128);
        if (elected) {
          if (ep.accumulate) tma_reduce_add_2d(&map_c, buf, col0, row0);
          else               tma_store_2d(&map_c, buf, col0, row0);
          bulk_commit_group();
        }
      };
      float va[32], vb[32];
      tmem_ld32(t_addr, va);
      for (int c = 0; c < chunks; c += 2) {
        tmem_ld_wait();
        if (c + 1 < chunks) tmem_ld32(t_addr + (c + 1) * 32, vb);
        emit(va, n0 + j * tn + c * 32);
        if (c + 1 < chunks) {
          tmem_ld_wait();
          if (c + 2 < chunks) tmem_ld32(t_addr + (c + 2) * 32, va);
          emit(vb, n0 + j * tn + (c + 1) * 32);
        }
      }
      fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(acc_empty0_addr);
      acc_phase ^= 1;
    }
    if (elected) bulk_wait_all();     // stores done before shared memory goes away
  }

  fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) { fence_after_sync(); tmem_dealloc_pair(tmem_base, TMEM_COLS); }
  if (threadIdx.x == 0 && *abort_flag) raise_status(status, SAPO_ST_WAIT_TIMEOUT);
  SAPO_CLOCK_END(sched.stats_id);
}

}  // namespace sapo
