// Tile shapes and the static work schedule of the tensor-core GEMM kernels: which CTA pair takes
// which output tile (or K range of a tile), in which order, and how a ragged last wave is cut
// along K.  No method arithmetic here.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"
#include "umma.cuh"

namespace sapo {
using namespace umma;


constexpr int BM = 128;            // accumulator rows per CTA (TMEM lanes)
constexpr int PAIR_M = 256;        // rows of a tile: two CTAs of a cluster share it
constexpr int BN = 256;            // accumulator columns per tile (at most)
constexpr int BK = 128;            // K depth of a pipeline stage: two 64-element (128-byte) row segments
constexpr int UMMA_K = 16;
constexpr int STAGES = 3;
constexpr int GEMM_THREADS = 320;  // warp 0: TMA, warp 1: MMA, warps 2-9: epilogue
constexpr uint32_t A_STAGE_BYTES = BM * BK * 2;         // this CTA's 128 rows of A
constexpr uint32_t B_STAGE_BYTES = (BN / 2) * BK * 2;   // this CTA's half of the tile's B columns
constexpr uint32_t BOX_BYTES = 128 * 128;    // one 128-row box: half the K depth of a K-major operand,
                                             // or 64 columns x full K depth of an MN-major one
constexpr uint32_t TMEM_COLS = 512;          // two accumulators of 256 columns
constexpr size_t GEMM_SMEM_BYTES = 1024 + STAGES * (A_STAGE_BYTES + B_STAGE_BYTES) + 256;
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;
constexpr float EXP_CAP = 1.2676506002282294e30f;   // 2^100: a row sum of exponentials at or beyond this is out of range (fused call)

// Static tile schedule: `num_units` work units, each one 256-row block and a run of n-blocks,
// dealt round-robin to the CTA pairs.
struct Sched {
  int32_t num_m_blocks, num_n_blocks, n_per_unit, units_per_m, num_units, num_k_blocks;
  int32_t m_fastest;  // 1: neighbouring pairs share the B tile; 0: they share the A tile
  int32_t group_m;    // m_fastest only: row blocks per group; a group's A rows are meant to stay in L2
                      // while the schedule walks all n-units for it
  int32_t N;          // true extent of the n dimension
  int32_t tile_n;     // columns per tile (a multiple of 32, at most 256)
  int32_t n_cover;    // columns the epilogue visits (>= N; the dz panel is padded to 64)
  int32_t panel_nvt;  // 64-column tiles per token block of the dz panel (tiled A operands)
  // Units [0, dp_units) are dealt whole, round-robin, to the pairs.  The sk_tiles units after
  // them would leave a last wave partly empty; when cutting helps, each of them is cut along K
  // into sk_parts equal ranges and the sk_tiles * sk_parts parts are dealt round-robin, K range
  // slowest: the last wave gets shorter, and pairs that work at the same time are on the same
  // K range of different tiles, so they still share the B tiles they stream through L2.  A part
  // leaves a partial accumulator in scratch; a small second kernel adds the parts of each tile
  // in order.
  int32_t dp_units, sk_tiles, sk_parts;
  int32_t k_split_ok; // the epilogue has scratch for K-split parts
  int32_t part_ld;    // columns of a partial tile in scratch (256, or 512 for the two-accumulator kernel)
  int32_t max_parts;  // partial tiles of that width the scratch holds
  int32_t min_part_k; // shortest K range (in stages) worth a part
  // Wide-tile kernel only: one bit per 128-token block, set when any of its tokens has a
  // non-zero gradient factor (nullptr: every block counts).  mask_dim 1: the blocks are rows of
  // the output (a tile whose two blocks are both clear is stored as zeros without any MMA);
  // mask_dim 2: they are slices of the contraction (stages of a clear block are left out).
  const uint32_t* active_mask;
  int32_t mask_words, mask_dim;
  // A size only the device knows (the number of active tokens after compaction), read by
  // every CTA at start-up: dyn_dim 1 = it is M (rows), 2 = it is K (contraction length).
  const int32_t* dyn_count;
  int32_t dyn_dim;
  int32_t skip_if_empty;  // dyn_dim 2 only: a zero-length contraction launches no work at all
  int32_t stats_id;   // row of the wait-cycle counters this launch adds to (instrumented builds)
  long long wait_limit;   // SM clocks after which a barrier wait gives up (SAPO_ST_WAIT_TIMEOUT)
};

// A-operand rows fetched in place from two source buffers (the rollout stores) instead of from a
// packed copy: for every 128-token block a list of boxes, each 2^k consecutive source rows that go
// to consecutive rows of the block (a run of tokens of one sequence, cut into powers of two).
struct NoGather {};
struct GatherArgs {
  CUtensorMap maps[2][8];     // [buffer][log2 rows]: boxes of 64 columns x 2^k rows, 128-byte swizzle
  const uint64_t* boxes;      // [blocks][128]: bits 0-6 first row in the block, 7-9 log2 rows, 10 buffer, 16.. source row
  const int32_t* n_boxes;     // [blocks]: boxes | rows they cover << 16
  int64_t rows;               // token rows of this launch (those past it are not fetched)
};
constexpr uint32_t GATHER_LIST_BYTES = 128 * 8;

constexpr int PARTIAL_FLOATS = PAIR_M * BN;   // one partial accumulator tile: 256 x 256 fp32
constexpr int MAX_PAIRS_SCRATCH = 96;          // CTA pairs a launch may use (a B200 has 74)
constexpr int MAX_PARTS_SCRATCH = 3 * MAX_PAIRS_SCRATCH;   // K-split parts the scratch holds
// partial tiles are 256 rows by 256 columns, or by 512 for the wide-tile kernel: sized for those
constexpr size_t KSPLIT_SCRATCH_BYTES = (size_t)MAX_PARTS_SCRATCH * 2 * PARTIAL_FLOATS * sizeof(float);

// Decide whether (and how finely) to cut the tiles of a ragged last wave along K (see Sched).
// With `rem` tiles left over and s parts per tile the tail takes ceil(rem s / pairs) / s of a
// tile's time instead of 1; every part also pays a pipeline fill and an exposed epilogue,
// counted here as 2 % of a tile.
__host__ __device__ inline void split_last_wave(Sched& s, int pairs) {
  s.dp_units = s.num_units; s.sk_tiles = 0; s.sk_parts = 1;
  if (!s.k_split_ok || pairs <= 0 || s.n_per_unit != 1) return;
  const int rem = s.num_units % pairs;
  if (rem == 0) return;
  int best = 1; float best_cost = 1.f;
  for (int parts = 2; parts <= 8; ++parts) {
    if (s.num_k_blocks / parts < s.min_part_k) break;   // keep every range long enough to be worth a pipeline fill
    if (rem * parts > s.max_parts) break;
    const int rounds = (rem * parts + pairs - 1) / pairs;
    const float cost = (float)rounds / (float)parts + 0.02f * (float)rounds;
    if (cost < best_cost - 0.05f) { best_cost = cost; best = parts; }
  }
  if (best == 1) return;
  s.dp_units = s.num_units - rem;
  s.sk_tiles = rem;
  s.sk_parts = best;
}

// Fill in what depends on a device-side size; every CTA (and the fix-up kernel) does the same.
__device__ __forceinline__ void finalize_sched(Sched& s, int pairs) {
  if (s.dyn_dim == 0) return;
  const int32_t n = *s.dyn_count;
  if (s.dyn_dim == 1) {
    s.num_m_blocks = (n + PAIR_M - 1) / PAIR_M;
    s.num_units = s.num_m_blocks * s.units_per_m;
  } else {
    s.num_k_blocks = (n + BK - 1) / BK;
    if (n == 0 && s.skip_if_empty) s.num_units = 0;   // adding an empty sum: leave the output alone
  }
  split_last_wave(s, pairs);
}

__device__ __forceinline__ void decode_unit(const Sched& s, int unit, int& mb, int& un,
                                            int& n_begin, int& n_end) {
  if (s.m_fastest) {
    // groups of group_m row blocks; inside a group the row block runs fastest, then the n-unit
    const int per_group = s.group_m * s.units_per_m;
    const int g = unit / per_group, r = unit - g * per_group;
    const int rows_here = min(s.group_m, s.num_m_blocks - g * s.group_m);
    un = r / rows_here;
    mb = g * s.group_m + (r - un * rows_here);
  }
  else             { mb = unit / s.units_per_m;  un = unit - mb * s.units_per_m; }
  n_begin = un * s.n_per_unit;
  n_end = min(n_begin + s.n_per_unit, s.num_n_blocks);
}

// The work of one CTA pair, in order: its whole units, then its share of the K-split parts.
// Every role of both CTAs walks the same list.
struct WorkList {
  const Sched& s; int pair, n_pairs, i, tail_i;
  __device__ __forceinline__ WorkList(const Sched& s_, int pair_, int n_pairs_)
      : s(s_), pair(pair_), n_pairs(n_pairs_), i(0), tail_i(0) {}
  // slot: -1 = the tile's whole K range (normal epilogue); otherwise the scratch slot of the part
  __device__ __forceinline__ bool next(int& pmb, int& un, int& n_begin, int& n_end, int& kb0, int& kb1,
                                       int& slot) {
    const int unit = pair + i * n_pairs;
    if (unit < s.dp_units) {
      ++i;
      decode_unit(s, unit, pmb, un, n_begin, n_end);
      kb0 = 0; kb1 = s.num_k_blocks; slot = -1;
      return true;
    }
    const int part = pair + tail_i * n_pairs;       // part j of tile t has index j * sk_tiles + t
    if (part < s.sk_tiles * s.sk_parts) {
      ++tail_i;
      const int j = part / s.sk_tiles, t = part - j * s.sk_tiles;
      decode_unit(s, s.dp_units + t, pmb, un, n_begin, n_end);
      kb0 = (int)((long long)s.num_k_blocks * j / s.sk_parts);
      kb1 = (int)((long long)s.num_k_blocks * (j + 1) / s.sk_parts);
      slot = part;
      return true;
    }
    return false;
  }
};

// columns of a tile the MMA computes: the tile width, or on the last tile what is left,
// rounded up to 32 so that each CTA's half stays a multiple of 16
__device__ __forceinline__ int tile_n_eff(const Sched& s, int nb) {
  const int left = s.N - nb * s.tile_n;
  return left >= s.tile_n ? s.tile_n : ((left + 31) & ~31);
}

}  // namespace sapo
