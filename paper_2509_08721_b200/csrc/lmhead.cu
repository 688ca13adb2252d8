// LM-head projection fused with the policy loss, forward and backward, on the Blackwell
// tensor cores (tcgen05 MMA, accumulators in tensor memory, operands staged by TMA).
//
// One persistent, warp-specialised GEMM kernel (128 x 256 output tiles, 64-deep K blocks)
// serves four contractions; they differ only in operand majors and in the epilogue that
// drains the accumulator:
//   forward      S = hidden . W^T      epilogue: running max / sum-exp / target logit per token
//   backward dz  S = hidden . W^T      epilogue: dz = g (onehot - exp(S - lse)) -> bf16 panel,
//                                      stored as contiguous [128 token x 64 vocab] tiles
//   backward dH  dH = dz . W           epilogue: fp32 store
//   backward dW  dW = dz^T . hidden    epilogue: fp32 store / accumulate
// The [tokens x vocab] logits never reach global memory (paper Section 3.2 asks for the
// token-level values of every rollout under the node's policy; Section 4.2 gives the
// clipped objective the epilogue tail evaluates).
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"
#include "compact.cuh"
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
constexpr uint32_t STAGING_BYTES = 2 * 128 * 128;   // dz epilogue: one 16 KB panel tile per column half
constexpr size_t GEMM_SMEM_BYTES = 1024 + STAGES * (A_STAGE_BYTES + B_STAGE_BYTES) + 256;
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;
constexpr float EXP_CAP = 1.2676506002282294e30f;   // 2^100: cap of a stored exponential (fused call)

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
};

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

// ---------------------------------------------------------------------------- epilogues
// Each epilogue thread owns one accumulator row (TMEM lane) of the tile.

// What a staged epilogue needs to move finished 64-column groups through shared memory.
struct StageCtx {
  uint32_t buf;          // shared address of this column half's 16 KB staging tile
  int bar_id;            // named barrier of the four warps that share it
  bool elected;          // the one thread that issues and tracks the TMA stores
  const CUtensorMap* map;
};

// A thread's 64 finished bf16 entries of a panel row (two 32-column chunks as 16 pairs each)
// go to the staging tile, and the tile leaves as one 16 KB TMA store: wait until the previous
// store has read the staging tile, write this row (128 bytes, in 128-byte-swizzle order) and
// hand the tile to the TMA.  Called by all 128 threads that share the staging tile.
__device__ __forceinline__ void store_panel_group(const StageCtx& cx, int r, const uint32_t (&pk)[2][16],
                                                  int tile_row0, int col0_of_group) {
  if (cx.elected) bulk_wait_read_all();
  named_barrier_sync(cx.bar_id, 128);
  #pragma unroll
  for (int q = 0; q < 8; ++q)
    st_shared_v4(cx.buf + r * 128 + ((q ^ (r & 7)) << 4),
                 pk[q >> 2][4 * (q & 3)], pk[q >> 2][4 * (q & 3) + 1],
                 pk[q >> 2][4 * (q & 3) + 2], pk[q >> 2][4 * (q & 3) + 3]);
  fence_proxy_async_smem();
  named_barrier_sync(cx.bar_id, 128);
  if (cx.elected) {
    tma_store_2d(cx.map, cx.buf, 0, tile_row0 + (col0_of_group >> 6) * BM);
    bulk_commit_group();
  }
}

// Forward: online log-sum-exp in the base-2 domain plus the logit of the chosen token.
struct FwdEpi {
  static constexpr bool STAGED = false;
  static constexpr bool STREAMK = false;
  template <class P> __device__ static void set_dynamic(P&, const Sched&) {}

  struct Params {
    const int32_t* ids; float* pm; float* ps; float* pz;  // partials [n_splits][T]
    int64_t T; int32_t V;
  };
  float m, s, zy; int32_t y; int64_t row;
  __device__ __forceinline__ void begin_unit(const Params& p, int mb, int r) {
    row = (int64_t)mb * BM + r;
    m = -INFINITY; s = 0.f; zy = 0.f;
    y = row < p.T ? p.ids[row] : -1;
  }
  template <int HALF>
  __device__ __forceinline__ void chunk(const Params& p, float (&v)[32], int col0, const StageCtx&) {
    if (col0 >= p.V) return;
    if (col0 + 32 > p.V) {
      #pragma unroll
      for (int j = 0; j < 32; ++j) if (col0 + j >= p.V) v[j] = -INFINITY;
    }
    const int yr = y - col0;
    if (yr >= 0 && yr < 32) {
      #pragma unroll
      for (int j = 0; j < 32; ++j) if (j == yr) zy = v[j];
    }
    float cmax = v[0];
    #pragma unroll
    for (int j = 1; j < 32; ++j) cmax = fmaxf(cmax, v[j]);
    const float m_new = fmaxf(m, cmax * LOG2E);
    float acc = s * ex2(m - m_new);          // first chunk: ex2(-inf) = 0
    #pragma unroll
    for (int j = 0; j < 32; ++j) acc += ex2(fmaf(v[j], LOG2E, -m_new));
    s = acc; m = m_new;
  }
  // two threads share a row (one per column half of the tiles): each leaves its own partial
  __device__ __forceinline__ void end_unit(const Params& p, int un, int col_half) {
    if (row < p.T) {
      const int64_t o = (int64_t)(2 * un + col_half) * p.T + row;
      p.pm[o] = m; p.ps[o] = s; p.pz[o] = zy;
    }
  }
};

// Backward, first contraction: dz[t,v] = g_t ([v == y_t] - exp(z[t,v] - lse_t)), to bf16.
// The panel is a sequence of [128 token x 64 vocab] tiles of 16 KB, tile (tb, vt) at index
// tb * nvt + vt, each tile row-major: both later contractions then fetch whole contiguous
// tiles with one TMA box.  Rows past the last token and columns past V are written as zeros,
// because those consumers cannot tell them from data.  A finished 64-column group is staged in
// shared memory (128-byte swizzle) and leaves as one 16 KB TMA store.
struct DzEpi {
  static constexpr bool STAGED = true;
  static constexpr bool STREAMK = false;
  template <class P> __device__ static void set_dynamic(P& p, const Sched& s) {
    if (s.dyn_dim == 1) p.M = *s.dyn_count;
  }
  struct Params {
    const int32_t* ids; const float* lse; const float* gscale;
    int64_t M; int32_t V; int32_t nvt;
  };
  float g, l2; int32_t y; int32_t tile_row0; int r; bool in_panel;
  __device__ __forceinline__ void begin_unit(const Params& p, int mb, int r_) {
    const int64_t row = (int64_t)mb * BM + r_;
    const bool valid = row < p.M;
    in_panel = (int64_t)mb * BM < p.M;   // the odd CTA of the last pair may own no token block
    r = r_;
    tile_row0 = mb * p.nvt * BM;          // first panel row of this token block
    g = valid ? p.gscale[row] : 0.f;
    l2 = valid ? p.lse[row] * LOG2E : 0.f;
    y = valid ? p.ids[row] : -1;
  }
  __device__ __forceinline__ void group_begin(const StageCtx&) {}
  // dz of 32 columns, kept in registers as 16 bf16 pairs until the whole 64-column group is done
  uint32_t pk[2][16];
  template <int HALF>   // which 32-column half of the group (a compile-time register choice)
  __device__ __forceinline__ void chunk(const Params& p, float (&v)[32], int col0, const StageCtx&) {
    if (!in_panel) return;
    uint32_t (&packed)[16] = pk[HALF];
    if (g == 0.f) {
      #pragma unroll
      for (int j = 0; j < 16; ++j) packed[j] = 0u;
    } else {
      const float ng = -g;
      #pragma unroll
      for (int j = 0; j < 32; ++j) v[j] = ng * ex2(fmaf(v[j], LOG2E, -l2));
      const int yr = y - col0;
      if (yr >= 0 && yr < 32) {            // the chunk that holds the chosen token
        #pragma unroll
        for (int j = 0; j < 32; ++j) if (j == yr) v[j] += g;
      }
      if (col0 + 32 > p.V) {               // ragged end of the vocabulary
        #pragma unroll
        for (int j = 0; j < 32; ++j) if (col0 + j >= p.V) v[j] = 0.f;
      }
      #pragma unroll
      for (int j = 0; j < 16; ++j) {
        __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
        packed[j] = *reinterpret_cast<uint32_t*>(&h);
      }
    }
  }
  __device__ __forceinline__ void group_end(const Params&, int col0_of_group, const StageCtx& cx) {
    if (in_panel) store_panel_group(cx, r, pk, tile_row0, col0_of_group);
  }
  __device__ __forceinline__ void end_unit(const Params&, int, int) {}
};

// Forward of the fused call: e[t,v] = exp(z[t,v] - c_t) against a per-token reference c_t that
// is known before the pass (see sapo_policy_loss_fwd_bwd), so no running maximum is needed:
// the epilogue adds the fp32 exponentials up per token and leaves them, rounded to bf16, in
// the tiled panel (same layout as DzEpi) for the backward contractions, which then need no
// second pass over the logits.  Exponentials are capped at 2^100, so that sums and products
// with them stay finite and a zero row scale later still gives zero (a token that reaches the
// cap is reported, see fused_tail_kernel).  Rows past the last token and columns past V hold zeros.
struct ExpEpi {
  static constexpr bool STAGED = true;
  static constexpr bool STREAMK = false;
  template <class P> __device__ static void set_dynamic(P&, const Sched&) {}
  struct Params {
    const float* c2;      // [M] reference of each token, in the base-2 domain (c_t * log2 e)
    float* ps;            // [2 * n_splits][M] partial sums of exponentials
    int64_t M; int32_t V; int32_t nvt;
  };
  float c, sum; int32_t tile_row0; int r; bool valid, in_panel; int64_t row;
  uint32_t pk[2][16];
  __device__ __forceinline__ void begin_unit(const Params& p, int mb, int r_) {
    row = (int64_t)mb * BM + r_;
    valid = row < p.M;
    in_panel = (int64_t)mb * BM < p.M;
    r = r_;
    tile_row0 = mb * p.nvt * BM;
    c = valid ? p.c2[row] : 0.f;
    sum = 0.f;
  }
  __device__ __forceinline__ void group_begin(const StageCtx&) {}
  template <int HALF>
  __device__ __forceinline__ void chunk(const Params& p, float (&v)[32], int col0, const StageCtx&) {
    if (!in_panel) return;
    uint32_t (&packed)[16] = pk[HALF];
    if (!valid || col0 >= p.V) {
      #pragma unroll
      for (int j = 0; j < 16; ++j) packed[j] = 0u;
      return;
    }
    const float cap = EXP_CAP;
    #pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = fminf(ex2(fmaf(v[j], LOG2E, -c)), cap);
    if (col0 + 32 > p.V) {               // ragged end of the vocabulary
      #pragma unroll
      for (int j = 0; j < 32; ++j) if (col0 + j >= p.V) v[j] = 0.f;
    }
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
    #pragma unroll
    for (int j = 0; j < 32; j += 4) { a0 += v[j]; a1 += v[j + 1]; a2 += v[j + 2]; a3 += v[j + 3]; }
    sum += (a0 + a1) + (a2 + a3);
    #pragma unroll
    for (int j = 0; j < 16; ++j) {
      __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
      packed[j] = *reinterpret_cast<uint32_t*>(&h);
    }
  }
  __device__ __forceinline__ void group_end(const Params&, int col0_of_group, const StageCtx& cx) {
    if (in_panel) store_panel_group(cx, r, pk, tile_row0, col0_of_group);
  }
  // two threads share a row (one per column half of the tiles): each leaves its own partial
  __device__ __forceinline__ void end_unit(const Params& p, int un, int col_half) {
    if (valid) p.ps[(int64_t)(2 * un + col_half) * p.M + row] = sum;
  }
};

// Plain fp32 output tile, optionally added to what is already there.
struct StoreEpi {
  static constexpr bool STAGED = false;
  static constexpr bool STREAMK = true;
  // row_map (optional): output row of each accumulator row (rows of compacted tokens go back
  // to their packed positions)
  // row_scale (optional): factor applied to each accumulator row before it is stored
  struct Params { float* C; int64_t ldc; int64_t M; int32_t N; int32_t accumulate; float* partials;
                  const int32_t* row_map; const float* row_scale; };
  template <class P> __device__ static void set_dynamic(P& p, const Sched& s) {
    if (s.dyn_dim == 1) p.M = *s.dyn_count;
  }
  int64_t row; bool valid; float* part; int n0; float scale;
  __device__ __forceinline__ void begin_unit(const Params& p, int mb, int r) {
    row = (int64_t)mb * BM + r;
    valid = row < p.M;
    scale = (valid && p.row_scale != nullptr) ? p.row_scale[row] : 1.f;
    if (valid && p.row_map != nullptr) row = p.row_map[row];
    part = nullptr;
  }
  // a K-split part of a tile goes to scratch slot `slot` instead: rows [128 rank, +128) of a
  // 256 x 256 fp32 tile, column 0 = the tile's first column
  __device__ __forceinline__ void set_dest(const Params& p, int slot, int rank, int r, int n0_, int part_ld) {
    n0 = n0_;
    part = slot < 0 ? nullptr
                    : p.partials + ((size_t)slot * PAIR_M + (size_t)(rank * BM + r)) * part_ld;
  }
  template <int HALF>
  __device__ __forceinline__ void chunk(const Params& p, float (&v)[32], int col0, const StageCtx&) {
    if (part != nullptr) {
      float4* dst = reinterpret_cast<float4*>(part + (col0 - n0));
      #pragma unroll
      for (int q = 0; q < 8; ++q) dst[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
      return;
    }
    if (!valid) return;
    float4* dst = reinterpret_cast<float4*>(p.C + row * p.ldc + col0);
    #pragma unroll
    for (int q = 0; q < 8; ++q) {
      if (col0 + 4 * q < p.N) {          // N is a multiple of 4
        float4 o = make_float4(scale * v[4 * q], scale * v[4 * q + 1], scale * v[4 * q + 2],
                               scale * v[4 * q + 3]);
        if (p.accumulate) { const float4 c = dst[q]; o.x += c.x; o.y += c.y; o.z += c.z; o.w += c.w; }
        dst[q] = o;
      }
    }
  }
  __device__ __forceinline__ void end_unit(const Params&, int, int) {}
};

// Adds up the K-split parts of each tile the GEMM kernel left in scratch and stores the sum.
// Part order is fixed (by pair index), so the result does not depend on timing.
__global__ void __launch_bounds__(256)
streamk_fixup_kernel(const Sched s_arg, const StoreEpi::Params p_arg, int pairs) {
  Sched s = s_arg;
  StoreEpi::Params p = p_arg;
  finalize_sched(s, pairs);
  StoreEpi::set_dynamic(p, s);
  const int t = blockIdx.x >> 5;                 // K-split tile
  if (t >= s.sk_tiles) return;
  const int row_begin = (blockIdx.x & 31) * 8;   // 8 of its 256 rows per block
  if (s.sk_parts <= 1) return;                   // whole tiles were stored by their pair
  int pmb, un, n_begin, n_end;
  decode_unit(s, s.dp_units + t, pmb, un, n_begin, n_end);
  const int n0 = n_begin * s.tile_n;
  const size_t part_floats = (size_t)PAIR_M * s.part_ld;
  // 8 rows x (columns / 4) float4 items per block; N, tile widths and leading dimensions are multiples of 4
  const int n4 = min(s.tile_n, p.N - n0) >> 2;
  for (int item = threadIdx.x; item < 8 * n4; item += blockDim.x) {
    const int rr = row_begin + item / n4, c4 = item - (item / n4) * n4;
    int64_t row = (int64_t)pmb * PAIR_M + rr;
    if (row >= p.M) continue;
    const float scale = p.row_scale != nullptr ? p.row_scale[row] : 1.f;
    if (p.row_map != nullptr) row = p.row_map[row];
    const float* src = p.partials + (size_t)t * part_floats + (size_t)rr * s.part_ld + 4 * c4;
    float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
    #pragma unroll 4
    for (int j = 0; j < s.sk_parts; ++j) {
      const float4 v = *reinterpret_cast<const float4*>(src + (size_t)j * s.sk_tiles * part_floats);
      sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
    }
    float4* dst = reinterpret_cast<float4*>(p.C + row * p.ldc + n0 + 4 * c4);
    float4 o = make_float4(scale * sum.x, scale * sum.y, scale * sum.z, scale * sum.w);
    if (p.accumulate) { const float4 c = *dst; o.x += c.x; o.y += c.y; o.z += c.z; o.w += c.w; }
    *dst = o;
  }
}

// Optional instrumentation (compile with -DSAPO_WAIT_STATS): cycles each role spends waiting.
#ifdef SAPO_WAIT_STATS
__device__ unsigned long long g_wait_stats[4][8];
#define SAPO_TIMED(slot, expr) ([&] { const long long t0_ = clock64(); const bool r_ = (expr); \
                                      wait_cycles[slot] += clock64() - t0_; return r_; }())
#define SAPO_STATS_DECL long long wait_cycles[8] = {0, 0, 0, 0, 0, 0, 0, 0}; const long long role_t0 = clock64();
#define SAPO_STATS_FLUSH(total_slot) do { wait_cycles[total_slot] += clock64() - role_t0; \
    for (int i_ = 0; i_ < 8; ++i_) if (wait_cycles[i_]) \
      atomicAdd(&g_wait_stats[sched.stats_id & 3][i_], (unsigned long long)wait_cycles[i_]); } while (0)
#else
#define SAPO_TIMED(slot, expr) (expr)
#define SAPO_STATS_DECL
#define SAPO_STATS_FLUSH(total_slot) do {} while (0)
#endif

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
template <int A_KIND, bool B_MN, class Epi>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
umma_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const __grid_constant__ CUtensorMap map_c,   // output tiles of a staged epilogue
                 const Sched sched_arg, const typename Epi::Params ep_arg, int32_t* status) {
  Sched sched = sched_arg;
  typename Epi::Params ep = ep_arg;
  finalize_sched(sched, (int)(gridDim.x >> 1));
  Epi::set_dynamic(ep, sched);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + STAGES * A_STAGE_BYTES;
  uint8_t* staging = smem + STAGES * (A_STAGE_BYTES + B_STAGE_BYTES);   // STAGED epilogues only
  uint64_t* bars = reinterpret_cast<uint64_t*>(staging + (Epi::STAGED ? STAGING_BYTES : 0));
  uint64_t* full = bars;                 // [STAGES] TMA -> MMA          (even CTA's are used)
  uint64_t* empty = bars + STAGES;       // [STAGES] MMA -> TMA          (each CTA waits on its own)
  uint64_t* acc_full = bars + 2 * STAGES;      // [2] MMA -> epilogue    (each CTA waits on its own)
  uint64_t* acc_empty = bars + 2 * STAGES + 2; // [2] epilogue -> MMA    (even CTA's are used)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr bool A_MN = (A_KIND & 1) != 0;
  const uint32_t rank = cluster_cta_rank();
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], 16); }
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
    constexpr int A_BOXES = A_KIND == 2 ? 1 : 2;
    WorkList work(sched, pair, num_pairs);
    int pmb, un, n_begin, n_end, kb0, kb1, slot;
    while (ok && work.next(pmb, un, n_begin, n_end, kb0, kb1, slot)) {
      const int mb = 2 * pmb + (int)rank;                 // this CTA's 128-row block
      for (int nb = n_begin; ok && nb < n_end; ++nb) {
        const int half = tile_n_eff(sched, nb) >> 1;       // B columns this CTA stages
        const int b_boxes = B_MN ? ((half + 63) >> 6) : 2;
        const uint32_t tx = 2 * (A_STAGE_BYTES + b_boxes * BOX_BYTES);
        const bool mine = lane < A_BOXES + b_boxes;
        const bool is_a = lane < A_BOXES;
        const int bi = is_a ? lane : lane - A_BOXES;
        const CUtensorMap* map = is_a ? &map_a : &map_b;
        const uint32_t dst_off = is_a ? bi * BOX_BYTES : STAGES * A_STAGE_BYTES + bi * BOX_BYTES;
        const bool mn = is_a ? A_MN : B_MN;
        // m or n coordinate of the box (an MN-major box covers 64 of them, a K-major one 128)
        const int row0 = is_a ? mb * BM + (mn ? 64 * bi : 0)
                              : nb * sched.tile_n + (int)rank * half + (mn ? 64 * bi : 0);
        const int k_off = mn ? 0 : 64 * bi;                // K-major boxes split the stage's K depth
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!SAPO_TIMED(0, mbar_wait(&empty[stage], phase ^ 1, abort_flag))) { ok = false; break; }
          if (rank == 0 && lane == 0) mbar_arrive_expect_tx(&full[stage], tx);
          if (mine) {
            uint8_t* dst = smem + dst_off + stage * (is_a ? A_STAGE_BYTES : B_STAGE_BYTES);
            const uint32_t bar = full0_addr + stage * 8;
            if (is_a && A_KIND == 2)        // vocab tiles 2 kb and 2 kb + 1 of token block mb: 256 rows
              tma_load_2d_pair(dst, map, bar, 0, (mb * sched.panel_nvt + 2 * kb) * BM);
            else if (is_a && A_KIND == 3)   // token block kb, vocab tile 2 mb + bi: all 128 rows
              tma_load_2d_pair(dst, map, bar, 0, (kb * sched.panel_nvt + 2 * mb + bi) * BM);
            else if (mn) tma_load_2d_pair(dst, map, bar, row0, kb * BK);
            else         tma_load_2d_pair(dst, map, bar, kb * BK + k_off, row0);
          }
          in_flight |= 1u << stage;
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
    if (lane == 0) SAPO_STATS_FLUSH(4);
    if (!ok && rank == 0 && lane == 0) {
      // give copies already issued a bounded chance to land before the pair leaves
      for (int i = 0; i < STAGES; ++i) {
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
        if (!SAPO_TIMED(2, mbar_wait(&acc_empty[acc], acc_phase ^ 1, abort_flag))) { ok = false; break; }
        fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!SAPO_TIMED(1, mbar_wait(&full[stage], phase, abort_flag))) { ok = false; break; }
          fence_after_sync();
          const uint32_t a_addr = smem_u32(smem_a + stage * A_STAGE_BYTES);
          const uint32_t b_addr = smem_u32(smem_b + stage * B_STAGE_BYTES);
          #pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
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
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (ok) {                                  // accumulator complete, in both CTAs
          mma_commit_pair(acc_full_addr[0] + acc * 8);
          mma_commit_pair(acc_full_addr[1] + acc * 8);
        }
        if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      }
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
    StageCtx cx;
    cx.buf = smem_u32(staging) + col_half * (STAGING_BYTES / 2);
    cx.bar_id = 1 + col_half;
    cx.elected = quad == 0 && lane == 0;
    cx.map = &map_c;
    WorkList work(sched, pair, num_pairs);
    int pmb, un, n_begin, n_end, kb0, kb1, slot;
    while (ok && work.next(pmb, un, n_begin, n_end, kb0, kb1, slot)) {
      epi.begin_unit(ep, 2 * pmb + (int)rank, r);
      if constexpr (Epi::STREAMK) epi.set_dest(ep, slot, (int)rank, r, n_begin * sched.tile_n, sched.part_ld);
      for (int nb = n_begin; ok && nb < n_end; ++nb) {
        if (!SAPO_TIMED(3, mbar_wait(&acc_full[acc], acc_phase, abort_flag))) { ok = false; break; }
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
          if constexpr (Epi::STAGED) epi.group_begin(cx);
          epi.template chunk<0>(ep, va, n0 + c * 32, cx);
          if (c + 1 < c_end) {
            tmem_ld_wait();
            if (c + 2 < c_end && c + 2 < c_tmem) tmem_ld32(t_addr + (c + 2) * 32, va);
            if (c + 1 >= c_tmem || kb1 == kb0) {
              #pragma unroll
              for (int j = 0; j < 32; ++j) vb[j] = 0.f;
            }
            epi.template chunk<1>(ep, vb, n0 + (c + 1) * 32, cx);
          }
          if constexpr (Epi::STAGED) epi.group_end(ep, n0 + c * 32, cx);
        }
        fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(acc_empty0_addr + acc * 8);
        if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      }
      if (ok) epi.end_unit(ep, un, col_half);
    }
    if (Epi::STAGED && cx.elected) bulk_wait_all();   // stores done before shared memory goes away
    if (threadIdx.x == 64) SAPO_STATS_FLUSH(6);
  }

  // neither CTA may leave while the other can still touch its shared or tensor memory
  fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) { fence_after_sync(); tmem_dealloc_pair(tmem_base, TMEM_COLS); }
  if (threadIdx.x == 0 && *abort_flag) raise_status(status, SAPO_ST_WAIT_TIMEOUT);
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
                  const __grid_constant__ CUtensorMap map_c,   // the fp32 output, boxes of 32 columns x 128 rows
                  const Sched sched_arg, const StoreEpi::Params ep_arg, int32_t* status) {
  static_assert(A_KIND == 2 || A_KIND == 3, "panel operands only");
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
        if (!mbar_wait(&empty[stage], phase ^ 1, abort_flag)) { ok = false; break; }
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
      if (!mbar_wait(acc_empty, acc_phase ^ 1, abort_flag)) { ok = false; break; }
      fence_after_sync();
      if (A_KIND == 2 && !rows_active(pmb)) kb1 = kb0;
      bool first = true;                       // the first stage that runs overwrites the accumulators
      uint32_t word = 0;
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!stage_active(kb, kb0, word)) continue;
        if (!mbar_wait(&full[stage], phase, abort_flag)) { ok = false; break; }
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
  } else if (warp >= 2) {
    // ------------------------------------------------------------ epilogue (8 warps, both CTAs)
    // warps 2-5 drain the first accumulator, warps 6-9 the second; one TMEM lane quadrant each
    const int quad = warp & 3;
    const int j = (warp - 2) >> 2;
    const int r = quad * 32 + lane;
    uint32_t acc_phase = 0;
    bool ok = true;
    StoreEpi epi;
    StageCtx cx{};
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
      if (!mbar_wait(acc_full, acc_phase, abort_flag)) { ok = false; break; }
      fence_after_sync();
      const uint32_t t_addr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + j * BN;
      const int chunks = (tn + 31) >> 5;
      const int row0 = (2 * pmb + (int)rank) * BM;      // first output row of this CTA's half of the tile
      // One 32-column chunk of this thread's row.  A K-split part goes to scratch with plain
      // stores.  A whole tile goes through the staging tile of this accumulator (128-byte rows,
      // 128-byte swizzle) and leaves as one TMA store, or TMA add when accumulating, of
      // 128 rows x 32 columns: full lines, and rows / columns outside the output are clipped.
      auto emit = [&](float (&v)[32], int col0) {
        if (!any) {
          #pragma unroll
          for (int q = 0; q < 32; ++q) v[q] = 0.f;
        }
        if (epi.part != nullptr) { epi.template chunk<0>(ep, v, col0, cx); return; }
        if (col0 >= ep.N || row0 >= ep.M) return;      // nothing of this box lies inside the output
        if (elected) bulk_wait_read_all();
        named_barrier_sync(1 + j, 128);
        #pragma unroll
        for (int q = 0; q < 8; ++q)
          st_shared_v4(buf + r * 128 + ((q ^ (r & 7)) << 4),
                       __float_as_uint(epi.scale * v[4 * q]), __float_as_uint(epi.scale * v[4 * q + 1]),
                       __float_as_uint(epi.scale * v[4 * q + 2]), __float_as_uint(epi.scale * v[4 * q + 3]));
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
}

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

// One block per sequence: merge the vocab-split partials, then the clipped surrogate.
__global__ void __launch_bounds__(256) loss_tail_kernel(TailArgs a) {
  __shared__ double sh[8];
  for (int32_t s = blockIdx.x; s < a.S; s += gridDim.x) {
    const int32_t t0 = a.cu[s], t1 = a.cu[s + 1];
    const int32_t Ts = t1 - t0;
    const float A = a.adv[s];
    // weight of a token of this sequence: 1/(S T_s) (mean of token means) or 1/T (token mean)
    const float w = Ts <= 0 ? 0.f : (a.loss_agg == 0 ? 1.f / ((float)a.S * (float)Ts) : 1.f / (float)a.T);
    double acc = 0.0;
    for (int32_t t = t0 + threadIdx.x; t < t1; t += 256) {
      float M = -INFINITY;
      for (int i = 0; i < a.n_splits; ++i) M = fmaxf(M, a.pm[(int64_t)i * a.T + t]);
      float sum = 0.f, zy = 0.f;
      for (int i = 0; i < a.n_splits; ++i) {
        const int64_t o = (int64_t)i * a.T + t;
        sum += a.ps[o] * exp2f(a.pm[o] - M);
        zy += a.pz[o];
      }
      const float lse = (M + log2f(sum)) * LN2;
      const int32_t y = a.ids[t];
      const bool bad = y < 0 || y >= a.V;
      if (bad) raise_status(a.status, SAPO_ST_BAD_TOKEN_ID);
      const float lp = bad ? 0.f : zy - lse;
      const float rho = bad ? 0.f : expf(lp - a.old_logp[t]);
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
}

// loss = -(1/S) sum_s seq_surr[s], or with token-level aggregation -(1/T) sum_s T_s seq_surr[s]
__global__ void __launch_bounds__(256)
loss_final_kernel(const float* seq_surr, const int32_t* cu, int32_t S, int64_t T, int32_t loss_agg, float* loss) {
  __shared__ double sh[8];
  double acc = 0.0;
  for (int32_t s = threadIdx.x; s < S; s += 256)
    acc += loss_agg == 0 ? (double)seq_surr[s] : (double)seq_surr[s] * (double)(cu[s + 1] - cu[s]);
  const double tot = block_sum_256(acc, sh);
  const double n = loss_agg == 0 ? (double)S : (double)T;
  if (threadIdx.x == 0) *loss = n > 0 ? (float)(-tot / n) : 0.f;
}

// ---------------------------------------------------------------------------- fused call: small kernels
// Before the forward pass of the fused call: the logit of the chosen token, z_y[t] = <h_t, W_y>,
// as a plain fp32 dot product (one warp per token), and the reference of the exponentials
//   c_t = z_y[t] - old_logp[t],
// which equals lse_t when the policy has not moved since old_logp was taken and is off by
// log(ratio_t) otherwise: exp(z - c_t) then stays within a few powers of e of a probability.
// c2 is c_t * log2(e).  A token id outside [0, V) gets z_y = c = 0 (the tail reports it).
__global__ void __launch_bounds__(256)
target_logit_kernel(const __nv_bfloat16* __restrict__ hidden, int64_t ldh, const __nv_bfloat16* __restrict__ W,
                    int64_t ldw, const int32_t* __restrict__ ids, const float* __restrict__ old_logp,
                    int64_t T, int32_t H, int32_t V, float* __restrict__ zy, float* __restrict__ c2) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int64_t n_warps = (int64_t)gridDim.x * 8;
  for (int64_t t = warp; t < T; t += n_warps) {
    const int32_t y = ids[t];
    float acc = 0.f;
    if (y >= 0 && y < V) {
      const uint4* a = reinterpret_cast<const uint4*>(hidden + t * ldh);
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
      zy[t] = ok ? acc : 0.f;
      c2[t] = ok ? (acc - old_logp[t]) * LOG2E : 0.f;
    }
  }
}

struct FusedTailArgs {
  const float* ps; int32_t n_parts; int64_t t0, tc;        // partial sums [n_parts][tc] of this token chunk
  const float* zy; const float* c2;                        // [T]
  const int32_t* ids; int32_t V; const float* old_logp; const float* adv; const int32_t* cu; int32_t S;
  int64_t T; float lo_edge, hi_edge, grad_scale; int32_t loss_agg; float kl_beta; const float* ref_logp;
  float* logp; float* lse; float* ratio; float* surr; float* gscale; float* obj;   // [T]
  float* row_scale;                                        // [tc]
  __nv_bfloat16* panel; int32_t nvt;                       // exponentials of the chunk
  const __nv_bfloat16* hidden; int64_t ldh; int32_t H; __nv_bfloat16* hs;   // hs [tc, H] = row_scale * hidden
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
  for (int64_t lr = warp; lr < a.tc; lr += n_warps) {
    const int64_t t = a.t0 + lr;
    float part = 0.f;
    for (int i = lane; i < a.n_parts; i += 32) part += a.ps[(int64_t)i * a.tc + lr];
    #pragma unroll
    for (int d = 16; d > 0; d >>= 1) part += __shfl_xor_sync(0xffffffffu, part, d);
    const float sum = part;
    // the sequence of this token: last s with cu[s] <= t
    int lo = 0, hi = a.S - 1;
    while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if ((int64_t)a.cu[mid] <= t) lo = mid; else hi = mid - 1; }
    const int32_t Ts = a.cu[lo + 1] - a.cu[lo];
    const float A = a.adv[lo];
    const float w = Ts <= 0 ? 0.f : (a.loss_agg == 0 ? 1.f / ((float)a.S * (float)Ts) : 1.f / (float)a.T);
    const int32_t y = a.ids[t];
    const bool bad_id = y < 0 || y >= a.V;
    // a capped exponential, or a sum that left the fp32 range: the reference was too far off
    const bool bad_range = !(sum < EXP_CAP) || !(sum > 1.f / EXP_CAP);
    const bool bad = bad_id || bad_range;
    const float c2 = a.c2[t], zy = a.zy[t];
    const float lse = bad_range ? 0.f : (c2 + log2f(sum)) * LN2;
    const float lp = bad ? 0.f : zy - lse;
    const float rho = bad ? 0.f : expf(lp - a.old_logp[t]);
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
      if (bad_range) raise_status(a.status, SAPO_ST_EXP_RANGE);
      a.lse[t] = lse; a.logp[t] = lp; a.ratio[t] = rho; a.surr[t] = u; a.gscale[t] = g; a.obj[t] = obj;
      a.row_scale[lr] = scale;
      if (scale != 0.f && a.active_mask != nullptr)
        atomicOr(&a.active_mask[lr >> 12], 1u << ((lr >> 7) & 31));
      if (!bad) {
        const float ey = ex2(fmaf(zy, LOG2E, -c2));
        const int64_t tile = (lr >> 7) * a.nvt + (y >> 6);
        a.panel[(tile * BM + (lr & 127)) * 64 + (y & 63)] = __float2bfloat16_rn(ey - sum);
      }
    }
    const uint4* src = reinterpret_cast<const uint4*>(a.hidden + t * a.ldh);
    uint4* dst = reinterpret_cast<uint4*>(a.hs + lr * (int64_t)a.H);
    for (int i = lane; i < a.H / 8; i += 32) {
      uint4 x = src[i];
      __nv_bfloat162* px = reinterpret_cast<__nv_bfloat162*>(&x);
      #pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 f = __bfloat1622float2(px[j]);
        px[j] = __floats2bfloat162_rn(scale * f.x, scale * f.y);
      }
      dst[i] = x;
    }
  }
}

// seq_surr[s] = mean over the tokens of s of obj[t] (same summation order as loss_tail_kernel)
__global__ void __launch_bounds__(256)
seq_mean_kernel(const float* __restrict__ obj, const int32_t* __restrict__ cu, int32_t S, float* seq_surr) {
  __shared__ double sh[8];
  for (int32_t s = blockIdx.x; s < S; s += gridDim.x) {
    const int32_t t0 = cu[s], t1 = cu[s + 1];
    double acc = 0.0;
    for (int32_t t = t0 + threadIdx.x; t < t1; t += 256) acc += (double)obj[t];
    const double tot = block_sum_256(acc, sh);
    if (threadIdx.x == 0) seq_surr[s] = t1 > t0 ? (float)(tot / (double)(t1 - t0)) : 0.f;
  }
}

// ---------------------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 matrix [outer, inner] with `ld` elements between rows; boxes are 64 elements wide
// (128 bytes, 128-byte swizzle) and `box_outer` rows high.  Out-of-range elements read as 0.
static bool make_map(CUtensorMap* map, const void* base, int64_t inner, int64_t outer, int64_t ld,
                     int box_outer) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr || inner <= 0 || outer <= 0) return false;
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {64u, (cuuint32_t)box_outer};
  cuuint32_t estr[2] = {1u, 1u};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// fp32 matrix [outer, inner] with `ld` elements between rows, for stores of 32-column x 128-row
// boxes (128 bytes wide, 128-byte swizzle); elements outside the matrix are not written.
static bool make_map_f32_out(CUtensorMap* map, const float* base, int64_t inner, int64_t outer, int64_t ld) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr || inner <= 0 || outer <= 0) return false;
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 4};
  cuuint32_t box[2] = {32u, 128u};
  cuuint32_t estr[2] = {1u, 1u};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static Sched make_sched(int64_t M, int64_t N, int64_t K, int n_splits, bool m_fastest, int tile_align = 32) {
  Sched s{};
  s.num_m_blocks = (int32_t)ceil_div<int64_t>(M, PAIR_M);
  const int64_t tiles = ceil_div<int64_t>(N, BN);
  s.tile_n = (int32_t)round_up<int64_t>(ceil_div<int64_t>(N, tiles), tile_align);   // equal-width tiles
  s.num_n_blocks = (int32_t)ceil_div<int64_t>(N, s.tile_n);
  s.n_per_unit = n_splits > 0 ? ceil_div(s.num_n_blocks, n_splits) : 1;
  s.units_per_m = ceil_div(s.num_n_blocks, s.n_per_unit);
  s.num_units = s.num_m_blocks * s.units_per_m;
  s.num_k_blocks = (int32_t)ceil_div<int64_t>(K, BK);
  s.m_fastest = m_fastest ? 1 : 0;
  // row blocks whose A rows (256 x K bf16 each) fit in about 48 MB of the 126 MB L2
  {
    const int64_t fit = (48ll << 20) / (PAIR_M * (int64_t)K * 2);
    s.group_m = (int32_t)(fit < 1 ? 1 : (fit > s.num_m_blocks ? s.num_m_blocks : fit));
    if (s.group_m < 1) s.group_m = 1;
  }
  s.N = (int32_t)N;
  s.n_cover = (int32_t)N;
  s.panel_nvt = 0;
  s.dp_units = s.num_units; s.sk_tiles = 0; s.sk_parts = 1;
  s.k_split_ok = 0; s.dyn_count = nullptr; s.dyn_dim = 0; s.skip_if_empty = 0;
  s.part_ld = BN; s.max_parts = MAX_PARTS_SCRATCH; s.min_part_k = 16;
  s.active_mask = nullptr; s.mask_words = 0; s.mask_dim = 0;
  return s;
}

// Number of vocab splits of the forward pass: enough units to keep every CTA pair busy when
// there are few token blocks, never more than there are vocab tiles.
static int fwd_splits(int64_t T, int32_t V, int64_t K, int sms) {
  const int64_t pairs = sms / 2 > 0 ? sms / 2 : 1;
  const int64_t mb = ceil_div<int64_t>(T, PAIR_M);
  const int64_t nb = ceil_div<int64_t>(V, BN);
  int64_t best = 1; double best_eff = 0.0;
  for (int64_t sp = 1; sp <= 160 && sp <= nb; ++sp) {
    const int64_t per = ceil_div(nb, sp);
    const int64_t units = mb * ceil_div(nb, per);
    const double eff = (double)units / (double)(ceil_div<int64_t>(units, pairs) * pairs);
    if (eff > best_eff + 1e-9) { best_eff = eff; best = sp; }
    if (units >= 8 * pairs) break;
  }
  // a wave of pairs should not span more row blocks than stay resident in L2 (see Sched::group_m)
  const int64_t fit = (48ll << 20) / (PAIR_M * (int64_t)K * 2);
  const int64_t group = fit < 1 ? 1 : fit;
  if (group < pairs && group < mb) {
    const int64_t want = ceil_div(pairs, group);
    if (best < want) best = want < nb ? want : nb;
  }
  const int64_t per = ceil_div(nb, best);
  return (int)ceil_div(nb, per);
}

template <int A_KIND, bool B_MN, class Epi>
static int launch_gemm(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mc, const Sched& sched,
                       const typename Epi::Params& ep, int32_t* status, cudaStream_t st, int kernel_id) {
  auto kern = umma_gemm_kernel<A_KIND, B_MN, Epi>;
  static int max_pairs = 0;     // CTA pairs the device can hold at once, found on first use
  if (sched.num_units <= 0) return SAPO_OK;
  Sched sc = sched;
  sc.stats_id = (kernel_id == SAPO_K_FWD_GEMM || kernel_id == SAPO_K_FWD_EXP) ? 0 : kernel_id - SAPO_K_BWD_DZ + 1;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(GEMM_THREADS, 1, 1);
  constexpr size_t smem_bytes = GEMM_SMEM_BYTES + (Epi::STAGED ? STAGING_BYTES : 0);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (max_pairs == 0) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes) !=
        cudaSuccess)
      return SAPO_ERR_CUDA;
    const int sms = sm_count();
    if (sms <= 0) return SAPO_ERR_CUDA;
    cfg.gridDim = dim3(sms & ~1, 1, 1);
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n <= 0) return SAPO_ERR_CUDA;
    max_pairs = n < sms / 2 ? n : sms / 2;
    if (max_pairs > MAX_PAIRS_SCRATCH) max_pairs = MAX_PAIRS_SCRATCH;
  }
  int pairs = sched.num_units < max_pairs ? sched.num_units : max_pairs;
  if (sc.dyn_dim != 0) pairs = max_pairs;          // sized on the device: bring every pair
  if constexpr (Epi::STREAMK) {
    sc.k_split_ok = ep.partials != nullptr ? 1 : 0;
    if (sc.dyn_dim == 0) {
      split_last_wave(sc, max_pairs);
      if (sc.sk_tiles > 0) pairs = max_pairs;
    }
  }
  cfg.gridDim = dim3(2 * pairs, 1, 1);
  {
    KernelScope scope(kernel_id, st);
    if (cudaLaunchKernelEx(&cfg, kern, ma, mb, mc, sc, ep, status) != cudaSuccess) return SAPO_ERR_CUDA;
  }
  if constexpr (Epi::STREAMK) {
    // with a device-side size the number of K-split tiles is not known here: launch for the
    // most there can be, the kernel drops the blocks it does not need
    const int fix_tiles = sc.dyn_dim != 0 ? (sc.k_split_ok ? pairs - 1 : 0) : sc.sk_tiles;
    if (fix_tiles > 0) {
      KernelScope scope(SAPO_K_STREAMK_FIXUP, st);
      streamk_fixup_kernel<<<fix_tiles * 32, 256, 0, st>>>(sc, ep, pairs);
    }
  }
  return check_launch();
}

// Schedule of the wide-tile kernel: equal-width tiles of up to 512 columns (two accumulators),
// 64-deep stages, partial tiles of 512 columns in the K-split scratch.
static Sched make_sched_wide(int64_t M, int64_t N, int64_t K) {
  Sched s = make_sched(M, N, K, 0, /*m_fastest=*/false);
  const int64_t tiles = ceil_div<int64_t>(N, 2 * BN);
  s.tile_n = (int32_t)round_up<int64_t>(ceil_div<int64_t>(N, tiles), 64);
  s.num_n_blocks = (int32_t)ceil_div<int64_t>(N, s.tile_n);
  s.n_per_unit = 1;
  s.units_per_m = s.num_n_blocks;
  s.num_units = s.num_m_blocks * s.units_per_m;
  s.num_k_blocks = (int32_t)ceil_div<int64_t>(K, BK2);
  s.dp_units = s.num_units;
  s.part_ld = 2 * BN; s.max_parts = MAX_PARTS_SCRATCH; s.min_part_k = 32;
  return s;
}
// the wide tiles pay off once the output is at least one full accumulator wide
static bool use_wide_tiles(int32_t N) { return N >= BN; }

template <int A_KIND>
static int launch_gemm_wide(const CUtensorMap& ma, const CUtensorMap& mb, const Sched& sched,
                            const StoreEpi::Params& ep, int32_t* status, cudaStream_t st, int kernel_id) {
  CUtensorMap mc;
  if (!make_map_f32_out(&mc, ep.C, ep.N, ep.M, ep.ldc)) return SAPO_ERR_CUDA;
  auto kern = umma_gemm2_kernel<A_KIND>;
  static int max_pairs = 0;
  if (sched.num_units <= 0) return SAPO_OK;
  Sched sc = sched;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(GEMM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = GEMM2_SMEM_BYTES;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (max_pairs == 0) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GEMM2_SMEM_BYTES) !=
        cudaSuccess)
      return SAPO_ERR_CUDA;
    const int sms = sm_count();
    if (sms <= 0) return SAPO_ERR_CUDA;
    cfg.gridDim = dim3(sms & ~1, 1, 1);
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n <= 0) return SAPO_ERR_CUDA;
    max_pairs = n < sms / 2 ? n : sms / 2;
    if (max_pairs > MAX_PAIRS_SCRATCH) max_pairs = MAX_PAIRS_SCRATCH;
  }
  int pairs = sched.num_units < max_pairs ? sched.num_units : max_pairs;
  sc.k_split_ok = ep.partials != nullptr ? 1 : 0;
  split_last_wave(sc, max_pairs);
  if (sc.sk_tiles > 0) pairs = max_pairs;
  cfg.gridDim = dim3(2 * pairs, 1, 1);
  {
    KernelScope scope(kernel_id, st);
    if (cudaLaunchKernelEx(&cfg, kern, ma, mb, mc, sc, ep, status) != cudaSuccess) return SAPO_ERR_CUDA;
  }
  if (sc.sk_tiles > 0) {
    KernelScope scope(SAPO_K_STREAMK_FIXUP, st);
    streamk_fixup_kernel<<<sc.sk_tiles * 32, 256, 0, st>>>(sc, ep, pairs);
  }
  return check_launch();
}

// The two contractions over a filled panel (dz, or the exponentials of the single-pass call):
//   dhidden[0:tc] = row_scale . (panel . W)       (M = tokens, N = H, K = vocabulary)
//   dW_head   (+)= panel^T . X                    (M = vocabulary, N = H, K = tokens)
// X is hidden (or its row-scaled copy), [tc, ldx].  Wide tiles when H allows.
static int launch_grad_gemms(const __nv_bfloat16* panel, int64_t panel_rows, int32_t nvt,
                             const __nv_bfloat16* W, int64_t ldw, const __nv_bfloat16* X, int64_t ldx,
                             int64_t tc, int32_t H, int32_t V, int64_t Vp, float* dhidden,
                             const float* row_scale, float* dW_head, int accumulate, float* partials,
                             const uint32_t* active_mask, int32_t* status, cudaStream_t st) {
  StoreEpi::Params ep_h{dhidden, H, tc, H, 0, partials, nullptr, row_scale};
  StoreEpi::Params ep_w{dW_head, H, V, H, accumulate, partials, nullptr, nullptr};
  if (use_wide_tiles(H)) {
    CUtensorMap map_p_tile, map_p_half, map_w64, map_x64;
    if (!make_map(&map_p_tile, panel, 64, panel_rows, 64, BM) || !make_map(&map_p_half, panel, 64, panel_rows, 64, 64) ||
        !make_map(&map_w64, W, H, V, ldw, 64) || !make_map(&map_x64, X, H, tc, ldx, 64))
      return SAPO_ERR_CUDA;
    // blocks of tokens without any gradient (zero-advantage groups, runs of clipped tokens) are
    // left out of both contractions when the caller knows them
    const int32_t mask_words = (int32_t)ceil_div<int64_t>(ceil_div<int64_t>(tc, BM), 32);
    const bool masked = active_mask != nullptr && mask_words <= MASK_WORDS_MAX;
    Sched sh = make_sched_wide(tc, H, Vp);
    sh.panel_nvt = nvt;
    if (masked) { sh.active_mask = active_mask; sh.mask_words = mask_words; sh.mask_dim = 1; }
    int rc = launch_gemm_wide<2>(map_p_tile, map_w64, sh, ep_h, status, st, SAPO_K_BWD_DH);
    if (rc != SAPO_OK) return rc;
    Sched sw = make_sched_wide(V, H, tc);
    sw.panel_nvt = nvt;
    if (masked) { sw.active_mask = active_mask; sw.mask_words = mask_words; sw.mask_dim = 2; }
    return launch_gemm_wide<3>(map_p_half, map_x64, sw, ep_w, status, st, SAPO_K_BWD_DW);
  }
  CUtensorMap map_p_two, map_p_tile, map_w_mn, map_x_mn;
  if (!make_map(&map_p_two, panel, 64, panel_rows, 64, 256) || !make_map(&map_p_tile, panel, 64, panel_rows, 64, BM) ||
      !make_map(&map_w_mn, W, H, V, ldw, 128) || !make_map(&map_x_mn, X, H, tc, ldx, 128))
    return SAPO_ERR_CUDA;
  Sched sh = make_sched(tc, H, Vp, 0, /*m_fastest=*/false);
  sh.panel_nvt = nvt;
  int rc = launch_gemm<2, true, StoreEpi>(map_p_two, map_w_mn, map_p_two, sh, ep_h, status, st, SAPO_K_BWD_DH);
  if (rc != SAPO_OK) return rc;
  Sched sw = make_sched(V, H, tc, 0, /*m_fastest=*/false);
  sw.panel_nvt = nvt;
  return launch_gemm<3, true, StoreEpi>(map_p_tile, map_x_mn, map_p_tile, sw, ep_w, status, st, SAPO_K_BWD_DW);
}

static int launch_split(const float* X, int64_t ld, int64_t R, int32_t H, __nv_bfloat16* out, int mode,
                        cudaStream_t st) {
  const int64_t n = R * (int64_t)H;
  int64_t blocks = ceil_div<int64_t>(n, 256);
  const int64_t cap = (int64_t)sm_count() * 16;
  if (blocks > cap) blocks = cap;
  if (blocks <= 0) return SAPO_OK;
  KernelScope scope(SAPO_K_SPLIT_BF16, st);
  split_bf16_kernel<<<(int)blocks, 256, 0, st>>>(X, ld, R, H, out, mode);
  return check_launch();
}

static bool shapes_ok(int64_t T, int32_t H, int32_t V) {
  return T >= 1 && T <= 0x7fffff00LL && H >= 8 && (H % 8) == 0 && H <= 65536 && V >= 1 && V <= 0x7fffff00;
}
static int64_t padded_vocab(int32_t V) { return round_up<int64_t>(V, 128); }

struct FwdLayout { size_t partials, a_split, b_split, total; int n_splits; };
static FwdLayout fwd_layout(int64_t T, int32_t H, int32_t V, int32_t dtype, int sms) {
  FwdLayout L{};
  L.n_splits = fwd_splits(T, V, dtype == SAPO_DTYPE_F32 ? 3 * (int64_t)H : (int64_t)H, sms);
  size_t off = 0;
  L.partials = off; off += round_up<size_t>((size_t)3 * 2 * L.n_splits * T * sizeof(float), 256);
  if (dtype == SAPO_DTYPE_F32) {
    L.a_split = off; off += round_up<size_t>((size_t)T * 3 * H * 2, 256);
    L.b_split = off; off += round_up<size_t>((size_t)V * 3 * H * 2, 256);
  }
  L.total = off;
  return L;
}

struct BwdLayout { size_t a_hi, b_hi, partials, panel, fixed; size_t bytes_per_row; };
static BwdLayout bwd_layout(int64_t T, int32_t H, int32_t V, int32_t dtype) {
  BwdLayout L{};
  size_t off = 0;
  if (dtype == SAPO_DTYPE_F32) {
    L.a_hi = off; off += round_up<size_t>((size_t)T * H * 2, 256);
    L.b_hi = off; off += round_up<size_t>((size_t)V * H * 2, 256);
  }
  L.partials = off; off += KSPLIT_SCRATCH_BYTES;
  L.panel = off; L.fixed = off;
  L.bytes_per_row = (size_t)padded_vocab(V) * 2;
  return L;
}
constexpr int64_t PANEL_ROWS_PREFERRED = 32768;

// Scratch of the fused call: per-token vectors for all T tokens, then what one token chunk
// needs (row scales, partial sums, the scaled copy of hidden), the K-split scratch, the
// per-sequence sums when the caller does not want them, and the panel of exponentials.
constexpr int FUSED_MAX_SPLITS = 160;
struct FusedLayout { size_t zy, c2, obj, seq, mask, partials, fixed; size_t bytes_per_row; };
static FusedLayout fused_layout(int64_t T, int32_t H, int32_t V, int32_t S) {
  FusedLayout L{};
  size_t off = 0;
  auto take = [&](size_t bytes) { const size_t at = off; off += round_up<size_t>(bytes, 256); return at; };
  L.zy = take((size_t)T * 4);
  L.c2 = take((size_t)T * 4);
  L.obj = take((size_t)T * 4);
  L.seq = take((size_t)(S > 0 ? S : 1) * 4);
  L.mask = take((size_t)MASK_WORDS_MAX * 4);
  L.partials = take(KSPLIT_SCRATCH_BYTES);
  L.fixed = off;
  // per chunk row: panel row, scaled hidden row, row scale, partial sums
  L.bytes_per_row = (size_t)padded_vocab(V) * 2 + (size_t)H * 2 + 4 + (size_t)2 * FUSED_MAX_SPLITS * 4;
  return L;
}
// where the per-chunk arrays sit for a chunk capacity of `rows` (a multiple of 128)
struct FusedChunk { size_t row_scale, ps, hs, panel; };
static FusedChunk fused_chunk(const FusedLayout& L, int64_t rows, int32_t H) {
  FusedChunk C{};
  size_t off = L.fixed;
  auto take = [&](size_t bytes) { const size_t at = off; off += round_up<size_t>(bytes, 256); return at; };
  C.row_scale = take((size_t)rows * 4);
  C.ps = take((size_t)rows * 2 * FUSED_MAX_SPLITS * 4);
  C.hs = take((size_t)rows * H * 2);
  C.panel = take(0);
  return C;
}
constexpr size_t FUSED_CHUNK_SLACK = 4 * 256;   // alignment padding between the per-chunk arrays

// Scratch of the compacting backward in front of the regular backward's: scan counters, the
// active-token list, compacted per-token vectors and hidden rows.
struct ActiveLayout { size_t counts, n_active, chunk_counts, act_idx, ids, lse, g, hidden, total; };
constexpr int MAX_ACTIVE_CHUNKS = 4096;
static ActiveLayout active_layout(int64_t T, int32_t H) {
  ActiveLayout L{};
  size_t off = 0;
  const size_t n_blocks = (size_t)ceil_div<int64_t>(T, COMPACT_BLOCK);
  auto take = [&](size_t bytes) { const size_t at = off; off += round_up<size_t>(bytes, 256); return at; };
  L.counts = take(n_blocks * 4);
  L.n_active = take(4);
  L.chunk_counts = take((size_t)MAX_ACTIVE_CHUNKS * 4);
  L.act_idx = take((size_t)T * 4);
  L.ids = take((size_t)T * 4);
  L.lse = take((size_t)T * 4);
  L.g = take((size_t)T * 4);
  L.hidden = take((size_t)round_up<int64_t>(T, 128) * H * 2);
  L.total = off;
  return L;
}

// chunk_counts[c] = active tokens that fall into chunk c of `chunk_rows` compacted rows
__global__ void chunk_counts_kernel(const int32_t* n_active, int64_t chunk_rows, int32_t n_chunks,
                                    int32_t* chunk_counts) {
  for (int c = threadIdx.x; c < n_chunks; c += blockDim.x) {
    const int64_t left = (int64_t)*n_active - (int64_t)c * chunk_rows;
    chunk_counts[c] = (int32_t)(left <= 0 ? 0 : (left < chunk_rows ? left : chunk_rows));
  }
}

}  // namespace sapo

// =============================================================================== C ABI
extern "C" size_t sapo_workspace_bytes(int32_t which, int64_t T, int32_t H, int32_t V, int32_t dtype) {
  using namespace sapo;
  if (!shapes_ok(T, H, V) || (dtype != SAPO_DTYPE_BF16 && dtype != SAPO_DTYPE_F32)) return 0;
  if (which == SAPO_WS_FWD) {
    int sms = sm_count();
    if (sms <= 0) sms = 148;
    return fwd_layout(T, H, V, dtype, sms).total;
  }
  if (which == SAPO_WS_FUSED) {
    if (dtype != SAPO_DTYPE_BF16) return 0;
    const FusedLayout L = fused_layout(T, H, V, /*S=*/(int32_t)(T < 0x7fffffff ? T : 0x7fffffff));
    const int64_t rows = T < PANEL_ROWS_PREFERRED ? T : PANEL_ROWS_PREFERRED;
    return L.fixed + FUSED_CHUNK_SLACK + (size_t)round_up<int64_t>(rows, BM) * L.bytes_per_row;
  }
  if (which == SAPO_WS_BWD || which == SAPO_WS_BWD_ACTIVE) {
    const BwdLayout L = bwd_layout(T, H, V, dtype);
    const int64_t rows = T < PANEL_ROWS_PREFERRED ? T : PANEL_ROWS_PREFERRED;
    const size_t extra = which == SAPO_WS_BWD_ACTIVE ? active_layout(T, H).total : 0;
    return extra + L.fixed + (size_t)round_up<int64_t>(rows, BM) * L.bytes_per_row;
  }
  return 0;
}

extern "C" size_t sapo_workspace_bytes_min(int32_t which, int64_t T, int32_t H, int32_t V, int32_t dtype) {
  using namespace sapo;
  if (which != SAPO_WS_BWD && which != SAPO_WS_FUSED) return sapo_workspace_bytes(which, T, H, V, dtype);
  if (!shapes_ok(T, H, V) || (dtype != SAPO_DTYPE_BF16 && dtype != SAPO_DTYPE_F32)) return 0;
  if (which == SAPO_WS_FUSED) {
    if (dtype != SAPO_DTYPE_BF16) return 0;
    const FusedLayout L = fused_layout(T, H, V, (int32_t)(T < 0x7fffffff ? T : 0x7fffffff));
    return L.fixed + FUSED_CHUNK_SLACK + (size_t)BM * L.bytes_per_row;
  }
  const BwdLayout L = bwd_layout(T, H, V, dtype);
  return L.fixed + (size_t)BM * L.bytes_per_row;
}

extern "C" int sapo_policy_loss_fwd(const void* hidden, const void* W_head, int32_t dtype,
                                    int64_t T, int32_t H, int32_t V, int64_t ld_hidden, int64_t ld_W,
                                    const int32_t* ids, const float* old_logp, const float* adv,
                                    const int32_t* cu_seqlens, int32_t S, const sapo_loss_cfg* h_cfg,
                                    float* logp, float* lse, float* ratio, float* surr, float* gscale,
                                    float* seq_surr, float* loss,
                                    void* workspace, size_t workspace_bytes,
                                    int32_t* status, void* stream) {
  using namespace sapo;
  if (!hidden || !W_head || !ids || !old_logp || !adv || !cu_seqlens || !h_cfg || !logp || !lse ||
      !ratio || !surr || !gscale || !loss || !workspace || !status || S < 1)
    return SAPO_ERR_INVALID_ARG;
  if (dtype != SAPO_DTYPE_BF16 && dtype != SAPO_DTYPE_F32) return SAPO_ERR_INVALID_ARG;
  if (T < 1 || H < 1 || V < 1 || ld_hidden < H || ld_W < H) return SAPO_ERR_INVALID_ARG;
  if (!shapes_ok(T, H, V)) return SAPO_ERR_UNSUPPORTED_SHAPE;
  const int esz = dtype == SAPO_DTYPE_BF16 ? 2 : 4;
  if (!aligned16(hidden) || !aligned16(W_head) || !aligned16(workspace) || (ld_hidden * esz) % 16 ||
      (ld_W * esz) % 16)
    return SAPO_ERR_INVALID_ARG;
  if (!(h_cfg->eps_low >= 0.f) || !(h_cfg->eps_high >= 0.f)) return SAPO_ERR_INVALID_ARG;
  if ((h_cfg->loss_agg != 0 && h_cfg->loss_agg != 1) || (h_cfg->kl_beta != 0.f && !h_cfg->ref_logp))
    return SAPO_ERR_INVALID_ARG;
  const int sms = sm_count();
  if (sms <= 0) return SAPO_ERR_CUDA;
  const FwdLayout L = fwd_layout(T, H, V, dtype, sms);
  // seq_surr scratch lives behind the layout when the caller does not want it
  const size_t need = L.total + (seq_surr ? 0 : round_up<size_t>((size_t)S * sizeof(float), 256));
  if (workspace_bytes < need) return SAPO_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  float* pm = reinterpret_cast<float*>(ws + L.partials);
  float* ps = pm + (size_t)2 * L.n_splits * T;
  float* pz = ps + (size_t)2 * L.n_splits * T;
  float* seq_out = seq_surr ? seq_surr : reinterpret_cast<float*>(ws + L.total);

  const void* A = hidden; const void* B = W_head;
  int64_t K = H, lda = ld_hidden, ldb = ld_W;
  if (dtype == SAPO_DTYPE_F32) {
    __nv_bfloat16* a3 = reinterpret_cast<__nv_bfloat16*>(ws + L.a_split);
    __nv_bfloat16* b3 = reinterpret_cast<__nv_bfloat16*>(ws + L.b_split);
    int rc = launch_split(static_cast<const float*>(hidden), ld_hidden, T, H, a3, 0, st);
    if (rc != SAPO_OK) return rc;
    rc = launch_split(static_cast<const float*>(W_head), ld_W, V, H, b3, 1, st);
    if (rc != SAPO_OK) return rc;
    A = a3; B = b3; K = 3 * (int64_t)H; lda = K; ldb = K;
  }
  CUtensorMap map_a, map_b;
  if (!make_map(&map_a, A, K, T, lda, BM) || !make_map(&map_b, B, K, V, ldb, 128)) return SAPO_ERR_CUDA;
  const Sched sched = make_sched(T, V, K, L.n_splits, /*m_fastest=*/true);
  FwdEpi::Params ep{ids, pm, ps, pz, T, V};
  int rc = launch_gemm<0, false, FwdEpi>(map_a, map_b, map_a, sched, ep, status, st, SAPO_K_FWD_GEMM);
  if (rc != SAPO_OK) return rc;

  TailArgs ta{};
  ta.pm = pm; ta.ps = ps; ta.pz = pz; ta.T = T;
  ta.n_splits = 2 * sched.units_per_m;   // one partial per vocab split and column half
  ta.ids = ids; ta.V = V; ta.old_logp = old_logp; ta.adv = adv; ta.cu = cu_seqlens; ta.S = S;
  ta.lo_edge = 1.f - h_cfg->eps_low; ta.hi_edge = 1.f + h_cfg->eps_high; ta.grad_scale = h_cfg->grad_scale;
  ta.loss_agg = h_cfg->loss_agg; ta.kl_beta = h_cfg->kl_beta; ta.ref_logp = h_cfg->ref_logp;
  ta.logp = logp; ta.lse = lse; ta.ratio = ratio; ta.surr = surr; ta.gscale = gscale; ta.seq_surr = seq_out;
  ta.status = status;
  const int tail_blocks = S < sms * 8 ? S : sms * 8;
  { KernelScope scope(SAPO_K_LOSS_TAIL, st); loss_tail_kernel<<<tail_blocks, 256, 0, st>>>(ta); }
  { KernelScope scope(SAPO_K_LOSS_FINAL, st); loss_final_kernel<<<1, 256, 0, st>>>(seq_out, cu_seqlens, S, T, h_cfg->loss_agg, loss); }
  return check_launch();
}

// ------------------------------------------------------------------------------------------
// Forward pass for callers that cannot obtain device memory of their own.
//
// Some hosts of this library may not allocate: a plugin inside a serving process whose
// memory pool is fixed at start-up, code that runs after the process has handed all of its
// device memory to another allocator, or a latency-critical loop in which cudaMalloc (which
// synchronises the device) is forbidden.  For them the forward scratch lives in this array,
// which belongs to the library image: every GPU that loads the library holds these
// SAPO_STATIC_SCRATCH_BYTES until the process exits, whether or not the entry point is used.
static __device__ __align__(256) unsigned char g_static_fwd_scratch[SAPO_STATIC_SCRATCH_BYTES];

namespace sapo {
constexpr int MAX_DEVICES = 64;
// Device address of the array on each GPU.  In host code the symbol's name is only a handle;
// the address a kernel can use has to be asked for, once per device, with that device current.
static void* g_static_scratch_ptr[MAX_DEVICES] = {nullptr};

static int static_scratch(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return SAPO_ERR_CUDA;
  if (g_static_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_fwd_scratch) != cudaSuccess || p == nullptr) return SAPO_ERR_CUDA;
    g_static_scratch_ptr[dev] = p;
  }
  *out = g_static_scratch_ptr[dev];
  return SAPO_OK;
}
}  // namespace sapo

extern "C" int sapo_policy_loss_fwd_static(const void* hidden, const void* W_head, int32_t dtype,
                                           int64_t T, int32_t H, int32_t V, int64_t ld_hidden,
                                           int64_t ld_W, const int32_t* ids, const float* old_logp,
                                           const float* adv, const int32_t* cu_seqlens, int32_t S,
                                           const sapo_loss_cfg* h_cfg, float* logp, float* lse,
                                           float* ratio, float* surr, float* gscale, float* seq_surr,
                                           float* loss, int32_t* status, void* stream) {
  using namespace sapo;
  // fp32 operands would need bf16 copies of hidden and W_head in the scratch: far beyond it
  if (dtype != SAPO_DTYPE_BF16) return SAPO_ERR_UNSUPPORTED_SHAPE;
  if (T < 1 || S < 1 || !shapes_ok(T, H, V)) return SAPO_ERR_INVALID_ARG;
  int sms = sm_count();
  if (sms <= 0) return SAPO_ERR_CUDA;
  const size_t need = fwd_layout(T, H, V, dtype, sms).total +
                      (seq_surr ? 0 : round_up<size_t>((size_t)S * sizeof(float), 256));
  if (need > (size_t)SAPO_STATIC_SCRATCH_BYTES) return SAPO_ERR_STATIC_SCRATCH_EXCEEDED;
  void* scratch = nullptr;
  const int rc = static_scratch(&scratch);
  if (rc != SAPO_OK) return rc;
  // Nothing in the scratch has to start at zero: the vocab-split partials and the per-sequence
  // sums are written for every token / sequence of this call before anything reads them.
  return sapo_policy_loss_fwd(hidden, W_head, dtype, T, H, V, ld_hidden, ld_W, ids, old_logp, adv,
                              cu_seqlens, S, h_cfg, logp, lse, ratio, surr, gscale, seq_surr, loss,
                              scratch, (size_t)SAPO_STATIC_SCRATCH_BYTES, status, stream);
}

extern "C" int sapo_policy_loss_bwd(const void* hidden, const void* W_head, int32_t dtype,
                                    int64_t T, int32_t H, int32_t V, int64_t ld_hidden, int64_t ld_W,
                                    const int32_t* ids, const float* lse, const float* gscale,
                                    float* dhidden, float* dW_head, int32_t accumulate_dW,
                                    void* workspace, size_t workspace_bytes,
                                    int32_t* status, void* stream) {
  using namespace sapo;
  if (!hidden || !W_head || !ids || !lse || !gscale || !dhidden || !dW_head || !workspace || !status)
    return SAPO_ERR_INVALID_ARG;
  if (dtype != SAPO_DTYPE_BF16 && dtype != SAPO_DTYPE_F32) return SAPO_ERR_INVALID_ARG;
  if (T < 1 || H < 1 || V < 1 || ld_hidden < H || ld_W < H) return SAPO_ERR_INVALID_ARG;
  if (!shapes_ok(T, H, V)) return SAPO_ERR_UNSUPPORTED_SHAPE;
  const int esz = dtype == SAPO_DTYPE_BF16 ? 2 : 4;
  if (!aligned16(hidden) || !aligned16(W_head) || !aligned16(workspace) || !aligned16(dhidden) ||
      !aligned16(dW_head) || (ld_hidden * esz) % 16 || (ld_W * esz) % 16)
    return SAPO_ERR_INVALID_ARG;
  const BwdLayout L = bwd_layout(T, H, V, dtype);
  if (workspace_bytes < L.fixed + (size_t)BM * L.bytes_per_row) return SAPO_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);

  const __nv_bfloat16* A = static_cast<const __nv_bfloat16*>(hidden);
  const __nv_bfloat16* B = static_cast<const __nv_bfloat16*>(W_head);
  int64_t lda = ld_hidden, ldb = ld_W;
  if (dtype == SAPO_DTYPE_F32) {
    __nv_bfloat16* a1 = reinterpret_cast<__nv_bfloat16*>(ws + L.a_hi);
    __nv_bfloat16* b1 = reinterpret_cast<__nv_bfloat16*>(ws + L.b_hi);
    int rc = launch_split(static_cast<const float*>(hidden), ld_hidden, T, H, a1, 2, st);
    if (rc != SAPO_OK) return rc;
    rc = launch_split(static_cast<const float*>(W_head), ld_W, V, H, b1, 2, st);
    if (rc != SAPO_OK) return rc;
    A = a1; B = b1; lda = H; ldb = H;
  }
  const int64_t Vp = padded_vocab(V);
  const int32_t nvt = (int32_t)(Vp / 64);
  __nv_bfloat16* panel = reinterpret_cast<__nv_bfloat16*>(ws + L.panel);
  float* partials = reinterpret_cast<float*>(ws + L.partials);
  // whole 128-token blocks of the panel that fit; a chunk never ends inside a block it cannot hold
  const int64_t rows_fit = ((int64_t)((workspace_bytes - L.fixed) / L.bytes_per_row) / BM) * BM;
  const int64_t chunk_rows = rows_fit >= T ? T : rows_fit;
  if (chunk_rows <= 0) return SAPO_ERR_WORKSPACE_TOO_SMALL;

  // W as the K-major B operand of the logit recompute
  CUtensorMap map_w_kmajor;
  if (!make_map(&map_w_kmajor, B, H, V, ldb, 128)) return SAPO_ERR_CUDA;

  for (int64_t t0 = 0; t0 < T; t0 += chunk_rows) {
    const int64_t tc = (T - t0) < chunk_rows ? (T - t0) : chunk_rows;
    const __nv_bfloat16* A0 = A + t0 * lda;
    const int64_t panel_rows = ceil_div<int64_t>(tc, BM) * nvt * BM;   // 128-byte rows of the tiled panel
    CUtensorMap map_h_kmajor, map_p_tile;
    if (!make_map(&map_h_kmajor, A0, H, tc, lda, BM) || !make_map(&map_p_tile, panel, 64, panel_rows, 64, BM))
      return SAPO_ERR_CUDA;
    // dz panel: recompute logits tile by tile
    {
      Sched sched = make_sched(tc, V, H, 0, /*m_fastest=*/true, /*tile_align=*/64);
      sched.n_cover = (int32_t)Vp;
      DzEpi::Params ep{ids + t0, lse + t0, gscale + t0, tc, V, nvt};
      int rc = launch_gemm<0, false, DzEpi>(map_h_kmajor, map_w_kmajor, map_p_tile, sched, ep, status, st, SAPO_K_BWD_DZ);
      if (rc != SAPO_OK) return rc;
    }
    // dhidden[t0:t0+tc] = dz . W         (M = tokens, N = H, K = V)
    // dW (+)= dz^T . hidden               (M = V, N = H, K = tokens)
    const int rc = launch_grad_gemms(panel, panel_rows, nvt, B, ldb, A0, lda, tc, H, V, Vp,
                                     dhidden + t0 * (int64_t)H, nullptr, dW_head,
                                     (t0 > 0 || accumulate_dW) ? 1 : 0, partials, nullptr, status, st);
    if (rc != SAPO_OK) return rc;
  }
  return SAPO_OK;
}

// ------------------------------------------------------------------------------------------
// Backward over the active tokens only (g_t != 0): same results as sapo_policy_loss_bwd, less
// tensor work when many tokens are inactive.  The number of active tokens stays on the device:
// the GEMM kernels read it when they start, so the call does not synchronise.
extern "C" int sapo_policy_loss_bwd_active(const void* hidden, const void* W_head, int32_t dtype,
                                           int64_t T, int32_t H, int32_t V, int64_t ld_hidden, int64_t ld_W,
                                           const int32_t* ids, const float* lse, const float* gscale,
                                           float* dhidden, float* dW_head, int32_t accumulate_dW,
                                           int32_t* n_active_out,
                                           void* workspace, size_t workspace_bytes,
                                           int32_t* status, void* stream) {
  using namespace sapo;
  if (!hidden || !W_head || !ids || !lse || !gscale || !dhidden || !dW_head || !workspace || !status)
    return SAPO_ERR_INVALID_ARG;
  if (dtype != SAPO_DTYPE_BF16 && dtype != SAPO_DTYPE_F32) return SAPO_ERR_INVALID_ARG;
  if (T < 1 || H < 1 || V < 1 || ld_hidden < H || ld_W < H) return SAPO_ERR_INVALID_ARG;
  if (!shapes_ok(T, H, V)) return SAPO_ERR_UNSUPPORTED_SHAPE;
  const int esz = dtype == SAPO_DTYPE_BF16 ? 2 : 4;
  if (!aligned16(hidden) || !aligned16(W_head) || !aligned16(workspace) || !aligned16(dhidden) ||
      !aligned16(dW_head) || (ld_hidden * esz) % 16 || (ld_W * esz) % 16)
    return SAPO_ERR_INVALID_ARG;
  const ActiveLayout AL = active_layout(T, H);
  const BwdLayout L = bwd_layout(T, H, V, dtype);
  if (workspace_bytes < AL.total + L.fixed + (size_t)BM * L.bytes_per_row) return SAPO_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* ws0 = static_cast<uint8_t*>(workspace);
  uint8_t* ws = ws0 + AL.total;                                   // the regular backward's layout
  const size_t ws_bytes = workspace_bytes - AL.total;
  int32_t* counts = reinterpret_cast<int32_t*>(ws0 + AL.counts);
  int32_t* n_active = reinterpret_cast<int32_t*>(ws0 + AL.n_active);
  int32_t* chunk_counts = reinterpret_cast<int32_t*>(ws0 + AL.chunk_counts);
  int32_t* act_idx = reinterpret_cast<int32_t*>(ws0 + AL.act_idx);
  int32_t* ids_act = reinterpret_cast<int32_t*>(ws0 + AL.ids);
  float* lse_act = reinterpret_cast<float*>(ws0 + AL.lse);
  float* g_act = reinterpret_cast<float*>(ws0 + AL.g);
  __nv_bfloat16* hidden_act = reinterpret_cast<__nv_bfloat16*>(ws0 + AL.hidden);

  const __nv_bfloat16* A = static_cast<const __nv_bfloat16*>(hidden);
  const __nv_bfloat16* B = static_cast<const __nv_bfloat16*>(W_head);
  int64_t lda = ld_hidden, ldb = ld_W;
  if (dtype == SAPO_DTYPE_F32) {
    __nv_bfloat16* a1 = reinterpret_cast<__nv_bfloat16*>(ws + L.a_hi);
    __nv_bfloat16* b1 = reinterpret_cast<__nv_bfloat16*>(ws + L.b_hi);
    int rc = launch_split(static_cast<const float*>(hidden), ld_hidden, T, H, a1, 2, st);
    if (rc != SAPO_OK) return rc;
    rc = launch_split(static_cast<const float*>(W_head), ld_W, V, H, b1, 2, st);
    if (rc != SAPO_OK) return rc;
    A = a1; B = b1; lda = H; ldb = H;
  }
  const int64_t Vp = padded_vocab(V);
  const int32_t nvt = (int32_t)(Vp / 64);
  __nv_bfloat16* panel = reinterpret_cast<__nv_bfloat16*>(ws + L.panel);
  float* partials = reinterpret_cast<float*>(ws + L.partials);
  const int64_t rows_fit = ((int64_t)((ws_bytes - L.fixed) / L.bytes_per_row) / BM) * BM;
  const int64_t chunk_rows = rows_fit >= T ? round_up<int64_t>(T, BM) : rows_fit;
  if (chunk_rows <= 0) return SAPO_ERR_WORKSPACE_TOO_SMALL;
  const int64_t n_chunks = ceil_div<int64_t>(T, chunk_rows);
  if (n_chunks > MAX_ACTIVE_CHUNKS) return SAPO_ERR_WORKSPACE_TOO_SMALL;

  // 1. which tokens take part, in order; compacted copies of what the GEMMs read per token
  const int sms = sm_count();
  if (sms <= 0) return SAPO_ERR_CUDA;
  const int n_blocks = (int)ceil_div<int64_t>(T, COMPACT_BLOCK);
  {
    KernelScope scope(SAPO_K_COMPACT, st);
    active_count_kernel<<<n_blocks, COMPACT_BLOCK, 0, st>>>(gscale, T, counts);
  }
  { KernelScope scope(SAPO_K_COMPACT, st); active_scan_kernel<<<1, 1024, 0, st>>>(counts, n_blocks, n_active); }
  {
    KernelScope scope(SAPO_K_COMPACT, st);
    active_assign_kernel<<<n_blocks, COMPACT_BLOCK, 0, st>>>(gscale, lse, ids, T, counts, act_idx, ids_act,
                                                             lse_act, g_act, dhidden, H);
  }
  {
    KernelScope scope(SAPO_K_COMPACT, st);
    int64_t blocks = ceil_div<int64_t>(T, 8);
    if (blocks > (int64_t)sms * 8) blocks = (int64_t)sms * 8;
    active_gather_kernel<<<(int)blocks, 256, 0, st>>>(A, lda, H, act_idx, n_active, hidden_act);
  }
  { KernelScope scope(SAPO_K_COMPACT, st); chunk_counts_kernel<<<1, 256, 0, st>>>(n_active, chunk_rows, (int32_t)n_chunks, chunk_counts); }
  if (n_active_out != nullptr &&
      cudaMemcpyAsync(n_active_out, n_active, sizeof(int32_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return SAPO_ERR_CUDA;

  // 2. the three contractions over at most T compacted rows; their true count is read on the device
  CUtensorMap map_w_kmajor, map_w_mn;
  if (!make_map(&map_w_kmajor, B, H, V, ldb, 128) || !make_map(&map_w_mn, B, H, V, ldb, 128))
    return SAPO_ERR_CUDA;
  for (int64_t c = 0; c < n_chunks; ++c) {
    const int64_t t0 = c * chunk_rows;
    const int64_t tc = (T - t0) < chunk_rows ? (T - t0) : chunk_rows;     // upper bound of this chunk
    const int64_t tc_pad = round_up<int64_t>(tc, BM);
    const __nv_bfloat16* A0 = hidden_act + t0 * (int64_t)H;
    const int64_t panel_rows = ceil_div<int64_t>(tc, BM) * nvt * BM;
    CUtensorMap map_h_kmajor, map_h_mn, map_p_two, map_p_tile;
    if (!make_map(&map_h_kmajor, A0, H, tc_pad, H, BM) || !make_map(&map_h_mn, A0, H, tc_pad, H, 128) ||
        !make_map(&map_p_two, panel, 64, panel_rows, 64, 256) ||
        !make_map(&map_p_tile, panel, 64, panel_rows, 64, BM))
      return SAPO_ERR_CUDA;
    const int32_t* count = chunk_counts + c;
    {
      Sched sched = make_sched(tc, V, H, 0, /*m_fastest=*/true, /*tile_align=*/64);
      sched.n_cover = (int32_t)Vp;
      sched.dyn_count = count; sched.dyn_dim = 1;
      DzEpi::Params ep{ids_act + t0, lse_act + t0, g_act + t0, tc, V, nvt};
      int rc = launch_gemm<0, false, DzEpi>(map_h_kmajor, map_w_kmajor, map_p_tile, sched, ep, status, st, SAPO_K_BWD_DZ);
      if (rc != SAPO_OK) return rc;
    }
    {
      Sched sched = make_sched(tc, H, Vp, 0, /*m_fastest=*/false);
      sched.panel_nvt = nvt;
      sched.dyn_count = count; sched.dyn_dim = 1;
      StoreEpi::Params ep{dhidden, H, tc, H, 0, partials, act_idx + t0, nullptr};   // rows go back to their tokens
      int rc = launch_gemm<2, true, StoreEpi>(map_p_two, map_w_mn, map_p_two, sched, ep, status, st, SAPO_K_BWD_DH);
      if (rc != SAPO_OK) return rc;
    }
    {
      const int acc = (c > 0 || accumulate_dW) ? 1 : 0;
      Sched sched = make_sched(V, H, tc, 0, /*m_fastest=*/false);
      sched.panel_nvt = nvt;
      sched.dyn_count = count; sched.dyn_dim = 2; sched.skip_if_empty = acc;
      StoreEpi::Params ep{dW_head, H, V, H, acc, partials, nullptr, nullptr};
      int rc = launch_gemm<3, true, StoreEpi>(map_p_tile, map_h_mn, map_p_tile, sched, ep, status, st, SAPO_K_BWD_DW);
      if (rc != SAPO_OK) return rc;
    }
  }
  return SAPO_OK;
}

// ------------------------------------------------------------------------------------------
// Loss and both gradients in one call, without a second pass over the logits: the forward
// epilogue leaves exp(z - c_t) in the panel, and the two backward contractions read it.
extern "C" int sapo_policy_loss_fwd_bwd(const void* hidden, const void* W_head, int32_t dtype,
                                        int64_t T, int32_t H, int32_t V, int64_t ld_hidden, int64_t ld_W,
                                        const int32_t* ids, const float* old_logp, const float* adv,
                                        const int32_t* cu_seqlens, int32_t S, const sapo_loss_cfg* h_cfg,
                                        float* logp, float* lse, float* ratio, float* surr, float* gscale,
                                        float* seq_surr, float* loss,
                                        float* dhidden, float* dW_head, int32_t accumulate_dW,
                                        void* workspace, size_t workspace_bytes,
                                        int32_t* status, void* stream) {
  using namespace sapo;
  if (!hidden || !W_head || !ids || !old_logp || !adv || !cu_seqlens || !h_cfg || !logp || !lse ||
      !ratio || !surr || !gscale || !loss || !dhidden || !dW_head || !workspace || !status || S < 1)
    return SAPO_ERR_INVALID_ARG;
  if (dtype != SAPO_DTYPE_BF16 && dtype != SAPO_DTYPE_F32) return SAPO_ERR_INVALID_ARG;
  if (T < 1 || H < 1 || V < 1 || ld_hidden < H || ld_W < H) return SAPO_ERR_INVALID_ARG;
  if (!seq_surr && S > T) return SAPO_ERR_INVALID_ARG;   // the built-in per-sequence scratch holds T entries
  if (!shapes_ok(T, H, V)) return SAPO_ERR_UNSUPPORTED_SHAPE;
  if (dtype != SAPO_DTYPE_BF16) return SAPO_ERR_UNSUPPORTED_SHAPE;   // fp32 operands: use the separate calls
  if (!aligned16(hidden) || !aligned16(W_head) || !aligned16(workspace) || !aligned16(dhidden) ||
      !aligned16(dW_head) || (ld_hidden * 2) % 16 || (ld_W * 2) % 16)
    return SAPO_ERR_INVALID_ARG;
  if (!(h_cfg->eps_low >= 0.f) || !(h_cfg->eps_high >= 0.f)) return SAPO_ERR_INVALID_ARG;
  if ((h_cfg->loss_agg != 0 && h_cfg->loss_agg != 1) || (h_cfg->kl_beta != 0.f && !h_cfg->ref_logp))
    return SAPO_ERR_INVALID_ARG;
  const int sms = sm_count();
  if (sms <= 0) return SAPO_ERR_CUDA;
  const FusedLayout L = fused_layout(T, H, V, (int32_t)(T < 0x7fffffff ? T : 0x7fffffff));
  if (workspace_bytes < L.fixed + FUSED_CHUNK_SLACK + (size_t)BM * L.bytes_per_row)
    return SAPO_ERR_WORKSPACE_TOO_SMALL;
  const int64_t rows_fit =
      ((int64_t)((workspace_bytes - L.fixed - FUSED_CHUNK_SLACK) / L.bytes_per_row) / BM) * BM;
  const int64_t chunk_rows = rows_fit >= T ? round_up<int64_t>(T, BM) : rows_fit;   // capacity, a multiple of 128
  const FusedChunk CL = fused_chunk(L, chunk_rows, H);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  float* zy = reinterpret_cast<float*>(ws + L.zy);
  float* c2 = reinterpret_cast<float*>(ws + L.c2);
  float* obj = reinterpret_cast<float*>(ws + L.obj);
  float* seq_out = seq_surr ? seq_surr : reinterpret_cast<float*>(ws + L.seq);
  float* partials = reinterpret_cast<float*>(ws + L.partials);
  uint32_t* active_mask = reinterpret_cast<uint32_t*>(ws + L.mask);
  float* row_scale = reinterpret_cast<float*>(ws + CL.row_scale);
  float* ps = reinterpret_cast<float*>(ws + CL.ps);
  __nv_bfloat16* hs = reinterpret_cast<__nv_bfloat16*>(ws + CL.hs);
  __nv_bfloat16* panel = reinterpret_cast<__nv_bfloat16*>(ws + CL.panel);
  const __nv_bfloat16* A = static_cast<const __nv_bfloat16*>(hidden);
  const __nv_bfloat16* B = static_cast<const __nv_bfloat16*>(W_head);
  const int64_t Vp = padded_vocab(V);
  const int32_t nvt = (int32_t)(Vp / 64);

  // 1. chosen-token logits and the reference of the exponentials, all tokens
  {
    int64_t blocks = ceil_div<int64_t>(T, 8);
    if (blocks > (int64_t)sms * 8) blocks = (int64_t)sms * 8;
    KernelScope scope(SAPO_K_TARGET_LOGIT, st);
    target_logit_kernel<<<(int)blocks, 256, 0, st>>>(A, ld_hidden, B, ld_W, ids, old_logp, T, H, V, zy, c2);
  }
  CUtensorMap map_w_kmajor;
  if (!make_map(&map_w_kmajor, B, H, V, ld_W, 128)) return SAPO_ERR_CUDA;

  for (int64_t t0 = 0; t0 < T; t0 += chunk_rows) {
    const int64_t tc = (T - t0) < chunk_rows ? (T - t0) : chunk_rows;
    const __nv_bfloat16* A0 = A + t0 * ld_hidden;
    const int64_t panel_rows = ceil_div<int64_t>(tc, BM) * nvt * BM;
    CUtensorMap map_h_kmajor, map_p_tile;
    if (!make_map(&map_h_kmajor, A0, H, tc, ld_hidden, BM) || !make_map(&map_p_tile, panel, 64, panel_rows, 64, BM))
      return SAPO_ERR_CUDA;
    // 2. exponentials of the chunk -> panel, their sums per token and vocab split
    int n_splits = fwd_splits(tc, V, H, sms);
    if (n_splits > FUSED_MAX_SPLITS) n_splits = FUSED_MAX_SPLITS;
    Sched fs = make_sched(tc, V, H, n_splits, /*m_fastest=*/true, /*tile_align=*/64);
    fs.n_cover = (int32_t)Vp;
    {
      ExpEpi::Params ep{c2 + t0, ps, tc, V, nvt};
      int rc = launch_gemm<0, false, ExpEpi>(map_h_kmajor, map_w_kmajor, map_p_tile, fs, ep, status, st, SAPO_K_FWD_EXP);
      if (rc != SAPO_OK) return rc;
    }
    // 3. per-token loss terms, row scales, the chosen-token entries of the panel, scaled hidden rows
    {
      FusedTailArgs ta{};
      ta.ps = ps; ta.n_parts = 2 * fs.units_per_m; ta.t0 = t0; ta.tc = tc;
      ta.zy = zy; ta.c2 = c2; ta.ids = ids; ta.V = V; ta.old_logp = old_logp; ta.adv = adv;
      ta.cu = cu_seqlens; ta.S = S; ta.T = T;
      ta.lo_edge = 1.f - h_cfg->eps_low; ta.hi_edge = 1.f + h_cfg->eps_high; ta.grad_scale = h_cfg->grad_scale;
      ta.loss_agg = h_cfg->loss_agg; ta.kl_beta = h_cfg->kl_beta; ta.ref_logp = h_cfg->ref_logp;
      ta.logp = logp; ta.lse = lse; ta.ratio = ratio; ta.surr = surr; ta.gscale = gscale; ta.obj = obj;
      ta.row_scale = row_scale; ta.panel = panel; ta.nvt = nvt;
      ta.hidden = A; ta.ldh = ld_hidden; ta.H = H; ta.hs = hs; ta.status = status;
      // one bit per 128-token block of the chunk that has a token with a gradient
      const bool masked = ceil_div<int64_t>(ceil_div<int64_t>(tc, BM), 32) <= MASK_WORDS_MAX;
      ta.active_mask = masked ? active_mask : nullptr;
      if (masked && cudaMemsetAsync(active_mask, 0, (size_t)MASK_WORDS_MAX * 4, st) != cudaSuccess) return SAPO_ERR_CUDA;
      int64_t blocks = ceil_div<int64_t>(tc, 8);
      if (blocks > (int64_t)sms * 8) blocks = (int64_t)sms * 8;
      KernelScope scope(SAPO_K_FUSED_TAIL, st);
      fused_tail_kernel<<<(int)blocks, 256, 0, st>>>(ta);
    }
    // 4. dhidden[t0:t0+tc] = a_t (e' . W)     (M = tokens, N = H, K = V)
    // 5. dW (+)= e'^T . (a_t h_t)            (M = V, N = H, K = tokens)
    const int rc = launch_grad_gemms(panel, panel_rows, nvt, B, ld_W, hs, H, tc, H, V, Vp,
                                     dhidden + t0 * (int64_t)H, row_scale, dW_head,
                                     (t0 > 0 || accumulate_dW) ? 1 : 0, partials, active_mask, status, st);
    if (rc != SAPO_OK) return rc;
  }
  // 6. per-sequence means and the loss
  const int seq_blocks = S < sms * 8 ? S : sms * 8;
  { KernelScope scope(SAPO_K_LOSS_TAIL, st); seq_mean_kernel<<<seq_blocks, 256, 0, st>>>(obj, cu_seqlens, S, seq_out); }
  { KernelScope scope(SAPO_K_LOSS_FINAL, st); loss_final_kernel<<<1, 256, 0, st>>>(seq_out, cu_seqlens, S, T, h_cfg->loss_agg, loss); }
  return check_launch();
}

#ifdef SAPO_WAIT_STATS
// Rows: forward, dz, dH, dW.  Columns: [0] TMA waits on free stages, [1] MMA waits on filled
// stages, [2] MMA waits on a free accumulator, [3] one epilogue thread's waits on a full
// accumulator, [4..6] total cycles of the TMA / MMA / that epilogue thread, summed over CTAs
// and launches since the last reset; [7] the longest MMA-thread time of any CTA.
extern "C" int sapo_debug_wait_stats(unsigned long long* h_out, int32_t reset) {
  if (h_out && cudaMemcpyFromSymbol(h_out, sapo::g_wait_stats, sizeof(unsigned long long) * 32) != cudaSuccess)
    return SAPO_ERR_CUDA;
  if (reset) {
    unsigned long long z[32] = {0};
    if (cudaMemcpyToSymbol(sapo::g_wait_stats, z, sizeof(z)) != cudaSuccess) return SAPO_ERR_CUDA;
  }
  return SAPO_OK;
}
#endif
