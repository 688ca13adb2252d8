// What happens to an accumulator tile once the tensor cores have finished it: the four epilogues
// of the GEMM kernels (online log-sum-exp of the forward, dz of the separate backward, the
// exponential panel of the single-pass call, plain fp32 stores) and the fix-up of K-split tiles.
#pragma once

#include "gemm_sched.cuh"

namespace sapo {
using namespace umma;

// ---------------------------------------------------------------------------- epilogues
// Each epilogue thread owns one accumulator row (TMEM lane) of the tile.

// Panel rows go straight from the epilogue threads' registers to global memory.  A tile row is
// 128 contiguous bytes (64 bf16); a thread writes it as 32-byte stores, each a whole sector.
// (Staging the tile in shared memory for one TMA store per tile was measured slower: the kernel's
// operand traffic already fills the shared-memory bandwidth, and the staged copy cost the MMA
// issuer 4-5 % more cycles per launch.)
// 16 finished bf16 entries (32 bytes, one sector) of a panel row: columns [col0, col0 + 16) of the
// tile row `r` of token block `tile_row0`.
__device__ __forceinline__ void store_panel_16(__nv_bfloat16* panel, int64_t panel_rows, int r, int tile_row0,
                                               int col0, const uint32_t (&w)[8]) {
  const int64_t prow = (int64_t)tile_row0 + (int64_t)(col0 >> 6) * BM + r;
  if (!SAPO_IN_BOUNDS(prow >= 0 && prow < panel_rows && r < BM)) return;
  uint8_t* dst = reinterpret_cast<uint8_t*>(panel) +
                 ((size_t)tile_row0 + (size_t)(col0 >> 6) * BM + (size_t)r) * 128 + (size_t)(col0 & 63) * 2;
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"l"(dst), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
               : "memory");
}

// Forward: online log-sum-exp in the base-2 domain plus the logit of the chosen token.
// ENT: also the running sum of 2^(x - m) z, from which the tail forms the entropy of the row's
// distribution, H = lse - sum_v p_v z_v (one more multiply-add per logit, so it is a variant).
template <bool ENT>
struct FwdEpiT {
  static constexpr bool PANEL = false;
  static constexpr bool STREAMK = false;
  template <class P> __device__ static void set_dynamic(P&, const Sched&) {}

  struct Params {
    const int32_t* ids; float* pm; float* ps; float* pz;  // partials [n_splits][T]
    float* pe;                                             // ENT: partial sums of 2^(x - m) z
    int64_t T; int32_t V;
    int32_t id_offset;                                     // first vocabulary entry of W (a vocab shard), else 0
    int32_t parts_cap;                                     // partials per token the arrays hold (checked builds)
  };
  float m, s, zy, sz; int32_t y; int64_t row;
  __device__ __forceinline__ void begin_unit(const Params& p, int mb, int r) {
    row = (int64_t)mb * BM + r;
    m = -INFINITY; s = 0.f; zy = 0.f; sz = 0.f;
    y = row < p.T ? p.ids[row] - p.id_offset : -1;          // outside [0, V): the chosen token is not in these columns
  }
  template <int HALF>
  __device__ __forceinline__ void chunk(const Params& p, float (&v)[32], int col0) {
    if (col0 >= p.V) return;
    if (col0 + 32 > p.V) {
      // columns past the vocabulary: far below any logit, but finite so that 0 * z stays 0
      #pragma unroll
      for (int j = 0; j < 32; ++j) if (col0 + j >= p.V) v[j] = -1e30f;
    }
    const int yr = y - col0;
    if (yr >= 0 && yr < 32 && y < p.V) {
      #pragma unroll
      for (int j = 0; j < 32; ++j) if (j == yr) zy = v[j];
    }
    float cmax = v[0];
    #pragma unroll
    for (int j = 1; j < 32; ++j) cmax = fmaxf(cmax, v[j]);
    const float m_new = fmaxf(m, cmax * LOG2E);
    const float rescale = ex2(m - m_new);    // first chunk: ex2(-inf) = 0
    float acc = s * rescale;
    float acc_z = sz * rescale;
    #pragma unroll
    for (int j = 0; j < 32; ++j) {
      const float e = ex2(fmaf(v[j], LOG2E, -m_new));
      acc += e;
      if constexpr (ENT) acc_z = fmaf(e, v[j], acc_z);
    }
    s = acc; m = m_new; sz = acc_z;
  }
  // two threads share a row (one per column half of the tiles): each leaves its own partial
  __device__ __forceinline__ void end_unit(const Params& p, int un, int col_half) {
    if (row < p.T && SAPO_IN_BOUNDS(2 * un + col_half < p.parts_cap)) {
      const int64_t o = (int64_t)(2 * un + col_half) * p.T + row;
      p.pm[o] = m; p.ps[o] = s; p.pz[o] = zy;
      if constexpr (ENT) p.pe[o] = sz;
    }
  }
};
using FwdEpi = FwdEpiT<false>;

// Backward, first contraction: dz[t,v] = g_t ([v == y_t] - exp(z[t,v] - lse_t)), to bf16.
// The panel is a sequence of [128 token x 64 vocab] tiles of 16 KB, tile (tb, vt) at index
// tb * nvt + vt, each tile row-major: both later contractions then fetch whole contiguous
// tiles with one TMA box.  Rows past the last token and columns past V are written as zeros,
// because those consumers cannot tell them from data.  A finished 64-column group of a row is
// written by its thread (store_panel_group).
struct DzEpi {
  static constexpr bool PANEL = true;
  static constexpr bool STREAMK = false;
  template <class P> __device__ static void set_dynamic(P& p, const Sched& s) {
    if (s.dyn_dim == 1) p.M = *s.dyn_count;
  }
  struct Params {
    const int32_t* ids; const float* lse; const float* gscale;
    int64_t M; int32_t V; int32_t nvt;
    __nv_bfloat16* panel;
    int32_t id_offset;     // first vocabulary entry of W (a vocab shard), else 0
    int64_t panel_rows;    // 128-byte rows the panel holds (checked builds)
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
    y = valid ? p.ids[row] - p.id_offset : -1;
  }
  // dz of 32 columns; every 16 finished columns (32 bytes of the row) are stored at once, so the
  // stores of the eight epilogue warps trickle out between their arithmetic instead of leaving
  // the SM in bursts of whole rows
  template <int HALF>   // which 32-column half of the 64-column group (kept for symmetry with the other epilogues)
  __device__ __forceinline__ void chunk(const Params& p, float (&v)[32], int col0) {
    if (!in_panel) return;
    uint32_t w[8];
    if (g == 0.f) {
      #pragma unroll
      for (int j = 0; j < 8; ++j) w[j] = 0u;
      store_panel_16(p.panel, p.panel_rows, r, tile_row0, col0, w);
      store_panel_16(p.panel, p.panel_rows, r, tile_row0, col0 + 16, w);
      return;
    }
    const float ng = -g;
    const int yr = y - col0;
    #pragma unroll
    for (int h = 0; h < 2; ++h) {
      #pragma unroll
      for (int j = 16 * h; j < 16 * h + 16; ++j) v[j] = ng * ex2(fmaf(v[j], LOG2E, -l2));
      if (yr >= 16 * h && yr < 16 * h + 16) {            // the columns that hold the chosen token
        #pragma unroll
        for (int j = 16 * h; j < 16 * h + 16; ++j) if (j == yr) v[j] += g;
      }
      if (col0 + 16 * h + 16 > p.V) {                     // ragged end of the vocabulary
        #pragma unroll
        for (int j = 16 * h; j < 16 * h + 16; ++j) if (col0 + j >= p.V) v[j] = 0.f;
      }
      #pragma unroll
      for (int j = 0; j < 8; ++j) {
        __nv_bfloat162 b2 = __floats2bfloat162_rn(v[16 * h + 2 * j], v[16 * h + 2 * j + 1]);
        w[j] = *reinterpret_cast<uint32_t*>(&b2);
      }
      store_panel_16(p.panel, p.panel_rows, r, tile_row0, col0 + 16 * h, w);
    }
  }
  __device__ __forceinline__ void group_end(const Params&, int) {}
  __device__ __forceinline__ void end_unit(const Params&, int, int) {}
};

// Forward of the fused call: e[t,v] = exp(z[t,v] - c_t) against a per-token reference c_t that
// is known before the pass (see sapo_policy_loss_fwd_bwd), so no running maximum is needed:
// the epilogue adds the fp32 exponentials up per token and leaves them, rounded to bf16, in
// the tiled panel (same layout as DzEpi) for the backward contractions, which then need no
// second pass over the logits.  Nothing is clamped here: a token whose exponentials leave the
// safe range (2^100 and beyond, infinite or NaN) shows in its sum, and fused_tail_kernel then
// reports it and clears its panel row, so that the backward contractions only ever see finite
// entries.  Rows past the last token and columns past V hold zeros.
template <bool ENT>     // ENT: also sum_v e[t,v] z[t,v] per token (for the entropy, see FwdEpiT)
struct ExpEpiT {
  static constexpr bool PANEL = true;
  static constexpr bool STREAMK = false;
  template <class P> __device__ static void set_dynamic(P&, const Sched&) {}
  struct Params {
    const float* c2;      // [M] reference of each token, in the base-2 domain (c_t * log2 e)
    float* ps;            // [2 * n_splits][M] partial sums of exponentials
    float* pe;            // ENT: [2 * n_splits][M] partial sums of e z
    int64_t M; int32_t V; int32_t nvt;
    __nv_bfloat16* panel;
    int64_t panel_rows;   // 128-byte rows the panel holds, and
    int32_t parts_cap;    // partials per token the arrays hold (checked builds)
    // optional: one bit per 128-token block of the whole batch, set when some token of the block
    // can have a gradient; the panel rows of a clear block are not written (its sums still are).
    // blk0 = index of this launch's first block in that array
    const uint32_t* need; int32_t blk0;
  };
  float c, sum, sz; int32_t tile_row0; int r; bool valid, in_panel, store; int64_t row;
  __device__ __forceinline__ void begin_unit(const Params& p, int mb, int r_) {
    row = (int64_t)mb * BM + r_;
    valid = row < p.M;
    in_panel = (int64_t)mb * BM < p.M;
    store = p.need == nullptr || ((p.need[(p.blk0 + mb) >> 5] >> ((p.blk0 + mb) & 31)) & 1u) != 0u;
    r = r_;
    tile_row0 = mb * p.nvt * BM;
    c = valid ? p.c2[row] : 0.f;
    sum = 0.f; sz = 0.f;
  }
  template <int HALF>
  __device__ __forceinline__ void chunk(const Params& p, float (&v)[32], int col0) {
    if (!in_panel) return;
    uint32_t w[8];
    if (!valid || col0 >= p.V) {
      if (!store) return;
      #pragma unroll
      for (int j = 0; j < 8; ++j) w[j] = 0u;
      store_panel_16(p.panel, p.panel_rows, r, tile_row0, col0, w);
      store_panel_16(p.panel, p.panel_rows, r, tile_row0, col0 + 16, w);
      return;
    }
    // every 16 finished columns (32 bytes of the row) are stored at once: see DzEpi
    #pragma unroll
    for (int h = 0; h < 2; ++h) {
      #pragma unroll
      for (int j = 16 * h; j < 16 * h + 16; ++j) {
        const float e = ex2(fmaf(v[j], LOG2E, -c));
        // (columns past the vocabulary hold z = 0 from the zero-filled load: they add nothing)
        if constexpr (ENT) sz = fmaf((col0 + j < p.V) ? e : 0.f, v[j], sz);
        v[j] = e;
      }
      if (col0 + 16 * h + 16 > p.V) {                     // ragged end of the vocabulary
        #pragma unroll
        for (int j = 16 * h; j < 16 * h + 16; ++j) if (col0 + j >= p.V) v[j] = 0.f;
      }
      float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
      #pragma unroll
      for (int j = 16 * h; j < 16 * h + 16; j += 4) { a0 += v[j]; a1 += v[j + 1]; a2 += v[j + 2]; a3 += v[j + 3]; }
      sum += (a0 + a1) + (a2 + a3);
      if (store) {
        #pragma unroll
        for (int j = 0; j < 8; ++j) {
          __nv_bfloat162 b2 = __floats2bfloat162_rn(v[16 * h + 2 * j], v[16 * h + 2 * j + 1]);
          w[j] = *reinterpret_cast<uint32_t*>(&b2);
        }
        store_panel_16(p.panel, p.panel_rows, r, tile_row0, col0 + 16 * h, w);
      }
    }
  }
  __device__ __forceinline__ void group_end(const Params&, int) {}
  // two threads share a row (one per column half of the tiles): each leaves its own partial
  __device__ __forceinline__ void end_unit(const Params& p, int un, int col_half) {
    if (valid && SAPO_IN_BOUNDS(2 * un + col_half < p.parts_cap)) {
      p.ps[(int64_t)(2 * un + col_half) * p.M + row] = sum;
      if constexpr (ENT) p.pe[(int64_t)(2 * un + col_half) * p.M + row] = sz;
    }
  }
};
using ExpEpi = ExpEpiT<false>;

// 32 floats -> 16 packed bf16 pairs, each value scaled first
__device__ __forceinline__ void pack_bf16_32(const float (&v)[32], float scale, uint32_t (&w)[16]) {
  #pragma unroll
  for (int j = 0; j < 16; ++j) {
    __nv_bfloat162 b2 = __floats2bfloat162_rn(scale * v[2 * j], scale * v[2 * j + 1]);
    w[j] = *reinterpret_cast<uint32_t*>(&b2);
  }
}
// 8 bf16 (one 16-byte vector) + 8 floats -> 8 bf16
__device__ __forceinline__ uint4 add_bf16x8(uint4 c, const float* x) {
  __nv_bfloat162* pc = reinterpret_cast<__nv_bfloat162*>(&c);
  #pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float2 f = __bfloat1622float2(pc[j]);
    pc[j] = __floats2bfloat162_rn(f.x + x[2 * j], f.y + x[2 * j + 1]);
  }
  return c;
}

// Plain output tile (fp32, or bf16 when out_bf16 is set), optionally added to what is already there.
struct StoreEpi {
  static constexpr bool PANEL = false;
  static constexpr bool STREAMK = true;
  // row_map (optional): output row of each accumulator row (rows of compacted tokens go back
  // to their packed positions)
  // row_scale (optional): factor applied to each accumulator row before it is stored
  struct Params { void* C; int64_t ldc; int64_t M; int32_t N; int32_t accumulate; float* partials;
                  const int32_t* row_map; const float* row_scale; int32_t out_bf16;
                  int64_t out_rows; int32_t parts_cap; };   // rows of C, K-split parts the scratch holds (checked builds)
  template <class P> __device__ static void set_dynamic(P& p, const Sched& s) {
    if (s.dyn_dim == 1) p.M = *s.dyn_count;
  }
  int64_t row; bool valid; float* part; int n0; float scale;
  __device__ __forceinline__ void begin_unit(const Params& p, int mb, int r) {
    row = (int64_t)mb * BM + r;
    valid = row < p.M;
    scale = (valid && p.row_scale != nullptr) ? p.row_scale[row] : 1.f;
    if (valid && p.row_map != nullptr) row = p.row_map[row];
    if (valid && !SAPO_IN_BOUNDS(row >= 0 && row < p.out_rows)) valid = false;
    part = nullptr;
  }
  // a K-split part of a tile goes to scratch slot `slot` instead: rows [128 rank, +128) of a
  // 256 x 256 fp32 tile, column 0 = the tile's first column
  __device__ __forceinline__ void set_dest(const Params& p, int slot, int rank, int r, int n0_, int part_ld) {
    n0 = n0_;
    part = slot < 0 ? nullptr
                    : p.partials + ((size_t)slot * PAIR_M + (size_t)(rank * BM + r)) * part_ld;
    if (slot >= 0 && !SAPO_IN_BOUNDS(slot < p.parts_cap)) { part = nullptr; valid = false; }
  }
  template <int HALF>
  __device__ __forceinline__ void chunk(const Params& p, float (&v)[32], int col0) {
    if (scale == 0.f) {                    // a row without a gradient: exact zeros, whatever was contracted
      #pragma unroll
      for (int j = 0; j < 32; ++j) v[j] = 0.f;
    }
    if (part != nullptr) {
      float4* dst = reinterpret_cast<float4*>(part + (col0 - n0));
      #pragma unroll
      for (int q = 0; q < 8; ++q) dst[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
      return;
    }
    if (!valid) return;
    if (p.out_bf16) {                      // N is a multiple of 8: 16-byte vectors of 8 bf16
      uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.C) + row * p.ldc + col0);
      #pragma unroll
      for (int q = 0; q < 4; ++q) {
        if (col0 + 8 * q < p.N) {
          float x[8];
          #pragma unroll
          for (int j = 0; j < 8; ++j) x[j] = scale * v[8 * q + j];
          uint4 o;
          if (p.accumulate) o = add_bf16x8(dst[q], x);
          else              o = add_bf16x8(make_uint4(0u, 0u, 0u, 0u), x);
          dst[q] = o;
        }
      }
      return;
    }
    float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(p.C) + row * p.ldc + col0);
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
    float4 o = make_float4(scale * sum.x, scale * sum.y, scale * sum.z, scale * sum.w);
    if (scale == 0.f) o = make_float4(0.f, 0.f, 0.f, 0.f);
    if (p.out_bf16) {
      __nv_bfloat162* dst = reinterpret_cast<__nv_bfloat162*>(reinterpret_cast<__nv_bfloat16*>(p.C) + row * p.ldc + n0 + 4 * c4);
      if (p.accumulate) {
        const float2 c0 = __bfloat1622float2(dst[0]), c1 = __bfloat1622float2(dst[1]);
        o.x += c0.x; o.y += c0.y; o.z += c1.x; o.w += c1.y;
      }
      dst[0] = __floats2bfloat162_rn(o.x, o.y);
      dst[1] = __floats2bfloat162_rn(o.z, o.w);
      continue;
    }
    float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(p.C) + row * p.ldc + n0 + 4 * c4);
    if (p.accumulate) { const float4 c = *dst; o.x += c.x; o.y += c.y; o.z += c.z; o.w += c.w; }
    *dst = o;
  }
}

// Optional instrumentation (compile with -DSAPO_WAIT_STATS): cycles each role spends waiting.
#ifdef SAPO_WAIT_STATS
__device__ unsigned long long g_wait_stats[4][12];   // [8] SM cycles, [9] nanoseconds, [10] launches of CTA 0
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
#define SAPO_CLOCK_BEGIN const long long clk_c0_ = clock64(); const unsigned long long clk_n0_ = global_ns();
#define SAPO_CLOCK_END(id) do { if (blockIdx.x == 0 && threadIdx.x == 0) { \
    atomicAdd(&g_wait_stats[(id) & 3][8], (unsigned long long)(clock64() - clk_c0_)); \
    atomicAdd(&g_wait_stats[(id) & 3][9], global_ns() - clk_n0_); \
    atomicAdd(&g_wait_stats[(id) & 3][10], 1ull); } } while (0)
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
#define SAPO_CLOCK_BEGIN
#define SAPO_CLOCK_END(id) do {} while (0)
#endif

}  // namespace sapo
