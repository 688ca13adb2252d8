// LM-head projection fused with the policy loss, forward and backward, on the Blackwell
// tensor cores (tcgen05 MMA, accumulators in tensor memory, operands staged by TMA): host side
// and C ABI.  The kernels live in gemm_kernels.cuh (with gemm_sched.cuh, gemm_epilogues.cuh) and
// loss_kernels.cuh.  Contractions, all on CTA pairs with 256-row tiles:
//   forward        S = hidden . W^T    epilogue: running max / sum-exp / target logit per token
//   backward dz    S = hidden . W^T    epilogue: dz = g (onehot - exp(S - lse)) -> bf16 panel,
//                                      stored as contiguous [128 token x 64 vocab] tiles
//   single pass    S = hidden . W^T    epilogue: exp(S - c_t) -> the same panel, sums per token
//   dhidden        dH = panel . W      fp32 store (wide tiles when H >= 256)
//   dW_head        dW = panel^T . X    fp32 store / accumulate (X = hidden or its scaled copy)
// The [tokens x vocab] logits never reach global memory (paper Section 3.2 asks for the
// token-level values of every rollout under the node's policy; Section 4.2 gives the
// clipped objective the loss tail evaluates).
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"
#include "compact.cuh"
#include "umma.cuh"
#include "gemm_sched.cuh"
#include "gemm_epilogues.cuh"
#include "gemm_kernels.cuh"
#include "loss_kernels.cuh"

namespace sapo {
using namespace umma;

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
// (bf16 outputs: the same boxes are 64 bytes wide and take the 64-byte swizzle)
static bool make_map_out(CUtensorMap* map, const void* base, bool bf16, int64_t inner, int64_t outer, int64_t ld) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr || inner <= 0 || outer <= 0) return false;
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
  cuuint64_t strides[1] = {(cuuint64_t)ld * (bf16 ? 2 : 4)};
  cuuint32_t box[2] = {32u, 128u};
  cuuint32_t estr[2] = {1u, 1u};
  return fn(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
            const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            bf16 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static Sched make_sched(int64_t M, int64_t N, int64_t K, int n_splits, bool m_fastest, int tile_align = 32,
                        int bk = BK) {
  Sched s{};
  s.num_m_blocks = (int32_t)ceil_div<int64_t>(M, PAIR_M);
  const int64_t tiles = ceil_div<int64_t>(N, BN);
  s.tile_n = (int32_t)round_up<int64_t>(ceil_div<int64_t>(N, tiles), tile_align);   // equal-width tiles
  s.num_n_blocks = (int32_t)ceil_div<int64_t>(N, s.tile_n);
  s.n_per_unit = n_splits > 0 ? ceil_div(s.num_n_blocks, n_splits) : 1;
  s.units_per_m = ceil_div(s.num_n_blocks, s.n_per_unit);
  s.num_units = s.num_m_blocks * s.units_per_m;
  s.num_k_blocks = (int32_t)ceil_div<int64_t>(K, bk);
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
  s.wait_limit = WAIT_LIMIT_CLOCKS;
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

// Stage shape of the three projections hidden . W^T (forward, dz, single pass): K depth and ring length
// (a ring of seven 64-deep stages was measured 15-20 % slower: twice the barrier rounds per MMA)
constexpr int FWD_BK = BK, FWD_STAGES = STAGES;

template <int A_KIND, bool B_MN, class Epi, int BKT = BK, int NSTAGE = STAGES, class Gather = NoGather>
static int launch_gemm(const CUtensorMap& ma, const CUtensorMap& mb, const Sched& sched,
                       const typename Epi::Params& ep, int32_t* status, cudaStream_t st, int kernel_id,
                       const Gather& ga = Gather{}) {
  auto kern = umma_gemm_kernel<A_KIND, B_MN, Epi, BKT, NSTAGE, Gather>;
  // CTA pairs the device can hold at once; found, together with the kernel's shared-memory
  // opt-in, on the first use on each device
  static int max_pairs_of[MAX_DEVICES] = {0};
  const int dev = current_device();
  if (dev < 0) return SAPO_ERR_CUDA;
  int& max_pairs = max_pairs_of[dev];
  if (sched.num_units <= 0) return SAPO_OK;
  Sched sc = sched;
  sc.stats_id = (kernel_id == SAPO_K_FWD_GEMM || kernel_id == SAPO_K_FWD_EXP) ? 0 : kernel_id - SAPO_K_BWD_DZ + 1;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.blockDim = dim3(GEMM_THREADS, 1, 1);
  constexpr size_t smem_bytes = 1024 + (size_t)NSTAGE * (BM + BN / 2) * BKT * 2 + 256 +
                                (std::is_same<Gather, NoGather>::value ? 0 : GATHER_LIST_BYTES);
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
    if (cudaLaunchKernelEx(&cfg, kern, ma, mb, sc, ep, status, ga) != cudaSuccess) return SAPO_ERR_CUDA;
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
  if (!make_map_out(&mc, ep.C, ep.out_bf16 != 0, ep.N, ep.M, ep.ldc)) return SAPO_ERR_CUDA;
  auto kern = umma_gemm2_kernel<A_KIND>;
  static int max_pairs_of[MAX_DEVICES] = {0};   // as in launch_gemm: per device, found on first use
  const int dev = current_device();
  if (dev < 0) return SAPO_ERR_CUDA;
  int& max_pairs = max_pairs_of[dev];
  if (sched.num_units <= 0) return SAPO_OK;
  Sched sc = sched;
  sc.stats_id = kernel_id - SAPO_K_BWD_DZ + 1;
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
                             int64_t tc, int32_t H, int32_t V, int64_t Vp, void* dhidden, bool dh_bf16,
                             const float* row_scale, void* dW_head, bool dw_bf16, int accumulate, float* partials,
                             const uint32_t* active_mask, int32_t* status, cudaStream_t st) {
  StoreEpi::Params ep_h{dhidden, H, tc, H, 0, partials, nullptr, row_scale, dh_bf16 ? 1 : 0, tc, MAX_PARTS_SCRATCH};
  StoreEpi::Params ep_w{dW_head, H, V, H, accumulate, partials, nullptr, nullptr, dw_bf16 ? 1 : 0, V, MAX_PARTS_SCRATCH};
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
  int rc = launch_gemm<2, true, StoreEpi>(map_p_two, map_w_mn, sh, ep_h, status, st, SAPO_K_BWD_DH);
  if (rc != SAPO_OK) return rc;
  Sched sw = make_sched(V, H, tc, 0, /*m_fastest=*/false);
  sw.panel_nvt = nvt;
  return launch_gemm<3, true, StoreEpi>(map_p_tile, map_x_mn, sw, ep_w, status, st, SAPO_K_BWD_DW);
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
// max_splits > 0 caps the number of vocab splits (fewer splits: less scratch, the same results up
// to the order in which the partial sums of a token are added)
static FwdLayout fwd_layout(int64_t T, int32_t H, int32_t V, int32_t dtype, int sms, int max_splits = 0,
                            bool entropy = true) {
  FwdLayout L{};
  L.n_splits = fwd_splits(T, V, dtype == SAPO_DTYPE_F32 ? 3 * (int64_t)H : (int64_t)H, sms);
  if (max_splits > 0 && L.n_splits > max_splits) L.n_splits = max_splits;
  size_t off = 0;
  // per vocab split and column half: running max, sum, target logit (and the entropy's sum)
  L.partials = off; off += round_up<size_t>((size_t)(entropy ? 4 : 3) * 2 * L.n_splits * T * sizeof(float), 256);
  if (dtype == SAPO_DTYPE_F32) {
    L.a_split = off; off += round_up<size_t>((size_t)T * 3 * H * 2, 256);
    L.b_split = off; off += round_up<size_t>((size_t)V * 3 * H * 2, 256);
  }
  L.total = off;
  return L;
}

// out_bf16: room for an fp32 copy of dW_head, in which the token chunks are summed before the
// result is rounded to bf16 once
struct BwdLayout { size_t a_hi, b_hi, partials, dw_acc, panel, fixed; size_t bytes_per_row; };
static BwdLayout bwd_layout(int64_t T, int32_t H, int32_t V, int32_t dtype, bool out_bf16 = false) {
  BwdLayout L{};
  size_t off = 0;
  if (out_bf16) { L.dw_acc = off; off += round_up<size_t>((size_t)V * H * 4, 256); }
  if (dtype == SAPO_DTYPE_F32) {
    L.a_hi = off; off += round_up<size_t>((size_t)T * H * 2, 256);
    L.b_hi = off; off += round_up<size_t>((size_t)V * H * 2, 256);
  }
  L.partials = off; off += KSPLIT_SCRATCH_BYTES;
  L.panel = off; L.fixed = off;
  L.bytes_per_row = (size_t)padded_vocab(V) * 2;
  return L;
}
// Token rows of the panel the workspace queries ask for.  Measured (hidden 896 and 1536, vocab
// 151936): a step over chunks of 16384 tokens is within 0.3 % of one over chunks of 32768, chunks
// of 8192 cost 2-3 %, of 2048 about 15 %; a batch of up to 20480 tokens is fastest in one piece.
// Longer batches are cut into equal chunks of at most 16384 tokens (rounded up to whole
// 128-token blocks), so that no short ragged chunk is left at the end.
constexpr int64_t PANEL_ROWS_TARGET = 16384;
constexpr int64_t PANEL_ROWS_ONE_PIECE = 20480;
static int64_t equal_chunk_rows(int64_t T, int64_t max_rows) {     // max_rows: a multiple of 128
  const int64_t n = ceil_div<int64_t>(T, max_rows);
  const int64_t rows = round_up<int64_t>(ceil_div<int64_t>(T, n), BM);
  return rows < max_rows ? rows : max_rows;
}
// Waves of CTA pairs the dhidden contraction of a `rows`-token chunk takes, in units of one tile's
// time, by the schedule's own rule for its last wave.  Of the three big kernels it is the one whose
// tile count follows the chunk size (2 to 7 column tiles per 256-token block), so it decides how
// well a chunk size fills the machine.
static double dhidden_waves(int64_t rows, int32_t H, int32_t V, int pairs) {
  Sched s = make_sched_wide(rows, H, padded_vocab(V));
  s.k_split_ok = 1;
  split_last_wave(s, pairs);
  if (s.sk_tiles == 0) return (double)ceil_div(s.num_units, pairs);
  const int rounds = ceil_div(s.sk_tiles * s.sk_parts, pairs);
  return (double)(s.dp_units / pairs) + (double)rounds / s.sk_parts + 0.02 * rounds;
}
// Panel rows the workspace queries ask for.  A batch of up to 20 480 tokens is taken whole.  A
// longer one is cut into equal chunks of at most 20 480 tokens when a chunk's hidden rows still
// sit in the share of L2 the forward pass counts on (48 MB), of at most 16 384 otherwise; among
// the five smallest chunk counts that allow, the one whose dhidden contraction wastes least of
// its last wave (plus a twentieth of a tile's time per chunk for what every chunk costs anyway).
static int64_t preferred_panel_rows(int64_t T, int32_t H, int32_t V) {
  if (T <= PANEL_ROWS_ONE_PIECE) return round_up<int64_t>(T, BM);
  const int64_t cap = PANEL_ROWS_ONE_PIECE * (int64_t)H * 2 <= (48ll << 20) ? PANEL_ROWS_ONE_PIECE : PANEL_ROWS_TARGET;
  if (!use_wide_tiles(H)) return equal_chunk_rows(T, cap);
  const int sms = sm_count();
  const int pairs = sms >= 2 ? sms / 2 : 74;
  const int64_t n_min = ceil_div<int64_t>(T, cap);
  int64_t best_rows = 0; double best_cost = 0.0;
  for (int64_t n = n_min; n < n_min + 5; ++n) {
    const int64_t rows = round_up<int64_t>(ceil_div<int64_t>(T, n), BM);
    const double cost = (double)n * (dhidden_waves(rows, H, V, pairs) + 0.05);
    if (best_rows == 0 || cost < best_cost - 1e-9) { best_rows = rows; best_cost = cost; }
  }
  return best_rows;
}

// Scratch of the fused call: per-token vectors for all T tokens, then what one token chunk
// needs (row scales, partial sums, the scaled copy of hidden), the K-split scratch, the
// per-sequence sums when the caller does not want them, and the panel of exponentials.
constexpr int FUSED_MAX_SPLITS = 160;
struct FusedLayout { size_t zy, c2, obj, seq, mask, need, partials, dw_acc, boxes, n_boxes, fixed; size_t bytes_per_row; };
static FusedLayout fused_layout(int64_t T, int32_t H, int32_t V, int32_t S, bool out_bf16 = false,
                                bool gather = false) {
  FusedLayout L{};
  size_t off = 0;
  auto take = [&](size_t bytes) { const size_t at = off; off += round_up<size_t>(bytes, 256); return at; };
  if (out_bf16) L.dw_acc = take((size_t)V * H * 4);
  if (gather) {      // the box list of every 128-token block (hidden rows read in place)
    const size_t n_blocks = (size_t)ceil_div<int64_t>(T, BM);
    L.boxes = take(n_blocks * 128 * 8);
    L.n_boxes = take(n_blocks * 4);
  }
  L.zy = take((size_t)T * 4);
  L.c2 = take((size_t)T * 4);
  L.obj = take((size_t)T * 4);
  L.seq = take((size_t)(S > 0 ? S : 1) * 4);
  L.mask = take((size_t)MASK_WORDS_MAX * 4);
  L.need = take((size_t)ceil_div<int64_t>(ceil_div<int64_t>(T, BM), 32) * 4);
  L.partials = take(KSPLIT_SCRATCH_BYTES);
  L.fixed = off;
  // per chunk row: panel row, scaled hidden row, row scale, partial sums
  L.bytes_per_row = (size_t)padded_vocab(V) * 2 + (size_t)H * 2 + 4 + (size_t)2 * 2 * FUSED_MAX_SPLITS * 4;
  return L;
}
// where the per-chunk arrays sit for a chunk capacity of `rows` (a multiple of 128)
struct FusedChunk { size_t row_scale, ps, pe, hs, panel; };
static FusedChunk fused_chunk(const FusedLayout& L, int64_t rows, int32_t H) {
  FusedChunk C{};
  size_t off = L.fixed;
  auto take = [&](size_t bytes) { const size_t at = off; off += round_up<size_t>(bytes, 256); return at; };
  C.row_scale = take((size_t)rows * 4);
  C.ps = take((size_t)rows * 2 * FUSED_MAX_SPLITS * 4);
  C.pe = take((size_t)rows * 2 * FUSED_MAX_SPLITS * 4);
  C.hs = take((size_t)rows * H * 2);
  C.panel = take(0);
  return C;
}
constexpr size_t FUSED_CHUNK_SLACK = 5 * 256;   // alignment padding between the per-chunk arrays

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

// dst (bf16) = src (fp32), or dst + src when adding: the one rounding of a dW_head that was summed
// over token chunks in fp32.  n is a multiple of 8.
__global__ void __launch_bounds__(256)
round_to_bf16_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, int64_t n, int add) {
  for (int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 8; i < n; i += (int64_t)gridDim.x * blockDim.x * 8) {
    const float4 a = *reinterpret_cast<const float4*>(src + i), b = *reinterpret_cast<const float4*>(src + i + 4);
    const float x[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    uint4* d = reinterpret_cast<uint4*>(dst + i);
    *d = add_bf16x8(add ? *d : make_uint4(0u, 0u, 0u, 0u), x);
  }
}
static int launch_round_to_bf16(const float* src, void* dst, int64_t n, int add, cudaStream_t st) {
  int64_t blocks = ceil_div<int64_t>(n / 8, 256);
  const int64_t cap = (int64_t)sm_count() * 8;
  if (blocks > cap) blocks = cap;
  if (blocks <= 0) return SAPO_OK;
  KernelScope scope(SAPO_K_STREAMK_FIXUP, st);
  round_to_bf16_kernel<<<(int)blocks, 256, 0, st>>>(src, static_cast<__nv_bfloat16*>(dst), n, add);
  return check_launch();
}

// chunk_counts[c] = active tokens that fall into chunk c of `chunk_rows` compacted rows
__global__ void chunk_counts_kernel(const int32_t* n_active, int64_t chunk_rows, int32_t n_chunks,
                                    int32_t* chunk_counts) {
  for (int c = threadIdx.x; c < n_chunks; c += blockDim.x) {
    const int64_t left = (int64_t)*n_active - (int64_t)c * chunk_rows;
    chunk_counts[c] = (int32_t)(left <= 0 ? 0 : (left < chunk_rows ? left : chunk_rows));
  }
}

// Host-side checks of the forward's arguments (everything but the scratch), in the order the
// header documents.
static int fwd_check_args(const void* hidden, const void* W_head, int32_t dtype, int64_t T, int32_t H, int32_t V,
                          int64_t ld_hidden, int64_t ld_W, const int32_t* ids, const float* old_logp,
                          const float* adv, const int32_t* cu_seqlens, int32_t S, const sapo_loss_cfg* h_cfg,
                          const float* logp, const float* lse, const float* ratio, const float* surr,
                          const float* gscale, const float* loss, const int32_t* status) {
  if (!hidden || !W_head || !ids || !old_logp || !adv || !cu_seqlens || !h_cfg || !logp || !lse ||
      !ratio || !surr || !gscale || !loss || !status || S < 1)
    return SAPO_ERR_INVALID_ARG;
  if (dtype != SAPO_DTYPE_BF16 && dtype != SAPO_DTYPE_F32) return SAPO_ERR_INVALID_ARG;
  if (T < 1 || H < 1 || V < 1 || ld_hidden < H || ld_W < H) return SAPO_ERR_INVALID_ARG;
  if (!shapes_ok(T, H, V)) return SAPO_ERR_UNSUPPORTED_SHAPE;
  const int esz = dtype == SAPO_DTYPE_BF16 ? 2 : 4;
  if (!aligned16(hidden) || !aligned16(W_head) || (ld_hidden * esz) % 16 || (ld_W * esz) % 16)
    return SAPO_ERR_INVALID_ARG;
  if (!(h_cfg->eps_low >= 0.f) || !(h_cfg->eps_high >= 0.f)) return SAPO_ERR_INVALID_ARG;
  if ((h_cfg->loss_agg != 0 && h_cfg->loss_agg != 1) || (h_cfg->kl_beta != 0.f && !h_cfg->ref_logp))
    return SAPO_ERR_INVALID_ARG;
  return SAPO_OK;
}

}  // namespace sapo

// =============================================================================== C ABI
extern "C" size_t sapo_workspace_bytes(int32_t which, int64_t T, int32_t H, int32_t V, int32_t dtype) {
  using namespace sapo;
  const bool out_bf16 = (which & SAPO_WS_OUT_BF16) != 0;
  const bool gather = (which & SAPO_WS_GATHER) != 0;
  which &= ~(SAPO_WS_OUT_BF16 | SAPO_WS_GATHER);
  if (!shapes_ok(T, H, V) || (dtype != SAPO_DTYPE_BF16 && dtype != SAPO_DTYPE_F32)) return 0;
  if (which == SAPO_WS_FWD) {
    int sms = sm_count();
    if (sms <= 0) sms = 148;
    return fwd_layout(T, H, V, dtype, sms).total;
  }
  if (which == SAPO_WS_FUSED) {
    if (dtype != SAPO_DTYPE_BF16) return 0;
    const FusedLayout L = fused_layout(T, H, V, /*S=*/(int32_t)(T < 0x7fffffff ? T : 0x7fffffff), out_bf16, gather);
    return L.fixed + FUSED_CHUNK_SLACK + (size_t)preferred_panel_rows(T, H, V) * L.bytes_per_row;
  }
  if (which == SAPO_WS_BWD || which == SAPO_WS_BWD_ACTIVE) {
    const BwdLayout L = bwd_layout(T, H, V, dtype, out_bf16);
    const size_t extra = which == SAPO_WS_BWD_ACTIVE ? active_layout(T, H).total : 0;
    return extra + L.fixed + (size_t)preferred_panel_rows(T, H, V) * L.bytes_per_row;
  }
  return 0;
}

extern "C" size_t sapo_workspace_bytes_min(int32_t which, int64_t T, int32_t H, int32_t V, int32_t dtype) {
  using namespace sapo;
  const bool out_bf16 = (which & SAPO_WS_OUT_BF16) != 0;
  const bool gather = (which & SAPO_WS_GATHER) != 0;
  const int32_t flags = SAPO_WS_OUT_BF16 | SAPO_WS_GATHER;
  if ((which & ~flags) != SAPO_WS_BWD && (which & ~flags) != SAPO_WS_FUSED)
    return sapo_workspace_bytes(which, T, H, V, dtype);
  which &= ~flags;
  if (!shapes_ok(T, H, V) || (dtype != SAPO_DTYPE_BF16 && dtype != SAPO_DTYPE_F32)) return 0;
  if (which == SAPO_WS_FUSED) {
    if (dtype != SAPO_DTYPE_BF16) return 0;
    const FusedLayout L = fused_layout(T, H, V, (int32_t)(T < 0x7fffffff ? T : 0x7fffffff), out_bf16, gather);
    return L.fixed + FUSED_CHUNK_SLACK + (size_t)BM * L.bytes_per_row;
  }
  const BwdLayout L = bwd_layout(T, H, V, dtype, out_bf16);
  return L.fixed + (size_t)BM * L.bytes_per_row;
}

namespace sapo {
// The LM-head projection of the forward: hidden . W^T on the tensor cores with the online
// log-sum-exp epilogue, leaving per token one (max, sum, target logit[, entropy sum]) partial per
// vocab split and column half.  id_offset: first vocabulary entry of W when it is a shard.
static int fwd_project(const void* hidden, const void* W_head, int32_t dtype, int64_t T, int32_t H, int32_t V,
                       int64_t ld_hidden, int64_t ld_W, const int32_t* ids, int32_t id_offset, const FwdLayout& L,
                       uint8_t* ws, float* pm, float* ps, float* pz, float* pe, int32_t* status, cudaStream_t st,
                       int* n_parts) {
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
  const Sched sched = make_sched(T, V, K, L.n_splits, /*m_fastest=*/true, 32, FWD_BK);
  *n_parts = 2 * sched.units_per_m;   // one partial per vocab split and column half
  if (pe != nullptr) {
    FwdEpiT<true>::Params ep{ids, pm, ps, pz, pe, T, V, id_offset, 2 * L.n_splits};
    return launch_gemm<0, false, FwdEpiT<true>, FWD_BK, FWD_STAGES>(map_a, map_b, sched, ep, status, st, SAPO_K_FWD_GEMM);
  }
  FwdEpi::Params ep{ids, pm, ps, pz, nullptr, T, V, id_offset, 2 * L.n_splits};
  return launch_gemm<0, false, FwdEpi, FWD_BK, FWD_STAGES>(map_a, map_b, sched, ep, status, st, SAPO_K_FWD_GEMM);
}

// The loss tail over merged or unmerged partials, then the loss itself.
static int launch_tail(const TailArgs& ta, int32_t loss_agg, float* loss, int sms, cudaStream_t st) {
  // one block per sequence; at least enough blocks to zero-fill, at a few thousand tokens each,
  // the outputs of tokens that belong to no sequence (T may be the caller's buffer capacity)
  int64_t tail_blocks = ceil_div<int64_t>(ta.T, 4096);
  if (tail_blocks < ta.S) tail_blocks = ta.S;
  if (tail_blocks > (int64_t)sms * 8) tail_blocks = (int64_t)sms * 8;
  { KernelScope scope(SAPO_K_LOSS_TAIL, st); loss_tail_kernel<<<(int)tail_blocks, 256, 0, st>>>(ta); }
  { KernelScope scope(SAPO_K_LOSS_FINAL, st); loss_final_kernel<<<1, 256, 0, st>>>(ta.seq_surr, ta.cu, ta.S, ta.T, loss_agg, loss); }
  return check_launch();
}

static int fwd_impl(const void* hidden, const void* W_head, int32_t dtype,
                    int64_t T, int32_t H, int32_t V, int64_t ld_hidden, int64_t ld_W,
                    const int32_t* ids, const float* old_logp, const float* adv,
                    const int32_t* cu_seqlens, int32_t S, const sapo_loss_cfg* h_cfg,
                    float* logp, float* lse, float* ratio, float* surr, float* gscale,
                    float* seq_surr, float* loss,
                    void* workspace, size_t workspace_bytes,
                    int32_t* status, void* stream, int max_splits) {
  int rc0 = fwd_check_args(hidden, W_head, dtype, T, H, V, ld_hidden, ld_W, ids, old_logp, adv, cu_seqlens, S,
                           h_cfg, logp, lse, ratio, surr, gscale, loss, status);
  if (rc0 != SAPO_OK) return rc0;
  if (!workspace || !aligned16(workspace)) return SAPO_ERR_INVALID_ARG;
  const int sms = sm_count();
  if (sms <= 0) return SAPO_ERR_CUDA;
  const bool want_entropy = h_cfg->entropy != nullptr;
  const FwdLayout L = fwd_layout(T, H, V, dtype, sms, max_splits, want_entropy);
  // seq_surr scratch lives behind the layout when the caller does not want it
  const size_t need = L.total + (seq_surr ? 0 : round_up<size_t>((size_t)S * sizeof(float), 256));
  if (workspace_bytes < need) return SAPO_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  float* pm = reinterpret_cast<float*>(ws + L.partials);
  float* ps = pm + (size_t)2 * L.n_splits * T;
  float* pz = ps + (size_t)2 * L.n_splits * T;
  float* pe = want_entropy ? pz + (size_t)2 * L.n_splits * T : nullptr;
  float* seq_out = seq_surr ? seq_surr : reinterpret_cast<float*>(ws + L.total);

  int n_parts = 0;
  int rc = fwd_project(hidden, W_head, dtype, T, H, V, ld_hidden, ld_W, ids, /*id_offset=*/0, L, ws, pm, ps, pz, pe,
                       status, st, &n_parts);
  if (rc != SAPO_OK) return rc;

  TailArgs ta{};
  ta.pm = pm; ta.ps = ps; ta.pz = pz; ta.T = T; ta.part_stride = T;
  ta.pe = pe; ta.entropy = h_cfg->entropy;
  ta.n_splits = n_parts;
  ta.ids = ids; ta.V = V; ta.old_logp = old_logp; ta.adv = adv; ta.cu = cu_seqlens; ta.S = S;
  ta.lo_edge = 1.f - h_cfg->eps_low; ta.hi_edge = 1.f + h_cfg->eps_high; ta.grad_scale = h_cfg->grad_scale;
  ta.loss_agg = h_cfg->loss_agg; ta.kl_beta = h_cfg->kl_beta; ta.ref_logp = h_cfg->ref_logp;
  ta.logp = logp; ta.lse = lse; ta.ratio = ratio; ta.surr = surr; ta.gscale = gscale; ta.seq_surr = seq_out;
  ta.status = status;
  return launch_tail(ta, h_cfg->loss_agg, loss, sms, st);
}
}  // namespace sapo

extern "C" int sapo_policy_loss_fwd(const void* hidden, const void* W_head, int32_t dtype,
                                    int64_t T, int32_t H, int32_t V, int64_t ld_hidden, int64_t ld_W,
                                    const int32_t* ids, const float* old_logp, const float* adv,
                                    const int32_t* cu_seqlens, int32_t S, const sapo_loss_cfg* h_cfg,
                                    float* logp, float* lse, float* ratio, float* surr, float* gscale,
                                    float* seq_surr, float* loss,
                                    void* workspace, size_t workspace_bytes,
                                    int32_t* status, void* stream) {
  return sapo::fwd_impl(hidden, W_head, dtype, T, H, V, ld_hidden, ld_W, ids, old_logp, adv, cu_seqlens, S, h_cfg,
                        logp, lse, ratio, surr, gscale, seq_surr, loss, workspace, workspace_bytes, status, stream,
                        /*max_splits=*/0);
}

// ------------------------------------------------------------------------------------------
// The forward in two halves, for a vocabulary that is sharded over ranks (each rank holds rows
// [vocab_offset, vocab_offset + V_shard) of W_head and all tokens): the projection of one shard,
// reduced to one (max, sum, target logit) triple per token, and the loss tail over the triples of
// all shards once they have been gathered into local memory.
extern "C" int sapo_lmhead_lse_partial(const void* hidden, const void* W_shard, int32_t dtype,
                                       int64_t T, int32_t H, int32_t V_shard, int64_t ld_hidden, int64_t ld_W,
                                       const int32_t* ids, int32_t vocab_offset, float* triple,
                                       void* workspace, size_t workspace_bytes, int32_t* status, void* stream) {
  using namespace sapo;
  if (!hidden || !W_shard || !ids || !triple || !workspace || !status) return SAPO_ERR_INVALID_ARG;
  if (dtype != SAPO_DTYPE_BF16 && dtype != SAPO_DTYPE_F32) return SAPO_ERR_INVALID_ARG;
  if (T < 1 || H < 1 || V_shard < 1 || ld_hidden < H || ld_W < H || vocab_offset < 0) return SAPO_ERR_INVALID_ARG;
  if (!shapes_ok(T, H, V_shard)) return SAPO_ERR_UNSUPPORTED_SHAPE;
  const int esz = dtype == SAPO_DTYPE_BF16 ? 2 : 4;
  if (!aligned16(hidden) || !aligned16(W_shard) || !aligned16(workspace) || (ld_hidden * esz) % 16 || (ld_W * esz) % 16)
    return SAPO_ERR_INVALID_ARG;
  const int sms = sm_count();
  if (sms <= 0) return SAPO_ERR_CUDA;
  const FwdLayout L = fwd_layout(T, H, V_shard, dtype, sms, 0, /*entropy=*/false);
  if (workspace_bytes < L.total) return SAPO_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  float* pm = reinterpret_cast<float*>(ws + L.partials);
  float* ps = pm + (size_t)2 * L.n_splits * T;
  float* pz = ps + (size_t)2 * L.n_splits * T;
  int n_parts = 0;
  int rc = fwd_project(hidden, W_shard, dtype, T, H, V_shard, ld_hidden, ld_W, ids, vocab_offset, L, ws, pm, ps, pz,
                       nullptr, status, st, &n_parts);
  if (rc != SAPO_OK) return rc;
  int64_t blocks = ceil_div<int64_t>(T, 256);
  if (blocks > (int64_t)sms * 8) blocks = (int64_t)sms * 8;
  { KernelScope scope(SAPO_K_LOSS_TAIL, st); merge_partials_kernel<<<(int)blocks, 256, 0, st>>>(pm, ps, pz, n_parts, T, triple); }
  return check_launch();
}

extern "C" int sapo_policy_loss_from_partials(const float* triples, int32_t n_parts, int64_t T, int32_t V,
                                              const int32_t* ids, const float* old_logp, const float* adv,
                                              const int32_t* cu_seqlens, int32_t S, const sapo_loss_cfg* h_cfg,
                                              float* logp, float* lse, float* ratio, float* surr, float* gscale,
                                              float* seq_surr, float* loss, int32_t* status, void* stream) {
  using namespace sapo;
  if (!triples || !ids || !old_logp || !adv || !cu_seqlens || !h_cfg || !logp || !lse || !ratio || !surr ||
      !gscale || !seq_surr || !loss || !status || S < 1 || n_parts < 1 || T < 1 || V < 1)
    return SAPO_ERR_INVALID_ARG;
  if (!(h_cfg->eps_low >= 0.f) || !(h_cfg->eps_high >= 0.f)) return SAPO_ERR_INVALID_ARG;
  if ((h_cfg->loss_agg != 0 && h_cfg->loss_agg != 1) || (h_cfg->kl_beta != 0.f && !h_cfg->ref_logp))
    return SAPO_ERR_INVALID_ARG;
  if (h_cfg->entropy != nullptr) return SAPO_ERR_UNSUPPORTED_SHAPE;   // the triples do not carry its sum
  const int sms = sm_count();
  if (sms <= 0) return SAPO_ERR_CUDA;
  TailArgs ta{};
  ta.pm = triples; ta.ps = triples + T; ta.pz = triples + 2 * T; ta.T = T; ta.part_stride = 3 * T;
  ta.pe = nullptr; ta.entropy = nullptr;
  ta.n_splits = n_parts;
  ta.ids = ids; ta.V = V; ta.old_logp = old_logp; ta.adv = adv; ta.cu = cu_seqlens; ta.S = S;
  ta.lo_edge = 1.f - h_cfg->eps_low; ta.hi_edge = 1.f + h_cfg->eps_high; ta.grad_scale = h_cfg->grad_scale;
  ta.loss_agg = h_cfg->loss_agg; ta.kl_beta = h_cfg->kl_beta; ta.ref_logp = h_cfg->ref_logp;
  ta.logp = logp; ta.lse = lse; ta.ratio = ratio; ta.surr = surr; ta.gscale = gscale; ta.seq_surr = seq_surr;
  ta.status = status;
  return launch_tail(ta, h_cfg->loss_agg, loss, sms, static_cast<cudaStream_t>(stream));
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
  // the same checks, in the same order, as the regular forward; then what only this entry limits
  const int rc0 = fwd_check_args(hidden, W_head, dtype, T, H, V, ld_hidden, ld_W, ids, old_logp, adv, cu_seqlens,
                                 S, h_cfg, logp, lse, ratio, surr, gscale, loss, status);
  if (rc0 != SAPO_OK) return rc0;
  // fp32 operands would need bf16 copies of hidden and W_head in the scratch: far beyond it
  if (dtype != SAPO_DTYPE_BF16) return SAPO_ERR_UNSUPPORTED_SHAPE;
  int sms = sm_count();
  if (sms <= 0) return SAPO_ERR_CUDA;
  // The forward likes one set of partials per vocab split (24 bytes per token and split); take
  // as many of the splits it would choose as the array holds, at least one.
  const size_t seq_bytes = seq_surr ? 0 : round_up<size_t>((size_t)S * sizeof(float), 256);
  if (seq_bytes >= (size_t)SAPO_STATIC_SCRATCH_BYTES) return SAPO_ERR_STATIC_SCRATCH_EXCEEDED;
  const size_t avail = (size_t)SAPO_STATIC_SCRATCH_BYTES - seq_bytes;
  const bool want_entropy = h_cfg->entropy != nullptr;
  const size_t per_token = want_entropy ? 32 : 24;
  int max_splits = (int)(avail / (per_token * (size_t)T) > 4096 ? 4096 : avail / (per_token * (size_t)T));
  while (max_splits >= 1 && fwd_layout(T, H, V, dtype, sms, max_splits, want_entropy).total > avail) --max_splits;
  if (max_splits < 1) return SAPO_ERR_STATIC_SCRATCH_EXCEEDED;
  void* scratch = nullptr;
  const int rc = static_scratch(&scratch);
  if (rc != SAPO_OK) return rc;
  // Nothing in the scratch has to start at zero: the vocab-split partials and the per-sequence
  // sums are written for every token / sequence of this call before anything reads them.
  return fwd_impl(hidden, W_head, dtype, T, H, V, ld_hidden, ld_W, ids, old_logp, adv,
                  cu_seqlens, S, h_cfg, logp, lse, ratio, surr, gscale, seq_surr, loss,
                  scratch, (size_t)SAPO_STATIC_SCRATCH_BYTES, status, stream, max_splits);
}

namespace sapo {
static int bwd_impl(const void* hidden, const void* W_head, int32_t dtype,
                    int64_t T, int32_t H, int32_t V, int64_t ld_hidden, int64_t ld_W,
                    const int32_t* ids, int32_t vocab_offset, const float* lse, const float* gscale,
                    void* dhidden, void* dW_head, int32_t out_dtype, int32_t accumulate_dW,
                    void* workspace, size_t workspace_bytes,
                    int32_t* status, void* stream) {
  if (!hidden || !W_head || !ids || !lse || !gscale || !dhidden || !dW_head || !workspace || !status)
    return SAPO_ERR_INVALID_ARG;
  if (dtype != SAPO_DTYPE_BF16 && dtype != SAPO_DTYPE_F32) return SAPO_ERR_INVALID_ARG;
  if (out_dtype != SAPO_DTYPE_BF16 && out_dtype != SAPO_DTYPE_F32) return SAPO_ERR_INVALID_ARG;
  const bool out_bf16 = out_dtype == SAPO_DTYPE_BF16;
  if (T < 1 || H < 1 || V < 1 || ld_hidden < H || ld_W < H) return SAPO_ERR_INVALID_ARG;
  if (!shapes_ok(T, H, V)) return SAPO_ERR_UNSUPPORTED_SHAPE;
  const int esz = dtype == SAPO_DTYPE_BF16 ? 2 : 4;
  if (!aligned16(hidden) || !aligned16(W_head) || !aligned16(workspace) || !aligned16(dhidden) ||
      !aligned16(dW_head) || (ld_hidden * esz) % 16 || (ld_W * esz) % 16)
    return SAPO_ERR_INVALID_ARG;
  const BwdLayout L = bwd_layout(T, H, V, dtype, out_bf16);
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
  if (rows_fit <= 0) return SAPO_ERR_WORKSPACE_TOO_SMALL;
  const int64_t chunk_rows = rows_fit >= T ? T : equal_chunk_rows(T, rows_fit);   // equal chunks: no short last one
  // a bf16 dW_head that is summed over several chunks, or added to what the caller holds, is formed
  // in fp32 scratch and rounded once at the end
  const bool dw_via_acc = out_bf16 && (chunk_rows < T || accumulate_dW);
  float* dw_acc = reinterpret_cast<float*>(ws + L.dw_acc);
  const size_t out_esz = out_bf16 ? 2 : 4;

  // W as the K-major B operand of the logit recompute
  CUtensorMap map_w_kmajor;
  if (!make_map(&map_w_kmajor, B, H, V, ldb, 128)) return SAPO_ERR_CUDA;

  for (int64_t t0 = 0; t0 < T; t0 += chunk_rows) {
    const int64_t tc = (T - t0) < chunk_rows ? (T - t0) : chunk_rows;
    const __nv_bfloat16* A0 = A + t0 * lda;
    const int64_t panel_rows = ceil_div<int64_t>(tc, BM) * nvt * BM;   // 128-byte rows of the tiled panel
    CUtensorMap map_h_kmajor;
    if (!make_map(&map_h_kmajor, A0, H, tc, lda, BM)) return SAPO_ERR_CUDA;
    // dz panel: recompute logits tile by tile
    {
      Sched sched = make_sched(tc, V, H, 0, /*m_fastest=*/true, /*tile_align=*/64, FWD_BK);
      sched.n_cover = (int32_t)Vp;
      DzEpi::Params ep{ids + t0, lse + t0, gscale + t0, tc, V, nvt, panel, vocab_offset, panel_rows};
      int rc = launch_gemm<0, false, DzEpi, FWD_BK, FWD_STAGES>(map_h_kmajor, map_w_kmajor, sched, ep, status, st, SAPO_K_BWD_DZ);
      if (rc != SAPO_OK) return rc;
    }
    // dhidden[t0:t0+tc] = dz . W         (M = tokens, N = H, K = V)
    // dW (+)= dz^T . hidden               (M = V, N = H, K = tokens)
    const int rc = launch_grad_gemms(panel, panel_rows, nvt, B, ldb, A0, lda, tc, H, V, Vp,
                                     static_cast<uint8_t*>(dhidden) + (size_t)t0 * H * out_esz, out_bf16, nullptr,
                                     dw_via_acc ? (void*)dw_acc : dW_head, out_bf16 && !dw_via_acc,
                                     dw_via_acc ? (t0 > 0 ? 1 : 0) : ((t0 > 0 || accumulate_dW) ? 1 : 0),
                                     partials, nullptr, status, st);
    if (rc != SAPO_OK) return rc;
  }
  if (dw_via_acc) return launch_round_to_bf16(dw_acc, dW_head, (int64_t)V * H, accumulate_dW ? 1 : 0, st);
  return SAPO_OK;
}
}  // namespace sapo

extern "C" int sapo_policy_loss_bwd(const void* hidden, const void* W_head, int32_t dtype,
                                    int64_t T, int32_t H, int32_t V, int64_t ld_hidden, int64_t ld_W,
                                    const int32_t* ids, const float* lse, const float* gscale,
                                    void* dhidden, void* dW_head, int32_t out_dtype, int32_t accumulate_dW,
                                    void* workspace, size_t workspace_bytes,
                                    int32_t* status, void* stream) {
  return sapo::bwd_impl(hidden, W_head, dtype, T, H, V, ld_hidden, ld_W, ids, 0, lse, gscale, dhidden, dW_head,
                        out_dtype, accumulate_dW, workspace, workspace_bytes, status, stream);
}

// The same for one vocabulary shard: W_shard holds rows [vocab_offset, vocab_offset + V_shard) of
// W_head, lse is the log-sum-exp over the WHOLE vocabulary; dhidden receives this shard's share of
// the sum over v (to be added up over the shards), dW_shard the shard's rows of dW_head.
extern "C" int sapo_policy_loss_bwd_shard(const void* hidden, const void* W_shard, int32_t dtype,
                                          int64_t T, int32_t H, int32_t V_shard, int64_t ld_hidden, int64_t ld_W,
                                          const int32_t* ids, int32_t vocab_offset, const float* lse,
                                          const float* gscale, void* dhidden, void* dW_shard, int32_t out_dtype,
                                          int32_t accumulate_dW, void* workspace, size_t workspace_bytes,
                                          int32_t* status, void* stream) {
  if (vocab_offset < 0) return SAPO_ERR_INVALID_ARG;
  return sapo::bwd_impl(hidden, W_shard, dtype, T, H, V_shard, ld_hidden, ld_W, ids, vocab_offset, lse, gscale,
                        dhidden, dW_shard, out_dtype, accumulate_dW, workspace, workspace_bytes, status, stream);
}

// ------------------------------------------------------------------------------------------
// Backward over the active tokens only (g_t != 0): same results as sapo_policy_loss_bwd, less
// tensor work when many tokens are inactive.  The number of active tokens stays on the device:
// the GEMM kernels read it when they start, so the call does not synchronise.
extern "C" int sapo_policy_loss_bwd_active(const void* hidden, const void* W_head, int32_t dtype,
                                           int64_t T, int32_t H, int32_t V, int64_t ld_hidden, int64_t ld_W,
                                           const int32_t* ids, const float* lse, const float* gscale,
                                           void* dhidden, void* dW_head, int32_t out_dtype, int32_t accumulate_dW,
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
  if (out_dtype != SAPO_DTYPE_BF16 && out_dtype != SAPO_DTYPE_F32) return SAPO_ERR_INVALID_ARG;
  const bool out_bf16 = out_dtype == SAPO_DTYPE_BF16;
  const ActiveLayout AL = active_layout(T, H);
  const BwdLayout L = bwd_layout(T, H, V, dtype, out_bf16);
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
  const bool dw_via_acc = out_bf16 && (n_chunks > 1 || accumulate_dW);   // summed in fp32 scratch, rounded once at the end
  float* dw_acc = reinterpret_cast<float*>(ws + L.dw_acc);

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
                                                             lse_act, g_act, dhidden, (int64_t)H * (out_bf16 ? 2 : 4));
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
      Sched sched = make_sched(tc, V, H, 0, /*m_fastest=*/true, /*tile_align=*/64, FWD_BK);
      sched.n_cover = (int32_t)Vp;
      sched.dyn_count = count; sched.dyn_dim = 1;
      DzEpi::Params ep{ids_act + t0, lse_act + t0, g_act + t0, tc, V, nvt, panel, 0, panel_rows};
      int rc = launch_gemm<0, false, DzEpi, FWD_BK, FWD_STAGES>(map_h_kmajor, map_w_kmajor, sched, ep, status, st, SAPO_K_BWD_DZ);
      if (rc != SAPO_OK) return rc;
    }
    {
      Sched sched = make_sched(tc, H, Vp, 0, /*m_fastest=*/false);
      sched.panel_nvt = nvt;
      sched.dyn_count = count; sched.dyn_dim = 1;
      StoreEpi::Params ep{dhidden, H, tc, H, 0, partials, act_idx + t0, nullptr, out_bf16 ? 1 : 0, T,
                          MAX_PARTS_SCRATCH};   // rows go back to their tokens
      int rc = launch_gemm<2, true, StoreEpi>(map_p_two, map_w_mn, sched, ep, status, st, SAPO_K_BWD_DH);
      if (rc != SAPO_OK) return rc;
    }
    {
      const int acc = dw_via_acc ? (c > 0 ? 1 : 0) : ((c > 0 || accumulate_dW) ? 1 : 0);
      Sched sched = make_sched(V, H, tc, 0, /*m_fastest=*/false);
      sched.panel_nvt = nvt;
      sched.dyn_count = count; sched.dyn_dim = 2; sched.skip_if_empty = acc;
      StoreEpi::Params ep{dw_via_acc ? (void*)dw_acc : dW_head, H, V, H, acc, partials, nullptr, nullptr,
                          (out_bf16 && !dw_via_acc) ? 1 : 0, V, MAX_PARTS_SCRATCH};
      int rc = launch_gemm<3, true, StoreEpi>(map_p_tile, map_h_mn, sched, ep, status, st, SAPO_K_BWD_DW);
      if (rc != SAPO_OK) return rc;
    }
  }
  if (dw_via_acc) return launch_round_to_bf16(dw_acc, dW_head, (int64_t)V * H, accumulate_dW ? 1 : 0, st);
  return SAPO_OK;
}

// ------------------------------------------------------------------------------------------
// Loss and both gradients in one call, without a second pass over the logits: the forward
// epilogue leaves exp(z - c_t) in the panel, and the two backward contractions read it.
namespace sapo {
// Where the hidden rows are read in place: the two rollout stores and each packed token's row.
struct HiddenSource { const void* local; const void* ext; int64_t n_local, n_ext; const int64_t* tok_src; };

static int fused_impl(const void* hidden, const HiddenSource* src, const void* W_head, int32_t dtype,
                                        int64_t T, int32_t H, int32_t V, int64_t ld_hidden, int64_t ld_W,
                                        const int32_t* ids, const float* old_logp, const float* adv,
                                        const int32_t* cu_seqlens, int32_t S, const sapo_loss_cfg* h_cfg,
                                        float* logp, float* lse, float* ratio, float* surr, float* gscale,
                                        float* seq_surr, float* loss,
                                        void* dhidden, void* dW_head, int32_t out_dtype, int32_t accumulate_dW,
                                        void* workspace, size_t workspace_bytes,
                                        int32_t* status, void* stream) {
  const bool gather = src != nullptr;
  if (gather && (!src->tok_src || src->n_local < 0 || src->n_ext < 0 || (src->n_local > 0 && !src->local) ||
                 (src->n_ext > 0 && !src->ext) || src->n_local > 0x7fffff00LL || src->n_ext > 0x7fffff00LL))
    return SAPO_ERR_INVALID_ARG;
  if ((!gather && !hidden) || !W_head || !ids || !old_logp || !adv || !cu_seqlens || !h_cfg || !logp || !lse ||
      !ratio || !surr || !gscale || !loss || !dhidden || !dW_head || !workspace || !status || S < 1)
    return SAPO_ERR_INVALID_ARG;
  if (dtype != SAPO_DTYPE_BF16 && dtype != SAPO_DTYPE_F32) return SAPO_ERR_INVALID_ARG;
  if (T < 1 || H < 1 || V < 1 || ld_hidden < H || ld_W < H) return SAPO_ERR_INVALID_ARG;
  if (!seq_surr && S > T) return SAPO_ERR_INVALID_ARG;   // the built-in per-sequence scratch holds T entries
  if (!shapes_ok(T, H, V)) return SAPO_ERR_UNSUPPORTED_SHAPE;
  if (dtype != SAPO_DTYPE_BF16) return SAPO_ERR_UNSUPPORTED_SHAPE;   // fp32 operands: use the separate calls
  if ((!gather && !aligned16(hidden)) || !aligned16(W_head) || !aligned16(workspace) || !aligned16(dhidden) ||
      !aligned16(dW_head) || (ld_hidden * 2) % 16 || (ld_W * 2) % 16)
    return SAPO_ERR_INVALID_ARG;
  if (gather && (!aligned16(src->local) || !aligned16(src->ext))) return SAPO_ERR_INVALID_ARG;
  if (!(h_cfg->eps_low >= 0.f) || !(h_cfg->eps_high >= 0.f)) return SAPO_ERR_INVALID_ARG;
  if ((h_cfg->loss_agg != 0 && h_cfg->loss_agg != 1) || (h_cfg->kl_beta != 0.f && !h_cfg->ref_logp))
    return SAPO_ERR_INVALID_ARG;
  const int sms = sm_count();
  if (sms <= 0) return SAPO_ERR_CUDA;
  if (out_dtype != SAPO_DTYPE_BF16 && out_dtype != SAPO_DTYPE_F32) return SAPO_ERR_INVALID_ARG;
  const bool out_bf16 = out_dtype == SAPO_DTYPE_BF16;
  const FusedLayout L = fused_layout(T, H, V, (int32_t)(T < 0x7fffffff ? T : 0x7fffffff), out_bf16, gather);
  if (workspace_bytes < L.fixed + FUSED_CHUNK_SLACK + (size_t)BM * L.bytes_per_row)
    return SAPO_ERR_WORKSPACE_TOO_SMALL;
  const int64_t rows_fit =
      ((int64_t)((workspace_bytes - L.fixed - FUSED_CHUNK_SLACK) / L.bytes_per_row) / BM) * BM;
  // capacity of a chunk, a multiple of 128; equal chunks, so that no short one is left at the end
  const int64_t chunk_rows = rows_fit >= T ? round_up<int64_t>(T, BM) : equal_chunk_rows(T, rows_fit);
  const FusedChunk CL = fused_chunk(L, chunk_rows, H);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  // a bf16 dW_head that is summed over several chunks, or added to what the caller holds, is formed
  // in fp32 scratch and rounded once at the end
  const bool dw_via_acc = out_bf16 && (chunk_rows < T || accumulate_dW);
  float* dw_acc = reinterpret_cast<float*>(ws + L.dw_acc);
  const size_t out_esz = out_bf16 ? 2 : 4;
  float* zy = reinterpret_cast<float*>(ws + L.zy);
  float* c2 = reinterpret_cast<float*>(ws + L.c2);
  float* obj = reinterpret_cast<float*>(ws + L.obj);
  float* seq_out = seq_surr ? seq_surr : reinterpret_cast<float*>(ws + L.seq);
  float* partials = reinterpret_cast<float*>(ws + L.partials);
  uint32_t* active_mask = reinterpret_cast<uint32_t*>(ws + L.mask);
  float* row_scale = reinterpret_cast<float*>(ws + CL.row_scale);
  float* ps = reinterpret_cast<float*>(ws + CL.ps);
  float* pe = reinterpret_cast<float*>(ws + CL.pe);
  const bool want_entropy = h_cfg->entropy != nullptr;
  __nv_bfloat16* hs = reinterpret_cast<__nv_bfloat16*>(ws + CL.hs);
  __nv_bfloat16* panel = reinterpret_cast<__nv_bfloat16*>(ws + CL.panel);
  const __nv_bfloat16* A = static_cast<const __nv_bfloat16*>(hidden);
  const __nv_bfloat16* B = static_cast<const __nv_bfloat16*>(W_head);
  const int64_t Vp = padded_vocab(V);
  const int32_t nvt = (int32_t)(Vp / 64);
  RowSource rows{A, nullptr, ld_hidden, nullptr, 0, 0};
  GatherArgs ga{};
  uint64_t* boxes = reinterpret_cast<uint64_t*>(ws + L.boxes);
  int32_t* n_boxes = reinterpret_cast<int32_t*>(ws + L.n_boxes);
  if (gather) {
    rows = RowSource{static_cast<const __nv_bfloat16*>(src->local), static_cast<const __nv_bfloat16*>(src->ext),
                     ld_hidden, src->tok_src, src->n_local, src->n_ext};
    // boxes of 64 columns x 2^k rows over each rollout store, and the box list of every 128-token block
    for (int side = 0; side < 2; ++side) {
      const void* base = side == 0 ? src->local : src->ext;
      const int64_t n = side == 0 ? src->n_local : src->n_ext;
      for (int k = 0; k < 8; ++k)
        if (!make_map(&ga.maps[side][k], n > 0 ? base : (const void*)W_head, H, n > 0 ? n : 1, ld_hidden, 1 << k))
          return SAPO_ERR_CUDA;
    }
    const int64_t n_blocks = ceil_div<int64_t>(T, BM);
    KernelScope scope(SAPO_K_COMPACT, st);
    gather_boxes_kernel<<<(int)ceil_div<int64_t>(n_blocks, 128), 128, 0, st>>>(src->tok_src, T, src->n_local,
                                                                               src->n_ext, boxes, n_boxes, status);
  }

  // Blocks of 128 tokens whose sequences all have a zero advantage get log-probs but no gradient
  // (without a KL term): the forward leaves their panel rows unwritten and both contractions
  // skip them.  Only where the contractions do skip by block: wide tiles, a chunk's block bits
  // within what those kernels hold.
  uint32_t* need = nullptr;
  if (use_wide_tiles(H) && h_cfg->kl_beta == 0.f &&
      ceil_div<int64_t>(ceil_div<int64_t>(chunk_rows < T ? chunk_rows : T, BM), 32) <= MASK_WORDS_MAX) {
    need = reinterpret_cast<uint32_t*>(ws + L.need);
    if (cudaMemsetAsync(need, 0, (size_t)ceil_div<int64_t>(ceil_div<int64_t>(T, BM), 32) * 4, st) != cudaSuccess)
      return SAPO_ERR_CUDA;
  }
  // 1. chosen-token logits and the reference of the exponentials, all tokens
  {
    int64_t blocks = ceil_div<int64_t>(T, 8);
    if (blocks > (int64_t)sms * 8) blocks = (int64_t)sms * 8;
    KernelScope scope(SAPO_K_TARGET_LOGIT, st);
    target_logit_kernel<<<(int)blocks, 256, 0, st>>>(rows, B, ld_W, ids, old_logp, T, H, V, zy, c2,
                                                     adv, cu_seqlens, S, need);
  }
  CUtensorMap map_w_kmajor;
  if (!make_map(&map_w_kmajor, B, H, V, ld_W, 128)) return SAPO_ERR_CUDA;

  for (int64_t t0 = 0; t0 < T; t0 += chunk_rows) {
    const int64_t tc = (T - t0) < chunk_rows ? (T - t0) : chunk_rows;
    const int64_t panel_rows = ceil_div<int64_t>(tc, BM) * nvt * BM;
    CUtensorMap map_h_kmajor;
    if (gather) {
      map_h_kmajor = ga.maps[0][7];        // unused by the gathering kernel
      ga.boxes = boxes + (size_t)(t0 / BM) * 128;
      ga.n_boxes = n_boxes + t0 / BM;
      ga.rows = tc;
    } else if (!make_map(&map_h_kmajor, A + t0 * ld_hidden, H, tc, ld_hidden, BM)) {
      return SAPO_ERR_CUDA;
    }
    // 2. exponentials of the chunk -> panel, their sums per token and vocab split
    int n_splits = fwd_splits(tc, V, H, sms);
    if (n_splits > FUSED_MAX_SPLITS) n_splits = FUSED_MAX_SPLITS;
    Sched fs = make_sched(tc, V, H, n_splits, /*m_fastest=*/true, /*tile_align=*/64, FWD_BK);
    fs.n_cover = (int32_t)Vp;
    {
      int rc;
      if (want_entropy) {
        ExpEpiT<true>::Params ep{c2 + t0, ps, pe, tc, V, nvt, panel, panel_rows, 2 * FUSED_MAX_SPLITS, need, (int32_t)(t0 / BM)};
        rc = gather ? launch_gemm<0, false, ExpEpiT<true>, FWD_BK, FWD_STAGES, GatherArgs>(map_h_kmajor, map_w_kmajor, fs, ep, status, st, SAPO_K_FWD_EXP, ga)
                    : launch_gemm<0, false, ExpEpiT<true>, FWD_BK, FWD_STAGES>(map_h_kmajor, map_w_kmajor, fs, ep, status, st, SAPO_K_FWD_EXP);
      } else {
        ExpEpi::Params ep{c2 + t0, ps, nullptr, tc, V, nvt, panel, panel_rows, 2 * FUSED_MAX_SPLITS, need, (int32_t)(t0 / BM)};
        rc = gather ? launch_gemm<0, false, ExpEpi, FWD_BK, FWD_STAGES, GatherArgs>(map_h_kmajor, map_w_kmajor, fs, ep, status, st, SAPO_K_FWD_EXP, ga)
                    : launch_gemm<0, false, ExpEpi, FWD_BK, FWD_STAGES>(map_h_kmajor, map_w_kmajor, fs, ep, status, st, SAPO_K_FWD_EXP);
      }
      if (rc != SAPO_OK) return rc;
    }
    // 3. per-token loss terms, row scales, the chosen-token entries of the panel, scaled hidden rows
    {
      FusedTailArgs ta{};
      ta.ps = ps; ta.n_parts = 2 * fs.units_per_m; ta.t0 = t0; ta.tc = tc;
      ta.pe = pe; ta.entropy = h_cfg->entropy;
      ta.zy = zy; ta.c2 = c2; ta.ids = ids; ta.V = V; ta.old_logp = old_logp; ta.adv = adv;
      ta.cu = cu_seqlens; ta.S = S; ta.T = T;
      ta.lo_edge = 1.f - h_cfg->eps_low; ta.hi_edge = 1.f + h_cfg->eps_high; ta.grad_scale = h_cfg->grad_scale;
      ta.loss_agg = h_cfg->loss_agg; ta.kl_beta = h_cfg->kl_beta; ta.ref_logp = h_cfg->ref_logp;
      ta.logp = logp; ta.lse = lse; ta.ratio = ratio; ta.surr = surr; ta.gscale = gscale; ta.obj = obj;
      ta.row_scale = row_scale; ta.panel = panel; ta.nvt = nvt; ta.panel_rows = panel_rows;
      ta.rows = rows; ta.H = H; ta.hs = hs; ta.status = status;
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
                                     static_cast<uint8_t*>(dhidden) + (size_t)t0 * H * out_esz, out_bf16, row_scale,
                                     dw_via_acc ? (void*)dw_acc : dW_head, out_bf16 && !dw_via_acc,
                                     dw_via_acc ? (t0 > 0 ? 1 : 0) : ((t0 > 0 || accumulate_dW) ? 1 : 0),
                                     partials, active_mask, status, st);
    if (rc != SAPO_OK) return rc;
  }
  if (dw_via_acc) {
    const int rc = launch_round_to_bf16(dw_acc, dW_head, (int64_t)V * H, accumulate_dW ? 1 : 0, st);
    if (rc != SAPO_OK) return rc;
  }
  // 6. per-sequence means and the loss
  const int seq_blocks = S < sms * 8 ? S : sms * 8;
  { KernelScope scope(SAPO_K_LOSS_TAIL, st); seq_mean_kernel<<<seq_blocks, 256, 0, st>>>(obj, cu_seqlens, S, T, seq_out, status); }
  { KernelScope scope(SAPO_K_LOSS_FINAL, st); loss_final_kernel<<<1, 256, 0, st>>>(seq_out, cu_seqlens, S, T, h_cfg->loss_agg, loss); }
  return check_launch();
}
}  // namespace sapo

extern "C" int sapo_policy_loss_fwd_bwd(const void* hidden, const void* W_head, int32_t dtype,
                                        int64_t T, int32_t H, int32_t V, int64_t ld_hidden, int64_t ld_W,
                                        const int32_t* ids, const float* old_logp, const float* adv,
                                        const int32_t* cu_seqlens, int32_t S, const sapo_loss_cfg* h_cfg,
                                        float* logp, float* lse, float* ratio, float* surr, float* gscale,
                                        float* seq_surr, float* loss,
                                        void* dhidden, void* dW_head, int32_t out_dtype, int32_t accumulate_dW,
                                        void* workspace, size_t workspace_bytes,
                                        int32_t* status, void* stream) {
  if (!hidden) return SAPO_ERR_INVALID_ARG;
  return sapo::fused_impl(hidden, nullptr, W_head, dtype, T, H, V, ld_hidden, ld_W, ids, old_logp, adv, cu_seqlens, S,
                          h_cfg, logp, lse, ratio, surr, gscale, seq_surr, loss, dhidden, dW_head, out_dtype,
                          accumulate_dW, workspace, workspace_bytes, status, stream);
}

// The same with the hidden states read in place from the two rollout stores (no packed copy):
// tok_src is what sapo_pack_rollouts wrote, n_*_tokens the number of token rows of each store.
extern "C" int sapo_policy_loss_fwd_bwd_gather(const void* local_hidden, int64_t n_local_tokens,
                                               const void* ext_hidden, int64_t n_ext_tokens, const int64_t* tok_src,
                                               const void* W_head, int32_t dtype,
                                               int64_t T, int32_t H, int32_t V, int64_t ld_hidden, int64_t ld_W,
                                               const int32_t* ids, const float* old_logp, const float* adv,
                                               const int32_t* cu_seqlens, int32_t S, const sapo_loss_cfg* h_cfg,
                                               float* logp, float* lse, float* ratio, float* surr, float* gscale,
                                               float* seq_surr, float* loss,
                                               void* dhidden, void* dW_head, int32_t out_dtype, int32_t accumulate_dW,
                                               void* workspace, size_t workspace_bytes,
                                               int32_t* status, void* stream) {
  const sapo::HiddenSource src{local_hidden, ext_hidden, n_local_tokens, n_ext_tokens, tok_src};
  return sapo::fused_impl(nullptr, &src, W_head, dtype, T, H, V, ld_hidden, ld_W, ids, old_logp, adv, cu_seqlens, S,
                          h_cfg, logp, lse, ratio, surr, gscale, seq_surr, loss, dhidden, dW_head, out_dtype,
                          accumulate_dW, workspace, workspace_bytes, status, stream);
}

namespace sapo {
long long bounds_violations_lmhead() { return read_bounds_violations(); }
}  // namespace sapo

// ------------------------------------------------------------------------------------------
// The bounded wait, made to run out on purpose: one thread waits on a barrier nobody arrives at.
namespace sapo {
__global__ void wait_timeout_probe_kernel(long long limit_clocks, int32_t* status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) { mbar_init(&bar, 1); abort_flag = 0; fence_mbar_init(); }
  __syncthreads();
  if (threadIdx.x == 0 && !mbar_wait(&bar, 0, &abort_flag, limit_clocks)) raise_status(status, SAPO_ST_WAIT_TIMEOUT);
}
}  // namespace sapo

extern "C" int sapo_debug_wait_timeout(int64_t limit_clocks, int32_t* status, void* stream) {
  if (!status || limit_clocks < 0 || limit_clocks > 100000000) return SAPO_ERR_INVALID_ARG;   // at most ~50 ms
  sapo::wait_timeout_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>((long long)limit_clocks, status);
  return sapo::check_launch();
}

#ifdef SAPO_WAIT_STATS
// Rows: forward, dz, dH, dW.  Columns: [0] TMA waits on free stages, [1] MMA waits on filled
// stages, [2] MMA waits on a free accumulator, [3] one epilogue thread's waits on a full
// accumulator, [4..6] total cycles of the TMA / MMA / that epilogue thread, summed over CTAs
// and launches since the last reset; [7] the longest MMA-thread time of any CTA; [8] SM cycles and
// [9] nanoseconds that CTA 0 of each launch was alive, [10] the number of launches: [8] / [9] is the
// SM clock (GHz) the kernel actually ran at.  12 columns per row.
extern "C" int sapo_debug_wait_stats(unsigned long long* h_out, int32_t reset) {
  if (h_out && cudaMemcpyFromSymbol(h_out, sapo::g_wait_stats, sizeof(unsigned long long) * 48) != cudaSuccess)
    return SAPO_ERR_CUDA;
  if (reset) {
    unsigned long long z[48] = {0};
    if (cudaMemcpyToSymbol(sapo::g_wait_stats, z, sizeof(z)) != cudaSuccess) return SAPO_ERR_CUDA;
  }
  return SAPO_OK;
}
#endif
