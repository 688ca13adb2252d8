// sapo_pack_rollouts: gather the selected local and external rollouts into one varlen,
// token-major batch (paper Section 3.2, training-set equation; Algorithm 1 "Assemble
// training set").  Two kernels: a one-block scan that lays out the sequences, and an
// HBM-bound row gather.  All integer work and copies are exact.
#include "common.cuh"

namespace sapo {

struct PackArgs {
  // selection
  const int32_t* qol; const int32_t* local_idx; const int32_t* qoe; const int32_t* ext_idx;
  int32_t Q;
  // sources
  const uint8_t* hid[2]; const int32_t* ids[2]; const float* old[2];
  const int64_t* off[2]; const float* rew[2]; int32_t n_roll[2];
  // outputs
  uint8_t* o_hid; int32_t* o_ids; float* o_old; float* o_rew;
  int32_t* cu; int32_t* seq_group; uint8_t* seq_is_ext; int32_t* seq_src;
  int32_t* tok_seq; uint8_t* tok_mask; int32_t* group_offsets;
  int64_t* tok_src;          // optional: source row of every packed token (bit 62: external buffer)
  int32_t* n_tokens; int32_t* n_seqs;
  int64_t max_tokens; int32_t max_seqs;
  int64_t row_bytes;
  int32_t tokens_per_warp;   // length of the runs of packed tokens a warp copies (even)
  int32_t* status;
};

constexpr int SCAN_THREADS = 1024;

// first group q with go(q+1) > s, where go(q) = qol[q] + qoe[q] is non-decreasing
__device__ __forceinline__ int32_t group_of(const PackArgs& a, int32_t s) {
  int32_t lo = 0, hi = a.Q;            // answer in [0, Q)
  while (lo < hi) {
    int32_t mid = (lo + hi) >> 1;
    if (a.qol[mid + 1] + a.qoe[mid + 1] > s) hi = mid; else lo = mid + 1;
  }
  return lo;
}

__global__ void __launch_bounds__(SCAN_THREADS) pack_scan_kernel(PackArgs a) {
  __shared__ int64_t warp_sums[SCAN_THREADS / 32];
  __shared__ int64_t running;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t S64 = (int64_t)a.qol[a.Q] + (int64_t)a.qoe[a.Q];
  if (S64 > a.max_seqs || S64 < 0) {
    if (tid == 0) {
      raise_status(a.status, SAPO_ST_SEQ_OVERFLOW);
      *a.n_tokens = 0; *a.n_seqs = 0; a.cu[0] = 0;
    }
    for (int q = tid; q <= a.Q; q += SCAN_THREADS) a.group_offsets[q] = 0;
    return;
  }
  const int32_t S = (int32_t)S64;
  for (int q = tid; q <= a.Q; q += SCAN_THREADS) a.group_offsets[q] = a.qol[q] + a.qoe[q];
  if (tid == 0) { running = 0; a.cu[0] = 0; }
  __syncthreads();

  for (int32_t base = 0; base < S; base += SCAN_THREADS) {
    const int32_t s = base + tid;
    int64_t len = 0;
    if (s < S) {
      const int32_t q = group_of(a, s);
      const int32_t r = s - (a.qol[q] + a.qoe[q]);
      const int32_t Iq = a.qol[q + 1] - a.qol[q];
      const int side = r < Iq ? 0 : 1;
      const int32_t idx = side == 0 ? a.local_idx[a.qol[q] + r] : a.ext_idx[a.qoe[q] + (r - Iq)];
      float rew = 0.f;
      if (idx < 0 || idx >= a.n_roll[side]) {
        raise_status(a.status, SAPO_ST_BAD_INDEX);
      } else {
        len = a.off[side][idx + 1] - a.off[side][idx];
        if (len <= 0) { len = 0; raise_status(a.status, SAPO_ST_EMPTY_SEQUENCE); }
        rew = a.rew[side][idx];
      }
      a.seq_group[s] = q;
      a.seq_is_ext[s] = (uint8_t)side;
      a.seq_src[s] = idx;
      a.o_rew[s] = rew;
    }
    // inclusive block scan of len
    int64_t x = len;
    #pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      int64_t y = __shfl_up_sync(0xffffffffu, x, d);
      if (lane >= d) x += y;
    }
    if (lane == 31) warp_sums[warp] = x;
    __syncthreads();
    if (warp == 0) {
      int64_t w = warp_sums[lane];
      #pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        int64_t y = __shfl_up_sync(0xffffffffu, w, d);
        if (lane >= d) w += y;
      }
      warp_sums[lane] = w;
    }
    __syncthreads();
    const int64_t incl = running + (warp > 0 ? warp_sums[warp - 1] : 0) + x;
    if (s < S) a.cu[s + 1] = (int32_t)(incl < a.max_tokens ? incl : a.max_tokens);
    __syncthreads();
    if (tid == SCAN_THREADS - 1) running = incl;
    __syncthreads();
  }
  if (tid == 0) {
    int64_t total = running;
    if (total > a.max_tokens) { raise_status(a.status, SAPO_ST_TOKEN_OVERFLOW); total = a.max_tokens; }
    *a.n_tokens = (int32_t)total;
    *a.n_seqs = S;
  }
}

// A warp copies runs of tokens_per_warp consecutive packed tokens (16 for batches that fill
// the device several times over, 8 below that, so that small batches still spread over all
// SMs): one binary search per run,
// then it walks the sequence table, re-reading a sequence's source only when the run crosses
// into the next sequence.  Rows move as 16-byte vectors; the loads of two tokens (up to eight
// per lane) are issued before the first store.
constexpr int ROW_VECS_PER_LANE = 4;     // 16-byte vectors of one row a lane holds at a time

__global__ void __launch_bounds__(256, 3) pack_copy_kernel(PackArgs a) {
  const int lane = threadIdx.x & 31;
  const int64_t warp0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  const int32_t T = *a.n_tokens, S = *a.n_seqs;
  const bool vec = (a.row_bytes & 15) == 0;
  const int n4 = (int)(a.row_bytes >> 4);
  const bool two_at_once = vec && n4 <= 32 * ROW_VECS_PER_LANE;
  const int tpw = a.tokens_per_warp;
  // Slots past the last packed token: mask 0, sequence -1 and an all-zero row, id and log-prob, so
  // that the whole capacity can be scored without reading the token count back to the host.
  for (int64_t t = T + warp0; t < a.max_tokens; t += n_warps) {
    if (lane == 0 && a.tok_src != nullptr) a.tok_src[t] = -1;
    if (a.o_hid == nullptr) {
      if (lane == 0) { a.o_ids[t] = 0; a.o_old[t] = 0.f; a.tok_seq[t] = -1; a.tok_mask[t] = 0; }
      continue;
    }
    uint8_t* to = a.o_hid + t * a.row_bytes;
    if (vec) {
      uint4* t4 = reinterpret_cast<uint4*>(to);
      for (int j = lane; j < n4; j += 32) t4[j] = make_uint4(0u, 0u, 0u, 0u);
    } else {
      uint16_t* t2 = reinterpret_cast<uint16_t*>(to);
      for (int j = lane; j < (int)(a.row_bytes >> 1); j += 32) t2[j] = 0;
    }
    if (lane == 0) { a.o_ids[t] = 0; a.o_old[t] = 0.f; a.tok_seq[t] = -1; a.tok_mask[t] = 0; }
  }
  for (int64_t t0 = warp0 * tpw; t0 < T; t0 += n_warps * tpw) {
    int32_t s = 0;
    {
      // first s with cu[s+1] > t0 (zero-length sequences share a start; take the one that owns t0)
      int32_t lo = 0, hi = S;
      while (lo < hi) {
        int32_t mid = (lo + hi) >> 1;
        if (a.cu[mid + 1] > t0) hi = mid; else lo = mid + 1;
      }
      s = lo;
    }
    // the sequence the walk is in: its end, its side and the source token of its first token
    int32_t seq_end = -1, seq_begin = 0, side = 0;
    int64_t src0 = 0;
    auto locate = [&](int64_t t) -> int64_t {       // source token of packed token t (t < T)
      if (t >= seq_end) {
        while (a.cu[s + 1] <= t) ++s;
        seq_begin = a.cu[s]; seq_end = a.cu[s + 1];
        side = a.seq_is_ext[s];
        src0 = a.off[side][a.seq_src[s]];
      }
      return src0 + (t - seq_begin);
    };
    auto finish = [&](int64_t t, int64_t src) {     // the per-token scalars
      if (lane == 0 && SAPO_IN_BOUNDS(t >= 0 && t < a.max_tokens && src >= 0 && src < a.off[side][a.n_roll[side]])) {
        a.o_ids[t] = a.ids[side][src];
        a.o_old[t] = a.old[side][src];
        a.tok_seq[t] = s;
        a.tok_mask[t] = 1;
        if (a.tok_src != nullptr) a.tok_src[t] = src | ((int64_t)side << 62);
      }
    };
    if (a.o_hid == nullptr) {
      // no copy of the hidden rows was asked for (the caller reads them in place through tok_src)
      for (int i = 0; i < tpw && t0 + i < T; ++i) finish(t0 + i, locate(t0 + i));
      continue;
    }
    for (int i = 0; i < tpw; i += 2) {
      const int64_t ta = t0 + i, tb = ta + 1;
      if (ta >= T) break;
      const bool have_b = tb < T;
      if (two_at_once) {
        // all loads of the two tokens (rows, ids, old log-probs) are issued before the first store,
        // so the pair costs one round trip to memory, not one per dependent load-store pair
        const int64_t sa = locate(ta);
        const int32_t seq_a = s, side_a = side;
        const uint4* fa = reinterpret_cast<const uint4*>(a.hid[side] + sa * a.row_bytes);
        uint4 va[ROW_VECS_PER_LANE], vb[ROW_VECS_PER_LANE];
        #pragma unroll
        for (int q = 0; q < ROW_VECS_PER_LANE; ++q) if (lane + 32 * q < n4) va[q] = __ldg(fa + lane + 32 * q);
        const bool ok_a = lane == 0 && SAPO_IN_BOUNDS(ta < a.max_tokens && sa >= 0 && sa < a.off[side][a.n_roll[side]]);
        int32_t id_a = 0, id_b = 0; float old_a = 0.f, old_b = 0.f;
        if (ok_a) { id_a = a.ids[side][sa]; old_a = a.old[side][sa]; }
        int64_t sb = 0; int32_t seq_b = 0, side_b = 0; bool ok_b = false;
        if (have_b) {
          sb = locate(tb);
          seq_b = s; side_b = side;
          const uint4* fb = reinterpret_cast<const uint4*>(a.hid[side] + sb * a.row_bytes);
          #pragma unroll
          for (int q = 0; q < ROW_VECS_PER_LANE; ++q) if (lane + 32 * q < n4) vb[q] = __ldg(fb + lane + 32 * q);
          ok_b = lane == 0 && SAPO_IN_BOUNDS(tb < a.max_tokens && sb >= 0 && sb < a.off[side][a.n_roll[side]]);
          if (ok_b) { id_b = a.ids[side][sb]; old_b = a.old[side][sb]; }
        }
        uint4* oa = reinterpret_cast<uint4*>(a.o_hid + ta * a.row_bytes);
        #pragma unroll
        for (int q = 0; q < ROW_VECS_PER_LANE; ++q) if (lane + 32 * q < n4) oa[lane + 32 * q] = va[q];
        if (ok_a) {
          a.o_ids[ta] = id_a; a.o_old[ta] = old_a; a.tok_seq[ta] = seq_a; a.tok_mask[ta] = 1;
          if (a.tok_src != nullptr) a.tok_src[ta] = sa | ((int64_t)side_a << 62);
        }
        if (have_b) {
          uint4* ob = reinterpret_cast<uint4*>(a.o_hid + tb * a.row_bytes);
          #pragma unroll
          for (int q = 0; q < ROW_VECS_PER_LANE; ++q) if (lane + 32 * q < n4) ob[lane + 32 * q] = vb[q];
          if (ok_b) {
            a.o_ids[tb] = id_b; a.o_old[tb] = old_b; a.tok_seq[tb] = seq_b; a.tok_mask[tb] = 1;
            if (a.tok_src != nullptr) a.tok_src[tb] = sb | ((int64_t)side_b << 62);
          }
        }
        continue;
      }
      // wide or unaligned rows: one token at a time
      for (int k = 0; k < 2; ++k) {
        const int64_t t = ta + k;
        if (t >= T) break;
        const int64_t src = locate(t);
        const uint8_t* from = a.hid[side] + src * a.row_bytes;
        uint8_t* to = a.o_hid + t * a.row_bytes;
        if (vec) {
          const uint4* f4 = reinterpret_cast<const uint4*>(from);
          uint4* t4 = reinterpret_cast<uint4*>(to);
          for (int j = lane; j < n4; j += 128) {
            uint4 v0, v1, v2, v3;
            v0 = __ldg(f4 + j);
            if (j + 32 < n4) v1 = __ldg(f4 + j + 32);
            if (j + 64 < n4) v2 = __ldg(f4 + j + 64);
            if (j + 96 < n4) v3 = __ldg(f4 + j + 96);
            t4[j] = v0;
            if (j + 32 < n4) t4[j + 32] = v1;
            if (j + 64 < n4) t4[j + 64] = v2;
            if (j + 96 < n4) t4[j + 96] = v3;
          }
        } else {
          const uint16_t* f2 = reinterpret_cast<const uint16_t*>(from);
          uint16_t* t2 = reinterpret_cast<uint16_t*>(to);
          const int n2 = (int)(a.row_bytes >> 1);
          for (int j = lane; j < n2; j += 32) t2[j] = f2[j];
        }
        finish(t, src);
      }
    }
  }
}

long long bounds_violations_pack() { return read_bounds_violations(); }

}  // namespace sapo

extern "C" int sapo_pack_rollouts(const sapo_rollout_buf* h_local, const sapo_rollout_buf* h_ext,
                                  const sapo_selection* h_sel, int32_t H, int32_t dtype,
                                  const sapo_packed* h_out, int32_t* status, void* stream) {
  using namespace sapo;
  if (!h_local || !h_ext || !h_sel || !h_out || !status) return SAPO_ERR_INVALID_ARG;
  if (H <= 0 || (dtype != SAPO_DTYPE_BF16 && dtype != SAPO_DTYPE_F32)) return SAPO_ERR_INVALID_ARG;
  if (h_sel->Q < 0 || h_out->max_tokens < 0 || h_out->max_tokens > 0x7fffff00LL ||
      h_out->max_seqs < 0 || h_local->n_rollouts < 0 || h_ext->n_rollouts < 0)
    return SAPO_ERR_INVALID_ARG;
  if (!h_sel->q_offsets_local || !h_sel->q_offsets_ext || !h_out->cu_seqlens ||
      !h_out->n_tokens || !h_out->n_seqs || !h_out->group_offsets)
    return SAPO_ERR_INVALID_ARG;
  // every array a kernel will touch must be there: a NULL would only show as a device fault
  if (h_out->max_seqs > 0 && (!h_out->rewards || !h_out->seq_group || !h_out->seq_is_ext || !h_out->seq_src))
    return SAPO_ERR_INVALID_ARG;
  if (h_out->max_tokens > 0 && (!h_out->ids || !h_out->old_logp || !h_out->tok_seq || !h_out->tok_mask))
    return SAPO_ERR_INVALID_ARG;
  // the packed copy of the hidden rows is optional, but then the map to the source rows is not
  if (h_out->max_tokens > 0 && !h_out->hidden && !h_out->tok_src) return SAPO_ERR_INVALID_ARG;
  // (the index lists may be NULL: a side nobody picks from has an empty list, and only the
  // device knows the list lengths; the scan never reads an empty list)
  const sapo_rollout_buf* src_bufs[2] = {h_local, h_ext};
  for (int i = 0; i < 2; ++i)
    if (src_bufs[i]->n_rollouts > 0 && (!src_bufs[i]->hidden || !src_bufs[i]->ids || !src_bufs[i]->old_logp ||
                                        !src_bufs[i]->offsets || !src_bufs[i]->rewards))
      return SAPO_ERR_INVALID_ARG;
  PackArgs a{};
  a.qol = h_sel->q_offsets_local; a.local_idx = h_sel->local_idx;
  a.qoe = h_sel->q_offsets_ext;   a.ext_idx = h_sel->ext_idx; a.Q = h_sel->Q;
  const sapo_rollout_buf* b[2] = {h_local, h_ext};
  for (int i = 0; i < 2; ++i) {
    a.hid[i] = static_cast<const uint8_t*>(b[i]->hidden); a.ids[i] = b[i]->ids;
    a.old[i] = b[i]->old_logp; a.off[i] = b[i]->offsets; a.rew[i] = b[i]->rewards;
    a.n_roll[i] = b[i]->n_rollouts;
  }
  a.o_hid = static_cast<uint8_t*>(h_out->hidden); a.o_ids = h_out->ids; a.o_old = h_out->old_logp;
  a.o_rew = h_out->rewards; a.cu = h_out->cu_seqlens; a.seq_group = h_out->seq_group;
  a.seq_is_ext = h_out->seq_is_ext; a.seq_src = h_out->seq_src; a.tok_seq = h_out->tok_seq;
  a.tok_mask = h_out->tok_mask; a.group_offsets = h_out->group_offsets; a.tok_src = h_out->tok_src;
  a.n_tokens = h_out->n_tokens; a.n_seqs = h_out->n_seqs;
  a.max_tokens = h_out->max_tokens; a.max_seqs = h_out->max_seqs;
  a.row_bytes = (int64_t)H * (dtype == SAPO_DTYPE_BF16 ? 2 : 4);
  if (a.o_hid != nullptr && (!aligned16(a.o_hid) || !aligned16(a.hid[0]) || !aligned16(a.hid[1]))) {
    if ((a.row_bytes & 15) == 0) return SAPO_ERR_INVALID_ARG;
  }
  a.status = status;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  { KernelScope scope(SAPO_K_PACK_SCAN, st); pack_scan_kernel<<<1, SCAN_THREADS, 0, st>>>(a); }
  if (a.max_tokens > 0) {
    const int sms = sm_count();
    if (sms <= 0) return SAPO_ERR_CUDA;
    a.tokens_per_warp = a.max_tokens >= (int64_t)sms * 64 * 16 ? 16 : 8;
    const int64_t warps_wanted = (a.max_tokens + a.tokens_per_warp - 1) / a.tokens_per_warp;
    int blocks = (int)((warps_wanted + 7) / 8);
    const int max_blocks = sms * resident_blocks_per_sm(pack_copy_kernel, 256);   // the whole grid resident at once (three per SM)
    if (blocks > max_blocks) blocks = max_blocks;
    KernelScope scope(SAPO_K_PACK_COPY, st);
    pack_copy_kernel<<<blocks, 256, 0, st>>>(a);
  }
  return check_launch();
}
