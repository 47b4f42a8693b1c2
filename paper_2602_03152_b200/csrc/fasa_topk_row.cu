// TopK-I (Sec. 4.1) for score rows, one CTA per row.
//
// The cluster kernel's select-only form cuts a row over several CTAs that hold its keys in
// shared memory; with many rows its CTAs run in rounds and every round pays the whole chain of
// cluster barriers.  Here a row belongs to ONE CTA of 1024 threads that never stores the keys:
// it reads the row (4 bytes per token, from L2 after the first time) once per radix level,
//   A. an 11-bit histogram of all keys -> the bin that holds the budget-th largest key;
//   B. while that bin holds more keys than the candidate list does, another level over the
//      keys of that bin alone (11 more bits, then the last 10);
//   C. one more pass that writes the bit masks of the keys in higher bins and lists the keys
//      of the bin (the candidates); the selection finishes on the list with block-level 7-bit
//      passes, and the candidates' mask bits are settled by re-reading just their scores;
//   D. the masks become ascending positions (equal keys lowest index first = a stable sort).
// No cluster, no barrier beyond the block's own; all rows of a launch are resident at once up
// to one per SM, so the launch costs one chain, not one per round.
#include "fasa_common.cuh"
#include "fasa_score_core.cuh"

namespace {

constexpr int kRT = 1024;               // threads per CTA (one CTA per SM)
constexpr int kRW = kRT / 32;
constexpr int kRBins = 2048;
constexpr int kRGroups = kRBins / 32;
constexpr int kRCand = 8192;            // keys of one bin that the CTA finishes from a list
constexpr int kRFinBits = 7;
constexpr int kRFinBins = 1 << kRFinBits;
constexpr int kRU = 4;                  // 16-byte loads a thread keeps in flight
constexpr int kRRep = 4;                // copies of the histogram: lane l adds to copy l % 4, so that the keys a warp
constexpr int kRStride = kRBins + 8;    // crowds into one bin collide four times less; copies start 8 banks apart

struct RowParams {
  const float* scores;                  // [rows][max_len]
  const int32_t* seq_lens;
  int32_t* idx;
  int32_t* n_sel;
  int32_t* status;
  int rows_per_seq, max_len, n_sink, n_recent, budget, n_sel_max, q_len;
};

__device__ __forceinline__ uint32_t row_incl_scan(uint32_t v, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += t;
  }
  return v;
}

// Among per-lane counts v (lane 0 first), the lane where the running sum reaches kth.
__device__ __forceinline__ bool row_find_kth(uint32_t v, uint32_t kth, int lane, int* hit_lane, uint32_t* residual) {
  const uint32_t incl = row_incl_scan(v, lane);
  const uint32_t hits = __ballot_sync(0xffffffffu, incl >= kth);
  if (hits == 0u) return false;
  const int first = __ffs(hits) - 1;
  *hit_lane = first;
  *residual = kth - __shfl_sync(0xffffffffu, incl - v, first);
  return true;
}

// Block-wide: the bin of `hist` (nb <= 2048, a multiple of 32) that holds the kth largest entry,
// counted from the highest bin down; *residual = its rank inside the bin, *in_bin = the bin's count.
// Called by all threads (kth <= number of entries); two block barriers; uses s_grp.
__device__ __forceinline__ void row_block_find(const uint32_t* hist, int nb, uint32_t kth, uint32_t* s_grp, int warp,
                                               int lane, uint32_t* bin, uint32_t* residual, uint32_t* in_bin) {
  const int ng = nb / 32;
  for (int g = warp; g < kRGroups; g += kRW) {
    uint32_t x = 0;
    if (g < ng) {
#pragma unroll
      for (int r = 0; r < kRRep; ++r) x += hist[r * kRStride + g * 32 + lane];
    }
    const uint32_t v = __reduce_add_sync(0xffffffffu, x);
    if (lane == 0) s_grp[g] = v;
  }
  __syncthreads();
  const uint32_t lo = s_grp[kRGroups - 2 - 2 * lane], hi = s_grp[kRGroups - 1 - 2 * lane];   // lane 0: the two highest groups
  int hit = 31;
  uint32_t res = 1;
  if (!row_find_kth(lo + hi, kth, lane, &hit, &res)) { hit = 31; res = 1; }
  const uint32_t first = __shfl_sync(0xffffffffu, hi, hit);
  int g = kRGroups - 1 - 2 * hit;
  if (first < res) { res -= first; --g; }
  uint32_t v = 0;                                   // lane 0 = highest bin of the group
#pragma unroll
  for (int r = 0; r < kRRep; ++r) v += hist[r * kRStride + g * 32 + 31 - lane];
  int hit2 = 31;
  uint32_t res2 = 1;
  if (!row_find_kth(v, res, lane, &hit2, &res2)) { hit2 = 31; res2 = 1; }
  *bin = (uint32_t)(g * 32 + 31 - hit2);
  *residual = res2;
  *in_bin = __shfl_sync(0xffffffffu, v, hit2);
  __syncthreads();                                  // (s_grp and hist may be rewritten)
}

__global__ void __launch_bounds__(kRT, 1) topk_row_kernel(const RowParams p) {
  extern __shared__ __align__(16) unsigned char rsm[];
  __shared__ uint32_t s_grp[kRGroups];
  __shared__ unsigned long long s_wcnt[kRW];
  __shared__ uint32_t s_fin[3][kRFinBins];
  __shared__ uint32_t s_ncand;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int u = blockIdx.x, b = u / p.rows_per_seq;
  uint32_t* hist = reinterpret_cast<uint32_t*>(rsm);
  uint32_t* cand = hist + kRRep * kRStride;
  uint32_t* my_hist = hist + (lane & (kRRep - 1)) * kRStride;
  uint32_t* s_mg = cand + kRCand;                   // keys above the threshold (first: in higher bins)
  uint32_t* s_me = s_mg + (p.max_len >> 5) + 1;     // keys equal to it (first: the candidates)

  int len_raw = p.seq_lens[b];
  if (p.q_len > 1) {                                // rows of a block of queries: query t sees q_len - 1 - t fewer positions
    const int t = (u % p.rows_per_seq) / (p.rows_per_seq / p.q_len);
    if (len_raw >= 0 && len_raw <= p.max_len) len_raw = max(0, len_raw - (p.q_len - 1 - t));
  }
  const int len = clamp_len(len_raw, p.max_len, p.status);
  const long long k_budget = p.budget > 0 ? (long long)p.budget : ((long long)(-p.budget) * len + 999) / 1000;
  const int sink = min(len, p.n_sink);
  const int n_forced = sink + min(p.n_recent, len - sink);
  long long ktot_ll = min((long long)len, (long long)n_forced + k_budget);
  if (ktot_ll > p.n_sel_max) {
    ktot_ll = p.n_sel_max;
    if (tid == 0) atomicOr(p.status, FASA_DEV_NSEL_CLAMPED);
  }
  const uint32_t ktot = (uint32_t)ktot_ll;
  if (ktot == 0) {                                  // (uniform: an empty sequence)
    if (tid == 0) p.n_sel[u] = 0;
    return;
  }
  for (int i = tid; i < kRRep * kRStride; i += kRT) hist[i] = 0u;
  for (int i = tid; i < 3 * kRFinBins; i += kRT) (&s_fin[0][0])[i] = 0u;
  if (tid == 0) s_ncand = 0u;
  __syncthreads();

  const float* srow = p.scores + (int64_t)u * p.max_len;
  const bool vec_ok = (reinterpret_cast<uintptr_t>(srow) & 15) == 0;
  // One radix level: counts digit (key >> shift) & mask of the keys whose bits above `above` equal prefix.
  // A thread keeps kRU 16-byte loads in flight (2 KB per warp) and asks for the next batch before it
  // works on the one that has arrived: what an SM can pull follows the bytes its warps have
  // outstanding, and a row is read at most a handful of times, each time in full.
  // positions [free_lo, free_hi) are not forced: their key is the score's order key, capped below the forced one
  const int free_lo = sink, free_hi = len - min(p.n_recent, len - sink);
  auto plain_key = [](float sc) -> uint32_t {
    const uint32_t k = fasa_order_key(sc);
    return k == 0xffffffffu ? 0xfffffffeu : k;
  };
  auto load_batch = [&](float4 (&v)[kRU], int i0) {
#pragma unroll
    for (int r = 0; r < kRU; ++r) {
      const int i = i0 + r * kRT * 4;
      v[r] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (vec_ok && i + 3 < len) {
        v[r] = *reinterpret_cast<const float4*>(srow + i);
      } else {
        if (i < len) v[r].x = srow[i];
        if (i + 1 < len) v[r].y = srow[i + 1];
        if (i + 2 < len) v[r].z = srow[i + 2];
        if (i + 3 < len) v[r].w = srow[i + 3];
      }
    }
  };
  auto count_pass = [&](uint32_t prefix, int above, int shift, uint32_t mask) {
    float4 v[kRU], nxt[kRU];
    load_batch(v, tid * 4);
    for (int i0 = tid * 4; i0 < len; i0 += kRT * 4 * kRU) {          // (not uniform; nothing below needs it to be)
      load_batch(nxt, i0 + kRT * 4 * kRU);                           // (past the end: no loads)
#pragma unroll
      for (int r = 0; r < kRU; ++r) {
        const int i = i0 + r * kRT * 4;
        const float sv[4] = {v[r].x, v[r].y, v[r].z, v[r].w};
        if (i >= free_lo && i + 3 < free_hi) {     // no forced position among the four: the plain key
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const uint32_t key = plain_key(sv[e]);
            if (above >= 32 || (key >> above) == prefix) atomicAdd(&my_hist[(key >> shift) & mask], 1u);
          }
        } else {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            if (i + e < len) {
              const uint32_t key = fasa_item_key(sv[e], i + e, len, p.n_sink, p.n_recent);
              if (above >= 32 || (key >> above) == prefix) atomicAdd(&my_hist[(key >> shift) & mask], 1u);
            }
          }
        }
      }
#pragma unroll
      for (int r = 0; r < kRU; ++r) v[r] = nxt[r];
    }
  };

  // ---- A, B: radix levels until the bin of the ktot-th key is small enough for the list ----------
  uint32_t prefix = 0, kth = ktot, thr = 0, tie_quota = 0, in_bin = 0;
  int shift = 32;
  bool done = false, collect = false;
#pragma unroll 1
  for (int level = 0; level < 3; ++level) {
    const int bits = level == 2 ? 10 : 11;
    if (level > 0) {
      for (int i = tid; i < kRRep * kRStride; i += kRT) hist[i] = 0u;
      __syncthreads();
    }
    count_pass(prefix, shift, shift - bits, (1u << bits) - 1u);
    __syncthreads();
    uint32_t bin = 0, res = 1;
    row_block_find(hist, 1 << bits, kth, s_grp, warp, lane, &bin, &res, &in_bin);
    prefix = (prefix << bits) | bin;
    kth = res;
    shift -= bits;
    if (in_bin == kth) {            // every key of this bin is selected: its other bits do not matter
      thr = prefix << shift;
      tie_quota = 0xffffffffu;
      done = true;
      break;
    }
    if (shift == 0) {               // all 32 bits are fixed: the bin holds the keys equal to the threshold
      thr = prefix;
      tie_quota = kth;
      done = true;
      break;
    }
    if (in_bin <= (uint32_t)kRCand) {
      collect = true;
      break;
    }
  }

  // ---- C: the masks (and the candidates): a warp takes 128 consecutive tokens per step ----------
  const int n_words = (len + 31) >> 5;
  auto load_blocks = [&](float (&sv)[8], int blk0) {
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int i = blk0 * 128 + 32 * e + lane;
      sv[e] = i < len ? srow[i] : 0.f;
    }
  };
  // The step's body exists in three forms: two for blocks without forced positions or a ragged end
  // (threshold known / only its leading bits known), where a key costs a handful of instructions, and
  // the general one.
  auto emit = [&](uint32_t ma, uint32_t mc, int w, bool same, uint32_t key) {
    if (lane == 0) { s_mg[w] = ma; s_me[w] = mc; }
    if (collect && mc) {
      uint32_t base = 0;
      if (lane == 0) base = atomicAdd(&s_ncand, (uint32_t)__popc(mc));
      base = __shfl_sync(0xffffffffu, base, 0);
      const uint32_t slot = base + __popc(mc & ((1u << lane) - 1u));
      if (same && slot < (uint32_t)kRCand) cand[slot] = key;
    }
  };
  float sv[8], sv_next[8];
  load_blocks(sv, warp * 2);
  for (int blk0 = warp * 2; blk0 * 128 < len; blk0 += kRW * 2) {    // uniform over the warp; two blocks of 128 tokens
    load_blocks(sv_next, blk0 + kRW * 2);                           // (past the end: no loads)
    const int first = blk0 * 128;
    if (first >= free_lo && first + 256 <= free_hi) {               // uniform over the warp
      if (done) {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const uint32_t key = plain_key(sv[e]);
          const bool same = key == thr;
          emit(__ballot_sync(0xffffffffu, key > thr), __ballot_sync(0xffffffffu, same), blk0 * 4 + e, same, key);
        }
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const uint32_t key = plain_key(sv[e]), top = key >> shift;
          const bool same = top == prefix;
          emit(__ballot_sync(0xffffffffu, top > prefix), __ballot_sync(0xffffffffu, same), blk0 * 4 + e, same, key);
        }
      }
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int i = first + 32 * e + lane;
        const bool in = i < len;
        const uint32_t key = in ? fasa_item_key(sv[e], i, len, p.n_sink, p.n_recent) : 0u;
        bool above, same;
        if (done) {
          above = in && key > thr;
          same = in && key == thr;
        } else {
          above = in && (key >> shift) > prefix;
          same = in && (key >> shift) == prefix;
        }
        const uint32_t ma = __ballot_sync(0xffffffffu, above), mc = __ballot_sync(0xffffffffu, same);
        if (blk0 * 4 + e < n_words) emit(ma, mc, blk0 * 4 + e, same, key);
      }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) sv[e] = sv_next[e];
  }
  __syncthreads();
  const int words_per_warp = (n_words + kRW - 1) / kRW;
  const int w0 = min(n_words, warp * words_per_warp), w1 = min(n_words, w0 + words_per_warp);
  if (collect) {
    // block-level radix passes over the candidates' remaining bits, kRFinBits at a time; every warp
    // scans the small histogram itself, so a pass costs one block barrier
    int rem = shift;
#pragma unroll 1
    for (int fp = 0; rem > 0 && !done; ++fp) {
      const int wbits = rem < kRFinBits ? rem : kRFinBits;
      const int sh = rem - wbits;
      uint32_t* fh = s_fin[fp];
      for (int i = tid; i < (int)in_bin; i += kRT) {
        const uint32_t key = cand[i];
        if ((key >> rem) == prefix) atomicAdd(&fh[(key >> sh) & (uint32_t)((1 << wbits) - 1)], 1u);
      }
      __syncthreads();
      uint32_t c4[4];                               // lane l owns the four bins 127 - 4 l .. 124 - 4 l (highest first)
#pragma unroll
      for (int j = 0; j < 4; ++j) c4[j] = fh[kRFinBins - 1 - 4 * lane - j];
      int hit = 0;
      uint32_t res2 = 1;
      if (!row_find_kth(c4[0] + c4[1] + c4[2] + c4[3], kth, lane, &hit, &res2)) { hit = 0; res2 = 1; }
      uint32_t digit = 0, cnt = 0;
      bool found = false;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t c = __shfl_sync(0xffffffffu, c4[j], hit);
        if (!found) {
          if (c >= res2) { digit = (uint32_t)(kRFinBins - 1 - 4 * hit - j); cnt = c; found = true; }
          else res2 -= c;
        }
      }
      prefix = (prefix << wbits) | digit;
      kth = res2;
      rem = sh;
      if (cnt == kth && rem > 0) {  // the rest of this bin is selected whole
        thr = prefix << rem;
        tie_quota = 0xffffffffu;
        done = true;
      }
    }
    if (!done) {
      thr = prefix;
      tie_quota = kth;
      done = true;
    }
    // the candidates' bits: a lane re-reads the scores behind the bits of its own words
    for (int w = w0 + lane; w < w1; w += 32) {
      uint32_t mc = s_me[w], mg = s_mg[w], me = 0u;
      while (mc) {
        const int j = __ffs(mc) - 1;
        mc &= mc - 1;
        const int i = 32 * w + j;
        const uint32_t key = fasa_item_key(srow[i], i, len, p.n_sink, p.n_recent);
        if (key > thr) mg |= 1u << j;
        else if (key == thr) me |= 1u << j;
      }
      s_mg[w] = mg;
      s_me[w] = me;
    }
  }

  // ---- D: ascending compaction (a lane owns one word of every 32 of its warp's run) -------------
  {
    uint32_t g_tot = 0, e_tot = 0;
    for (int w = w0 + lane; w < w1; w += 32) {
      g_tot += __popc(s_mg[w]);
      e_tot += __popc(s_me[w]);
    }
    g_tot = __reduce_add_sync(0xffffffffu, g_tot);
    e_tot = __reduce_add_sync(0xffffffffu, e_tot);
    if (lane == 0) s_wcnt[warp] = ((unsigned long long)g_tot << 32) | e_tot;
  }
  __syncthreads();
  uint32_t g_run, e_run;          // selected keys before this warp's run: above / equal to the threshold
  {
    const unsigned long long mine = s_wcnt[lane];   // (kRW = 32: a warp per lane)
    unsigned long long incl = mine;
#pragma unroll
    for (int o = 1; o < kRW; o <<= 1) {
      const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    const unsigned long long before = __shfl_sync(0xffffffffu, incl - mine, warp);
    g_run = (uint32_t)(before >> 32);
    e_run = (uint32_t)before;
  }
  int32_t* out_idx = p.idx + (int64_t)u * p.n_sel_max;
  for (int wb = w0; wb < w1; wb += 32) {           // uniform over the warp
    const int w = wb + lane;
    const uint32_t mg = w < w1 ? s_mg[w] : 0u, me = w < w1 ? s_me[w] : 0u;
    const uint32_t cnt = (__popc(mg) << 16) | __popc(me), incl = row_incl_scan(cnt, lane);
    uint32_t g_before = g_run + ((incl - cnt) >> 16), e_before = e_run + ((incl - cnt) & 0xffffu);
    const uint32_t all = __shfl_sync(0xffffffffu, incl, 31);
    g_run += all >> 16;
    e_run += all & 0xffffu;
    uint32_t m = mg | me;
    while (m) {
      const int j = __ffs(m) - 1;
      m &= m - 1;
      uint32_t pos = 0xffffffffu;
      if ((mg >> j) & 1u) { pos = g_before + min(e_before, tie_quota); ++g_before; }
      else { if (e_before < tie_quota) pos = g_before + e_before; ++e_before; }
      if (pos < ktot) out_idx[pos] = 32 * w + j;   // (positions are < ktot by construction)
    }
  }
  if (tid == 0) p.n_sel[u] = (int32_t)ktot;
}

}  // namespace

// Longest row the kernel takes: its two bit masks must fit in shared memory beside the histogram
// and the candidate list.
static constexpr int kTopkRowMaxLen = 524288;

bool fasa_topk_row_ok(const fasa_ctx* ctx) { return ctx->cfg.max_len <= kTopkRowMaxLen; }

int32_t fasa_topk_row_launch(fasa_ctx* ctx, const float* scores, const int32_t* seq_lens, int32_t budget,
                             int32_t n_sel_max, int32_t* idx, int32_t* n_sel, int rows_per_seq, int n_sink,
                             int n_recent, cudaStream_t stream, int q_len) {
  const fasa_config_t& c = ctx->cfg;
  RowParams p;
  p.scores = scores; p.seq_lens = seq_lens; p.idx = idx; p.n_sel = n_sel; p.status = ctx->d_status;
  p.rows_per_seq = rows_per_seq; p.max_len = c.max_len; p.n_sink = n_sink; p.n_recent = n_recent;
  p.budget = budget; p.n_sel_max = n_sel_max; p.q_len = q_len;
  const size_t smem = (size_t)(kRRep * kRStride + kRCand) * 4 + 2 * ((size_t)(c.max_len >> 5) + 1) * 4;
  cudaError_t e = cudaFuncSetAttribute((const void*)topk_row_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)((size_t)(kRRep * kRStride + kRCand) * 4 + 2 * ((size_t)(kTopkRowMaxLen >> 5) + 1) * 4));
  if (e == cudaSuccess) {
    topk_row_kernel<<<(unsigned)(c.batch * rows_per_seq), kRT, smem, stream>>>(p);
    e = cudaGetLastError();
  }
  ctx->launches += 1;
  FASA_CUDA_TRY(ctx, e);
  return FASA_OK;
}
