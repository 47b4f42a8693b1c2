// One decode step in one launch: UpdateCache -> TIP scoring -> TopK-I -> FAC (Algorithm 2's
// order; Sec. 4.1-4.2, Eq. 6-7).
//
// One thread-block cluster per selection unit: a (batch, KV head) pair, or the part of a KV
// head's query heads that shares an index set.  The CTAs of the cluster cut the unit's cached
// tokens into contiguous slices and
//   0. (append form) the CTA whose slice ends the sequence writes the new K, V and proxy rows;
//   1. stream their slice of the tiled proxy-K buffer once (16-byte loads in tensor-core
//      fragment order, scored with mma.sync), keep every token's selection key in shared
//      memory and histogram its top 11 bits;
//   2. find the budget-th largest key by an MSB-first radix select.  A radix pass (11, 11, 10
//      bits) costs one cluster barrier: before it every CTA PUSHES the sums of its 32-bin
//      groups into every peer's shared memory, after it every warp locates the group from its
//      local copy, fetches that group's 32 bins from the peers through distributed shared
//      memory and locates the bin, redundantly and without a block barrier.  As soon as the
//      bin that holds the budget-th key has few keys cluster-wide (normally after the first
//      pass), every CTA pushes its keys of that bin to all peers (second barrier) and each CTA
//      finishes the selection on its own copy with block-level passes;
//   3. write the selected positions in ascending order (ballot masks + prefix sums, equal keys
//      lowest index first, so the result equals a stable sort).  The number of selected tokens
//      in lower-ranked CTAs follows from what step 2 has already fetched (their bin counts and
//      their pushed keys), so no barrier is needed here;
//   4. attend, each CTA over an equal share of the index list (one barrier makes the peers'
//      parts of the list visible): K/V rows gathered by index with an online softmax;
//   5. push their partial results into the shared memory of the CTA that finishes each output
//      (one last barrier), which merges them locally.
// Scores, histograms and split-K partials never travel through HBM: the launch moves the
// proxy rows of every token, the K/V rows of the selected tokens, q and the outputs.
//
// Cluster barriers per launch: the split set-up barrier, then normally four (first histogram,
// candidate keys, index list, merge); up to six when many keys share the leading bits of the
// budget-th key.  Each is reached by all
// threads of all CTAs of a cluster the same number of times: every decision around one is taken
// from cluster-wide integer sums that are identical in every warp of every CTA.  The whole-step
// form ends with the merge barrier; the select-only forms end with the last barrier of the
// selection, after which no CTA touches a peer's shared memory.  No thread spins on anything.
#include <cooperative_groups.h>

#include <type_traits>

#include "fasa_cluster_merge.cuh"
#include "fasa_common.cuh"
#include "fasa_score_core.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int kFT = 512;               // threads per CTA; two CTAs share an SM (64 registers per thread):
                                       // what one SM can pull from HBM grows with its resident warps
constexpr int kFBins = 2048;           // bins of the widest radix pass
constexpr int kPartStride = kMergePartStride - 2;   // m, l, acc[128] (+ 2 words of padding in shared memory)
constexpr int kCapMax = 22528;         // keys a CTA can hold (88 KB of shared memory)
constexpr int kCapPair = 16384;        // ... and still leave room for a second CTA on the SM
constexpr int kMaxCs = kMergeMaxCs;     // CTAs per cluster at most
constexpr int kGroups = kFBins / 32;   // 32-bin groups of the widest radix pass
constexpr int kCandCap = 4096;         // keys of one bin that the cluster finishes locally
constexpr int kFinBits = 7;            // bits per block-level pass of that local finish
constexpr int kFinBins = 1 << kFinBits;
constexpr int kHP = 4;                 // query heads per attention pass

// Dynamic shared memory of one CTA holding `cap` keys (bytes from the start):
//   keys[cap] | hist1 (8 KB) | sums1 (4 KB) | 4 KB | sums0 (4 KB) | hist0 (8 KB) | masks
// hist0 / hist1: the histograms of even / odd radix passes; sums0 / sums1: the group sums that
// every CTA of the cluster pushes here before the barrier of an even / odd pass, [rank][group].
// The candidate keys pushed after pass 0 land in hist1 .. the spare 4 KB (nothing else uses
// them then), those pushed after pass 1 in the spare 4 KB .. hist0 (read by peers during pass
// 0 only).  The attention phase reuses the area from its start (keys, histograms and masks are
// dead by then; no peer writes here after the last barrier of the selection).
struct FusedSmem {
  int keys, hist1, sums1, spare, sums0, hist0, mask, sel_end;
  int acc, part, p, al, m, l, att_end;
  int total;
};
__host__ __device__ inline FusedSmem fused_smem_layout(int cap, int kFW = kFT / 32) {   // kFW: warps per CTA
  FusedSmem L;
  L.keys = 0;
  L.hist1 = cap * 4;
  L.sums1 = L.hist1 + kFBins * 4;
  L.spare = L.sums1 + kMaxCs * kGroups * 4;
  L.sums0 = L.spare + 4096;
  L.hist0 = L.sums0 + kMaxCs * kGroups * 4;
  L.mask = L.hist0 + kFBins * 4;
  L.sel_end = L.mask + 2 * (cap / 32 + 1) * 4;     // one bit per key: above / equal to the threshold
  L.acc = 0;                                       // [kFW][kHP][128] fp32
  L.part = L.acc + kFW * kHP * FASA_HEAD_DIM * 4;  // [8][kPartStride + 2]
  L.p = L.part + FASA_MAX_GROUP * (kPartStride + 2) * 4;   // [kFW][16]
  L.al = L.p + kFW * 16 * 4;                       // [kFW][kHP]
  L.m = L.al + kFW * kHP * 4;
  L.l = L.m + kFW * kHP * 4;
  L.att_end = L.l + kFW * kHP * 4;
  L.total = L.sel_end > L.att_end ? L.sel_end : L.att_end;
  return L;
}
static_assert(kFBins * 4 + kMaxCs * kGroups * 4 + 4096 == kCandCap * 4, "candidate area");

struct FusedParams {
  const uint16_t* q;
  const uint16_t* k;
  const uint16_t* v;
  const unsigned char* proxy;
  const int32_t* seq_lens;
  const int16_t* chan;
  // append-then-step form (all null / unused otherwise): the new token's rows, the buffers
  // they are written to, the length to update and a per-sequence arrival counter
  const uint16_t* k_new;
  const uint16_t* v_new;
  uint16_t* k_w;
  uint16_t* v_w;
  unsigned char* proxy_w;
  int32_t* seq_lens_w;
  int32_t* arrive;
  int shift_clusters, shift_ctas;   // phase shift of grids that run in rounds: clusters / CTAs resident at once (0: none)
  float* scores;           // nullable
  int32_t* idx;
  int32_t* n_sel;
  float* out;
  float* out_mirror;       // nullable: a second copy of out (mapped host memory of the host-buffer step)
  float* lse;              // nullable
  int32_t* status;
  int n_q_heads, n_kv_heads, n_sets, group, max_len, chunks, n_sink, n_recent, budget, n_sel_max;   // group: query heads of a unit
  int max_reduce;          // score of a KV head = max over its query heads instead of their sum
  int q_len;               // select-only form over blocks of queries: rows per sequence are (query, set) pairs,
                           // query t sees q_len - 1 - t fewer positions (0 or 1: plain rows)
  int64_t ksb, ksh, kst, vsb, vsh, vst;
  float scale_log2;        // softmax_scale * log2(e)
  PageMap pm;              // paged caches (all zero: contiguous)
};

__device__ __forceinline__ uint2 ld_stream_u2(const void* p) {
  uint2 r;
  asm volatile("ld.global.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(r.x), "=r"(r.y) : "l"(p) : "memory");
  return r;
}

// The two halves of a cluster barrier (cluster.sync() = arrive + wait), for all threads of all
// CTAs alike: what a thread wrote before its arrive is visible to every thread after its wait.
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t t = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += t;
  }
  return v;
}

// Among per-lane counts v (lane 0 first), finds the lane where the running sum reaches kth.
// Returns true when found; *hit_lane and *residual (= kth minus the sum before that lane) are
// then uniform over the warp.  *total is the sum over the warp.
__device__ __forceinline__ bool warp_find_kth(uint32_t v, uint32_t kth, int lane, int* hit_lane,
                                              uint32_t* residual, uint32_t* total) {
  const uint32_t incl = warp_incl_scan(v, lane);
  *total = __shfl_sync(0xffffffffu, incl, 31);
  const uint32_t hits = __ballot_sync(0xffffffffu, incl >= kth);
  if (hits == 0u) return false;
  const int first = __ffs(hits) - 1;
  const uint32_t before = __shfl_sync(0xffffffffu, incl - v, first);
  *hit_lane = first;
  *residual = kth - before;
  return true;
}

// A tile's 16-channel blocks are taken NG groups of KB at a time (KB = 1, 2, 4; NG = 2 only with
// KB = 4, for more than 4 blocks), which bounds the registers the loads in flight need.
// MODE 0: the whole step.  MODE 1: TopK-I alone (fasa_topk): the keys come from a score buffer
// instead of the proxy stream, and the kernel ends after the index list is written.  MODE 2:
// the step without its attention phase (large selections are attended by the split-K
// tensor-core kernel instead).
// PAGED: K, V and the proxy are page pools behind a block table (compiled separately, so that
// the contiguous form keeps its plain address arithmetic within 64 registers).
// NT: threads per CTA: 512 (two CTAs per SM) or 1024 (one CTA per SM with twice the slice).
template <int KB, int NG, int MODE, bool PAGED = false, int NT = 512>
__global__ void __launch_bounds__(NT, NT == 512 ? 2 : 1)
fused_decode_kernel(const FusedParams p) {
  constexpr int kFT = NT;                  // (shadow the file-level constants inside this kernel)
  constexpr int kFW = NT / 32;
  cg::cluster_group cluster = cg::this_cluster();
  const int cs = (int)cluster.num_blocks();
  const int crank = (int)cluster.block_rank();
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int warp = tid >> 5;
  const int u = blockIdx.y;
  const SelUnit su = sel_unit(u, p.n_sets, p.group, p.n_q_heads, p.n_kv_heads);
  const int h = su.h;
  const int b = su.b;

  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ unsigned long long s_wcnt[kFW];
  __shared__ uint32_t s_fin[3][kFinBins];          // histograms of the local finish (one per pass)
  __shared__ __align__(8) uint32_t s_gsum[3][2][kGroups];   // per radix pass: cluster-wide group sums, and those of the lower ranks (added by the peers)
  __shared__ uint32_t s_fine[3][2][32];            // per radix pass: the bins of the group that holds the kth key, same two sums
  __shared__ uint32_t s_mine[kGroups];             // this CTA's group sums of the current pass
  __shared__ uint32_t s_ncand, s_cgt, s_ceq;       // candidates found here; pushed keys of lower ranks above / equal to the threshold
  __shared__ int s_len_old;
  constexpr int GP = FASA_MAX_GROUP;     // query heads a KV head can serve
  constexpr int HP = kHP;                // heads per attention pass
  __shared__ __align__(16) float s_q[GP][FASA_HEAD_DIM];
  __shared__ __align__(16) uint16_t s_qraw[GP][FASA_HEAD_DIM];   // the unit's query rows as stored (scoring operand)
  __shared__ int16_t s_chan[8 * FASA_MAX_DOM / 4];               // the head's channel table
  __shared__ ClusterMergeSmem s_merge;                            // pushed by the cluster: the partial results this CTA finishes

  // ---- slices -------------------------------------------------------------------------
  // Append-then-step: one thread reads the length for the whole CTA, so that the CTA's arrival
  // (below) certifies that it no longer needs the old value; the last CTA of the sequence to
  // arrive stores the new length.  Nothing waits on the counter.
  // Loads that depend on nothing are issued first, so their (cold) latencies overlap: the
  // length, this thread's 16 bytes of the unit's query rows and its entry of the channel table.
  // The scoring operand (query values at the dominant channels) is gathered from the staged
  // copies in shared memory after the set-up barrier: no load waits on another load's result.
  const bool append = MODE != 1 && p.k_new != nullptr;
  int len_raw = 0;
  if (!append || tid == 0) len_raw = p.seq_lens[b];
  uint4 q_stage = make_uint4(0u, 0u, 0u, 0u);
  if (MODE != 1 && tid < FASA_MAX_GROUP * (FASA_HEAD_DIM / 8) && tid / (FASA_HEAD_DIM / 8) < p.group)
    q_stage = *reinterpret_cast<const uint4*>(p.q + su.q0 * FASA_HEAD_DIM + tid * 8);
  int16_t chan_stage = -1;
  if (MODE != 1 && tid < p.chunks * 8) chan_stage = p.chan[h * p.chunks * 8 + tid];
  if (MODE == 1 && p.q_len > 1) {
    const int t = (u % p.n_sets) / (p.n_sets / p.q_len);        // the query of this row
    if (len_raw >= 0 && len_raw <= p.max_len) len_raw = max(0, len_raw - (p.q_len - 1 - t));   // (a bad length is left for clamp_len to flag)
  }
  int len_old;
  if (append) {
    if (tid == 0) s_len_old = clamp_len(len_raw, p.max_len, p.status);
    __syncthreads();
    len_old = s_len_old;
  } else {
    len_old = clamp_len(len_raw, p.max_len, p.status);
  }
  const bool grows = append && len_old < p.max_len;
  const int len = len_old + (grows ? 1 : 0);
  if (append && tid == 0) {
    if (!grows && crank == 0) atomicOr(p.status, FASA_DEV_APPEND_FULL);
    __threadfence();
    const int total = p.n_sets * cs;
    if (atomicAdd(&p.arrive[b], 1) == total - 1) {
      p.seq_lens_w[b] = len;
      p.arrive[b] = 0;
    }
  }
  const int per = (((len + cs - 1) / cs) + 31) & ~31;          // <= the capacity the host sized
  const int c0 = min(len, crank * per);
  const int c1 = min(len, c0 + per);
  const int nloc = c1 - c0;
  // Phase shift.  A grid of several rounds of CTAs runs in lock-step: streams that run side by side
  // share HBM evenly and end together, after which all their CTAs select at the same time and HBM
  // idles for the length of a select chain, round after round.  Every second cluster of the FIRST
  // round therefore starts late by a little under half the time the round's streams take (its own
  // slice stands for the average; 6.4 bytes per ns is about what the memory delivers), which puts
  // the two halves of the machine out of phase for the rest of the launch: one half streams while
  // the other selects.  Measured: batch 16 at 64-128 K 177.9 -> 167.9 us, batch 32 at 64 K
  // 225.9 -> 189.2 us.  The wait is a sleep bounded by the clock; nothing is waited for.
  if (MODE != 1 && p.shift_ctas > 0 && (int)blockIdx.y < p.shift_clusters && (blockIdx.y & 1)) {
    const float ns = 0.45f * (float)p.shift_ctas * (float)nloc * (float)(p.chunks * 16) * (1.0f / 6400.0f);
    const unsigned long long want = (unsigned long long)fminf(ns, 200000.0f);
    unsigned long long t0, t1;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    do {
      __nanosleep(1000);
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
    } while (t1 - t0 < want);
  }
  const int cap = (((p.max_len + cs - 1) / cs) + 31) & ~31;
  const FusedSmem sl = fused_smem_layout(cap, kFW);
  uint32_t* keys = reinterpret_cast<uint32_t*>(smem_raw + sl.keys);
  uint32_t* hist0 = reinterpret_cast<uint32_t*>(smem_raw + sl.hist0);
  uint32_t* hist1 = reinterpret_cast<uint32_t*>(smem_raw + sl.hist1);
  uint32_t* s_mask = reinterpret_cast<uint32_t*>(smem_raw + sl.mask);

  const long long k_budget =
      p.budget > 0 ? (long long)p.budget : ((long long)(-p.budget) * len + 999) / 1000;
  const int sink = min(len, p.n_sink);
  const int n_forced = sink + min(p.n_recent, len - sink);
  long long ktot_ll = min((long long)len, (long long)n_forced + k_budget);
  if (ktot_ll > p.n_sel_max) {
    ktot_ll = p.n_sel_max;
    if (crank == 0 && tid == 0) atomicOr(p.status, FASA_DEV_NSEL_CLAMPED);
  }
  const uint32_t ktot = (uint32_t)ktot_ll;

  // The first proxy loads leave before the rest of the set-up (histogram clearing, query
  // staging, its barrier), whose latency they then hide.  A warp keeps about four 16-byte
  // loads per lane in flight (more do not raise what a warp can pull); the SM's bandwidth
  // comes from its 32 resident warps.  Only the CTA that is about to write the new token's
  // rows has to wait for them.
  constexpr int TPI = KB == 1 ? 4 : 2;                        // tiles per warp iteration (even)
  const ProxyGeom pg = proxy_geom(p.chunks);
  const int n_blocks = pg.n16 + pg.n8;
  const unsigned char* unit = p.proxy + (int64_t)su.kv * ((p.max_len + 15) >> 4) * pg.tile_bytes;
  float* srow = p.scores ? p.scores + (int64_t)u * p.max_len : nullptr;
  const int tiles_alloc = (p.max_len + 15) >> 4;
  // Paged caches: the tiles of a batch are located through the block table.  The table is read
  // one batch ahead (tp_next) so that its latency overlaps the proxy loads in flight.
  const unsigned char* tp[PAGED ? TPI : 1];
  const unsigned char* tp_next[PAGED ? TPI : 1];
  auto locate = [&](const unsigned char* (&out)[PAGED ? TPI : 1], int T) {
    if constexpr (PAGED) {
#pragma unroll
      for (int j = 0; j < TPI; ++j)
        out[j] = p.proxy + proxy_tile_offset(p.pm, b, h, p.n_kv_heads, min(T + j, tiles_alloc - 1), tiles_alloc,
                                             pg.tile_bytes, (T + j) * 16 < c1 ? p.status : nullptr);
    }
  };
  auto fetch = [&](uint4 (&a)[TPI][KB], int T, int grp) {      // (paged: tp holds the tiles of batch T)
#pragma unroll
    for (int j = 0; j < TPI; ++j) {
      const unsigned char* tile;
      if constexpr (PAGED) tile = tp[j];
      else tile = unit + (int64_t)(T + j) * pg.tile_bytes;
      load_tile<KB>(a[j], tile, pg, lane, (T + j) * 16 < c1, grp * KB);
    }
  };
  const int step = kFW * TPI;
  int T = ((crank * per) >> 4) + warp * TPI;                  // slices start on a tile boundary
  const bool own_new = grows && c0 <= len_old && len_old < c1;
  uint4 a[TPI][KB];
  if (MODE != 1) locate(tp, T);
  if (MODE != 1 && !own_new) fetch(a, T, 0);

  if (own_new) {
    // this CTA's slice holds the new row: K and V copies (16 lanes each) and the packed
    // dominant-FC pairs of the key (one lane per 16-byte chunk), as in fasa_kv_append.  When
    // several units share a KV head each writes the same values, and reads back its own.
    const uint16_t* ksrc = p.k_new + (int64_t)su.kv * FASA_HEAD_DIM;
    const ProxyGeom pg = proxy_geom(p.chunks);
    // where the row goes: the sequence's own cache, or (paged) the page of position len_old; a
    // table entry outside the pool drops the row
    int64_t koff = b * p.ksb + h * p.ksh + (int64_t)len_old * p.kst;
    int64_t voff = b * p.vsb + h * p.vsh + (int64_t)len_old * p.vst;
    int64_t poff = (int64_t)su.kv * ((p.max_len + 15) >> 4) * pg.tile_bytes;
    int prow = len_old;
    bool row_ok = true;
    if constexpr (PAGED) {
      const int page = page_of(p.pm, b, len_old);
      row_ok = page_ok(p.pm, page);
      if (!row_ok && tid == 0) atomicOr(p.status, FASA_DEV_PAGE_CLAMPED);
      prow = len_old & ((1 << p.pm.shift) - 1);
      koff = page * p.ksb + h * p.ksh + (int64_t)prow * p.kst;
      voff = page * p.vsb + h * p.vsh + (int64_t)prow * p.vst;
      poff = ((int64_t)page * p.n_kv_heads + h) * (1 << (p.pm.shift - 4)) * pg.tile_bytes;
    }
    if (!row_ok) {
    } else if (tid < 16) {
      *reinterpret_cast<uint4*>(p.k_w + koff + tid * 8) = *reinterpret_cast<const uint4*>(ksrc + tid * 8);
    } else if (tid < 32) {
      const int c = tid - 16;
      *reinterpret_cast<uint4*>(p.v_w + voff + c * 8) =
          *reinterpret_cast<const uint4*>(p.v_new + (int64_t)su.kv * FASA_HEAD_DIM + c * 8);
    } else if (tid - 32 < 4 * p.chunks) {
      const int w = tid - 32;                       // one dominant FC = one 4-byte channel pair
      const int16_t* ch = p.chan + h * p.chunks * 8 + 2 * w;
      const int ch0 = ch[0], ch1 = ch[1];
      const uint32_t lo = ch0 >= 0 ? ksrc[ch0] : 0u;
      const uint32_t hi = ch1 >= 0 ? ksrc[ch1] : 0u;
      *reinterpret_cast<uint32_t*>(p.proxy_w + poff + proxy_word_offset(pg, prow, w)) = lo | (hi << 16);
    }
  }
  for (int i = tid; i < kFBins; i += kFT) { hist0[i] = 0u; hist1[i] = 0u; }
  for (int i = tid; i < 3 * kFinBins; i += kFT) (&s_fin[0][0])[i] = 0u;
  for (int i = tid; i < 3 * 2 * kGroups; i += kFT) (&s_gsum[0][0][0])[i] = 0u;
  for (int i = tid; i < 3 * 2 * 32; i += kFT) (&s_fine[0][0][0])[i] = 0u;
  if (tid == 0) { s_ncand = 0u; s_cgt = 0u; s_ceq = 0u; }
  if (MODE != 1 && tid < GP * (FASA_HEAD_DIM / 8))
    *reinterpret_cast<uint4*>(&s_qraw[tid / (FASA_HEAD_DIM / 8)][(tid % (FASA_HEAD_DIM / 8)) * 8]) = q_stage;
  if (MODE != 1 && tid < p.chunks * 8) s_chan[tid] = chan_stage;
  // query, scaled into the base-2 logit domain, for the attention phase
  if (MODE == 0 && tid < GP * (FASA_HEAD_DIM / 8)) {
    const int g = tid / (FASA_HEAD_DIM / 8), c = (tid % (FASA_HEAD_DIM / 8)) * 8;
    const uint4 w = q_stage;
    const float2 f0 = bf16x2_to_f32x2(w.x), f1 = bf16x2_to_f32x2(w.y), f2 = bf16x2_to_f32x2(w.z), f3 = bf16x2_to_f32x2(w.w);
    const float sc = p.scale_log2;
    *reinterpret_cast<float4*>(&s_q[g][c]) = make_float4(f0.x * sc, f0.y * sc, f1.x * sc, f1.y * sc);
    *reinterpret_cast<float4*>(&s_q[g][c + 4]) = make_float4(f2.x * sc, f2.y * sc, f3.x * sc, f3.y * sc);
  }
  __syncthreads();
  // This CTA runs and its totals are cleared: the peers may add to them from now on.  Each CTA
  // waits for the others' arrival only when it is about to touch them, after its stream.
  cluster_arrive();
  ScoreFrag<KB> f[NG];
  if constexpr (MODE != 1) {
#pragma unroll
    for (int grp = 0; grp < NG; ++grp)
      load_score_b<KB>(f[grp], &s_qraw[0][0], s_chan, p.chunks, p.group, lane, grp * KB);
  }

  // ---- 1. scoring stream -> keys + first histogram ------------------------------------------
  if constexpr (MODE == 1) {
    // keys from the caller's score buffer, four consecutive tokens per thread
    const float* sin = p.scores + (int64_t)u * p.max_len;
    const bool vec_ok = ((reinterpret_cast<uintptr_t>(sin) & 15) == 0);
    for (int i = c0 + tid * 4; i < c1; i += kFT * 4) {
      float sv[4] = {0.f, 0.f, 0.f, 0.f};
      if (vec_ok && i + 3 < c1) {
        const float4 v4 = *reinterpret_cast<const float4*>(sin + i);
        sv[0] = v4.x; sv[1] = v4.y; sv[2] = v4.z; sv[3] = v4.w;
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if (i + e < c1) sv[e] = sin[i + e];
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        if (i + e < c1) {
          const uint32_t key = fasa_item_key(sv[e], i + e, len, p.n_sink, p.n_recent);
          atomicAdd(&hist0[key >> 21], 1u);
          keys[i + e - c0] = key;
        }
      }
    }
  } else {
    if (own_new) fetch(a, T, 0);                              // (the new row is in place now)
    locate(tp_next, T + step);
    // The loop exists twice.  When the head's dominant channels fill whole 16-channel blocks and
    // exactly the KB x NG blocks this kernel is compiled for (4 n_dom = 32 KB NG: 8, 16, 32 or 64
    // FCs), a tile's loads and products need no run-time test of the geometry: the loads of a batch
    // then leave back to back, which is worth a quarter of what one SM can pull on its own.
    auto stream = [&](auto exact_tag) {
      constexpr bool EXACT = decltype(exact_tag)::value;
      auto fetch_x = [&](uint4 (&aa)[TPI][KB], int TT, int grp) {
        if constexpr (EXACT) {
#pragma unroll
          for (int j = 0; j < TPI; ++j) {
            const unsigned char* tile;
            if constexpr (PAGED) tile = tp[j];
            else tile = unit + (int64_t)(TT + j) * (KB * NG * 512);
            const bool ok = (TT + j) * 16 < c1;
#pragma unroll
            for (int i = 0; i < KB; ++i)
              aa[j][i] = ok ? ld_proxy_u4(tile + (grp * KB + i) * 512 + lane * 16) : make_uint4(0u, 0u, 0u, 0u);
          }
        } else {
          fetch(aa, TT, grp);
        }
      };
      while (T * 16 < c1) {       // uniform over the warp
        float c[TPI][4];
#pragma unroll
        for (int j = 0; j < TPI; ++j) c[j][0] = c[j][1] = c[j][2] = c[j][3] = 0.f;
#pragma unroll
        for (int grp = 0; grp < NG; ++grp) {
#pragma unroll
          for (int j = 0; j < TPI; ++j) {
            if constexpr (EXACT) {
#pragma unroll
              for (int kb = 0; kb < KB; ++kb) mma_bf16_16816(c[j], a[j][kb], f[grp].b[kb]);
            } else {
              mma_tile<KB>(c[j], a[j], f[grp], n_blocks - grp * KB);
            }
          }
          // the registers are free again: the next group, or the next batch of tiles, at once
          if (grp + 1 < NG) {
            fetch_x(a, T, grp + 1);
          } else if ((T + step) * 16 < c1) {
            if constexpr (PAGED) {
#pragma unroll
              for (int j = 0; j < TPI; ++j) tp[j] = tp_next[j];
            }
            fetch_x(a, T + step, 0);
            locate(tp_next, T + 2 * step);
          }
        }
#pragma unroll
        for (int pr = 0; pr < TPI / 2; ++pr) {
          float a_lo, a_hi, b_lo, b_hi, sc;
          if (p.max_reduce) {     // uniform
            reduce_heads<true>(c[2 * pr], p.group, lane, a_lo, a_hi);
            reduce_heads<true>(c[2 * pr + 1], p.group, lane, b_lo, b_hi);
          } else {
            reduce_heads<false>(c[2 * pr], p.group, lane, a_lo, a_hi);
            reduce_heads<false>(c[2 * pr + 1], p.group, lane, b_lo, b_hi);
          }
          const int row = (T + 2 * pr) * 16 + pick_row_of_pair(lane, a_lo, a_hi, b_lo, b_hi, sc);
          if (row < c1) {
            const uint32_t key = fasa_item_key(sc, row, len, p.n_sink, p.n_recent);
            atomicAdd(&hist0[key >> 21], 1u);
            keys[row - c0] = key;
            if (srow) srow[row] = sc;
          }
        }
        T += step;
      }
    };
    if (pg.n8 == 0 && pg.n16 == KB * NG) stream(std::true_type{});
    else stream(std::false_type{});
  }
  __syncthreads();

  // ---- 2. radix select of the ktot-th largest key ------------------------------------------
  // Every value that steers this phase (the bin found, the keys still wanted from it, the
  // number of keys it holds) is computed by every warp of every CTA from the same cluster-wide
  // integer sums, hence identical everywhere: loops and barriers end for the whole cluster at
  // once.  `lower_gt` / `lower_eq` count, over the lower-ranked CTAs, the keys above the
  // threshold found so far and the keys equal to it: the compaction's cluster-wide prefix.
  cluster_wait();               // (set-up barrier, second half: every peer has started and cleared its totals)
  uint32_t prefix = 0, kth = ktot, thr = 0, tie_quota = 0, lower_gt = 0, lower_eq = 0;
  bool done = false;            // thr and tie_quota are final
  bool peers_idle = false;      // a barrier has passed since the last access to a peer's memory
  bool have_masks = false;      // s_mask already holds (higher bins, candidates) per block of 128 keys
  // Bit masks over the keys: word w covers keys 32 w .. 32 w + 31.  A warp owns a contiguous run
  // of words, a lane one word of every 32 of them: after the first pass over the keys all work
  // is per word, without ballots.
  const int n_words = (nloc + 31) >> 5;
  const int words_per_warp = (n_words + kFW - 1) / kFW;
  const int w0 = min(n_words, warp * words_per_warp), w1 = min(n_words, w0 + words_per_warp);
  uint32_t* s_mg = s_mask;                       // keys above the threshold (first: in higher bins)
  uint32_t* s_me = s_mask + (cap / 32 + 1);      // keys equal to it (first: the candidates)
#pragma unroll 1
  for (int pass = 0; pass < 3 && !done; ++pass) {
    const int bits = pass == 2 ? 10 : 11;
    const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
    const int nb = 1 << bits;
    const int ng = nb / 32;
    uint32_t* buf = (pass & 1) ? hist1 : hist0;
    if (pass > 0) {
      if (pass == 2) {          // (hist0: its remote readers of pass 0 are past the barrier of pass 1)
        for (int i = tid; i < nb; i += kFT) buf[i] = 0u;
        __syncthreads();
      }
#pragma unroll 4
      for (int i = tid * 4; i < nloc; i += kFT * 4) {
        const uint4 kq = *reinterpret_cast<const uint4*>(&keys[i]);
        const uint32_t kv[4] = {kq.x, kq.y, kq.z, kq.w};
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if (i + e < nloc && (kv[e] >> (shift + bits)) == prefix)
            atomicAdd(&buf[(kv[e] >> shift) & (uint32_t)(nb - 1)], 1u);
      }
      __syncthreads();
    }
    {
      // Group sums: each warp reduces its groups side by side; after a block barrier warp r
      // ADDS them into CTA r's totals (coalesced remote atomics, zeros skipped: scores crowd
      // into few groups), and into CTA r's totals of lower ranks if this CTA ranks below r.
      // After the cluster barrier every CTA holds the cluster-wide sums, already reduced.
      constexpr int GPW = kGroups / kFW;
      uint32_t v[GPW];
#pragma unroll
      for (int j = 0; j < GPW; ++j) {
        const int g = warp + j * kFW;
        v[j] = g < ng ? buf[g * 32 + lane] : 0u;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1)
#pragma unroll
        for (int j = 0; j < GPW; ++j) v[j] += __shfl_xor_sync(0xffffffffu, v[j], o);
      if (lane == 0) {
#pragma unroll
        for (int j = 0; j < GPW; ++j) s_mine[warp + j * kFW] = v[j];
      }
      __syncthreads();
      if (warp < cs) {
        uint32_t* tot = cluster.map_shared_rank(&s_gsum[pass][0][0], warp);
        uint32_t* low = cluster.map_shared_rank(&s_gsum[pass][1][0], warp);
#pragma unroll
        for (int j = 0; j < kGroups / 32; ++j) {
          const uint32_t x = s_mine[lane + 32 * j];
          if (x) {
            atomicAdd(tot + lane + 32 * j, x);
            if (crank < warp) atomicAdd(low + lane + 32 * j, x);
          }
        }
      }
    }
    cluster.sync();   // one per radix pass: all group sums have arrived, all histograms are complete

    // (a) every warp finds the group of 32 bins that holds the kth key from the local totals:
    // lane l owns groups 63 - 2 l and 62 - 2 l (highest first)
    uint32_t res, above_lower;                 // above_lower: keys of lower ranks in higher bins
    int group_id;
    {
      const uint2 t2 = *reinterpret_cast<const uint2*>(&s_gsum[pass][0][kGroups - 2 - 2 * lane]);   // (.y, .x) = (first, second)
      const uint2 l2 = *reinterpret_cast<const uint2*>(&s_gsum[pass][1][kGroups - 2 - 2 * lane]);
      int hit = 31;
      uint32_t tot = 0;
      res = 1;
      if (!warp_find_kth(t2.x + t2.y, kth, lane, &hit, &res, &tot)) { hit = 31; res = 1; }   // cannot fail: kth <= number of keys
      above_lower = __reduce_add_sync(0xffffffffu, lane < hit ? l2.x + l2.y : 0u);
      const uint32_t first = __shfl_sync(0xffffffffu, t2.y, hit), first_low = __shfl_sync(0xffffffffu, l2.y, hit);
      group_id = kGroups - 1 - 2 * hit;
      if (first < res) {
        res -= first;
        above_lower += first_low;
        --group_id;
      }
    }
    // (b) warp r fetches the 32 bins of that group from CTA r (one transaction) and adds them to
    // the block's totals; after a block barrier every warp locates the bin
    if (warp < cs) {
      const uint32_t x = cluster.map_shared_rank(buf, warp)[group_id * 32 + 31 - lane];   // lane 0 = highest bin
      if (x) {
        atomicAdd(&s_fine[pass][0][lane], x);
        if (warp < crank) atomicAdd(&s_fine[pass][1][lane], x);
      }
    }
    __syncthreads();
    uint32_t in_bin, bin_lower;                // keys in the bin: cluster-wide / in lower ranks
    {
      const uint32_t v = s_fine[pass][0][lane], vl = s_fine[pass][1][lane];
      int hit = 31;
      uint32_t tot = 0, res2 = 1;
      if (!warp_find_kth(v, res, lane, &hit, &res2, &tot)) { hit = 31; res2 = 1; }
      in_bin = __shfl_sync(0xffffffffu, v, hit);
      bin_lower = __shfl_sync(0xffffffffu, vl, hit);
      above_lower += __reduce_add_sync(0xffffffffu, lane < hit ? vl : 0u);
      prefix = (prefix << bits) | (uint32_t)(group_id * 32 + 31 - hit);
      kth = res2;
    }
    lower_gt += above_lower;
    peers_idle = false;

    if (in_bin == kth) {            // every key of this bin is selected: its other bits do not matter
      thr = prefix << shift;
      tie_quota = 0xffffffffu;
      lower_gt += bin_lower;
      done = true;
    } else if (pass == 2) {         // all 32 bits are fixed: the bin holds the keys equal to the threshold
      thr = prefix;
      tie_quota = kth;
      lower_eq = bin_lower;
      done = true;
    } else if (in_bin <= (uint32_t)kCandCap) {
      // ---- few keys share this prefix: every CTA gets all of them and finishes on its own ----
      // CTA r's keys occupy [sum of lower ranks' counts, + its own count) of every copy.
      uint32_t* cand = reinterpret_cast<uint32_t*>(smem_raw + (pass == 0 ? sl.hist1 : sl.spare));
      // One pass over the keys: masks of the keys in higher bins (selected for certain) and of
      // the keys in this bin (the candidates, decided once the threshold is known); then the
      // candidates themselves are appended, with one counter update per warp.
      have_masks = true;
      {
        uint32_t cnt = 0;
#pragma unroll 4
        for (int w = w0; w < w1; ++w) {
          const int i = 32 * w + lane;
          const uint32_t top = keys[i] >> shift;
          const uint32_t ma = __ballot_sync(0xffffffffu, i < nloc && top > prefix);
          const uint32_t mc = __ballot_sync(0xffffffffu, i < nloc && top == prefix);
          if (lane == 0) { s_mg[w] = ma; s_me[w] = mc; }
          cnt += __popc(mc);
        }
        uint32_t base = 0;
        if (lane == 0 && cnt) base = atomicAdd(&s_ncand, cnt);
        base = __shfl_sync(0xffffffffu, base, 0) + bin_lower;
        __syncwarp();
        for (int wb = w0; wb < w1; wb += 32) {     // uniform over the warp
          const int w = wb + lane;
          uint32_t m = w < w1 ? s_me[w] : 0u;
          const uint32_t c = __popc(m), incl = warp_incl_scan(c, lane);
          uint32_t slot = base + incl - c;
          base += __shfl_sync(0xffffffffu, incl, 31);
          while (m) {
            const int j = __ffs(m) - 1;
            m &= m - 1;
            if (slot < (uint32_t)kCandCap) cand[slot] = keys[32 * w + j];
            ++slot;
          }
        }
      }
      __syncthreads();
      if (warp < cs && warp != crank) {          // this CTA's run of keys, to CTA `warp`, coalesced
        const uint32_t n_own = min(s_ncand, (uint32_t)kCandCap - min(bin_lower, (uint32_t)kCandCap));
        uint32_t* dst = cluster.map_shared_rank(cand, warp) + bin_lower;
        for (uint32_t i = lane; i < n_own; i += 32) dst[i] = cand[bin_lower + i];
      }
      cluster.sync();   // every CTA holds every candidate; no peer is touched from here to the merge
      peers_idle = true;
      // block-level radix passes over the remaining `shift` bits, kFinBits at a time; every
      // warp scans the small histogram itself, so a pass costs one block barrier
      int rem = shift;
#pragma unroll 1
      for (int fp = 0; rem > 0 && !done; ++fp) {
        const int wbits = rem < kFinBits ? rem : kFinBits;
        const int sh = rem - wbits;
        uint32_t* fh = s_fin[fp];
        for (int i = tid; i < (int)in_bin; i += kFT) {
          const uint32_t key = cand[i];
          if ((key >> rem) == prefix) atomicAdd(&fh[(key >> sh) & (uint32_t)((1 << wbits) - 1)], 1u);
        }
        __syncthreads();
        // lane l owns the four bins 127 - 4 l .. 124 - 4 l (highest first)
        uint32_t c4[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) c4[j] = fh[kFinBins - 1 - 4 * lane - j];
        int hit = 0;
        uint32_t res2 = 1, tot = 0;
        if (!warp_find_kth(c4[0] + c4[1] + c4[2] + c4[3], kth, lane, &hit, &res2, &tot)) { hit = 0; res2 = 1; }
        uint32_t digit = 0, cnt = 0;
        bool found = false;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t c = __shfl_sync(0xffffffffu, c4[j], hit);
          if (!found) {
            if (c >= res2) { digit = (uint32_t)(kFinBins - 1 - 4 * hit - j); cnt = c; found = true; }
            else res2 -= c;
          }
        }
        prefix = (prefix << wbits) | digit;
        kth = res2;
        rem = sh;
        if (cnt == kth && rem > 0) {     // the rest of this bin is selected whole
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
      // pushed keys of the lower-ranked CTAs against the threshold (they lie in [0, bin_lower))
      {
        uint32_t ngt = 0, neq = 0;
        for (int i = tid; i < (int)bin_lower; i += kFT) {
          const uint32_t key = cand[i];
          ngt += key > thr ? 1u : 0u;
          neq += key == thr ? 1u : 0u;
        }
        ngt = __reduce_add_sync(0xffffffffu, ngt);
        neq = __reduce_add_sync(0xffffffffu, neq);
        if (lane == 0 && (ngt | neq)) { atomicAdd(&s_cgt, ngt); atomicAdd(&s_ceq, neq); }
      }
    }
  }
  // The attention phase reuses the histograms, and a CTA of the select-only forms may leave:
  // both only once no peer can still be reading this CTA's bins.
  if (!peers_idle) cluster.sync();

  // ---- 3. ascending compaction ---------------------------------------------------------------
  // (a) the masks of the keys above / equal to the threshold: from the keys (ballots), or,
  // where the select phase has left the masks of the higher bins and of the candidates, by
  // looking at the candidates alone, each lane at the bits of its own words; (b) the warps'
  // totals give each warp its offset (one block barrier); (c) every lane turns the set bits of
  // its words into positions of the index list (prefix over the lanes by shuffles).  Equal
  // keys are taken lowest index first, so the result equals a stable sort.
  {
    uint32_t g_tot = 0, e_tot = 0;
    if (have_masks) {
      for (int w = w0 + lane; w < w1; w += 32) {
        uint32_t mc = s_me[w], mg = s_mg[w], me = 0u;
        while (mc) {
          const int j = __ffs(mc) - 1;
          mc &= mc - 1;
          const uint32_t key = keys[32 * w + j];
          if (key > thr) mg |= 1u << j;
          else if (key == thr) me |= 1u << j;
        }
        s_mg[w] = mg;
        s_me[w] = me;
        g_tot += __popc(mg);
        e_tot += __popc(me);
      }
      g_tot = __reduce_add_sync(0xffffffffu, g_tot);
      e_tot = __reduce_add_sync(0xffffffffu, e_tot);
    } else {
#pragma unroll 4
      for (int w = w0; w < w1; ++w) {
        const int i = 32 * w + lane;
        const uint32_t key = keys[i];
        const uint32_t mg = __ballot_sync(0xffffffffu, i < nloc && key > thr);
        const uint32_t me = __ballot_sync(0xffffffffu, i < nloc && key == thr);
        if (lane == 0) { s_mg[w] = mg; s_me[w] = me; }
        g_tot += __popc(mg);
        e_tot += __popc(me);
      }
    }
    if (lane == 0) s_wcnt[warp] = ((unsigned long long)g_tot << 32) | e_tot;
  }
  __syncthreads();            // the warps' totals; the candidate counts of the select phase
  uint32_t g_run, e_run;        // selected keys before this warp's run: above / equal to the threshold
  {
    static_assert(kFW <= 32, "one lane per warp total");
    const unsigned long long mine = lane < kFW ? s_wcnt[lane] : 0ull;
    unsigned long long incl = mine;
#pragma unroll
    for (int o = 1; o < kFW; o <<= 1) {
      const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    const unsigned long long before = __shfl_sync(0xffffffffu, incl - mine, warp);
    const unsigned long long all = __shfl_sync(0xffffffffu, incl, kFW - 1);
    // selected tokens of the lower-ranked CTAs: from the bin counts and the pushed keys that
    // the select phase has seen, no barrier needed
    const uint32_t gb = lower_gt + s_cgt, eb = lower_eq + s_ceq;
    g_run = gb + (uint32_t)(before >> 32);
    e_run = eb + (uint32_t)before;
  }
  {
    int32_t* out_idx = p.idx + (int64_t)u * p.n_sel_max;
    for (int wb = w0; wb < w1; wb += 32) {         // uniform over the warp
      const int w = wb + lane;
      const uint32_t mg = w < w1 ? s_mg[w] : 0u, me = w < w1 ? s_me[w] : 0u;
      // counts of the lower lanes' words, packed (a word holds at most 32 keys, a CTA < 65536)
      const uint32_t cnt = (__popc(mg) << 16) | __popc(me), incl = warp_incl_scan(cnt, lane);
      uint32_t g_before = g_run + ((incl - cnt) >> 16), e_before = e_run + ((incl - cnt) & 0xffffu);
      const uint32_t all = __shfl_sync(0xffffffffu, incl, 31);
      g_run += all >> 16;
      e_run += all & 0xffffu;
      uint32_t m = mg | me;
      while (m) {
        const int j = __ffs(m) - 1;
        m &= m - 1;
        // (positions are < ktot by construction; the comparison keeps a write inside the
        // list whatever the scores hold)
        uint32_t pos = 0xffffffffu;
        if ((mg >> j) & 1u) { pos = g_before + min(e_before, tie_quota); ++g_before; }
        else { if (e_before < tie_quota) pos = g_before + e_before; ++e_before; }
        if (pos < ktot) out_idx[pos] = c0 + 32 * w + j;
      }
    }
    if (crank == 0 && tid == 0) p.n_sel[u] = (int32_t)ktot;
  }
  if constexpr (MODE != 0) return;   // (no peer reads this CTA's memory after the selection's last barrier)

  // ---- 4. attention over this CTA's share of the selected rows -----------------------------
  // Register-lean form (64 registers per thread): four query heads per pass (two passes for
  // groups of 5-8 heads; the second pass finds the rows in L2), four rows per warp step, a
  // lane owning 4 channels of every row.  The 16 partial logits (4 rows x 4 heads) of a step
  // are completed by a transposing xor-shuffle reduction, one shuffle per value.
  constexpr int R = 4;
  // The selected tokens are dealt out evenly: CTA r attends to rows [r, r + 1) * ktot / cs of the
  // index list, whoever selected them (scores cluster by position, so the CTAs' own selections
  // can differ several times in size); this costs one cluster barrier, after which the list
  // written by the peers is visible.
  cluster.sync();               // the index list is complete
  const int a0 = (int)(((long long)ktot * crank) / cs);
  const int a1 = (int)(((long long)ktot * (crank + 1)) / cs);
  // The attention phase's working arrays take over the key / histogram area: every read of
  // it, local or remote, happened before the selection's last barrier or the block barrier above.
  float* s_acc = reinterpret_cast<float*>(smem_raw + sl.acc);                        // [kFW][HP][128]
  float (*s_part)[kPartStride + 2] = reinterpret_cast<float (*)[kPartStride + 2]>(smem_raw + sl.part);
  float (*s_p)[16] = reinterpret_cast<float (*)[16]>(smem_raw + sl.p);
  float (*s_al)[HP] = reinterpret_cast<float (*)[HP]>(smem_raw + sl.al);
  float (*s_m)[HP] = reinterpret_cast<float (*)[HP]>(smem_raw + sl.m);
  float (*s_l)[HP] = reinterpret_cast<float (*)[HP]>(smem_raw + sl.l);
  const int n_hp = (p.group + HP - 1) / HP;
  for (int hp = 0; hp < n_hp; ++hp) {                          // uniform
    float2 acc[HP][2];
#pragma unroll
    for (int g = 0; g < HP; ++g) acc[g][0] = acc[g][1] = make_float2(0.f, 0.f);
    float m_run = -INFINITY, l_run = 0.f;   // of value (lane >> 1) = row * 4 + head
    const int32_t* irow = p.idx + (int64_t)u * p.n_sel_max;
    const uint16_t* kbase = p.k + b * p.ksb + h * p.ksh + lane * 4;
    const uint16_t* vbase = p.v + b * p.vsb + h * p.vsh + lane * 4;
    const int my_g = (lane >> 1) & 3;
    const int my_i = lane >> 3;
    for (int base = a0 + warp * R; base < a1; base += kFW * R) {
      // all row indices first, then all row loads: nothing waits on a previous row (rows
      // past the end repeat the last one and are masked below)
      int tok[R];
#pragma unroll
      for (int i = 0; i < R; ++i) tok[i] = __ldcg(irow + min(base + i, a1 - 1));
      uint2 kk[R], vv[R];
#pragma unroll
      for (int i = 0; i < R; ++i) {
        const int t = min(max(tok[i], 0), p.max_len - 1);
        if constexpr (PAGED) {
          kk[i] = ld_stream_u2(p.k + lane * 4 + cache_row(p.pm, b, h, t, p.ksb, p.ksh, p.kst, p.status));
          vv[i] = ld_stream_u2(p.v + lane * 4 + cache_row(p.pm, b, h, t, p.vsb, p.vsh, p.vst, p.status));
        } else {
          kk[i] = ld_stream_u2(kbase + (int64_t)t * p.kst);
          vv[i] = ld_stream_u2(vbase + (int64_t)t * p.vst);
        }
      }
      float part[16];
#pragma unroll
      for (int g = 0; g < HP; ++g) {
        const float4 qg = *reinterpret_cast<const float4*>(&s_q[hp * HP + g][lane * 4]);
#pragma unroll
        for (int i = 0; i < R; ++i) {
          const float2 k0 = bf16x2_to_f32x2(kk[i].x), k1 = bf16x2_to_f32x2(kk[i].y);
          part[i * HP + g] = qg.x * k0.x + qg.y * k0.y + qg.z * k1.x + qg.w * k1.y;
        }
      }
      // transposing reduction: lane L ends with the full sum of value L >> 1
      float logit;
      {
        float p8[8], p4[4], p2[2];
        const bool u16 = (lane & 16) != 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float send = u16 ? part[i] : part[i + 8];
          const float keep = u16 ? part[i + 8] : part[i];
          p8[i] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
        }
        const bool u8 = (lane & 8) != 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float send = u8 ? p8[i] : p8[i + 4];
          const float keep = u8 ? p8[i + 4] : p8[i];
          p4[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
        }
        const bool u4 = (lane & 4) != 0;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const float send = u4 ? p4[i] : p4[i + 2];
          const float keep = u4 ? p4[i + 2] : p4[i];
          p2[i] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
        }
        const bool u2 = (lane & 2) != 0;
        const float send = u2 ? p2[0] : p2[1];
        const float keep = u2 ? p2[1] : p2[0];
        logit = keep + __shfl_xor_sync(0xffffffffu, send, 2);
        logit += __shfl_xor_sync(0xffffffffu, logit, 1);
      }
      if (!(base + my_i < a1 && hp * HP + my_g < p.group)) logit = -INFINITY;
      float bmax = logit;                                      // over the 4 rows of this head
      bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 8));
      bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 16));
      const float m_new = fmaxf(m_run, bmax);
      const float m_safe = m_new == -INFINITY ? 0.f : m_new;
      const float alpha = exp2f(m_run - m_safe);
      const float pr = exp2f(logit - m_safe);
      l_run = l_run * alpha + pr;
      m_run = m_new;
      if ((lane & 1) == 0) {
        s_p[warp][lane >> 1] = pr;
        if (lane < 2 * HP) s_al[warp][lane >> 1] = alpha;      // row 0 lanes: one per head
      }
      __syncwarp();
#pragma unroll
      for (int g = 0; g < HP; ++g) {
        const float al = s_al[warp][g];
        const float2 a2 = make_float2(al, al);
        acc[g][0] = __ffma2_rn(acc[g][0], a2, make_float2(0.f, 0.f));
        acc[g][1] = __ffma2_rn(acc[g][1], a2, make_float2(0.f, 0.f));
      }
#pragma unroll
      for (int i = 0; i < R; ++i) {
        const float2 v0 = bf16x2_to_f32x2(vv[i].x), v1 = bf16x2_to_f32x2(vv[i].y);
        const float4 pi = *reinterpret_cast<const float4*>(&s_p[warp][i * HP]);
        const float pg4[4] = {pi.x, pi.y, pi.z, pi.w};
#pragma unroll
        for (int g = 0; g < HP; ++g) {
          const float2 p2 = make_float2(pg4[g], pg4[g]);
          acc[g][0] = __ffma2_rn(p2, v0, acc[g][0]);
          acc[g][1] = __ffma2_rn(p2, v1, acc[g][1]);
        }
      }
      __syncwarp();
    }
    // the four row lanes of a head add their partial sums of probabilities
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 8);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 16);

    // ---- 5a. combine the warps of this CTA for these heads ---------------------------------
    if (lane < 2 * HP && (lane & 1) == 0) {
      s_m[warp][lane >> 1] = m_run;
      s_l[warp][lane >> 1] = l_run;
    }
#pragma unroll
    for (int g = 0; g < HP; ++g)
      *reinterpret_cast<float4*>(&s_acc[((warp * HP) + g) * FASA_HEAD_DIM + lane * 4]) =
          make_float4(acc[g][0].x, acc[g][0].y, acc[g][1].x, acc[g][1].y);
    __syncthreads();
    for (int o = tid; o < HP * FASA_HEAD_DIM; o += kFT) {
      const int g = o / FASA_HEAD_DIM, c = o % FASA_HEAD_DIM;
      float mx = -INFINITY;
#pragma unroll
      for (int w = 0; w < kFW; ++w) mx = fmaxf(mx, s_m[w][g]);
      float av = 0.f, l = 0.f;
#pragma unroll
      for (int w = 0; w < kFW; ++w) {
        const float ms = s_m[w][g];
        const float wt = ms == -INFINITY ? 0.f : exp2f(ms - mx);
        av += wt * s_acc[((w * HP) + g) * FASA_HEAD_DIM + c];
        l += wt * s_l[w][g];
      }
      s_part[hp * HP + g][2 + c] = av;
      if (c == 0) {
        s_part[hp * HP + g][0] = mx;
        s_part[hp * HP + g][1] = l;
      }
    }
    __syncthreads();                                           // s_acc / s_m are reused by the next pass
  }
  // ---- 5b. merge across the cluster (one barrier; see fasa_cluster_merge.cuh) -------------------
  cluster_merge_store<kFT>(cluster, s_part, s_merge, p.group, su.q0, p.out, p.out_mirror, p.lse);
}

size_t fused_smem_bytes(int cap) { return (size_t)fused_smem_layout(cap).total; }

using FusedFn = void (*)(const FusedParams);

template <int MODE, bool PAGED>
FusedFn fused_variant(int chunks) {
  const int nb = (chunks + 1) / 2;      // 16-channel blocks per tile, the 8-channel one included
  if (nb <= 1) return fused_decode_kernel<1, 1, MODE, PAGED>;
  if (nb <= 2) return fused_decode_kernel<2, 1, MODE, PAGED>;
  if (nb <= 4) return fused_decode_kernel<4, 1, MODE, PAGED>;
  return fused_decode_kernel<4, 2, MODE, PAGED>;
}

FusedFn fused_fn(int chunks, bool paged = false) {
  return paged ? fused_variant<0, true>(chunks) : fused_variant<0, false>(chunks);
}

FusedFn topk_fn() { return fused_decode_kernel<1, 1, 1>; }

// The wide form of the step: 1024 threads, one CTA per SM.
template <int MODE, bool PAGED>
FusedFn wide_variant(int chunks) {
  const int nb = (chunks + 1) / 2;
  if (nb <= 1) return fused_decode_kernel<1, 1, MODE, PAGED, 1024>;
  if (nb <= 2) return fused_decode_kernel<2, 1, MODE, PAGED, 1024>;
  if (nb <= 4) return fused_decode_kernel<4, 1, MODE, PAGED, 1024>;
  return fused_decode_kernel<4, 2, MODE, PAGED, 1024>;
}
FusedFn wide_fn(int chunks, bool paged) { return paged ? wide_variant<0, true>(chunks) : wide_variant<0, false>(chunks); }
FusedFn wide_select_fn(int chunks, bool paged) { return paged ? wide_variant<2, true>(chunks) : wide_variant<2, false>(chunks); }
constexpr int kCapWide = 40960;        // keys a 1024-thread CTA can hold (one CTA per SM)

FusedFn select_fn(int chunks, bool paged = false) {         // the step without attention
  return paged ? fused_variant<2, true>(chunks) : fused_variant<2, false>(chunks);
}

}  // namespace

// Decides once per context whether and how the fused kernel runs: the smallest cluster whose
// CTAs can hold their slice of max_len keys, grown while that leaves SMs idle, then shrunk
// again if the device cannot co-schedule a cluster of that size.
int fasa_fused_plan(fasa_ctx* ctx) {
  const fasa_config_t& c = ctx->cfg;
  ctx->fused_cs = 0;
  ctx->fused_smem = 0;
  ctx->fused_step_ok = 1;
  const int units = c.batch * ctx->n_sets;
  const bool paged = c.page_size > 0;
  FusedFn fn = fused_fn(ctx->chunks, paged);
  auto cap_of = [&](int cs) { return (((c.max_len + cs - 1) / cs) + 31) & ~31; };
  // Two CTAs per SM can be resident; a cluster is doubled while the whole grid still fits
  // in one wave of them and every CTA keeps at least 512 tokens.
  const int slots = 2 * ctx->n_sm;
  int want = 1;
  while (want < 16 && cap_of(want) > kCapPair) want *= 2;
  while (want < 16 && units * want * 2 <= slots && c.max_len / (2 * want) >= 512) want *= 2;
  if (cudaFuncSetAttribute((const void*)fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
    cudaGetLastError();
    if (want > 8) want = 8;
  }
  for (int cs = want; cs >= 1; cs /= 2) {
    const int cap = cap_of(cs);
    if (cap > kCapMax) break;
    const size_t smem = fused_smem_bytes(cap);
    // The opt-in limit is a property of the kernel, shared by every context of the process:
    // it is set to the most any context can ask for, not to what this one needs.
    const int smem_limit = (int)fused_smem_bytes(kCapMax);
    if (cudaFuncSetAttribute((const void*)fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_limit) != cudaSuccess) {
      cudaGetLastError();
      continue;
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)cs, (unsigned)units, 1);
    cfg.blockDim = dim3(kFT, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cs;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n_clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&n_clusters, (const void*)fn, &cfg) != cudaSuccess || n_clusters < 1) {
      cudaGetLastError();
      continue;
    }
    // the select-only forms of the kernel run with the same cluster shape
    if (cudaFuncSetAttribute((const void*)topk_fn(), cudaFuncAttributeMaxDynamicSharedMemorySize, smem_limit) != cudaSuccess ||
        cudaFuncSetAttribute((const void*)select_fn(ctx->chunks, paged), cudaFuncAttributeMaxDynamicSharedMemorySize, smem_limit) != cudaSuccess ||
        (cs > 8 && (cudaFuncSetAttribute((const void*)topk_fn(), cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess ||
                    cudaFuncSetAttribute((const void*)select_fn(ctx->chunks, paged), cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess))) {
      cudaGetLastError();
      continue;
    }
    ctx->fused_cs = cs;
    ctx->fused_smem = smem;
    // The wide form.  When the 512-thread grid has more CTAs than SMs, SMs hold pairs of CTAs that
    // share their ~44 GB/s while lone CTAs (in a single wave: batch 8 x 8 heads at 64 K) end their
    // stream at 28 us against 50 us, and grids of several rounds run twice as many select chains.
    // Half as many CTAs of 1024 threads with twice the slice each sit alone on their SMs and
    // stream at the same rate: 74 -> 70 us there, 68 -> 57 us for batch 5, 210 -> 203 us for the
    // four-round grid of batch 16 at 64-128 K.
    ctx->step_threads = kFT;
    ctx->step_cs = cs;
    ctx->step_smem = smem;
    ctx->step_resident = n_clusters;
    const long long ctas = (long long)units * cs;
    // (not down to clusters of one CTA: batch 32 x 4 heads of 7 query heads at 16 K lost 3-6 % that way)
    if (cs >= 4 && ctas > ctx->n_sm && cap_of(cs / 2) <= kCapWide) {
      const int cs_w = cs / 2;
      const size_t smem_w = (size_t)fused_smem_layout(cap_of(cs_w), 32).total;
      const int limit_w = (int)fused_smem_layout(kCapWide, 32).total;
      FusedFn fw = wide_fn(ctx->chunks, paged), fs = wide_select_fn(ctx->chunks, paged);
      cudaLaunchConfig_t cw;
      memset(&cw, 0, sizeof(cw));
      cw.gridDim = dim3((unsigned)cs_w, (unsigned)units, 1);
      cw.blockDim = dim3(1024, 1, 1);
      cw.dynamicSmemBytes = smem_w;
      cudaLaunchAttribute aw[1];
      aw[0].id = cudaLaunchAttributeClusterDimension;
      aw[0].val.clusterDim.x = (unsigned)cs_w;
      aw[0].val.clusterDim.y = 1;
      aw[0].val.clusterDim.z = 1;
      cw.attrs = aw;
      cw.numAttrs = 1;
      int n_w = 0;
      if (cudaFuncSetAttribute((const void*)fw, cudaFuncAttributeMaxDynamicSharedMemorySize, limit_w) == cudaSuccess &&
          cudaFuncSetAttribute((const void*)fs, cudaFuncAttributeMaxDynamicSharedMemorySize, limit_w) == cudaSuccess &&
          cudaOccupancyMaxActiveClusters(&n_w, (const void*)fw, &cw) == cudaSuccess && n_w >= 1) {
        ctx->step_threads = 1024;
        ctx->step_cs = cs_w;
        ctx->step_smem = smem_w;
        ctx->step_resident = n_w;
      } else {
        cudaGetLastError();
      }
    }
    return cs;
  }
  return 0;
}

int32_t fasa_fused_launch(fasa_ctx* ctx, const void* q, const void* k_cache, const void* v_cache,
                          const void* proxy_k, const int32_t* seq_lens, int32_t budget,
                          int32_t n_sel_max, float* scores, int32_t* idx, int32_t* n_sel,
                          float* out, float* lse, const void* k_new, const void* v_new,
                          cudaStream_t stream, bool with_attention, float* out_mirror) {
  const fasa_config_t& c = ctx->cfg;
  FusedParams p;
  p.out_mirror = out_mirror;
  p.q = (const uint16_t*)q; p.k = (const uint16_t*)k_cache; p.v = (const uint16_t*)v_cache;
  p.proxy = (const unsigned char*)proxy_k; p.seq_lens = seq_lens; p.chan = ctx->d_chan;
  p.k_new = (const uint16_t*)k_new; p.v_new = (const uint16_t*)v_new;
  p.k_w = (uint16_t*)k_cache; p.v_w = (uint16_t*)v_cache; p.proxy_w = (unsigned char*)proxy_k;
  p.seq_lens_w = (int32_t*)seq_lens; p.arrive = ctx->d_arrive;
  p.shift_clusters = 0; p.shift_ctas = 0;
  p.scores = scores; p.idx = idx; p.n_sel = n_sel; p.out = out; p.lse = lse; p.status = ctx->d_status;
  p.n_q_heads = c.n_q_heads; p.n_kv_heads = c.n_kv_heads; p.n_sets = ctx->n_sets; p.group = ctx->sel_heads; p.max_len = c.max_len;
  p.chunks = ctx->chunks; p.n_sink = c.n_sink; p.n_recent = c.n_recent; p.budget = budget;
  p.n_sel_max = n_sel_max;
  p.max_reduce = c.group_reduce;
  p.q_len = 1;
  p.ksb = c.k_stride_b; p.ksh = c.k_stride_h; p.kst = c.k_stride_t;
  p.vsb = c.v_stride_b; p.vsh = c.v_stride_h; p.vst = c.v_stride_t;
  p.scale_log2 = c.softmax_scale * 1.4426950408889634f;
  p.pm = fasa_page_map(ctx);
  if (!fasa_pages_ready(ctx)) return FASA_ERR_INVALID_ARG;
  const bool paged = c.page_size > 0;
  FusedFn fn = with_attention ? fused_fn(ctx->chunks, paged) : select_fn(ctx->chunks, paged);
  // (the step's own shape: 512 threads and the context's cluster size, or the wide form)
  const bool wide = ctx->step_threads == 1024;
  if (wide) fn = with_attention ? wide_fn(ctx->chunks, paged) : wide_select_fn(ctx->chunks, paged);
  const int threads = wide ? 1024 : kFT, cs_l = wide ? ctx->step_cs : ctx->fused_cs;
  const size_t smem_l = wide ? ctx->step_smem : ctx->fused_smem;

  // (from one and a half rounds of CTAs on: see the kernel)
  if (ctx->step_resident > 0 && 2ll * c.batch * ctx->n_sets >= 3ll * ctx->step_resident) {
    p.shift_clusters = ctx->step_resident;
    p.shift_ctas = ctx->step_resident * cs_l;
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)cs_l, (unsigned)(c.batch * ctx->n_sets), 1);
  cfg.blockDim = dim3((unsigned)threads, 1, 1);
  cfg.dynamicSmemBytes = smem_l;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)cs_l;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, fn, p);
  ctx->launches += 1;
  FASA_CUDA_TRY(ctx, e);
  return FASA_OK;
}

// TopK-I alone with the cluster kernel's selection phases (fasa_topk).
int32_t fasa_fused_topk_launch(fasa_ctx* ctx, const float* scores, const int32_t* seq_lens,
                               int32_t budget, int32_t n_sel_max, int32_t* idx, int32_t* n_sel,
                               cudaStream_t stream) {
  return fasa_fused_topk_rows(ctx, scores, seq_lens, budget, n_sel_max, idx, n_sel, ctx->n_sets,
                              ctx->cfg.n_sink, ctx->cfg.n_recent, stream);
}

// TopK-I over rows_per_seq score rows per sequence (row r of the buffer belongs to sequence
// r / rows_per_seq), with the given forced positions instead of the context's.
int32_t fasa_fused_topk_rows(fasa_ctx* ctx, const float* scores, const int32_t* seq_lens,
                             int32_t budget, int32_t n_sel_max, int32_t* idx, int32_t* n_sel,
                             int rows_per_seq, int n_sink, int n_recent, cudaStream_t stream, int q_len) {
  const fasa_config_t& c = ctx->cfg;
  // Many long rows (batch 16 at 64-128 K, blocks of queries, calibration): clusters would run in
  // rounds, each paying the whole chain of cluster barriers; one CTA per row is faster there (128 rows
  // of 64-128 K: 64 -> 53 us; calibration of 512 samples at 64-128 K: 18.5 -> 11.6 ms; eight queries
  // per sequence at batch 8, 64 K: 133 -> 105 us).  For few rows and for short ones the cluster form
  // wins (64 rows of 64 K: 21 against 31 us; 8 rows of 32 K: 16 against 23 us; 2080 rows of 32 K: 387
  // against 420 us).
  if (fasa_topk_row_ok(ctx) &&
      (((long long)c.batch * rows_per_seq >= ctx->n_sm * 3 / 4 && c.max_len >= 65536) || ctx->topk_rows))
    return fasa_topk_row_launch(ctx, scores, seq_lens, budget, n_sel_max, idx, n_sel, rows_per_seq, n_sink, n_recent, stream, q_len);
  FusedParams p;
  memset(&p, 0, sizeof(p));
  p.seq_lens = seq_lens; p.scores = const_cast<float*>(scores); p.idx = idx; p.n_sel = n_sel;
  p.status = ctx->d_status;
  // (the select-only form uses the unit index for its score row and its sequence alone)
  p.n_q_heads = rows_per_seq; p.n_kv_heads = 1; p.n_sets = rows_per_seq; p.group = 1; p.max_len = c.max_len;
  p.chunks = ctx->chunks; p.n_sink = n_sink; p.n_recent = n_recent; p.budget = budget;
  p.n_sel_max = n_sel_max;
  p.q_len = q_len;
  // The context's cluster size suits its own number of rows (few rows: wide clusters, so the
  // whole GPU works on them).  A launch with many more rows takes the narrowest cluster that
  // holds a row's keys: more rows are then resident at once.
  int cs = ctx->fused_cs;
  auto cap_of = [&](int n) { return (((c.max_len + n - 1) / n) + 31) & ~31; };
  if (rows_per_seq > ctx->n_sets) {
    cs = 1;
    while (cs < ctx->fused_cs && cap_of(cs) > kCapPair) cs *= 2;
  }
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)cs, (unsigned)(c.batch * rows_per_seq), 1);
  cfg.blockDim = dim3(kFT, 1, 1);
  cfg.dynamicSmemBytes = cs == ctx->fused_cs ? ctx->fused_smem : fused_smem_bytes(cap_of(cs));
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)cs;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, topk_fn(), p);
  ctx->launches += 1;
  FASA_CUDA_TRY(ctx, e);
  return FASA_OK;
}
