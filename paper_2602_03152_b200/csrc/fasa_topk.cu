// TopK-I (Sec. 4.1): per (batch, KV head) the `budget` best-scoring positions plus the
// forced sink / recent positions, written in ascending order.
//
// One thread-block cluster per unit.  Each CTA of the cluster owns a contiguous slice of
// the unit's scores and loads it ONCE into registers as order-preserving 32-bit keys.
// The k-th largest key is found by an MSB-first radix select (11 + 11 + 10 bits): every
// CTA histograms its slice in shared memory, the cluster adds the histograms through
// distributed shared memory, and every CTA locates the threshold bin redundantly, so
// one cluster barrier per pass suffices.  A final pass writes the indices with a prefix
// sum over (key > T, key == T) counts: equal keys are taken lowest index first, which
// makes the result deterministic and identical to a stable sort.
#include <cooperative_groups.h>

#include "fasa_common.cuh"
#include "fasa_score_core.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int kTopkThreads = 1024;
constexpr int kTopkItems = 16;                         // keys a thread can hold
constexpr int kTopkCtaCap = kTopkThreads * kTopkItems;  // 16384 scores per CTA in registers
constexpr int kMaxBins = 2048;

// Block-wide inclusive scan of a 64-bit value (1024 threads).
__device__ __forceinline__ unsigned long long block_scan_incl(unsigned long long v,
                                                              unsigned long long* warp_tot) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    unsigned long long t = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += t;
  }
  __syncthreads();  // a previous scan may still be reading warp_tot
  if (lane == 31) warp_tot[warp] = v;
  __syncthreads();
  if (warp == 0) {
    unsigned long long w = warp_tot[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      unsigned long long t = __shfl_up_sync(0xffffffffu, w, o);
      if (lane >= o) w += t;
    }
    warp_tot[lane] = w;
  }
  __syncthreads();
  if (warp > 0) v += warp_tot[warp - 1];
  return v;
}

template <bool CACHED>
__global__ void __launch_bounds__(kTopkThreads, 1)
topk_kernel(const float* __restrict__ scores, const int32_t* __restrict__ seq_lens, int budget,
            int n_sel_max, int32_t* __restrict__ idx, int32_t* __restrict__ n_sel,
            int32_t* __restrict__ status, int n_sets, int max_len, int n_sink, int n_recent) {
  cg::cluster_group cluster = cg::this_cluster();
  const int cs = (int)cluster.num_blocks();
  const int crank = (int)cluster.block_rank();
  const int tid = threadIdx.x;
  const int u = blockIdx.y;
  const int b = u / n_sets;
  const int len = clamp_len(seq_lens[b], max_len, status);

  // Selection size: forced positions come on top of the budget.
  const long long k_budget = budget > 0 ? (long long)budget : ((long long)(-budget) * len + 999) / 1000;
  const int sink = min(len, n_sink);
  const int n_forced = sink + min(n_recent, len - sink);
  long long ktot_ll = min((long long)len, (long long)n_forced + k_budget);
  if (ktot_ll > n_sel_max) {
    ktot_ll = n_sel_max;
    if (crank == 0 && tid == 0) atomicOr(status, FASA_DEV_NSEL_CLAMPED);
  }
  const uint32_t ktot = (uint32_t)ktot_ll;
  if (ktot == 0) {  // uniform over the cluster
    if (crank == 0 && tid == 0) n_sel[u] = 0;
    return;
  }

  __shared__ uint32_t hist[2][kMaxBins];
  __shared__ unsigned long long s_warp[32];
  __shared__ unsigned long long s_tot;
  __shared__ uint32_t s_bin, s_kth, s_cnt;

  // Slice of this CTA and of this thread (contiguous, in index order).
  const int per = ((len + cs - 1) / cs + 3) & ~3;
  const int c0 = min(len, crank * per);
  const int c1 = min(len, c0 + per);
  const int ipt = ((per + kTopkThreads - 1) / kTopkThreads + 3) & ~3;
  const int j0 = c0 + tid * ipt;
  const float* srow = scores + (int64_t)u * max_len;

  uint32_t keys[kTopkItems];
  uint32_t vmask = 0;
  if (CACHED) {
    const bool vec_ok = (((uintptr_t)srow) & 15) == 0;
#pragma unroll
    for (int i = 0; i < kTopkItems; i += 4) {
      float s[4] = {0.f, 0.f, 0.f, 0.f};
      const int j = j0 + i;
      if (i < ipt && j < c1) {
        if (vec_ok && j + 3 < c1) {
          float4 v = *reinterpret_cast<const float4*>(srow + j);
          s[0] = v.x; s[1] = v.y; s[2] = v.z; s[3] = v.w;
        } else {
#pragma unroll
          for (int e = 0; e < 4; ++e)
            if (j + e < c1) s[e] = srow[j + e];
        }
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const bool ok = (i < ipt) && (j + e < c1);
        keys[i + e] = ok ? fasa_item_key(s[e], j + e, len, n_sink, n_recent) : 0u;
        vmask |= ok ? (1u << (i + e)) : 0u;
      }
    }
  }

  // Applies f(key, j) to this thread's items in index order.
  auto for_items = [&](auto&& f) {
    if (CACHED) {
#pragma unroll
      for (int i = 0; i < kTopkItems; ++i)
        if ((vmask >> i) & 1u) f(keys[i], j0 + i);
    } else {
      for (int i = 0; i < ipt; ++i) {
        const int j = j0 + i;
        if (j < c1) f(fasa_item_key(srow[j], j, len, n_sink, n_recent), j);
      }
    }
  };

  // ---- radix select of the ktot-th largest key --------------------------------------
  uint32_t prefix = 0, kth = ktot, thr = 0, tie_quota = 0;
  bool done = false;
#pragma unroll 1
  for (int pass = 0; pass < 3 && !done; ++pass) {
    const int bits = pass == 2 ? 10 : 11;
    const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
    const int nb = 1 << bits;
    uint32_t* buf = hist[pass & 1];
    for (int i = tid; i < nb; i += kTopkThreads) buf[i] = 0;
    __syncthreads();
    for_items([&](uint32_t key, int) {
      if (pass == 0 || (key >> (shift + bits)) == prefix)
        atomicAdd(&buf[(key >> shift) & (uint32_t)(nb - 1)], 1u);
    });
    cluster.sync();

    // Cluster-wide counts of two adjacent bins per thread, walking down from the top bin.
    const int rb0 = 2 * tid, rb1 = 2 * tid + 1;
    uint32_t n0 = 0, n1 = 0;
    if (rb0 < nb) {
      for (int r = 0; r < cs; ++r) {
        const uint32_t* rbuf = cluster.map_shared_rank(buf, r);
        n0 += rbuf[nb - 1 - rb0];
        n1 += rbuf[nb - 1 - rb1];
      }
    }
    const uint32_t incl = (uint32_t)block_scan_incl((unsigned long long)(n0 + n1), s_warp);
    const uint32_t excl = incl - n0 - n1;
    if (excl < kth && kth <= excl + n0) {
      s_bin = (uint32_t)(nb - 1 - rb0); s_kth = kth - excl; s_cnt = n0;
    } else if (excl + n0 < kth && kth <= excl + n0 + n1) {
      s_bin = (uint32_t)(nb - 1 - rb1); s_kth = kth - excl - n0; s_cnt = n1;
    }
    __syncthreads();
    prefix = (prefix << bits) | s_bin;
    kth = s_kth;
    if (s_cnt == kth) {          // the whole bin is needed: no finer pass required
      thr = prefix << shift;
      tie_quota = 0xffffffffu;
      done = true;
    }
    __syncthreads();             // s_bin / s_kth / s_cnt are rewritten by the next pass
  }
  if (!done) { thr = prefix; tie_quota = kth; }

  // ---- ascending-index compaction ----------------------------------------------------
  uint32_t n_gt = 0, n_eq = 0;
  for_items([&](uint32_t key, int) {
    n_gt += key > thr;
    n_eq += key == thr;
  });
  const unsigned long long mine = ((unsigned long long)n_gt << 32) | n_eq;
  const unsigned long long incl64 = block_scan_incl(mine, s_warp);
  if (tid == kTopkThreads - 1) s_tot = incl64;
  cluster.sync();
  unsigned long long before = incl64 - mine;
  for (int r = 0; r < crank; ++r) before += *cluster.map_shared_rank(&s_tot, r);
  uint32_t g_run = (uint32_t)(before >> 32), e_run = (uint32_t)before;
  int32_t* out = idx + (int64_t)u * n_sel_max;
  for_items([&](uint32_t key, int j) {
    if (key > thr) {
      out[g_run + min(e_run, tie_quota)] = j;
      ++g_run;
    } else if (key == thr) {
      if (e_run < tie_quota) out[g_run + e_run] = j;
      ++e_run;
    }
  });
  if (crank == 0 && tid == 0) n_sel[u] = (int32_t)ktot;
  cluster.sync();  // no CTA may leave while a peer can still read its shared memory
}

}  // namespace

extern "C" int32_t fasa_topk(fasa_ctx_t* ctx, const float* scores, const int32_t* seq_lens,
                             int32_t budget, int32_t n_sel_max, int32_t* idx, int32_t* n_sel,
                             void* workspace, void* stream) {
  (void)workspace;  // the selection keeps its state in registers and shared memory
  if (!ctx || !scores || !seq_lens || !idx || !n_sel || budget == 0 || n_sel_max <= 0)
    return FASA_ERR_INVALID_ARG;
  if (budget < -1000) return FASA_ERR_INVALID_ARG;
  const fasa_config_t& c = ctx->cfg;
  const int units = c.batch * ctx->n_sets;
  // The cluster kernel's selection phases (keys in shared memory, one barrier per radix pass,
  // mask compaction) serve wherever a cluster shape exists for this context; the
  // register-resident kernel below remains for the rest (max_len beyond 16 x 22528).
  if (ctx->use_fused && ctx->fused_cs > 0)
    return fasa_fused_topk_launch(ctx, scores, seq_lens, budget, n_sel_max, idx, n_sel, (cudaStream_t)stream);

  // Cluster size: enough CTAs to hold max_len scores in registers, more when few units
  // would leave SMs idle (down to 2048 scores per CTA).
  int cs = 1;
  while (cs < 8 && (long long)cs * kTopkCtaCap < c.max_len) cs *= 2;
  while (cs < 8 && units * cs < ctx->n_sm && c.max_len / (cs * 2) >= 2048) cs *= 2;
  const bool cached = (long long)cs * kTopkCtaCap >= c.max_len;

  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)cs, (unsigned)units, 1);
  cfg.blockDim = dim3(kTopkThreads, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = (cudaStream_t)stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)cs;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e;
  if (cached)
    e = cudaLaunchKernelEx(&cfg, topk_kernel<true>, scores, seq_lens, (int)budget, (int)n_sel_max,
                           idx, n_sel, ctx->d_status, (int)ctx->n_sets, (int)c.max_len,
                           (int)c.n_sink, (int)c.n_recent);
  else
    e = cudaLaunchKernelEx(&cfg, topk_kernel<false>, scores, seq_lens, (int)budget, (int)n_sel_max,
                           idx, n_sel, ctx->d_status, (int)ctx->n_sets, (int)c.max_len,
                           (int)c.n_sink, (int)c.n_recent);
  ctx->launches += 1;
  FASA_CUDA_TRY(ctx, e);
  return FASA_OK;
}
