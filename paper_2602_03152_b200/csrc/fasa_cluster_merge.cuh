// Merge of split-K attention partials inside one thread-block cluster (the second half of
// flash decoding: m* = max_s m_s, out = sum_s 2^(m_s - m*) acc_s / sum_s 2^(m_s - m*) l_s),
// shared by the one-launch decode step and by the split-K attention kernel.
//
// CTA r of the cluster finishes outputs [r * per_o, (r + 1) * per_o) of the unit's
// group * 128 outputs.  Every CTA PUSHES its partial values for those outputs into r's shared
// memory (consecutive threads write consecutive words of one peer, so the distributed-shared-
// memory traffic is a few wide transactions); after ONE cluster barrier r combines from local
// memory only: no CTA reads a peer afterwards, so none has to wait for the others to leave.
#pragma once

#include <cooperative_groups.h>

#include "fasa_common.cuh"

constexpr int kMergePartStride = FASA_HEAD_DIM + 4;   // a head's partial in shared memory: m, l, acc[128], padding
constexpr int kMergeMaxCs = 16;                        // CTAs per cluster at most

// What the peers write into: must not share memory with anything the owning CTA still uses
// when the first peer finishes its part.
struct ClusterMergeSmem {
  float racc[FASA_MAX_GROUP * FASA_HEAD_DIM + kMergeMaxCs];   // [rank][per_o]: accumulators of this CTA's outputs
  float rml[kMergeMaxCs][FASA_MAX_GROUP][2];                 // every CTA's (m, l) per head
};

// part[g] = (m, l, acc[128]) of head g of this CTA, base-2 logit domain, complete and visible to
// the whole block.  NT threads call this together, in every CTA of the cluster (the cluster
// size must be a power of two <= 16).  out / lse rows start at query head q0; out_mirror and
// lse may be null.
template <int NT>
__device__ __forceinline__ void cluster_merge_store(cooperative_groups::cluster_group& cluster,
                                                    const float (*part)[kMergePartStride], ClusterMergeSmem& sm,
                                                    int group, int64_t q0, float* out, float* out_mirror, float* lse) {
  const int cs = (int)cluster.num_blocks();
  const int crank = (int)cluster.block_rank();
  const int tid = threadIdx.x;
  constexpr int GP = FASA_MAX_GROUP;
  const int n_out = group * FASA_HEAD_DIM;
  const int per_o = (n_out + cs - 1) / cs;
  for (int o = tid; o < n_out; o += NT) {
    const int r = o / per_o, ol = o % per_o;
    float* dst = cluster.map_shared_rank(&sm.racc[0], r);
    dst[crank * per_o + ol] = part[o / FASA_HEAD_DIM][2 + o % FASA_HEAD_DIM];
  }
  for (int i = tid; i < cs * GP; i += NT) {
    const int r = i / GP, g = i % GP;
    float* dst = cluster.map_shared_rank(&sm.rml[0][0][0], r);
    dst[(crank * GP + g) * 2 + 0] = part[g][0];
    dst[(crank * GP + g) * 2 + 1] = part[g][1];
  }
  cluster.sync();   // the merge barrier: every CTA's partial results have arrived
  const int opp = NT / cs;                   // outputs per pass
  const int r = tid % cs, tl = tid / cs;
  for (int t0 = 0; t0 < per_o; t0 += opp) {  // uniform trip count
    const int t = t0 + tl;
    const int o = crank * per_o + t;
    const bool ok = t < per_o && o < n_out;
    const int g = ok ? o / FASA_HEAD_DIM : 0;
    const float ms = sm.rml[r][g][0], ls = sm.rml[r][g][1];
    const float as = ok ? sm.racc[r * per_o + t] : 0.f;
    float mx = ms;
    for (int off = cs >> 1; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
    const float wt = ms == -INFINITY ? 0.f : exp2f(ms - mx);
    float av = wt * as, l = wt * ls;
    for (int off = cs >> 1; off > 0; off >>= 1) {
      av += __shfl_xor_sync(0xffffffffu, av, off);
      l += __shfl_xor_sync(0xffffffffu, l, off);
    }
    if (ok && r == 0) {
      const int c = o % FASA_HEAD_DIM;
      const int64_t hq = q0 + g;
      const float ov = l > 0.f ? av / l : 0.f;
      out[hq * FASA_HEAD_DIM + c] = ov;
      if (out_mirror) out_mirror[hq * FASA_HEAD_DIM + c] = ov;
      if (lse && c == 0) lse[hq] = l > 0.f ? (mx + log2f(l)) * 0.6931471805599453f : -INFINITY;
    }
  }
}
