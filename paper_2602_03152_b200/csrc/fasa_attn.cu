// FAC (Sec. 4.2, Eq. 6-7) and the dense FKV path (Sec. 5.1): split-K flash decoding with an
// online softmax, rows gathered by index for the sparse form, followed by a merge pass.
//
// Two kernels compute the partial results of a split.
//   decode_attn_mma_kernel (the default): the GQA group (<= 8 query heads) is the N = 8 of
//     mma.m16n8k16, so both products of the step run on tensor cores; described above the
//     kernel.
//   decode_attn_kernel (step mode 0, the first version): a KV row (128 bf16 = 256 bytes) is
//     read by a half-warp, 16 bytes per lane; a lane owns 8 channels of every row it sees and
//     keeps, for up to 4 query heads of the group, its slice of q and of the output
//     accumulator in registers, so one K/V row serves the whole group from a single load.
//     Groups of 5-8 heads use both half-warps of a warp on the same row (the second load is
//     merged by the coalescer).  Logits of a batch of 8 rows are completed with a transposing
//     xor-shuffle reduction (8 shuffles per head per batch); probabilities travel back to all
//     lanes through shared memory.  All multiply-adds are packed two-wide fp32 FMAs.
// decode_attn_merge_kernel then combines the splits of every (sequence, query head).  Where a
// unit needs at most 8 splits (selections up to 16384 rows), the splits of a unit form one
// thread-block cluster instead and merge through distributed shared memory inside the same
// launch: no partial result touches HBM, no second launch, no workspace.
#include <mutex>

#include "fasa_cluster_merge.cuh"
#include "fasa_common.cuh"
#include "fasa_score_core.cuh"

namespace cg = cooperative_groups;

namespace {

// Split-K partials of fasa_sparse_decode_attn_static: lives in the library image, so every
// GPU that loads the library holds these bytes until the process exits.
constexpr size_t kStaticScratchBytes = FASA_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kAttnThreads = 128;
constexpr int kAttnHalfWarps = kAttnThreads / 16;  // 8
constexpr int kRB = 8;                              // rows per half-warp batch
constexpr int kPartialStride = FASA_HEAD_DIM + 2;   // m, l, acc[128] (base-2 domain)

struct AttnParams {
  const uint16_t* q;
  const uint16_t* k;
  const uint16_t* v;
  const int32_t* idx;      // sparse: [units][n_sel_max]
  const int32_t* n_rows;   // sparse: n_sel [units]; dense: seq_lens [batch]
  float* partial;          // [batch][n_q_heads][n_splits][kPartialStride]
  float* out;              // (cluster form: merged in the same launch)
  float* out_mirror;       // (cluster form, nullable: a second copy of out, e.g. mapped host memory)
  float* lse;
  int32_t* status;
  int n_q_heads, n_kv_heads, n_sets, group, max_len, n_sel_max, n_cap, chunk, n_splits;   // a unit = `group` query heads; n_sets units per sequence
  int64_t ksb, ksh, kst, vsb, vsh, vst;
  PageMap pm;              // paged caches (all zero: contiguous)
  float scale_log2;        // softmax_scale * log2(e)
  fasa_ksplit ks;          // split key cache (KSPLIT kernels): k holds the non-dominant channels only
  int q_len;               // blocks of queries (tensor-core kernel, sparse form): a "sequence" of the grid is a
                           // (sequence, query) pair and reads the cache of sequence b / q_len; 1 otherwise
};

// GP: heads per half-warp (1..4).  HWS: half-warps sharing a row (1: group <= 4, 2: group <= 8).
template <int GP, int HWS, bool SPARSE>
__global__ void __launch_bounds__(kAttnThreads)
decode_attn_kernel(const AttnParams p) {
  const int u = blockIdx.y;
  const SelUnit su = sel_unit(u, p.n_sets, p.group, p.n_q_heads, p.n_kv_heads);
  const int h = su.h;
  const int b = su.b;
  int n;
  if (SPARSE) {
    n = p.n_rows[u];
    if (n < 0 || n > p.n_cap) {
      atomicOr(p.status, FASA_DEV_NSEL_CLAMPED);
      n = n < 0 ? 0 : p.n_cap;
    }
  } else {
    n = clamp_len(p.n_rows[b], p.max_len, p.status);
  }
  const int split = blockIdx.x;
  const int r0 = split * p.chunk;
  if (r0 >= n) return;
  const int r1 = min(n, r0 + p.chunk);

  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int l16 = lane & 15;
  const int hw = lane >> 4;
  const int hwid = warp * 2 + hw;                          // half-warp within the CTA
  constexpr int kSlots = kAttnHalfWarps / HWS;             // row-batch streams per CTA
  constexpr int kWarpRows = kRB * (2 / HWS);               // rows one warp covers per iteration
  const int g0 = HWS == 1 ? 0 : hw * GP;                   // first head (within the group) of this half-warp

  __shared__ __align__(16) float s_p[kAttnHalfWarps][kRB][4];
  __shared__ __align__(16) float s_acc[kAttnHalfWarps][GP][FASA_HEAD_DIM];
  __shared__ float s_m[kAttnHalfWarps][GP];
  __shared__ float s_l[kAttnHalfWarps][GP];

  // q slice of this lane, pre-multiplied by scale * log2(e): logits live in the base-2 domain.
  float2 qf[GP][4];
#pragma unroll
  for (int g = 0; g < GP; ++g) {
    const bool head_ok = g0 + g < p.group;
    const uint16_t* qp =
        p.q + (su.q0 + (head_ok ? g0 + g : 0)) * FASA_HEAD_DIM + l16 * 8;
    uint4 w = *reinterpret_cast<const uint4*>(qp);
    const float sc = head_ok ? p.scale_log2 : 0.f;
    float2 t;
    t = bf16x2_to_f32x2(w.x); qf[g][0] = make_float2(t.x * sc, t.y * sc);
    t = bf16x2_to_f32x2(w.y); qf[g][1] = make_float2(t.x * sc, t.y * sc);
    t = bf16x2_to_f32x2(w.z); qf[g][2] = make_float2(t.x * sc, t.y * sc);
    t = bf16x2_to_f32x2(w.w); qf[g][3] = make_float2(t.x * sc, t.y * sc);
  }

  float2 acc[GP][4];
  float m[GP], lsum[GP];
#pragma unroll
  for (int g = 0; g < GP; ++g) {
    m[g] = -INFINITY;
    lsum[g] = 0.f;
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[g][e] = make_float2(0.f, 0.f);
  }

  const uint16_t* kbase = p.k + l16 * 8;
  const uint16_t* vbase = p.v + l16 * 8;
  const int32_t* irow = SPARSE ? p.idx + (int64_t)u * p.n_sel_max : nullptr;
  // The row of the batch whose finished logit lands in this lane after the reduction.
  const int my_row = ((l16 >> 3) & 1) * 4 + ((l16 >> 2) & 1) * 2 + ((l16 >> 1) & 1);

  // The trip count is the same for both half-warps of a warp (the shuffles below name all
  // 32 lanes); a half-warp whose batch starts past r1 runs it fully masked.
  for (int wbase = r0 + warp * kWarpRows; wbase < r1; wbase += (kAttnThreads / 32) * kWarpRows) {
    const int base = wbase + (HWS == 1 ? hw * kRB : 0);
    // all row indices first, then all row loads, so that no load waits on a previous row
    int tok[kRB];
#pragma unroll
    for (int i = 0; i < kRB; ++i) {
      const int r = base + i;
      tok[i] = SPARSE ? (r < r1 ? __ldg(irow + r) : 0) : r;
    }
    uint4 kk[kRB], vv[kRB];
#pragma unroll
    for (int i = 0; i < kRB; ++i) {
      const int r = base + i;
      if (r < r1) {
        int t = tok[i];
        if (SPARSE && (t < 0 || t >= p.max_len)) {
          atomicOr(p.status, FASA_DEV_IDX_CLAMPED);
          t = 0;
        }
        if (p.pm.table != nullptr) {
          kk[i] = ld_stream_u4(kbase + cache_row(p.pm, b, h, t, p.ksb, p.ksh, p.kst, p.status));
          vv[i] = ld_stream_u4(vbase + cache_row(p.pm, b, h, t, p.vsb, p.vsh, p.vst, p.status));
        } else {
          kk[i] = ld_stream_u4(kbase + b * p.ksb + h * p.ksh + (int64_t)t * p.kst);
          vv[i] = ld_stream_u4(vbase + b * p.vsb + h * p.vsh + (int64_t)t * p.vst);
        }
      } else {
        kk[i] = make_uint4(0u, 0u, 0u, 0u);
        vv[i] = make_uint4(0u, 0u, 0u, 0u);
      }
    }

    float alpha[GP];
#pragma unroll
    for (int g = 0; g < GP; ++g) {
      // partial logits of the 8 rows over this lane's 8 channels
      float part[kRB];
#pragma unroll
      for (int i = 0; i < kRB; ++i) part[i] = dot8(qf[g], kk[i]);
      // transposing reduction over the 16 lanes: 8 -> 4 -> 2 -> 1 rows per lane
      float p4[4], p2[2], p1;
      {
        const bool up = (l16 & 8) != 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float send = up ? part[i] : part[i + 4];
          const float keep = up ? part[i + 4] : part[i];
          p4[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
        }
      }
      {
        const bool up = (l16 & 4) != 0;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const float send = up ? p4[i] : p4[i + 2];
          const float keep = up ? p4[i + 2] : p4[i];
          p2[i] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
        }
      }
      {
        const bool up = (l16 & 2) != 0;
        const float send = up ? p2[0] : p2[1];
        const float keep = up ? p2[1] : p2[0];
        p1 = keep + __shfl_xor_sync(0xffffffffu, send, 2);
      }
      p1 += __shfl_xor_sync(0xffffffffu, p1, 1);
      const float logit = (base + my_row < r1) ? p1 : -INFINITY;
      float bmax = logit;
      bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 8));
      bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 4));
      bmax = fmaxf(bmax, __shfl_xor_sync(0xffffffffu, bmax, 2));
      const float m_new = fmaxf(m[g], bmax);
      // m_new is finite here: the batch holds at least one real row with finite inputs.
      const float m_safe = m_new == -INFINITY ? 0.f : m_new;
      alpha[g] = exp2f(m[g] - m_safe);
      const float pr = exp2f(logit - m_safe);
      lsum[g] = lsum[g] * alpha[g] + ((l16 & 1) ? 0.f : pr);
      m[g] = m_new;
      if ((l16 & 1) == 0) s_p[hwid][my_row][g] = pr;
    }
    __syncwarp();

#pragma unroll
    for (int g = 0; g < GP; ++g) {
      const float2 a2 = make_float2(alpha[g], alpha[g]);
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[g][e] = __ffma2_rn(acc[g][e], a2, make_float2(0.f, 0.f));
    }
#pragma unroll
    for (int i = 0; i < kRB; ++i) {
      const float4 pi = *reinterpret_cast<const float4*>(&s_p[hwid][i][0]);
      const float pg[4] = {pi.x, pi.y, pi.z, pi.w};
      float2 vf[4];
      vf[0] = bf16x2_to_f32x2(vv[i].x);
      vf[1] = bf16x2_to_f32x2(vv[i].y);
      vf[2] = bf16x2_to_f32x2(vv[i].z);
      vf[3] = bf16x2_to_f32x2(vv[i].w);
#pragma unroll
      for (int g = 0; g < GP; ++g) {
        const float2 p2 = make_float2(pg[g], pg[g]);
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[g][e] = __ffma2_rn(p2, vf[e], acc[g][e]);
      }
    }
    __syncwarp();  // s_p is rewritten by the next batch
  }

  // ---- combine the half-warps of this CTA, then write one partial per head -----------
#pragma unroll
  for (int g = 0; g < GP; ++g) {
    float l = lsum[g];
    l += __shfl_xor_sync(0xffffffffu, l, 8);
    l += __shfl_xor_sync(0xffffffffu, l, 4);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    if (l16 == 0) {
      s_m[hwid][g] = m[g];
      s_l[hwid][g] = l;
    }
    float4* dst = reinterpret_cast<float4*>(&s_acc[hwid][g][l16 * 8]);
    dst[0] = make_float4(acc[g][0].x, acc[g][0].y, acc[g][1].x, acc[g][1].y);
    dst[1] = make_float4(acc[g][2].x, acc[g][2].y, acc[g][3].x, acc[g][3].y);
  }
  __syncthreads();

  const int c = threadIdx.x;  // one channel per thread
  for (int gl = 0; gl < p.group; ++gl) {
    const int gi = HWS == 1 ? gl : gl % GP;      // index inside the half-warp
    const int hsel = HWS == 1 ? 0 : gl / GP;     // which half of each warp holds it
    float mx = -INFINITY;
#pragma unroll
    for (int s = 0; s < kSlots; ++s) {
      const int hwi = HWS == 1 ? s : s * 2 + hsel;
      mx = fmaxf(mx, s_m[hwi][gi]);
    }
    float a = 0.f, l = 0.f;
#pragma unroll
    for (int s = 0; s < kSlots; ++s) {
      const int hwi = HWS == 1 ? s : s * 2 + hsel;
      const float ms = s_m[hwi][gi];
      const float w = ms == -INFINITY ? 0.f : exp2f(ms - mx);
      a += w * s_acc[hwi][gi][c];
      l += w * s_l[hwi][gi];
    }
    float* dst = p.partial +
                 ((su.q0 + gl) * p.n_splits + split) * kPartialStride;
    dst[2 + c] = a;
    if (c == 0) {
      dst[0] = mx;
      dst[1] = l;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Tensor-core form.  With a GQA group of G query heads the two products of a decode step are
// [rows x 128] . [128 x G] (logits) and [128 x rows] . [rows x G] (output, transposed): G <= 8
// is exactly the N = 8 of mma.m16n8k16.  The scalar kernel above spends ~60 instructions per
// K/V row per four heads and is bound by instruction issue (0.67 of the copy bandwidth at
// G = 4, 0.3 at G = 7); here a warp handles 16 rows with 8 + 16 MMAs.
//   - K and V rows go to shared memory with 16-byte cp.async copies (row stride padded by 16
//     bytes, so ldmatrix reads them without bank conflicts);
//   - logits: A = K tile via ldmatrix.x4, B = q (bf16, exact) in registers; the softmax scale
//     is applied to the fp32 result;
//   - online softmax per head on the accumulator fragment (a thread owns heads 2t, 2t+1 of
//     rows g, g+8; row maxima and sums by xor-shuffles over g);
//   - output: A = V^T via ldmatrix.x4.trans, B = P^T.  P is split into two bf16 terms
//     (p = hi + lo, error 2^-17 p) because one bf16 term would cost up to 2^-9 |v| of the
//     2e-3 tolerance; two MMAs per block.
constexpr int kMmaThreads = 128;
constexpr int kMmaWarps = kMmaThreads / 32;
constexpr int kRowPad = FASA_HEAD_DIM + 8;          // bf16 elements per staged row (272 bytes)

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(void* dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr(dst)), "l"(src) : "memory");
}
// The same through L1 ("cache all levels"): rows that live in page-locked HOST memory cross the
// host link in full 128-byte requests this way, at twice the rate of the L2-only form (measured:
// 50 vs 25 GB/s of a 55 GB/s link); for rows in HBM the L2-only form above is the faster one.
__device__ __forceinline__ void cp_async16_ca(void* dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(smem_addr(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async4(void* dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_addr(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// waits until at most N of this thread's committed groups are still in flight
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* row) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_addr(row)));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* row) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_addr(row)));
}
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// round-to-nearest-even fp32 -> bf16 bits (finite inputs)
__device__ __forceinline__ uint32_t f32_to_bf16_bits(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u + 0x7fffu + ((u >> 16) & 1u)) >> 16;
}

struct MmaSmem {
  uint16_t k[kMmaWarps][16][kRowPad];
  uint16_t v[kMmaWarps][16][kRowPad];
  uint16_t p_hi[kMmaWarps][8][16];                  // P^T: [head][row]
  uint16_t p_lo[kMmaWarps][8][16];
};

// Programmatic dependent launch: these kernels may be scheduled while the kernel before them
// on the stream is still draining (their launch latency then overlaps its tail).  They wait
// here until that kernel has completed and its writes are visible, and let their own
// successor be scheduled early in turn.  Launched the ordinary way, both are no-ops.
__device__ __forceinline__ void pdl_wait_for_predecessor() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_release_successor() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// cluster_x > 0: the CTAs of a grid row form one thread-block cluster of that size.
template <typename Kernel, typename... Args>
cudaError_t launch_after_predecessor(Kernel kernel, dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                     int cluster_x, Args... args) {
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.numAttrs = 1;
  if (cluster_x > 0) {
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)cluster_x;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  }
  cfg.attrs = attr;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// CLUSTER: the splits of a unit are the CTAs of one cluster (grid.x = cluster size) and merge
// in the same launch; otherwise each split writes its partial result for the merge kernel.
// HOSTMEM: K and V rows are copied through L1 (caches in page-locked host memory).  KSPLIT
// (Algorithm 2's Combine; sparse, contiguous, HOSTMEM): a key row is assembled in shared memory
// from its non-dominant channels (p.k, ascending channel order, the part that crosses the host
// link) followed by its dominant channels in proxy order (from the GPU-resident proxy); the
// query operand is loaded in the same channel order, so the logits are the same dot products
// summed in another order.
template <bool SPARSE, bool PAGED, bool CLUSTER, bool HOSTMEM = false, bool KSPLIT = false>
__global__ void __launch_bounds__(kMmaThreads)
decode_attn_mma_kernel(const AttnParams p) {
  __shared__ ClusterMergeSmem s_merge;              // (CLUSTER only: written by the peers)
  pdl_wait_for_predecessor();
  pdl_release_successor();
  const int u = blockIdx.y;
  const SelUnit su = sel_unit(u, p.n_sets, p.group, p.n_q_heads, p.n_kv_heads);
  const int h = su.h;
  const int b = su.b;
  int n;
  if (SPARSE) {
    n = p.n_rows[u];
    if (n < 0 || n > p.n_cap) {
      atomicOr(p.status, FASA_DEV_NSEL_CLAMPED);
      n = n < 0 ? 0 : p.n_cap;
    }
  } else {
    n = clamp_len(p.n_rows[b], p.max_len, p.status);
  }
  const int split = blockIdx.x;
  // In a cluster the splits share the rows the unit actually has (every CTA stays for the merge
  // anyway, and with rows far below the bound a fixed split size would leave most of them idle
  // while they hold their place on an SM); otherwise the split size is the planned one, which
  // the merge kernel knows.
  const int chunk = CLUSTER ? min(p.chunk, max(32, ((n + (int)gridDim.x - 1) / (int)gridDim.x + 31) & ~31)) : p.chunk;
  const int r0 = min(n, split * chunk);
  if (!CLUSTER && r0 >= n) return;
  const int r1 = min(n, r0 + chunk);

  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;

  extern __shared__ __align__(16) unsigned char attn_smem_raw[];
  MmaSmem& sm = *reinterpret_cast<MmaSmem*>(attn_smem_raw);

  // B operand of the logits: q[head g][channels], bf16 as stored, for the 8 blocks of 16 channels
  uint32_t qb[8][2];
  {
    const uint16_t* qh = p.q + (su.q0 + (g < p.group ? g : 0)) * FASA_HEAD_DIM;
    // position c of an assembled key row holds channel ndchan[c] (c < nd) or chan[c - nd]
    auto q_at = [&](int c) -> uint32_t {
      const int ch = c < p.ks.nd ? p.ks.ndchan[h * p.ks.nd + c] : p.ks.chan[h * p.ks.chunks * 8 + c - p.ks.nd];
      return qh[ch];
    };
#pragma unroll
    for (int kb = 0; kb < 8; ++kb) {
      uint32_t w0, w1;
      if constexpr (KSPLIT) {
        w0 = q_at(kb * 16 + 2 * t) | (q_at(kb * 16 + 2 * t + 1) << 16);
        w1 = q_at(kb * 16 + 2 * t + 8) | (q_at(kb * 16 + 2 * t + 9) << 16);
      } else {
        w0 = *reinterpret_cast<const uint32_t*>(qh + kb * 16 + 2 * t);
        w1 = *reinterpret_cast<const uint32_t*>(qh + kb * 16 + 2 * t + 8);
      }
      qb[kb][0] = g < p.group ? w0 : 0u;
      qb[kb][1] = g < p.group ? w1 : 0u;
    }
  }

  float acc[8][4];                                  // out^T: [16-channel block][frag], heads 2t, 2t+1
#pragma unroll
  for (int cb = 0; cb < 8; ++cb) acc[cb][0] = acc[cb][1] = acc[cb][2] = acc[cb][3] = 0.f;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};

  const int32_t* irow = SPARSE ? p.idx + (int64_t)u * p.n_sel_max : nullptr;

  // The CTA's slice of the index list goes to shared memory in one coalesced read (checked
  // once): a tile then costs one memory round trip (its rows), not two (its indices first).
  int32_t* s_idx = reinterpret_cast<int32_t*>(attn_smem_raw + sizeof(MmaSmem));
  if (SPARSE) {
    for (int i = threadIdx.x; i < r1 - r0; i += kMmaThreads) {
      int tok = __ldg(irow + r0 + i);
      if (tok < 0 || tok >= p.max_len) {
        atomicOr(p.status, FASA_DEV_IDX_CLAMPED);
        tok = 0;
      }
      if constexpr (KSPLIT) {
        // a row that is resident on the GPU is entered as -1 - slot: it is then copied from there
        if (p.ks.res.tags != nullptr) {
          const int slot = fasa_resident_slot(p.ks.res, tok);
          if (slot >= 0 && p.ks.res.tags[(int64_t)su.kv * p.ks.res.slots_pad + slot] == tok) tok = -1 - slot;
        }
      }
      s_idx[i] = tok;
    }
    __syncthreads();
  }

  // Staging of a tile's 16 K rows (or V rows): lane l copies chunk (l % 16) of rows 2j + l / 16.
  // The K and the V buffer of a warp are two pipeline stages: the next tile's K rows are
  // requested as soon as this tile's logits are done (they travel during the output
  // product), its V rows as soon as the output product is done (they travel during the next
  // logits), so memory stays busy while the warp computes.  One cp.async group per buffer
  // fill, an empty group when there is no next tile, so "all but the newest group" always
  // names the buffer that is needed next.
  const int bc = b / p.q_len;                       // the sequence whose cache this unit reads
  const uint16_t* kunit = PAGED ? p.k : p.k + bc * p.ksb + h * p.ksh;
  const uint16_t* vunit = PAGED ? p.v : p.v + bc * p.vsb + h * p.vsh;
  auto stage = [&](uint16_t (*dst)[kRowPad], const uint16_t* unit, int64_t sb, int64_t sh, int64_t st, int base) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int row = 2 * j + (lane >> 4);
      const int r = min(base + row, r1 - 1);        // rows past the end repeat the last one (masked below)
      const int tok = SPARSE ? s_idx[r - r0] : r;
      const int c8 = (lane & 15) * 8;
      // (contiguous caches keep the plain address arithmetic: the page map costs registers)
      if constexpr (PAGED) cp_async16(&dst[row][c8], unit + cache_row(p.pm, bc, h, tok, sb, sh, st, p.status) + c8);
      else if constexpr (HOSTMEM) cp_async16_ca(&dst[row][c8], unit + (int64_t)tok * st + c8);
      else cp_async16(&dst[row][c8], unit + (int64_t)tok * st + c8);
    }
  };
  // Combine: the 16 key rows of a tile from their two homes
  const ProxyGeom ks_pg = proxy_geom(KSPLIT ? p.ks.chunks : 1);
  const unsigned char* ks_proxy = KSPLIT ? p.ks.proxy + (int64_t)su.kv * ((p.max_len + 15) >> 4) * ks_pg.tile_bytes : nullptr;
  const uint16_t* res_rows = KSPLIT && p.ks.res.tags ? p.ks.res.rows + (int64_t)su.kv * p.ks.res.slots * 2 * FASA_HEAD_DIM : nullptr;
  auto stage_split_k = [&](uint16_t (*dst)[kRowPad], int base) {
    const int nd_chunks = p.ks.nd >> 3, words = 4 * p.ks.chunks;
    for (int c = lane; c < 16 * nd_chunks; c += 32) {                 // the part that crosses the link
      const int row = c / nd_chunks, ch = c % nd_chunks;
      const int tok = s_idx[min(base + row, r1 - 1) - r0];
      if (tok >= 0) cp_async16_ca(&dst[row][ch * 8], kunit + (int64_t)tok * p.kst + ch * 8);
    }
    for (int c = lane; c < 16 * words; c += 32) {                     // the dominant pairs, from the proxy
      const int row = c / words, w = c % words;
      const int tok = s_idx[min(base + row, r1 - 1) - r0];
      if (tok >= 0) cp_async4(&dst[row][p.ks.nd + 2 * w], ks_proxy + proxy_word_offset(ks_pg, tok, w));
    }
    if (res_rows != nullptr) {                                        // resident rows: whole assembled key rows
      for (int c = lane; c < 16 * 16; c += 32) {
        const int row = c >> 4, ch = c & 15;
        const int tok = s_idx[min(base + row, r1 - 1) - r0];
        if (tok < 0) cp_async16(&dst[row][ch * 8], res_rows + (int64_t)(-1 - tok) * 2 * FASA_HEAD_DIM + ch * 8);
      }
    }
  };
  // value rows of a tile with a split key cache: from the host, or from the resident rows
  auto stage_split_v = [&](uint16_t (*dst)[kRowPad], int base) {
    for (int c = lane; c < 16 * 16; c += 32) {
      const int row = c >> 4, ch = c & 15;
      const int tok = s_idx[min(base + row, r1 - 1) - r0];
      if (tok >= 0) cp_async16_ca(&dst[row][ch * 8], vunit + (int64_t)tok * p.vst + ch * 8);
      else cp_async16(&dst[row][ch * 8], res_rows + (int64_t)(-1 - tok) * 2 * FASA_HEAD_DIM + FASA_HEAD_DIM + ch * 8);
    }
  };
  auto stage_v = [&](int base) {
    if constexpr (KSPLIT) stage_split_v(sm.v[warp], base);
    else stage(sm.v[warp], vunit, p.vsb, p.vsh, p.vst, base);
  };
  auto stage_k = [&](int base) {
    if constexpr (KSPLIT) stage_split_k(sm.k[warp], base);
    else stage(sm.k[warp], kunit, p.ksb, p.ksh, p.kst, base);
  };
  constexpr int kTileStep = kMmaWarps * 16;
  if (r0 + warp * 16 < r1) stage_k(r0 + warp * 16);
  cp_async_commit();
  if (r0 + warp * 16 < r1) stage_v(r0 + warp * 16);
  cp_async_commit();

  for (int base = r0 + warp * 16; base < r1; base += kTileStep) {   // uniform over the warp
    const bool more = base + kTileStep < r1;
    cp_async_wait<1>();                             // this tile's K rows have landed
    __syncwarp();

    // ---- logits: D[16 rows x 8 heads] ---------------------------------------------------------
    float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int kb = 0; kb < 8; ++kb) {
      uint32_t a[4];
      // matrices: (rows 0-7, ch 0-7), (rows 8-15, ch 0-7), (rows 0-7, ch 8-15), (rows 8-15, ch 8-15)
      ldmatrix_x4(a, &sm.k[warp][(lane & 7) + 8 * ((lane >> 3) & 1)][kb * 16 + 8 * (lane >> 4)]);
      mma16816(c, a, qb[kb][0], qb[kb][1]);
    }
    // thread: c0, c1 = row g, heads 2t, 2t+1; c2, c3 = row g + 8
    const bool ok_lo = base + g < r1, ok_hi = base + g + 8 < r1;
    float lg[4];
    lg[0] = ok_lo ? c[0] * p.scale_log2 : -INFINITY;
    lg[1] = ok_lo ? c[1] * p.scale_log2 : -INFINITY;
    lg[2] = ok_hi ? c[2] * p.scale_log2 : -INFINITY;
    lg[3] = ok_hi ? c[3] * p.scale_log2 : -INFINITY;
    float alpha[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      float bm = fmaxf(lg[e], lg[2 + e]);
      bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 4));
      bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 8));
      bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 16));
      const float m_new = fmaxf(m_run[e], bm);
      const float m_safe = m_new == -INFINITY ? 0.f : m_new;
      alpha[e] = exp2f(m_run[e] - m_safe);
      lg[e] = exp2f(lg[e] - m_safe);
      lg[2 + e] = exp2f(lg[2 + e] - m_safe);
      l_run[e] = l_run[e] * alpha[e] + lg[e] + lg[2 + e];   // this thread's rows; the g lanes are added at the end
      m_run[e] = m_new;
    }
    // P^T[head][row] as two bf16 terms
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int head = 2 * t + (e & 1), row = g + 8 * (e >> 1);
      const uint32_t hi = f32_to_bf16_bits(lg[e]);
      const float rest = lg[e] - __uint_as_float(hi << 16);
      sm.p_hi[warp][head][row] = (uint16_t)hi;
      sm.p_lo[warp][head][row] = (uint16_t)f32_to_bf16_bits(rest);
    }
    __syncwarp();                                   // P is visible; every lane is done with the K buffer
    if (more) stage_k(base + kTileStep);
    cp_async_commit();
    cp_async_wait<1>();                             // this tile's V rows have landed
    __syncwarp();
    // B operand of the output product: B[k = row][n = head g]: rows 2t, 2t+1 and 2t+8, 2t+9
    const uint32_t ph0 = *reinterpret_cast<const uint32_t*>(&sm.p_hi[warp][g][2 * t]);
    const uint32_t ph1 = *reinterpret_cast<const uint32_t*>(&sm.p_hi[warp][g][2 * t + 8]);
    const uint32_t pl0 = *reinterpret_cast<const uint32_t*>(&sm.p_lo[warp][g][2 * t]);
    const uint32_t pl1 = *reinterpret_cast<const uint32_t*>(&sm.p_lo[warp][g][2 * t + 8]);

    // ---- output: out^T[16 ch x 8 heads] += V^T[16 ch x 16 rows] . P^T[16 rows x 8 heads] ------
#pragma unroll
    for (int cb = 0; cb < 8; ++cb) {
      acc[cb][0] *= alpha[0]; acc[cb][1] *= alpha[1]; acc[cb][2] *= alpha[0]; acc[cb][3] *= alpha[1];
      uint32_t a[4];
      // source blocks (token rows x channels), transposed on load:
      // (rows 0-7, ch 0-7), (rows 0-7, ch 8-15), (rows 8-15, ch 0-7), (rows 8-15, ch 8-15)
      ldmatrix_x4_trans(a, &sm.v[warp][(lane & 7) + 8 * (lane >> 4)][cb * 16 + 8 * ((lane >> 3) & 1)]);
      mma16816(acc[cb], a, ph0, ph1);
      mma16816(acc[cb], a, pl0, pl1);
    }
    __syncwarp();                                   // every lane is done with the V buffer
    if (more) stage_v(base + kTileStep);
    cp_async_commit();
  }
  cp_async_wait<0>();

  // ---- this warp's (m, l, acc) per head; the g lanes add their sums -------------------------------
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 4);
    l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 8);
    l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 16);
  }
  __syncthreads();                                  // staging memory becomes the combine area
  float* s_acc = reinterpret_cast<float*>(attn_smem_raw);                 // [warps][8 heads][128]
  float* s_ml = s_acc + kMmaWarps * 8 * FASA_HEAD_DIM;                    // [warps][8 heads][2]
#pragma unroll
  for (int cb = 0; cb < 8; ++cb) {
    s_acc[(warp * 8 + 2 * t) * FASA_HEAD_DIM + cb * 16 + g] = acc[cb][0];
    s_acc[(warp * 8 + 2 * t + 1) * FASA_HEAD_DIM + cb * 16 + g] = acc[cb][1];
    s_acc[(warp * 8 + 2 * t) * FASA_HEAD_DIM + cb * 16 + g + 8] = acc[cb][2];
    s_acc[(warp * 8 + 2 * t + 1) * FASA_HEAD_DIM + cb * 16 + g + 8] = acc[cb][3];
  }
  if (g == 0) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      s_ml[(warp * 8 + 2 * t + e) * 2 + 0] = m_run[e];
      s_ml[(warp * 8 + 2 * t + e) * 2 + 1] = l_run[e];
    }
  }
  __syncthreads();
  const int cch = threadIdx.x;                      // one channel per thread
  // (CLUSTER: this CTA's partial per head goes to shared memory behind the combine area)
  float (*s_part)[kMergePartStride] = reinterpret_cast<float (*)[kMergePartStride]>(s_ml + kMmaWarps * 8 * 2);
  for (int gl = 0; gl < p.group; ++gl) {
    float mx = -INFINITY;
#pragma unroll
    for (int w = 0; w < kMmaWarps; ++w) mx = fmaxf(mx, s_ml[(w * 8 + gl) * 2]);
    float a = 0.f, l = 0.f;
#pragma unroll
    for (int w = 0; w < kMmaWarps; ++w) {
      const float ms = s_ml[(w * 8 + gl) * 2];
      const float wt = ms == -INFINITY ? 0.f : exp2f(ms - mx);
      a += wt * s_acc[(w * 8 + gl) * FASA_HEAD_DIM + cch];
      l += wt * s_ml[(w * 8 + gl) * 2 + 1];
    }
    float* dst = CLUSTER ? &s_part[gl][0] : p.partial + ((su.q0 + gl) * p.n_splits + split) * kPartialStride;
    dst[2 + cch] = a;
    if (cch == 0) {
      dst[0] = mx;
      dst[1] = l;
    }
  }
  if constexpr (CLUSTER) {
    __syncthreads();
    cg::cluster_group cluster = cg::this_cluster();
    cluster_merge_store<kMmaThreads>(cluster, s_part, s_merge, p.group, su.q0, p.out, p.out_mirror, p.lse);
  }
}

// Merge pass: one CTA per (batch, query head); thread (c, j) takes channel c of the splits
// s = j, j + 4, ... so that four chains of dependent loads run side by side, then the four
// partial merges are merged.
constexpr int kMergeWays = 4;
template <bool SPARSE>
__global__ void __launch_bounds__(FASA_HEAD_DIM * kMergeWays)
decode_attn_merge_kernel(const float* __restrict__ partial, const int32_t* __restrict__ n_rows,
                         float* __restrict__ out, float* __restrict__ lse,
                         int32_t* __restrict__ status, int n_q_heads, int n_sets, int group,
                         int max_len, int n_cap, int chunk, int n_splits) {
  pdl_wait_for_predecessor();
  const int bh = blockIdx.x;
  const int b = bh / n_q_heads;
  const int hq = bh % n_q_heads;
  int n;
  if (SPARSE) {
    n = n_rows[b * n_sets + hq / group];
    n = n < 0 ? 0 : (n > n_cap ? n_cap : n);
  } else {
    n = n_rows[b];
    n = n < 0 ? 0 : (n > max_len ? max_len : n);
  }
  const int ns = min(n_splits, (n + chunk - 1) / chunk);
  const int c = threadIdx.x % FASA_HEAD_DIM;
  const int j = threadIdx.x / FASA_HEAD_DIM;
  const float* src = partial + (int64_t)bh * n_splits * kPartialStride;
  __shared__ float s_m[kMergeWays], s_l[kMergeWays];
  __shared__ float s_a[kMergeWays][FASA_HEAD_DIM];
  float mx = -INFINITY;
  for (int s = j; s < ns; s += kMergeWays) mx = fmaxf(mx, src[s * kPartialStride]);
  float a = 0.f, l = 0.f;
  for (int s = j; s < ns; s += kMergeWays) {
    const float ms = src[s * kPartialStride];
    const float w = ms == -INFINITY ? 0.f : exp2f(ms - mx);
    a += w * src[s * kPartialStride + 2 + c];
    l += w * src[s * kPartialStride + 1];
  }
  s_a[j][c] = a;
  if (c == 0) {
    s_m[j] = mx;
    s_l[j] = l;
  }
  __syncthreads();
  if (j != 0) return;
  float m_all = -INFINITY;
#pragma unroll
  for (int k = 0; k < kMergeWays; ++k) m_all = fmaxf(m_all, s_m[k]);
  float a_all = 0.f, l_all = 0.f;
#pragma unroll
  for (int k = 0; k < kMergeWays; ++k) {
    const float w = s_m[k] == -INFINITY ? 0.f : exp2f(s_m[k] - m_all);
    a_all += w * s_a[k][c];
    l_all += w * s_l[k];
  }
  out[(int64_t)bh * FASA_HEAD_DIM + c] = (ns > 0 && l_all > 0.f) ? a_all / l_all : 0.f;
  if (lse && c == 0)
    lse[bh] = (ns > 0 && l_all > 0.f) ? (m_all + log2f(l_all)) * 0.6931471805599453f : -INFINITY;
}

// out_mirror (nullable): a second destination of out; *mirrored tells whether it was written
// (only the form that merges inside the attention launch can do that).
template <bool SPARSE>
int32_t launch_attn(fasa_ctx* ctx, const void* q, const void* k, const void* v,
                    const int32_t* idx, const int32_t* n_rows, int n_upper, int n_sel_max,
                    float* out, float* lse, void* workspace, cudaStream_t s, float* out_mirror = nullptr,
                    bool* mirrored = nullptr, int q_len = 1, const fasa_ksplit* ksplit = nullptr) {
  if (mirrored) *mirrored = false;
  const fasa_config_t& c = ctx->cfg;
  if (!fasa_pages_ready(ctx)) return FASA_ERR_INVALID_ARG;
  // the dense pass treats a KV head with all its query heads as the unit
  const int n_sets = SPARSE ? ctx->n_sets : c.n_kv_heads;
  const int G = SPARSE ? ctx->sel_heads : ctx->group;
  const int n_seq = c.batch * q_len;                // rows of the grid's "batch" axis
  const fasa_split_plan plan = fasa_plan_splits(ctx, n_upper, n_seq * n_sets);
  AttnParams p;
  p.q_len = q_len;
  memset(&p.ks, 0, sizeof(p.ks));
  if (ksplit) p.ks = *ksplit;
  // caches in page-locked host memory are copied through L1 (contiguous caches, tensor-core kernel)
  const bool host = c.page_size == 0 && ctx->use_fused && (ksplit != nullptr || fasa_on_host(ctx, k));
  p.q = (const uint16_t*)q; p.k = (const uint16_t*)k; p.v = (const uint16_t*)v;
  p.idx = idx; p.n_rows = n_rows; p.partial = (float*)workspace; p.out = nullptr; p.out_mirror = nullptr; p.lse = nullptr; p.status = ctx->d_status;
  p.n_q_heads = c.n_q_heads; p.n_kv_heads = c.n_kv_heads; p.n_sets = n_sets; p.group = G;
  p.max_len = c.max_len; p.n_sel_max = n_sel_max; p.n_cap = n_upper; p.chunk = plan.chunk; p.n_splits = plan.n_splits;
  p.ksb = c.k_stride_b; p.ksh = c.k_stride_h; p.kst = c.k_stride_t;
  p.vsb = c.v_stride_b; p.vsh = c.v_stride_h; p.vst = c.v_stride_t;
  p.pm = fasa_page_map(ctx);
  p.scale_log2 = c.softmax_scale * 1.4426950408889634f;
  dim3 grid((unsigned)plan.n_splits, (unsigned)(n_seq * n_sets));
  if (ctx->use_fused) {   // default: the tensor-core kernel (mode 0 keeps the scalar one)
    static_assert(sizeof(MmaSmem) >= ((size_t)kMmaWarps * 8 * (FASA_HEAD_DIM + 2) + 8 * kMergePartStride) * sizeof(float),
                  "combine area");
    const int max_smem = (int)(sizeof(MmaSmem) + 2080 * sizeof(int32_t));
    // One launch where the splits of a unit fit a portable cluster: the split count becomes a
    // power of two <= 8 (the nearest to the planned one) and the cluster merges by itself.
    int cs = 1;
    while (cs < 8 && cs * 3 < plan.n_splits * 2) cs *= 2;          // nearest power of two, ties up
    int cchunk = ((n_upper + cs - 1) / cs + 31) / 32 * 32;
    while (cs < 8 && cchunk > 2048) { cs *= 2; cchunk = ((n_upper + cs - 1) / cs + 31) / 32 * 32; }
    if (cchunk <= 2048) {
      p.chunk = cchunk; p.n_splits = cs; p.out = out; p.out_mirror = out_mirror; p.lse = lse;
      if (mirrored) *mirrored = out_mirror != nullptr;
      auto fn = c.page_size > 0 ? decode_attn_mma_kernel<SPARSE, true, true> : decode_attn_mma_kernel<SPARSE, false, true>;
      if (host) fn = decode_attn_mma_kernel<SPARSE, false, true, true>;
      if constexpr (SPARSE) { if (ksplit) fn = decode_attn_mma_kernel<true, false, true, true, true>; }
      const size_t smem = sizeof(MmaSmem) + (SPARSE ? (size_t)cchunk * sizeof(int32_t) : 0);
      FASA_CUDA_TRY(ctx, cudaFuncSetAttribute((const void*)fn, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem));
      FASA_CUDA_TRY(ctx, launch_after_predecessor(fn, dim3((unsigned)cs, grid.y), dim3(kMmaThreads), smem, s, cs, p));
      FASA_LAUNCH_CHECK(ctx);
      return FASA_OK;
    }
    auto fn = c.page_size > 0 ? decode_attn_mma_kernel<SPARSE, true, false> : decode_attn_mma_kernel<SPARSE, false, false>;
    if (host) fn = decode_attn_mma_kernel<SPARSE, false, false, true>;
    if constexpr (SPARSE) { if (ksplit) fn = decode_attn_mma_kernel<true, false, false, true, true>; }
    // (+ the slice of the index list: chunk <= 2048 rows)
    const size_t smem = sizeof(MmaSmem) + (SPARSE ? (size_t)plan.chunk * sizeof(int32_t) : 0);
    FASA_CUDA_TRY(ctx, cudaFuncSetAttribute((const void*)fn, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem));
    FASA_CUDA_TRY(ctx, launch_after_predecessor(fn, grid, dim3(kMmaThreads), smem, s, 0, p));
  } else if (G == 1) decode_attn_kernel<1, 1, SPARSE><<<grid, kAttnThreads, 0, s>>>(p);
  else if (G == 2) decode_attn_kernel<2, 1, SPARSE><<<grid, kAttnThreads, 0, s>>>(p);
  else if (G == 3) decode_attn_kernel<3, 1, SPARSE><<<grid, kAttnThreads, 0, s>>>(p);
  else if (G == 4) decode_attn_kernel<4, 1, SPARSE><<<grid, kAttnThreads, 0, s>>>(p);
  else if (G <= 6) decode_attn_kernel<3, 2, SPARSE><<<grid, kAttnThreads, 0, s>>>(p);
  else decode_attn_kernel<4, 2, SPARSE><<<grid, kAttnThreads, 0, s>>>(p);
  FASA_LAUNCH_CHECK(ctx);
  FASA_CUDA_TRY(ctx, launch_after_predecessor(
      decode_attn_merge_kernel<SPARSE>, dim3((unsigned)(n_seq * c.n_q_heads)), dim3(FASA_HEAD_DIM * kMergeWays),
      (size_t)0, s, 0, (const float*)workspace, n_rows, out, lse, ctx->d_status, (int)c.n_q_heads, (int)n_sets,
      (int)G, (int)c.max_len, (int)n_upper, (int)plan.chunk, (int)plan.n_splits));
  FASA_LAUNCH_CHECK(ctx);
  return FASA_OK;
}

bool aligned(const void* p, uintptr_t a) { return ((uintptr_t)p & (a - 1)) == 0; }

}  // namespace

extern "C" int32_t fasa_sparse_decode_attn(fasa_ctx_t* ctx, const void* q, const void* k_cache,
                                           const void* v_cache, const int32_t* idx,
                                           const int32_t* n_sel, int32_t n_sel_max, float* out,
                                           float* lse, void* workspace, void* stream) {
  if (!ctx || !q || !k_cache || !v_cache || !idx || !n_sel || !out || !workspace || n_sel_max <= 0)
    return FASA_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(k_cache, 16) || !aligned(v_cache, 16) || !aligned(workspace, 256))
    return FASA_ERR_INVALID_ARG;
  const int n_upper = n_sel_max < ctx->cfg.max_len ? n_sel_max : ctx->cfg.max_len;
  return launch_attn<true>(ctx, q, k_cache, v_cache, idx, n_sel, n_upper, n_sel_max, out, lse,
                           workspace, (cudaStream_t)stream);
}

// fasa_sparse_decode_attn with a second destination for the output (the host-buffer step).
int32_t fasa_sparse_attn_mirrored(fasa_ctx* ctx, const void* q, const void* k_cache, const void* v_cache,
                                  const int32_t* idx, const int32_t* n_sel, int32_t n_sel_max, float* out,
                                  float* lse, void* workspace, cudaStream_t stream, float* out_mirror, bool* mirrored) {
  const int n_upper = n_sel_max < ctx->cfg.max_len ? n_sel_max : ctx->cfg.max_len;
  return launch_attn<true>(ctx, q, k_cache, v_cache, idx, n_sel, n_upper, n_sel_max, out, lse, workspace, stream,
                           out_mirror, mirrored);
}

// FAC over a split key cache (Algorithm 2: Combine, then Eq. 6-7): k_nondom holds the non-dominant
// channels of every key, the proxy their dominant ones.
int32_t fasa_attn_split_keys(fasa_ctx* ctx, const void* q, const void* k_nondom, const void* v_cache, const void* proxy_k,
                             const int32_t* idx, const int32_t* n_sel, int32_t n_sel_max, float* out, float* lse,
                             void* workspace, cudaStream_t stream) {
  const fasa_config_t& c = ctx->cfg;
  fasa_ksplit ks;
  ks.proxy = (const unsigned char*)proxy_k; ks.ndchan = ctx->d_ndchan; ks.chan = ctx->d_chan;
  ks.chunks = ctx->chunks; ks.nd = FASA_HEAD_DIM - 2 * c.n_dom;
  ks.res = fasa_resident_of(ctx);
  // (the kernel addresses k_nondom with the K strides: rows of nd elements, dense per unit)
  fasa_ctx tmp = *ctx;
  tmp.cfg.k_stride_t = ks.nd;
  tmp.cfg.k_stride_h = (int64_t)c.max_len * ks.nd;
  tmp.cfg.k_stride_b = tmp.cfg.k_stride_h * c.n_kv_heads;
  const int n_upper = n_sel_max < c.max_len ? n_sel_max : c.max_len;
  int32_t st = launch_attn<true>(&tmp, q, k_nondom, v_cache, idx, n_sel, n_upper, n_sel_max, out, lse, workspace, stream,
                                 nullptr, nullptr, 1, &ks);
  ctx->launches = tmp.launches;
  memcpy(ctx->cuda_err, tmp.cuda_err, sizeof(ctx->cuda_err));
  return st;
}

extern "C" int32_t fasa_sparse_decode_attn_batched(fasa_ctx_t* ctx, const void* q, const void* k_cache,
                                                   const void* v_cache, const int32_t* idx, const int32_t* n_sel,
                                                   int32_t q_len, int32_t n_sel_max, float* out, float* lse,
                                                   void* workspace, void* stream) {
  if (!ctx || !q || !k_cache || !v_cache || !idx || !n_sel || !out || !workspace || n_sel_max <= 0)
    return FASA_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(k_cache, 16) || !aligned(v_cache, 16) || !aligned(workspace, 256))
    return FASA_ERR_INVALID_ARG;
  if (q_len < 1 || q_len > FASA_MAX_QLEN || !ctx->use_fused) return FASA_ERR_UNSUPPORTED;   // (tensor-core kernel only)
  if ((long long)ctx->cfg.batch * q_len * ctx->n_sets > 65535) return FASA_ERR_UNSUPPORTED;
  const int n_upper = n_sel_max < ctx->cfg.max_len ? n_sel_max : ctx->cfg.max_len;
  // (beyond 16384 rows per unit the splits no longer merge inside one cluster, and the workspace
  // is sized for single queries)
  if (q_len > 1 && n_upper > 16384) return FASA_ERR_UNSUPPORTED;
  return launch_attn<true>(ctx, q, k_cache, v_cache, idx, n_sel, n_upper, n_sel_max, out, lse, workspace,
                           (cudaStream_t)stream, nullptr, nullptr, q_len);
}

extern "C" int32_t fasa_full_decode_attn(fasa_ctx_t* ctx, const void* q, const void* k_cache,
                                         const void* v_cache, const int32_t* seq_lens, float* out,
                                         float* lse, void* workspace, void* stream) {
  if (!ctx || !q || !k_cache || !v_cache || !seq_lens || !out || !workspace)
    return FASA_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(k_cache, 16) || !aligned(v_cache, 16) || !aligned(workspace, 256))
    return FASA_ERR_INVALID_ARG;
  return launch_attn<false>(ctx, q, k_cache, v_cache, nullptr, seq_lens, ctx->cfg.max_len, 0, out,
                            lse, workspace, (cudaStream_t)stream);
}

// ---- variant for callers that cannot allocate device memory --------------------------------

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_ptr[kMaxDevices];   // device address of g_static_scratch, per device ordinal
}  // namespace

extern "C" int32_t fasa_sparse_decode_attn_static(fasa_ctx_t* ctx, const void* q,
                                                  const void* k_cache, const void* v_cache,
                                                  const int32_t* idx, const int32_t* n_sel,
                                                  int32_t n_sel_max, float* out, float* lse,
                                                  void* stream) {
  if (!ctx || !q || !k_cache || !v_cache || !idx || !n_sel || !out || n_sel_max <= 0)
    return FASA_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(k_cache, 16) || !aligned(v_cache, 16)) return FASA_ERR_INVALID_ARG;
  const fasa_config_t& c = ctx->cfg;
  const int n_upper = n_sel_max < c.max_len ? n_sel_max : c.max_len;
  const fasa_split_plan plan = fasa_plan_splits(ctx, n_upper, c.batch * ctx->n_sets);
  const size_t need = (size_t)c.batch * c.n_q_heads * (size_t)plan.n_splits * kPartialStride * sizeof(float);
  if (need > kStaticScratchBytes) return FASA_ERR_WORKSPACE;

  // The symbol names a different copy of the array on each device: its address is looked up
  // once per device, with that device current (the name itself is not a device pointer).
  int dev = -1;
  FASA_CUDA_TRY(ctx, cudaGetDevice(&dev));
  if (dev != ctx->device || dev < 0 || dev >= kMaxDevices) return FASA_ERR_INVALID_ARG;
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[dev]) {
      void* p = nullptr;
      FASA_CUDA_TRY(ctx, cudaGetSymbolAddress(&p, g_static_scratch));
      g_scratch_ptr[dev] = p;
    }
    scratch = g_scratch_ptr[dev];
  }
  return launch_attn<true>(ctx, q, k_cache, v_cache, idx, n_sel, n_upper, n_sel_max, out, lse,
                           scratch, (cudaStream_t)stream);
}
