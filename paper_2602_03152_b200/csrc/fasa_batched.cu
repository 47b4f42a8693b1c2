// Blocks of query tokens (q_len = T > 1 per sequence: speculative or multi-token decoding).
//
// The method is defined per query q_t (Sec. 4.1: S_t and T_t; Sec. 4.2, Eq. 6-7: the output of
// q_t), so a block of T queries is T decode steps that happen to read the same cache: query t of
// the block sits at cache position L - T + t (L = seq_lens[b] counts the block's own keys, already
// appended), sees the rows up to its own, and gets its own scores, index set and output.  What
// the T steps share is the proxy-K stream: scoring all of them is ONE pass over it,
//     S[L x (G T)] = P[L x 2F] . Q[2F x (G T)],
// a real matrix product (N up to 64 columns), after which the G columns of each query are
// reduced.  This is the one dense contraction of the path, and it runs on the fifth-generation
// tensor cores: tcgen05.mma with both operands in shared memory and the fp32 accumulator in
// tensor memory (TMEM), read back with tcgen05.ld for the reduction over the group.
//
// fc_score_batched_kernel, per CTA (128 threads, a run of 128-token tiles of one unit):
//   - B operand: the unit's query values at the head's dominant channels, [N x K] K-major, built
//     once in shared memory in the canonical no-swizzle layout (8-row x 16-byte core matrices);
//   - A operand: 128 proxy rows [128 x K].  The proxy lives in HBM in the fragment order of the
//     warp-level tensor-core instruction (fasa_score_core.cuh); each warp pulls two 16-token
//     tiles with coalesced 16-byte loads and scatters their four 4-byte words per lane into the
//     core-matrix layout (conflict-free: the 32 lanes of a store fill 128 contiguous bytes);
//   - one thread issues K / 16 tcgen05.mma (M 128, N 16..64, bf16 x bf16 -> fp32) and commits
//     them to an mbarrier;
//   - epilogue: thread r owns token row r: tcgen05.ld of its N columns (column 8 g + t = head g,
//     query t, so the registers of a head are indexed statically), sum (or max) over the G heads
//     of each query, rows past a query's own position are not written.
// Two A buffers, two accumulators (32 or 64 TMEM columns each) and two register stages: the
// product of tile i+1 is issued before the epilogue of tile i, while the loads of tiles i+2 and
// i+3 travel.  Several CTAs share an SM (64 or 128 TMEM columns each; the shared memory is padded
// so that the CTAs of an SM never ask for more than its 512 columns).  The wait on the mbarrier
// is bounded: on expiry the kernel raises FASA_DEV_TIMEOUT, frees its tensor memory and returns.
//
// Selection and attention of the block reuse the cluster kernel's selection phases and the
// split-K tensor-core attention with (sequence, query) pairs as rows.
#include <type_traits>

#include "fasa_common.cuh"
#include "fasa_score_core.cuh"

namespace {

constexpr int kBT = 128;          // threads per CTA
constexpr int kBM = 128;          // tokens per MMA tile (the M of the instruction)
constexpr long long kWaitCycles = 400000000ll;   // bound of the wait for a product, in SM clocks (~0.2 s)

struct BatchedParams {
  const uint16_t* q;            // [batch][q_len][n_q_heads][128]
  const unsigned char* proxy;
  const int32_t* seq_lens;
  const int16_t* chan;
  float* scores;                // [batch][q_len][n_sets][max_len]
  int32_t* status;
  int n_q_heads, n_kv_heads, n_sets, group, max_len, chunks, q_len, n_cols, tiles_per_cta, max_reduce;
  PageMap pm;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Shared-memory matrix descriptor of a K-major operand without swizzling: rows in groups of 8,
// a group's 16-byte chunks 128 bytes apart (leading byte offset), groups `group_stride` bytes
// apart (stride byte offset); descriptor version 1.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr, uint32_t group_stride) {
  return (uint64_t)((smem_addr >> 4) & 0x3fffu) | ((uint64_t)(128u >> 4) << 16) |
         ((uint64_t)((group_stride >> 4) & 0x3fffu) << 32) | (1ull << 46);
}

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  const uint32_t zero = 0u;
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(zero)
      : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Byte offset of 4-byte word `w` (channels 2w, 2w+1 of the proxy row) of row `r` in an operand
// tile whose rows have `chunks_pad` 16-byte chunks.
__device__ __forceinline__ uint32_t operand_word(int r, int w, int chunks_pad) {
  return (uint32_t)((r >> 3) * chunks_pad * 128 + (w >> 2) * 128 + (r & 7) * 16 + (w & 3) * 4);
}

// KB: 16-channel blocks per proxy tile rounded up to 1, 2, 4 or 8 (the registers of the loads in
// flight).  Columns of the product: n = 8 g + t for head g of the set and query t of the block
// (a fixed 8 columns per head, so that the reduction over the heads indexes registers statically).
// EXACT: contiguous caches whose dominant channels fill exactly KB whole 16-channel blocks (8, 16,
// 32, 64 FCs), so loads and stores need no run-time test of the tile geometry or of a page map
// (the kernel is bound by the instructions it issues per tile, not by HBM).
template <int KB, bool MAXRED, bool EXACT>
__global__ void __launch_bounds__(kBT)
fc_score_batched_kernel(const BatchedParams p) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int u = blockIdx.y;
  const SelUnit su = sel_unit(u, p.n_sets, p.group, p.n_q_heads, p.n_kv_heads);
  const int b = su.b, h = su.h;
  const int hs = u % p.n_sets;
  const int len = clamp_len(p.seq_lens[b], p.max_len, p.status);
  const int mt0 = blockIdx.x * p.tiles_per_cta;
  const int mt1 = min(min((p.max_len + kBM - 1) / kBM, mt0 + p.tiles_per_cta), (len + kBM - 1) / kBM);
  if (mt0 >= mt1) return;                           // (uniform over the CTA; nothing allocated yet)

  extern __shared__ __align__(128) unsigned char bsm[];
  __shared__ __align__(8) unsigned long long s_bar[2];
  __shared__ uint32_t s_tmem;
  const ProxyGeom pg = proxy_geom(p.chunks);
  const int n_blocks = pg.n16 + pg.n8;              // 16-channel blocks per proxy tile, the 8-channel one included
  const int chunks_pad = (p.chunks + 1) & ~1;       // K of an instruction is 16 channels = two chunks
  const int words = 4 * p.chunks;                   // 4-byte words (channel pairs) per proxy row
  const int a_bytes = kBM * chunks_pad * 16;
  unsigned char* smA = bsm;                                            // 2 x [128 rows][chunks_pad x 16 B]
  unsigned char* smB = bsm + 2 * a_bytes;                              // [n_cols rows][chunks_pad x 16 B]
  const int tiles_alloc = (p.max_len + 15) >> 4;
  const int acc_cols = p.n_cols <= 32 ? 32 : 64;    // columns of one accumulator; two are allocated

  // ---- set-up: tensor memory, the barriers, the B operand, zeroed A buffers (their padding stays zero) ----
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(2 * acc_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&s_bar[0])), "r"(1) : "memory");
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&s_bar[1])), "r"(1) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = tid; i < (2 * kBM + p.n_cols) * chunks_pad * 4; i += kBT) reinterpret_cast<uint32_t*>(bsm)[i] = 0u;
  __syncthreads();
  {
    const int G = p.group, T = p.q_len;
    const int16_t* chan_h = p.chan + h * p.chunks * 8;
    for (int i = tid; i < T * G * words; i += kBT) {
      const int c = i / words, w = i % words;
      const int g = c / T, t = c % T;
      const uint16_t* qrow = p.q + (((int64_t)b * T + t) * p.n_q_heads + hs * G + g) * FASA_HEAD_DIM;
      const int c0 = chan_h[2 * w], c1 = chan_h[2 * w + 1];
      const uint32_t lo = c0 >= 0 ? qrow[c0] : 0u, hi = c1 >= 0 ? qrow[c1] : 0u;
      *reinterpret_cast<uint32_t*>(smB + operand_word(8 * g + t, w, chunks_pad)) = lo | (hi << 16);
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = s_tmem;

  // instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, N = n_cols, M = 128
  const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_cols >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
  const uint32_t a_addr = smem_u32(smA), b_addr = smem_u32(smB);
  const uint32_t group_stride = (uint32_t)chunks_pad * 128u;

  // a warp brings proxy tiles 2 warp, 2 warp + 1 of every 128-token tile (16 tokens each)
  // two register stages: tile i + 1 waits in one while the loads of tile i + 2 fill the other
  uint4 a0[2][KB], a1[2][KB];
  const unsigned char* unit_base = p.proxy + (int64_t)su.kv * tiles_alloc * (KB * 512);   // (EXACT)
  float* const score_row0 = p.scores + ((int64_t)b * p.q_len * p.n_sets + hs) * p.max_len;    // query 0 of this unit
  const int64_t score_stride = (int64_t)p.n_sets * p.max_len;                                // one query to the next
  auto fetch = [&](uint4 (&a)[2][KB], int mt) {
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int T16 = mt * 8 + warp * 2 + j;
      const bool ok = T16 < tiles_alloc && T16 * 16 < len;
      const unsigned char* tile = p.proxy;
      if constexpr (EXACT) tile = unit_base + (int64_t)T16 * (KB * 512);
      else if (ok) tile += proxy_tile_offset(p.pm, b, h, p.n_kv_heads, T16, tiles_alloc, pg.tile_bytes, p.status);
#pragma unroll
      for (int kb = 0; kb < KB; ++kb) {
        if constexpr (EXACT) {
          a[j][kb] = ok ? ld_proxy_u4(tile + kb * 512 + lane * 16) : make_uint4(0u, 0u, 0u, 0u);
          continue;
        }
        a[j][kb] = make_uint4(0u, 0u, 0u, 0u);
        if (ok && kb < pg.n16) {
          a[j][kb] = ld_proxy_u4(tile + kb * 512 + lane * 16);
        } else if (ok && kb == pg.n16 && pg.n8) {
          const uint2 w2 = ld_proxy_u2(tile + pg.n16 * 512 + lane * 8);
          a[j][kb] = make_uint4(w2.x, w2.y, 0u, 0u);
        }
      }
    }
  };
  // lane 4 g + t of a block holds words (row g, t), (row g + 8, t), (row g, t + 4), (row g + 8, t + 4)
  // of the block's 8 words; the 8-channel block only the first two
  auto scatter = [&](const uint4 (&a)[2][KB], int buf) {
    const int g = lane >> 2, t = lane & 3;
    unsigned char* base = smA + buf * a_bytes + g * 16 + t * 4;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      unsigned char* rowg = base + ((warp * 2 + j) * 2) * group_stride;   // rows g and (next group) g + 8 of this 16-token tile
#pragma unroll
      for (int kb = 0; kb < KB; ++kb) {
        if (EXACT || kb < n_blocks) {
          *reinterpret_cast<uint32_t*>(rowg + kb * 256) = a[j][kb].x;
          *reinterpret_cast<uint32_t*>(rowg + group_stride + kb * 256) = a[j][kb].y;
          if (EXACT || kb < pg.n16) {
            *reinterpret_cast<uint32_t*>(rowg + kb * 256 + 128) = a[j][kb].z;
            *reinterpret_cast<uint32_t*>(rowg + group_stride + kb * 256 + 128) = a[j][kb].w;
          }
        }
      }
    }
  };
  // the products of one 128-token tile, from A buffer `buf` into accumulator `buf`, then the commit
  auto product = [&](int buf) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    for (int k2 = 0; k2 < chunks_pad / 2; ++k2)
      umma_bf16(tmem + buf * acc_cols, umma_desc(a_addr + buf * a_bytes + k2 * 256, group_stride),
                umma_desc(b_addr + k2 * 256, group_stride), idesc, k2 > 0 ? 1u : 0u);
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&s_bar[buf])) : "memory");
  };

  // Two A buffers, two accumulators, two register stages: the product of tile i + 1 is issued
  // before the epilogue of tile i, and the loads of tiles i + 2 and i + 3 are in flight meanwhile.
  bool timed_out = false;
  // one tile: `nxt` holds tile mt + 1 (scattered here, then refilled with tile mt + 3)
  auto tile_step = [&](int mt, uint4 (&nxt)[2][KB]) {
    const int i = mt - mt0, buf = i & 1;
    if (mt + 1 < mt1) {
      scatter(nxt, buf ^ 1);                        // (the buffer's last reader, the product of tile i - 1, was waited for)
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");       // these stores are read by the tensor core
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");   // (the tcgen05.ld of tile i - 1 are done)
      __syncthreads();
      if (tid == 0) product(buf ^ 1);
      if (mt + 3 < mt1) fetch(nxt, mt + 3);
    }
    {
      uint32_t done = 0;
      const uint32_t parity = (uint32_t)(i >> 1) & 1u;
      const long long t_wait = clock64();
      while (!done) {                               // a product takes microseconds; the bound is a fraction of a second
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(smem_u32(&s_bar[buf])), "r"(parity) : "memory");
        if (!done && clock64() - t_wait > kWaitCycles) break;
      }
      if (!done) {
        if (lane == 0) atomicOr(p.status, FASA_DEV_TIMEOUT);
        timed_out = true;
      }
      timed_out = __syncthreads_or(timed_out ? 1 : 0) != 0;             // leave together
    }
    if (timed_out) return;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    // ---- epilogue: thread r owns token row r of the tile; 16 columns = two heads x 8 queries ----
    const int j = mt * kBM + tid;
    const int G = p.group, T = p.q_len;
    float red[8];                                   // one value per query of the block
#pragma unroll
    for (int t = 0; t < 8; ++t) red[t] = MAXRED ? -INFINITY : 0.f;
#pragma unroll
    for (int c16 = 0; c16 < 4; ++c16) {
      if (c16 * 16 < p.n_cols) {                    // uniform
        float v[16];
        tmem_ld16(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * acc_cols + c16 * 16), v);
        const bool second = 2 * c16 + 1 < G;        // (an odd group leaves the last 8 columns empty)
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          if (MAXRED) red[t] = fmaxf(red[t], second ? fmaxf(v[t], v[8 + t]) : v[t]);
          else red[t] += v[t] + v[8 + t];
        }
      }
    }
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      if (t < T && j < len - (T - 1 - t))
        score_row0[t * score_stride + j] = red[t] + 0.0f;   // (-0 becomes +0)
    }
  };
  fetch(a0, mt0);
  scatter(a0, 0);
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();
  if (tid == 0) product(0);
  if (mt0 + 1 < mt1) fetch(a1, mt0 + 1);
  if (mt0 + 2 < mt1) fetch(a0, mt0 + 2);
  for (int mt = mt0; mt < mt1 && !timed_out; mt += 2) {                 // uniform over the CTA
    tile_step(mt, a1);
    if (mt + 1 < mt1 && !timed_out) tile_step(mt + 1, a0);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(2 * acc_cols) : "memory");
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

}  // namespace

extern "C" int32_t fasa_fc_score_batched(fasa_ctx_t* ctx, const void* q, const void* proxy_k,
                                         const int32_t* seq_lens, int32_t q_len, float* scores, void* stream) {
  if (!ctx || !q || !proxy_k || !seq_lens || !scores || !fasa_pages_ready(ctx)) return FASA_ERR_INVALID_ARG;
  if (!aligned16(proxy_k) || ((uintptr_t)q & 1) || ((uintptr_t)scores & 3)) return FASA_ERR_INVALID_ARG;
  if (q_len < 1 || q_len > FASA_MAX_QLEN) return FASA_ERR_UNSUPPORTED;
  const fasa_config_t& c = ctx->cfg;
  if ((long long)c.batch * q_len * ctx->n_sets > 65535) return FASA_ERR_UNSUPPORTED;
  BatchedParams p;
  p.q = (const uint16_t*)q; p.proxy = (const unsigned char*)proxy_k; p.seq_lens = seq_lens; p.chan = ctx->d_chan;
  p.scores = scores; p.status = ctx->d_status;
  p.n_q_heads = c.n_q_heads; p.n_kv_heads = c.n_kv_heads; p.n_sets = ctx->n_sets; p.group = ctx->sel_heads;
  p.max_len = c.max_len; p.chunks = ctx->chunks; p.q_len = q_len;
  p.n_cols = (8 * ctx->sel_heads + 15) / 16 * 16;      // 8 columns per head of the set
  p.max_reduce = c.group_reduce;
  p.pm = fasa_page_map(ctx);
  const int units = c.batch * ctx->n_sets;
  const int m_tiles = (c.max_len + kBM - 1) / kBM;
  const int chunks_pad = (ctx->chunks + 1) & ~1;
  const int nb = (ctx->chunks + 1) / 2;                // 16-channel blocks per tile, the 8-channel one included
  // shared memory: two A buffers and B; at least 1/8 (1/4 with the wide accumulators) of an SM's, so
  // that the CTAs of an SM together never ask for more than its 512 columns of tensor memory
  const int acc_cols = p.n_cols <= 32 ? 32 : 64;
  const int ctas_per_sm = 512 / (2 * acc_cols);
  size_t smem = (size_t)(2 * kBM + p.n_cols) * chunks_pad * 16;
  const size_t floor_smem = (size_t)(227 * 1024) / (ctas_per_sm + 1) + 1024;
  if (smem < floor_smem) smem = floor_smem;
  // one wave of CTAs where the tiles allow it: a unit's tiles are cut into as many runs as fit
  const int slots = ctas_per_sm * ctx->n_sm;
  const int runs = units >= slots ? 1 : slots / units;
  p.tiles_per_cta = (m_tiles + runs - 1) / runs;
  if (p.tiles_per_cta < 4) p.tiles_per_cta = m_tiles < 4 ? m_tiles : 4;
  dim3 grid((unsigned)((m_tiles + p.tiles_per_cta - 1) / p.tiles_per_cta), (unsigned)units);
  auto go = [&](auto fn) -> cudaError_t {
    cudaError_t e = cudaFuncSetAttribute((const void*)fn, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
    if (e != cudaSuccess) return e;
    fn<<<grid, kBT, smem, (cudaStream_t)stream>>>(p);
    return cudaGetLastError();
  };
  const bool mx = c.group_reduce != 0;
  const int kb_of = nb <= 1 ? 1 : (nb <= 2 ? 2 : (nb <= 4 ? 4 : 8));
  const bool exact = ctx->chunks % 2 == 0 && ctx->chunks / 2 == kb_of && c.page_size == 0;
  auto pick = [&](auto kb_tag) -> cudaError_t {
    constexpr int K = decltype(kb_tag)::value;
    if (exact) return mx ? go(fc_score_batched_kernel<K, true, true>) : go(fc_score_batched_kernel<K, false, true>);
    return mx ? go(fc_score_batched_kernel<K, true, false>) : go(fc_score_batched_kernel<K, false, false>);
  };
  cudaError_t e;
  if (kb_of == 1) e = pick(std::integral_constant<int, 1>{});
  else if (kb_of == 2) e = pick(std::integral_constant<int, 2>{});
  else if (kb_of == 4) e = pick(std::integral_constant<int, 4>{});
  else e = pick(std::integral_constant<int, 8>{});
  FASA_CUDA_TRY(ctx, e);
  FASA_LAUNCH_CHECK(ctx);
  return FASA_OK;
}

// TopK-I of every query of the block: rows (sequence, query, index set) of the score buffer,
// each with the length its query sees.
extern "C" int32_t fasa_topk_batched(fasa_ctx_t* ctx, const float* scores, const int32_t* seq_lens, int32_t q_len,
                                     int32_t budget, int32_t n_sel_max, int32_t* idx, int32_t* n_sel, void* stream) {
  if (!ctx || !scores || !seq_lens || !idx || !n_sel || budget == 0 || budget < -1000 || n_sel_max <= 0)
    return FASA_ERR_INVALID_ARG;
  if (q_len < 1 || q_len > FASA_MAX_QLEN) return FASA_ERR_UNSUPPORTED;
  if (!(ctx->fused_cs > 0)) return FASA_ERR_UNSUPPORTED;            // needs the cluster kernel's selection phases
  if ((long long)ctx->cfg.batch * q_len * ctx->n_sets > 65535) return FASA_ERR_UNSUPPORTED;
  return fasa_fused_topk_rows(ctx, scores, seq_lens, budget, n_sel_max, idx, n_sel, q_len * ctx->n_sets,
                              ctx->cfg.n_sink, ctx->cfg.n_recent, (cudaStream_t)stream, q_len);
}

extern "C" int32_t fasa_decode_step_batched(fasa_ctx_t* ctx, const void* q, const void* k_cache, const void* v_cache,
                                            const void* proxy_k, const int32_t* seq_lens, int32_t q_len, int32_t budget,
                                            int32_t n_sel_max, float* scores, int32_t* idx, int32_t* n_sel, float* out,
                                            float* lse, void* workspace, void* stream) {
  if (!scores || !workspace) return FASA_ERR_INVALID_ARG;
  if (!ctx || !q || !k_cache || !v_cache || !idx || !n_sel || !out || !aligned16(q) || !aligned16(k_cache) ||
      !aligned16(v_cache) || ((uintptr_t)workspace & 255) || n_sel_max <= 0 || budget == 0 || budget < -1000)
    return FASA_ERR_INVALID_ARG;                                    // (everything the later calls would refuse)
  if (!(ctx->fused_cs > 0)) return FASA_ERR_UNSUPPORTED;
  int32_t st = fasa_fc_score_batched(ctx, q, proxy_k, seq_lens, q_len, scores, stream);
  if (st != FASA_OK) return st;
  st = fasa_topk_batched(ctx, scores, seq_lens, q_len, budget, n_sel_max, idx, n_sel, stream);
  if (st != FASA_OK) return st;
  return fasa_sparse_decode_attn_batched(ctx, q, k_cache, v_cache, idx, n_sel, q_len, n_sel_max, out, lse, workspace, stream);
}
