// The memory-optimised variant (FASA-M, Algorithm 2) with the key cache SPLIT as the algorithm
// states it: the dominant part of every key (C_key^dom) is the GPU-resident proxy-K buffer, the
// non-dominant part (C_key^nondom) and the values (C_val) live in page-locked host memory.  Per
// step only the selected tokens' non-dominant key channels and value rows cross the host link
// (512 - 4 n_dom bytes per token instead of 512); the attention kernel Combines a key row in
// shared memory from its two homes (fasa_attn.cu, KSPLIT).
//
// k_nondom: bf16 [batch][n_kv_heads][max_len][128 - 2 n_dom], the channels of a key that are not
// among its head's dominant ones, in ascending channel order.  Needs n_dom to be a multiple of 4
// (the row is then a whole number of 16-byte chunks and the proxy row has no padding) and
// contiguous caches.
#include "fasa_common.cuh"
#include "fasa_score_core.cuh"

namespace {

constexpr int kSplitRows = 16;

// A CTA takes 16 rows of one (batch, KV head) unit.  APPEND: the rows are new tokens (k_src /
// v_src = [units][n_new][128]); their non-dominant channels go to k_nondom, their dominant pairs
// to the proxy, their value rows to v_cache, at rows old length + n; the last CTA of a sequence
// to report in stores the new length.  Otherwise: k_src is a full key cache ([units][max_len][128]
// through the K strides) and only k_nondom rows j < seq_lens[b] are written.
template <bool APPEND>
__global__ void __launch_bounds__(256)
split_rows_kernel(const uint16_t* __restrict__ k_src, const uint16_t* __restrict__ v_src, uint16_t* __restrict__ k_nondom,
                  uint16_t* __restrict__ v_cache, unsigned char* __restrict__ proxy, const int32_t* seq_lens,
                  int32_t* seq_lens_w, int32_t* arrive, const int16_t* __restrict__ chan,
                  const int16_t* __restrict__ ndchan, int32_t* __restrict__ status, int n_new, int n_kv_heads,
                  int max_len, int chunks, int nd, int64_t ksb, int64_t ksh, int64_t kst, int64_t vsb, int64_t vsh,
                  int64_t vst, const fasa_resident res) {
  __shared__ __align__(16) uint16_t s_k[kSplitRows][FASA_HEAD_DIM];
  const int u = blockIdx.y, h = u % n_kv_heads, b = u / n_kv_heads, tid = threadIdx.x;
  const int len = clamp_len(seq_lens[b], max_len, status);
  const int n0 = blockIdx.x * kSplitRows;
  if (APPEND) {
    __syncthreads();                                     // every thread has read the old length
    if (tid == 0) {
      __threadfence();
      if (atomicAdd(&arrive[b], 1) == n_kv_heads * (int)gridDim.x - 1) {
        const int grown = len + n_new;
        seq_lens_w[b] = grown > max_len ? max_len : grown;
        arrive[b] = 0;
      }
    }
  }
  const int n_src = APPEND ? n_new : len;
  const int first = APPEND ? len + n0 : n0;              // destination row of source row n0
  if (n0 >= n_src) return;
  // Resident rows (APPEND): an appended row that is a sink position, or one of the last n_recent of
  // the grown sequence, is also kept on the GPU, assembled as the attention kernel reads it.
  const int grown_len = min(max_len, len + n_new);
  auto res_slot_of = [&](int pos) -> int {
    if (!APPEND || res.tags == nullptr || pos >= max_len) return -1;
    if (pos >= res.n_sink && pos < grown_len - res.n_recent) return -1;
    return fasa_resident_slot(res, pos);
  };
  uint16_t* res_unit = APPEND && res.tags ? res.rows + (int64_t)u * res.slots * 2 * FASA_HEAD_DIM : nullptr;
  if (APPEND && first + min(kSplitRows, n_src - n0) > max_len && tid == 0) atomicOr(status, FASA_DEV_APPEND_FULL);
  const int r = tid >> 4, c8 = (tid & 15) * 8;
  const bool row_ok = n0 + r < n_src && first + r < max_len;
  uint4 kx = make_uint4(0u, 0u, 0u, 0u);
  if (row_ok) {
    const uint16_t* ks = APPEND ? k_src + ((int64_t)u * n_new + n0 + r) * FASA_HEAD_DIM
                                : k_src + b * ksb + h * ksh + (int64_t)(first + r) * kst;
    kx = *reinterpret_cast<const uint4*>(ks + c8);
    if (APPEND) {
      const uint4 vx = *reinterpret_cast<const uint4*>(v_src + ((int64_t)u * n_new + n0 + r) * FASA_HEAD_DIM + c8);
      *reinterpret_cast<uint4*>(v_cache + b * vsb + h * vsh + (int64_t)(first + r) * vst + c8) = vx;
      const int slot = res_slot_of(first + r);
      if (slot >= 0) {
        *reinterpret_cast<uint4*>(res_unit + (int64_t)slot * 2 * FASA_HEAD_DIM + FASA_HEAD_DIM + c8) = vx;
        if (c8 == 0) res.tags[(int64_t)u * res.slots_pad + slot] = first + r;
      }
    }
  }
  *reinterpret_cast<uint4*>(&s_k[r][c8]) = kx;
  __syncthreads();
  // non-dominant channels, two per thread and store
  const int16_t* nch = ndchan + h * nd;
  uint16_t* dst_unit = k_nondom + (int64_t)u * max_len * nd;
  for (int i = tid; i < kSplitRows * (nd / 2); i += 256) {
    const int rr = i / (nd / 2), w = i % (nd / 2);
    if (n0 + rr >= n_src || first + rr >= max_len) continue;
    const uint32_t lo = s_k[rr][nch[2 * w]], hi = s_k[rr][nch[2 * w + 1]];
    *reinterpret_cast<uint32_t*>(dst_unit + (int64_t)(first + rr) * nd + 2 * w) = lo | (hi << 16);
    const int slot = res_slot_of(first + rr);
    if (slot >= 0) *reinterpret_cast<uint32_t*>(res_unit + (int64_t)slot * 2 * FASA_HEAD_DIM + 2 * w) = lo | (hi << 16);
  }
  if (APPEND) {
    const ProxyGeom pg = proxy_geom(chunks);
    const int words = 4 * chunks;
    const int16_t* ch = chan + h * chunks * 8;
    unsigned char* punit = proxy + (int64_t)u * ((max_len + 15) >> 4) * pg.tile_bytes;
    for (int i = tid; i < kSplitRows * words; i += 256) {
      const int rr = i / words, w = i % words;
      if (n0 + rr >= n_src || first + rr >= max_len) continue;
      const uint32_t lo = s_k[rr][ch[2 * w]], hi = s_k[rr][ch[2 * w + 1]];
      *reinterpret_cast<uint32_t*>(punit + proxy_word_offset(pg, first + rr, w)) = lo | (hi << 16);
      const int slot = res_slot_of(first + rr);
      if (slot >= 0) *reinterpret_cast<uint32_t*>(res_unit + (int64_t)slot * 2 * FASA_HEAD_DIM + nd + 2 * w) = lo | (hi << 16);
    }
  }
}

// Fills the resident rows of one (batch, KV head) unit from the split caches as they stand: the
// sink positions and the last n_recent positions of the sequence.  One warp per row.
__global__ void __launch_bounds__(256)
resident_build_kernel(const uint16_t* __restrict__ k_nondom, const uint16_t* __restrict__ v_cache,
                      const unsigned char* __restrict__ proxy, const int32_t* __restrict__ seq_lens,
                      int32_t* __restrict__ status, int n_kv_heads, int max_len, int chunks, int nd, int64_t vsb,
                      int64_t vsh, int64_t vst, const fasa_resident res) {
  const int u = blockIdx.x, h = u % n_kv_heads, b = u / n_kv_heads;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int len = clamp_len(seq_lens[b], max_len, status);
  const ProxyGeom pg = proxy_geom(chunks);
  const unsigned char* punit = proxy + (int64_t)u * ((max_len + 15) >> 4) * pg.tile_bytes;
  for (int s = warp; s < res.slots; s += 8) {
    // the position this slot holds now, if any
    int pos = -1;
    if (s < res.n_sink) {
      if (s < len) pos = s;
    } else if (len > res.n_sink) {
      const int lo = max(res.n_sink, len - res.n_recent);       // first position of the window
      const int cand = lo + ((s - res.n_sink) - (lo - res.n_sink) % res.n_recent + res.n_recent) % res.n_recent;
      if (cand < len) pos = cand;
    }
    uint16_t* row = res.rows + ((int64_t)u * res.slots + s) * 2 * FASA_HEAD_DIM;
    if (pos >= 0) {
      for (int c = lane; c < nd / 2; c += 32)
        reinterpret_cast<uint32_t*>(row)[c] = reinterpret_cast<const uint32_t*>(k_nondom + ((int64_t)u * max_len + pos) * nd)[c];
      for (int w = lane; w < 4 * chunks; w += 32)
        reinterpret_cast<uint32_t*>(row + nd)[w] = *reinterpret_cast<const uint32_t*>(punit + proxy_word_offset(pg, pos, w));
      for (int c = lane; c < FASA_HEAD_DIM / 2; c += 32)
        reinterpret_cast<uint32_t*>(row + FASA_HEAD_DIM)[c] =
            reinterpret_cast<const uint32_t*>(v_cache + b * vsb + h * vsh + (int64_t)pos * vst)[c];
    }
    if (lane == 0) res.tags[(int64_t)u * res.slots_pad + s] = pos;
  }
}

bool split_ok(const fasa_ctx* ctx) { return ctx->d_ndchan != nullptr && ctx->cfg.page_size == 0; }
bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

}  // namespace

extern "C" int32_t fasa_m_nondom_row_elems(int32_t n_dom) {
  if (n_dom < 1 || n_dom >= FASA_HEAD_DIM / 2 || n_dom % 4 != 0) return 0;
  return FASA_HEAD_DIM - 2 * n_dom;
}

extern "C" int32_t fasa_m_split(fasa_ctx_t* ctx, const void* k_cache, void* k_nondom, const int32_t* seq_lens,
                                void* stream) {
  if (!ctx || !k_cache || !k_nondom || !seq_lens || !aligned16(k_cache) || !aligned16(k_nondom)) return FASA_ERR_INVALID_ARG;
  if (!split_ok(ctx)) return FASA_ERR_UNSUPPORTED;
  const fasa_config_t& c = ctx->cfg;
  dim3 grid((unsigned)((c.max_len + kSplitRows - 1) / kSplitRows), (unsigned)(c.batch * c.n_kv_heads));
  split_rows_kernel<false><<<grid, 256, 0, (cudaStream_t)stream>>>(
      (const uint16_t*)k_cache, nullptr, (uint16_t*)k_nondom, nullptr, nullptr, seq_lens, nullptr, nullptr, ctx->d_chan,
      ctx->d_ndchan, ctx->d_status, 0, c.n_kv_heads, c.max_len, ctx->chunks, FASA_HEAD_DIM - 2 * c.n_dom, c.k_stride_b,
      c.k_stride_h, c.k_stride_t, c.v_stride_b, c.v_stride_h, c.v_stride_t, fasa_resident{});
  FASA_LAUNCH_CHECK(ctx);
  return FASA_OK;
}

extern "C" int32_t fasa_m_kv_append(fasa_ctx_t* ctx, void* k_nondom, void* v_cache, void* proxy_k, int32_t* seq_lens,
                                    const void* k_new, const void* v_new, int32_t n_new, void* stream) {
  if (!ctx || !k_nondom || !v_cache || !proxy_k || !seq_lens || !k_new || !v_new || n_new <= 0) return FASA_ERR_INVALID_ARG;
  if (!aligned16(k_nondom) || !aligned16(v_cache) || !aligned16(proxy_k) || !aligned16(k_new) || !aligned16(v_new))
    return FASA_ERR_INVALID_ARG;
  if (!split_ok(ctx)) return FASA_ERR_UNSUPPORTED;
  const fasa_config_t& c = ctx->cfg;
  dim3 grid((unsigned)((n_new + kSplitRows - 1) / kSplitRows), (unsigned)(c.batch * c.n_kv_heads));
  split_rows_kernel<true><<<grid, 256, 0, (cudaStream_t)stream>>>(
      (const uint16_t*)k_new, (const uint16_t*)v_new, (uint16_t*)k_nondom, (uint16_t*)v_cache, (unsigned char*)proxy_k,
      seq_lens, seq_lens, ctx->d_arrive, ctx->d_chan, ctx->d_ndchan, ctx->d_status, n_new, c.n_kv_heads, c.max_len,
      ctx->chunks, FASA_HEAD_DIM - 2 * c.n_dom, c.k_stride_b, c.k_stride_h, c.k_stride_t, c.v_stride_b, c.v_stride_h,
      c.v_stride_t, fasa_resident_of(ctx));
  FASA_LAUNCH_CHECK(ctx);
  return FASA_OK;
}

// ---- GPU-resident copies of the rows every step attends to -------------------------------------
fasa_resident fasa_resident_of(const fasa_ctx* ctx) {
  fasa_resident r;
  memset(&r, 0, sizeof(r));
  if (ctx->m_resident == nullptr) return r;
  const fasa_config_t& c = ctx->cfg;
  r.n_sink = c.n_sink;
  r.n_recent = c.n_recent;
  r.slots = c.n_sink + c.n_recent;
  r.slots_pad = (r.slots + 3) & ~3;
  r.tags = (int32_t*)ctx->m_resident;
  r.rows = (uint16_t*)((unsigned char*)ctx->m_resident + (size_t)c.batch * c.n_kv_heads * r.slots_pad * sizeof(int32_t));
  return r;
}

extern "C" int64_t fasa_m_resident_bytes(const fasa_ctx_t* ctx) {
  if (!ctx || !split_ok(ctx)) return 0;
  const fasa_config_t& c = ctx->cfg;
  const int64_t slots = c.n_sink + c.n_recent, slots_pad = (slots + 3) & ~3;
  if (slots == 0) return 0;
  return (int64_t)c.batch * c.n_kv_heads * (slots_pad * 4 + slots * 2 * FASA_HEAD_DIM * 2);
}

extern "C" int32_t fasa_m_set_resident(fasa_ctx_t* ctx, void* resident, void* stream) {
  if (!ctx) return FASA_ERR_INVALID_ARG;
  if (resident == nullptr) {
    ctx->m_resident = nullptr;
    return FASA_OK;
  }
  if (!aligned16(resident)) return FASA_ERR_INVALID_ARG;
  if (fasa_m_resident_bytes(ctx) == 0) return FASA_ERR_UNSUPPORTED;
  const fasa_config_t& c = ctx->cfg;
  const size_t tag_bytes = (size_t)c.batch * c.n_kv_heads * (((size_t)c.n_sink + c.n_recent + 3) & ~(size_t)3) * sizeof(int32_t);
  FASA_CUDA_TRY(ctx, cudaMemsetAsync(resident, 0xff, tag_bytes, (cudaStream_t)stream));   // every tag -1: nothing held
  ctx->m_resident = resident;
  return FASA_OK;
}

extern "C" int32_t fasa_m_resident_build(fasa_ctx_t* ctx, const void* k_nondom, const void* v_cache, const void* proxy_k,
                                         const int32_t* seq_lens, void* stream) {
  if (!ctx || !k_nondom || !v_cache || !proxy_k || !seq_lens || !aligned16(k_nondom) || !aligned16(v_cache) ||
      !aligned16(proxy_k))
    return FASA_ERR_INVALID_ARG;
  if (!split_ok(ctx) || ctx->m_resident == nullptr) return FASA_ERR_UNSUPPORTED;
  const fasa_config_t& c = ctx->cfg;
  resident_build_kernel<<<(unsigned)(c.batch * c.n_kv_heads), 256, 0, (cudaStream_t)stream>>>(
      (const uint16_t*)k_nondom, (const uint16_t*)v_cache, (const unsigned char*)proxy_k, seq_lens, ctx->d_status,
      c.n_kv_heads, c.max_len, ctx->chunks, FASA_HEAD_DIM - 2 * c.n_dom, c.v_stride_b, c.v_stride_h, c.v_stride_t,
      fasa_resident_of(ctx));
  FASA_LAUNCH_CHECK(ctx);
  return FASA_OK;
}

extern "C" int32_t fasa_m_sparse_decode_attn(fasa_ctx_t* ctx, const void* q, const void* k_nondom, const void* v_cache,
                                             const void* proxy_k, const int32_t* idx, const int32_t* n_sel,
                                             int32_t n_sel_max, float* out, float* lse, void* workspace, void* stream) {
  if (!ctx || !q || !k_nondom || !v_cache || !proxy_k || !idx || !n_sel || !out || !workspace || n_sel_max <= 0)
    return FASA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_nondom) || !aligned16(v_cache) || !aligned16(proxy_k) || ((uintptr_t)workspace & 255))
    return FASA_ERR_INVALID_ARG;
  if (!split_ok(ctx) || !ctx->use_fused) return FASA_ERR_UNSUPPORTED;
  return fasa_attn_split_keys(ctx, q, k_nondom, v_cache, proxy_k, idx, n_sel, n_sel_max, out, lse, workspace,
                              (cudaStream_t)stream);
}

extern "C" int32_t fasa_m_decode_step(fasa_ctx_t* ctx, const void* q, const void* k_new, const void* v_new, void* k_nondom,
                                      void* v_cache, void* proxy_k, int32_t* seq_lens, int32_t budget, int32_t n_sel_max,
                                      float* scores, int32_t* idx, int32_t* n_sel, float* out, float* lse, void* workspace,
                                      void* stream) {
  if (!ctx || !q || !k_nondom || !v_cache || !proxy_k || !seq_lens || !idx || !n_sel || !out || !workspace ||
      budget == 0 || budget < -1000 || n_sel_max <= 0 || (k_new == nullptr) != (v_new == nullptr))
    return FASA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k_nondom) || !aligned16(v_cache) || !aligned16(proxy_k) || !aligned16(k_new) ||
      !aligned16(v_new) || ((uintptr_t)workspace & 255) || (scores && ((uintptr_t)scores & 3)))
    return FASA_ERR_INVALID_ARG;
  if (!split_ok(ctx) || !(ctx->use_fused && ctx->fused_step_ok && ctx->fused_cs > 0)) return FASA_ERR_UNSUPPORTED;
  int32_t st;
  if (k_new) {                                    // Algorithm 2's order: UpdateCache (Split) first
    st = fasa_m_kv_append(ctx, k_nondom, v_cache, proxy_k, seq_lens, k_new, v_new, 1, stream);
    if (st != FASA_OK) return st;
  }
  // TIP + TopK-I on the GPU-resident proxy (the key and value caches are not touched)
  st = fasa_fused_launch(ctx, q, proxy_k, proxy_k, proxy_k, seq_lens, budget, n_sel_max, scores, idx, n_sel, nullptr,
                         nullptr, nullptr, nullptr, (cudaStream_t)stream, false);
  if (st != FASA_OK) return st;
  return fasa_attn_split_keys(ctx, q, k_nondom, v_cache, proxy_k, idx, n_sel, n_sel_max, out, lse, workspace,
                              (cudaStream_t)stream);
}
