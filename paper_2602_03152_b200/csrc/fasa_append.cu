// Cache update: K/V rows plus the packed dominant-FC proxy rows (Algorithm 2: Split,
// UpdateCache), and the one-off proxy build from an existing key cache.
#include "fasa_common.cuh"
#include "fasa_score_core.cuh"

namespace {

// Where row `pos` of (sequence b, KV head h) is written.  Paged caches: a table entry outside
// the pool drops the row (ok = false) instead of redirecting the write.
struct RowDst {
  int64_t k, v;          // element offsets into the K and V caches
  int64_t proxy_unit;    // byte offset of the (page, head) or (sequence, head) proxy block
  int proxy_row;         // row inside that block
  bool ok;
};
__device__ __forceinline__ RowDst row_dst(const PageMap& m, int b, int h, int n_kv_heads, int pos, int max_len,
                                          int tile_bytes, int64_t ksb, int64_t ksh, int64_t kst, int64_t vsb,
                                          int64_t vsh, int64_t vst, int32_t* status) {
  RowDst d;
  d.ok = true;
  if (m.table == nullptr) {
    d.k = b * ksb + h * ksh + (int64_t)pos * kst;
    d.v = b * vsb + h * vsh + (int64_t)pos * vst;
    d.proxy_unit = (int64_t)(b * n_kv_heads + h) * ((max_len + 15) >> 4) * tile_bytes;
    d.proxy_row = pos;
    return d;
  }
  const int page = page_of(m, b, pos);
  if (!page_ok(m, page)) {
    atomicOr(status, FASA_DEV_PAGE_CLAMPED);
    d.ok = false;
    d.k = d.v = d.proxy_unit = 0;
    d.proxy_row = 0;
    return d;
  }
  const int in_page = pos & ((1 << m.shift) - 1);
  d.k = page * ksb + h * ksh + (int64_t)in_page * kst;
  d.v = page * vsb + h * vsh + (int64_t)in_page * vst;
  d.proxy_unit = ((int64_t)page * n_kv_heads + h) * (1 << (m.shift - 4)) * tile_bytes;
  d.proxy_row = in_page;
  return d;
}

// 128 threads per appended row: 16 copy the K row, 16 the V row (16 bytes each), up to 64
// write the proxy words (one dominant FC = one 4-byte channel pair each) to their places in
// the tiled proxy layout.
__global__ void __launch_bounds__(256)
kv_append_kernel(uint16_t* __restrict__ k_cache, uint16_t* __restrict__ v_cache,
                 unsigned char* __restrict__ proxy, const int32_t* seq_lens /* same memory as seq_lens_w */,
                 const uint16_t* __restrict__ k_new, const uint16_t* __restrict__ v_new,
                 const int16_t* __restrict__ chan, int32_t* __restrict__ status, int n_rows,
                 int n_new, int n_kv_heads, int max_len, int chunks, int64_t ksb, int64_t ksh,
                 int64_t kst, int64_t vsb, int64_t vsh, int64_t vst, int32_t* seq_lens_w,
                 int32_t* arrive, const PageMap pm) {
  const int row = blockIdx.x * 2 + (threadIdx.x >> 7);
  const bool live = row < n_rows;
  const int t = threadIdx.x & 127;
  const int n = live ? row % n_new : 0;
  const int u = live ? row / n_new : 0;  // unit = b * n_kv_heads + h
  const int h = u % n_kv_heads;
  const int b = u / n_kv_heads;
  const int len = live ? clamp_len(seq_lens[b], max_len, status) : 0;
  // The length is updated here too: once every thread of the CTA has read the old value
  // (barrier), one thread per row reports in; the last of the sequence's n_kv_heads * n_new
  // rows to do so stores the new length.  Nobody waits on the counter.
  __syncthreads();
  if (live && t == 0) {
    __threadfence();
    if (atomicAdd(&arrive[b], 1) == n_kv_heads * n_new - 1) {
      const int grown = len + n_new;
      seq_lens_w[b] = grown > max_len ? max_len : grown;
      arrive[b] = 0;
    }
  }
  if (!live) return;
  const int pos = len + n;
  if (pos >= max_len) {
    if (t == 0) atomicOr(status, FASA_DEV_APPEND_FULL);
    return;
  }
  const uint16_t* ksrc = k_new + (int64_t)row * FASA_HEAD_DIM;
  const ProxyGeom pg = proxy_geom(chunks);
  const RowDst d = row_dst(pm, b, h, n_kv_heads, pos, max_len, pg.tile_bytes, ksb, ksh, kst, vsb, vsh, vst, status);
  if (!d.ok) return;
  if (t < 16) {
    uint4 x = *reinterpret_cast<const uint4*>(ksrc + t * 8);
    *reinterpret_cast<uint4*>(k_cache + d.k + t * 8) = x;
  } else if (t < 32) {
    const int c = t - 16;
    uint4 x = *reinterpret_cast<const uint4*>(v_new + (int64_t)row * FASA_HEAD_DIM + c * 8);
    *reinterpret_cast<uint4*>(v_cache + d.v + c * 8) = x;
  } else if (t - 32 < 4 * chunks) {
    const int w = t - 32;
    const int16_t* ch = chan + h * chunks * 8 + 2 * w;
    const int c0 = ch[0], c1 = ch[1];
    const uint32_t lo = c0 >= 0 ? ksrc[c0] : 0u;
    const uint32_t hi = c1 >= 0 ? ksrc[c1] : 0u;
    *reinterpret_cast<uint32_t*>(proxy + d.proxy_unit + proxy_word_offset(pg, d.proxy_row, w)) = lo | (hi << 16);
  }
}

// Many rows at once (a prompt's cache update, or the proxy build of a cache written by other
// means): a CTA takes 16 consecutive rows of one (batch, KV head) unit.  The 16 key rows go
// through shared memory once: from there they are copied to the cache with 16-byte stores and
// their dominant-FC pairs are picked for the proxy, so the keys are read from HBM a single time
// with full-width loads.  APPEND: source = the new rows, destination row = old length + n, and
// the CTA reports in on the sequence's arrival counter (the last one stores the new length).
// Otherwise: source = the cache rows themselves, j < seq_lens[b].
constexpr int kBulkRows = 16;
template <bool APPEND, bool PAGED>
__global__ void __launch_bounds__(256)
bulk_rows_kernel(uint16_t* k_cache, uint16_t* __restrict__ v_cache, unsigned char* __restrict__ proxy,
                 const int32_t* seq_lens /* same memory as seq_lens_w */, const uint16_t* __restrict__ k_new,
                 const uint16_t* __restrict__ v_new, const int16_t* __restrict__ chan,
                 int32_t* __restrict__ status, int n_new, int n_kv_heads, int max_len, int chunks,
                 int64_t ksb, int64_t ksh, int64_t kst, int64_t vsb, int64_t vsh, int64_t vst,
                 int32_t* seq_lens_w, int32_t* arrive, const PageMap pm_arg) {
  const PageMap pm = PAGED ? pm_arg : PageMap{nullptr, 0, 0, 0};   // contiguous: the translation folds away
  __shared__ __align__(16) uint16_t s_k[kBulkRows][FASA_HEAD_DIM];
  const int u = blockIdx.y;
  const int h = u % n_kv_heads;
  const int b = u / n_kv_heads;
  const int tid = threadIdx.x;
  const int len = clamp_len(seq_lens[b], max_len, status);
  const int n0 = blockIdx.x * kBulkRows;                 // first row of this CTA (new-row index, or cache row)
  if (APPEND) {
    __syncthreads();                                     // every thread has read the old length
    if (tid == 0) {
      const int total = n_kv_heads * (int)gridDim.x;
      if (atomicAdd(&arrive[b], 1) == total - 1) {
        const int grown = len + n_new;
        seq_lens_w[b] = grown > max_len ? max_len : grown;
        arrive[b] = 0;
      }
    }
  }
  const int n_src = APPEND ? n_new : len;                // rows that exist at the source
  const int first = APPEND ? len + n0 : n0;              // destination row of source row n0
  if (n0 >= n_src) return;
  if (APPEND && first + min(kBulkRows, n_src - n0) > max_len && tid == 0) atomicOr(status, FASA_DEV_APPEND_FULL);
  const int r = tid >> 4, c8 = (tid & 15) * 8;
  const ProxyGeom pg = proxy_geom(chunks);
  const bool row_ok = n0 + r < n_src && first + r < max_len;
  uint4 kx = make_uint4(0u, 0u, 0u, 0u);
  if (row_ok) {
    const RowDst d = row_dst(pm, b, h, n_kv_heads, first + r, max_len, pg.tile_bytes, ksb, ksh, kst, vsb, vsh, vst, status);
    if (d.ok) {
      const uint16_t* ksrc = APPEND ? k_new + ((int64_t)u * n_new + n0 + r) * FASA_HEAD_DIM : k_cache + d.k;
      kx = *reinterpret_cast<const uint4*>(ksrc + c8);
      if (APPEND) {
        *reinterpret_cast<uint4*>(k_cache + d.k + c8) = kx;
        *reinterpret_cast<uint4*>(v_cache + d.v + c8) =
            *reinterpret_cast<const uint4*>(v_new + ((int64_t)u * n_new + n0 + r) * FASA_HEAD_DIM + c8);
      }
    }
  }
  *reinterpret_cast<uint4*>(&s_k[r][c8]) = kx;
  __syncthreads();
  const int words = 4 * chunks;
  const int16_t* ch = chan + h * chunks * 8;
  for (int i = tid; i < kBulkRows * words; i += 256) {
    const int rr = i / words, w = i % words;
    if (n0 + rr >= n_src || first + rr >= max_len) continue;
    const RowDst d = row_dst(pm, b, h, n_kv_heads, first + rr, max_len, pg.tile_bytes, ksb, ksh, kst, vsb, vsh, vst, status);
    if (!d.ok) continue;
    const int c0 = ch[2 * w], c1 = ch[2 * w + 1];
    const uint32_t lo = c0 >= 0 ? s_k[rr][c0] : 0u;
    const uint32_t hi = c1 >= 0 ? s_k[rr][c1] : 0u;
    *reinterpret_cast<uint32_t*>(proxy + d.proxy_unit + proxy_word_offset(pg, d.proxy_row, w)) = lo | (hi << 16);
  }
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

}  // namespace

extern "C" int32_t fasa_kv_append(fasa_ctx_t* ctx, void* k_cache, void* v_cache, void* proxy_k,
                                  int32_t* seq_lens, const void* k_new, const void* v_new,
                                  int32_t n_new, void* stream) {
  if (!ctx || !k_cache || !v_cache || !proxy_k || !seq_lens || !k_new || !v_new || n_new <= 0)
    return FASA_ERR_INVALID_ARG;
  if (!aligned16(k_cache) || !aligned16(v_cache) || !aligned16(proxy_k) || !aligned16(k_new) ||
      !aligned16(v_new) || !fasa_pages_ready(ctx))
    return FASA_ERR_INVALID_ARG;
  const fasa_config_t& c = ctx->cfg;
  long long n_rows = (long long)c.batch * c.n_kv_heads * n_new;
  if (n_rows > (1ll << 30)) return FASA_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  if (n_new >= kBulkRows) {
    dim3 grid((unsigned)((n_new + kBulkRows - 1) / kBulkRows), (unsigned)(c.batch * c.n_kv_heads));
    auto bulk = c.page_size > 0 ? bulk_rows_kernel<true, true> : bulk_rows_kernel<true, false>;
    bulk<<<grid, 256, 0, s>>>(
        (uint16_t*)k_cache, (uint16_t*)v_cache, (unsigned char*)proxy_k, seq_lens, (const uint16_t*)k_new,
        (const uint16_t*)v_new, ctx->d_chan, ctx->d_status, n_new, c.n_kv_heads, c.max_len, ctx->chunks,
        c.k_stride_b, c.k_stride_h, c.k_stride_t, c.v_stride_b, c.v_stride_h, c.v_stride_t, seq_lens, ctx->d_arrive,
        fasa_page_map(ctx));
  } else {
    kv_append_kernel<<<(unsigned)((n_rows + 1) / 2), 256, 0, s>>>(
        (uint16_t*)k_cache, (uint16_t*)v_cache, (unsigned char*)proxy_k, seq_lens, (const uint16_t*)k_new,
        (const uint16_t*)v_new, ctx->d_chan, ctx->d_status, (int)n_rows, n_new, c.n_kv_heads,
        c.max_len, ctx->chunks, c.k_stride_b, c.k_stride_h, c.k_stride_t, c.v_stride_b,
        c.v_stride_h, c.v_stride_t, seq_lens, ctx->d_arrive, fasa_page_map(ctx));
  }
  FASA_LAUNCH_CHECK(ctx);
  return FASA_OK;
}

extern "C" int32_t fasa_proxy_build(fasa_ctx_t* ctx, const void* k_cache, void* proxy_k,
                                    const int32_t* seq_lens, void* stream) {
  if (!ctx || !k_cache || !proxy_k || !seq_lens) return FASA_ERR_INVALID_ARG;
  if (!aligned16(k_cache) || !aligned16(proxy_k) || !fasa_pages_ready(ctx)) return FASA_ERR_INVALID_ARG;
  const fasa_config_t& c = ctx->cfg;
  dim3 grid((unsigned)((c.max_len + kBulkRows - 1) / kBulkRows), (unsigned)(c.batch * c.n_kv_heads));
  auto build = c.page_size > 0 ? bulk_rows_kernel<false, true> : bulk_rows_kernel<false, false>;
  build<<<grid, 256, 0, (cudaStream_t)stream>>>(
      const_cast<uint16_t*>((const uint16_t*)k_cache), nullptr, (unsigned char*)proxy_k, seq_lens, nullptr, nullptr,
      ctx->d_chan, ctx->d_status, 0, c.n_kv_heads, c.max_len, ctx->chunks, c.k_stride_b, c.k_stride_h,
      c.k_stride_t, 0, 0, 0, nullptr, nullptr, fasa_page_map(ctx));
  FASA_LAUNCH_CHECK(ctx);
  return FASA_OK;
}

// ---- staging of the host-buffer step ---------------------------------------------------------
namespace {
// Copies three device-addressable (mapped host) buffers to device memory in one launch, 16 bytes
// per thread and iteration; sizes are multiples of 16 bytes.
__global__ void __launch_bounds__(256)
stage_copy_kernel(uint4* __restrict__ d0, const uint4* __restrict__ s0, int n0, uint4* __restrict__ d1,
                  const uint4* __restrict__ s1, uint4* __restrict__ d2, const uint4* __restrict__ s2, int n12) {
  const int total = n0 + 2 * n12;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    if (i < n0) d0[i] = s0[i];
    else if (i < n0 + n12) d1[i - n0] = s1[i - n0];
    else d2[i - n0 - n12] = s2[i - n0 - n12];
  }
}
}  // namespace

cudaError_t fasa_stage_from_mapped(void* dq, const void* sq, size_t q_bytes, void* dk, const void* sk, void* dv,
                                   const void* sv, size_t kv_bytes, cudaStream_t stream) {
  const int n0 = (int)(q_bytes / 16), n12 = (int)(kv_bytes / 16);
  const int total = n0 + 2 * n12;
  const int blocks = total < 256 * 256 ? (total + 255) / 256 : 256;
  stage_copy_kernel<<<blocks > 0 ? blocks : 1, 256, 0, stream>>>((uint4*)dq, (const uint4*)sq, n0, (uint4*)dk, (const uint4*)sk,
                                                               (uint4*)dv, (const uint4*)sv, n12);
  return cudaGetLastError();
}
