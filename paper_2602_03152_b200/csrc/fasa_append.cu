// Cache update: K/V rows plus the packed dominant-FC proxy rows (Algorithm 2: Split,
// UpdateCache), and the one-off proxy build from an existing key cache.
#include "fasa_common.cuh"
#include "fasa_score_core.cuh"

namespace {

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
                 int32_t* arrive) {
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
  if (t < 16) {
    uint4 x = *reinterpret_cast<const uint4*>(ksrc + t * 8);
    *reinterpret_cast<uint4*>(k_cache + b * ksb + h * ksh + pos * kst + t * 8) = x;
  } else if (t < 32) {
    const int c = t - 16;
    uint4 x = *reinterpret_cast<const uint4*>(v_new + (int64_t)row * FASA_HEAD_DIM + c * 8);
    *reinterpret_cast<uint4*>(v_cache + b * vsb + h * vsh + pos * vst + c * 8) = x;
  } else if (t - 32 < 4 * chunks) {
    const int w = t - 32;
    const ProxyGeom pg = proxy_geom(chunks);
    const int16_t* ch = chan + h * chunks * 8 + 2 * w;
    const int c0 = ch[0], c1 = ch[1];
    const uint32_t lo = c0 >= 0 ? ksrc[c0] : 0u;
    const uint32_t hi = c1 >= 0 ? ksrc[c1] : 0u;
    unsigned char* unit = proxy + (int64_t)u * ((max_len + 15) >> 4) * pg.tile_bytes;
    *reinterpret_cast<uint32_t*>(unit + proxy_word_offset(pg, pos, w)) = lo | (hi << 16);
  }
}

// One thread per proxy word of rows 0 .. seq_lens[b]-1.
__global__ void __launch_bounds__(256)
proxy_build_kernel(const uint16_t* __restrict__ k_cache, unsigned char* __restrict__ proxy,
                   const int32_t* __restrict__ seq_lens, const int16_t* __restrict__ chan,
                   int32_t* __restrict__ status, int n_kv_heads, int max_len, int chunks,
                   int64_t ksb, int64_t ksh, int64_t kst) {
  const int u = blockIdx.y;
  const int h = u % n_kv_heads;
  const int b = u / n_kv_heads;
  const int len = clamp_len(seq_lens[b], max_len, status);
  const int words = 4 * chunks;
  const int64_t item = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int j = (int)(item / words);
  const int w = (int)(item % words);
  if (j >= len) return;
  const ProxyGeom pg = proxy_geom(chunks);
  const int16_t* ch = chan + h * chunks * 8 + 2 * w;
  const uint16_t* ksrc = k_cache + b * ksb + h * ksh + (int64_t)j * kst;
  const int c0 = ch[0], c1 = ch[1];
  const uint32_t lo = c0 >= 0 ? ksrc[c0] : 0u;
  const uint32_t hi = c1 >= 0 ? ksrc[c1] : 0u;
  unsigned char* unit = proxy + (int64_t)u * ((max_len + 15) >> 4) * pg.tile_bytes;
  *reinterpret_cast<uint32_t*>(unit + proxy_word_offset(pg, j, w)) = lo | (hi << 16);
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

}  // namespace

extern "C" int32_t fasa_kv_append(fasa_ctx_t* ctx, void* k_cache, void* v_cache, void* proxy_k,
                                  int32_t* seq_lens, const void* k_new, const void* v_new,
                                  int32_t n_new, void* stream) {
  if (!ctx || !k_cache || !v_cache || !proxy_k || !seq_lens || !k_new || !v_new || n_new <= 0)
    return FASA_ERR_INVALID_ARG;
  if (!aligned16(k_cache) || !aligned16(v_cache) || !aligned16(proxy_k) || !aligned16(k_new) ||
      !aligned16(v_new))
    return FASA_ERR_INVALID_ARG;
  const fasa_config_t& c = ctx->cfg;
  long long n_rows = (long long)c.batch * c.n_kv_heads * n_new;
  if (n_rows > (1ll << 30)) return FASA_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  kv_append_kernel<<<(unsigned)((n_rows + 1) / 2), 256, 0, s>>>(
      (uint16_t*)k_cache, (uint16_t*)v_cache, (unsigned char*)proxy_k, seq_lens, (const uint16_t*)k_new,
      (const uint16_t*)v_new, ctx->d_chan, ctx->d_status, (int)n_rows, n_new, c.n_kv_heads,
      c.max_len, ctx->chunks, c.k_stride_b, c.k_stride_h, c.k_stride_t, c.v_stride_b,
      c.v_stride_h, c.v_stride_t, seq_lens, ctx->d_arrive);
  FASA_LAUNCH_CHECK(ctx);
  return FASA_OK;
}

extern "C" int32_t fasa_proxy_build(fasa_ctx_t* ctx, const void* k_cache, void* proxy_k,
                                    const int32_t* seq_lens, void* stream) {
  if (!ctx || !k_cache || !proxy_k || !seq_lens) return FASA_ERR_INVALID_ARG;
  if (!aligned16(k_cache) || !aligned16(proxy_k)) return FASA_ERR_INVALID_ARG;
  const fasa_config_t& c = ctx->cfg;
  long long items = (long long)c.max_len * ctx->chunks * 4;
  dim3 grid((unsigned)((items + 255) / 256), (unsigned)(c.batch * c.n_kv_heads));
  proxy_build_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>(
      (const uint16_t*)k_cache, (unsigned char*)proxy_k, seq_lens, ctx->d_chan, ctx->d_status,
      c.n_kv_heads, c.max_len, ctx->chunks, c.k_stride_b, c.k_stride_h, c.k_stride_t);
  FASA_LAUNCH_CHECK(ctx);
  return FASA_OK;
}
