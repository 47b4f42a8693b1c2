// TIP scoring (Sec. 4.1): S[j] = reduce_g sum_{i in I_dom} alpha^(i)_g[j], streamed from the
// tiled proxy-K buffer.  Every proxy byte is read once: a warp fetches whole 512-byte blocks
// (16 bytes per lane, already in tensor-core fragment order) and turns 16 tokens x 16
// channels x up to 8 query heads into partial scores with one mma.sync; several tiles are in
// flight per warp, and the first batch of loads is issued before the sequence length, the
// channel table and the query are known.
#include <type_traits>

#include "fasa_common.cuh"
#include "fasa_score_core.cuh"

namespace {

constexpr int kScoreThreads = 256;
constexpr int kScoreWarps = kScoreThreads / 32;

// Tiles a warp handles per iteration (even; about 8 loads in flight per lane).
template <int KB>
struct TilesPerIter {
  static constexpr int value = KB == 1 ? 8 : (KB == 2 ? 4 : 2);
};

// KB = 16-channel blocks per tile rounded up to a power of two (1, 2, 4, 8).
template <int KB, bool MAXRED, bool PAGED>
__global__ void __launch_bounds__(kScoreThreads)
fc_score_kernel(const uint16_t* __restrict__ q, const unsigned char* __restrict__ proxy,
                const int32_t* __restrict__ seq_lens, const int16_t* __restrict__ chan,
                float* __restrict__ scores, int32_t* __restrict__ status, int n_q_heads,
                int n_kv_heads, int n_sets, int group, int max_len, int chunks, int tiles_per_cta,
                const PageMap pm) {
  constexpr int TPI = TilesPerIter<KB>::value;
  const int u = blockIdx.y;
  const SelUnit su = sel_unit(u, n_sets, group, n_q_heads, n_kv_heads);
  const int h = su.h;
  const int b = su.b;
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const ProxyGeom pg = proxy_geom(chunks);
  const int n_blocks = pg.n16 + pg.n8;
  const int tiles_alloc = (max_len + 15) >> 4;
  const int cta_tile0 = blockIdx.x * tiles_per_cta;
  const int cta_tile1 = min(tiles_alloc, cta_tile0 + tiles_per_cta);
  // (contiguous caches: plain pointer arithmetic, as compiled without the page map)
  const unsigned char* unit = proxy + (int64_t)su.kv * tiles_alloc * pg.tile_bytes;
  auto tile_at = [&](int T, int32_t* report) {
    if constexpr (PAGED) return proxy + proxy_tile_offset(pm, b, h, n_kv_heads, T, tiles_alloc, pg.tile_bytes, report);
    else return unit + (int64_t)T * pg.tile_bytes;
  };

  // First batch of loads: every tile up to max_len is allocated, so reading past the
  // sequence length is harmless and overlaps with the loads of the length and the query.
  int T = cta_tile0 + warp * TPI;
  uint4 a[TPI][KB];
#pragma unroll
  for (int j = 0; j < TPI; ++j)
    load_tile<KB>(a[j], tile_at(PAGED ? min(T + j, tiles_alloc - 1) : T + j, nullptr), pg, lane, T + j < cta_tile1);

  const int len = clamp_len(seq_lens[b], max_len, status);
  if (cta_tile0 * 16 >= len) return;
  const int row1 = min(len, cta_tile1 * 16);
  if constexpr (PAGED) {
#pragma unroll
    for (int j = 0; j < TPI; ++j)
      if ((T + j) * 16 < row1) proxy_tile_check(pm, b, T + j, status);
  }

  ScoreFrag<KB> f;
  load_score_b<KB>(f, q + su.q0 * FASA_HEAD_DIM,
                   chan + h * chunks * 8, chunks, group, lane);
  float* srow = scores + (int64_t)u * max_len;
  // Paged caches: the pages of the batch of tiles after this one are looked up one iteration
  // ahead, so that the table reads overlap the proxy loads in flight instead of preceding them.
  const unsigned char* ahead[TPI];
  auto look_ahead = [&](int Tn) {
    if constexpr (PAGED) {
#pragma unroll
      for (int j = 0; j < TPI; ++j)
        ahead[j] = tile_at(min(Tn + j, tiles_alloc - 1), (Tn + j) * 16 < row1 ? status : nullptr);
    }
  };
  look_ahead(T + kScoreWarps * TPI);

  // The loop exists twice: when the dominant channels fill exactly KB whole 16-channel blocks
  // (8, 16, 32 FCs), loads and products need no run-time test of the tile geometry.
  auto stream = [&](auto exact_tag) {
    constexpr bool EXACT = decltype(exact_tag)::value;
    while (T * 16 < row1) {       // uniform over the warp
      float s_lo[TPI], s_hi[TPI];
#pragma unroll
      for (int j = 0; j < TPI; ++j) {
        if constexpr (EXACT) {
          float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int kb = 0; kb < KB; ++kb) mma_bf16_16816(c, a[j][kb], f.b[kb]);
          reduce_heads<MAXRED>(c, group, lane, s_lo[j], s_hi[j]);
        } else {
          score_tile<KB, MAXRED>(a[j], f, n_blocks, group, lane, s_lo[j], s_hi[j]);
        }
      }
      const int next = T + kScoreWarps * TPI;
      if (next * 16 < row1) {
#pragma unroll
        for (int j = 0; j < TPI; ++j) {
          const unsigned char* tile = PAGED ? ahead[j] : tile_at(next + j, nullptr);
          const bool ok = (next + j) * 16 < row1;
          if constexpr (EXACT) {
#pragma unroll
            for (int kb = 0; kb < KB; ++kb)
              a[j][kb] = ok ? ld_proxy_u4(tile + kb * 512 + lane * 16) : make_uint4(0u, 0u, 0u, 0u);
          } else {
            load_tile<KB>(a[j], tile, pg, lane, ok);
          }
        }
        look_ahead(next + kScoreWarps * TPI);
      }
#pragma unroll
      for (int p = 0; p < TPI / 2; ++p) {
        float v;
        const int row = (T + 2 * p) * 16 + pick_row_of_pair(lane, s_lo[2 * p], s_hi[2 * p], s_lo[2 * p + 1], s_hi[2 * p + 1], v);
        if (row < row1) srow[row] = v;
      }
      T = next;
    }
  };
  if (pg.n8 == 0 && pg.n16 == KB) stream(std::true_type{});
  else stream(std::false_type{});
}

template <int KB>
void launch_score(fasa_ctx* ctx, const void* q, const void* proxy, const int32_t* seq_lens,
                  float* scores, cudaStream_t s) {
  const fasa_config_t& c = ctx->cfg;
  const int units = c.batch * ctx->n_sets;
  // Enough CTAs to cover the SMs several times, at least one warp iteration each.
  constexpr int kStep = TilesPerIter<KB>::value * kScoreWarps;
  const int tiles = (c.max_len + 15) / 16;
  const int want_ctas = (8 * ctx->n_sm + units - 1) / units;
  int per = (tiles + want_ctas - 1) / want_ctas;
  per = (per + kStep - 1) / kStep * kStep;
  dim3 grid((unsigned)((tiles + per - 1) / per), (unsigned)units);
  auto go = [&](auto kernel) {
    kernel<<<grid, kScoreThreads, 0, s>>>(
        (const uint16_t*)q, (const unsigned char*)proxy, seq_lens, ctx->d_chan, scores, ctx->d_status,
        c.n_q_heads, c.n_kv_heads, ctx->n_sets, ctx->sel_heads, c.max_len, ctx->chunks, per, fasa_page_map(ctx));
  };
  const bool paged = c.page_size > 0;
  if (c.group_reduce == 0) paged ? go(fc_score_kernel<KB, false, true>) : go(fc_score_kernel<KB, false, false>);
  else paged ? go(fc_score_kernel<KB, true, true>) : go(fc_score_kernel<KB, true, false>);
}

}  // namespace

extern "C" int32_t fasa_fc_score(fasa_ctx_t* ctx, const void* q, const void* proxy_k,
                                 const int32_t* seq_lens, float* scores, void* stream) {
  if (!ctx || !q || !proxy_k || !seq_lens || !scores || !fasa_pages_ready(ctx)) return FASA_ERR_INVALID_ARG;
  if (((uintptr_t)proxy_k & 15) != 0 || ((uintptr_t)q & 1) != 0 || ((uintptr_t)scores & 3) != 0)
    return FASA_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  const int nb = (ctx->chunks + 1) / 2;      // 16-channel blocks per tile, the 8-channel one included
  if (nb <= 1) launch_score<1>(ctx, q, proxy_k, seq_lens, scores, s);
  else if (nb <= 2) launch_score<2>(ctx, q, proxy_k, seq_lens, scores, s);
  else if (nb <= 4) launch_score<4>(ctx, q, proxy_k, seq_lens, scores, s);
  else launch_score<8>(ctx, q, proxy_k, seq_lens, scores, s);
  FASA_LAUNCH_CHECK(ctx);
  return FASA_OK;
}
