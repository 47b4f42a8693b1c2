// TIP scoring (Sec. 4.1): S[j] = reduce_g sum_{i in I_dom} alpha^(i)_g[j], streamed from the
// packed proxy-K buffer.  HBM-bound: every proxy byte is read once with 128-bit loads that
// are contiguous across the warp, each thread keeps UNROLL loads in flight, and the lanes
// that share a row combine their partial sums with xor-shuffles.
#include "fasa_common.cuh"
#include "fasa_score_core.cuh"

namespace {

constexpr int kScoreThreads = 256;
constexpr int kScoreUnroll = 8;

// LPR = lanes per proxy row (power of two >= chunks).  MAXRED = reduce the group by max
// (one dot product per query head) instead of by sum (one dot product with sum_g q_g).
template <int LPR, bool MAXRED>
__global__ void __launch_bounds__(kScoreThreads)
fc_score_kernel(const uint16_t* __restrict__ q, const uint4* __restrict__ proxy,
                const int32_t* __restrict__ seq_lens, const int16_t* __restrict__ chan,
                float* __restrict__ scores, int32_t* __restrict__ status, int n_q_heads,
                int n_kv_heads, int group, int max_len, int chunks, int rows_per_cta) {
  constexpr int RPL = 32 / LPR;                 // rows covered by one warp-wide load
  constexpr int RPI = RPL * kScoreUnroll;       // rows per warp iteration

  const int u = blockIdx.y;
  const int h = u % n_kv_heads;
  const int b = u / n_kv_heads;
  const int cta_row0 = blockIdx.x * rows_per_cta;
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int sub = lane & (LPR - 1);             // which 16-byte chunk of the row
  const int grp = lane / LPR;                   // which row of the warp-wide load
  const bool live = sub < chunks;
  const uint4* prow = proxy + (int64_t)u * max_len * chunks;

  // The first batch of proxy loads is issued before anything else is known: rows up to
  // max_len are allocated, so reading past the sequence length is harmless, and the loads of
  // the length, the channel table and the query overlap with the stream instead of
  // preceding it.
  const int alloc_row1 = min(max_len, cta_row0 + rows_per_cta);
  int base = cta_row0 + warp * RPI;
  uint4 x[kScoreUnroll];
#pragma unroll
  for (int i = 0; i < kScoreUnroll; ++i) {
    const int row = base + i * RPL + grp;
    x[i] = (live && row < alloc_row1) ? ld_stream_u4(prow + (int64_t)row * chunks + sub)
                                      : make_uint4(0u, 0u, 0u, 0u);
  }

  const int len = clamp_len(seq_lens[b], max_len, status);
  if (cta_row0 >= len) return;
  const int cta_row1 = min(len, cta_row0 + rows_per_cta);

  ScoreQ<MAXRED> sq;
  load_score_q<MAXRED>(sq, q + ((int64_t)b * n_q_heads + (int64_t)h * group) * FASA_HEAD_DIM,
                       chan + h * chunks * 8 + (live ? sub : 0) * 8, group, live);
  float* srow = scores + (int64_t)u * max_len;

  while (base < cta_row1) {
    float s[kScoreUnroll];
#pragma unroll
    for (int i = 0; i < kScoreUnroll; ++i) s[i] = score_row<LPR, MAXRED>(sq, x[i], group);
    const int next = base + (kScoreThreads / 32) * RPI;
    if (next < cta_row1) {
#pragma unroll
      for (int i = 0; i < kScoreUnroll; ++i) {
        const int row = next + i * RPL + grp;
        x[i] = (live && row < cta_row1) ? ld_stream_u4(prow + (int64_t)row * chunks + sub)
                                        : make_uint4(0u, 0u, 0u, 0u);
      }
    }
#pragma unroll
    for (int i = 0; i < kScoreUnroll; ++i) {
      const int row = base + i * RPL + grp;
      if (sub == 0 && row < cta_row1) srow[row] = s[i];
    }
    base = next;
  }
}

template <int LPR>
void launch_score(fasa_ctx* ctx, const void* q, const void* proxy, const int32_t* seq_lens,
                  float* scores, cudaStream_t s) {
  const fasa_config_t& c = ctx->cfg;
  const int units = c.batch * c.n_kv_heads;
  // Enough CTAs to cover the SMs several times, at least one warp iteration each.
  constexpr int RPI_CTA = (32 / LPR) * kScoreUnroll * (kScoreThreads / 32);
  int want_ctas = (8 * ctx->n_sm + units - 1) / units;
  int rows = (c.max_len + want_ctas - 1) / want_ctas;
  rows = (rows + RPI_CTA - 1) / RPI_CTA * RPI_CTA;
  if (rows < RPI_CTA) rows = RPI_CTA;
  dim3 grid((unsigned)((c.max_len + rows - 1) / rows), (unsigned)units);
  if (c.group_reduce == 0)
    fc_score_kernel<LPR, false><<<grid, kScoreThreads, 0, s>>>(
        (const uint16_t*)q, (const uint4*)proxy, seq_lens, ctx->d_chan, scores, ctx->d_status,
        c.n_q_heads, c.n_kv_heads, ctx->group, c.max_len, ctx->chunks, rows);
  else
    fc_score_kernel<LPR, true><<<grid, kScoreThreads, 0, s>>>(
        (const uint16_t*)q, (const uint4*)proxy, seq_lens, ctx->d_chan, scores, ctx->d_status,
        c.n_q_heads, c.n_kv_heads, ctx->group, c.max_len, ctx->chunks, rows);
}

}  // namespace

extern "C" int32_t fasa_fc_score(fasa_ctx_t* ctx, const void* q, const void* proxy_k,
                                 const int32_t* seq_lens, float* scores, void* stream) {
  if (!ctx || !q || !proxy_k || !seq_lens || !scores) return FASA_ERR_INVALID_ARG;
  if (((uintptr_t)proxy_k & 15) != 0 || ((uintptr_t)q & 1) != 0 || ((uintptr_t)scores & 3) != 0)
    return FASA_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  const int ch = ctx->chunks;
  if (ch <= 1) launch_score<1>(ctx, q, proxy_k, seq_lens, scores, s);
  else if (ch <= 2) launch_score<2>(ctx, q, proxy_k, seq_lens, scores, s);
  else if (ch <= 4) launch_score<4>(ctx, q, proxy_k, seq_lens, scores, s);
  else if (ch <= 8) launch_score<8>(ctx, q, proxy_k, seq_lens, scores, s);
  else launch_score<16>(ctx, q, proxy_k, seq_lens, scores, s);
  FASA_LAUNCH_CHECK(ctx);
  return FASA_OK;
}
