// TIP scoring (Sec. 4.1): S[j] = reduce_g sum_{i in I_dom} alpha^(i)_g[j], streamed from the
// packed proxy-K buffer.  HBM-bound: every proxy byte is read once with 128-bit loads that
// are contiguous across the warp, each thread keeps UNROLL loads in flight, and the lanes
// that share a row combine their partial sums with xor-shuffles.
#include "fasa_common.cuh"

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
  constexpr int NG = MAXRED ? FASA_MAX_GROUP : 1;

  const int u = blockIdx.y;
  const int h = u % n_kv_heads;
  const int b = u / n_kv_heads;
  const int len = clamp_len(seq_lens[b], max_len, status);
  const int cta_row0 = blockIdx.x * rows_per_cta;
  if (cta_row0 >= len) return;
  const int cta_row1 = min(len, cta_row0 + rows_per_cta);

  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int sub = lane & (LPR - 1);             // which 16-byte chunk of the row
  const int grp = lane / LPR;                   // which row of the warp-wide load
  const bool live = sub < chunks;

  // This lane's 8 query values (summed over the group, or kept per head for MAXRED).
  float2 qv[NG][4];
#pragma unroll
  for (int g = 0; g < NG; ++g)
#pragma unroll
    for (int e = 0; e < 4; ++e) qv[g][e] = make_float2(0.f, 0.f);
  if (live) {
    const int16_t* ch = chan + h * chunks * 8 + sub * 8;
    const uint16_t* qb = q + ((int64_t)b * n_q_heads + (int64_t)h * group) * FASA_HEAD_DIM;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int c0 = ch[2 * e], c1 = ch[2 * e + 1];
      for (int g = 0; g < group; ++g) {
        const float x = c0 >= 0 ? bf16_bits_to_f32(qb[g * FASA_HEAD_DIM + c0]) : 0.f;
        const float y = c1 >= 0 ? bf16_bits_to_f32(qb[g * FASA_HEAD_DIM + c1]) : 0.f;
        if (MAXRED) {
#pragma unroll
          for (int gg = 0; gg < NG; ++gg)
            if (gg == g) qv[gg][e] = make_float2(x, y);
        } else {
          qv[0][e].x += x;
          qv[0][e].y += y;
        }
      }
    }
  }

  const uint4* prow = proxy + (int64_t)u * max_len * chunks;
  float* srow = scores + (int64_t)u * max_len;

  for (int base = cta_row0 + warp * RPI; base < cta_row1; base += (kScoreThreads / 32) * RPI) {
    uint4 x[kScoreUnroll];
#pragma unroll
    for (int i = 0; i < kScoreUnroll; ++i) {
      const int row = base + i * RPL + grp;
      x[i] = (live && row < cta_row1) ? ld_stream_u4(prow + (int64_t)row * chunks + sub)
                                      : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int i = 0; i < kScoreUnroll; ++i) {
      float s;
      if (!MAXRED) {
        s = dot8(qv[0], x[i]);
#pragma unroll
        for (int o = LPR / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      } else {
        s = -INFINITY;
#pragma unroll
        for (int g = 0; g < NG; ++g) {
          if (g < group) {
            float sg = dot8(qv[g], x[i]);
#pragma unroll
            for (int o = LPR / 2; o > 0; o >>= 1) sg += __shfl_xor_sync(0xffffffffu, sg, o);
            s = fmaxf(s, sg);
          }
        }
      }
      const int row = base + i * RPL + grp;
      if (sub == 0 && row < cta_row1) srow[row] = s + 0.0f;  // -0 becomes +0
    }
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
