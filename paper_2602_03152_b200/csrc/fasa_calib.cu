// Offline calibration of the dominant FCs (Algorithm 1): the contextual agreement CA of every
// FC with the full head (Sec. 3.3, Eq. 4), accumulated over samples, and the choice of the F
// FCs with the highest mean.
//
// One call takes a batch of (query, key cache) pairs laid out as for a decode step.  A sample
// is a (sequence, query head) pair.  Three stages, all on the caller's stream:
//   1. calib_score_kernel: the 64 single-FC raw scores alpha^(i)[j] (Eq. 3) and their sum, the
//      full-head raw scores alpha[j] (Eq. 2), as 65 fp32 rows per sample;
//   2. TopK-I of each of the 65 rows (the cluster kernel's select-only form, the same code
//      that serves fasa_topk, no forced positions);
//   3. calib_intersect_kernel: |TopK-I(alpha) n TopK-I(alpha^(i))| for every i, added to the
//      caller's running counts.
// Which index enters a top-k set is decided by fp32 values with a fixed evaluation order:
// alpha^(i) = fl(q_c0 k_c0 + q_c1 k_c1) (the products of bf16 values are exact in fp32) and
// alpha = ((alpha^(0) + alpha^(1)) + alpha^(2)) + ...; equal scores keep the lower index.
#include <algorithm>
#include <vector>

#include "fasa_common.cuh"

namespace {

constexpr int kFc = FASA_HEAD_DIM / 2;        // FCs per head
constexpr int kRows = kFc + 1;                // score rows per sample: the FCs, then the full head
constexpr int kCalibWarps = 4;
constexpr int kPad = 33;                      // row stride of the staging tile (bank-conflict free)

// grid (ceil(max_len / (32 * kCalibWarps)), batch * n_q_heads); a warp takes 32 consecutive
// tokens: lane l evaluates FCs l and l + 32 of one token at a time (coalesced 2-byte loads of
// the key row), the tile is transposed through shared memory and every score row is written
// with coalesced 128-byte stores.
template <bool PAGED>
__global__ void __launch_bounds__(kCalibWarps * 32)
calib_score_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k,
                   const int32_t* __restrict__ seq_lens, float* __restrict__ scores,
                   int32_t* __restrict__ status, int n_q_heads, int n_kv_heads, int max_len, int pairing,
                   int64_t ksb, int64_t ksh, int64_t kst, const PageMap pm) {
  const int u = blockIdx.y;
  const int b = u / n_q_heads, hq = u % n_q_heads;
  const int h = hq / (n_q_heads / n_kv_heads);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int len = clamp_len(seq_lens[b], max_len, status);
  const int base = (blockIdx.x * kCalibWarps + warp) * 32;
  if (base >= len) return;
  __shared__ float tile[kCalibWarps][kRows * kPad];
  float* s = tile[warp];

  // channels of FC l and FC l + 32
  int c[2][2];
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const int i = lane + 32 * e;
    c[e][0] = pairing == 0 ? i : 2 * i;
    c[e][1] = pairing == 0 ? i + kFc : 2 * i + 1;
  }
  const uint16_t* qrow = q + ((int64_t)b * n_q_heads + hq) * FASA_HEAD_DIM;
  float qv[2][2];
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    qv[e][0] = bf16_bits_to_f32(qrow[c[e][0]]);
    qv[e][1] = bf16_bits_to_f32(qrow[c[e][1]]);
  }
  const int n_tok = min(32, len - base);
  for (int tt = 0; tt < n_tok; ++tt) {
    const uint16_t* krow = PAGED ? k + cache_row(pm, b, h, base + tt, ksb, ksh, kst, status)
                                 : k + b * ksb + h * ksh + (int64_t)(base + tt) * kst;
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const float p0 = qv[e][0] * bf16_bits_to_f32(krow[c[e][0]]);     // exact
      const float p1 = qv[e][1] * bf16_bits_to_f32(krow[c[e][1]]);     // exact
      s[(lane + 32 * e) * kPad + tt] = __fadd_rn(p0, p1) + 0.0f;       // one rounding; -0 becomes +0
    }
  }
  __syncwarp();
  if (lane < n_tok) {
    float acc = 0.0f;
    for (int i = 0; i < kFc; ++i) acc = __fadd_rn(acc, s[i * kPad + lane]);
    s[kFc * kPad + lane] = acc + 0.0f;
  }
  __syncwarp();
  float* out = scores + (int64_t)u * kRows * max_len + base;
  if (lane < n_tok)
    for (int i = 0; i < kRows; ++i) out[(int64_t)i * max_len + lane] = s[i * kPad + lane];
}

// One CTA per sample: the full head's index list goes to shared memory, every warp then takes
// FC lists in turn and looks each of their indices up by binary search (both lists ascending).
__global__ void __launch_bounds__(256)
calib_intersect_kernel(const int32_t* __restrict__ idx, const int32_t* __restrict__ seq_lens,
                       unsigned long long* __restrict__ counts, unsigned long long* __restrict__ n_used,
                       int n_q_heads, int max_len, int top_k) {
  extern __shared__ int32_t full[];
  const int u = blockIdx.x;
  const int b = u / n_q_heads, hq = u % n_q_heads;
  int len = seq_lens[b];
  len = len > max_len ? max_len : len;
  if (len <= top_k) return;                   // every position is selected: not a sample
  const int32_t* lists = idx + (int64_t)u * kRows * top_k;
  for (int i = threadIdx.x; i < top_k; i += blockDim.x) full[i] = lists[(int64_t)kFc * top_k + i];
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  for (int i = warp; i < kFc; i += n_warps) {
    const int32_t* mine = lists + (int64_t)i * top_k;
    int common = 0;
    for (int e = lane; e < top_k; e += 32) {
      const int32_t want = mine[e];
      int lo = 0, hi = top_k;                 // first position with full[pos] >= want
      while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (full[mid] < want) lo = mid + 1;
        else hi = mid;
      }
      common += (lo < top_k && full[lo] == want) ? 1 : 0;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) common += __shfl_xor_sync(0xffffffffu, common, o);
    if (lane == 0 && common > 0) atomicAdd(&counts[(int64_t)hq * kFc + i], (unsigned long long)common);
  }
  if (threadIdx.x == 0) atomicAdd(&n_used[hq], 1ull);
}

struct CalibLayout {
  size_t scores, idx, n_sel, total;
};

CalibLayout calib_layout(const fasa_ctx* ctx, int top_k) {
  const fasa_config_t& c = ctx->cfg;
  const size_t samples = (size_t)c.batch * c.n_q_heads;
  CalibLayout l;
  l.scores = 0;
  l.idx = fasa_align_up(samples * kRows * (size_t)c.max_len * sizeof(float), 256);
  l.n_sel = l.idx + fasa_align_up(samples * kRows * (size_t)top_k * sizeof(int32_t), 256);
  l.total = l.n_sel + fasa_align_up(samples * kRows * sizeof(int32_t), 256);
  return l;
}

bool calib_args_ok(const fasa_ctx* ctx, int top_k) {
  const fasa_config_t& c = ctx->cfg;
  return top_k >= 1 && top_k <= c.max_len && top_k <= 8192 &&
         (long long)c.batch * c.n_q_heads * kRows <= 65535;      // grid.y of the select launch
}

}  // namespace

extern "C" int32_t fasa_calib_workspace_bytes(const fasa_ctx_t* ctx, int32_t top_k, size_t* out_bytes) {
  if (!ctx || !out_bytes) return FASA_ERR_INVALID_ARG;
  if (!calib_args_ok(ctx, top_k)) return FASA_ERR_UNSUPPORTED;
  *out_bytes = calib_layout(ctx, top_k).total;
  return FASA_OK;
}

extern "C" int32_t fasa_calib_accumulate(fasa_ctx_t* ctx, const void* q, const void* k_cache,
                                         const int32_t* seq_lens, int32_t top_k, int64_t* ca_counts,
                                         int64_t* n_used, void* workspace, void* stream) {
  if (!ctx || !q || !k_cache || !seq_lens || !ca_counts || !n_used || !workspace) return FASA_ERR_INVALID_ARG;
  if (((uintptr_t)workspace & 255) != 0 || ((uintptr_t)ca_counts & 7) != 0 || ((uintptr_t)n_used & 7) != 0)
    return FASA_ERR_INVALID_ARG;
  if (!fasa_pages_ready(ctx)) return FASA_ERR_INVALID_ARG;
  if (!calib_args_ok(ctx, top_k) || ctx->fused_cs <= 0) return FASA_ERR_UNSUPPORTED;
  const fasa_config_t& c = ctx->cfg;
  cudaStream_t s = (cudaStream_t)stream;
  const CalibLayout l = calib_layout(ctx, top_k);
  float* scores = reinterpret_cast<float*>((char*)workspace + l.scores);
  int32_t* idx = reinterpret_cast<int32_t*>((char*)workspace + l.idx);
  int32_t* n_sel = reinterpret_cast<int32_t*>((char*)workspace + l.n_sel);
  const int samples = c.batch * c.n_q_heads;

  dim3 grid((unsigned)((c.max_len + 32 * kCalibWarps - 1) / (32 * kCalibWarps)), (unsigned)samples);
  auto score = c.page_size > 0 ? calib_score_kernel<true> : calib_score_kernel<false>;
  score<<<grid, kCalibWarps * 32, 0, s>>>(
      (const uint16_t*)q, (const uint16_t*)k_cache, seq_lens, scores, ctx->d_status, c.n_q_heads, c.n_kv_heads,
      c.max_len, c.rope_pairing, c.k_stride_b, c.k_stride_h, c.k_stride_t, fasa_page_map(ctx));
  FASA_LAUNCH_CHECK(ctx);
  const int32_t st = fasa_fused_topk_rows(ctx, scores, seq_lens, top_k, top_k, idx, n_sel, c.n_q_heads * kRows,
                                          0, 0, s);
  if (st != FASA_OK) return st;
  calib_intersect_kernel<<<samples, 256, (size_t)top_k * sizeof(int32_t), s>>>(
      idx, seq_lens, reinterpret_cast<unsigned long long*>(ca_counts),
      reinterpret_cast<unsigned long long*>(n_used), c.n_q_heads, c.max_len, top_k);
  FASA_LAUNCH_CHECK(ctx);
  return FASA_OK;
}

extern "C" int32_t fasa_calib_select(int32_t n_q_heads, int32_t n_kv_heads, const int64_t* ca_counts_host,
                                     const int64_t* n_used_host, int32_t top_k, int32_t n_dom,
                                     int32_t* dom_fc_host, double* mean_ca_host) {
  if (!ca_counts_host || !n_used_host || !dom_fc_host) return FASA_ERR_INVALID_ARG;
  if (n_q_heads <= 0 || n_kv_heads <= 0 || n_q_heads % n_kv_heads != 0 || top_k < 1) return FASA_ERR_INVALID_ARG;
  if (n_dom < 1 || n_dom > kFc) return FASA_ERR_UNSUPPORTED;
  const int group = n_q_heads / n_kv_heads;
  for (int h = 0; h < n_kv_heads; ++h) {
    // the query heads of a KV head read the same keys: their samples are pooled
    int64_t sum[kFc] = {0}, samples = 0;
    for (int g = h * group; g < (h + 1) * group; ++g) {
      samples += n_used_host[g];
      for (int i = 0; i < kFc; ++i) sum[i] += ca_counts_host[(int64_t)g * kFc + i];
    }
    int order[kFc];
    for (int i = 0; i < kFc; ++i) order[i] = i;
    std::stable_sort(order, order + kFc, [&](int a, int b) { return sum[a] > sum[b]; });   // equal means: lower FC first
    std::sort(order, order + n_dom);
    for (int r = 0; r < n_dom; ++r) dom_fc_host[(int64_t)h * n_dom + r] = order[r];
    if (mean_ca_host)
      for (int i = 0; i < kFc; ++i)
        mean_ca_host[(int64_t)h * kFc + i] = samples > 0 ? (double)sum[i] / ((double)samples * (double)top_k) : 0.0;
  }
  return FASA_OK;
}
