// Context, validation, workspace sizing and the composite calls of the C ABI.
#include <algorithm>
#include <new>
#include <vector>

#include "fasa_common.cuh"

namespace {

bool valid_cfg(const fasa_config_t& c, int32_t* why) {
  *why = FASA_ERR_INVALID_ARG;
  if (c.batch <= 0 || c.n_q_heads <= 0 || c.n_kv_heads <= 0 || c.max_len <= 0) return false;
  if (c.n_sink < 0 || c.n_recent < 0) return false;
  if (c.softmax_scale < 0.f || c.softmax_scale != c.softmax_scale) return false;
  *why = FASA_ERR_UNSUPPORTED;
  if (c.head_dim != FASA_HEAD_DIM) return false;
  if (c.n_dom < 1 || c.n_dom > FASA_MAX_DOM) return false;
  if (c.n_q_heads % c.n_kv_heads != 0) return false;
  if (c.n_q_heads / c.n_kv_heads > FASA_MAX_GROUP) return false;
  if (c.rope_pairing != 0 && c.rope_pairing != 1) return false;
  if (c.group_reduce != 0 && c.group_reduce != 1) return false;
  if (c.page_size != 0) {
    if (c.page_size < 16 || (c.page_size & (c.page_size - 1)) != 0 || c.n_pages < 1) return false;
  }
  if (c.select_heads < 0) return false;
  const int group = c.n_q_heads / c.n_kv_heads;
  const int per_set = c.select_heads > 0 ? c.select_heads : group;
  if (group % per_set != 0) return false;
  if ((long long)c.batch * (c.n_q_heads / per_set) > 65535) return false;  // grid.y
  return true;
}

bool fill_strides(int64_t& sb, int64_t& sh, int64_t& st, const fasa_config_t& c) {
  if (sb == 0 && sh == 0 && st == 0) {
    st = FASA_HEAD_DIM;
    sh = (int64_t)(c.page_size > 0 ? c.page_size : c.max_len) * FASA_HEAD_DIM;   // rows per head of a page / a sequence
    sb = sh * c.n_kv_heads;
    return true;
  }
  // rows are read with 16-byte loads
  return st >= FASA_HEAD_DIM && st % 8 == 0 && sh % 8 == 0 && sb % 8 == 0 && sh > 0 && sb > 0;
}

}  // namespace

extern "C" int32_t fasa_proxy_row_elems(int32_t n_dom) {
  if (n_dom < 1 || n_dom > FASA_MAX_DOM) return 0;
  return 8 * ((n_dom + 3) / 4);
}

extern "C" int32_t fasa_proxy_bytes(const fasa_ctx_t* ctx, size_t* out_bytes) {
  if (!ctx || !out_bytes) return FASA_ERR_INVALID_ARG;
  const fasa_config_t& c = ctx->cfg;
  const size_t rows = (size_t)((c.max_len + 15) / 16) * 16;
  *out_bytes = c.page_size > 0 ? (size_t)c.n_pages * c.n_kv_heads * c.page_size * ctx->row_elems * 2
                               : (size_t)c.batch * c.n_kv_heads * rows * ctx->row_elems * 2;
  return FASA_OK;
}

extern "C" int32_t fasa_create(const fasa_config_t* cfg, const int32_t* dom_fc_host,
                               fasa_ctx_t** out) {
  if (!cfg || !dom_fc_host || !out) return FASA_ERR_INVALID_ARG;
  *out = nullptr;
  int32_t why;
  if (!valid_cfg(*cfg, &why)) return why;

  fasa_ctx* ctx = new (std::nothrow) fasa_ctx();
  if (!ctx) return FASA_ERR_INVALID_ARG;
  memset(ctx, 0, sizeof(*ctx));
  ctx->cfg = *cfg;
  fasa_config_t& c = ctx->cfg;
  if (!fill_strides(c.k_stride_b, c.k_stride_h, c.k_stride_t, c) ||
      !fill_strides(c.v_stride_b, c.v_stride_h, c.v_stride_t, c)) {
    delete ctx;
    return FASA_ERR_INVALID_ARG;
  }
  if (c.softmax_scale == 0.f) c.softmax_scale = 0.08838834764831845f;  // 1/sqrt(128)
  ctx->group = c.n_q_heads / c.n_kv_heads;
  ctx->sel_heads = c.select_heads > 0 ? c.select_heads : ctx->group;
  ctx->n_sets = c.n_q_heads / ctx->sel_heads;
  if (c.page_size > 0) {
    while ((1 << ctx->page_shift) < c.page_size) ++ctx->page_shift;
    ctx->pages_per_seq = (c.max_len + c.page_size - 1) / c.page_size;
  }
  ctx->chunks = (c.n_dom + 3) / 4;
  ctx->row_elems = 8 * ctx->chunks;

  // Channel table: dominant FCs sorted ascending, FC r of head h at elements 2r, 2r+1.
  std::vector<int16_t> chan((size_t)c.n_kv_heads * ctx->row_elems, (int16_t)-1);
  for (int h = 0; h < c.n_kv_heads; ++h) {
    std::vector<int32_t> fcs(dom_fc_host + (size_t)h * c.n_dom, dom_fc_host + (size_t)(h + 1) * c.n_dom);
    std::sort(fcs.begin(), fcs.end());
    for (int r = 0; r < c.n_dom; ++r) {
      bool bad = fcs[r] < 0 || fcs[r] >= FASA_HEAD_DIM / 2 || (r > 0 && fcs[r] == fcs[r - 1]);
      if (bad) {
        delete ctx;
        return FASA_ERR_INVALID_ARG;
      }
      int c0 = c.rope_pairing == 0 ? fcs[r] : 2 * fcs[r];
      int c1 = c.rope_pairing == 0 ? fcs[r] + FASA_HEAD_DIM / 2 : 2 * fcs[r] + 1;
      chan[(size_t)h * ctx->row_elems + 2 * r] = (int16_t)c0;
      chan[(size_t)h * ctx->row_elems + 2 * r + 1] = (int16_t)c1;
    }
  }

  // the complement of each head's dominant channels, ascending (split key cache)
  std::vector<int16_t> ndchan;
  if (c.n_dom % 4 == 0 && c.n_dom < FASA_HEAD_DIM / 2 && c.page_size == 0) {
    const int nd = FASA_HEAD_DIM - 2 * c.n_dom;
    ndchan.resize((size_t)c.n_kv_heads * nd);
    for (int h = 0; h < c.n_kv_heads; ++h) {
      bool dom[FASA_HEAD_DIM] = {false};
      for (int i = 0; i < 2 * c.n_dom; ++i) dom[chan[(size_t)h * ctx->row_elems + i]] = true;
      int n = 0;
      for (int ch = 0; ch < FASA_HEAD_DIM; ++ch)
        if (!dom[ch]) ndchan[(size_t)h * nd + n++] = (int16_t)ch;
    }
  }

  cudaError_t e = cudaGetDevice(&ctx->device);
  cudaDeviceProp prop;
  if (e == cudaSuccess) e = cudaGetDeviceProperties(&prop, ctx->device);
  if (e == cudaSuccess && prop.major != 10) {
    delete ctx;
    return FASA_ERR_UNSUPPORTED;  // built for sm_100a only
  }
  if (e == cudaSuccess) ctx->n_sm = prop.multiProcessorCount;
  if (e == cudaSuccess) e = cudaMalloc(&ctx->d_chan, chan.size() * sizeof(int16_t));
  if (e == cudaSuccess) e = cudaMalloc(&ctx->d_status, 256);
  if (e == cudaSuccess) e = cudaMalloc(&ctx->d_arrive, (size_t)c.batch * sizeof(int32_t));
  if (e == cudaSuccess) e = cudaMemset(ctx->d_arrive, 0, (size_t)c.batch * sizeof(int32_t));
  if (e == cudaSuccess)
    e = cudaMemcpy(ctx->d_chan, chan.data(), chan.size() * sizeof(int16_t), cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemset(ctx->d_status, 0, 256);
  if (e == cudaSuccess && !ndchan.empty()) {
    e = cudaMalloc(&ctx->d_ndchan, ndchan.size() * sizeof(int16_t));
    if (e == cudaSuccess) e = cudaMemcpy(ctx->d_ndchan, ndchan.data(), ndchan.size() * sizeof(int16_t), cudaMemcpyHostToDevice);
  }
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    cudaFree(ctx->d_chan);
    cudaFree(ctx->d_ndchan);
    cudaFree(ctx->d_status);
    cudaFree(ctx->d_arrive);
    delete ctx;
    return FASA_ERR_CUDA;
  }
  fasa_fused_plan(ctx);
  ctx->use_fused = 1;
  *out = ctx;
  return FASA_OK;
}

// Whether a K/V cache pointer is host memory (the memory-optimised variant keeps the caches in
// page-locked host memory): asked of the driver once per pointer, a decode loop passes the same one.
bool fasa_on_host(fasa_ctx* ctx, const void* p) {
  if (ctx->cache_seen == p && p) return ctx->cache_on_host != 0;
  cudaPointerAttributes at;
  bool host = false;
  if (cudaPointerGetAttributes(&at, p) == cudaSuccess) host = at.type == cudaMemoryTypeHost;
  else cudaGetLastError();
  ctx->cache_seen = p;
  ctx->cache_on_host = host ? 1 : 0;
  return host;
}

extern "C" int32_t fasa_set_block_table(fasa_ctx_t* ctx, const int32_t* block_table) {
  if (!ctx || !block_table || ctx->cfg.page_size == 0) return FASA_ERR_INVALID_ARG;
  ctx->block_table = block_table;
  return FASA_OK;
}

extern "C" int32_t fasa_destroy(fasa_ctx_t* ctx) {
  if (!ctx) return FASA_ERR_INVALID_ARG;
  cudaFree(ctx->d_chan);
  cudaFree(ctx->d_ndchan);
  cudaFree(ctx->d_status);
  cudaFree(ctx->d_arrive);
  delete ctx;
  return FASA_OK;
}

extern "C" const char* fasa_status_string(int32_t s) {
  switch (s) {
    case FASA_OK: return "ok";
    case FASA_ERR_INVALID_ARG: return "invalid argument";
    case FASA_ERR_UNSUPPORTED: return "unsupported configuration";
    case FASA_ERR_WORKSPACE: return "workspace too small for this selection size";
    case FASA_ERR_CUDA: return "CUDA runtime error";
    case FASA_ERR_TIMEOUT: return "timeout";
    default: return "unknown status";
  }
}

extern "C" const char* fasa_last_cuda_error(const fasa_ctx_t* ctx) {
  return ctx ? ctx->cuda_err : "";
}

extern "C" int32_t fasa_set_step_mode(fasa_ctx_t* ctx, int32_t mode) {
  if (!ctx || mode < 0 || mode > 2) return FASA_ERR_INVALID_ARG;
  ctx->use_fused = mode != 0;
  ctx->topk_rows = mode == 2;
  return FASA_OK;
}

extern "C" int32_t fasa_step_cluster_size(const fasa_ctx_t* ctx) {
  return ctx && ctx->use_fused && ctx->fused_step_ok ? (ctx->fused_cs > 0 ? ctx->step_cs : 0) : 0;
}

extern "C" int64_t fasa_launch_count(const fasa_ctx_t* ctx) { return ctx ? ctx->launches : 0; }

extern "C" int32_t fasa_get_device_status(fasa_ctx_t* ctx, void* stream, int32_t* host_out) {
  if (!ctx || !host_out) return FASA_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  FASA_CUDA_TRY(ctx, cudaMemcpyAsync(host_out, ctx->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  FASA_CUDA_TRY(ctx, cudaMemsetAsync(ctx->d_status, 0, sizeof(int32_t), s));
  FASA_CUDA_TRY(ctx, cudaStreamSynchronize(s));
  return FASA_OK;
}

// Splits: enough CTAs to fill the GPU a few times over, between 64 and 2048 rows each.
static int split_count_bound(const fasa_ctx* ctx, int n_upper, int units) {
  const int target = 4 * (ctx->n_sm > 0 ? ctx->n_sm : 148);
  const int want = std::max((target + units - 1) / units, (n_upper + 2047) / 2048);
  const int most = (n_upper + 63) / 64;
  return std::max(1, std::min(want, most));   // non-decreasing in n_upper, non-increasing in units
}

fasa_split_plan fasa_plan_splits(const fasa_ctx* ctx, int n_upper, int units) {
  const int n = split_count_bound(ctx, n_upper, units);
  int chunk = (n_upper + n - 1) / n;
  chunk = (chunk + 31) / 32 * 32;
  fasa_split_plan p;
  p.chunk = chunk;
  p.n_splits = std::max(1, (n_upper + chunk - 1) / chunk);  // <= n
  return p;
}

// The partial-result area is sized for the largest split count any call can use
// (the bound at max_len for the fewest units a launch can have, one per KV head), so it does
// not depend on the selection size.
extern "C" int32_t fasa_workspace_bytes(const fasa_ctx_t* ctx, int32_t n_sel_max, size_t* out_bytes) {
  if (!ctx || !out_bytes || n_sel_max < 0) return FASA_ERR_INVALID_ARG;
  const int n = split_count_bound(ctx, ctx->cfg.max_len, ctx->cfg.batch * ctx->cfg.n_kv_heads);
  size_t per_split = (size_t)ctx->cfg.batch * ctx->cfg.n_q_heads * (FASA_HEAD_DIM + 2) * sizeof(float);
  *out_bytes = fasa_align_up(per_split * (size_t)n, 256) + 256;
  return FASA_OK;
}

// The cluster kernel attends to groups of more than four query heads in two passes over the
// selected rows.  From HBM the second pass hits L2; from caches in page-locked host memory every
// row would cross the host link twice (measured at 28 / 4 heads: 531 us against 282 us through
// the tensor-core kernel, which reads a row once for up to eight heads): given a workspace, such
// steps hand the attention over whatever the selection size.
static bool fasa_host_rows_twice(fasa_ctx* ctx, const void* k_cache, const void* workspace) {
  return workspace != nullptr && ctx->sel_heads > 4 && ctx->cfg.page_size == 0 && fasa_on_host(ctx, k_cache);
}

// What fasa_fc_score, fasa_topk and fasa_sparse_decode_attn require of the arguments they share
// with the composite calls.
static bool three_kernel_args_ok(const fasa_ctx* ctx, const void* q, const void* k_cache, const void* v_cache,
                                 const void* proxy_k, const float* scores, const void* workspace) {
  return scores && workspace && fasa_pages_ready(ctx) && !((uintptr_t)proxy_k & 15) && !((uintptr_t)q & 15) &&
         !((uintptr_t)scores & 3) && !((uintptr_t)k_cache & 15) && !((uintptr_t)v_cache & 15) &&
         !((uintptr_t)workspace & 255);
}

extern "C" int32_t fasa_decode_step(fasa_ctx_t* ctx, const void* q, const void* k_cache,
                                    const void* v_cache, const void* proxy_k,
                                    const int32_t* seq_lens, int32_t budget, int32_t n_sel_max,
                                    float* scores, int32_t* idx, int32_t* n_sel, float* out,
                                    float* lse, void* workspace, void* stream) {
  if (!ctx || !q || !k_cache || !v_cache || !proxy_k || !seq_lens || !idx || !n_sel || !out ||
      budget == 0 || budget < -1000 || n_sel_max <= 0)
    return FASA_ERR_INVALID_ARG;
  if (ctx->use_fused && ctx->fused_step_ok && ctx->fused_cs > 0) {
    if (((uintptr_t)proxy_k & 15) || ((uintptr_t)q & 15) || ((uintptr_t)k_cache & 15) ||
        ((uintptr_t)v_cache & 15) || (scores && ((uintptr_t)scores & 3)))
      return FASA_ERR_INVALID_ARG;
    if (!fasa_pages_ready(ctx)) return FASA_ERR_INVALID_ARG;
    if (fasa_attend_separately(ctx, n_sel_max, workspace) || fasa_host_rows_twice(ctx, k_cache, workspace)) {
      if ((uintptr_t)workspace & 255) return FASA_ERR_INVALID_ARG;   // (what the second launch would refuse)
      int32_t st2 = fasa_fused_launch(ctx, q, k_cache, v_cache, proxy_k, seq_lens, budget, n_sel_max, scores,
                                      idx, n_sel, out, lse, nullptr, nullptr, (cudaStream_t)stream, false);
      if (st2 != FASA_OK) return st2;
      return fasa_sparse_decode_attn(ctx, q, k_cache, v_cache, idx, n_sel, n_sel_max, out, lse, workspace, stream);
    }
    return fasa_fused_launch(ctx, q, k_cache, v_cache, proxy_k, seq_lens, budget, n_sel_max, scores,
                             idx, n_sel, out, lse, nullptr, nullptr, (cudaStream_t)stream);
  }
  // three kernels: everything any of them would refuse is refused before the first is enqueued
  if (!three_kernel_args_ok(ctx, q, k_cache, v_cache, proxy_k, scores, workspace)) return FASA_ERR_INVALID_ARG;
  int32_t st = fasa_fc_score(ctx, q, proxy_k, seq_lens, scores, stream);
  if (st != FASA_OK) return st;
  st = fasa_topk(ctx, scores, seq_lens, budget, n_sel_max, idx, n_sel, workspace, stream);
  if (st != FASA_OK) return st;
  return fasa_sparse_decode_attn(ctx, q, k_cache, v_cache, idx, n_sel, n_sel_max, out, lse,
                                 workspace, stream);
}

// out_mirror (nullable): device-accessible second destination of `out`; *mirrored tells whether
// the path taken wrote it.
static int32_t append_decode_step_impl(fasa_ctx_t* ctx, const void* q, const void* k_new,
                                       const void* v_new, void* k_cache, void* v_cache,
                                       void* proxy_k, int32_t* seq_lens, int32_t budget,
                                       int32_t n_sel_max, float* scores, int32_t* idx,
                                       int32_t* n_sel, float* out, float* lse, void* workspace,
                                       void* stream, float* out_mirror, bool* mirrored) {
  *mirrored = false;
  if (!ctx || !q || !k_new || !v_new || !k_cache || !v_cache || !proxy_k || !seq_lens || !idx ||
      !n_sel || !out || budget == 0 || budget < -1000 || n_sel_max <= 0)
    return FASA_ERR_INVALID_ARG;
  if (ctx->use_fused && ctx->fused_step_ok && ctx->fused_cs > 0) {
    if (((uintptr_t)proxy_k & 15) || ((uintptr_t)q & 15) || ((uintptr_t)k_cache & 15) ||
        ((uintptr_t)v_cache & 15) || ((uintptr_t)k_new & 15) || ((uintptr_t)v_new & 15) ||
        (scores && ((uintptr_t)scores & 3)))
      return FASA_ERR_INVALID_ARG;
    if (!fasa_pages_ready(ctx)) return FASA_ERR_INVALID_ARG;
    if (fasa_attend_separately(ctx, n_sel_max, workspace) || fasa_host_rows_twice(ctx, k_cache, workspace)) {
      if ((uintptr_t)workspace & 255) return FASA_ERR_INVALID_ARG;   // (what the second launch would refuse)
      int32_t st2 = fasa_fused_launch(ctx, q, k_cache, v_cache, proxy_k, seq_lens, budget, n_sel_max, scores,
                                      idx, n_sel, out, lse, k_new, v_new, (cudaStream_t)stream, false);
      if (st2 != FASA_OK) return st2;
      return fasa_sparse_attn_mirrored(ctx, q, k_cache, v_cache, idx, n_sel, n_sel_max, out, lse, workspace,
                                       (cudaStream_t)stream, out_mirror, mirrored);
    }
    *mirrored = out_mirror != nullptr;
    return fasa_fused_launch(ctx, q, k_cache, v_cache, proxy_k, seq_lens, budget, n_sel_max, scores,
                             idx, n_sel, out, lse, k_new, v_new, (cudaStream_t)stream, true, out_mirror);
  }
  // append + three kernels: the arguments of all four calls are checked before the cache grows,
  // so that a caller who repairs an argument and retries does not append the token twice
  if (!three_kernel_args_ok(ctx, q, k_cache, v_cache, proxy_k, scores, workspace) || ((uintptr_t)k_new & 15) ||
      ((uintptr_t)v_new & 15))
    return FASA_ERR_INVALID_ARG;
  int32_t st = fasa_kv_append(ctx, k_cache, v_cache, proxy_k, seq_lens, k_new, v_new, 1, stream);
  if (st != FASA_OK) return st;
  return fasa_decode_step(ctx, q, k_cache, v_cache, proxy_k, seq_lens, budget, n_sel_max, scores, idx,
                          n_sel, out, lse, workspace, stream);
}

extern "C" int32_t fasa_append_decode_step(fasa_ctx_t* ctx, const void* q, const void* k_new,
                                           const void* v_new, void* k_cache, void* v_cache,
                                           void* proxy_k, int32_t* seq_lens, int32_t budget,
                                           int32_t n_sel_max, float* scores, int32_t* idx,
                                           int32_t* n_sel, float* out, float* lse, void* workspace,
                                           void* stream) {
  bool mirrored;
  return append_decode_step_impl(ctx, q, k_new, v_new, k_cache, v_cache, proxy_k, seq_lens, budget, n_sel_max,
                                 scores, idx, n_sel, out, lse, workspace, stream, nullptr, &mirrored);
}

extern "C" int32_t fasa_select_step(fasa_ctx_t* ctx, const void* q, const void* k_new,
                                    const void* v_new, void* k_cache, void* v_cache, void* proxy_k,
                                    int32_t* seq_lens, int32_t budget, int32_t n_sel_max,
                                    float* scores, int32_t* idx, int32_t* n_sel, void* stream) {
  if (!ctx || !q || !k_cache || !v_cache || !proxy_k || !seq_lens || !idx || !n_sel || budget == 0 ||
      budget < -1000 || n_sel_max <= 0 || (k_new == nullptr) != (v_new == nullptr))
    return FASA_ERR_INVALID_ARG;
  if (!(ctx->use_fused && ctx->fused_step_ok && ctx->fused_cs > 0)) return FASA_ERR_UNSUPPORTED;
  if (((uintptr_t)proxy_k & 15) || ((uintptr_t)q & 15) || ((uintptr_t)k_cache & 15) || ((uintptr_t)v_cache & 15) ||
      ((uintptr_t)k_new & 15) || ((uintptr_t)v_new & 15) || (scores && ((uintptr_t)scores & 3)) ||
      !fasa_pages_ready(ctx))
    return FASA_ERR_INVALID_ARG;
  return fasa_fused_launch(ctx, q, k_cache, v_cache, proxy_k, seq_lens, budget, n_sel_max, scores, idx, n_sel,
                           nullptr, nullptr, k_new, v_new, (cudaStream_t)stream, false);
}

extern "C" int32_t fasa_stage_bytes(const fasa_ctx_t* ctx, size_t* out_bytes) {
  if (!ctx || !out_bytes) return FASA_ERR_INVALID_ARG;
  const fasa_config_t& c = ctx->cfg;
  size_t qb = fasa_align_up((size_t)c.batch * c.n_q_heads * FASA_HEAD_DIM * 2, 256);
  size_t kb = fasa_align_up((size_t)c.batch * c.n_kv_heads * FASA_HEAD_DIM * 2, 256);
  *out_bytes = qb + 2 * kb;
  return FASA_OK;
}

extern "C" int32_t fasa_decode_step_host(fasa_ctx_t* ctx, const void* q_host,
                                         const void* k_new_host, const void* v_new_host,
                                         void* dev_stage, void* k_cache, void* v_cache,
                                         void* proxy_k, int32_t* seq_lens, int32_t budget,
                                         int32_t n_sel_max, float* scores, int32_t* idx,
                                         int32_t* n_sel, float* out, float* out_host,
                                         void* workspace, void* stream) {
  if (!ctx || !q_host || !k_new_host || !v_new_host || !dev_stage || !out_host || !out)
    return FASA_ERR_INVALID_ARG;
  const fasa_config_t& c = ctx->cfg;
  cudaStream_t s = (cudaStream_t)stream;
  size_t q_bytes = (size_t)c.batch * c.n_q_heads * FASA_HEAD_DIM * 2;
  size_t kv_bytes = (size_t)c.batch * c.n_kv_heads * FASA_HEAD_DIM * 2;
  char* dq = (char*)dev_stage;
  char* dk = dq + fasa_align_up(q_bytes, 256);
  char* dv = dk + fasa_align_up(kv_bytes, 256);
  // Pinned (page-locked, mapped) host buffers need no copy call: where the step is a single wave
  // of one launch its kernel reads them in place (the few KB cross the host link inside the
  // launch); where it is several launches or several waves of CTAs, one small kernel first
  // brings all three to the staging area, so that no CTA's start waits on the link.  Anything
  // else is copied to the staging area with cudaMemcpyAsync.  The driver is asked about a
  // pointer once: a decode loop passes the same buffers every step.
  auto mapped = [&](int slot, const void* hp) -> void* {
    if (ctx->host_seen[slot] == hp) return ctx->host_mapped[slot];
    cudaPointerAttributes at;
    void* dp = nullptr;
    if (cudaPointerGetAttributes(&at, hp) == cudaSuccess) {
      if (at.type == cudaMemoryTypeHost) dp = at.devicePointer;
    } else {
      cudaGetLastError();
    }
    ctx->host_seen[slot] = hp;
    ctx->host_mapped[slot] = dp;
    return dp;
  };
  const void* mq = mapped(0, q_host);
  const void* mk = mapped(1, k_new_host);
  const void* mv = mapped(2, v_new_host);
  const bool all_mapped = mq && mk && mv && !((uintptr_t)mq & 15) && !((uintptr_t)mk & 15) && !((uintptr_t)mv & 15);
  const bool one_wave_one_launch = ctx->use_fused && ctx->fused_cs > 0 && !fasa_attend_separately(ctx, n_sel_max, workspace) &&
                                   (long long)c.batch * ctx->n_sets * ctx->fused_cs <= 2ll * ctx->n_sm;
  if (all_mapped && one_wave_one_launch) {
    dq = (char*)mq; dk = (char*)mk; dv = (char*)mv;
  } else if (all_mapped) {
    FASA_CUDA_TRY(ctx, fasa_stage_from_mapped(dq, mq, q_bytes, dk, mk, dv, mv, kv_bytes, s));
    ctx->launches += 1;
  } else {
    FASA_CUDA_TRY(ctx, cudaMemcpyAsync(dq, q_host, q_bytes, cudaMemcpyHostToDevice, s));
    FASA_CUDA_TRY(ctx, cudaMemcpyAsync(dk, k_new_host, kv_bytes, cudaMemcpyHostToDevice, s));
    FASA_CUDA_TRY(ctx, cudaMemcpyAsync(dv, v_new_host, kv_bytes, cudaMemcpyHostToDevice, s));
  }
  // A pinned out_host is written by the step's kernel itself (next to `out`), where the path
  // taken has a single kernel to do it; otherwise `out` is copied back.
  float* mo = (float*)mapped(3, out_host);
  if ((uintptr_t)mo & 3) mo = nullptr;
  bool mirrored = false;
  int32_t st = append_decode_step_impl(ctx, dq, dk, dv, k_cache, v_cache, proxy_k, seq_lens, budget, n_sel_max,
                                       scores, idx, n_sel, out, nullptr, workspace, stream, mo, &mirrored);
  if (st != FASA_OK) return st;
  size_t o_bytes = (size_t)c.batch * c.n_q_heads * FASA_HEAD_DIM * sizeof(float);
  if (!mirrored) FASA_CUDA_TRY(ctx, cudaMemcpyAsync(out_host, out, o_bytes, cudaMemcpyDeviceToHost, s));
  FASA_CUDA_TRY(ctx, cudaStreamSynchronize(s));
  return FASA_OK;
}
