// Shared declarations of the FASA CUDA library (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include "fasa.h"

#define FASA_HEAD_DIM 128
#define FASA_MAX_GROUP 8
#define FASA_MAX_DOM 64

// Context: the normalised configuration plus a small device table.
struct fasa_ctx {
  fasa_config_t cfg;      // strides and softmax_scale filled in
  int group;              // query heads per KV head
  int sel_heads;          // query heads that share one index set (a divisor of group)
  int n_sets;             // index sets (selection units) per sequence = n_q_heads / sel_heads
  int chunks;             // 16-byte chunks per proxy row = ceil(n_dom / 4)
  int row_elems;          // bf16 elements per proxy row = 8 * chunks
  int device;
  int n_sm;
  const int32_t* block_table;  // paged caches: device [batch][pages_per_seq], caller-owned; null until set
  int page_shift;         // log2(page_size), 0 for contiguous caches
  int pages_per_seq;      // ceil(max_len / page_size)
  int16_t* d_chan;        // device [n_kv_heads][row_elems]: K channel of each proxy element, -1 = padding
  void* m_resident;       // memory-optimised variant: the caller's buffer of GPU-resident sink / recent rows (null: none)
  int16_t* d_ndchan;      // device [n_kv_heads][128 - 2 n_dom]: the other channels of each head, ascending (null
                          // unless n_dom is a multiple of 4: the split key cache of the memory-optimised variant)
  int32_t* d_status;      // device status word (FASA_DEV_* bits)
  int32_t* d_arrive;      // device [batch]: CTAs of a sequence that have read its length (append-then-step)
  int fused_cs;           // cluster size of the cluster kernel (step and top-k), 0 = not available
  int fused_step_ok;      // the one-launch step supports this configuration
  size_t fused_smem;      // its dynamic shared memory
  int step_threads;       // the decode step's own shape: 512 threads with fused_cs CTAs per cluster, or the wide
  int step_cs;            // form (1024 threads, one CTA per SM, half the cluster) where that evens out the stream
  size_t step_smem;
  int step_resident;      // clusters of the step's shape that the device holds at once
  int use_fused;          // fasa_decode_step takes the one-launch kernel when it is available
  int topk_rows;          // fasa_topk by the one-CTA-per-row kernel whatever the number of rows (fasa_set_step_mode 2)
  // host-buffer step: the last host pointers seen and what the device can use in their place
  // (null: not page-locked + mapped), so that a decode loop with fixed buffers asks the driver once
  const void* host_seen[4];
  void* host_mapped[4];
  const void* cache_seen;   // the last K/V cache pointer asked about, and whether it is host memory
  int cache_on_host;
  long long launches;     // kernels launched through this context
  char cuda_err[256];
};

// Records a CUDA failure in the context and returns FASA_ERR_CUDA from the caller.
#define FASA_CUDA_TRY(ctx, expr)                                                       \
  do {                                                                                 \
    cudaError_t e_ = (expr);                                                           \
    if (e_ != cudaSuccess) {                                                           \
      snprintf((ctx)->cuda_err, sizeof((ctx)->cuda_err), "%.120s: %.100s", #expr,      \
               cudaGetErrorString(e_));                                                \
      return FASA_ERR_CUDA;                                                            \
    }                                                                                  \
  } while (0)

#define FASA_LAUNCH_CHECK(ctx)                                                         \
  do {                                                                                 \
    (ctx)->launches += 1;                                                              \
    FASA_CUDA_TRY(ctx, cudaGetLastError());                                            \
  } while (0)

// How the attention kernels cut a list of at most n_upper rows per unit into splits, given
// the number of units (grid.y) of the launch.
struct fasa_split_plan {
  int n_splits;   // grid.x
  int chunk;      // rows per split (multiple of 32)
};
fasa_split_plan fasa_plan_splits(const fasa_ctx* ctx, int n_upper, int units);

// One-launch decode step (fasa_fused.cu): plan at context creation, launch per step.
int fasa_fused_plan(fasa_ctx* ctx);
int32_t fasa_fused_launch(fasa_ctx* ctx, const void* q, const void* k_cache, const void* v_cache,
                          const void* proxy_k, const int32_t* seq_lens, int32_t budget,
                          int32_t n_sel_max, float* scores, int32_t* idx, int32_t* n_sel,
                          float* out, float* lse, const void* k_new, const void* v_new,
                          cudaStream_t stream, bool with_attention = true, float* out_mirror = nullptr);
// Large selections are attended by the split-K tensor-core kernel rather than inside the
// cluster kernel (whose attention phase runs on CUDA cores at 64 registers per thread).  When
// the cluster kernel's grid needs several waves of CTAs, every wave pays for its attention
// phase with idle HBM while one split-K launch covers all units at once: the hand-over then
// starts at much smaller selections (measured at B 16 x 8 heads, 64-128 K: 202 vs 223 us at
// budget 256, 218 vs 250 us at 1024).
static inline bool fasa_attend_separately(const fasa_ctx* ctx, int n_sel_max, const void* workspace) {
  const long long rows = (long long)n_sel_max * ((ctx->sel_heads + 3) / 4);
  const long long ctas = (long long)ctx->cfg.batch * ctx->n_sets * ctx->fused_cs;
  const bool several_waves = ctas > 2ll * ctx->n_sm;
  // One wave: the two extra launches pay off once a unit has ~512 rows to attend and the
  // units together ~24 K (B 8 x 8 heads, 64 K: 82.9 vs 86.0 us at budget 512, 87.0 vs 98.3 us
  // at 1024; B 32 x 4 heads with 7 query heads each, context 4096: 48.2 vs 63.5 us; a batch-1
  // step with 8 units stays in one launch: 28.7 vs 33.7 us at budget 512).
  const long long all_rows = rows * ctx->cfg.batch * ctx->n_sets;
  return workspace != nullptr &&
         (rows >= 2048 || (several_waves && rows >= 256) || (rows >= 512 && all_rows >= 24576));
}

cudaError_t fasa_stage_from_mapped(void* dq, const void* sq, size_t q_bytes, void* dk, const void* sk, void* dv,
                                   const void* sv, size_t kv_bytes, cudaStream_t stream);

int32_t fasa_sparse_attn_mirrored(fasa_ctx* ctx, const void* q, const void* k_cache, const void* v_cache,
                                  const int32_t* idx, const int32_t* n_sel, int32_t n_sel_max, float* out,
                                  float* lse, void* workspace, cudaStream_t stream, float* out_mirror, bool* mirrored);

// Split key cache (memory-optimised variant): what the attention kernels need besides k_nondom.
// The rows every step attends to (the sink positions and the recent window) can stay on the GPU:
// a slot per sink position and a ring of n_recent slots for the positions behind them, each
// tagged with the position it holds.  A slot holds the key row as the attention kernel
// assembles it (non-dominant channels, then the dominant pairs in proxy order) and the value row.
struct fasa_resident {
  int32_t* tags;                // [batch * n_kv_heads][slots_pad]: position held by each slot, -1 = none
  uint16_t* rows;               // [batch * n_kv_heads][slots][2][128]
  int slots, slots_pad, n_sink, n_recent;   // tags == nullptr: no resident rows
};
__host__ __device__ inline int fasa_resident_slot(const fasa_resident& r, int tok) {
  if (tok < r.n_sink) return tok;
  return r.n_recent > 0 ? r.n_sink + (tok - r.n_sink) % r.n_recent : -1;
}
struct fasa_ksplit {
  const unsigned char* proxy;   // the dominant part, on the GPU
  const int16_t* ndchan;        // [n_kv_heads][nd]
  const int16_t* chan;          // [n_kv_heads][2 n_dom]
  int chunks, nd;               // 16-byte chunks per proxy row; non-dominant channels per key
  fasa_resident res;            // rows that need not cross the host link
};
fasa_resident fasa_resident_of(const fasa_ctx* ctx);
int32_t fasa_attn_split_keys(fasa_ctx* ctx, const void* q, const void* k_nondom, const void* v_cache, const void* proxy_k,
                             const int32_t* idx, const int32_t* n_sel, int32_t n_sel_max, float* out, float* lse,
                             void* workspace, cudaStream_t stream);
bool fasa_on_host(fasa_ctx* ctx, const void* p);

bool fasa_topk_row_ok(const fasa_ctx* ctx);
int32_t fasa_topk_row_launch(fasa_ctx* ctx, const float* scores, const int32_t* seq_lens, int32_t budget,
                             int32_t n_sel_max, int32_t* idx, int32_t* n_sel, int rows_per_seq, int n_sink,
                             int n_recent, cudaStream_t stream, int q_len);
int32_t fasa_fused_topk_launch(fasa_ctx* ctx, const float* scores, const int32_t* seq_lens,
                               int32_t budget, int32_t n_sel_max, int32_t* idx, int32_t* n_sel,
                               cudaStream_t stream);

// q_len > 1: the rows of a sequence are (query, set) pairs, query-major, and query t of the
// block sees seq_lens[b] - (q_len - 1 - t) positions.
int32_t fasa_fused_topk_rows(fasa_ctx* ctx, const float* scores, const int32_t* seq_lens,
                             int32_t budget, int32_t n_sel_max, int32_t* idx, int32_t* n_sel,
                             int rows_per_seq, int n_sink, int n_recent, cudaStream_t stream, int q_len = 1);

// Paged caches: how a (sequence, token) pair finds its page.  All zero = contiguous caches.
struct PageMap {
  const int32_t* table;   // [batch][pages_per_seq]: physical page of each logical page
  int shift;              // log2(tokens per page)
  int pages_per_seq;
  int n_pages;
};
static inline PageMap fasa_page_map(const fasa_ctx* ctx) {
  PageMap m;
  m.table = ctx->block_table;
  m.shift = ctx->page_shift;
  m.pages_per_seq = ctx->pages_per_seq;
  m.n_pages = ctx->cfg.n_pages;
  return m;
}
// Paged contexts need their block table before any call that touches a cache.
static inline bool fasa_pages_ready(const fasa_ctx* ctx) { return ctx->cfg.page_size == 0 || ctx->block_table != nullptr; }

static inline size_t fasa_align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

#ifdef __CUDACC__

// Two bf16 packed in a 32-bit word -> two fp32 (exact).
__device__ __forceinline__ float2 bf16x2_to_f32x2(uint32_t w) {
  return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}

__device__ __forceinline__ float bf16_bits_to_f32(uint16_t b) {
  return __uint_as_float(((uint32_t)b) << 16);
}

// 128-bit read-only load that does not allocate in L1 (streamed once).
__device__ __forceinline__ uint4 ld_stream_u4(const void* p) {
  uint4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p));
  return r;
}

// Dot product of 8 fp32 (as 4 float2) with 8 bf16 (one uint4), packed FMAs.
__device__ __forceinline__ float dot8(const float2 (&q)[4], const uint4& k) {
  float2 a = make_float2(0.f, 0.f);
  a = __ffma2_rn(q[0], bf16x2_to_f32x2(k.x), a);
  a = __ffma2_rn(q[1], bf16x2_to_f32x2(k.y), a);
  a = __ffma2_rn(q[2], bf16x2_to_f32x2(k.z), a);
  a = __ffma2_rn(q[3], bf16x2_to_f32x2(k.w), a);
  return a.x + a.y;
}

__device__ __forceinline__ bool page_ok(const PageMap& m, int page) { return page >= 0 && page < m.n_pages; }
__device__ __forceinline__ int page_of(const PageMap& m, int b, int tok) {
  return __ldg(m.table + (int64_t)b * m.pages_per_seq + (tok >> m.shift));
}
// Element offset of row `tok` of (sequence b, KV head h) in a K or V cache, for reading: an
// entry outside the pool reads page 0 and raises the status bit.
__device__ __forceinline__ int64_t cache_row(const PageMap& m, int b, int h, int tok, int64_t sb, int64_t sh,
                                             int64_t st, int32_t* status) {
  if (m.table == nullptr) return b * sb + h * sh + (int64_t)tok * st;
  int page = page_of(m, b, tok);
  if (!page_ok(m, page)) {
    atomicOr(status, FASA_DEV_PAGE_CLAMPED);
    page = 0;
  }
  return page * sb + h * sh + (int64_t)(tok & ((1 << m.shift) - 1)) * st;
}
// Byte offset of the proxy tile of token tile T (tokens 16 T .. 16 T + 15) of (b, h).
// status == nullptr: a speculative read (a tile that may lie past the sequence's end, where no
// page need be mapped) - page 0 is read and nothing is reported.
__device__ __forceinline__ int64_t proxy_tile_offset(const PageMap& m, int b, int h, int n_kv_heads, int T,
                                                     int tiles_per_unit, int tile_bytes, int32_t* status) {
  if (m.table == nullptr) return ((int64_t)(b * n_kv_heads + h) * tiles_per_unit + T) * tile_bytes;
  int page = (T >> (m.shift - 4)) < m.pages_per_seq ? page_of(m, b, T << 4) : -1;
  if (!page_ok(m, page)) {
    if (status) atomicOr(status, FASA_DEV_PAGE_CLAMPED);
    page = 0;
  }
  const int tpp = 1 << (m.shift - 4);           // tiles per page
  return (((int64_t)page * n_kv_heads + h) * tpp + (T & (tpp - 1))) * tile_bytes;
}

// Reports (status bit) a token tile whose page is not in the pool; for tiles that were read
// speculatively and turned out to be part of the sequence.
__device__ __forceinline__ void proxy_tile_check(const PageMap& m, int b, int T, int32_t* status) {
  if (m.table != nullptr && !page_ok(m, page_of(m, b, T << 4))) atomicOr(status, FASA_DEV_PAGE_CLAMPED);
}

// A selection unit: `heads` consecutive query heads of one sequence that share an index set
// (Sec. 4.1 keeps a set per head; by default all heads of a KV head share one).  Unit u of
// the grid is set hs = u % n_sets of sequence b = u / n_sets.
struct SelUnit {
  int b;        // sequence
  int h;        // KV head whose cache the unit reads
  int kv;       // b * n_kv_heads + h: index of that cache (K, V, proxy, appended rows)
  int64_t q0;   // b * n_q_heads + first query head of the unit: row of q, out and lse
};
__device__ __forceinline__ SelUnit sel_unit(int u, int n_sets, int heads, int n_q_heads, int n_kv_heads) {
  SelUnit s;
  const int hs = u % n_sets;
  s.b = u / n_sets;
  s.h = hs / (n_sets / n_kv_heads);
  s.kv = s.b * n_kv_heads + s.h;
  s.q0 = (int64_t)s.b * n_q_heads + (int64_t)hs * heads;
  return s;
}

__device__ __forceinline__ int clamp_len(int len, int max_len, int32_t* status) {
  if (len < 0 || len > max_len) {
    atomicOr(status, FASA_DEV_LEN_CLAMPED);
    len = len < 0 ? 0 : max_len;
  }
  return len;
}

#endif  // __CUDACC__
