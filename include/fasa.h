/*
 * fasa.h - C ABI of the B200 (sm_100a) decode-time hot path of FASA,
 * Frequency-Aware Sparse Attention (arxiv 2602.03152).
 *
 * One decode step per (batch b, KV head h) - or per smaller set of query heads, see
 * "Index sets" below - in the paper's order:
 *   fasa_kv_append          cache update, incl. the dominant part of the key cache
 *                           (C_key^dom of Algorithm 2, kept here as a packed
 *                           "proxy-K" side buffer)
 *   fasa_fc_score           TIP: S_t = sum_{i in I_dom} alpha^(i)       (Sec. 4.1)
 *   fasa_topk               T_t = TopK-I(S_t, N_fac)                    (Sec. 4.1)
 *   fasa_sparse_decode_attn FAC: Softmax(q K_T^T / sqrt(d)) V_T         (Sec. 4.2, Eq. 6-7)
 *   fasa_full_decode_attn   full-KV attention, the FKV baseline         (Sec. 5.1)
 *
 * Conventions
 *   - Every tensor argument is a DEVICE pointer owned by the caller unless its
 *     name ends in _host.  The library owns only the context and a few hundred
 *     bytes of device tables inside it.  Nothing is allocated per call.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*; NULL = the
 *     legacy default stream) and return without synchronising, except where
 *     stated.  A non-zero return means nothing was enqueued by that call.
 *   - bf16 = IEEE binary32 upper half, 2 bytes.  head_dim is 128.
 *   - Layouts are row-major.  K and V: [batch][n_kv_heads][max_len][128] bf16
 *     (or the strides in fasa_config_t), keys stored post-RoPE at their
 *     absolute positions.  q: [batch][n_q_heads][128] bf16, post-RoPE; query
 *     head g belongs to KV head g / (n_q_heads / n_kv_heads).
 *   - Where the caches live.  k_cache and v_cache (not proxy_k) may instead be page-locked
 *     host memory that the device can address (cudaHostAlloc / cudaHostRegister under
 *     unified addressing): this is the memory-optimised variant of the method (FASA-M,
 *     Algorithm 2), which keeps only the dominant part of the key cache - here the proxy-K
 *     buffer - on the GPU.  Every call works unchanged: scoring and selection run on the
 *     GPU-resident proxy, the attention kernels fetch just the selected K/V rows across
 *     the host link by index (no host-side gather, no staging copy), and the append calls
 *     store the new rows there.  GPU memory per cached token drops from 512 bytes to
 *     proxy_row_elems * 2 (64 at n_dom = 16); a step then moves n_sel * 512 bytes per
 *     (batch, KV head) over the link, which bounds it.  The dense path over host-resident
 *     caches streams the whole cache over the link and is only useful as a reference.
 *     The attention calls ask the driver once per k_cache pointer whether it is host memory
 *     (rows in host memory are copied through L1, which doubles the link's throughput) and
 *     remember the answer for the last pointer seen: k_cache and v_cache must be of the same
 *     kind, and a buffer must not change its kind while keeping its address.
 *   - Paged caches (page_size > 0).  K, V and the proxy are pools of n_pages pages of
 *     page_size tokens, shared by the sequences; a block table, int32
 *     [batch][ceil(max_len / page_size)] on the device, names the physical page of every
 *     logical page of a sequence (fasa_set_block_table; the caller owns it and may rewrite
 *     it between calls, in stream order).  K and V: [n_pages][n_kv_heads][page_size][128],
 *     or any layout the stride fields describe with stride_b read as the PAGE stride;
 *     proxy: [n_pages][n_kv_heads][page_size / 16 tiles], fasa_proxy_bytes() in all.
 *     Token positions everywhere else (seq_lens, idx, scores) stay logical.  Reads through
 *     an entry outside [0, n_pages) use page 0 and set FASA_DEV_PAGE_CLAMPED, writes through
 *     one are dropped.  Every call takes paged caches, the one-launch step included.
 *   - Frequency chunk (FC) i, 0 <= i < 64, is the channel pair (i, i+64) with
 *     rope_pairing 0 (rotate-half layout) or (2i, 2i+1) with rope_pairing 1
 *     (the paper's Eq. 1 layout).  An FC is never split (Appendix, design choices).
 *   - Proxy-K buffer: fasa_proxy_bytes() bytes, 16-byte aligned, zero-filled once by
 *     the caller.  Per (batch, kv head) it holds ceil(max_len / 16) tiles of 16 tokens;
 *     a token owns proxy_row_elems = 8 * ceil(n_dom / 4) bf16 values: for the head's
 *     dominant FCs sorted ascending, the pairs (K[j][c0], K[j][c1]), zero padded.
 *     Inside a tile the values are stored in the operand order of the tensor-core
 *     instruction that scores them (blocks of 16 channels, 512 bytes each, lane
 *     4g+t of a warp owning {P[g][2t..2t+1], P[g+8][2t..2t+1], P[g][2t+8..2t+9],
 *     P[g+8][2t+8..2t+9]}; a trailing block of 8 channels, 256 bytes, when
 *     ceil(n_dom / 4) is odd).  Only fasa_kv_append, fasa_proxy_build and
 *     fasa_append_decode_step write it; treat it as opaque.
 *   - Index sets.  The paper keeps one index set T_t per (layer, head) (Sec. 4.1).  With
 *     grouped-query attention the default here is one set per KV head, scored by all its
 *     query heads together, so that each selected K/V row is gathered once per KV head.
 *     select_heads = s makes every s consecutive query heads share a set instead (s = 1:
 *     a set per query head, the paper's literal reading; s must divide n_q_heads /
 *     n_kv_heads).  With n_sets = n_q_heads / s sets per sequence, set hs covers query
 *     heads hs*s .. hs*s+s-1 and reads the cache of their KV head; scores, idx and n_sel
 *     have n_sets rows per sequence wherever the text below says n_kv_heads (I_dom, K, V
 *     and the proxy stay per KV head).  Gathered K/V traffic grows by the group size / s.
 *   - Data-dependent problems (a sequence longer than max_len, an index out of
 *     range) never fault: the kernel clamps and ORs a bit into a device status
 *     word read by fasa_get_device_status.
 *   - One context, one stream order.  The status word and the per-sequence arrival
 *     counters with which the appending calls update seq_lens belong to the context.
 *     Calls on the same context must therefore be ordered on the device (one stream, or
 *     streams joined by events): two appending calls of one context that overlap corrupt
 *     the length update without any error.  Different contexts are independent (apart from
 *     the shared array of fasa_sparse_decode_attn_static, see there).
 */
#ifndef FASA_H_
#define FASA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FASA_OK                 0
#define FASA_ERR_INVALID_ARG   -1   /* null pointer, non-positive size, bad alignment      */
#define FASA_ERR_UNSUPPORTED   -2   /* head_dim != 128, n_dom outside 1..64, group > 8 ... */
#define FASA_ERR_WORKSPACE     -3   /* n_sel_max / budget larger than the workspace covers */
#define FASA_ERR_CUDA          -4   /* a CUDA runtime call failed (see fasa_last_cuda_error) */
#define FASA_ERR_TIMEOUT       -5   /* reserved: no kernel waits for another; see FASA_DEV_TIMEOUT */

/* Bits of the device status word. */
#define FASA_DEV_LEN_CLAMPED    1   /* a seq_lens entry was < 0 or > max_len               */
#define FASA_DEV_APPEND_FULL    2   /* kv_append ran out of rows; the excess was dropped   */
#define FASA_DEV_IDX_CLAMPED    4   /* sparse attention met an index outside [0, max_len)  */
#define FASA_DEV_NSEL_CLAMPED   8   /* n_sel exceeded n_sel_max                            */
#define FASA_DEV_PAGE_CLAMPED  16   /* a block-table entry was < 0 or >= n_pages           */
#define FASA_DEV_TIMEOUT       32   /* a bounded wait inside a kernel ran out; results of  */
                                    /* that launch are undefined, the context stays usable */

typedef struct fasa_ctx fasa_ctx_t;

typedef struct {
  int32_t batch, n_q_heads, n_kv_heads, head_dim; /* head_dim must be 128                  */
  int32_t max_len;        /* rows allocated per (b, kv head) in K, V, proxy and scores     */
  int32_t n_dom;          /* F = N_tip: dominant FCs per KV head, 1..64                    */
  int32_t rope_pairing;   /* 0: FC i = (i, i+64); 1: FC i = (2i, 2i+1)                     */
  int32_t group_reduce;   /* score of an index set over its query heads: 0 sum, 1 max      */
  int32_t select_heads;   /* query heads that share one index set: 0 => all heads of a KV  */
                          /* head; 1 => a set per query head; else a divisor of the group  */
  int32_t n_sink;         /* first n_sink positions are always selected                    */
  int32_t n_recent;       /* last n_recent positions are always selected                   */
  float   softmax_scale;  /* 0 => 1/sqrt(head_dim)                                         */
  int64_t k_stride_b, k_stride_h, k_stride_t; /* in elements; all 0 => dense layout above  */
  int64_t v_stride_b, v_stride_h, v_stride_t; /* stride_t must be a multiple of 8          */
  int32_t page_size;      /* 0: one contiguous cache per sequence; else tokens per page    */
                          /* (a power of two >= 16) of a paged cache, see "Paged caches"   */
  int32_t n_pages;        /* pages in the pool (paged caches only)                         */
} fasa_config_t;

/* ---- context (off the hot path) ----------------------------------------- */

/* Validates cfg, sorts each head's dominant-FC list and uploads the channel
 * table to the current device.  dom_fc_host: [n_kv_heads][n_dom] distinct FC
 * indices in 0..63 (the calibrated I_dom of Sec. 4.1; Algorithm 1 produces it).
 * Synchronises the device once.  Errors: INVALID_ARG (null, duplicate or
 * out-of-range FC), UNSUPPORTED, CUDA. */
int32_t fasa_create(const fasa_config_t* cfg, const int32_t* dom_fc_host, fasa_ctx_t** out);
int32_t fasa_destroy(fasa_ctx_t* ctx);

/* Paged caches: the block table the calls after this one translate token positions with
 * (device pointer, int32 [batch][ceil(max_len / page_size)], kept by reference).
 * INVALID_ARG for a context with page_size == 0 or a null table. */
int32_t fasa_set_block_table(fasa_ctx_t* ctx, const int32_t* block_table);

/* bf16 values per token in the proxy-K buffer for n_dom dominant FCs: 8 * ceil(n_dom / 4). */
int32_t fasa_proxy_row_elems(int32_t n_dom);
/* Size of the proxy-K buffer of this context:
 * batch * n_kv_heads * 16 * ceil(max_len / 16) * proxy_row_elems * 2 bytes, or
 * n_pages * n_kv_heads * page_size * proxy_row_elems * 2 bytes for paged caches. */
int32_t fasa_proxy_bytes(const fasa_ctx_t* ctx, size_t* out_bytes);

/* Bytes of caller-provided scratch that fasa_topk, the two attention calls and
 * fasa_decode_step need for selections of at most n_sel_max tokens.  The
 * workspace must be 256-byte aligned; its contents need not be preserved
 * between calls, and two calls that overlap on the GPU need separate ones. */
int32_t fasa_workspace_bytes(const fasa_ctx_t* ctx, int32_t n_sel_max, size_t* out_bytes);

const char* fasa_status_string(int32_t status);
/* Text of the last CUDA error a call of this library met in this thread's context. */
const char* fasa_last_cuda_error(const fasa_ctx_t* ctx);
/* Synchronises `stream`, copies the device status word to *host_out and clears it. */
int32_t fasa_get_device_status(fasa_ctx_t* ctx, void* stream, int32_t* host_out);
/* Number of kernels this context has launched so far (host-side counter). */
int64_t fasa_launch_count(const fasa_ctx_t* ctx);

/* ---- cache update (Algorithm 2: Split + UpdateCache) -------------------- */

/* Appends n_new rows per (b, kv head): K and V rows go to rows seq_lens[b] ..
 * seq_lens[b]+n_new-1 of the caches, the dominant-FC slices of the new keys go
 * to the same rows of proxy_k, then seq_lens[b] += n_new (on the device, in
 * stream order).  k_new, v_new: bf16 [batch][n_kv_heads][n_new][128], post-RoPE.
 * Rows that would pass max_len are dropped and FASA_DEV_APPEND_FULL is set.
 * One launch: a row per half-CTA for a few rows, 16 rows per CTA (keys staged in
 * shared memory once) from n_new = 16 on, the size of a prompt. */
int32_t fasa_kv_append(fasa_ctx_t* ctx, void* k_cache, void* v_cache, void* proxy_k,
                       int32_t* seq_lens, const void* k_new, const void* v_new,
                       int32_t n_new, void* stream);

/* Fills proxy_k rows 0 .. seq_lens[b]-1 from a key cache that was written by
 * other means (a prefill): the Split of Algorithm 2 applied to the whole cache. */
int32_t fasa_proxy_build(fasa_ctx_t* ctx, const void* k_cache, void* proxy_k,
                         const int32_t* seq_lens, void* stream);

/* ---- TIP: importance scores (Sec. 4.1) ---------------------------------- */

/* scores[b][h][j] = reduce_{g in group(h)} sum_{i in I_dom(h)}
 *                   (q[b][g][c0(i)] K[j][c0(i)] + q[b][g][c1(i)] K[j][c1(i)])
 * for j < seq_lens[b], read from proxy_k; exact bf16 products accumulated in fp32 per
 * query head on tensor cores, the heads then reduced in fp32; no scaling.
 * scores: fp32 [batch][n_kv_heads][max_len] (n_sets rows per sequence with select_heads,
 * here and for idx / n_sel below; see "Index sets"); entries at j >= seq_lens[b] are left
 * untouched.  -0 is stored as +0. */
int32_t fasa_fc_score(fasa_ctx_t* ctx, const void* q, const void* proxy_k,
                      const int32_t* seq_lens, float* scores, void* stream);

/* ---- TopK-I (Sec. 4.1) --------------------------------------------------- */

/* Per (b, h) with L = seq_lens[b]: forced = positions < n_sink or >= L - n_recent;
 * T = forced U the `budget` best-scoring other positions, higher score first and
 * lower index first among equal scores; n_sel = min(L, |forced| + budget).
 * budget > 0 is N_fac itself; budget < 0 means ceil(-budget/1000 * L) (device-side,
 * so a length that grows each step needs no host round trip).
 * idx: int32 [batch][n_kv_heads][n_sel_max], ascending; entries past n_sel are
 * left untouched.  n_sel: int32 [batch][n_kv_heads].  If n_sel would exceed
 * n_sel_max the selection is cut to the n_sel_max best and FASA_DEV_NSEL_CLAMPED
 * is set.  NaN scores rank above +inf (their sign bit clear) or below -inf. */
int32_t fasa_topk(fasa_ctx_t* ctx, const float* scores, const int32_t* seq_lens,
                  int32_t budget, int32_t n_sel_max, int32_t* idx, int32_t* n_sel,
                  void* workspace, void* stream);

/* ---- FAC (Sec. 4.2, Eq. 6-7) and FKV (Sec. 5.1) -------------------------- */

/* out[b][g][:] = sum_j p_j V[idx_j],  p = softmax_j(q[b][g] . K[idx_j] * scale) over
 * the n_sel[b][h] rows listed in idx (any order, rows used as stored).  fp32
 * accumulation; out fp32 [batch][n_q_heads][128]; lse (nullable) fp32
 * [batch][n_q_heads] = log sum_j exp(logit_j).  n_sel == 0 gives out = 0,
 * lse = -inf.  Split over the selection; the splits of a unit merge inside the same launch (they
 * form one thread-block cluster) up to n_sel_max = 16384, through `workspace` and a second
 * kernel beyond. */
int32_t fasa_sparse_decode_attn(fasa_ctx_t* ctx, const void* q, const void* k_cache,
                                const void* v_cache, const int32_t* idx, const int32_t* n_sel,
                                int32_t n_sel_max, float* out, float* lse, void* workspace,
                                void* stream);

/* The same over all rows j < seq_lens[b], no index list. */
int32_t fasa_full_decode_attn(fasa_ctx_t* ctx, const void* q, const void* k_cache,
                              const void* v_cache, const int32_t* seq_lens, float* out,
                              float* lse, void* workspace, void* stream);

/* ---- for callers that cannot allocate ------------------------------------ */

/* Size of the built-in scratch area of fasa_sparse_decode_attn_static (bytes). */
#define FASA_STATIC_SCRATCH_BYTES (4u << 20)

/* (No counterpart in the paper: a packaging variant of fasa_sparse_decode_attn.)
 * Some callers have no way to hand the library a workspace: code that runs where
 * cudaMalloc is off limits (inside a memory pool it does not own, under a plugin
 * interface that passes only inputs and outputs, in a real-time loop that may not
 * touch the allocator).  For them this call computes exactly what
 * fasa_sparse_decode_attn computes, with the split-K partial results kept in a
 * fixed FASA_STATIC_SCRATCH_BYTES array that is part of the library image; each
 * GPU that loads the library holds that array until the process exits.  The call
 * allocates and frees nothing, on the host or the device.
 *   - Arguments, layouts and results: as fasa_sparse_decode_attn, minus `workspace`.
 *   - Limit: batch * n_q_heads * n_splits * 130 * 4 bytes must fit the array, where
 *     n_splits is the split count the library picks for n_sel_max (at most
 *     ceil(n_sel_max / 64)); otherwise FASA_ERR_WORKSPACE is returned and nothing is
 *     enqueued.  Configuration 1 of the benchmarks needs 0.1 MB, configuration 2 1.4 MB.
 *   - The context's device must be current (FASA_ERR_INVALID_ARG otherwise).  The first
 *     call on a device looks up the array's device address (a CUDA runtime query, no
 *     allocation; where the CUDA runtime loads modules lazily, that query is also what
 *     places the library's module, array included, on the device); make that first call
 *     before any stream capture begins.  The address is remembered per device for the
 *     life of the process and does not survive a cudaDeviceReset.
 *   - All calls in the process share the one array per device.  Nothing in it has to
 *     start at zero (every partial that is read was written by the same call), but
 *     two calls whose kernels overlap on the GPU (different streams, or different
 *     contexts on the same device) race on it: keep them on one stream, or ordered. */
int32_t fasa_sparse_decode_attn_static(fasa_ctx_t* ctx, const void* q, const void* k_cache,
                                       const void* v_cache, const int32_t* idx,
                                       const int32_t* n_sel, int32_t n_sel_max, float* out,
                                       float* lse, void* stream);

/* ---- whole step ---------------------------------------------------------- */

/* Scoring, selection and attention of one step, on one stream with no host round trip.
 * idx and n_sel are outputs too; so is scores unless it is NULL.
 *
 * Mode 1 (default where available): ONE kernel, one thread-block cluster per (batch, KV
 * head); scores, histograms and split partials stay in (distributed) shared memory, so
 * `workspace` may be NULL and `scores` may be NULL (they are then not written).  Available
 * when ceil(max_len / 16) <= 22528 and the device can co-schedule such a cluster;
 * fasa_step_cluster_size tells.
 * When a workspace is given and the selection is large (n_sel_max * ceil(heads per set / 4)
 * >= 2048; >= 512 when all units together reach 24576 such rows; >= 256 when the cluster
 * kernel's grid exceeds two CTAs per SM), mode 1 ends the
 * cluster kernel after the selection and attends with the split-K tensor-core kernel of
 * fasa_sparse_decode_attn (two launches instead of one; three beyond 16384 selected rows).  The
 * same hand-over happens, whatever the selection size, when the caches are page-locked host
 * memory and an index set serves more than four query heads (the cluster kernel would fetch
 * every row twice over the host link).
 * Mode 0, and every configuration mode 1 cannot take: fasa_fc_score -> fasa_topk ->
 * fasa_sparse_decode_attn; scores and workspace are then required (INVALID_ARG if NULL).
 * Both modes select identical index sets; outputs agree to fp32 rounding.
 * n_sel_max is also the bound the launch shapes are planned with (route, split count): a
 * caller that knows the current lengths should pass the tightest bound it can (e.g.
 * ceil(0.189 * L) + n_sink + n_recent for a permille budget) rather than the bound at
 * max_len; idx is addressed with whatever n_sel_max is passed as its row stride. */
int32_t fasa_set_step_mode(fasa_ctx_t* ctx, int32_t mode);
/* (The mode also selects the kernel behind fasa_topk: the cluster kernel's selection phases
 * in mode 1, a register-resident cluster kernel in mode 0; the results are identical.  Launches
 * with more score rows than the step has units - fasa_topk_batched, the calibration - take a
 * third kernel, one CTA per row, which re-reads the row once per radix level instead of
 * holding its keys; mode 2 is mode 1 with that kernel behind fasa_topk as well, for rows of
 * up to 524288 tokens.) */
/* Cluster size mode 1 runs with for this context; 0 = fasa_decode_step uses mode 0. */
int32_t fasa_step_cluster_size(const fasa_ctx_t* ctx);
int32_t fasa_decode_step(fasa_ctx_t* ctx, const void* q, const void* k_cache,
                         const void* v_cache, const void* proxy_k, const int32_t* seq_lens,
                         int32_t budget, int32_t n_sel_max, float* scores, int32_t* idx,
                         int32_t* n_sel, float* out, float* lse, void* workspace, void* stream);

/* Algorithm 2's order for one new token per sequence: UpdateCache (K, V and the dominant
 * part of the key cache), then the step above on the grown cache; seq_lens[b] += 1 on the
 * device.  k_new, v_new: bf16 [batch][n_kv_heads][1][128], post-RoPE, 16-byte aligned.
 * In mode 1 the append happens inside the same kernel (the CTA whose slice ends the
 * sequence writes the three rows before it scores them), so the whole step is one launch;
 * otherwise it is fasa_kv_append followed by fasa_decode_step.  A full cache drops the
 * token and sets FASA_DEV_APPEND_FULL, as fasa_kv_append does. */
int32_t fasa_append_decode_step(fasa_ctx_t* ctx, const void* q, const void* k_new,
                                const void* v_new, void* k_cache, void* v_cache, void* proxy_k,
                                int32_t* seq_lens, int32_t budget, int32_t n_sel_max,
                                float* scores, int32_t* idx, int32_t* n_sel, float* out,
                                float* lse, void* workspace, void* stream);

/* Token importance prediction and selection of one step in ONE launch (TIP then TopK-I,
 * Sec. 4.1): what fasa_decode_step does before it attends, for callers that run their own
 * attention over the selected rows (or want the index sets alone).  Outputs idx, n_sel and,
 * unless NULL, scores, exactly as fasa_fc_score followed by fasa_topk give them.  k_new and
 * v_new (both NULL, or both bf16 [batch][n_kv_heads][1][128]) make it the appending form:
 * UpdateCache first, as in fasa_append_decode_step, and seq_lens[b] += 1.  Only the cluster
 * kernel provides this: FASA_ERR_UNSUPPORTED when fasa_step_cluster_size is 0. */
int32_t fasa_select_step(fasa_ctx_t* ctx, const void* q, const void* k_new, const void* v_new,
                         void* k_cache, void* v_cache, void* proxy_k, int32_t* seq_lens,
                         int32_t budget, int32_t n_sel_max, float* scores, int32_t* idx,
                         int32_t* n_sel, void* stream);

/* ---- blocks of query tokens (q_len > 1) ----------------------------------- */

/* Most query tokens per sequence that the batched calls take. */
#define FASA_MAX_QLEN 8

/* The method is defined per query token q_t (Sec. 4.1: S_t, T_t; Sec. 4.2, Eq. 6-7), so a block
 * of q_len queries per sequence - speculative or multi-token decoding - is q_len decode steps
 * over one cache: query t (0 <= t < q_len) is the query of cache row seq_lens[b] - q_len + t
 * (the block's own keys are already appended, e.g. by fasa_kv_append with n_new = q_len), it
 * sees rows j < seq_lens[b] - (q_len - 1 - t), sink / recent positions are those of that range,
 * and it has its own scores, its own index set and its own output.  Layouts gain a query axis
 * after the batch axis: q bf16 [batch][q_len][n_q_heads][128]; scores fp32
 * [batch][q_len][n_sets][max_len]; idx [batch][q_len][n_sets][n_sel_max]; n_sel
 * [batch][q_len][n_sets]; out fp32 [batch][q_len][n_q_heads][128]; lse [batch][q_len][n_q_heads].
 * What the q_len steps share is the proxy stream: fasa_fc_score_batched reads it ONCE and
 * scores all queries as one matrix product P[L x 2F] . Q[2F x (heads per set * q_len)] on the
 * tcgen05 tensor cores (fp32 accumulation in tensor memory), then reduces each query's heads
 * (sum, or max with group_reduce = 1).  q_len = 1 gives the results of the single-query calls
 * up to the rounding order of the fp32 accumulation.  fasa_topk_batched and
 * fasa_sparse_decode_attn_batched are fasa_topk and fasa_sparse_decode_attn over the
 * (sequence, query) pairs; fasa_decode_step_batched runs the three on one stream (scores and
 * workspace required).  Status FASA_ERR_UNSUPPORTED: q_len outside [1, FASA_MAX_QLEN],
 * batch * q_len * n_sets > 65535, (selection) a context without
 * a cluster shape (fasa_step_cluster_size == 0), or (attention, q_len > 1) n_sel_max > 16384. */
int32_t fasa_fc_score_batched(fasa_ctx_t* ctx, const void* q, const void* proxy_k,
                              const int32_t* seq_lens, int32_t q_len, float* scores, void* stream);
int32_t fasa_topk_batched(fasa_ctx_t* ctx, const float* scores, const int32_t* seq_lens,
                          int32_t q_len, int32_t budget, int32_t n_sel_max, int32_t* idx,
                          int32_t* n_sel, void* stream);
int32_t fasa_sparse_decode_attn_batched(fasa_ctx_t* ctx, const void* q, const void* k_cache,
                                        const void* v_cache, const int32_t* idx,
                                        const int32_t* n_sel, int32_t q_len, int32_t n_sel_max,
                                        float* out, float* lse, void* workspace, void* stream);
int32_t fasa_decode_step_batched(fasa_ctx_t* ctx, const void* q, const void* k_cache,
                                 const void* v_cache, const void* proxy_k, const int32_t* seq_lens,
                                 int32_t q_len, int32_t budget, int32_t n_sel_max, float* scores,
                                 int32_t* idx, int32_t* n_sel, float* out, float* lse,
                                 void* workspace, void* stream);

/* ---- memory-optimised variant with a split key cache (FASA-M, Algorithm 2) -------------- */

/* Algorithm 2 keeps the dominant part of the key cache on the GPU (here: the proxy-K buffer)
 * and moves the rest - the non-dominant key channels and the values - to the CPU; per step it
 * selects on the GPU, transfers K^nondom_T and V_T for the selected tokens only, and Combines
 * the key rows before the attention.  Besides handing whole-row caches in host memory to the
 * ordinary calls (see "Where the caches live"), the library therefore takes the key cache in
 * that split form:
 *   k_nondom  bf16 [batch][n_kv_heads][max_len][fasa_m_nondom_row_elems(n_dom)]: of every key
 *             the 128 - 2 n_dom channels that are NOT dominant for its head, ascending; meant
 *             for page-locked, device-addressable host memory (device memory works too);
 *   v_cache   as everywhere else, likewise in host memory; proxy_k on the GPU.
 * A selected token then costs 512 - 4 n_dom bytes on the host link instead of 512, and a group
 * of up to 8 query heads reads each row once.  Requirements: n_dom a multiple of 4 (otherwise
 * fasa_m_nondom_row_elems returns 0 and the calls FASA_ERR_UNSUPPORTED), contiguous caches.
 *   fasa_m_split        Split of an existing full key cache: writes k_nondom rows j < seq_lens[b]
 *                       (the proxy comes from fasa_proxy_build).
 *   fasa_m_kv_append    Split + UpdateCache of n_new new tokens per sequence: their dominant pairs
 *                       to the proxy, the other channels to k_nondom, the value rows to v_cache;
 *                       seq_lens[b] += n_new.  Arguments as fasa_kv_append.
 *   fasa_m_sparse_decode_attn   Combine + FAC (Eq. 6-7): the key rows of idx are assembled in
 *                       shared memory from k_nondom and the proxy.  The logits are the same dot
 *                       products as in fasa_sparse_decode_attn, summed in another channel order
 *                       (results agree to fp32 rounding, not bit for bit).
 *   fasa_m_decode_step  Algorithm 2's loop body: (k_new / v_new non-NULL: Split + UpdateCache,)
 *                       TIP and TopK-I on the proxy (the cluster kernel, one launch), then the
 *                       call above.  Needs a cluster shape (fasa_step_cluster_size > 0). */
int32_t fasa_m_nondom_row_elems(int32_t n_dom);
int32_t fasa_m_split(fasa_ctx_t* ctx, const void* k_cache, void* k_nondom, const int32_t* seq_lens,
                     void* stream);
int32_t fasa_m_kv_append(fasa_ctx_t* ctx, void* k_nondom, void* v_cache, void* proxy_k,
                         int32_t* seq_lens, const void* k_new, const void* v_new, int32_t n_new,
                         void* stream);
int32_t fasa_m_sparse_decode_attn(fasa_ctx_t* ctx, const void* q, const void* k_nondom,
                                  const void* v_cache, const void* proxy_k, const int32_t* idx,
                                  const int32_t* n_sel, int32_t n_sel_max, float* out, float* lse,
                                  void* workspace, void* stream);
int32_t fasa_m_decode_step(fasa_ctx_t* ctx, const void* q, const void* k_new, const void* v_new,
                           void* k_nondom, void* v_cache, void* proxy_k, int32_t* seq_lens,
                           int32_t budget, int32_t n_sel_max, float* scores, int32_t* idx,
                           int32_t* n_sel, float* out, float* lse, void* workspace, void* stream);

/* Rows that need not cross the host link (Sec. 4.3 pairs the memory-optimised variant with
 * prefetching; Algorithm 2, appendix).  The only rows of a step that are known before its
 * selection ends are the forced ones: the n_sink first positions and the n_recent last ones
 * (Sec. 4.1's T_t always contains them here).  With a resident buffer registered they are kept
 * on the GPU for good instead of being fetched every step: fasa_m_kv_append stores every
 * appended row that is a sink position or among the last n_recent of the grown sequence into
 * its slot (a slot per sink position, a ring of n_recent slots behind them, each tagged with
 * the position it holds), and fasa_m_sparse_decode_attn / fasa_m_decode_step copy a selected
 * row from there whenever the tag of its slot names it, from the host otherwise.  Outputs are
 * bit-identical with and without the buffer.
 *   fasa_m_resident_bytes   size of the buffer: per (sequence, KV head) n_sink + n_recent slots of
 *                           512 bytes (the key row as the kernel assembles it + the value row)
 *                           and a 4-byte tag each; 0 when n_sink + n_recent = 0 or the split key
 *                           cache is not available for this configuration.
 *   fasa_m_set_resident     registers the caller's DEVICE buffer (16-byte aligned, kept by
 *                           reference, caller-owned; NULL switches the feature off) and enqueues
 *                           the clearing of its tags on `stream`.  UNSUPPORTED when
 *                           fasa_m_resident_bytes is 0.
 *   fasa_m_resident_build   fills the slots from split caches that already hold tokens (after
 *                           fasa_m_split, or after the buffer was registered late): reads the
 *                           forced rows of the current lengths from k_nondom / v_cache / proxy_k.
 * Like the block table, the buffer belongs to the calls of one context in stream order. */
int64_t fasa_m_resident_bytes(const fasa_ctx_t* ctx);
int32_t fasa_m_set_resident(fasa_ctx_t* ctx, void* resident, void* stream);
int32_t fasa_m_resident_build(fasa_ctx_t* ctx, const void* k_nondom, const void* v_cache,
                              const void* proxy_k, const int32_t* seq_lens, void* stream);

/* End-to-end step from HOST buffers: q_host, k_new_host, v_new_host (layouts as
 * fasa_kv_append with n_new = 1) -> fasa_append_decode_step -> out copied to out_host
 * (fp32 [batch][n_q_heads][128]); synchronises the stream.  Inputs in pinned (page-locked,
 * mapped) host memory need no copy call: a step that is one launch of one wave of CTAs reads
 * them in place, across the host link; otherwise one small kernel brings them to the device
 * staging area dev_stage (>= fasa_stage_bytes) first.  Pageable inputs are copied there with
 * three asynchronous copies.  A pinned out_host is written by the step's last kernel itself.
 * The context remembers what the driver said about the last four host pointers it saw, so a
 * loop that passes the same buffers asks once; a buffer must therefore not change its kind
 * (pageable / page-locked) while keeping its address between two calls. */
int32_t fasa_stage_bytes(const fasa_ctx_t* ctx, size_t* out_bytes);
int32_t fasa_decode_step_host(fasa_ctx_t* ctx, const void* q_host, const void* k_new_host,
                              const void* v_new_host, void* dev_stage, void* k_cache,
                              void* v_cache, void* proxy_k, int32_t* seq_lens, int32_t budget,
                              int32_t n_sel_max, float* scores, int32_t* idx, int32_t* n_sel,
                              float* out, float* out_host, void* workspace, void* stream);

/* ---- offline calibration of the dominant FCs (Algorithm 1) ---------------- */

/* Contextual agreement (Sec. 3.3, Eq. 4) of each FC i with the full head, for a batch laid
 * out as for a decode step: a sample is a (sequence b, query head g) pair with
 * seq_lens[b] > top_k (shorter sequences select every position and are skipped).  For each
 * sample and each FC i the call adds
 *     | TopK-I(alpha, top_k)  n  TopK-I(alpha^(i), top_k) |          ( = top_k * CA )
 * to ca_counts[g][i] and 1 to n_used[g], where alpha^(i)[j] = q[c0(i)] K[j][c0(i)] +
 * q[c1(i)] K[j][c1(i)] are the single-FC raw scores (Eq. 3) and alpha their sum over the
 * 64 FCs, both in fp32 (alpha^(i) rounded once, alpha accumulated in ascending i); TopK-I
 * ranks higher scores first and lower indices first among equal scores.
 * q: bf16 [batch][n_q_heads][128]; k_cache as everywhere; ca_counts: int64
 * [n_q_heads][64] and n_used: int64 [n_q_heads], device, 8-byte aligned, zeroed by the
 * caller before the first call and carried from call to call (Stage 1 of Algorithm 1).
 * workspace: fasa_calib_workspace_bytes(ctx, top_k) bytes = batch * n_q_heads * 65 *
 * (max_len + top_k + 1) * 4 plus padding, 256-byte aligned.  The context's n_dom, sinks,
 * budget and select_heads play no part.  Three kernels on `stream`, no synchronisation.
 * UNSUPPORTED: top_k outside 1..min(max_len, 8192), batch * n_q_heads * 65 > 65535, or a
 * max_len the cluster kernel cannot take (fasa_step_cluster_size() == 0). */
int32_t fasa_calib_workspace_bytes(const fasa_ctx_t* ctx, int32_t top_k, size_t* out_bytes);
int32_t fasa_calib_accumulate(fasa_ctx_t* ctx, const void* q, const void* k_cache,
                              const int32_t* seq_lens, int32_t top_k, int64_t* ca_counts,
                              int64_t* n_used, void* workspace, void* stream);

/* Stage 2 of Algorithm 1, on the host (no GPU work): from counts and sample numbers copied
 * back by the caller, the mean CA of FC i for KV head h over all samples of the query
 * heads that share h, and I_dom(h) = the n_dom FCs with the highest mean (a lower index
 * first among equal means), written ascending to dom_fc_host [n_kv_heads][n_dom] - the
 * table fasa_create takes.  mean_ca_host (nullable): double [n_kv_heads][64]. */
int32_t fasa_calib_select(int32_t n_q_heads, int32_t n_kv_heads, const int64_t* ca_counts_host,
                          const int64_t* n_used_host, int32_t top_k, int32_t n_dom,
                          int32_t* dom_fc_host, double* mean_ca_host);

#ifdef __cplusplus
}
#endif
#endif /* FASA_H_ */
