// Inner pieces of TIP scoring (Sec. 4.1) shared by the stand-alone scoring kernel, the fused
// decode-step kernel and the cache-append kernels: the tiled layout of the proxy-K buffer and
// the tensor-core evaluation of  S[j] = reduce_g sum_{i in I_dom} alpha_g^(i)[j].
//
// Scoring a KV head is the skinny matrix product  P[L x 2F] . Q[2F x G]  (proxy rows times the
// dominant channels of the G query heads of the group) followed by a reduction over the G
// columns.  It is evaluated with mma.sync.m16n8k16 (bf16 inputs, fp32 accumulation): one
// instruction covers 16 tokens x 16 channels x 8 heads, where the scalar form needs about
// forty instructions per 8 tokens and is bound by instruction issue, not by HBM.
//
// Proxy layout.  Tokens are grouped in tiles of 16 rows.  A token has 8 * chunks proxy
// channels (chunks = ceil(F / 4); channel 2r, 2r+1 = the pair (K[c0], K[c1]) of the r-th
// dominant FC in ascending order, zero padded).  A tile stores, one after another,
//   n16 = chunks / 2 blocks of 16 channels, 512 bytes each: lane l = 4 g + t of a warp owns
//       16 bytes = the A fragment of mma.m16n8k16: words
//       { P[g][2t..2t+1], P[g+8][2t..2t+1], P[g][2t+8..2t+9], P[g+8][2t+8..2t+9] }
//       (rows relative to the tile, channels relative to the block), and
//   n8 = chunks % 2 block of 8 channels, 256 bytes: lane l owns 8 bytes =
//       { P[g][2t..2t+1], P[g+8][2t..2t+1] }.
// A warp therefore reads a block with one fully coalesced 16-byte (8-byte) load per lane and
// feeds it to the tensor core unchanged.  A tile takes 16 * 16 * chunks bytes, the same as
// 16 plain rows; a unit's buffer holds ceil(max_len / 16) tiles.
#pragma once

#include "fasa_common.cuh"

struct ProxyGeom {
  int chunks;      // 16-byte units per token
  int n16, n8;     // blocks per tile
  int tile_bytes;  // 256 * chunks
};

__host__ __device__ inline ProxyGeom proxy_geom(int chunks) {
  ProxyGeom g;
  g.chunks = chunks;
  g.n16 = chunks >> 1;
  g.n8 = chunks & 1;
  g.tile_bytes = 256 * chunks;
  return g;
}

// Byte offset, inside one unit's proxy buffer, of the 4-byte word that holds channel pair w
// (channels 2w, 2w+1; 0 <= w < 4 * chunks) of token `row`.
__host__ __device__ inline int64_t proxy_word_offset(const ProxyGeom& pg, int row, int w) {
  const int tile = row >> 4, r = row & 15, g = r & 7, hi = r >> 3;
  const int kb = w >> 3, wi = w & 7;
  int64_t off = (int64_t)tile * pg.tile_bytes;
  if (kb < pg.n16) {
    const int t = wi & 3, reg = (wi >> 2) * 2 + hi;
    off += kb * 512 + (g * 4 + t) * 16 + reg * 4;
  } else {                       // the 8-channel block: wi < 4
    off += pg.n16 * 512 + (g * 4 + wi) * 8 + hi * 4;
  }
  return off;
}

#ifdef __CUDACC__

// B fragments (query side) of one lane for up to KB blocks of 16 channels.
template <int KB>
struct ScoreFrag {
  uint32_t b[KB][2];
};

// q_unit: first query head of the KV head; chan_h: the head's 8 * chunks channel ids (-1 =
// padding).  Column n = lane / 4 of the B matrix is query head n (zero for n >= group).
template <int KB>
__device__ __forceinline__ void load_score_b(ScoreFrag<KB>& f, const uint16_t* __restrict__ q_unit,
                                             const int16_t* __restrict__ chan_h, int chunks,
                                             int group, int lane, int kb0 = 0) {
  const int n = lane >> 2, t = lane & 3;
  const int n_chan = chunks * 8;
#pragma unroll
  for (int kb = 0; kb < KB; ++kb) {
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      uint32_t w = 0u;
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int ci = (kb0 + kb) * 16 + half * 8 + 2 * t + e;
        uint32_t v = 0u;
        if (ci < n_chan && n < group) {
          const int ch = chan_h[ci];
          if (ch >= 0) v = q_unit[n * FASA_HEAD_DIM + ch];
        }
        w |= v << (16 * e);
      }
      f.b[kb][half] = w;
    }
  }
}

__device__ __forceinline__ uint4 ld_proxy_u4(const void* p) {
  uint4 r;
  asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
               : "l"(p)
               : "memory");
  return r;
}

__device__ __forceinline__ uint2 ld_proxy_u2(const void* p) {
  uint2 r;
  asm volatile("ld.global.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(r.x), "=r"(r.y) : "l"(p) : "memory");
  return r;
}

// The A fragments of blocks kb0 .. kb0 + KB - 1 of one tile (this lane's share).  `tile` points
// at the tile's first byte; when `ok` is false nothing is read.  Loads go through the coherent path: in the
// append-then-step form the last row of the cache is written earlier in the same launch.
template <int KB>
__device__ __forceinline__ void load_tile(uint4 (&a)[KB], const unsigned char* tile, const ProxyGeom& pg,
                                          int lane, bool ok, int kb0 = 0) {
#pragma unroll
  for (int i = 0; i < KB; ++i) {
    const int kb = kb0 + i;
    a[i] = make_uint4(0u, 0u, 0u, 0u);
    if (ok && kb < pg.n16) {
      a[i] = ld_proxy_u4(tile + kb * 512 + lane * 16);
    } else if (ok && kb == pg.n16 && pg.n8) {
      const uint2 w = ld_proxy_u2(tile + pg.n16 * 512 + lane * 8);
      a[i] = make_uint4(w.x, w.y, 0u, 0u);
    }
  }
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint4& a, const uint32_t (&b)[2]) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b[0]), "r"(b[1]));
}

// Adds the products of up to KB blocks (n_left of them exist) of one tile to c.
template <int KB>
__device__ __forceinline__ void mma_tile(float (&c)[4], const uint4 (&a)[KB], const ScoreFrag<KB>& f, int n_left) {
#pragma unroll
  for (int kb = 0; kb < KB; ++kb)
    if (kb < n_left) mma_bf16_16816(c, a[kb], f.b[kb]);     // uniform over the warp
}

// Reduces the head columns of a tile's accumulators: every lane of quad g (lanes 4g .. 4g+3)
// returns the score of row g in s_lo and of row g + 8 in s_hi.  MAXRED reduces the group by
// max instead of by sum.  -0 is turned into +0 so that equal scores have equal bit patterns.
template <bool MAXRED>
__device__ __forceinline__ void reduce_heads(const float (&c)[4], int group, int lane, float& s_lo, float& s_hi) {
  if (!MAXRED) {
    s_lo = c[0] + c[1];                                     // heads 2t and 2t+1; absent heads are exact zeros
    s_hi = c[2] + c[3];
#pragma unroll
    for (int o = 1; o <= 2; o <<= 1) {
      s_lo += __shfl_xor_sync(0xffffffffu, s_lo, o);
      s_hi += __shfl_xor_sync(0xffffffffu, s_hi, o);
    }
  } else {
    const int h0 = 2 * (lane & 3);
    const float ninf = -INFINITY;
    s_lo = fmaxf(h0 < group ? c[0] : ninf, h0 + 1 < group ? c[1] : ninf);
    s_hi = fmaxf(h0 < group ? c[2] : ninf, h0 + 1 < group ? c[3] : ninf);
#pragma unroll
    for (int o = 1; o <= 2; o <<= 1) {
      s_lo = fmaxf(s_lo, __shfl_xor_sync(0xffffffffu, s_lo, o));
      s_hi = fmaxf(s_hi, __shfl_xor_sync(0xffffffffu, s_hi, o));
    }
  }
  s_lo += 0.0f;
  s_hi += 0.0f;
}

// Scores of the 16 tokens of one tile.  Every lane of quad g (lanes 4g .. 4g+3) returns the
// score of row g in s_lo and of row g + 8 in s_hi.  MAXRED reduces the group by max instead
// of by sum.  -0 is turned into +0 so that equal scores have equal bit patterns.
template <int KB, bool MAXRED>
__device__ __forceinline__ void score_tile(const uint4 (&a)[KB], const ScoreFrag<KB>& f, int n_blocks,
                                           int group, int lane, float& s_lo, float& s_hi) {
  float c[4] = {0.f, 0.f, 0.f, 0.f};
  mma_tile<KB>(c, a, f, n_blocks);
  reduce_heads<MAXRED>(c, group, lane, s_lo, s_hi);
}

// After two tiles (A, B) every lane takes one of the 32 rows: t = lane % 4 picks
// (A, g), (A, g+8), (B, g), (B, g+8).  Returns the row offset relative to tile A's first row.
__device__ __forceinline__ int pick_row_of_pair(int lane, float a_lo, float a_hi, float b_lo, float b_hi,
                                                float& v) {
  const int t = lane & 3, g = lane >> 2;
  v = t == 0 ? a_lo : (t == 1 ? a_hi : (t == 2 ? b_lo : b_hi));
  return (t >> 1) * 16 + g + 8 * (t & 1);
}

// Order-preserving map from fp32 to uint32 (larger float <=> larger key).
__device__ __forceinline__ uint32_t fasa_order_key(float f) {
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Selection key of position j: forced (sink / recent) positions outrank every score, and
// scores are capped just below them.
__device__ __forceinline__ uint32_t fasa_item_key(float s, int j, int len, int n_sink, int n_recent) {
  if (j < n_sink || j >= len - n_recent) return 0xffffffffu;
  const uint32_t k = fasa_order_key(s);
  return k == 0xffffffffu ? 0xfffffffeu : k;
}

#endif  // __CUDACC__
