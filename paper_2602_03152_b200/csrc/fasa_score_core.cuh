// Inner pieces of TIP scoring (Sec. 4.1) shared by the stand-alone scoring kernel and the
// fused decode-step kernel: how a lane obtains its slice of the (group-reduced) query and
// how the lanes of one proxy row combine their partial dot products.
#pragma once

#include "fasa_common.cuh"

// A proxy row is `chunks` 16-byte chunks; LPR lanes (a power of two >= chunks) share a row
// and lane `sub` owns chunk `sub` (8 bf16 = 4 channel pairs).  With the sum reduction the
// group's query heads are added once into registers (NG = 1); with the max reduction each
// head keeps its own slice (NG = FASA_MAX_GROUP).
template <bool MAXRED>
struct ScoreQ {
  static constexpr int NG = MAXRED ? FASA_MAX_GROUP : 1;
  float2 v[NG][4];
};

// q_unit points at the first query head of the KV head; ch at this lane's 8 channel ids.
template <bool MAXRED>
__device__ __forceinline__ void load_score_q(ScoreQ<MAXRED>& sq, const uint16_t* __restrict__ q_unit,
                                             const int16_t* __restrict__ ch, int group, bool live) {
  constexpr int NG = ScoreQ<MAXRED>::NG;
#pragma unroll
  for (int g = 0; g < NG; ++g)
#pragma unroll
    for (int e = 0; e < 4; ++e) sq.v[g][e] = make_float2(0.f, 0.f);
  if (!live) return;
  // the 8 channel ids of this lane in one 16-byte load
  const uint4 cw = *reinterpret_cast<const uint4*>(ch);
  const uint32_t cws[4] = {cw.x, cw.y, cw.z, cw.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const int c0 = (int)(int16_t)(cws[e] & 0xffffu);
    const int c1 = (int)(int16_t)(cws[e] >> 16);
    for (int g = 0; g < group; ++g) {
      const float x = c0 >= 0 ? bf16_bits_to_f32(q_unit[g * FASA_HEAD_DIM + c0]) : 0.f;
      const float y = c1 >= 0 ? bf16_bits_to_f32(q_unit[g * FASA_HEAD_DIM + c1]) : 0.f;
      if (MAXRED) {
#pragma unroll
        for (int gg = 0; gg < NG; ++gg)
          if (gg == g) sq.v[gg][e] = make_float2(x, y);
      } else {
        sq.v[0][e].x += x;
        sq.v[0][e].y += y;
      }
    }
  }
}

// Score of the row whose chunk `x` this lane holds; every lane of the row gets the result.
// -0 is turned into +0 so that equal scores have equal bit patterns.
template <int LPR, bool MAXRED>
__device__ __forceinline__ float score_row(const ScoreQ<MAXRED>& sq, const uint4& x, int group) {
  float s;
  if (!MAXRED) {
    s = dot8(sq.v[0], x);
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  } else {
    s = -INFINITY;
#pragma unroll
    for (int g = 0; g < ScoreQ<MAXRED>::NG; ++g) {
      if (g < group) {
        float sg = dot8(sq.v[g], x);
#pragma unroll
        for (int o = LPR / 2; o > 0; o >>= 1) sg += __shfl_xor_sync(0xffffffffu, sg, o);
        s = fmaxf(s, sg);
      }
    }
  }
  return s + 0.0f;
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
