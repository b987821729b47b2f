// Log-sum-exp merge of the partial records of one (new token, query head) by one warp (a7).
// Shared by the combine kernel and by the tensor-core attention kernel's own merge, so that both
// give the same bits: the records are taken in slot order, eight at a time, with a running maximum.
#pragma once

#include "aspd_internal.cuh"

namespace aspd {

template <typename T> __device__ inline T combine_from_f32(float x);
template <> __device__ inline float combine_from_f32<float>(float x) { return x; }
template <> __device__ inline __nv_bfloat16 combine_from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Records p0 .. p0 + n - 1 of KV-head group member g; lane owns D / 32 consecutive output elements.
// The records are read past L1 (ld.global.cg): inside the attention kernel they were written by
// other CTAs of the same launch.
// PREFETCH: the next eight records are requested before the current eight are folded in (same
// arithmetic in the same order, so the same bits; a row cut into 37 parts then costs about one
// memory round trip plus five short steps instead of five round trips).
template <typename T, int D, bool PREFETCH = false>
__device__ __forceinline__ void combine_row(const float* __restrict__ ws_o, const float2* __restrict__ ws_ml, int p0, int n, int G,
                                            int g, int lane, T* __restrict__ dst) {
  constexpr int EPL = D / 32;
  float M = -INFINITY, L = 0.f, acc[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
  auto fetch = [&](int b0, float2& ml, float (&v)[8][EPL]) {
    const int cnt = min(8, n - b0);
    ml = make_float2(-INFINITY, 0.f);
    if (lane < cnt) ml = __ldcg(ws_ml + (size_t)(p0 + b0 + lane) * G + g);
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const float* row = ws_o + ((size_t)(p0 + b0 + min(u, cnt - 1)) * G + g) * D + lane * EPL;
      if constexpr (EPL == 4) {
        const float4 x = __ldcg(reinterpret_cast<const float4*>(row));
        v[u][0] = x.x; v[u][1] = x.y; v[u][2] = x.z; v[u][3] = x.w;
      } else {
        const float2 x = __ldcg(reinterpret_cast<const float2*>(row));
        v[u][0] = x.x; v[u][1] = x.y;
      }
    }
  };
  float2 ml, ml_next = make_float2(-INFINITY, 0.f);
  float v[8][EPL], v_next[8][EPL];
  if (PREFETCH && n > 0) fetch(0, ml, v);
  for (int b0 = 0; b0 < n; b0 += 8) {
    const int cnt = min(8, n - b0);
    if constexpr (PREFETCH) {
      if (b0 + 8 < n) fetch(b0 + 8, ml_next, v_next);
    } else {
      fetch(b0, ml, v);
    }
    float mb = ml.y > 0.f ? ml.x : -INFINITY;     // records of chunks with no visible key have sum 0
#pragma unroll
    for (int o = 4; o; o >>= 1) mb = fmaxf(mb, __shfl_xor_sync(0xffffffffu, mb, o));
    mb = __shfl_sync(0xffffffffu, mb, 0);         // maximum over the eight records (lanes 0..7)
    const float m_new = fmaxf(M, mb);
    const float alpha = m_new == -INFINITY ? 1.f : exp2f(M - m_new);   // M = -inf: alpha = 0
    L *= alpha;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] *= alpha;
    M = m_new;
    const float wt = (lane < cnt && ml.y > 0.f) ? exp2f(ml.x - M) : 0.f;
    float lw = ml.y * wt;
#pragma unroll
    for (int o = 4; o; o >>= 1) lw += __shfl_xor_sync(0xffffffffu, lw, o);
    L += __shfl_sync(0xffffffffu, lw, 0);
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const float wi = __shfl_sync(0xffffffffu, wt, u);
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[e] += wi != 0.f ? v[u][e] * wi : 0.f;   // a skipped record may hold anything
    }
    if constexpr (PREFETCH) {
      ml = ml_next;
#pragma unroll
      for (int u = 0; u < 8; ++u)
#pragma unroll
        for (int e = 0; e < EPL; ++e) v[u][e] = v_next[u][e];
    }
  }
  const float inv = 1.f / L;
#pragma unroll
  for (int e = 0; e < EPL; ++e) dst[lane * EPL + e] = combine_from_f32<T>(acc[e] * inv);
}

}  // namespace aspd
