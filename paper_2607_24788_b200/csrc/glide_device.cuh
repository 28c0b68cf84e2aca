// Small device helpers shared by the decode and prefill kernels.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>

#include "glide_internal.h"

namespace glide {

constexpr float kLog2e = 1.4426950408889634f;

template <typename T>
struct TypeTag {
  using type = T;
};
template <int N>
struct IntTag {
  static constexpr int value = N;
};

// Calls f(TypeTag<T>, IntTag<D>, IntTag<G>) for the configured dtype / head_dim / group size.
template <typename F>
int dispatch_config(int dtype, int D, int G, F &&f) {
#define GLIDE_DISPATCH_G(TT, DD)                                   \
  switch (G) {                                                     \
    case 1: return f(TypeTag<TT>{}, IntTag<DD>{}, IntTag<1>{});    \
    case 2: return f(TypeTag<TT>{}, IntTag<DD>{}, IntTag<2>{});    \
    case 4: return f(TypeTag<TT>{}, IntTag<DD>{}, IntTag<4>{});    \
    case 8: return f(TypeTag<TT>{}, IntTag<DD>{}, IntTag<8>{});    \
    default: return int(GLIDE_ERR_UNSUPPORTED);                    \
  }
  if (dtype == GLIDE_F32) {
    if (D == 64) { GLIDE_DISPATCH_G(float, 64) }
    if (D == 128) { GLIDE_DISPATCH_G(float, 128) }
  } else {
    if (D == 64) { GLIDE_DISPATCH_G(__nv_bfloat16, 64) }
    if (D == 128) { GLIDE_DISPATCH_G(__nv_bfloat16, 128) }
  }
#undef GLIDE_DISPATCH_G
  return int(GLIDE_ERR_UNSUPPORTED);
}

// E consecutive elements (E in {2,4}) -> fp32.  p must be aligned to E * sizeof(T).
template <typename T, int E>
__device__ __forceinline__ void load_elems(const T *p, float (&x)[E]) {
  static_assert(E == 2 || E == 4, "E");
  if constexpr (sizeof(T) == 4) {
    if constexpr (E == 4) {
      float4 v = *reinterpret_cast<const float4 *>(p);
      x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    } else {
      float2 v = *reinterpret_cast<const float2 *>(p);
      x[0] = v.x; x[1] = v.y;
    }
  } else {
    if constexpr (E == 4) {
      uint2 v = *reinterpret_cast<const uint2 *>(p);
      x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xffff0000u);
      x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xffff0000u);
    } else {
      uint32_t v = *reinterpret_cast<const uint32_t *>(p);
      x[0] = __uint_as_float(v << 16); x[1] = __uint_as_float(v & 0xffff0000u);
    }
  }
}

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void from_f32(float *p, float x) { *p = x; }
__device__ __forceinline__ void from_f32(__nv_bfloat16 *p, float x) { *p = __float2bfloat16_rn(x); }

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}
__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}

// phi(x) = softmax over the D entries of one row, one warp per row, lane holds E = D/32 entries.
template <int E>
__device__ __forceinline__ void warp_phi(float (&x)[E]) {
  float mx = x[0];
#pragma unroll
  for (int i = 1; i < E; ++i) mx = fmaxf(mx, x[i]);
  mx = warp_max(mx);
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < E; ++i) {
    x[i] = exp2f((x[i] - mx) * kLog2e);
    s += x[i];
  }
  s = warp_sum(s);
  const float inv = 1.0f / s;
#pragma unroll
  for (int i = 0; i < E; ++i) x[i] *= inv;
}

// Projection of the learned feature map for N vectors held by a warp (lane: entries lane*E .. lane*E+E-1 of each):
// y += (rows [il0*E, il1*E) of W)^T x, with the head's d x d matrix W read row by row (row i: 32 lanes x E consecutive
// entries, coalesced).  The rows are fetched UB * E at a time into registers before any of them is used, so that
// many loads are in flight per lane.  y is in the same lane layout.
template <typename T, int D, int N, int UB>
__device__ __forceinline__ void warp_project_rows(const T *W, const float (&x)[N][D / 32], float (&y)[N][D / 32],
                                                  int il_begin, int il_end) {
  constexpr int E = D / 32;
  const int lane = threadIdx.x & 31;
  for (int il0 = il_begin; il0 < il_end; il0 += UB) {
    float w[UB * E][E];
#pragma unroll
    for (int u = 0; u < UB * E; ++u) load_elems<T, E>(W + size_t(il0 * E + u) * D + lane * E, w[u]);
#pragma unroll
    for (int u = 0; u < UB * E; ++u) {
#pragma unroll
      for (int n = 0; n < N; ++n) {
        const float xi = __shfl_sync(0xffffffffu, x[n][u % E], il0 + u / E);
#pragma unroll
        for (int e = 0; e < E; ++e) y[n][e] = fmaf(xi, w[u][e], y[n][e]);
      }
    }
  }
}

// Learned feature map of N vectors held by a warp: y = W^T x, then the two softmax halves; lo / hi receive
// softmax(y) and softmax(-y) in the lane layout of x.
template <typename T, int D, int N, int UB = 2>
__device__ __forceinline__ void warp_phi_learned(const T *W, const float (&x)[N][D / 32], float (&lo)[N][D / 32],
                                                 float (&hi)[N][D / 32]) {
  constexpr int E = D / 32;
  static_assert(32 % UB == 0, "batches of rows");
#pragma unroll
  for (int n = 0; n < N; ++n)
#pragma unroll
    for (int e = 0; e < E; ++e) lo[n][e] = 0.f;
  warp_project_rows<T, D, N, UB>(W, x, lo, 0, 32);
#pragma unroll
  for (int n = 0; n < N; ++n) {
#pragma unroll
    for (int e = 0; e < E; ++e) hi[n][e] = -lo[n][e];
    warp_phi<E>(lo[n]);
    warp_phi<E>(hi[n]);
  }
}

// One key/value row folded into a per-warp online softmax over G heads (log2 domain).
template <int E, int G>
__device__ __forceinline__ void online_row(const float (&qr)[G][E], const float (&kx)[E], const float (&vx)[E],
                                           float (&m)[G], float (&l)[G], float (&acc)[G][E]) {
#pragma unroll
  for (int h = 0; h < G; ++h) {
    float part = 0.f;
#pragma unroll
    for (int i = 0; i < E; ++i) part = fmaf(qr[h][i], kx[i], part);
    const float sc = warp_sum(part);
    const float mn = fmaxf(m[h], sc);
    const float corr = exp2f(m[h] - mn);
    const float pw = exp2f(sc - mn);
    l[h] = fmaf(l[h], corr, pw);
#pragma unroll
    for (int i = 0; i < E; ++i) acc[h][i] = fmaf(acc[h][i], corr, pw * vx[i]);
    m[h] = mn;
  }
}

}  // namespace glide
