// GLIDE prefill: append T prompt tokens, chunk by chunk (C tokens per chunk).
//
// For a layer with window w the linear part of query i sums over tokens j <= i - w, i.e. it is
// ordinary causal (inclusive) linear attention on the stream delayed by w tokens:
// k'_i = k_{i-w}, v'_i = v_{i-w}.  Per chunk, in stream order:
//   1. phi kernel    phi(k') of the chunk's delayed tokens -> scratch (fp32)
//   2. attn kernel   per query: sliding-window online softmax over ring-or-call rows, the readout
//                    phi(q) S / phi(q) z of the state at chunk start, the intra-chunk delayed terms
//                    (phi(q).phi(k'_j)) v'_j, merged under the shared normaliser -> out
//   3. state kernel  S += phi(K'_c)^T V'_c, z += sum phi(K'_c)   (fp32 carry)
//   4. ring kernel   the chunk's newest min(C, cap) tokens -> slot (position mod cap)
// The delayed rows and the window rows older than the call come from the ring, which step 4 of
// the same chunk overwrites only after steps 1-3 have read it.
#include <algorithm>
#include <type_traits>

#include "glide_device.cuh"

namespace glide {

namespace {

constexpr int kPrefillThreads = 128;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return uint32_t(__cvta_generic_to_shared(p)); }
// 16 bytes global -> shared; a false `valid` writes zeros and reads nothing
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid) {
  const int bytes = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

template <typename T>
struct RowSource {
  const T *ringK, *ringV;   // unit base: [cap][D]
  const T *callK, *callV;   // (layer, sequence) base: [T][Hkv][D], already offset to KV head g
  int64_t n0, cap;
  int64_t call_stride;      // Hkv * D
  __device__ __forceinline__ const T *k(int64_t j, int D) const {
    return j >= n0 ? callK + (j - n0) * call_stride : ringK + (j % cap) * D;
  }
  __device__ __forceinline__ const T *v(int64_t j, int D) const {
    return j >= n0 ? callV + (j - n0) * call_stride : ringV + (j % cap) * D;
  }
  // gate of token j (gated contexts): from the call's gates, or from the ring of gates; 1 when the call has none
  const float *ringG, *callG;   // unit base [cap]; (layer, sequence) base [T][Hkv], already offset to KV head g
  int64_t gate_stride;          // Hkv
  __device__ __forceinline__ float gate(int64_t j) const {
    return j >= n0 ? (callG ? callG[(j - n0) * gate_stride] : 1.f) : ringG[j % cap];
  }
};

template <typename T, int D>
__device__ __forceinline__ RowSource<T> make_source(const PrefillParams &p, const LayerDev &ld, int lrel, int b, int g) {
  RowSource<T> s;
  const size_t unit_rows = (size_t(b + p.b0) * p.Hkv + g) * size_t(ld.cap);   // b + b0: the sequence's slot in the context
  s.ringK = reinterpret_cast<const T *>(p.ws + ld.ringK) + unit_rows * D;
  s.ringV = reinterpret_cast<const T *>(p.ws + ld.ringV) + unit_rows * D;
  const size_t seq = (size_t(lrel) * p.B + b) * size_t(p.T) * p.Hkv * D + size_t(g) * D;
  s.callK = reinterpret_cast<const T *>(p.k) + seq;
  s.callV = reinterpret_cast<const T *>(p.v) + seq;
  s.n0 = p.n0;
  s.cap = ld.cap > 0 ? ld.cap : 1;
  s.call_stride = int64_t(p.Hkv) * D;
  s.ringG = p.gated ? reinterpret_cast<const float *>(p.ws + ld.ringG) + unit_rows : nullptr;
  s.callG = p.gate ? p.gate + (size_t(lrel) * p.B + b) * size_t(p.T) * p.Hkv + g : nullptr;
  s.gate_stride = p.Hkv;
  return s;
}

// 1. phi of the delayed keys of this chunk: one warp per (unit, kTokPerWarp consecutive chunk tokens), the rows'
// loads issued together (with one row per warp the kernel was bound by the latency of its single load)
constexpr int kTokPerWarp = 4;
template <typename T, int D, int DP>
__global__ void __launch_bounds__(kPrefillThreads) prefill_phi_kernel(const PrefillParams p) {
  constexpr int E = D / 32;
  const int lane = threadIdx.x & 31;
  const int64_t wid = (int64_t(blockIdx.x) * kPrefillThreads + threadIdx.x) >> 5;
  const int64_t units = int64_t(p.layer_count) * p.B * p.Hkv;
  const int groups = (p.C + kTokPerWarp - 1) / kTokPerWarp;
  if (wid >= units * groups) return;
  const int i0 = int(wid % groups) * kTokPerWarp;
  const int64_t u = wid / groups;
  const int g = int(u % p.Hkv);
  const int b = int((u / p.Hkv) % p.B);
  const int lrel = int(u / (int64_t(p.Hkv) * p.B));
  const LayerDev ld = p.layers[p.layer_begin + lrel];
  if (!ld.evicts) return;
  const RowSource<T> src = make_source<T, D>(p, ld, lrel, b, g);
  float x[kTokPerWarp][E];
  bool valid[kTokPerWarp];
#pragma unroll
  for (int r = 0; r < kTokPerWarp; ++r) {
    const int64_t j = p.n0 + p.c0 + i0 + r - ld.wlin;  // delayed token
    valid[r] = i0 + r < p.C && j >= 0;
    if (valid[r]) load_elems<T, E>(src.k(j, D) + lane * E, x[r]);
  }
  if constexpr (DP == D) {
#pragma unroll
    for (int r = 0; r < kTokPerWarp; ++r) {
      if (!valid[r]) continue;   // warp-uniform
      warp_phi<E>(x[r]);
      float *dst = p.phik + (size_t(u) * p.Cmax + i0 + r) * D + lane * E;
#pragma unroll
      for (int e = 0; e < E; ++e) dst[e] = x[r][e];
      if (p.phik16) {   // the same row rounded to bf16 for the tensor-core attention kernel
        __nv_bfloat16 *d16 = reinterpret_cast<__nv_bfloat16 *>(p.phik16) + (size_t(u) * p.Cmax + i0 + r) * D + lane * E;
#pragma unroll
        for (int e = 0; e < E; ++e) d16[e] = __float2bfloat16_rn(x[r][e]);
      }
    }
  } else {
#pragma unroll
    for (int r = 0; r < kTokPerWarp; ++r)
      if (!valid[r])
#pragma unroll
        for (int e = 0; e < E; ++e) x[r][e] = 0.f;
    float lo[kTokPerWarp][E], hi[kTokPerWarp][E];
    const T *W = reinterpret_cast<const T *>(p.wk) + (size_t(p.layer_begin + lrel) * p.Hkv + g) * D * D;
    warp_phi_learned<T, D, kTokPerWarp>(W, x, lo, hi);
#pragma unroll
    for (int r = 0; r < kTokPerWarp; ++r) {
      if (!valid[r]) continue;
      float *dst = p.phik + (size_t(u) * p.Cmax + i0 + r) * DP + lane * E;
#pragma unroll
      for (int e = 0; e < E; ++e) {
        dst[e] = lo[r][e];
        dst[D + e] = hi[r][e];
      }
      if (p.phik16) {   // the two halves rounded to bf16, each in its own array, for the tensor-core attention kernel
        __nv_bfloat16 *d16 = reinterpret_cast<__nv_bfloat16 *>(p.phik16) + (size_t(u) * p.Cmax + i0 + r) * D + lane * E;
        const size_t half = size_t(p.units_cap) * p.Cmax * D;
#pragma unroll
        for (int e = 0; e < E; ++e) {
          d16[e] = __float2bfloat16_rn(lo[r][e]);
          d16[half + e] = __float2bfloat16_rn(hi[r][e]);
        }
      }
    }
  }
}

// 1c. (gated contexts) running sums of log(gate) over the chunk's delayed tokens: gcum[i] = sum over the valid delayed
// indices ii <= i of log gate(k'_ii).  exp(gcum[i] - gcum[ii]) is then the decay a delayed token ii has suffered when
// delayed token i has entered the state, exp(gcum[i]) the decay of the state the chunk started from.
// One thread per unit, sequential over the chunk (C <= 1024).
template <typename T, int D>
__global__ void __launch_bounds__(kPrefillThreads) prefill_gcum_kernel(const PrefillParams p) {
  const int64_t u = int64_t(blockIdx.x) * kPrefillThreads + threadIdx.x;
  const int64_t units = int64_t(p.layer_count) * p.B * p.Hkv;
  if (u >= units) return;
  const int g = int(u % p.Hkv);
  const int b = int((u / p.Hkv) % p.B);
  const int lrel = int(u / (int64_t(p.Hkv) * p.B));
  const LayerDev ld = p.layers[p.layer_begin + lrel];
  if (!ld.evicts) return;
  const RowSource<T> src = make_source<T, D>(p, ld, lrel, b, g);
  float run = 0.f;
  for (int i = 0; i < p.C; ++i) {
    const int64_t j = p.n0 + p.c0 + i - ld.wlin;
    if (j >= 0) run += logf(src.gate(j));
    p.gcum[size_t(u) * p.Cmax + i] = run;
  }
}

// 2. outputs: one warp per (unit, query token), G heads at once
template <typename T, int D, int G, int DP>
__global__ void __launch_bounds__(kPrefillThreads) prefill_attn_kernel(const PrefillParams p) {
  constexpr int E = D / 32;
  constexpr int NW = kPrefillThreads / 32;
  constexpr int NH = DP / D;   // halves of the feature vector: lane holds entries lane*E .. +E-1 of each
  __shared__ float sm_phiq[NW][G][DP];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t wid = int64_t(blockIdx.x) * NW + warp;
  const int64_t units = int64_t(p.layer_count) * p.B * p.Hkv;
  if (wid >= units * p.C) return;
  const int i = int(wid % p.C);
  const int64_t u = wid / p.C;
  const int g = int(u % p.Hkv);
  const int b = int((u / p.Hkv) % p.B);
  const int lrel = int(u / (int64_t(p.Hkv) * p.B));
  const LayerDev ld = p.layers[p.layer_begin + lrel];
  const RowSource<T> src = make_source<T, D>(p, ld, lrel, b, g);
  const int64_t tq = p.n0 + p.c0 + i;  // absolute position of the query
  const int ub = (b + p.b0) * p.Hkv + g;

  float qr[G][E];
  const T *qbase = reinterpret_cast<const T *>(p.q) + ((size_t(lrel) * p.B + b) * size_t(p.T) + size_t(p.c0 + i)) * p.H * D;
#pragma unroll
  for (int h = 0; h < G; ++h) {
    const int head = p.heads_of[g * G + h];
    load_elems<T, E>(qbase + size_t(head) * D + lane * E, qr[h]);
    if constexpr (DP == D) {
      float x[E];
#pragma unroll
      for (int e = 0; e < E; ++e) x[e] = qr[h][e];
      warp_phi<E>(x);
#pragma unroll
      for (int e = 0; e < E; ++e) sm_phiq[warp][h][lane * E + e] = x[e];
    } else {
      float x[1][E], lo[1][E], hi[1][E];
#pragma unroll
      for (int e = 0; e < E; ++e) x[0][e] = qr[h][e];
      warp_phi_learned<T, D, 1>(reinterpret_cast<const T *>(p.wq) + (size_t(p.layer_begin + lrel) * p.H + head) * D * D, x,
                                lo, hi);
#pragma unroll
      for (int e = 0; e < E; ++e) {
        sm_phiq[warp][h][lane * E + e] = lo[0][e];
        sm_phiq[warp][h][D + lane * E + e] = hi[0][e];
      }
    }
#pragma unroll
    for (int e = 0; e < E; ++e) qr[h][e] *= p.scale_log2;
  }
  __syncwarp();

  // window part: tokens max(0, tq - w + 1) .. tq
  float acc[G][E], m[G], l[G];
#pragma unroll
  for (int h = 0; h < G; ++h) {
    m[h] = -CUDART_INF_F;
    l[h] = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) acc[h][e] = 0.f;
  }
  int64_t w_lo = tq - ld.w + 1;
  if (w_lo < 0) w_lo = 0;
  for (int64_t j = w_lo; j <= tq; j += 2) {
    float kx[2][E], vx[2][E];
    const bool two = j + 1 <= tq;
    load_elems<T, E>(src.k(j, D) + lane * E, kx[0]);
    load_elems<T, E>(src.v(j, D) + lane * E, vx[0]);
    if (two) {
      load_elems<T, E>(src.k(j + 1, D) + lane * E, kx[1]);
      load_elems<T, E>(src.v(j + 1, D) + lane * E, vx[1]);
    }
    online_row<E, G>(qr, kx[0], vx[0], m, l, acc);
    if (two) online_row<E, G>(qr, kx[1], vx[1], m, l, acc);
  }

  // linear part on the delayed stream
  float lin[G][E], bl[G];
#pragma unroll
  for (int h = 0; h < G; ++h) {
    bl[h] = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) lin[h][e] = 0.f;
  }
  if (ld.evicts && tq >= ld.wlin) {
    const int64_t folded_at_chunk_start = p.n0 + p.c0 - ld.wlin;  // tokens < this are in S,z
    // gated: the decays come from the running sums of log(gate) over the chunk's delayed tokens
    const float *gc = p.gated ? p.gcum + size_t(u) * p.Cmax : nullptr;
    const float g_own = gc ? gc[i] : 0.f;
    if (folded_at_chunk_start > 0) {
      const float *Sb = reinterpret_cast<const float *>(p.ws + ld.S) + size_t(ub) * DP * D;
      const float *zb = reinterpret_cast<const float *>(p.ws + ld.z) + size_t(ub) * DP;
      const float dec0 = gc ? expf(g_own) : 1.f;   // what the state of the chunk's start has decayed to by now
      for (int r = 0; r < DP; ++r) {
        float s[E];
        load_elems<float, E>(Sb + size_t(r) * D + lane * E, s);
#pragma unroll
        for (int h = 0; h < G; ++h) {
          const float f = sm_phiq[warp][h][r] * dec0;
#pragma unroll
          for (int e = 0; e < E; ++e) lin[h][e] = fmaf(f, s[e], lin[h][e]);
        }
      }
#pragma unroll
      for (int h = 0; h < G; ++h) {
        float part = 0.f;
#pragma unroll
        for (int nh = 0; nh < NH; ++nh) {
          float zz[E];
          load_elems<float, E>(zb + nh * D + lane * E, zz);
#pragma unroll
          for (int e = 0; e < E; ++e) part = fmaf(sm_phiq[warp][h][nh * D + lane * E + e], zz[e], part);
        }
        bl[h] = warp_sum(part) * dec0;
      }
    }
    // delayed tokens of this chunk, up to and including the query's own delayed token
    const float *pk = p.phik + size_t(u) * p.Cmax * DP;
    int i_lo = 0;
    if (folded_at_chunk_start < 0) i_lo = int(-folded_at_chunk_start);  // delayed index < 0 does not exist
    for (int ii = i_lo; ii <= i; ++ii) {
      const int64_t j = p.n0 + p.c0 + ii - ld.wlin;
      float fk[NH][E], vx[E];
#pragma unroll
      for (int nh = 0; nh < NH; ++nh) load_elems<float, E>(pk + size_t(ii) * DP + nh * D + lane * E, fk[nh]);
      load_elems<T, E>(src.v(j, D) + lane * E, vx);
      const float dec = gc ? expf(g_own - gc[ii]) : 1.f;
#pragma unroll
      for (int h = 0; h < G; ++h) {
        float part = 0.f;
#pragma unroll
        for (int nh = 0; nh < NH; ++nh)
#pragma unroll
          for (int e = 0; e < E; ++e) part = fmaf(sm_phiq[warp][h][nh * D + lane * E + e], fk[nh][e], part);
        const float c = warp_sum(part) * dec;
        bl[h] += c;
#pragma unroll
        for (int e = 0; e < E; ++e) lin[h][e] = fmaf(c, vx[e], lin[h][e]);
      }
    }
  }

  // shared normaliser, or the sum of the two separately normalised terms (an empty term counts as zero)
  T *obase = reinterpret_cast<T *>(p.out) + ((size_t(lrel) * p.B + b) * size_t(p.T) + size_t(p.c0 + i)) * p.H * D;
  if (ld.merge != GLIDE_MERGE_SHARED) {
#pragma unroll
    for (int h = 0; h < G; ++h) {
      const float iw = l[h] > 0.f ? 1.0f / l[h] : 0.f, il = bl[h] > 0.f ? 1.0f / bl[h] : 0.f;
      const int head = p.heads_of[g * G + h];
#pragma unroll
      for (int e = 0; e < E; ++e) from_f32(obase + size_t(head) * D + lane * E + e, fmaf(acc[h][e], iw, lin[h][e] * il));
    }
    return;
  }
#pragma unroll
  for (int h = 0; h < G; ++h) {
    const float M = bl[h] > 0.f ? fmaxf(m[h], 0.f) : m[h];   // the floor belongs to the linear terms (logit 0)
    const float fw = m[h] == -CUDART_INF_F ? 0.f : exp2f(m[h] - M);
    const float fl = bl[h] > 0.f ? exp2f(-M) : 0.f;
    const float inv = 1.0f / fmaf(l[h], fw, fl * bl[h]);
    const int head = p.heads_of[g * G + h];
#pragma unroll
    for (int e = 0; e < E; ++e)
      from_f32(obase + size_t(head) * D + lane * E + e, (acc[h][e] * fw + fl * lin[h][e]) * inv);
  }
}

// 3. S += phi(K'_c)^T V'_c ; z += sum phi(K'_c) in fp32 on the CUDA cores (the carry keeps fp32 precision, which
// a bf16 or tf32 tensor-core product of phi(K') would not).  One CTA per (unit, block of 64 state rows): the
// chunk's phi(K') columns and V' rows are staged through shared memory 32 tokens at a time and every thread
// accumulates an 8 x (D/16) register tile of rank-1 updates (rows ty*4..+3 and 32+ty*4..+3, columns tx*4..+3 and,
// for D = 128, 64+tx*4..+3: 16-byte shared-memory reads without bank conflicts).
constexpr int kStateRows = 64;    // state rows per CTA
constexpr int kStateTok = 32;     // tokens per shared-memory stage
// V values of one shared-memory row chunk as fp32 (the stage holds the rows in the I/O dtype)
__device__ __forceinline__ void stage_v4(const float *p, float (&x)[4]) {
  const float4 v = *reinterpret_cast<const float4 *>(p);
  x[0] = v.x, x[1] = v.y, x[2] = v.z, x[3] = v.w;
}
__device__ __forceinline__ void stage_v4(const __nv_bfloat16 *p, float (&x)[4]) {
  const uint2 v = *reinterpret_cast<const uint2 *>(p);
  x[0] = __uint_as_float(v.x << 16), x[1] = __uint_as_float(v.x & 0xffff0000u);
  x[2] = __uint_as_float(v.y << 16), x[3] = __uint_as_float(v.y & 0xffff0000u);
}
template <typename T, int D>
__global__ void __launch_bounds__(kPrefillThreads) prefill_state_kernel(const PrefillParams p) {
  static_assert(kPrefillThreads == 128, "8 x 16 thread grid");
  constexpr int CG = D / 64;                      // column groups of 4 per thread
  // two stages, filled by cp.async while the other one is consumed: phi columns (fp32), then V' rows (I/O dtype)
  constexpr int kPhiBytes = kStateTok * kStateRows * 4;
  constexpr int kVBytes = kStateTok * D * int(sizeof(T));
  constexpr int kVChunks = D * int(sizeof(T)) / 16;   // 16-byte chunks per V row
  __shared__ __align__(16) unsigned char stage[2][kPhiBytes + kVBytes];
  const int dp = p.dp;
  const int blocks_per_unit = dp / kStateRows;
  const int64_t u = blockIdx.x / blocks_per_unit;
  const int rb = blockIdx.x % blocks_per_unit;
  const int g = int(u % p.Hkv);
  const int b = int((u / p.Hkv) % p.B);
  const int lrel = int(u / (int64_t(p.Hkv) * p.B));
  const LayerDev ld = p.layers[p.layer_begin + lrel];
  if (!ld.evicts) return;
  const int64_t first = p.n0 + p.c0 - ld.wlin;    // delayed token of chunk index 0
  const int i_lo = first < 0 ? int(first < -int64_t(p.C) ? p.C : -first) : 0;
  if (i_lo >= p.C) return;
  const RowSource<T> src = make_source<T, D>(p, ld, lrel, b, g);
  const int ub = (b + p.b0) * p.Hkv + g;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const float *pk = p.phik + size_t(u) * p.Cmax * dp + rb * kStateRows;
  const float *gc = p.gated ? p.gcum + size_t(u) * p.Cmax : nullptr;
  const float g_end = gc ? gc[p.C - 1] : 0.f;
  float acc[8][4 * CG];
#pragma unroll
  for (int r = 0; r < 8; ++r)
#pragma unroll
    for (int c = 0; c < 4 * CG; ++c) acc[r][c] = 0.f;
  float zacc = 0.f;   // threads 0..63: z of row rb*64 + tid
  // tokens past the chunk's end are filled with zeros (cp.async with a source size of 0)
  auto issue = [&](int buf, int i0) {
    const int nt = min(kStateTok, p.C - i0);
    const uint32_t sphi = smem_u32(stage[buf]), sv = sphi + kPhiBytes;
    for (int e = tid; e < kStateTok * (kStateRows / 4); e += kPrefillThreads) {
      const int i = e / (kStateRows / 4), c4 = e % (kStateRows / 4);
      cp_async16(sphi + uint32_t(i * kStateRows + c4 * 4) * 4u, pk + size_t(i0 + (i < nt ? i : 0)) * dp + c4 * 4, i < nt);
    }
    for (int e = tid; e < kStateTok * kVChunks; e += kPrefillThreads) {
      const int i = e / kVChunks, c = e % kVChunks;
      const unsigned char *row = reinterpret_cast<const unsigned char *>(src.v(first + i0 + (i < nt ? i : 0), D));
      cp_async16(sv + uint32_t(i * kVChunks + c) * 16u, row + c * 16, i < nt);
    }
    cp_async_commit();
  };
  issue(0, i_lo);
  int buf = 0;
  for (int i0 = i_lo; i0 < p.C; i0 += kStateTok, buf ^= 1) {
    if (i0 + kStateTok < p.C) {
      issue(buf ^ 1, i0 + kStateTok);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      cp_async_wait_all();
    }
    __syncthreads();
    const float *sphi = reinterpret_cast<const float *>(stage[buf]);
    const T *sv = reinterpret_cast<const T *>(stage[buf] + kPhiBytes);
#pragma unroll 4
    for (int i = 0; i < kStateTok; ++i) {
      const float4 fa = *reinterpret_cast<const float4 *>(sphi + i * kStateRows + ty * 4);
      const float4 fb = *reinterpret_cast<const float4 *>(sphi + i * kStateRows + 32 + ty * 4);
      // gated: what this token has decayed to by the end of the chunk (tokens past the chunk's end are zero rows)
      const float dc = (gc && i0 + i < p.C) ? expf(g_end - gc[i0 + i]) : 1.f;
      const float fr[8] = {fa.x * dc, fa.y * dc, fa.z * dc, fa.w * dc, fb.x * dc, fb.y * dc, fb.z * dc, fb.w * dc};
      float vc[4 * CG];
#pragma unroll
      for (int cg = 0; cg < CG; ++cg) {
        float x[4];
        stage_v4(sv + i * D + cg * 64 + tx * 4, x);
        vc[cg * 4 + 0] = x[0], vc[cg * 4 + 1] = x[1], vc[cg * 4 + 2] = x[2], vc[cg * 4 + 3] = x[3];
      }
#pragma unroll
      for (int r = 0; r < 8; ++r)
#pragma unroll
        for (int c = 0; c < 4 * CG; ++c) acc[r][c] = fmaf(fr[r], vc[c], acc[r][c]);
    }
    if (tid < kStateRows) {
#pragma unroll 8
      for (int i = 0; i < kStateTok; ++i)
        zacc = fmaf(sphi[i * kStateRows + tid], (gc && i0 + i < p.C) ? expf(g_end - gc[i0 + i]) : 1.f, zacc);
    }
    __syncthreads();   // the stage is refilled by the next iteration's issue
  }
  float *Sb = reinterpret_cast<float *>(p.ws + ld.S) + size_t(ub) * dp * D + size_t(rb) * kStateRows * D;
  const float dec_all = gc ? expf(g_end) : 1.f;   // the state the chunk started from, after the whole chunk has entered
#pragma unroll
  for (int r = 0; r < 8; ++r) {
    const int row = (r >> 2) * 32 + ty * 4 + (r & 3);
#pragma unroll
    for (int cg = 0; cg < CG; ++cg) {
      float4 *dst = reinterpret_cast<float4 *>(Sb + size_t(row) * D + cg * 64 + tx * 4);
      float4 cur = *dst;
      cur.x = fmaf(cur.x, dec_all, acc[r][cg * 4 + 0]);
      cur.y = fmaf(cur.y, dec_all, acc[r][cg * 4 + 1]);
      cur.z = fmaf(cur.z, dec_all, acc[r][cg * 4 + 2]);
      cur.w = fmaf(cur.w, dec_all, acc[r][cg * 4 + 3]);
      *dst = cur;
    }
  }
  if (tid < kStateRows) {
    float *zb = reinterpret_cast<float *>(p.ws + ld.z) + size_t(ub) * dp + rb * kStateRows;
    zb[tid] = fmaf(zb[tid], dec_all, zacc);
  }
}

// 1b. (sum-of-terms merges on the tcgen05 kernel) running sums of phi(K') over the chunk: zcum[i] = sum over the valid
// delayed indices ii <= i of phi(k'_ii); a row's linear normaliser is then phi(q) . (z + zcum[own index]).
// One thread per (unit, feature), sequential over the chunk (C <= 1024).
template <int D>
__global__ void __launch_bounds__(kPrefillThreads) prefill_zcum_kernel(const PrefillParams p) {
  const int64_t idx = int64_t(blockIdx.x) * kPrefillThreads + threadIdx.x;
  const int64_t units = int64_t(p.layer_count) * p.B * p.Hkv;
  const int dp = p.dp;
  if (idx >= units * dp) return;
  const int r = int(idx % dp);
  const int64_t u = idx / dp;
  const int lrel = int(u / (int64_t(p.Hkv) * p.B));
  const LayerDev ld = p.layers[p.layer_begin + lrel];
  if (!ld.evicts) return;
  const int64_t first = p.n0 + p.c0 - ld.wlin;
  const int i_lo = first < 0 ? int(first < -int64_t(p.C) ? p.C : -first) : 0;
  const float *pk = p.phik + size_t(u) * p.Cmax * dp + r;
  float *zc = p.zcum + size_t(u) * p.Cmax * dp + r;
  float run = 0.f;
  for (int i = 0; i < p.C; ++i) {
    if (i >= i_lo) run += pk[size_t(i) * dp];
    zc[size_t(i) * dp] = run;
  }
}

// 4. ring fill: the chunk's newest min(C, cap) tokens; one warp per (unit, kTokPerWarp consecutive chunk tokens)
template <typename T, int D>
__global__ void __launch_bounds__(kPrefillThreads) prefill_ring_kernel(const PrefillParams p) {
  constexpr int E = D / 32;
  const int lane = threadIdx.x & 31;
  const int64_t wid = (int64_t(blockIdx.x) * kPrefillThreads + threadIdx.x) >> 5;
  const int64_t units = int64_t(p.layer_count) * p.B * p.Hkv;
  const int groups = (p.C + kTokPerWarp - 1) / kTokPerWarp;
  if (wid >= units * groups) return;
  const int i0 = int(wid % groups) * kTokPerWarp;
  const int64_t u = wid / groups;
  const int g = int(u % p.Hkv);
  const int b = int((u / p.Hkv) % p.B);
  const int lrel = int(u / (int64_t(p.Hkv) * p.B));
  const LayerDev ld = p.layers[p.layer_begin + lrel];
  if (ld.cap == 0) return;
  T kx[kTokPerWarp][E], vx[kTokPerWarp][E];
  bool valid[kTokPerWarp];
#pragma unroll
  for (int r = 0; r < kTokPerWarp; ++r) {
    const int i = i0 + r;
    valid[r] = i < p.C && int64_t(i) >= int64_t(p.C) - ld.cap;   // older tokens of the chunk are overwritten anyway
    if (valid[r]) {
      const size_t src = (((size_t(lrel) * p.B + b) * size_t(p.T) + size_t(p.c0 + i)) * p.Hkv + g) * D + lane * E;
      const T *ks = reinterpret_cast<const T *>(p.k) + src;
      const T *vs = reinterpret_cast<const T *>(p.v) + src;
#pragma unroll
      for (int e = 0; e < E; ++e) {
        kx[r][e] = ks[e];
        vx[r][e] = vs[e];
      }
    }
  }
#pragma unroll
  for (int r = 0; r < kTokPerWarp; ++r) {
    if (!valid[r]) continue;
    const int64_t j = p.n0 + p.c0 + i0 + r;
    const size_t dst = ((size_t(b + p.b0) * p.Hkv + g) * size_t(ld.cap) + size_t(j % ld.cap)) * D + lane * E;
    T *kd = reinterpret_cast<T *>(p.ws + ld.ringK) + dst;
    T *vd = reinterpret_cast<T *>(p.ws + ld.ringV) + dst;
#pragma unroll
    for (int e = 0; e < E; ++e) {
      kd[e] = kx[r][e];
      vd[e] = vx[r][e];
    }
    if (p.gated && lane == 0) {   // the token's gate waits in the ring with it
      const size_t slot = (size_t(b + p.b0) * p.Hkv + g) * size_t(ld.cap) + size_t(j % ld.cap);
      reinterpret_cast<float *>(p.ws + ld.ringG)[slot] =
          p.gate ? p.gate[((size_t(lrel) * p.B + b) * size_t(p.T) + size_t(p.c0 + i0 + r)) * p.Hkv + g] : 1.f;
    }
  }
}

// bf16 copy of the state of every unit of the call as it is before the chunk's state update: what the tcgen05 attention
// kernel multiplies phi(Q) with (one 16-byte store per thread).  With the learned map S has 2 d rows: rows d .. 2d - 1
// go to the second half of the array.
__global__ void __launch_bounds__(kPrefillThreads) prefill_s16_kernel(const PrefillParams p) {
  constexpr int D = 128;
  const int64_t id = int64_t(blockIdx.x) * kPrefillThreads + threadIdx.x;   // 8 consecutive entries of one unit's S
  const int64_t per_unit = int64_t(p.dp) * D / 8;
  const int64_t u = id / per_unit;
  if (u >= int64_t(p.layer_count) * p.B * p.Hkv) return;
  const int g = int(u % p.Hkv);
  const int b = int((u / p.Hkv) % p.B);
  const int lrel = int(u / (int64_t(p.Hkv) * p.B));
  const LayerDev ld = p.layers[p.layer_begin + lrel];
  if (!ld.evicts) return;
  const size_t e0 = size_t(id % per_unit) * 8;   // entry of S [dp][d]
  const float *src = reinterpret_cast<const float *>(p.ws + ld.S) + (size_t(b + p.b0) * p.Hkv + g) * size_t(p.dp) * D + e0;
  const float4 f0 = *reinterpret_cast<const float4 *>(src), f1 = *reinterpret_cast<const float4 *>(src + 4);
  __nv_bfloat162 o[4] = {__floats2bfloat162_rn(f0.x, f0.y), __floats2bfloat162_rn(f0.z, f0.w),
                         __floats2bfloat162_rn(f1.x, f1.y), __floats2bfloat162_rn(f1.z, f1.w)};
  const size_t half = e0 / (size_t(D) * D);
  *reinterpret_cast<uint4 *>(reinterpret_cast<__nv_bfloat16 *>(p.s16) + half * size_t(p.units_cap) * D * D + size_t(u) * D * D +
                             (e0 - half * D * D)) = *reinterpret_cast<const uint4 *>(o);
}

}  // namespace

int launch_prefill(glide_ctx *ctx, int layer_begin, int layer_count, int64_t T, const void *q, const void *k,
                   const void *v, const float *gate, void *out, int seq, int64_t n0, cudaStream_t stream) {
  PrefillParams p{};
  p.ws = ctx->ws;
  p.layers = reinterpret_cast<const LayerDev *>(ctx->ws + ctx->off_layers);
  p.heads_of = reinterpret_cast<const int32_t *>(ctx->ws + ctx->off_heads);
  p.ctl = reinterpret_cast<Control *>(ctx->ws + ctx->off_ctl);
  p.phik = reinterpret_cast<float *>(ctx->ws + ctx->off_phik);
  p.zcum = reinterpret_cast<float *>(ctx->ws + ctx->off_zcum);
  p.merge = ctx->cfg.merge;
  p.q = q;
  p.k = k;
  p.v = v;
  p.out = out;
  p.n0 = n0;
  p.T = T;
  p.Cmax = ctx->prefill_chunk;
  p.layer_begin = layer_begin;
  p.layer_count = layer_count;
  p.L = ctx->cfg.n_layers;
  p.B = seq < 0 ? ctx->cfg.batch : 1;
  p.b0 = seq < 0 ? 0 : seq;
  p.H = ctx->cfg.n_q_heads;
  p.Hkv = ctx->cfg.n_kv_heads;
  p.scale_log2 = ctx->scale * kLog2e;
  p.phi = ctx->cfg.phi;
  p.dp = ctx->dp;
  p.wq = ctx->cfg.phi_wq;
  p.wk = ctx->cfg.phi_wk;
  p.gated = ctx->cfg.gated;
  p.gate = gate;
  p.gcum = reinterpret_cast<float *>(ctx->ws + ctx->off_gcum);
  const int64_t units = int64_t(layer_count) * p.B * p.Hkv;
  const bool plain = ctx->cfg.phi == GLIDE_PHI_SOFTMAX && !ctx->cfg.gated;   // what the tensor-core kernels compute
  int impl = ctx->cfg.prefill_impl;
  // the tcgen05 kernel also takes the learned map under the shared normaliser (its two halves as two linear parts)
  const bool tc_kind = !ctx->cfg.gated && (ctx->cfg.phi == GLIDE_PHI_SOFTMAX || ctx->cfg.merge == GLIDE_MERGE_SHARED);
  if (impl == GLIDE_PREFILL_AUTO)
    impl = (tc_kind && prefill_attn_mma_supported(ctx) && ctx->cfg.decode_impl != GLIDE_DECODE_FMA) ? GLIDE_PREFILL_TCGEN05
                                                                                                : GLIDE_PREFILL_FMA;
  // the tcgen05 kernel needs the ring descriptors of the tensor-core decode kernels (absent when decode_impl asks
  // for the CUDA-core kernel); without them the call uses the mma.sync kernel
  const bool use_tc = impl == GLIDE_PREFILL_TCGEN05 && tc_kind && prefill_attn_tc_supported(ctx);
  p.phik16 = use_tc && out ? ctx->ws + ctx->off_phik16 : nullptr;
  p.s16 = use_tc && out ? ctx->ws + ctx->off_s16 : nullptr;
  p.phiq16 = use_tc && out && ctx->off_phiq16 ? ctx->ws + ctx->off_phiq16 : nullptr;
  p.units_cap = int64_t(ctx->cfg.n_layers) * ctx->cfg.batch * ctx->cfg.n_kv_heads;
  // (the mma.sync kernel has the shared normaliser only: the other merges fall through to the CUDA-core kernel)
  const bool use_mma = plain && (impl == GLIDE_PREFILL_MMA_SYNC || (impl == GLIDE_PREFILL_TCGEN05 && !use_tc)) &&
                       prefill_attn_mma_supported(ctx) && ctx->cfg.merge == GLIDE_MERGE_SHARED;
  // carry of the chunk scan: tensor cores with an error-free three-way bf16 split of phi(K') (bf16, d = 128), or the
  // CUDA-core kernel (fp32 I/O, d = 64, and whenever the CUDA-core prefill is asked for)
  const bool state_mma = !ctx->cfg.gated && prefill_state_mma_supported(ctx) && impl != GLIDE_PREFILL_FMA;   // (either feature map)
  bool any_evicts = false;
  for (int l = layer_begin; l < layer_begin + layer_count; ++l) any_evicts = any_evicts || ctx->layers[l].evicts;

  auto run_chunks = [&](auto tt, auto dd, auto gg, auto pp) -> int {
    using TT = typename decltype(tt)::type;
    constexpr int D = decltype(dd)::value, G = decltype(gg)::value, DP = decltype(pp)::value;
    for (int64_t c0 = 0; c0 < T; c0 += p.Cmax) {
      p.c0 = c0;
      p.C = int(std::min<int64_t>(p.Cmax, T - c0));
      const int64_t warps = units * p.C;
      const unsigned warp_blocks = unsigned((warps * 32 + kPrefillThreads - 1) / kPrefillThreads);
      const int64_t warps4 = units * ((p.C + kTokPerWarp - 1) / kTokPerWarp);
      const unsigned warp4_blocks = unsigned((warps4 * 32 + kPrefillThreads - 1) / kPrefillThreads);
      // the learned map's projections of the delayed keys go to the tensor cores for bf16 / d = 128 unless the
      // CUDA-core prefill was asked for
      constexpr bool kCanProject = DP == 2 * D && D == 128 && std::is_same<TT, __nv_bfloat16>::value;
      if (any_evicts && kCanProject && impl != GLIDE_PREFILL_FMA) {
        if (launch_prefill_project(ctx, p, true, stream) != GLIDE_OK) return GLIDE_ERR_CUDA;
      } else if (any_evicts) {
        prefill_phi_kernel<TT, D, DP><<<warp4_blocks, kPrefillThreads, 0, stream>>>(p);
      }
      if (any_evicts && p.gated)
        prefill_gcum_kernel<TT, D><<<unsigned((units + kPrefillThreads - 1) / kPrefillThreads), kPrefillThreads, 0, stream>>>(p);
      if (out) {
        if (use_tc) {
          if (any_evicts)
            prefill_s16_kernel<<<unsigned((units * (int64_t(p.dp) * 128 / 8) + kPrefillThreads - 1) / kPrefillThreads), kPrefillThreads, 0, stream>>>(p);
          if (any_evicts && p.phiq16 && launch_prefill_project(ctx, p, false, stream) != GLIDE_OK) return GLIDE_ERR_CUDA;
          if (any_evicts && p.merge != GLIDE_MERGE_SHARED)
            prefill_zcum_kernel<D><<<unsigned((units * D + kPrefillThreads - 1) / kPrefillThreads), kPrefillThreads, 0, stream>>>(p);
          if (launch_prefill_attn_tc(ctx, p, stream) != GLIDE_OK) return GLIDE_ERR_CUDA;
        } else if (use_mma) {
          if (launch_prefill_attn_mma(ctx, p, stream) != GLIDE_OK) return GLIDE_ERR_CUDA;
        } else {
          prefill_attn_kernel<TT, D, G, DP><<<warp_blocks, kPrefillThreads, 0, stream>>>(p);
        }
      }
      if (any_evicts) {
        if (state_mma) {
          if (launch_prefill_state_mma(ctx, p, stream) != GLIDE_OK) return GLIDE_ERR_CUDA;
        } else {
          prefill_state_kernel<TT, D><<<unsigned(units * (DP / kStateRows)), kPrefillThreads, 0, stream>>>(p);
        }
      }
      prefill_ring_kernel<TT, D><<<warp4_blocks, kPrefillThreads, 0, stream>>>(p);
      if (cudaGetLastError() != cudaSuccess) return GLIDE_ERR_CUDA;
    }
    return GLIDE_OK;
  };
  int rc = dispatch_config(ctx->cfg.io_dtype, ctx->cfg.head_dim, ctx->G, [&](auto tt, auto dd, auto gg) -> int {
    constexpr int D = decltype(dd)::value;
    if (ctx->dp == D) return run_chunks(tt, dd, gg, IntTag<D>{});
    return run_chunks(tt, dd, gg, IntTag<2 * D>{});
  });
  if (rc) return rc;
  return seq < 0 ? launch_advance(ctx, layer_begin, layer_count, T, stream) : GLIDE_OK;
}

}  // namespace glide
