// GLIDE prefill outputs on the tensor cores (bf16 I/O, head_dim 128).
//
// One CTA owns 128 query rows of one (layer, sequence, KV head) unit: 128/G consecutive tokens of the
// current chunk times the G query heads of the KV head (row = token * G + head), 16 rows per warp.
//   window part   flash-style loop over 64-key tiles of the sliding window (ring rows for tokens older
//                 than the call, the call's own rows otherwise): S = Q K^T (mma.sync m16n8k16, bf16 in,
//                 fp32 out), causal + window mask per row, online softmax in the log2 domain, O += P V;
//   linear part   with m* = max(window max, 0) fixed per row, the weights of the older tokens are
//                 phi(q) . phi(k'_j) * 2^-m*, no exponential:
//                   inter-chunk  O += (phi(Q) 2^-m*) S,  l += (phi(Q) 2^-m*) z   (state at chunk start, bf16 copy of S)
//                   intra-chunk  C = phi(Q) phi(K')^T over the chunk's delayed tokens, masked to j' <= i,
//                                O += C V',  l += rowsum(C)
//   out = O / l  (shared normaliser), bf16.
// K/V/phi(K') tiles are staged with cp.async into XOR-swizzled shared memory so that every ldmatrix is
// bank-conflict free.  The fp32 state update of the chunk stays in prefill_state_kernel.
#include <algorithm>

#include "glide_device.cuh"

namespace glide {

namespace {

constexpr int kD = 128;
constexpr int kRows = 128;      // query rows per CTA
constexpr int kKT = 64;         // keys per tile
constexpr int kThreads = 256;
constexpr int kRowBytes = kD * 2;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return uint32_t(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ uint32_t swz(int row, int chunk) { return uint32_t(row * kRowBytes + ((chunk ^ (row & 7)) << 4)); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid) {
  const int bytes = valid ? 16 : 0;   // 0: the 16 destination bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi, float &lo_r, float &hi_r) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  lo_r = __low2float(v);
  hi_r = __high2float(v);
  return *reinterpret_cast<const uint32_t *>(&v);
}
__device__ __forceinline__ uint32_t scale2(uint32_t x, float f) {   // bf16x2 times a scalar
  __nv_bfloat162 v = *reinterpret_cast<const __nv_bfloat162 *>(&x);
  v = __hmul2(v, __float2bfloat162_rn(f));
  return *reinterpret_cast<const uint32_t *>(&v);
}
__device__ __forceinline__ float quad_max(float x) {
  x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 1));
  return fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 2));
}
__device__ __forceinline__ float quad_sum(float x) {
  x += __shfl_xor_sync(0xffffffffu, x, 1);
  return x + __shfl_xor_sync(0xffffffffu, x, 2);
}

struct Smem {
  unsigned char q[kRows * kRowBytes];        // Q, later phi(Q) in place
  unsigned char k[2][kKT * kRowBytes];
  unsigned char v[2][kKT * kRowBytes];
  float z[kD];
};

template <int G>
__global__ void __launch_bounds__(kThreads, 1) prefill_attn_mma_kernel(const PrefillParams p) {
  using bf16 = __nv_bfloat16;
  constexpr int TOK = kRows / G;   // tokens per CTA
  extern __shared__ __align__(128) unsigned char smem_raw[];
  Smem &sm = *reinterpret_cast<Smem *>(smem_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tiles_per_chunk = (p.C + TOK - 1) / TOK;
  const int64_t u = blockIdx.x / tiles_per_chunk;
  const int tok0 = int(blockIdx.x % tiles_per_chunk) * TOK;   // chunk-relative first token of this CTA
  const int g = int(u % p.Hkv);
  const int b = int((u / p.Hkv) % p.B);
  const int lrel = int(u / (int64_t(p.Hkv) * p.B));
  const LayerDev ld = p.layers[p.layer_begin + lrel];
  const int ntok = min(TOK, p.C - tok0);                      // valid tokens of this CTA
  const int64_t tq0 = p.n0 + p.c0 + tok0;                     // absolute position of the first token
  const int64_t tq_last = tq0 + ntok - 1;
  const int64_t w = ld.w;
  const int64_t cap = ld.cap > 0 ? ld.cap : 1;

  const size_t unit_rows = (size_t(b + p.b0) * p.Hkv + g) * size_t(ld.cap);
  const bf16 *ringK = reinterpret_cast<const bf16 *>(p.ws + ld.ringK) + unit_rows * kD;
  const bf16 *ringV = reinterpret_cast<const bf16 *>(p.ws + ld.ringV) + unit_rows * kD;
  const size_t seq = (size_t(lrel) * p.B + b) * size_t(p.T);
  const bf16 *callK = reinterpret_cast<const bf16 *>(p.k) + (seq * p.Hkv + g) * kD;
  const bf16 *callV = reinterpret_cast<const bf16 *>(p.v) + (seq * p.Hkv + g) * kD;
  const int64_t call_stride = int64_t(p.Hkv) * kD;

  const uint32_t sQ = smem_u32(sm.q);
  const uint32_t sK[2] = {smem_u32(sm.k[0]), smem_u32(sm.k[1])};
  const uint32_t sV[2] = {smem_u32(sm.v[0]), smem_u32(sm.v[1])};

  // rows of token j (absolute) -> shared tile; tokens outside [0, j_max] are zero-filled
  auto load_rows = [&](uint32_t dstK, uint32_t dstV, int64_t j0, int64_t j_max, bool want_k, bool want_v) {
#pragma unroll
    for (int i = 0; i < kKT * 16 / kThreads; ++i) {
      const int id = tid + kThreads * i;
      const int row = id >> 4, c = id & 15;
      const int64_t j = j0 + row;
      const bool valid = j >= 0 && j <= j_max;
      const int64_t jj = valid ? j : 0;
      const size_t off_call = size_t(jj >= p.n0 ? jj - p.n0 : 0) * call_stride + c * 8;
      const size_t off_ring = size_t(uint32_t(jj) % uint32_t(cap)) * kD + c * 8;
      const bool from_call = jj >= p.n0;
      if (want_k) cp_async16(dstK + swz(row, c), from_call ? callK + off_call : ringK + off_ring, valid);
      if (want_v) cp_async16(dstV + swz(row, c), from_call ? callV + off_call : ringV + off_ring, valid);
    }
  };

  // ---- Q tile ------------------------------------------------------------------------------------
  {
    const bf16 *qbase = reinterpret_cast<const bf16 *>(p.q) + (seq + size_t(p.c0 + tok0)) * p.H * kD;
#pragma unroll
    for (int i = 0; i < kRows * 16 / kThreads; ++i) {
      const int id = tid + kThreads * i;
      const int row = id >> 4, c = id & 15;
      const int tok = row / G, hh = row - tok * G;
      const bool valid = tok < ntok;
      const int head = p.heads_of[g * G + hh];
      cp_async16(sQ + swz(row, c), qbase + (size_t(valid ? tok : 0) * p.H + head) * kD + c * 8, valid);
    }
    cp_async_commit();
  }
  // first window tile
  const bool has_window = w > 0;
  int64_t j_lo = tq0 - w + 1;
  if (j_lo < 0) j_lo = 0;
  const int n_wtiles = has_window ? int((tq_last - j_lo) / kKT) + 1 : 0;
  if (n_wtiles > 0) {
    load_rows(sK[0], sV[0], j_lo, tq_last, true, true);
    cp_async_commit();
    cp_async_wait<1>();
  } else {
    cp_async_wait<0>();
  }
  __syncthreads();

  const int r0 = warp * 16;
  uint32_t qf[kD / 16][4];
  {
    const int row = r0 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
    for (int ks = 0; ks < kD / 16; ++ks) ldsm_x4(qf[ks], sQ + swz(row, 2 * ks + (lane >> 4)));
  }
  __syncwarp();
  const bool linear = ld.evicts && tq_last >= w;
  if (linear) {
    // phi(q) of this warp's 16 rows, in place (only this warp touches these rows)
#pragma unroll
    for (int rr = 0; rr < 16; rr += 4) {
      float x[4][4];
#pragma unroll
      for (int n = 0; n < 4; ++n) {
        const uint2 raw = *reinterpret_cast<const uint2 *>(sm.q + swz(r0 + rr + n, lane >> 1) + (lane & 1) * 8);
        x[n][0] = __uint_as_float(raw.x << 16);
        x[n][1] = __uint_as_float(raw.x & 0xffff0000u);
        x[n][2] = __uint_as_float(raw.y << 16);
        x[n][3] = __uint_as_float(raw.y & 0xffff0000u);
      }
      float mx[4], sum[4];
#pragma unroll
      for (int n = 0; n < 4; ++n) mx[n] = fmaxf(fmaxf(x[n][0], x[n][1]), fmaxf(x[n][2], x[n][3]));
#pragma unroll
      for (int o = 16; o > 0; o >>= 1)
#pragma unroll
        for (int n = 0; n < 4; ++n) mx[n] = fmaxf(mx[n], __shfl_xor_sync(0xffffffffu, mx[n], o));
#pragma unroll
      for (int n = 0; n < 4; ++n) {
        sum[n] = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          x[n][i] = ex2((x[n][i] - mx[n]) * kLog2e);
          sum[n] += x[n][i];
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1)
#pragma unroll
        for (int n = 0; n < 4; ++n) sum[n] += __shfl_xor_sync(0xffffffffu, sum[n], o);
#pragma unroll
      for (int n = 0; n < 4; ++n) {
        const float inv = __frcp_rn(sum[n]);
        const __nv_bfloat162 lo = __floats2bfloat162_rn(x[n][0] * inv, x[n][1] * inv);
        const __nv_bfloat162 hi = __floats2bfloat162_rn(x[n][2] * inv, x[n][3] * inv);
        uint2 outw;
        outw.x = *reinterpret_cast<const uint32_t *>(&lo);
        outw.y = *reinterpret_cast<const uint32_t *>(&hi);
        *reinterpret_cast<uint2 *>(sm.q + swz(r0 + rr + n, lane >> 1) + (lane & 1) * 8) = outw;
      }
    }
    __syncwarp();
  }

  // ---- accumulators: thread holds rows r0 + lane/4 (e = 0,1) and r0 + lane/4 + 8 (e = 2,3) -----------------
  float o[kD / 8][4];
#pragma unroll
  for (int nt = 0; nt < kD / 8; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;
  float m_row[2] = {-CUDART_INF_F, -CUDART_INF_F}, l_row[2] = {0.f, 0.f};
  const int rowA = r0 + (lane >> 2), rowB = rowA + 8;
  const int64_t tokA = tq0 + rowA / G, tokB = tq0 + rowB / G;     // absolute token of the two rows
  const int colk = (lane & 3) * 2;

  // P (or C) fragments times a V-like tile: O += P V
  auto pv = [&](const float (&s)[kKT / 8][4], uint32_t vbase) {
#pragma unroll
    for (int kk = 0; kk < kKT / 16; ++kk) {
      uint32_t a[4];
      float r_[8];
      a[0] = pack2(s[2 * kk][0], s[2 * kk][1], r_[0], r_[1]);
      a[1] = pack2(s[2 * kk][2], s[2 * kk][3], r_[2], r_[3]);
      a[2] = pack2(s[2 * kk + 1][0], s[2 * kk + 1][1], r_[4], r_[5]);
      a[3] = pack2(s[2 * kk + 1][2], s[2 * kk + 1][3], r_[6], r_[7]);
      l_row[0] += r_[0] + r_[1] + r_[4] + r_[5];   // sums of the weights as the tensor core sees them
      l_row[1] += r_[2] + r_[3] + r_[6] + r_[7];
      const int krow = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
      for (int dp = 0; dp < kD / 16; ++dp) {
        uint32_t bfr[4];
        ldsm_x4_trans(bfr, vbase + swz(krow, 2 * dp + (lane >> 4)));
        mma16816(o[2 * dp], a, bfr[0], bfr[1]);
        mma16816(o[2 * dp + 1], a, bfr[2], bfr[3]);
      }
    }
  };
  // S = A K^T for this warp's 16 rows against a 64-row K-like tile
  auto qk = [&](float (&s)[kKT / 8][4], const uint32_t (&af)[kD / 16][4], uint32_t kbase) {
#pragma unroll
    for (int nt = 0; nt < kKT / 8; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < kD / 16; ++ks) {
#pragma unroll
      for (int np = 0; np < kKT / 16; ++np) {
        uint32_t bfr[4];
        const int krow = np * 16 + (lane & 7) + ((lane >> 4) & 1) * 8;
        ldsm_x4(bfr, kbase + swz(krow, 2 * ks + ((lane >> 3) & 1)));
        mma16816(s[2 * np], af[ks], bfr[0], bfr[1]);
        mma16816(s[2 * np + 1], af[ks], bfr[2], bfr[3]);
      }
    }
  };

  // ---- window part -------------------------------------------------------------------------------------
  for (int t = 0; t < n_wtiles; ++t) {
    const int buf = t & 1;
    if (t + 1 < n_wtiles) {
      load_rows(sK[buf ^ 1], sV[buf ^ 1], j_lo + int64_t(t + 1) * kKT, tq_last, true, true);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    const int64_t j0 = j_lo + int64_t(t) * kKT;
    float s[kKT / 8][4];
    qk(s, qf, sK[buf]);
    // keys of the tile are inside every row's window and not in its future?
    const bool interior = j0 + kKT - 1 <= tq0 && j0 > tq_last - w;
#pragma unroll
    for (int nt = 0; nt < kKT / 8; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float x = s[nt][e] * p.scale_log2;
        if (!interior) {
          const int64_t j = j0 + nt * 8 + colk + (e & 1);
          const int64_t tok = (e & 2) ? tokB : tokA;
          if (j > tok || j <= tok - w) x = -CUDART_INF_F;
        }
        s[nt][e] = x;
      }
    }
    float mx[2] = {-CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
    for (int nt = 0; nt < kKT / 8; ++nt) {
      mx[0] = fmaxf(mx[0], fmaxf(s[nt][0], s[nt][1]));
      mx[1] = fmaxf(mx[1], fmaxf(s[nt][2], s[nt][3]));
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      mx[h] = quad_max(mx[h]);
      const float mn = fmaxf(m_row[h], mx[h]);
      const float corr = mn == -CUDART_INF_F ? 1.f : ex2(m_row[h] - mn);
      l_row[h] *= corr;
#pragma unroll
      for (int nt = 0; nt < kD / 8; ++nt) {
        o[nt][2 * h] *= corr;
        o[nt][2 * h + 1] *= corr;
      }
      m_row[h] = mn;
      const float ms = mn == -CUDART_INF_F ? 0.f : mn;
#pragma unroll
      for (int nt = 0; nt < kKT / 8; ++nt) {
        s[nt][2 * h] = ex2(s[nt][2 * h] - ms);
        s[nt][2 * h + 1] = ex2(s[nt][2 * h + 1] - ms);
      }
    }
    pv(s, sV[buf]);
    __syncthreads();   // the other buffer is refilled in the next iteration
  }

  // ---- linear part --------------------------------------------------------------------------------------
  if (linear) {   // uniform over the CTA
    float fl[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      // a row without evicted tokens keeps its own reference and gets phi(q) = 0: the floor belongs to the linear terms
      const bool has_lin = (h ? tokB : tokA) >= w;
      const float M = has_lin ? fmaxf(m_row[h], 0.f) : m_row[h];
      const float fw = m_row[h] == -CUDART_INF_F ? 0.f : ex2(m_row[h] - M);
      fl[h] = has_lin ? ex2(-M) : 0.f;
      l_row[h] *= fw;
#pragma unroll
      for (int nt = 0; nt < kD / 8; ++nt) {
        o[nt][2 * h] *= fw;
        o[nt][2 * h + 1] *= fw;
      }
    }
    // phi(Q) fragments scaled by 2^-m* of their row (registers of the Q fragments are reused)
    {
      const int row = r0 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
      for (int ks = 0; ks < kD / 16; ++ks) {
        ldsm_x4(qf[ks], sQ + swz(row, 2 * ks + (lane >> 4)));
        qf[ks][0] = scale2(qf[ks][0], fl[0]);
        qf[ks][2] = scale2(qf[ks][2], fl[0]);
        qf[ks][1] = scale2(qf[ks][1], fl[1]);
        qf[ks][3] = scale2(qf[ks][3], fl[1]);
      }
    }
    const int ub = (b + p.b0) * p.Hkv + g;
    const int64_t folded = p.n0 + p.c0 - w;   // tokens below this index are in S, z at the start of the chunk
    if (folded > 0) {
      // inter-chunk: the state as a bf16 "V tile" (features on the key axis), two halves of 64 rows
      const float *Sg = reinterpret_cast<const float *>(p.ws + ld.S) + size_t(ub) * kD * kD;
      const float *zg = reinterpret_cast<const float *>(p.ws + ld.z) + size_t(ub) * kD;
#pragma unroll
      for (int i = 0; i < kD * 16 / kThreads; ++i) {
        const int id = tid + kThreads * i;
        const int row = id >> 4, c = id & 15;
        const float4 f0 = *reinterpret_cast<const float4 *>(Sg + size_t(row) * kD + c * 8);
        const float4 f1 = *reinterpret_cast<const float4 *>(Sg + size_t(row) * kD + c * 8 + 4);
        const __nv_bfloat162 h0 = __floats2bfloat162_rn(f0.x, f0.y), h1 = __floats2bfloat162_rn(f0.z, f0.w);
        const __nv_bfloat162 h2 = __floats2bfloat162_rn(f1.x, f1.y), h3 = __floats2bfloat162_rn(f1.z, f1.w);
        uint4 pk;
        pk.x = *reinterpret_cast<const uint32_t *>(&h0);
        pk.y = *reinterpret_cast<const uint32_t *>(&h1);
        pk.z = *reinterpret_cast<const uint32_t *>(&h2);
        pk.w = *reinterpret_cast<const uint32_t *>(&h3);
        *reinterpret_cast<uint4 *>(sm.v[row >> 6] + swz(row & 63, c)) = pk;
      }
      if (tid < kD) sm.z[tid] = zg[tid];
      __syncthreads();
#pragma unroll
      for (int half = 0; half < 2; ++half) {
#pragma unroll
        for (int kk = 0; kk < kKT / 16; ++kk) {
          const int ks = half * 4 + kk;   // features 16 ks .. 16 ks + 15
          const int krow = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
          for (int dp = 0; dp < kD / 16; ++dp) {
            uint32_t bfr[4];
            ldsm_x4_trans(bfr, sV[half] + swz(krow, 2 * dp + (lane >> 4)));
            mma16816(o[2 * dp], qf[ks], bfr[0], bfr[1]);
            mma16816(o[2 * dp + 1], qf[ks], bfr[2], bfr[3]);
          }
          // l += (phi(q) 2^-m*) . z over these 16 features: a0,a2 belong to row A, a1,a3 to row B
          const float z0 = sm.z[ks * 16 + colk], z1 = sm.z[ks * 16 + colk + 1];
          const float z8 = sm.z[ks * 16 + colk + 8], z9 = sm.z[ks * 16 + colk + 9];
          const uint32_t a0 = qf[ks][0], a1 = qf[ks][1], a2 = qf[ks][2], a3 = qf[ks][3];
          l_row[0] += __uint_as_float(a0 << 16) * z0 + __uint_as_float(a0 & 0xffff0000u) * z1 +
                      __uint_as_float(a2 << 16) * z8 + __uint_as_float(a2 & 0xffff0000u) * z9;
          l_row[1] += __uint_as_float(a1 << 16) * z0 + __uint_as_float(a1 & 0xffff0000u) * z1 +
                      __uint_as_float(a3 << 16) * z8 + __uint_as_float(a3 & 0xffff0000u) * z9;
        }
      }
      __syncthreads();
    }
    // intra-chunk: delayed tokens of this chunk up to the tile's last token
    const int i_lo = folded < 0 ? int(-folded < int64_t(p.C) ? -folded : int64_t(p.C)) : 0;
    const int i_hi = tok0 + ntok - 1;
    const float *pk = p.phik + size_t(u) * p.Cmax * kD;
    for (int i0 = i_lo & ~(kKT - 1); i0 <= i_hi; i0 += kKT) {
      // phi(K') tile: fp32 scratch -> bf16, swizzled; V' tile: rows of the delayed tokens
#pragma unroll
      for (int i = 0; i < kKT * 16 / kThreads; ++i) {
        const int id = tid + kThreads * i;
        const int row = id >> 4, c = id & 15;
        const int ii = i0 + row;
        uint4 pkd = make_uint4(0u, 0u, 0u, 0u);
        if (ii >= i_lo && ii <= i_hi) {
          const float4 f0 = *reinterpret_cast<const float4 *>(pk + size_t(ii) * kD + c * 8);
          const float4 f1 = *reinterpret_cast<const float4 *>(pk + size_t(ii) * kD + c * 8 + 4);
          const __nv_bfloat162 h0 = __floats2bfloat162_rn(f0.x, f0.y), h1 = __floats2bfloat162_rn(f0.z, f0.w);
          const __nv_bfloat162 h2 = __floats2bfloat162_rn(f1.x, f1.y), h3 = __floats2bfloat162_rn(f1.z, f1.w);
          pkd.x = *reinterpret_cast<const uint32_t *>(&h0);
          pkd.y = *reinterpret_cast<const uint32_t *>(&h1);
          pkd.z = *reinterpret_cast<const uint32_t *>(&h2);
          pkd.w = *reinterpret_cast<const uint32_t *>(&h3);
        }
        *reinterpret_cast<uint4 *>(sm.k[0] + swz(row, c)) = pkd;
      }
      // delayed token of chunk index ii is token n0 + c0 + ii - w; indices outside [i_lo, i_hi] are zero-filled
      {
        const int64_t jbase = p.n0 + p.c0 - w;
#pragma unroll
        for (int i = 0; i < kKT * 16 / kThreads; ++i) {
          const int id = tid + kThreads * i;
          const int row = id >> 4, c = id & 15;
          const int ii = i0 + row;
          const bool valid = ii >= i_lo && ii <= i_hi;
          const int64_t jj = valid ? jbase + ii : 0;
          const bool from_call = jj >= p.n0;
          const size_t off_call = size_t(from_call ? jj - p.n0 : 0) * call_stride + c * 8;
          const size_t off_ring = size_t(uint32_t(jj) % uint32_t(cap)) * kD + c * 8;
          cp_async16(sV[0] + swz(row, c), from_call ? callV + off_call : ringV + off_ring, valid);
        }
        cp_async_commit();
        cp_async_wait<0>();
      }
      __syncthreads();
      float s[kKT / 8][4];
      qk(s, qf, sK[0]);   // already carries 2^-m* of the row
#pragma unroll
      for (int nt = 0; nt < kKT / 8; ++nt) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int ii = i0 + nt * 8 + colk + (e & 1);
          const int tl = tok0 + ((e & 2) ? rowB : rowA) / G;   // chunk-relative token of the row
          if (ii > tl || ii < i_lo) s[nt][e] = 0.f;
        }
      }
      pv(s, sV[0]);
      __syncthreads();
    }
  }

  // ---- shared normaliser and store ------------------------------------------------------------------------
  bf16 *obase = reinterpret_cast<bf16 *>(p.out) + (seq + size_t(p.c0 + tok0)) * p.H * kD;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const float lsum = quad_sum(l_row[h]);
    const int row = h ? rowB : rowA;
    const int tok = row / G, hh = row - tok * G;
    if (tok < ntok) {
      const float inv = 1.0f / lsum;
      const int head = p.heads_of[g * G + hh];
      bf16 *op = obase + (size_t(tok) * p.H + head) * kD;
#pragma unroll
      for (int nt = 0; nt < kD / 8; ++nt)
        *reinterpret_cast<__nv_bfloat162 *>(op + nt * 8 + colk) = __floats2bfloat162_rn(o[nt][2 * h] * inv, o[nt][2 * h + 1] * inv);
    }
  }
}

}  // namespace

namespace {
// Learned feature map of the chunk's query rows for the tcgen05 attention kernel: Y = X W on the tensor cores (X: 128
// tokens of one query head, bf16; W: the head's d x d projection; fp32 accumulation), then phi = [softmax(Y);
// softmax(-Y)] per row, written as bf16 into the two half arrays, row (unit, token, head of the group).
// One CTA of 8 warps per (layer, sequence, query head, 128 tokens); a warp owns 16 rows, whose 128 outputs sit in its
// accumulator fragments (a row's entries across the four lanes of a quad).
constexpr int kProjRows = 128;
struct ProjSmem {
  unsigned char x[kProjRows * kRowBytes];   // swizzled [token][128] bf16
  unsigned char w[kD * kRowBytes];          // swizzled [i][j] bf16
};
// KEYS: the same for the chunk's delayed keys k'_i = k_(i - w) of one unit (ring rows for tokens older than the call, the
// call's rows otherwise; the KV head's projection): fp32 rows [unit][chunk][2d] for the carry and the bf16 halves.
template <int G, bool KEYS>
__global__ void __launch_bounds__(kThreads) prefill_project_mma_kernel(const PrefillParams p) {
  using bf16 = __nv_bfloat16;
  extern __shared__ __align__(128) unsigned char proj_raw[];
  ProjSmem &sm = *reinterpret_cast<ProjSmem *>(proj_raw);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int blocks_per_head = (p.C + kProjRows - 1) / kProjRows;
  const int i0 = int(blockIdx.x % blocks_per_head) * kProjRows;
  const int64_t uh = blockIdx.x / blocks_per_head;   // (unit, head of the group); KEYS: the unit
  const int hh = KEYS ? 0 : int(uh % G);
  const int64_t u = KEYS ? uh : uh / G;
  const int g = int(u % p.Hkv);
  const int b = int((u / p.Hkv) % p.B);
  const int lrel = int(u / (int64_t(p.Hkv) * p.B));
  const LayerDev ld = p.layers[p.layer_begin + lrel];
  if (!ld.evicts) return;
  const int head = p.heads_of[g * G + hh];
  const int ntok = min(kProjRows, p.C - i0);
  const size_t seq = (size_t(lrel) * p.B + b) * size_t(p.T);
  const bf16 *qrow = reinterpret_cast<const bf16 *>(p.q) + (seq + size_t(p.c0 + i0)) * p.H * kD + size_t(head) * kD;
  const bf16 *callK = reinterpret_cast<const bf16 *>(p.k) + (seq * p.Hkv + g) * kD;
  const uint64_t cap = ld.cap > 0 ? uint64_t(ld.cap) : 1u;
  const bf16 *ringK = reinterpret_cast<const bf16 *>(p.ws + ld.ringK) + (size_t(b + p.b0) * p.Hkv + g) * size_t(ld.cap) * kD;
  const int64_t j0 = p.n0 + p.c0 + i0 - ld.wlin;   // the delayed token of the tile's first row
  const bf16 *W = KEYS ? reinterpret_cast<const bf16 *>(p.wk) + (size_t(p.layer_begin + lrel) * p.Hkv + g) * kD * kD
                       : reinterpret_cast<const bf16 *>(p.wq) + (size_t(p.layer_begin + lrel) * p.H + head) * kD * kD;
  const uint32_t sX = smem_u32(sm.x), sW = smem_u32(sm.w);
  for (int id = tid; id < kProjRows * 16; id += kThreads) {
    const int r = id >> 4, c = id & 15;
    if (KEYS) {
      const int64_t j = j0 + r;
      const bool valid = r < ntok && j >= 0;
      const bf16 *src = !valid ? callK : (j >= p.n0 ? callK + size_t(j - p.n0) * p.Hkv * kD : ringK + size_t(uint64_t(j) % cap) * kD);
      cp_async16(sX + swz(r, c), src + c * 8, valid);
    } else {
      cp_async16(sX + swz(r, c), qrow + size_t(r < ntok ? r : 0) * p.H * kD + c * 8, r < ntok);
    }
  }
  for (int id = tid; id < kD * 16; id += kThreads) {
    const int r = id >> 4, c = id & 15;
    cp_async16(sW + swz(r, c), W + size_t(r) * kD + c * 8, true);
  }
  cp_async_commit();
  cp_async_wait<0>();
  __syncthreads();

  const int r0 = warp * 16;
  float y[kD / 8][4];
#pragma unroll
  for (int nt = 0; nt < kD / 8; ++nt) y[nt][0] = y[nt][1] = y[nt][2] = y[nt][3] = 0.f;
#pragma unroll
  for (int ks = 0; ks < kD / 16; ++ks) {
    uint32_t af[4];
    ldsm_x4(af, sX + swz(r0 + (lane & 7) + ((lane >> 3) & 1) * 8, 2 * ks + (lane >> 4)));
    const int krow = ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
    for (int dp = 0; dp < kD / 16; ++dp) {
      uint32_t bfr[4];
      ldsm_x4_trans(bfr, sW + swz(krow, 2 * dp + (lane >> 4)));
      mma16816(y[2 * dp], af, bfr[0], bfr[1]);
      mma16816(y[2 * dp + 1], af, bfr[2], bfr[3]);
    }
  }
  // rows r0 + lane / 4 (entries [.][0], [.][1]) and that + 8 (entries [.][2], [.][3]); columns nt * 8 + (lane & 3) * 2 + {0, 1}
  constexpr float kLog2e = 1.4426950408889634f;
#pragma unroll
  for (int rr = 0; rr < 2; ++rr) {
    float mx = -CUDART_INF_F, mn = CUDART_INF_F;
#pragma unroll
    for (int nt = 0; nt < kD / 8; ++nt) {
      mx = fmaxf(mx, fmaxf(y[nt][2 * rr], y[nt][2 * rr + 1]));
      mn = fminf(mn, fminf(y[nt][2 * rr], y[nt][2 * rr + 1]));
    }
    mx = quad_max(mx);
    mn = -quad_max(-mn);
    float sp = 0.f, sn = 0.f;
    float ep[kD / 8][2], en[kD / 8][2];
#pragma unroll
    for (int nt = 0; nt < kD / 8; ++nt)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        ep[nt][e] = ex2((y[nt][2 * rr + e] - mx) * kLog2e);
        en[nt][e] = ex2((mn - y[nt][2 * rr + e]) * kLog2e);
        sp += ep[nt][e];
        sn += en[nt][e];
      }
    const float ip = 1.0f / quad_sum(sp), in = 1.0f / quad_sum(sn);
    const int tok = r0 + (lane >> 2) + rr * 8;
    if (tok >= ntok || (KEYS && j0 + tok < 0)) continue;
    const int col = (lane & 3) * 2;
    if (KEYS) {
      float *d32 = p.phik + (size_t(u) * p.Cmax + i0 + tok) * (2 * kD) + col;
#pragma unroll
      for (int nt = 0; nt < kD / 8; ++nt) {
        *reinterpret_cast<float2 *>(d32 + nt * 8) = make_float2(ep[nt][0] * ip, ep[nt][1] * ip);
        *reinterpret_cast<float2 *>(d32 + kD + nt * 8) = make_float2(en[nt][0] * in, en[nt][1] * in);
      }
    }
    bf16 *dst = KEYS ? reinterpret_cast<bf16 *>(p.phik16) + (size_t(u) * p.Cmax + i0 + tok) * kD + col
                     : reinterpret_cast<bf16 *>(p.phiq16) + ((size_t(u) * p.Cmax + i0 + tok) * G + hh) * kD + col;
    const size_t half = KEYS ? size_t(p.units_cap) * p.Cmax * kD : size_t(p.units_cap) * p.Cmax * G * kD;
    if (dst != nullptr && (!KEYS || p.phik16)) {
#pragma unroll
      for (int nt = 0; nt < kD / 8; ++nt) {
        *reinterpret_cast<__nv_bfloat162 *>(dst + nt * 8) = __floats2bfloat162_rn(ep[nt][0] * ip, ep[nt][1] * ip);
        *reinterpret_cast<__nv_bfloat162 *>(dst + half + nt * 8) = __floats2bfloat162_rn(en[nt][0] * in, en[nt][1] * in);
      }
    }
  }
}
}  // namespace

// phi_W of the chunk's query rows (keys = false) or of its delayed keys (keys = true) on the tensor cores (see the kernel)
int launch_prefill_project(glide_ctx *ctx, const PrefillParams &p, bool keys, cudaStream_t stream) {
  const int64_t units = int64_t(p.layer_count) * p.B * p.Hkv;
  auto launch = [&](auto gg) -> int {
    constexpr int G = decltype(gg)::value;
    auto run = [&](auto kern, int64_t blocks) -> int {
      if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sizeof(ProjSmem))) != cudaSuccess) {
        cudaGetLastError();
        return GLIDE_ERR_CUDA;
      }
      kern<<<unsigned(blocks), kThreads, sizeof(ProjSmem), stream>>>(p);
      return cudaGetLastError() == cudaSuccess ? GLIDE_OK : GLIDE_ERR_CUDA;
    };
    const int64_t tiles = (p.C + kProjRows - 1) / kProjRows;
    return keys ? run(prefill_project_mma_kernel<G, true>, units * tiles) : run(prefill_project_mma_kernel<G, false>, units * G * tiles);
  };
  switch (ctx->G) {
    case 1: return launch(IntTag<1>{});
    case 2: return launch(IntTag<2>{});
    case 4: return launch(IntTag<4>{});
    case 8: return launch(IntTag<8>{});
    default: return GLIDE_ERR_UNSUPPORTED;
  }
}

bool prefill_attn_mma_supported(const glide_ctx *ctx) {
  return ctx->cfg.io_dtype == GLIDE_BF16 && ctx->cfg.head_dim == kD;
}

int launch_prefill_attn_mma(glide_ctx *ctx, const PrefillParams &p, cudaStream_t stream) {
  const int64_t units = int64_t(p.layer_count) * p.B * p.Hkv;
  auto launch = [&](auto gg) -> int {
    constexpr int G = decltype(gg)::value;
    constexpr int TOK = kRows / G;
    auto kern = prefill_attn_mma_kernel<G>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sizeof(Smem))) != cudaSuccess) {
      cudaGetLastError();
      return GLIDE_ERR_CUDA;
    }
    const int64_t blocks = units * ((p.C + TOK - 1) / TOK);
    kern<<<unsigned(blocks), kThreads, sizeof(Smem), stream>>>(p);
    return cudaGetLastError() == cudaSuccess ? GLIDE_OK : GLIDE_ERR_CUDA;
  };
  switch (ctx->G) {
    case 1: return launch(IntTag<1>{});
    case 2: return launch(IntTag<2>{});
    case 4: return launch(IntTag<4>{});
    case 8: return launch(IntTag<8>{});
    default: return GLIDE_ERR_UNSUPPORTED;
  }
}

}  // namespace glide
