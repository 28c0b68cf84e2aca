// GLIDE prefill outputs on the 5th-generation tensor cores (tcgen05 + TMEM), bf16 I/O, head_dim 128.
//
// One CTA (128 threads) owns 128 query rows of one (layer, sequence, KV head) unit -- 128/G consecutive
// tokens of the chunk times the G query heads (row = token * G + head) -- and thread r owns row r, which
// is also TMEM lane r.
//   window part   128-key tiles of the sliding window (ring rows for tokens older than the call, the call's
//                 own rows otherwise) are staged with cp.async into the 128-byte-swizzled K-major / MN-major
//                 layouts tcgen05.mma reads.  One elected thread issues S = Q K^T (8 x m128n128k16) into TMEM
//                 columns [0,128); every thread reads its row with tcgen05.ld, masks, takes the row maximum
//                 without any shuffle, writes P = 2^(s - m_ref) as bf16 into the swizzled A-operand layout,
//                 and the elected thread issues O += P V into TMEM columns [128,256).  The reference m_ref is
//                 lazy: O is rescaled in TMEM (tcgen05.ld / tcgen05.st) only when a row's maximum grows by
//                 more than 2^8.  K tiles are prefetched two tiles ahead, V tiles one.
//   linear part   with m* = max(m_ref, 0) per row: phi(Q) 2^-m* (bf16, K-major) times a bf16 copy of the state
//                 (inter-chunk), and C = phi(Q) phi(K')^T masked to j' <= i, then C V' (intra-chunk), through the
//                 same two MMAs; l accumulates the matching sums.
//   out = O / l, bf16, one contiguous 256-byte row per thread.
// Every mbarrier wait is bounded; on a time-out the CTA records kDevWaitTimeout, skips the remaining work,
// frees its TMEM columns and returns.
#include <algorithm>

#include "glide_device.cuh"

namespace glide {

namespace {

constexpr int kD = 128;
constexpr int kRows = 128;
constexpr int kKT = 128;             // keys per tile
constexpr int kThreads = 128;
constexpr uint32_t kTileBytes = 32768;   // [2 boxes][128 rows][64 bf16]
constexpr uint32_t kBoxBytes = 16384;
constexpr uint32_t kWaitLimit = 1u << 20;
constexpr float kLazy = 8.0f;        // rescale O only when the row maximum grows by more than 2^8

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return uint32_t(__cvta_generic_to_shared(p)); }
// byte offset of 16-byte chunk c16 (0..15) of row `row` inside a [2][128][64] bf16 tile with 128-byte swizzle
__device__ __forceinline__ uint32_t sw128(int row, int c16) {
  return uint32_t((c16 >> 3) * kBoxBytes + row * 128 + (((c16 & 7) ^ (row & 7)) << 4));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid) {
  const int bytes = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// shared-memory matrix descriptor, 128-byte swizzle
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= uint64_t((saddr & 0x3FFFF) >> 4);
  d |= uint64_t((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= uint64_t((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= uint64_t(1) << 46;
  d |= uint64_t(2) << 61;
  return d;
}
// instruction descriptor: fp32 accumulate, bf16 A and B, M = N = 128; b_mn: B operand is MN-major
__device__ __forceinline__ uint32_t make_idesc(bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn ? (1u << 16) : 0u) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
}
__device__ __forceinline__ void mma_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok = 0;
  for (uint32_t spin = 0; spin < kWaitLimit && !ok; ++spin)
    asm volatile("{.reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p;}"
                 : "=r"(ok)
                 : "r"(bar), "r"(parity)
                 : "memory");
  return ok != 0;
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
      "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]),
      "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]),
      "r"(r[31])
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

struct Smem {
  unsigned char q[kTileBytes];       // Q, later phi(Q) 2^-m*
  unsigned char p[kTileBytes];       // P (or C): A operand of the second MMA
  unsigned char k[2][kTileBytes];    // K tiles / phi(K') tile
  unsigned char v[2][kTileBytes];    // V tiles / bf16 state / V' tile
  float z[kD];
  uint64_t bar;                      // completion of the MMAs issued so far
  uint32_t tmem_base;
  int failed;
};


template <int G>
__global__ void __launch_bounds__(kThreads, 1) prefill_attn_tc_kernel(const PrefillParams p) {
  using bf16 = __nv_bfloat16;
  constexpr int TOK = kRows / G;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  Smem &sm = *reinterpret_cast<Smem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, warp = tid >> 5;
  const int tiles_per_chunk = (p.C + TOK - 1) / TOK;
  const int64_t u = blockIdx.x / tiles_per_chunk;
  const int tok0 = int(blockIdx.x % tiles_per_chunk) * TOK;
  const int g = int(u % p.Hkv);
  const int b = int((u / p.Hkv) % p.B);
  const int lrel = int(u / (int64_t(p.Hkv) * p.B));
  const LayerDev ld = p.layers[p.layer_begin + lrel];
  const int ntok = min(TOK, p.C - tok0);
  const int64_t tq0 = p.n0 + p.c0 + tok0;
  const int64_t tq_last = tq0 + ntok - 1;
  const int64_t w = ld.w;
  const uint32_t cap = ld.cap > 0 ? uint32_t(ld.cap) : 1u;

  const size_t unit_rows = (size_t(b) * p.Hkv + g) * size_t(ld.cap);
  const bf16 *ringK = reinterpret_cast<const bf16 *>(p.ws + ld.ringK) + unit_rows * kD;
  const bf16 *ringV = reinterpret_cast<const bf16 *>(p.ws + ld.ringV) + unit_rows * kD;
  const size_t seq = (size_t(lrel) * p.B + b) * size_t(p.T);
  const bf16 *callK = reinterpret_cast<const bf16 *>(p.k) + (seq * p.Hkv + g) * kD;
  const bf16 *callV = reinterpret_cast<const bf16 *>(p.v) + (seq * p.Hkv + g) * kD;
  const int64_t call_stride = int64_t(p.Hkv) * kD;

  // a time-out recorded by an earlier CTA ends the launch quickly
  if (*reinterpret_cast<volatile int32_t *>(&p.ctl->status) == kDevWaitTimeout) return;

  const uint32_t sQ = smem_u32(sm.q), sP = smem_u32(sm.p);
  const uint32_t sK[2] = {smem_u32(sm.k[0]), smem_u32(sm.k[1])};
  const uint32_t sV[2] = {smem_u32(sm.v[0]), smem_u32(sm.v[1])};
  const uint32_t bar = smem_u32(&sm.bar);

  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    sm.failed = 0;
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 256;" ::"r"(smem_u32(&sm.tmem_base)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  const uint32_t tS = tmem + (uint32_t(warp * 32) << 16);         // this warp's lanes, columns [0,128): S / C
  const uint32_t tO = tS + 128;                                    // columns [128,256): O
  uint32_t phase = 0;
  bool failed = false;

  // rows of tokens j0 .. j0+127 (absolute) of K or V -> swizzled tile; tokens outside [0, j_max] are zero-filled
  auto load_rows = [&](uint32_t dst, bool is_v, int64_t j0, int64_t j_max) {
    const bf16 *ring = is_v ? ringV : ringK;
    const bf16 *call = is_v ? callV : callK;
#pragma unroll 4
    for (int i = 0; i < kKT * 16 / kThreads; ++i) {
      const int id = tid + kThreads * i;
      const int r = id >> 4, c = id & 15;
      const int64_t j = j0 + r;
      const bool valid = j >= 0 && j <= j_max;
      const int64_t jj = valid ? j : 0;
      const bool from_call = jj >= p.n0;
      const bf16 *src = from_call ? call + size_t(jj - p.n0) * call_stride : ring + size_t(uint32_t(jj) % cap) * kD;
      cp_async16(dst + sw128(r, c), src + c * 8, valid);
    }
  };
  // 8 MMAs of one 128 x 128 x 128 product; B K-major (S = A B^T) or MN-major (O += A B)
  auto issue_mma = [&](uint32_t tmem_d, uint32_t a_tile, uint32_t b_tile, bool b_mn, bool accumulate) {
    const uint32_t idesc = make_idesc(b_mn);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      const uint64_t adesc = make_desc(a_tile + (ks >> 2) * kBoxBytes + (ks & 3) * 32, 16, 1024);
      const uint64_t bdesc = b_mn ? make_desc(b_tile + ks * 2048, kBoxBytes, 1024)
                                  : make_desc(b_tile + (ks >> 2) * kBoxBytes + (ks & 3) * 32, 16, 1024);
      mma_f16(tmem_d, adesc, bdesc, idesc, (accumulate || ks > 0) ? 1u : 0u);
    }
  };
  // all threads wait for the MMAs committed so far; `failed` stays uniform over the warp
  auto wait_mma = [&]() {
    __syncwarp();
    bool bad = failed;
    if (!bad && !mbar_wait(bar, phase & 1u)) {
      bad = true;
      sm.failed = 1;
    }
    failed = __any_sync(0xffffffffu, bad);
    ++phase;
    tc_fence_after();
  };
  // multiply this thread's O row by f (warp-collective TMEM read-modify-write)
  auto scale_o = [&](float f) {
#pragma unroll 1
    for (int c0 = 0; c0 < kD; c0 += 32) {
      uint32_t r[32];
      tmem_ld32(tO + c0, r);
#pragma unroll
      for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * f);
      tmem_st32(tO + c0, r);
    }
  };

  const int row = tid;
  const int tok_r = row / G, hh = row - tok_r * G;
  const int64_t tok_abs = tq0 + tok_r;

  // ---- prologue: Q and the first tiles ---------------------------------------------------------------
  const bool has_window = w > 0;
  int64_t j_lo = tq0 - w + 1;
  if (j_lo < 0) j_lo = 0;
  const int n_wtiles = has_window ? int((tq_last - j_lo) / kKT) + 1 : 0;
  {
    const bf16 *qbase = reinterpret_cast<const bf16 *>(p.q) + (seq + size_t(p.c0 + tok0)) * p.H * kD;
#pragma unroll 4
    for (int i = 0; i < kRows * 16 / kThreads; ++i) {
      const int id = tid + kThreads * i;
      const int r = id >> 4, c = id & 15;
      const int tk = r / G, h2 = r - tk * G;
      const bool valid = tk < ntok;
      cp_async16(sQ + sw128(r, c), qbase + (size_t(valid ? tk : 0) * p.H + p.heads_of[g * G + h2]) * kD + c * 8, valid);
    }
    if (n_wtiles > 0) load_rows(sK[0], false, j_lo, tq_last);
    cp_async_commit();
    if (n_wtiles > 1) load_rows(sK[1], false, j_lo + kKT, tq_last);
    if (n_wtiles > 0) load_rows(sV[0], true, j_lo, tq_last);
    cp_async_commit();
  }
  bool o_init = false;   // O holds a valid accumulation (uniform over the CTA)
  if (n_wtiles > 0) {
    cp_async_wait<1>();
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      issue_mma(tmem, sQ, sK[0], false, false);
      mma_commit(bar);
    }
  }

  float m_ref = -CUDART_INF_F, l_sum = 0.f;
  // ---- window part -------------------------------------------------------------------------------------
  for (int t = 0; t < n_wtiles; ++t) {
    wait_mma();   // S(t) is in TMEM, O += P V of tile t-1 has finished
    if (t + 2 < n_wtiles) load_rows(sK[t & 1], false, j_lo + int64_t(t + 2) * kKT, tq_last);
    if (t + 1 < n_wtiles) load_rows(sV[(t + 1) & 1], true, j_lo + int64_t(t + 1) * kKT, tq_last);
    cp_async_commit();
    const int64_t j0 = j_lo + int64_t(t) * kKT;
    const bool interior = j0 + kKT - 1 <= tq0 && j0 > tq_last - w;
    if (!failed) {
      // pass 1: row maximum of the masked, scaled logits
      float mx = -CUDART_INF_F;
#pragma unroll 1
      for (int c0 = 0; c0 < kKT; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tS + c0, r);
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const int64_t j = j0 + c0 + i;
          const bool ok = interior || (j <= tok_abs && j > tok_abs - w);
          if (ok) mx = fmaxf(mx, __uint_as_float(r[i]) * p.scale_log2);
        }
      }
      // lazy reference: move it (and rescale O, l) only when the maximum grows by more than 2^kLazy
      float f = 1.f;
      if (mx > m_ref + kLazy || (m_ref == -CUDART_INF_F && mx > -CUDART_INF_F)) {
        f = m_ref == -CUDART_INF_F ? 0.f : ex2(m_ref - mx);
        m_ref = mx;
      }
      if (o_init && __any_sync(0xffffffffu, f != 1.f)) scale_o(f);
      l_sum *= f;
      const float mr = m_ref == -CUDART_INF_F ? 0.f : m_ref;
      // pass 2: P = 2^(s - m_ref) as bf16 into the swizzled A-operand layout; the row sum uses the rounded weights
#pragma unroll 1
      for (int c0 = 0; c0 < kKT; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(tS + c0, r);
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          uint32_t pk[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float pv[2];
#pragma unroll
            for (int z2 = 0; z2 < 2; ++z2) {
              const int i = q4 * 8 + e * 2 + z2;
              const int64_t j = j0 + c0 + i;
              const bool ok = interior || (j <= tok_abs && j > tok_abs - w);
              pv[z2] = ok ? ex2(__uint_as_float(r[i]) * p.scale_log2 - mr) : 0.f;
            }
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(pv[0], pv[1]);
            l_sum += __low2float(h2) + __high2float(h2);
            pk[e] = *reinterpret_cast<const uint32_t *>(&h2);
          }
          *reinterpret_cast<uint4 *>(sm.p + sw128(row, (c0 >> 3) + q4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        }
      }
    }
    cp_async_wait<1>();
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      issue_mma(tmem + 128, sP, sV[t & 1], true, o_init);
      if (t + 1 < n_wtiles) issue_mma(tmem, sQ, sK[(t + 1) & 1], false, false);
      mma_commit(bar);
    }
    o_init = true;
  }
  if (n_wtiles > 0) wait_mma();
  cp_async_wait<0>();
  __syncthreads();   // every thread's copies into the Q tile have landed before rows are overwritten

  // ---- linear part --------------------------------------------------------------------------------------
  const bool linear = ld.evicts && tq_last >= w;
  if (linear) {
    const float M = fmaxf(m_ref, 0.f);
    const float fw = m_ref == -CUDART_INF_F ? 0.f : ex2(m_ref - M);
    const float fl = ex2(-M);
    if (o_init && !failed && __any_sync(0xffffffffu, fw != 1.f)) scale_o(fw);
    l_sum *= fw;
    // phi(q) of this thread's row, times 2^-m*, as bf16 (kept packed in registers and written to the Q tile)
    uint32_t phq[kD / 2];
    {
      const bf16 *qrow = reinterpret_cast<const bf16 *>(p.q) +
                         ((seq + size_t(p.c0 + tok0 + (tok_r < ntok ? tok_r : 0))) * p.H + p.heads_of[g * G + hh]) * kD;
#pragma unroll
      for (int i = 0; i < kD / 8; ++i) {
        const uint4 v4 = *reinterpret_cast<const uint4 *>(qrow + i * 8);
        phq[i * 4 + 0] = v4.x;
        phq[i * 4 + 1] = v4.y;
        phq[i * 4 + 2] = v4.z;
        phq[i * 4 + 3] = v4.w;
      }
      float mx = -CUDART_INF_F;
#pragma unroll
      for (int i = 0; i < kD / 2; ++i)
        mx = fmaxf(mx, fmaxf(__uint_as_float(phq[i] << 16), __uint_as_float(phq[i] & 0xffff0000u)));
      float sum = 0.f;
#pragma unroll
      for (int i = 0; i < kD / 2; ++i)
        sum += ex2((__uint_as_float(phq[i] << 16) - mx) * kLog2e) + ex2((__uint_as_float(phq[i] & 0xffff0000u) - mx) * kLog2e);
      const float sc = fl * __frcp_rn(sum);
#pragma unroll
      for (int i = 0; i < kD / 2; ++i) {
        const __nv_bfloat162 h2 = __floats2bfloat162_rn(ex2((__uint_as_float(phq[i] << 16) - mx) * kLog2e) * sc,
                                                        ex2((__uint_as_float(phq[i] & 0xffff0000u) - mx) * kLog2e) * sc);
        phq[i] = *reinterpret_cast<const uint32_t *>(&h2);
      }
#pragma unroll
      for (int c = 0; c < 16; ++c)
        *reinterpret_cast<uint4 *>(sm.q + sw128(row, c)) = make_uint4(phq[c * 4], phq[c * 4 + 1], phq[c * 4 + 2], phq[c * 4 + 3]);
    }
    const int ub = b * p.Hkv + g;
    const int64_t folded = p.n0 + p.c0 - w;   // tokens below this index are in S, z at the start of the chunk
    if (folded > 0) {
      // inter-chunk: O += (phi(Q) 2^-m*) S with a bf16 copy of the state as the MN-major B tile
      const float *Sg = reinterpret_cast<const float *>(p.ws + ld.S) + size_t(ub) * kD * kD;
      const float *zg = reinterpret_cast<const float *>(p.ws + ld.z) + size_t(ub) * kD;
#pragma unroll 4
      for (int i = 0; i < kD * 16 / kThreads; ++i) {
        const int id = tid + kThreads * i;
        const int r = id >> 4, c = id & 15;
        const float4 f0 = *reinterpret_cast<const float4 *>(Sg + size_t(r) * kD + c * 8);
        const float4 f1 = *reinterpret_cast<const float4 *>(Sg + size_t(r) * kD + c * 8 + 4);
        const __nv_bfloat162 h0 = __floats2bfloat162_rn(f0.x, f0.y), h1 = __floats2bfloat162_rn(f0.z, f0.w);
        const __nv_bfloat162 h2 = __floats2bfloat162_rn(f1.x, f1.y), h3 = __floats2bfloat162_rn(f1.z, f1.w);
        *reinterpret_cast<uint4 *>(sm.v[0] + sw128(r, c)) =
            make_uint4(*reinterpret_cast<const uint32_t *>(&h0), *reinterpret_cast<const uint32_t *>(&h1),
                       *reinterpret_cast<const uint32_t *>(&h2), *reinterpret_cast<const uint32_t *>(&h3));
      }
      sm.z[tid] = zg[tid];
      fence_async_smem();
      tc_fence_before();
      __syncthreads();
      if (tid == 0) {
        tc_fence_after();
        issue_mma(tmem + 128, sQ, sV[0], true, o_init);
        mma_commit(bar);
      }
      o_init = true;
      float dot = 0.f;
#pragma unroll
      for (int i = 0; i < kD / 2; ++i)
        dot += __uint_as_float(phq[i] << 16) * sm.z[2 * i] + __uint_as_float(phq[i] & 0xffff0000u) * sm.z[2 * i + 1];
      l_sum += dot;
      wait_mma();
    } else {
      fence_async_smem();
      __syncthreads();
    }
    // intra-chunk: delayed tokens of this chunk up to the tile's last token, 128 at a time
    const int i_lo = folded < 0 ? int(-folded < int64_t(p.C) ? -folded : int64_t(p.C)) : 0;
    const int i_hi = tok0 + ntok - 1;
    const int tl = tok0 + tok_r;   // chunk-relative token of this row
    const float *pkp = p.phik + size_t(u) * p.Cmax * kD;
    for (int i0 = i_lo & ~(kKT - 1); i0 <= i_hi; i0 += kKT) {
      // phi(K') tile (fp32 scratch -> bf16, K-major) and the delayed tokens' V rows (MN-major)
#pragma unroll 4
      for (int i = 0; i < kKT * 16 / kThreads; ++i) {
        const int id = tid + kThreads * i;
        const int r = id >> 4, c = id & 15;
        const int ii = i0 + r;
        uint4 pkd = make_uint4(0u, 0u, 0u, 0u);
        if (ii >= i_lo && ii <= i_hi) {
          const float4 f0 = *reinterpret_cast<const float4 *>(pkp + size_t(ii) * kD + c * 8);
          const float4 f1 = *reinterpret_cast<const float4 *>(pkp + size_t(ii) * kD + c * 8 + 4);
          const __nv_bfloat162 h0 = __floats2bfloat162_rn(f0.x, f0.y), h1 = __floats2bfloat162_rn(f0.z, f0.w);
          const __nv_bfloat162 h2 = __floats2bfloat162_rn(f1.x, f1.y), h3 = __floats2bfloat162_rn(f1.z, f1.w);
          pkd = make_uint4(*reinterpret_cast<const uint32_t *>(&h0), *reinterpret_cast<const uint32_t *>(&h1),
                           *reinterpret_cast<const uint32_t *>(&h2), *reinterpret_cast<const uint32_t *>(&h3));
        }
        *reinterpret_cast<uint4 *>(sm.k[0] + sw128(r, c)) = pkd;
        const bool valid = ii >= i_lo && ii <= i_hi;
        const int64_t jj = valid ? p.n0 + p.c0 - w + ii : 0;
        const bool from_call = jj >= p.n0;
        const bf16 *src = from_call ? callV + size_t(jj - p.n0) * call_stride : ringV + size_t(uint32_t(jj) % cap) * kD;
        cp_async16(sV[1] + sw128(r, c), src + c * 8, valid);
      }
      cp_async_commit();
      cp_async_wait<0>();
      fence_async_smem();
      tc_fence_before();
      __syncthreads();
      if (tid == 0) {
        tc_fence_after();
        issue_mma(tmem, sQ, sK[0], false, false);   // C = (phi(Q) 2^-m*) phi(K')^T
        mma_commit(bar);
      }
      wait_mma();
      if (!failed) {
#pragma unroll 1
        for (int c0 = 0; c0 < kKT; c0 += 32) {
          uint32_t r[32];
          tmem_ld32(tS + c0, r);
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            uint32_t pk[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              float pv[2];
#pragma unroll
              for (int z2 = 0; z2 < 2; ++z2) {
                const int i = q4 * 8 + e * 2 + z2;
                const int ii = i0 + c0 + i;
                pv[z2] = (ii <= tl && ii >= i_lo) ? __uint_as_float(r[i]) : 0.f;
              }
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(pv[0], pv[1]);
              l_sum += __low2float(h2) + __high2float(h2);
              pk[e] = *reinterpret_cast<const uint32_t *>(&h2);
            }
            *reinterpret_cast<uint4 *>(sm.p + sw128(row, (c0 >> 3) + q4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
          }
        }
      }
      fence_async_smem();
      tc_fence_before();
      __syncthreads();
      if (tid == 0) {
        tc_fence_after();
        issue_mma(tmem + 128, sP, sV[1], true, o_init);
        mma_commit(bar);
      }
      o_init = true;
      wait_mma();
    }
  }

  // ---- shared normaliser and store: one contiguous 256-byte row per thread ------------------------------------
  __syncthreads();
  if (sm.failed) {
    if (tid == 0) atomicExch(&p.ctl->status, kDevWaitTimeout);
  } else if (o_init) {
    const bool store = tok_r < ntok;   // the TMEM loads below are warp-collective: only the store is per row
    const float inv = store ? 1.0f / l_sum : 0.f;
    bf16 *op = reinterpret_cast<bf16 *>(p.out) + ((seq + size_t(p.c0 + tok0 + (store ? tok_r : 0))) * p.H + p.heads_of[g * G + hh]) * kD;
#pragma unroll 1
    for (int c0 = 0; c0 < kD; c0 += 32) {
      uint32_t r[32];
      tmem_ld32(tO + c0, r);
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        uint32_t pk[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(r[q4 * 8 + e * 2]) * inv, __uint_as_float(r[q4 * 8 + e * 2 + 1]) * inv);
          pk[e] = *reinterpret_cast<const uint32_t *>(&h2);
        }
        if (store) *reinterpret_cast<uint4 *>(op + c0 + q4 * 8) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 256;" ::"r"(tmem) : "memory");
}

}  // namespace

bool prefill_attn_tc_supported(const glide_ctx *ctx) {
  return ctx->cfg.io_dtype == GLIDE_BF16 && ctx->cfg.head_dim == kD;
}

int launch_prefill_attn_tc(glide_ctx *ctx, const PrefillParams &p, cudaStream_t stream) {
  const int64_t units = int64_t(p.layer_count) * p.B * p.Hkv;
  auto launch = [&](auto gg) -> int {
    constexpr int G = decltype(gg)::value;
    constexpr int TOK = kRows / G;
    auto kern = prefill_attn_tc_kernel<G>;
    const size_t smem = sizeof(Smem) + 1024;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess) {
      cudaGetLastError();
      return GLIDE_ERR_CUDA;
    }
    const int64_t blocks = units * ((p.C + TOK - 1) / TOK);
    kern<<<unsigned(blocks), kThreads, smem, stream>>>(p);
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
