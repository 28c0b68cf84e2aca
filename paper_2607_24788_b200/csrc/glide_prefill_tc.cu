// GLIDE prefill outputs on the 5th-generation tensor cores (tcgen05 + TMEM + TMA), bf16 I/O, head_dim 128.
//
// One CTA (10 warps) owns 256 query rows of one (layer, sequence, KV head) unit: two row tiles X = A, B of 128
// rows each, a row being (token, query head of the group), row = token * G + head.
//   warps 0-3   softmax of tile A: thread r owns row r = TMEM lane r
//   warps 4-7   softmax of tile B
//   warp 8      one elected thread issues every tcgen05.mma
//   warp 9      one elected thread issues the TMA loads of the K and V tiles
// Window part, per 128-key tile t (keys are tokens j0 + 0..127, j0 a multiple of 16):
//   loader    K_t and V_t as 16-token boxes (ring rows for tokens older than the call, the call's rows otherwise)
//             into a ring of five 32 KiB buffers (kStages), 128-byte swizzle, completion on an mbarrier
//   MMA       S_X = Q_X K_t^T into TMEM (8 x m128n128k16), committed to an mbarrier the softmax warps wait on
//   softmax   tcgen05.ld of the own row, mask, row maximum without any shuffle, P = 2^(s - m_ref) as bf16 into
//             the swizzled A-operand layout in shared memory; the reference m_ref is lazy: O is rescaled in
//             TMEM only when the maximum grows by more than 2^8
//   MMA       O_X += P_X V_t (V as the MN-major B operand), then S_X of the next tile: while one row tile is
//             in its softmax the tensor core works for the other
// TMEM columns: S_A [0,128) S_B [128,256) O_A [256,384) O_B [384,512).
// Linear part (after the window tiles, the whole CTA in step): with a common reference M = max(m_ref, -64) per
// row, phi(Q) 2^-M as bf16 times a bf16 copy of the state (inter-chunk), and C = phi(Q) phi(K')^T masked to
// j' <= i, then C V' (intra-chunk), through the same MMAs; l accumulates the matching sums.  out = O / l.
// Every mbarrier wait is bounded; on a time-out the CTA records kDevWaitTimeout, leaves its loops, frees its TMEM
// columns and returns.
#include <cuda.h>
#include <cstring>

#include <algorithm>

#include "glide_device.cuh"

namespace glide {

namespace {

constexpr int kD = 128;
constexpr int kRows = 128;            // rows per row tile
constexpr int kKT = 128;              // keys per tile
constexpr int kGroup = 16;            // tokens per TMA box
constexpr int kSoftmaxThreads = 256;
constexpr int kThreads = 320;
constexpr int kMmaWarp = 8, kLoadWarp = 9;
constexpr uint32_t kTileBytes = 32768;   // [2 boxes][128 rows][64 bf16]
constexpr uint32_t kBoxBytes = 16384;
constexpr uint32_t kGroupBytes = kGroup * 128;   // one 16-token box of 64 columns
constexpr uint32_t kWaitLimit = 1u << 20;
constexpr float kLazy = 8.0f;         // rescale O only when the row maximum grows by more than 2^8
constexpr int kStages = 5;

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
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
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
// 8 MMAs of one 128 x 128 x 128 product; B K-major (D = A B^T) or MN-major (D (+)= A B)
__device__ __forceinline__ void issue_mma(uint32_t tmem_d, uint32_t a_tile, uint32_t b_tile, bool b_mn, bool accumulate) {
  const uint32_t idesc = make_idesc(b_mn);
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    const uint64_t adesc = make_desc(a_tile + (ks >> 2) * kBoxBytes + (ks & 3) * 32, 16, 1024);
    const uint64_t bdesc = b_mn ? make_desc(b_tile + ks * 2048, kBoxBytes, 1024)
                                : make_desc(b_tile + (ks >> 2) * kBoxBytes + (ks & 3) * 32, 16, 1024);
    mma_f16(tmem_d, adesc, bdesc, idesc, (accumulate || ks > 0) ? 1u : 0u);
  }
}
// the same product with the A operand in TMEM: lane = row, 32-bit column c = elements 2c (low half) and 2c+1 of
// the row, 8 columns per k16 step; B MN-major in shared memory
__device__ __forceinline__ void issue_mma_ts(uint32_t tmem_d, uint32_t tmem_a, uint32_t b_tile, bool accumulate) {
  const uint32_t idesc = make_idesc(true);
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    const uint64_t bdesc = make_desc(b_tile + ks * 2048, kBoxBytes, 1024);
    const uint32_t acc = (accumulate || ks > 0) ? 1u : 0u;
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(tmem_d),
        "r"(tmem_a + ks * 8), "l"(bdesc), "r"(idesc), "r"(acc)
        : "memory");
  }
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait; gives up early when another thread of the CTA has already timed out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *failed) {
  for (uint32_t spin = 0; spin < kWaitLimit; ++spin) {
    uint32_t ok;
    asm volatile("{.reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p;}"
                 : "=r"(ok)
                 : "r"(bar), "r"(parity)
                 : "memory");
    if (ok) return true;
    if ((spin & 1023u) == 1023u && *failed) return false;
  }
  *failed = 1;
  return false;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void *tmap, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(tmap), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const void *tmap, int c0, int c1, int c2, int c3, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(dst),
      "l"(tmap), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
      : "memory");
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
// the same load without the wait: the registers are valid only after tmem_wait_ld()
__device__ __forceinline__ void tmem_ld32_nowait(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
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


// (no wait: the caller issues tmem_wait_st() once after its last store)
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]),
      "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

#ifdef GLIDE_PF_CLOCKS
// debug builds only: clock cycles per phase of thread 0 of every CTA, summed over the CTAs ([8] phases, [8] = CTAs)
__device__ unsigned long long g_pf_clk[16];
#define PF_CLK(i)                                                   \
  do {                                                              \
    if (threadIdx.x == 0) {                                         \
      const long long now_ = clock64();                             \
      atomicAdd(&g_pf_clk[i], (unsigned long long)(now_ - pf_t_));  \
      pf_t_ = now_;                                                 \
    }                                                               \
  } while (0)
#else
#define PF_CLK(i) do { } while (0)
#endif

struct Smem {
  unsigned char q[2][kTileBytes];        // Q_A, Q_B; later phi(Q) 2^-m*
  unsigned char kv[kStages][kTileBytes]; // K and V tiles in turn; linear part: bf16 state, phi(K') tile, V' tile
  float z[2 * kD];                       // z of the unit (both halves with the learned map)
  uint64_t bar_full[kStages];            // TMA bytes of the buffer have landed
  uint64_t bar_free[kStages];            // the MMAs that read the buffer have completed
  uint64_t bar_q[2];                     // Q_X staged (128 arrivals)
  uint64_t bar_s[2];                     // S_X of the current tile is in TMEM
  uint64_t bar_p[2];                     // P_X of the current tile is in TMEM (128 arrivals)
  uint64_t bar_done;                     // every window MMA has completed
  uint64_t bar_lin;                      // linear part: the MMAs issued so far have completed
  uint64_t bar_state;                    // the bf16 copy of S and z of the unit have landed
  uint64_t bar_pk[2];                    // the phi(K') tile of an intra-chunk step has landed (even / odd steps)
  uint64_t bar_vp[2];                    // the V' tile of the first / second intra-chunk step has landed (2 arrivals)
  uint32_t tmem_base;
  int failed;
};
static_assert(sizeof(Smem) + 1024 <= 232448, "shared memory of one CTA");

// the call's K (or V) rows as a 4-D tensor {d, Hkv, T, layers x sequences}: boxes of 16 tokens x 64 columns of one KV head
struct CallMaps {
  CUtensorMap k, v;         // boxes of 16 tokens
  CUtensorMap k128, v128;   // boxes of a whole 128-key tile
};

template <int G, bool SUM, bool PHI2>
__global__ void __launch_bounds__(kThreads, 1)   // 10 warps = 3 on one scheduler: 168 registers per thread at most
prefill_attn_tc_kernel(const PrefillParams p, const CUtensorMap *ring_maps, const __grid_constant__ CallMaps cm) {
  using bf16 = __nv_bfloat16;
  constexpr int TOKT = kRows / G;    // tokens per row tile
  constexpr int TOKC = 2 * TOKT;     // tokens per CTA
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  Smem &sm = *reinterpret_cast<Smem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int ctas_per_chunk = (p.C + TOKC - 1) / TOKC;
  const int64_t u = blockIdx.x / ctas_per_chunk;
  const int tok0 = int(blockIdx.x % ctas_per_chunk) * TOKC;
  const int g = int(u % p.Hkv);
  const int b = int((u / p.Hkv) % p.B);
  const int lrel = int(u / (int64_t(p.Hkv) * p.B));
  const int layer = p.layer_begin + lrel;
  const LayerDev ld = p.layers[layer];
  const int ntok = min(TOKC, p.C - tok0);
  const int ntokA = min(TOKT, ntok), ntokB = ntok - ntokA;
  const bool hasB = ntokB > 0;
  const int64_t tq0 = p.n0 + p.c0 + tok0;
  const int64_t tq_last = tq0 + ntok - 1;
  const int64_t w = ld.w;
  const int64_t wl = ld.wlin;                      // delay of the linear stream: w, or 0 when the state holds every token
  constexpr bool sum_terms = SUM;                  // sum of two normalised terms instead of the shared normaliser
  const uint32_t cap = ld.cap > 0 ? uint32_t(ld.cap) : 1u;
  const size_t unit_rows = (size_t(b + p.b0) * p.Hkv + g) * size_t(ld.cap);   // b + b0: the sequence's slot in the context
  const size_t seq = (size_t(lrel) * p.B + b) * size_t(p.T);
  volatile int *failed = &sm.failed;
#ifdef GLIDE_PF_CLOCKS
  long long pf_t_ = clock64();
  if (threadIdx.x == 0) atomicAdd(&g_pf_clk[8], 1ull);
#endif

  // a time-out recorded by an earlier CTA ends the launch quickly
  if (*reinterpret_cast<volatile int32_t *>(&p.ctl->status) == kDevWaitTimeout) return;

  const bool has_window = w > 0;
  int64_t j_lo = tq0 - w + 1;
  if (j_lo < 0) j_lo = 0;
  j_lo &= ~int64_t(kGroup - 1);   // key tiles start at a multiple of the TMA box
  const int n_tiles = has_window ? int((tq_last - j_lo) / kKT) + 1 : 0;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&sm.bar_full[s]), 2);
      mbar_init(smem_u32(&sm.bar_free[s]), 1);
    }
    for (int x = 0; x < 2; ++x) {
      mbar_init(smem_u32(&sm.bar_q[x]), kRows);
      mbar_init(smem_u32(&sm.bar_s[x]), 1);
      mbar_init(smem_u32(&sm.bar_p[x]), kRows);
    }
    mbar_init(smem_u32(&sm.bar_done), 1);
    mbar_init(smem_u32(&sm.bar_lin), 1);
    mbar_init(smem_u32(&sm.bar_state), 1);
    mbar_init(smem_u32(&sm.bar_pk[0]), 1);
    mbar_init(smem_u32(&sm.bar_pk[1]), 1);
    mbar_init(smem_u32(&sm.bar_vp[0]), 2);
    mbar_init(smem_u32(&sm.bar_vp[1]), 2);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    sm.failed = 0;
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&sm.tmem_base)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // Token groups past the CTA's last token are never loaded (only the last tile has such groups), and what a
  // masked key's V row holds is multiplied by a zero weight, so it has to be finite: those rows of the buffer that
  // will hold the last V tile start at zero (earlier tiles that pass through the buffer leave real rows behind).
  if (n_tiles > 0) {
    const int last_slot = (2 * (n_tiles - 1) + 1) % kStages;
    const int64_t j0_last = j_lo + int64_t(n_tiles - 1) * kKT;
    const int first_skipped = int((tq_last - j0_last) / kGroup) + 1;   // groups [first_skipped, 8) are not loaded
    const int n16 = (kKT / kGroup - first_skipped) * int(kGroupBytes / 16);
    for (int half = 0; half < 2; ++half) {
      uint4 *dst = reinterpret_cast<uint4 *>(&sm.kv[last_slot][half * kBoxBytes + first_skipped * kGroupBytes]);
      for (int i = tid; i < n16; i += kThreads) dst[i] = make_uint4(0u, 0u, 0u, 0u);
    }
  }
  // Q_X: 128 rows x 16 chunks by the 128 threads of each row tile, asked for before the set-up's barrier so that the copy
  // runs while the other warps finish setting up (it needs nothing of that; nothing else writes these tiles).
  {
    const int Xq = (tid >> 7) & 1, rq = tid & 127;
    const int ntokXq = Xq ? ntokB : ntokA;
    if (tid < kSoftmaxThreads && ntokXq > 0) {
      const bf16 *qbase = reinterpret_cast<const bf16 *>(p.q) + (seq + size_t(p.c0 + tok0 + Xq * TOKT)) * p.H * kD;
      const uint32_t sQx = smem_u32(sm.q[Xq]);
#pragma unroll 4
      for (int i = 0; i < kRows * 16 / kRows; ++i) {
        const int id = rq + kRows * i;
        const int r = id >> 4, c = id & 15;
        const int tk = r / G, h2 = r - tk * G;
        const bool valid = tk < ntokXq;
        cp_async16(sQx + sw128(r, c), qbase + (size_t(valid ? tk : 0) * p.H + p.heads_of[g * G + h2]) * kD + c * 8, valid);
      }
      cp_async_commit();
    }
  }
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm.tmem_base;
  PF_CLK(0);
  const uint32_t sQ[2] = {smem_u32(sm.q[0]), smem_u32(sm.q[1])};
  const uint32_t sKV0 = smem_u32(sm.kv[0]);
  auto kv_addr = [&](int slot) { return sKV0 + uint32_t(slot) * kTileBytes; };
  // Linear part: what it needs is known now, so that the loader can fetch it behind the last key tiles.
  const bool linear = ld.evicts && tq_last >= wl;
  const int64_t folded = p.n0 + p.c0 - wl;   // tokens below this index are in S, z at the start of the chunk
  const bool need_state = linear && folded > 0;
  // intra-chunk steps: delayed tokens of this chunk up to the CTA's last token, 128 at a time
  const int i_lo = folded < 0 ? int(-folded < int64_t(p.C) ? -folded : int64_t(p.C)) : 0;
  const int i_hi = tok0 + ntok - 1;
  const int it0 = i_lo & ~(kKT - 1);
  const int n_itiles = (linear && it0 <= i_hi) ? (i_hi - it0) / kKT + 1 : 0;
  // Roles of the five buffers after the window loop, by the order in which the loop stops using them (load number
  // 2 n_tiles - 5 + k; a negative number is a buffer the loop never used): the first to come free receives the bf16
  // copy of the unit's state, the next two the phi(K') tiles of the first two intra-chunk steps (all three by TMA
  // while the last key tiles are still being processed), the last two the V' tiles of those steps.  Later steps
  // take the buffers of the step before the previous one.
  auto late_seq = [&](int k) { return 2 * n_tiles - kStages + k; };
  auto late_slot = [&](int k) { const int sq = late_seq(k); return sq >= 0 ? sq % kStages : sq + kStages; };
  const int slotSb = late_slot(0);
  const int slotPk[2] = {late_slot(1), late_slot(2)}, slotVp[2] = {late_slot(3), late_slot(4)};
  const CUtensorMap *map_pk = ring_maps + 5 * p.L, *map_s16 = map_pk + 1;
  auto load_pk = [&](int t) {   // one thread: the phi(K') rows of intra-chunk step t
    const uint32_t bar = smem_u32(&sm.bar_pk[t & 1]);
    const uint32_t dst = kv_addr(slotPk[t & 1]);
    const int y = int(u * p.Cmax) + it0 + t * kKT;
    mbar_expect_tx(bar, kTileBytes);
    tma_load_2d(dst, map_pk, 0, y, bar);
    tma_load_2d(dst + kBoxBytes, map_pk, 64, y, bar);
  };

  // ---- softmax threads: per-row state that lives across the window and the linear part ----------------------
  const int X = (tid >> 7) & 1;                   // row tile of this thread (softmax warps only)
  const int row = tid & 127;
  const int tok_r = row / G, hh = row - tok_r * G;
  const int ntokX = X ? ntokB : ntokA;
  const bool activeX = tid < kSoftmaxThreads && ntokX > 0;
  const int tl = tok0 + X * TOKT + tok_r;         // chunk-relative token of this row
  const int64_t tok_abs = p.n0 + p.c0 + tl;
  const uint32_t tS = tmem + (uint32_t((warp & 3) * 32) << 16) + uint32_t(X) * 128u;
  const uint32_t tO = tS + 256u;
  float m_ref = -CUDART_INF_F, l_sum = 0.f;

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
  // weights of one S row against reference mr (log2 domain) -> bf16 P row in the swizzled A layout; returns their sum
  auto write_p = [&](auto masked, int lo, int hi, float mr, float scale) -> float {
    constexpr bool kMasked = decltype(masked)::value;
    float sum0 = 0.f, sum1 = 0.f;
    uint32_t ra[32], rb[32];
    tmem_ld32_nowait(tS, ra);
#pragma unroll
    for (int c0 = 0; c0 < kKT; c0 += 32) {
      uint32_t (&r)[32] = ((c0 >> 5) & 1) ? rb : ra;
      uint32_t pk[16];
      tmem_wait_ld();
      // the next 32 columns are on their way while these are turned into weights; the store below touches
      // columns [c0/2, c0/2+16), which lie below c0+32 only when they have been read already
      if (c0 + 32 < kKT) tmem_ld32_nowait(tS + c0 + 32, ((c0 >> 5) & 1) ? ra : rb);
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        const int i = e * 2;
        float a0 = ex2(fmaf(__uint_as_float(r[i]), scale, -mr));
        float a1 = ex2(fmaf(__uint_as_float(r[i + 1]), scale, -mr));
        if (kMasked) {
          if (c0 + i < lo || c0 + i > hi) a0 = 0.f;
          if (c0 + i + 1 < lo || c0 + i + 1 > hi) a1 = 0.f;
        }
        pk[e] = pack_bf16x2(a0, a1);
        sum0 += __uint_as_float(pk[e] << 16);          // the sum uses the weights as the tensor core sees them
        sum1 += __uint_as_float(pk[e] & 0xffff0000u);
      }
      // P overwrites the S columns this thread has already consumed: keys c0..c0+31 -> columns c0/2..c0/2+15
      tmem_st16(tS + (c0 >> 1), pk);
    }
    tmem_wait_st();
    return sum0 + sum1;
  };
  // =========================== window part: warp-specialised ===========================
  if (tid < kSoftmaxThreads) {
    if (activeX) {
      cp_async_wait_all();   // Q_X (asked for before the set-up's barrier) has landed
      fence_async_smem();
      mbar_arrive(smem_u32(&sm.bar_q[X]));

      const int64_t tqX0 = tq0 + X * TOKT, tqX_last = tqX0 + ntokX - 1;
      bool o_written = false;   // a P V product has been accumulated into O_X (uniform over the row tile)
      for (int t = 0; t < n_tiles; ++t) {
        const bool got = mbar_wait(smem_u32(&sm.bar_s[X]), uint32_t(t) & 1u, failed);
        if (!__all_sync(0xffffffffu, got)) break;   // warp-uniform: the collectives below need every lane
        tc_fence_after();
        const int64_t j0 = j_lo + int64_t(t) * kKT;
        const bool interior = j0 + kKT - 1 <= tqX0 && j0 > tqX_last - w;
        // valid columns of this row: lo <= c <= hi
        int64_t lo64 = tok_abs - w + 1 - j0, hi64 = tok_abs - j0;
        const int lo = int(lo64 < 0 ? 0 : (lo64 > kKT ? kKT : lo64));
        const int hi = int(hi64 < -1 ? -1 : (hi64 > kKT - 1 ? kKT - 1 : hi64));
        // pass 1: row maximum of the valid raw scores (the scale is positive: it is applied to the maximum)
        float mx = -CUDART_INF_F;
#pragma unroll 1
        for (int c0 = 0; c0 < kKT; c0 += 32) {
          uint32_t r[32];
          tmem_ld32(tS + c0, r);
          float m4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
          if (interior) {
#pragma unroll
            for (int i = 0; i < 32; ++i) m4[i & 3] = fmaxf(m4[i & 3], __uint_as_float(r[i]));
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (c0 + i >= lo && c0 + i <= hi) m4[i & 3] = fmaxf(m4[i & 3], __uint_as_float(r[i]));
          }
          mx = fmaxf(mx, fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])));
        }
        mx *= p.scale_log2;
        // lazy reference: move it (and rescale O, l) only when the maximum grows by more than 2^kLazy
        float f = 1.f;
        if (mx > m_ref + kLazy || (m_ref == -CUDART_INF_F && mx > -CUDART_INF_F)) {
          f = m_ref == -CUDART_INF_F ? 0.f : ex2(m_ref - mx);
          m_ref = mx;
        }
        if (o_written && __any_sync(0xffffffffu, f != 1.f)) scale_o(f);
        l_sum *= f;
        const float mr = m_ref == -CUDART_INF_F ? 0.f : m_ref;
        if (interior) l_sum += write_p(IntTag<0>{}, lo, hi, mr, p.scale_log2);
        else l_sum += write_p(IntTag<1>{}, lo, hi, mr, p.scale_log2);
        tc_fence_before();      // this thread's TMEM accesses precede the MMAs that read P and overwrite S
        mbar_arrive(smem_u32(&sm.bar_p[X]));
        o_written = true;
      }
    }
    if (n_tiles > 0) mbar_wait(smem_u32(&sm.bar_done), 0u, failed);
    tc_fence_after();
  } else if (warp == kMmaWarp) {
    if (lane == 0 && n_tiles > 0) {
      bool ok = mbar_wait(smem_u32(&sm.bar_q[0]), 0u, failed);
      if (ok && hasB) ok = mbar_wait(smem_u32(&sm.bar_q[1]), 0u, failed);
      if (ok) ok = mbar_wait(smem_u32(&sm.bar_full[0]), 0u, failed);   // K_0
      if (ok) {
        tc_fence_after();
        issue_mma(tmem, sQ[0], kv_addr(0), false, false);
        mma_commit(smem_u32(&sm.bar_s[0]));
        if (hasB) {
          issue_mma(tmem + 128, sQ[1], kv_addr(0), false, false);
          mma_commit(smem_u32(&sm.bar_s[1]));
        }
        mma_commit(smem_u32(&sm.bar_free[0]));
      }
      for (int t = 0; t < n_tiles && ok; ++t) {
        const int seqV = 2 * t + 1, seqK = 2 * t + 2;
        const bool more = t + 1 < n_tiles;
        ok = mbar_wait(smem_u32(&sm.bar_full[seqV % kStages]), uint32_t(seqV / kStages) & 1u, failed);
        if (ok && more) ok = mbar_wait(smem_u32(&sm.bar_full[seqK % kStages]), uint32_t(seqK / kStages) & 1u, failed);
        for (int x = 0; x < 2 && ok; ++x) {
          if (x == 1 && !hasB) break;
          ok = mbar_wait(smem_u32(&sm.bar_p[x]), uint32_t(t) & 1u, failed);
          if (!ok) break;
          tc_fence_after();
          issue_mma_ts(tmem + 256 + x * 128, tmem + x * 128, kv_addr(seqV % kStages), t > 0);
          if (more) {
            issue_mma(tmem + x * 128, sQ[x], kv_addr(seqK % kStages), false, false);
            mma_commit(smem_u32(&sm.bar_s[x]));
          }
        }
        if (ok) {
          mma_commit(smem_u32(&sm.bar_free[seqV % kStages]));
          if (more) mma_commit(smem_u32(&sm.bar_free[seqK % kStages]));
        }
      }
      if (ok) mma_commit(smem_u32(&sm.bar_done));
    }
  } else if (warp == kLoadWarp) {
    // A 128-key tile is eight groups of 16 tokens.  A group that lies in one source (ring or call) and is contiguous
    // there is fetched by TMA, lane gi issuing the two boxes (column halves) of group gi so that the address
    // arithmetic of the groups runs in parallel.  A group that straddles the call boundary or a ring wrap is copied
    // row by row by the whole warp (at most a few per tile).  Each buffer's barrier takes two arrivals: the
    // expect-tx one before the TMA boxes are issued and a plain one after the row copies.
    const CUtensorMap *ringK = ring_maps + 3 * layer, *ringV = ringK + 1;
    const CUtensorMap *ringK128 = ring_maps + 3 * p.L + 2 * layer, *ringV128 = ringK128 + 1;
    const bf16 *ringKp = reinterpret_cast<const bf16 *>(p.ws + ld.ringK) + unit_rows * kD;
    const bf16 *ringVp = reinterpret_cast<const bf16 *>(p.ws + ld.ringV) + unit_rows * kD;
    const bf16 *callKp = reinterpret_cast<const bf16 *>(p.k) + (seq * p.Hkv + g) * kD;
    const bf16 *callVp = reinterpret_cast<const bf16 *>(p.v) + (seq * p.Hkv + g) * kD;
    const int64_t call_stride = int64_t(p.Hkv) * kD;
    const int gi = lane;
    // Rows of tokens j0 .. j0 + 127 (K or V) into buffer `slot` (the whole warp); rows of tokens below 0 are zero;
    // 16-row groups that lie wholly above j_max are zero too (zero_rest) or not written at all.  j0 need
    // not be a multiple of the box size: a ring row or a token of the call is a TMA coordinate like any other.
    auto load_tile = [&](int64_t j0, bool is_v, int slot, uint32_t bar, int64_t j_max, bool zero_rest) {
      const int64_t left = j_max - j0;                         // >= 0: the tile holds at least one valid token
      const int ngroups = left >= kKT - 1 ? kKT / kGroup : int(left / kGroup) + 1;
      // A full tile that lies in one source without a wrap takes two boxes of 128 rows (the layout in shared memory
      // is that of eight 16-row boxes).  Tiles that reach past the last token keep the 16-row path, which never
      // loads a later token's row.
      if (j0 >= 0) {
        const uint32_t slot_row0 = (j0 >> 32) == 0 ? uint32_t(j0) % cap : uint32_t(uint64_t(j0) % cap);
        const bool all_call = j0 >= p.n0;
        const bool all_ring = j0 + kKT <= p.n0 && slot_row0 + kKT <= cap;
        // (left >= kKT - 1: every row of the tile is a token up to the last one; eight groups alone would also
        // admit a last group that is only partly valid)
        if (left >= kKT - 1 && (all_call || all_ring)) {
          if (lane == 0) {
            mbar_expect_tx(bar, kTileBytes);
            const uint32_t dst = kv_addr(slot);
            if (all_call) {
              const CUtensorMap *m = is_v ? &cm.v128 : &cm.k128;
              tma_load_4d(dst, m, 0, g, int(j0 - p.n0), lrel * p.B + b, bar);
              tma_load_4d(dst + kBoxBytes, m, 64, g, int(j0 - p.n0), lrel * p.B + b, bar);
            } else {
              const CUtensorMap *m = is_v ? ringV128 : ringK128;
              const int y = int(unit_rows + slot_row0);
              tma_load_2d(dst, m, 0, y, bar);
              tma_load_2d(dst + kBoxBytes, m, 64, y, bar);
            }
            mbar_arrive(bar);   // the barrier's second arrival (after the row copies on the other path)
          }
          return;
        }
      }
      // this lane's group: where it comes from and whether one box covers it
      const int64_t j = j0 + gi * kGroup;
      const bool mine = gi < kKT / kGroup && (zero_rest || gi < ngroups);
      const bool from_call = j >= p.n0;
      const uint32_t slot_row = j < 0 ? 0u : ((j >> 32) == 0 ? uint32_t(j) % cap : uint32_t(uint64_t(j) % cap));
      const bool boxed = mine && gi < ngroups && j >= 0 && (from_call || (j + kGroup <= p.n0 && slot_row + kGroup <= cap));
      const unsigned boxed_mask = __ballot_sync(0xffffffffu, boxed);
      const unsigned manual_mask = __ballot_sync(0xffffffffu, mine && !boxed);
      if (lane == 0) mbar_expect_tx(bar, uint32_t(__popc(boxed_mask)) * 2u * kGroupBytes);
      __syncwarp();
      if (boxed) {
        const uint32_t dst = kv_addr(slot) + uint32_t(gi) * kGroupBytes;
        if (from_call) {
          const CUtensorMap *m = is_v ? &cm.v : &cm.k;
          tma_load_4d(dst, m, 0, g, int(j - p.n0), lrel * p.B + b, bar);
          tma_load_4d(dst + kBoxBytes, m, 64, g, int(j - p.n0), lrel * p.B + b, bar);
        } else {
          const CUtensorMap *m = is_v ? ringV : ringK;
          const int y = int(unit_rows + slot_row);
          tma_load_2d(dst, m, 0, y, bar);
          tma_load_2d(dst + kBoxBytes, m, 64, y, bar);
        }
      }
      for (unsigned mm = manual_mask; mm; mm &= mm - 1) {
        const int gm = __ffs(int(mm)) - 1;
        unsigned char *tile = sm.kv[slot];
#pragma unroll
        for (int i = 0; i < kGroup * 16 / 32; ++i) {
          const int id = lane + 32 * i;
          const int r = id >> 4, c = id & 15;
          const int64_t jj = j0 + gm * kGroup + r;
          uint4 val = make_uint4(0u, 0u, 0u, 0u);
          if (jj >= 0 && jj <= j_max) {
            const bf16 *src = jj >= p.n0 ? (is_v ? callVp : callKp) + size_t(jj - p.n0) * call_stride
                                         : (is_v ? ringVp : ringKp) + size_t(uint64_t(jj) % cap) * kD;
            val = *reinterpret_cast<const uint4 *>(src + c * 8);
          }
          *reinterpret_cast<uint4 *>(tile + sw128(gm * kGroup + r, c)) = val;
        }
      }
      fence_async_smem();   // the row copies are read by the tensor core (async proxy)
      __syncwarp();
      if (lane == 0) mbar_arrive(bar);
    };
    bool ok = true;
    for (int sq = 0; sq < 2 * n_tiles; ++sq) {
      const int t = sq >> 1, slot = sq % kStages;
      if (sq >= kStages) ok = mbar_wait(smem_u32(&sm.bar_free[slot]), uint32_t(sq / kStages - 1) & 1u, failed);
      if (!__all_sync(0xffffffffu, ok)) break;
      load_tile(j_lo + int64_t(t) * kKT, sq & 1, slot, smem_u32(&sm.bar_full[slot]), tq_last, false);
    }
    if (!PHI2 && lane == 0 && linear && !*failed) {
      // the linear part's operands into the buffers the window loop leaves first: the bf16 state (with z), then the
      // phi(K') tiles of the first two intra-chunk steps
      const int n_late = 1 + (n_itiles < 2 ? n_itiles : 2);
      for (int k = 0; k < n_late; ++k) {
        const int sq = late_seq(k);
        if (sq >= 0 && !mbar_wait(smem_u32(&sm.bar_free[sq % kStages]), uint32_t(sq / kStages) & 1u, failed)) break;
        if (k == 0) {
          if (!need_state) continue;
          const int ub = (b + p.b0) * p.Hkv + g;
          const uint32_t bar = smem_u32(&sm.bar_state);
          mbar_expect_tx(bar, kTileBytes + uint32_t(kD * sizeof(float)));
          tma_load_2d(kv_addr(slotSb), map_s16, 0, int(u * kD), bar);
          tma_load_2d(kv_addr(slotSb) + kBoxBytes, map_s16, 64, int(u * kD), bar);
          bulk_load(smem_u32(sm.z), p.ws + ld.z + size_t(ub) * kD * sizeof(float), uint32_t(kD * sizeof(float)), bar);
        } else {
          load_pk(k - 1);
        }
      }
    }
    __syncwarp();
    // the V rows of the delayed tokens of the first two intra-chunk steps, behind the window loop's last tiles (the
    // rows of tokens that do not exist yet, below 0, are zero: their weights are, and 0 x anything must stay 0)
    for (int t = 0; !PHI2 && t < n_itiles && t < 2 && __all_sync(0xffffffffu, ok && !*failed); ++t) {
      const int sq = late_seq(3 + t);
      if (sq >= 0) ok = mbar_wait(smem_u32(&sm.bar_free[sq % kStages]), uint32_t(sq / kStages) & 1u, failed);
      if (!__all_sync(0xffffffffu, ok)) break;
      load_tile(folded + it0 + int64_t(t) * kKT, true, slotVp[t], smem_u32(&sm.bar_vp[t]), tq_last, true);
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();

  PF_CLK(1);
  // =========================== linear part: the whole CTA in step ===========================
  // (no early exits from here on: every thread passes the same __syncthreads; after a time-out the waits return
  // at once and the results are discarded)
  // Operands: phi(Q) 2^-M from the softmax threads; the bf16 state and the phi(K') tiles by TMA (issued by the loader
  // behind the window loop, see above); the delayed tokens' V rows row by row (they come from the ring or from the
  // call, with a wrap or the call boundary anywhere) by the loader as well, with the key tiles' own routine.
  bool o_init = n_tiles > 0;   // O_X holds a valid accumulation (uniform over the CTA)
  uint32_t lin_phase = 0;
  const int mma_tid = kMmaWarp * 32;
  auto wait_lin = [&]() {
    mbar_wait(smem_u32(&sm.bar_lin), lin_phase & 1u, failed);
    ++lin_phase;
    tc_fence_after();
  };
  // C row of this thread -> bf16 over the same TMEM columns, masked to the delayed tokens j' <= i of the row (the
  // values already carry 2^-m*); the row's weight sum goes to l
  auto convert_c = [&](int i0) {
    if (activeX) {
      // C row -> bf16, masked to delayed tokens j' <= i of this row (the values already carry 2^-m*)
      float sum0 = 0.f, sum1 = 0.f;
      const int lo = i_lo - i0, hi = tl - i0;
      // a tile that lies wholly before the row tile's first token (and after the first delayed token) needs no mask
      const bool whole = i0 + kKT - 1 <= tok0 + X * TOKT && i0 >= i_lo;
      uint32_t ra[32], rb[32];
      tmem_ld32_nowait(tS, ra);
#pragma unroll
      for (int c0 = 0; c0 < kKT; c0 += 32) {
        uint32_t (&r)[32] = ((c0 >> 5) & 1) ? rb : ra;
        uint32_t pk[16];
        tmem_wait_ld();
        if (c0 + 32 < kKT) tmem_ld32_nowait(tS + c0 + 32, ((c0 >> 5) & 1) ? ra : rb);
        if (whole) {
#pragma unroll
          for (int e = 0; e < 16; ++e) pk[e] = pack_bf16x2(__uint_as_float(r[e * 2]), __uint_as_float(r[e * 2 + 1]));
        } else {
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const int i = c0 + e * 2;
            const float a0 = (i >= lo && i <= hi) ? __uint_as_float(r[e * 2]) : 0.f;
            const float a1 = (i + 1 >= lo && i + 1 <= hi) ? __uint_as_float(r[e * 2 + 1]) : 0.f;
            pk[e] = pack_bf16x2(a0, a1);
          }
        }
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          sum0 += __uint_as_float(pk[e] << 16);
          sum1 += __uint_as_float(pk[e] & 0xffff0000u);
        }
        tmem_st16(tS + (c0 >> 1), pk);
      }
      tmem_wait_st();
      if (!sum_terms) l_sum += sum0 + sum1;
    }
    PF_CLK(4);
  };
  if (linear && !PHI2) {
    const bf16 *ringV = reinterpret_cast<const bf16 *>(p.ws + ld.ringV) + unit_rows * kD;
    const bf16 *callV = reinterpret_cast<const bf16 *>(p.v) + (seq * p.Hkv + g) * kD;
    const int64_t call_stride = int64_t(p.Hkv) * kD;
    auto load_vp = [&](int t) {   // softmax threads, steps after the second: V rows of the delayed tokens (MN-major), zero where none
      const int i0 = it0 + t * kKT;
      const uint32_t dst = kv_addr(slotVp[t & 1]);
#pragma unroll 4
      for (int i = 0; i < kKT * 16 / kSoftmaxThreads; ++i) {
        const int id = tid + kSoftmaxThreads * i;
        const int r = id >> 4, c = id & 15;
        const int ii = i0 + r;
        const bool valid = ii >= i_lo && ii <= i_hi;
        const int64_t jj = valid ? folded + ii : 0;
        const bool from_call = jj >= p.n0;
        const uint32_t slot_row = (jj >> 32) == 0 ? uint32_t(jj) % cap : uint32_t(uint64_t(jj) % cap);
        const bf16 *src = from_call ? callV + size_t(jj - p.n0) * call_stride : ringV + size_t(slot_row) * kD;
        cp_async16(dst + sw128(r, c), src + c * 8, valid);
      }
      cp_async_commit();
    };
    uint32_t phq[kD / 2];                      // phi(q) 2^-m* of this row, packed bf16
    if (activeX) {
      // Any common reference M >= m_ref gives the same quotient O / l.  M = max(m_ref, 0) would rescale O for every
      // row whose window maximum is negative; a floor of -64 keeps 2^-M and everything scaled by it far inside the
      // fp32 / bf16 range (phi <= 1) and makes that rescale a rarity.
      // A row without evicted tokens (position below the window size) keeps its own reference and gets phi(q) = 0:
      // a floor there would only push its window weights towards underflow.
      // Sum of two normalised terms instead: the window part is normalised now (O / l), and phi(q) is divided by the
      // row's linear normaliser phi(q) . (z + running sum of phi(K') up to the row's own delayed token), so that what
      // the linear products add to O is the normalised linear term; the final division is by 1.
      const bool has_lin = tok_abs >= wl;
      const float M = has_lin ? fmaxf(m_ref, -64.f) : m_ref;
      float fw = m_ref == -CUDART_INF_F ? 0.f : ex2(m_ref - M);
      const float fl = has_lin ? ex2(-M) : 0.f;
      if (sum_terms) fw = l_sum > 0.f ? 1.0f / l_sum : 0.f;
      if (o_init && __any_sync(0xffffffffu, fw != 1.f)) scale_o(fw);
      l_sum = sum_terms ? 1.f : l_sum * fw;
      if (sum_terms && need_state) mbar_wait(smem_u32(&sm.bar_state), 0u, failed);   // z is needed for the normaliser
      // this row of Q is still in the shared tile (every S product has completed)
#pragma unroll
      for (int i = 0; i < kD / 8; ++i) {
        const uint4 v4 = *reinterpret_cast<const uint4 *>(sm.q[X] + sw128(row, i));
        phq[i * 4 + 0] = v4.x;
        phq[i * 4 + 1] = v4.y;
        phq[i * 4 + 2] = v4.z;
        phq[i * 4 + 3] = v4.w;
      }
      float mx = -CUDART_INF_F;
#pragma unroll
      for (int i = 0; i < kD / 2; ++i)
        mx = fmaxf(mx, fmaxf(__uint_as_float(phq[i] << 16), __uint_as_float(phq[i] & 0xffff0000u)));
      // one pass of exponentials: kept as packed bf16, normalised by the sum of the unrounded values afterwards
      float sum0 = 0.f, sum1 = 0.f, dz0 = 0.f, dz1 = 0.f;
      const float mxl = mx * kLog2e;
      const float4 *zrow = reinterpret_cast<const float4 *>(p.zcum + (size_t(u) * p.Cmax + size_t(tok_r < ntokX ? tl : tok0)) * kD);
#pragma unroll
      for (int i4 = 0; i4 < kD / 4; ++i4) {
        float zz[4] = {0.f, 0.f, 0.f, 0.f};
        if (sum_terms) {
          const float4 zc = __ldg(zrow + i4);
          zz[0] = zc.x, zz[1] = zc.y, zz[2] = zc.z, zz[3] = zc.w;
          if (need_state) {
#pragma unroll
            for (int e = 0; e < 4; ++e) zz[e] += sm.z[i4 * 4 + e];
          }
        }
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          const int i = i4 * 2 + hf;
          const float e0 = ex2(fmaf(__uint_as_float(phq[i] << 16), kLog2e, -mxl));
          const float e1 = ex2(fmaf(__uint_as_float(phq[i] & 0xffff0000u), kLog2e, -mxl));
          sum0 += e0;
          sum1 += e1;
          dz0 = fmaf(e0, zz[hf * 2], dz0);
          dz1 = fmaf(e1, zz[hf * 2 + 1], dz1);
          phq[i] = pack_bf16x2(e0, e1);
        }
      }
      // shared normaliser: phi(q) 2^-M;  sum of terms: phi(q) / (phi(q) . z_row) = e / (e . z_row)
      const float dz = dz0 + dz1;
      const float sc = sum_terms ? ((has_lin && dz > 0.f) ? 1.0f / dz : 0.f) : fl * __frcp_rn(sum0 + sum1);
#pragma unroll
      for (int i = 0; i < kD / 2; ++i)
        phq[i] = pack_bf16x2(__uint_as_float(phq[i] << 16) * sc, __uint_as_float(phq[i] & 0xffff0000u) * sc);
#pragma unroll
      for (int c = 0; c < 16; ++c)
        *reinterpret_cast<uint4 *>(sm.q[X] + sw128(row, c)) = make_uint4(phq[c * 4], phq[c * 4 + 1], phq[c * 4 + 2], phq[c * 4 + 3]);
    }
    PF_CLK(10);
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    PF_CLK(2);
    // inter-chunk product into O and the first intra-chunk C in one batch
    if (tid == mma_tid) {
      tc_fence_after();
      if (need_state) {
        mbar_wait(smem_u32(&sm.bar_state), 0u, failed);
        issue_mma(tmem + 256, sQ[0], kv_addr(slotSb), true, o_init);
        if (hasB) issue_mma(tmem + 384, sQ[1], kv_addr(slotSb), true, o_init);
      }
      if (n_itiles > 0) {
        mbar_wait(smem_u32(&sm.bar_pk[0]), 0u, failed);
        issue_mma(tmem, sQ[0], kv_addr(slotPk[0]), false, false);   // C_X = (phi(Q_X) 2^-m*) phi(K')^T
        if (hasB) issue_mma(tmem + 128, sQ[1], kv_addr(slotPk[0]), false, false);
      }
      if (need_state || n_itiles > 0) mma_commit(smem_u32(&sm.bar_lin));
    }
    if (need_state && activeX) {
      mbar_wait(smem_u32(&sm.bar_state), 0u, failed);   // z has landed
      float dot = 0.f;
#pragma unroll
      for (int i = 0; i < kD / 2; ++i)
        dot += __uint_as_float(phq[i] << 16) * sm.z[2 * i] + __uint_as_float(phq[i] & 0xffff0000u) * sm.z[2 * i + 1];
      if (!sum_terms) l_sum += dot;
    }
    if (need_state || n_itiles > 0) wait_lin();
    if (need_state) o_init = true;
    PF_CLK(3);
    for (int t = 0; t < n_itiles; ++t) {
      const int i0 = it0 + t * kKT;
      convert_c(i0);
      if (t >= 2 && tid < kSoftmaxThreads) cp_async_wait_all();   // (steps after the second: rows copied by these threads)
      fence_async_smem();
      tc_fence_before();
      __syncthreads();
      if (tid == mma_tid) {
        if (t < 2) mbar_wait(smem_u32(&sm.bar_vp[t]), 0u, failed);   // the loader's V' tile
        tc_fence_after();
        issue_mma_ts(tmem + 256, tmem, kv_addr(slotVp[t & 1]), o_init);
        if (hasB) issue_mma_ts(tmem + 384, tmem + 128, kv_addr(slotVp[t & 1]), o_init);
        if (t + 1 < n_itiles) {   // the next step's C follows in the same batch (the tensor pipe keeps the order)
          mbar_wait(smem_u32(&sm.bar_pk[(t + 1) & 1]), uint32_t((t + 1) >> 1) & 1u, failed);
          issue_mma(tmem, sQ[0], kv_addr(slotPk[(t + 1) & 1]), false, false);
          if (hasB) issue_mma(tmem + 128, sQ[1], kv_addr(slotPk[(t + 1) & 1]), false, false);
        }
        mma_commit(smem_u32(&sm.bar_lin));
      }
      wait_lin();
      PF_CLK(5);
      o_init = true;
      if (t + 2 < n_itiles) {   // this step's buffers are free again: the operands of the step after the next
        if (tid == mma_tid) load_pk(t + 2);
        if (tid < kSoftmaxThreads) load_vp(t + 2);
      }
    }
  }

  // Learned feature map (shared normaliser): phi(q) = [softmax(W^T q); softmax(-W^T q)] has 2 d entries, and
  // phi(q)^T S, phi(q)^T z and phi(Q) phi(K')^T are sums over its two halves; every half is a linear part of the
  // kind above with its own 128-column tensors.  phi(Q) comes from a kernel in front of this one (the projections
  // differ per head, and a row tile mixes the heads of the group), as bf16 rows that this thread only scales by
  // 2^-M.  Everything arrives by TMA after the window loop (the Q tiles and all five K/V buffers are free then):
  // phi+ of the two row tiles in the Q tiles, phi- in buffers 0 and 1, the state halves and then the phi(K') halves of
  // each intra-chunk step in buffers 2 and 3, the step's V' rows in buffer 4.
  if (linear && PHI2) {
    const bf16 *ringV = reinterpret_cast<const bf16 *>(p.ws + ld.ringV) + unit_rows * kD;
    const bf16 *callV = reinterpret_cast<const bf16 *>(p.v) + (seq * p.Hkv + g) * kD;
    const int64_t call_stride = int64_t(p.Hkv) * kD;
    auto load_vp = [&](int t) {   // softmax threads: V rows of the delayed tokens of step t (MN-major), zero where none
      const int i0 = it0 + t * kKT;
      const uint32_t dst = kv_addr(4);
#pragma unroll 4
      for (int i = 0; i < kKT * 16 / kSoftmaxThreads; ++i) {
        const int id = tid + kSoftmaxThreads * i;
        const int r = id >> 4, c = id & 15;
        const int ii = i0 + r;
        const bool valid = ii >= i_lo && ii <= i_hi;
        const int64_t jj = valid ? folded + ii : 0;
        const bool from_call = jj >= p.n0;
        const uint32_t slot_row = (jj >> 32) == 0 ? uint32_t(jj) % cap : uint32_t(uint64_t(jj) % cap);
        const bf16 *src = from_call ? callV + size_t(jj - p.n0) * call_stride : ringV + size_t(slot_row) * kD;
        cp_async16(dst + sw128(r, c), src + c * 8, valid);
      }
      cp_async_commit();
    };
    const CUtensorMap *map_pq = map_pk + 2;
    const int rows_q = int(p.units_cap) * p.Cmax * G, rows_s = int(p.units_cap) * kD, rows_k = int(p.units_cap) * p.Cmax;
    auto tma_tile = [&](uint32_t dst, const CUtensorMap *m, int y, uint32_t bar) {
      tma_load_2d(dst, m, 0, y, bar);
      tma_load_2d(dst + kBoxBytes, m, 64, y, bar);
    };
    if (tid == mma_tid) {
      const uint32_t bar = smem_u32(&sm.bar_state);
      mbar_expect_tx(bar, (hasB ? 4u : 2u) * kTileBytes + (need_state ? 2u * kTileBytes + uint32_t(2 * kD * sizeof(float)) : 0u));
      for (int hf = 0; hf < 2; ++hf)
        for (int x = 0; x < 2; ++x) {
          if (x == 1 && !hasB) break;
          tma_tile(hf == 0 ? sQ[x] : kv_addr(x), map_pq, hf * rows_q + (int(u) * p.Cmax + tok0 + x * TOKT) * G, bar);
        }
      if (need_state) {
        const int ub = (b + p.b0) * p.Hkv + g;
        tma_tile(kv_addr(2), map_s16, int(u) * kD, bar);
        tma_tile(kv_addr(3), map_s16, rows_s + int(u) * kD, bar);
        bulk_load(smem_u32(sm.z), p.ws + ld.z + size_t(ub) * 2 * kD * sizeof(float), uint32_t(2 * kD * sizeof(float)), bar);
      }
    }
    if (tid < kSoftmaxThreads && n_itiles > 0) load_vp(0);
    float dot = 0.f;
    if (activeX) {
      const bool has_lin = tok_abs >= wl;
      const float M = has_lin ? fmaxf(m_ref, -64.f) : m_ref;   // (the reference of the shared normaliser, as above)
      const float fw = m_ref == -CUDART_INF_F ? 0.f : ex2(m_ref - M);
      const float fl = has_lin ? ex2(-M) : 0.f;
      if (o_init && __any_sync(0xffffffffu, fw != 1.f)) scale_o(fw);
      l_sum *= fw;
      mbar_wait(smem_u32(&sm.bar_state), 0u, failed);
      // this thread's row of phi+ and of phi-: times 2^-M, back as bf16; the dot with z uses the rounded values
#pragma unroll 1
      for (int hf = 0; hf < 2; ++hf) {
        unsigned char *tile = hf == 0 ? sm.q[X] : sm.kv[X];
#pragma unroll
        for (int c = 0; c < 16; ++c) {
          uint4 v4 = *reinterpret_cast<const uint4 *>(tile + sw128(row, c));
          uint32_t w4[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            w4[e] = pack_bf16x2(__uint_as_float(w4[e] << 16) * fl, __uint_as_float(w4[e] & 0xffff0000u) * fl);
            if (need_state)
              dot += __uint_as_float(w4[e] << 16) * sm.z[hf * kD + c * 8 + e * 2] +
                     __uint_as_float(w4[e] & 0xffff0000u) * sm.z[hf * kD + c * 8 + e * 2 + 1];
          }
          *reinterpret_cast<uint4 *>(tile + sw128(row, c)) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
        }
      }
    }
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    if (need_state) {
      if (tid == mma_tid) {
        tc_fence_after();
        mbar_wait(smem_u32(&sm.bar_state), 0u, failed);
        for (int x = 0; x < 2; ++x) {
          if (x == 1 && !hasB) break;
          issue_mma(tmem + 256 + x * 128, sQ[x], kv_addr(2), true, o_init);
          issue_mma(tmem + 256 + x * 128, kv_addr(x), kv_addr(3), true, true);
        }
        mma_commit(smem_u32(&sm.bar_lin));
      }
      if (activeX) l_sum += dot;
      wait_lin();
      o_init = true;
    }
    for (int t = 0; t < n_itiles; ++t) {
      const int i0 = it0 + t * kKT;
      if (tid == mma_tid) {
        // buffers 2 and 3 are free: the products that read them have completed
        const uint32_t bar = smem_u32(&sm.bar_pk[0]);
        mbar_expect_tx(bar, 2u * kTileBytes);
        tma_tile(kv_addr(2), map_pk, int(u) * p.Cmax + i0, bar);
        tma_tile(kv_addr(3), map_pk, rows_k + int(u) * p.Cmax + i0, bar);
        mbar_wait(bar, uint32_t(t) & 1u, failed);
        tc_fence_after();
        for (int x = 0; x < 2; ++x) {
          if (x == 1 && !hasB) break;
          issue_mma(tmem + x * 128, sQ[x], kv_addr(2), false, false);      // C_X = phi+(Q_X) phi+(K')^T ...
          issue_mma(tmem + x * 128, kv_addr(x), kv_addr(3), false, true);  // ... + phi-(Q_X) phi-(K')^T
        }
        mma_commit(smem_u32(&sm.bar_lin));
      }
      wait_lin();
      convert_c(i0);
      if (tid < kSoftmaxThreads) cp_async_wait_all();   // the step's V' rows
      fence_async_smem();
      tc_fence_before();
      __syncthreads();
      if (tid == mma_tid) {
        tc_fence_after();
        issue_mma_ts(tmem + 256, tmem, kv_addr(4), o_init);
        if (hasB) issue_mma_ts(tmem + 384, tmem + 128, kv_addr(4), o_init);
        mma_commit(smem_u32(&sm.bar_lin));
      }
      wait_lin();
      o_init = true;
      if (t + 1 < n_itiles && tid < kSoftmaxThreads) load_vp(t + 1);
    }
  }
  // ---- shared normaliser and store: one contiguous 256-byte row per thread ------------------------------------
  __syncthreads();
  const bool bad = sm.failed != 0;
  if (bad) {
    if (tid == 0) atomicExch(&p.ctl->status, kDevWaitTimeout);
  } else if (activeX && o_init) {
    const bool store = tok_r < ntokX;   // the TMEM loads below are warp-collective: only the store is per row
    const float inv = store ? 1.0f / l_sum : 0.f;
    bf16 *op = reinterpret_cast<bf16 *>(p.out) +
               ((seq + size_t(p.c0 + (store ? tl : tok0))) * p.H + p.heads_of[g * G + hh]) * kD;
    uint32_t ra[32], rb[32];
    tmem_ld32_nowait(tO, ra);
#pragma unroll
    for (int c0 = 0; c0 < kD; c0 += 32) {
      uint32_t (&r)[32] = ((c0 >> 5) & 1) ? rb : ra;
      tmem_wait_ld();
      if (c0 + 32 < kD) tmem_ld32_nowait(tO + c0 + 32, ((c0 >> 5) & 1) ? ra : rb);   // the next columns are on their way
#pragma unroll
      for (int q4 = 0; q4 < 4; ++q4) {
        uint32_t pk[4];
#pragma unroll
        for (int e = 0; e < 4; ++e)
          pk[e] = pack_bf16x2(__uint_as_float(r[q4 * 8 + e * 2]) * inv, __uint_as_float(r[q4 * 8 + e * 2 + 1]) * inv);
        if (store) *reinterpret_cast<uint4 *>(op + c0 + q4 * 8) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  PF_CLK(6);
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
}

}  // namespace


// The kernel needs the ring descriptors made for the tensor-core decode kernels.
#ifdef GLIDE_PF_CLOCKS
extern "C" int glide_debug_pf_clocks(unsigned long long *host16, int reset) {
  if (cudaMemcpyFromSymbol(host16, g_pf_clk, sizeof(g_pf_clk)) != cudaSuccess) return 6;
  if (reset) {
    unsigned long long z[16] = {};
    if (cudaMemcpyToSymbol(g_pf_clk, z, sizeof(z)) != cudaSuccess) return 6;
  }
  return 0;
}
#endif

bool prefill_attn_tc_supported(const glide_ctx *ctx) {
  return ctx->cfg.io_dtype == GLIDE_BF16 && ctx->cfg.head_dim == kD && ctx->decode_kind >= 1 && ctx->off_phik16 != 0;
}

namespace {
typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                             const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeFn tensor_map_encoder() {
  static EncodeFn fn = [] {
    void *f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess || !f ||
        q != cudaDriverEntryPointSuccess) {
      cudaGetLastError();
      f = nullptr;
    }
    return reinterpret_cast<EncodeFn>(f);
  }();
  return fn;
}
}  // namespace

int launch_prefill_attn_tc(glide_ctx *ctx, const PrefillParams &p, cudaStream_t stream) {
  EncodeFn encode = tensor_map_encoder();
  if (!encode) return GLIDE_ERR_CUDA;
  CallMaps cm;
  {
    const cuuint64_t dims[4] = {cuuint64_t(kD), cuuint64_t(p.Hkv), cuuint64_t(p.T), cuuint64_t(p.layer_count) * cuuint64_t(p.B)};
    const cuuint64_t strides[3] = {cuuint64_t(kD) * 2, cuuint64_t(p.Hkv) * kD * 2, cuuint64_t(p.T) * p.Hkv * kD * 2};
    const cuuint32_t box[4] = {64, 1, kGroup, 1}, box128[4] = {64, 1, kKT, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    memset(&cm, 0, sizeof(cm));
    // (a whole-tile box is used only for tiles that lie inside the call: calls shorter than a tile never need it)
    for (int kv = 0; kv < (p.T >= kKT ? 4 : 2); ++kv) {
      CUtensorMap *m = kv == 0 ? &cm.k : kv == 1 ? &cm.v : kv == 2 ? &cm.k128 : &cm.v128;
      CUresult r = encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>((kv & 1) == 0 ? p.k : p.v), dims,
                          strides, kv < 2 ? box : box128, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (r != CUDA_SUCCESS) return GLIDE_ERR_UNSUPPORTED;
    }
  }
  const CUtensorMap *ring_maps = reinterpret_cast<const CUtensorMap *>(ctx->ws + ctx->off_tmaps);
  const int64_t units = int64_t(p.layer_count) * p.B * p.Hkv;
  auto launch = [&](auto gg) -> int {
    constexpr int G = decltype(gg)::value;
    constexpr int TOKC = 2 * kRows / G;
    const size_t smem = sizeof(Smem) + 1024;
    const int64_t blocks = units * ((p.C + TOKC - 1) / TOKC);
    auto run = [&](auto kern) -> int {
      if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess) {
        cudaGetLastError();
        return GLIDE_ERR_CUDA;
      }
      kern<<<unsigned(blocks), kThreads, smem, stream>>>(p, ring_maps, cm);
      return cudaGetLastError() == cudaSuccess ? GLIDE_OK : GLIDE_ERR_CUDA;
    };
    if (p.phiq16) return run(prefill_attn_tc_kernel<G, false, true>);   // learned map (shared normaliser only)
    return p.merge == GLIDE_MERGE_SHARED ? run(prefill_attn_tc_kernel<G, false, false>) : run(prefill_attn_tc_kernel<G, true, false>);
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
