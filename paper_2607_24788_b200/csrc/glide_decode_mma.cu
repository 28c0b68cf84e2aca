// Fused GLIDE decode step for bf16 I/O on sm_100a: persistent, barrier-free, one launch per step.
//
// Every WARP is an autonomous worker that pulls work items from the static longest-first list
// through an atomic counter (the list and the ticket/merge protocol are those of glide_decode.cu):
//
//   window item -- the warp streams its run of ring slots through a private 3-stage shared-memory
//     ring of 16-key tiles.  One lane issues TMA tensor loads (cp.async.bulk.tensor.2d, 128-byte
//     swizzle, completion on an mbarrier) for K and V boxes; all lanes then run the tile on the
//     tensor cores: S = K_tile Q^T (keys on M, the KV head's query heads on N, zero padded to 8),
//     online softmax in the log2 domain on the accumulator fragment, P transposed in registers
//     (movmatrix) and O^T += V_tile^T P.  HBM traffic is the K/V rows exactly once for all G heads.
//   state item  -- the warp folds the token leaving the window into its block of S rows
//     (S += phi(k) v^T, z += phi(k), fp32, in place) and reads the updated rows out against phi(q).
//
// The warp holding the last ticket of a unit merges the partials under the shared normaliser,
// writes the output and stores k,v into the ring slot.  No warp waits on another warp; the only
// waits are on the warp's own TMA mbarriers, and those are bounded.
#include <cuda.h>

#include "glide_device.cuh"

namespace glide {

namespace {

constexpr int kTileKeys = 16;

// Optional per-warp event trace (debug builds only: -DGLIDE_TRACE).
#ifdef GLIDE_TRACE
__device__ unsigned long long *g_trace = nullptr;   // [warps][64] of (code << 56 | globaltimer ns)
#define GLIDE_TRACE_EVENT(code)                                                                    \
  do {                                                                                             \
    if (g_trace && lane == 0 && trace_n < 64) {                                                    \
      unsigned long long now;                                                                      \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));                                      \
      g_trace[(size_t(blockIdx.x) * (blockDim.x >> 5) + (threadIdx.x >> 5)) * 64 + trace_n++] =    \
          (static_cast<unsigned long long>(code) << 56) | (now & 0x00ffffffffffffffull);           \
    }                                                                                              \
  } while (0)
#else
#define GLIDE_TRACE_EVENT(code) do { } while (0)
#endif
constexpr uint32_t kWaitLimit = 1u << 24;   // polls of one mbarrier before giving up

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return uint32_t(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void *tmap, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(tmap), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
  return y;
}
// two fp32 -> packed bf16x2 (lo in the low half), and the rounded values back as fp32
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi, float &lo_r, float &hi_r) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  lo_r = __low2float(v);
  hi_r = __high2float(v);
  return *reinterpret_cast<const uint32_t *>(&v);
}
__device__ __forceinline__ float quad_col_max(float x) {  // over the 8 lanes that share lane % 4
  x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 4));
  x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 8));
  return fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 16));
}
__device__ __forceinline__ float quad_col_sum(float x) {
  x += __shfl_xor_sync(0xffffffffu, x, 4);
  x += __shfl_xor_sync(0xffffffffu, x, 8);
  return x + __shfl_xor_sync(0xffffffffu, x, 16);
}

struct WarpPipe {
  uint32_t stages;   // shared address of this warp's stage ring
  uint32_t bars;     // shared address of this warp's mbarriers (8 bytes each)
  uint32_t phases;   // bit s = parity the next wait on stage s expects
  bool failed;       // a wait ran out
};

// ---- window item ---------------------------------------------------------------------------
template <int D, int G, int STAGES>
__device__ __forceinline__ void window_item_mma(const DecodeParams &p, const void *tmapK, const void *tmapV,
                                                const WorkItem &it, const LayerDev &ld, int64_t t, int b, int g,
                                                float *rec, WarpPipe &pipe, int lane) {
  using bf16 = __nv_bfloat16;
  constexpr int KS = D / 16;                        // k-steps of QK^T = m-tiles of PV
  constexpr int BOXES = D / 64;                     // 128-byte wide TMA boxes per row
  constexpr uint32_t BOX_BYTES = kTileKeys * 128;   // 2 KiB
  constexpr uint32_t TILE_BYTES = BOXES * BOX_BYTES;
  const int col2 = (lane & 3) * 2;                  // this thread's head columns: col2, col2 + 1
  const int hrow = lane >> 2;

  // Q^T as the B operand (k = feature, n = head); heads >= G are zero padding
  uint32_t qb[KS][2];
  {
    const bool valid = hrow < G;
    const int head = valid ? p.heads_of[g * G + hrow] : 0;
    const uint32_t *qrow =
        reinterpret_cast<const uint32_t *>(reinterpret_cast<const bf16 *>(p.q) + ((size_t(it.layer) * p.B + b) * p.H + head) * D);
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qb[ks][0] = valid ? qrow[ks * 8 + (lane & 3)] : 0u;
      qb[ks][1] = valid ? qrow[ks * 8 + 4 + (lane & 3)] : 0u;
    }
  }
  float o[KS][4];
#pragma unroll
  for (int mt = 0; mt < KS; ++mt) o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f;
  float m0 = -CUDART_INF_F, m1 = -CUDART_INF_F, l0 = 0.f, l1 = 0.f;

  // valid slots: [0, t) while the ring is filling, afterwards all but t mod cap
  const int64_t lim64 = t < ld.cap ? t : ld.cap;
  const int cur = int(t % ld.cap);
  const int end = min(it.begin + it.count, int(lim64));
  const int ntiles = end > it.begin ? (end - it.begin + kTileKeys - 1) / kTileKeys : 0;
  const int row0 = int((size_t(b) * p.Hkv + g) * size_t(ld.cap)) + it.begin;  // row in the layer's [rows][D] tensor

  auto issue = [&](int tile, int stage) {
    if (lane == 0) {
      const uint32_t bar = pipe.bars + stage * 8;
      const uint32_t dst = pipe.stages + stage * 2 * TILE_BYTES;
      // earlier generic-proxy accesses to this stage (state scratch, zeroed rows) precede the async-proxy fill
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      mbar_expect_tx(bar, 2 * TILE_BYTES);
      const int y = row0 + tile * kTileKeys;
#pragma unroll
      for (int bx = 0; bx < BOXES; ++bx) {
        tma_load_2d(dst + bx * BOX_BYTES, tmapK, bx * 64, y, bar);
        tma_load_2d(dst + TILE_BYTES + bx * BOX_BYTES, tmapV, bx * 64, y, bar);
      }
    }
  };

  const int pre = ntiles < STAGES ? ntiles : STAGES;
  for (int s = 0; s < pre; ++s) issue(s, s);

  int stage = 0;
  for (int tile = 0; tile < ntiles; ++tile) {
    // wait for this stage's bytes (bounded)
    {
      const uint32_t bar = pipe.bars + stage * 8;
      const uint32_t parity = (pipe.phases >> stage) & 1u;
      uint32_t spins = 0;
      while (!mbar_try_wait(bar, parity)) {
        if (++spins > kWaitLimit) {
          pipe.failed = true;
          break;
        }
      }
      pipe.phases ^= 1u << stage;
      if (__any_sync(0xffffffffu, pipe.failed)) {
        pipe.failed = true;
        return;
      }
    }
    const uint32_t Kst = pipe.stages + stage * 2 * TILE_BYTES;
    const uint32_t Vst = Kst + TILE_BYTES;
    const int slot0 = it.begin + tile * kTileKeys;
    const bool ragged = slot0 + kTileKeys > end || (cur >= slot0 && cur < slot0 + kTileKeys);

    if (ragged) {
      // rows that are not window tokens get zero V so that 0 * garbage cannot make a NaN
      for (int r = 0; r < kTileKeys; ++r) {
        const int s = slot0 + r;
        if ((s >= end || s == cur) && lane < BOXES * 8)
          *reinterpret_cast<uint4 *>(__cvta_shared_to_generic(Vst + (lane >> 3) * BOX_BYTES + r * 128 + (lane & 7) * 16)) =
              make_uint4(0u, 0u, 0u, 0u);
      }
      __syncwarp();
    }

    // S[key][head] = K_tile Q^T
    float s[4] = {0.f, 0.f, 0.f, 0.f};
    {
      const int r = (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        const int c = (ks & 3) * 2 + (lane >> 4);
        uint32_t a[4];
        ldmatrix_x4(a, Kst + (ks >> 2) * BOX_BYTES + r * 128 + ((c ^ (r & 7)) << 4));
        mma_bf16(s, a, qb[ks]);
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) s[i] *= p.scale_log2;
    if (ragged) {
      const int k0 = slot0 + hrow, k1 = k0 + 8;
      if (k0 >= end || k0 == cur) s[0] = s[1] = -CUDART_INF_F;
      if (k1 >= end || k1 == cur) s[2] = s[3] = -CUDART_INF_F;
    }
    // online softmax, per head column, log2 domain
    const float mx0 = quad_col_max(fmaxf(s[0], s[2]));
    const float mx1 = quad_col_max(fmaxf(s[1], s[3]));
    const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
    if (__any_sync(0xffffffffu, mn0 != m0 || mn1 != m1)) {
      const float c0 = mn0 == -CUDART_INF_F ? 1.f : exp2f(m0 - mn0);
      const float c1 = mn1 == -CUDART_INF_F ? 1.f : exp2f(m1 - mn1);
      l0 *= c0;
      l1 *= c1;
#pragma unroll
      for (int mt = 0; mt < KS; ++mt) {
        o[mt][0] *= c0;
        o[mt][2] *= c0;
        o[mt][1] *= c1;
        o[mt][3] *= c1;
      }
      m0 = mn0;
      m1 = mn1;
    }
    const float ms0 = m0 == -CUDART_INF_F ? 0.f : m0, ms1 = m1 == -CUDART_INF_F ? 0.f : m1;
    float p0, p1, p2, p3;
    uint32_t pb[2];
    pb[0] = pack_bf16(exp2f(s[0] - ms0), exp2f(s[1] - ms1), p0, p1);
    pb[1] = pack_bf16(exp2f(s[2] - ms0), exp2f(s[3] - ms1), p2, p3);
    l0 += p0 + p2;   // the row sum uses the weights as the tensor core will see them
    l1 += p1 + p3;
    pb[0] = movmatrix_trans(pb[0]);   // P[key][head] fragment -> B operand (k = key, n = head)
    pb[1] = movmatrix_trans(pb[1]);
    // O^T[feature][head] += V_tile^T P
    {
      const int j = lane >> 3;
      const int r = (lane & 7) + (j >> 1) * 8;
#pragma unroll
      for (int mt = 0; mt < KS; ++mt) {
        const int c = (mt & 3) * 2 + (j & 1);
        uint32_t a[4];
        ldmatrix_x4_trans(a, Vst + (mt >> 2) * BOX_BYTES + r * 128 + ((c ^ (r & 7)) << 4));
        mma_bf16(o[mt], a, pb);
      }
    }
    __syncwarp();   // every lane has finished reading this stage before it is refilled
    if (tile + STAGES < ntiles) issue(tile + STAGES, stage);
    stage = stage + 1 == STAGES ? 0 : stage + 1;
  }

  // partial record: acc [G][D], m [G], l [G]
  l0 = quad_col_sum(l0);
  l1 = quad_col_sum(l1);
#pragma unroll
  for (int mt = 0; mt < KS; ++mt) {
    const int d0 = mt * 16 + hrow;
    if (col2 < G) {
      rec[col2 * D + d0] = o[mt][0];
      rec[col2 * D + d0 + 8] = o[mt][2];
    }
    if (col2 + 1 < G) {
      rec[(col2 + 1) * D + d0] = o[mt][1];
      rec[(col2 + 1) * D + d0 + 8] = o[mt][3];
    }
  }
  if (hrow == 0) {
    if (col2 < G) {
      rec[G * D + col2] = m0;
      rec[G * D + G + col2] = l0;
    }
    if (col2 + 1 < G) {
      rec[G * D + col2 + 1] = m1;
      rec[G * D + G + col2 + 1] = l1;
    }
  }
}

// ---- state item ----------------------------------------------------------------------------
template <int D, int G>
__device__ __forceinline__ void state_item_warp(const DecodeParams &p, const WorkItem &it, const LayerDev &ld, int64_t t,
                                                int b, int g, float *rec, float *scratch, int lane) {
  using bf16 = __nv_bfloat16;
  constexpr int E = D / 32;
  constexpr int LPR = D / 4;      // lanes per state row (float4 each)
  constexpr int RPI = 32 / LPR;   // rows per warp iteration
  constexpr int U = 8;            // row iterations in flight
  if (!(ld.w == 0 || t >= ld.w)) return;
  const int ub = b * p.Hkv + g;
  const bf16 *ke, *ve;
  if (ld.w == 0) {
    ke = reinterpret_cast<const bf16 *>(p.k) + size_t(it.unit) * D;
    ve = reinterpret_cast<const bf16 *>(p.v) + size_t(it.unit) * D;
  } else {
    const size_t row = (size_t(ub) * size_t(ld.cap) + size_t(t % ld.cap)) * D;
    ke = reinterpret_cast<const bf16 *>(p.ws + ld.ringK) + row;
    ve = reinterpret_cast<const bf16 *>(p.ws + ld.ringV) + row;
  }
  float *s_phik = scratch;            // [D]
  float *s_ve = scratch + D;          // [D]
  float *s_phiq = scratch + 2 * D;    // [G][D]
  {
    float x[E], y[E];
    load_elems<bf16, E>(ke + lane * E, x);
    load_elems<bf16, E>(ve + lane * E, y);
    warp_phi<E>(x);
#pragma unroll
    for (int i = 0; i < E; ++i) {
      s_phik[lane * E + i] = x[i];
      s_ve[lane * E + i] = y[i];
    }
#pragma unroll
    for (int h = 0; h < G; ++h) {
      const int head = p.heads_of[g * G + h];
      load_elems<bf16, E>(reinterpret_cast<const bf16 *>(p.q) + ((size_t(it.layer) * p.B + b) * p.H + head) * D + lane * E, x);
      warp_phi<E>(x);
#pragma unroll
      for (int i = 0; i < E; ++i) s_phiq[h * D + lane * E + i] = x[i];
    }
  }
  __syncwarp();

  const int c4 = lane % LPR, rsub = lane / LPR;
  const int r_end = it.begin + it.count;
  float *Sb = reinterpret_cast<float *>(p.ws + ld.S) + size_t(ub) * D * D;
  const float4 v4 = *reinterpret_cast<const float4 *>(s_ve + c4 * 4);
  float4 a[G];
#pragma unroll
  for (int h = 0; h < G; ++h) a[h] = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int rb = it.begin; rb < r_end; rb += U * RPI) {
    float4 sv[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int r = rb + u * RPI + rsub;
      if (r < r_end) sv[u] = *reinterpret_cast<const float4 *>(Sb + size_t(r) * D + c4 * 4);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int r = rb + u * RPI + rsub;
      if (r < r_end) {
        const float pk = s_phik[r];
        float4 s = sv[u];
        s.x = fmaf(pk, v4.x, s.x);
        s.y = fmaf(pk, v4.y, s.y);
        s.z = fmaf(pk, v4.z, s.z);
        s.w = fmaf(pk, v4.w, s.w);
        *reinterpret_cast<float4 *>(Sb + size_t(r) * D + c4 * 4) = s;
#pragma unroll
        for (int h = 0; h < G; ++h) {
          const float f = s_phiq[h * D + r];
          a[h].x = fmaf(f, s.x, a[h].x);
          a[h].y = fmaf(f, s.y, a[h].y);
          a[h].z = fmaf(f, s.z, a[h].z);
          a[h].w = fmaf(f, s.w, a[h].w);
        }
      }
    }
  }
  if (RPI > 1) {  // D = 64: two rows per iteration, fold the halves of the warp
#pragma unroll
    for (int h = 0; h < G; ++h) {
      a[h].x += __shfl_xor_sync(0xffffffffu, a[h].x, 16);
      a[h].y += __shfl_xor_sync(0xffffffffu, a[h].y, 16);
      a[h].z += __shfl_xor_sync(0xffffffffu, a[h].z, 16);
      a[h].w += __shfl_xor_sync(0xffffffffu, a[h].w, 16);
    }
  }
  if (rsub == 0) {
#pragma unroll
    for (int h = 0; h < G; ++h) *reinterpret_cast<float4 *>(rec + h * D + c4 * 4) = a[h];
  }
  // z rows of this block and the b_h readout
  float *zb = reinterpret_cast<float *>(p.ws + ld.z) + size_t(ub) * D;
  float bp[G];
#pragma unroll
  for (int h = 0; h < G; ++h) bp[h] = 0.f;
  for (int r = it.begin + lane; r < r_end; r += 32) {
    const float zn = zb[r] + s_phik[r];
    zb[r] = zn;
#pragma unroll
    for (int h = 0; h < G; ++h) bp[h] = fmaf(s_phiq[h * D + r], zn, bp[h]);
  }
#pragma unroll
  for (int h = 0; h < G; ++h) {
    const float bs = warp_sum(bp[h]);
    if (lane == 0) {
      rec[G * D + h] = bs;
      rec[G * D + G + h] = 0.f;
    }
  }
  __syncwarp();
}

// ---- merge (the warp with the unit's last ticket) -------------------------------------------
template <int D, int G>
__device__ __forceinline__ void merge_unit_warp(const DecodeParams &p, const WorkItem &it, const LayerDev &ld, int64_t t,
                                                int b, int g, float *scratch, int scratch_floats, int lane) {
  using bf16 = __nv_bfloat16;
  constexpr int E = D / 32;
  const int ub = b * p.Hkv + g;
  const int n_win = ld.n_win_items, n_st = ld.n_state_items;
  const int per_unit = n_win + n_st;
  const float *rec0 = p.partials + ld.part_base + size_t(ub) * per_unit * p.rec_floats;
  const bool has_win = ld.cap > 0;
  const bool has_state = n_st > 0 && (ld.w == 0 || t >= ld.w);
  const bool cached = n_win * G <= scratch_floats;   // per-partial rescale factors kept in the warp's scratch
  const bf16 *kt = reinterpret_cast<const bf16 *>(p.k) + size_t(it.unit) * D;
  const bf16 *vt = reinterpret_cast<const bf16 *>(p.v) + size_t(it.unit) * D;

  float scur[G], M[G], inv[G];
  float kx[E];
  load_elems<bf16, E>(kt + lane * E, kx);
#pragma unroll
  for (int h = 0; h < G; ++h) {
    scur[h] = -CUDART_INF_F;
    if (has_win) {
      const int head = p.heads_of[g * G + h];
      float qx[E];
      load_elems<bf16, E>(reinterpret_cast<const bf16 *>(p.q) + ((size_t(it.layer) * p.B + b) * p.H + head) * D + lane * E, qx);
      float part = 0.f;
#pragma unroll
      for (int i = 0; i < E; ++i) part = fmaf(qx[i], kx[i], part);
      scur[h] = warp_sum(part) * p.scale_log2;
    }
  }
  // m* = max(window max, current logit, 0 if the state holds tokens: its terms have logit 0; without them a floor
  // would only push the window weights towards underflow); the partial maxima are read once, lane-strided
#pragma unroll
  for (int h = 0; h < G; ++h) {
    float mx = has_state ? fmaxf(scur[h], 0.f) : scur[h];
    for (int i = lane; i < n_win; i += 32) mx = fmaxf(mx, __ldcg(rec0 + size_t(i) * p.rec_floats + G * D + h));
    M[h] = warp_max(mx);
  }
#pragma unroll
  for (int h = 0; h < G; ++h) {
    float den = 0.f;
    for (int i = lane; i < n_win; i += 32) {
      const float *r = rec0 + size_t(i) * p.rec_floats;
      const float f = exp2f(__ldcg(r + G * D + h) - M[h]);
      if (cached) scratch[i * G + h] = f;
      den = fmaf(__ldcg(r + G * D + G + h), f, den);
    }
    float bs = 0.f;
    if (has_state)
      for (int i = lane; i < n_st; i += 32) bs += __ldcg(rec0 + size_t(n_win + i) * p.rec_floats + G * D + h);
    den = warp_sum(den) + (has_win ? exp2f(scur[h] - M[h]) : 0.f) + (has_state ? exp2f(-M[h]) * warp_sum(bs) : 0.f);
    inv[h] = 1.0f / den;
  }
  __syncwarp();
  bf16 *outp = reinterpret_cast<bf16 *>(p.out);
#pragma unroll
  for (int j = 0; j * 128 < G * D; ++j) {
    const int idx = (j * 32 + lane) * 4;   // four consecutive features of one head per lane
    if (idx >= G * D) break;
    const int h = idx / D, c = idx - h * D;
    float Mh = 0.f, invh = 0.f, scurh = 0.f;
#pragma unroll
    for (int hh = 0; hh < G; ++hh)       // register select: no dynamically indexed arrays
      if (hh == h) {
        Mh = M[hh];
        invh = inv[hh];
        scurh = scur[hh];
      }
    float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
    if (cached) {
      constexpr int MU = 8;   // independent loads in flight
      for (int i0 = 0; i0 < n_win; i0 += MU) {
        float4 a[MU];
#pragma unroll
        for (int u = 0; u < MU; ++u)
          if (i0 + u < n_win) a[u] = __ldcg(reinterpret_cast<const float4 *>(rec0 + size_t(i0 + u) * p.rec_floats + idx));
#pragma unroll
        for (int u = 0; u < MU; ++u)
          if (i0 + u < n_win) {
            const float f = scratch[(i0 + u) * G + h];
            num.x = fmaf(a[u].x, f, num.x);
            num.y = fmaf(a[u].y, f, num.y);
            num.z = fmaf(a[u].z, f, num.z);
            num.w = fmaf(a[u].w, f, num.w);
          }
      }
    } else {
      for (int i = 0; i < n_win; ++i) {
        const float *r = rec0 + size_t(i) * p.rec_floats;
        const float f = exp2f(__ldcg(r + G * D + h) - Mh);
        const float4 a = __ldcg(reinterpret_cast<const float4 *>(r + idx));
        num.x = fmaf(a.x, f, num.x);
        num.y = fmaf(a.y, f, num.y);
        num.z = fmaf(a.z, f, num.z);
        num.w = fmaf(a.w, f, num.w);
      }
    }
    if (has_win) {
      const float f = exp2f(scurh - Mh);
      float vx[4];
      load_elems<bf16, 4>(vt + c, vx);
      num.x = fmaf(f, vx[0], num.x);
      num.y = fmaf(f, vx[1], num.y);
      num.z = fmaf(f, vx[2], num.z);
      num.w = fmaf(f, vx[3], num.w);
    }
    if (has_state) {
      float4 asum = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int i = 0; i < n_st; ++i) {
        const float4 a = __ldcg(reinterpret_cast<const float4 *>(rec0 + size_t(n_win + i) * p.rec_floats + idx));
        asum.x += a.x;
        asum.y += a.y;
        asum.z += a.z;
        asum.w += a.w;
      }
      const float f = exp2f(-Mh);
      num.x = fmaf(f, asum.x, num.x);
      num.y = fmaf(f, asum.y, num.y);
      num.z = fmaf(f, asum.z, num.z);
      num.w = fmaf(f, asum.w, num.w);
    }
    const int head = p.heads_of[g * G + h];
    const __nv_bfloat162 lo = __floats2bfloat162_rn(num.x * invh, num.y * invh);
    const __nv_bfloat162 hi = __floats2bfloat162_rn(num.z * invh, num.w * invh);
    uint2 packed;
    packed.x = *reinterpret_cast<const uint32_t *>(&lo);
    packed.y = *reinterpret_cast<const uint32_t *>(&hi);
    *reinterpret_cast<uint2 *>(outp + ((size_t(it.layer) * p.B + b) * p.H + head) * D + c) = packed;
  }
  if (has_win) {  // all readers of slot t mod cap are done: store the new row (bit copy)
    const size_t row = (size_t(ub) * size_t(ld.cap) + size_t(t % ld.cap)) * D;
    bf16 *Kd = reinterpret_cast<bf16 *>(p.ws + ld.ringK) + row;
    bf16 *Vd = reinterpret_cast<bf16 *>(p.ws + ld.ringV) + row;
    if constexpr (E == 4) {
      *reinterpret_cast<uint2 *>(Kd + lane * 4) = *reinterpret_cast<const uint2 *>(kt + lane * 4);
      *reinterpret_cast<uint2 *>(Vd + lane * 4) = *reinterpret_cast<const uint2 *>(vt + lane * 4);
    } else {
      *reinterpret_cast<uint32_t *>(Kd + lane * 2) = *reinterpret_cast<const uint32_t *>(kt + lane * 2);
      *reinterpret_cast<uint32_t *>(Vd + lane * 2) = *reinterpret_cast<const uint32_t *>(vt + lane * 2);
    }
  }
  __syncwarp();
}

template <int D, int G, int WARPS, int STAGES>
__global__ void __launch_bounds__(WARPS * 32, 1) glide_decode_mma_kernel(const DecodeParams p, const CUtensorMap *tmaps) {
  constexpr uint32_t STAGE_BYTES = 2 * kTileKeys * D * 2;   // K tile + V tile
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t bars[WARPS][STAGES];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // 1024-byte aligned stage ring per warp (the 128-byte swizzle repeats every 1024 bytes)
  unsigned char *base = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char *my_stages = base + size_t(warp) * STAGES * STAGE_BYTES;
  WarpPipe pipe;
  pipe.stages = smem_u32(my_stages);
  pipe.bars = smem_u32(&bars[warp][0]);
  pipe.phases = 0;
  pipe.failed = false;
  if (lane == 0) {
    for (int s = 0; s < STAGES; ++s) mbar_init(pipe.bars + s * 8, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncwarp();
  const int units_per_layer = p.B * p.Hkv;

#ifdef GLIDE_TRACE
  int trace_n = 0;
#endif
  GLIDE_TRACE_EVENT(1);
  for (;;) {
    int idx = 0;
    if (lane == 0) idx = atomicAdd(&p.ctl->work_counter, 1);
    idx = __shfl_sync(0xffffffffu, idx, 0);
    GLIDE_TRACE_EVENT(2);
    if (idx >= p.n_items) break;
    const WorkItem it = p.items[idx];
    if (it.layer < 0 || it.layer >= p.L || it.unit < 0) {
      if (lane == 0) atomicExch(p.status, kDevBadItem);
      continue;
    }
    if (it.layer < p.layer_begin || it.layer >= p.layer_begin + p.layer_count) continue;   // not a layer of this launch
    const LayerDev ld = p.layers[it.layer];
    const int ub = it.unit - it.layer * units_per_layer;
    const int b = ub / p.Hkv, g = ub - b * p.Hkv;
    const int64_t t = p.n_dev[it.layer] + (p.seq_off ? p.seq_off[b] : 0);   // position of this sequence
    if (t < 0) continue;   // parked slot: nothing is read or written for it (every item of the unit takes this branch)
    const int per_unit = ld.n_win_items + ld.n_state_items;
    float *rec = p.partials + ld.part_base + (size_t(ub) * per_unit + it.part) * p.rec_floats;
    GLIDE_TRACE_EVENT(it.kind == kItemWindow ? 3 : 4);
    if (it.kind == kItemWindow) {
      window_item_mma<D, G, STAGES>(p, tmaps + 3 * it.layer, tmaps + 3 * it.layer + 1, it, ld, t, b, g, rec, pipe, lane);
      if (pipe.failed) {  // a TMA never completed: record it and stop taking work
        if (lane == 0) atomicExch(p.status, kDevWaitTimeout);
        break;
      }
    } else {
      state_item_warp<D, G>(p, it, ld, t, b, g, rec, reinterpret_cast<float *>(my_stages), lane);
    }
    GLIDE_TRACE_EVENT(5);
    __threadfence();
    __syncwarp();
    GLIDE_TRACE_EVENT(6);
    int last = 0;
    if (lane == 0) last = atomicAdd(&p.tickets[it.unit], 1) == per_unit - 1;
    last = __shfl_sync(0xffffffffu, last, 0);
    GLIDE_TRACE_EVENT(7);
    if (last) {
      __threadfence();
      merge_unit_warp<D, G>(p, it, ld, t, b, g, reinterpret_cast<float *>(my_stages), int(STAGES * STAGE_BYTES / 4), lane);
      if (lane == 0) p.tickets[it.unit] = 0;
      GLIDE_TRACE_EVENT(8);
    }
  }
  GLIDE_TRACE_EVENT(9);
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    if (atomicAdd(&p.ctl->done_counter, 1) == int(gridDim.x) - 1) {
      p.ctl->work_counter = 0;
      p.ctl->done_counter = 0;
      for (int l = 0; l < p.layer_count; ++l) p.n_dev[p.layer_begin + l] += 1;
      __threadfence();
    }
  }
}

constexpr int kMmaWarps = 8;
constexpr int kMmaStages = 3;

template <int D>
constexpr size_t mma_smem_bytes() {
  return size_t(kMmaWarps) * kMmaStages * (2 * kTileKeys * D * 2) + 1024;
}

template <typename F>
int dispatch_mma(int D, int G, F &&f) {
#define GLIDE_MMA_G(DD)                                  \
  switch (G) {                                           \
    case 1: return f(IntTag<DD>{}, IntTag<1>{});         \
    case 2: return f(IntTag<DD>{}, IntTag<2>{});         \
    case 4: return f(IntTag<DD>{}, IntTag<4>{});         \
    case 8: return f(IntTag<DD>{}, IntTag<8>{});         \
    default: return int(GLIDE_ERR_UNSUPPORTED);          \
  }
  if (D == 64) { GLIDE_MMA_G(64) }
  if (D == 128) { GLIDE_MMA_G(128) }
#undef GLIDE_MMA_G
  return int(GLIDE_ERR_UNSUPPORTED);
}

}  // namespace

int build_ring_tensor_maps(glide_ctx *ctx) {
  // tensor maps: per layer the K ring and the V ring as [rows = B*Hkv*cap][D] bf16, 64 x 16 boxes, 128-byte swizzle
  typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                               const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                               CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  void *fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess) {
    cudaGetLastError();
    return GLIDE_ERR_CUDA;
  }
  EncodeFn encode = reinterpret_cast<EncodeFn>(fn);
  const int L = ctx->cfg.n_layers, D = ctx->cfg.head_dim;
  ctx->tmaps_host.assign((size_t(L) * 5 + 3) * sizeof(CUtensorMap), 0);
  ctx->tmaps_kv4d = D == 128;
  CUtensorMap *maps = reinterpret_cast<CUtensorMap *>(ctx->tmaps_host.data());
  for (int l = 0; l < L; ++l) {
    const LayerDev &ld = ctx->layers[l];
    if (ld.cap == 0) continue;
    const cuuint64_t rows = cuuint64_t(ctx->cfg.batch) * ctx->cfg.n_kv_heads * cuuint64_t(ld.cap);
    const cuuint64_t dims[2] = {cuuint64_t(D), rows};
    const cuuint64_t strides[1] = {cuuint64_t(D) * 2};
    const cuuint32_t box[2] = {64, kTileKeys};
    const cuuint32_t estr[2] = {1, 1};
    for (int kv = 0; kv < 2; ++kv) {
      void *gptr = ctx->ws + (kv == 0 ? ld.ringK : ld.ringV);
      CUresult r = encode(&maps[3 * l + kv], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, gptr, dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (r != CUDA_SUCCESS) return GLIDE_ERR_CUDA;
      // the same ring with boxes of a whole 128-key tile (prefill: tiles that neither wrap nor cross into the call);
      // these maps follow the 3 L maps of the decode kernels
      if (D == 128 && ld.cap >= 128) {
        const cuuint32_t box128[2] = {64, 128};
        r = encode(&maps[3 * L + 2 * l + kv], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, gptr, dims, strides, box128, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return GLIDE_ERR_CUDA;
      }
    }
    if (D == 128 && ctx->tmaps_kv4d) {
      // K and V rings of the layer as one 4-D tensor [kv][half][row][64]: a single TMA then fills a whole
      // window stage in the layout the 2-D boxes produce (K halves, then V halves)
      const cuuint64_t dims4[4] = {64, rows, 2, 2};
      const cuuint64_t strides4[3] = {cuuint64_t(D) * 2, 128, cuuint64_t(ld.ringV - ld.ringK)};
      const cuuint32_t box4[4] = {64, kTileKeys, 2, 2};
      const cuuint32_t estr4[4] = {1, 1, 1, 1};
      CUresult r = encode(&maps[3 * l + 2], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, ctx->ws + ld.ringK, dims4, strides4, box4,
                          estr4, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (r != CUDA_SUCCESS) ctx->tmaps_kv4d = false;   // the driver refused the strides: keep the 2-D boxes
    }
  }
  if (D == 128 && ctx->off_phik16 != 0) {
    // prefill scratch as [rows][128] bf16 with boxes of a whole 128-row tile: phi(K') rows of the chunk ([unit][chunk]
    // rows), the bf16 copy of S ([unit][128] rows) and, for the learned map, phi(Q) ([unit][chunk][G] rows); with the
    // learned map every array holds its two 128-column halves one after the other
    const cuuint64_t units = cuuint64_t(L) * ctx->cfg.batch * ctx->cfg.n_kv_heads;
    const cuuint64_t halves = cuuint64_t(ctx->dp / D);
    const cuuint64_t strides[1] = {cuuint64_t(D) * 2};
    const cuuint32_t box128[2] = {64, 128};
    const cuuint32_t estr[2] = {1, 1};
    for (int i = 0; i < (ctx->off_phiq16 ? 3 : 2); ++i) {
      const cuuint64_t rows = halves * units * (i == 0 ? cuuint64_t(ctx->prefill_chunk) : i == 1 ? cuuint64_t(D) : cuuint64_t(ctx->prefill_chunk) * ctx->G);
      const cuuint64_t dims[2] = {cuuint64_t(D), rows};
      const size_t base = i == 0 ? ctx->off_phik16 : i == 1 ? ctx->off_s16 : ctx->off_phiq16;
      CUresult r = encode(&maps[5 * L + i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ctx->ws + base, dims, strides, box128, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (r != CUDA_SUCCESS) return GLIDE_ERR_CUDA;
    }
  }
  return GLIDE_OK;
}

int mma_decode_setup(glide_ctx *ctx) {
  return dispatch_mma(ctx->cfg.head_dim, ctx->G, [&](auto dd, auto gg) -> int {
    constexpr int DD = decltype(dd)::value, GG = decltype(gg)::value;
    auto kern = glide_decode_mma_kernel<DD, GG, kMmaWarps, kMmaStages>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(mma_smem_bytes<DD>())) != cudaSuccess) {
      cudaGetLastError();
      return GLIDE_ERR_CUDA;
    }
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kMmaWarps * 32, mma_smem_bytes<DD>()) != cudaSuccess ||
        per_sm < 1) {
      cudaGetLastError();
      return GLIDE_ERR_CUDA;
    }
    ctx->decode_grid = std::max(1, std::min((ctx->n_items + kMmaWarps - 1) / kMmaWarps, ctx->sm_count * per_sm));
    return GLIDE_OK;
  });
}

#ifdef GLIDE_TRACE
extern "C" int glide_debug_set_trace(void *dev_buf) {
  return cudaMemcpyToSymbol(g_trace, &dev_buf, sizeof(void *)) == cudaSuccess ? 0 : 6;
}
#endif

int launch_decode_mma(glide_ctx *ctx, const DecodeParams &p, cudaStream_t stream) {
  const CUtensorMap *tmaps = reinterpret_cast<const CUtensorMap *>(ctx->ws + ctx->off_tmaps);
  return dispatch_mma(ctx->cfg.head_dim, ctx->G, [&](auto dd, auto gg) -> int {
    constexpr int DD = decltype(dd)::value, GG = decltype(gg)::value;
    glide_decode_mma_kernel<DD, GG, kMmaWarps, kMmaStages>
        <<<ctx->decode_grid, kMmaWarps * 32, mma_smem_bytes<DD>(), stream>>>(p, tmaps);
    if (cudaGetLastError() != cudaSuccess) return GLIDE_ERR_CUDA;
    return GLIDE_OK;
  });
}

}  // namespace glide
