// Fused GLIDE decode step for bf16, head_dim 128: statically scheduled streaming kernel (sm_100a).
//
// The step's whole traffic is laid out as one stream of equal-sized tiles, unit after unit
// (unit = layer x sequence x KV head, largest first):
//   state tile  -- 16 rows of the unit's S (8 KiB fp32) plus the 16 matching z entries,
//   window tile -- 16 ring slots: a 16x128 bf16 K box and V box (8 KiB).
// The host cuts the stream into one contiguous, equally heavy range per CTA (one CTA per SM) and
// describes it by a short segment list (one segment per unit the range touches).  Inside a CTA tile
// i of the range belongs to warp i mod 8.  Every warp owns a ring of TMA stages and keeps it full
// ACROSS unit boundaries: lane 0 issues cp.async.bulk(.tensor) loads for the warp's next tiles as
// stages drain, so the memory pipe never empties while a unit is being finished.
//   window tile: S = K_tile Q^T on the tensor cores (keys on M, query heads on N), online softmax
//                in the log2 domain, P transposed in registers, O^T += V_tile^T P;
//   state tile:  S += phi(k_e) v_e^T and z += phi(k_e) in place (fp32), readout phi(q_h)^T S, phi(q_h)^T z.
// The linear readout is folded into the warp's softmax partial as a term with logit 0 (exact: the
// shared normaliser's reference m* is max(window max, 0)), so a unit needs ONE (m, l, acc) record per
// warp.  When a unit's segment ends the 8 warps reduce their records in shared memory; a unit that
// lies inside one CTA is finished right there (current token's own term, normalise, write, ring
// append) without touching global scratch.  Only units cut by a CTA boundary go through one global
// record per CTA and a ticket; the last CTA merges those few records.  No CTA waits for another.
#include <cuda.h>

#include <algorithm>

#include "glide_device.cuh"

namespace glide {

namespace {

constexpr int kD = 128;
constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kTileRows = 16;
constexpr uint32_t kStageBytes = 2 * kTileRows * kD * 2;   // 8 KiB: K box + V box, or 16 fp32 state rows
constexpr uint32_t kBoxBytes = kTileRows * 128;            // one 64-column TMA box
constexpr uint32_t kTileKV = 2 * kBoxBytes;                // K (or V) part of a window stage
constexpr uint32_t kWaitLimit = 1u << 24;
constexpr int kHdrSlots = 3;

// Optional per-warp event trace (debug builds only: -DGLIDE_TRACE).
#ifdef GLIDE_TRACE
__device__ unsigned long long *g_stream_trace = nullptr;   // [warps][64] of (code << 56 | globaltimer ns)
#define GLIDE_TRACE_EVENT(code)                                                                        \
  do {                                                                                                 \
    if (g_stream_trace && lane == 0 && trace_n < 64) {                                                 \
      unsigned long long now;                                                                          \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));                                          \
      g_stream_trace[(size_t(blockIdx.x) * kWarps + (threadIdx.x >> 5)) * 64 + trace_n++] =            \
          (static_cast<unsigned long long>(code) << 56) | (now & 0x00ffffffffffffffull);               \
    }                                                                                                  \
  } while (0)
#else
#define GLIDE_TRACE_EVENT(code) do { } while (0)
#endif

// ---- PTX wrappers --------------------------------------------------------------------------
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
// Bounded wait: false if the barrier did not flip within kWaitLimit polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity))
    if (++spins > kWaitLimit) return false;
  return true;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void *tmap, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(tmap), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
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
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
  uint32_t y;
  asm("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
  return y;
}
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
__device__ __forceinline__ float lds_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ float4 lds_f32x4(uint32_t addr) {
  float4 v;
  asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
  return v;
}
// ---- schedule walking ------------------------------------------------------------------------
__device__ __forceinline__ float ex2_approx(float x) {   // 2^x, 2 ulp, 2^-inf = 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float exp2_or_zero(float m, float M) { return m == -CUDART_INF_F ? 0.f : ex2_approx(m - M); }

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const void *tmap, int c0, int c1, int c2, int c3, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(dst),
      "l"(tmap), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
      : "memory");
}

__device__ __forceinline__ bool seg_evicting(const StreamSegment &s, int64_t t) {
  return s.evicts && (s.w == 0 || t >= int64_t(s.w));
}

// A warp's position in the CTA's tile range with the fields of its current segment cached in registers.
struct Cursor {
  int i;         // CTA-relative index of this warp's next candidate tile
  int seg;       // segment that holds it
  int tile0, tile_end, n_state, state0, win0;
  int n_valid_win;   // window tiles of the segment that hold window tokens at this position
  int evicting;
};
struct TileRef {
  int seg;
  int index;     // state tile (rows 16*index ..) or window tile (slots 16*index ..) within the unit
  bool is_state;
};

__device__ __forceinline__ void cursor_load(Cursor &c, const StreamSegment *segs, int64_t t) {
  const StreamSegment &s = segs[c.seg];
  c.tile0 = s.tile0;
  c.n_state = s.n_state;
  c.state0 = s.state0;
  c.win0 = s.win0;
  c.tile_end = s.tile0 + s.n_state + s.n_win;
  const int64_t lim = t < int64_t(s.cap) ? t : int64_t(s.cap);
  int nv = int((lim + kTileRows - 1) / kTileRows) - s.win0;
  c.n_valid_win = nv < 0 ? 0 : (nv > s.n_win ? s.n_win : nv);
  c.evicting = seg_evicting(s, t) ? 1 : 0;
}

// Next tile of this warp that has work; the issuing lane and the consuming warp walk the same sequence.
__device__ __forceinline__ bool next_tile(Cursor &c, const StreamSegment *segs, int nseg, int ntiles, int64_t t,
                                          TileRef &ref) {
  while (c.i < ntiles) {
    if (c.i >= c.tile_end) {
      do { ++c.seg; } while (c.seg + 1 < nseg && c.i >= segs[c.seg].tile0 + segs[c.seg].n_state + segs[c.seg].n_win);
      cursor_load(c, segs, t);
    }
    const int local = c.i - c.tile0;
    bool valid;
    if (local < c.n_state) {
      ref.is_state = true;
      ref.index = c.state0 + local;
      valid = c.evicting != 0;
    } else {
      ref.is_state = false;
      ref.index = c.win0 + local - c.n_state;
      valid = local - c.n_state < c.n_valid_win;
    }
    ref.seg = c.seg;
    c.i += kWarps;
    if (valid) return true;
  }
  return false;
}

template <int G>
struct Layout {
  static constexpr int kRecFloats = (G * kD + 2 * G + 3) / 4 * 4;
  static constexpr uint32_t kHdrBytes = G * 256 + 4 * 256;   // q rows | k_e | v_e | k_t | v_t
};

// phi = softmax over the 128 entries of N rows at once (lane holds 4 entries of each row); the N
// reductions are interleaved so that their shuffle latencies overlap.
template <int N>
__device__ __forceinline__ void warp_phi_multi(float (&x)[N][4]) {
  float mx[N], sm[N];
#pragma unroll
  for (int n = 0; n < N; ++n) mx[n] = fmaxf(fmaxf(x[n][0], x[n][1]), fmaxf(x[n][2], x[n][3]));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1)
#pragma unroll
    for (int n = 0; n < N; ++n) mx[n] = fmaxf(mx[n], __shfl_xor_sync(0xffffffffu, mx[n], o));
#pragma unroll
  for (int n = 0; n < N; ++n) {
    sm[n] = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[n][i] = exp2f((x[n][i] - mx[n]) * kLog2e);
      sm[n] += x[n][i];
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1)
#pragma unroll
    for (int n = 0; n < N; ++n) sm[n] += __shfl_xor_sync(0xffffffffu, sm[n], o);
#pragma unroll
  for (int n = 0; n < N; ++n) {
    const float inv = 1.0f / sm[n];
#pragma unroll
    for (int i = 0; i < 4; ++i) x[n][i] *= inv;
  }
}

// ---- the kernel -----------------------------------------------------------------------------
template <int G, int STAGES>
__global__ void __launch_bounds__(kThreads, 1)
glide_decode_stream_kernel(const DecodeParams p, const StreamParams sp) {
  using bf16 = __nv_bfloat16;
  using L = Layout<G>;
  constexpr int KS = kD / 16;
  constexpr int VPT = (G * kD + kThreads - 1) / kThreads;   // combined values per thread at a flush

  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char *base = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char *sm_stages = base;                                                  // [kWarps][STAGES][8 KiB]
  float *sm_rec = reinterpret_cast<float *>(sm_stages + size_t(kWarps) * STAGES * kStageBytes);   // [kWarps][kRecFloats]
  unsigned char *sm_hdr = reinterpret_cast<unsigned char *>(sm_rec + kWarps * L::kRecFloats);     // [3][kHdrBytes]
  float *sm_z = reinterpret_cast<float *>(sm_hdr + kHdrSlots * L::kHdrBytes);                    // [kWarps][STAGES][16]
  StreamSegment *sm_segs = reinterpret_cast<StreamSegment *>(sm_z + kWarps * STAGES * 16);      // [max_segs]
  uint64_t *sm_bars = reinterpret_cast<uint64_t *>(sm_segs + sp.max_segs);                        // [kWarps*STAGES + 3]
  float *sm_scur = reinterpret_cast<float *>(sm_bars + kWarps * STAGES + kHdrSlots);             // [8]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
#ifdef GLIDE_TRACE
  int trace_n = 0;
#endif
  GLIDE_TRACE_EVENT(1);
  const int64_t t = p.n_dev[0];   // every layer is at the same position (checked by the host)
  const int col2 = (lane & 3) * 2, hrow = lane >> 2;
  const int seg_begin = sp.cta_seg_begin[blockIdx.x];
  const int nseg = sp.cta_seg_begin[blockIdx.x + 1] - seg_begin;
  if (nseg > 0) {
    const uint4 *src = reinterpret_cast<const uint4 *>(sp.segs + seg_begin);
    uint4 *dst = reinterpret_cast<uint4 *>(sm_segs);
    for (int i = tid; i < nseg * int(sizeof(StreamSegment) / 16); i += kThreads) dst[i] = src[i];
  }
  const uint32_t my_stages = smem_u32(sm_stages + size_t(warp) * STAGES * kStageBytes);
  unsigned char *my_stages_ptr = sm_stages + size_t(warp) * STAGES * kStageBytes;
  const uint32_t my_bars = smem_u32(sm_bars + warp * STAGES);
  const uint32_t my_z = smem_u32(sm_z + warp * STAGES * 16);
  const float *my_z_ptr = sm_z + warp * STAGES * 16;
  const uint32_t hdr_bars = smem_u32(sm_bars + kWarps * STAGES);
  if (lane == 0)
    for (int s = 0; s < STAGES; ++s) mbar_init(my_bars + s * 8, 1);
  if (tid == 0)
    for (int s = 0; s < kHdrSlots; ++s) mbar_init(hdr_bars + s * 8, 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  fence_async_smem();
  __syncthreads();

  const int ntiles = nseg > 0 ? sm_segs[nseg - 1].tile0 + sm_segs[nseg - 1].n_state + sm_segs[nseg - 1].n_win : 0;
  const int units_per_layer = p.B * p.Hkv;
  bool failed = false;

  // ---- header (q rows, evicted k/v, current k/v) of segment s -> slot s % 3, issued by thread 0 -----
  auto issue_header = [&](int s) {
    const StreamSegment &sg = sm_segs[s];
    const uint32_t bar = hdr_bars + (s % kHdrSlots) * 8;
    const uint32_t dst = smem_u32(sm_hdr + size_t(s % kHdrSlots) * L::kHdrBytes);
    const bool ev = seg_evicting(sg, t);
    const int ub = sg.unit - sg.layer * units_per_layer;
    const int b = ub / p.Hkv, g = ub - b * p.Hkv;
    mbar_expect_tx(bar, G * 256 + 512 + (ev ? 512 : 0));
    const bf16 *qb = reinterpret_cast<const bf16 *>(p.q) + (size_t(sg.layer) * p.B + b) * p.H * kD;
    if (sp.heads_contiguous) {
      bulk_load(dst, qb + size_t(p.heads_of[g * G]) * kD, G * 256, bar);
    } else {
      for (int h = 0; h < G; ++h) bulk_load(dst + h * 256, qb + size_t(p.heads_of[g * G + h]) * kD, 256, bar);
    }
    const bf16 *kt = reinterpret_cast<const bf16 *>(p.k) + size_t(sg.unit) * kD;
    const bf16 *vt = reinterpret_cast<const bf16 *>(p.v) + size_t(sg.unit) * kD;
    bulk_load(dst + G * 256 + 512, kt, 256, bar);
    bulk_load(dst + G * 256 + 768, vt, 256, bar);
    if (ev) {
      if (sg.w == 0) {   // no ring: the current token is the one folded into the state
        bulk_load(dst + G * 256, kt, 256, bar);
        bulk_load(dst + G * 256 + 256, vt, 256, bar);
      } else {
        const LayerDev &ld = p.layers[sg.layer];
        const size_t row = (size_t(sg.row_base) + size_t(t % int64_t(sg.cap))) * kD;
        bulk_load(dst + G * 256, reinterpret_cast<const bf16 *>(p.ws + ld.ringK) + row, 256, bar);
        bulk_load(dst + G * 256 + 256, reinterpret_cast<const bf16 *>(p.ws + ld.ringV) + row, 256, bar);
      }
    }
  };
  if (tid == 0) {
    if (nseg > 0) issue_header(0);
    if (nseg > 1) issue_header(1);
  }

  // ---- tile issue (lane 0 of each warp) ---------------------------------------------------------
  Cursor icur;
  icur.i = warp;
  icur.seg = 0;
  icur.tile_end = 0;
  if (nseg > 0) cursor_load(icur, sm_segs, t);
  int issue_stage = 0;
  auto issue_next = [&]() {
    if (lane == 0) {
      TileRef r;
      if (next_tile(icur, sm_segs, nseg, ntiles, t, r)) {
        const StreamSegment &sg = sm_segs[r.seg];
        const uint32_t bar = my_bars + issue_stage * 8;
        const uint32_t dst = my_stages + issue_stage * kStageBytes;
        if (r.is_state) {
          mbar_expect_tx(bar, kStageBytes + 64);
          const float *Sg = reinterpret_cast<const float *>(p.ws + size_t(sg.S_off256) * 256) + size_t(r.index) * kTileRows * kD;
          const float *zg = reinterpret_cast<const float *>(p.ws + size_t(sg.z_off256) * 256) + r.index * kTileRows;
          bulk_load(dst, Sg, kStageBytes, bar);
          bulk_load(my_z + issue_stage * 64, zg, 64, bar);
        } else {
          mbar_expect_tx(bar, kStageBytes);
          const CUtensorMap *tk = reinterpret_cast<const CUtensorMap *>(sp.tmaps) + 3 * sg.layer;
          const int y = sg.row_base + r.index * kTileRows;
          if (sp.kv4d) {
            tma_load_4d(dst, tk + 2, 0, y, 0, 0, bar);   // K halves then V halves: [kv][half][row][64]
          } else {
            tma_load_2d(dst, tk, 0, y, bar);
            tma_load_2d(dst + kBoxBytes, tk, 64, y, bar);
            tma_load_2d(dst + kTileKV, tk + 1, 0, y, bar);
            tma_load_2d(dst + kTileKV + kBoxBytes, tk + 1, 64, y, bar);
          }
        }
        issue_stage = issue_stage + 1 == STAGES ? 0 : issue_stage + 1;
      }
    }
  };
  for (int s = 0; s < STAGES; ++s) issue_next();
  GLIDE_TRACE_EVENT(2);

  // ---- per-unit register state ------------------------------------------------------------------
  uint32_t qb[KS][2];
  float o[KS][4];
  float m0 = -CUDART_INF_F, m1 = -CUDART_INF_F, l0 = 0.f, l1 = 0.f;
  float phi[G + 1][4];     // phi(q_h) for the G heads, then phi(k_e); lane holds entries 4*lane .. 4*lane+3
  float ve[4];
  float4 a[G];
  float bp[G];
  bool had_state = false, phi_ready = false;
  int acc_seg = -1;        // segment the accumulators belong to
  int win_end = 0, win_cur = 0;   // window tokens live in slots [0, win_end) except slot win_cur
  uint32_t phases = 0;     // parity expected by the next wait on each stage
  int stage = 0;

  auto wait_header = [&](int s) {
    if (!mbar_wait(hdr_bars + (s % kHdrSlots) * 8, uint32_t(s / kHdrSlots) & 1u)) failed = true;
  };

  // q fragments of segment s into registers; accumulators cleared
  auto load_unit = [&](int s) {
    const StreamSegment &sg = sm_segs[s];
    wait_header(s);
    const uint32_t *hq = reinterpret_cast<const uint32_t *>(sm_hdr + size_t(s % kHdrSlots) * L::kHdrBytes);
    const bool valid = hrow < G;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      qb[ks][0] = valid ? hq[hrow * 64 + ks * 8 + (lane & 3)] : 0u;
      qb[ks][1] = valid ? hq[hrow * 64 + ks * 8 + 4 + (lane & 3)] : 0u;
    }
    if (sg.cap > 0) {
      const int64_t lim = t < int64_t(sg.cap) ? t : int64_t(sg.cap);
      win_end = int(lim);
      win_cur = int(t % int64_t(sg.cap));
    }
#pragma unroll
    for (int mt = 0; mt < KS; ++mt) o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f;
    m0 = m1 = -CUDART_INF_F;
    l0 = l1 = 0.f;
#pragma unroll
    for (int h = 0; h < G; ++h) {
      a[h] = make_float4(0.f, 0.f, 0.f, 0.f);
      bp[h] = 0.f;
    }
    had_state = false;
    phi_ready = false;
    acc_seg = s;
  };

  // feature maps of the unit's queries and of the evicted key (first state tile of a segment only)
  auto load_phi = [&](int s) {
    const bf16 *h0 = reinterpret_cast<const bf16 *>(sm_hdr + size_t(s % kHdrSlots) * L::kHdrBytes);
#pragma unroll
    for (int h = 0; h < G; ++h) load_elems<bf16, 4>(h0 + h * kD + lane * 4, phi[h]);
    load_elems<bf16, 4>(h0 + G * kD + lane * 4, phi[G]);
    load_elems<bf16, 4>(h0 + (G + 1) * kD + lane * 4, ve);
    warp_phi_multi<G + 1>(phi);
    phi_ready = true;
  };

  // ---- window tile ------------------------------------------------------------------------------
  auto consume_window = [&](int wtile, uint32_t stage_addr) {
    const uint32_t Kst = stage_addr, Vst = stage_addr + kTileKV;
    const int slot0 = wtile * kTileRows;
    const bool ragged = slot0 + kTileRows > win_end || (win_cur >= slot0 && win_cur < slot0 + kTileRows);
    if (ragged) {   // rows that are not window tokens get zero V so that 0 * garbage cannot make a NaN
      for (int r = 0; r < kTileRows; ++r) {
        const int s = slot0 + r;
        if ((s >= win_end || s == win_cur) && lane < 16)
          *reinterpret_cast<uint4 *>(__cvta_shared_to_generic(Vst + (lane >> 3) * kBoxBytes + r * 128 + (lane & 7) * 16)) =
              make_uint4(0u, 0u, 0u, 0u);
      }
      fence_async_smem();   // these generic-proxy writes precede the next async-proxy fill of the stage
      __syncwarp();
    }
    float s[4] = {0.f, 0.f, 0.f, 0.f}, s2[4] = {0.f, 0.f, 0.f, 0.f};   // two chains over the feature dimension
    {
      const int r = (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
      for (int ks = 0; ks < KS; ks += 2) {
        const int c = (ks & 3) * 2 + (lane >> 4);
        uint32_t af[4], ag[4];
        ldmatrix_x4(af, Kst + (ks >> 2) * kBoxBytes + r * 128 + ((c ^ (r & 7)) << 4));
        ldmatrix_x4(ag, Kst + (ks >> 2) * kBoxBytes + r * 128 + (((c + 2) ^ (r & 7)) << 4));
        mma_bf16(s, af, qb[ks]);
        mma_bf16(s2, ag, qb[ks + 1]);
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) s[i] = (s[i] + s2[i]) * p.scale_log2;
    if (ragged) {
      const int k0 = slot0 + hrow, k1 = k0 + 8;
      if (k0 >= win_end || k0 == win_cur) s[0] = s[1] = -CUDART_INF_F;
      if (k1 >= win_end || k1 == win_cur) s[2] = s[3] = -CUDART_INF_F;
    }
    const float mx0 = quad_col_max(fmaxf(s[0], s[2]));
    const float mx1 = quad_col_max(fmaxf(s[1], s[3]));
    const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
    if (mn0 != m0 || mn1 != m1) {   // lanes of one head column agree; columns may diverge
      const float c0 = mn0 == -CUDART_INF_F ? 1.f : ex2_approx(m0 - mn0);
      const float c1 = mn1 == -CUDART_INF_F ? 1.f : ex2_approx(m1 - mn1);
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
    __syncwarp();
    const float ms0 = m0 == -CUDART_INF_F ? 0.f : m0, ms1 = m1 == -CUDART_INF_F ? 0.f : m1;
    float p0, p1, p2, p3;
    uint32_t pb[2];
    pb[0] = pack_bf16(ex2_approx(s[0] - ms0), ex2_approx(s[1] - ms1), p0, p1);
    pb[1] = pack_bf16(ex2_approx(s[2] - ms0), ex2_approx(s[3] - ms1), p2, p3);
    l0 += p0 + p2;   // the row sum uses the weights as the tensor core sees them
    l1 += p1 + p3;
    pb[0] = movmatrix_trans(pb[0]);
    pb[1] = movmatrix_trans(pb[1]);
    {
      const int j = lane >> 3;
      const int r = (lane & 7) + (j >> 1) * 8;
#pragma unroll
      for (int mt = 0; mt < KS; ++mt) {
        const int c = (mt & 3) * 2 + (j & 1);
        uint32_t af[4];
        ldmatrix_x4_trans(af, Vst + (mt >> 2) * kBoxBytes + r * 128 + ((c ^ (r & 7)) << 4));
        mma_bf16(o[mt], af, pb);
      }
    }
  };

  // ---- state tile: 16 rows of S and z, updated in place and read out ------------------------------
  auto consume_state = [&](const StreamSegment &sg, int stile, const float4 *st, const float *zs) {
    float *Sg = reinterpret_cast<float *>(p.ws + size_t(sg.S_off256) * 256) + size_t(stile) * kTileRows * kD;
    float *zg = reinterpret_cast<float *>(p.ws + size_t(sg.z_off256) * 256) + stile * kTileRows;
    const int src0 = stile * 4;   // lane that holds phi entries of the tile's first row (4 rows per lane)
#pragma unroll
    for (int r = 0; r < kTileRows; ++r) {
      float4 s = st[r * (kD / 4) + lane];
      const float pk = __shfl_sync(0xffffffffu, phi[G][r & 3], src0 + (r >> 2));
      s.x = fmaf(pk, ve[0], s.x);
      s.y = fmaf(pk, ve[1], s.y);
      s.z = fmaf(pk, ve[2], s.z);
      s.w = fmaf(pk, ve[3], s.w);
      *reinterpret_cast<float4 *>(Sg + r * kD + lane * 4) = s;
#pragma unroll
      for (int h = 0; h < G; ++h) {
        const float f = __shfl_sync(0xffffffffu, phi[h][r & 3], src0 + (r >> 2));
        a[h].x = fmaf(f, s.x, a[h].x);
        a[h].y = fmaf(f, s.y, a[h].y);
        a[h].z = fmaf(f, s.z, a[h].z);
        a[h].w = fmaf(f, s.w, a[h].w);
      }
    }
    // z: lane r < 16 owns row r of the tile
    const int zsrc = src0 + ((lane & 15) >> 2);
    float zn = 0.f;
#pragma unroll
    for (int h = 0; h <= G; ++h) {
      float f = 0.f;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float v = __shfl_sync(0xffffffffu, phi[(h + G) % (G + 1)][j], zsrc);   // phi(k_e) first, then the heads
        if ((lane & 3) == j) f = v;
      }
      if (h == 0) {
        if (lane < 16) {
          zn = zs[lane] + f;
          zg[lane] = zn;
        }
      } else if (lane < 16) {
        bp[h - 1] = fmaf(f, zn, bp[h - 1]);
      }
    }
    had_state = true;
  };

  // ---- end of a segment: reduce the 8 warps, finish or hand over the unit -----------------------------
  auto flush = [&](int s) {
    GLIDE_TRACE_EVENT(6);
    const StreamSegment &sg = sm_segs[s];
    float *rec = sm_rec + warp * L::kRecFloats;
    const bool mine = acc_seg == s;
    // 1. this warp's record (m, l, acc) in shared memory
    if (mine) {
      const float lq0 = quad_col_sum(l0), lq1 = quad_col_sum(l1);
#pragma unroll
      for (int mt = 0; mt < KS; ++mt) {
        const int d0 = mt * 16 + hrow;
        if (col2 < G) {
          rec[col2 * kD + d0] = o[mt][0];
          rec[col2 * kD + d0 + 8] = o[mt][2];
        }
        if (col2 + 1 < G) {
          rec[(col2 + 1) * kD + d0] = o[mt][1];
          rec[(col2 + 1) * kD + d0 + 8] = o[mt][3];
        }
      }
      if (hrow == 0) {
        if (col2 < G) {
          rec[G * kD + col2] = m0;
          rec[G * kD + G + col2] = lq0;
        }
        if (col2 + 1 < G) {
          rec[G * kD + col2 + 1] = m1;
          rec[G * kD + G + col2 + 1] = lq1;
        }
      }
      __syncwarp();
      if (had_state) {   // fold the linear readout in as a term with logit 0
        float mh[G], lh[G], bs[G];
#pragma unroll
        for (int h = 0; h < G; ++h) {
          mh[h] = rec[G * kD + h];
          lh[h] = rec[G * kD + G + h];
          bs[h] = bp[h];
        }
#pragma unroll
        for (int o2 = 16; o2 > 0; o2 >>= 1)
#pragma unroll
          for (int h = 0; h < G; ++h) bs[h] += __shfl_xor_sync(0xffffffffu, bs[h], o2);
        __syncwarp();
#pragma unroll
        for (int h = 0; h < G; ++h) {
          const float mn = fmaxf(mh[h], 0.f);
          const float fo = exp2_or_zero(mh[h], mn), fl = ex2_approx(-mn);
          float4 *ap = reinterpret_cast<float4 *>(rec + h * kD + lane * 4);
          float4 v = *ap;
          v.x = fmaf(v.x, fo, a[h].x * fl);
          v.y = fmaf(v.y, fo, a[h].y * fl);
          v.z = fmaf(v.z, fo, a[h].z * fl);
          v.w = fmaf(v.w, fo, a[h].w * fl);
          *ap = v;
          if (lane == 0) {
            rec[G * kD + h] = mn;
            rec[G * kD + G + h] = fmaf(lh[h], fo, bs[h] * fl);
          }
        }
      }
    } else {
      for (int i = lane; i < G * kD; i += 32) rec[i] = 0.f;
      if (lane < G) {
        rec[G * kD + lane] = -CUDART_INF_F;
        rec[G * kD + G + lane] = 0.f;
      }
    }
    // the current token's own logit, one head per warp (needed by whoever finishes the unit)
    const unsigned char *hdr = sm_hdr + size_t(s % kHdrSlots) * L::kHdrBytes;
    const bool has_win = sg.cap > 0;
    if (warp < G && has_win) {
      if (!mine) wait_header(s);
      float qx[4], kx[4];
      load_elems<bf16, 4>(reinterpret_cast<const bf16 *>(hdr) + warp * kD + lane * 4, qx);
      load_elems<bf16, 4>(reinterpret_cast<const bf16 *>(hdr + G * 256 + 512) + lane * 4, kx);
      float part = 0.f;
#pragma unroll
      for (int i = 0; i < 4; ++i) part = fmaf(qx[i], kx[i], part);
      part = warp_sum(part) * p.scale_log2;
      if (lane == 0) sm_scur[warp] = part;
    }
    __syncthreads();   // A: records and logits visible
    if (tid == 0 && s + 2 < nseg) issue_header(s + 2);   // slot of segment s-1, fully consumed before A

    // 2. combine the 8 records: thread owns VPT consecutive features of one head
    const int idx0 = tid * VPT;
    const bool active = idx0 < G * kD;
    const int h = active ? idx0 / kD : 0, c = idx0 - h * kD;
    float M = -CUDART_INF_F, lsum = 0.f, val[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) val[i] = 0.f;
    if (active) {
      float mw[kWarps];
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {
        mw[w] = sm_rec[w * L::kRecFloats + G * kD + h];
        M = fmaxf(M, mw[w]);
      }
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {
        const float *r = sm_rec + w * L::kRecFloats;
        const float f = exp2_or_zero(mw[w], M);
        lsum = fmaf(r[G * kD + G + h], f, lsum);
#pragma unroll
        for (int i = 0; i < VPT; ++i) val[i] = fmaf(r[idx0 + i], f, val[i]);
      }
    }
    const int ub = sg.unit - sg.layer * units_per_layer;
    const int b = ub / p.Hkv, g = ub - b * p.Hkv;
    float scur_all[G];   // warp 0 may finish the unit after barrier B, when sm_scur is being rewritten
#pragma unroll
    for (int hh = 0; hh < G; ++hh) scur_all[hh] = has_win ? sm_scur[hh] : -CUDART_INF_F;

    if (sg.part < 0) {
      // the whole unit lives in this CTA: add the current token, normalise, write, append to the ring
      if (active) {
        float sc = -CUDART_INF_F;
#pragma unroll
        for (int hh = 0; hh < G; ++hh)
          if (hh == h) sc = scur_all[hh];
        const float Mf = fmaxf(fmaxf(M, sc), 0.f);
        const float fr = exp2_or_zero(M, Mf), fc = exp2_or_zero(sc, Mf);
        const float inv = 1.0f / fmaf(lsum, fr, fc);
        const bf16 *vt = reinterpret_cast<const bf16 *>(hdr + G * 256 + 768);
        const int head = p.heads_of[g * G + h];
        bf16 *op = reinterpret_cast<bf16 *>(p.out) + ((size_t(sg.layer) * p.B + b) * p.H + head) * kD + c;
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
          const float num = fmaf(val[i], fr, has_win ? fc * __bfloat162float(vt[c + i]) : 0.f);
          op[i] = __float2bfloat16_rn(num * inv);
        }
      }
      if (has_win && tid < 128) {   // bit copy of the new k,v rows into slot t mod cap
        const LayerDev &ld = p.layers[sg.layer];
        const size_t row = (size_t(sg.row_base) + size_t(t % int64_t(sg.cap))) * kD;
        const uint32_t *srcw = reinterpret_cast<const uint32_t *>(hdr + G * 256 + 512);   // k_t (64 words) | v_t (64 words)
        uint32_t *dstw = reinterpret_cast<uint32_t *>(reinterpret_cast<bf16 *>(p.ws + (tid < 64 ? ld.ringK : ld.ringV)) + row);
        dstw[tid & 63] = srcw[tid];
      }
    } else if (active) {
      // unit cut by a CTA boundary: one global record per CTA
      float *grec = p.partials + (size_t(sg.rec0) + sg.part) * p.rec_floats;
#pragma unroll
      for (int i = 0; i < VPT; ++i) grec[idx0 + i] = val[i];
      if (c == 0) {
        grec[G * kD + h] = M;
        grec[G * kD + G + h] = lsum;
      }
    }
    __syncthreads();   // B: record area and logits may be rewritten; the CTA's global record is complete

    if (sg.part >= 0 && warp == 0) {
      // Warp 0 takes the unit's ticket while the other warps go on; the last ticket merges the few records.
      int last = 0;
      if (lane == 0) {
        __threadfence();
        last = atomicAdd(&p.tickets[sg.unit], 1) == sg.n_parts - 1;
      }
      last = __shfl_sync(0xffffffffu, last, 0);
      if (last) {
        __threadfence();
        const float *r0 = p.partials + size_t(sg.rec0) * p.rec_floats;
        const bf16 *vt = reinterpret_cast<const bf16 *>(hdr + G * 256 + 768);
#pragma unroll
        for (int hh = 0; hh < G; ++hh) {
          float Mg = fmaxf(scur_all[hh], 0.f);
          for (int i = 0; i < sg.n_parts; ++i) Mg = fmaxf(Mg, __ldcg(r0 + size_t(i) * p.rec_floats + G * kD + hh));
          float lg = 0.f;
          float4 vg = make_float4(0.f, 0.f, 0.f, 0.f);
          for (int i = 0; i < sg.n_parts; ++i) {
            const float *r = r0 + size_t(i) * p.rec_floats;
            const float f = exp2_or_zero(__ldcg(r + G * kD + hh), Mg);
            lg = fmaf(__ldcg(r + G * kD + G + hh), f, lg);
            const float4 av = __ldcg(reinterpret_cast<const float4 *>(r + hh * kD + lane * 4));
            vg.x = fmaf(av.x, f, vg.x);
            vg.y = fmaf(av.y, f, vg.y);
            vg.z = fmaf(av.z, f, vg.z);
            vg.w = fmaf(av.w, f, vg.w);
          }
          const float fc = exp2_or_zero(scur_all[hh], Mg);
          const float inv = 1.0f / (lg + fc);
          float vx[4] = {0.f, 0.f, 0.f, 0.f};
          if (has_win) load_elems<bf16, 4>(vt + lane * 4, vx);
          const int head = p.heads_of[g * G + hh];
          const __nv_bfloat162 lo = __floats2bfloat162_rn(fmaf(fc, vx[0], vg.x) * inv, fmaf(fc, vx[1], vg.y) * inv);
          const __nv_bfloat162 hi = __floats2bfloat162_rn(fmaf(fc, vx[2], vg.z) * inv, fmaf(fc, vx[3], vg.w) * inv);
          uint2 packed;
          packed.x = *reinterpret_cast<const uint32_t *>(&lo);
          packed.y = *reinterpret_cast<const uint32_t *>(&hi);
          *reinterpret_cast<uint2 *>(reinterpret_cast<bf16 *>(p.out) + ((size_t(sg.layer) * p.B + b) * p.H + head) * kD + lane * 4) = packed;
        }
        if (has_win) {
          const LayerDev &ld = p.layers[sg.layer];
          const size_t row = (size_t(sg.row_base) + size_t(t % int64_t(sg.cap))) * kD;
          const uint2 *srcw = reinterpret_cast<const uint2 *>(hdr + G * 256 + 512);
          reinterpret_cast<uint2 *>(reinterpret_cast<bf16 *>(p.ws + ld.ringK) + row)[lane] = srcw[lane];
          reinterpret_cast<uint2 *>(reinterpret_cast<bf16 *>(p.ws + ld.ringV) + row)[lane] = srcw[32 + lane];
        }
        if (lane == 0) p.tickets[sg.unit] = 0;
      }
    }
    GLIDE_TRACE_EVENT(7);
  };

  // ---- main loop --------------------------------------------------------------------------------------
  Cursor ccur;
  ccur.i = warp;
  ccur.seg = 0;
  ccur.tile_end = 0;
  if (nseg > 0) cursor_load(ccur, sm_segs, t);
  int next_flush = 0;
  TileRef ref;
  while (next_tile(ccur, sm_segs, nseg, ntiles, t, ref)) {
    while (next_flush < ref.seg) flush(next_flush++);
    if (acc_seg != ref.seg) load_unit(ref.seg);
    if (ref.is_state && !phi_ready) load_phi(ref.seg);
    if (!failed && !mbar_wait(my_bars + stage * 8, (phases >> stage) & 1u)) failed = true;
    phases ^= 1u << stage;
    failed = __any_sync(0xffffffffu, failed);
    GLIDE_TRACE_EVENT(ref.is_state ? 4 : 3);
    if (!failed) {
      if (ref.is_state)
        consume_state(sm_segs[ref.seg], ref.index, reinterpret_cast<const float4 *>(my_stages_ptr + stage * kStageBytes),
                      my_z_ptr + stage * 16);
      else
        consume_window(ref.index, my_stages + stage * kStageBytes);
    }
    stage = stage + 1 == STAGES ? 0 : stage + 1;
    __syncwarp();   // every lane is done with the stage before it is refilled
    if (!failed) issue_next();
    GLIDE_TRACE_EVENT(5);
  }
  while (next_flush < nseg) flush(next_flush++);
  if (failed && lane == 0) atomicExch(&p.ctl->status, kDevWaitTimeout);
  GLIDE_TRACE_EVENT(9);

  __syncthreads();
  if (tid == 0) {
    __threadfence();
    if (atomicAdd(&p.ctl->done_counter, 1) == int(gridDim.x) - 1) {
      p.ctl->work_counter = 0;
      p.ctl->done_counter = 0;
      for (int l = 0; l < p.L; ++l) p.n_dev[l] += 1;
      __threadfence();
    }
  }
}

template <int G, int STAGES>
size_t stream_smem_bytes(int max_segs) {
  using L = Layout<G>;
  return 1024 + size_t(kWarps) * STAGES * kStageBytes + size_t(kWarps) * L::kRecFloats * 4 + size_t(kHdrSlots) * L::kHdrBytes +
         size_t(kWarps) * STAGES * 64 + size_t(max_segs) * sizeof(StreamSegment) + size_t(kWarps * STAGES + kHdrSlots) * 8 +
         8 * 4;
}

template <typename F>
int dispatch_stream(int G, F &&f) {
  switch (G) {
    case 1: return f(IntTag<1>{}, IntTag<3>{});
    case 2: return f(IntTag<2>{}, IntTag<3>{});
    case 4: return f(IntTag<4>{}, IntTag<3>{});
    case 8: return f(IntTag<8>{}, IntTag<2>{});
    default: return int(GLIDE_ERR_UNSUPPORTED);
  }
}

}  // namespace

// Cuts the tile stream into `n_ctas` equally heavy ranges (state tiles weigh 2: read + write).
void build_stream_schedule(const glide_ctx *ctx, int n_ctas, std::vector<StreamSegment> *segs,
                           std::vector<int32_t> *cta_seg_begin, int *max_segs_per_cta, size_t *n_records) {
  const int L = ctx->cfg.n_layers, B = ctx->cfg.batch, Hkv = ctx->cfg.n_kv_heads, d = ctx->cfg.head_dim;
  const int64_t units_per_layer = int64_t(B) * Hkv;
  struct UnitTiles {
    int layer, unit;
    int n_state, n_win;
  };
  std::vector<int> order(L);
  for (int l = 0; l < L; ++l) order[l] = l;
  auto layer_weight = [&](int l) -> int64_t {
    const LayerDev &ld = ctx->layers[l];
    return (ld.evicts ? 2 * int64_t(d / kTileRows) : 0) + (ld.cap + kTileRows - 1) / kTileRows;
  };
  std::stable_sort(order.begin(), order.end(), [&](int x, int y) { return layer_weight(x) > layer_weight(y); });
  std::vector<UnitTiles> units;
  int64_t total_w = 0;
  for (int l : order) {
    const LayerDev &ld = ctx->layers[l];
    for (int64_t u = 0; u < units_per_layer; ++u) {
      UnitTiles ut{l, int(int64_t(l) * units_per_layer + u), ld.evicts ? d / kTileRows : 0,
                   int((ld.cap + kTileRows - 1) / kTileRows)};
      units.push_back(ut);
      total_w += 2 * int64_t(ut.n_state) + ut.n_win;
    }
  }
  segs->clear();
  cta_seg_begin->assign(size_t(n_ctas) + 1, 0);
  *max_segs_per_cta = 0;
  size_t records = 0;
  // walk the stream; CTA c takes tiles while the cumulative weight stays below (c+1) * total / n_ctas
  size_t ui = 0;
  int st_done = 0, win_done = 0;   // progress inside units[ui]
  int64_t cum = 0;
  std::vector<std::vector<size_t>> unit_segs(units.size());
  for (int c = 0; c < n_ctas; ++c) {
    (*cta_seg_begin)[c] = int32_t(segs->size());
    const int64_t target = (c + 1 == n_ctas) ? total_w : (total_w * (c + 1) + n_ctas - 1) / n_ctas;
    int tile0 = 0;
    while (ui < units.size() && cum < target) {
      const UnitTiles &ut = units[ui];
      const LayerDev &ld = ctx->layers[ut.layer];
      int64_t room = target - cum;
      StreamSegment sg{};
      sg.unit = ut.unit;
      sg.layer = ut.layer;
      sg.tile0 = tile0;
      sg.state0 = st_done;
      sg.n_state = int(std::min<int64_t>(ut.n_state - st_done, (room + 1) / 2));
      room -= 2 * int64_t(sg.n_state);
      sg.win0 = win_done;
      sg.n_win = (st_done + sg.n_state == ut.n_state) ? int(std::min<int64_t>(ut.n_win - win_done, std::max<int64_t>(room, 0))) : 0;
      if (sg.n_state == 0 && sg.n_win == 0 && (ut.n_state - st_done > 0 || ut.n_win - win_done > 0)) break;   // range full
      const int64_t ub = ut.unit - int64_t(ut.layer) * units_per_layer;
      sg.row_base = int32_t(ub * ld.cap);
      sg.cap = int32_t(ld.cap);
      sg.w = int32_t(std::min<int64_t>(ld.w, INT32_MAX));
      sg.evicts = ld.evicts;
      sg.S_off256 = int32_t((ld.S + size_t(ub) * d * d * 4) / 256);
      sg.z_off256 = int32_t((ld.z + size_t(ub) * d * 4) / 256);
      st_done += sg.n_state;
      win_done += sg.n_win;
      cum += 2 * int64_t(sg.n_state) + sg.n_win;
      tile0 += sg.n_state + sg.n_win;
      unit_segs[ui].push_back(segs->size());
      segs->push_back(sg);
      if (st_done == ut.n_state && win_done == ut.n_win) {
        ++ui;
        st_done = win_done = 0;
      }
    }
    *max_segs_per_cta = std::max<int>(*max_segs_per_cta, int(segs->size()) - (*cta_seg_begin)[c]);
  }
  (*cta_seg_begin)[n_ctas] = int32_t(segs->size());
  for (size_t u = 0; u < units.size(); ++u) {
    const std::vector<size_t> &list = unit_segs[u];
    if (list.size() == 1) {
      (*segs)[list[0]].part = -1;
      (*segs)[list[0]].n_parts = 1;
      (*segs)[list[0]].rec0 = 0;
    } else {
      for (size_t i = 0; i < list.size(); ++i) {
        (*segs)[list[i]].part = int32_t(i);
        (*segs)[list[i]].n_parts = int32_t(list.size());
        (*segs)[list[i]].rec0 = int32_t(records);
      }
      records += list.size();
    }
  }
  *n_records = records;
}

int stream_decode_supported(const glide_ctx *ctx) {
  return ctx->cfg.io_dtype == GLIDE_BF16 && ctx->cfg.head_dim == kD;
}

int stream_decode_setup(glide_ctx *ctx) {
  const int n_ctas = ctx->sm_count;
  int max_segs = 0;
  size_t n_records = 0;
  build_stream_schedule(ctx, n_ctas, &ctx->stream_segs, &ctx->stream_cta_begin, &max_segs, &n_records);
  ctx->stream_max_segs = std::max(max_segs, 1);
  if (ctx->stream_segs.size() > ctx->stream_seg_capacity || n_records > ctx->stream_rec_capacity) return GLIDE_ERR_UNSUPPORTED;
  bool contiguous = true;
  for (int g = 0; g < ctx->cfg.n_kv_heads; ++g)
    for (int i = 1; i < ctx->G; ++i)
      contiguous = contiguous && ctx->heads_of[size_t(g) * ctx->G + i] == ctx->heads_of[size_t(g) * ctx->G] + i;
  ctx->stream_heads_contiguous = contiguous;
  return dispatch_stream(ctx->G, [&](auto gg, auto ss) -> int {
    constexpr int G = decltype(gg)::value, S = decltype(ss)::value;
    const size_t smem = stream_smem_bytes<G, S>(ctx->stream_max_segs);
    int dev_max = 0;
    if (cudaDeviceGetAttribute(&dev_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, ctx->device) != cudaSuccess) {
      cudaGetLastError();
      return GLIDE_ERR_CUDA;
    }
    if (smem > size_t(dev_max)) return GLIDE_ERR_UNSUPPORTED;   // too many segments per CTA for the table
    auto kern = glide_decode_stream_kernel<G, S>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess) {
      cudaGetLastError();
      return GLIDE_ERR_CUDA;
    }
    ctx->stream_smem = smem;
    ctx->decode_grid = n_ctas;
    return GLIDE_OK;
  });
}

#ifdef GLIDE_TRACE
extern "C" int glide_debug_set_stream_trace(void *dev_buf) {
  return cudaMemcpyToSymbol(g_stream_trace, &dev_buf, sizeof(void *)) == cudaSuccess ? 0 : 6;
}
#endif

int launch_decode_stream(glide_ctx *ctx, const DecodeParams &p, cudaStream_t stream) {
  StreamParams sp{};
  sp.segs = reinterpret_cast<const StreamSegment *>(ctx->ws + ctx->off_stream_segs);
  sp.cta_seg_begin = reinterpret_cast<const int32_t *>(ctx->ws + ctx->off_stream_cta);
  sp.tmaps = reinterpret_cast<const CUtensorMap_st *>(ctx->ws + ctx->off_tmaps);
  sp.max_segs = ctx->stream_max_segs;
  sp.heads_contiguous = ctx->stream_heads_contiguous ? 1 : 0;
  sp.kv4d = ctx->tmaps_kv4d ? 1 : 0;
  return dispatch_stream(ctx->G, [&](auto gg, auto ss) -> int {
    constexpr int G = decltype(gg)::value, S = decltype(ss)::value;
    glide_decode_stream_kernel<G, S><<<ctx->decode_grid, kThreads, ctx->stream_smem, stream>>>(p, sp);
    if (cudaGetLastError() != cudaSuccess) return GLIDE_ERR_CUDA;
    return GLIDE_OK;
  });
}

}  // namespace glide
