// Fused GLIDE decode step for bf16, head_dim 128: statically scheduled streaming kernel (sm_100a).
//
// The step's whole traffic is laid out as one stream of equal-sized tiles, unit after unit
// (unit = layer x sequence x KV head, largest first):
//   state tile  -- 16 rows of the unit's S (8 KiB fp32) plus the 16 matching z entries,
//   window tile -- 16 ring slots: a 16x128 bf16 K box and V box (8 KiB).
// The host cuts the stream into one contiguous, equally heavy range per WARP (8 warps per CTA, one
// CTA per SM) and describes each range by a short segment list (one segment per unit it touches).
// A warp is an autonomous worker: it owns a ring of TMA stages and keeps it full ACROSS unit
// boundaries (lane 0 issues cp.async.bulk / cp.async.bulk.tensor loads as stages drain), and a small
// header buffer into which the next unit's q rows, evicted k/v rows and current k/v rows are
// prefetched while the current unit streams.  There is no CTA-wide barrier after set-up.
//   window tile: S = K_tile Q^T on the tensor cores (keys on M, query heads on N), online softmax
//                in the log2 domain, P transposed in registers, O^T += V_tile^T P;
//   state tile:  S += phi(k_e) v_e^T and z += phi(k_e) in place (fp32), readout phi(q_h)^T S, phi(q_h)^T z.
// The linear readout is folded into the softmax partial as a term with logit 0 (exact: the shared
// normaliser's reference m* is max(window max, 0)), so a unit needs ONE (m, l, acc) record per warp.
// A unit that lies inside one warp's range is finished by that warp alone (current token's own term,
// normalise, write, ring append) without touching global scratch.  Units shared by warps of one CTA are
// reduced in shared memory by the last of them to arrive.  Only units cut by a CTA boundary go through global
// scratch: one record per CTA, every value stored beside the launch's tag in one 8-byte word, and a ticket per
// unit taken with a relaxed atomic (no fence between the record and the ticket: the tags say when a value has
// arrived).  The warp that draws a unit's last ticket merges the records at the end of its range, polling the
// words it is about to use until they carry the tag: every one of them has been stored by then, so the poll
// never waits for a CTA that is not running.  Like the waits on the warp's own mbarriers it is bounded, and a
// wait that runs out sets the context's status word.
#include <cuda.h>

#include <algorithm>

#include "glide_device.cuh"
#include "glide_trace.cuh"

namespace glide {

namespace {

constexpr int kD = 128;
constexpr int kWarps = kStreamWarps;
constexpr int kThreads = kWarps * 32;
constexpr int kTileRows = 16;
constexpr uint32_t kStageBytes = 2 * kTileRows * kD * 2;   // 8 KiB: K box + V box, or 16 fp32 state rows
constexpr uint32_t kBoxBytes = kTileRows * 128;            // one 64-column TMA box
constexpr uint32_t kTileKV = 2 * kBoxBytes;                // K (or V) part of a window stage
constexpr uint32_t kWaitLimit = 1u << 24;
constexpr int kHdrSlots = 3;
#ifndef GLIDE_STREAM_STAGES
#define GLIDE_STREAM_STAGES 2
#endif
// schedule weights: cost of a state tile, a window tile and of starting a unit in a range
#ifndef GLIDE_W_STATE
#define GLIDE_W_STATE 15
#define GLIDE_W_WIN 10
#define GLIDE_W_UNIT 27
#endif
#ifndef GLIDE_STREAM_MAX_PARTS
#define GLIDE_STREAM_MAX_PARTS 8
#endif
#ifndef GLIDE_W_GROUP
#define GLIDE_W_GROUP 0   // extra weight of a segment whose unit is shared with other warps of the CTA
#endif
#ifndef GLIDE_STREAM_FILL
#define GLIDE_STREAM_FILL 100
#endif
#ifndef GLIDE_STREAM_TMAP_PREFETCH
#define GLIDE_STREAM_TMAP_PREFETCH 1
#endif
#ifndef GLIDE_W_MIN_CTA
#define GLIDE_W_MIN_CTA 128   // least weight worth a CTA of its own (about ten tiles)
#endif
#ifndef GLIDE_W_EDGE
#define GLIDE_W_EDGE 40
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
__device__ __forceinline__ void bulk_store(void *dst, uint32_t src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
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
__device__ __forceinline__ void prefetch_tensormap(const void *tmap) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(tmap) : "memory");
}
// ---- records of units cut across CTAs: every 4-byte value travels with the launch's tag in one 8-byte store ------
// A 64-bit store is a single access, so a reader that sees the tag sees the value: no fence orders the record
// before the unit's ticket: whoever draws the last ticket polls the pairs it is about to use.
__device__ __forceinline__ unsigned long long ll_pack(float v, uint32_t tag) {
  return (static_cast<unsigned long long>(tag) << 32) | __float_as_uint(v);
}
__device__ __forceinline__ void ll_store2(unsigned long long *dst, float a, float b, uint32_t tag) {   // dst 16-byte aligned
  asm volatile("st.relaxed.gpu.global.v2.u64 [%0], {%1, %2};" ::"l"(dst), "l"(ll_pack(a, tag)), "l"(ll_pack(b, tag)) : "memory");
}
__device__ __forceinline__ void ll_store1(unsigned long long *dst, float a, uint32_t tag) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(dst), "l"(ll_pack(a, tag)) : "memory");
}
__device__ __forceinline__ bool ll_load2(const unsigned long long *src, uint32_t tag, float &a, float &b) {
  unsigned long long x, y;
  asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(x), "=l"(y) : "l"(src) : "memory");
  a = __uint_as_float(uint32_t(x));
  b = __uint_as_float(uint32_t(y));
  return uint32_t(x >> 32) == tag && uint32_t(y >> 32) == tag;
}
__device__ __forceinline__ bool ll_load1(const unsigned long long *src, uint32_t tag, float &a) {
  unsigned long long x;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(x) : "l"(src) : "memory");
  a = __uint_as_float(uint32_t(x));
  return uint32_t(x >> 32) == tag;
}
// 8-byte load that stays where it is written (ahead of the polling loop it is meant to overlap with)
__device__ __forceinline__ uint2 ld_u2_pinned(const void *src) {
  uint2 v;
  asm volatile("ld.global.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(src));
  return v;
}
__device__ __forceinline__ bool ll_load4(const unsigned long long *src, uint32_t tag, float4 &v) {   // four consecutive pairs
  const bool a = ll_load2(src, tag, v.x, v.y);
  const bool b = ll_load2(src + 2, tag, v.z, v.w);
  return a && b;
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

// (PARKABLE: the launch has slot offsets, so a position may be negative = a parked slot; the instantiation for level
// batches carries none of the checks)
template <bool PARKABLE>
__device__ __forceinline__ bool seg_evicting(const StreamSegment &s, int64_t t) {
  // evicts bit 0: the layer has a state; bit 1: the token folded at a step is the current one (no ring, or a state
  // that holds every token), otherwise the one that leaves the window
  if (PARKABLE && t < 0) return false;
  return (s.evicts & 1) && ((s.evicts & 2) || t >= int64_t(s.w));
}
// window tiles of the segment that hold window tokens at position t
template <bool PARKABLE>
__device__ __forceinline__ int seg_valid_win(const StreamSegment &s, int64_t t) {
  if (PARKABLE && t < 0) return 0;
  const int64_t lim = t < int64_t(s.cap) ? t : int64_t(s.cap);
  const int nv = int((lim + kTileRows - 1) / kTileRows) - s.win0;
  return nv < 0 ? 0 : (nv > s.n_win ? s.n_win : nv);
}

// A position in the warp's range: segment, tile within the segment, and the segment's tile counts.
// ring slot of position t (t >= 0): 32-bit arithmetic while the position allows it (a 64-bit remainder is a call)
__device__ __forceinline__ int slot_of(int64_t t, int cap) {
  return t <= int64_t(0x7fffffff) ? int(uint32_t(t) % uint32_t(cap)) : int(t % int64_t(cap));
}

struct Cursor {
  int seg;
  int k;          // next tile of the segment: [0, n_state_eff) state tiles, then window tiles
  int n_state_eff, n_total;
};

template <bool PARKABLE>
__device__ __forceinline__ void cursor_enter(Cursor &c, const StreamSegment *segs, int64_t t) {
  const StreamSegment &s = segs[c.seg];
  c.k = 0;
  c.n_state_eff = seg_evicting<PARKABLE>(s, t) ? s.n_state : 0;
  c.n_total = c.n_state_eff + seg_valid_win<PARKABLE>(s, t);
}

// Records.  Shared normaliser: (acc[G][d], m[G], l[G]) with the linear readout already folded in as a term with
// logit 0.  Sum of two normalised terms (SUM): the window part as above and, kRecW floats further on, the linear
// part (a[G][d], b[G]) kept apart.
template <int G, bool SUM = false>
struct Layout {
  static constexpr int kRecW = (G * kD + 2 * G + 3) / 4 * 4;
  static constexpr int kRecFloats = SUM ? 2 * kRecW : kRecW;
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
      x[n][i] = ex2_approx((x[n][i] - mx[n]) * kLog2e);
      sm[n] += x[n][i];
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1)
#pragma unroll
    for (int n = 0; n < N; ++n) sm[n] += __shfl_xor_sync(0xffffffffu, sm[n], o);
#pragma unroll
  for (int n = 0; n < N; ++n) {
    const float inv = __frcp_rn(sm[n]);
#pragma unroll
    for (int i = 0; i < 4; ++i) x[n][i] *= inv;
  }
}

template <int N>
__device__ __forceinline__ void warp_sum_multi(float (&x)[N]) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1)
#pragma unroll
    for (int n = 0; n < N; ++n) x[n] += __shfl_xor_sync(0xffffffffu, x[n], o);
}

// ---- the kernel -----------------------------------------------------------------------------
// MODE bit 0: the sum of two normalised terms instead of the shared normaliser; bit 1: the learned feature map
// (feature dimension 2 kD: 16 state tiles per unit, and every state tile arrives with its 16 entries of phi(q_h) and
// of phi(k_e), which the feature kernel in front of this launch has written)
template <int G, int STAGES, int MODE, bool RAGGED>
__global__ void __launch_bounds__(kThreads, GLIDE_STREAM_CTAS_PER_SM)
glide_decode_stream_kernel(const DecodeParams p, const StreamParams sp) {
  using bf16 = __nv_bfloat16;
  constexpr bool SUM = (MODE & 1) != 0, PHI2 = (MODE & 2) != 0;
  constexpr int kPhiTile = (G + 1) * 16;   // floats of feature values per state tile
  using L = Layout<G, SUM>;
  constexpr int KS = kD / 16;

  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char *base = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char *sm_stages = base;                                                  // [kWarps][STAGES][8 KiB]
  unsigned char *sm_hdr = sm_stages + size_t(kWarps) * STAGES * kStageBytes;        // [kWarps][kHdrBytes]
  float *sm_z = reinterpret_cast<float *>(sm_hdr + kWarps * L::kHdrBytes);           // [kWarps][STAGES][16]
  StreamSegment *sm_segs = reinterpret_cast<StreamSegment *>(sm_z + kWarps * STAGES * 16);   // [max_segs]
  uint64_t *sm_bars = reinterpret_cast<uint64_t *>(sm_segs + sp.max_segs);          // [kWarps][STAGES + 1]
  int *sm_ctr = reinterpret_cast<int *>(sm_bars + kWarps * (STAGES + 1));             // [kStreamMaxGroups]
  float *sm_phi = reinterpret_cast<float *>(sm_ctr + kStreamMaxGroups);               // PHI2: [kWarps][STAGES][kPhiTile]
  float *sm_pool = sm_phi + (PHI2 ? kWarps * STAGES * kPhiTile : 0);                  // [pool slots][kRecFloats]
  int64_t *sm_t = reinterpret_cast<int64_t *>(base + sp.t_off);                       // [max_segs], behind the pool

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  GLIDE_TRACE_DECL;
  GLIDE_TRACE_EVENT(1);
  // Programmatic dependent launch: the next launch in the stream may start its prologue on SMs this grid has
  // left; whatever an earlier kernel wrote is read only after griddepcontrol.wait below.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int col2 = (lane & 3) * 2, hrow = lane >> 2;
  // the CTA's slice of the segment list: offsets come with the kernel parameters (no dependent global load)
  const int cta_seg_begin = sp.cta_seg_begin[blockIdx.x];
  const int cta_nseg = sp.cta_seg_begin[blockIdx.x + 1] - cta_seg_begin;
  if (cta_nseg > 0) {
    const uint4 *src = reinterpret_cast<const uint4 *>(sp.segs + cta_seg_begin);
    uint4 *dst = reinterpret_cast<uint4 *>(sm_segs);
    for (int i = tid; i < cta_nseg * int(sizeof(StreamSegment) / 16); i += kThreads) dst[i] = src[i];
  }
  unsigned char *my_stages_ptr = sm_stages + size_t(warp) * STAGES * kStageBytes;
  const uint32_t my_stages = smem_u32(my_stages_ptr);
  unsigned char *my_hdr_ptr = sm_hdr + size_t(warp) * L::kHdrBytes;
  const uint32_t my_hdr = smem_u32(my_hdr_ptr);
  float *my_z_ptr = sm_z + warp * STAGES * 16;
  const uint32_t my_z = smem_u32(my_z_ptr);
  float *my_phi_ptr = sm_phi + warp * STAGES * kPhiTile;
  const uint32_t my_phi = smem_u32(my_phi_ptr);
  const uint32_t my_bars = smem_u32(sm_bars + warp * (STAGES + 1));
  const uint32_t hdr_bar = my_bars + STAGES * 8;
  if (tid < kStreamMaxGroups) sm_ctr[tid] = 0;
  if (lane == 0) {
    for (int s = 0; s <= STAGES; ++s) mbar_init(my_bars + s * 8, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_async_smem();
  }
  __syncthreads();   // segment table and barriers ready
  // A sequence's position is the layers' common counter, which comes with the launch, plus the sequence's own offset
  // (zero unless sequences were reset or prefilled one by one; written by copies from the host, never by a kernel,
  // so it may be read before the preceding kernel has completed).  Level batches (RAGGED false: an instantiation of
  // its own, so that the B = 1 step carries none of this) take the position from the launch parameters.
  constexpr bool ragged = RAGGED;
  if (ragged) {
    for (int i = tid; i < cta_nseg; i += kThreads) sm_t[i] = p.t_host + p.seq_off[(sm_segs[i].unit / p.Hkv) % p.B];
    __syncthreads();
  }
  auto pos_of = [&](int s) -> int64_t { return ragged ? sm_t[s] : p.t_host; };
#if GLIDE_STREAM_TMAP_PREFETCH
  // the ring descriptors are written when the context is created, never by a kernel: fetch the ones this
  // CTA's segments use before waiting for the preceding kernel
  if (tid < cta_nseg && sm_segs[tid].cap > 0)
    prefetch_tensormap(reinterpret_cast<const CUtensorMap *>(sp.tmaps) + 3 * sm_segs[tid].layer + (sp.kv4d ? 2 : 0));
#endif
  asm volatile("griddepcontrol.wait;" ::: "memory");   // the preceding kernel has completed and its writes are visible
  // every layer is at the same position (checked by the host); the host's copy of the counter comes with the
  // launch, which saves a dependent global load at the head of every warp's critical path
  // the device counters are not read by this kernel; one thread moves them on (no grid-wide completion count,
  // which would put an atomic round trip at the end of every CTA)
  if (blockIdx.x == 0)
    for (int l = tid; l < p.layer_count; l += kThreads) p.n_dev[p.layer_begin + l] = p.t_host + 1;
  // this warp's segments: the run of the CTA's list that carries its index
  int seg_lo = 0;
  while (seg_lo < cta_nseg && sm_segs[seg_lo].range < warp) ++seg_lo;
  int seg_hi = seg_lo;
  while (seg_hi < cta_nseg && sm_segs[seg_hi].range == warp) ++seg_hi;

  bool failed = false;

  // ---- header of segment s (q rows | k_e | v_e | k_t | v_t) into this warp's buffer, lane 0 ---------
  auto issue_header = [&](int s) {
    if (lane == 0) {
      const StreamSegment &sg = sm_segs[s];
      const int64_t t = pos_of(s);
      const bool ev = seg_evicting<RAGGED>(sg, t);
      fence_async_smem();
      mbar_expect_tx(hdr_bar, G * 256 + 512 + (ev ? 512 : 0));
      const bf16 *qall = reinterpret_cast<const bf16 *>(p.q);
      if (sp.heads_contiguous) {
        bulk_load(my_hdr, qall + size_t(sg.qrow0) * kD, G * 256, hdr_bar);
      } else {
        for (int h = 0; h < G; ++h)
          bulk_load(my_hdr + h * 256, qall + (size_t(sg.qrow0) + p.heads_of[sg.g * G + h]) * kD, 256, hdr_bar);
      }
      const bf16 *kt = reinterpret_cast<const bf16 *>(p.k) + size_t(sg.unit) * kD;
      const bf16 *vt = reinterpret_cast<const bf16 *>(p.v) + size_t(sg.unit) * kD;
      bulk_load(my_hdr + G * 256 + 512, kt, 256, hdr_bar);
      bulk_load(my_hdr + G * 256 + 768, vt, 256, hdr_bar);
      if (ev) {
        if (sg.evicts & 2) {   // the current token is the one folded into the state
          bulk_load(my_hdr + G * 256, kt, 256, hdr_bar);
          bulk_load(my_hdr + G * 256 + 256, vt, 256, hdr_bar);
        } else {
          const size_t row = (size_t(sg.row_base) + size_t(slot_of(t, sg.cap))) * kD;
          bulk_load(my_hdr + G * 256, reinterpret_cast<const bf16 *>(p.ws + size_t(sg.ringK_off256) * 256) + row, 256, hdr_bar);
          bulk_load(my_hdr + G * 256 + 256, reinterpret_cast<const bf16 *>(p.ws + size_t(sg.ringV_off256) * 256) + row, 256, hdr_bar);
        }
      }
    }
  };

  // ---- tile issue (lane 0) ------------------------------------------------------------------------
  Cursor icur;
  icur.seg = seg_lo;
  icur.k = icur.n_state_eff = icur.n_total = 0;
  if (seg_lo < seg_hi) cursor_enter<RAGGED>(icur, sm_segs, pos_of(icur.seg));
  int issue_stage = 0;
  auto issue_next = [&]() {
    if (lane == 0) {
      while (icur.seg < seg_hi && icur.k >= icur.n_total) {
        if (++icur.seg < seg_hi) cursor_enter<RAGGED>(icur, sm_segs, pos_of(icur.seg));
      }
      if (icur.seg < seg_hi) {
        const StreamSegment &sg = sm_segs[icur.seg];
        const uint32_t bar = my_bars + issue_stage * 8;
        const uint32_t dst = my_stages + issue_stage * kStageBytes;
        GLIDE_CHECK_OR(icur.k < icur.n_state_eff ? (sg.state0 + icur.k) * kTileRows < kD
                                                 : (sg.win0 + icur.k - icur.n_state_eff) * kTileRows < sg.cap,
                       p.status, (void)0);
        if (icur.k < icur.n_state_eff) {
          const int st = sg.state0 + icur.k;
          mbar_expect_tx(bar, kStageBytes + 64 + (PHI2 ? kPhiTile * 4 : 0));
          const float *Sg = reinterpret_cast<const float *>(p.ws + size_t(sg.S_off256) * 256) + size_t(st) * kTileRows * kD;
          const float *zg = reinterpret_cast<const float *>(p.ws + size_t(sg.z_off256) * 256) + st * kTileRows;
          bulk_load(dst, Sg, kStageBytes, bar);
          bulk_load(my_z + issue_stage * 64, zg, 64, bar);
          if (PHI2)   // the tile's rows of phi(q_h), h < G, and of phi(k_e): [unit][tile][G + 1][16]
            bulk_load(my_phi + issue_stage * kPhiTile * 4,
                      p.phit + (size_t(sg.unit) * (2 * kD / kTileRows) + st) * kPhiTile, kPhiTile * 4, bar);
        } else {
          const int wt = sg.win0 + icur.k - icur.n_state_eff;
          mbar_expect_tx(bar, kStageBytes);
          const CUtensorMap *tk = reinterpret_cast<const CUtensorMap *>(sp.tmaps) + 3 * sg.layer;
          const int y = sg.row_base + wt * kTileRows;
          if (sp.kv4d) {
            tma_load_4d(dst, tk + 2, 0, y, 0, 0, bar);   // K halves then V halves: [kv][half][row][64]
          } else {
            tma_load_2d(dst, tk, 0, y, bar);
            tma_load_2d(dst + kBoxBytes, tk, 64, y, bar);
            tma_load_2d(dst + kTileKV, tk + 1, 0, y, bar);
            tma_load_2d(dst + kTileKV + kBoxBytes, tk + 1, 64, y, bar);
          }
        }
        ++icur.k;
        issue_stage = issue_stage + 1 == STAGES ? 0 : issue_stage + 1;
      }
    }
  };
  if (seg_lo < seg_hi) issue_header(seg_lo);   // small and needed first
  for (int s = 0; s < STAGES; ++s) issue_next();
  GLIDE_TRACE_EVENT(2);

  // ---- per-unit register state ------------------------------------------------------------------
  uint32_t qb[KS][2];
  float o[KS][4];
  float m0, m1, l0, l1;
  float phi[G + 1][4];     // phi(q_h) for the G heads, then phi(k_e); lane holds entries 4*lane .. 4*lane+3
  float ve[4];
  float gamma = 1.f;       // gated recurrence: gate of the token that enters the state at this step
  float4 a[G];
  float bp[G];
  float scur[G];           // the current token's own logit per head (log2 domain)
  uint2 kt_bits, vt_bits;  // the current token's k and v entries 4*lane .. 4*lane+3 (bf16)
  int win_end = 0, win_cur = 0;   // window tokens live in slots [0, win_end) except slot win_cur
  uint32_t phases = 0;     // parity expected by the next wait on each stage; bit STAGES: header barrier
  int stage = 0;
  int n_pending = 0, pend0 = 0, pend1 = 0;   // segments of this range whose unit is shared with a neighbour (at most two)
  unsigned tick0 = 0, tick1 = 0;             // their tickets (lane 0)

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

  // ---- state tile: 16 rows of S and z, updated in the stage and stored back by the async proxy ---------
  // (nothing later in the warp waits for these bulk stores except the wait for all of them before it exits)
  auto consume_state = [&](const StreamSegment &sg, int stile, float4 *st, float *zs, uint32_t st_addr, uint32_t z_addr,
                           const float *sphi) {
    const int src0 = stile * 4;   // lane that holds phi entries of the tile's first row (4 rows per lane)
#pragma unroll
    for (int r = 0; r < kTileRows; ++r) {
      float4 s = st[r * (kD / 4) + lane];
      const float pk = PHI2 ? sphi[G * 16 + r] : __shfl_sync(0xffffffffu, phi[G][r & 3], src0 + (r >> 2));
      s.x = fmaf(pk, ve[0], gamma * s.x);   // (gamma = 1 without gates: the product is exact)
      s.y = fmaf(pk, ve[1], gamma * s.y);
      s.z = fmaf(pk, ve[2], gamma * s.z);
      s.w = fmaf(pk, ve[3], gamma * s.w);
      st[r * (kD / 4) + lane] = s;
#pragma unroll
      for (int h = 0; h < G; ++h) {
        const float f = PHI2 ? sphi[h * 16 + r] : __shfl_sync(0xffffffffu, phi[h][r & 3], src0 + (r >> 2));
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
      if (PHI2) {
        f = sphi[((h + G) % (G + 1)) * 16 + (lane & 15)];
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float v = __shfl_sync(0xffffffffu, phi[(h + G) % (G + 1)][j], zsrc);   // phi(k_e) first, then the heads
          if ((lane & 3) == j) f = v;
        }
      }
      if (h == 0) {
        if (lane < 16) {
          zn = fmaf(gamma, zs[lane], f);
          zs[lane] = zn;
        }
      } else if (lane < 16) {
        bp[h - 1] = fmaf(f, zn, bp[h - 1]);
      }
    }
    fence_async_smem();   // the updated rows are read by the async proxy
    __syncwarp();
    if (lane == 0) {
      float *Sg = reinterpret_cast<float *>(p.ws + size_t(sg.S_off256) * 256) + size_t(stile) * kTileRows * kD;
      float *zg = reinterpret_cast<float *>(p.ws + size_t(sg.z_off256) * 256) + stile * kTileRows;
      bulk_store(Sg, st_addr, kStageBytes);
      bulk_store(zg, z_addr, 64);
      bulk_commit();
      bulk_wait_read0();   // the stage may be refilled once the store has read it
    }
  };

  // the record of the segment that has just finished (after the loop: of the range's last segment, which the merge
  // below takes from here instead of reading it back from global memory)
  float mh[G], lh[G];
  float4 acc[G];
  int own_seg = -1;   // segment whose global record these registers still hold
  // ---- main loop over this warp's segments ------------------------------------------------------------
  for (int s = seg_lo; s < seg_hi && !failed; ++s) {
    const StreamSegment &sg = sm_segs[s];
    const int64_t t = pos_of(s);
    const bool ev = seg_evicting<RAGGED>(sg, t);
    const int n_state_eff = ev ? sg.n_state : 0;
    const int n_total = n_state_eff + seg_valid_win<RAGGED>(sg, t);
    const bool has_win = sg.cap > 0;

    // -- header: q fragments, current token, feature maps -> registers; then prefetch the next header --
    GLIDE_TRACE_EVENT(6);
    gamma = 1.f;
    if (p.gated && n_state_eff > 0) {
      // the gate of the token that enters the state: the current token's (no ring, or a state that holds every
      // token), else the one waiting in the ring of gates beside the token that leaves the window
      if (sg.evicts & 2) {
        if (p.gate) gamma = p.gate[sg.unit];
      } else {
        gamma = reinterpret_cast<const float *>(p.ws + p.layers[sg.layer].ringG)[size_t(sg.row_base) + size_t(slot_of(t, sg.cap))];
      }
    }
    if (!mbar_wait(hdr_bar, (phases >> STAGES) & 1u)) failed = true;
    phases ^= 1u << STAGES;
    if (__any_sync(0xffffffffu, failed)) {
      failed = true;
      break;
    }
    {
      const uint32_t *hq = reinterpret_cast<const uint32_t *>(my_hdr_ptr);
      const bool valid = hrow < G;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        qb[ks][0] = valid ? hq[hrow * 64 + ks * 8 + (lane & 3)] : 0u;
        qb[ks][1] = valid ? hq[hrow * 64 + ks * 8 + 4 + (lane & 3)] : 0u;
      }
      const bf16 *h0 = reinterpret_cast<const bf16 *>(my_hdr_ptr);
      kt_bits = *reinterpret_cast<const uint2 *>(h0 + (G + 2) * kD + lane * 4);
      vt_bits = *reinterpret_cast<const uint2 *>(h0 + (G + 3) * kD + lane * 4);
      float kx[4];
      load_elems<bf16, 4>(h0 + (G + 2) * kD + lane * 4, kx);
#pragma unroll
      for (int h = 0; h < G; ++h) {
        load_elems<bf16, 4>(h0 + h * kD + lane * 4, phi[h]);
        scur[h] = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) scur[h] = fmaf(phi[h][i], kx[i], scur[h]);
      }
      warp_sum_multi<G>(scur);
#pragma unroll
      for (int h = 0; h < G; ++h) scur[h] = has_win ? scur[h] * p.scale_log2 : -CUDART_INF_F;
      if (n_state_eff > 0) {
        load_elems<bf16, 4>(h0 + (G + 1) * kD + lane * 4, ve);
        if (!PHI2) {   // (the learned map's features arrive with the state tiles)
          load_elems<bf16, 4>(h0 + G * kD + lane * 4, phi[G]);
          warp_phi_multi<G + 1>(phi);
        }
      }
    }
    __syncwarp();
    if (s + 1 < seg_hi) issue_header(s + 1);
    // A parked slot (negative position; only batches with slot offsets have them) goes through the header hand-over
    // like every segment and then leaves: it has no tiles, and nothing of it is reduced or written.  All segments
    // of a unit share the position, so its group counters and records stay untouched as well.
    if (RAGGED && t < 0) continue;
    if (has_win) {
      const int64_t lim = t < int64_t(sg.cap) ? t : int64_t(sg.cap);
      win_end = int(lim);
      win_cur = slot_of(t, sg.cap);
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

    // -- tiles ------------------------------------------------------------------------------------------
    int last_stage = -1;
    for (int k = 0; k < n_total; ++k) {
      if (!mbar_wait(my_bars + stage * 8, (phases >> stage) & 1u)) failed = true;
      phases ^= 1u << stage;
      if (__any_sync(0xffffffffu, failed)) {
        failed = true;
        break;
      }
      GLIDE_TRACE_EVENT(k < n_state_eff ? 4 : 3);
      if (k < n_state_eff)
        consume_state(sg, sg.state0 + k, reinterpret_cast<float4 *>(my_stages_ptr + stage * kStageBytes),
                      my_z_ptr + stage * 16, my_stages + stage * kStageBytes, my_z + stage * 64,
                      my_phi_ptr + stage * kPhiTile);
      else
        consume_window(sg.win0 + k - n_state_eff, my_stages + stage * kStageBytes);
      last_stage = stage;
      stage = stage + 1 == STAGES ? 0 : stage + 1;
      __syncwarp();   // every lane is done with the stage before it is refilled
      if (k + 1 < n_total) issue_next();   // the last tile's stage first serves as scratch for the finish
    }
    if (failed) break;
    // -- finish: record (m, l, acc) in a common layout: lane holds features 4*lane..4*lane+3 of every head --
    if (n_total > n_state_eff) {   // window tiles were processed: move the accumulator fragments through the freed stage
      float *scr = reinterpret_cast<float *>(my_stages_ptr + last_stage * kStageBytes);
      const float lq0 = quad_col_sum(l0), lq1 = quad_col_sum(l1);
#pragma unroll
      for (int mt = 0; mt < KS; ++mt) {
        const int d0 = mt * 16 + hrow;
        if (col2 < G) {
          scr[col2 * kD + d0] = o[mt][0];
          scr[col2 * kD + d0 + 8] = o[mt][2];
        }
        if (col2 + 1 < G) {
          scr[(col2 + 1) * kD + d0] = o[mt][1];
          scr[(col2 + 1) * kD + d0 + 8] = o[mt][3];
        }
      }
      if (hrow == 0) {
        if (col2 < G) {
          scr[G * kD + col2] = m0;
          scr[G * kD + G + col2] = lq0;
        }
        if (col2 + 1 < G) {
          scr[G * kD + col2 + 1] = m1;
          scr[G * kD + G + col2 + 1] = lq1;
        }
      }
      __syncwarp();
#pragma unroll
      for (int h = 0; h < G; ++h) {
        mh[h] = scr[G * kD + h];
        lh[h] = scr[G * kD + G + h];
        acc[h] = *reinterpret_cast<const float4 *>(scr + h * kD + lane * 4);
      }
      fence_async_smem();   // the stage is refilled by the async proxy next
      __syncwarp();
    } else {
#pragma unroll
      for (int h = 0; h < G; ++h) {
        mh[h] = -CUDART_INF_F;
        lh[h] = 0.f;
        acc[h] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    if (n_total > 0) issue_next();   // the deferred refill
    if (n_state_eff > 0) warp_sum_multi<G>(bp);
    if (!SUM && n_state_eff > 0) {   // fold the linear readout in as a term with logit 0
#pragma unroll
      for (int h = 0; h < G; ++h) {
        const float mn = fmaxf(mh[h], 0.f);
        const float fo = exp2_or_zero(mh[h], mn), fl = ex2_approx(-mn);
        acc[h].x = fmaf(acc[h].x, fo, a[h].x * fl);
        acc[h].y = fmaf(acc[h].y, fo, a[h].y * fl);
        acc[h].z = fmaf(acc[h].z, fo, a[h].z * fl);
        acc[h].w = fmaf(acc[h].w, fo, a[h].w * fl);
        lh[h] = fmaf(lh[h], fo, bp[h] * fl);
        mh[h] = mn;
      }
    }
    if (sg.grp_size > 1) {
      // several warps of this CTA share the unit: records meet in shared memory, the last one to arrive
      // combines them and carries the unit on
      float *slot = sm_pool + size_t(sg.grp_slot0 + sg.grp_idx) * L::kRecFloats;
#pragma unroll
      for (int h = 0; h < G; ++h) {
        *reinterpret_cast<float4 *>(slot + h * kD + lane * 4) = acc[h];
        if (SUM) *reinterpret_cast<float4 *>(slot + L::kRecW + h * kD + lane * 4) = a[h];
        if (lane == 0) {
          slot[G * kD + h] = mh[h];
          slot[G * kD + G + h] = lh[h];
          if (SUM) slot[L::kRecW + G * kD + h] = bp[h];
        }
      }
      __syncwarp();
      int lastc = 0;
      if (lane == 0) {
        // shared-memory accesses of one SM are performed in order: the record written above (ordered by the
        // __syncwarp) is visible to whichever warp sees this arrival
        // (a relaxed atomic: a fence here would also wait for this warp's outstanding global stores)
        unsigned old;
        asm volatile("atom.relaxed.cta.shared.add.u32 %0, [%1], 1;" : "=r"(old) : "r"(smem_u32(&sm_ctr[sg.grp_ctr])) : "memory");
        lastc = int(old) == sg.grp_size - 1;
      }
      lastc = __shfl_sync(0xffffffffu, lastc, 0);
      GLIDE_TRACE_EVENT(21);
      if (!lastc) continue;
      // at most 8 records (one per warp); fully unrolled so that the shared-memory loads overlap
      const float *g0 = sm_pool + size_t(sg.grp_slot0) * L::kRecFloats;
      float fr[kWarps][G];
#pragma unroll
      for (int h = 0; h < G; ++h) {
        float Mg = -CUDART_INF_F;
#pragma unroll
        for (int i = 0; i < kWarps; ++i) {
          fr[i][h] = i < sg.grp_size ? g0[size_t(i) * L::kRecFloats + G * kD + h] : -CUDART_INF_F;
          Mg = fmaxf(Mg, fr[i][h]);
        }
        float lg = 0.f;
#pragma unroll
        for (int i = 0; i < kWarps; ++i) {
          fr[i][h] = exp2_or_zero(fr[i][h], Mg);
          if (i < sg.grp_size) lg = fmaf(g0[size_t(i) * L::kRecFloats + G * kD + G + h], fr[i][h], lg);
        }
        mh[h] = Mg;
        lh[h] = lg;
        acc[h] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int i = 0; i < kWarps; ++i) {
        if (i < sg.grp_size) {
#pragma unroll
          for (int h = 0; h < G; ++h) {
            const float4 av = *reinterpret_cast<const float4 *>(g0 + size_t(i) * L::kRecFloats + h * kD + lane * 4);
            acc[h].x = fmaf(av.x, fr[i][h], acc[h].x);
            acc[h].y = fmaf(av.y, fr[i][h], acc[h].y);
            acc[h].z = fmaf(av.z, fr[i][h], acc[h].z);
            acc[h].w = fmaf(av.w, fr[i][h], acc[h].w);
          }
        }
      }
      if (SUM) {   // the linear parts of the group's records simply add up
#pragma unroll
        for (int h = 0; h < G; ++h) {
          a[h] = make_float4(0.f, 0.f, 0.f, 0.f);
          bp[h] = 0.f;
        }
#pragma unroll
        for (int i = 0; i < kWarps; ++i) {
          if (i < sg.grp_size) {
#pragma unroll
            for (int h = 0; h < G; ++h) {
              const float4 av = *reinterpret_cast<const float4 *>(g0 + size_t(i) * L::kRecFloats + L::kRecW + h * kD + lane * 4);
              a[h].x += av.x;
              a[h].y += av.y;
              a[h].z += av.z;
              a[h].w += av.w;
              bp[h] += g0[size_t(i) * L::kRecFloats + L::kRecW + G * kD + h];
            }
          }
        }
      }
      GLIDE_TRACE_EVENT(22);
    }
    if (sg.part >= 0) {
      // the unit is cut by a CTA boundary: this CTA's record goes to global scratch, every value paired with the
      // launch's tag; the unit's last ticket merges the records (at the end of that warp's range).
      unsigned long long *grec = reinterpret_cast<unsigned long long *>(p.partials) + (size_t(sg.rec0) + sg.part) * p.rec_floats;
#pragma unroll
      for (int h = 0; h < G; ++h) {
        ll_store2(grec + h * kD + lane * 4, acc[h].x, acc[h].y, p.launch_tag);
        ll_store2(grec + h * kD + lane * 4 + 2, acc[h].z, acc[h].w, p.launch_tag);
        if (SUM) {
          ll_store2(grec + L::kRecW + h * kD + lane * 4, a[h].x, a[h].y, p.launch_tag);
          ll_store2(grec + L::kRecW + h * kD + lane * 4 + 2, a[h].z, a[h].w, p.launch_tag);
        }
        if (lane == 0) {
          ll_store1(grec + G * kD + h, mh[h], p.launch_tag);
          ll_store1(grec + G * kD + G + h, lh[h], p.launch_tag);
          if (SUM) ll_store1(grec + L::kRecW + G * kD + h, bp[h], p.launch_tag);
        }
      }
      // the unit's ticket, taken without a fence: the result is looked at only at the end of this warp's range, so
      // the round trip runs beside the tiles of the range's remaining segments
      unsigned tick = 0;
      if (lane == 0)
        asm volatile("atom.relaxed.gpu.global.add.u32 %0, [%1], 1;" : "=r"(tick) : "l"(p.tickets + sg.unit) : "memory");
      if (n_pending == 0) {
        pend0 = s;
        tick0 = tick;
      } else {
        pend1 = s;
        tick1 = tick;
      }
      ++n_pending;
      own_seg = s;
    } else {
      // the whole unit is in this range: current token's own term, shared normaliser, output row, ring append
      float vx[4];
      vx[0] = __uint_as_float(vt_bits.x << 16);
      vx[1] = __uint_as_float(vt_bits.x & 0xffff0000u);
      vx[2] = __uint_as_float(vt_bits.y << 16);
      vx[3] = __uint_as_float(vt_bits.y & 0xffff0000u);
#pragma unroll
      for (int h = 0; h < G; ++h) {
        // reference: the largest logit of the records (a record that includes the linear readout carries a
        // reference >= 0 already; without a state no floor is wanted: it would only push the window weights
        // towards underflow).  Sum of terms: the linear term a / b is added (an empty term counts as zero)
        const float Mf = fmaxf(mh[h], scur[h]);
        const float fr = exp2_or_zero(mh[h], Mf), fc = exp2_or_zero(scur[h], Mf);
        const float den = fmaf(lh[h], fr, fc);
        const float inv = (!SUM || den > 0.f) ? 1.0f / den : 0.f;
        const float il = (SUM && bp[h] > 0.f) ? 1.0f / bp[h] : 0.f;
        const int orow = sg.qrow0 + (sp.heads_contiguous ? h : p.heads_of[sg.g * G + h]);
        const __nv_bfloat162 lo = __floats2bfloat162_rn(fmaf(fmaf(acc[h].x, fr, fc * vx[0]), inv, SUM ? a[h].x * il : 0.f),
                                                        fmaf(fmaf(acc[h].y, fr, fc * vx[1]), inv, SUM ? a[h].y * il : 0.f));
        const __nv_bfloat162 hi = __floats2bfloat162_rn(fmaf(fmaf(acc[h].z, fr, fc * vx[2]), inv, SUM ? a[h].z * il : 0.f),
                                                        fmaf(fmaf(acc[h].w, fr, fc * vx[3]), inv, SUM ? a[h].w * il : 0.f));
        uint2 packed;
        packed.x = *reinterpret_cast<const uint32_t *>(&lo);
        packed.y = *reinterpret_cast<const uint32_t *>(&hi);
        *reinterpret_cast<uint2 *>(reinterpret_cast<bf16 *>(p.out) + size_t(orow) * kD + lane * 4) = packed;
      }
      if (has_win) {   // every reader of slot t mod cap is done: bit copy of the new rows
        const size_t row = (size_t(sg.row_base) + size_t(win_cur)) * kD;
        reinterpret_cast<uint2 *>(reinterpret_cast<bf16 *>(p.ws + size_t(sg.ringK_off256) * 256) + row)[lane] = kt_bits;
        reinterpret_cast<uint2 *>(reinterpret_cast<bf16 *>(p.ws + size_t(sg.ringV_off256) * 256) + row)[lane] = vt_bits;
        if (p.gated && lane == 0)   // the token's gate waits in the ring with it
          reinterpret_cast<float *>(p.ws + p.layers[sg.layer].ringG)[size_t(sg.row_base) + size_t(win_cur)] =
              p.gate ? p.gate[sg.unit] : 1.f;
      }
    }
  }
  GLIDE_TRACE_EVENT(14);

  // ---- units this range shares with other CTAs: whoever holds a unit's last ticket merges its records ---------------
  // (every record of the unit has been stored by then, though perhaps not arrived: the merge polls the tags.  It
  // never waits for a CTA that has not run yet, so launches that share the GPU cannot block each other.)
  if (n_pending > 0 && !failed) {
    GLIDE_TRACE_EVENT(12);
    for (int pi = 0; pi < n_pending && !failed; ++pi) {
      const StreamSegment &sg = sm_segs[pi == 0 ? pend0 : pend1];
      const int pseg = pi == 0 ? pend0 : pend1;
      // this warp's own record of the unit is still in registers when the unit's segment was the last of the range: it
      // is taken from there (same values, same place in the order of the merge) instead of being awaited from memory
      // (groups of 8 heads: the record is 40 registers wide and keeping it would spill; it is read back like the others)
      const int own = (G <= 4 && pseg == own_seg && pseg == seg_hi - 1) ? sg.part : -1;
      const bool has_win = sg.cap > 0;
      // reload the unit's query rows and current token (this warp may have moved on to another unit since);
      // every load of the merge's first batch is issued before anything is reduced
      const bf16 *qall = reinterpret_cast<const bf16 *>(p.q);
      const unsigned long long *r0 = reinterpret_cast<const unsigned long long *>(p.partials) + size_t(sg.rec0) * p.rec_floats;
      constexpr int RPB = 16 / G;   // records per batch (every value arrives as an 8-byte pair: two registers)
      const uint2 ktb = ld_u2_pinned(reinterpret_cast<const bf16 *>(p.k) + size_t(sg.unit) * kD + lane * 4);
      const uint2 vtb = ld_u2_pinned(reinterpret_cast<const bf16 *>(p.v) + size_t(sg.unit) * kD + lane * 4);
      int orow[G];
      uint2 qbits[G];
#pragma unroll
      for (int h = 0; h < G; ++h) {
        orow[h] = sg.qrow0 + (sp.heads_contiguous ? h : p.heads_of[sg.g * G + h]);
        qbits[h] = ld_u2_pinned(qall + size_t(orow[h]) * kD + lane * 4);
      }
      float me0 = -CUDART_INF_F, le0 = 0.f;
      float4 vv0[RPB][G];
      // one batch of records: polled until every pair this lane uses carries the launch's tag (bounded)
      auto load_batch = [&](int i0, float &me, float &le, uint32_t max_spins) -> bool {
        const int ri = i0 + lane / G, rh = lane % G;
        const int nb = sg.n_parts - i0 < RPB ? sg.n_parts - i0 : RPB;
        const bool mine = lane < RPB * G && ri < sg.n_parts;
        // every load is issued before any tag is looked at (records past the unit's last one re-read the batch's first)
        const unsigned long long *ml = r0 + size_t(mine ? ri : i0) * p.rec_floats + G * kD + rh;
        for (uint32_t spins = 0;; ++spins) {
          unsigned long long raw[RPB][G][4], rm, rl;
          asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(rm) : "l"(ml));
          asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(rl) : "l"(ml + G));
#pragma unroll
          for (int u = 0; u < RPB; ++u)
#pragma unroll
            for (int h = 0; h < G; ++h) {
              const unsigned long long *src = r0 + size_t(u < nb ? i0 + u : i0) * p.rec_floats + h * kD + lane * 4;
              asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(raw[u][h][0]), "=l"(raw[u][h][1]) : "l"(src));
              asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(raw[u][h][2]), "=l"(raw[u][h][3]) : "l"(src + 2));
            }
          uint32_t diff = (mine && ri != own) ? (uint32_t(rm >> 32) ^ p.launch_tag) | (uint32_t(rl >> 32) ^ p.launch_tag) : 0u;
#pragma unroll
          for (int u = 0; u < RPB; ++u)
#pragma unroll
            for (int h = 0; h < G; ++h) {
              const bool is_own = i0 + u == own;
#pragma unroll
              for (int c = 0; c < 4; ++c)
                if (!is_own && u < nb) diff |= uint32_t(raw[u][h][c] >> 32) ^ p.launch_tag;   // (slots past the last record are not used)
              vv0[u][h] = is_own ? acc[h]
                                 : make_float4(__uint_as_float(uint32_t(raw[u][h][0])), __uint_as_float(uint32_t(raw[u][h][1])),
                                               __uint_as_float(uint32_t(raw[u][h][2])), __uint_as_float(uint32_t(raw[u][h][3])));
            }
          me = mine ? __uint_as_float(uint32_t(rm)) : -CUDART_INF_F;
          le = mine ? __uint_as_float(uint32_t(rl)) : 0.f;
          if (mine && ri == own) {
#pragma unroll
            for (int h = 0; h < G; ++h)
              if (rh == h) {
                me = mh[h];
                le = lh[h];
              }
          }
          if (__all_sync(0xffffffffu, diff == 0)) return true;
          if (spins >= max_spins) return false;
        }
      };
      // The first batch is read once before the ticket is looked at, so that for the warp that turns out to hold the
      // last ticket the ticket's round trip and these loads run side by side (the other parts stored their records
      // before they took their tickets; this warp's own record is not awaited).  The others have read a few KiB of
      // L2 for nothing, at the idle end of their range.
      const bool early = load_batch(0, me0, le0, 0u);
      if (__shfl_sync(0xffffffffu, pi == 0 ? tick0 : tick1, 0) != unsigned(sg.n_parts - 1)) continue;
      if (!early && !load_batch(0, me0, le0, kWaitLimit >> 6)) {
        failed = true;
        break;
      }
      GLIDE_TRACE_EVENT(15);
      float sc[G];
      {
        float kx[4];
        kx[0] = __uint_as_float(ktb.x << 16);
        kx[1] = __uint_as_float(ktb.x & 0xffff0000u);
        kx[2] = __uint_as_float(ktb.y << 16);
        kx[3] = __uint_as_float(ktb.y & 0xffff0000u);
#pragma unroll
        for (int h = 0; h < G; ++h) {
          sc[h] = fmaf(__uint_as_float(qbits[h].x << 16), kx[0], 0.f);
          sc[h] = fmaf(__uint_as_float(qbits[h].x & 0xffff0000u), kx[1], sc[h]);
          sc[h] = fmaf(__uint_as_float(qbits[h].y << 16), kx[2], sc[h]);
          sc[h] = fmaf(__uint_as_float(qbits[h].y & 0xffff0000u), kx[3], sc[h]);
        }
        warp_sum_multi<G>(sc);
#pragma unroll
        for (int h = 0; h < G; ++h) sc[h] = has_win ? sc[h] * p.scale_log2 : -CUDART_INF_F;
      }
      GLIDE_TRACE_EVENT(16);
      // merge the records: maxima and sums first (one (record, head) pair per lane), then the vectors
      float Mg[G], lg[G];
      float4 macc[G];
#pragma unroll
      for (int h = 0; h < G; ++h) {
        Mg[h] = -CUDART_INF_F;
        lg[h] = 0.f;
        macc[h] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
      for (int i0 = 0; i0 < sg.n_parts; i0 += RPB) {
        const int rh = lane % G;
        const int nb = sg.n_parts - i0 < RPB ? sg.n_parts - i0 : RPB;
        float me = me0, le = le0;
        if (i0 > 0 && !load_batch(i0, me, le, kWaitLimit >> 6)) {   // further batches (units cut into more than RPB records)
          failed = true;
          break;
        }
        float Mn[G];
#pragma unroll
        for (int h = 0; h < G; ++h) Mn[h] = rh == h ? me : -CUDART_INF_F;
#pragma unroll
        for (int o2 = 16; o2 > 0; o2 >>= 1)
#pragma unroll
          for (int h = 0; h < G; ++h) Mn[h] = fmaxf(Mn[h], __shfl_xor_sync(0xffffffffu, Mn[h], o2));
        float fe = 0.f, lpart[G];
#pragma unroll
        for (int h = 0; h < G; ++h) {
          Mn[h] = fmaxf(Mn[h], Mg[h]);
          const float resc = exp2_or_zero(Mg[h], Mn[h]);
          lg[h] *= resc;
          macc[h].x *= resc;
          macc[h].y *= resc;
          macc[h].z *= resc;
          macc[h].w *= resc;
          Mg[h] = Mn[h];
          if (rh == h) fe = exp2_or_zero(me, Mn[h]);
          lpart[h] = rh == h ? le * fe : 0.f;
        }
        warp_sum_multi<G>(lpart);
#pragma unroll
        for (int h = 0; h < G; ++h) lg[h] += lpart[h];
#pragma unroll
        for (int u = 0; u < RPB; ++u)
#pragma unroll
          for (int h = 0; h < G; ++h)
            if (u < nb) {
              const float f = __shfl_sync(0xffffffffu, fe, u * G + h);
              macc[h].x = fmaf(vv0[u][h].x, f, macc[h].x);
              macc[h].y = fmaf(vv0[u][h].y, f, macc[h].y);
              macc[h].z = fmaf(vv0[u][h].z, f, macc[h].z);
              macc[h].w = fmaf(vv0[u][h].w, f, macc[h].w);
            }
      }
      GLIDE_TRACE_EVENT(17);
      float vx[4];
      vx[0] = __uint_as_float(vtb.x << 16);
      vx[1] = __uint_as_float(vtb.x & 0xffff0000u);
      vx[2] = __uint_as_float(vtb.y << 16);
      vx[3] = __uint_as_float(vtb.y & 0xffff0000u);
      float4 al[G];
      float bl[G];
      if (SUM) {   // linear parts of all records: plain sums
#pragma unroll
        for (int h = 0; h < G; ++h) {
          al[h] = make_float4(0.f, 0.f, 0.f, 0.f);
          bl[h] = 0.f;
        }
        for (int i = 0; i < sg.n_parts && !failed; ++i) {
#pragma unroll
          for (int h = 0; h < G; ++h) {
            float4 av = a[h];
            float bv = bp[h];
            uint32_t spins = 0;   // (the window half of the record carried the tag already: these follow at once)
            while (i != own && !__all_sync(0xffffffffu, ll_load4(r0 + size_t(i) * p.rec_floats + L::kRecW + h * kD + lane * 4, p.launch_tag, av) &&
                                                ll_load1(r0 + size_t(i) * p.rec_floats + L::kRecW + G * kD + h, p.launch_tag, bv)))
              if (++spins > (kWaitLimit >> 6)) {
                failed = true;
                break;
              }
            al[h].x += av.x;
            al[h].y += av.y;
            al[h].z += av.z;
            al[h].w += av.w;
            bl[h] += bv;
          }
        }
      }
#pragma unroll
      for (int h = 0; h < G; ++h) {
        const float Mf = fmaxf(Mg[h], sc[h]);
        const float fr = exp2_or_zero(Mg[h], Mf), fc = exp2_or_zero(sc[h], Mf);
        const float den = fmaf(lg[h], fr, fc);
        const float inv = (!SUM || den > 0.f) ? 1.0f / den : 0.f;
        const float il = (SUM && bl[h] > 0.f) ? 1.0f / bl[h] : 0.f;
        const __nv_bfloat162 lo = __floats2bfloat162_rn(fmaf(fmaf(macc[h].x, fr, fc * vx[0]), inv, SUM ? al[h].x * il : 0.f),
                                                        fmaf(fmaf(macc[h].y, fr, fc * vx[1]), inv, SUM ? al[h].y * il : 0.f));
        const __nv_bfloat162 hi = __floats2bfloat162_rn(fmaf(fmaf(macc[h].z, fr, fc * vx[2]), inv, SUM ? al[h].z * il : 0.f),
                                                        fmaf(fmaf(macc[h].w, fr, fc * vx[3]), inv, SUM ? al[h].w * il : 0.f));
        uint2 packed;
        packed.x = *reinterpret_cast<const uint32_t *>(&lo);
        packed.y = *reinterpret_cast<const uint32_t *>(&hi);
        *reinterpret_cast<uint2 *>(reinterpret_cast<bf16 *>(p.out) + size_t(orow[h]) * kD + lane * 4) = packed;
      }
      if (has_win) {
        const size_t row = (size_t(sg.row_base) + size_t(slot_of(pos_of(pi == 0 ? pend0 : pend1), sg.cap))) * kD;
        reinterpret_cast<uint2 *>(reinterpret_cast<bf16 *>(p.ws + size_t(sg.ringK_off256) * 256) + row)[lane] = ktb;
        reinterpret_cast<uint2 *>(reinterpret_cast<bf16 *>(p.ws + size_t(sg.ringV_off256) * 256) + row)[lane] = vtb;
        if (p.gated && lane == 0)
          reinterpret_cast<float *>(p.ws + p.layers[sg.layer].ringG)[row / kD] = p.gate ? p.gate[sg.unit] : 1.f;
      }
      if (lane == 0) p.tickets[sg.unit] = 0;   // for the next launch
      GLIDE_TRACE_EVENT(13);
    }
  }
  if (failed && lane == 0) atomicExch(p.status, kDevWaitTimeout);
  if (lane == 0) bulk_wait0();   // this warp's state stores have landed
  GLIDE_TRACE_EVENT(9);

}

template <int G, int STAGES, int MODE>
size_t stream_smem_bytes(int max_segs, int pool_slots) {
  using L = Layout<G, (MODE & 1) != 0>;
  return 1024 + size_t(kWarps) * STAGES * kStageBytes + size_t(kWarps) * L::kHdrBytes + size_t(kWarps) * STAGES * 64 +
         size_t(max_segs) * sizeof(StreamSegment) + size_t(kWarps) * (STAGES + 1) * 8 + size_t(kStreamMaxGroups) * 4 +
         ((MODE & 2) ? size_t(kWarps) * STAGES * (G + 1) * 64 : 0) + size_t(pool_slots) * L::kRecFloats * 4 +
         size_t(max_segs) * 8;
}

// the kernel's MODE for a context
int stream_mode(const glide_ctx *ctx) {
  return (ctx->cfg.phi == GLIDE_PHI_PROJ_SOFTMAX2 ? 2 : 0) | (ctx->cfg.merge != GLIDE_MERGE_SHARED ? 1 : 0);
}

// f(group size, stages, mode)
template <typename F>
int dispatch_stream(int G, int mode, F &&f) {
#define GLIDE_STREAM_CASE(GG)                                                                   \
  case GG:                                                                                      \
    return mode == 3   ? f(IntTag<GG>{}, IntTag<GLIDE_STREAM_STAGES>{}, IntTag<3>{})            \
           : mode == 2 ? f(IntTag<GG>{}, IntTag<GLIDE_STREAM_STAGES>{}, IntTag<2>{})            \
           : mode == 1 ? f(IntTag<GG>{}, IntTag<GLIDE_STREAM_STAGES>{}, IntTag<1>{})            \
                       : f(IntTag<GG>{}, IntTag<GLIDE_STREAM_STAGES>{}, IntTag<0>{});
  switch (G) {
    GLIDE_STREAM_CASE(1)
    GLIDE_STREAM_CASE(2)
    GLIDE_STREAM_CASE(4)
    GLIDE_STREAM_CASE(8)
    default: return int(GLIDE_ERR_UNSUPPORTED);
  }
#undef GLIDE_STREAM_CASE
}

}  // namespace

// Static schedule of the streaming kernel.  Weights are the measured relative costs of a state tile, a window
// tile and of a segment (header, feature maps, finish).
//   1. Units (layer x sequence x KV head) are packed whole into CTAs, heaviest first onto the least loaded CTA;
//      a unit heavier than a CTA's share is first cut into equal pieces.  So almost every unit lives inside one
//      CTA and is reduced in shared memory; only the oversized ones need global records and a merge.
//   2. Inside a CTA the list of pieces is cut into 8 contiguous ranges, one per warp, whose heaviest is as light as
//      a cut at tile boundaries allows (bisection on the limit of a greedy split).
// Schedule for the layers [layer_begin, layer_begin + layer_count).  Units and query rows are numbered relative to
// the first layer of the range (that is how a launch for the range addresses q, k, v and out); the
// layer index itself stays absolute (descriptors, layer table).
void build_stream_schedule(const glide_ctx *ctx, int layer_begin, int layer_count, int n_ranges, int pool_slots,
                           std::vector<StreamSegment> *segs, std::vector<int32_t> *range_seg_begin, int *max_segs_per_cta,
                           size_t *n_records) {
  constexpr int64_t kSegWeight = GLIDE_W_UNIT, kStateWeight = GLIDE_W_STATE, kWinWeight = GLIDE_W_WIN;
  const int B = ctx->cfg.batch, Hkv = ctx->cfg.n_kv_heads, d = ctx->cfg.head_dim;
  const int n_ctas = n_ranges / kWarps;
  const int64_t units_per_layer = int64_t(B) * Hkv;
  bool contiguous_heads = true;
  for (int g = 0; g < Hkv; ++g)
    for (int i = 1; i < ctx->G; ++i)
      contiguous_heads = contiguous_heads && ctx->heads_of[size_t(g) * ctx->G + i] == ctx->heads_of[size_t(g) * ctx->G] + i;

  struct Piece {   // a run of tiles of one unit: state tiles [st0, st0+nst), window tiles [w0, w0+nw)
    int layer, unit, uidx;
    int st0, nst, w0, nw;
    int64_t weight() const { return kStateWeight * nst + kWinWeight * nw + kSegWeight; }
  };
  std::vector<Piece> pieces;
  int64_t total_w = 0;
  int n_units = 0;
  for (int l = layer_begin; l < layer_begin + layer_count; ++l) {
    const LayerDev &ld = ctx->layers[l];
    for (int64_t u = 0; u < units_per_layer; ++u) {
      Piece pc{l, int(int64_t(l - layer_begin) * units_per_layer + u), n_units++, 0, ld.evicts ? ctx->dp / kTileRows : 0, 0,
               int((ld.cap + kTileRows - 1) / kTileRows)};
      pieces.push_back(pc);
      total_w += pc.weight();
    }
  }
  // Small problems (one layer, a short window, a small batch) do not have work for every CTA: below about ten
  // tiles per CTA the per-segment overheads and the number of records per merge grow faster than the streaming
  // time shrinks.  Units that are small themselves are then kept whole.
  constexpr int64_t kMinCtaWeight = GLIDE_W_MIN_CTA;
  int64_t max_unit_w = 0;
  for (const Piece &pc : pieces) max_unit_w = std::max(max_unit_w, pc.weight());
  const int n_used = int(std::max<int64_t>(1, std::min<int64_t>(n_ctas, total_w / kMinCtaWeight)));
  int64_t cta_share = std::max<int64_t>(1, (total_w + n_used - 1) / n_used);
  if (n_used < n_ctas && max_unit_w <= 2 * kMinCtaWeight) cta_share = std::max(cta_share, max_unit_w);
  std::vector<std::vector<size_t>> cta_pieces(size_t(std::max(n_ctas, 1)));
  std::vector<int64_t> cta_load(size_t(std::max(n_ctas, 1)), 0);
  // heaviest first
  std::vector<size_t> order(pieces.size());
  for (size_t i = 0; i < order.size(); ++i) order[i] = i;
  std::stable_sort(order.begin(), order.end(), [&](size_t x, size_t y) { return pieces[x].weight() > pieces[y].weight(); });
  // (a) units heavier than one CTA's share are laid out back to back over the first CTAs (state tiles first) and
  //     cut at cumulative targets, so that what one CTA leaves unused goes to the next one instead of piling up
  //     on the last; only these units need global records and a merge
  size_t oi = 0;
  int n_heavy_ctas = 0;
  int64_t heavy_slack = 0;
  {
    int64_t heavy_w = 0;
    size_t n_heavy = 0;
    while (n_heavy < order.size() && pieces[order[n_heavy]].weight() > cta_share) heavy_w += pieces[order[n_heavy++]].weight();
    // these CTAs end with the merge of their units' records: they may be given less than a full share
    const int64_t heavy_share = std::max<int64_t>(1, cta_share * GLIDE_STREAM_FILL / 100);
    int n_h = int(std::max<int64_t>(1, std::min<int64_t>(n_used, (heavy_w + heavy_share / 2) / heavy_share)));
    // Where spreading leaves a CTA only a few dozen tiles (a one-layer launch of a long window at a small batch), a
    // unit is cut into at most about GLIDE_STREAM_MAX_PARTS records: the merging warp reads them a few at a time, each
    // batch a round trip to L2, and that costs more than the shorter streams save.  Large problems keep every SM.
    if (heavy_w / n_h < 40 * kWinWeight) n_h = int(std::max<int64_t>(1, std::min<int64_t>(n_h, int64_t(GLIDE_STREAM_MAX_PARTS) * int64_t(n_heavy))));
    // every CTA boundary inside a unit opens one more piece with its own fixed cost
    const int64_t target = (heavy_w + int64_t(n_h) * kSegWeight) / n_h + 1;
    if (n_heavy > 0) {
      n_heavy_ctas = n_h;
      heavy_slack = cta_share - heavy_share;
    }
    int cta = 0;
    int64_t cum = 0;   // weight laid out so far over all heavy CTAs
    for (; oi < n_heavy; ++oi) {
      const Piece pc = pieces[order[oi]];
      int st_done = 0, w_done = 0;
      while (st_done < pc.nst || w_done < pc.nw) {
        const bool last_cta = cta + 1 >= n_h;
        int64_t room = last_cta ? INT64_MAX / 4 : int64_t(cta + 1) * target - cum - kSegWeight;
        if (!last_cta && room < 4 * kWinWeight) {   // not worth a piece: this CTA is full
          ++cta;
          continue;
        }
        Piece q = pc;
        q.st0 = pc.st0 + st_done;
        q.nst = int(std::min<int64_t>(pc.nst - st_done, room / kStateWeight));
        room -= kStateWeight * int64_t(q.nst);
        q.w0 = pc.w0 + w_done;
        q.nw = (st_done + q.nst == pc.nst) ? int(std::min<int64_t>(pc.nw - w_done, std::max<int64_t>(room, 0) / kWinWeight)) : 0;
        // a remainder of a few tiles is not worth a piece of its own either
        const int64_t rest = kStateWeight * int64_t(pc.nst - st_done - q.nst) + kWinWeight * int64_t(pc.nw - w_done - q.nw);
        if (q.nst + q.nw == 0 || rest < 4 * kWinWeight) {
          q.nst = pc.nst - st_done;
          q.nw = pc.nw - w_done;
        }
        st_done += q.nst;
        w_done += q.nw;
        pieces.push_back(q);
        cta_pieces[size_t(cta)].push_back(pieces.size() - 1);
        cta_load[size_t(cta)] += q.weight();
        cum += q.weight();
      }
    }
  }
  // CTAs beyond n_used stay empty
  for (size_t c = size_t(n_used); c < cta_load.size(); ++c) cta_load[c] = INT64_MAX / 2;
  // (b) every other unit goes whole onto the least loaded CTA (the share the heavy CTAs leave unused is not on offer)
  for (int c = 0; c < n_heavy_ctas; ++c) cta_load[size_t(c)] += heavy_slack;
  for (; oi < order.size(); ++oi) {
    size_t best = 0;
    for (size_t c = 1; c < cta_load.size(); ++c)
      if (cta_load[c] < cta_load[best]) best = c;
    cta_pieces[best].push_back(order[oi]);
    cta_load[best] += pieces[order[oi]].weight();
  }
  for (size_t c = size_t(n_used); c < cta_load.size(); ++c) cta_load[c] = 0;
  for (int c = 0; c < n_heavy_ctas; ++c) cta_load[size_t(c)] -= heavy_slack;

  segs->clear();
  range_seg_begin->assign(size_t(n_ranges) + 1, 0);
  std::vector<std::vector<size_t>> unit_segs;
  unit_segs.resize(size_t(n_units));
  std::vector<int> seg_range;
  // Runs of tiles of one piece: what a segment covers.
  struct Run {
    size_t piece;
    int st0, nst, w0, nw;
  };
  // The CTA's pieces cut into kWarps contiguous ranges whose heaviest is as light as possible: for a limit on a warp's
  // weight every warp takes, in order, whole pieces while they fit and then as many tiles of the next piece as fit
  // (a piece shared by several warps costs every one of them a record and a place in the reduction); the smallest
  // limit that places all tiles is found by bisection.
  constexpr int64_t kGroupWeight = GLIDE_W_GROUP;
  auto split_cta = [&](const std::vector<size_t> &list, int64_t limit, std::vector<std::vector<Run>> *out) -> bool {
    size_t pi = 0;
    int st_done = 0, w_done = 0;
    if (out) out->assign(size_t(kWarps), {});
    for (int wi = 0; wi < kWarps && pi < list.size(); ++wi) {
      int64_t cum = 0;
      bool empty = true;
      while (pi < list.size()) {
        const Piece &pc = pieces[list[pi]];
        const int rem_st = pc.nst - st_done, rem_w = pc.nw - w_done;
        const bool begun = st_done > 0 || w_done > 0;
        const int64_t whole = kSegWeight + (begun ? kGroupWeight : 0) + kStateWeight * rem_st + kWinWeight * rem_w;
        Run r{list[pi], pc.st0 + st_done, rem_st, pc.w0 + w_done, rem_w};
        bool full = false;
        if (cum + whole > limit && wi + 1 < kWarps) {
          int64_t room = limit - cum - kSegWeight - kGroupWeight;
          r.nst = int(std::max<int64_t>(0, std::min<int64_t>(rem_st, room / kStateWeight)));
          room -= kStateWeight * int64_t(r.nst);
          r.nw = r.nst == rem_st ? int(std::max<int64_t>(0, std::min<int64_t>(rem_w, room / kWinWeight))) : 0;
          if (r.nst + r.nw < (empty ? 1 : 2)) {   // a tile more does not fit (and one alone is not worth a segment)
            if (empty) return false;
            break;
          }
          full = true;
        } else if (cum + whole > limit) {
          return false;   // the last warp would have to take more than the limit
        }
        empty = false;
        cum += kSegWeight + ((begun || full) ? kGroupWeight : 0) + kStateWeight * r.nst + kWinWeight * r.nw;
        if (out) (*out)[size_t(wi)].push_back(r);
        st_done += r.nst;
        w_done += r.nw;
        if (st_done == pc.nst && w_done == pc.nw) {
          ++pi;
          st_done = w_done = 0;
        }
        if (full) break;
      }
    }
    return pi == list.size();
  };
  for (int cta = 0; cta < n_ctas; ++cta) {
    const std::vector<size_t> &list = cta_pieces[size_t(cta)];
    std::vector<std::vector<Run>> runs;
    runs.resize(size_t(kWarps));
    if (!list.empty()) {
      int64_t hi = 0;
      for (size_t i : list) hi += pieces[i].weight() + kGroupWeight;
      int64_t lo = hi / kWarps;   // lo - 1 is not enough, hi always is (one warp takes everything)
      while (lo < hi) {
        const int64_t mid = lo + (hi - lo) / 2;
        if (split_cta(list, mid, nullptr)) hi = mid; else lo = mid + 1;
      }
      split_cta(list, hi, &runs);
    }
    for (int wi = 0; wi < kWarps; ++wi) {
      const int c = cta * kWarps + wi;
      (*range_seg_begin)[size_t(c)] = int32_t(segs->size());
      for (const Run &r : runs[size_t(wi)]) {
        const Piece &pc = pieces[r.piece];
        const LayerDev &ld = ctx->layers[pc.layer];
        StreamSegment sg{};
        sg.n_state = r.nst;
        sg.n_win = r.nw;
        sg.unit = pc.unit;
        sg.layer = pc.layer;
        sg.range = wi;
        sg.state0 = r.st0;
        sg.win0 = r.w0;
        const int64_t ub = pc.unit - int64_t(pc.layer - layer_begin) * units_per_layer;
        sg.row_base = int32_t(ub * ld.cap);
        sg.cap = int32_t(ld.cap);
        sg.w = int32_t(std::min<int64_t>(ld.w, INT32_MAX));
        sg.evicts = ld.evicts ? (ld.wlin == 0 ? 3 : 1) : 0;
        sg.S_off256 = int32_t((ld.S + size_t(ub) * ctx->dp * d * 4) / 256);
        sg.z_off256 = int32_t((ld.z + size_t(ub) * ctx->dp * 4) / 256);
        sg.ringK_off256 = int32_t(ld.ringK / 256);
        sg.ringV_off256 = int32_t(ld.ringV / 256);
        sg.g = int32_t(ub % Hkv);
        {
          const int64_t b = ub / Hkv;
          const int64_t row = (int64_t(pc.layer - layer_begin) * B + b) * ctx->cfg.n_q_heads;
          sg.qrow0 = int32_t(row + (contiguous_heads ? ctx->heads_of[size_t(sg.g) * ctx->G] : 0));
        }
        unit_segs[size_t(pc.uidx)].push_back(segs->size());
        seg_range.push_back(c);
        segs->push_back(sg);
      }
    }
  }
  for (int c = n_ctas * kWarps; c <= n_ranges; ++c) (*range_seg_begin)[size_t(c)] = int32_t(segs->size());
  (*range_seg_begin)[size_t(n_ranges)] = int32_t(segs->size());
  *max_segs_per_cta = 0;
  for (int c = 0; c + kWarps <= n_ranges; c += kWarps)
    *max_segs_per_cta = std::max<int>(*max_segs_per_cta, (*range_seg_begin)[size_t(c + kWarps)] - (*range_seg_begin)[size_t(c)]);

  // Warps of one CTA that share a unit reduce their records in shared memory first (a "group"); only one
  // record per group goes to global scratch, and a unit that lies inside one group never touches it.
  size_t records = 0;
  std::vector<int> cta_slots(size_t(n_ctas) + 1, 0), cta_groups(size_t(n_ctas) + 1, 0);
  for (size_t u = 0; u < unit_segs.size(); ++u) {
    std::vector<size_t> &list = unit_segs[u];
    std::stable_sort(list.begin(), list.end(), [&](size_t x, size_t y) { return seg_range[x] < seg_range[y]; });
    std::vector<std::pair<size_t, size_t>> groups;   // [first, last) into list
    for (size_t i = 0; i < list.size();) {
      const int cta = seg_range[list[i]] / kWarps;
      size_t j = i + 1;
      while (j < list.size() && seg_range[list[j]] / kWarps == cta) ++j;
      const int need = int(j - i);
      if (need >= 2 && cta_slots[size_t(cta)] + need <= pool_slots && cta_groups[size_t(cta)] < kStreamMaxGroups) {
        for (size_t k = i; k < j; ++k) {
          StreamSegment &sg = (*segs)[list[k]];
          sg.grp_size = need;
          sg.grp_slot0 = cta_slots[size_t(cta)];
          sg.grp_idx = int(k - i);
          sg.grp_ctr = cta_groups[size_t(cta)];
        }
        cta_slots[size_t(cta)] += need;
        cta_groups[size_t(cta)] += 1;
        groups.emplace_back(i, j);
      } else {   // single warp, or no room left in the CTA's pool: every segment is its own group
        for (size_t k = i; k < j; ++k) {
          (*segs)[list[k]].grp_size = 1;
          groups.emplace_back(k, k + 1);
        }
      }
      i = j;
    }
    for (size_t gi = 0; gi < groups.size(); ++gi)
      for (size_t k = groups[gi].first; k < groups[gi].second; ++k) {
        StreamSegment &sg = (*segs)[list[k]];
        sg.part = groups.size() == 1 ? -1 : int32_t(gi);
        sg.n_parts = int32_t(groups.size());
        sg.rec0 = groups.size() == 1 ? 0 : int32_t(records);
      }
    if (groups.size() > 1) records += groups.size();
  }
  *n_records = records;
}

int stream_decode_supported(const glide_ctx *ctx) {
  return ctx->cfg.io_dtype == GLIDE_BF16 && ctx->cfg.head_dim == kD;
}

// Host-only part of the set-up: every schedule of the context for a device with n_ctas SMs and smem_limit bytes of
// shared memory per CTA; sizes the record pool so that stages, tables and pool fit.
int stream_decode_plan(glide_ctx *ctx, int n_ctas, size_t smem_limit) {
  const int L = ctx->cfg.n_layers;
  bool contiguous = true;
  for (int g = 0; g < ctx->cfg.n_kv_heads; ++g)
    for (int i = 1; i < ctx->G; ++i)
      contiguous = contiguous && ctx->heads_of[size_t(g) * ctx->G + i] == ctx->heads_of[size_t(g) * ctx->G] + i;
  ctx->stream_heads_contiguous = contiguous;
  return dispatch_stream(ctx->G, stream_mode(ctx), [&](auto gg, auto ss, auto mm) -> int {
    constexpr int G = decltype(gg)::value, S = decltype(ss)::value;
    constexpr int SUM = decltype(mm)::value;   // the kernel's MODE
    // The record pool for the shared-memory groups takes what the segment table leaves, up to kStreamPoolBytes: with
    // many small units per CTA (large batches) the table is large and hardly any unit is shared between warps.
    const int rec_bytes = ctx->stream_rec_floats * 4;
    int pool_slots = kStreamPoolBytes / rec_bytes;
    for (int attempt = 0;; ++attempt) {
      ctx->stream_scheds.clear();
      ctx->stream_segs.clear();
      ctx->stream_max_segs = 1;
      // [0]: all layers in one launch; [1 + l]: layer l alone, for callers that run other kernels between the layers
      const int n_sched = L > 1 ? L + 1 : 1;
      for (int si = 0; si < n_sched; ++si) {
        std::vector<StreamSegment> segs;
        glide_ctx::StreamSchedule sc;
        int max_segs = 0;
        size_t n_records = 0;
        build_stream_schedule(ctx, si == 0 ? 0 : si - 1, si == 0 ? L : 1, n_ctas * kWarps, pool_slots, &segs, &sc.range_begin,
                              &max_segs, &n_records);
        if (n_records > ctx->stream_rec_capacity) return GLIDE_ERR_UNSUPPORTED;
        sc.seg_base = ctx->stream_segs.size();
        sc.n_segs = segs.size();
        ctx->stream_segs.insert(ctx->stream_segs.end(), segs.begin(), segs.end());
        ctx->stream_max_segs = std::max(ctx->stream_max_segs, max_segs);
        ctx->stream_scheds.push_back(std::move(sc));
      }
      if (ctx->stream_segs.size() > ctx->stream_seg_capacity) return GLIDE_ERR_UNSUPPORTED;
      if (stream_smem_bytes<G, S, SUM>(ctx->stream_max_segs, pool_slots) <= smem_limit) break;
      const size_t without_pool = stream_smem_bytes<G, S, SUM>(ctx->stream_max_segs, 0);
      if (attempt > 0 || without_pool > smem_limit) return GLIDE_ERR_UNSUPPORTED;   // the table alone does not fit
      pool_slots = int((smem_limit - without_pool) / size_t(rec_bytes));
    }
    ctx->stream_smem = stream_smem_bytes<G, S, SUM>(ctx->stream_max_segs, pool_slots);
    ctx->decode_grid = n_ctas;
    return GLIDE_OK;
  });
}

int stream_decode_setup(glide_ctx *ctx) {
  const int n_ctas = std::min(ctx->sm_count * GLIDE_STREAM_CTAS_PER_SM, kMaxStreamCtas);
  int dev_max = 0;
  if (cudaDeviceGetAttribute(&dev_max, cudaDevAttrMaxSharedMemoryPerBlockOptin, ctx->device) != cudaSuccess) {
    cudaGetLastError();
    return GLIDE_ERR_CUDA;
  }
  const int rc = stream_decode_plan(ctx, n_ctas, size_t(dev_max));
  if (rc) return rc;
  return dispatch_stream(ctx->G, stream_mode(ctx), [&](auto gg, auto ss, auto mm) -> int {
    constexpr int G = decltype(gg)::value, S = decltype(ss)::value;
    constexpr int SUM = decltype(mm)::value;   // the kernel's MODE
    // the attribute belongs to the kernel, not to the context: ask for the device maximum so that contexts with
    // different schedules (different table sizes) can be alive together
    if (cudaFuncSetAttribute(glide_decode_stream_kernel<G, S, SUM, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             dev_max) != cudaSuccess ||
        cudaFuncSetAttribute(glide_decode_stream_kernel<G, S, SUM, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             dev_max) != cudaSuccess) {
      cudaGetLastError();
      return GLIDE_ERR_CUDA;
    }
    return GLIDE_OK;
  });
}

int launch_decode_stream(glide_ctx *ctx, const DecodeParams &p, int schedule, cudaStream_t stream) {
  if (schedule < 0 || size_t(schedule) >= ctx->stream_scheds.size()) return GLIDE_ERR_INVALID_ARG;
  const glide_ctx::StreamSchedule &sc = ctx->stream_scheds[size_t(schedule)];
  if (p.launch_tag == 1 && ctx->launch_wrapped) {
    // the launch counter has gone round: a record slot that no schedule has written for 2^32 launches could carry this
    // launch's tag already, so the records start from zero again (stream-ordered behind the preceding launch)
    if (cudaMemsetAsync(ctx->ws + ctx->off_partials, 0, ctx->off_stream_segs - ctx->off_partials, stream) != cudaSuccess) {
      cudaGetLastError();
      return GLIDE_ERR_CUDA;
    }
    ctx->launch_wrapped = false;
  }
  StreamParams sp{};
  sp.segs = reinterpret_cast<const StreamSegment *>(ctx->ws + ctx->off_stream_segs) + sc.seg_base;
  for (int c = 0; c <= ctx->decode_grid; ++c) sp.cta_seg_begin[c] = sc.range_begin[size_t(c) * kWarps];
  sp.tmaps = reinterpret_cast<const CUtensorMap_st *>(ctx->ws + ctx->off_tmaps);
  sp.max_segs = ctx->stream_max_segs;
  sp.heads_contiguous = ctx->stream_heads_contiguous ? 1 : 0;
  sp.kv4d = ctx->tmaps_kv4d ? 1 : 0;
  sp.t_off = int32_t(ctx->stream_smem - 1024 - size_t(ctx->stream_max_segs) * 8);
  return dispatch_stream(ctx->G, stream_mode(ctx), [&](auto gg, auto ss, auto mm) -> int {
    constexpr int G = decltype(gg)::value, S = decltype(ss)::value;
    constexpr int SUM = decltype(mm)::value;   // the kernel's MODE
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(unsigned(ctx->decode_grid));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = ctx->stream_smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
#ifdef GLIDE_NO_PDL
    cfg.numAttrs = 0;
#else
    cfg.numAttrs = 1;
#endif
    const cudaError_t err = p.seq_off ? cudaLaunchKernelEx(&cfg, glide_decode_stream_kernel<G, S, SUM, true>, p, sp)
                                      : cudaLaunchKernelEx(&cfg, glide_decode_stream_kernel<G, S, SUM, false>, p, sp);
    if (err != cudaSuccess) {
      cudaGetLastError();
      return GLIDE_ERR_CUDA;
    }
    return GLIDE_OK;
  });
}

}  // namespace glide
