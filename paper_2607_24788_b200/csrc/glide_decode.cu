// Fused GLIDE decode step: ONE persistent launch over all layers.
//
// CTAs pull work items from a static, longest-first list through an atomic counter:
//   window item  -- a run of ring slots of one (layer, sequence, KV head) unit: streams K/V rows
//                   once for all G query heads of the KV head, online softmax, writes a split-K
//                   partial (m, l, acc) to scratch;
//   state item   -- a block of rows of the unit's recurrent state: folds the token that leaves the
//                   window (S += phi(k) v^T, z += phi(k), in place, fp32) and reads the updated
//                   rows out against phi(q) of the G heads, writes a linear partial (a, b).
// Each finished item takes a ticket on its unit; the CTA that takes the last ticket merges the
// partials in fixed order with the current token's own term under the shared normaliser, writes
// the output, stores k,v in the ring slot and clears the ticket.  Nothing ever spins.
// The last CTA to leave the kernel resets the work counter and advances the position counters,
// so the step needs no host-side state and no second launch.
#include <algorithm>

#include "glide_device.cuh"

namespace glide {

namespace {

template <int D, int G>
constexpr int scratch_floats() {
  // window items: [warps][G][D+2]; state items: [row groups][G][D]; feature kernel: [D] + reductions
  constexpr int NW = kDecodeThreads / 32;
  constexpr int RPI = kDecodeThreads / (D / 4);
  return (NW * G * (D + 2) > RPI * G * D) ? NW * G * (D + 2) : RPI * G * D;
}

template <typename T, int D, int G, int DP = D>
struct DecodeSmem {
  float scratch[scratch_floats<D, G>()];
  float phiq[G][DP];
  float phik[DP];
  float ve[D];
  float scur[G];
  float M[G];
  float inv[G];
  float invl[G];   // sum-of-terms merges: 1 / (phi(q) z), or 0 while the state is empty
  int item;
  int last;
};

// ---- window item ---------------------------------------------------------------------------
template <typename T, int D, int G, int DP>
__device__ __forceinline__ void window_item(const DecodeParams &p, const WorkItem &it, const LayerDev &ld,
                                            int64_t t, int b, int g, float *rec, DecodeSmem<T, D, G, DP> &sm) {
  constexpr int E = D / 32;
  constexpr int NW = kDecodeThreads / 32;
  constexpr int U = 4;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const size_t unit_rows = (size_t(b) * p.Hkv + g) * size_t(ld.cap);
  const T *Kb = reinterpret_cast<const T *>(p.ws + ld.ringK) + unit_rows * D;
  const T *Vb = reinterpret_cast<const T *>(p.ws + ld.ringV) + unit_rows * D;

  float qr[G][E];
#pragma unroll
  for (int h = 0; h < G; ++h) {
    const int head = p.heads_of[g * G + h];
    const T *qp = reinterpret_cast<const T *>(p.q) + ((size_t(it.layer) * p.B + b) * p.H + head) * D + lane * E;
    load_elems<T, E>(qp, qr[h]);
#pragma unroll
    for (int i = 0; i < E; ++i) qr[h][i] *= p.scale_log2;
  }
  float acc[G][E], m[G], l[G];
#pragma unroll
  for (int h = 0; h < G; ++h) {
    m[h] = -CUDART_INF_F;
    l[h] = 0.f;
#pragma unroll
    for (int i = 0; i < E; ++i) acc[h][i] = 0.f;
  }
  // Valid rows: the window's tokens other than the current one.  While the ring is not full they
  // are slots [0, t); afterwards every slot but t mod cap, which holds the token leaving the window.
  const int64_t lim = t < ld.cap ? t : ld.cap;
  const int64_t cur = t % ld.cap;
  const int end = it.begin + it.count;
  for (int s0 = it.begin + warp; s0 < end; s0 += NW * U) {
    float kx[U][E], vx[U][E];
    bool ok[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int s = s0 + u * NW;
      ok[u] = s < end && s < lim && s != cur;
      if (ok[u]) {
        load_elems<T, E>(Kb + size_t(s) * D + lane * E, kx[u]);
        load_elems<T, E>(Vb + size_t(s) * D + lane * E, vx[u]);
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u)
      if (ok[u]) online_row<E, G>(qr, kx[u], vx[u], m, l, acc);
  }
  // combine the warps
  float *red = sm.scratch;  // [NW][G][D+2]
#pragma unroll
  for (int h = 0; h < G; ++h) {
    float *r = red + (size_t(warp) * G + h) * (D + 2);
#pragma unroll
    for (int i = 0; i < E; ++i) r[lane * E + i] = acc[h][i];
    if (lane == 0) {
      r[D] = m[h];
      r[D + 1] = l[h];
    }
  }
  __syncthreads();
  for (int idx = tid; idx < G * D; idx += kDecodeThreads) {
    const int h = idx / D, c = idx - h * D;
    float M = -CUDART_INF_F;
#pragma unroll
    for (int w = 0; w < NW; ++w) M = fmaxf(M, red[(size_t(w) * G + h) * (D + 2) + D]);
    float val = 0.f, lsum = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const float *r = red + (size_t(w) * G + h) * (D + 2);
      const float f = r[D] == -CUDART_INF_F ? 0.f : exp2f(r[D] - M);
      val = fmaf(r[c], f, val);
      lsum = fmaf(r[D + 1], f, lsum);
    }
    rec[idx] = val;
    if (c == 0) {
      rec[G * D + h] = M;
      rec[G * D + G + h] = lsum;
    }
  }
}

// ---- state item ----------------------------------------------------------------------------
// DP: the feature dimension (rows of S): D for the parameter-free map, 2 D for the learned map, whose phi(k_e) and
// phi(q_h) were written by the feature kernel in front of this launch (p.phit).  A gated context decays the rows by
// the gate of the token that enters the state.
template <typename T, int D, int G, int DP>
__device__ __forceinline__ void state_item(const DecodeParams &p, const WorkItem &it, const LayerDev &ld, int64_t t,
                                           int b, int g, float *rec, DecodeSmem<T, D, G, DP> &sm) {
  constexpr int E = D / 32;
  constexpr int NW = kDecodeThreads / 32;
  constexpr int TPR = D / 4;                   // threads per state row (float4 each)
  constexpr int RPI = kDecodeThreads / TPR;    // rows per iteration
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (t < ld.wlin) return;                     // nothing has reached the state yet: S,z are still zero
  const int ub = b * p.Hkv + g;
  const T *ke, *ve;
  float gamma = 1.f;                           // gate of the token that enters the state
  if (ld.wlin == 0) {  // no ring, or a state that holds every token: the current token is folded now
    ke = reinterpret_cast<const T *>(p.k) + size_t(it.unit) * D;
    ve = reinterpret_cast<const T *>(p.v) + size_t(it.unit) * D;
    if (p.gated && p.gate) gamma = p.gate[it.unit];
  } else {          // slot t mod cap holds token t - w
    const size_t slot = size_t(ub) * size_t(ld.cap) + size_t(t % ld.cap);
    ke = reinterpret_cast<const T *>(p.ws + ld.ringK) + slot * D;
    ve = reinterpret_cast<const T *>(p.ws + ld.ringV) + slot * D;
    if (p.gated) gamma = reinterpret_cast<const float *>(p.ws + ld.ringG)[slot];
  }
  const int r_end = it.begin + it.count;
  if constexpr (DP == D) {
    if (warp == 0) {
      float x[E], y[E];
      load_elems<T, E>(ke + lane * E, x);
      load_elems<T, E>(ve + lane * E, y);
      warp_phi<E>(x);
#pragma unroll
      for (int i = 0; i < E; ++i) {
        sm.phik[lane * E + i] = x[i];
        sm.ve[lane * E + i] = y[i];
      }
    }
    for (int h = warp; h < G; h += NW) {
      const int head = p.heads_of[g * G + h];
      float x[E];
      load_elems<T, E>(reinterpret_cast<const T *>(p.q) + ((size_t(it.layer) * p.B + b) * p.H + head) * D + lane * E, x);
      warp_phi<E>(x);
#pragma unroll
      for (int i = 0; i < E; ++i) sm.phiq[h][lane * E + i] = x[i];
    }
  } else {
    // the rows of this item from the feature kernel's output: [unit][DP / 16][G + 1][16]
    const float *ph = p.phit + size_t(it.unit - p.layer_begin * p.B * p.Hkv) * DP * (G + 1);
    for (int idx = tid; idx < (G + 1) * it.count; idx += kDecodeThreads) {
      const int h = idx / it.count, r = it.begin + idx % it.count;
      const float val = ph[(size_t(r >> 4) * (G + 1) + h) * 16 + (r & 15)];
      if (h < G) sm.phiq[h][r] = val; else sm.phik[r] = val;
    }
    for (int c = tid; c < D; c += kDecodeThreads) sm.ve[c] = to_f32(ve[c]);
  }
  __syncthreads();

  const int c4 = tid % TPR, rsub = tid / TPR;
  float *Sb = reinterpret_cast<float *>(p.ws + ld.S) + size_t(ub) * DP * D;
  const float4 v4 = *reinterpret_cast<const float4 *>(&sm.ve[c4 * 4]);
  float4 a[G];
#pragma unroll
  for (int h = 0; h < G; ++h) a[h] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
  for (int r = it.begin + rsub; r < r_end; r += RPI) {
    float4 *sp = reinterpret_cast<float4 *>(Sb + size_t(r) * D + c4 * 4);
    float4 s = *sp;
    const float pk = sm.phik[r];
    s.x = fmaf(pk, v4.x, gamma * s.x);
    s.y = fmaf(pk, v4.y, gamma * s.y);
    s.z = fmaf(pk, v4.z, gamma * s.z);
    s.w = fmaf(pk, v4.w, gamma * s.w);
    *sp = s;
#pragma unroll
    for (int h = 0; h < G; ++h) {
      const float f = sm.phiq[h][r];
      a[h].x = fmaf(f, s.x, a[h].x);
      a[h].y = fmaf(f, s.y, a[h].y);
      a[h].z = fmaf(f, s.z, a[h].z);
      a[h].w = fmaf(f, s.w, a[h].w);
    }
  }
  // z rows of this block and the b_h readout: warp 0
  if (warp == 0) {
    float *zb = reinterpret_cast<float *>(p.ws + ld.z) + size_t(ub) * DP;
    float bp[G];
#pragma unroll
    for (int h = 0; h < G; ++h) bp[h] = 0.f;
    for (int r = it.begin + lane; r < r_end; r += 32) {
      const float zn = fmaf(gamma, zb[r], sm.phik[r]);
      zb[r] = zn;
#pragma unroll
      for (int h = 0; h < G; ++h) bp[h] = fmaf(sm.phiq[h][r], zn, bp[h]);
    }
#pragma unroll
    for (int h = 0; h < G; ++h) {
      const float bs = warp_sum(bp[h]);
      if (lane == 0) {
        rec[G * D + h] = bs;
        rec[G * D + G + h] = 0.f;
      }
    }
  }
  float *red = sm.scratch;  // [RPI][G][D]
#pragma unroll
  for (int h = 0; h < G; ++h) *reinterpret_cast<float4 *>(red + (size_t(rsub) * G + h) * D + c4 * 4) = a[h];
  __syncthreads();
  for (int idx = tid; idx < G * D; idx += kDecodeThreads) {
    float val = 0.f;
#pragma unroll
    for (int rs = 0; rs < RPI; ++rs) val += red[size_t(rs) * G * D + idx];
    rec[idx] = val;
  }
}

// ---- merge (last ticket of a unit) -----------------------------------------------------------
template <typename T, int D, int G, int DP>
__device__ __forceinline__ void merge_unit(const DecodeParams &p, const WorkItem &it, const LayerDev &ld, int64_t t,
                                           int b, int g, DecodeSmem<T, D, G, DP> &sm) {
  constexpr int E = D / 32;
  constexpr int NW = kDecodeThreads / 32;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int ub = b * p.Hkv + g;
  const int per_unit = ld.n_win_items + ld.n_state_items;
  const float *rec0 = p.partials + ld.part_base + size_t(ub) * per_unit * p.rec_floats;
  const bool has_win = ld.cap > 0;
  const bool has_state = ld.n_state_items > 0 && t >= ld.wlin;
  const T *kt = reinterpret_cast<const T *>(p.k) + size_t(it.unit) * D;
  const T *vt = reinterpret_cast<const T *>(p.v) + size_t(it.unit) * D;

  if (has_win) {  // the current token's own logit, per head
    float kx[E];
    load_elems<T, E>(kt + lane * E, kx);
    for (int h = warp; h < G; h += NW) {
      const int head = p.heads_of[g * G + h];
      float qx[E];
      load_elems<T, E>(reinterpret_cast<const T *>(p.q) + ((size_t(it.layer) * p.B + b) * p.H + head) * D + lane * E, qx);
      float part = 0.f;
#pragma unroll
      for (int i = 0; i < E; ++i) part = fmaf(qx[i] * p.scale_log2, kx[i], part);
      part = warp_sum(part);
      if (lane == 0) sm.scur[h] = part;
    }
  }
  __syncthreads();
  if (tid < G) {
    const int h = tid;
    // shared normaliser: m* = max(window max, 0), the linear terms carry the factor exp(-m*) <= 1;
    // sum of two normalised terms: the window is normalised on its own, against its own maximum
    const bool shared = ld.merge == GLIDE_MERGE_SHARED;
    float M = (shared && has_state) ? 0.f : -CUDART_INF_F;   // the floor belongs to the linear terms (logit 0)
    for (int i = 0; i < ld.n_win_items; ++i) M = fmaxf(M, __ldcg(rec0 + size_t(i) * p.rec_floats + G * D + h));
    if (has_win) M = fmaxf(M, sm.scur[h]);
    float den = 0.f;
    for (int i = 0; i < ld.n_win_items; ++i) {
      const float *r = rec0 + size_t(i) * p.rec_floats;
      const float mi = __ldcg(r + G * D + h);
      den = fmaf(__ldcg(r + G * D + G + h), exp2f(mi - M), den);
    }
    if (has_win) den += exp2f(sm.scur[h] - M);
    float invl = 0.f;
    if (has_state) {
      float bsum = 0.f;
      for (int i = 0; i < ld.n_state_items; ++i)
        bsum += __ldcg(rec0 + size_t(ld.n_win_items + i) * p.rec_floats + G * D + h);
      if (shared) den = fmaf(exp2f(-M), bsum, den);
      else invl = bsum > 0.f ? 1.0f / bsum : 0.f;
    }
    sm.M[h] = M;
    sm.inv[h] = den > 0.f ? 1.0f / den : 0.f;   // den = 0 only for a sum-of-terms layer without a window
    sm.invl[h] = invl;
  }
  __syncthreads();
  T *outp = reinterpret_cast<T *>(p.out);
  for (int idx = tid; idx < G * D; idx += kDecodeThreads) {
    const int h = idx / D, c = idx - h * D;
    const float M = sm.M[h];
    float num = 0.f;
    for (int i = 0; i < ld.n_win_items; ++i) {
      const float *r = rec0 + size_t(i) * p.rec_floats;
      num = fmaf(__ldcg(r + idx), exp2f(__ldcg(r + G * D + h) - M), num);
    }
    if (has_win) num = fmaf(exp2f(sm.scur[h] - M), to_f32(vt[c]), num);
    float lin = 0.f;
    if (has_state) {
      float asum = 0.f;
      for (int i = 0; i < ld.n_state_items; ++i) asum += __ldcg(rec0 + size_t(ld.n_win_items + i) * p.rec_floats + idx);
      if (ld.merge == GLIDE_MERGE_SHARED) num = fmaf(exp2f(-M), asum, num);
      else lin = asum * sm.invl[h];
    }
    const int head = p.heads_of[g * G + h];
    from_f32(outp + ((size_t(it.layer) * p.B + b) * p.H + head) * D + c, fmaf(num, sm.inv[h], lin));
  }
  if (has_win) {  // every reader of slot t mod cap has finished: store the new row
    const size_t row = (size_t(ub) * size_t(ld.cap) + size_t(t % ld.cap)) * D;
    T *Kd = reinterpret_cast<T *>(p.ws + ld.ringK) + row;
    T *Vd = reinterpret_cast<T *>(p.ws + ld.ringV) + row;
    for (int c = tid; c < D; c += kDecodeThreads) {
      Kd[c] = kt[c];
      Vd[c] = vt[c];
    }
    if (p.gated && tid == 0)   // the token's gate waits in the ring with it
      reinterpret_cast<float *>(p.ws + ld.ringG)[size_t(ub) * size_t(ld.cap) + size_t(t % ld.cap)] =
          p.gate ? p.gate[it.unit] : 1.f;
  }
}

template <typename T, int D, int G, int DP>
__global__ void __launch_bounds__(kDecodeThreads) glide_decode_kernel(const DecodeParams p) {
  __shared__ DecodeSmem<T, D, G, DP> sm;
  const int tid = threadIdx.x;
  const int units_per_layer = p.B * p.Hkv;
  for (;;) {
    __syncthreads();
    if (tid == 0) sm.item = atomicAdd(&p.ctl->work_counter, 1);
    __syncthreads();
    const int idx = sm.item;
    if (idx >= p.n_items) break;
    const WorkItem it = p.items[idx];
    if (it.layer < 0 || it.layer >= p.L || it.unit < 0) {  // corrupted list: record and skip
      if (tid == 0) atomicExch(p.status, kDevBadItem);
      continue;
    }
    if (it.layer < p.layer_begin || it.layer >= p.layer_begin + p.layer_count) continue;   // not a layer of this launch
    const LayerDev ld = p.layers[it.layer];
    const int ub = it.unit - it.layer * units_per_layer;
    const int b = ub / p.Hkv, g = ub - b * p.Hkv;
    GLIDE_CHECK_OR(ub >= 0 && ub < units_per_layer && it.begin >= 0 && it.count >= 0 &&
                       it.begin + it.count <= (it.kind == kItemWindow ? ld.cap : int64_t(DP)),
                   p.status, continue);   // (uniform over the CTA: every thread sees the same item)
    const int64_t t = p.n_dev[it.layer] + (p.seq_off ? p.seq_off[b] : 0);   // position of this sequence
    if (t < 0) continue;   // parked slot: nothing is read or written for it (every item of the unit takes this branch)
    const int per_unit = ld.n_win_items + ld.n_state_items;
    float *rec = p.partials + ld.part_base + (size_t(ub) * per_unit + it.part) * p.rec_floats;
    if (it.kind == kItemWindow)
      window_item<T, D, G, DP>(p, it, ld, t, b, g, rec, sm);
    else
      state_item<T, D, G, DP>(p, it, ld, t, b, g, rec, sm);
    __threadfence();
    __syncthreads();
    if (tid == 0) sm.last = atomicAdd(&p.tickets[it.unit], 1) == per_unit - 1;
    __syncthreads();
    if (sm.last) {
      __threadfence();
      merge_unit<T, D, G, DP>(p, it, ld, t, b, g, sm);
      if (tid == 0) p.tickets[it.unit] = 0;
    }
  }
  if (tid == 0) {
    __threadfence();
    if (atomicAdd(&p.ctl->done_counter, 1) == int(gridDim.x) - 1) {
      // every CTA has drained the list: re-arm it and advance the positions
      p.ctl->work_counter = 0;
      p.ctl->done_counter = 0;
      for (int l = 0; l < p.layer_count; ++l) p.n_dev[p.layer_begin + l] += 1;
      __threadfence();
    }
  }
}

// ---- learned feature map of one decode step ------------------------------------------------------
// phi_W(x) = [softmax(W^T x); softmax(-W^T x)] of the step's queries and of the key that enters the state, for every
// unit of the launch, into p.phit [unit][DP / 16][G + 1][16] (row G: the key).  kPhiSplit warps per (layer, KV head,
// row of the group), each with its share of the rows of the head's d x d matrix: every lane owns D / 32 outputs
// (the partial sums of the warps meet in shared memory), the matrix is streamed row by row, coalesced, many rows in
// flight, for kPhiSeqs sequences of the batch at a time.
constexpr int kPhiSplit = 2;    // warps per matrix
constexpr int kPhiHeads = 2;    // matrices per CTA
template <typename T, int D, int G, int kPhiSeqs>
__global__ void __launch_bounds__(kPhiSplit * kPhiHeads * 32) glide_decode_phi_kernel(const DecodeParams p) {
  constexpr int DP = 2 * D;
  constexpr int E = D / 32;
  __shared__ float part[kPhiHeads][kPhiSplit][kPhiSeqs][D];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int hslot = warp / kPhiSplit, split = warp % kPhiSplit;
  const int total = p.layer_count * p.Hkv * (G + 1);
  int wid = blockIdx.x * kPhiHeads + hslot;
  const bool active = wid < total;
  if (!active) wid = total - 1;   // (keeps the warp in the CTA's barriers; it writes nothing)
  const int row = wid % (G + 1);
  const int g = (wid / (G + 1)) % p.Hkv;
  const int lrel = wid / ((G + 1) * p.Hkv);
  const int layer = p.layer_begin + lrel;
  const LayerDev ld = p.layers[layer];
  const bool has_work = active && !(row == G && !ld.evicts);
  const int head = row < G ? p.heads_of[g * G + row] : 0;
  const T *W = row < G ? reinterpret_cast<const T *>(p.wq) + (size_t(layer) * p.H + head) * D * D
                       : reinterpret_cast<const T *>(p.wk) + (size_t(layer) * p.Hkv + g) * D * D;
  // the per-item kernels index q, k, v with the absolute layer (their base pointers are moved back)
  const int lq = p.tensors_absolute ? layer : lrel;
  const int64_t n = p.n_dev[layer];
  for (int b0 = 0; b0 < p.B; b0 += kPhiSeqs) {
    float x[kPhiSeqs][E], y[kPhiSeqs][E];
    bool live[kPhiSeqs];
#pragma unroll
    for (int bi = 0; bi < kPhiSeqs; ++bi) {
      const int b = b0 + bi;
      live[bi] = false;
#pragma unroll
      for (int e = 0; e < E; ++e) x[bi][e] = y[bi][e] = 0.f;
      if (b >= p.B || !has_work) continue;
      const int64_t t = n + (p.seq_off ? p.seq_off[b] : 0);
      if (t < 0) continue;   // parked slot
      const int ub = b * p.Hkv + g;
      const T *src;
      if (row < G) {
        src = reinterpret_cast<const T *>(p.q) + ((size_t(lq) * p.B + b) * p.H + head) * D;
      } else if (t < ld.wlin) {
        continue;            // nothing enters the state at this step
      } else if (ld.wlin == 0) {
        src = reinterpret_cast<const T *>(p.k) + (size_t(lq) * p.B * p.Hkv + ub) * D;
      } else {
        src = reinterpret_cast<const T *>(p.ws + ld.ringK) + (size_t(ub) * size_t(ld.cap) + size_t(t % ld.cap)) * D;
      }
      live[bi] = true;
      load_elems<T, E>(src + lane * E, x[bi]);
    }
    if (has_work)
      warp_project_rows<T, D, kPhiSeqs, (sizeof(T) == 2 ? 8 : 4)>(W, x, y, split * (32 / kPhiSplit),
                                                                  (split + 1) * (32 / kPhiSplit));
    __syncthreads();   // the previous batch's partial sums have been read
    if (split > 0) {
#pragma unroll
      for (int bi = 0; bi < kPhiSeqs; ++bi)
#pragma unroll
        for (int e = 0; e < E; ++e) part[hslot][split][bi][lane * E + e] = y[bi][e];
    }
    __syncthreads();
    if (split == 0 && has_work) {
#pragma unroll
      for (int bi = 0; bi < kPhiSeqs; ++bi) {
        if (!live[bi]) continue;
        float lo[E], hi[E];
#pragma unroll
        for (int e = 0; e < E; ++e) {
          float sum = y[bi][e];
#pragma unroll
          for (int sp = 1; sp < kPhiSplit; ++sp) sum += part[hslot][sp][bi][lane * E + e];
          lo[e] = sum;
          hi[e] = -sum;
        }
        warp_phi<E>(lo);
        warp_phi<E>(hi);
        const size_t unit = (size_t(lrel) * p.B + (b0 + bi)) * p.Hkv + g;
        float *ph = p.phit + unit * DP * (G + 1);
#pragma unroll
        for (int e = 0; e < E; ++e) {
          const int j = lane * E + e;
          ph[(size_t(j >> 4) * (G + 1) + row) * 16 + (j & 15)] = lo[e];
          ph[(size_t((D + j) >> 4) * (G + 1) + row) * 16 + (j & 15)] = hi[e];
        }
      }
    }
  }
}

__global__ void glide_advance_kernel(int64_t *n_dev, int layer_begin, int layer_count, int64_t T) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < layer_count) n_dev[layer_begin + i] += T;
}

}  // namespace

// q, k, v, out are the tensors of the layer range [layer_begin, layer_begin + layer_count).  The per-item kernels
// index them with the absolute layer, so they get base pointers moved back by layer_begin layers (never
// dereferenced below the range); the streaming kernel's per-range schedules are numbered from the range's start.
DecodeParams make_decode_params(const glide_ctx *ctx, int layer_begin, int layer_count, const void *q, const void *k,
                                const void *v, void *out) {
  DecodeParams p{};
  if (ctx->decode_kind != 2 && layer_begin > 0) {
    const size_t row = size_t(ctx->cfg.head_dim) * ctx->elem * size_t(ctx->cfg.batch) * size_t(layer_begin);
    q = static_cast<const unsigned char *>(q) - row * ctx->cfg.n_q_heads;
    out = static_cast<unsigned char *>(out) - row * ctx->cfg.n_q_heads;
    k = static_cast<const unsigned char *>(k) - row * ctx->cfg.n_kv_heads;
    v = static_cast<const unsigned char *>(v) - row * ctx->cfg.n_kv_heads;
  }
  p.ws = ctx->ws;
  p.layers = reinterpret_cast<const LayerDev *>(ctx->ws + ctx->off_layers);
  p.items = reinterpret_cast<const WorkItem *>(ctx->ws + ctx->off_items);
  p.heads_of = reinterpret_cast<const int32_t *>(ctx->ws + ctx->off_heads);
  p.ctl = reinterpret_cast<Control *>(ctx->ws + ctx->off_ctl);
  p.status = &p.ctl->status;
  p.tickets = reinterpret_cast<int32_t *>(ctx->ws + ctx->off_tickets);
  p.partials = reinterpret_cast<float *>(ctx->ws + ctx->off_partials);
  p.n_dev = reinterpret_cast<int64_t *>(ctx->ws + ctx->off_ndev);
  p.seq_off = ctx->ragged ? reinterpret_cast<const int64_t *>(ctx->ws + ctx->off_seqoff) : nullptr;
  p.phit = ctx->cfg.phi == GLIDE_PHI_PROJ_SOFTMAX2 ? reinterpret_cast<float *>(ctx->ws + ctx->off_phit) : nullptr;
  p.wq = ctx->cfg.phi_wq;
  p.wk = ctx->cfg.phi_wk;
  p.dp = ctx->dp;
  p.gated = ctx->cfg.gated;
  p.gate = nullptr;
  p.tensors_absolute = ctx->decode_kind != 2;
  if (++ctx->launch_seq == 0) {   // tag 0 is what a never-written record holds
    ctx->launch_seq = 1;
    ctx->launch_wrapped = true;
  }
  p.launch_tag = ctx->launch_seq;
  p.q = q;
  p.k = k;
  p.v = v;
  p.out = out;
  p.n_items = ctx->n_items;
  p.L = ctx->cfg.n_layers;
  p.B = ctx->cfg.batch;
  p.H = ctx->cfg.n_q_heads;
  p.Hkv = ctx->cfg.n_kv_heads;
  p.rec_floats = ctx->decode_kind == 2 ? ctx->stream_rec_floats : ctx->rec_floats;
  p.scale_log2 = ctx->scale * kLog2e;
  p.t_host = ctx->n_host[size_t(layer_begin)];
  p.layer_begin = layer_begin;
  p.layer_count = layer_count;
  return p;
}

namespace {
// f(TypeTag<T>, IntTag<D>, IntTag<G>, IntTag<DP>) for the configured dtype, head_dim, group size and feature dimension
template <typename F>
int dispatch_decode(const glide_ctx *ctx, F &&f) {
  return dispatch_config(ctx->cfg.io_dtype, ctx->cfg.head_dim, ctx->G, [&](auto tt, auto dd, auto gg) -> int {
    constexpr int D = decltype(dd)::value;
    if (ctx->dp == D) return f(tt, dd, gg, IntTag<D>{});
    return f(tt, dd, gg, IntTag<2 * D>{});
  });
}
}  // namespace

int decode_occupancy(const glide_ctx *ctx, int *blocks_per_sm) {
  return dispatch_decode(ctx, [&](auto tt, auto dd, auto gg, auto pp) -> int {
    using T = typename decltype(tt)::type;
    constexpr int D = decltype(dd)::value, G = decltype(gg)::value, DP = decltype(pp)::value;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, glide_decode_kernel<T, D, G, DP>, kDecodeThreads,
                                                      0) != cudaSuccess) {
      cudaGetLastError();
      return GLIDE_ERR_CUDA;
    }
    return GLIDE_OK;
  });
}

// the step's learned features, in front of the decode kernel of the same layers
int launch_decode_phi(glide_ctx *ctx, const DecodeParams &p, cudaStream_t stream) {
  if (ctx->cfg.phi != GLIDE_PHI_PROJ_SOFTMAX2) return GLIDE_OK;
  return dispatch_config(ctx->cfg.io_dtype, ctx->cfg.head_dim, ctx->G, [&](auto tt, auto dd, auto gg) -> int {
    using T = typename decltype(tt)::type;
    constexpr int D = decltype(dd)::value, G = decltype(gg)::value;
    const unsigned mats = unsigned(p.layer_count) * unsigned(p.Hkv) * unsigned(G + 1);
    const unsigned grid = (mats + kPhiHeads - 1) / kPhiHeads, block = kPhiSplit * kPhiHeads * 32;
    // (a single sequence gets its own instantiation: no work for absent sequences)
    if (p.B == 1)
      glide_decode_phi_kernel<T, D, G, 1><<<grid, block, 0, stream>>>(p);
    else
      glide_decode_phi_kernel<T, D, G, 4><<<grid, block, 0, stream>>>(p);
    if (cudaGetLastError() != cudaSuccess) return GLIDE_ERR_CUDA;
    return GLIDE_OK;
  });
}

int launch_decode(glide_ctx *ctx, int layer_begin, int layer_count, const void *q, const void *k, const void *v,
                  const float *gate, void *out, cudaStream_t stream) {
  const int L = ctx->cfg.n_layers;
  if (ctx->decode_kind == 2 && layer_count != L) {
    // the streaming kernel has a schedule for the whole stack and one per layer: a partial range is one launch per layer
    const size_t qrow = size_t(ctx->cfg.head_dim) * ctx->elem * size_t(ctx->cfg.batch) * ctx->cfg.n_q_heads;
    const size_t krow = size_t(ctx->cfg.head_dim) * ctx->elem * size_t(ctx->cfg.batch) * ctx->cfg.n_kv_heads;
    for (int i = 0; i < layer_count; ++i) {
      DecodeParams pl = make_decode_params(ctx, layer_begin + i, 1, static_cast<const unsigned char *>(q) + qrow * i,
                                           static_cast<const unsigned char *>(k) + krow * i,
                                           static_cast<const unsigned char *>(v) + krow * i,
                                           static_cast<unsigned char *>(out) + qrow * i);
      pl.gate = gate ? gate + size_t(i) * ctx->cfg.batch * ctx->cfg.n_kv_heads : nullptr;
      int rc = launch_decode_phi(ctx, pl, stream);
      if (rc) return rc;
      rc = launch_decode_stream(ctx, pl, 1 + layer_begin + i, stream);
      if (rc) return rc;
    }
    return GLIDE_OK;
  }
  DecodeParams p = make_decode_params(ctx, layer_begin, layer_count, q, k, v, out);
  p.gate = gate;
  const int rc = launch_decode_phi(ctx, p, stream);
  if (rc) return rc;
  if (ctx->decode_kind == 2) return launch_decode_stream(ctx, p, 0, stream);
  if (ctx->decode_kind == 1) return launch_decode_mma(ctx, p, stream);
  return dispatch_decode(ctx, [&](auto tt, auto dd, auto gg, auto pp) -> int {
    using T = typename decltype(tt)::type;
    constexpr int D = decltype(dd)::value, G = decltype(gg)::value, DP = decltype(pp)::value;
    glide_decode_kernel<T, D, G, DP><<<ctx->decode_grid, kDecodeThreads, 0, stream>>>(p);
    if (cudaGetLastError() != cudaSuccess) return GLIDE_ERR_CUDA;
    return GLIDE_OK;
  });
}

// ---- allocation-free decode variant ---------------------------------------------------------------
// Split-K scratch of the CUDA-core decode kernel inside the library image instead of the caller's workspace.
// In host code `g_noalloc_scratch` is only a handle for the symbol, not a device address: the address is
// looked up once per device with cudaGetSymbolAddress and that pointer is what the kernel receives.
static __device__ __align__(256) unsigned char g_noalloc_scratch[GLIDE_NOALLOC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
unsigned char *g_noalloc_ptr[kMaxDevices] = {};   // device address of the buffer, per device (nullptr: not looked up yet)
}  // namespace

int launch_decode_noalloc(glide_ctx *ctx, const void *q, const void *k, const void *v, void *out, cudaStream_t stream) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    cudaGetLastError();
    return GLIDE_ERR_CUDA;
  }
  if (dev != ctx->device) return GLIDE_ERR_INVALID_ARG;   // the context lives on another device
  const size_t units = size_t(ctx->cfg.n_layers) * ctx->cfg.batch * ctx->cfg.n_kv_heads;
  const size_t tickets_off = 256;
  const size_t partials_off = tickets_off + (units * sizeof(int32_t) + 255) / 256 * 256;
  const size_t need = partials_off + ctx->item_part_floats * sizeof(float);
  if (need > size_t(GLIDE_NOALLOC_SCRATCH_BYTES)) return GLIDE_ERR_SCRATCH_LIMIT;
  if (!g_noalloc_ptr[dev]) {   // first call on this device: this device is current here
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) {
      cudaGetLastError();
      return GLIDE_ERR_CUDA;
    }
    g_noalloc_ptr[dev] = static_cast<unsigned char *>(ptr);
  }
  if (ctx->noalloc_grid == 0) {   // a host-side occupancy query, no allocation
    int per_sm = 0;
    if (decode_occupancy(ctx, &per_sm) != GLIDE_OK || per_sm < 1) return GLIDE_ERR_CUDA;
    ctx->noalloc_grid = std::max(1, std::min(ctx->n_items, ctx->sm_count * per_sm));
  }
  unsigned char *scratch = g_noalloc_ptr[dev];
  // control words and tickets must start at zero; the records are fully written before they are read
  if (cudaMemsetAsync(scratch, 0, partials_off, stream) != cudaSuccess) {
    cudaGetLastError();
    return GLIDE_ERR_CUDA;
  }
  DecodeParams p = make_decode_params(ctx, 0, ctx->cfg.n_layers, q, k, v, out);
  p.ctl = reinterpret_cast<Control *>(scratch);   // counters only: p.status stays the context's own word
  p.tickets = reinterpret_cast<int32_t *>(scratch + tickets_off);
  p.partials = reinterpret_cast<float *>(scratch + partials_off);
  p.rec_floats = ctx->rec_floats;   // this variant always runs the CUDA-core kernel and its record layout
  p.tensors_absolute = 1;
  const int rc = launch_decode_phi(ctx, p, stream);
  if (rc) return rc;
  return dispatch_decode(ctx, [&](auto tt, auto dd, auto gg, auto pp) -> int {
    using T = typename decltype(tt)::type;
    constexpr int D = decltype(dd)::value, G = decltype(gg)::value, DP = decltype(pp)::value;
    glide_decode_kernel<T, D, G, DP><<<ctx->noalloc_grid, kDecodeThreads, 0, stream>>>(p);
    if (cudaGetLastError() != cudaSuccess) return GLIDE_ERR_CUDA;
    return GLIDE_OK;
  });
}

int launch_advance(glide_ctx *ctx, int layer_begin, int layer_count, int64_t T, cudaStream_t stream) {
  int64_t *n_dev = reinterpret_cast<int64_t *>(ctx->ws + ctx->off_ndev);
  glide_advance_kernel<<<(layer_count + 63) / 64, 64, 0, stream>>>(n_dev, layer_begin, layer_count, T);
  if (cudaGetLastError() != cudaSuccess) return GLIDE_ERR_CUDA;
  return GLIDE_OK;
}

}  // namespace glide
