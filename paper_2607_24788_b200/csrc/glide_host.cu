// Host runtime of the GLIDE library: configuration checks, workspace layout, static decode
// work list, state export/import and bookkeeping.  No device memory is allocated here.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>

#include <nvtx3/nvToolsExt.h>

#include "glide_internal.h"

using namespace glide;

#ifndef GLIDE_RING_SKEW_BYTES
#define GLIDE_RING_SKEW_BYTES 66816          // 65 KiB + 1280 B
#endif
#ifndef GLIDE_RING_SKEW_MIN_BYTES
#define GLIDE_RING_SKEW_MIN_BYTES (size_t(1) << 30)
#endif
#ifndef GLIDE_STATE_ALIGN
#define GLIDE_STATE_ALIGN (2u << 20)
#endif

namespace {

// A named range around a call of the library, for timelines of profilers that follow NVTX (a no-op when none is
// attached: the header-only NVTX loader finds no tool and returns at once).
struct Range {
  explicit Range(const char *name) { nvtxRangePushA(name); }
  ~Range() { nvtxRangePop(); }
  Range(const Range &) = delete;
  Range &operator=(const Range &) = delete;
};

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

cudaStream_t as_stream(void *s) { return reinterpret_cast<cudaStream_t>(s); }

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int validate_config(const glide_config *c) {
  if (!c || !c->windows) return GLIDE_ERR_INVALID_ARG;
  if (c->n_layers < 1 || c->batch < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->max_tokens < 1)
    return GLIDE_ERR_INVALID_ARG;
  if (c->io_dtype != GLIDE_F32 && c->io_dtype != GLIDE_BF16) return GLIDE_ERR_INVALID_ARG;
  if (c->softmax_scale < 0.f || !std::isfinite(c->softmax_scale)) return GLIDE_ERR_INVALID_ARG;
  if (c->prefill_chunk < 0 || c->decode_chunk < 0 || c->decode_state_splits < 0) return GLIDE_ERR_INVALID_ARG;
  if (c->prefill_chunk % 16 != 0 || c->prefill_chunk > 1024) return GLIDE_ERR_INVALID_ARG;
  if (c->decode_impl < GLIDE_DECODE_AUTO || c->decode_impl > GLIDE_DECODE_STREAM) return GLIDE_ERR_INVALID_ARG;
  if (c->prefill_impl < GLIDE_PREFILL_AUTO || c->prefill_impl > GLIDE_PREFILL_FMA) return GLIDE_ERR_INVALID_ARG;
  if ((c->prefill_impl == GLIDE_PREFILL_MMA_SYNC || c->prefill_impl == GLIDE_PREFILL_TCGEN05) && c->io_dtype != GLIDE_BF16)
    return GLIDE_ERR_UNSUPPORTED;
  if ((c->prefill_impl == GLIDE_PREFILL_MMA_SYNC || c->prefill_impl == GLIDE_PREFILL_TCGEN05) && c->head_dim != 128)
    return GLIDE_ERR_UNSUPPORTED;
  if ((c->decode_impl == GLIDE_DECODE_MMA || c->decode_impl == GLIDE_DECODE_STREAM) && c->io_dtype != GLIDE_BF16)
    return GLIDE_ERR_UNSUPPORTED;
  for (int l = 0; l < c->n_layers; ++l)
    if (c->windows[l] < 0) return GLIDE_ERR_INVALID_ARG;
  if (c->phi != GLIDE_PHI_SOFTMAX && c->phi != GLIDE_PHI_PROJ_SOFTMAX2) return GLIDE_ERR_INVALID_ARG;
  if (c->gated != 0 && c->gated != 1) return GLIDE_ERR_INVALID_ARG;
  if (c->reserved_ != 0) return GLIDE_ERR_INVALID_ARG;
  if (c->phi == GLIDE_PHI_PROJ_SOFTMAX2) {
    if (!c->phi_wq || !c->phi_wk || !aligned16(c->phi_wq) || !aligned16(c->phi_wk)) return GLIDE_ERR_INVALID_ARG;
    // the learned map runs on the CUDA-core kernels, on the streaming decode kernel and (shared normaliser) on the
    // tcgen05 prefill kernel
    if (c->decode_impl == GLIDE_DECODE_MMA) return GLIDE_ERR_UNSUPPORTED;
    if (c->prefill_impl == GLIDE_PREFILL_MMA_SYNC) return GLIDE_ERR_UNSUPPORTED;
    if (c->prefill_impl == GLIDE_PREFILL_TCGEN05 && c->merge != GLIDE_MERGE_SHARED) return GLIDE_ERR_UNSUPPORTED;
  } else if (c->phi_wq || c->phi_wk) {
    return GLIDE_ERR_INVALID_ARG;
  }
  if (c->gated) {   // the gated recurrence runs on the CUDA-core kernels and on the streaming decode kernel
    if (c->decode_impl == GLIDE_DECODE_MMA) return GLIDE_ERR_UNSUPPORTED;
    if (c->prefill_impl == GLIDE_PREFILL_MMA_SYNC || c->prefill_impl == GLIDE_PREFILL_TCGEN05) return GLIDE_ERR_UNSUPPORTED;
  }
  if (c->merge < GLIDE_MERGE_SHARED || c->merge > GLIDE_MERGE_SUM_ALL) return GLIDE_ERR_INVALID_ARG;
  if (c->merge != GLIDE_MERGE_SHARED &&
      (c->decode_impl == GLIDE_DECODE_MMA || c->prefill_impl == GLIDE_PREFILL_MMA_SYNC))
    return GLIDE_ERR_UNSUPPORTED;   // sum-of-terms merges: not on the per-item tensor-core decode kernel nor on mma.sync
  if (c->head_dim != 64 && c->head_dim != 128) return GLIDE_ERR_UNSUPPORTED;
  if (c->n_q_heads % c->n_kv_heads != 0) return GLIDE_ERR_UNSUPPORTED;
  int G = c->n_q_heads / c->n_kv_heads;
  if (G != 1 && G != 2 && G != 4 && G != 8) return GLIDE_ERR_UNSUPPORTED;
  if (c->n_q_heads > 64) return GLIDE_ERR_UNSUPPORTED;
  if (c->max_tokens > (int64_t(1) << 30)) return GLIDE_ERR_UNSUPPORTED;
  if (c->q_to_kv) {
    std::vector<int> cnt(c->n_kv_heads, 0);
    for (int h = 0; h < c->n_q_heads; ++h) {
      int g = c->q_to_kv[h];
      if (g < 0 || g >= c->n_kv_heads) return GLIDE_ERR_INVALID_ARG;
      cnt[g]++;
    }
    for (int g = 0; g < c->n_kv_heads; ++g)
      if (cnt[g] != G) return GLIDE_ERR_UNSUPPORTED;
  }
  return GLIDE_OK;
}

}  // namespace

int glide::plan_context(const glide_config *cfg, glide_ctx *ctx, std::vector<WorkItem> *items) {
  int rc = validate_config(cfg);
  if (rc) return rc;
  ctx->cfg = *cfg;
  const int L = cfg->n_layers, B = cfg->batch, H = cfg->n_q_heads, Hkv = cfg->n_kv_heads, d = cfg->head_dim;
  ctx->G = H / Hkv;
  ctx->dp = cfg->phi == GLIDE_PHI_PROJ_SOFTMAX2 ? 2 * d : d;
  ctx->elem = cfg->io_dtype == GLIDE_F32 ? 4 : 2;
  ctx->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / std::sqrt(float(d));
  ctx->prefill_chunk = cfg->prefill_chunk ? cfg->prefill_chunk : 256;
  ctx->windows.assign(cfg->windows, cfg->windows + L);
  ctx->q_to_kv.resize(H);
  for (int h = 0; h < H; ++h) ctx->q_to_kv[h] = cfg->q_to_kv ? cfg->q_to_kv[h] : h / ctx->G;
  ctx->heads_of.assign(size_t(Hkv) * ctx->G, 0);
  {
    std::vector<int> fill(Hkv, 0);
    for (int h = 0; h < H; ++h) {
      int g = ctx->q_to_kv[h];
      ctx->heads_of[size_t(g) * ctx->G + fill[g]++] = h;
    }
  }
  ctx->cfg.windows = nullptr;
  ctx->cfg.q_to_kv = nullptr;
  const int dp = ctx->dp;
  ctx->n_host.assign(L, 0);
  ctx->seq_off.assign(size_t(cfg->batch), 0);
  ctx->parked.assign(size_t(cfg->batch), 0);
  ctx->rec_floats = int(align_up(size_t(ctx->G) * (d + 2), 4));
  ctx->stream_rec_floats = ctx->rec_floats * (cfg->merge == GLIDE_MERGE_SHARED ? 1 : 2);

  // window slots per split-K item: fixed by the caller, or 128 (512 for very long windows, to bound the
  // number of partials one merge has to read)
  auto chunk_of = [&](int64_t cap) -> int { return cfg->decode_chunk ? cfg->decode_chunk : (cap > 8192 ? 512 : 128); };
  const int splits = (cfg->decode_state_splits ? std::min<int>(cfg->decode_state_splits, d) : (d == 128 ? 4 : 2)) * (dp / d);
  const int64_t units_per_layer = int64_t(B) * Hkv;

  if (int64_t(L) * units_per_layer > (int64_t(1) << 30)) return GLIDE_ERR_UNSUPPORTED;   // unit indices are 32-bit
  ctx->layers.assign(L, LayerDev{});
  size_t part_floats = 0;
  int64_t n_items = 0;
  for (int l = 0; l < L; ++l) {
    LayerDev &ld = ctx->layers[l];
    ld.w = ctx->windows[l];
    ld.cap = std::min<int64_t>(ld.w, cfg->max_tokens);
    // ring rows of a layer are addressed with 32-bit TMA coordinates and 32-bit row indices in the schedules
    if (units_per_layer * ld.cap > int64_t(INT32_MAX) - 1024) return GLIDE_ERR_UNSUPPORTED;
    ld.merge = cfg->merge;
    ld.wlin = cfg->merge == GLIDE_MERGE_SUM_ALL ? 0 : ld.w;
    ld.evicts = ld.wlin < cfg->max_tokens ? 1 : 0;
    const int chunk = chunk_of(ld.cap);
    ld.n_win_items = int((ld.cap + chunk - 1) / chunk);
    ld.n_state_items = ld.evicts ? splits : 0;
    ld.part_base = part_floats;
    int per_unit = ld.n_win_items + ld.n_state_items;
    part_floats += size_t(units_per_layer) * per_unit * ctx->rec_floats;
    n_items += units_per_layer * per_unit;
  }
  if (n_items > (int64_t(1) << 30)) return GLIDE_ERR_UNSUPPORTED;
  ctx->n_items = int(n_items);

  // ---- workspace layout ----
  size_t off = 0;
  ctx->off_ctl = off;
  off = align_up(off + sizeof(Control), 256);
  ctx->off_ndev = off;
  off = align_up(off + sizeof(int64_t) * L, 256);
  ctx->off_layers = off;
  off = align_up(off + sizeof(LayerDev) * L, 256);
  ctx->off_heads = off;
  off = align_up(off + sizeof(int32_t) * H, 256);
  ctx->off_items = off;
  off = align_up(off + sizeof(WorkItem) * size_t(n_items), 256);
  ctx->off_tickets = off;
  off = align_up(off + sizeof(int32_t) * size_t(L) * units_per_layer, 256);
  ctx->off_partials = off;
  ctx->item_part_floats = part_floats;
  // the all-layer schedule plus one schedule per layer (glide_decode_step_layers)
  ctx->stream_rec_capacity = size_t(L) * units_per_layer + size_t(kMaxStreamCtas) * kStreamWarps;
  ctx->stream_seg_capacity = 2 * size_t(L) * units_per_layer + size_t(L + 1) * kMaxStreamCtas * kStreamWarps;
  // (the streaming kernel stores every value of a cross-CTA record beside the launch's tag: 8 bytes per value)
  part_floats = std::max(part_floats, 2 * ctx->stream_rec_capacity * size_t(ctx->stream_rec_floats));
  off = align_up(off + sizeof(float) * part_floats, 256);
  ctx->off_stream_segs = off;
  off = align_up(off + sizeof(StreamSegment) * ctx->stream_seg_capacity, 256);
  ctx->off_stream_cta = off;
  off = align_up(off + sizeof(int32_t) * (size_t(kMaxStreamCtas) * kStreamWarps + 1), 256);
  ctx->off_tmaps = off;
  // per layer 3 maps of 16-row boxes, then (from 3 L on) 2 of 128-row boxes, then the three bf16 scratch arrays of prefill
  off = align_up(off + size_t(128) * (5 * L + 3), 256);
  ctx->off_phik = off;
  off = align_up(off + sizeof(float) * size_t(L) * units_per_layer * ctx->prefill_chunk * dp, 256);
  ctx->off_zcum = off;   // running sums of phi(K') over the chunk: only the sum-of-terms merges use them
  if (cfg->merge != GLIDE_MERGE_SHARED)
    off = align_up(off + sizeof(float) * size_t(L) * units_per_layer * ctx->prefill_chunk * dp, 256);
  ctx->off_phit = off;   // learned feature map: phi(q_h), phi(k_e) of one decode step
  if (cfg->phi == GLIDE_PHI_PROJ_SOFTMAX2)
    off = align_up(off + sizeof(float) * size_t(L) * units_per_layer * dp * (ctx->G + 1), 256);
  ctx->off_gcum = off;   // gated: running sums of log(gate) over the chunk's delayed tokens
  if (cfg->gated) off = align_up(off + sizeof(float) * size_t(L) * units_per_layer * ctx->prefill_chunk, 256);
  // tcgen05 prefill kernel (bf16, head_dim 128, plain feature map): bf16 copies of the chunk's phi(K') rows and of S,
  // which its CTAs fetch by TMA instead of converting the fp32 arrays themselves
  if (cfg->io_dtype == GLIDE_BF16 && d == 128 && !cfg->gated &&
      (cfg->phi == GLIDE_PHI_SOFTMAX || cfg->merge == GLIDE_MERGE_SHARED)) {
    const size_t halves = size_t(dp / d);   // the learned map's two softmax halves are kept apart (one 128-column tensor each)
    ctx->off_phik16 = off;
    off = align_up(off + 2 * halves * size_t(L) * units_per_layer * ctx->prefill_chunk * d, 256);
    ctx->off_s16 = off;
    off = align_up(off + 2 * halves * size_t(L) * units_per_layer * d * d, 256);
    if (halves == 2) {
      ctx->off_phiq16 = off;
      off = align_up(off + 2 * halves * size_t(L) * units_per_layer * ctx->prefill_chunk * ctx->G * d, 256);
    }
  }
  ctx->off_seqoff = off;   // per-sequence position offsets
  off = align_up(off + sizeof(int64_t) * size_t(cfg->batch), 256);
  // the streamed arrays start on a 2 MiB boundary of the workspace whatever the sizes of the small tables before
  // them (measured on the B = 1 decode step: 31.5 us against 32.1 us with 64 KiB or 256 B alignment)
  off = align_up(off, size_t(GLIDE_STATE_ALIGN));
  ctx->off_state = off;
  for (int l = 0; l < L; ++l) {
    ctx->layers[l].S = off;
    off += sizeof(float) * size_t(units_per_layer) * dp * d;
  }
  for (int l = 0; l < L; ++l) {
    ctx->layers[l].z = off;
    off += sizeof(float) * size_t(units_per_layer) * dp;
  }
  ctx->state_bytes = off - ctx->off_state;
  off = align_up(off, 256);
  {
    // Where the rings start relative to the 2 MiB-aligned state is worth 1-2 % of the decode bandwidth, in opposite
    // directions for small and large contexts (measured: B = 1 / 115 MB of rings is 1.5 % faster with the rings
    // aligned, B = 16 / 1.8 GB and B = 4 / 4.2 GB are 0.8 % and 2 % faster with them 65 KiB + 1280 B further on).
    size_t ring_total = 0;
    for (int l = 0; l < L; ++l) ring_total += 2 * size_t(units_per_layer) * size_t(ctx->layers[l].cap) * d * ctx->elem;
    if (ring_total >= GLIDE_RING_SKEW_MIN_BYTES) off += size_t(GLIDE_RING_SKEW_BYTES);
  }
  ctx->off_ring = off;
  for (int l = 0; l < L; ++l) {
    size_t bytes = align_up(size_t(units_per_layer) * size_t(ctx->layers[l].cap) * d * ctx->elem, 256);
    ctx->layers[l].ringK = off;
    off += bytes;
    ctx->layers[l].ringV = off;
    off += bytes;
  }
  if (cfg->gated)
    for (int l = 0; l < L; ++l) {
      ctx->layers[l].ringG = off;
      off += align_up(sizeof(float) * size_t(units_per_layer) * size_t(ctx->layers[l].cap), 256);
    }
  ctx->total = align_up(off, 256);

  if (items) {
    items->clear();
    items->reserve(size_t(n_items));
    for (int l = 0; l < L; ++l) {
      const LayerDev &ld = ctx->layers[l];
      const int chunk = chunk_of(ld.cap);
      for (int64_t u = 0; u < units_per_layer; ++u) {
        int unit = int(int64_t(l) * units_per_layer + u);
        int part = 0;
        for (int i = 0; i < ld.n_win_items; ++i) {
          WorkItem it{};
          it.unit = unit;
          it.layer = l;
          it.kind = kItemWindow;
          it.part = part++;
          it.begin = i * chunk;
          it.count = int(std::min<int64_t>(chunk, ld.cap - int64_t(i) * chunk));
          items->push_back(it);
        }
        for (int i = 0; i < ld.n_state_items; ++i) {
          WorkItem it{};
          it.unit = unit;
          it.layer = l;
          it.kind = kItemState;
          it.part = part++;
          int r0 = int(int64_t(dp) * i / ld.n_state_items), r1 = int(int64_t(dp) * (i + 1) / ld.n_state_items);
          it.begin = r0;
          it.count = r1 - r0;
          items->push_back(it);
        }
      }
    }
    // Units with the most bytes first, a unit's items adjacent: the merge of a long-window unit (many
    // partials) then runs in the middle of the launch, and the tail is made of the cheapest units.
    const size_t elem = ctx->elem;
    auto layer_cost = [&](int l) -> size_t {
      const LayerDev &ld = ctx->layers[l];
      return size_t(ld.cap) * d * elem * 2 + (ld.evicts ? size_t(dp) * d * 4 * 2 : 0);
    };
    std::stable_sort(items->begin(), items->end(), [&](const WorkItem &a, const WorkItem &b) {
      const size_t ca = layer_cost(a.layer), cb = layer_cost(b.layer);
      if (ca != cb) return ca > cb;
      if (a.unit != b.unit) return a.unit < b.unit;
      return a.kind > b.kind;   // state rows first, then the window runs
    });
  }
  return GLIDE_OK;
}

extern "C" {

int glide_workspace_bytes(const glide_config *cfg, size_t *bytes_out) {
  if (!bytes_out) return GLIDE_ERR_INVALID_ARG;
  glide_ctx tmp;
  int rc = plan_context(cfg, &tmp, nullptr);
  if (rc) return rc;
  *bytes_out = tmp.total;
  return GLIDE_OK;
}

int glide_create(const glide_config *cfg, void *dev_workspace, size_t workspace_bytes, void *stream,
                 glide_ctx **ctx_out) {
  if (!ctx_out) return GLIDE_ERR_INVALID_ARG;
  Range range("glide_create");
  *ctx_out = nullptr;
  glide_ctx *ctx = new (std::nothrow) glide_ctx;
  if (!ctx) return GLIDE_ERR_INVALID_ARG;
  std::vector<WorkItem> items;
  int rc = plan_context(cfg, ctx, &items);
  if (rc) {
    delete ctx;
    return rc;
  }
  if (!dev_workspace || (reinterpret_cast<uintptr_t>(dev_workspace) & 255u)) {
    delete ctx;
    return GLIDE_ERR_INVALID_ARG;
  }
  if (workspace_bytes < ctx->total) {
    delete ctx;
    return GLIDE_ERR_WORKSPACE_TOO_SMALL;
  }
  ctx->ws = static_cast<unsigned char *>(dev_workspace);
  ctx->ws_bytes = workspace_bytes;
  cudaStream_t st = as_stream(stream);
  bool ok = cudaGetDevice(&ctx->device) == cudaSuccess &&
            cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device) == cudaSuccess;
  int per_sm = 0;
  // kernel choice: fp32 -> CUDA cores; bf16 -> streaming tensor-core kernel when it applies, else per-item one
  ctx->decode_kind = 0;
  if (ok && cfg->io_dtype == GLIDE_BF16 && cfg->decode_impl != GLIDE_DECODE_FMA) {
    ok = build_ring_tensor_maps(ctx) == GLIDE_OK;
    const bool want_stream = cfg->decode_impl == GLIDE_DECODE_AUTO || cfg->decode_impl == GLIDE_DECODE_STREAM;
    if (ok && want_stream && stream_decode_supported(ctx) && ctx->sm_count * GLIDE_STREAM_CTAS_PER_SM <= kMaxStreamCtas) {
      int rc2 = stream_decode_setup(ctx);
      if (rc2 == GLIDE_OK) ctx->decode_kind = 2;
      else if (rc2 != GLIDE_ERR_UNSUPPORTED) ok = false;
    }
    if (ok && ctx->decode_kind == 0) {
      if (cfg->decode_impl == GLIDE_DECODE_STREAM) {   // asked for explicitly but not applicable
        delete ctx;
        return GLIDE_ERR_UNSUPPORTED;
      }
      if (cfg->merge == GLIDE_MERGE_SHARED && cfg->phi == GLIDE_PHI_SOFTMAX && !cfg->gated) {
        ok = mma_decode_setup(ctx) == GLIDE_OK;
        ctx->decode_kind = 1;
      }   // the per-item tensor-core kernel has the shared normaliser and the parameter-free map only: other merges,
          // the learned map and gates use the CUDA-core kernel
    }
  }
  if (ok && ctx->decode_kind == 0) {
    ok = decode_occupancy(ctx, &per_sm) == GLIDE_OK && per_sm > 0;
    if (ok) ctx->decode_grid = std::max(1, std::min(ctx->n_items, ctx->sm_count * per_sm));
  }
  if (ok) {
    if (!ctx->tmaps_host.empty())
      ok = cudaMemcpyAsync(ctx->ws + ctx->off_tmaps, ctx->tmaps_host.data(), ctx->tmaps_host.size(),
                           cudaMemcpyHostToDevice, st) == cudaSuccess;
    if (ok && ctx->decode_kind == 2) {
      ok = cudaMemcpyAsync(ctx->ws + ctx->off_stream_segs, ctx->stream_segs.data(),
                           sizeof(StreamSegment) * ctx->stream_segs.size(), cudaMemcpyHostToDevice, st) == cudaSuccess &&
           true;
    }
    // control words, counters, tickets, S and z start at zero; so do the records (no launch has the tag 0)
    ok = ok && cudaMemsetAsync(ctx->ws, 0, ctx->off_layers, st) == cudaSuccess &&
         cudaMemsetAsync(ctx->ws + ctx->off_partials, 0, ctx->off_stream_segs - ctx->off_partials, st) == cudaSuccess &&
         cudaMemsetAsync(ctx->ws + ctx->off_seqoff, 0, sizeof(int64_t) * size_t(ctx->cfg.batch), st) == cudaSuccess &&
         cudaMemsetAsync(ctx->ws + ctx->off_tickets, 0, ctx->off_partials - ctx->off_tickets, st) == cudaSuccess &&
         cudaMemsetAsync(ctx->ws + ctx->off_state, 0, ctx->state_bytes, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(ctx->ws + ctx->off_layers, ctx->layers.data(), sizeof(LayerDev) * ctx->layers.size(),
                               cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(ctx->ws + ctx->off_heads, ctx->heads_of.data(), sizeof(int32_t) * ctx->heads_of.size(),
                               cudaMemcpyHostToDevice, st) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(ctx->ws + ctx->off_items, items.data(), sizeof(WorkItem) * items.size(),
                               cudaMemcpyHostToDevice, st) == cudaSuccess;
    // the host vectors above are pageable and go out of scope: finish the copies now
    ok = ok && cudaStreamSynchronize(st) == cudaSuccess;
  }
  if (!ok) {
    cudaGetLastError();
    delete ctx;
    return GLIDE_ERR_CUDA;
  }
  *ctx_out = ctx;
  return GLIDE_OK;
}

int glide_destroy(glide_ctx *ctx) {
  if (!ctx) return GLIDE_ERR_INVALID_ARG;
  delete ctx;
  return GLIDE_OK;
}

namespace {
// largest offset among the slots that hold a sequence (the parked ones are never stepped)
int64_t max_seq_off(const glide_ctx *ctx) {
  int64_t m = kParkedOffset;
  for (size_t b = 0; b < ctx->seq_off.size(); ++b)
    if (!ctx->parked[b]) m = std::max(m, ctx->seq_off[b]);
  return m;
}
bool layers_level(const glide_ctx *ctx) {
  for (size_t l = 1; l < ctx->n_host.size(); ++l)
    if (ctx->n_host[l] != ctx->n_host[0]) return false;
  return true;
}
// new offset of sequence b, on the host and (ordered on the stream) on the device
int set_seq_off(glide_ctx *ctx, int b, int64_t off, cudaStream_t st) {
  // pageable 8-byte source: the runtime stages it before returning
  if (cudaMemcpyAsync(ctx->ws + ctx->off_seqoff + sizeof(int64_t) * size_t(b), &off, sizeof(int64_t),
                      cudaMemcpyHostToDevice, st) != cudaSuccess) {
    cudaGetLastError();
    return GLIDE_ERR_CUDA;
  }
  ctx->seq_off[size_t(b)] = off;
  ctx->ragged = false;
  for (int64_t o : ctx->seq_off) ctx->ragged = ctx->ragged || o != 0;
  return GLIDE_OK;
}
}  // namespace

namespace {
int decode_step_layers(glide_ctx *ctx, int32_t layer_begin, int32_t layer_count, const void *q, const void *k,
                       const void *v, const float *gate, void *out, void *stream) {
  if (!ctx || !q || !k || !v || !out) return GLIDE_ERR_INVALID_ARG;
  Range range("glide_decode_step");
  if (layer_begin < 0 || layer_count < 1 || layer_begin + layer_count > ctx->cfg.n_layers) return GLIDE_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return GLIDE_ERR_INVALID_ARG;
  for (int l = layer_begin + 1; l < layer_begin + layer_count; ++l)
    if (ctx->n_host[l] != ctx->n_host[layer_begin]) return GLIDE_ERR_STATE;
  if (ctx->n_host[layer_begin] + max_seq_off(ctx) + 1 > ctx->cfg.max_tokens) return GLIDE_ERR_CAPACITY;
  int rc = launch_decode(ctx, layer_begin, layer_count, q, k, v, gate, out, as_stream(stream));
  if (rc) return rc;
  for (int l = layer_begin; l < layer_begin + layer_count; ++l) ctx->n_host[l] += 1;
  return GLIDE_OK;
}
}  // namespace

int glide_decode_step_layers(glide_ctx *ctx, int32_t layer_begin, int32_t layer_count, const void *q, const void *k,
                             const void *v, void *out, void *stream) {
  return decode_step_layers(ctx, layer_begin, layer_count, q, k, v, nullptr, out, stream);
}

int glide_decode_step_gated(glide_ctx *ctx, const void *q, const void *k, const void *v, const float *gate, void *out,
                            void *stream) {
  if (!ctx || !ctx->cfg.gated || !aligned16(gate)) return GLIDE_ERR_INVALID_ARG;
  return decode_step_layers(ctx, 0, ctx->cfg.n_layers, q, k, v, gate, out, stream);
}

int glide_decode_step(glide_ctx *ctx, const void *q, const void *k, const void *v, void *out, void *stream) {
  if (!ctx) return GLIDE_ERR_INVALID_ARG;
  return glide_decode_step_layers(ctx, 0, ctx->cfg.n_layers, q, k, v, out, stream);
}

int glide_decode_step_noalloc(glide_ctx *ctx, const void *q, const void *k, const void *v, void *out, void *stream) {
  if (!ctx || !q || !k || !v || !out) return GLIDE_ERR_INVALID_ARG;
  Range range("glide_decode_step_noalloc");
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return GLIDE_ERR_INVALID_ARG;
  const int L = ctx->cfg.n_layers;
  for (int l = 1; l < L; ++l)
    if (ctx->n_host[l] != ctx->n_host[0]) return GLIDE_ERR_STATE;
  if (ctx->n_host[0] + max_seq_off(ctx) + 1 > ctx->cfg.max_tokens) return GLIDE_ERR_CAPACITY;
  int rc = launch_decode_noalloc(ctx, q, k, v, out, as_stream(stream));
  if (rc) return rc;
  for (int l = 0; l < L; ++l) ctx->n_host[l] += 1;
  return GLIDE_OK;
}

namespace {
int prefill_layers(glide_ctx *ctx, int32_t layer_begin, int32_t layer_count, int64_t T, const void *q, const void *k,
                   const void *v, const float *gate, void *out, void *stream) {
  if (!ctx || !k || !v || T < 0) return GLIDE_ERR_INVALID_ARG;
  Range range("glide_prefill");
  if (out && !q) return GLIDE_ERR_INVALID_ARG;
  if (layer_begin < 0 || layer_count < 1 || layer_begin + layer_count > ctx->cfg.n_layers)
    return GLIDE_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return GLIDE_ERR_INVALID_ARG;
  for (int l = layer_begin + 1; l < layer_begin + layer_count; ++l)
    if (ctx->n_host[l] != ctx->n_host[layer_begin]) return GLIDE_ERR_STATE;
  // one call for all sequences needs them at one position
  for (size_t b = 0; b < ctx->seq_off.size(); ++b)
    if (ctx->seq_off[b] != ctx->seq_off[0] || ctx->parked[b]) return GLIDE_ERR_STATE;
  if (ctx->n_host[layer_begin] + ctx->seq_off[0] + T > ctx->cfg.max_tokens) return GLIDE_ERR_CAPACITY;
  if (T == 0) return GLIDE_OK;
  int rc = launch_prefill(ctx, layer_begin, layer_count, T, q, k, v, gate, out, -1,
                          ctx->n_host[layer_begin] + ctx->seq_off[0], as_stream(stream));
  if (rc) return rc;
  for (int l = layer_begin; l < layer_begin + layer_count; ++l) ctx->n_host[l] += T;
  return GLIDE_OK;
}
}  // namespace

int glide_prefill(glide_ctx *ctx, int32_t layer_begin, int32_t layer_count, int64_t T, const void *q, const void *k,
                  const void *v, void *out, void *stream) {
  return prefill_layers(ctx, layer_begin, layer_count, T, q, k, v, nullptr, out, stream);
}

int glide_prefill_gated(glide_ctx *ctx, int32_t layer_begin, int32_t layer_count, int64_t T, const void *q, const void *k,
                        const void *v, const float *gate, void *out, void *stream) {
  if (!ctx || !ctx->cfg.gated || !aligned16(gate)) return GLIDE_ERR_INVALID_ARG;
  return prefill_layers(ctx, layer_begin, layer_count, T, q, k, v, gate, out, stream);
}

int glide_prefill_seq(glide_ctx *ctx, int32_t b, int64_t T, const void *q, const void *k, const void *v, void *out,
                      void *stream) {
  if (!ctx || !k || !v || T < 0 || b < 0 || b >= ctx->cfg.batch) return GLIDE_ERR_INVALID_ARG;
  Range range("glide_prefill_seq");
  if (out && !q) return GLIDE_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return GLIDE_ERR_INVALID_ARG;
  if (!layers_level(ctx)) return GLIDE_ERR_STATE;
  if (ctx->parked[size_t(b)]) return GLIDE_ERR_STATE;   // a parked slot starts again with glide_reset_seq
  const int64_t n0 = ctx->n_host[0] + ctx->seq_off[size_t(b)];
  if (n0 + T > ctx->cfg.max_tokens) return GLIDE_ERR_CAPACITY;
  if (T == 0) return GLIDE_OK;
  int rc = launch_prefill(ctx, 0, ctx->cfg.n_layers, T, q, k, v, nullptr, out, b, n0, as_stream(stream));
  if (rc) return rc;
  return set_seq_off(ctx, b, ctx->seq_off[size_t(b)] + T, as_stream(stream));
}

int glide_reset_seq(glide_ctx *ctx, int32_t b, void *stream) {
  if (!ctx || b < 0 || b >= ctx->cfg.batch) return GLIDE_ERR_INVALID_ARG;
  if (!layers_level(ctx)) return GLIDE_ERR_STATE;
  cudaStream_t st = as_stream(stream);
  // S and z of the slot start at zero; ring rows need no clearing (slots at or beyond the position are never read)
  const size_t d = size_t(ctx->cfg.head_dim), Hkv = size_t(ctx->cfg.n_kv_heads);
  bool ok = true;
  for (const LayerDev &ld : ctx->layers) {
    const size_t dp = size_t(ctx->dp);
    ok = ok && cudaMemsetAsync(ctx->ws + ld.S + size_t(b) * Hkv * dp * d * 4, 0, Hkv * dp * d * 4, st) == cudaSuccess;
    ok = ok && cudaMemsetAsync(ctx->ws + ld.z + size_t(b) * Hkv * dp * 4, 0, Hkv * dp * 4, st) == cudaSuccess;
  }
  if (!ok) {
    cudaGetLastError();
    return GLIDE_ERR_CUDA;
  }
  ctx->parked[size_t(b)] = 0;
  return set_seq_off(ctx, b, -ctx->n_host[0], st);
}

int glide_park_seq(glide_ctx *ctx, int32_t b, void *stream) {
  if (!ctx || b < 0 || b >= ctx->cfg.batch) return GLIDE_ERR_INVALID_ARG;
  ctx->parked[size_t(b)] = 1;
  return set_seq_off(ctx, b, kParkedOffset, as_stream(stream));
}

int glide_seq_tokens(glide_ctx *ctx, int32_t b, int64_t *n_out) {
  if (!ctx || !n_out || b < 0 || b >= ctx->cfg.batch) return GLIDE_ERR_INVALID_ARG;
  if (!layers_level(ctx)) return GLIDE_ERR_STATE;
  if (ctx->parked[size_t(b)]) {
    *n_out = -1;
    return GLIDE_OK;
  }
  *n_out = ctx->n_host[0] + ctx->seq_off[size_t(b)];
  return GLIDE_OK;
}

int glide_seq_layer_info(glide_ctx *ctx, int32_t layer, int32_t b, void *stream, glide_layer_info_t *out) {
  if (!ctx || !out || layer < 0 || layer >= ctx->cfg.n_layers || b < 0 || b >= ctx->cfg.batch) return GLIDE_ERR_INVALID_ARG;
  if (ctx->parked[size_t(b)]) return GLIDE_ERR_STATE;   // a parked slot has no position
  int64_t n = 0, off = 0;
  cudaStream_t st = as_stream(stream);
  if (cudaMemcpyAsync(&n, ctx->ws + ctx->off_ndev + sizeof(int64_t) * layer, sizeof(int64_t), cudaMemcpyDeviceToHost,
                      st) != cudaSuccess ||
      cudaMemcpyAsync(&off, ctx->ws + ctx->off_seqoff + sizeof(int64_t) * size_t(b), sizeof(int64_t),
                      cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) {
    cudaGetLastError();
    return GLIDE_ERR_CUDA;
  }
  n += off;
  const LayerDev &ld = ctx->layers[layer];
  out->window = ld.w;
  out->capacity = ld.cap;
  out->n = n;
  out->count = std::min<int64_t>(n, ld.w);
  out->head_slot = ld.cap > 0 ? n % ld.cap : 0;
  out->n_evicted = std::max<int64_t>(0, n - ld.w);
  return GLIDE_OK;
}

int glide_layer_info(glide_ctx *ctx, int32_t layer, void *stream, glide_layer_info_t *out) {
  return glide_seq_layer_info(ctx, layer, 0, stream, out);
}

int glide_export_state(glide_ctx *ctx, int32_t layer, void *ringK, void *ringV, float *S, float *z, void *stream) {
  if (!ctx || layer < 0 || layer >= ctx->cfg.n_layers) return GLIDE_ERR_INVALID_ARG;
  const LayerDev &ld = ctx->layers[layer];
  const size_t units = size_t(ctx->cfg.batch) * ctx->cfg.n_kv_heads, d = ctx->cfg.head_dim;
  const size_t ring_bytes = units * size_t(ld.cap) * d * ctx->elem;
  cudaStream_t st = as_stream(stream);
  bool ok = true;
  if (ringK && ring_bytes) ok = ok && cudaMemcpyAsync(ringK, ctx->ws + ld.ringK, ring_bytes, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  if (ringV && ring_bytes) ok = ok && cudaMemcpyAsync(ringV, ctx->ws + ld.ringV, ring_bytes, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  const size_t dp = size_t(ctx->dp);
  if (S) ok = ok && cudaMemcpyAsync(S, ctx->ws + ld.S, units * dp * d * 4, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  if (z) ok = ok && cudaMemcpyAsync(z, ctx->ws + ld.z, units * dp * 4, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return GLIDE_ERR_CUDA;
  }
  return GLIDE_OK;
}

int glide_import_state(glide_ctx *ctx, int32_t layer, int64_t n, const void *ringK, const void *ringV, const float *S,
                       const float *z, void *stream) {
  if (!ctx || layer < 0 || layer >= ctx->cfg.n_layers || n < 0 || n > ctx->cfg.max_tokens)
    return GLIDE_ERR_INVALID_ARG;
  const LayerDev &ld = ctx->layers[layer];
  const size_t units = size_t(ctx->cfg.batch) * ctx->cfg.n_kv_heads, d = ctx->cfg.head_dim;
  const size_t ring_bytes = units * size_t(ld.cap) * d * ctx->elem;
  cudaStream_t st = as_stream(stream);
  bool ok = true;
  if (ringK && ring_bytes) ok = ok && cudaMemcpyAsync(ctx->ws + ld.ringK, ringK, ring_bytes, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  if (ringV && ring_bytes) ok = ok && cudaMemcpyAsync(ctx->ws + ld.ringV, ringV, ring_bytes, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  const size_t dp = size_t(ctx->dp);
  if (S) ok = ok && cudaMemcpyAsync(ctx->ws + ld.S, S, units * dp * d * 4, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  if (z) ok = ok && cudaMemcpyAsync(ctx->ws + ld.z, z, units * dp * 4, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  // the counter is a pageable 8-byte source: the runtime stages it before returning
  ok = ok && cudaMemcpyAsync(ctx->ws + ctx->off_ndev + sizeof(int64_t) * layer, &n, sizeof(int64_t),
                             cudaMemcpyHostToDevice, st) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return GLIDE_ERR_CUDA;
  }
  ctx->n_host[layer] = n;
  return GLIDE_OK;
}

namespace {
int copy_gates(glide_ctx *ctx, int32_t layer, float *out, const float *in, void *stream) {
  if (!ctx || layer < 0 || layer >= ctx->cfg.n_layers || (!out && !in)) return GLIDE_ERR_INVALID_ARG;
  if (!ctx->cfg.gated) return GLIDE_ERR_INVALID_ARG;
  const LayerDev &ld = ctx->layers[layer];
  const size_t bytes = sizeof(float) * size_t(ctx->cfg.batch) * ctx->cfg.n_kv_heads * size_t(ld.cap);
  if (bytes == 0) return GLIDE_OK;
  const cudaError_t e = out ? cudaMemcpyAsync(out, ctx->ws + ld.ringG, bytes, cudaMemcpyDeviceToDevice, as_stream(stream))
                            : cudaMemcpyAsync(ctx->ws + ld.ringG, in, bytes, cudaMemcpyDeviceToDevice, as_stream(stream));
  if (e != cudaSuccess) {
    cudaGetLastError();
    return GLIDE_ERR_CUDA;
  }
  return GLIDE_OK;
}
}  // namespace

int glide_export_gates(glide_ctx *ctx, int32_t layer, float *dev_gates, void *stream) {
  return copy_gates(ctx, layer, dev_gates, nullptr, stream);
}
int glide_import_gates(glide_ctx *ctx, int32_t layer, const float *dev_gates, void *stream) {
  return copy_gates(ctx, layer, nullptr, dev_gates, stream);
}

int glide_reset(glide_ctx *ctx, void *stream) {
  if (!ctx) return GLIDE_ERR_INVALID_ARG;
  cudaStream_t st = as_stream(stream);
  bool ok = cudaMemsetAsync(ctx->ws, 0, ctx->off_layers, st) == cudaSuccess &&
            cudaMemsetAsync(ctx->ws + ctx->off_seqoff, 0, sizeof(int64_t) * size_t(ctx->cfg.batch), st) == cudaSuccess &&
            cudaMemsetAsync(ctx->ws + ctx->off_tickets, 0, ctx->off_partials - ctx->off_tickets, st) == cudaSuccess &&
            cudaMemsetAsync(ctx->ws + ctx->off_state, 0, ctx->state_bytes, st) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    return GLIDE_ERR_CUDA;
  }
  std::fill(ctx->n_host.begin(), ctx->n_host.end(), 0);
  std::fill(ctx->seq_off.begin(), ctx->seq_off.end(), 0);
  std::fill(ctx->parked.begin(), ctx->parked.end(), 0);
  ctx->ragged = false;
  return GLIDE_OK;
}

int glide_device_status(glide_ctx *ctx, void *stream, int32_t *status_out) {
  if (!ctx || !status_out) return GLIDE_ERR_INVALID_ARG;
  cudaStream_t st = as_stream(stream);
  Control c{};
  if (cudaMemcpyAsync(&c, ctx->ws + ctx->off_ctl, sizeof(Control), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) {
    cudaGetLastError();
    return GLIDE_ERR_CUDA;
  }
  *status_out = c.status;
  return GLIDE_OK;
}

int glide_decode_launch_info(glide_ctx *ctx, int32_t *n_launches, int32_t *n_work_items, int32_t *grid_size) {
  if (!ctx) return GLIDE_ERR_INVALID_ARG;
  if (n_launches) *n_launches = ctx->cfg.phi == GLIDE_PHI_PROJ_SOFTMAX2 ? 2 : 1;   // the feature kernel, then the step
  if (n_work_items) *n_work_items = ctx->decode_kind == 2 ? int32_t(ctx->stream_scheds[0].n_segs) : ctx->n_items;
  if (grid_size) *grid_size = ctx->decode_grid;
  return GLIDE_OK;
}

int glide_stream_schedule(const glide_config *cfg, int32_t n_sms, int64_t smem_limit, int32_t *rows_out, int32_t max_rows,
                          int32_t *n_rows) {
  if (!n_rows || n_sms < 1 || n_sms * GLIDE_STREAM_CTAS_PER_SM > kMaxStreamCtas || smem_limit < 0 || max_rows < 0 ||
      (max_rows > 0 && !rows_out))
    return GLIDE_ERR_INVALID_ARG;
  glide_ctx ctx;
  int rc = plan_context(cfg, &ctx, nullptr);
  if (rc) return rc;
  if (!stream_decode_supported(&ctx) || cfg->decode_impl == GLIDE_DECODE_FMA || cfg->decode_impl == GLIDE_DECODE_MMA)
    return GLIDE_ERR_UNSUPPORTED;
  const int n_ctas = n_sms * GLIDE_STREAM_CTAS_PER_SM;
  rc = stream_decode_plan(&ctx, n_ctas, size_t(smem_limit));
  if (rc) return rc;
  const glide_ctx::StreamSchedule &sc = ctx.stream_scheds[0];
  *n_rows = int32_t(sc.n_segs);
  for (int c = 0; c < n_ctas; ++c)
    for (int i = sc.range_begin[size_t(c) * kStreamWarps]; i < sc.range_begin[size_t(c + 1) * kStreamWarps] && i < max_rows; ++i) {
      const StreamSegment &sg = ctx.stream_segs[sc.seg_base + size_t(i)];
      int32_t *r = rows_out + size_t(i) * 12;
      r[0] = c; r[1] = sg.range; r[2] = sg.unit; r[3] = sg.layer; r[4] = sg.n_state; r[5] = sg.state0; r[6] = sg.n_win;
      r[7] = sg.win0; r[8] = sg.grp_size; r[9] = sg.grp_size > 1 ? sg.grp_slot0 + sg.grp_idx : -1; r[10] = sg.part;
      r[11] = sg.n_parts;
    }
  return GLIDE_OK;
}

const char *glide_strerror(int code) {
  switch (code) {
    case GLIDE_OK: return "ok";
    case GLIDE_ERR_INVALID_ARG: return "invalid argument";
    case GLIDE_ERR_UNSUPPORTED: return "unsupported configuration";
    case GLIDE_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case GLIDE_ERR_CAPACITY: return "sequence capacity (max_tokens) exceeded";
    case GLIDE_ERR_STATE: return "layers are at different positions";
    case GLIDE_ERR_CUDA: return "CUDA runtime error";
    case GLIDE_ERR_SCRATCH_LIMIT: return "configuration needs more scratch than the library's built-in static buffer holds";
    default: return "unknown status";
  }
}

}  // extern "C"
