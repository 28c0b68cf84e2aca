// Internal structures shared by the host runtime and the kernels of the GLIDE library.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <vector>

#include "glide.h"

namespace glide {

constexpr int kDecodeThreads = 128;   // 4 warps per CTA
constexpr int kMaxGroup = 8;          // query heads per KV head
constexpr int64_t kParkedOffset = -(int64_t(1) << 61);   // slot offset of a parked slot: position < 0 at any counter

// Per-layer constants, resident in the workspace (device) and mirrored on the host.
struct LayerDev {
  int64_t w;            // configured window
  int64_t cap;          // ring slots: min(w, max_tokens)
  size_t ringK;         // byte offset in the workspace: [B][Hkv][cap][d] (I/O dtype)
  size_t ringV;
  size_t S;             // byte offset: [B][Hkv][d][d] fp32
  size_t z;             // byte offset: [B][Hkv][d] fp32
  size_t part_base;     // float index into the split-K scratch of this layer's first unit
  int32_t n_win_items;  // window work items per unit
  int32_t n_state_items;// state work items per unit (0 if the layer never evicts)
  int32_t evicts;       // 1 if the layer has a state that ever receives tokens: wlin < max_tokens
  int32_t merge;        // glide_merge
  int64_t wlin;         // a token enters the state wlin steps after it arrives: w, or 0 when the state holds all tokens
  size_t ringG;         // byte offset: gates of the ring's tokens [B][Hkv][cap] fp32 (gated contexts only)
  size_t pad2_;
};

// One work item of the decode kernel.
struct WorkItem {
  int32_t unit;    // (layer * B + b) * Hkv + g
  int32_t layer;
  int32_t kind;    // 0 window slots [begin, begin + count), 1 state rows [begin, begin + count)
  int32_t part;    // index of this item's partial record within the unit
  int32_t begin;
  int32_t count;
  int32_t pad0_, pad1_;
};

enum : int { kItemWindow = 0, kItemState = 1 };

// Device status codes (glide_device_status).
enum : int { kDevOk = 0, kDevBadSlot = 1, kDevBadItem = 2, kDevWaitTimeout = 3 };

// Range checks of a debug build (-DGLIDE_CHECKS): a ring slot, state row or unit index outside its bounds records
// kDevBadSlot in the status word and the access is skipped; nothing traps.  Absent from normal builds.
#ifdef GLIDE_CHECKS
#define GLIDE_CHECK_OR(cond, status_ptr, action)                 \
  do {                                                           \
    if (!(cond)) {                                               \
      atomicExch((status_ptr), glide::kDevBadSlot);              \
      action;                                                    \
    }                                                            \
  } while (0)
#else
#define GLIDE_CHECK_OR(cond, status_ptr, action) do { } while (0)
#endif

// Control words at the start of the workspace.
struct Control {
  int32_t work_counter;
  int32_t done_counter;
  int32_t status;
  int32_t pad_;
};

struct DecodeParams {
  unsigned char *ws;
  const LayerDev *layers;
  const WorkItem *items;
  const int32_t *heads_of;   // [Hkv][G] query heads of each KV head
  Control *ctl;              // work and completion counters (the allocation-free step keeps them in the static buffer)
  int32_t *status;           // the context's status word, in its workspace for every entry point (glide_device_status)
  int32_t *tickets;          // [units]: arrivals at a unit's global records; the last one merges and clears it
  float *partials;
  int64_t *n_dev;            // [L]
  const int64_t *seq_off;    // [B] position of sequence b minus the layer's counter; null when every offset is zero
  const void *q, *k, *v;
  void *out;
  int32_t n_items;
  int32_t L, B, H, Hkv;
  int32_t rec_floats;        // floats per partial record: G * (d + 2) rounded up to 4
  float scale_log2;          // softmax_scale * log2(e)
  int64_t t_host;            // position of the token being decoded as the host tracks it (= device counter)
  int32_t layer_begin, layer_count;   // layers of this launch; q, k, v, out are indexed with the absolute layer
  // learned feature map: the step's phi(q_h) and phi(k_e), written by the feature kernel in front of the decode kernel,
  // [unit][D_phi / 16][G + 1][16] fp32 (row G: the key that enters the state); null for the parameter-free map
  float *phit;
  const void *wq, *wk;       // [L][H][d][d], [L][Hkv][d][d] in the I/O dtype
  int32_t dp;                // feature dimension D_phi
  int32_t gated;
  const float *gate;         // this step's gates [L][B][Hkv] (indexed with the absolute layer), or null for gates of 1
  int32_t tensors_absolute;  // q, k, v, out are indexed with the absolute layer (per-item kernels) or from the range's first
  uint32_t launch_tag;       // streaming kernel: this launch's tag in the records of units cut across CTAs (never 0)
};

#ifndef GLIDE_STREAM_WARPS
#define GLIDE_STREAM_WARPS 8
#endif
#ifndef GLIDE_STREAM_CTAS_PER_SM
#define GLIDE_STREAM_CTAS_PER_SM 1
#endif
#ifndef GLIDE_STREAM_POOL_KB
#define GLIDE_STREAM_POOL_KB 56
#endif
constexpr int kMaxStreamCtas = 192 * GLIDE_STREAM_CTAS_PER_SM;   // CTAs the streaming decode kernel's schedule can address
constexpr int kStreamWarps = GLIDE_STREAM_WARPS;                 // warps (= ranges of the schedule) per CTA
constexpr int kStreamPoolBytes = GLIDE_STREAM_POOL_KB * 1024;    // shared-memory record slots for the CTA-level reduction
constexpr int kStreamMaxGroups = 32;          // reduction groups per CTA

// One segment of the streaming decode kernel's schedule: the part of one unit that falls into one warp's
// range of the tile stream (state tiles first, then window tiles).  64 bytes.
struct StreamSegment {
  int32_t unit, layer;
  int32_t range;             // warp (0..7) of the CTA that owns the segment
  int32_t n_state, state0;   // state tiles [state0, state0 + n_state): 16 rows of S each
  int32_t n_win, win0;       // window tiles [win0, win0 + n_win): 16 ring slots each
  int32_t part;              // this group's record among the unit's global records, -1 if the whole unit is in this group
  int32_t n_parts;           // records of the unit (ticket target)
  int32_t rec0;              // index of the unit's first record in the split-K scratch
  int32_t row_base;          // row of the unit's slot 0 in the layer's [rows][d] ring tensor
  int32_t cap;               // ring slots
  int32_t w;                 // window (clamped to INT32_MAX)
  int32_t evicts;
  int32_t S_off256, z_off256;        // workspace byte offsets / 256 of the unit's S and z
  int32_t ringK_off256, ringV_off256;  // workspace byte offsets / 256 of the layer's K and V rings
  int32_t qrow0;             // row of the KV head's first query head in the [L*B*H][d] q / out tensors
  int32_t g;                 // KV head index (for the head table when the groups are not contiguous)
  int32_t grp_size;          // warps of this CTA that share the unit (1: none); they reduce in shared memory first
  int32_t grp_slot0;         // first shared-memory record slot of the group
  int32_t grp_idx;           // this segment's slot within the group
  int32_t grp_ctr;           // the group's arrival counter in shared memory
};
static_assert(sizeof(StreamSegment) == 96, "StreamSegment is copied as 16-byte chunks");

struct StreamParams {
  const StreamSegment *segs;
  int32_t cta_seg_begin[kMaxStreamCtas + 1];   // first segment of every CTA (its 8 warps' ranges follow each other)
  const struct CUtensorMap_st *tmaps;   // [3 L]: K ring, V ring (2-D), K+V ring (4-D) per layer
  int32_t max_segs;
  int32_t heads_contiguous;
  int32_t kv4d;                    // the 4-D K+V map exists: one TMA per window tile
  int32_t t_off;                   // byte offset in the CTA's shared memory of the per-segment positions (int64 each)
};

struct PrefillParams {
  unsigned char *ws;
  const LayerDev *layers;
  const int32_t *heads_of;
  Control *ctl;
  float *phik;               // chunk scratch: [layer_count][B][Hkv][C][d] fp32, phi of the delayed keys
  void *phik16;              // tcgen05 kernel: the same rows as bf16 (read by TMA), [dp / d halves][units_cap * Cmax][d];
                             // nullptr when that kernel is not in use
  void *s16;                 // tcgen05 kernel: bf16 copy of every unit's S as it is at the start of the chunk,
                             // [dp / d halves][units_cap][d][d]
  void *phiq16;              // tcgen05 kernel, learned map: phi(q) of the chunk's query rows as bf16,
                             // [2 halves][units_cap * Cmax * G][d], row = (unit * Cmax + token) * G + head of the group
  int64_t units_cap;         // L * B * H_kv of the context: what separates the halves in the three arrays above
  float *zcum;               // sum-of-terms merges on the tcgen05 kernel: running sums of phik over the chunk, same shape
  int32_t merge;             // glide_merge
  const void *q, *k, *v;     // the call's inputs
  void *out;
  int64_t n0;                // tokens absorbed before this call (all layers of the call)
  int64_t T;                 // tokens of this call
  int64_t c0;                // first token (call-relative) of the current chunk
  int32_t C;                 // tokens in the current chunk
  int32_t Cmax;              // scratch stride (prefill_chunk)
  int32_t layer_begin, layer_count;
  int32_t L, B, H, Hkv;      // B: sequences of the call's tensors
  int32_t b0;                // sequence slot of the context that the call's sequence 0 is (0 unless one sequence is prefilled)
  float scale_log2;
  int32_t phi, dp;           // glide_phi and its feature dimension
  const void *wq, *wk;       // learned feature map: [L][H][d][d], [L][Hkv][d][d] in the I/O dtype
  int32_t gated;
  const float *gate;         // the call's gates [layer_count][B][T][Hkv], or null for gates of 1
  float *gcum;               // gated: running sums of log(gate) of the chunk's delayed tokens, [units][Cmax]
};

}  // namespace glide

struct glide_ctx {
  glide_config cfg;                 // pointers inside are not used after create
  std::vector<int64_t> windows;
  std::vector<int32_t> q_to_kv;
  std::vector<int32_t> heads_of;    // [Hkv][G]
  std::vector<glide::LayerDev> layers;
  std::vector<int64_t> n_host;      // mirror of the device counters
  std::vector<int64_t> seq_off;     // [B] mirror of the per-sequence offsets: sequence b of layer l is at n_host[l] + seq_off[b]
  bool ragged = false;              // some offset is not zero
  std::vector<char> parked;         // [B] slot holds no sequence: its offset makes every position negative
  std::vector<unsigned char> tmaps_host;  // TMA descriptors of the rings (bf16 tensor-core decode kernel)
  int decode_kind = 0;              // 0 CUDA-core kernel, 1 per-item tensor-core kernel, 2 streaming tensor-core kernel
  // schedules of the streaming kernel: [0] all layers; [1 + l] layer l alone (built when L > 1)
  struct StreamSchedule {
    size_t seg_base = 0;                 // index of its first segment in the device array
    size_t n_segs = 0;
    std::vector<int32_t> range_begin;    // first segment of every warp range, relative to seg_base
  };
  std::vector<StreamSchedule> stream_scheds;
  std::vector<glide::StreamSegment> stream_segs;   // all schedules, concatenated (host copy of the device array)
  int stream_max_segs = 0;
  bool stream_heads_contiguous = true;
  bool tmaps_kv4d = false;
  size_t stream_smem = 0;
  size_t stream_seg_capacity = 0, stream_rec_capacity = 0;
  size_t off_stream_segs = 0, off_stream_cta = 0;
  int G = 0;
  int dp = 0;                       // feature dimension of the linear part: d, or 2d for the learned map
  size_t off_phit = 0, off_gcum = 0;
  size_t off_phik16 = 0, off_s16 = 0, off_phiq16 = 0;   // bf16 scratch of the tcgen05 prefill kernel (0: not laid out)
  int device = 0;
  int sm_count = 0;
  int decode_grid = 0;
  int n_items = 0;
  int rec_floats = 0;
  mutable uint32_t launch_seq = 0;  // launches so far: the tag of the next launch's cross-CTA records
  mutable bool launch_wrapped = false;   // the counter has passed 2^32: the records are cleared before the next launch
  int stream_rec_floats = 0;        // record size of the streaming kernel (twice as large for the sum-of-terms merges)
  int prefill_chunk = 0;
  float scale = 0.f;
  size_t elem = 0;
  unsigned char *ws = nullptr;
  size_t ws_bytes = 0;
  // workspace regions (byte offsets)
  size_t off_ctl = 0, off_ndev = 0, off_seqoff = 0, off_layers = 0, off_heads = 0, off_items = 0, off_tickets = 0,
         off_partials = 0, off_tmaps = 0, off_phik = 0, off_zcum = 0, off_state = 0, off_ring = 0, total = 0;
  size_t state_bytes = 0;           // S and z of all layers (contiguous)
  size_t item_part_floats = 0;      // floats of split-K records the per-item work list needs
  int noalloc_grid = 0;             // grid of the allocation-free decode variant (0: not sized yet)
};

namespace glide {

// Layout planning shared by glide_workspace_bytes and glide_create (host only).
int plan_context(const glide_config *cfg, glide_ctx *ctx, std::vector<WorkItem> *items);

DecodeParams make_decode_params(const glide_ctx *ctx, int layer_begin, int layer_count, const void *q, const void *k,
                                const void *v, void *out);
int launch_prefill_project(glide_ctx *ctx, const PrefillParams &p, bool keys, cudaStream_t stream);   // learned map on the tensor cores
int build_ring_tensor_maps(glide_ctx *ctx);   // TMA descriptors of every layer's K and V ring (host copy)
int mma_decode_setup(glide_ctx *ctx);         // sizes the grid of the per-item tensor-core kernel
int stream_decode_supported(const glide_ctx *ctx);
int stream_decode_plan(glide_ctx *ctx, int n_ctas, size_t smem_limit);   // every schedule of the context (host only)
int stream_decode_setup(glide_ctx *ctx);      // builds the static schedule (host copy) and sizes the launch
int launch_decode_stream(glide_ctx *ctx, const DecodeParams &p, int schedule, cudaStream_t stream);
int launch_decode_mma(glide_ctx *ctx, const DecodeParams &p, cudaStream_t stream);
int launch_decode_noalloc(glide_ctx *ctx, const void *q, const void *k, const void *v, void *out, cudaStream_t stream);
int launch_decode(glide_ctx *ctx, int layer_begin, int layer_count, const void *q, const void *k, const void *v,
                  const float *gate, void *out, cudaStream_t stream);
int decode_occupancy(const glide_ctx *ctx, int *blocks_per_sm);
// seq < 0: the call's tensors hold all B sequences, the layers' counters advance; otherwise they hold sequence slot
// `seq` alone ([layer_count][1][T]...), which is at position n0, and no counter is touched
int launch_prefill(glide_ctx *ctx, int layer_begin, int layer_count, int64_t T, const void *q, const void *k,
                   const void *v, const float *gate, void *out, int seq, int64_t n0, cudaStream_t stream);
bool prefill_attn_tc_supported(const glide_ctx *ctx);
int launch_prefill_attn_tc(glide_ctx *ctx, const PrefillParams &p, cudaStream_t stream);
bool prefill_attn_mma_supported(const glide_ctx *ctx);
int launch_prefill_attn_mma(glide_ctx *ctx, const PrefillParams &p, cudaStream_t stream);
bool prefill_state_mma_supported(const glide_ctx *ctx);
int launch_prefill_state_mma(glide_ctx *ctx, const PrefillParams &p, cudaStream_t stream);
int launch_advance(glide_ctx *ctx, int layer_begin, int layer_count, int64_t T, cudaStream_t stream);

}  // namespace glide
