/*
 * glide.h -- C ABI of the B200 (sm_100a) GLIDE hybrid-attention library.
 *
 * The operation (paper Sec. III-B "GLIDE Attention", Eq. 7 with its two component
 * equations; Sec. II "Linearized Attention"; appendix Eq. 1-6): every layer l keeps a
 * ring buffer of its newest w_l keys/values and runs exact softmax attention over it;
 * a token that slides out of the window is folded into a recurrent linear-attention
 * state  S += phi(k) v^T,  z += phi(k)  (phi = softmax over the head features, fp32);
 * the output merges both parts under ONE normaliser:
 *
 *   O_t = (sum_W exp(scale q.k_j) v_j + phi(q)^T S) / (sum_W exp(scale q.k_j) + phi(q)^T z)
 *
 * with W = the newest w_l tokens including the current one and S,z holding every
 * older token.  w_l >= context gives causal softmax attention, w_l = 0 pure linear
 * attention.  Prefill over T tokens leaves the same state and outputs as T decode steps.
 *
 * Conventions for every call
 *   - All pointers named dev_* or documented "device" are device pointers on the
 *     CUDA device that was current at glide_create; "host" pointers are ordinary
 *     host memory.  Device buffers must be contiguous and 16-byte aligned.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls
 *     are asynchronous and stream-ordered; the library never synchronises the host on
 *     the hot path and never allocates device memory: the caller owns the workspace
 *     and every q/k/v/out buffer.  The library owns only the small host-side context.
 *   - Every call returns a glide_status code (0 = success).  Arguments are validated
 *     before anything is launched; a failing call changes no state.  Device code never
 *     traps: internal range checks and bounded waits record a code in a status word
 *     (glide_device_status).  Once that word is not zero the step that set it may have
 *     left a unit unfinished (outputs not written, a reduction counter not returned to
 *     zero): call glide_reset, or glide_import_state for every layer, before the context
 *     is used again.
 *   - The host context tracks every layer's position and hands it to each launch, and it
 *     advances its own bookkeeping per call.  A launch that is recorded once and replayed
 *     (a CUDA graph) would run again at the recorded position: issue every prefill and
 *     decode step through these calls.
 *   - Not thread-safe per context; different contexts are independent, also on the GPU: their launches may run on
 *     different streams at the same time (no kernel of the library waits for a thread block that is not running).
 */
#ifndef GLIDE_H_
#define GLIDE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct glide_ctx glide_ctx; /* opaque, host side */

typedef enum {
  GLIDE_OK = 0,
  GLIDE_ERR_INVALID_ARG = 1,         /* NULL / misaligned pointer, negative size, bad layer range */
  GLIDE_ERR_UNSUPPORTED = 2,         /* head_dim not in {64,128}, unequal GQA groups, group size not in {1,2,4,8} */
  GLIDE_ERR_WORKSPACE_TOO_SMALL = 3,
  GLIDE_ERR_CAPACITY = 4,            /* tokens absorbed + T would exceed max_tokens */
  GLIDE_ERR_STATE = 5,               /* decode with layers at different positions */
  GLIDE_ERR_CUDA = 6,                /* a CUDA runtime call or launch failed */
  GLIDE_ERR_SCRATCH_LIMIT = 7        /* glide_decode_step_noalloc: the split-K scratch would not fit the static buffer */
} glide_status;

typedef enum { GLIDE_F32 = 0, GLIDE_BF16 = 1 } glide_dtype;

/* Feature map of the linear part.  GLIDE_PHI_SOFTMAX is the paper's default
 * (Sec. III-B): phi(x) = softmax over the head_dim entries of x, no parameters,
 * feature dimension = head_dim.
 * GLIDE_PHI_PROJ_SOFTMAX2 is the learned map of the Hedgehog / LoLCATs line that the appendix' "Linear Attention"
 * lists among the kernels the method accepts (the paper prints no formula for it; this is the library's reading):
 * with one d x d matrix W per head, y = W^T x (y_j = sum_i x_i W[i][j]),
 *   phi_W(x) = [ softmax(y) ; softmax(-y) ],   feature dimension 2 * head_dim,
 * a matrix per layer and query head for the queries (phi_wq) and per layer and KV head for the keys (phi_wk).
 * S is then [2d][d] and z [2d] per KV head.  It runs on the CUDA-core kernels and, for bf16 I/O with head_dim 128,
 * the decode step on the streaming kernel and, under the shared normaliser, prefill outputs on the tcgen05 kernel
 * (decode_impl AUTO, FMA or STREAM; prefill_impl AUTO, FMA or, with GLIDE_MERGE_SHARED, TCGEN05). */
typedef enum { GLIDE_PHI_SOFTMAX = 0, GLIDE_PHI_PROJ_SOFTMAX2 = 1 } glide_phi;

/* How the window part and the linear part are merged (Sec. III-B "(+)"; appendix
 * "Retention-based SWA").  GLIDE_MERGE_SHARED is the shared normaliser above.  The other two are the appendix'
 * hybrid equations, a plain sum of two separately normalised terms:
 *   GLIDE_MERGE_SUM_EVICTED   phi(q) S / phi(q) z over the evicted tokens  +  window softmax
 *   GLIDE_MERGE_SUM_ALL       the same with a state that holds every token up to the current one (a token is
 *                             folded when it arrives, not when it leaves the window)
 * A term whose token set is empty counts as zero.  With bf16 I/O and head_dim 128 they run on the streaming decode
 * kernel and the tcgen05 prefill kernel, otherwise on the CUDA-core kernels (decode_impl must not be MMA,
 * prefill_impl must not be MMA_SYNC). */
typedef enum { GLIDE_MERGE_SHARED = 0, GLIDE_MERGE_SUM_EVICTED = 1, GLIDE_MERGE_SUM_ALL = 2 } glide_merge;

/* Decode kernel selection.  AUTO: for bf16 I/O the statically scheduled streaming tensor-core/TMA kernel
 * (head_dim 128) or the per-item tensor-core/TMA kernel; for fp32 I/O the CUDA-core kernel.  The others
 * force one kernel (GLIDE_ERR_UNSUPPORTED if it does not apply). */
typedef enum { GLIDE_DECODE_AUTO = 0, GLIDE_DECODE_MMA = 1, GLIDE_DECODE_FMA = 2, GLIDE_DECODE_STREAM = 3 } glide_decode_impl;

/* Kernel that computes the prefill outputs (bf16 I/O).  AUTO picks the fastest that applies.  MMA_SYNC and
 * TCGEN05 need head_dim 128.  For fp32 I/O only the CUDA-core kernel exists.  State, ring and counters do not
 * depend on the choice. */
typedef enum { GLIDE_PREFILL_AUTO = 0, GLIDE_PREFILL_MMA_SYNC = 1, GLIDE_PREFILL_TCGEN05 = 2, GLIDE_PREFILL_FMA = 3 } glide_prefill_impl;

typedef struct {
  int32_t n_layers;        /* L >= 1 */
  int32_t batch;           /* B >= 1 independent sequences of equal length */
  int32_t n_q_heads;       /* H */
  int32_t n_kv_heads;      /* H_kv, H % H_kv == 0 */
  int32_t head_dim;        /* d in {64, 128} */
  int32_t io_dtype;        /* glide_dtype of q, k, v, out and of the ring; S and z are always fp32 */
  int32_t phi;             /* glide_phi */
  int32_t merge;           /* glide_merge */
  const int64_t *windows;  /* host [n_layers]: w_l >= 0 (the layer-wise allocation w - delta_l, Sec. III-B).
                              w_l >= max_tokens never evicts: that layer is full softmax attention. Copied. */
  const int32_t *q_to_kv;  /* host [n_q_heads] KV head of each query head, or NULL for contiguous groups
                              h / (H/H_kv) (the Llama/Mistral GQA convention). Groups must be equal-sized. Copied. */
  int64_t max_tokens;      /* per-sequence capacity, prompt + generated tokens */
  float softmax_scale;     /* scale of the window logits; 0 selects 1/sqrt(head_dim) (appendix Eq. 1) */
  int32_t prefill_chunk;   /* tokens per chunk of the chunked linear scan; 0 selects 256; multiple of 16, <= 1024 */
  int32_t decode_chunk;    /* window slots per split-K work item of the decode kernel; 0 selects automatically */
  int32_t decode_state_splits; /* row blocks the S update/readout of one KV head is split into; 0 selects automatically */
  int32_t decode_impl;     /* glide_decode_impl */
  int32_t prefill_impl;    /* glide_prefill_impl */
  const void *phi_wq;      /* GLIDE_PHI_PROJ_SOFTMAX2: device [n_layers][n_q_heads][d][d] in the I/O dtype, row i column j
                              = W[i][j]; borrowed, must stay alive and unchanged until glide_destroy.  Else NULL. */
  const void *phi_wk;      /* likewise [n_layers][n_kv_heads][d][d] for the keys */
  int32_t gated;           /* 1: gated recurrence (Sec. III-B "GLA-style gating mechanisms"; the paper gives no formula,
                              the library's reading): every token brings a decay gamma in (0, 1] per KV head, which
                              waits in the ring with its key and value, and the state decays by the gate of the token
                              that enters it: S <- gamma S + phi(k) v^T, z <- gamma z + phi(k).  Gates are passed to
                              glide_prefill_gated / glide_decode_step_gated; the calls without gates use gamma = 1.
                              Decode: the streaming kernel (bf16, head_dim 128) or the CUDA-core kernel (decode_impl
                              AUTO, STREAM or FMA); prefill: the CUDA-core kernels (prefill_impl AUTO or FMA). */
  int32_t reserved_;       /* must be 0 */
} glide_config;

typedef struct {
  int64_t window;     /* w_l as configured */
  int64_t capacity;   /* ring slots allocated: min(w_l, max_tokens) */
  int64_t n;          /* tokens absorbed so far (device counter) */
  int64_t count;      /* valid ring entries: min(n, w_l) */
  int64_t head_slot;  /* slot the next token will be written to: n mod capacity (0 if capacity == 0) */
  int64_t n_evicted;  /* tokens folded into S,z so far: max(0, n - w_l) */
} glide_layer_info_t;

/* Bytes of device workspace glide_create needs for this configuration (rings, S, z,
 * split-K scratch, work lists, chunk-scan scratch).  Host only, no CUDA calls. */
int glide_workspace_bytes(const glide_config *cfg, size_t *bytes_out);

/* Set up the per-layer hybrid attention of Sec. III-B (Eq. 7: window softmax over the newest w_l = w - delta_l
 * tokens of layer l, linear state for the rest; the layer-wise allocation delta_l is the caller's, Sec. III-C) with
 * the KV cache of Sec. II "KV Cache" reduced to one ring of w_l slots per layer plus the state S, z of Sec. II
 * "Linearized Attention".
 * Build a context over caller-owned device memory `dev_workspace` (>= glide_workspace_bytes,
 * 256-byte aligned; a 2 MiB-aligned base is worth about 2 % on the smallest decode steps, because the library
 * places the streamed arrays on 2 MiB multiples of its offsets).  Sets the GQA head mapping and the per-layer windows, uploads the static
 * work lists and zeroes rings' bookkeeping, S and z on `stream`.  The workspace must stay
 * alive and untouched by the caller until glide_destroy. */
int glide_create(const glide_config *cfg, void *dev_workspace, size_t workspace_bytes, void *stream,
                 glide_ctx **ctx_out);

/* Prefill stage (Sec. II "KV Cache"; appendix "KV Cache"): append T prompt tokens to layers
 * [layer_begin, layer_begin + layer_count).  May be called repeatedly (chunked prefill); layers
 * may be prefilled in separate calls.
 *   dev_q   [layer_count][B][T][H][d]      (ignored when dev_out is NULL)
 *   dev_k,v [layer_count][B][T][H_kv][d]
 *   dev_out [layer_count][B][T][H][d] or NULL to build the state only.
 * Output i of the call attends to the newest w_l tokens up to and including itself (from the ring
 * and from this call) and, through S,z, to everything older.  Afterwards ring, S, z and counters
 * are exactly as T decode steps would leave them. */
int glide_prefill(glide_ctx *ctx, int32_t layer_begin, int32_t layer_count, int64_t T, const void *dev_q,
                  const void *dev_k, const void *dev_v, void *dev_out, void *stream);

/* Decode stage (Sec. II "KV Cache", decode; Sec. III-B Eq. 7 with its two component equations; the state fold is
 * Sec. II "Linearized Attention", S_i = S_{i-1} + phi(k_i)^T v_i, z_i = z_{i-1} + phi(k_i)^T): one token for every
 * layer and sequence, one fused launch.
 *   dev_q, dev_out [L][B][H][d];  dev_k, dev_v [L][B][H_kv][d].
 * Per layer: the token leaving the window (if any) is folded into S,z in place, the window is
 * streamed once for all query heads of a KV head, the linear readout uses the updated state, and
 * the merged output is written; then k,v are stored at slot n mod capacity and n advances.
 * All layers must be at the same position (GLIDE_ERR_STATE otherwise). */
int glide_decode_step(glide_ctx *ctx, const void *dev_q, const void *dev_k, const void *dev_v, void *dev_out,
                      void *stream);

/* glide_prefill and glide_decode_step of a context created with gated = 1 (GLIDE_ERR_INVALID_ARG otherwise), with
 * the tokens' gates: dev_gate fp32 [layer_count][B][T][H_kv] (prefill) or [L][B][H_kv] (decode), each in (0, 1];
 * NULL stands for gates of 1.  The gate of a token decays the state at the step the token enters it (Sec. III-B
 * "GLA-style gating mechanisms", see glide_config.gated). */
int glide_prefill_gated(glide_ctx *ctx, int32_t layer_begin, int32_t layer_count, int64_t T, const void *dev_q,
                        const void *dev_k, const void *dev_v, const float *dev_gate, void *dev_out, void *stream);
int glide_decode_step_gated(glide_ctx *ctx, const void *dev_q, const void *dev_k, const void *dev_v,
                            const float *dev_gate, void *dev_out, void *stream);

/* The same step for the layers [layer_begin, layer_begin + layer_count) only: what a model needs whose layer l + 1
 * computes its q, k, v from layer l's output (the setting of the paper's experiments, whose "Limitations & Future
 * Works" section names the kernel-launch overhead of small windows).  Tensors are those of the range:
 *   dev_q, dev_out [layer_count][B][H][d];  dev_k, dev_v [layer_count][B][H_kv][d].
 * The layers of the range must be at the same position; other layers are not touched, and glide_decode_step
 * needs all layers level again.  On the streaming kernel a range other than the whole stack is one launch per
 * layer (each with its own schedule); on the other kernels it is one launch. */
int glide_decode_step_layers(glide_ctx *ctx, int32_t layer_begin, int32_t layer_count, const void *dev_q,
                             const void *dev_k, const void *dev_v, void *dev_out, void *stream);

/* Decode step for callers that must not allocate.  (The paper has no counterpart: this is a deployment
 * variant of glide_decode_step, not part of the method.)
 *
 * Who needs it: a serving process that hands every byte of device memory to its own arena at start-up (KV
 * cache, weights) and from then on treats cudaMalloc as forbidden -- because it can fail when the arena has
 * taken the whole GPU, because it synchronises the device, or because the process runs under a budget that
 * audits allocations.  glide_decode_step itself never allocates either, but it keeps its split-K scratch
 * (control words, tickets, partial records) in the caller's workspace; a caller that wants the workspace to
 * hold only persistent state (rings, S, z, tables) and nothing transient can use this call instead: the same
 * step, computed by the CUDA-core decode kernel (any I/O dtype), with that scratch in a buffer that is part of
 * the library image: a file-scope `static __device__` array of GLIDE_NOALLOC_SCRATCH_BYTES (8 MiB), which
 * every GPU that loads the library holds until the process exits.
 *
 *   - Same arguments, layouts, state updates and error behaviour as glide_decode_step; results agree with it
 *     to the tolerance of the I/O dtype (a different kernel may round differently).  The status word of the
 *     device-side checks stays in the context's own workspace, as for every other call (glide_device_status);
 *     only the step's counters, tickets and partial records live in the static buffer.
 *   - Configurations whose scratch (256 + 4 * units + 4 * records bytes, a few KiB per work item) exceeds the
 *     static buffer are refused with GLIDE_ERR_SCRATCH_LIMIT before anything is launched.
 *   - Calls no cudaMalloc / cudaFree and no allocating library routine.  The first call on each device looks
 *     the buffer's device address up once (with that device current): make that first call outside any stream
 *     capture.
 *   - All contexts on a device share the one buffer.  It keeps the previous call's contents; the words that
 *     must start at zero are cleared on `stream` at the start of every call.  Two calls whose kernels overlap
 *     on the GPU (different streams) race on it: keep calls of this entry point stream-ordered per device. */
#define GLIDE_NOALLOC_SCRATCH_BYTES (8u << 20)
int glide_decode_step_noalloc(glide_ctx *ctx, const void *dev_q, const void *dev_k, const void *dev_v, void *dev_out,
                              void *stream);

/* ---- sequences of different lengths (continuous batching) -----------------------------------------
 * The method is defined per sequence (Sec. II "KV Cache", Sec. III-B): nothing couples the B sequences of a
 * context, so each slot b may hold a sequence of its own length.  The position of slot b at layer l is the layer's
 * counter (moved by glide_prefill and the decode steps, which advance every slot together) plus an offset of the
 * slot, which the three calls below change.  They act on all layers and need all layers level (GLIDE_ERR_STATE
 * otherwise).  A decode step advances every slot that is not parked by one token; the capacity check of a step is
 * against the longest such slot.  glide_prefill for all slots at once needs them at one position and none parked. */

/* Slot b starts an empty sequence: position 0, S and z zeroed (ring rows need no clearing).  Other slots are
 * untouched.  Stream-ordered. */
int glide_reset_seq(glide_ctx *ctx, int32_t b, void *stream);

/* glide_prefill for slot b alone, all layers: appends T tokens to that sequence.
 *   dev_q, dev_out [L][T][H][d] (dev_out NULL: state only);  dev_k, dev_v [L][T][H_kv][d]. */
int glide_prefill_seq(glide_ctx *ctx, int32_t b, int64_t T, const void *dev_q, const void *dev_k, const void *dev_v,
                      void *dev_out, void *stream);

/* Slot b holds no sequence from now on: decode steps skip it (its rows of q, k, v may be fetched but are not used --
 * they must stay addressable --, its rows of out and its ring, S and z are not written), so an idle slot costs no
 * window or state traffic.  glide_reset_seq starts a new
 * sequence in it; glide_prefill_seq and glide_seq_layer_info on a parked slot return GLIDE_ERR_STATE.  May be
 * called between the layer-range calls of a step.  Stream-ordered. */
int glide_park_seq(glide_ctx *ctx, int32_t b, void *stream);

/* Tokens slot b holds, as the host tracks them (no device access); -1 for a parked slot. */
int glide_seq_tokens(glide_ctx *ctx, int32_t b, int64_t *n_out);

/* Free the host context (the end of a sequence batch's life: the cache of Sec. II "KV Cache" is the caller's
 * workspace, which this call does not touch). */
int glide_destroy(glide_ctx *ctx);

/* ---- test / benchmark support -------------------------------------------------------------- */

/* Bookkeeping of one layer, read back from the device counters (synchronises `stream`): slot 0, or slot b. */
int glide_layer_info(glide_ctx *ctx, int32_t layer, void *stream, glide_layer_info_t *out);
int glide_seq_layer_info(glide_ctx *ctx, int32_t layer, int32_t b, void *stream, glide_layer_info_t *out);

/* Copy one layer's state to caller DEVICE buffers (any may be NULL):
 *   dev_ringK, dev_ringV [B][H_kv][capacity][d] in the I/O dtype (slot order);
 *   dev_S [B][H_kv][D_phi][d] fp32 with S[r][c] = sum phi(k)_r v_c;  dev_z [B][H_kv][D_phi] fp32
 *   (D_phi = d, or 2d with GLIDE_PHI_PROJ_SOFTMAX2). */
int glide_export_state(glide_ctx *ctx, int32_t layer, void *dev_ringK, void *dev_ringV, float *dev_S,
                       float *dev_z, void *stream);

/* Overwrite one layer's state from caller DEVICE buffers (same layouts; NULL leaves that part
 * as it is) and set the layer's counter to n (0 <= n <= max_tokens; slot offsets stay as they are). */
int glide_import_state(glide_ctx *ctx, int32_t layer, int64_t n, const void *dev_ringK, const void *dev_ringV,
                       const float *dev_S, const float *dev_z, void *stream);

/* The gates of a gated context's ring, one layer: dev_gates fp32 [B][H_kv][capacity] (slot order), copied out or in
 * like the ring rows above (glide_import_gates leaves the counter alone: call it beside glide_import_state). */
int glide_export_gates(glide_ctx *ctx, int32_t layer, float *dev_gates, void *stream);
int glide_import_gates(glide_ctx *ctx, int32_t layer, const float *dev_gates, void *stream);

/* Back to the empty state: counters, slot offsets, S and z zeroed (rings need no clearing). */
int glide_reset(glide_ctx *ctx, void *stream);

/* Status word written by device-side range checks (0 = none tripped).  Synchronises `stream`. */
int glide_device_status(glide_ctx *ctx, void *stream, int32_t *status_out);

/* Kernels one glide_decode_step launches and work items it processes (for launch accounting). */
int glide_decode_launch_info(glide_ctx *ctx, int32_t *n_launches, int32_t *n_work_items, int32_t *grid_size);

/* The streaming decode kernel's static schedule of one all-layer step (Sec. III-B: one unit of work per layer, sequence
 * and KV head: its window of w_l ring slots and its d x d state), as glide_create would build it on a device with
 * n_sms SMs and smem_limit bytes of shared memory per CTA.  Host only, no CUDA calls.  *n_rows receives the number
 * of segments; the first min(*n_rows, max_rows) are described in rows_out, 12 int32 each: {CTA, warp of the CTA,
 * unit, layer, state tiles, first state tile, window tiles, first window tile, warps of the CTA that share the unit
 * (1: none), the segment's shared-memory record slot (-1: none), index of the CTA's global record (-1: the unit lies
 * in one CTA), global records of the unit}.  A tile is 16 rows of S or 16 ring slots.  GLIDE_ERR_UNSUPPORTED when
 * the configuration does not run on that kernel. */
int glide_stream_schedule(const glide_config *cfg, int32_t n_sms, int64_t smem_limit, int32_t *rows_out, int32_t max_rows,
                          int32_t *n_rows);

/* Static, NUL-terminated description of a status code. */
const char *glide_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* GLIDE_H_ */
