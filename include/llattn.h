/*
 * llattn - sink+window attention over a rolling per-layer KV cache (sm_100a).
 *
 * C ABI of the inference hot path of a causal, chunk-wise autoregressive video
 * generator that keeps the first frame chunk as a permanent attention sink and
 * a short rolling window of recent frames (Sec. 3.3 "Short-window Attention",
 * "Frame Sink"), and rebuilds the window on a prompt switch (Sec. 3.1 "KV
 * Recache"; Algorithm 2).
 *
 * Conventions for every call
 *   - Return value: LL_OK (0) or a negative LL_ERR_* code.  On any error the
 *     cache's integer state is unchanged and ll_last_error() (thread-local)
 *     describes the failure.
 *   - "device" pointers are CUDA global memory owned by the caller, contiguous
 *     and 16-byte aligned; "host" pointers are ordinary process memory.
 *   - bf16 tensors are bfloat16 bit patterns.  Activations are token-major
 *     [tokens, heads, head_dim]; token n of a frame is grid cell
 *     (y, x) = (n / grid_w, n % grid_w).
 *   - Kernels are enqueued on the caller's stream and the call returns without
 *     synchronising.  The integer state lives on the host inside the handle
 *     and is updated by the call itself, so calls on one handle must be issued
 *     in program order from one thread, on one stream (or on streams the caller
 *     orders).  Handles are independent of each other.
 *   - No CPU fallback exists: without a CUDA device the compute calls fail with
 *     LL_ERR_CUDA.
 */
#ifndef LLATTN_H
#define LLATTN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ll_cache ll_cache;   /* opaque; owned by the library */
typedef void *ll_stream;            /* a cudaStream_t (NULL = default stream) */
typedef uint16_t ll_bf16;           /* bfloat16 bit pattern */

enum {
    LL_OK = 0,
    LL_ERR_INVALID_ARG = -1,        /* null/misaligned pointer, bad layer, bad size */
    LL_ERR_BAD_POSITION = -2,       /* frame_start / n_frames do not fit the stream state */
    LL_ERR_UNSUPPORTED_SHAPE = -3,  /* shape outside what the kernels were built for */
    LL_ERR_NO_STORAGE = -4,         /* compute call before ll_cache_bind_storage */
    LL_ERR_CUDA = -5,               /* a CUDA runtime/driver call failed */
    LL_ERR_DEVICE_TIMEOUT = -6,     /* a kernel gave up on a bounded wait (see ll_cache_device_status) */
    LL_ERR_DEVICE_CHECK = -7        /* a kernel's own bounds check, or a guard band of a debug handle, tripped */
};

#define LL_MAX_SLOTS 64             /* sink_frames + window_frames <= LL_MAX_SLOTS */
#define LL_MAX_RANGES 4             /* contiguous cache-row runs a query group can see */

/* Integer state of one layer's cache.  Bit-exact contract:
 *   frame f lives in slot f if f < S, else in slot S + (f - S) mod W;
 *   slot_frame[slot] is the absolute frame held there, -1 if empty.          */
typedef struct ll_state {
    int64_t end;                        /* frames appended so far */
    int32_t n_slots;                    /* S + W */
    int32_t ring_valid;                 /* ring slots that hold a frame */
    int32_t slot_frame[LL_MAX_SLOTS];
    int64_t n_appends;                  /* new-chunk appends */
    int64_t n_overwrites;               /* overwrite-newest appends */
    int64_t n_evictions;                /* frames replaced by a newer frame */
    int64_t n_recaches;
    int64_t n_attn_calls;
} ll_state;

/* ---- lifetime ----------------------------------------------------------- */

/* Create the host-side handle of one stream's cache: `layers` independent
 * per-layer caches of S = sink_frames pinned frames (Sec. 3.3 "Frame Sink")
 * plus a ring of W = window_frames frames (Sec. 3.3 "Short-window Attention";
 * W counts the chunk being generated), tokens_per_frame tokens each.
 * Requires head_dim in {64, 128}; chunk_frames >= 1; sink_frames and
 * window_frames multiples of chunk_frames; window_frames >= chunk_frames;
 * sink_frames + window_frames <= LL_MAX_SLOTS; window_frames / chunk_frames <= 24;
 * else LL_ERR_UNSUPPORTED_SHAPE.  Touches no device.  *out is owned by the
 * library until ll_cache_destroy. */
int ll_cache_create(int layers, int heads, int head_dim, int tokens_per_frame,
                    int chunk_frames, int sink_frames, int window_frames, ll_cache **out);

/* Frees the handle (host memory only; bound storage stays the caller's). */
void ll_cache_destroy(ll_cache *cache);

/* Bytes of device memory the caller must provide: an aux block (status words,
 * RoPE tables, and the scratch of the attention kernel: arrival counters and
 * 320 partial-result slots of 256 x (head_dim + 2) floats, 42.6 MB at head_dim
 * 128) followed by, per layer, K then V as
 * [heads][(S+W)*tokens_per_frame rows][head_dim] bf16, sink rows first.
 * The scratch is shared by all layers of the handle: one more reason why calls
 * on one handle must be ordered. */
size_t ll_cache_storage_bytes(const ll_cache *cache);

/* Attach caller-owned device memory (`dev`, >= ll_cache_storage_bytes, 1024-byte
 * aligned).  Zero-fills it on `stream` (rows of empty slots may be fetched by
 * partially valid tiles and must hold finite numbers) and encodes the TMA
 * descriptors.  The memory must outlive every later call on the handle. */
int ll_cache_bind_storage(ll_cache *cache, void *dev, size_t bytes, ll_stream stream);

/* 8-bit cache storage.  (The paper's appendix "Quantization" reports an INT8 variant of
 * the whole model; it defines no cache format.  This one is the library's: the rotated
 * keys and the values are kept as E4M3 codes - 1 sign, 4 exponent bits with bias 7, 3
 * mantissa bits, largest magnitude 448, no infinities - times one fp32 scale per layer
 * and head: code = E4M3(fl32(x) / scale), round to nearest even, saturating.)
 *
 * ll_cache_set_kv_format must come before ll_cache_bind_storage and changes
 * ll_cache_storage_bytes: per layer K and V take heads*(S+W)*tokens_per_frame*head_dim
 * bytes each (half of bf16), and the aux block grows by ONE bf16 K/V pair of a layer's
 * size, shared by all layers: an attention call first expands the visible rows' codes
 * into it (exactly: every E4M3 value is a bf16 value) and then runs the same kernel as
 * the bf16 path, with the scales folded into the softmax scale (keys) and into the
 * final normalisation (values).  Net effect at 30 layers of the benchmark shape: 1.84 GB
 * instead of 3.45 GB resident.  Queries stay bf16.
 *
 * ll_cache_set_kv_scales: k_scale, v_scale are HOST arrays of `heads` positive floats
 * for one layer (default 1.0 everywhere); they apply to rows written afterwards, and an
 * attention call uses the scales in force when it is made, so set them before the
 * layer's first append and leave them alone while rows written under them are resident.
 * Copied to the device on `stream`.
 *
 * With LL_KV_E4M3: ll_rope_append_kv, ll_sink_window_attn (also batched, and mixed with
 * bf16 caches in one launch), ll_recache and ll_clip_append_attn work as documented;
 * ll_norm_rope_append_kv returns LL_ERR_UNSUPPORTED_SHAPE. */
#define LL_KV_BF16 0
#define LL_KV_E4M3 1
int ll_cache_set_kv_format(ll_cache *cache, int format);
int ll_cache_set_kv_scales(ll_cache *cache, int layer, const float *k_scale, const float *v_scale,
                           ll_stream stream);

/* Byte offset, inside the bound storage, of head `head` of layer `layer`'s K
 * (which = 0) or V (which = 1) matrix: (S+W)*tokens_per_frame rows of head_dim
 * bf16 (or E4M3 bytes), row = slot * tokens_per_frame + token.  For tests and
 * checkpointing. */
int ll_cache_kv_offset(const ll_cache *cache, int layer, int which, int head, size_t *offset);

/* ---- the hot path --------------------------------------------------------- */

/* Fused 3-D RoPE + K/V append (Algorithm 2: every pass of a chunk writes the
 * chunk's K/V into the cache before attending; the final clean pass commits it.
 * Slot rule: Sec. 3.3 "Frame Sink").
 *   q, k, v   device, bf16 [n_frames*grid_h*grid_w, heads, head_dim]; q may be
 *             NULL when q_out is NULL.
 *   q_out     device, same shape as q, nullable: receives RoPE(q) (may alias q).
 *   n_frames  must equal chunk_frames; grid_h*grid_w must equal tokens_per_frame.
 *   frame_start == end      : a new chunk; evicts the frames W behind it, end += C.
 *   frame_start == end - C  : overwrites the newest chunk in place (state unchanged).
 *   anything else           : LL_ERR_BAD_POSITION.
 * RoPE: the D/2 rotation pairs are split t|h|w with n_h = n_w = D/6 (floor) and
 * n_t = D/2 - 2*n_h pairs; pair j is elements (2j, 2j+1); pair i of an axis with
 * n_a pairs turns by pos * rope_theta^(-i/n_a); t is the absolute frame index.
 * K rows are stored rotated, V rows verbatim.  The arithmetic is fp32 on
 * fp64-accurate sine/cosine tables kept in the aux block.  The tables are
 * rebuilt only when the grid, rope_theta or the resident range of frames
 * changes - until a call on the handle is recorded into a CUDA graph: from then
 * on every append of the handle, recorded or not, enqueues the small table
 * kernel in front of itself, so a replayed graph never reads tables that a
 * later call has moved. */
int ll_rope_append_kv(ll_cache *cache, int layer, const ll_bf16 *q, const ll_bf16 *k,
                      const ll_bf16 *v, int64_t frame_start, int n_frames,
                      int grid_h, int grid_w, float rope_theta, ll_bf16 *q_out,
                      ll_stream stream);

/* The same with the base model's q/k normalisation in front (the paper does not
 * define it; this is the RMS norm over a token's whole row of heads*head_dim
 * elements with a learned gain, applied before the rotation):
 *   x_hat[e] = x[e] / sqrt(mean_e(x[e]^2) + eps) * gain[e]
 * for q (gain_q) and k (gain_k), in fp32, then RoPE and append as above; v is
 * stored as it comes.  One pass over q, k, v instead of a norm kernel followed
 * by ll_rope_append_kv.
 *   gain_q, gain_k  [heads*head_dim] fp32, device, 16-byte aligned; gain_q may
 *                   be null when q_out is null
 *   eps >= 0
 * Everything else (positions, state, errors) as ll_rope_append_kv. */
int ll_norm_rope_append_kv(ll_cache *cache, int layer, const ll_bf16 *q, const ll_bf16 *k,
                           const ll_bf16 *v, const float *gain_q, const float *gain_k, float eps,
                           int64_t frame_start, int n_frames, int grid_h, int grid_w,
                           float rope_theta, ll_bf16 *q_out, ll_stream stream);

/* The QKV projection of a DiT self-attention layer (Sec. 3.1: the block this path sits
 * in; the projection itself is the base model's, the paper does not restate it) with the
 * front end of the path in the GEMM's epilogue: one tcgen05 GEMM
 *     y = x W^T + b,   q | k | v = y
 * whose accumulators go through the optional q/k RMS norm (as in
 * ll_norm_rope_append_kv), the 3-D rotation and the append without a round trip
 * through memory: v rows and rotated k rows land in the cache, rotated q in q_out.
 *   x        device, bf16 [n_frames*tokens_per_frame, d_model]; d_model a multiple of 8
 *   w_qkv    device, bf16 [3*heads*head_dim, d_model]: q features, then k, then v
 *   bias     device, fp32 [3*heads*head_dim], nullable
 *   gain_q, gain_k  device, fp32 [heads*head_dim]; both NULL: no norm
 *   q_out    device, bf16 [tokens, heads, head_dim]
 * With the norm, a token's factor 1/sqrt(mean(q^2) + eps) is known only when all its
 * heads are done, and they are computed by different thread blocks.  So q_out receives
 * rotate(gain * q) WITHOUT that factor and q_row_scale[token] (device, fp32 [tokens])
 * receives the factor: pass both to ll_sink_window_attn_scaled, which folds the factor
 * into the row's softmax scale.  k rows are completed inside the call (a second small
 * kernel), for which it needs `workspace`: device, 256-byte aligned, at least
 * ll_qkv_proj_workspace_bytes (4 bytes per k element of a chunk plus a table of partial
 * sums), caller-owned, free again when the call's kernels have run.  Without the norm
 * q_row_scale and workspace may be NULL.
 * heads*head_dim must be a multiple of 256 or of 192; bf16 caches only; positions, state and errors
 * as ll_rope_append_kv. */
size_t ll_qkv_proj_workspace_bytes(const ll_cache *cache);
int ll_qkv_proj_append(ll_cache *cache, int layer, const ll_bf16 *x, int d_model, const ll_bf16 *w_qkv,
                       const float *bias, const float *gain_q, const float *gain_k, float eps,
                       int64_t frame_start, int n_frames, int grid_h, int grid_w, float rope_theta,
                       ll_bf16 *q_out, float *q_row_scale, void *workspace, size_t workspace_bytes,
                       ll_stream stream);

/* Sink+window attention of the newest chunk's queries (Sec. 3.3): every query
 * attends to all sink rows and all resident window rows (the chunk itself
 * included; bidirectional inside the chunk), softmax scale 1/sqrt(head_dim).
 *   q_roped   device, bf16 [n_q_frames*tokens_per_frame, heads, head_dim], after RoPE.
 *   q_frame_start must equal end - C and n_q_frames must equal C.
 *   out       device, bf16, same shape as q_roped.
 *   lse_out   device, float [heads, n_q_frames*tokens_per_frame], nullable:
 *             natural-log softmax denominators.
 * QK^T and PV run on tcgen05 tensor cores with fp32 accumulation in TMEM; the
 * softmax is fp32 (weights rounded to bf16 for the PV product, the denominator
 * summed from the unrounded values).  The result is run-to-run deterministic. */
int ll_sink_window_attn(ll_cache *cache, int layer, const ll_bf16 *q_roped,
                        int64_t q_frame_start, int n_q_frames, ll_bf16 *out,
                        float *lse_out, ll_stream stream);

/* The same with one extra factor per query row on the scores (q_row_scale: device, fp32
 * [n_q_frames*tokens_per_frame], 16-byte aligned; NULL = 1): row i attends with
 * softmax scale q_row_scale[i]/sqrt(head_dim).  For queries whose normalisation factor
 * was left out of q_roped (ll_qkv_proj_append). */
int ll_sink_window_attn_scaled(ll_cache *cache, int layer, const ll_bf16 *q_roped, const float *q_row_scale,
                               int64_t q_frame_start, int n_q_frames, ll_bf16 *out, float *lse_out,
                               ll_stream stream);

/* The same for several independent streams in ONE launch (serving: the streams
 * of a batch sit at different positions, with windows filled to different
 * degrees and possibly of different sizes; Sec. 3.3's attention per stream is
 * unchanged).  Each item is one ll_sink_window_attn call's arguments; the
 * caches must agree in heads and head_dim and may differ in everything else,
 * no (cache, layer) may appear twice, n_items <= LL_MAX_BATCH.  The kernel
 * divides the work of all items between the SMs together, so small or
 * partly filled windows do not leave SMs idle.  The scratch of items[0].cache
 * is used; the usual rule (calls on a handle are ordered) extends to every
 * handle named.  On error nothing is launched and no state changes. */
#define LL_MAX_BATCH 8
typedef struct ll_attn_item {
    ll_cache *cache;
    int32_t layer;
    int32_t n_q_frames;                 /* must equal the cache's chunk_frames */
    const ll_bf16 *q_roped;
    int64_t q_frame_start;              /* must equal end - chunk_frames */
    ll_bf16 *out;
    float *lse_out;                     /* nullable */
} ll_attn_item;
int ll_sink_window_attn_batched(const ll_attn_item *items, int n_items, ll_stream stream);

/* Dense attention of n_q queries over n_k keys, no mask and no RoPE: the
 * cross-attention to the prompt that alternates with the self-attention layers
 * and through which the recache re-encodes the prefix under the new prompt
 * (Sec. 3.1).  Same kernel as ll_sink_window_attn, reading K and V where the
 * projection left them.
 *   q [n_q, heads, head_dim], k and v [n_k, heads, head_dim], bf16, device,
 *   16-byte aligned; heads and head_dim are the handle's.  The handle lends its
 *   scratch and status words; its caches and integer state are not touched
 *   (calls on a handle are ordered by the caller, as everywhere).
 *   out [n_q, heads, head_dim] bf16; lse_out [heads, n_q] fp32, nullable. */
int ll_cross_attn(ll_cache *cache, const ll_bf16 *q, int64_t n_q, const ll_bf16 *k, const ll_bf16 *v,
                  int64_t n_k, ll_bf16 *out, float *lse_out, ll_stream stream);

/* A clip of several chunks in one step (Sec. 3.3 "Consistency between Training
 * and Inference": the resident cache is the S sink frames, the last frames of
 * the preceding context and the T frames of the current clip, attended under
 * the same sink + local-window rule as at inference; also the way to prefill a
 * stream from an existing video).  Forward only.
 *   q, k, v             [n_frames*tokens_per_frame, heads, head_dim], raw
 *   frame_start         must equal end; n_frames a positive multiple of
 *                       chunk_frames, at most 24 chunks
 *   attn_window_frames  W_a, the local window a chunk attends over (counts the
 *                       chunk itself), a multiple of chunk_frames.  The ring
 *                       must hold the first chunk's window until the last chunk
 *                       is in: window_frames >= W_a + n_frames - chunk_frames,
 *                       else LL_ERR_UNSUPPORTED_SHAPE.
 * Appends all n_frames (RoPE on K, slots and eviction as n_frames/chunk_frames
 * calls of ll_rope_append_kv would), writes RoPE(q) to q_out, then attends: a
 * query of the chunk ending at frame e sees the sink frames below e and the
 * frames [max(S, e - W_a), e).  Every chunk gets what chunk-by-chunk decoding
 * on a cache with window_frames = W_a would give it.  out/lse_out as for
 * ll_sink_window_attn with n_frames*tokens_per_frame rows.  On error nothing is
 * launched and no state changes. */
int ll_clip_append_attn(ll_cache *cache, int layer, const ll_bf16 *q, const ll_bf16 *k,
                        const ll_bf16 *v, int64_t frame_start, int n_frames,
                        int attn_window_frames, int grid_h, int grid_w, float rope_theta,
                        ll_bf16 *q_out, ll_bf16 *out, float *lse_out, ll_stream stream);

/* Backward of ll_clip_append_attn: gradients of a scalar loss through the clip step (Sec. 3.3
 * "Consistency between Training and Inference": the clip's T frames carry gradients, the sink
 * and the preceding context are detached; Algorithm 1 back-propagates the newest clip's loss).
 * Call it while the cache is as the forward left it (frame_start + n_frames == end; same
 * attn_window_frames, grid and rope_theta).
 *   q_roped  the forward's q_out; out, lse: the forward's outputs (lse is required here);
 *   d_out    gradient of the loss with respect to out, bf16 [n_frames*tokens_per_frame, heads, head_dim]
 *   dq, dk, dv  bf16, same shape: gradients with respect to the q, k, v that were handed to the
 *            forward (BEFORE the rotation: dq and dk are turned back through it); dk, dv cover
 *            the clip's own keys only.
 *   workspace  device, 256-byte aligned, >= ll_clip_backward_workspace_bytes (one float per query
 *            row and head), caller-owned.
 * With s_ij the scaled scores over the keys visible to row i and p = softmax(s):
 *   dv_j = sum_i p_ij d_out_i;  dS_ij = p_ij (d_out_i.v_j - d_out_i.out_i);
 *   dq_i = sum_j dS_ij k_j / sqrt(D);  dk_j = sum_i dS_ij q_i / sqrt(D).
 * P and dS are rounded to bf16 for the tensor-core products (fp32 accumulation); every element is
 * accumulated by one thread block in one order, so the result is run-to-run deterministic.  bf16
 * caches only.  State is not changed. */
size_t ll_clip_backward_workspace_bytes(const ll_cache *cache, int n_frames);
int ll_clip_attn_backward(ll_cache *cache, int layer, const ll_bf16 *q_roped, const ll_bf16 *out,
                          const ll_bf16 *d_out, const float *lse, int64_t frame_start, int n_frames,
                          int attn_window_frames, int grid_h, int grid_w, float rope_theta,
                          ll_bf16 *dq, ll_bf16 *dk, ll_bf16 *dv, void *workspace, size_t workspace_bytes,
                          ll_stream stream);

/* KV-recache (Sec. 3.1; Sec. 3.3 last paragraph: only the most recent W frames
 * are rebuilt; the sink is left alone).  q, k, v hold fresh activations for the
 * resident window frames [r0, end), r0 = max(S, end - W), oldest first.
 *   n_frames  must equal end - r0 (0 while only sink frames exist: no work).
 * Re-ropes and overwrites those frames' ring rows (slot table and end
 * unchanged), then attends all their queries block-causally: a query of chunk c
 * sees the sink and window frames [r0, (c+1)*C).  out/lse_out as above with
 * n_frames*tokens_per_frame rows; q_out nullable receives RoPE(q). */
int ll_recache(ll_cache *cache, int layer, const ll_bf16 *q, const ll_bf16 *k,
               const ll_bf16 *v, int n_frames, int grid_h, int grid_w, float rope_theta,
               ll_bf16 *q_out, ll_bf16 *out, float *lse_out, ll_stream stream);

/* Forget everything in every layer (Algorithm 2 "C <- []"): end = 0, all slots
 * empty, counters kept.  Stored bytes are not cleared: the next stream writes
 * over them slot by slot, and until a slot is rewritten its stale rows may
 * still be fetched by the ragged last tile of a neighbouring slot's keys (they
 * are masked out of the softmax but pass through the PV product with weight
 * zero), so they must hold finite numbers.  Rows written by this library from
 * finite inputs always do. */
int ll_cache_reset(ll_cache *cache);

/* 3-D RoPE of a query tensor without any device allocation.  (The paper has no
 * counterpart: this entry point exists for integration, not for the method.)
 *
 * Who it is for: code that must not, or cannot, obtain device memory at the
 * time of the call - a serving process whose memory manager has already taken
 * the whole GPU, a component that is forbidden to allocate after start-up so
 * its latency stays predictable, a plug-in that is handed tensors but no
 * allocator.  Such a caller cannot provide the storage block that
 * ll_cache_bind_storage wants, and that block is where ll_rope_append_kv keeps
 * its sine/cosine tables.  Here the tables live in a fixed array inside the
 * library image instead (180 KB, present on every GPU that loads the library
 * for as long as the process runs), and the call itself never calls cudaMalloc,
 * cudaFree or anything else that allocates.
 *
 *   q, q_out  device, bf16 [n_frames*grid_h*grid_w, heads, head_dim], 16-byte
 *             aligned; q_out may alias q.  Caller-owned, as everywhere else.
 *   result    q_out = RoPE(q), the same values ll_rope_append_kv writes to its
 *             q_out for the same frame_start, grid and rope_theta.
 *   limits    head_dim 64 or 128; n_frames <= LL_STATIC_MAX_FRAMES;
 *             grid_h + grid_w <= LL_STATIC_MAX_GRID_SUM.  Larger requests are
 *             refused with LL_ERR_UNSUPPORTED_SHAPE (the fixed array cannot hold
 *             their tables) and ll_last_error() says which limit was hit.
 *   sharing   all calls on a GPU use the one array.  A call first writes the
 *             table entries it needs and then reads them, on `stream`, so it does
 *             not depend on what an earlier call left there; but two calls that
 *             are in flight on the same GPU at the same time (two streams, two
 *             threads) overwrite each other's tables.  Order them.
 *   set-up    the first call on each device looks up where that device's copy
 *             of the array lives (once, with that device current).  Make that
 *             first call outside of any stream capture. */
#define LL_STATIC_MAX_FRAMES 64
#define LL_STATIC_MAX_GRID_SUM 1024
int ll_rope_q_static(const ll_bf16 *q, ll_bf16 *q_out, int heads, int head_dim,
                     int64_t frame_start, int n_frames, int grid_h, int grid_w,
                     float rope_theta, ll_stream stream);

/* ---- state, diagnostics ----------------------------------------------------- */

int ll_cache_get_state(const ll_cache *cache, int layer, ll_state *out);

/* Restore a state saved by ll_cache_get_state (checkpoint/resume); validates
 * that every resident frame sits in the slot the slot rule gives it. */
int ll_cache_set_state(ll_cache *cache, int layer, const ll_state *state);

/* Cache-row runs [start, start+len) (row = slot*tokens_per_frame + token) that
 * the queries of frames [q_frame_start, q_frame_start + chunk_frames) can see
 * given the current state; lo_floor hides window frames older than it (pass 0
 * for decode).  Writes up to LL_MAX_RANGES pairs, returns the count in
 * *n_ranges.  Host-only; used by the attention calls and by tests. */
int ll_cache_visible_ranges(const ll_cache *cache, int layer, int64_t q_frame_start,
                            int64_t lo_floor, int64_t *starts, int64_t *lens, int *n_ranges);

/* Bookkeeping-only mode (on != 0): compute calls validate arguments and update
 * the integer state but launch nothing and need no device or storage.  For
 * planning and host-side tests; outputs are NOT produced. */
int ll_cache_set_dry_run(ll_cache *cache, int on);

/* Synchronise `stream`, read the aux status words and clear them.  LL_OK, or
 * LL_ERR_DEVICE_TIMEOUT if a kernel abandoned a bounded wait (its outputs are
 * then invalid); ll_last_error() names the role and barrier.  On a time-out
 * the call also zeroes the arrival counters of the split-column merge, which
 * the abandoned launch left mid-count, so the handle can be used again.
 * LL_ERR_DEVICE_CHECK: an append kernel was handed a storage slot outside the
 * layer and refused to write (it never is with the slot rule above; the check
 * costs one comparison), or - for a handle created while the environment
 * variable LL_DEBUG was set to something other than 0 - one of the two 4 KB
 * guard bands that such a handle keeps in front of and behind its K/V region
 * no longer holds its pattern (ll_cache_storage_bytes accounts for the bands). */
int ll_cache_device_status(ll_cache *cache, ll_stream stream);

/* Kernel launches made by this process through the library so far. */
int64_t ll_launch_count(void);

const char *ll_last_error(void);
const char *ll_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LLATTN_H */
