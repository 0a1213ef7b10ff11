/*
 * llattn_debug.h - test and tuning hooks of the llattn library.
 *
 * Nothing here is on the hot path and no compute call of llattn.h uses any of
 * it.  The functions are exported from the same shared library so that the
 * test-suite can reach the kernel's work division, the bounded-wait machinery
 * and a slow triage kernel through the C ABI.  Conventions (return codes,
 * pointer ownership, ll_last_error) are those of llattn.h.
 */
#ifndef LLATTN_DEBUG_H
#define LLATTN_DEBUG_H

#include "llattn.h"

#ifdef __cplusplus
extern "C" {
#endif

/* Test-only triage kernel: the same computation as ll_sink_window_attn with one
 * thread block per (query row, head) and plain fp32 FMAs.  Never used by the
 * calls above. */
int ll_debug_attn_simt(ll_cache *cache, int layer, const ll_bf16 *q_roped,
                       int64_t q_frame_start, int n_q_frames, ll_bf16 *out,
                       float *lse_out, ll_stream stream);

/* Test-only: exercise the bounded-wait machinery the kernels share.  Enqueues a
 * one-warp kernel that waits on a barrier nobody completes, gives up after
 * limit_ms (1..1000), records the time-out in the status words and returns
 * normally; the next ll_cache_device_status then reports
 * LL_ERR_DEVICE_TIMEOUT (barrier 99, iteration 7) and clears the record.
 * Attention launches enqueued while the record stands skip their work. */
int ll_debug_wait_timeout(ll_cache *cache, int limit_ms, ll_stream stream);

/* How the attention kernel would divide the work of a call, given the current
 * state (host-only; for tests and tuning).  recache = 0: ll_sink_window_attn of
 * the newest chunk; recache = 1: ll_recache of the resident window.  sm_count > 0
 * overrides the SM count of the storage's device (148 when no storage is bound).
 * Per query group g: tiles[g] query tiles of 256 rows per head (so heads *
 * tiles[g] columns), n_kt[g] key tiles (steps) per column.  The columns of all
 * groups are numbered through (group g's first is col_begin[g]); the first
 * n_waves * n_ctas go out whole, CTA i taking columns i, i + n_ctas, ... (of
 * group g these are its first wave_cols[g]).  The steps of the other columns
 * are laid end to end (group g's from step_begin[g]) and cut into n_shares
 * shares: CTA i takes shared steps [share_begin[k], share_begin[k + 1]) with
 * k = share_of_cta[i], or none when that is -1.  Shares are sized so that
 * whole columns plus share come to the same number of steps on every CTA.
 * When the columns are short (merging the parts of a split column would cost
 * more than splitting saves) nothing is shared: the last wave is partial,
 * columns numbered all_cols and up do not exist, and n_shares is 0.
 * ll_debug_attn_plan_batched: the same for ll_sink_window_attn_batched of the
 * newest chunk of every item (only cache and layer of an item are read). */
#define LL_MAX_GROUPS 24
#define LL_MAX_CTAS 160
typedef struct ll_attn_plan {
    int32_t n_ctas;
    int32_t n_groups;
    int32_t heads;
    int32_t n_waves;
    int32_t n_shares;
    int32_t all_cols;
    int64_t shared_steps;
    int32_t tiles[LL_MAX_GROUPS];
    int32_t n_kt[LL_MAX_GROUPS];
    int32_t col_begin[LL_MAX_GROUPS];
    int32_t wave_cols[LL_MAX_GROUPS];
    int64_t step_begin[LL_MAX_GROUPS];
    int32_t share_begin[LL_MAX_CTAS + 1];
    int32_t share_of_cta[LL_MAX_CTAS];
} ll_attn_plan;
int ll_debug_attn_plan(ll_cache *cache, int layer, int recache, int sm_count, ll_attn_plan *out);
int ll_debug_attn_plan_batched(const ll_attn_item *items, int n_items, int sm_count, ll_attn_plan *out);

/* Byte offsets, inside the bound storage, of the regions of the aux block that
 * the attention kernel and the bounded waits write: the status words and the
 * arrival counters of the split-column merge (Sec. 3.3's attention needs
 * neither; they belong to this implementation).  Any out pointer may be NULL.
 * Host-only; lets a test check that ll_cache_device_status leaves both regions
 * clean after a reported time-out. */
int ll_debug_aux_layout(const ll_cache *cache, size_t *status_offset, size_t *status_bytes,
                        size_t *counters_offset, size_t *counters_bytes);

/* Where the guard bands of a handle created under LL_DEBUG sit inside its storage (byte
 * offsets) and how long each is.  Lets a test overwrite one from the host and see
 * ll_cache_device_status report it.  LL_ERR_INVALID_ARG for a handle without bands. */
int ll_debug_guard_layout(const ll_cache *cache, size_t *front_offset, size_t *back_offset, size_t *bytes);

#ifdef __cplusplus
}
#endif
#endif /* LLATTN_DEBUG_H */
