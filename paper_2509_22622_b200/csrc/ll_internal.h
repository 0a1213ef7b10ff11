// Internal declarations shared by the host code and the kernel translation units.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "llattn.h"
#include "llattn_debug.h"

namespace ll {

constexpr int kMaxGroups = 24;        // query groups (chunks) one attention launch can hold
constexpr int kMaxItems = 8;          // (cache, layer, q, out) tuples one attention launch can serve
constexpr int kTTabFrames = 256;      // frames covered by the resident t-axis RoPE table
constexpr int kTTabAlign = 128;       // table base is a multiple of this many frames
constexpr int kStatusWords = 64;      // uint32 words at the head of the aux block
constexpr int kQTileRows = 256;       // query rows of one work column (two 128-row MMA tiles)
constexpr int kKeyTile = 128;         // keys per MMA tile
constexpr int kMaxCtas = 160;         // persistent CTAs one attention launch may use
constexpr int kSlabs = 16;            // 16-row warp slabs in a work column (2 tiles x 8)

// status word 0 is non-zero when a kernel abandoned a wait; words 1.. hold details
enum StatusCode : uint32_t {
    kStatusOk = 0,
    kStatusTimeout = 1,
    kStatusBadRow = 2,                // an append kernel was handed a storage slot outside the layer
};

#ifdef __CUDACC__
// First come, first served: the record stays until the host has read it.
__device__ __forceinline__ void record_status(uint32_t *status, uint32_t code, uint32_t a, uint32_t b)
{
    if (atomicCAS(status, 0u, code) == 0u) {
        status[1] = a;
        status[2] = b;
        status[3] = 0;
        status[4] = blockIdx.x; status[5] = blockIdx.y; status[6] = blockIdx.z;
        __threadfence();
    }
}
#endif

struct LayerState {
    int64_t end = 0;
    int32_t slot_frame[LL_MAX_SLOTS];
    int64_t n_appends = 0, n_overwrites = 0, n_evictions = 0, n_recaches = 0, n_attn = 0;
};

// One group of query rows that share a visible key set.  The group's work is
// heads x tiles columns (a column = kQTileRows query rows of one head, numbered
// head-major), each n_kt steps long (a step = one kKeyTile-key tile).  The
// columns of all groups of a launch are numbered through, group after group;
// the first n_waves * n_ctas of them are handed out whole, CTA i taking columns
// i, i + n_ctas, ..., and the steps of the columns left over are laid end to
// end and cut into one share per CTA, sized so that every CTA ends up with the
// same number of steps (whole columns of groups with different key counts
// weigh differently).  When the columns are so short that merging the parts of a
// split column would cost more than it saves, the last columns go out whole as
// a partial wave instead and nothing is shared.
struct AttnGroup {
    int item;                         // which (cache, layer, q, out) of the launch the group belongs to
    int q_begin;                      // first query row of the group in its item's q tensor
    int q_rows;                       // rows in the group
    int tiles;                        // query tiles of kQTileRows rows
    int n_kt;                         // key tiles (steps) per column
    int col_begin;                    // launch-wide number of the group's first column
    int wave_cols;                    // the group's first wave_cols columns are handed out whole
    long long step_begin;             // shared steps of all earlier groups
    int n_ranges;
    int k_start[LL_MAX_RANGES];       // visible cache-row runs
    int k_len[LL_MAX_RANGES];
};

// Bytes of the arrival counters of the split-column merge (one per share and 16-row slab).
inline size_t counters_bytes() { return (size_t)kMaxCtas * kSlabs * sizeof(uint32_t); }

// Bytes of one partial-result slot: both tiles' unnormalised O rows in fp32 plus
// (reference max, sum) per row.
inline size_t attn_slot_bytes(int head_dim) { return (size_t)kQTileRows * (head_dim + 2) * sizeof(float); }

// What differs between the items of a batched launch (the K/V and Q tensor maps are in AttnMaps).
struct AttnItem {
    ll_bf16 *out;                     // [nq_total, H, D]
    float *lse;                       // [H, nq_total] or null
    const float *k_scale;             // [H] per-head factor on the keys (8-bit caches), or null
    const float *v_scale;             // [H] per-head factor on the values, or null
    const float *q_scale;             // [nq_total] per-row factor on the queries, or null
    int nq_total;                     // rows of this item's q / out
    int pad;
};

struct AttnMaps {
    CUtensorMap q[kMaxItems], k[kMaxItems], v[kMaxItems];
};

struct AttnParams {
    int n_groups;
    int n_items;
    int heads;
    int nq_total;                     // rows of q / out of item 0 (the triage kernel serves one item)
    int n_ctas;                       // grid.x: persistent CTAs
    int kv_token_major;               // K/V maps are [token][head][dim] (dense attention) instead of [head][row][dim]
    int n_waves;                      // whole-column waves (the last may be partial: columns >= all_cols do not exist)
    int all_cols;                     // columns of all groups
    int n_shares;                     // non-empty shares of the shared steps
    long long total_steps;            // shared steps of all groups
    int64_t rows_per_head;            // (S+W)*P
    float scale_log2;                 // log2(e) / sqrt(D)
    const ll_bf16 *q;                 // [nq_total, H, D]
    ll_bf16 *out;                     // [nq_total, H, D]
    float *lse;                       // [H, nq_total] or null
    const ll_bf16 *kbase;             // layer K: [H][rows][D]
    const ll_bf16 *vbase;             // layer V
    uint32_t *status;                 // aux status words
    float *partial;                   // 2 * kMaxCtas slots of attn_slot_bytes (two per share)
    uint32_t *counters;               // kMaxCtas * kSlabs arrival counters (per share), zero between launches
    AttnItem item[kMaxItems];
    AttnGroup g[kMaxGroups];
    int share_begin[kMaxCtas + 1];    // share k = shared steps [share_begin[k], share_begin[k + 1]), k < n_shares
    short share_of_cta[kMaxCtas];     // the share a CTA takes, -1 for none; shares go to CTAs in rising order
};

struct RopeAppendParams {
    const ll_bf16 *q, *k, *v;         // [n_tokens, H, D]; q may be null
    ll_bf16 *q_out;                   // nullable
    void *kcache, *vcache;            // layer base, [H][rows][D] of bf16 or of E4M3 codes
    const float *k_scale, *v_scale;   // [H], 8-bit caches only: codes hold value / scale
    const float2 *t_tab;              // entry of the call's first frame: [frame][n_t] (cos, sin)
    const float2 *h_tab;              // [grid_h][n_h]
    const float2 *w_tab;              // [grid_w][n_w]
    int64_t rows_per_head;
    int n_tokens, heads, P, grid_w;
    int n_t, n_h;                     // pairs of the t and h bands (w band takes the rest)
    int slot[LL_MAX_SLOTS];           // storage slot of the call's i-th frame
    uint32_t *status;                 // aux status words
    int n_slots;                      // S + W: a slot outside [0, n_slots) is refused by the kernel
};

// QKV projection with norm, rotation and append in its epilogue (qkv_gemm.cu).
struct QkvParams {
    int n_tokens, d_model, heads, head_dim;
    int m_tiles, n_tiles;             // tiles of 128 tokens x tile_n output features
    int tile_n, ssq_slots;            // 256 or 192; 2 * H*D / tile_n slots of the sum of squares per token
    int P, grid_w, n_t, n_h;
    int with_norm;
    float eps;
    const float *bias;                // [3*H*D] or null
    const float *gain_q, *gain_k;     // [H*D] (with_norm)
    const float2 *t_tab, *h_tab, *w_tab;   // as in RopeAppendParams
    ll_bf16 *q_out;                   // [n_tokens, H, D]: rotated q (without the norm's row factor)
    float *q_row_scale;               // [n_tokens] (with_norm): the norm's factor of every q row
    ll_bf16 *kcache, *vcache;         // layer base, [H][rows][D]
    int64_t rows_per_head;
    float *k_park;                    // [n_tokens, H*D] fp32 (with_norm): rotated k without its row factor
    float *ssq;                       // [2][n_tokens][ssq_slots] (with_norm): sums of squares per half tile, q then k
    uint32_t *status;
    int slot[LL_MAX_SLOTS];
};
cudaError_t launch_qkv_gemm(const QkvParams &p, const CUtensorMap &xmap, const CUtensorMap &wmap, int sm_count,
                            cudaStream_t stream);

// Backward of the clip step (attn_bwd.cu): the forward's query groups and key runs, plus where
// the clip's own rows sit in the cache.
struct BwdParams {
    int n_groups, heads, head_dim, nq_total;
    float scale;                      // 1 / sqrt(D)
    float scale_log2;                 // log2(e) / sqrt(D)
    const ll_bf16 *q, *out, *d_out;   // [nq_total, H, D]; q is the rotated query
    const float *lse;                 // [H, nq_total], natural log (the forward's)
    float *delta;                     // [H, nq_total] workspace: sum_d d_out * out
    ll_bf16 *dq, *dk, *dv;            // [nq_total, H, D]
    uint32_t *status;
    int P, grid_w, n_t, n_h;
    const float2 *t_tab, *h_tab, *w_tab;   // t_tab at the clip's first frame
    int64_t rows_per_head;
    int n_kruns;                      // runs of cache rows that hold the clip's frames
    int krun_start[4], krun_len[4];
    int n_ktiles;                     // 128-row tiles over those runs
    int n_qtiles;                     // 128-row query tiles over all groups
    int slot_clip_frame[LL_MAX_SLOTS];     // index of the clip frame a slot holds, -1: not the clip's
    AttnGroup g[kMaxGroups];
};
struct BwdMaps { CUtensorMap q, d_out, k, v; };
cudaError_t launch_attn_backward(const BwdParams &p, const BwdMaps &maps, cudaStream_t stream);

// kernel launchers (each returns the cudaError of the launch)
cudaError_t launch_rope_tables(float2 *t_tab, int64_t t_base, int n_t_frames, int n_t,
                               float2 *h_tab, int grid_h, float2 *w_tab, int grid_w, int n_hw,
                               float theta, bool do_t, bool do_hw, cudaStream_t stream);
cudaError_t launch_rope_append(const RopeAppendParams &p, int head_dim, cudaStream_t stream);
cudaError_t launch_rope_append_e4m3(const RopeAppendParams &p, int head_dim, cudaStream_t stream);
// E4M3 codes of the cache-row runs [start, start + len) of every head -> bf16 values (the codes
// themselves, scales not applied) at the same rows of a bf16 matrix set of the same shape
constexpr int kMaxStageRuns = LL_MAX_SLOTS / 2 + 1;
struct StageParams {
    const uint8_t *k8, *v8;           // [H][rows][D] codes
    ll_bf16 *k16, *v16;               // [H][rows][D]
    int64_t rows_per_head;
    int heads, n_runs;
    int start[kMaxStageRuns], len[kMaxStageRuns];
};
cudaError_t launch_stage_e4m3(const StageParams &p, int head_dim, cudaStream_t stream);
cudaError_t launch_norm_rope_append(const RopeAppendParams &p, int head_dim, const float *gain_q, const float *gain_k,
                                    float eps, cudaStream_t stream);
cudaError_t launch_attn_sm100(const AttnParams &p, int head_dim, const AttnMaps &maps, cudaStream_t stream);
cudaError_t launch_attn_simt(const AttnParams &p, int head_dim, cudaStream_t stream);
// what the probe of the bounded-wait machinery records as barrier and iteration
constexpr int kProbeBarrierId = 99;
constexpr int kProbeIteration = 7;
cudaError_t launch_wait_probe(uint32_t *status, uint64_t limit_ns, cudaStream_t stream);

void count_launch(int n = 1);
void set_last_error(const char *msg);     // what ll_last_error() returns on this thread

}  // namespace ll

struct ll_cache {
    int L, H, D, P, C, S, W;
    int n_slots;
    int64_t rows;                     // (S+W)*P cache rows per head
    std::vector<ll::LayerState> layers;
    bool dry_run = false;
    bool debug = false;               // LL_DEBUG=1 at create time: guard bands around the K/V region
    size_t off_guard0 = 0, off_guard1 = 0;

    char *storage = nullptr;
    size_t storage_bytes = 0;
    // aux block layout (byte offsets from storage)
    size_t off_status = 0, off_ttab = 0, off_hwtab = 0, off_counters = 0, off_partial = 0, aux_bytes = 0;
    int sm_count = 0;                 // of the device the storage lives on
    size_t kv_bytes = 0;              // one K (or V) matrix set of one layer in bf16: H*rows*D*2
    size_t kv_store_bytes = 0;        // the same as stored: kv_bytes, or half of it for E4M3 codes
    std::vector<CUtensorMap> kmap, vmap;
    // 8-bit storage: codes per layer, one bf16 staging pair shared by all layers, scales [L][2][H]
    int kv_format = LL_KV_BF16;
    size_t off_scales = 0, off_stage = 0;
    CUtensorMap stage_kmap, stage_vmap;
    std::vector<float> scales;        // host copy, [L][2][H]

    // Tensor maps of caller tensors met recently (q of the attention calls, k/v of the dense ones):
    // a map depends on address and shape only, and encoding one costs more than a microsecond.
    struct CachedMap { const void *base; uint64_t d2; uint32_t box1, box2; CUtensorMap map; };
    std::vector<CachedMap> map_cache;
    size_t map_cache_next = 0;

    // which RoPE tables are resident
    bool hw_valid = false;
    int tab_gh = 0, tab_gw = 0;
    float tab_theta = 0.f;
    int64_t t_base = -1;
    bool tables_per_call = false;     // set by the first captured call: every append then rebuilds its tables
};
