// Host side of the library: handle, integer cache state, argument checks,
// TMA descriptor encoding and kernel dispatch.  No tensor arithmetic here.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>

#include <nvtx3/nvToolsExt.h>

#include "ll_internal.h"

namespace {

// NVTX range around a compute call (the kernels it enqueues show up under it in a timeline),
// only when the environment variable LL_NVTX is set to something other than 0.
bool nvtx_on()
{
    static const bool on = [] { const char *e = getenv("LL_NVTX"); return e && e[0] && e[0] != '0'; }();
    return on;
}
struct Range {
    bool on;
    Range(const char *what, int layer, long long frame) : on(nvtx_on())
    {
        if (!on) return;
        char buf[96];
        snprintf(buf, sizeof buf, "%s layer %d frame %lld", what, layer, frame);
        nvtxRangePushA(buf);
    }
    ~Range() { if (on) nvtxRangePop(); }
};

thread_local std::string g_err;
std::atomic<int64_t> g_launches{0};

int fail(int code, const char *fmt, ...)
{
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    g_err = buf;
    return code;
}

int cuda_fail(cudaError_t e, const char *what)
{
    return fail(LL_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

void rope_split(int D, int *n_t, int *n_h)
{
    *n_h = D / 6;
    *n_t = D / 2 - 2 * (D / 6);
}

// Slot rule: sink frames are pinned, later frames roll through the ring.
int slot_of(const ll_cache *c, int64_t f)
{
    return f < c->S ? (int)f : c->S + (int)((f - c->S) % c->W);
}

bool layer_ok(const ll_cache *c, int layer) { return c && layer >= 0 && layer < c->L; }

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                  const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                  const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// 3-D bf16 tensor map with 128-byte swizzle; box = {64 elements, box1, box2}.
int encode_map(CUtensorMap *m, const void *base, uint64_t d0, uint64_t d1, uint64_t d2,
               uint64_t stride1_bytes, uint64_t stride2_bytes, uint32_t box1, uint32_t box2)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return fail(LL_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t dims[3] = {d0, d1, d2};
    cuuint64_t strides[2] = {stride1_bytes, stride2_bytes};
    cuuint32_t box[3] = {64, box1, box2};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides,
                    box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(LL_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
    return LL_OK;
}

char *layer_k(const ll_cache *c, int layer) { return c->storage + c->aux_bytes + (size_t)layer * 2 * c->kv_store_bytes; }
char *layer_v(const ll_cache *c, int layer) { return layer_k(c, layer) + c->kv_store_bytes; }
const float *layer_scales(const ll_cache *c, int layer, int which)
{
    return reinterpret_cast<const float *>(c->storage + c->off_scales) + ((size_t)layer * 2 + which) * c->H;
}

constexpr size_t kGuardBytes = 4096;
constexpr int kGuardByte = 0xA5;

// Offsets of the aux block's parts and the size of a stored K (or V) matrix set.
void compute_layout(ll_cache *c)
{
    int n_t, n_h;
    rope_split(c->D, &n_t, &n_h);
    c->off_status = 0;
    c->off_ttab = align_up(ll::kStatusWords * sizeof(uint32_t), 256);
    c->off_hwtab = align_up(c->off_ttab + (size_t)ll::kTTabFrames * n_t * sizeof(float2), 256);
    // grid_h + grid_w <= tokens_per_frame + 1 for any grid with grid_h*grid_w == tokens_per_frame
    c->off_counters = align_up(c->off_hwtab + (size_t)(c->P + 1) * n_h * sizeof(float2), 256);
    c->off_partial = align_up(c->off_counters + ll::counters_bytes(), 1024);
    size_t end = align_up(c->off_partial + 2 * (size_t)ll::kMaxCtas * ll::attn_slot_bytes(c->D), 1024);
    c->kv_bytes = (size_t)c->H * c->rows * c->D * sizeof(ll_bf16);
    c->kv_store_bytes = c->kv_bytes;
    c->off_scales = c->off_stage = 0;
    if (c->kv_format == LL_KV_E4M3) {
        c->kv_store_bytes = c->kv_bytes / 2;
        c->off_scales = end;
        c->off_stage = align_up(c->off_scales + (size_t)c->L * 2 * c->H * sizeof(float), 1024);
        end = align_up(c->off_stage + 2 * c->kv_bytes, 1024);
    }
    c->off_guard0 = c->off_guard1 = 0;
    if (c->debug) {
        // a band of a fixed pattern right in front of the K/V region (and one behind it, see
        // ll_cache_storage_bytes): a kernel that writes outside the layers' rows trips one
        c->off_guard0 = end;
        end += kGuardBytes;
    }
    c->aux_bytes = end;
}

// Visible cache-row runs for queries of the chunk holding q_frame_start.
int visible_ranges(const ll_cache *c, int layer, int64_t q_frame_start, int64_t lo_floor,
                   int64_t *starts, int64_t *lens, int *n_ranges)
{
    const ll::LayerState &st = c->layers[layer];
    if (q_frame_start < 0 || q_frame_start >= st.end)
        return fail(LL_ERR_BAD_POSITION, "query frame %lld is outside the stream [0, %lld)",
                    (long long)q_frame_start, (long long)st.end);
    const int64_t hi = (q_frame_start / c->C + 1) * c->C;
    int64_t lo = std::max<int64_t>(std::max<int64_t>(c->S, hi - c->W), lo_floor);
    bool seen[LL_MAX_SLOTS] = {false};
    auto mark = [&](int64_t f) -> bool {
        int s = slot_of(c, f);
        if (st.slot_frame[s] != (int32_t)f) return false;
        seen[s] = true;
        return true;
    };
    for (int64_t f = 0; f < std::min<int64_t>(c->S, hi); ++f)
        if (!mark(f)) return fail(LL_ERR_BAD_POSITION, "sink frame %lld is not resident", (long long)f);
    for (int64_t f = lo; f < hi; ++f)
        if (!mark(f)) return fail(LL_ERR_BAD_POSITION, "window frame %lld is not resident", (long long)f);
    int n = 0;
    for (int s = 0; s < c->n_slots;) {
        if (!seen[s]) { ++s; continue; }
        int e = s;
        while (e < c->n_slots && seen[e]) ++e;
        if (n >= LL_MAX_RANGES) return fail(LL_ERR_UNSUPPORTED_SHAPE, "visible set needs more than %d runs", LL_MAX_RANGES);
        starts[n] = (int64_t)s * c->P;
        lens[n] = (int64_t)(e - s) * c->P;
        ++n;
        s = e;
    }
    *n_ranges = n;
    return LL_OK;
}

// Make sure the RoPE tables cover frames [f0, f1) and this grid/theta.
//
// Normally the tables are rebuilt only when the grid, theta or the resident window of
// kTTabFrames frames changes, and the host remembers what is resident.  A call recorded
// into a CUDA graph cannot rely on that memory: the graph may be replayed after other calls
// on the handle have moved the tables, and a replay moves them back without the host
// seeing it.  So from the first captured call on, every append of the handle (recorded or
// not) brings its own tables: the table kernel is enqueued in front of it, for exactly the
// frames it needs.
int ensure_tables(ll_cache *c, int64_t f0, int64_t f1, int gh, int gw, float theta, cudaStream_t stream)
{
    int n_t, n_h;
    rope_split(c->D, &n_t, &n_h);
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess) {
        cap = cudaStreamCaptureStatusNone;
        (void)cudaGetLastError();
    }
    if (cap == cudaStreamCaptureStatusActive) c->tables_per_call = true;
    bool do_hw = !(c->hw_valid && c->tab_gh == gh && c->tab_gw == gw && c->tab_theta == theta);
    bool do_t = do_hw || c->t_base < 0 || f0 < c->t_base || f1 > c->t_base + ll::kTTabFrames;
    int64_t base = do_t ? f0 / ll::kTTabAlign * ll::kTTabAlign : c->t_base;
    int n_frames = ll::kTTabFrames;
    if (c->tables_per_call) {
        do_t = do_hw = true;
        base = f0;
        n_frames = (int)(f1 - f0);
        if (n_frames > ll::kTTabFrames) return fail(LL_ERR_UNSUPPORTED_SHAPE, "more than %d frames in one call", ll::kTTabFrames);
    }
    if (!do_t && !do_hw) return LL_OK;
    float2 *t_tab = reinterpret_cast<float2 *>(c->storage + c->off_ttab);
    float2 *h_tab = reinterpret_cast<float2 *>(c->storage + c->off_hwtab);
    float2 *w_tab = h_tab + (size_t)gh * n_h;
    cudaError_t e = ll::launch_rope_tables(t_tab, base, n_frames, n_t, h_tab, gh, w_tab, gw, n_h,
                                           theta, do_t, do_hw, stream);
    if (e != cudaSuccess) return cuda_fail(e, "rope table kernel");
    c->t_base = base;
    c->hw_valid = true; c->tab_gh = gh; c->tab_gw = gw; c->tab_theta = theta;
    return LL_OK;
}

int need_storage(const ll_cache *c)
{
    if (!c->storage) return fail(LL_ERR_NO_STORAGE, "no device storage bound (call ll_cache_bind_storage)");
    return LL_OK;
}

int fill_rope_params(ll_cache *c, int layer, const ll_bf16 *q, const ll_bf16 *k, const ll_bf16 *v,
                     ll_bf16 *q_out, int64_t frame_start, int n_frames, int gw, ll::RopeAppendParams *p)
{
    int n_t, n_h;
    rope_split(c->D, &n_t, &n_h);
    p->q = q; p->k = k; p->v = v; p->q_out = q_out;
    p->kcache = layer_k(c, layer);
    p->vcache = layer_v(c, layer);
    p->k_scale = c->kv_format == LL_KV_E4M3 ? layer_scales(c, layer, 0) : nullptr;
    p->v_scale = c->kv_format == LL_KV_E4M3 ? layer_scales(c, layer, 1) : nullptr;
    const float2 *t_tab = reinterpret_cast<const float2 *>(c->storage + c->off_ttab);
    p->t_tab = t_tab + (size_t)(frame_start - c->t_base) * n_t;
    p->h_tab = reinterpret_cast<const float2 *>(c->storage + c->off_hwtab);
    p->w_tab = p->h_tab + (size_t)c->tab_gh * n_h;
    p->rows_per_head = c->rows;
    p->n_tokens = n_frames * c->P;
    p->heads = c->H; p->P = c->P; p->grid_w = gw;
    p->n_t = n_t; p->n_h = n_h;
    for (int i = 0; i < n_frames; ++i) p->slot[i] = slot_of(c, frame_start + i);
    p->status = reinterpret_cast<uint32_t *>(c->storage + c->off_status);
    p->n_slots = c->n_slots;
    return LL_OK;
}

cudaError_t launch_append(const ll_cache *c, const ll::RopeAppendParams &p, cudaStream_t stream)
{
    return c->kv_format == LL_KV_E4M3 ? ll::launch_rope_append_e4m3(p, c->D, stream)
                                      : ll::launch_rope_append(p, c->D, stream);
}

// One (cache, layer, q, out) of an attention launch and the chunks of queries it brings.
struct AttnCall {
    ll_cache *c;
    int layer;
    const ll_bf16 *q;
    ll_bf16 *out;
    float *lse;
    int n_groups;
    int64_t group_frame_start[ll::kMaxGroups];
    int64_t lo_floor;                             // non-sink frames older than this are hidden from every group ...
    int64_t group_lo_floor[ll::kMaxGroups];       // ... and from group g those older than this (0: no extra limit)
    // dense attention (dense_keys > 0): one group of dense_rows queries over all dense_keys rows of the
    // token-major k/v tensors given here; the cache lends its shape and scratch only
    int64_t dense_rows, dense_keys;
    const ll_bf16 *dense_k, *dense_v;
    const float *q_scale;                         // per-row factor on the queries, or null
};

// Divide the columns of all groups between the CTAs (one persistent CTA per SM).  The
// columns are numbered through, group after group.  While a CTA's worth of them is
// left they go out whole, one per CTA and wave (CTAs on the same head then walk the keys
// in step and share each K/V tile through L2).  The steps of the columns left over are
// laid end to end and cut into shares: a CTA's share is what it lacks to the common
// level T of steps, after its whole columns; CTAs already above T take none.
void plan_work(ll::AttnParams *p, int sms, long long all_cols, long long all_steps)
{
    const bool waves = all_cols >= sms;
    p->n_ctas = waves ? sms : (int)std::min<long long>(sms, all_steps);
    p->n_waves = waves ? (int)(all_cols / sms) : 0;
    p->all_cols = (int)all_cols;
    {
        // Short columns: splitting the leftover columns saves at most their length minus an even
        // share, and costs every part a trip through the scratch slots (about kMergeSteps steps'
        // worth).  When that does not pay, the leftover goes out whole as one more, partial wave.
        constexpr long long kMergeSteps = 3;
        const long long first_left = (long long)p->n_waves * sms;
        long long left_steps = 0, left_longest = 0;
        for (int g = 0; g < p->n_groups; ++g) {
            const ll::AttnGroup &G = p->g[g];
            const long long cols = (long long)p->heads * G.tiles;
            const long long left = std::min(cols, std::max<long long>(0, G.col_begin + cols - first_left));
            left_steps += left * G.n_kt;
            if (left > 0) left_longest = std::max<long long>(left_longest, G.n_kt);
        }
        if (left_steps > 0 && left_longest <= (left_steps + sms - 1) / sms + kMergeSteps) {
            p->n_waves += 1;
            p->n_ctas = (int)std::min<long long>(sms, all_cols);
        }
    }
    const long long whole_cols = std::min<long long>((long long)p->n_waves * p->n_ctas, all_cols);
    long long steps = 0;
    for (int g = 0; g < p->n_groups; ++g) {
        ll::AttnGroup &G = p->g[g];
        const long long cols = (long long)p->heads * G.tiles;
        G.wave_cols = (int)std::min(cols, std::max<long long>(0, whole_cols - G.col_begin));
        G.step_begin = steps;
        steps += (cols - G.wave_cols) * G.n_kt;
    }
    p->total_steps = steps;
    // steps each CTA gets as whole columns
    long long load[ll::kMaxCtas] = {};
    for (int g = 0; g < p->n_groups && p->n_ctas > 0; ++g) {
        // of the columns [0, x) CTA i takes those congruent to i: (x + n - 1 - i) / n of them
        const ll::AttnGroup &G = p->g[g];
        const long long lo = G.col_begin, hi = G.col_begin + G.wave_cols, n = p->n_ctas;
        for (int i = 0; i < p->n_ctas; ++i)
            load[i] += ((hi + n - 1 - i) / n - (lo + n - 1 - i) / n) * G.n_kt;
    }
    // the highest level T that the shared steps can fill: sum over CTAs of max(0, T - load) <= steps
    auto fill = [&](long long T) {
        long long need = 0;
        for (int i = 0; i < p->n_ctas; ++i) need += std::max<long long>(0, T - load[i]);
        return need;
    };
    long long lo = 0, hi = 0;
    for (int i = 0; i < p->n_ctas; ++i) hi = std::max(hi, load[i]);
    hi += steps + 1;                                     // fill(hi) > steps
    while (hi - lo > 1) {
        const long long mid = lo + (hi - lo) / 2;
        if (fill(mid) <= steps) lo = mid; else hi = mid;
    }
    const long long T = lo;
    long long extra = steps - fill(T);                   // fewer than the CTAs at or below T: one more step each
    int k = 0;
    p->share_begin[0] = 0;
    for (int i = 0; i < p->n_ctas; ++i) {
        long long size = std::max<long long>(0, T - load[i]);
        if (load[i] <= T && extra > 0) { ++size; --extra; }
        p->share_of_cta[i] = size > 0 ? (short)k : (short)-1;
        if (size > 0) {
            p->share_begin[k + 1] = p->share_begin[k] + (int)size;
            ++k;
        }
    }
    p->n_shares = k;
}

// Fill the launch parameters of one launch serving `n_calls` calls: every call's query chunks
// become groups, each split into query tiles, and the work is divided between the CTAs.
// Scratch and status words are those of the first call's cache.
int build_attn_params(const AttnCall *calls, int n_calls, ll::AttnParams *p)
{
    if (n_calls < 1 || n_calls > ll::kMaxItems) return fail(LL_ERR_UNSUPPORTED_SHAPE, "between 1 and %d items per launch", ll::kMaxItems);
    ll_cache *c0 = calls[0].c;
    memset(p, 0, sizeof *p);
    p->n_items = n_calls;
    p->heads = c0->H;
    p->rows_per_head = c0->rows;
    p->scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)c0->D));
    p->q = calls[0].q; p->out = calls[0].out; p->lse = calls[0].lse;
    p->kbase = reinterpret_cast<const ll_bf16 *>(c0->storage ? layer_k(c0, calls[0].layer) : nullptr);
    p->vbase = reinterpret_cast<const ll_bf16 *>(c0->storage ? layer_v(c0, calls[0].layer) : nullptr);
    p->status = reinterpret_cast<uint32_t *>(c0->storage ? c0->storage + c0->off_status : nullptr);
    p->partial = reinterpret_cast<float *>(c0->storage ? c0->storage + c0->off_partial : nullptr);
    p->counters = reinterpret_cast<uint32_t *>(c0->storage ? c0->storage + c0->off_counters : nullptr);
    const int sms = std::min(c0->sm_count > 0 ? c0->sm_count : 148, ll::kMaxCtas);
    long long all_steps = 0, all_cols = 0;
    int ng = 0;
    for (int i = 0; i < n_calls; ++i) {
        const AttnCall &call = calls[i];
        ll_cache *c = call.c;
        if (c->H != c0->H || c->D != c0->D)
            return fail(LL_ERR_UNSUPPORTED_SHAPE, "the items of one launch must agree in heads and head_dim");
        if (ng + call.n_groups > ll::kMaxGroups) return fail(LL_ERR_UNSUPPORTED_SHAPE, "more than %d query groups", ll::kMaxGroups);
        const bool dense = call.dense_keys > 0;
        if (dense && n_calls != 1) return fail(LL_ERR_INVALID_ARG, "dense attention does not share a launch");
        const int rows_per_group = dense ? (int)call.dense_rows : c->C * c->P;
        const int tiles = (rows_per_group + ll::kQTileRows - 1) / ll::kQTileRows;
        p->kv_token_major = dense ? 1 : 0;
        p->item[i].out = call.out;
        p->item[i].lse = call.lse;
        const bool e4m3 = !dense && c->kv_format == LL_KV_E4M3 && c->storage;
        p->item[i].q_scale = call.q_scale;
        p->item[i].k_scale = e4m3 ? layer_scales(c, call.layer, 0) : nullptr;
        p->item[i].v_scale = e4m3 ? layer_scales(c, call.layer, 1) : nullptr;
        p->item[i].nq_total = call.n_groups * rows_per_group;
        for (int g = 0; g < call.n_groups; ++g, ++ng) {
            ll::AttnGroup &G = p->g[ng];
            G.item = i;
            G.q_begin = g * rows_per_group;
            G.q_rows = rows_per_group;
            G.tiles = tiles;
            int64_t starts[LL_MAX_RANGES], lens[LL_MAX_RANGES];
            int n = 0;
            if (dense) {
                starts[0] = 0;
                lens[0] = call.dense_keys;
                n = 1;
            } else {
                int st = visible_ranges(c, call.layer, call.group_frame_start[g],
                                        std::max(call.lo_floor, call.group_lo_floor[g]), starts, lens, &n);
                if (st != LL_OK) return st;
            }
            G.n_ranges = n;
            G.n_kt = 0;
            for (int r = 0; r < n; ++r) {
                G.k_start[r] = (int)starts[r];
                G.k_len[r] = (int)lens[r];
                G.n_kt += (int)((lens[r] + ll::kKeyTile - 1) / ll::kKeyTile);
            }
            G.col_begin = (int)all_cols;
            all_cols += (long long)c->H * tiles;
            all_steps += (long long)c->H * tiles * G.n_kt;
        }
    }
    if (all_steps > INT32_MAX) return fail(LL_ERR_UNSUPPORTED_SHAPE, "too much work for one launch");
    p->n_groups = ng;
    p->nq_total = p->item[0].nq_total;
    plan_work(p, sms, all_cols, all_steps);
    return LL_OK;
}

// Map of a token-major [tokens, H, D] tensor of the caller (box: 64 elements x 1 head x 128 tokens),
// from the handle's small cache when this address and length were seen before.
int token_major_map(ll_cache *c, CUtensorMap *out, const void *base, uint64_t tokens)
{
    for (const auto &e : c->map_cache)
        if (e.base == base && e.d2 == tokens) { *out = e.map; return LL_OK; }
    int st = encode_map(out, base, (uint64_t)c->D, (uint64_t)c->H, tokens, (uint64_t)c->D * 2, (uint64_t)c->H * c->D * 2, 1, 128);
    if (st != LL_OK) return st;
    constexpr size_t kEntries = 16;
    ll_cache::CachedMap e{base, tokens, 1, 128, *out};
    if (c->map_cache.size() < kEntries) c->map_cache.push_back(e);
    else c->map_cache[c->map_cache_next++ % kEntries] = e;
    return LL_OK;
}

int launch_attention(const AttnCall *calls, int n_calls, const ll::AttnParams &p, cudaStream_t stream, bool simt)
{
    ll_cache *c0 = calls[0].c;
    if (simt) {
        cudaError_t e = ll::launch_attn_simt(p, c0->D, stream);
        return e == cudaSuccess ? LL_OK : cuda_fail(e, "simt attention kernel");
    }
    ll::AttnMaps maps;
    memset(&maps, 0, sizeof maps);
    for (int i = 0; i < n_calls; ++i) {
        ll_cache *c = calls[i].c;
        int st = token_major_map(c, &maps.q[i], calls[i].q, (uint64_t)p.item[i].nq_total);
        if (st != LL_OK) return st;
        if (calls[i].dense_keys > 0) {
            // token-major K/V: coordinates (dim, head, token), a tile = 128 tokens of one head
            st = token_major_map(c, &maps.k[i], calls[i].dense_k, (uint64_t)calls[i].dense_keys);
            if (st != LL_OK) return st;
            st = token_major_map(c, &maps.v[i], calls[i].dense_v, (uint64_t)calls[i].dense_keys);
            if (st != LL_OK) return st;
            continue;
        }
        if (c->kv_format == LL_KV_E4M3) {
            // expand the codes of every cache row some group of this call can see into the bf16
            // staging pair the kernel reads (the union of the groups' runs, merged by slot)
            bool seen[LL_MAX_SLOTS] = {false};
            for (int g = 0; g < p.n_groups; ++g) {
                if (p.g[g].item != i) continue;
                for (int r = 0; r < p.g[g].n_ranges; ++r)
                    for (int sl = p.g[g].k_start[r] / c->P; sl < (p.g[g].k_start[r] + p.g[g].k_len[r]) / c->P; ++sl)
                        seen[sl] = true;
            }
            ll::StageParams sp;
            memset(&sp, 0, sizeof sp);
            sp.k8 = reinterpret_cast<const uint8_t *>(layer_k(c, calls[i].layer));
            sp.v8 = reinterpret_cast<const uint8_t *>(layer_v(c, calls[i].layer));
            sp.k16 = reinterpret_cast<ll_bf16 *>(c->storage + c->off_stage);
            sp.v16 = reinterpret_cast<ll_bf16 *>(c->storage + c->off_stage + c->kv_bytes);
            sp.rows_per_head = c->rows;
            sp.heads = c->H;
            for (int sl = 0; sl < c->n_slots;) {
                if (!seen[sl]) { ++sl; continue; }
                int e = sl;
                while (e < c->n_slots && seen[e]) ++e;
                sp.start[sp.n_runs] = sl * c->P;
                sp.len[sp.n_runs] = (e - sl) * c->P;
                ++sp.n_runs;                                   // at most n_slots / 2 + 1 <= kMaxStageRuns runs
                sl = e;
            }
            cudaError_t es = ll::launch_stage_e4m3(sp, c->D, stream);
            if (es != cudaSuccess) return cuda_fail(es, "staging kernel of the 8-bit cache");
            maps.k[i] = c->stage_kmap;
            maps.v[i] = c->stage_vmap;
            continue;
        }
        maps.k[i] = c->kmap[calls[i].layer];
        maps.v[i] = c->vmap[calls[i].layer];
    }
    cudaError_t e = ll::launch_attn_sm100(p, c0->D, maps, stream);
    return e == cudaSuccess ? LL_OK : cuda_fail(e, "sink+window attention kernel");
}

// Checks of one decode item (the newest chunk's queries of one layer of one cache).
int check_decode_item(ll_cache *c, int layer, const ll_bf16 *q_roped, int64_t q_frame_start, int n_q_frames,
                      ll_bf16 *out, float *lse_out)
{
    if (!layer_ok(c, layer)) return fail(LL_ERR_INVALID_ARG, "bad cache handle or layer %d", layer);
    ll::LayerState &st = c->layers[layer];
    if (n_q_frames != c->C) return fail(LL_ERR_BAD_POSITION, "n_q_frames %d != chunk_frames %d", n_q_frames, c->C);
    if (st.end < c->C || q_frame_start != st.end - c->C)
        return fail(LL_ERR_BAD_POSITION, "queries must be the newest chunk: q_frame_start %lld, end %lld",
                    (long long)q_frame_start, (long long)st.end);
    if (!c->dry_run) {
        if (!q_roped || !out) return fail(LL_ERR_INVALID_ARG, "null q_roped or out");
        if (!aligned16(q_roped) || !aligned16(out) || (lse_out && !aligned16(lse_out)))
            return fail(LL_ERR_INVALID_ARG, "q_roped/out/lse_out must be 16-byte aligned");
        int s = need_storage(c);
        if (s != LL_OK) return s;
    }
    return LL_OK;
}

int attn_entry(ll_cache *c, int layer, const ll_bf16 *q_roped, int64_t q_frame_start, int n_q_frames,
               ll_bf16 *out, float *lse_out, ll_stream stream, bool simt, const float *q_scale = nullptr)
{
    Range range("ll_sink_window_attn", layer, (long long)q_frame_start);
    int s = check_decode_item(c, layer, q_roped, q_frame_start, n_q_frames, out, lse_out);
    if (s != LL_OK) return s;
    if (simt && c->kv_format != LL_KV_BF16) return fail(LL_ERR_UNSUPPORTED_SHAPE, "the triage kernel reads bf16 caches only");
    AttnCall call{c, layer, q_roped, out, lse_out, 1, {q_frame_start}, 0};
    call.q_scale = q_scale;
    ll::AttnParams p;
    s = build_attn_params(&call, 1, &p);
    if (s != LL_OK) return s;
    if (!c->dry_run) {
        s = launch_attention(&call, 1, p, (cudaStream_t)stream, simt);
        if (s != LL_OK) return s;
    }
    c->layers[layer].n_attn += 1;
    return LL_OK;
}

}  // namespace

namespace ll {
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
void set_last_error(const char *msg) { g_err = msg; }
}  // namespace ll

extern "C" {

const char *ll_last_error(void) { return g_err.c_str(); }
const char *ll_version(void) { return "llattn 0.1 (sm_100a)"; }
int64_t ll_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int ll_cache_create(int layers, int heads, int head_dim, int tokens_per_frame, int chunk_frames,
                    int sink_frames, int window_frames, ll_cache **out)
{
    if (!out) return fail(LL_ERR_INVALID_ARG, "out is null");
    *out = nullptr;
    if (layers <= 0 || heads <= 0 || tokens_per_frame <= 0 || chunk_frames <= 0 || sink_frames < 0 ||
        window_frames <= 0)
        return fail(LL_ERR_INVALID_ARG, "non-positive size");
    if (head_dim != 64 && head_dim != 128)
        return fail(LL_ERR_UNSUPPORTED_SHAPE, "head_dim %d: only 64 and 128 are built", head_dim);
    if (sink_frames % chunk_frames || window_frames % chunk_frames || window_frames < chunk_frames)
        return fail(LL_ERR_UNSUPPORTED_SHAPE, "sink_frames and window_frames must be multiples of chunk_frames");
    if (sink_frames + window_frames > LL_MAX_SLOTS)
        return fail(LL_ERR_UNSUPPORTED_SHAPE, "sink_frames + window_frames > %d", LL_MAX_SLOTS);
    if (window_frames / chunk_frames > ll::kMaxGroups)
        return fail(LL_ERR_UNSUPPORTED_SHAPE, "window_frames / chunk_frames > %d", ll::kMaxGroups);
    int64_t rows = (int64_t)(sink_frames + window_frames) * tokens_per_frame;
    if (rows > (1ll << 30) || (int64_t)window_frames * tokens_per_frame > (1ll << 30))
        return fail(LL_ERR_UNSUPPORTED_SHAPE, "cache rows per head exceed 2^30");

    ll_cache *c = new ll_cache();
    c->L = layers; c->H = heads; c->D = head_dim; c->P = tokens_per_frame;
    c->C = chunk_frames; c->S = sink_frames; c->W = window_frames;
    c->n_slots = sink_frames + window_frames;
    c->rows = rows;
    c->layers.resize(layers);
    for (auto &l : c->layers)
        for (int s = 0; s < LL_MAX_SLOTS; ++s) l.slot_frame[s] = -1;
    c->scales.assign((size_t)layers * 2 * heads, 1.f);
    const char *dbg = getenv("LL_DEBUG");
    c->debug = dbg && dbg[0] && dbg[0] != '0';
    compute_layout(c);
    *out = c;
    return LL_OK;
}

void ll_cache_destroy(ll_cache *cache) { delete cache; }

size_t ll_cache_storage_bytes(const ll_cache *c)
{
    if (!c) return 0;
    return c->aux_bytes + (size_t)c->L * 2 * c->kv_store_bytes + (c->debug ? kGuardBytes : 0);
}

int ll_cache_bind_storage(ll_cache *c, void *dev, size_t bytes, ll_stream stream)
{
    if (!c || !dev) return fail(LL_ERR_INVALID_ARG, "null handle or storage");
    if (reinterpret_cast<uintptr_t>(dev) & 1023u) return fail(LL_ERR_INVALID_ARG, "storage must be 1024-byte aligned");
    if (bytes < ll_cache_storage_bytes(c))
        return fail(LL_ERR_INVALID_ARG, "storage too small: %zu < %zu bytes", bytes, ll_cache_storage_bytes(c));
    if (c->dry_run) return fail(LL_ERR_INVALID_ARG, "handle is in bookkeeping-only mode");
    cudaError_t e = cudaMemsetAsync(dev, 0, ll_cache_storage_bytes(c), (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(storage)");
    if (c->debug) {
        c->off_guard1 = c->aux_bytes + (size_t)c->L * 2 * c->kv_store_bytes;
        e = cudaMemsetAsync(static_cast<char *>(dev) + c->off_guard0, kGuardByte, kGuardBytes, (cudaStream_t)stream);
        if (e == cudaSuccess)
            e = cudaMemsetAsync(static_cast<char *>(dev) + c->off_guard1, kGuardByte, kGuardBytes, (cudaStream_t)stream);
        if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync(guard bands)");
    }
    cudaPointerAttributes attr;
    int sms = 0;
    e = cudaPointerGetAttributes(&attr, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, attr.device);
    if (e != cudaSuccess) return cuda_fail(e, "query of the storage's device");
    c->sm_count = sms;
    std::vector<CUtensorMap> km(c->L), vm(c->L);
    char *base = static_cast<char *>(dev) + c->aux_bytes;
    if (c->kv_format == LL_KV_E4M3) {
        // the attention kernel reads the bf16 staging pair, whichever layer was expanded into it
        char *k = static_cast<char *>(dev) + c->off_stage;
        int s = encode_map(&c->stage_kmap, k, c->D, (uint64_t)c->rows, c->H, (uint64_t)c->D * 2,
                           (uint64_t)c->rows * c->D * 2, 128, 1);
        if (s != LL_OK) return s;
        s = encode_map(&c->stage_vmap, k + c->kv_bytes, c->D, (uint64_t)c->rows, c->H, (uint64_t)c->D * 2,
                       (uint64_t)c->rows * c->D * 2, 128, 1);
        if (s != LL_OK) return s;
        e = cudaMemcpyAsync(static_cast<char *>(dev) + c->off_scales, c->scales.data(), c->scales.size() * sizeof(float),
                            cudaMemcpyHostToDevice, (cudaStream_t)stream);
        if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync(scales)");
    }
    for (int l = 0; l < c->L && c->kv_format == LL_KV_BF16; ++l) {
        char *k = base + (size_t)l * 2 * c->kv_bytes;
        int s = encode_map(&km[l], k, c->D, (uint64_t)c->rows, c->H, (uint64_t)c->D * 2,
                           (uint64_t)c->rows * c->D * 2, 128, 1);
        if (s != LL_OK) return s;
        s = encode_map(&vm[l], k + c->kv_bytes, c->D, (uint64_t)c->rows, c->H, (uint64_t)c->D * 2,
                       (uint64_t)c->rows * c->D * 2, 128, 1);
        if (s != LL_OK) return s;
    }
    c->kmap.swap(km); c->vmap.swap(vm);
    c->storage = static_cast<char *>(dev);
    c->storage_bytes = bytes;
    c->hw_valid = false; c->t_base = -1;
    return LL_OK;
}

int ll_cache_set_kv_format(ll_cache *c, int format)
{
    if (!c) return fail(LL_ERR_INVALID_ARG, "null handle");
    if (format != LL_KV_BF16 && format != LL_KV_E4M3) return fail(LL_ERR_INVALID_ARG, "unknown cache format %d", format);
    if (c->storage) return fail(LL_ERR_INVALID_ARG, "the cache format is fixed once storage is bound");
    static_assert(LL_MAX_SLOTS / 2 + 1 <= ll::kMaxStageRuns, "staging run list too short");
    c->kv_format = format;
    compute_layout(c);
    return LL_OK;
}

int ll_cache_set_kv_scales(ll_cache *c, int layer, const float *k_scale, const float *v_scale, ll_stream stream)
{
    if (!layer_ok(c, layer) || !k_scale || !v_scale) return fail(LL_ERR_INVALID_ARG, "bad argument to ll_cache_set_kv_scales");
    if (c->kv_format != LL_KV_E4M3) return fail(LL_ERR_INVALID_ARG, "scales belong to the 8-bit cache format");
    for (int h = 0; h < c->H; ++h)
        if (!(k_scale[h] > 0.f) || !(v_scale[h] > 0.f) || !std::isfinite(k_scale[h]) || !std::isfinite(v_scale[h]))
            return fail(LL_ERR_INVALID_ARG, "scales must be positive and finite");
    float *dst = c->scales.data() + (size_t)layer * 2 * c->H;
    memcpy(dst, k_scale, c->H * sizeof(float));
    memcpy(dst + c->H, v_scale, c->H * sizeof(float));
    if (c->storage && !c->dry_run) {
        cudaError_t e = cudaMemcpyAsync(c->storage + c->off_scales + (size_t)layer * 2 * c->H * sizeof(float), dst,
                                        2 * c->H * sizeof(float), cudaMemcpyHostToDevice, (cudaStream_t)stream);
        if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync(scales)");
    }
    return LL_OK;
}

int ll_cache_kv_offset(const ll_cache *c, int layer, int which, int head, size_t *offset)
{
    if (!layer_ok(c, layer) || !offset || which < 0 || which > 1 || head < 0 || head >= c->H)
        return fail(LL_ERR_INVALID_ARG, "bad argument to ll_cache_kv_offset");
    *offset = c->aux_bytes + (size_t)layer * 2 * c->kv_store_bytes + (size_t)which * c->kv_store_bytes +
              (size_t)head * (c->kv_store_bytes / c->H);
    return LL_OK;
}

namespace {
// ll_rope_append_kv, and with gains given ll_norm_rope_append_kv.
int append_entry(ll_cache *c, int layer, const ll_bf16 *q, const ll_bf16 *k, const ll_bf16 *v,
                 const float *gain_q, const float *gain_k, float eps, bool with_norm,
                 int64_t frame_start, int n_frames, int grid_h, int grid_w, float rope_theta,
                 ll_bf16 *q_out, ll_stream stream)
{
    Range range(with_norm ? "ll_norm_rope_append_kv" : "ll_rope_append_kv", layer, (long long)frame_start);
    if (!layer_ok(c, layer)) return fail(LL_ERR_INVALID_ARG, "bad cache handle or layer %d", layer);
    if (grid_h <= 0 || grid_w <= 0 || (int64_t)grid_h * grid_w != c->P)
        return fail(LL_ERR_INVALID_ARG, "grid %dx%d does not give %d tokens per frame", grid_h, grid_w, c->P);
    if (!(rope_theta > 0.f)) return fail(LL_ERR_INVALID_ARG, "rope_theta must be positive");
    if (with_norm && c->kv_format != LL_KV_BF16)
        return fail(LL_ERR_UNSUPPORTED_SHAPE, "the fused norm is built for bf16 caches only");
    if (n_frames != c->C) return fail(LL_ERR_BAD_POSITION, "n_frames %d != chunk_frames %d", n_frames, c->C);
    ll::LayerState &st = c->layers[layer];
    const bool is_new = frame_start == st.end;
    const bool is_over = st.end >= c->C && frame_start == st.end - c->C;
    if (!is_new && !is_over)
        return fail(LL_ERR_BAD_POSITION, "frame_start %lld is neither end (%lld) nor end - chunk_frames",
                    (long long)frame_start, (long long)st.end);
    if (frame_start + n_frames > INT32_MAX) return fail(LL_ERR_BAD_POSITION, "frame index exceeds int32");
    if (!c->dry_run) {
        if (!k || !v) return fail(LL_ERR_INVALID_ARG, "null k or v");
        if (q_out && !q) return fail(LL_ERR_INVALID_ARG, "q_out given without q");
        if (!aligned16(k) || !aligned16(v) || !aligned16(q) || !aligned16(q_out))
            return fail(LL_ERR_INVALID_ARG, "q/k/v/q_out must be 16-byte aligned");
        if (with_norm && (!gain_k || (q_out && !gain_q))) return fail(LL_ERR_INVALID_ARG, "null gain");
        if (with_norm && (!aligned16(gain_q) || !aligned16(gain_k)))
            return fail(LL_ERR_INVALID_ARG, "gains must be 16-byte aligned");
        int s = need_storage(c);
        if (s != LL_OK) return s;
        s = ensure_tables(c, frame_start, frame_start + n_frames, grid_h, grid_w, rope_theta, (cudaStream_t)stream);
        if (s != LL_OK) return s;
        ll::RopeAppendParams p;
        fill_rope_params(c, layer, q_out ? q : nullptr, k, v, q_out, frame_start, n_frames, grid_w, &p);
        cudaError_t e = with_norm ? ll::launch_norm_rope_append(p, c->D, gain_q, gain_k, eps, (cudaStream_t)stream)
                                  : launch_append(c, p, (cudaStream_t)stream);
        if (e != cudaSuccess) return cuda_fail(e, "rope+append kernel");
    }
    if (is_new) {
        for (int i = 0; i < n_frames; ++i) {
            int64_t f = frame_start + i;
            int s = slot_of(c, f);
            if (st.slot_frame[s] >= 0 && st.slot_frame[s] != (int32_t)f) st.n_evictions += 1;
            st.slot_frame[s] = (int32_t)f;
        }
        st.end += n_frames;
        st.n_appends += 1;
    } else {
        st.n_overwrites += 1;
    }
    return LL_OK;
}
}  // namespace

int ll_rope_append_kv(ll_cache *c, int layer, const ll_bf16 *q, const ll_bf16 *k, const ll_bf16 *v,
                      int64_t frame_start, int n_frames, int grid_h, int grid_w, float rope_theta,
                      ll_bf16 *q_out, ll_stream stream)
{
    return append_entry(c, layer, q, k, v, nullptr, nullptr, 0.f, false, frame_start, n_frames, grid_h, grid_w,
                        rope_theta, q_out, stream);
}

int ll_norm_rope_append_kv(ll_cache *c, int layer, const ll_bf16 *q, const ll_bf16 *k, const ll_bf16 *v,
                           const float *gain_q, const float *gain_k, float eps, int64_t frame_start, int n_frames,
                           int grid_h, int grid_w, float rope_theta, ll_bf16 *q_out, ll_stream stream)
{
    if (!(eps >= 0.f)) return fail(LL_ERR_INVALID_ARG, "eps must be non-negative");
    return append_entry(c, layer, q, k, v, gain_q, gain_k, eps, true, frame_start, n_frames, grid_h, grid_w,
                        rope_theta, q_out, stream);
}

int ll_sink_window_attn(ll_cache *c, int layer, const ll_bf16 *q_roped, int64_t q_frame_start,
                        int n_q_frames, ll_bf16 *out, float *lse_out, ll_stream stream)
{
    return attn_entry(c, layer, q_roped, q_frame_start, n_q_frames, out, lse_out, stream, false);
}

int ll_sink_window_attn_scaled(ll_cache *c, int layer, const ll_bf16 *q_roped, const float *q_row_scale,
                               int64_t q_frame_start, int n_q_frames, ll_bf16 *out, float *lse_out, ll_stream stream)
{
    if (q_row_scale && !aligned16(q_row_scale)) return fail(LL_ERR_INVALID_ARG, "q_row_scale must be 16-byte aligned");
    return attn_entry(c, layer, q_roped, q_frame_start, n_q_frames, out, lse_out, stream, false, q_row_scale);
}

size_t ll_qkv_proj_workspace_bytes(const ll_cache *c)
{
    if (!c) return 0;
    const size_t tokens = (size_t)c->C * c->P, hd = (size_t)c->H * c->D;
    // parked fp32 k rows, then the per-tile sums of squares of q and k
    return align_up(tokens * hd * sizeof(float), 256) + align_up(2 * tokens * ((hd + 95) / 96) * sizeof(float), 256);
}

int ll_qkv_proj_append(ll_cache *c, int layer, const ll_bf16 *x, int d_model, const ll_bf16 *w_qkv, const float *bias,
                       const float *gain_q, const float *gain_k, float eps, int64_t frame_start, int n_frames,
                       int grid_h, int grid_w, float rope_theta, ll_bf16 *q_out, float *q_row_scale,
                       void *workspace, size_t workspace_bytes, ll_stream stream)
{
    if (!layer_ok(c, layer)) return fail(LL_ERR_INVALID_ARG, "bad cache handle or layer %d", layer);
    if (grid_h <= 0 || grid_w <= 0 || (int64_t)grid_h * grid_w != c->P)
        return fail(LL_ERR_INVALID_ARG, "grid %dx%d does not give %d tokens per frame", grid_h, grid_w, c->P);
    if (!(rope_theta > 0.f)) return fail(LL_ERR_INVALID_ARG, "rope_theta must be positive");
    Range range("ll_qkv_proj_append", layer, (long long)frame_start);
    if (d_model < 64 || d_model % 8) return fail(LL_ERR_UNSUPPORTED_SHAPE, "d_model must be a multiple of 8, at least 64");
    if (((c->H * c->D) % 256 && (c->H * c->D) % 192) || c->H * c->D > 8192)
        return fail(LL_ERR_UNSUPPORTED_SHAPE, "heads * head_dim must be a multiple of 256 or of 192, at most 8192");
    if (c->kv_format != LL_KV_BF16) return fail(LL_ERR_UNSUPPORTED_SHAPE, "the fused projection is built for bf16 caches only");
    const bool with_norm = gain_q || gain_k;
    if (with_norm && (!gain_q || !gain_k || !(eps >= 0.f))) return fail(LL_ERR_INVALID_ARG, "both gains and eps >= 0 are needed for the norm");
    if (n_frames != c->C) return fail(LL_ERR_BAD_POSITION, "n_frames %d != chunk_frames %d", n_frames, c->C);
    ll::LayerState &st = c->layers[layer];
    const bool is_new = frame_start == st.end;
    const bool is_over = st.end >= c->C && frame_start == st.end - c->C;
    if (!is_new && !is_over)
        return fail(LL_ERR_BAD_POSITION, "frame_start %lld is neither end (%lld) nor end - chunk_frames",
                    (long long)frame_start, (long long)st.end);
    if (frame_start + n_frames > INT32_MAX) return fail(LL_ERR_BAD_POSITION, "frame index exceeds int32");
    if (!c->dry_run) {
        if (!x || !w_qkv || !q_out) return fail(LL_ERR_INVALID_ARG, "null x, w_qkv or q_out");
        if (!aligned16(x) || !aligned16(w_qkv) || !aligned16(q_out) || !aligned16(bias) || !aligned16(gain_q) ||
            !aligned16(gain_k) || !aligned16(q_row_scale) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
            return fail(LL_ERR_INVALID_ARG, "pointers must be 16-byte aligned (workspace: 256)");
        if (with_norm && (!q_row_scale || !workspace || workspace_bytes < ll_qkv_proj_workspace_bytes(c)))
            return fail(LL_ERR_INVALID_ARG, "the norm needs q_row_scale and a workspace of ll_qkv_proj_workspace_bytes");
        int s = need_storage(c);
        if (s != LL_OK) return s;
        s = ensure_tables(c, frame_start, frame_start + n_frames, grid_h, grid_w, rope_theta, (cudaStream_t)stream);
        if (s != LL_OK) return s;
        ll::RopeAppendParams rp;
        fill_rope_params(c, layer, nullptr, nullptr, nullptr, nullptr, frame_start, n_frames, grid_w, &rp);
        ll::QkvParams p;
        memset(&p, 0, sizeof p);
        p.n_tokens = n_frames * c->P; p.d_model = d_model; p.heads = c->H; p.head_dim = c->D;
        p.m_tiles = (p.n_tokens + 127) / 128;
        {
            // tile width: the one whose last round of tiles leaves the SMs less idle
            const int hd = c->H * c->D, sms = c->sm_count > 0 ? c->sm_count : 148;
            long long best = -1;
            for (int tn : {256, 192}) {
                if (hd % tn) continue;
                const long long tiles = (long long)p.m_tiles * (3 * hd / tn), cost = (tiles + sms - 1) / sms * tn;
                if (best < 0 || cost < best) { best = cost; p.tile_n = tn; }
            }
            p.n_tiles = 3 * hd / p.tile_n;
            p.ssq_slots = 2 * hd / p.tile_n;
        }
        p.P = c->P; p.grid_w = grid_w; p.n_t = rp.n_t; p.n_h = rp.n_h;
        p.with_norm = with_norm ? 1 : 0; p.eps = eps;
        p.bias = bias; p.gain_q = gain_q; p.gain_k = gain_k;
        p.t_tab = rp.t_tab; p.h_tab = rp.h_tab; p.w_tab = rp.w_tab;
        p.q_out = q_out; p.q_row_scale = q_row_scale;
        p.kcache = static_cast<ll_bf16 *>(rp.kcache); p.vcache = static_cast<ll_bf16 *>(rp.vcache);
        p.rows_per_head = c->rows;
        p.k_park = static_cast<float *>(workspace);
        p.ssq = reinterpret_cast<float *>(static_cast<char *>(workspace) +
                                          align_up((size_t)p.n_tokens * c->H * c->D * sizeof(float), 256));
        p.status = reinterpret_cast<uint32_t *>(c->storage + c->off_status);
        for (int i = 0; i < n_frames; ++i) p.slot[i] = rp.slot[i];
        CUtensorMap xmap, wmap;
        s = encode_map(&xmap, x, (uint64_t)d_model, (uint64_t)p.n_tokens, 1, (uint64_t)d_model * 2,
                       (uint64_t)p.n_tokens * d_model * 2, 128, 1);
        if (s != LL_OK) return s;
        s = encode_map(&wmap, w_qkv, (uint64_t)d_model, (uint64_t)3 * c->H * c->D, 1, (uint64_t)d_model * 2,
                       (uint64_t)3 * c->H * c->D * d_model * 2, (uint32_t)p.tile_n, 1);
        if (s != LL_OK) return s;
        cudaError_t e = ll::launch_qkv_gemm(p, xmap, wmap, c->sm_count > 0 ? c->sm_count : 148, (cudaStream_t)stream);
        if (e != cudaSuccess) return cuda_fail(e, "qkv projection kernel");
    }
    if (is_new) {
        for (int i = 0; i < n_frames; ++i) {
            int64_t f = frame_start + i;
            int sl = slot_of(c, f);
            if (st.slot_frame[sl] >= 0 && st.slot_frame[sl] != (int32_t)f) st.n_evictions += 1;
            st.slot_frame[sl] = (int32_t)f;
        }
        st.end += n_frames;
        st.n_appends += 1;
    } else {
        st.n_overwrites += 1;
    }
    return LL_OK;
}

int ll_sink_window_attn_batched(const ll_attn_item *items, int n_items, ll_stream stream)
{
    Range range("ll_sink_window_attn_batched items", n_items, 0);
    if (!items || n_items < 1) return fail(LL_ERR_INVALID_ARG, "no items");
    if (n_items > LL_MAX_BATCH) return fail(LL_ERR_UNSUPPORTED_SHAPE, "more than %d items", LL_MAX_BATCH);
    static_assert(LL_MAX_BATCH == ll::kMaxItems, "header and kernel disagree on the batch limit");
    AttnCall calls[ll::kMaxItems];
    for (int i = 0; i < n_items; ++i) {
        const ll_attn_item &it = items[i];
        int s = check_decode_item(it.cache, it.layer, it.q_roped, it.q_frame_start, it.n_q_frames, it.out, it.lse_out);
        if (s != LL_OK) return s;
        if (it.cache->dry_run != items[0].cache->dry_run)
            return fail(LL_ERR_INVALID_ARG, "bookkeeping-only and real handles cannot share a launch");
        for (int j = 0; j < i; ++j)
            if (items[j].cache == it.cache && items[j].layer == it.layer)
                return fail(LL_ERR_INVALID_ARG, "items %d and %d name the same layer of the same cache", j, i);
        calls[i] = AttnCall{it.cache, it.layer, it.q_roped, it.out, it.lse_out, 1, {it.q_frame_start}, 0};
    }
    ll::AttnParams p;
    int s = build_attn_params(calls, n_items, &p);
    if (s != LL_OK) return s;
    if (!items[0].cache->dry_run) {
        s = launch_attention(calls, n_items, p, (cudaStream_t)stream, false);
        if (s != LL_OK) return s;
    }
    for (int i = 0; i < n_items; ++i) items[i].cache->layers[items[i].layer].n_attn += 1;
    return LL_OK;
}

int ll_debug_attn_simt(ll_cache *c, int layer, const ll_bf16 *q_roped, int64_t q_frame_start,
                       int n_q_frames, ll_bf16 *out, float *lse_out, ll_stream stream)
{
    return attn_entry(c, layer, q_roped, q_frame_start, n_q_frames, out, lse_out, stream, true);
}

int ll_recache(ll_cache *c, int layer, const ll_bf16 *q, const ll_bf16 *k, const ll_bf16 *v, int n_frames,
               int grid_h, int grid_w, float rope_theta, ll_bf16 *q_out, ll_bf16 *out, float *lse_out,
               ll_stream stream)
{
    if (!layer_ok(c, layer)) return fail(LL_ERR_INVALID_ARG, "bad cache handle or layer %d", layer);
    if (grid_h <= 0 || grid_w <= 0 || (int64_t)grid_h * grid_w != c->P)
        return fail(LL_ERR_INVALID_ARG, "grid %dx%d does not give %d tokens per frame", grid_h, grid_w, c->P);
    if (!(rope_theta > 0.f)) return fail(LL_ERR_INVALID_ARG, "rope_theta must be positive");
    ll::LayerState &st = c->layers[layer];
    const int64_t r0 = std::max<int64_t>(c->S, st.end - c->W);
    Range range("ll_recache", layer, (long long)r0);
    const int64_t resident = std::max<int64_t>(0, st.end - r0);
    if (n_frames != resident)
        return fail(LL_ERR_BAD_POSITION, "n_frames %d != resident window frames %lld", n_frames, (long long)resident);
    if (n_frames == 0) return LL_OK;
    const int n_groups = n_frames / c->C;
    int64_t gstart[ll::kMaxGroups];
    for (int g = 0; g < n_groups; ++g) gstart[g] = r0 + (int64_t)g * c->C;
    if (!c->dry_run) {
        if (!q || !k || !v || !q_out || !out) return fail(LL_ERR_INVALID_ARG, "null q/k/v/q_out/out");
        if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(q_out) || !aligned16(out) ||
            (lse_out && !aligned16(lse_out)))
            return fail(LL_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
        int s = need_storage(c);
        if (s != LL_OK) return s;
    }
    AttnCall call{c, layer, q_out, out, lse_out, n_groups, {}, r0};
    for (int g = 0; g < n_groups; ++g) call.group_frame_start[g] = gstart[g];
    ll::AttnParams ap;
    int s = build_attn_params(&call, 1, &ap);
    if (s != LL_OK) return s;
    if (!c->dry_run) {
        s = ensure_tables(c, r0, st.end, grid_h, grid_w, rope_theta, (cudaStream_t)stream);
        if (s != LL_OK) return s;
        ll::RopeAppendParams rp;
        fill_rope_params(c, layer, q, k, v, q_out, r0, n_frames, grid_w, &rp);
        cudaError_t e = launch_append(c, rp, (cudaStream_t)stream);
        if (e != cudaSuccess) return cuda_fail(e, "rope+append kernel (recache)");
        s = launch_attention(&call, 1, ap, (cudaStream_t)stream, false);
        if (s != LL_OK) return s;
    }
    st.n_recaches += 1;
    return LL_OK;
}

int ll_cross_attn(ll_cache *c, const ll_bf16 *q, int64_t n_q, const ll_bf16 *k, const ll_bf16 *v, int64_t n_k,
                  ll_bf16 *out, float *lse_out, ll_stream stream)
{
    Range range("ll_cross_attn keys", (int)n_k, 0);
    if (!c) return fail(LL_ERR_INVALID_ARG, "null handle");
    if (n_q <= 0 || n_k <= 0) return fail(LL_ERR_INVALID_ARG, "n_q and n_k must be positive");
    if (n_q > (1ll << 30) || n_k > (1ll << 30)) return fail(LL_ERR_UNSUPPORTED_SHAPE, "more than 2^30 queries or keys");
    if (!c->dry_run) {
        if (!q || !k || !v || !out) return fail(LL_ERR_INVALID_ARG, "null q/k/v/out");
        if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || (lse_out && !aligned16(lse_out)))
            return fail(LL_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
        int s = need_storage(c);
        if (s != LL_OK) return s;
    }
    AttnCall call{c, 0, q, out, lse_out, 1, {}, 0, {}, n_q, n_k, k, v};
    ll::AttnParams p;
    int s = build_attn_params(&call, 1, &p);
    if (s != LL_OK) return s;
    if (!c->dry_run) {
        s = launch_attention(&call, 1, p, (cudaStream_t)stream, false);
        if (s != LL_OK) return s;
    }
    return LL_OK;
}

int ll_clip_append_attn(ll_cache *c, int layer, const ll_bf16 *q, const ll_bf16 *k, const ll_bf16 *v,
                        int64_t frame_start, int n_frames, int attn_window_frames, int grid_h, int grid_w,
                        float rope_theta, ll_bf16 *q_out, ll_bf16 *out, float *lse_out, ll_stream stream)
{
    if (!layer_ok(c, layer)) return fail(LL_ERR_INVALID_ARG, "bad cache handle or layer %d", layer);
    if (grid_h <= 0 || grid_w <= 0 || (int64_t)grid_h * grid_w != c->P)
        return fail(LL_ERR_INVALID_ARG, "grid %dx%d does not give %d tokens per frame", grid_h, grid_w, c->P);
    if (!(rope_theta > 0.f)) return fail(LL_ERR_INVALID_ARG, "rope_theta must be positive");
    Range range("ll_clip_append_attn", layer, (long long)frame_start);
    if (n_frames <= 0 || n_frames % c->C)
        return fail(LL_ERR_BAD_POSITION, "n_frames %d is not a positive multiple of chunk_frames %d", n_frames, c->C);
    const int n_groups = n_frames / c->C;
    if (n_groups > ll::kMaxGroups) return fail(LL_ERR_UNSUPPORTED_SHAPE, "more than %d chunks in a clip", ll::kMaxGroups);
    if (attn_window_frames < c->C || attn_window_frames % c->C)
        return fail(LL_ERR_INVALID_ARG, "attn_window_frames %d is not a positive multiple of chunk_frames", attn_window_frames);
    if ((int64_t)attn_window_frames + n_frames - c->C > c->W)
        return fail(LL_ERR_UNSUPPORTED_SHAPE,
                    "the ring (%d frames) is shorter than attn_window_frames + n_frames - chunk_frames = %lld: the first "
                    "chunk's window would be evicted before it is read",
                    c->W, (long long)attn_window_frames + n_frames - c->C);
    ll::LayerState &st = c->layers[layer];
    if (frame_start != st.end)
        return fail(LL_ERR_BAD_POSITION, "frame_start %lld is not the end of the stream (%lld)", (long long)frame_start,
                    (long long)st.end);
    if (frame_start + n_frames > INT32_MAX) return fail(LL_ERR_BAD_POSITION, "frame index exceeds int32");
    if (!c->dry_run) {
        if (!q || !k || !v || !q_out || !out) return fail(LL_ERR_INVALID_ARG, "null q/k/v/q_out/out");
        if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(q_out) || !aligned16(out) ||
            (lse_out && !aligned16(lse_out)))
            return fail(LL_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
        int s = need_storage(c);
        if (s != LL_OK) return s;
    }
    // the clip's frames take their slots first (the plan below reads the slot table); undone on error
    const ll::LayerState saved = st;
    for (int i = 0; i < n_frames; ++i) {
        const int64_t f = frame_start + i;
        const int slot = slot_of(c, f);
        if (st.slot_frame[slot] >= 0 && st.slot_frame[slot] != (int32_t)f) st.n_evictions += 1;
        st.slot_frame[slot] = (int32_t)f;
    }
    st.end += n_frames;
    st.n_appends += n_groups;
    AttnCall call{c, layer, q_out, out, lse_out, n_groups, {}, 0, {}};
    for (int g = 0; g < n_groups; ++g) {
        call.group_frame_start[g] = frame_start + (int64_t)g * c->C;
        call.group_lo_floor[g] = call.group_frame_start[g] + c->C - attn_window_frames;
    }
    ll::AttnParams ap;
    int s = build_attn_params(&call, 1, &ap);
    if (s == LL_OK && !c->dry_run) {
        s = ensure_tables(c, frame_start, frame_start + n_frames, grid_h, grid_w, rope_theta, (cudaStream_t)stream);
        if (s == LL_OK) {
            ll::RopeAppendParams rp;
            fill_rope_params(c, layer, q, k, v, q_out, frame_start, n_frames, grid_w, &rp);
            cudaError_t e = launch_append(c, rp, (cudaStream_t)stream);
            if (e != cudaSuccess) s = cuda_fail(e, "rope+append kernel (clip)");
        }
        if (s == LL_OK) s = launch_attention(&call, 1, ap, (cudaStream_t)stream, false);
    }
    if (s != LL_OK) {
        st = saved;
        return s;
    }
    st.n_attn += 1;
    return LL_OK;
}

size_t ll_clip_backward_workspace_bytes(const ll_cache *c, int n_frames)
{
    if (!c || n_frames <= 0) return 0;
    return align_up((size_t)c->H * n_frames * c->P * sizeof(float), 256);
}

int ll_clip_attn_backward(ll_cache *c, int layer, const ll_bf16 *q_roped, const ll_bf16 *out, const ll_bf16 *d_out,
                          const float *lse, int64_t frame_start, int n_frames, int attn_window_frames, int grid_h,
                          int grid_w, float rope_theta, ll_bf16 *dq, ll_bf16 *dk, ll_bf16 *dv, void *workspace,
                          size_t workspace_bytes, ll_stream stream)
{
    Range range("ll_clip_attn_backward", layer, (long long)frame_start);
    if (!layer_ok(c, layer)) return fail(LL_ERR_INVALID_ARG, "bad cache handle or layer %d", layer);
    if (grid_h <= 0 || grid_w <= 0 || (int64_t)grid_h * grid_w != c->P)
        return fail(LL_ERR_INVALID_ARG, "grid %dx%d does not give %d tokens per frame", grid_h, grid_w, c->P);
    if (!(rope_theta > 0.f)) return fail(LL_ERR_INVALID_ARG, "rope_theta must be positive");
    if (c->kv_format != LL_KV_BF16) return fail(LL_ERR_UNSUPPORTED_SHAPE, "the backward pass is built for bf16 caches only");
    if (n_frames <= 0 || n_frames % c->C)
        return fail(LL_ERR_BAD_POSITION, "n_frames %d is not a positive multiple of chunk_frames %d", n_frames, c->C);
    const int n_groups = n_frames / c->C;
    if (n_groups > ll::kMaxGroups) return fail(LL_ERR_UNSUPPORTED_SHAPE, "more than %d chunks in a clip", ll::kMaxGroups);
    if (attn_window_frames < c->C || attn_window_frames % c->C)
        return fail(LL_ERR_INVALID_ARG, "attn_window_frames %d is not a positive multiple of chunk_frames", attn_window_frames);
    if ((int64_t)attn_window_frames + n_frames - c->C > c->W)
        return fail(LL_ERR_UNSUPPORTED_SHAPE, "the ring (%d frames) cannot have held this clip's windows", c->W);
    ll::LayerState &st = c->layers[layer];
    if (frame_start < 0 || frame_start + n_frames != st.end)
        return fail(LL_ERR_BAD_POSITION, "the clip [%lld, %lld) is not the newest %d frames of the stream (end %lld)",
                    (long long)frame_start, (long long)frame_start + n_frames, n_frames, (long long)st.end);
    if ((int64_t)n_frames * c->P > INT32_MAX / 2) return fail(LL_ERR_UNSUPPORTED_SHAPE, "clip too long");
    if (c->dry_run) return LL_OK;
    if (!q_roped || !out || !d_out || !lse || !dq || !dk || !dv || !workspace)
        return fail(LL_ERR_INVALID_ARG, "null tensor or workspace");
    if (!aligned16(q_roped) || !aligned16(out) || !aligned16(d_out) || !aligned16(lse) || !aligned16(dq) || !aligned16(dk) ||
        !aligned16(dv) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return fail(LL_ERR_INVALID_ARG, "pointers must be 16-byte aligned (workspace: 256)");
    if (workspace_bytes < ll_clip_backward_workspace_bytes(c, n_frames))
        return fail(LL_ERR_INVALID_ARG, "workspace smaller than ll_clip_backward_workspace_bytes");
    int s = need_storage(c);
    if (s != LL_OK) return s;
    // the forward's query groups and key runs
    AttnCall call{c, layer, q_roped, nullptr, nullptr, n_groups, {}, 0, {}};
    for (int g = 0; g < n_groups; ++g) {
        call.group_frame_start[g] = frame_start + (int64_t)g * c->C;
        call.group_lo_floor[g] = call.group_frame_start[g] + c->C - attn_window_frames;
    }
    ll::AttnParams ap;
    s = build_attn_params(&call, 1, &ap);
    if (s != LL_OK) return s;
    s = ensure_tables(c, frame_start, frame_start + n_frames, grid_h, grid_w, rope_theta, (cudaStream_t)stream);
    if (s != LL_OK) return s;
    ll::RopeAppendParams rp;
    fill_rope_params(c, layer, nullptr, nullptr, nullptr, nullptr, frame_start, n_frames, grid_w, &rp);
    ll::BwdParams p;
    memset(&p, 0, sizeof p);
    p.n_groups = n_groups; p.heads = c->H; p.head_dim = c->D; p.nq_total = n_frames * c->P;
    p.scale = (float)(1.0 / std::sqrt((double)c->D));
    p.scale_log2 = ap.scale_log2;
    p.q = q_roped; p.out = out; p.d_out = d_out; p.lse = lse; p.delta = static_cast<float *>(workspace);
    p.dq = dq; p.dk = dk; p.dv = dv;
    p.status = reinterpret_cast<uint32_t *>(c->storage + c->off_status);
    p.P = c->P; p.grid_w = grid_w; p.n_t = rp.n_t; p.n_h = rp.n_h;
    p.t_tab = rp.t_tab; p.h_tab = rp.h_tab; p.w_tab = rp.w_tab;
    p.rows_per_head = c->rows;
    for (int g = 0; g < n_groups; ++g) {
        p.g[g] = ap.g[g];
        p.n_qtiles += (ap.g[g].q_rows + 127) / 128;
    }
    // where the clip's frames sit: contiguous slots make runs of cache rows
    for (int sl = 0; sl < LL_MAX_SLOTS; ++sl) p.slot_clip_frame[sl] = -1;
    for (int i = 0; i < n_frames; ++i) p.slot_clip_frame[slot_of(c, frame_start + i)] = i;
    for (int sl = 0; sl < c->n_slots;) {
        if (p.slot_clip_frame[sl] < 0) { ++sl; continue; }
        int e = sl;
        while (e < c->n_slots && p.slot_clip_frame[e] >= 0) ++e;
        if (p.n_kruns >= 4) return fail(LL_ERR_UNSUPPORTED_SHAPE, "the clip's frames sit in more than 4 runs of slots");
        p.krun_start[p.n_kruns] = sl * c->P;
        p.krun_len[p.n_kruns] = (e - sl) * c->P;
        p.n_ktiles += (p.krun_len[p.n_kruns] + 127) / 128;
        ++p.n_kruns;
        sl = e;
    }
    ll::BwdMaps maps;
    memset(&maps, 0, sizeof maps);
    s = token_major_map(c, &maps.q, q_roped, (uint64_t)p.nq_total);
    if (s == LL_OK) s = token_major_map(c, &maps.d_out, d_out, (uint64_t)p.nq_total);
    if (s != LL_OK) return s;
    maps.k = c->kmap[layer];
    maps.v = c->vmap[layer];
    cudaError_t e = ll::launch_attn_backward(p, maps, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e, "clip backward kernels");
    return LL_OK;
}

namespace {
void copy_plan(const ll::AttnParams &p, ll_attn_plan *out)
{
    memset(out, 0, sizeof *out);
    out->n_ctas = p.n_ctas;
    out->n_groups = p.n_groups;
    out->heads = p.heads;
    out->n_waves = p.n_waves;
    out->n_shares = p.n_shares;
    out->all_cols = p.all_cols;
    out->shared_steps = p.total_steps;
    for (int k = 0; k <= p.n_shares; ++k) out->share_begin[k] = p.share_begin[k];
    for (int i = 0; i < p.n_ctas; ++i) out->share_of_cta[i] = p.share_of_cta[i];
    for (int g = 0; g < p.n_groups; ++g) {
        out->tiles[g] = p.g[g].tiles;
        out->n_kt[g] = p.g[g].n_kt;
        out->col_begin[g] = p.g[g].col_begin;
        out->wave_cols[g] = p.g[g].wave_cols;
        out->step_begin[g] = p.g[g].step_begin;
    }
}
}  // namespace

int ll_debug_attn_plan_batched(const ll_attn_item *items, int n_items, int sm_count, ll_attn_plan *out)
{
    if (!items || !out || n_items < 1 || n_items > LL_MAX_BATCH)
        return fail(LL_ERR_INVALID_ARG, "bad argument to ll_debug_attn_plan_batched");
    AttnCall calls[ll::kMaxItems];
    for (int i = 0; i < n_items; ++i) {
        const ll_attn_item &it = items[i];
        if (!layer_ok(it.cache, it.layer)) return fail(LL_ERR_INVALID_ARG, "bad cache handle or layer in item %d", i);
        const ll::LayerState &st = it.cache->layers[it.layer];
        if (st.end < it.cache->C) return fail(LL_ERR_BAD_POSITION, "no chunk has been appended yet");
        calls[i] = AttnCall{it.cache, it.layer, nullptr, nullptr, nullptr, 1, {st.end - it.cache->C}, 0};
    }
    ll_cache *c0 = items[0].cache;
    const int saved = c0->sm_count;
    if (sm_count > 0) c0->sm_count = sm_count;
    ll::AttnParams p;
    const int s = build_attn_params(calls, n_items, &p);
    c0->sm_count = saved;
    if (s != LL_OK) return s;
    copy_plan(p, out);
    return LL_OK;
}

int ll_debug_attn_plan(ll_cache *c, int layer, int recache, int sm_count, ll_attn_plan *out)
{
    if (!layer_ok(c, layer) || !out) return fail(LL_ERR_INVALID_ARG, "bad argument to ll_debug_attn_plan");
    static_assert(LL_MAX_GROUPS == ll::kMaxGroups && LL_MAX_CTAS == ll::kMaxCtas, "header and kernel disagree on a limit");
    const ll::LayerState &st = c->layers[layer];
    int n_groups = 1;
    int64_t gstart[ll::kMaxGroups];
    int64_t lo_floor = 0;
    if (recache) {
        const int64_t r0 = std::max<int64_t>(c->S, st.end - c->W);
        n_groups = (int)(std::max<int64_t>(0, st.end - r0) / c->C);
        for (int g = 0; g < n_groups; ++g) gstart[g] = r0 + (int64_t)g * c->C;
        lo_floor = r0;
    } else {
        if (st.end < c->C) return fail(LL_ERR_BAD_POSITION, "no chunk has been appended yet");
        gstart[0] = st.end - c->C;
    }
    memset(out, 0, sizeof *out);
    if (n_groups == 0) return LL_OK;
    const int saved = c->sm_count;
    if (sm_count > 0) c->sm_count = sm_count;
    AttnCall call{c, layer, nullptr, nullptr, nullptr, n_groups, {}, lo_floor};
    for (int g = 0; g < n_groups; ++g) call.group_frame_start[g] = gstart[g];
    ll::AttnParams p;
    const int s = build_attn_params(&call, 1, &p);
    c->sm_count = saved;
    if (s != LL_OK) return s;
    copy_plan(p, out);
    return LL_OK;
}

int ll_debug_wait_timeout(ll_cache *c, int limit_ms, ll_stream stream)
{
    if (!c) return fail(LL_ERR_INVALID_ARG, "null handle");
    if (limit_ms < 1 || limit_ms > 1000) return fail(LL_ERR_INVALID_ARG, "limit_ms must be in [1, 1000]");
    int s = need_storage(c);
    if (s != LL_OK) return s;
    cudaError_t e = ll::launch_wait_probe(reinterpret_cast<uint32_t *>(c->storage + c->off_status),
                                          (uint64_t)limit_ms * 1000000ull, (cudaStream_t)stream);
    return e == cudaSuccess ? LL_OK : cuda_fail(e, "wait probe kernel");
}

int ll_debug_aux_layout(const ll_cache *c, size_t *status_offset, size_t *status_bytes, size_t *counters_offset,
                        size_t *counters_bytes)
{
    if (!c) return fail(LL_ERR_INVALID_ARG, "null handle");
    if (status_offset) *status_offset = c->off_status;
    if (status_bytes) *status_bytes = ll::kStatusWords * sizeof(uint32_t);
    if (counters_offset) *counters_offset = c->off_counters;
    if (counters_bytes) *counters_bytes = ll::counters_bytes();
    return LL_OK;
}

int ll_debug_guard_layout(const ll_cache *c, size_t *front_offset, size_t *back_offset, size_t *bytes)
{
    if (!c) return fail(LL_ERR_INVALID_ARG, "null handle");
    if (!c->debug) return fail(LL_ERR_INVALID_ARG, "the handle was not created with LL_DEBUG set");
    if (front_offset) *front_offset = c->off_guard0;
    if (back_offset) *back_offset = c->aux_bytes + (size_t)c->L * 2 * c->kv_store_bytes;
    if (bytes) *bytes = kGuardBytes;
    return LL_OK;
}

int ll_cache_reset(ll_cache *c)
{
    if (!c) return fail(LL_ERR_INVALID_ARG, "null handle");
    for (auto &l : c->layers) {
        l.end = 0;
        for (int s = 0; s < LL_MAX_SLOTS; ++s) l.slot_frame[s] = -1;
    }
    return LL_OK;
}

int ll_cache_get_state(const ll_cache *c, int layer, ll_state *out)
{
    if (!layer_ok(c, layer) || !out) return fail(LL_ERR_INVALID_ARG, "bad argument to ll_cache_get_state");
    const ll::LayerState &st = c->layers[layer];
    memset(out, 0, sizeof *out);
    out->end = st.end;
    out->n_slots = c->n_slots;
    int ring = 0;
    for (int s = 0; s < LL_MAX_SLOTS; ++s) {
        out->slot_frame[s] = s < c->n_slots ? st.slot_frame[s] : -1;
        if (s >= c->S && s < c->n_slots && st.slot_frame[s] >= 0) ++ring;
    }
    out->ring_valid = ring;
    out->n_appends = st.n_appends; out->n_overwrites = st.n_overwrites;
    out->n_evictions = st.n_evictions; out->n_recaches = st.n_recaches;
    out->n_attn_calls = st.n_attn;
    return LL_OK;
}

int ll_cache_set_state(ll_cache *c, int layer, const ll_state *in)
{
    if (!layer_ok(c, layer) || !in) return fail(LL_ERR_INVALID_ARG, "bad argument to ll_cache_set_state");
    if (in->n_slots != c->n_slots || in->end < 0 || in->end % c->C)
        return fail(LL_ERR_INVALID_ARG, "state does not belong to a cache of this shape");
    for (int s = 0; s < c->n_slots; ++s) {
        int32_t f = in->slot_frame[s];
        if (f < 0) continue;
        if (f >= in->end || slot_of(c, f) != s)
            return fail(LL_ERR_INVALID_ARG, "slot %d holds frame %d, which the slot rule does not allow", s, f);
    }
    ll::LayerState &st = c->layers[layer];
    st.end = in->end;
    for (int s = 0; s < LL_MAX_SLOTS; ++s) st.slot_frame[s] = s < c->n_slots ? in->slot_frame[s] : -1;
    st.n_appends = in->n_appends; st.n_overwrites = in->n_overwrites;
    st.n_evictions = in->n_evictions; st.n_recaches = in->n_recaches; st.n_attn = in->n_attn_calls;
    return LL_OK;
}

int ll_cache_visible_ranges(const ll_cache *c, int layer, int64_t q_frame_start, int64_t lo_floor,
                            int64_t *starts, int64_t *lens, int *n_ranges)
{
    if (!layer_ok(c, layer) || !starts || !lens || !n_ranges)
        return fail(LL_ERR_INVALID_ARG, "bad argument to ll_cache_visible_ranges");
    return visible_ranges(c, layer, q_frame_start, lo_floor, starts, lens, n_ranges);
}

int ll_cache_set_dry_run(ll_cache *c, int on)
{
    if (!c) return fail(LL_ERR_INVALID_ARG, "null handle");
    c->dry_run = on != 0;
    return LL_OK;
}

int ll_cache_device_status(ll_cache *c, ll_stream stream)
{
    if (!c) return fail(LL_ERR_INVALID_ARG, "null handle");
    int s = need_storage(c);
    if (s != LL_OK) return s;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
    uint32_t w[ll::kStatusWords];
    e = cudaMemcpy(w, c->storage + c->off_status, sizeof w, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpy(status)");
    if (w[0] == ll::kStatusOk && c->debug) {
        std::vector<unsigned char> band_buf(2 * kGuardBytes);
        unsigned char *band = band_buf.data();
        e = cudaMemcpy(band, c->storage + c->off_guard0, kGuardBytes, cudaMemcpyDeviceToHost);
        if (e == cudaSuccess) e = cudaMemcpy(band + kGuardBytes, c->storage + c->off_guard1, kGuardBytes, cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpy(guard bands)");
        for (size_t i = 0; i < 2 * kGuardBytes; ++i)
            if (band[i] != kGuardByte)
                return fail(LL_ERR_DEVICE_CHECK, "guard band %s the K/V region overwritten at byte %zu",
                            i < kGuardBytes ? "in front of" : "behind", i % kGuardBytes);
    }
    if (w[0] == ll::kStatusOk) return LL_OK;
    // A CTA that gave up, and every CTA that then skipped its work, never made its arrival on
    // the split-column counters, so the counters of that launch are left mid-count: clear them
    // together with the record, or the next launch that splits a column would merge too early.
    e = cudaMemset(c->storage + c->off_status, 0, sizeof w);
    if (e == cudaSuccess) e = cudaMemset(c->storage + c->off_counters, 0, ll::counters_bytes());
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemset(status, counters)");
    if (w[0] == ll::kStatusBadRow)
        return fail(LL_ERR_DEVICE_CHECK, "an append kernel refused storage slot %u of the call's frame %u (block %u)",
                    w[1], w[2], w[4]);
    return fail(LL_ERR_DEVICE_TIMEOUT,
                "a kernel gave up on a bounded wait: code %u role %u barrier %u iteration %u block (%u,%u,%u)",
                w[0], w[1], w[2], w[3], w[4], w[5], w[6]);
}

}  // extern "C"
