// Sink+window attention on tcgen05 tensor cores (sm_100a).
//
// Work decomposition.  A *column* is up to 256 query rows of one head (two
// 128-row MMA tiles, "lanes" 0 and 1) and a *step* is one 128-key tile of that
// column's visible cache rows.  One persistent CTA runs per SM.  The columns of
// all query groups of a launch (one per chunk of queries, of one or several
// streams) are numbered through.  As long as there is a column for every CTA,
// columns are handed out whole: the CTAs of a head then walk the keys in step and
// each K/V tile is fetched from HBM once and shared through L2.  The steps of the
// columns left over are laid end to end and cut into one share per CTA, sized on
// the host so that every SM ends up with the same number of steps whatever the
// number and length of the columns (very short columns go out whole instead).
// A column whose steps fall into several CTAs is finished by whichever of them
// arrives last:
// every part leaves its unnormalised O rows, reference maxima and sums in a
// scratch slot, bumps the column's arrival counter, and the last one merges the
// parts and writes the output.  Nothing waits on another CTA.
//
// Inside a CTA (640 threads):
//   warp 16 (one lane)  TMA producer: the column's Q tiles, then K_j V_j K_j+1 ...
//                       into a ring of 128-byte-swizzled shared-memory stages
//   warps 17, 18        MMA issuers of lane 0 and lane 1 (one elected thread each):
//                       S_w = Q_w K_j^T and O_w += P_w V_j, all operands in shared
//                       memory, accumulators in TMEM
//   warps 0-15          softmax: warp (w, q, h) owns the 16 rows 32q + 16h .. of
//                       lane w; its threads read S with the 16x256b TMEM shape, so
//                       a row lives in the four threads of a quad.  P (bf16) goes to
//                       a swizzled shared-memory tile, 64 keys at a time and as soon as
//                       a 64-key piece is computed (its registers are then free for
//                       the next piece).  The rows' reference maxima move, and O is
//                       rescaled in TMEM, only when a weight computed against the old
//                       reference would have been large.
//   P does not go back over S: a lane's S buffer is free as soon as its softmax
//   warps hold the tile in registers, so the MMA warp issues QK of step j+1 while
//   the softmax of step j is still running, and the softmax warps find the next S
//   waiting.  The tensor pipe then sees, per lane and step, PV(first half), QK(next),
//   PV(second half), whenever their inputs arrive.  A share of the exponentials can be
//   evaluated with a cubic on the FMA pipe instead of the special-function unit
//   (kPolyMask: none at head_dim 128, a quarter at head_dim 64, as measured).
//
// TMEM columns: S_0 | S_1 | O_0 | O_1 (fp32).  The visible keys are a short list of
// contiguous cache-row runs (sink, ring, wrapped ring); softmax does not care about
// key order, so the only masking is the ragged last tile of each run.
//
// Every mbarrier wait is bounded: a role that waits longer than kWaitLimitNs
// records a status word, raises the CTA's abort flag, and all roles drain to the
// common exit where TMEM is released.
#include <cuda_bf16.h>

#include <atomic>

#include "bounded_wait.cuh"
#include "exp2_poly.cuh"
#include "ll_internal.h"
#include "ptx.cuh"

namespace ll {

namespace {

using namespace ptx;

constexpr int kThreads = 640;
constexpr int kSoftmaxWarps = 16;
constexpr int kTmaWarp = 16;
constexpr int kMmaWarp = 17;
// A piece's 16 weights per thread and row were safe to compute if they sum to less than this:
// no weight can exceed the sum, and a score too far above the row's reference shows up as a
// weight of at least 2^127 on the special-function unit and of just under 256 (the top of its
// clamped range) on the polynomial path.
constexpr float kSafeSum = 128.f;
// Register reallocation draws on what the CTA was launched with: 640 threads x 96
// registers = (16 softmax warps x 104 + 4 producer-group warps x 64) x 32.  A
// request beyond that total would block forever.
constexpr int kLaunchRegs = 96;
constexpr int kSoftmaxRegs = 104;
constexpr int kProducerRegs = 64;
static_assert(kSoftmaxWarps * kSoftmaxRegs + (kThreads / 32 - kSoftmaxWarps) * kProducerRegs <= (kThreads / 32) * kLaunchRegs,
              "setmaxnreg targets exceed the CTA's register allocation");
// 8-key groups (bit k of 16 per 128-key tile) whose exponentials use the cubic instead of the
// special-function unit.  head_dim 128: none - the special-function unit is not what a step
// waits for, and the cubic's ten instructions per pair cost time and power (0.4027 ms against
// 0.4047 ms with one group in four, 0.4218 ms with two; 0.4664 / 0.4715 / 0.4915 ms in a long
// loop at the power cap).  head_dim 64 has twice the exponentials per flop and is bound by
// them: one group in four (0.681 ms against 0.726 ms with none, 0.684 / 0.683 ms with one in
// eight / three in eight, 24 heads on the same grid).
template <int D> constexpr uint32_t kPolyMask = D == 64 ? 0x8888u : 0x0000u;

template <int D>
struct Cfg {
    static constexpr int kAtoms = D / 64;                   // 128-byte swizzle atoms per row
    static constexpr int kAtomBytes = 128 * 128;            // 128 rows x 128 bytes
    static constexpr int kTileBytes = kAtoms * kAtomBytes;  // one 128-row tile of Q, K or V
    static constexpr int kPBytes = 2 * kAtomBytes;          // one lane's P: 128 rows x 128 keys
    static constexpr int kStages = (D == 128) ? 3 : 8;
    static constexpr int kSmemTiles = 2 * kTileBytes + 2 * kPBytes + kStages * kTileBytes;
    static constexpr int kSmemBytes = kSmemTiles + 1024 /*barriers*/ + 1024 /*alignment slack*/;
    static constexpr int kTmemCols = 512;
    static constexpr int kColS = 0;                         // S_w at kColS + 128 w
    static constexpr int kColO = 256;                       // O_w at kColO + D w
    static constexpr int kOChunks = D / 64;                 // 64-column pieces of an O row
};

// barrier indices inside the shared barrier array (+ lane or + stage)
enum Bar {
    kQFull = 0, kQEmpty = 2, kSFull = 4, kSEmpty = 6, kPFull = 8, kPEmpty = 10, kOFull = 12, kOEmpty = 14,
    kKvFull = 16, kKvEmpty = 24, kNumBars = 32
};

// Walks the visible key tiles of a group: runs in order, 128 rows at a time.
struct KeyIter {
    const AttnGroup *g;
    int r, off;
    __device__ KeyIter(const AttnGroup *grp, int first_tile) : g(grp), r(0), off(0)
    {
        while (first_tile > 0) {
            const int nt = (g->k_len[r] + kKeyTile - 1) / kKeyTile;
            if (first_tile >= nt) { first_tile -= nt; ++r; }
            else { off = first_tile * kKeyTile; first_tile = 0; }
        }
    }
    __device__ int row() const { return g->k_start[r] + off; }
    __device__ int valid() const { return min(kKeyTile, g->k_len[r] - off); }
    __device__ void next()
    {
        off += kKeyTile;
        if (off >= g->k_len[r]) { ++r; off = 0; }
    }
};

// One CTA's piece of one column.
struct Segment {
    int g, head, tile;      // the column
    int kt0, kt1;           // its steps [kt0, kt1) run here
    int q0;                 // first query row of the column
    int rows_valid;         // live rows of the 256
    int n_sub;              // live 128-row tiles
    int col_begin;          // shared-step index of the column's first step (split columns only)
};

// A CTA's work in order: its whole columns, wave by wave, then its share of the steps
// that are left.  Every role of the CTA walks the same sequence.
struct WorkIter {
    const AttnParams &p;
    int cta, g, wave, share;
    int u, end;
    __device__ WorkIter(const AttnParams &prm, int cta_)
        : p(prm), cta(cta_), g(0), wave(0), share(prm.share_of_cta[cta_]), u(0), end(0)
    {
        if (share >= 0) {
            u = p.share_begin[share];
            end = p.share_begin[share + 1];
        }
    }
    __device__ void fill(Segment &s, int grp, int col, int kt0, int kt1) const
    {
        const AttnGroup &G = p.g[grp];
        s.g = grp;
        s.head = col / G.tiles;
        s.tile = col - s.head * G.tiles;
        s.kt0 = kt0;
        s.kt1 = kt1;
        s.q0 = G.q_begin + s.tile * kQTileRows;
        s.rows_valid = min(kQTileRows, G.q_rows - s.tile * kQTileRows);
        s.n_sub = s.rows_valid > 128 ? 2 : 1;
    }
    __device__ bool next(Segment &s)
    {
        if (wave < p.n_waves) {
            const int col = wave * p.n_ctas + cta;                  // launch-wide column number
            ++wave;
            if (col < p.all_cols) {
                while (col >= p.g[g].col_begin + p.heads * p.g[g].tiles) ++g;
                fill(s, g, col - p.g[g].col_begin, 0, p.g[g].n_kt);
                s.col_begin = 0;
                return true;
            }
        }
        if (u >= end) return false;
        int gg = 0;
        while (gg + 1 < p.n_groups && u >= p.g[gg + 1].step_begin) ++gg;
        const AttnGroup &G = p.g[gg];
        const int off = u - (int)G.step_begin;
        const int col = off / G.n_kt;
        const int kt0 = off - col * G.n_kt;
        const int kt1 = min(G.n_kt, kt0 + (end - u));
        fill(s, gg, G.wave_cols + col, kt0, kt1);
        s.col_begin = u - kt0;
        u += kt1 - kt0;
        return true;
    }
};

// -inf into the registers of one 64-column piece (first column col0) whose key is not valid.
__device__ __forceinline__ void mask_piece(uint32_t *v, int col0, int cq, int nvalid)
{
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        if (col0 + 8 * k + cq >= nvalid) v[4 * k] = v[4 * k + 2] = 0xff800000u;
        if (col0 + 8 * k + cq + 1 >= nvalid) v[4 * k + 1] = v[4 * k + 3] = 0xff800000u;
    }
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
attn_sm100_kernel(const __grid_constant__ AttnParams p, const __grid_constant__ AttnMaps maps)
{
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t q_smem = smem_base;                                  // 2 tiles
    const uint32_t p_smem = smem_base + 2 * C::kTileBytes;              // one 64-key P tile per lane
    const uint32_t kv_smem = p_smem + 2 * C::kPBytes;                   // kStages tiles
    const uint32_t bars = smem_base + C::kSmemTiles;                    // kNumBars x 8 bytes
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem_gen + C::kSmemTiles + kNumBars * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    auto bar = [&](int i) -> uint32_t { return bars + 8u * (uint32_t)i; };

    // (the shuffle tells the compiler that the warp index is the same in all lanes, which
    // keeps the role code of the MMA warps on the uniform datapath)
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
    const int lane = threadIdx.x & 31;
    const int cta = blockIdx.x;

    // ---- setup ------------------------------------------------------------------
    if (threadIdx.x == 0) {
        for (int i = 0; i < kNumBars; ++i) {
            uint32_t count = 1;
            if ((i >= kSEmpty && i < kSEmpty + 2) || (i >= kPFull && i < kPFull + 2) || (i >= kOEmpty && i < kOEmpty + 2))
                count = kSoftmaxWarps / 2;                                     // one arrival per softmax warp of the lane
            if (i == kQEmpty || i >= kKvEmpty) count = 2;                      // both MMA warps release Q and every K/V stage
            mbar_init(bar(i), count);
        }
        // an earlier CTA already gave up on a wait: this one does not start (flag value 2)
        *abort_flag = (*reinterpret_cast<volatile uint32_t *>(p.status) != kStatusOk) ? 2 : 0;
        fence_mbar_init();
    }
    if (warp == kTmaWarp) {
        tmem_alloc(smem_u32(tmem_slot), C::kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;

    WaitCtx ctx{abort_flag, p.status, warp};
    const bool skip = *abort_flag != 0;
    auto wait = [&](int bar_id, uint32_t parity, int iter) -> bool {
        return wait_bar(bar(bar_id), parity & 1u, ctx, bar_id, iter);
    };

    if (warp >= kSoftmaxWarps) {
        // Register reallocation: the softmax warps hold half an S row pair per thread,
        // the producer warpgroup (TMA, MMA and two idle warps) needs little.
        setmaxnreg_dec<kProducerRegs>();
        if (skip) {
            // an earlier CTA gave up: nothing to do
        } else if (warp == kTmaWarp && lane == 0) {
            // =========================== TMA producer ===========================
            [&]() {
                for (int i = 0; i < p.n_items; ++i) {
                    prefetch_tensormap(&maps.q[i]);
                    prefetch_tensormap(&maps.k[i]);
                    prefetch_tensormap(&maps.v[i]);
                }
                uint32_t n = 0;                 // K/V tiles issued so far
                uint32_t seg = 0;
                Segment s;
                for (WorkIter it(p, cta); it.next(s); ++seg) {
                    // Tile order K_0, K_1, V_0, K_2, V_1, ... : the QK of a step is issued a whole
                    // softmax ahead of the step's PV, so K runs one step ahead of V and three stages
                    // (the V in use, the K in use, one in flight) keep both fed.
                    KeyIter kit_k(&p.g[s.g], s.kt0), kit_v(&p.g[s.g], s.kt0);
                    const int item = p.g[s.g].item;
                    const CUtensorMap *qmap = &maps.q[item], *kmap = &maps.k[item], *vmap = &maps.v[item];
                    auto load_kv = [&](const CUtensorMap *m, int row) -> bool {
                        const int stage = n % C::kStages;
                        if (!wait(kKvEmpty + stage, (n / C::kStages) ^ 1u, (int)n)) return false;
                        mbar_arrive_expect_tx(bar(kKvFull + stage), C::kTileBytes);
                        for (int a = 0; a < C::kAtoms; ++a)
                            tma_load_3d(kv_smem + stage * C::kTileBytes + a * C::kAtomBytes, m,
                                        bar(kKvFull + stage), a * 64, p.kv_token_major ? s.head : row,
                                        p.kv_token_major ? row : s.head);
                        ++n;
                        return true;
                    };
                    // the first key tile goes out before Q: it needs no Q buffer and is in
                    // flight while the previous column's last products drain
                    if (!load_kv(kmap, kit_k.row())) return;
                    if (seg > 0 && !wait(kQEmpty, seg - 1, (int)seg)) return;
                    for (int w = 0; w < s.n_sub; ++w) {
                        mbar_arrive_expect_tx(bar(kQFull + w), C::kTileBytes);
                        for (int a = 0; a < C::kAtoms; ++a)
                            tma_load_3d(q_smem + w * C::kTileBytes + a * C::kAtomBytes, qmap, bar(kQFull + w),
                                        a * 64, s.head, s.q0 + 128 * w);
                    }
                    for (int j = s.kt0; j < s.kt1; ++j) {
                        if (j + 1 < s.kt1) {
                            kit_k.next();
                            if (!load_kv(kmap, kit_k.row())) return;
                        }
                        if (!load_kv(vmap, kit_v.row())) return;
                        kit_v.next();
                    }
                }
            }();
        } else if (warp == kMmaWarp || warp == kMmaWarp + 1) {
            // ====================== MMA issuer of lane w = warp - kMmaWarp ======================
            // One issuing warp per lane.  Both walk the same K/V ring and both release every
            // stage (a lane that sits a column out releases it unused).  All 32 lanes walk the
            // loops and the waits, so that addresses and descriptors are warp-uniform values;
            // one elected lane issues the MMAs, commits and arrivals.
            [&]() {
                const int w = warp - kMmaWarp;
                const bool elected = elect_one();
                constexpr uint32_t idesc_qk = idesc_bf16_f32(128, 128, 0, 0);
                constexpr uint32_t idesc_pv = idesc_bf16_f32(128, D, 0, 1);
                constexpr uint32_t hi = smem_desc_hi_sw128(1024);
                const uint32_t t_sw = tmem + C::kColS + 128 * w, t_ow = tmem + C::kColO + D * w;
                // S_w = Q_w K^T: both operands K-major, 64-element atoms, 16 elements (32 bytes) per MMA
                const uint32_t q_lo = smem_desc_lo(q_smem + w * C::kTileBytes, 16);
                const uint32_t k_lo0 = smem_desc_lo(kv_smem, 16);
                // O_w += P_w V: P K-major (one 64-key atom, 16 keys = 32 bytes per MMA); V is MN-major:
                // 8-key groups 1024 bytes apart, 64-wide d atoms kAtomBytes apart
                const uint32_t p_lo = smem_desc_lo(p_smem + w * C::kPBytes, 16);
                const uint32_t v_lo0 = smem_desc_lo(kv_smem, C::kAtomBytes);
                auto issue_qk = [&](uint32_t stage) {
                    const uint32_t k_lo = k_lo0 + stage * (C::kTileBytes >> 4);
                    if (elected) {
#pragma unroll
                        for (int kk = 0; kk < D / 16; ++kk) {
                            const uint32_t off = ((kk / 4) * C::kAtomBytes + (kk % 4) * 32) >> 4;
                            mma_ss(t_sw, smem_desc_join(q_lo + off, hi), smem_desc_join(k_lo + off, hi), idesc_qk, kk > 0);
                        }
                    }
                    __syncwarp();
                };
                auto issue_pv = [&](uint32_t stage, bool first) {
                    const uint32_t v_lo = v_lo0 + stage * (C::kTileBytes >> 4);
                    if (elected) {
#pragma unroll
                        for (int kk = 0; kk < kKeyTile / 16; ++kk)
                            mma_ss(t_ow, smem_desc_join(p_lo + (((kk / 4) * C::kAtomBytes + (kk % 4) * 32) >> 4), hi),
                                   smem_desc_join(v_lo + ((kk * 2048) >> 4), hi), idesc_pv, (!first || kk > 0) ? 1u : 0u);
                    }
                    __syncwarp();
                };
                auto commit = [&](int bar_id) { if (elected) tc_commit(bar(bar_id)); };
                auto arrive = [&](int bar_id) { if (elected) mbar_arrive(bar(bar_id)); };
                // tile n of the producer's sequence K_0, K_1, V_0, K_2, V_1, ... sits in stage n % kStages
                auto kv_wait = [&](uint32_t n) -> bool { return wait(kKvFull + n % C::kStages, n / C::kStages, (int)n); };
                uint32_t n0 = 0;                // producer index of the column's first tile
                uint32_t sc = 0;                // steps this lane has been through
                uint32_t oc = 0;                // columns this lane took part in so far
                uint32_t seg = 0;
                Segment s;
                for (WorkIter it(p, cta); it.next(s); ++seg) {
                    const int n_steps = s.kt1 - s.kt0;
                    if (w >= s.n_sub) {
                        // not this lane's column: pass every stage on once its tile has landed, and
                        // the Q buffers once the previous column's release is complete
                        for (int t = 0; t < 2 * n_steps; ++t) {
                            if (!kv_wait(n0 + t)) return;
                            arrive(kKvEmpty + (n0 + t) % C::kStages);
                        }
                        n0 += 2 * n_steps;
                        if (seg > 0 && !wait(kQEmpty, seg - 1, (int)seg)) return;
                        arrive(kQEmpty);
                        continue;
                    }
                    if (!wait(kQFull + w, oc, 0)) return;
                    // QK of the column's first step: its S buffer was read out by the last softmax
                    if (!kv_wait(n0)) return;
                    if (sc > 0 && !wait(kSEmpty + w, sc - 1, (int)sc)) return;
                    tc_fence_after_sync();
                    issue_qk(n0 % C::kStages);
                    commit(kSFull + w);
                    commit(kKvEmpty + n0 % C::kStages);
                    if (n_steps == 1) commit(kQEmpty);
                    for (int j = 0; j < n_steps; ++j, ++sc) {
                        const bool more = j + 1 < n_steps;
                        const uint32_t nk = n0 + 2 * j + 1;                     // K_j+1 (if any)
                        const uint32_t nv = more ? nk + 1 : nk;                 // V_j
                        // QK of the next step as soon as the softmax warps hold S_j in registers
                        if (more) {
                            if (!kv_wait(nk)) return;
                            if (!wait(kSEmpty + w, sc, (int)sc)) return;
                            tc_fence_after_sync();
                            issue_qk(nk % C::kStages);
                            commit(kSFull + w);
                            commit(kKvEmpty + nk % C::kStages);
                            if (j + 2 == n_steps) commit(kQEmpty);               // the column's last QK is in the pipe
                        }
                        if (!kv_wait(nv)) return;
                        // the previous column's O rows must have been read out
                        if (j == 0 && oc > 0 && !wait(kOEmpty + w, oc - 1, (int)oc)) return;
                        if (!wait(kPFull + w, sc, (int)sc)) return;
                        tc_fence_after_sync();
                        issue_pv(nv % C::kStages, j == 0);
                        commit(kPEmpty + w);
                        commit(kKvEmpty + nv % C::kStages);
                        if (!more) commit(kOFull + w);
                    }
                    n0 += 2 * n_steps;
                    ++oc;
                }
            }();
        }
    } else {
        // ============================= softmax warps =============================
        setmaxnreg_inc<kSoftmaxRegs>();
        if (!skip) [&]() {
            const int q = warp & 3;                        // TMEM lane quarter this warp may touch
            const int w = warp >> 3;                       // lane (query tile) of the column
            const int h = (warp >> 2) & 1;                 // which 16 rows of the quarter
            const uint32_t lane_off = (uint32_t)(32 * q + 16 * h) << 16;
            const uint32_t t_s = tmem + lane_off + C::kColS + 128 * w;
            const uint32_t t_o = tmem + lane_off + C::kColO + D * w;
            const int row_a = 32 * q + 16 * h + (lane >> 2);   // row of registers 4k+{0,1}; 4k+{2,3} are row_a + 8
            const int cq = 2 * (lane & 3);                     // first of this thread's two columns in each group of 8
            const int slab = w * 8 + q * 2 + h;
            // P goes to shared memory with stmatrix: of the warp's 16 rows x 64 keys, one call
            // stores four 8-row x 8-key blocks (a block row = one 16-byte chunk); lane 8m + r gives the
            // address of row r of the block holding chunk m, which sits at chunk position m ^ r.
            // Chunks 4..7 are at the same address ^ 64, the second eight rows 1024 bytes on.
            const uint32_t p_at = p_smem + w * C::kPBytes + (uint32_t)(32 * q + 16 * h + (lane & 7)) * 128 +
                                  ((uint32_t)((lane >> 3) ^ (lane & 7)) << 4);
            uint32_t sc = 0, oc = 0;
            Segment s;
            for (WorkIter it(p, cta); it.next(s);) {
                if (w >= s.n_sub) continue;
                const AttnGroup &G = p.g[s.g];
                KeyIter kit(&G, s.kt0);
                // log2(e)/sqrt(D), times the head's key scale when the cache holds 8-bit codes
                const float *k_scale = p.item[G.item].k_scale;
                const float c = k_scale ? p.scale_log2 * __ldg(k_scale + s.head) : p.scale_log2;
                // ... and times the query row's own factor when the caller brings one (a q/k norm whose
                // per-token factor was left out of the stored q)
                float c_a = c, c_b = c;
                if (const float *q_scale = p.item[G.item].q_scale) {
                    const int r = 128 * w + row_a;
                    if (r < s.rows_valid) c_a *= __ldg(q_scale + s.q0 + r);
                    if (r + 8 < s.rows_valid) c_b *= __ldg(q_scale + s.q0 + r + 8);
                }
                float m_a = -INFINITY, m_b = -INFINITY;
                uint64_t acc_a = 0ull, acc_b = 0ull;       // two partial sums per row
                for (int j = s.kt0; j < s.kt1; ++j, kit.next(), ++sc) {
                    if (!__all_sync(0xffffffffu, wait(kSFull + w, sc, j))) return;
                    tc_fence_after_sync();
                    const int nvalid = kit.valid();
                    // The tile is taken in two 64-key pieces.  A piece's exponentials are computed
                    // against the rows' current reference maxima straight away; its sums then tell
                    // whether that was safe (no weight can exceed the sum).  Only when some sum in
                    // the warp is large or not finite - always on a column's first piece, where the
                    // references are -inf - are the exact row maxima taken, the references moved,
                    // what has been accumulated rescaled, and the piece redone.
#pragma unroll
                    for (int piece = 0; piece < 2; ++piece) {
                        uint32_t v[32];
                        uint32_t pp[16];                           // the piece's P: 16 rows x 64 keys per warp
                        tmem_ld_16x256b_x8(t_s + 64 * piece, v);
                        tmem_wait_ld();
                        if (piece == 1) {
                            // the whole tile is in registers now: the S buffer may take the next QK
                            tc_fence_before_sync();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(bar(kSEmpty + w));
                        }
                        if (nvalid < kKeyTile) mask_piece(v, 64 * piece, cq, nvalid);
                        uint64_t ts_a = 0ull, ts_b = 0ull;         // the piece's sums, two partials per row
                        {
                            const uint64_t na2 = pack2(-m_a, -m_a), nb2 = pack2(-m_b, -m_b);
                            const uint64_t c2a = pack2(c_a, c_a), c2b = pack2(c_b, c_b);
                            const PolyRow ra{c_a * (1.f / 128.f), ((float)kPolyLow - m_a) * (1.f / 128.f)};
                            const PolyRow rb{c_b * (1.f / 128.f), ((float)kPolyLow - m_b) * (1.f / 128.f)};
                            // Four 8-key groups at a time, stage by stage, so that the exponentials of a
                            // batch are all in flight before the first result is needed.
#pragma unroll
                            for (int g = 0; g < 2; ++g) {
                                uint64_t xa[4], xb[4];
#pragma unroll
                                for (int kk = 0; kk < 4; ++kk) {
                                    const int k = 4 * g + kk;
                                    if (!((kPolyMask<D> >> (8 * piece + k)) & 1u)) {
                                        xa[kk] = fma2(pack2(as_f(v[4 * k]), as_f(v[4 * k + 1])), c2a, na2);
                                        xb[kk] = fma2(pack2(as_f(v[4 * k + 2]), as_f(v[4 * k + 3])), c2b, nb2);
                                    }
                                }
#pragma unroll
                                for (int kk = 0; kk < 4; ++kk) {
                                    const int k = 4 * g + kk;
                                    if ((kPolyMask<D> >> (8 * piece + k)) & 1u) {
                                        xa[kk] = exp2_poly2(as_f(v[4 * k]), as_f(v[4 * k + 1]), ra);
                                        xb[kk] = exp2_poly2(as_f(v[4 * k + 2]), as_f(v[4 * k + 3]), rb);
                                    } else {
                                        xa[kk] = exp2_sfu2(xa[kk]);
                                        xb[kk] = exp2_sfu2(xb[kk]);
                                    }
                                }
#pragma unroll
                                for (int kk = 0; kk < 4; ++kk) {
                                    const int k = 4 * g + kk;
                                    ts_a = add2(ts_a, xa[kk]);
                                    ts_b = add2(ts_b, xb[kk]);
                                    float a0, a1, b0, b1;
                                    unpack2(xa[kk], a0, a1);
                                    unpack2(xb[kk], b0, b1);
                                    pp[2 * k] = cvt_bf16x2(a0, a1);        // key 8k + cq in the low half
                                    pp[2 * k + 1] = cvt_bf16x2(b0, b1);
                                }
                            }
                        }
                        float sa, sb;
                        {
                            float x0, x1;
                            unpack2(ts_a, x0, x1);
                            sa = x0 + x1;
                            unpack2(ts_b, x0, x1);
                            sb = x0 + x1;
                        }
                        if (__any_sync(0xffffffffu, !(sa < kSafeSum) || !(sb < kSafeSum))) {
                            // exact maxima of the piece's rows: 16 columns per thread, then across the quad
                            float ta = fmaxf(as_f(v[0]), as_f(v[1])), tb = fmaxf(as_f(v[2]), as_f(v[3]));
#pragma unroll
                            for (int k = 1; k < 8; ++k) {
                                ta = max3(ta, as_f(v[4 * k]), as_f(v[4 * k + 1]));
                                tb = max3(tb, as_f(v[4 * k + 2]), as_f(v[4 * k + 3]));
                            }
                            ta = fmaxf(ta, __shfl_xor_sync(0xffffffffu, ta, 1));
                            tb = fmaxf(tb, __shfl_xor_sync(0xffffffffu, tb, 1));
                            ta = fmaxf(ta, __shfl_xor_sync(0xffffffffu, ta, 2)) * c_a;
                            tb = fmaxf(tb, __shfl_xor_sync(0xffffffffu, tb, 2)) * c_b;
                            const bool fresh = j == s.kt0 && piece == 0;     // nothing accumulated yet
                            const float new_a = fresh ? ta : fmaxf(m_a, ta), new_b = fresh ? tb : fmaxf(m_b, tb);
                            const float al_a = fresh ? 0.f : ex2(m_a - new_a), al_b = fresh ? 0.f : ex2(m_b - new_b);
                            m_a = new_a;
                            m_b = new_b;
                            acc_a = fma2(acc_a, pack2(al_a, al_a), 0ull);
                            acc_b = fma2(acc_b, pack2(al_b, al_b), 0ull);
                            if (piece == 1) {
                                // the first piece's P already sits in shared memory, against the old
                                // references: take it back, rescale, store again (nobody else reads it
                                // before this step's hand-over)
                                __syncwarp();
#pragma unroll
                                for (int half = 0; half < 2; ++half) {
                                    const uint32_t at = half ? (p_at ^ 64u) : p_at;
                                    uint32_t ra0, ra1, ra2, ra3, rb0, rb1, rb2, rb3;
                                    ldmatrix_x4(at, ra0, ra1, ra2, ra3);
                                    ldmatrix_x4(at + 8 * 128, rb0, rb1, rb2, rb3);
                                    auto scale = [](uint32_t x, float al) {
                                        return cvt_bf16x2(as_f(x << 16) * al, as_f(x & 0xffff0000u) * al);
                                    };
                                    __syncwarp();
                                    stmatrix_x4(at, scale(ra0, al_a), scale(ra1, al_a), scale(ra2, al_a), scale(ra3, al_a));
                                    stmatrix_x4(at + 8 * 128, scale(rb0, al_b), scale(rb1, al_b), scale(rb2, al_b), scale(rb3, al_b));
                                }
                            }
                            if (j != s.kt0) {
                                // The O rows hold every earlier tile of the column: once the last PV issued
                                // (the previous step's) has completed they can be rescaled; this step's PV
                                // waits for this step's P.
                                if (!__all_sync(0xffffffffu, wait(kPEmpty + w, sc - 1, (int)sc))) return;
                                tc_fence_after_sync();
#pragma unroll 1
                                for (int ch = 0; ch < C::kOChunks; ++ch) {
                                    uint32_t o[32];
                                    tmem_ld_16x256b_x8(t_o + 64 * ch, o);
                                    tmem_wait_ld();
#pragma unroll
                                    for (int k = 0; k < 8; ++k) {
                                        o[4 * k] = as_u(as_f(o[4 * k]) * al_a);
                                        o[4 * k + 1] = as_u(as_f(o[4 * k + 1]) * al_a);
                                        o[4 * k + 2] = as_u(as_f(o[4 * k + 2]) * al_b);
                                        o[4 * k + 3] = as_u(as_f(o[4 * k + 3]) * al_b);
                                    }
                                    tmem_st_16x256b_x8(t_o + 64 * ch, o);
                                }
                                tmem_wait_st();
                                tc_fence_before_sync();
                            }
                            // the piece again, against the new references
                            const uint64_t na2 = pack2(-m_a, -m_a), nb2 = pack2(-m_b, -m_b);
                            const uint64_t c2a = pack2(c_a, c_a), c2b = pack2(c_b, c_b);
                            ts_a = ts_b = 0ull;
#pragma unroll
                            for (int k = 0; k < 8; ++k) {
                                const uint64_t pa = exp2_sfu2(fma2(pack2(as_f(v[4 * k]), as_f(v[4 * k + 1])), c2a, na2));
                                const uint64_t pb = exp2_sfu2(fma2(pack2(as_f(v[4 * k + 2]), as_f(v[4 * k + 3])), c2b, nb2));
                                ts_a = add2(ts_a, pa);
                                ts_b = add2(ts_b, pb);
                                float a0, a1, b0, b1;
                                unpack2(pa, a0, a1);
                                unpack2(pb, b0, b1);
                                pp[2 * k] = cvt_bf16x2(a0, a1);
                                pp[2 * k + 1] = cvt_bf16x2(b0, b1);
                            }
                        }
                        acc_a = add2(acc_a, ts_a);
                        acc_b = add2(acc_b, ts_b);
                        // The piece's P (bf16) goes into the lane's shared-memory tile straight away (the
                        // first piece's once the PV that read the previous step's P has completed), so
                        // its registers are free while the second piece is computed.  The tile is the
                        // K-major, 128-byte-swizzled A operand of PV: one 64-key atom per piece, row r at
                        // r * 128 bytes, its 16-byte chunk k (8 keys) at chunk position k ^ (r % 8).
                        if (piece == 0 && sc > 0 && !__all_sync(0xffffffffu, wait(kPEmpty + w, sc - 1, (int)sc))) return;
                        {
                            const uint32_t at = p_at + piece * C::kAtomBytes;
                            stmatrix_x4(at, pp[0], pp[2], pp[4], pp[6]);                       // rows a, chunks 0..3
                            stmatrix_x4(at ^ 64u, pp[8], pp[10], pp[12], pp[14]);               // rows a, chunks 4..7
                            stmatrix_x4(at + 8 * 128, pp[1], pp[3], pp[5], pp[7]);              // rows a + 8
                            stmatrix_x4((at ^ 64u) + 8 * 128, pp[9], pp[11], pp[13], pp[15]);
                        }
                    }
                    fence_proxy_async_smem();                      // the stores above are read by the tensor pipe
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(kPFull + w));
                }

                // ---- the column's (or this part's) O rows are complete ----
                if (!__all_sync(0xffffffffu, wait(kOFull + w, oc, s.kt1))) return;
                tc_fence_after_sync();
                float l_a, l_b;
                {
                    float x0, x1;
                    unpack2(acc_a, x0, x1);
                    l_a = x0 + x1;
                    unpack2(acc_b, x0, x1);
                    l_b = x0 + x1;
                    l_a += __shfl_xor_sync(0xffffffffu, l_a, 1);
                    l_b += __shfl_xor_sync(0xffffffffu, l_b, 1);
                    l_a += __shfl_xor_sync(0xffffffffu, l_a, 2);
                    l_b += __shfl_xor_sync(0xffffffffu, l_b, 2);
                }
                const int row = 128 * w + row_a;               // row inside the column
                const bool live_a = row < s.rows_valid, live_b = row + 8 < s.rows_valid;
                const AttnItem &item = p.item[G.item];
                ll_bf16 *dst_a = item.out + ((size_t)(s.q0 + row) * p.heads + s.head) * D;
                ll_bf16 *dst_b = dst_a + (size_t)8 * p.heads * D;
                float *lse_a = item.lse ? item.lse + (size_t)s.head * item.nq_total + s.q0 + row : nullptr;

                bool finish = true;            // this warp writes the output rows
                int i0 = 0, n_parts = 1;
                const bool whole = s.kt0 == 0 && s.kt1 == G.n_kt;
                const size_t slot_floats = (size_t)kQTileRows * (D + 2);
                if (!whole) {
                    // leave this part in its slot and count the arrival
                    // (the parts of a column sit in consecutive shares; i0 = the share with its first step)
                    const int own = p.share_of_cta[cta];
                    int i1 = own;
                    i0 = own;
                    while (p.share_begin[i0] > s.col_begin) --i0;
                    while (p.share_begin[i1 + 1] < s.col_begin + G.n_kt) ++i1;
                    n_parts = i1 - i0 + 1;
                    float *slot = p.partial + (size_t)(2 * own + (s.kt0 == 0 ? 1 : 0)) * slot_floats;
#pragma unroll 1
                    for (int ch = 0; ch < C::kOChunks; ++ch) {
                        uint32_t o[32];
                        tmem_ld_16x256b_x8(t_o + 64 * ch, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            float2 *dst = reinterpret_cast<float2 *>(slot) +
                                          ((size_t)(slab * (D / 8) + 8 * ch + k) * 2) * 32 + lane;
                            dst[0] = make_float2(as_f(o[4 * k]), as_f(o[4 * k + 1]));
                            dst[32] = make_float2(as_f(o[4 * k + 2]), as_f(o[4 * k + 3]));
                        }
                    }
                    if ((lane & 3) == 0) {
                        float2 *ml = reinterpret_cast<float2 *>(slot + (size_t)kQTileRows * D) + slab * 16 + (lane >> 2);
                        ml[0] = make_float2(m_a, l_a);
                        ml[8] = make_float2(m_b, l_b);
                    }
                    __threadfence();
                    __syncwarp();
                    uint32_t arrived = 0;
                    if (lane == 0) arrived = atomicAdd(p.counters + i0 * kSlabs + slab, 1u);
                    arrived = __shfl_sync(0xffffffffu, arrived, 0);
                    finish = arrived == (uint32_t)(n_parts - 1);
                    if (finish) {
                        if (lane == 0) p.counters[i0 * kSlabs + slab] = 0;    // ready for the next launch
                        __threadfence();
                    }
                }
                if (finish) {
                    // the slot of part i, and this thread's two (max, sum) pairs in it
                    auto part_slot = [&](int i) -> const float * {
                        return p.partial + (size_t)(2 * i + (i == i0 ? 1 : 0)) * slot_floats;
                    };
                    auto part_ml = [&](const float *slot) -> const float2 * {
                        return reinterpret_cast<const float2 *>(slot + (size_t)kQTileRows * D) + slab * 16 + (lane >> 2);
                    };
                    // Reference maximum and sum over all parts.  A split column is merged from the
                    // slots alone, the own part included, in the order of the parts, so the result
                    // does not depend on which part happened to arrive last.
                    float mm_a = m_a, mm_b = m_b, ll_a = l_a, ll_b = l_b;
                    if (!whole) {
                        for (int i = i0; i < i0 + n_parts; ++i) {
                            const float2 *ml = part_ml(part_slot(i));
                            mm_a = fmaxf(mm_a, __ldcg(ml).x);
                            mm_b = fmaxf(mm_b, __ldcg(ml + 8).x);
                        }
                        ll_a = ll_b = 0.f;
                        for (int i = i0; i < i0 + n_parts; ++i) {
                            const float2 *ml = part_ml(part_slot(i));
                            const float2 pa = __ldcg(ml), pb = __ldcg(ml + 8);
                            ll_a = fmaf(pa.y, ex2(pa.x - mm_a), ll_a);
                            ll_b = fmaf(pb.y, ex2(pb.x - mm_b), ll_b);
                        }
                    }
                    const float v_scale = item.v_scale ? __ldg(item.v_scale + s.head) : 1.f;   // 8-bit caches: value codes x scale
                    const float inv_a = v_scale / ll_a, inv_b = v_scale / ll_b;
#pragma unroll 1
                    for (int ch = 0; ch < C::kOChunks; ++ch) {
                        uint32_t o[32];
                        if (whole) {
                            tmem_ld_16x256b_x8(t_o + 64 * ch, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int k = 0; k < 8; ++k) {
                                o[4 * k] = as_u(as_f(o[4 * k]) * inv_a);
                                o[4 * k + 1] = as_u(as_f(o[4 * k + 1]) * inv_a);
                                o[4 * k + 2] = as_u(as_f(o[4 * k + 2]) * inv_b);
                                o[4 * k + 3] = as_u(as_f(o[4 * k + 3]) * inv_b);
                            }
                        } else {
#pragma unroll
                            for (int k = 0; k < 32; ++k) o[k] = 0u;
                            for (int i = i0; i < i0 + n_parts; ++i) {
                                const float *slot = part_slot(i);
                                const float2 *ml = part_ml(slot);
                                const float wa = ex2(__ldcg(ml).x - mm_a) * inv_a, wb = ex2(__ldcg(ml + 8).x - mm_b) * inv_b;
#pragma unroll
                                for (int k = 0; k < 8; ++k) {
                                    const float2 *src = reinterpret_cast<const float2 *>(slot) +
                                                        ((size_t)(slab * (D / 8) + 8 * ch + k) * 2) * 32 + lane;
                                    const float2 xa = __ldcg(src), xb = __ldcg(src + 32);
                                    o[4 * k] = as_u(fmaf(xa.x, wa, as_f(o[4 * k])));
                                    o[4 * k + 1] = as_u(fmaf(xa.y, wa, as_f(o[4 * k + 1])));
                                    o[4 * k + 2] = as_u(fmaf(xb.x, wb, as_f(o[4 * k + 2])));
                                    o[4 * k + 3] = as_u(fmaf(xb.y, wb, as_f(o[4 * k + 3])));
                                }
                            }
                        }
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            const int col = 64 * ch + 8 * k + cq;
                            if (live_a)
                                *reinterpret_cast<uint32_t *>(dst_a + col) = cvt_bf16x2(as_f(o[4 * k]), as_f(o[4 * k + 1]));
                            if (live_b)
                                *reinterpret_cast<uint32_t *>(dst_b + col) = cvt_bf16x2(as_f(o[4 * k + 2]), as_f(o[4 * k + 3]));
                        }
                    }
                    if (lse_a && (lane & 3) == 0) {
                        if (live_a) lse_a[0] = (mm_a + log2f(ll_a)) * 0.6931471805599453f;
                        if (live_b) lse_a[8] = (mm_b + log2f(ll_b)) * 0.6931471805599453f;
                    }
                }
                // the O columns may be overwritten by the next column's first PV
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kOEmpty + w));
                ++oc;
            }
        }();
    }

    // ---- common exit -------------------------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag == 1) {
        // give copies and MMAs that may still be in flight time to land before the
        // shared and tensor memory go back to the SM
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == kTmaWarp) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(tmem, C::kTmemCols);
    }
}

// The bounded-wait machinery on its own: one warp waits on a barrier that nobody will ever
// complete, gives up after limit_ns, leaves the record and returns normally.
__global__ void wait_probe_kernel(uint32_t *status, unsigned long long limit_ns)
{
    __shared__ uint64_t never;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&never), 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();
    WaitCtx ctx{&abort_flag, status, (int)(threadIdx.x >> 5)};
    wait_bar(smem_u32(&never), 0, ctx, kProbeBarrierId, kProbeIteration, limit_ns);
}

}  // namespace

cudaError_t launch_wait_probe(uint32_t *status, uint64_t limit_ns, cudaStream_t stream)
{
    wait_probe_kernel<<<1, 32, 0, stream>>>(status, (unsigned long long)limit_ns);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_attn_sm100(const AttnParams &p, int head_dim, const AttnMaps &maps, cudaStream_t stream)
{
    if (p.n_ctas <= 0) return cudaSuccess;
    dim3 grid((unsigned)p.n_ctas);
    cudaError_t e;
    // Once per device and head size: the in-kernel register reallocation assumes the launch
    // allocation it was sized for, and the kernel needs its dynamic shared memory opted in.
    constexpr int kMaxDevices = 64;
    static std::atomic<unsigned char> prepared[kMaxDevices][2];
    int dev = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const int which = head_dim == 128 ? 1 : 0;
    if (dev < 0 || dev >= kMaxDevices || !prepared[dev][which].load(std::memory_order_acquire)) {
        cudaFuncAttributes fa;
        e = which ? cudaFuncGetAttributes(&fa, attn_sm100_kernel<128>) : cudaFuncGetAttributes(&fa, attn_sm100_kernel<64>);
        if (e != cudaSuccess) return e;
        if (fa.numRegs != kLaunchRegs) return cudaErrorLaunchOutOfResources;
        e = which ? cudaFuncSetAttribute(attn_sm100_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<128>::kSmemBytes)
                  : cudaFuncSetAttribute(attn_sm100_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<64>::kSmemBytes);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < kMaxDevices) prepared[dev][which].store(1, std::memory_order_release);
    }
    if (which) attn_sm100_kernel<128><<<grid, kThreads, Cfg<128>::kSmemBytes, stream>>>(p, maps);
    else       attn_sm100_kernel<64><<<grid, kThreads, Cfg<64>::kSmemBytes, stream>>>(p, maps);
    count_launch();
    return cudaGetLastError();
}

}  // namespace ll
