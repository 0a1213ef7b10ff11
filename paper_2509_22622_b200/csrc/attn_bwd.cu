// Backward of the clip step on tcgen05 tensor cores (sm_100a): gradients of a loss with respect to
// the clip's q, k, v given the gradient of the attention output.
//
// With s_ij = q_i.k_j / sqrt(D) over the keys visible to row i, p_ij = exp(s_ij - lse_i):
//   delta_i = d_out_i . out_i                                  (delta kernel)
//   dP_ij = d_out_i . v_j,   dS_ij = p_ij (dP_ij - delta_i)
//   dq_i = sum_j dS_ij k_j / sqrt(D)                            (dq kernel, one CTA per query tile)
//   dk_j = sum_i dS_ij q_i / sqrt(D),  dv_j = sum_i p_ij d_out_i   (dkdv kernel, one CTA per key tile)
// q, k are the rotated tensors; dq and dk are turned back through the rotation before they are
// stored.  Only the clip's own keys get dk, dv (the sink and the context are detached).
//
// Two kernels instead of one with atomics: every gradient element is accumulated by one CTA in one
// order, so the result is run-to-run deterministic, at the price of forming S and dP twice.  Both
// kernels are plain: one warp loads (TMA) and issues the MMAs, four warps (one thread per tile row,
// the 32x32b TMEM shape) turn S and dP into P and dS in shared memory; a tile pair's steps run one
// after the other, with only the next operand load in flight.
#include <cuda_bf16.h>

#include "bounded_wait.cuh"
#include "ll_internal.h"
#include "ptx.cuh"

namespace ll {

namespace {

using namespace ptx;

constexpr int kBwdThreads = 160;                       // four compute warps, one load/issue warp
constexpr int kTile = 128;

__device__ __forceinline__ float as_f(uint32_t u) { return __uint_as_float(u); }

__device__ __forceinline__ void tmem_ld_32x32b_x32(uint32_t taddr, uint32_t *r)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr)
                 : "memory");
}

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// Meeting point of the four compute warps (hardware barrier 1; 0 is __syncthreads).
__device__ __forceinline__ void compute_sync() { asm volatile("barrier.sync 1, 128;" ::: "memory"); }

// delta[h][i] = sum_d d_out[i][h][d] * out[i][h][d]: one warp per (row, head).
template <int D>
__global__ void __launch_bounds__(256) bwd_delta_kernel(const __grid_constant__ BwdParams p)
{
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= (long long)p.nq_total * p.heads) return;
    const long long row = warp / p.heads;
    const int head = (int)(warp % p.heads);
    const size_t off = ((size_t)row * p.heads + head) * D;
    float s = 0.f;
    for (int d = 2 * lane; d < D; d += 64) {
        const uint32_t a = *reinterpret_cast<const uint32_t *>(p.out + off + d);
        const uint32_t b = *reinterpret_cast<const uint32_t *>(p.d_out + off + d);
        s = fmaf(as_f(a << 16), as_f(b << 16), s);
        s = fmaf(as_f(a & 0xffff0000u), as_f(b & 0xffff0000u), s);
    }
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) s += __shfl_xor_sync(0xffffffffu, s, m);
    if (lane == 0) p.delta[(size_t)head * p.nq_total + row] = s;
}

// One row of a 128 x 128 score tile and of the matching dP tile (TMEM, fp32) to P and/or dS
// (bf16) in 128-byte-swizzled shared-memory tiles laid out [row][key]: two 64-key atoms of
// 128 rows x 128 bytes, row r's 16-byte chunk k at chunk position k ^ (r % 8).
//   p = 2^(s * c - lse2), ds = p * (dp - delta); columns whose bit in `valid` is clear, and rows
//   that are not live, give zeros.
__device__ __forceinline__ void row_to_p_ds(uint32_t t_s, uint32_t t_dp, int row, bool live, float c, float lse2,
                                            float delta, const uint32_t (&valid)[4], uint32_t p_tile, uint32_t ds_tile)
{
#pragma unroll 1
    for (int ch = 0; ch < 4; ++ch) {
        uint32_t s[32], dp[32];
        tmem_ld_32x32b_x32(t_s + 32 * ch, s);
        tmem_ld_32x32b_x32(t_dp + 32 * ch, dp);
        tmem_wait_ld();
        uint32_t pw[16], dw[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            float p0 = ex2(fmaf(as_f(s[2 * i]), c, -lse2)), p1 = ex2(fmaf(as_f(s[2 * i + 1]), c, -lse2));
            if (!live || !((valid[ch] >> (2 * i)) & 1u)) p0 = 0.f;
            if (!live || !((valid[ch] >> (2 * i + 1)) & 1u)) p1 = 0.f;
            pw[i] = cvt_bf16x2(p0, p1);
            dw[i] = cvt_bf16x2(p0 * (as_f(dp[2 * i]) - delta), p1 * (as_f(dp[2 * i + 1]) - delta));
        }
        // 32 keys = four 16-byte chunks of this row, in atom ch / 2
        const uint32_t row_off = (uint32_t)(ch >> 1) * (128 * 128) + (uint32_t)row * 128;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t chunk = (uint32_t)(((ch & 1) * 4 + k) ^ (row & 7)) << 4;
            if (p_tile) st_shared_v4(p_tile + row_off + chunk, pw[4 * k], pw[4 * k + 1], pw[4 * k + 2], pw[4 * k + 3]);
            st_shared_v4(ds_tile + row_off + chunk, dw[4 * k], dw[4 * k + 1], dw[4 * k + 2], dw[4 * k + 3]);
        }
    }
}

// 128 rows x D fp32 in TMEM (row = thread), times `mul`, optionally turned back through the
// rotation of the row's grid position, rounded to bf16 and stored at dst (one head row of D).
template <int D, bool kRotateBack>
__device__ __forceinline__ void store_grad_row(uint32_t taddr, float mul, ll_bf16 *dst, const BwdParams &p, int frame,
                                               int y, int x, bool live)
{
    constexpr int kNh = D / 6, kNt = D / 2 - 2 * kNh;
    const float2 *t_row = p.t_tab + (size_t)frame * kNt, *h_row = p.h_tab + (size_t)y * kNh, *w_row = p.w_tab + (size_t)x * kNh;
#pragma unroll
    for (int ch = 0; ch < D / 32; ++ch) {
        uint32_t r[32];
        tmem_ld_32x32b_x32(taddr + 32 * ch, r);
        tmem_wait_ld();
        uint32_t o[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            float a = as_f(r[2 * i]) * mul, b = as_f(r[2 * i + 1]) * mul;
            if (kRotateBack) {
                const int j = 16 * ch + i;
                const float2 cs = j < kNt ? __ldg(t_row + j) : j < kNt + kNh ? __ldg(h_row + (j - kNt)) : __ldg(w_row + (j - kNt - kNh));
                const float a2 = fmaf(a, cs.x, b * cs.y), b2 = fmaf(b, cs.x, -(a * cs.y));
                a = a2;
                b = b2;
            }
            o[i] = cvt_bf16x2(a, b);
        }
        if (live) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
                reinterpret_cast<uint4 *>(dst + 32 * ch)[i] = make_uint4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
        }
    }
}

// Walks the 128-row key tiles of a group's visible runs.
struct RunTiles {
    const AttnGroup *g;
    int r, off;
    __device__ RunTiles(const AttnGroup *grp) : g(grp), r(0), off(0) {}
    __device__ int row() const { return g->k_start[r] + off; }
    __device__ int valid() const { return min(kTile, g->k_len[r] - off); }
    __device__ void next()
    {
        off += kTile;
        if (off >= g->k_len[r]) { ++r; off = 0; }
    }
};


template <int D>
struct BwdCfg {
    static constexpr int kAtomBytes = 128 * 128;
    static constexpr int kTileBytes = (D / 64) * kAtomBytes;     // 128 rows x D bf16
    static constexpr int kPBytes = 2 * kAtomBytes;               // 128 rows x 128 keys bf16
};

// MMA helpers: all tiles are 128-byte-swizzled, 128 rows, tile base 1024-byte aligned.
// K-major operand [rows][64-element atoms]: slice kk (16 elements) of the contraction.
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t tile, int kk)
{
    constexpr uint32_t hi = smem_desc_hi_sw128(1024);
    return smem_desc_join(smem_desc_lo(tile, 16) + (uint32_t)(((kk / 4) * (128 * 128) + (kk % 4) * 32) >> 4), hi);
}
// MN-major operand: the tile's rows are the contraction index, its columns the M (or N) index;
// slice kk = rows 16 kk .. 16 kk + 15.
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t tile, int kk)
{
    constexpr uint32_t hi = smem_desc_hi_sw128(1024);
    return smem_desc_join(smem_desc_lo(tile, 128 * 128) + (uint32_t)((kk * 2048) >> 4), hi);
}

__device__ __forceinline__ void key_mask(int nvalid, uint32_t (&valid)[4])
{
#pragma unroll
    for (int ch = 0; ch < 4; ++ch)
        valid[ch] = nvalid >= 32 * (ch + 1) ? 0xffffffffu : nvalid > 32 * ch ? ((1u << (nvalid - 32 * ch)) - 1u) : 0u;
}

// ---- dq: one CTA per (128-row query tile, head) ---------------------------------------------
template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1)
bwd_dq_kernel(const __grid_constant__ BwdParams p, const __grid_constant__ BwdMaps maps)
{
    using C = BwdCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t q_s = base, do_s = q_s + C::kTileBytes, k_s = do_s + C::kTileBytes, v_s = k_s + 2 * C::kTileBytes,
                   ds_s = v_s + 2 * C::kTileBytes, bars = ds_s + C::kPBytes;
    enum { kQFull = 0, kKvFull = 1, kKvEmpty = 3, kSFull = 5, kDsFull = 6, kDone = 7, kBars = 8 };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(gen + (bars - base) + kBars * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    auto bar = [&](int i) -> uint32_t { return bars + 8u * (uint32_t)i; };
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const int head = blockIdx.y;
    // which group and tile of it
    int g = 0, tile = blockIdx.x;
    while (tile >= (p.g[g].q_rows + kTile - 1) / kTile) { tile -= (p.g[g].q_rows + kTile - 1) / kTile; ++g; }
    const AttnGroup &G = p.g[g];
    const int q0 = G.q_begin + tile * kTile, rows = min(kTile, G.q_rows - tile * kTile);
    const int n_kt = G.n_kt;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kBars; ++i) mbar_init(bar(i), 1);
        *abort_flag = (*reinterpret_cast<volatile uint32_t *>(p.status) != kStatusOk) ? 2 : 0;
        fence_mbar_init();
    }
    if (warp == 4) { tmem_alloc(smem_u32(tmem_slot), 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    WaitCtx ctx{abort_flag, p.status, warp};
    auto wait = [&](int bar_id, uint32_t parity, int iter) -> bool { return wait_bar(bar(bar_id), parity & 1u, ctx, bar_id, iter); };
    const bool skip = *abort_flag != 0;
    const uint32_t t_s = tmem, t_dp = tmem + 128, t_dq = tmem + 256;

    if (skip) {
    } else if (warp == 4) {
        if (lane == 0) [&]() {
            constexpr uint32_t idesc_s = idesc_bf16_f32(128, 128, 0, 0), idesc_dq = idesc_bf16_f32(128, D, 0, 1);
            auto load_kv = [&](int j, int row) {
                const int b = j & 1;
                mbar_arrive_expect_tx(bar(kKvFull + b), 2 * C::kTileBytes);
                for (int a = 0; a < D / 64; ++a) {
                    tma_load_3d(k_s + b * C::kTileBytes + a * C::kAtomBytes, &maps.k, bar(kKvFull + b), a * 64, row, head);
                    tma_load_3d(v_s + b * C::kTileBytes + a * C::kAtomBytes, &maps.v, bar(kKvFull + b), a * 64, row, head);
                }
            };
            mbar_arrive_expect_tx(bar(kQFull), 2 * C::kTileBytes);
            for (int a = 0; a < D / 64; ++a) {
                tma_load_3d(q_s + a * C::kAtomBytes, &maps.q, bar(kQFull), a * 64, head, q0);
                tma_load_3d(do_s + a * C::kAtomBytes, &maps.d_out, bar(kQFull), a * 64, head, q0);
            }
            RunTiles kt(&G);
            load_kv(0, kt.row());
            if (!wait(kQFull, 0, 0)) return;
            for (int j = 0; j < n_kt; ++j) {
                const int b = j & 1;
                if (j + 1 < n_kt) {
                    kt.next();
                    if (j + 1 >= 2 && !wait(kKvEmpty + ((j + 1) & 1), ((j + 1) >> 1) - 1, j)) return;
                    load_kv(j + 1, kt.row());
                }
                if (!wait(kKvFull + b, j >> 1, j)) return;
                tc_fence_after_sync();
                for (int kk = 0; kk < D / 16; ++kk)
                    mma_ss(t_s, desc_kmajor(q_s, kk), desc_kmajor(k_s + b * C::kTileBytes, kk), idesc_s, kk > 0);
                for (int kk = 0; kk < D / 16; ++kk)
                    mma_ss(t_dp, desc_kmajor(do_s, kk), desc_kmajor(v_s + b * C::kTileBytes, kk), idesc_s, kk > 0);
                tc_commit(bar(kSFull));
                if (!wait(kDsFull, j, j)) return;
                tc_fence_after_sync();
                for (int kk = 0; kk < kTile / 16; ++kk)
                    mma_ss(t_dq, desc_kmajor(ds_s, kk), desc_mnmajor(k_s + b * C::kTileBytes, kk), idesc_dq, (j > 0 || kk > 0) ? 1u : 0u);
                tc_commit(bar(kKvEmpty + b));
            }
            tc_commit(bar(kDone));
        }();
    } else {
        bool alive = true;
        auto wait_c = [&](int bar_id, uint32_t parity, int iter) {
            if (alive && !__all_sync(0xffffffffu, wait(bar_id, parity, iter))) alive = false;
        };
        const int row = threadIdx.x;                             // tile row = TMEM lane
        const bool live = row < rows;
        const uint32_t lane_off = (uint32_t)(32 * warp) << 16;
        const size_t stat = (size_t)head * p.nq_total + q0 + (live ? row : 0);
        const float lse2 = p.lse[stat] * 1.4426950408889634f, delta = p.delta[stat];
        RunTiles kt(&G);
        for (int j = 0; j < n_kt; ++j, kt.next()) {
            uint32_t valid[4];
            key_mask(kt.valid(), valid);
            wait_c(kSFull, j, j);
            tc_fence_after_sync();
            row_to_p_ds(t_s + lane_off, t_dp + lane_off, row, live, p.scale_log2, lse2, delta, valid, 0u, ds_s);
            fence_proxy_async_smem();
            tc_fence_before_sync();
            compute_sync();
            if (threadIdx.x == 0) mbar_arrive(bar(kDsFull));
        }
        wait_c(kDone, 0, n_kt);
        tc_fence_after_sync();
        const int token = q0 + (live ? row : 0);
        const int frame = token / p.P, cell = token % p.P;
        if (alive)
            store_grad_row<D, true>(t_dq + lane_off, p.scale, p.dq + ((size_t)token * p.heads + head) * D, p, frame,
                                    cell / p.grid_w, cell % p.grid_w, live);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag == 1) {
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 4) { __syncwarp(); tc_fence_after_sync(); tmem_dealloc(tmem, 512); }
}


// Which of the 128 cache rows starting at r0 a group can see (bit c of word c / 32 = row r0 + c).
__device__ __forceinline__ bool group_mask(const AttnGroup &G, int r0, uint32_t (&valid)[4])
{
    valid[0] = valid[1] = valid[2] = valid[3] = 0u;
    bool any = false;
    for (int r = 0; r < G.n_ranges; ++r) {
        const int lo = max(G.k_start[r], r0) - r0, hi = min(G.k_start[r] + G.k_len[r], r0 + kTile) - r0;
        for (int c = lo; c < hi; ++c) valid[c >> 5] |= 1u << (c & 31);
        any |= hi > lo;
    }
    return any;
}

// ---- dk, dv: one CTA per (128-row tile of the clip's cache rows, head) -----------------------
template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1)
bwd_dkdv_kernel(const __grid_constant__ BwdParams p, const __grid_constant__ BwdMaps maps)
{
    using C = BwdCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t k_s = base, v_s = k_s + C::kTileBytes, q_s = v_s + C::kTileBytes, do_s = q_s + C::kTileBytes,
                   p_s = do_s + C::kTileBytes, ds_s = p_s + C::kPBytes, bars = ds_s + C::kPBytes;
    enum { kKvFull = 0, kQdFull = 1, kSFull = 2, kPdsFull = 3, kStepDone = 4, kBars = 5 };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(gen + (bars - base) + kBars * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    auto bar = [&](int i) -> uint32_t { return bars + 8u * (uint32_t)i; };
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const int head = blockIdx.y;
    // the tile's first cache row and the end of the run it belongs to
    int run = 0, t = blockIdx.x;
    while (t >= (p.krun_len[run] + kTile - 1) / kTile) { t -= (p.krun_len[run] + kTile - 1) / kTile; ++run; }
    const int r0 = p.krun_start[run] + t * kTile, run_end = p.krun_start[run] + p.krun_len[run];

    if (threadIdx.x == 0) {
        for (int i = 0; i < kBars; ++i) mbar_init(bar(i), 1);
        *abort_flag = (*reinterpret_cast<volatile uint32_t *>(p.status) != kStatusOk) ? 2 : 0;
        fence_mbar_init();
    }
    if (warp == 4) { tmem_alloc(smem_u32(tmem_slot), 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    WaitCtx ctx{abort_flag, p.status, warp};
    auto wait = [&](int bar_id, uint32_t parity, int iter) -> bool { return wait_bar(bar(bar_id), parity & 1u, ctx, bar_id, iter); };
    const bool skip = *abort_flag != 0;
    const uint32_t t_s = tmem, t_dp = tmem + 128, t_dk = tmem + 256, t_dv = tmem + 256 + D;

    if (skip) {
    } else if (warp == 4) {
        if (lane == 0) [&]() {
            constexpr uint32_t idesc_s = idesc_bf16_f32(128, 128, 0, 0), idesc_g = idesc_bf16_f32(128, D, 1, 1);
            mbar_arrive_expect_tx(bar(kKvFull), 2 * C::kTileBytes);
            for (int a = 0; a < D / 64; ++a) {
                tma_load_3d(k_s + a * C::kAtomBytes, &maps.k, bar(kKvFull), a * 64, r0, head);
                tma_load_3d(v_s + a * C::kAtomBytes, &maps.v, bar(kKvFull), a * 64, r0, head);
            }
            if (!wait(kKvFull, 0, 0)) return;
            uint32_t step = 0;
            for (int g = 0; g < p.n_groups; ++g) {
                const AttnGroup &G = p.g[g];
                uint32_t valid[4];
                if (!group_mask(G, r0, valid)) continue;
                for (int i = 0; i * kTile < G.q_rows; ++i, ++step) {
                    // the previous step's products have read Q, dO, P and dS
                    if (step > 0 && !wait(kStepDone, step - 1, (int)step)) return;
                    mbar_arrive_expect_tx(bar(kQdFull), 2 * C::kTileBytes);
                    for (int a = 0; a < D / 64; ++a) {
                        tma_load_3d(q_s + a * C::kAtomBytes, &maps.q, bar(kQdFull), a * 64, head, G.q_begin + i * kTile);
                        tma_load_3d(do_s + a * C::kAtomBytes, &maps.d_out, bar(kQdFull), a * 64, head, G.q_begin + i * kTile);
                    }
                    if (!wait(kQdFull, step, (int)step)) return;
                    tc_fence_after_sync();
                    for (int kk = 0; kk < D / 16; ++kk)
                        mma_ss(t_s, desc_kmajor(q_s, kk), desc_kmajor(k_s, kk), idesc_s, kk > 0);
                    for (int kk = 0; kk < D / 16; ++kk)
                        mma_ss(t_dp, desc_kmajor(do_s, kk), desc_kmajor(v_s, kk), idesc_s, kk > 0);
                    tc_commit(bar(kSFull));
                    if (!wait(kPdsFull, step, (int)step)) return;
                    tc_fence_after_sync();
                    // dV += P^T dO and dK += dS^T Q: the contraction runs over the 128 query rows
                    for (int kk = 0; kk < kTile / 16; ++kk)
                        mma_ss(t_dv, desc_mnmajor(p_s, kk), desc_mnmajor(do_s, kk), idesc_g, (step > 0 || kk > 0) ? 1u : 0u);
                    for (int kk = 0; kk < kTile / 16; ++kk)
                        mma_ss(t_dk, desc_mnmajor(ds_s, kk), desc_mnmajor(q_s, kk), idesc_g, (step > 0 || kk > 0) ? 1u : 0u);
                    tc_commit(bar(kStepDone));
                }
            }
        }();
    } else {
        bool alive = true;
        auto wait_c = [&](int bar_id, uint32_t parity, int iter) {
            if (alive && !__all_sync(0xffffffffu, wait(bar_id, parity, iter))) alive = false;
        };
        const int row = threadIdx.x;
        const uint32_t lane_off = (uint32_t)(32 * warp) << 16;
        uint32_t step = 0;
        for (int g = 0; g < p.n_groups; ++g) {
            const AttnGroup &G = p.g[g];
            uint32_t valid[4];
            if (!group_mask(G, r0, valid)) continue;
            for (int i = 0; i * kTile < G.q_rows; ++i, ++step) {
                const bool live = i * kTile + row < G.q_rows;
                const size_t stat = (size_t)head * p.nq_total + G.q_begin + (live ? i * kTile + row : 0);
                const float lse2 = p.lse[stat] * 1.4426950408889634f, delta = p.delta[stat];
                wait_c(kSFull, step, (int)step);
                tc_fence_after_sync();
                row_to_p_ds(t_s + lane_off, t_dp + lane_off, row, live, p.scale_log2, lse2, delta, valid, p_s, ds_s);
                fence_proxy_async_smem();
                tc_fence_before_sync();
                compute_sync();
                if (threadIdx.x == 0) mbar_arrive(bar(kPdsFull));
            }
        }
        // this thread's key row: stored only if it is one of the clip's rows inside this run
        const int r = r0 + row;
        const int slot = r / p.P, cell = r % p.P;
        const int cf = (r < run_end && slot < LL_MAX_SLOTS) ? p.slot_clip_frame[slot] : -1;
        const bool live = cf >= 0;
        const size_t token = live ? (size_t)cf * p.P + cell : 0;
        if (step > 0) wait_c(kStepDone, step - 1, (int)step);
        tc_fence_after_sync();
        if (alive && step > 0) {
            store_grad_row<D, true>(t_dk + lane_off, p.scale, p.dk + (token * p.heads + head) * D, p, live ? cf : 0,
                                    cell / p.grid_w, cell % p.grid_w, live);
            store_grad_row<D, false>(t_dv + lane_off, 1.f, p.dv + (token * p.heads + head) * D, p, 0, 0, 0, live);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag == 1) {
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 4) { __syncwarp(); tc_fence_after_sync(); tmem_dealloc(tmem, 512); }
}

}  // namespace

cudaError_t launch_attn_backward(const BwdParams &p, const BwdMaps &maps, cudaStream_t stream)
{
    const int D = p.head_dim;
    const size_t tile = (size_t)128 * D * 2, ptile = 2 * 128 * 128;
    const int smem_dq = (int)(6 * tile + ptile + 2048), smem_kv = (int)(4 * tile + 2 * ptile + 2048);
    cudaError_t e;
    if (D == 128) {
        e = cudaFuncSetAttribute(bwd_dq_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_dq);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(bwd_dkdv_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_kv);
    } else {
        e = cudaFuncSetAttribute(bwd_dq_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_dq);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(bwd_dkdv_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_kv);
    }
    if (e != cudaSuccess) return e;
    const long long warps = (long long)p.nq_total * p.heads;
    const unsigned dblocks = (unsigned)((warps * 32 + 255) / 256);
    if (D == 128) bwd_delta_kernel<128><<<dblocks, 256, 0, stream>>>(p); else bwd_delta_kernel<64><<<dblocks, 256, 0, stream>>>(p);
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    dim3 gq((unsigned)p.n_qtiles, (unsigned)p.heads), gk((unsigned)p.n_ktiles, (unsigned)p.heads);
    if (D == 128) bwd_dq_kernel<128><<<gq, kBwdThreads, smem_dq, stream>>>(p, maps);
    else          bwd_dq_kernel<64><<<gq, kBwdThreads, smem_dq, stream>>>(p, maps);
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (D == 128) bwd_dkdv_kernel<128><<<gk, kBwdThreads, smem_kv, stream>>>(p, maps);
    else          bwd_dkdv_kernel<64><<<gk, kBwdThreads, smem_kv, stream>>>(p, maps);
    count_launch();
    return cudaGetLastError();
}

}  // namespace ll
