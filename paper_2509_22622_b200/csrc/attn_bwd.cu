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
// kernels have one warp that loads (TMA) and issues the MMAs (all its lanes walk the loop so that
// descriptors are warp-uniform; one elected lane issues) and eight compute warps (one thread per
// tile row and 64-key half, the 32x32b TMEM shape).  The compute warps take S into registers and
// release its tensor memory at once, so the next step's S is formed while they are in the
// exponentials; dP is read only for the last multiply.
#include <cuda_bf16.h>

#include "bounded_wait.cuh"
#include "exp2_poly.cuh"
#include "ll_internal.h"
#include "ptx.cuh"

namespace ll {

namespace {

using namespace ptx;

constexpr int kBwdThreads = 288;                       // eight compute warps, one load/issue warp
constexpr int kIssueWarp = 8;
constexpr int kDkdvThreads = 320;                      // the dk/dv kernel adds a load warp
constexpr int kLoadWarp = 9;
constexpr int kTile = 128;

__device__ __forceinline__ void tmem_ld_32x32b_x32(uint32_t taddr, uint32_t *r)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr)
                 : "memory");
}

__device__ __forceinline__ void tmem_st_32x32b_x32(uint32_t taddr, const uint32_t *r)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
                 : "memory");
}

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

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

// Half `half` of the D columns of 128 rows x D fp32 in TMEM (row = thread), times `mul`,
// optionally turned back through the rotation of the row's grid position, rounded to bf16 and
// stored at dst (one head row of D).
template <int D, bool kRotateBack>
__device__ __forceinline__ void store_grad_row(uint32_t taddr, float mul, ll_bf16 *dst, const BwdParams &p, int frame,
                                               int y, int x, bool live, int half)
{
    constexpr int kNh = D / 6, kNt = D / 2 - 2 * kNh;
    const float2 *t_row = p.t_tab + (size_t)frame * kNt, *h_row = p.h_tab + (size_t)y * kNh, *w_row = p.w_tab + (size_t)x * kNh;
#pragma unroll
    for (int c = 0; c < D / 64; ++c) {
        const int ch = half * (D / 64) + c;
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

// MMA helpers: all tiles are 128-byte-swizzled, 128 rows, tile base 1024-byte aligned.  The low
// descriptor word of a tile is formed once; a slice of the contraction adds a constant to it.
//   K-major operand [rows][64-element atoms]: slice kk = 16 elements of the contraction.
//   MN-major operand: the tile's rows are the contraction index, its columns the M (or N) index;
//   slice kk = rows 16 kk .. 16 kk + 15.
__device__ __forceinline__ uint32_t lo_kmajor(uint32_t tile) { return smem_desc_lo(tile, 16); }
__device__ __forceinline__ uint32_t lo_mnmajor(uint32_t tile) { return smem_desc_lo(tile, 128 * 128); }
__host__ __device__ constexpr uint32_t slice_kmajor(int kk) { return (uint32_t)(((kk / 4) * (128 * 128) + (kk % 4) * 32) >> 4); }
__host__ __device__ constexpr uint32_t slice_mnmajor(int kk) { return (uint32_t)((kk * 2048) >> 4); }

// Slices kBegin .. kEnd - 1 of D (+)= A B; kAMn / kBMn say which operand is MN-major.  The first
// slice accumulates iff `acc_first`.
template <int kBegin, int kEnd, bool kAMn, bool kBMn>
__device__ __forceinline__ void mma_slices(uint32_t d, uint32_t a_lo, uint32_t b_lo, uint32_t idesc, uint32_t acc_first)
{
    constexpr uint32_t hi = smem_desc_hi_sw128(1024);
#pragma unroll
    for (int kk = kBegin; kk < kEnd; ++kk)
        mma_ss(d, smem_desc_join(a_lo + (kAMn ? slice_mnmajor(kk) : slice_kmajor(kk)), hi),
               smem_desc_join(b_lo + (kBMn ? slice_mnmajor(kk) : slice_kmajor(kk)), hi), idesc, kk > kBegin ? 1u : acc_first);
}

__device__ __forceinline__ void key_mask(int nvalid, uint32_t (&valid)[4])
{
#pragma unroll
    for (int ch = 0; ch < 4; ++ch)
        valid[ch] = nvalid >= 32 * (ch + 1) ? 0xffffffffu : nvalid > 32 * ch ? ((1u << (nvalid - 32 * ch)) - 1u) : 0u;
}

// This thread's 64 columns of a score row (fp32 words in s) to the weights p = 2^(s c - lse2),
// in place; columns whose bit in vlo (first 32) / vhi is clear give zero.  (Moving a quarter or
// a half of the exponentials to the FMA-pipe polynomial of the forward kernel made the pass
// slower, 8.46 and 8.59 ms against 8.35 ms at the 21-frame clip, so all of them stay on the
// special-function unit.)
__device__ __forceinline__ void scores_to_weights(uint32_t (&s)[64], float c, float lse2, uint32_t vlo, uint32_t vhi)
{
    const uint64_t c2 = pack2(c, c), nl2 = pack2(-lse2, -lse2);
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        float e0, e1;
        unpack2(exp2_sfu2(fma2(pack2(as_f(s[2 * i]), as_f(s[2 * i + 1])), c2, nl2)), e0, e1);
        s[2 * i] = __float_as_uint(e0);
        s[2 * i + 1] = __float_as_uint(e1);
    }
    if ((vlo & vhi) != 0xffffffffu) {
#pragma unroll
        for (int i = 0; i < 64; ++i)
            if (!(((i < 32 ? vlo : vhi) >> (i & 31)) & 1u)) s[i] = 0u;
    }
}

// dS = p (dP - delta) of this thread's 64 columns (32-column chunks ch0, ch0 + 1 of tile row
// `row`), rounded to bf16, into the swizzled [row][key] tile; the weights themselves too when
// p_tile is not 0.
__device__ __forceinline__ void store_ds(const uint32_t (&pw)[64], uint32_t t_dp, int row, int ch0, float delta, uint32_t p_tile,
                                         uint32_t ds_tile)
{
    const uint64_t nd2 = pack2(-delta, -delta);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int ch = ch0 + h;
        uint32_t dp[32];
        tmem_ld_32x32b_x32(t_dp + 32 * ch, dp);
        tmem_wait_ld();
        uint32_t dw[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            float d0, d1;
            unpack2(mul2(pack2(as_f(pw[32 * h + 2 * i]), as_f(pw[32 * h + 2 * i + 1])),
                         add2(pack2(as_f(dp[2 * i]), as_f(dp[2 * i + 1])), nd2)), d0, d1);
            dw[i] = cvt_bf16x2(d0, d1);
        }
        const uint32_t row_off = (uint32_t)(ch >> 1) * (128 * 128) + (uint32_t)row * 128;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t chunk = (uint32_t)(((ch & 1) * 4 + k) ^ (row & 7)) << 4;
            st_shared_v4(ds_tile + row_off + chunk, dw[4 * k], dw[4 * k + 1], dw[4 * k + 2], dw[4 * k + 3]);
            if (p_tile) {
                const int b = 32 * h + 8 * k;
                st_shared_v4(p_tile + row_off + chunk, cvt_bf16x2(as_f(pw[b]), as_f(pw[b + 1])), cvt_bf16x2(as_f(pw[b + 2]), as_f(pw[b + 3])),
                             cvt_bf16x2(as_f(pw[b + 4]), as_f(pw[b + 5])), cvt_bf16x2(as_f(pw[b + 6]), as_f(pw[b + 7])));
            }
        }
    }
}

// ---- dq: one CTA per (128-row query tile, head) ---------------------------------------------
// The tile's Q and dO rows are the stationary A operands of S = Q K^T and dP = dO V^T: they are
// written once into tensor memory (bf16, two elements per column), so those products read only
// K and V from shared memory.  Eight compute warps share a step (thread = tile row x 64-key
// half).  Per 128-key step j the tensor pipe runs S(j+1) | dQ(j-1) | dP(j) ...: the compute warps
// take S(j) into registers and release it at once, so S(j+1) is formed while they are in the
// exponentials; dP(j) is only needed for the last multiply, dS = P (dP - delta), after which
// dQ(j) and dP(j+1) are issued.  K and V tiles sit in three stages; K is needed until the
// step's dQ product, V only until its dP.
//   tensor memory columns: S 0..127, dP 128..255, dQ 256..256+D-1, Q 384.., dO 448..
template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1)
bwd_dq_kernel(const __grid_constant__ BwdParams p, const __grid_constant__ BwdMaps maps)
{
    using C = BwdCfg<D>;
    constexpr int kStages = 3;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t k_s = base, v_s = k_s + kStages * C::kTileBytes, ds_s = v_s + kStages * C::kTileBytes, bars = ds_s + C::kPBytes;
    enum { kKFull = 0, kVFull = 3, kKEmpty = 6, kVEmpty = 9, kSFull = 12, kSFree = 13, kDpFull = 14, kDsFull = 15, kDone = 16, kBars = 17 };
    constexpr int kComputeWarps = 8;
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
        for (int i = 0; i < kBars; ++i) mbar_init(bar(i), (i == kSFree || i == kDsFull) ? kComputeWarps : 1);
        *abort_flag = (*reinterpret_cast<volatile uint32_t *>(p.status) != kStatusOk) ? 2 : 0;
        fence_mbar_init();
    }
    if (warp == kIssueWarp) { tmem_alloc(smem_u32(tmem_slot), 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    WaitCtx ctx{abort_flag, p.status, warp};
    auto wait = [&](int bar_id, uint32_t parity, int iter) -> bool { return wait_bar(bar(bar_id), parity & 1u, ctx, bar_id, iter); };
    const bool skip = *abort_flag != 0;
    const uint32_t t_s = tmem, t_dp = tmem + 128, t_dq = tmem + 256, t_q = tmem + 384, t_do = tmem + 448;

    // the tile's Q rows (warps 0-3) and dO rows (warps 4-7) into tensor memory; rows past the
    // group's end become zeros
    if (!skip && warp != kIssueWarp) {
        const int row = threadIdx.x & 127, half = threadIdx.x >> 7;
        const bool live = row < rows;
        const uint4 *src = reinterpret_cast<const uint4 *>((half ? p.d_out : p.q) + ((size_t)(q0 + (live ? row : 0)) * p.heads + head) * D);
        const uint32_t dst = (half ? t_do : t_q) + ((uint32_t)(32 * (warp & 3)) << 16);
#pragma unroll
        for (int c = 0; c < D / 64; ++c) {
            uint32_t w[32];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint4 u = live ? __ldg(src + 8 * c + i) : make_uint4(0u, 0u, 0u, 0u);
                w[4 * i] = u.x; w[4 * i + 1] = u.y; w[4 * i + 2] = u.z; w[4 * i + 3] = u.w;
            }
            tmem_st_32x32b_x32(dst + 32 * c, w);
        }
        tmem_wait_st();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();

    if (skip) {
    } else if (warp == kIssueWarp) {
        // All 32 lanes walk the loop and the waits, so that addresses and descriptors are
        // warp-uniform values; one elected lane issues the copies, the MMAs and the commits.
        [&]() {
            const bool elected = elect_one();
            constexpr uint32_t idesc_s = idesc_bf16_f32(128, 128, 0, 0), idesc_dq = idesc_bf16_f32(128, D, 0, 1);
            constexpr uint32_t hi = smem_desc_hi_sw128(1024);
            RunTiles kt(&G);                                     // walks ahead of the products: tile of the next load
            int loaded = 0;
            auto load_kv = [&]() {                               // K and V tiles of step `loaded`
                const int st = loaded % kStages, row = kt.row();
                if (elected) {
                    mbar_arrive_expect_tx(bar(kKFull + st), C::kTileBytes);
                    for (int a = 0; a < D / 64; ++a)
                        tma_load_3d(k_s + st * C::kTileBytes + a * C::kAtomBytes, &maps.k, bar(kKFull + st), a * 64, row, head);
                    mbar_arrive_expect_tx(bar(kVFull + st), C::kTileBytes);
                    for (int a = 0; a < D / 64; ++a)
                        tma_load_3d(v_s + st * C::kTileBytes + a * C::kAtomBytes, &maps.v, bar(kVFull + st), a * 64, row, head);
                }
                __syncwarp();
                ++loaded;
                kt.next();
            };
            auto commit = [&](int bar_id) { if (elected) tc_commit(bar(bar_id)); };
            const uint32_t k_lo = lo_kmajor(k_s), v_lo = lo_kmajor(v_s), ds_lo = lo_kmajor(ds_s);
            auto issue_s = [&](int j) -> bool {                  // S(j) = Q K(j)^T
                const int st = j % kStages;
                if (!wait(kKFull + st, j / kStages, j)) return false;
                tc_fence_after_sync();
                const uint32_t b_lo = k_lo + ((uint32_t)(st * C::kTileBytes) >> 4);
                if (elected) {
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk)
                        mma_ts(t_s, t_q + 8 * kk, smem_desc_join(b_lo + slice_kmajor(kk), hi), idesc_s, kk > 0);
                }
                __syncwarp();
                commit(kSFull);
                return true;
            };
            auto issue_dp = [&](int j) -> bool {                 // dP(j) = dO V(j)^T
                const int st = j % kStages;
                if (!wait(kVFull + st, j / kStages, j)) return false;
                tc_fence_after_sync();
                const uint32_t b_lo = v_lo + ((uint32_t)(st * C::kTileBytes) >> 4);
                if (elected) {
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk)
                        mma_ts(t_dp, t_do + 8 * kk, smem_desc_join(b_lo + slice_kmajor(kk), hi), idesc_s, kk > 0);
                }
                __syncwarp();
                commit(kDpFull);
                commit(kVEmpty + st);
                return true;
            };
            for (int i = 0; i < kStages && i < n_kt; ++i) load_kv();
            if (!issue_s(0) || !issue_dp(0)) return;
            for (int j = 0; j < n_kt; ++j) {
                const int st = j % kStages;
                if (j >= 1 && j + 2 < n_kt) {                    // the stage step j - 1 used takes step j + 2
                    const int free_st = (j - 1) % kStages;
                    if (!wait(kVEmpty + free_st, (j - 1) / kStages, j) || !wait(kKEmpty + free_st, (j - 1) / kStages, j)) return;
                    load_kv();
                }
                if (j + 1 < n_kt) {
                    if (!wait(kSFree, j, j)) return;             // S(j) is in the compute warps' registers
                    if (!issue_s(j + 1)) return;
                }
                if (!wait(kDsFull, j, j)) return;                // dS(j) is in shared memory, dP(j) has been read
                tc_fence_after_sync();
                const uint32_t k_mn = lo_mnmajor(k_s + st * C::kTileBytes);
                if (elected) mma_slices<0, 8, false, true>(t_dq, ds_lo, k_mn, idesc_dq, j > 0 ? 1u : 0u);
                __syncwarp();
                commit(kKEmpty + st);
                if (j + 1 < n_kt && !issue_dp(j + 1)) return;
            }
            commit(kDone);
        }();
    } else {
        bool alive = true;
        auto wait_c = [&](int bar_id, uint32_t parity, int iter) {
            if (alive && !__all_sync(0xffffffffu, wait(bar_id, parity, iter))) alive = false;
        };
        const int row = threadIdx.x & 127, half = threadIdx.x >> 7;      // tile row = TMEM lane; 64-key half
        const bool live = row < rows;
        const uint32_t lane_off = (uint32_t)(32 * (warp & 3)) << 16;
        const size_t stat = (size_t)head * p.nq_total + q0 + (live ? row : 0);
        const float lse2 = p.lse[stat] * 1.4426950408889634f, delta = p.delta[stat];
        RunTiles kt(&G);
        for (int j = 0; j < n_kt; ++j, kt.next()) {
            uint32_t valid[4];
            key_mask(kt.valid(), valid);
            wait_c(kSFull, j, j);
            tc_fence_after_sync();
            uint32_t w[64];
            tmem_ld_32x32b_x32(t_s + lane_off + 64 * half, w);
            tmem_ld_32x32b_x32(t_s + lane_off + 64 * half + 32, w + 32);
            tmem_wait_ld();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kSFree));
            scores_to_weights(w, p.scale_log2, lse2, live ? (half ? valid[2] : valid[0]) : 0u, live ? (half ? valid[3] : valid[1]) : 0u);
            wait_c(kDpFull, j, j);
            tc_fence_after_sync();
            store_ds(w, t_dp + lane_off, row, 2 * half, delta, 0u, ds_s);
            fence_proxy_async_smem();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kDsFull));
        }
        wait_c(kDone, 0, n_kt);
        tc_fence_after_sync();
        const int token = q0 + (live ? row : 0);
        const int frame = token / p.P, cell = token % p.P;
        if (alive)
            store_grad_row<D, true>(t_dq + lane_off, p.scale, p.dq + ((size_t)token * p.heads + head) * D, p, frame,
                                    cell / p.grid_w, cell % p.grid_w, live, half);
    }
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag == 1) {
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == kIssueWarp) { __syncwarp(); tc_fence_after_sync(); tmem_dealloc(tmem, 512); }
}


// Which of the 128 cache rows starting at r0 a group can see (bit c of word c / 32 = row r0 + c).
__device__ __forceinline__ bool group_mask(const AttnGroup &G, int r0, uint32_t (&valid)[4])
{
    valid[0] = valid[1] = valid[2] = valid[3] = 0u;
    bool any = false;
    for (int r = 0; r < G.n_ranges; ++r) {
        const int lo = max(G.k_start[r], r0) - r0, hi = min(G.k_start[r] + G.k_len[r], r0 + kTile) - r0;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const int a = min(max(lo - 32 * w, 0), 32), b = min(max(hi - 32 * w, 0), 32);
            if (b > a) valid[w] |= (b == 32 ? 0xffffffffu : (1u << b) - 1u) & ~((1u << a) - 1u);
        }
        any |= hi > lo;
    }
    return any;
}

// Whether any of the 128 cache rows starting at r0 is visible to the group.
__device__ __forceinline__ bool group_sees(const AttnGroup &G, int r0)
{
    bool any = false;
    for (int r = 0; r < G.n_ranges; ++r)
        any |= min(G.k_start[r] + G.k_len[r], r0 + kTile) > max(G.k_start[r], r0);
    return any;
}

// The (group, 128-row query tile) pairs a key tile takes part in, in order.  The group's first row
// and tile count are kept, so a step inside a group costs an increment.
struct QTiles {
    const BwdParams &p;
    int r0, g, i, tiles, q_begin;
    __device__ QTiles(const BwdParams &params, int first_row) : p(params), r0(first_row), g(-1), i(0), tiles(0), q_begin(0) { next(); }
    __device__ bool done() const { return g >= p.n_groups; }
    __device__ int q_row() const { return q_begin + i * kTile; }
    __device__ void next()
    {
        if (++i < tiles) return;
        i = 0;
        for (++g; g < p.n_groups; ++g) {
            const AttnGroup &G = p.g[g];
            if (G.q_rows > 0 && group_sees(G, r0)) {
                tiles = (G.q_rows + kTile - 1) / kTile;
                q_begin = G.q_begin;
                return;
            }
        }
    }
};

// ---- dk, dv: one CTA per (128-row tile of the clip's cache rows, head) -----------------------
// K and V of the tile stay in shared memory; per step j one query tile's Q and dO stream in.
// The tensor pipe runs, per step,  S(j+1) | dV(j) | dK(j) | dP(j+1):  the eight compute warps
// take S(j) into registers and release it at once, so S(j+1) is formed while they are in the
// exponentials; dP(j) is only needed for dS = P (dP - delta), after which P and dS go to shared
// memory as the MN-major A operands of dV += P^T dO and dK += dS^T Q.
// Shared memory has room for three streamed tiles beside K, V, P and dS, so Q is loaded twice:
//   slot j % 2:  Q(j) for S(j), then (once S(j) is done) dO(j) for dP(j) and dV(j), then Q(j+2)
//   slot C:      Q(j) for dK(j), then Q(j+1)
// which gives every load about one step of lead.  The loads have a warp of their own (warp 9),
// so that the MMA issuer (warp 8) never sits in a wait for a slot while products could be issued.
template <int D>
__global__ void __launch_bounds__(kDkdvThreads, 1)
bwd_dkdv_kernel(const __grid_constant__ BwdParams p, const __grid_constant__ BwdMaps maps)
{
    using C = BwdCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t k_s = base, v_s = k_s + C::kTileBytes, slot_s = v_s + C::kTileBytes, c_s = slot_s + 2 * C::kTileBytes,
                   p_s = c_s + C::kTileBytes, ds_s = p_s + C::kPBytes, bars = ds_s + C::kPBytes;
    enum { kKvFull = 0, kSlotFull = 1, kCFull = 3, kSFull = 4, kSFree = 5, kDpFull = 6, kDsFull = 7, kSlotFree = 8, kCFree = 10, kBars = 11 };
    constexpr int kComputeWarps = 8;
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
        for (int i = 0; i < kBars; ++i) mbar_init(bar(i), (i == kSFree || i == kDsFull) ? kComputeWarps : 1);
        *abort_flag = (*reinterpret_cast<volatile uint32_t *>(p.status) != kStatusOk) ? 2 : 0;
        fence_mbar_init();
    }
    if (warp == kIssueWarp) { tmem_alloc(smem_u32(tmem_slot), 512); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = *tmem_slot;
    WaitCtx ctx{abort_flag, p.status, warp};
    auto wait = [&](int bar_id, uint32_t parity, int iter) -> bool { return wait_bar(bar(bar_id), parity & 1u, ctx, bar_id, iter); };
    const bool skip = *abort_flag != 0;
    const uint32_t t_s = tmem, t_dp = tmem + 128, t_dk = tmem + 256, t_dv = tmem + 256 + D;

    if (skip) {
    } else if (warp == kLoadWarp) {
        // ---- loads: all lanes walk the loop, one elected lane issues the copies ----
        [&]() {
            const bool elected = elect_one();
            auto load_tile = [&](uint32_t dst, const CUtensorMap *map, int bar_id, int q_row) {
                if (elected) {
                    mbar_arrive_expect_tx(bar(bar_id), C::kTileBytes);
                    for (int a = 0; a < D / 64; ++a) tma_load_3d(dst + a * C::kAtomBytes, map, bar(bar_id), a * 64, head, q_row);
                }
                __syncwarp();
            };
            // first rows of the query tiles of steps j, j + 1, j + 2 (-1: no such step)
            QTiles qt(p, r0);
            auto take = [&]() -> int { if (qt.done()) return -1; const int r = qt.q_row(); qt.next(); return r; };
            int row_j = take(), row_j1 = take(), row_j2 = take();
            if (row_j < 0) return;
            if (elected) {
                mbar_arrive_expect_tx(bar(kKvFull), 2 * C::kTileBytes);
                for (int a = 0; a < D / 64; ++a) {
                    tma_load_3d(k_s + a * C::kAtomBytes, &maps.k, bar(kKvFull), a * 64, r0, head);
                    tma_load_3d(v_s + a * C::kAtomBytes, &maps.v, bar(kKvFull), a * 64, r0, head);
                }
            }
            __syncwarp();
            load_tile(slot_s, &maps.q, kSlotFull + 0, row_j);
            if (row_j1 >= 0) load_tile(slot_s + C::kTileBytes, &maps.q, kSlotFull + 1, row_j1);
            load_tile(c_s, &maps.q, kCFull, row_j);
            if (!wait(kSFull, 0, 0)) return;                     // S(0) has read Q(0): its slot takes dO(0)
            load_tile(slot_s, &maps.d_out, kSlotFull + 0, row_j);
            for (int j = 0; row_j1 >= 0; ++j) {
                const int sl = j & 1;
                if (!wait(kSFull, j + 1, j)) return;             // S(j+1) has read Q(j+1): its slot takes dO(j+1)
                load_tile(slot_s + (sl ^ 1) * C::kTileBytes, &maps.d_out, kSlotFull + (sl ^ 1), row_j1);
                if (row_j2 >= 0) {                               // dV(j) has read dO(j): its slot takes Q(j+2)
                    if (!wait(kSlotFree + sl, j >> 1, j)) return;
                    load_tile(slot_s + sl * C::kTileBytes, &maps.q, kSlotFull + sl, row_j2);
                }
                if (!wait(kCFree, j, j)) return;                 // dK(j) has read Q(j)
                load_tile(c_s, &maps.q, kCFull, row_j1);
                row_j = row_j1;
                row_j1 = row_j2;
                row_j2 = take();
            }
        }();
    } else if (warp == kIssueWarp) {
        // ---- MMA issue: all lanes walk the loop and the waits, one elected lane issues ----
        [&]() {
            const bool elected = elect_one();
            constexpr uint32_t idesc_s = idesc_bf16_f32(128, 128, 0, 0), idesc_g = idesc_bf16_f32(128, D, 1, 1);
            auto commit = [&](int bar_id) { if (elected) tc_commit(bar(bar_id)); };
            int n_steps = 0;
            for (QTiles qt(p, r0); !qt.done(); qt.next()) ++n_steps;
            if (n_steps == 0) return;
            const uint32_t k_k = lo_kmajor(k_s), v_k = lo_kmajor(v_s), p_mn = lo_mnmajor(p_s), ds_mn = lo_mnmajor(ds_s), c_mn = lo_mnmajor(c_s);
            // a slot's fills alternate Q (for S) and dO: waits see parity 0 for Q, 1 for dO
            auto issue_s = [&](int j) -> bool {
                const int sl = j & 1;
                if (!wait(kSlotFull + sl, 0, j)) return false;
                tc_fence_after_sync();
                if (elected) mma_slices<0, D / 16, false, false>(t_s, lo_kmajor(slot_s + sl * C::kTileBytes), k_k, idesc_s, 0u);
                __syncwarp();
                commit(kSFull);
                return true;
            };
            auto issue_dp = [&](int j) -> bool {
                const int sl = j & 1;
                if (!wait(kSlotFull + sl, 1, j)) return false;
                tc_fence_after_sync();
                if (elected) mma_slices<0, D / 16, false, false>(t_dp, lo_kmajor(slot_s + sl * C::kTileBytes), v_k, idesc_s, 0u);
                __syncwarp();
                commit(kDpFull);
                return true;
            };
            if (!wait(kKvFull, 0, 0)) return;
            if (!issue_s(0) || !issue_dp(0)) return;
            for (int j = 0; j < n_steps; ++j) {
                const int sl = j & 1;
                const bool more = j + 1 < n_steps;
                if (more) {
                    if (!wait(kSFree, j, j)) return;             // S(j) is in the compute warps' registers
                    if (!issue_s(j + 1)) return;
                }
                if (!wait(kDsFull, j, j)) return;                // P(j) and dS(j) are in shared memory, dP(j) has been read
                tc_fence_after_sync();
                // dV += P^T dO and dK += dS^T Q: the contraction runs over the 128 query rows
                if (elected) mma_slices<0, kTile / 16, true, true>(t_dv, p_mn, lo_mnmajor(slot_s + sl * C::kTileBytes), idesc_g, j > 0 ? 1u : 0u);
                __syncwarp();
                commit(kSlotFree + sl);
                if (!wait(kCFull, j, j)) return;
                tc_fence_after_sync();
                if (elected) mma_slices<0, kTile / 16, true, true>(t_dk, ds_mn, c_mn, idesc_g, j > 0 ? 1u : 0u);
                __syncwarp();
                commit(kCFree);
                if (more && !issue_dp(j + 1)) return;
            }
        }();
    } else {
        bool alive = true;
        auto wait_c = [&](int bar_id, uint32_t parity, int iter) {
            if (alive && !__all_sync(0xffffffffu, wait(bar_id, parity, iter))) alive = false;
        };
        const int row = threadIdx.x & 127, half = threadIdx.x >> 7;
        const uint32_t lane_off = (uint32_t)(32 * (warp & 3)) << 16;
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
                uint32_t w[64];
                tmem_ld_32x32b_x32(t_s + lane_off + 64 * half, w);
                tmem_ld_32x32b_x32(t_s + lane_off + 64 * half + 32, w + 32);
                tmem_wait_ld();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kSFree));
                scores_to_weights(w, p.scale_log2, lse2, live ? (half ? valid[2] : valid[0]) : 0u, live ? (half ? valid[3] : valid[1]) : 0u);
                wait_c(kDpFull, step, (int)step);
                if (step > 0) wait_c(kCFree, step - 1, (int)step);       // the last step's products have read P and dS
                tc_fence_after_sync();
                store_ds(w, t_dp + lane_off, row, 2 * half, delta, p_s, ds_s);
                fence_proxy_async_smem();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kDsFull));
            }
        }
        // this thread's key row: stored only if it is one of the clip's rows inside this run
        const int r = r0 + row;
        const int slot = r / p.P, cell = r % p.P;
        const int cf = (r < run_end && slot < LL_MAX_SLOTS) ? p.slot_clip_frame[slot] : -1;
        const bool live = cf >= 0;
        const size_t token = live ? (size_t)cf * p.P + cell : 0;
        if (step > 0) wait_c(kCFree, step - 1, (int)step);
        tc_fence_after_sync();
        if (alive && step > 0) {
            store_grad_row<D, true>(t_dk + lane_off, p.scale, p.dk + (token * p.heads + head) * D, p, live ? cf : 0,
                                    cell / p.grid_w, cell % p.grid_w, live, half);
            store_grad_row<D, false>(t_dv + lane_off, 1.f, p.dv + (token * p.heads + head) * D, p, 0, 0, 0, live, half);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag == 1) {
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == kIssueWarp) { __syncwarp(); tc_fence_after_sync(); tmem_dealloc(tmem, 512); }
}

}  // namespace

cudaError_t launch_attn_backward(const BwdParams &p, const BwdMaps &maps, cudaStream_t stream)
{
    const int D = p.head_dim;
    const size_t tile = (size_t)128 * D * 2, ptile = 2 * 128 * 128;
    const int smem_dq = (int)(6 * tile + ptile + 2048), smem_kv = (int)(5 * tile + 2 * ptile + 2048);
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
    if (D == 128) bwd_dkdv_kernel<128><<<gk, kDkdvThreads, smem_kv, stream>>>(p, maps);
    else          bwd_dkdv_kernel<64><<<gk, kDkdvThreads, smem_kv, stream>>>(p, maps);
    count_launch();
    return cudaGetLastError();
}

}  // namespace ll
