// QKV projection with the path's front end in its epilogue (sm_100a):
//
//   y = x W^T + b          x [n_tokens, d_model] bf16, W [3*H*D, d_model] bf16, fp32 accumulation
//   q | k | v = y          (the rows of W are the q features, then k, then v)
//   q, k: optional RMS norm over the token's whole row of H*D elements with a learned gain,
//         then the 3-D rotation;  rotated q -> q_out, rotated k and raw v -> the cache rows.
//
// The GEMM is a persistent tcgen05 kernel: CTA tile 128 tokens x TN output features, TN = 256
// or 192 (whichever leaves the SMs less idle in the last round of tiles: 3*H*D / TN tiles per
// 128 tokens over the SM count), K blocks of 64 through a TMA ring of 4 (TN 256) or 5 (TN 192)
// stages, accumulators double-buffered in TMEM (2 x TN columns) so that the epilogue of a tile
// runs under the main loop of the next.  Warp 0 (one lane): TMA producer.  Warp 1 (one elected
// lane): MMA issuer.  Warps 4-11: epilogue, one thread per token row and half of the tile's
// features (the 32x32b TMEM shape).
//
// The norm needs the sum of squares of a token's whole q (or k) row, which is spread over
// H*D/256 tiles that run on different SMs at different times.  The factor is one scalar per
// token and everything after it is linear, so a tile stores rotate(gain * y) without it and
// leaves its part of the sum of squares in a table (one slot per token and half tile: no atomics,
// the sum is taken in a fixed order).  For q the scalar then travels with q_out to the
// attention call as a per-row softmax scale; for k a small second kernel applies it: the
// epilogue parks the un-normalised rotated k rows in fp32 in the caller's workspace and the
// second kernel scales, rounds once to bf16 and writes the cache rows.
#include <cuda_bf16.h>

#include "bounded_wait.cuh"
#include "ll_internal.h"
#include "ptx.cuh"

namespace ll {

namespace {

using namespace ptx;

constexpr int kGemmThreads = 384;                      // TMA, MMA, two idle warps, eight epilogue warps
constexpr int kTileM = 128, kBlockK = 64;
constexpr int kABytes = kTileM * kBlockK * 2;          // 16 KB

template <int TN>
struct GemmCfg {
    static_assert(TN == 256 || TN == 192, "tile widths built");
    static constexpr int kStages = TN == 256 ? 4 : 5;
    static constexpr int kBBytes = TN * kBlockK * 2;   // 32 KB or 24 KB
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kSmem = kStages * kStageBytes + 1024 /*barriers*/ + 1024 /*alignment*/;
    // barrier indices
    static constexpr int kFull = 0, kEmpty = kStages, kAccFull = 2 * kStages, kAccEmpty = 2 * kStages + 2, kBars = 2 * kStages + 4;
};

__device__ __forceinline__ void tmem_ld_32x32b_x32(uint32_t taddr, uint32_t *r)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr)
                 : "memory");
}

// What an epilogue thread knows about its token row.
struct EpiRow {
    int which;                         // 0 q, 1 k, 2 v (a tile never straddles them)
    int token, HD;
    bool live, park;                   // park: k under the norm, fp32, finished by the second kernel
    size_t cache_row;
    const float *gain;
    const float2 *t_row, *h_row, *w_row;
};

// 32 features of one token row (first feature cw inside q, k or v, n inside the 3*H*D outputs;
// kD0 = cw % D, so which band - t, h or w - a rotation pair belongs to is known at compile time
// and its (cos, sin) comes from one of three row pointers at a fixed offset): bias, sum of
// squares, gain, rotation, stores.
template <int D, int kD0>
__device__ __forceinline__ void epilogue_piece(const QkvParams &p, const EpiRow &e, uint32_t taddr, int n, int cw, float &ssq)
{
    constexpr int kNh = D / 6, kNt = D / 2 - 2 * kNh;  // pairs of the h (= w) and t bands
    uint32_t r[32];
    tmem_ld_32x32b_x32(taddr, r);
    tmem_wait_ld();
    const int head = cw / D;
    float v[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
    if (p.bias) {
        const float4 *bp = reinterpret_cast<const float4 *>(p.bias + n);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float4 bb = __ldg(bp + i);
            v[4 * i] += bb.x; v[4 * i + 1] += bb.y; v[4 * i + 2] += bb.z; v[4 * i + 3] += bb.w;
        }
    }
    if (e.which < 2) {
#pragma unroll
        for (int i = 0; i < 32; ++i) ssq = fmaf(v[i], v[i], ssq);
        if (p.with_norm) {
            const float4 *gp = reinterpret_cast<const float4 *>(e.gain + cw);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float4 gg = __ldg(gp + i);
                v[4 * i] *= gg.x; v[4 * i + 1] *= gg.y; v[4 * i + 2] *= gg.z; v[4 * i + 3] *= gg.w;
            }
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            constexpr int j0 = kD0 / 2;
            const int j = j0 + i;                      // rotation pair inside the head row (compile time)
            const float2 cs = j < kNt ? __ldg(e.t_row + j) : j < kNt + kNh ? __ldg(e.h_row + (j - kNt)) : __ldg(e.w_row + (j - kNt - kNh));
            const float a = v[2 * i], b = v[2 * i + 1];
            v[2 * i] = fmaf(a, cs.x, -(b * cs.y));
            v[2 * i + 1] = fmaf(a, cs.y, b * cs.x);
        }
    }
    if (!e.live) return;
    if (e.park) {
        float4 *dst = reinterpret_cast<float4 *>(p.k_park + (size_t)e.token * e.HD + cw);
#pragma unroll
        for (int i = 0; i < 8; ++i) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
    } else {
        ll_bf16 *dst;
        if (e.which == 0) dst = p.q_out + ((size_t)e.token * p.heads + head) * D + kD0;
        else              dst = (e.which == 1 ? p.kcache : p.vcache) + ((size_t)head * p.rows_per_head + e.cache_row) * D + kD0;
        uint32_t o[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) o[i] = cvt_bf16x2(v[2 * i], v[2 * i + 1]);
#pragma unroll
        for (int i = 0; i < 4; ++i)
            reinterpret_cast<uint4 *>(dst)[i] = make_uint4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
    }
}

// One token row of half a 128 x TN accumulator tile (TN / 2 features: `half` 0 or 1), 32
// features at a time; returns the half's sum of squares.
template <int D, int TN>
__device__ __forceinline__ float epilogue_half(const QkvParams &p, uint32_t taddr, int token, int n0, int half)
{
    constexpr int kNh = D / 6, kNt = D / 2 - 2 * kNh;
    constexpr int kHalf = TN / 2;
    EpiRow e;
    e.HD = p.heads * D;
    e.which = n0 / e.HD;
    e.live = token < p.n_tokens;
    e.token = token;
    const int tok = e.live ? token : 0;
    const int frame = tok / p.P, cell = tok % p.P;
    e.cache_row = (size_t)p.slot[frame] * p.P + cell;
    e.park = e.which == 1 && p.with_norm;
    e.gain = e.which == 0 ? p.gain_q : p.gain_k;
    e.t_row = p.t_tab + (size_t)frame * kNt;
    e.h_row = p.h_tab + (size_t)(cell / p.grid_w) * kNh;
    e.w_row = p.w_tab + (size_t)(cell % p.grid_w) * kNh;
    const int cw0 = n0 - e.which * e.HD + kHalf * half;    // this half's first feature inside q, k or v
    float ssq = 0.f;
#pragma unroll 1
    for (int ch = 0; ch < kHalf / 32; ++ch) {
        const int cw = cw0 + 32 * ch, n = n0 + kHalf * half + 32 * ch;
        const uint32_t t = taddr + kHalf * half + 32 * ch;
        switch (cw % D) {                                  // the same for the whole warp
        case 0: epilogue_piece<D, 0>(p, e, t, n, cw, ssq); break;
        case 32: epilogue_piece<D, 32>(p, e, t, n, cw, ssq); break;
        default:
            if constexpr (D == 128) {
                if (cw % D == 64) epilogue_piece<D, 64>(p, e, t, n, cw, ssq);
                else              epilogue_piece<D, 96>(p, e, t, n, cw, ssq);
            }
            break;
        }
    }
    return ssq;
}

template <int D, int TN>
__global__ void __launch_bounds__(kGemmThreads, 1)
qkv_gemm_kernel(const __grid_constant__ QkvParams p, const __grid_constant__ CUtensorMap xmap,
                const __grid_constant__ CUtensorMap wmap)
{
    using G = GemmCfg<TN>;
    constexpr int kGemmStages = G::kStages, kStageBytes = G::kStageBytes, kTileN = TN, kGemmBars = G::kBars;
    constexpr int kFull = G::kFull, kEmpty = G::kEmpty, kAccFull = G::kAccFull, kAccEmpty = G::kAccEmpty;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t bars = smem_base + kGemmStages * kStageBytes;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem_gen + kGemmStages * kStageBytes + kGemmBars * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    auto bar = [&](int i) -> uint32_t { return bars + 8u * (uint32_t)i; };
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int i = 0; i < kGemmBars; ++i) mbar_init(bar(i), (i >= kAccEmpty) ? 8u : 1u);   // eight epilogue warps free a buffer
        *abort_flag = (*reinterpret_cast<volatile uint32_t *>(p.status) != kStatusOk) ? 2 : 0;
        fence_mbar_init();
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(tmem_slot), 512);
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
    const int n_kb = (p.d_model + kBlockK - 1) / kBlockK;
    const int n_tiles = p.m_tiles * p.n_tiles;

    if (skip) {
        // an earlier kernel gave up on a wait: nothing to do
    } else if (warp == 0 && lane == 0) {
        // ---- TMA producer: tiles in the order all roles walk them; n runs fastest so that the
        // CTAs of a wave share x rows and stream the weights (which stay in L2 anyway) ----
        prefetch_tensormap(&xmap);
        prefetch_tensormap(&wmap);
        uint32_t n = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
            const int m0 = (tile / p.n_tiles) * kTileM, n0 = (tile % p.n_tiles) * kTileN;
            for (int kb = 0; kb < n_kb; ++kb, ++n) {
                const int stage = n % kGemmStages;
                if (!wait(kEmpty + stage, (n / kGemmStages) ^ 1u, (int)n)) goto done;
                mbar_arrive_expect_tx(bar(kFull + stage), kStageBytes);
                const uint32_t a = smem_base + stage * kStageBytes;
                tma_load_3d(a, &xmap, bar(kFull + stage), kb * kBlockK, m0, 0);
                tma_load_3d(a + kABytes, &wmap, bar(kFull + stage), kb * kBlockK, n0, 0);
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer ----
        const bool elected = elect_one();
        constexpr uint32_t idesc = idesc_bf16_f32(kTileM, kTileN, 0, 0);
        constexpr uint32_t hi = smem_desc_hi_sw128(1024);
        uint32_t n = 0, t = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++t) {
            const uint32_t buf = t & 1u;
            // the epilogue has read this accumulator buffer out (two tiles ago)
            if (t >= 2 && !wait(kAccEmpty + buf, (t >> 1) - 1, (int)t)) goto done;
            tc_fence_after_sync();
            for (int kb = 0; kb < n_kb; ++kb, ++n) {
                const int stage = n % kGemmStages;
                if (!wait(kFull + stage, n / kGemmStages, (int)n)) goto done;
                tc_fence_after_sync();
                if (elected) {
                    const uint32_t a_lo = smem_desc_lo(smem_base + stage * kStageBytes, 16);
                    const uint32_t b_lo = smem_desc_lo(smem_base + stage * kStageBytes + kABytes, 16);
#pragma unroll
                    for (int kk = 0; kk < kBlockK / 16; ++kk)
                        mma_ss(tmem + buf * kTileN, smem_desc_join(a_lo + ((kk * 32) >> 4), hi),
                               smem_desc_join(b_lo + ((kk * 32) >> 4), hi), idesc, (kb > 0 || kk > 0) ? 1u : 0u);
                    tc_commit(bar(kEmpty + stage));
                    if (kb == n_kb - 1) tc_commit(bar(kAccFull + buf));
                }
                __syncwarp();
            }
        }
    } else if (warp >= 4) {
        // ---- epilogue: thread = one token row of one half (128 features) of the tile ----
        const int q4 = warp & 3, half = (warp - 4) >> 2;
        uint32_t t = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++t) {
            const uint32_t buf = t & 1u;
            const int m0 = (tile / p.n_tiles) * kTileM, n0 = (tile % p.n_tiles) * kTileN;
            if (!__all_sync(0xffffffffu, wait(kAccFull + buf, t >> 1, (int)t))) goto done;
            tc_fence_after_sync();
            const int token = m0 + 32 * q4 + lane;
            const float ssq = epilogue_half<D, TN>(p, tmem + buf * kTileN + ((uint32_t)(32 * q4) << 16), token, n0, half);
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kAccEmpty + buf));
            // the half's part of the row's sum of squares: one slot per token and half tile
            const int HD = p.heads * D;
            if (p.with_norm && n0 < 2 * HD && token < p.n_tokens) {
                const int which = n0 / HD;
                p.ssq[((size_t)which * p.n_tokens + token) * p.ssq_slots + 2 * ((n0 - which * HD) / kTileN) + half] = ssq;
            }
        }
    }
done:
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag == 1) {
        const uint64_t t0 = globaltimer_ns();
        while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 0) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(tmem, 512);
    }
}

// The norm's second step, one thread block per token: the row factors from the sums of squares
// per half tile (added in feature order), q's to q_row_scale, k's applied to the parked fp32
// row, which is rounded once to bf16 into the cache row.  One thread per 8 features.
__global__ void __launch_bounds__(1024)
qkv_finish_kernel(const __grid_constant__ QkvParams p)
{
    __shared__ float r_sh[2];
    const int HD = p.heads * p.head_dim;
    const int tiles = p.ssq_slots;
    const int token = blockIdx.x;
    if (threadIdx.x < 2) {
        const float *src = p.ssq + ((size_t)threadIdx.x * p.n_tokens + token) * tiles;
        float sum = 0.f;
        for (int t = 0; t < tiles; ++t) sum += src[t];
        r_sh[threadIdx.x] = 1.f / sqrtf(fmaf(sum, 1.f / (float)HD, p.eps));
    }
    __syncthreads();
    const float rk = r_sh[1];
    if (threadIdx.x == 0) p.q_row_scale[token] = r_sh[0];
    const int f0 = threadIdx.x * 8, head = f0 / p.head_dim, d0 = f0 % p.head_dim;
    const int frame = token / p.P, cell = token % p.P;
    const size_t cache_row = (size_t)p.slot[frame] * p.P + cell;
    const float4 *src = reinterpret_cast<const float4 *>(p.k_park + (size_t)token * HD + f0);
    const float4 a = src[0], b = src[1];
    *reinterpret_cast<uint4 *>(p.kcache + ((size_t)head * p.rows_per_head + cache_row) * p.head_dim + d0) =
        make_uint4(cvt_bf16x2(a.x * rk, a.y * rk), cvt_bf16x2(a.z * rk, a.w * rk), cvt_bf16x2(b.x * rk, b.y * rk),
                   cvt_bf16x2(b.z * rk, b.w * rk));
}

}  // namespace

cudaError_t launch_qkv_gemm(const QkvParams &p, const CUtensorMap &xmap, const CUtensorMap &wmap, int sm_count,
                            cudaStream_t stream)
{
    const int n_tiles = p.m_tiles * p.n_tiles;
    if (n_tiles <= 0) return cudaSuccess;
    const int grid = n_tiles < sm_count ? n_tiles : sm_count;
    cudaError_t e = cudaErrorInvalidValue;
#define LL_GEMM_CASE(DD, TT)                                                                                                  \
    if (p.head_dim == DD && p.tile_n == TT) {                                                                                  \
        e = cudaFuncSetAttribute(qkv_gemm_kernel<DD, TT>, cudaFuncAttributeMaxDynamicSharedMemorySize, GemmCfg<TT>::kSmem);   \
        if (e != cudaSuccess) return e;                                                                                        \
        qkv_gemm_kernel<DD, TT><<<grid, kGemmThreads, GemmCfg<TT>::kSmem, stream>>>(p, xmap, wmap);                            \
        e = cudaGetLastError();                                                                                                \
    }
    LL_GEMM_CASE(128, 256)
    LL_GEMM_CASE(128, 192)
    LL_GEMM_CASE(64, 256)
    LL_GEMM_CASE(64, 192)
#undef LL_GEMM_CASE
    count_launch();
    if (e != cudaSuccess || !p.with_norm) return e;
    qkv_finish_kernel<<<(unsigned)p.n_tokens, p.heads * p.head_dim / 8, 0, stream>>>(p);
    count_launch();
    return cudaGetLastError();
}

}  // namespace ll
