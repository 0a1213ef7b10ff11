// Sink+window attention on tcgen05 tensor cores (sm_100a).
//
// One CTA owns up to 256 query rows of one head (two 128-row MMA tiles) and
// streams that head's visible cache rows past them in 128-key tiles:
//
//   warp 8  (one lane)  TMA producer: Q tiles once, then K_0 V_0 K_1 V_1 ... into a
//                       ring of 128-byte-swizzled shared-memory stages
//   warp 9  (one lane)  MMA issuer: S_w = Q_w K_j^T (operands in shared memory,
//                       accumulator in TMEM), O_w += P_w V_j (P read from TMEM)
//   warps 0-3 / 4-7     softmax warpgroup of query tile 0 / 1: one thread per
//                       query row reads its S row from TMEM, keeps the running
//                       max and sum in fp32, writes P (bf16) back over S, and
//                       rescales O in TMEM only when the max moved by > 2^8
//
// While one warpgroup runs its softmax the tensor pipe works on the other
// tile's MMAs.  TMEM columns: S_0 | S_1 | O_0 | O_1 (fp32), P_w aliases the
// first half of S_w.  The visible keys are a short list of contiguous cache-row
// runs (sink, ring, wrapped ring); softmax does not care about key order, so
// the only masking is the ragged last tile of each run.
//
// Every wait is bounded: a role that waits longer than kWaitLimitNs records a
// status word, raises the CTA's abort flag, and all roles drain to the common
// exit where TMEM is released.
#include <cuda_bf16.h>

#include "ll_internal.h"
#include "ptx.cuh"

namespace ll {

namespace {

using namespace ptx;

constexpr int kThreads = 384;
constexpr int kTmaWarp = 8;
constexpr int kMmaWarp = 9;
constexpr uint64_t kWaitLimitNs = 2000000000ull;    // 2 s
constexpr float kRescaleThreshold = 8.f;            // log2 units
// 384 threads start with 168 registers each; (2 * 224 + 56) * 128 is the same total
constexpr int kSoftmaxRegs = 224;
constexpr int kProducerRegs = 56;

template <int D>
struct Cfg {
    static constexpr int kAtoms = D / 64;                   // 128-byte swizzle atoms per row
    static constexpr int kAtomBytes = 128 * 128;            // 128 rows x 128 bytes
    static constexpr int kTileBytes = kAtoms * kAtomBytes;  // one 128-row tile of Q, K or V
    static constexpr int kStages = (D == 128) ? 5 : 8;
    static constexpr int kSmemTiles = (2 + kStages) * kTileBytes;
    static constexpr int kSmemBytes = kSmemTiles + 1024 /*barriers*/ + 1024 /*alignment slack*/;
    static constexpr int kTmemCols = 512;
    static constexpr int kColS = 0;                         // S_w at kColS + 128 w
    static constexpr int kColO = 256;                       // O_w at kColO + D w
};

// barrier indices inside the shared barrier array
enum Bar { kQFull = 0, kSFull = 2, kPFull = 4, kOFull = 6, kKvFull = 8 /* + stage */, kKvEmpty = 24 /* + stage */, kNumBars = 40 };

// Walks the visible key tiles of a group: runs in order, 128 rows at a time.
struct KeyIter {
    const AttnGroup *g;
    int r, off;
    __device__ KeyIter(const AttnGroup *grp) : g(grp), r(0), off(0) {}
    __device__ int row() const { return g->k_start[r] + off; }
    __device__ int valid() const { return min(kKeyTile, g->k_len[r] - off); }
    __device__ void next()
    {
        off += kKeyTile;
        if (off >= g->k_len[r]) { ++r; off = 0; }
    }
};

__device__ int count_key_tiles(const AttnGroup &g)
{
    int n = 0;
    for (int r = 0; r < g.n_ranges; ++r) n += (g.k_len[r] + kKeyTile - 1) / kKeyTile;
    return n;
}

struct WaitCtx {
    volatile int *abort_flag;
    uint32_t *status;
    int role;
};

// Bounded wait on an mbarrier phase.  Returns false when the CTA is aborting.
__device__ __forceinline__ bool wait_slow(uint32_t bar, uint32_t parity, const WaitCtx &ctx, int bar_id, int iter)
{
    const uint64_t t0 = globaltimer_ns();
    uint32_t spins = 0;
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 63u) == 0) {
            if (*ctx.abort_flag) return false;
            if (globaltimer_ns() - t0 > kWaitLimitNs) {
                *ctx.abort_flag = 1;
                if (atomicCAS(ctx.status, 0u, (uint32_t)kStatusTimeout) == 0u) {
                    ctx.status[1] = (uint32_t)ctx.role;
                    ctx.status[2] = (uint32_t)bar_id;
                    ctx.status[3] = (uint32_t)iter;
                    ctx.status[4] = blockIdx.x; ctx.status[5] = blockIdx.y; ctx.status[6] = blockIdx.z;
                    __threadfence();
                }
                return false;
            }
        }
    }
}

__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, const WaitCtx &ctx, int bar_id, int iter)
{
    if (mbar_try_wait(bar, parity)) return true;
    return wait_slow(bar, parity, ctx, bar_id, iter);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&t);
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
attn_sm100_kernel(const __grid_constant__ AttnParams p, const __grid_constant__ CUtensorMap qmap,
                  const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap)
{
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t q_smem = smem_base;                                  // 2 tiles
    const uint32_t kv_smem = smem_base + 2 * C::kTileBytes;             // kStages tiles
    const uint32_t bars = smem_base + C::kSmemTiles;                    // kNumBars x 8 bytes
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem_gen + C::kSmemTiles + kNumBars * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    auto bar = [&](int i) -> uint32_t { return bars + 8u * (uint32_t)i; };

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int head = blockIdx.y;

    // ---- which query rows and which keys ----------------------------------
    int g = 0;
    while (g + 1 < p.n_groups && (int)blockIdx.x >= p.g[g + 1].tile_begin) ++g;
    const AttnGroup &G = p.g[g];
    const int local_tile = blockIdx.x - G.tile_begin;
    const int q0 = G.q_begin + local_tile * kQTileRows;                  // first query row of the CTA
    const int rows_valid = min(kQTileRows, G.q_rows - local_tile * kQTileRows);
    const int n_sub = rows_valid > 128 ? 2 : 1;                          // live 128-row tiles
    const int n_kt = count_key_tiles(G);

    // ---- setup ------------------------------------------------------------------
    if (threadIdx.x == 0) {
        for (int i = 0; i < kNumBars; ++i) {
            uint32_t count = 1;
            if (i == kPFull || i == kPFull + 1) count = 128;
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

    // Register reallocation: the softmax warpgroups hold a whole S row per thread, the
    // producer warpgroup (TMA, MMA and two idle warps) needs little.
    if (warp >= 8) {
        setmaxnreg_dec<kProducerRegs>();
    if (skip) {
        // an earlier CTA gave up: nothing to do
    } else if (warp == kTmaWarp) {
        // =========================== TMA producer ===========================
        if (lane == 0) {
            prefetch_tensormap(&qmap);
            prefetch_tensormap(&kmap);
            prefetch_tensormap(&vmap);
            for (int w = 0; w < n_sub; ++w) {
                mbar_arrive_expect_tx(bar(kQFull + w), C::kTileBytes);
                for (int a = 0; a < C::kAtoms; ++a)
                    tma_load_3d(q_smem + w * C::kTileBytes + a * C::kAtomBytes, &qmap, bar(kQFull + w),
                                a * 64, head, q0 + 128 * w);
            }
            KeyIter it(&G);
            bool ok = true;
            for (int j = 0; j < n_kt && ok; ++j, it.next()) {
                const int row = it.row();
                for (int kv = 0; kv < 2 && ok; ++kv) {
                    const int n = 2 * j + kv;
                    const int stage = n % C::kStages;
                    const uint32_t phase = (uint32_t)(n / C::kStages) & 1u;
                    ok = wait_bar(bar(kKvEmpty + stage), phase ^ 1u, ctx, kKvEmpty + stage, n);
                    if (!ok) break;
                    mbar_arrive_expect_tx(bar(kKvFull + stage), C::kTileBytes);
                    const CUtensorMap *m = kv ? &vmap : &kmap;
                    for (int a = 0; a < C::kAtoms; ++a)
                        tma_load_3d(kv_smem + stage * C::kTileBytes + a * C::kAtomBytes, m,
                                    bar(kKvFull + stage), a * 64, row, head);
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // ============================ MMA issuer ============================
        if (lane == 0) {
            constexpr uint32_t idesc_qk = idesc_bf16_f32(128, 128, 0, 0);
            constexpr uint32_t idesc_pv = idesc_bf16_f32(128, D, 0, 1);
            // S_w = Q_w K^T: both operands K-major, 64-element atoms, 16 elements (32 bytes) per MMA
            auto issue_qk = [&](int w, int stage) {
                const uint32_t qa = q_smem + w * C::kTileBytes;
                const uint32_t kb = kv_smem + stage * C::kTileBytes;
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (kk / 4) * C::kAtomBytes + (kk % 4) * 32;
                    mma_ss(tmem + C::kColS + 128 * w, smem_desc_sw128(qa + off, 16, 1024),
                           smem_desc_sw128(kb + off, 16, 1024), idesc_qk, kk > 0);
                }
            };
            // O_w += P_w V: P from TMEM (16 keys = 8 packed columns per MMA); V is MN-major:
            // 8-key groups 1024 bytes apart, 64-wide d atoms kAtomBytes apart
            auto issue_pv = [&](int w, int stage, bool first) {
                const uint32_t vb = kv_smem + stage * C::kTileBytes;
#pragma unroll
                for (int kk = 0; kk < kKeyTile / 16; ++kk) {
                    mma_ts(tmem + C::kColO + D * w, tmem + C::kColS + 128 * w + 8 * kk,
                           smem_desc_sw128(vb + kk * 2048, C::kAtomBytes, 1024), idesc_pv,
                           (!first || kk > 0) ? 1u : 0u);
                }
            };
            bool ok = true;
            for (int w = 0; w < n_sub && ok; ++w) ok = wait_bar(bar(kQFull + w), 0, ctx, kQFull + w, 0);
            if (ok) ok = wait_bar(bar(kKvFull + 0), 0, ctx, kKvFull, 0);
            if (ok) {
                tc_fence_after_sync();
                for (int w = 0; w < n_sub; ++w) {
                    issue_qk(w, 0);
                    tc_commit(bar(kSFull + w));
                }
                tc_commit(bar(kKvEmpty + 0));
            }
            for (int j = 0; j < n_kt && ok; ++j) {
                const int nv = 2 * j + 1, nk = 2 * j + 2;
                const int sv = nv % C::kStages, sk = nk % C::kStages;
                const bool more = j + 1 < n_kt;
                ok = wait_bar(bar(kKvFull + sv), (uint32_t)(nv / C::kStages) & 1u, ctx, kKvFull + sv, nv);
                if (ok && more) ok = wait_bar(bar(kKvFull + sk), (uint32_t)(nk / C::kStages) & 1u, ctx, kKvFull + sk, nk);
                for (int w = 0; w < n_sub && ok; ++w) {
                    ok = wait_bar(bar(kPFull + w), (uint32_t)j & 1u, ctx, kPFull + w, j);
                    if (!ok) break;
                    tc_fence_after_sync();
                    issue_pv(w, sv, j == 0);
                    if (more) {
                        issue_qk(w, sk);
                        tc_commit(bar(kSFull + w));
                    } else {
                        tc_commit(bar(kOFull + w));
                    }
                }
                if (ok) {
                    tc_commit(bar(kKvEmpty + sv));
                    if (more) tc_commit(bar(kKvEmpty + sk));
                }
            }
        }
    }
    } else {
        // ========================= softmax warpgroups =========================
        setmaxnreg_inc<kSoftmaxRegs>();
        const int w = warp >> 2;                       // query tile of this warpgroup
        if (!skip && w < n_sub) {
            const int r = threadIdx.x & 127;           // row inside the tile = TMEM lane
            const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
            const uint32_t t_s = tmem + lane_base + C::kColS + 128 * w;
            const uint32_t t_o = tmem + lane_base + C::kColO + D * w;
            const float c = p.scale_log2;
            float m = -INFINITY, l = 0.f;
            KeyIter it(&G);
            bool ok = true;
            for (int j = 0; j < n_kt; ++j, it.next()) {
                ok = __all_sync(0xffffffffu, wait_bar(bar(kSFull + w), (uint32_t)j & 1u, ctx, kSFull + w, j));
                if (!ok) break;
                tc_fence_after_sync();
                const int nvalid = it.valid();
                // ---- pass 1: row max of the tile (the values are fetched again below) ----
                float m_tile;
                uint32_t ca[32], cb[32];
                {
                    uint32_t v[128];
#pragma unroll
                    for (int i = 0; i < 4; ++i) tmem_ld32(t_s + 32 * i, v + 32 * i);
                    tmem_wait_ld();
                    tmem_ld32(t_s, ca);                    // chunk 0 of pass 2, in flight during the max
                    if (nvalid < kKeyTile) {
#pragma unroll
                        for (int i = 0; i < 128; ++i)
                            if (i >= nvalid) v[i] = 0xff800000u;   // -inf
                    }
                    float mc[4];
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        mc[ch] = fmaxf(__uint_as_float(v[32 * ch]), __uint_as_float(v[32 * ch + 1]));
#pragma unroll
                        for (int i = 2; i < 32; i += 2)
                            mc[ch] = max3(mc[ch], __uint_as_float(v[32 * ch + i]), __uint_as_float(v[32 * ch + i + 1]));
                    }
                    m_tile = max3(mc[0], mc[1], fmaxf(mc[2], mc[3])) * c;
                }
                if (j == 0) {
                    m = m_tile;
                } else {
                    const bool grow = m_tile > m + kRescaleThreshold;
                    if (__any_sync(0xffffffffu, grow)) {
                        // rescale the running sum and the O row; PV of tile j-1 has completed
                        // (the commit that released S_j covers it) and PV of tile j is not issued yet
                        const float alpha = grow ? ex2(m - m_tile) : 1.f;
                        if (grow) m = m_tile;
                        l *= alpha;
#pragma unroll
                        for (int i = 0; i < D / 32; ++i) {
                            uint32_t o[32];
                            tmem_ld32(t_o + 32 * i, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int u = 0; u < 32; ++u) o[u] = __float_as_uint(__uint_as_float(o[u]) * alpha);
                            tmem_st32(t_o + 32 * i, o);
                        }
                    }
                }
                // ---- pass 2: p = 2^(s*c - m) in 32-key chunks; P chunk k (16 packed columns)
                //      lands on S columns that chunks <= k no longer need ----
                const uint64_t c2 = pack2(c, c);
                const uint64_t nm2 = pack2(-m, -m);
                uint64_t acc[2] = {0ull, 0ull};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    uint32_t *cur = (k & 1) ? cb : ca;
                    uint32_t *nxt = (k & 1) ? ca : cb;
                    tmem_wait_ld();
                    if (k < 3) tmem_ld32(t_s + 32 * (k + 1), nxt);
                    if (nvalid < kKeyTile) {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (32 * k + i >= nvalid) cur[i] = 0xff800000u;
                    }
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const uint64_t t2 = fma2(pack2(__uint_as_float(cur[2 * i]), __uint_as_float(cur[2 * i + 1])), c2, nm2);
                        float t0, t1;
                        unpack2(t2, t0, t1);
                        const float p0 = ex2(t0), p1 = ex2(t1);
                        acc[i & 1] = add2(acc[i & 1], pack2(p0, p1));
                        pk[i] = pack_bf16(p0, p1);         // key 2i in the low half
                    }
                    tmem_st16(t_s + 16 * k, pk);
                }
                float sum0, sum1;
                unpack2(add2(acc[0], acc[1]), sum0, sum1);
                l += sum0 + sum1;
                tmem_wait_st();
                tc_fence_before_sync();
                mbar_arrive(bar(kPFull + w));
            }
            // ---- epilogue: O / l -> bf16 -> global ---------------------------
            if (ok) ok = __all_sync(0xffffffffu, wait_bar(bar(kOFull + w), 0, ctx, kOFull + w, n_kt));
            if (ok) {
                tc_fence_after_sync();
                const int row = 128 * w + r;
                const bool live = row < rows_valid;
                const float inv_l = 1.f / l;
                ll_bf16 *dst = p.out + ((size_t)(q0 + row) * p.heads + head) * D;
#pragma unroll
                for (int i = 0; i < D / 32; ++i) {
                    uint32_t o[32];
                    tmem_ld32(t_o + 32 * i, o);
                    tmem_wait_ld();
                    if (live) {
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            uint4 pk;
                            pk.x = pack_bf16(__uint_as_float(o[8 * u + 0]) * inv_l, __uint_as_float(o[8 * u + 1]) * inv_l);
                            pk.y = pack_bf16(__uint_as_float(o[8 * u + 2]) * inv_l, __uint_as_float(o[8 * u + 3]) * inv_l);
                            pk.z = pack_bf16(__uint_as_float(o[8 * u + 4]) * inv_l, __uint_as_float(o[8 * u + 5]) * inv_l);
                            pk.w = pack_bf16(__uint_as_float(o[8 * u + 6]) * inv_l, __uint_as_float(o[8 * u + 7]) * inv_l);
                            *reinterpret_cast<uint4 *>(dst + 32 * i + 8 * u) = pk;
                        }
                    }
                }
                if (live && p.lse)
                    p.lse[(size_t)head * p.nq_total + q0 + row] = (m + log2f(l)) * 0.6931471805599453f;
            }
        }
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

}  // namespace

cudaError_t launch_attn_sm100(const AttnParams &p, int head_dim, const CUtensorMap &qmap, const CUtensorMap &kmap,
                              const CUtensorMap &vmap, cudaStream_t stream)
{
    dim3 grid((unsigned)p.total_qtiles, (unsigned)p.heads);
    cudaError_t e;
    if (head_dim == 128) {
        e = cudaFuncSetAttribute(attn_sm100_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<128>::kSmemBytes);
        if (e != cudaSuccess) return e;
        attn_sm100_kernel<128><<<grid, kThreads, Cfg<128>::kSmemBytes, stream>>>(p, qmap, kmap, vmap);
    } else {
        e = cudaFuncSetAttribute(attn_sm100_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<64>::kSmemBytes);
        if (e != cudaSuccess) return e;
        attn_sm100_kernel<64><<<grid, kThreads, Cfg<64>::kSmemBytes, stream>>>(p, qmap, kmap, vmap);
    }
    count_launch();
    return cudaGetLastError();
}

}  // namespace ll
