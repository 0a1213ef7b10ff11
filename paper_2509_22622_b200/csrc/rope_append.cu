// Fused 3-D RoPE + K/V append (HBM-bound).
//
// One thread owns one 16-byte vector (8 bf16 = 4 rotation pairs) of one token
// for a group of kHeadsPerThread heads: it fetches the four (cos, sin) pairs
// once (they depend on the token's (t, y, x) only, not on the head and not on
// Q vs K), then streams Q, K, V of its heads through registers.  All global
// accesses are 16-byte vectors; 16 consecutive threads cover one 256-byte head
// row, so reads of the token-major inputs and writes of the head-major cache
// rows are fully coalesced.
#include <cuda_bf16.h>

#include "ll_internal.h"
#include "rope_math.cuh"

namespace ll {

namespace {

constexpr int kHeadsPerThread = 4;
constexpr int kThreads = 256;

// fp64-accurate sine/cosine tables, rounded once to fp32.
//   t_tab[(f - t_base) * n_t + i] = (cos, sin)(f * theta^(-i/n_t))
//   h_tab[y * n_hw + i], w_tab[x * n_hw + i] likewise with n_hw pairs per axis
__global__ void rope_table_kernel(float2 *t_tab, long long t_base, int n_t_frames, int n_t,
                                  float2 *h_tab, int grid_h, float2 *w_tab, int grid_w, int n_hw,
                                  double theta, int do_t, int do_hw)
{
    const int n_tt = do_t ? n_t_frames * n_t : 0;
    const int n_hh = do_hw ? grid_h * n_hw : 0;
    const int n_ww = do_hw ? grid_w * n_hw : 0;
    for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < n_tt + n_hh + n_ww;
         idx += gridDim.x * blockDim.x) {
        double pos; int i, n_a; float2 *dst;
        if (idx < n_tt) {
            pos = (double)(t_base + idx / n_t); i = idx % n_t; n_a = n_t; dst = t_tab + idx;
        } else if (idx < n_tt + n_hh) {
            int j = idx - n_tt;
            pos = (double)(j / n_hw); i = j % n_hw; n_a = n_hw; dst = h_tab + j;
        } else {
            int j = idx - n_tt - n_hh;
            pos = (double)(j / n_hw); i = j % n_hw; n_a = n_hw; dst = w_tab + j;
        }
        double ang = pos * pow(theta, -(double)i / (double)n_a);
        double s, c;
        sincos(ang, &s, &c);
        *dst = make_float2((float)c, (float)s);
    }
}

__device__ __forceinline__ uint4 ld16(const ll_bf16 *p) { return *reinterpret_cast<const uint4 *>(p); }
__device__ __forceinline__ void st16(ll_bf16 *p, uint4 v) { *reinterpret_cast<uint4 *>(p) = v; }

__device__ __forceinline__ uint4 rotate_vec(uint4 x, const float2 (&cs)[4])
{
    return make_uint4(rotate_pair(x.x, cs[0]), rotate_pair(x.y, cs[1]),
                      rotate_pair(x.z, cs[2]), rotate_pair(x.w, cs[3]));
}

template <int D>
__global__ void __launch_bounds__(kThreads)
rope_append_kernel(const __grid_constant__ RopeAppendParams p)
{
    constexpr int kVecs = D / 8;                       // 16-byte vectors per head row
    const int head_groups = (p.heads + kHeadsPerThread - 1) / kHeadsPerThread;
    const long long gid = (long long)blockIdx.x * kThreads + threadIdx.x;
    const int vec = (int)(gid % kVecs);
    const long long rest = gid / kVecs;
    const int hg = (int)(rest % head_groups);
    const long long token = rest / head_groups;
    if (token >= p.n_tokens) return;

    const int frame = (int)(token / p.P);
    const int cell = (int)(token % p.P);
    const int y = cell / p.grid_w, x = cell % p.grid_w;
    if ((unsigned)p.slot[frame] >= (unsigned)p.n_slots) {         // never with the host's slot rule: refuse, report
        record_status(p.status, kStatusBadRow, (uint32_t)p.slot[frame], (uint32_t)frame);
        return;
    }

    float2 cs[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int j = vec * 4 + u;                     // rotation pair inside the head row
        const float2 *src;
        if (j < p.n_t)             src = p.t_tab + (size_t)frame * p.n_t + j;
        else if (j < p.n_t + p.n_h) src = p.h_tab + (size_t)y * p.n_h + (j - p.n_t);
        else                        src = p.w_tab + (size_t)x * p.n_h + (j - p.n_t - p.n_h);
        cs[u] = __ldg(src);
    }

    const int h0 = hg * kHeadsPerThread;
    const size_t in_base = ((size_t)token * p.heads + h0) * D + (size_t)vec * 8;
    const size_t cache_row = (size_t)p.slot[frame] * p.P + cell;

    uint4 kq[kHeadsPerThread], kk[kHeadsPerThread], kv[kHeadsPerThread];
#pragma unroll
    for (int u = 0; u < kHeadsPerThread; ++u) {
        if (h0 + u < p.heads) {
            kk[u] = ld16(p.k + in_base + (size_t)u * D);
            kv[u] = ld16(p.v + in_base + (size_t)u * D);
            if (p.q_out) kq[u] = ld16(p.q + in_base + (size_t)u * D);
        }
    }
#pragma unroll
    for (int u = 0; u < kHeadsPerThread; ++u) {
        if (h0 + u < p.heads) {
            const size_t dst = (((size_t)(h0 + u)) * p.rows_per_head + cache_row) * D + (size_t)vec * 8;
            st16(static_cast<ll_bf16 *>(p.kcache) + dst, rotate_vec(kk[u], cs));
            st16(static_cast<ll_bf16 *>(p.vcache) + dst, kv[u]);
            if (p.q_out) st16(p.q_out + in_base + (size_t)u * D, rotate_vec(kq[u], cs));
        }
    }
}

// ---- the same into an 8-bit cache ---------------------------------------------------------
//
// K (rotated, fp32) and V are divided by their head's scale (IEEE division) and rounded to
// E4M3, round to nearest even, saturating; a thread's eight elements make one 8-byte store, 16
// consecutive threads cover a 128-byte cache row.  Q is rotated to bf16 as in the bf16 kernel.
__device__ __forceinline__ uint2 quantise_vec(const float (&x)[8], float scale)
{
    uint32_t c[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) c[u] = cvt_e4m3x2(__fdiv_rn(x[2 * u], scale), __fdiv_rn(x[2 * u + 1], scale));
    return make_uint2(c[0] | (c[1] << 16), c[2] | (c[3] << 16));
}

template <int D>
__global__ void __launch_bounds__(kThreads)
rope_append_e4m3_kernel(const __grid_constant__ RopeAppendParams p)
{
    constexpr int kVecs = D / 8;
    const int head_groups = (p.heads + kHeadsPerThread - 1) / kHeadsPerThread;
    const long long gid = (long long)blockIdx.x * kThreads + threadIdx.x;
    const int vec = (int)(gid % kVecs);
    const long long rest = gid / kVecs;
    const int hg = (int)(rest % head_groups);
    const long long token = rest / head_groups;
    if (token >= p.n_tokens) return;

    const int frame = (int)(token / p.P);
    const int cell = (int)(token % p.P);
    const int y = cell / p.grid_w, x = cell % p.grid_w;
    if ((unsigned)p.slot[frame] >= (unsigned)p.n_slots) {         // never with the host's slot rule: refuse, report
        record_status(p.status, kStatusBadRow, (uint32_t)p.slot[frame], (uint32_t)frame);
        return;
    }
    float2 cs[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int j = vec * 4 + u;
        const float2 *src;
        if (j < p.n_t)             src = p.t_tab + (size_t)frame * p.n_t + j;
        else if (j < p.n_t + p.n_h) src = p.h_tab + (size_t)y * p.n_h + (j - p.n_t);
        else                        src = p.w_tab + (size_t)x * p.n_h + (j - p.n_t - p.n_h);
        cs[u] = __ldg(src);
    }
    const int h0 = hg * kHeadsPerThread;
    const size_t in_base = ((size_t)token * p.heads + h0) * D + (size_t)vec * 8;
    const size_t cache_row = (size_t)p.slot[frame] * p.P + cell;
    uint8_t *kc = static_cast<uint8_t *>(p.kcache), *vc = static_cast<uint8_t *>(p.vcache);
#pragma unroll
    for (int u = 0; u < kHeadsPerThread; ++u) {
        if (h0 + u >= p.heads) break;
        const uint4 k = ld16(p.k + in_base + (size_t)u * D);
        const uint4 v = ld16(p.v + in_base + (size_t)u * D);
        const uint32_t kw[4] = {k.x, k.y, k.z, k.w}, vw[4] = {v.x, v.y, v.z, v.w};
        float kr[8], vr[8];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            rotate_pair_f32(kw[t], cs[t], kr[2 * t], kr[2 * t + 1]);
            vr[2 * t] = __uint_as_float(vw[t] << 16);
            vr[2 * t + 1] = __uint_as_float(vw[t] & 0xffff0000u);
        }
        const size_t dst = (((size_t)(h0 + u)) * p.rows_per_head + cache_row) * D + (size_t)vec * 8;
        *reinterpret_cast<uint2 *>(kc + dst) = quantise_vec(kr, __ldg(p.k_scale + h0 + u));
        *reinterpret_cast<uint2 *>(vc + dst) = quantise_vec(vr, __ldg(p.v_scale + h0 + u));
        if (p.q_out) st16(p.q_out + in_base + (size_t)u * D, rotate_vec(ld16(p.q + in_base + (size_t)u * D), cs));
    }
}

// Codes of the listed cache-row runs, all heads, K and V: to bf16 at the same rows of the
// staging pair.  One thread converts 16 codes (one 16-byte load, two 16-byte stores).
template <int D>
__global__ void __launch_bounds__(kThreads)
stage_e4m3_kernel(const __grid_constant__ StageParams p)
{
    constexpr int kVecs = D / 16;                      // 16-code vectors per row
    long long gid = (long long)blockIdx.x * kThreads + threadIdx.x;
    const int vec = (int)(gid % kVecs);
    gid /= kVecs;
    int run = 0;
    long long rows_before = 0;
    // threads are numbered run by run, within a run head-major over its rows
    while (run < p.n_runs && gid >= rows_before + (long long)p.len[run] * p.heads) {
        rows_before += (long long)p.len[run] * p.heads;
        ++run;
    }
    if (run >= p.n_runs) return;
    const long long r = gid - rows_before;
    const int head = (int)(r / p.len[run]);
    const long long row = p.start[run] + r % p.len[run];
    const size_t off = ((size_t)head * p.rows_per_head + row) * D + (size_t)vec * 16;
    auto expand = [&](const uint8_t *src, ll_bf16 *dst) {
        const uint4 c = *reinterpret_cast<const uint4 *>(src + off);
        const uint32_t w[4] = {c.x, c.y, c.z, c.w};
        uint32_t o[8];
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            o[2 * t] = e4m3x2_to_bf16x2(w[t] & 0xffffu);
            o[2 * t + 1] = e4m3x2_to_bf16x2(w[t] >> 16);
        }
        st16(dst + off, make_uint4(o[0], o[1], o[2], o[3]));
        st16(dst + off + 8, make_uint4(o[4], o[5], o[6], o[7]));
    };
    expand(p.k8, p.k16);
    expand(p.v8, p.v16);
}

// ---- the same with the RMS norm of q and k in front -----------------------------------
//
// One warp owns one token.  Its lanes take the row's 16-byte vectors round-robin; a first
// pass over q and k sums the squares (fp32, then a butterfly over the warp), a second pass
// scales by the row's factor and the gain, rotates and stores.  Rows of up to 192 vectors
// (1536 elements at head_dim 128) stay in registers between the passes; longer ones are
// read again (from L1/L2).  The row stride in vectors (32) is a multiple of the vectors per head (8 or
// 16), so a lane meets the same four rotation pairs in every vector it owns and fetches
// their (cos, sin) once.
__device__ __forceinline__ float sum_squares(uint4 x)
{
    float s = 0.f;
    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const float a = __uint_as_float(w[u] << 16), b = __uint_as_float(w[u] & 0xffff0000u);
        s = fmaf(a, a, s);
        s = fmaf(b, b, s);
    }
    return s;
}

__device__ __forceinline__ uint32_t norm_rotate_pair(uint32_t packed, float r, float2 gain, float2 cs)
{
    const float a = __uint_as_float(packed << 16) * r * gain.x;
    const float b = __uint_as_float(packed & 0xffff0000u) * r * gain.y;
    const float r0 = fmaf(a, cs.x, -(b * cs.y));
    const float r1 = fmaf(a, cs.y, b * cs.x);
    __nv_bfloat162 o = __floats2bfloat162_rn(r0, r1);
    return *reinterpret_cast<uint32_t *>(&o);
}

__device__ __forceinline__ uint4 norm_rotate_vec(uint4 x, float r, const float *gain, const float2 (&cs)[4])
{
    const float4 g0 = *reinterpret_cast<const float4 *>(gain), g1 = *reinterpret_cast<const float4 *>(gain + 4);
    return make_uint4(norm_rotate_pair(x.x, r, make_float2(g0.x, g0.y), cs[0]),
                      norm_rotate_pair(x.y, r, make_float2(g0.z, g0.w), cs[1]),
                      norm_rotate_pair(x.z, r, make_float2(g1.x, g1.y), cs[2]),
                      norm_rotate_pair(x.w, r, make_float2(g1.z, g1.w), cs[3]));
}

// kIters > 0: the row's vectors fit kIters per lane and stay in registers between the two
// passes (one read of q, k, v from memory); kIters == 0: any row length, second pass re-reads.
template <int D, int kIters>
__global__ void __launch_bounds__(kThreads)
norm_rope_append_kernel(const __grid_constant__ RopeAppendParams p, const float *__restrict__ gain_q,
                        const float *__restrict__ gain_k, float eps)
{
    constexpr int kVecs = D / 8;                       // 16-byte vectors per head row
    static_assert(32 % kVecs == 0, "a lane must meet the same rotation pairs in all its vectors");
    constexpr int kHeld = kIters > 0 ? kIters : 1;
    const int lane = threadIdx.x & 31;
    const long long token = (long long)blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
    if (token >= p.n_tokens) return;
    const int row_vecs = p.heads * kVecs;
    const int frame = (int)(token / p.P);
    const int cell = (int)(token % p.P);
    const int y = cell / p.grid_w, x = cell % p.grid_w;
    if ((unsigned)p.slot[frame] >= (unsigned)p.n_slots) {         // never with the host's slot rule: refuse, report
        record_status(p.status, kStatusBadRow, (uint32_t)p.slot[frame], (uint32_t)frame);
        return;
    }
    const size_t in_base = (size_t)token * row_vecs * 8;
    const bool with_q = p.q_out != nullptr;

    uint4 hq[kHeld], hk[kHeld], hv[kHeld];
    float sq = 0.f, sk = 0.f;
    if (kIters > 0) {
#pragma unroll
        for (int i = 0; i < kHeld; ++i) {
            const int v = lane + 32 * i;
            if (v < row_vecs) {
                hk[i] = ld16(p.k + in_base + (size_t)v * 8);
                hv[i] = ld16(p.v + in_base + (size_t)v * 8);
                if (with_q) hq[i] = ld16(p.q + in_base + (size_t)v * 8);
            }
        }
#pragma unroll
        for (int i = 0; i < kHeld; ++i) {
            if (lane + 32 * i < row_vecs) {
                sk += sum_squares(hk[i]);
                if (with_q) sq += sum_squares(hq[i]);
            }
        }
    } else {
        for (int v = lane; v < row_vecs; v += 32) {
            sk += sum_squares(ld16(p.k + in_base + (size_t)v * 8));
            if (with_q) sq += sum_squares(ld16(p.q + in_base + (size_t)v * 8));
        }
    }
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) {
        sq += __shfl_xor_sync(0xffffffffu, sq, m);
        sk += __shfl_xor_sync(0xffffffffu, sk, m);
    }
    const float inv_n = 1.f / (float)(row_vecs * 8);
    const float rq = 1.f / sqrtf(fmaf(sq, inv_n, eps)), rk = 1.f / sqrtf(fmaf(sk, inv_n, eps));

    const int vec = lane % kVecs;                      // the lane's vector inside every head row it meets
    float2 cs[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int j = vec * 4 + u;
        const float2 *src;
        if (j < p.n_t)             src = p.t_tab + (size_t)frame * p.n_t + j;
        else if (j < p.n_t + p.n_h) src = p.h_tab + (size_t)y * p.n_h + (j - p.n_t);
        else                        src = p.w_tab + (size_t)x * p.n_h + (j - p.n_t - p.n_h);
        cs[u] = __ldg(src);
    }
    const size_t cache_row = (size_t)p.slot[frame] * p.P + cell;
    auto emit = [&](int v, uint4 xq, uint4 xk, uint4 xv) {
        const int head = v / kVecs;
        const size_t src = in_base + (size_t)v * 8;
        const size_t dst = ((size_t)head * p.rows_per_head + cache_row) * D + (size_t)vec * 8;
        st16(static_cast<ll_bf16 *>(p.kcache) + dst, norm_rotate_vec(xk, rk, gain_k + (size_t)v * 8, cs));
        st16(static_cast<ll_bf16 *>(p.vcache) + dst, xv);
        if (with_q) st16(p.q_out + src, norm_rotate_vec(xq, rq, gain_q + (size_t)v * 8, cs));
    };
    if (kIters > 0) {
#pragma unroll
        for (int i = 0; i < kHeld; ++i) {
            const int v = lane + 32 * i;
            if (v < row_vecs) emit(v, hq[i], hk[i], hv[i]);
        }
    } else {
        for (int v = lane; v < row_vecs; v += 32) {
            const size_t src = in_base + (size_t)v * 8;
            emit(v, with_q ? ld16(p.q + src) : make_uint4(0, 0, 0, 0), ld16(p.k + src), ld16(p.v + src));
        }
    }
}

template <int D>
void launch_norm_variant(const RopeAppendParams &p, const float *gain_q, const float *gain_k, float eps,
                         unsigned blocks, cudaStream_t stream)
{
    const int iters = (p.heads * (D / 8) + 31) / 32;
    if (iters <= 2)      norm_rope_append_kernel<D, 2><<<blocks, kThreads, 0, stream>>>(p, gain_q, gain_k, eps);
    else if (iters <= 4) norm_rope_append_kernel<D, 4><<<blocks, kThreads, 0, stream>>>(p, gain_q, gain_k, eps);
    else if (iters <= 6) norm_rope_append_kernel<D, 6><<<blocks, kThreads, 0, stream>>>(p, gain_q, gain_k, eps);
    else                 norm_rope_append_kernel<D, 0><<<blocks, kThreads, 0, stream>>>(p, gain_q, gain_k, eps);
}

}  // namespace

cudaError_t launch_norm_rope_append(const RopeAppendParams &p, int head_dim, const float *gain_q, const float *gain_k,
                                    float eps, cudaStream_t stream)
{
    const unsigned blocks = (unsigned)((p.n_tokens + kThreads / 32 - 1) / (kThreads / 32));
    if (blocks == 0) return cudaSuccess;
    if (head_dim == 128) launch_norm_variant<128>(p, gain_q, gain_k, eps, blocks, stream);
    else                 launch_norm_variant<64>(p, gain_q, gain_k, eps, blocks, stream);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_rope_tables(float2 *t_tab, int64_t t_base, int n_t_frames, int n_t, float2 *h_tab,
                               int grid_h, float2 *w_tab, int grid_w, int n_hw, float theta, bool do_t,
                               bool do_hw, cudaStream_t stream)
{
    int total = (do_t ? n_t_frames * n_t : 0) + (do_hw ? (grid_h + grid_w) * n_hw : 0);
    if (total == 0) return cudaSuccess;
    int blocks = (total + 127) / 128;
    rope_table_kernel<<<blocks, 128, 0, stream>>>(t_tab, (long long)t_base, n_t_frames, n_t, h_tab, grid_h,
                                                  w_tab, grid_w, n_hw, (double)theta, do_t, do_hw);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_rope_append_e4m3(const RopeAppendParams &p, int head_dim, cudaStream_t stream)
{
    const int head_groups = (p.heads + kHeadsPerThread - 1) / kHeadsPerThread;
    const long long threads = (long long)p.n_tokens * head_groups * (head_dim / 8);
    const unsigned blocks = (unsigned)((threads + kThreads - 1) / kThreads);
    if (blocks == 0) return cudaSuccess;
    if (head_dim == 128) rope_append_e4m3_kernel<128><<<blocks, kThreads, 0, stream>>>(p);
    else                 rope_append_e4m3_kernel<64><<<blocks, kThreads, 0, stream>>>(p);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_stage_e4m3(const StageParams &p, int head_dim, cudaStream_t stream)
{
    long long rows = 0;
    for (int i = 0; i < p.n_runs; ++i) rows += (long long)p.len[i] * p.heads;
    const long long threads = rows * (head_dim / 16);
    const unsigned blocks = (unsigned)((threads + kThreads - 1) / kThreads);
    if (blocks == 0) return cudaSuccess;
    if (head_dim == 128) stage_e4m3_kernel<128><<<blocks, kThreads, 0, stream>>>(p);
    else                 stage_e4m3_kernel<64><<<blocks, kThreads, 0, stream>>>(p);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_rope_append(const RopeAppendParams &p, int head_dim, cudaStream_t stream)
{
    const int head_groups = (p.heads + kHeadsPerThread - 1) / kHeadsPerThread;
    const long long threads = (long long)p.n_tokens * head_groups * (head_dim / 8);
    const unsigned blocks = (unsigned)((threads + kThreads - 1) / kThreads);
    if (blocks == 0) return cudaSuccess;
    if (head_dim == 128) rope_append_kernel<128><<<blocks, kThreads, 0, stream>>>(p);
    else                 rope_append_kernel<64><<<blocks, kThreads, 0, stream>>>(p);
    count_launch();
    return cudaGetLastError();
}

}  // namespace ll
