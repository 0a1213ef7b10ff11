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

// Rotate one packed pair (lo = element 2j, hi = element 2j+1) in fp32.
__device__ __forceinline__ uint32_t rotate_pair(uint32_t packed, float2 cs)
{
    float a = __uint_as_float(packed << 16);
    float b = __uint_as_float(packed & 0xffff0000u);
    float r0 = fmaf(a, cs.x, -(b * cs.y));
    float r1 = fmaf(a, cs.y, b * cs.x);
    __nv_bfloat162 o = __floats2bfloat162_rn(r0, r1);   // .x (low half) = r0
    return *reinterpret_cast<uint32_t *>(&o);
}

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
            st16(p.kcache + dst, rotate_vec(kk[u], cs));
            st16(p.vcache + dst, kv[u]);
            if (p.q_out) st16(p.q_out + in_base + (size_t)u * D, rotate_vec(kq[u], cs));
        }
    }
}

}  // namespace

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
