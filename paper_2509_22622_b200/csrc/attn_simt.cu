// Test-only triage kernel: sink+window attention with plain fp32 FMAs, one
// thread block per (query row, head).  It reads the same launch parameters as
// the tensor-core kernel, so a disagreement between the two isolates a fault to
// the tensor-core data path rather than to the cache layout or the visible
// ranges.  The library's compute calls never dispatch to it.
#include <cuda_bf16.h>

#include "ll_internal.h"

namespace ll {

namespace {

constexpr int kThreads = 128;

__device__ __forceinline__ float bf16_bits_to_float(ll_bf16 b) { return __uint_as_float((uint32_t)b << 16); }

template <int D>
__global__ void __launch_bounds__(kThreads)
attn_simt_kernel(const __grid_constant__ AttnParams p)
{
    __shared__ float q_s[D];
    __shared__ float s_s[kThreads];
    __shared__ float red[kThreads / 32];

    const int row = blockIdx.x;
    const int head = blockIdx.y;
    const int tid = threadIdx.x;

    int g = 0;
    while (g + 1 < p.n_groups && row >= p.g[g + 1].q_begin) ++g;
    const AttnGroup &G = p.g[g];

    const ll_bf16 *qrow = p.q + ((size_t)row * p.heads + head) * D;
    for (int d = tid; d < D; d += kThreads) q_s[d] = bf16_bits_to_float(qrow[d]);
    __syncthreads();

    const ll_bf16 *K = p.kbase + (size_t)head * p.rows_per_head * D;
    const ll_bf16 *V = p.vbase + (size_t)head * p.rows_per_head * D;

    float m = -INFINITY, l = 0.f, acc = 0.f;     // thread `tid` owns output dim tid (tid < D)
    for (int r = 0; r < G.n_ranges; ++r) {
        for (int j0 = 0; j0 < G.k_len[r]; j0 += kThreads) {
            const int j = j0 + tid;
            float s = -INFINITY;
            if (j < G.k_len[r]) {
                const ll_bf16 *krow = K + (size_t)(G.k_start[r] + j) * D;
                float dot = 0.f;
                for (int d = 0; d < D; d += 8) {
                    uint4 kk = *reinterpret_cast<const uint4 *>(krow + d);
                    const uint32_t w[4] = {kk.x, kk.y, kk.z, kk.w};
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        dot = fmaf(q_s[d + 2 * u], __uint_as_float(w[u] << 16), dot);
                        dot = fmaf(q_s[d + 2 * u + 1], __uint_as_float(w[u] & 0xffff0000u), dot);
                    }
                }
                s = dot * p.scale_log2;              // scores in log2 units
            }
            // block max of this tile
            float mx = s;
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            if ((tid & 31) == 0) red[tid >> 5] = mx;
            __syncthreads();
            mx = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
            const float m_new = fmaxf(m, mx);
            const float alpha = exp2f(m - m_new);    // 0 on the first tile (m = -inf)
            const float pj = exp2f(s - m_new);       // 0 for masked keys
            s_s[tid] = pj;
            __syncthreads();
            const int n_here = min(kThreads, G.k_len[r] - j0);
            float lsum = 0.f, a = 0.f;
            for (int t = 0; t < n_here; ++t) {
                const float pt = s_s[t];
                lsum += pt;
                if (tid < D) a = fmaf(pt, bf16_bits_to_float(V[(size_t)(G.k_start[r] + j0 + t) * D + tid]), a);
            }
            l = l * alpha + lsum;
            acc = acc * alpha + a;
            m = m_new;
            __syncthreads();
        }
    }
    if (tid < D) {
        p.out[((size_t)row * p.heads + head) * D + tid] = __bfloat16_as_ushort(__float2bfloat16_rn(acc / l));
    }
    if (tid == 0 && p.lse) p.lse[(size_t)head * p.nq_total + row] = (m + log2f(l)) * 0.6931471805599453f;
}

}  // namespace

cudaError_t launch_attn_simt(const AttnParams &p, int head_dim, cudaStream_t stream)
{
    dim3 grid((unsigned)p.nq_total, (unsigned)p.heads);
    if (head_dim == 128) attn_simt_kernel<128><<<grid, kThreads, 0, stream>>>(p);
    else                 attn_simt_kernel<64><<<grid, kThreads, 0, stream>>>(p);
    count_launch();
    return cudaGetLastError();
}

}  // namespace ll
