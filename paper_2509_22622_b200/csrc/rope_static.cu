// ll_rope_q_static: the 3-D RoPE of a query tensor for callers that cannot
// allocate device memory.
//
// The other entry points keep their sine/cosine tables in the storage block the
// caller allocated and bound to a cache handle.  This one needs no handle and no
// storage: its tables live in a fixed array that is part of the library image,
// so every GPU that loads the library carries those 180 KB until the process
// exits.  Nothing on this path calls cudaMalloc, cudaFree or any routine that
// allocates.
//
// Sharing rules that follow from the fixed array:
//   - every call on a device writes its tables into the same array and then
//     reads them back in the rotation kernel, both on the caller's stream.  Two
//     calls that run at the same time on one GPU (different streams, or
//     different host threads without ordering) race on the tables;
//   - the array keeps whatever the previous call left.  Each call rewrites
//     every table entry it is going to read before reading it, so nothing in
//     the array has to start at zero.
#include <cuda_bf16.h>

#include <mutex>

#include "ll_internal.h"
#include "rope_math.cuh"

namespace {

// One frame-axis table for up to LL_STATIC_MAX_FRAMES frames of at most 24
// rotation pairs, then the row and column tables for up to
// LL_STATIC_MAX_GRID_SUM positions of at most 21 pairs (head_dim <= 128).
constexpr int kMaxTPairs = 24;
constexpr int kMaxHwPairs = 21;
constexpr int kTEntries = LL_STATIC_MAX_FRAMES * kMaxTPairs;
constexpr int kHwEntries = LL_STATIC_MAX_GRID_SUM * kMaxHwPairs;
constexpr int kMaxDevices = 64;

// In host code this name is only a handle for cudaGetSymbolAddress; it is not
// an address a kernel can be given.
static __device__ __align__(256) float2 g_rope_scratch[kTEntries + kHwEntries];

std::mutex g_setup_mutex;
float2 *g_scratch_addr[kMaxDevices];   // device address of g_rope_scratch, per device ordinal

// One thread rotates one 16-byte vector (4 pairs) of one head row of one token.  q_out may be
// q itself (each thread reads its vector before it writes it), so neither pointer is
// declared free of aliases.
template <int D>
__global__ void __launch_bounds__(256)
rope_q_static_kernel(const ll_bf16 *q, ll_bf16 *q_out, const float2 *t_tab,
                     const float2 *h_tab, const float2 *w_tab, long long n_tokens, int heads, int P, int grid_w,
                     int n_t, int n_h)
{
    constexpr int kVecs = D / 8;
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int vec = (int)(gid % kVecs);
    const long long row = gid / kVecs;                 // token * heads + head
    if (row >= n_tokens * heads) return;
    const long long token = row / heads;
    const int frame = (int)(token / P);
    const int cell = (int)(token % P);
    const int y = cell / grid_w, x = cell % grid_w;
    float2 cs[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int j = vec * 4 + u;
        const float2 *src;
        if (j < n_t)            src = t_tab + (size_t)frame * n_t + j;
        else if (j < n_t + n_h) src = h_tab + (size_t)y * n_h + (j - n_t);
        else                    src = w_tab + (size_t)x * n_h + (j - n_t - n_h);
        cs[u] = *src;
    }
    const size_t off = (size_t)row * D + (size_t)vec * 8;
    uint4 v = *reinterpret_cast<const uint4 *>(q + off);
    v.x = ll::rotate_pair(v.x, cs[0]);
    v.y = ll::rotate_pair(v.y, cs[1]);
    v.z = ll::rotate_pair(v.z, cs[2]);
    v.w = ll::rotate_pair(v.w, cs[3]);
    *reinterpret_cast<uint4 *>(q_out + off) = v;
}

}  // namespace

extern "C" int ll_rope_q_static(const ll_bf16 *q, ll_bf16 *q_out, int heads, int head_dim,
                                int64_t frame_start, int n_frames, int grid_h, int grid_w,
                                float rope_theta, ll_stream stream)
{
    auto fail = [](int code, const char *msg) {
        ll::set_last_error(msg);
        return code;
    };
    if (!q || !q_out) return fail(LL_ERR_INVALID_ARG, "null q or q_out");
    if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(q_out)) & 15u)
        return fail(LL_ERR_INVALID_ARG, "q and q_out must be 16-byte aligned");
    if (head_dim != 64 && head_dim != 128) return fail(LL_ERR_UNSUPPORTED_SHAPE, "head_dim must be 64 or 128");
    if (heads <= 0 || grid_h <= 0 || grid_w <= 0 || n_frames <= 0 || frame_start < 0 || !(rope_theta > 0.f))
        return fail(LL_ERR_INVALID_ARG, "non-positive size, negative frame_start or non-positive rope_theta");
    if (n_frames > LL_STATIC_MAX_FRAMES)
        return fail(LL_ERR_UNSUPPORTED_SHAPE, "n_frames exceeds LL_STATIC_MAX_FRAMES: the fixed table cannot hold it");
    if ((int64_t)grid_h + grid_w > LL_STATIC_MAX_GRID_SUM)
        return fail(LL_ERR_UNSUPPORTED_SHAPE,
                    "grid_h + grid_w exceeds LL_STATIC_MAX_GRID_SUM: the fixed table cannot hold it");
    if (frame_start + n_frames > INT32_MAX) return fail(LL_ERR_BAD_POSITION, "frame index exceeds int32");

    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(LL_ERR_CUDA, cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices) return fail(LL_ERR_CUDA, "device ordinal out of range");
    float2 *tab = nullptr;
    {
        // set-up, once per device and with that device current: ask the runtime where
        // this device's copy of the array lives
        std::lock_guard<std::mutex> lock(g_setup_mutex);
        if (!g_scratch_addr[dev]) {
            void *p = nullptr;
            e = cudaGetSymbolAddress(&p, g_rope_scratch);
            if (e != cudaSuccess) return fail(LL_ERR_CUDA, cudaGetErrorString(e));
            g_scratch_addr[dev] = static_cast<float2 *>(p);
        }
        tab = g_scratch_addr[dev];
    }

    const int n_h = head_dim / 6;
    const int n_t = head_dim / 2 - 2 * n_h;
    float2 *t_tab = tab;
    float2 *h_tab = tab + kTEntries;
    float2 *w_tab = h_tab + (size_t)grid_h * n_h;
    cudaStream_t s = (cudaStream_t)stream;
    e = ll::launch_rope_tables(t_tab, frame_start, n_frames, n_t, h_tab, grid_h, w_tab, grid_w, n_h, rope_theta,
                               true, true, s);
    if (e != cudaSuccess) return fail(LL_ERR_CUDA, cudaGetErrorString(e));
    const int P = grid_h * grid_w;
    const long long n_tokens = (long long)n_frames * P;
    const long long threads = n_tokens * heads * (head_dim / 8);
    const unsigned blocks = (unsigned)((threads + 255) / 256);
    if (head_dim == 128)
        rope_q_static_kernel<128><<<blocks, 256, 0, s>>>(q, q_out, t_tab, h_tab, w_tab, n_tokens, heads, P, grid_w, n_t, n_h);
    else
        rope_q_static_kernel<64><<<blocks, 256, 0, s>>>(q, q_out, t_tab, h_tab, w_tab, n_tokens, heads, P, grid_w, n_t, n_h);
    ll::count_launch();
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(LL_ERR_CUDA, cudaGetErrorString(e));
    return LL_OK;
}
