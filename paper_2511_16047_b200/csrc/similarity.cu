// Inter-scale key similarity (Sec. 4.3, Eq. 4): ss = || k_i - resize(k_{i-1}) ||^2.
//
// One thread per (item, output token, 8-channel chunk): it reads 16 bytes of the current
// scale's keys and the four bilinear neighbours from the previous scale (which is at most as
// large, so those reads are served by L1/L2 after the first touch), interpolates in fp32 and
// accumulates the squared differences.  Blocks reduce in fp64 into a partials array; a second
// single-block kernel adds the partials in a fixed order, so the result is reproducible.
#include <mutex>

#include "../../include/amskv.h"
#include "kernels.cuh"

namespace amskv {

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ void unpack8(const uint4& raw, float (&f)[8])
{
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 v = __bfloat1622float2(h[i]);
        f[2 * i] = v.x;
        f[2 * i + 1] = v.y;
    }
}

__device__ __forceinline__ double block_sum(double v, double* smem)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) smem[warp] = v;
    __syncthreads();
    double total = 0.0;
    if (threadIdx.x == 0)
        for (int w = 0; w < kThreads / 32; ++w) total += smem[w];
    return total;  // valid in thread 0
}

// source coordinate of output pixel i: (i + 0.5) * s_in / s_out - 0.5, clamped to [0, s_in - 1]
__device__ __forceinline__ void tap(int i, float ratio, int s_in, int& i0, int& i1, float& w)
{
    float f = ((float)i + 0.5f) * ratio - 0.5f;
    f = fminf(fmaxf(f, 0.f), (float)(s_in - 1));
    i0 = (int)floorf(f);
    i1 = min(i0 + 1, s_in - 1);
    w = f - (float)i0;
}

// Index is uint32_t whenever the chunk count allows it: the per-chunk index arithmetic (two divisions by
// run-time values) is what this kernel spends its instructions on, and 64-bit division costs several
// times the 32-bit one.
template <int D, typename Index>
__global__ void __launch_bounds__(kThreads)
similarity_partial_kernel(const uint4* __restrict__ K_prev, int32_t s_prev, const uint4* __restrict__ K_cur,
                          int32_t s_cur, int64_t total_chunks_, double* __restrict__ partials)
{
    const Index total_chunks = (Index)total_chunks_;
    constexpr int CPT = D / 8;
    __shared__ double smem[kThreads / 32];
    const float ratio = (float)s_prev / (float)s_cur;
    const int32_t t_cur = s_cur * s_cur, t_prev = s_prev * s_prev;
    double acc = 0.0;
    // Two chunks per thread and iteration, all ten loads issued before either is used: a thread's one
    // 16-byte HBM load per iteration would leave the memory system a third full.
    constexpr int kPer = 2;
    const Index stride = (Index)gridDim.x * kThreads;
    for (Index base = (Index)blockIdx.x * kThreads + threadIdx.x; base < total_chunks; base += kPer * stride) {
        uint4 cur[kPer], t00[kPer], t01[kPer], t10[kPer], t11[kPer];
        float wy[kPer], wx[kPer];
        bool live[kPer];
#pragma unroll
        for (int u = 0; u < kPer; ++u) {
            const Index idx = base + (Index)u * stride;
            live[u] = idx < total_chunks && idx >= base;   // (the second test catches wrap-around of a narrow index)
            const Index safe = live[u] ? idx : base;
            const Index tok_global = safe / CPT;
            const int32_t ch = (int32_t)(safe - tok_global * CPT);
            const Index item = tok_global / (Index)t_cur;
            const int32_t tok = (int32_t)(tok_global - item * (Index)t_cur);
            const int32_t y = tok / s_cur, x = tok - y * s_cur;
            int y0, y1, x0, x1;
            tap(y, ratio, s_prev, y0, y1, wy[u]);
            tap(x, ratio, s_prev, x0, x1, wx[u]);
            const uint4* P = K_prev + (int64_t)item * t_prev * CPT + ch;
            cur[u] = __ldcs(K_cur + safe);
            t00[u] = __ldg(P + (int64_t)(y0 * s_prev + x0) * CPT);
            t01[u] = __ldg(P + (int64_t)(y0 * s_prev + x1) * CPT);
            t10[u] = __ldg(P + (int64_t)(y1 * s_prev + x0) * CPT);
            t11[u] = __ldg(P + (int64_t)(y1 * s_prev + x1) * CPT);
        }
#pragma unroll
        for (int u = 0; u < kPer; ++u) {
            float c[8], v00[8], v01[8], v10[8], v11[8];
            unpack8(cur[u], c);
            unpack8(t00[u], v00);
            unpack8(t01[u], v01);
            unpack8(t10[u], v10);
            unpack8(t11[u], v11);
            float part = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const float top = v00[i] + wx[u] * (v01[i] - v00[i]);
                const float bot = v10[i] + wx[u] * (v11[i] - v10[i]);
                const float diff = c[i] - (top + wy[u] * (bot - top));
                part = fmaf(diff, diff, part);
            }
            if (live[u]) acc += (double)part;
        }
    }
    const double total = block_sum(acc, smem);
    if (threadIdx.x == 0) partials[blockIdx.x] = total;
}

__global__ void __launch_bounds__(kThreads)
similarity_final_kernel(const double* __restrict__ partials, int n, double* __restrict__ out)
{
    __shared__ double smem[kThreads / 32];
    double acc = 0.0;
    for (int i = threadIdx.x; i < n; i += kThreads) acc += partials[i];
    const double total = block_sum(acc, smem);
    if (threadIdx.x == 0) *out = total;
}

}  // namespace

cudaError_t launch_similarity(const __nv_bfloat16* K_prev, int32_t side_prev, const __nv_bfloat16* K_cur,
                              int32_t side_cur, int64_t items, int32_t D, double* out_ss, double* partials,
                              cudaStream_t stream)
{
    const int64_t total = items * side_cur * side_cur * (D / 8);
    int64_t blocks = (total + kThreads - 1) / kThreads;
    if (blocks > kSimilarityMaxBlocks) blocks = kSimilarityMaxBlocks;
    if (blocks < 1) blocks = 1;
    // the grid-stride loop adds gridDim * kThreads to an index below total: keep that sum inside 32 bits
    const bool narrow = total + 2ll * kSimilarityMaxBlocks * kThreads < (1ll << 32);
    const uint4* kp = (const uint4*)K_prev;
    const uint4* kc = (const uint4*)K_cur;
    if (D == 64) {
        if (narrow) similarity_partial_kernel<64, uint32_t><<<(unsigned)blocks, kThreads, 0, stream>>>(kp, side_prev, kc, side_cur, total, partials);
        else similarity_partial_kernel<64, int64_t><<<(unsigned)blocks, kThreads, 0, stream>>>(kp, side_prev, kc, side_cur, total, partials);
    } else {
        if (narrow) similarity_partial_kernel<128, uint32_t><<<(unsigned)blocks, kThreads, 0, stream>>>(kp, side_prev, kc, side_cur, total, partials);
        else similarity_partial_kernel<128, int64_t><<<(unsigned)blocks, kThreads, 0, stream>>>(kp, side_prev, kc, side_cur, total, partials);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    similarity_final_kernel<<<1, kThreads, 0, stream>>>(partials, (int)blocks, out_ss);
    count_launch(2);
    return cudaGetLastError();
}

}  // namespace amskv

// ---------------------------------------------------------------- entry point without allocation
//
// Scratch for the per-block partial sums of amskv_layer_similarity_static, resident in every
// device that loads this library until the process exits (16 KB).  In host code the name
// g_static_partials is only a stand-in for the symbol: it is never passed to a kernel.  The
// device address is looked up once per device with cudaGetSymbolAddress (below) and that
// pointer is what the kernels get.
namespace amskv {
namespace {

static __device__ __align__(256) double g_static_partials[kSimilarityMaxBlocks];

constexpr int kMaxDevices = 64;
// 16-byte chunks one call may cover: 2^30 chunks = 16 GiB of current-scale keys, which keeps
// every thread's grid-stride loop at or below 2048 iterations over the fixed 2048 partials.
constexpr int64_t kStaticMaxChunks = 1ll << 30;

std::mutex g_static_mutex;
double* g_static_addr[kMaxDevices] = {};

// Device address of g_static_partials on the current device; looked up on first use.
int static_partials(double** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { (void)cudaGetLastError(); return AMSKV_ERR_CUDA; }
    if (dev < 0 || dev >= kMaxDevices) return AMSKV_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_partials) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return AMSKV_ERR_CUDA;
        }
        g_static_addr[dev] = static_cast<double*>(p);
    }
    *out = g_static_addr[dev];
    return AMSKV_OK;
}

}  // namespace
}  // namespace amskv

extern "C" int amskv_layer_similarity_static(const void* K_prev, int side_prev, const void* K_cur, int side_cur,
                                             int rows, int heads, int head_dim, double* out_ss, void* stream)
{
    using namespace amskv;
    if (!K_prev || !K_cur || !out_ss) return AMSKV_ERR_INVALID;
    if ((reinterpret_cast<uintptr_t>(K_prev) & 15u) || (reinterpret_cast<uintptr_t>(K_cur) & 15u) ||
        (reinterpret_cast<uintptr_t>(out_ss) & 7u))
        return AMSKV_ERR_INVALID;
    if (side_prev < 1 || side_cur < 1 || side_prev > 4096 || side_cur > 4096 || rows < 1 || heads < 1)
        return AMSKV_ERR_INVALID;
    if (head_dim != 64 && head_dim != 128) return AMSKV_ERR_UNSUPPORTED;
    const int64_t items = (int64_t)rows * heads;
    const int64_t per_item = (int64_t)side_cur * side_cur * (head_dim / 8);
    if (items > kStaticMaxChunks / per_item) return AMSKV_ERR_UNSUPPORTED;  // beyond the stated maximum
    double* partials = nullptr;
    const int rc = static_partials(&partials);
    if (rc != AMSKV_OK) return rc;
    // Every partial the final kernel reads is written by the first kernel of the same call, so
    // nothing left in the array by an earlier call is ever read and nothing needs clearing.
    const cudaError_t e = launch_similarity((const __nv_bfloat16*)K_prev, side_prev, (const __nv_bfloat16*)K_cur,
                                            side_cur, items, head_dim, out_ss, partials,
                                            static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { (void)cudaGetLastError(); return AMSKV_ERR_CUDA; }
    return AMSKV_OK;
}
