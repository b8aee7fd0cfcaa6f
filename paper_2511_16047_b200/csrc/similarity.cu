// Inter-scale key similarity (Sec. 4.3, Eq. 4): ss = || k_i - resize(k_{i-1}) ||^2.
//
// One thread per (item, output token, 16-channel piece): it reads 32 bytes of the current
// scale's keys and the four bilinear neighbours from the previous scale (which is at most as
// large, so those reads are served by L1/L2 after the first touch), interpolates in fp32 and
// accumulates the squared differences (fp32 over the 16 channels of a thread's piece, fp64 beyond).
// Blocks reduce in fp64 into a partials array; a second single-block kernel adds the partials
// in a fixed order, so the result is reproducible.
#include <mutex>

#include "../../include/amskv.h"
#include "kernels.cuh"

namespace amskv {

namespace {

constexpr int kThreads = 256;

// A bf16 is the upper half of the fp32 with the same value: each 32-bit word holds two of them, widened
// by one shift (the low one) and one mask (the high one).
__device__ __forceinline__ void unpack8(const uint4& raw, float (&f)[8])
{
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

// d = a * b + c on two packed fp32 lanes (one instruction on sm_100)
__device__ __forceinline__ void fma2(float& d0, float& d1, float a0, float a1, float b0, float b1, float c0, float c1)
{
    asm("{\n"
        ".reg .b64 ra, rb, rc, rd;\n"
        "mov.b64 ra, {%2, %3};\n"
        "mov.b64 rb, {%4, %5};\n"
        "mov.b64 rc, {%6, %7};\n"
        "fma.rn.f32x2 rd, ra, rb, rc;\n"
        "mov.b64 {%0, %1}, rd;\n"
        "}\n"
        : "=f"(d0), "=f"(d1)
        : "f"(a0), "f"(a1), "f"(b0), "f"(b1), "f"(c0), "f"(c1));
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

// Work is cut into units of (item, part of the item's chunks), one unit per block iteration, so that the
// per-chunk index arithmetic has no run-time division: the token is a shift of the chunk index, its row
// comes from a multiplication by a precomputed reciprocal (exact for every token index below 2^24 and
// side up to 4096: y = (tok * ceil(2^36 / s)) >> 36), and the one division per unit is by the number of
// parts.  The interpolation uses the four tap weights directly: diff = c - sum_j w_j v_j, four
// multiply-adds per channel.
template <int D>
__global__ void __launch_bounds__(kThreads)
similarity_partial_kernel(const uint4* __restrict__ K_prev, int32_t s_prev, const uint4* __restrict__ K_cur,
                          int32_t s_cur, int64_t items, int64_t units, int32_t parts, int32_t part_chunks,
                          int32_t items_per_unit, uint64_t inv_s_cur, double* __restrict__ partials)
{
    constexpr int CPT = D / 16;                      // 32-byte pieces per token; a thread takes one piece at a time
    constexpr int kShift = (D == 64) ? 2 : 3;
    __shared__ double smem[kThreads / 32];
    const float ratio = (float)s_prev / (float)s_cur;
    const int32_t t_cur = s_cur * s_cur, t_prev = s_prev * s_prev;
    const int32_t item_chunks = t_cur * CPT;
    double acc = 0.0;
    for (int64_t unit = blockIdx.x; unit < units; unit += gridDim.x) {
        int64_t item;
        int32_t end, first;
        if (items_per_unit > 1) {
            // coarse scales: an item has fewer pieces than the block has threads, so a unit is several items
            const int32_t sub = (int32_t)threadIdx.x / item_chunks;
            item = unit * items_per_unit + sub;
            end = (sub < items_per_unit && item < items) ? item_chunks : 0;
            first = (int32_t)threadIdx.x - sub * item_chunks;
            if (end == 0) item = 0;
        } else {
            item = unit / parts;
            const int32_t part = (int32_t)(unit - item * parts);
            const int32_t begin = part * part_chunks;
            end = min(begin + part_chunks, item_chunks);
            first = begin + (int32_t)threadIdx.x;
        }
        const uint4* C = K_cur + item * item_chunks * 2;
        const uint4* P = K_prev + item * (int64_t)t_prev * CPT * 2;
        // A piece is two adjacent 16-byte chunks of one token, so the token's taps and weights are computed
        // once for both, and all ten loads are issued before any is used.
        for (int32_t idx = first; idx < end; idx += kThreads) {
            const int32_t tok = idx >> kShift, ch = idx & (CPT - 1);
            const int32_t y = (int32_t)(((uint64_t)(uint32_t)tok * inv_s_cur) >> 36), x = tok - y * s_cur;
            int y0, y1, x0, x1;
            float wy, wx;
            tap(y, ratio, s_prev, y0, y1, wy);
            tap(x, ratio, s_prev, x0, x1, wx);
            const float w11 = wy * wx, w10 = wy - w11, w01 = wx - w11, w00 = 1.f - wy - w01;
            const float n00 = -w00, n01 = -w01, n10 = -w10, n11 = -w11;
            const uint4* Pc = P + 2 * ch;
            const uint4* p00 = Pc + (y0 * s_prev + x0) * (2 * CPT);
            const uint4* p01 = Pc + (y0 * s_prev + x1) * (2 * CPT);
            const uint4* p10 = Pc + (y1 * s_prev + x0) * (2 * CPT);
            const uint4* p11 = Pc + (y1 * s_prev + x1) * (2 * CPT);
            uint4 cur[2], t00[2], t01[2], t10[2], t11[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                cur[h] = __ldcs(C + 2 * idx + h);
                t00[h] = __ldg(p00 + h);
                t01[h] = __ldg(p01 + h);
                t10[h] = __ldg(p10 + h);
                t11[h] = __ldg(p11 + h);
            }
            float p0 = 0.f, p1 = 0.f;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                float c[8], v00[8], v01[8], v10[8], v11[8];
                unpack8(cur[h], c);
                unpack8(t00[h], v00);
                unpack8(t01[h], v01);
                unpack8(t10[h], v10);
                unpack8(t11[h], v11);
#pragma unroll
                for (int i = 0; i < 8; i += 2) {
                    float d0, d1;
                    fma2(d0, d1, n00, n00, v00[i], v00[i + 1], c[i], c[i + 1]);
                    fma2(d0, d1, n01, n01, v01[i], v01[i + 1], d0, d1);
                    fma2(d0, d1, n10, n10, v10[i], v10[i + 1], d0, d1);
                    fma2(d0, d1, n11, n11, v11[i], v11[i + 1], d0, d1);
                    fma2(p0, p1, d0, d1, d0, d1, p0, p1);
                }
            }
            acc += (double)(p0 + p1);
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
    const int32_t cpt = D / 16;   // the kernel works in 32-byte pieces
    const int64_t item_chunks = (int64_t)side_cur * side_cur * cpt;
    if (item_chunks >= (1ll << 31) || (int64_t)side_cur * side_cur >= (1ll << 24) + 1) return cudaErrorInvalidValue;
    // units of (item, part): enough of them to fill the partials array, none smaller than a few block iterations
    int64_t parts = (kSimilarityMaxBlocks + items - 1) / items;
    const int64_t max_parts = (item_chunks + 4 * kThreads - 1) / (4 * kThreads);
    if (parts > max_parts) parts = max_parts;
    if (parts < 1) parts = 1;
    const int32_t part_chunks = (int32_t)((item_chunks + parts - 1) / parts);
    parts = (item_chunks + part_chunks - 1) / part_chunks;
    int64_t units = items * parts;
    int32_t items_per_unit = 1;
    if (2 * item_chunks <= kThreads) {
        items_per_unit = (int32_t)(kThreads / item_chunks);
        parts = 1;
        units = (items + items_per_unit - 1) / items_per_unit;
    }
    int64_t blocks = units < kSimilarityMaxBlocks ? units : kSimilarityMaxBlocks;
    if (blocks < 1) blocks = 1;
    const uint64_t inv = ((1ull << 36) + (uint64_t)side_cur - 1) / (uint64_t)side_cur;
    const uint4* kp = (const uint4*)K_prev;
    const uint4* kc = (const uint4*)K_cur;
    if (D == 64)
        similarity_partial_kernel<64><<<(unsigned)blocks, kThreads, 0, stream>>>(
            kp, side_prev, kc, side_cur, items, units, (int32_t)parts, part_chunks, items_per_unit, inv, partials);
    else
        similarity_partial_kernel<128><<<(unsigned)blocks, kThreads, 0, stream>>>(
            kp, side_prev, kc, side_cur, items, units, (int32_t)parts, part_chunks, items_per_unit, inv, partials);
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
