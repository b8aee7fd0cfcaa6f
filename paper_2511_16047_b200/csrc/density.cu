// Attention density (Sec. 4.1): how much attention the queries of a scale pay to each retained
// segment, per key token of that segment.
//
// An analysis tool, not part of the generation step: it recomputes the softmax of the attend call
// on the CUDA cores in two passes over the retained keys (pass 1: row maximum and row sum; pass 2:
// the normalised probabilities, summed per piece of the cache) and adds the sums, weighted by
// 1 / (rows * tokens of the run), into a [heads, runs] table of doubles with atomic adds.  Eight
// lanes share one query row as in the CUDA-core attention kernel; a CTA never spans two items, so
// its partial sums are first combined in shared memory.
#include "kernels.cuh"

namespace amskv {

namespace {

constexpr int kThreads = 128;
constexpr int kLanesPerRow = 8;
constexpr int kRowsPerCta = kThreads / kLanesPerRow;

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int N>
__device__ __forceinline__ void load_bf16(const __nv_bfloat16* p, float (&f)[N])
{
#pragma unroll
    for (int c = 0; c < N / 8; ++c) {
        const uint4 raw = __ldg(reinterpret_cast<const uint4*>(p) + c);
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 v = __bfloat1622float2(h[i]);
            f[c * 8 + 2 * i] = v.x;
            f[c * 8 + 2 * i + 1] = v.y;
        }
    }
}

template <int D>
__global__ void __launch_bounds__(kThreads)
density_kernel(const __nv_bfloat16* __restrict__ Q, int64_t q_row, int64_t q_head, int64_t q_tok,
               const __nv_bfloat16* __restrict__ region, int32_t capacity, const DensityPieces pieces, int32_t T,
               int32_t heads, int32_t ctas_per_item, float scale_log2, double inv_rows, double* __restrict__ out)
{
    constexpr int DPL = D / kLanesPerRow;
    __shared__ double acc[kMaxDensityPieces];
    for (int i = threadIdx.x; i < pieces.n; i += kThreads) acc[i] = 0.0;
    __syncthreads();
    const int32_t item = blockIdx.x / ctas_per_item;
    const int32_t qi = (blockIdx.x - item * ctas_per_item) * kRowsPerCta + (int32_t)threadIdx.x / kLanesPerRow;
    const int sub = threadIdx.x % kLanesPerRow;
    const bool live = qi < T;
    const int32_t row = item / heads, head = item - row * heads;

    float q[DPL];
    load_bf16<DPL>(Q + row * q_row + head * q_head + (int64_t)min(qi, T - 1) * q_tok + sub * DPL, q);
#pragma unroll
    for (int d = 0; d < DPL; ++d) q[d] *= scale_log2;
    const __nv_bfloat16* kbase = region + (int64_t)item * (2ll * capacity * D) + sub * DPL;

    auto logit = [&](int32_t tok) {
        float k[DPL];
        load_bf16<DPL>(kbase + (int64_t)tok * D, k);
        float s = 0.f;
#pragma unroll
        for (int d = 0; d < DPL; ++d) s = fmaf(q[d], k[d], s);
        s += __shfl_xor_sync(0xffffffffu, s, 1);
        s += __shfl_xor_sync(0xffffffffu, s, 2);
        s += __shfl_xor_sync(0xffffffffu, s, 4);
        return s;
    };
    // pass 1: row maximum, then row sum against it
    float m = -INFINITY;
    for (int p = 0; p < pieces.n; ++p)
        for (int32_t t = 0; t < pieces.len[p]; ++t) m = fmaxf(m, logit(pieces.start[p] + t));
    float l = 0.f;
    for (int p = 0; p < pieces.n; ++p)
        for (int32_t t = 0; t < pieces.len[p]; ++t) l += fast_exp2(logit(pieces.start[p] + t) - m);
    const float inv_l = 1.f / l;
    // pass 2: probability mass per piece
    for (int p = 0; p < pieces.n; ++p) {
        float mass = 0.f;
        for (int32_t t = 0; t < pieces.len[p]; ++t) mass += fast_exp2(logit(pieces.start[p] + t) - m) * inv_l;
        if (live && sub == 0) atomicAdd(&acc[p], (double)mass);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < pieces.n; i += kThreads)
        atomicAdd(out + (int64_t)head * pieces.n_runs + pieces.run[i], acc[i] * inv_rows * pieces.weight[i]);
}

}  // namespace

cudaError_t launch_density(const Strided& Q, const LayerRegion& region, const DensityPieces& pieces, int32_t T,
                           int32_t rows, int32_t heads, int32_t D, float softmax_scale, double* out, cudaStream_t stream)
{
    const int64_t items = (int64_t)rows * heads;
    if (items == 0 || pieces.n == 0) return cudaSuccess;
    const int32_t ctas_per_item = (T + kRowsPerCta - 1) / kRowsPerCta;
    const int64_t blocks = items * ctas_per_item;
    if (blocks > 0x7fffffffll) return cudaErrorInvalidValue;
    cudaError_t e = cudaMemsetAsync(out, 0, sizeof(double) * (size_t)heads * pieces.n_runs, stream);
    if (e != cudaSuccess) return e;
    const float scale_log2 = softmax_scale * 1.4426950408889634f;
    const double inv_rows = 1.0 / (double)rows;
    if (D == 64)
        density_kernel<64><<<(unsigned)blocks, kThreads, 0, stream>>>((const __nv_bfloat16*)Q.ptr, Q.row, Q.head, Q.token,
                                                                      region.base, region.capacity, pieces, T, heads,
                                                                      ctas_per_item, scale_log2, inv_rows, out);
    else
        density_kernel<128><<<(unsigned)blocks, kThreads, 0, stream>>>((const __nv_bfloat16*)Q.ptr, Q.row, Q.head, Q.token,
                                                                       region.base, region.capacity, pieces, T, heads,
                                                                       ctas_per_item, scale_log2, inv_rows, out);
    count_launch();
    return cudaGetLastError();
}

}  // namespace amskv
