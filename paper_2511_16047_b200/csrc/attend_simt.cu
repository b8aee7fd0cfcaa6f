// Small-query attention on the CUDA cores.
//
// The coarse scales have 1-16 query tokens per (row, head), so the work is a few dot
// products per byte read: HBM-bound.  Eight lanes share one query row; each lane owns
// D/8 channels, so one key (or value) row is read by the eight lanes as consecutive
// 16-byte loads straight from global memory, and rows that share an item hit L1/L2.
// Softmax is the running-max form, updated once per four keys.  The kernel is correct for
// any number of query tokens and serves as the CUDA-core alternative to the tensor-core
// kernel at every scale.
#include "kernels.cuh"

namespace amskv {

namespace {

constexpr int kThreads = 128;
constexpr int kLanesPerRow = 8;
constexpr int kKeysPerStep = 4;

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int N>
__device__ __forceinline__ void load_bf16(const __nv_bfloat16* p, float (&f)[N])
{
    static_assert(N % 8 == 0, "16-byte granules");
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
attend_simt_kernel(const __nv_bfloat16* __restrict__ Q, int64_t q_row, int64_t q_head, int64_t q_tok,
                   __nv_bfloat16* __restrict__ O, int64_t o_row, int64_t o_head, int64_t o_tok,
                   const __nv_bfloat16* __restrict__ region, int32_t capacity, const RangeList ranges, int32_t T,
                   int32_t heads, int64_t total_rows, float scale_log2, const __nv_bfloat16* __restrict__ ext_k,
                   const __nv_bfloat16* __restrict__ ext_v, int64_t e_row, int64_t e_head, int64_t e_tok, int ext_range)
{
    constexpr int DPL = D / kLanesPerRow;  // channels per lane
    const int64_t tid = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    const int sub = (int)(tid % kLanesPerRow);
    int64_t g = tid / kLanesPerRow;
    const bool live = g < total_rows;
    if (!live) g = total_rows - 1;  // keep the lane in the shuffles; its result is dropped
    const int64_t item = g / T;
    const int32_t qi = (int32_t)(g - item * T);
    const int32_t row = (int32_t)(item / heads);
    const int32_t head = (int32_t)(item - (int64_t)row * heads);

    float q[DPL];
    load_bf16<DPL>(Q + row * q_row + head * q_head + qi * q_tok + sub * DPL, q);
#pragma unroll
    for (int d = 0; d < DPL; ++d) q[d] *= scale_log2;  // logits in log2 units

    const __nv_bfloat16* kbase = region + item * (2ll * capacity * D) + sub * DPL;
    const __nv_bfloat16* vbase = kbase + (int64_t)capacity * D;

    float m = -INFINITY, l = 0.f;
    float o[DPL];
#pragma unroll
    for (int d = 0; d < DPL; ++d) o[d] = 0.f;

    for (int r = 0; r < ranges.n; ++r) {
        // range `ext_range` (if any) is the current scale in the caller's own K and V tensors
        const bool ext = r == ext_range;
        const __nv_bfloat16* kb = ext ? ext_k + row * e_row + head * e_head + sub * DPL : kbase;
        const __nv_bfloat16* vb = ext ? ext_v + row * e_row + head * e_head + sub * DPL : vbase;
        const int64_t tstride = ext ? e_tok : (int64_t)D;
        const int32_t end = ranges.r[r].start + ranges.r[r].len;
        for (int32_t tok = ranges.r[r].start; tok < end; tok += kKeysPerStep) {
            float s[kKeysPerStep];
            float v[kKeysPerStep][DPL];
#pragma unroll
            for (int u = 0; u < kKeysPerStep; ++u) {
                if (tok + u < end) {
                    float k[DPL];
                    load_bf16<DPL>(kb + (int64_t)(tok + u) * tstride, k);
                    load_bf16<DPL>(vb + (int64_t)(tok + u) * tstride, v[u]);
                    float acc = 0.f;
#pragma unroll
                    for (int d = 0; d < DPL; ++d) acc = fmaf(q[d], k[d], acc);
                    s[u] = acc;
                } else {
                    s[u] = 0.f;
#pragma unroll
                    for (int d = 0; d < DPL; ++d) v[u][d] = 0.f;
                }
            }
#pragma unroll
            for (int u = 0; u < kKeysPerStep; ++u) {
                s[u] += __shfl_xor_sync(0xffffffffu, s[u], 1);
                s[u] += __shfl_xor_sync(0xffffffffu, s[u], 2);
                s[u] += __shfl_xor_sync(0xffffffffu, s[u], 4);
                if (tok + u >= end) s[u] = -INFINITY;
            }
            float m_new = m;
#pragma unroll
            for (int u = 0; u < kKeysPerStep; ++u) m_new = fmaxf(m_new, s[u]);
            const float a = fast_exp2(m - m_new);  // 0 on the first step (m = -inf)
            float p[kKeysPerStep];
            float psum = 0.f;
#pragma unroll
            for (int u = 0; u < kKeysPerStep; ++u) {
                p[u] = fast_exp2(s[u] - m_new);
                psum += p[u];
            }
            l = fmaf(l, a, psum);
#pragma unroll
            for (int d = 0; d < DPL; ++d) {
                float acc = o[d] * a;
#pragma unroll
                for (int u = 0; u < kKeysPerStep; ++u) acc = fmaf(p[u], v[u][d], acc);
                o[d] = acc;
            }
            m = m_new;
        }
    }

    if (live) {
        const float inv = 1.f / l;
        __nv_bfloat16* dst = O + row * o_row + head * o_head + qi * o_tok + sub * DPL;
#pragma unroll
        for (int c = 0; c < DPL / 8; ++c) {
            uint4 raw;
            __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&raw);
#pragma unroll
            for (int i = 0; i < 4; ++i)
                h[i] = __floats2bfloat162_rn(o[c * 8 + 2 * i] * inv, o[c * 8 + 2 * i + 1] * inv);
            reinterpret_cast<uint4*>(dst)[c] = raw;
        }
    }
}

}  // namespace

cudaError_t launch_attend_simt(const Strided& Q, const Strided& O, const LayerRegion& region, const RangeList& ranges,
                               int32_t T, int32_t rows, int32_t heads, int32_t D, float softmax_scale,
                               cudaStream_t stream, const CurrentScaleSource* cur)
{
    const __nv_bfloat16* ek = cur ? (const __nv_bfloat16*)cur->K.ptr : nullptr;
    const __nv_bfloat16* ev = cur ? (const __nv_bfloat16*)cur->V.ptr : nullptr;
    const int64_t e_row = cur ? cur->K.row : 0, e_head = cur ? cur->K.head : 0, e_tok = cur ? cur->K.token : 0;
    const int ext_range = cur ? ranges.n - 1 : -1;
    if (cur && (cur->store || cur->V.row != e_row || cur->V.head != e_head || cur->V.token != e_tok)) return cudaErrorNotSupported;
    const int64_t total_rows = (int64_t)rows * heads * T;
    if (total_rows == 0) return cudaSuccess;
    const int64_t threads = total_rows * kLanesPerRow;
    const int64_t blocks = (threads + kThreads - 1) / kThreads;
    if (blocks > 0x7fffffffll) return cudaErrorInvalidValue;
    const float scale_log2 = softmax_scale * 1.4426950408889634f;
    if (D == 64) {
        attend_simt_kernel<64><<<(unsigned)blocks, kThreads, 0, stream>>>(
            (const __nv_bfloat16*)Q.ptr, Q.row, Q.head, Q.token, (__nv_bfloat16*)O.ptr, O.row, O.head, O.token,
            region.base, region.capacity, ranges, T, heads, total_rows, scale_log2, ek, ev, e_row, e_head, e_tok, ext_range);
    } else {
        attend_simt_kernel<128><<<(unsigned)blocks, kThreads, 0, stream>>>(
            (const __nv_bfloat16*)Q.ptr, Q.row, Q.head, Q.token, (__nv_bfloat16*)O.ptr, O.row, O.head, O.token,
            region.base, region.capacity, ranges, T, heads, total_rows, scale_log2, ek, ev, e_row, e_head, e_tok, ext_range);
    }
    count_launch();
    return cudaGetLastError();
}

}  // namespace amskv
