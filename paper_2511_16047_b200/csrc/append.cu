// Append: copies one scale's K and V ([rows, heads, T, D] bf16, strided) into the layer's
// slot for that segment (Algorithm 1, "append the i-th scale").  Pure byte movement, 16 bytes
// per access; eviction itself moves no data (the evicted segment is the slot's old tenant).
#include "kernels.cuh"

namespace amskv {

namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 4;

template <int D>
__global__ void __launch_bounds__(kThreads)
append_kernel(const uint4* __restrict__ Ksrc, const uint4* __restrict__ Vsrc, int64_t k_row, int64_t k_head,
              int64_t k_tok, int64_t v_row, int64_t v_head, int64_t v_tok, uint4* __restrict__ dst, int32_t capacity,
              int32_t token_offset, int32_t T, int32_t heads, int64_t total_chunks)
{
    constexpr int CPT = D / 8;  // 16-byte chunks per token
    const int64_t chunks_per_item = (int64_t)T * CPT;
    const int64_t item_stride = 2ll * capacity * CPT;     // chunks
    const int64_t v_shift = (int64_t)capacity * CPT;       // values sit behind the keys
    const int64_t step = (int64_t)gridDim.x * kThreads * kUnroll;
    for (int64_t base = (int64_t)blockIdx.x * kThreads * kUnroll + threadIdx.x; base < total_chunks; base += step) {
        uint4 kv[kUnroll], vv[kUnroll];
        int64_t d[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int64_t idx = base + (int64_t)u * kThreads;
            d[u] = -1;
            if (idx < total_chunks) {
                const int64_t item = idx / chunks_per_item;
                const int32_t rem = (int32_t)(idx - item * chunks_per_item);
                const int32_t tok = rem / CPT;
                const int32_t ch = rem - tok * CPT;
                const int32_t row = (int32_t)(item / heads);
                const int32_t head = (int32_t)(item - (int64_t)row * heads);
                // strides are in elements and multiples of 8, so they divide into chunks
                const int64_t ks = (row * k_row + head * k_head + tok * k_tok) / 8 + ch;
                const int64_t vs = (row * v_row + head * v_head + tok * v_tok) / 8 + ch;
                kv[u] = __ldcs(Ksrc + ks);
                vv[u] = __ldcs(Vsrc + vs);
                d[u] = item * item_stride + (int64_t)(token_offset + tok) * CPT + ch;
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            if (d[u] >= 0) {
                dst[d[u]] = kv[u];
                dst[d[u] + v_shift] = vv[u];
            }
        }
    }
}

}  // namespace

cudaError_t launch_append(const Strided& K, const Strided& V, const LayerRegion& region, int32_t token_offset,
                          int32_t T, int32_t rows, int32_t heads, int32_t D, cudaStream_t stream)
{
    const int64_t total = (int64_t)rows * heads * T * (D / 8);
    if (total == 0) return cudaSuccess;
    int64_t blocks = (total + (int64_t)kThreads * kUnroll - 1) / ((int64_t)kThreads * kUnroll);
    if (blocks > (1 << 20)) blocks = 1 << 20;
    auto* dst = reinterpret_cast<uint4*>(region.base);
    if (D == 64) {
        append_kernel<64><<<(unsigned)blocks, kThreads, 0, stream>>>(
            (const uint4*)K.ptr, (const uint4*)V.ptr, K.row, K.head, K.token, V.row, V.head, V.token, dst,
            region.capacity, token_offset, T, heads, total);
    } else {
        append_kernel<128><<<(unsigned)blocks, kThreads, 0, stream>>>(
            (const uint4*)K.ptr, (const uint4*)V.ptr, K.row, K.head, K.token, V.row, V.head, V.token, dst,
            region.capacity, token_offset, T, heads, total);
    }
    count_launch();
    return cudaGetLastError();
}

}  // namespace amskv
