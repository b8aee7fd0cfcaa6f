// Append: copies one scale's K and V ([rows, heads, T, D] bf16, strided) into the layer's
// slot for that segment (the step of Algorithm 1 in which a new scale joins the cache).  Pure byte movement, 16 bytes
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


// ---------------------------------------------------------------- bulk-copy form
// For token-contiguous inputs one item's K (or V) of a scale is one contiguous block on both sides,
// so it can move as bulk asynchronous copies: global -> shared -> global through a small ring of
// shared-memory stages, driven by a single thread.  A CTA needs 32 threads, a handful of registers
// and 24 KB of shared memory, so it also fits beside the attention kernel's CTAs on an SM: an append
// enqueued on a second stream (the next layer's, say) runs in the memory bandwidth attention leaves.
constexpr int kBulkStages = 3;
constexpr uint32_t kBulkChunk = 8192;            // bytes per stage
constexpr uint32_t kBulkSmem = kBulkStages * kBulkChunk;
constexpr uint32_t kBulkSpinLimit = 1u << 24;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__global__ void __launch_bounds__(32)
append_bulk_kernel(const char* __restrict__ Ksrc, const char* __restrict__ Vsrc, int64_t src_item_bytes,
                   char* __restrict__ dst, int64_t dst_item_bytes, int64_t v_shift_bytes, int64_t dst_offset_bytes,
                   uint32_t block_bytes, uint32_t chunks_per_block, int64_t total_chunks, int* __restrict__ status)
{
    extern __shared__ __align__(128) uint8_t bulk_smem[];
    __shared__ uint64_t full[kBulkStages];
    if (threadIdx.x != 0) return;
    for (int s = 0; s < kBulkStages; ++s)
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(&full[s])) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");

    // chunk c of this CTA: global chunk index blockIdx.x + c * gridDim.x
    const int64_t mine = blockIdx.x < total_chunks ? (total_chunks - 1 - blockIdx.x) / gridDim.x + 1 : 0;
    auto locate = [&](int64_t c, const char*& src, char*& out, uint32_t& bytes) {
        const int64_t idx = (int64_t)blockIdx.x + c * gridDim.x;
        const int64_t blk = idx / chunks_per_block;          // (item, K or V)
        const uint32_t part = (uint32_t)(idx - blk * chunks_per_block);
        const int64_t item = blk >> 1;
        const bool is_v = (blk & 1) != 0;
        const uint32_t off = part * kBulkChunk;
        bytes = min(kBulkChunk, block_bytes - off);
        src = (is_v ? Vsrc : Ksrc) + item * src_item_bytes + off;
        out = dst + item * dst_item_bytes + (is_v ? v_shift_bytes : 0) + dst_offset_bytes + off;
    };
    auto issue_load = [&](int64_t c) {
        const char* src;
        char* out;
        uint32_t bytes;
        locate(c, src, out, bytes);
        const uint32_t stage = (uint32_t)(c % kBulkStages);
        const uint32_t bar = smem_addr(&full[stage]);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_addr(bulk_smem + stage * kBulkChunk)), "l"(src), "r"(bytes), "r"(bar)
                     : "memory");
    };
    for (int64_t c = 0; c < mine && c < kBulkStages; ++c) issue_load(c);
    for (int64_t c = 0; c < mine; ++c) {
        const uint32_t stage = (uint32_t)(c % kBulkStages);
        const uint32_t bar = smem_addr(&full[stage]);
        const uint32_t parity = (uint32_t)((c / kBulkStages) & 1);
        uint32_t done = 0;
        for (uint32_t i = 0; i < kBulkSpinLimit && !done; ++i) {
            asm volatile(
                "{\n"
                ".reg .pred p;\n"
                "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
                "selp.u32 %0, 1, 0, p;\n"
                "}\n"
                : "=r"(done)
                : "r"(bar), "r"(parity)
                : "memory");
        }
        if (!done) {
            // a copy that never landed: record it, stop issuing, and give the loads still in flight a
            // bounded time to land before the CTA hands its shared memory back
            if (status) atomicCAS(status, 0, (int)kStatusTmaTimeout);
            for (int64_t c2 = c + 1; c2 < mine && c2 < c + kBulkStages; ++c2) {
                const uint32_t bar2 = smem_addr(&full[c2 % kBulkStages]);
                const uint32_t parity2 = (uint32_t)((c2 / kBulkStages) & 1);
                uint32_t landed = 0;
                for (uint32_t i = 0; i < kBulkSpinLimit && !landed; ++i) {
                    asm volatile(
                        "{\n"
                        ".reg .pred p;\n"
                        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
                        "selp.u32 %0, 1, 0, p;\n"
                        "}\n"
                        : "=r"(landed)
                        : "r"(bar2), "r"(parity2)
                        : "memory");
                }
            }
            break;
        }
        const char* src;
        char* out;
        uint32_t bytes;
        locate(c, src, out, bytes);
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                     ::"l"(out), "r"(smem_addr(bulk_smem + stage * kBulkChunk)), "r"(bytes)
                     : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        // refill the stage of the previous chunk once its store has read it (the store just issued may
        // still be reading its own stage)
        if (c >= 1 && c - 1 + kBulkStages < mine) {
            asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
            issue_load(c - 1 + kBulkStages);
        }
    }
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // stores complete before the CTA's shared memory goes away
}

}  // namespace

cudaError_t launch_append(const Strided& K, const Strided& V, const LayerRegion& region, int32_t token_offset,
                          int32_t T, int32_t rows, int32_t heads, int32_t D, bool bulk, int* status, int sm_count,
                          cudaStream_t stream)
{
    const int64_t total = (int64_t)rows * heads * T * (D / 8);
    if (total == 0) return cudaSuccess;
    const int64_t block_bytes = (int64_t)T * D * 2;
    const bool contiguous = K.token == D && V.token == D && K.head == (int64_t)T * D && V.head == (int64_t)T * D &&
                            K.row == (int64_t)heads * T * D && V.row == (int64_t)heads * T * D;
    if (bulk && contiguous && block_bytes >= 4096 && block_bytes < (1ll << 31)) {
        static SharedMemoryOptIn opt_in;
        const cudaError_t oe = opt_in.ensure(append_bulk_kernel, (int)kBulkSmem);
        if (oe != cudaSuccess) return oe;
        const uint32_t cpb = (uint32_t)((block_bytes + kBulkChunk - 1) / kBulkChunk);
        const int64_t total_chunks = (int64_t)rows * heads * 2 * cpb;
        int64_t grid = (int64_t)(sm_count > 0 ? sm_count : 148) * 8;
        if (grid > total_chunks) grid = total_chunks;
        append_bulk_kernel<<<(unsigned)grid, 32, kBulkSmem, stream>>>(
            (const char*)K.ptr, (const char*)V.ptr, block_bytes, (char*)region.base, 4ll * region.capacity * D,
            2ll * region.capacity * D, 2ll * token_offset * D, (uint32_t)block_bytes, cpb, total_chunks, status);
        count_launch();
        return cudaGetLastError();
    }
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
