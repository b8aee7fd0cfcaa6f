// Small-query attention: one warp per (row, head) item, for the coarse scales whose retained
// keys fit one register tile (at most 32 keys, at most 16 queries: measured, the paired
// tensor-memory kernel is faster beyond that).
//
// At these scales an item is a few kilobytes of K and V and a handful of query rows, so the
// work is HBM-bound and what matters is that every item is fetched once, with whole sectors,
// by many independent warps.  A warp reads Q, K and V straight from global memory in the
// register layout of the warp-level matrix instruction (each load instruction takes 16
// contiguous bytes from each of eight token rows; the neighbouring 16 bytes of the sector are
// the next load's), computes the whole score row block S = Q K^T in registers
// (mma.sync.m16n8k16, bf16 in, fp32 out), takes the softmax in one pass (no running maximum is
// needed when the whole row is present), rounds P to bf16, multiplies by V (transposed in
// registers with movmatrix) and stores out = P V / rowsum.  No shared memory, no barriers.
// The legacy warp-level tensor instruction is enough here: a launch moves a few hundred MB and
// needs well under a tenth of the tensor throughput the big scales need.
#include "kernels.cuh"

namespace amskv {

namespace {

constexpr int kWarpsPerCta = 4;
constexpr int kMaxKeyTiles = kSmallMaxKeys / 8;   // 8-key column tiles of S

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// D (16x8, fp32) += A (16x16, bf16, row-major) * B (16x8, bf16, column-major)
__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// transposes an 8x8 matrix of 16-bit elements held one row per four lanes
__device__ __forceinline__ uint32_t transpose_8x8(uint32_t x)
{
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}

// arena token of the i-th retained key (i < total); ranges are in ascending position order
__device__ __forceinline__ int32_t key_token(const RangeList& rl, int32_t i)
{
    int r = 0;
    for (; r < rl.n - 1; ++r) {
        if (i < rl.r[r].len) break;
        i -= rl.r[r].len;
    }
    return rl.r[r].start + i;
}

template <int D>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
attend_small_kernel(const __nv_bfloat16* __restrict__ Q, int64_t q_row, int64_t q_head, int64_t q_tok,
                    __nv_bfloat16* __restrict__ O, int64_t o_row, int64_t o_head, int64_t o_tok,
                    const __nv_bfloat16* __restrict__ region, int32_t capacity, const RangeList ranges, int32_t T,
                    int32_t heads, int32_t n_items, float scale_log2)
{
    constexpr int kKSteps = D / 16;     // 16-channel steps of Q K^T
    constexpr int kOTiles = D / 8;      // 8-channel column tiles of O
    const int lane = threadIdx.x & 31;
    const int item = blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
    if (item >= n_items) return;        // whole warps leave together: nothing below synchronises across warps
    const int quad = lane >> 2, col2 = (lane & 3) * 2;
    const int32_t L = ranges.total;
    const int n_key_tiles = (L + 7) >> 3;
    const int n_key_steps = (L + 15) >> 4;
    const int32_t row = item / heads, head = item - row * heads;
    const __nv_bfloat16* qbase = Q + row * q_row + head * q_head;
    const __nv_bfloat16* kbase = region + (int64_t)item * (2ll * capacity * D);
    const __nv_bfloat16* vbase = kbase + (int64_t)capacity * D;
    __nv_bfloat16* obase = O + row * o_row + head * o_head;

    // The key this lane addresses in column tile t of S (token quad of that tile), and in the second
    // product the two keys of 16-key step s (tokens quad and quad + 8).  Keys past the end are
    // clamped to the last one; their scores are masked, so their probabilities are exactly zero.
    const uint32_t* krow[kMaxKeyTiles];   // key row, as 32-bit words, at this lane's channel pair
#pragma unroll
    for (int t = 0; t < kMaxKeyTiles; ++t) {
        const int32_t i = min(t * 8 + quad, L - 1);
        krow[t] = reinterpret_cast<const uint32_t*>(kbase + (int64_t)key_token(ranges, i) * D + col2);
    }

    for (int m0 = 0; m0 < T; m0 += 16) {
        // ---- Q fragments of query rows m0 + quad and m0 + quad + 8 (clamped; rows past T are not stored)
        const int32_t r0 = min(m0 + quad, T - 1), r1 = min(m0 + quad + 8, T - 1);
        const uint32_t* q0 = reinterpret_cast<const uint32_t*>(qbase + r0 * q_tok + col2);
        const uint32_t* q1 = reinterpret_cast<const uint32_t*>(qbase + r1 * q_tok + col2);
        uint32_t qa[kKSteps][4];
#pragma unroll
        for (int ks = 0; ks < kKSteps; ++ks) {
            qa[ks][0] = __ldg(q0 + ks * 8);
            qa[ks][1] = __ldg(q1 + ks * 8);
            qa[ks][2] = __ldg(q0 + ks * 8 + 4);
            qa[ks][3] = __ldg(q1 + ks * 8 + 4);
        }
        // ---- S = Q K^T : this lane holds S[quad][t*8 + col2 .. +1] and S[quad + 8][same] of every tile t
        float s[kMaxKeyTiles][4];
#pragma unroll
        for (int t = 0; t < kMaxKeyTiles; ++t) {
            s[t][0] = s[t][1] = s[t][2] = s[t][3] = 0.f;
            if (t < n_key_tiles) {
#pragma unroll
                for (int ks = 0; ks < kKSteps; ++ks) mma_16816(s[t], qa[ks], __ldg(krow[t] + ks * 8), __ldg(krow[t] + ks * 8 + 4));
            }
        }
        // ---- softmax over the whole row (two rows per lane; a row is spread over the four lanes of a quad)
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int t = 0; t < kMaxKeyTiles; ++t) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const bool live = t * 8 + col2 + e < L;
                if (!live) s[t][e] = s[t][2 + e] = -INFINITY;
            }
            mx0 = fmaxf(mx0, fmaxf(s[t][0], s[t][1]));
            mx1 = fmaxf(mx1, fmaxf(s[t][2], s[t][3]));
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        const float nb0 = -mx0 * scale_log2, nb1 = -mx1 * scale_log2;
        float l0 = 0.f, l1 = 0.f;
        uint32_t p[kMaxKeyTiles][2];   // P as bf16 pairs: [t][0] row quad, [t][1] row quad + 8
#pragma unroll
        for (int t = 0; t < kMaxKeyTiles; ++t) {
            const float p00 = fast_exp2(fmaf(s[t][0], scale_log2, nb0)), p01 = fast_exp2(fmaf(s[t][1], scale_log2, nb0));
            const float p10 = fast_exp2(fmaf(s[t][2], scale_log2, nb1)), p11 = fast_exp2(fmaf(s[t][3], scale_log2, nb1));
            l0 += p00 + p01;
            l1 += p10 + p11;
            p[t][0] = pack_bf16(p00, p01);
            p[t][1] = pack_bf16(p10, p11);
        }
        l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
        l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
        // ---- O = P V : two adjacent column tiles of S are one 16-key step of the second product
        float o[kOTiles][4];
#pragma unroll
        for (int c = 0; c < kOTiles; ++c) o[c][0] = o[c][1] = o[c][2] = o[c][3] = 0.f;
#pragma unroll
        for (int st = 0; st < kMaxKeyTiles / 2; ++st) {
            if (st < n_key_steps) {
                const uint32_t pa[4] = {p[2 * st][0], p[2 * st][1], p[2 * st + 1][0], p[2 * st + 1][1]};
                const int32_t i0 = min(st * 16 + quad, L - 1), i1 = min(st * 16 + 8 + quad, L - 1);
                const uint32_t* v0 = reinterpret_cast<const uint32_t*>(vbase + (int64_t)key_token(ranges, i0) * D + col2);
                const uint32_t* v1 = reinterpret_cast<const uint32_t*>(vbase + (int64_t)key_token(ranges, i1) * D + col2);
#pragma unroll
                for (int c = 0; c < kOTiles; ++c) {
                    // V[key quad][channels c*8 + col2 ..] read row-wise, then transposed to the B layout
                    const uint32_t b0 = transpose_8x8(__ldg(v0 + c * 4));
                    const uint32_t b1 = transpose_8x8(__ldg(v1 + c * 4));
                    mma_16816(o[c], pa, b0, b1);
                }
            }
        }
        // ---- out = O / l
        const float inv0 = 1.f / l0, inv1 = 1.f / l1;
        const bool st0 = m0 + quad < T, st1 = m0 + quad + 8 < T;
        uint32_t* out0 = reinterpret_cast<uint32_t*>(obase + (int64_t)(m0 + quad) * o_tok + col2);
        uint32_t* out1 = reinterpret_cast<uint32_t*>(obase + (int64_t)(m0 + quad + 8) * o_tok + col2);
#pragma unroll
        for (int c = 0; c < kOTiles; ++c) {
            if (st0) out0[c * 4] = pack_bf16(o[c][0] * inv0, o[c][1] * inv0);
            if (st1) out1[c * 4] = pack_bf16(o[c][2] * inv1, o[c][3] * inv1);
        }
    }
}

}  // namespace

bool small_supported(int32_t T, int32_t total_keys) { return T <= kSmallMaxQueries && total_keys >= 1 && total_keys <= kSmallMaxKeys; }

cudaError_t launch_attend_small(const Strided& Q, const Strided& O, const LayerRegion& region, const RangeList& ranges,
                                int32_t T, int32_t rows, int32_t heads, int32_t D, float softmax_scale,
                                cudaStream_t stream)
{
    if (!small_supported(T, ranges.total)) return cudaErrorInvalidValue;
    const int64_t items = (int64_t)rows * heads;
    if (items == 0) return cudaSuccess;
    if (items > 0x3fffffffll) return cudaErrorInvalidValue;
    const int64_t blocks = (items + kWarpsPerCta - 1) / kWarpsPerCta;
    const float scale_log2 = softmax_scale * 1.4426950408889634f;
    if (D == 64) {
        attend_small_kernel<64><<<(unsigned)blocks, kWarpsPerCta * 32, 0, stream>>>(
            (const __nv_bfloat16*)Q.ptr, Q.row, Q.head, Q.token, (__nv_bfloat16*)O.ptr, O.row, O.head, O.token,
            region.base, region.capacity, ranges, T, heads, (int32_t)items, scale_log2);
    } else {
        attend_small_kernel<128><<<(unsigned)blocks, kWarpsPerCta * 32, 0, stream>>>(
            (const __nv_bfloat16*)Q.ptr, Q.row, Q.head, Q.token, (__nv_bfloat16*)O.ptr, O.row, O.head, O.token,
            region.base, region.capacity, ranges, T, heads, (int32_t)items, scale_log2);
    }
    count_launch();
    return cudaGetLastError();
}

}  // namespace amskv
