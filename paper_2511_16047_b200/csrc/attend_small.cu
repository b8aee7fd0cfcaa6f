// Small-query attention: one warp per (row, head) item, for the coarse scales whose retained
// keys fit one register tile (at most 32 keys, at most 16 queries: measured, the paired
// tensor-memory kernel is faster beyond that), optionally with the append of the scale fused in.
//
// At these scales an item is a few kilobytes of K and V and a handful of query rows, so the
// work is HBM-bound and what matters is that every item is fetched once, with 16-byte accesses,
// by many independent warps that each have all their loads in flight at once.
//
// Every global access is 16 bytes per lane.  Lane (g = lane / 4, q = lane % 4) reads, of token row g
// of an 8-row tile, the 16-byte pieces q, q + 4, ... (8 channels each).  The warp-level matrix
// instruction (mma.sync.m16n8k16, bf16 in, fp32 out) does not care which channel sits in which slot of
// its contraction dimension as long as both operands agree, so the four 32-bit words of a piece are
// used directly as fragment registers: words 0 and 1 are one 16-channel step of Q K^T, words 2 and 3 the
// next -- for the query rows (A operand) and the key rows (B operand) alike.  No shuffle, no shared
// memory.  For the second product V is read the same way and each word is transposed in registers
// (movmatrix); the output columns then come out permuted such that a lane ends up with 8 consecutive
// channels of its query row: one 16-byte store.
//
// S = Q K^T for the whole row block sits in registers, softmax is a single pass (no running maximum
// is needed when the whole row is present), P is rounded to bf16, out = P V / rowsum.
//
// Fused append: the keys and values of the current scale are read from the caller's tensors instead
// of the cache (they are the last keys of the row) and the very registers that feed the products are
// also stored to the scale's place in the cache.
//
// The legacy warp-level tensor instruction is enough here: a launch moves a few hundred MB and
// needs well under a tenth of the tensor throughput the big scales need.
#include "kernels.cuh"

namespace amskv {

namespace {

constexpr int kWarpsPerCta = 4;
static_assert(kSmallMaxKeys == 32, "the register tile is instantiated for 1, 2 and 4 eight-key tiles");

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// D (16x8, fp32) += A (16x16, bf16, row-major) * B (16x8, bf16, column-major)
__device__ __forceinline__ void mma_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                          uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
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
__device__ __forceinline__ uint32_t word_of(const uint4& v, int i) { return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w; }

// arena token of the i-th cached key (i < total); ranges are in ascending position order
__device__ __forceinline__ int32_t key_token(const RangeList& rl, int32_t i)
{
    int r = 0;
    for (; r < rl.n - 1; ++r) {
        if (i < rl.r[r].len) break;
        i -= rl.r[r].len;
    }
    return rl.r[r].start + i;
}

// The current scale in the caller's tensors (kExt): its T tokens are the last keys of every row.
struct SmallExt {
    const __nv_bfloat16* K;
    const __nv_bfloat16* V;
    int64_t row, head, tok;   // element strides, the same for K and V
    int32_t dst;              // first position of the scale in the per-item region
    int32_t store;            // also write the scale there
};

// kTiles: 8-key tiles a row can have (1, 2 or 4): the register tile is sized for it, so the coarsest scales,
// whose rows are a handful of keys, run with more warps per SM -- their launches are bound by how many
// independent items are in flight, not by arithmetic.
template <int D, bool kExt, int kTiles>
__global__ void __launch_bounds__(kWarpsPerCta * 32, D == 64 ? (kTiles == 1 ? 6 : 4) : (kTiles == 1 ? 3 : 2))
attend_small_kernel(const __nv_bfloat16* __restrict__ Q, int64_t q_row, int64_t q_head, int64_t q_tok,
                    __nv_bfloat16* __restrict__ O, int64_t o_row, int64_t o_head, int64_t o_tok,
                    __nv_bfloat16* __restrict__ region, int32_t capacity, const RangeList ranges, int32_t T,
                    int32_t heads, int32_t n_items, float scale_log2, const SmallExt ext)
{
    constexpr int kPieces = D / 32;     // 16-byte pieces of a token row per lane (the lane's pieces are q + 4h)
    const int lane = threadIdx.x & 31;
    const int item = blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
    if (item >= n_items) return;        // whole warps leave together: nothing below synchronises across warps
    const int g = lane >> 2, q = lane & 3;
    const int32_t Lc = ranges.total;                 // keys read from the cache
    const int32_t L = Lc + (kExt ? T : 0);           // all keys of a row
    const int n_key_tiles = (L + 7) >> 3;
    const int n_key_steps = (L + 15) >> 4;
    const int32_t row = item / heads, head = item - row * heads;
    const __nv_bfloat16* qbase = Q + row * q_row + head * q_head;
    __nv_bfloat16* kbase = region + (int64_t)item * (2ll * capacity * D);
    const int64_t v_shift = (int64_t)capacity * D;   // values sit behind the keys
    __nv_bfloat16* obase = O + row * o_row + head * o_head;

    // The key this lane addresses in 8-key tile t (key 8t + g).  Keys past the end are clamped to the last
    // one; their scores are masked, so their probabilities are exactly zero, and they are never stored.
    // kp / vp: this lane's first piece of that key's K and V rows; kd: where the key goes in the cache
    // when the append is fused in (null for cached keys and for clamped duplicates).
    const uint4* kp[kTiles];
    const uint4* vp[kTiles];
    uint4* kd[kTiles];
#pragma unroll
    for (int t = 0; t < kTiles; ++t) {
        const int32_t i = min(t * 8 + g, L - 1);
        kd[t] = nullptr;
        if (kExt && i >= Lc) {
            const int64_t off = row * ext.row + head * ext.head + (int64_t)(i - Lc) * ext.tok + 8 * q;
            kp[t] = reinterpret_cast<const uint4*>(ext.K + off);
            vp[t] = reinterpret_cast<const uint4*>(ext.V + off);
            if (ext.store && t * 8 + g < L) kd[t] = reinterpret_cast<uint4*>(kbase + (int64_t)(ext.dst + i - Lc) * D + 8 * q);
        } else {
            const __nv_bfloat16* p = kbase + (int64_t)key_token(ranges, i) * D + 8 * q;
            kp[t] = reinterpret_cast<const uint4*>(p);
            vp[t] = reinterpret_cast<const uint4*>(p + v_shift);
        }
    }

    for (int m0 = 0; m0 < T; m0 += 16) {
        // ---- Q pieces of query rows m0 + g and m0 + g + 8 (clamped; rows past T are not stored)
        const int32_t r0 = min(m0 + g, T - 1), r1 = min(m0 + g + 8, T - 1);
        const uint4* q0 = reinterpret_cast<const uint4*>(qbase + r0 * q_tok + 8 * q);
        const uint4* q1 = reinterpret_cast<const uint4*>(qbase + r1 * q_tok + 8 * q);
        uint4 qa0[kPieces], qa1[kPieces];
#pragma unroll
        for (int h = 0; h < kPieces; ++h) {
            qa0[h] = __ldg(q0 + 4 * h);
            qa1[h] = __ldg(q1 + 4 * h);
        }
        // ---- K pieces of every tile: all loads are issued before the first product needs one
        uint4 kk[kTiles][kPieces];
#pragma unroll
        for (int t = 0; t < kTiles; ++t) {
            if (t < n_key_tiles) {
#pragma unroll
                for (int h = 0; h < kPieces; ++h) kk[t][h] = __ldg(kp[t] + 4 * h);
            }
        }
        // ---- V pieces likewise (nothing the softmax computes is needed to fetch them), except with the
        // largest register tile, where holding them through the softmax costs more in resident warps than the
        // earlier fetch gains (measured): there they are fetched when the second product starts
        constexpr bool kEarlyV = kTiles < 4;
        uint4 vv[kTiles][kPieces];
#pragma unroll
        for (int t = 0; t < kTiles; ++t) {
            if (kEarlyV && t < 2 * n_key_steps) {
#pragma unroll
                for (int h = 0; h < kPieces; ++h) vv[t][h] = __ldg(vp[t] + 4 * h);
            }
        }
        // ---- S = Q K^T : this lane holds S[g][8t + 2q .. +1] and S[g + 8][same] of every tile t
        float s[kTiles][4];
#pragma unroll
        for (int t = 0; t < kTiles; ++t) {
            s[t][0] = s[t][1] = s[t][2] = s[t][3] = 0.f;
            if (t < n_key_tiles) {
#pragma unroll
                for (int h = 0; h < kPieces; ++h) {
                    mma_16816(s[t], qa0[h].x, qa1[h].x, qa0[h].y, qa1[h].y, kk[t][h].x, kk[t][h].y);
                    mma_16816(s[t], qa0[h].z, qa1[h].z, qa0[h].w, qa1[h].w, kk[t][h].z, kk[t][h].w);
                }
                if (kExt && m0 == 0 && kd[t] != nullptr) {
#pragma unroll
                    for (int h = 0; h < kPieces; ++h) kd[t][4 * h] = kk[t][h];
                }
            }
        }
        // ---- softmax over the whole row (two rows per lane; a row is spread over the four lanes of a quad)
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int t = 0; t < kTiles; ++t) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const bool live = t * 8 + 2 * q + e < L;
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
        uint32_t p[kTiles + (kTiles & 1)][2];   // P as bf16 pairs: [t][0] row g, [t][1] row g + 8
        if (kTiles & 1) p[kTiles][0] = p[kTiles][1] = 0u;
#pragma unroll
        for (int t = 0; t < kTiles; ++t) {
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
        // ---- O = P V : two adjacent key tiles are one 16-key step of the second product.  Word m of piece h
        // of the V rows, transposed, is the B operand of output tile (h, m), whose column n is channel
        // 32h + 8 (n / 2) + 2m + (n % 2): lane (g, q) ends up with channels 32h + 8q .. + 7 of its rows.
        float o[kPieces][4][4];
#pragma unroll
        for (int h = 0; h < kPieces; ++h)
#pragma unroll
            for (int m = 0; m < 4; ++m) o[h][m][0] = o[h][m][1] = o[h][m][2] = o[h][m][3] = 0.f;
#pragma unroll
        for (int st = 0; st < (kTiles + 1) / 2; ++st) {
            if (st < n_key_steps) {
                if (!kEarlyV) {
#pragma unroll
                    for (int h = 0; h < kPieces; ++h) {
                        vv[2 * st][h] = __ldg(vp[2 * st] + 4 * h);
                        vv[kTiles > 1 ? 2 * st + 1 : 0][h] = __ldg(vp[kTiles > 1 ? 2 * st + 1 : 0] + 4 * h);
                    }
                }
                const uint4(&v0)[kPieces] = vv[2 * st];
                const uint4(&v1)[kPieces] = vv[kTiles > 1 ? 2 * st + 1 : 0];   // (a one-tile row has no second half: P is zero there)
                if (kExt && m0 == 0) {
                    if (kd[2 * st] != nullptr) {
#pragma unroll
                        for (int h = 0; h < kPieces; ++h) (kd[2 * st] + v_shift / 8)[4 * h] = v0[h];
                    }
                    if (kTiles > 1 && kd[kTiles > 1 ? 2 * st + 1 : 0] != nullptr) {
#pragma unroll
                        for (int h = 0; h < kPieces; ++h) (kd[kTiles > 1 ? 2 * st + 1 : 0] + v_shift / 8)[4 * h] = v1[h];
                    }
                }
#pragma unroll
                for (int h = 0; h < kPieces; ++h) {
#pragma unroll
                    for (int m = 0; m < 4; ++m) {
                        const uint32_t b0 = transpose_8x8(word_of(v0[h], m));
                        const uint32_t b1 = transpose_8x8(word_of(v1[h], m));
                        mma_16816(o[h][m], p[2 * st][0], p[2 * st][1], p[2 * st + 1][0], p[2 * st + 1][1], b0, b1);
                    }
                }
            }
        }
        // ---- out = O / l : 16 bytes (8 consecutive channels) per lane, piece and row
        const float inv0 = 1.f / l0, inv1 = 1.f / l1;
        const bool st0 = m0 + g < T, st1 = m0 + g + 8 < T;
        uint4* out0 = reinterpret_cast<uint4*>(obase + (int64_t)(m0 + g) * o_tok + 8 * q);
        uint4* out1 = reinterpret_cast<uint4*>(obase + (int64_t)(m0 + g + 8) * o_tok + 8 * q);
#pragma unroll
        for (int h = 0; h < kPieces; ++h) {
            if (st0)
                out0[4 * h] = make_uint4(pack_bf16(o[h][0][0] * inv0, o[h][0][1] * inv0), pack_bf16(o[h][1][0] * inv0, o[h][1][1] * inv0),
                                         pack_bf16(o[h][2][0] * inv0, o[h][2][1] * inv0), pack_bf16(o[h][3][0] * inv0, o[h][3][1] * inv0));
            if (st1)
                out1[4 * h] = make_uint4(pack_bf16(o[h][0][2] * inv1, o[h][0][3] * inv1), pack_bf16(o[h][1][2] * inv1, o[h][1][3] * inv1),
                                         pack_bf16(o[h][2][2] * inv1, o[h][2][3] * inv1), pack_bf16(o[h][3][2] * inv1, o[h][3][3] * inv1));
        }
    }
}

// A scale of one token whose only key is itself (the first scale of a schedule): softmax over one key is
// exactly 1, so out = V bit for bit; with the append fused in the same launch also stores K and V.
// One 16-byte piece per thread.
template <int D>
__global__ void __launch_bounds__(256)
single_key_kernel(const uint4* __restrict__ K, const uint4* __restrict__ V, int64_t e_row, int64_t e_head,
                  uint4* __restrict__ O, int64_t o_row, int64_t o_head, uint4* __restrict__ region, int32_t capacity,
                  int32_t dst, int32_t store, int32_t heads, int64_t n_pieces)
{
    constexpr int CPT = D / 8;   // 16-byte pieces per token
    const int64_t idx = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (idx >= n_pieces) return;
    const int64_t item = idx / CPT;
    const int32_t ch = (int32_t)(idx - item * CPT);
    const int32_t row = (int32_t)(item / heads), head = (int32_t)(item - (int64_t)row * heads);
    const uint4 v = __ldg(V + (row * e_row + head * e_head) / 8 + ch);
    O[(row * o_row + head * o_head) / 8 + ch] = v;
    if (store) {
        const uint4 k = __ldg(K + (row * e_row + head * e_head) / 8 + ch);
        uint4* kd = region + item * (2ll * capacity * CPT) + (int64_t)dst * CPT + ch;
        kd[0] = k;
        kd[(int64_t)capacity * CPT] = v;
    }
}

}  // namespace

bool small_supported(int32_t T, int32_t total_keys) { return T <= kSmallMaxQueries && total_keys >= 1 && total_keys <= kSmallMaxKeys; }

cudaError_t launch_attend_small(const Strided& Q, const Strided& O, const LayerRegion& region, const RangeList& ranges,
                                int32_t T, int32_t rows, int32_t heads, int32_t D, float softmax_scale,
                                cudaStream_t stream, const CurrentScaleSource* cur)
{
    const int32_t total = ranges.total + (cur ? T : 0);
    if (!small_supported(T, total)) return cudaErrorInvalidValue;
    const int64_t items = (int64_t)rows * heads;
    if (items == 0) return cudaSuccess;
    if (items > 0x3fffffffll) return cudaErrorInvalidValue;
    SmallExt ext;
    memset(&ext, 0, sizeof(ext));
    if (cur) {
        if (cur->V.row != cur->K.row || cur->V.head != cur->K.head || cur->V.token != cur->K.token) return cudaErrorNotSupported;
        ext.K = (const __nv_bfloat16*)cur->K.ptr;
        ext.V = (const __nv_bfloat16*)cur->V.ptr;
        ext.row = cur->K.row;
        ext.head = cur->K.head;
        ext.tok = cur->K.token;
        ext.dst = cur->dst;
        ext.store = cur->store ? 1 : 0;
    }
    if (cur && T == 1 && ranges.total == 0) {
        // the scale's single token is its only key
        const int64_t n_pieces = items * (D / 8);
        const int64_t blocks = (n_pieces + 255) / 256;
        if (D == 64)
            single_key_kernel<64><<<(unsigned)blocks, 256, 0, stream>>>(
                (const uint4*)ext.K, (const uint4*)ext.V, ext.row, ext.head, (uint4*)O.ptr, O.row, O.head, (uint4*)region.base,
                region.capacity, ext.dst, ext.store, heads, n_pieces);
        else
            single_key_kernel<128><<<(unsigned)blocks, 256, 0, stream>>>(
                (const uint4*)ext.K, (const uint4*)ext.V, ext.row, ext.head, (uint4*)O.ptr, O.row, O.head, (uint4*)region.base,
                region.capacity, ext.dst, ext.store, heads, n_pieces);
        count_launch();
        return cudaGetLastError();
    }
    const int64_t blocks = (items + kWarpsPerCta - 1) / kWarpsPerCta;
    const float scale_log2 = softmax_scale * 1.4426950408889634f;
#define AMSKV_SMALL_LAUNCH(DD, EXT, TILES)                                                                            \
    attend_small_kernel<DD, EXT, TILES><<<(unsigned)blocks, kWarpsPerCta * 32, 0, stream>>>(                          \
        (const __nv_bfloat16*)Q.ptr, Q.row, Q.head, Q.token, (__nv_bfloat16*)O.ptr, O.row, O.head, O.token, region.base, \
        region.capacity, ranges, T, heads, (int32_t)items, scale_log2, ext)
#define AMSKV_SMALL_TILES(DD, EXT)                                                                                    \
    do {                                                                                                              \
        if (total <= 8) AMSKV_SMALL_LAUNCH(DD, EXT, 1);                                                               \
        else if (total <= 16) AMSKV_SMALL_LAUNCH(DD, EXT, 2);                                                         \
        else AMSKV_SMALL_LAUNCH(DD, EXT, 4);                                                                          \
    } while (0)
    if (D == 64) {
        if (cur) AMSKV_SMALL_TILES(64, true);
        else AMSKV_SMALL_TILES(64, false);
    } else {
        if (cur) AMSKV_SMALL_TILES(128, true);
        else AMSKV_SMALL_TILES(128, false);
    }
#undef AMSKV_SMALL_TILES
#undef AMSKV_SMALL_LAUNCH
    count_launch();
    return cudaGetLastError();
}

}  // namespace amskv
