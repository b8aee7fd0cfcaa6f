// Tensor-core attention for sm_100a: softmax(scale * Q K^T) V over the resident token ranges
// of one layer, with both products on tcgen05 and both accumulators in tensor memory.
//
// Work unit = (row, head, 128-query tile).  A CTA is persistent and walks its units; inside a
// unit it walks 64-token key/value tiles of the resident ranges.
//   warp 4      TMA producer: Q tile per unit (double-buffered for head_dim 64), K and V tiles
//               through a ring of stages, 16 tokens per bulk copy so a range's tail tile reads
//               only the 16-token groups it needs
//   warp 5      issues tcgen05.mma: S_j = Q K_j^T (128 x 64, fp32, two TMEM buffers) one tile
//               ahead of O += P_j V_j, so the softmax warps always find the next S ready
//   warps 0-3   one query row per thread (row = TMEM lane): read S with tcgen05.ld, running-max
//               softmax in exp2 form, write P as bf16 into a swizzled shared tile, and at the end
//               of the unit read O, divide by the row sum and store bf16 to global memory
// The accumulator O is rescaled in place only when the row maximum grew by more than 2^8 since
// the reference maximum was taken, so for well-conditioned logits it is never touched.
// Two CTAs share an SM.  Every wait is bounded: a wait that gives up records a status code
// and the CTA winds down.
#include <cuda.h>  // CUtensorMap and enums only; the encoder is fetched from the driver at run time

#include "kernels.cuh"
#include "sm100_ptx.cuh"

namespace amskv {

namespace {

constexpr int kQRows = 128;       // query rows per tile = TMEM lanes
constexpr int kQBoxRows = 32;     // query rows per bulk copy
constexpr int kKT = 64;           // key/value tokens per tile
constexpr int kKVBoxRows = 16;    // tokens per bulk copy
constexpr int kThreads = 192;
constexpr int kProducerWarp = 4;
constexpr int kMmaWarp = 5;
constexpr int kMaxStages = 4;
constexpr float kRescaleLog2 = 8.f;

template <int D>
struct Cfg {
    static constexpr int kHalves = D / 64;                      // 128-byte swizzle atoms per row
    static constexpr int kStages = (D == 64) ? 4 : 2;
    static constexpr int kQBufs = (D == 64) ? 2 : 1;
    static constexpr uint32_t kQBytes = kQRows * D * 2;
    static constexpr uint32_t kQHalfBytes = kQRows * 128;
    static constexpr uint32_t kKVBytes = kKT * D * 2;           // one K (or V) tile
    static constexpr uint32_t kKVHalfBytes = kKT * 128;
    static constexpr uint32_t kStageBytes = 2 * kKVBytes;
    static constexpr uint32_t kPBytes = kQRows * kKT * 2;
    static constexpr uint32_t kTileBytes = kQBufs * kQBytes + kStages * kStageBytes + kPBytes;
    static constexpr uint32_t kSmemBytes = 1024 + kTileBytes;   // barriers + alignment slack in front
    static constexpr uint32_t kTmemCols = 256;                  // S x2 (64 each) + O (D)
    static constexpr uint32_t kSCol = 0, kOCol = 2 * kKT;
    static constexpr int kCtasPerSm = 2;
};

struct Barriers {
    uint64_t q_full[2], q_empty[2];
    uint64_t kv_full[kMaxStages], kv_empty[kMaxStages];
    uint64_t s_full[2];
    uint64_t p_full, p_empty, o_full, o_empty;
    uint32_t tmem_base;
    int abort_flag;
};

// ---------------------------------------------------------------- PTX wrappers
// (the common ones come from sm100_ptx.cuh; below are the forms only this kernel uses)
using namespace ptx;

// D (+)= A * B with both operands described in shared memory by full 64-bit descriptors
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate)
{
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// 32 / 64 consecutive fp32 columns of this thread's TMEM lane; return after the data has arrived.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32])
{
    uint32_t r[32];
    ptx::tmem_ld32(taddr, r);
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, float (&v)[64])
{
    uint32_t r[64];
    ptx::tmem_ld64(taddr, r);
#pragma unroll
    for (int i = 0; i < 64; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};\n"
        "tcgen05.wait::st.sync.aligned;\n"
        ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
        "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
        "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])),
        "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])), "r"(__float_as_uint(v[16])),
        "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
        "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])),
        "r"(__float_as_uint(v[23])), "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])),
        "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])), "r"(__float_as_uint(v[28])),
        "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
        : "memory");
}


// Shared-memory matrix descriptor for a 128-byte-swizzled tile whose rows are 128 bytes:
// start address, leading and stride byte offsets in 16-byte units, descriptor version 1,
// layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46) | (2ull << 61);
}

// Tile j of the resident ranges: first token and number of valid tokens (<= 64).
__device__ __forceinline__ void tile_at(const RangeList& rl, int j, int32_t& t0, int32_t& valid)
{
    int r = 0;
    for (; r < rl.n - 1; ++r) {
        const int nt = (rl.r[r].len + kKT - 1) / kKT;
        if (j < nt) break;
        j -= nt;
    }
    t0 = rl.r[r].start + j * kKT;
    valid = min(kKT, rl.r[r].start + rl.r[r].len - t0);
}

// ---------------------------------------------------------------- kernel
template <int D>
__global__ void __launch_bounds__(kThreads, Cfg<D>::kCtasPerSm)
attend_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                 const __grid_constant__ CUtensorMap v_map, __nv_bfloat16* __restrict__ O, int64_t o_row,
                 int64_t o_head, int64_t o_tok, const RangeList ranges, int32_t T, int32_t heads, int64_t n_units,
                 int32_t nqt, int32_t n_tiles, int3 qpos, float scale_log2, int* __restrict__ status)
{
    using C = Cfg<D>;
    extern __shared__ uint8_t smem_raw[];
    Barriers* bars = reinterpret_cast<Barriers*>(smem_raw);
    volatile int* abort_flag = &bars->abort_flag;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + (uint32_t)sizeof(Barriers) + 1023u) & ~1023u;
    const uint32_t q_smem = tiles;
    const uint32_t kv_smem = q_smem + C::kQBufs * C::kQBytes;
    const uint32_t p_smem = kv_smem + C::kStages * C::kStageBytes;
    uint8_t* p_generic = smem_raw + (p_smem - raw);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    const bool layout_ok = (tiles + C::kTileBytes) <= (raw + C::kSmemBytes);
    if (threadIdx.x == 0) {
        bars->abort_flag = 0;
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bars->q_full[b]), 1);
            mbar_init(smem_u32(&bars->q_empty[b]), 1);
            mbar_init(smem_u32(&bars->s_full[b]), 1);
        }
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(smem_u32(&bars->kv_full[s]), 1);
            mbar_init(smem_u32(&bars->kv_empty[s]), 1);
        }
        mbar_init(smem_u32(&bars->p_full), 4);
        mbar_init(smem_u32(&bars->p_empty), 1);
        mbar_init(smem_u32(&bars->o_full), 1);
        mbar_init(smem_u32(&bars->o_empty), 4);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
        if (!layout_ok) report(status, kStatusSyncTimeout, abort_flag);
    }
    if (warp == kProducerWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)),
                     "r"(C::kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars->tmem_base;
    const uint32_t s_tmem = tmem + C::kSCol, o_tmem = tmem + C::kOCol;

    const uint32_t q_full0 = smem_u32(&bars->q_full[0]), q_empty0 = smem_u32(&bars->q_empty[0]);
    const uint32_t s_full0 = smem_u32(&bars->s_full[0]);
    const uint32_t p_full = smem_u32(&bars->p_full), p_empty = smem_u32(&bars->p_empty);
    const uint32_t o_full = smem_u32(&bars->o_full), o_empty = smem_u32(&bars->o_empty);
    const uint32_t kv_full0 = smem_u32(&bars->kv_full[0]), kv_empty0 = smem_u32(&bars->kv_empty[0]);

    // units of this CTA: u = blockIdx.x + n * gridDim.x, n = 0 .. my_units-1; every unit has n_tiles tiles
    const uint32_t my_units = blockIdx.x < n_units ? (uint32_t)((n_units - 1 - blockIdx.x) / gridDim.x + 1) : 0u;
    const uint32_t total_tiles = my_units * (uint32_t)n_tiles;

    if (layout_ok && warp == kProducerWarp) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t g = 0;
            uint32_t armed[kMaxStages] = {0, 0, 0, 0};
            bool ok = true;
            for (uint32_t n = 0; ok && n < my_units; ++n) {
                const int64_t u = (int64_t)blockIdx.x + (int64_t)n * gridDim.x;
                const int64_t item = u / nqt;
                const int32_t qt = (int32_t)(u - item * nqt);
                const int32_t row = (int32_t)(item / heads), head = (int32_t)(item - (int64_t)row * heads);
                const int32_t valid_rows = min(kQRows, T - qt * kQRows);
                const uint32_t qb = n % C::kQBufs, quse = n / C::kQBufs;
                if (!mbar_wait(q_empty0 + 8 * qb, (quse & 1u) ^ 1u, abort_flag)) { report(status, kStatusTmaTimeout, abort_flag); ok = false; break; }
                const int qboxes = (valid_rows + kQBoxRows - 1) / kQBoxRows;
                const uint32_t qf = q_full0 + 8 * qb;
                mbar_expect_tx(qf, (uint32_t)qboxes * kQBoxRows * D * 2);
                int c[4] = {0, 0, 0, 0};
                c[qpos.y] = head;
                c[qpos.z] = row;
                for (int bx = 0; bx < qboxes; ++bx) {
                    c[qpos.x] = qt * kQRows + bx * kQBoxRows;
#pragma unroll
                    for (int h = 0; h < C::kHalves; ++h)
                        tma_load_4d(q_smem + qb * C::kQBytes + h * C::kQHalfBytes + bx * kQBoxRows * 128, &q_map, qf,
                                    h * 64, c[1], c[2], c[3]);
                }
                for (int j = 0; j < n_tiles; ++j, ++g) {
                    int32_t t0, valid;
                    tile_at(ranges, j, t0, valid);
                    const uint32_t stage = g % C::kStages, use = g / C::kStages;
                    if (!mbar_wait(kv_empty0 + 8 * stage, (use & 1u) ^ 1u, abort_flag)) { report(status, kStatusTmaTimeout, abort_flag); ok = false; break; }
                    const uint32_t full = kv_full0 + 8 * stage;
                    const int nch = (valid + 15) >> 4;
                    mbar_expect_tx(full, (uint32_t)nch * kKVBoxRows * D * 2 * 2);
                    const uint32_t k_dst = kv_smem + stage * C::kStageBytes, v_dst = k_dst + C::kKVBytes;
                    for (int bx = 0; bx < nch; ++bx) {
#pragma unroll
                        for (int h = 0; h < C::kHalves; ++h) {
                            tma_load_3d(k_dst + h * C::kKVHalfBytes + bx * kKVBoxRows * 128, &k_map, full, h * 64,
                                        t0 + bx * kKVBoxRows, (int)item);
                            tma_load_3d(v_dst + h * C::kKVHalfBytes + bx * kKVBoxRows * 128, &v_map, full, h * 64,
                                        t0 + bx * kKVBoxRows, (int)item);
                        }
                    }
                    armed[stage] = use + 1;
                }
            }
            if (!ok) {
                // wind down: let the copies that were issued land before the CTA gives its shared memory back
                for (int s = 0; s < C::kStages; ++s)
                    if (armed[s]) {
                        for (uint32_t i = 0; i < kSpinLimit; ++i)
                            if (mbar_try_wait(kv_full0 + 8 * s, (armed[s] - 1) & 1u)) break;
                    }
            }
        }
    } else if (layout_ok && warp == kMmaWarp) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0 && total_tiles > 0) {
            bool ok = true;
            const uint32_t idesc_pv = make_idesc(kQRows, D, 1);
            // S for flat tile gs: Q of its unit times K of its stage, into S buffer gs % 2
            auto issue_s = [&](uint32_t gs) -> bool {
                const uint32_t n = gs / (uint32_t)n_tiles, j = gs - n * (uint32_t)n_tiles;
                const uint32_t qb = n % C::kQBufs, quse = n / C::kQBufs;
                const uint32_t stage = gs % C::kStages, use = gs / C::kStages;
                int32_t t0, valid;
                tile_at(ranges, (int)j, t0, valid);
                const uint32_t nch = (uint32_t)(valid + 15) >> 4;
                if (j == 0 && !mbar_wait(q_full0 + 8 * qb, quse & 1u, abort_flag)) return false;
                if (!mbar_wait(kv_full0 + 8 * stage, use & 1u, abort_flag)) return false;
                tc_fence_after();
                const uint32_t q_src = q_smem + qb * C::kQBytes;
                const uint32_t k_src = kv_smem + stage * C::kStageBytes;
                const uint32_t idesc_s = make_idesc(kQRows, nch * 16, 0);
                const uint32_t d = s_tmem + (gs & 1u) * kKT;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t a = q_src + (ks >> 2) * C::kQHalfBytes + (ks & 3) * 32;
                    const uint32_t b = k_src + (ks >> 2) * C::kKVHalfBytes + (ks & 3) * 32;
                    umma_bf16(d, make_smem_desc(a, 16, 1024), make_smem_desc(b, 16, 1024), idesc_s, ks > 0);
                }
                umma_commit(s_full0 + 8 * (gs & 1u));
                if (j == (uint32_t)n_tiles - 1) umma_commit(q_empty0 + 8 * qb);
                return true;
            };
            ok = issue_s(0);
            for (uint32_t g = 0; ok && g < total_tiles; ++g) {
                // S runs one tile ahead.  Its buffer was last read by the softmax of tile g-1, whose
                // arrival on p_full was awaited in the previous iteration.
                if (g + 1 < total_tiles && !issue_s(g + 1)) { ok = false; break; }
                const uint32_t n = g / (uint32_t)n_tiles, j = g - n * (uint32_t)n_tiles;
                const uint32_t stage = g % C::kStages;
                int32_t t0, valid;
                tile_at(ranges, (int)j, t0, valid);
                const uint32_t nch = (uint32_t)(valid + 15) >> 4;
                if (!mbar_wait(p_full, g & 1u, abort_flag)) { ok = false; break; }
                if (j == 0 && !mbar_wait(o_empty, (n & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                // O (+)= P_j V_j : M = 128, N = D channels, K = 16 * nch tokens; V is read MN-major
                const uint32_t v_src = kv_smem + stage * C::kStageBytes + C::kKVBytes;
                for (uint32_t ks = 0; ks < nch; ++ks) {
                    const uint64_t a = make_smem_desc(p_smem + ks * 32, 16, 1024);
                    const uint64_t b = make_smem_desc(v_src + ks * 2048, C::kKVHalfBytes, 1024);
                    umma_bf16(o_tmem, a, b, idesc_pv, (j > 0 || ks > 0) ? 1u : 0u);
                }
                umma_commit(kv_empty0 + 8 * stage);
                umma_commit(p_empty);
                if (j == (uint32_t)n_tiles - 1) umma_commit(o_full);
            }
            if (!ok) report(status, kStatusMmaTimeout, abort_flag);
        }
    } else if (layout_ok) {
        // ------------------------------------------------------------ softmax + epilogue (warps 0-3)
        const uint32_t lane_base = ((uint32_t)(warp * 32)) << 16;
        const int r = warp * 32 + lane;  // query row inside the tile = TMEM lane
        uint8_t* prow = p_generic + r * 128;
        uint32_t g = 0;
        bool ok = true;
        for (uint32_t n = 0; ok && n < my_units; ++n) {
            const int64_t u = (int64_t)blockIdx.x + (int64_t)n * gridDim.x;
            const int64_t item = u / nqt;
            const int32_t qt = (int32_t)(u - item * nqt);
            const int32_t valid_rows = min(kQRows, T - qt * kQRows);
            const bool warp_live = warp * 32 < valid_rows;
            float m_ref = 0.f, l = 0.f;
            for (int j = 0; j < n_tiles; ++j, ++g) {
                int32_t t0, valid;
                tile_at(ranges, j, t0, valid);
                if (!__all_sync(0xffffffffu, mbar_wait(s_full0 + 8 * (g & 1u), (g >> 1) & 1u, abort_flag))) { report(status, kStatusSyncTimeout, abort_flag); ok = false; break; }
                tc_fence_after();
                if (warp_live) {
                    const int nch = (valid + 15) >> 4;
                    float s[kKT];
                    tmem_ld64(s_tmem + (g & 1u) * kKT + lane_base, s);
                    if (valid < kKT) {
#pragma unroll
                        for (int i = 0; i < kKT; ++i)
                            if (i >= valid) s[i] = -INFINITY;
                    }
                    float mt = s[0];
#pragma unroll
                    for (int i = 1; i < kKT; ++i) mt = fmaxf(mt, s[i]);
                    bool grow = false;
                    if (j == 0) m_ref = mt;
                    else grow = (mt - m_ref) * scale_log2 > kRescaleLog2;
                    const bool any_grow = __any_sync(0xffffffffu, grow);
                    float alpha = 1.f;
                    if (grow) {
                        alpha = fast_exp2((m_ref - mt) * scale_log2);
                        m_ref = mt;
                        l *= alpha;
                    }
                    const float neg = -m_ref * scale_log2;
                    uint32_t pk[kKT / 2];
                    float sum = 0.f;
#pragma unroll
                    for (int i = 0; i < kKT / 2; ++i) {
                        const float p0 = fast_exp2(fmaf(s[2 * i], scale_log2, neg));
                        const float p1 = fast_exp2(fmaf(s[2 * i + 1], scale_log2, neg));
                        sum += p0 + p1;
                        const __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
                        pk[i] = *reinterpret_cast<const uint32_t*>(&h);
                    }
                    l += sum;
                    // the previous tile's P V product must be done before P is overwritten or O is rescaled
                    if (!__all_sync(0xffffffffu, mbar_wait(p_empty, (g & 1u) ^ 1u, abort_flag))) { report(status, kStatusSyncTimeout, abort_flag); ok = false; break; }
                    if (any_grow) {
                        tc_fence_after();
#pragma unroll
                        for (int cblk = 0; cblk < D / 32; ++cblk) {
                            float o[32];
                            tmem_ld32(o_tmem + lane_base + cblk * 32, o);
#pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] *= alpha;
                            tmem_st32(o_tmem + lane_base + cblk * 32, o);
                        }
                    }
#pragma unroll
                    for (int c = 0; c < kKT / 8; ++c) {
                        if (c * 8 < nch * 16)
                            *reinterpret_cast<uint4*>(prow + ((c ^ (r & 7)) << 4)) =
                                make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
                    }
                }
                else {
                    // A warp without live rows still may not run ahead: its arrival for tile g+1 must not be
                    // counted in the phase of tile g, so it too waits for the previous P V product.
                    if (!__all_sync(0xffffffffu, mbar_wait(p_empty, (g & 1u) ^ 1u, abort_flag))) { report(status, kStatusSyncTimeout, abort_flag); ok = false; break; }
                }
                tc_fence_before();
                fence_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full);
            }
            if (!ok) break;
            // epilogue: out = O / l
            if (!__all_sync(0xffffffffu, mbar_wait(o_full, n & 1u, abort_flag))) { report(status, kStatusSyncTimeout, abort_flag); ok = false; break; }
            tc_fence_after();
            if (warp_live) {
                const float inv = 1.f / l;
                const int32_t row = (int32_t)(item / heads), head = (int32_t)(item - (int64_t)row * heads);
                __nv_bfloat16* dst = O + row * o_row + head * o_head + (int64_t)(qt * kQRows + r) * o_tok;
#pragma unroll
                for (int cblk = 0; cblk < D / 32; ++cblk) {
                    float o[32];
                    tmem_ld32(o_tmem + lane_base + cblk * 32, o);
                    if (r < valid_rows) {
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint4 pk;
                            __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&pk);
#pragma unroll
                            for (int i = 0; i < 4; ++i)
                                h[i] = __floats2bfloat162_rn(o[c * 8 + 2 * i] * inv, o[c * 8 + 2 * i + 1] * inv);
                            reinterpret_cast<uint4*>(dst + cblk * 32)[c] = pk;
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(o_empty);
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == kProducerWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(C::kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encoder()
{
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            return (EncodeTiledFn) nullptr;
        }
        return (EncodeTiledFn)p;
    }();
    return fn;
}

bool encode_map(CUtensorMap* out, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides_bytes,
                const cuuint32_t* box)
{
    EncodeTiledFn fn = encoder();
    if (!fn) return false;
    cuuint32_t ones[4] = {1, 1, 1, 1};
    const CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), dims,
                          strides_bytes, box, ones, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

template <int D>
cudaError_t launch(const CUtensorMap& qm, const CUtensorMap& km, const CUtensorMap& vm, const Strided& O,
                   const RangeList& ranges, int32_t T, int32_t heads, int64_t units, int32_t nqt, int32_t n_tiles,
                   int3 qpos, float scale_log2, int* status, int sm_count, cudaStream_t stream)
{
    using C = Cfg<D>;
    static SharedMemoryOptIn opt_in;
    const cudaError_t oe = opt_in.ensure(attend_tc_kernel<D>, (int)C::kSmemBytes);
    if (oe != cudaSuccess) return oe;
    int64_t grid = (int64_t)sm_count * C::kCtasPerSm;
    if (grid > units) grid = units;
    attend_tc_kernel<D><<<(unsigned)grid, kThreads, C::kSmemBytes, stream>>>(
        qm, km, vm, (__nv_bfloat16*)O.ptr, O.row, O.head, O.token, ranges, T, heads, units, nqt, n_tiles, qpos,
        scale_log2, status);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

bool tc_supported(int32_t D) { return D == 64 || D == 128; }

bool tc_encode_kv_maps(const LayerRegion& region, int64_t items, int32_t D, int box_rows, void* k_map_out,
                       void* v_map_out)
{
    static_assert(sizeof(CUtensorMap) == 128, "tensor map blob size");
    const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)region.capacity, (cuuint64_t)items};
    const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)region.capacity * D * 2 * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    CUtensorMap km, vm;
    if (!encode_map(&km, region.base, 3, dims, strides, box)) return false;
    if (!encode_map(&vm, region.base + (int64_t)region.capacity * D, 3, dims, strides, box)) return false;
    memcpy(k_map_out, &km, sizeof(km));
    memcpy(v_map_out, &vm, sizeof(vm));
    return true;
}

bool tc_encode_kv_store_maps(const LayerRegion& region, int64_t items, int32_t D, int box_rows, int32_t token_extent,
                             void* k_map_out, void* v_map_out)
{
    if (token_extent < 1 || token_extent > region.capacity) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)token_extent, (cuuint64_t)items};
    const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)region.capacity * D * 2 * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    CUtensorMap km, vm;
    if (!encode_map(&km, region.base, 3, dims, strides, box)) return false;
    if (!encode_map(&vm, region.base + (int64_t)region.capacity * D, 3, dims, strides, box)) return false;
    memcpy(k_map_out, &km, sizeof(km));
    memcpy(v_map_out, &vm, sizeof(vm));
    return true;
}

// Q as a rank-4 tensor: channels, then token / head / row ordered by ascending stride.  pos[0..2]
// receive the coordinate index (1..3) of the token, head and row dimensions.
bool tc_encode_q_map(const Strided& Q, int32_t T, int32_t rows, int32_t heads, int32_t D, int box_rows, void* map_out,
                     int pos[3])
{
    struct Dim { cuuint64_t size; int64_t stride; int which; };
    Dim d[3] = {{(cuuint64_t)T, Q.token, 0}, {(cuuint64_t)heads, Q.head, 1}, {(cuuint64_t)rows, Q.row, 2}};
    for (int a = 0; a < 3; ++a)
        for (int b = a + 1; b < 3; ++b)
            if (d[b].stride < d[a].stride) { Dim t = d[a]; d[a] = d[b]; d[b] = t; }
    cuuint64_t dims[4] = {(cuuint64_t)D, d[0].size, d[1].size, d[2].size};
    cuuint64_t strides[3] = {(cuuint64_t)d[0].stride * 2, (cuuint64_t)d[1].stride * 2, (cuuint64_t)d[2].stride * 2};
    cuuint32_t box[4] = {64, 1, 1, 1};
    for (int a = 0; a < 3; ++a) {
        pos[d[a].which] = a + 1;
        if (d[a].which == 0) box[a + 1] = (cuuint32_t)box_rows;
        if (d[a].stride == 0) strides[a] = 16;  // a broadcast dimension of extent 1
    }
    CUtensorMap qm;
    if (!encode_map(&qm, Q.ptr, 4, dims, strides, box)) return false;
    memcpy(map_out, &qm, sizeof(qm));
    return true;
}

cudaError_t launch_attend_tc(const Strided& Q, const Strided& O, const LayerRegion& region, const void* k_map,
                             const void* v_map, const RangeList& ranges, int32_t T, int32_t rows, int32_t heads,
                             int32_t D, float softmax_scale, int* status, int sm_count, cudaStream_t stream)
{
    (void)region;
    if (ranges.n < 1 || ranges.total < 1 || T < 1) return cudaErrorInvalidValue;
    CUtensorMap qm;
    int pos[3];
    if (!tc_encode_q_map(Q, T, rows, heads, D, kQBoxRows, &qm, pos)) return cudaErrorNotSupported;
    CUtensorMap km, vm;
    memcpy(&km, k_map, sizeof(km));
    memcpy(&vm, v_map, sizeof(vm));
    const int32_t nqt = (T + kQRows - 1) / kQRows;
    const int64_t units = (int64_t)rows * heads * nqt;
    int32_t n_tiles = 0;
    for (int i = 0; i < ranges.n; ++i) n_tiles += (ranges.r[i].len + kKT - 1) / kKT;
    const int3 qpos = make_int3(pos[0], pos[1], pos[2]);
    const float scale_log2 = softmax_scale * 1.4426950408889634f;
    if (D == 64)
        return launch<64>(qm, km, vm, O, ranges, T, heads, units, nqt, n_tiles, qpos, scale_log2, status, sm_count, stream);
    return launch<128>(qm, km, vm, O, ranges, T, heads, units, nqt, n_tiles, qpos, scale_log2, status, sm_count, stream);
}

}  // namespace amskv
