// Tensor-core attention for sm_100a, paired form: softmax(scale * Q K^T) V over the resident
// token ranges of one layer, both products on tcgen05 with every accumulator in tensor memory.
//
// A CTA is persistent and walks "pairs".  A pair is two streams, A and B, each a (row, head,
// 128-query tile) that runs through the same number of 64-token key/value tiles:
//   * more than 128 query tokens: the two streams are two query tiles of ONE item, so each
//     key/value tile is fetched into shared memory once and used by both;
//   * at most 128 query tokens: the two streams are two different items with their own tiles.
// Stream B is absent when the pair has no second member.
//   warps 0-3    softmax group of stream A: one query row per thread (row = TMEM lane)
//   warps 4-7    softmax group of stream B
//   warp 8       TMA producer of the key/value tiles (ring of stages, 16 tokens per bulk copy so a
//                range's tail tile reads only the 16-token groups it needs)
//   warp 9       issues tcgen05.mma for both streams, alternating between them
// Per stream and tile: S = Q K^T (128 x 64 fp32 in TMEM) -> the group reads S with tcgen05.ld,
// exponentiates in exp2 form against a reference maximum, packs P to bf16 and writes it back
// over S with tcgen05.st -> O += P V with P read from TMEM.  S and P share their columns, so
// there is no shared-memory tile for P.  While one group exponentiates, the tensor pipe works
// for the other.  The reference maximum of a row is the maximum of its first tile; O and the
// row sum are rescaled only when a later tile exceeds it by more than 2^8, so for
// well-conditioned logits they are never touched.  Launches of three key tiles or more (kLazy)
// do not even take the later tiles' maxima: a tile is exponentiated against the reference as it
// stands, and only a row whose tile sum leaves the range (beyond 2^64, or not a number) makes
// its warp take the true maxima, rescale and form the tile again.  The first lane of each group fetches its
// next query tile as soon as the last S of the current one has landed.
// Every wait is bounded: a wait that gives up records a status code, all roles wind down,
// copies in flight are awaited and the tensor memory is freed.
#include "kernels.cuh"
#include "sm100_ptx.cuh"

namespace amskv {

namespace {

constexpr int kQRows = 128;       // query rows per tile = TMEM lanes
constexpr int kMaxDenRuns = 16;   // runs of attended tokens a density launch can tell apart
constexpr int kQBoxRows = 32;     // query rows per bulk copy
constexpr int kKT = 64;           // key/value tokens per tile
constexpr int kKVBoxRows = 16;    // tokens per bulk copy
constexpr int kGroupWarps = 4;
constexpr int kProducerWarp = 8;
constexpr int kMmaWarp = 9;        // first MMA-issuing warp; Cfg<D>::kMmaWarps of them
constexpr int kMaxStages = 4;
constexpr float kRescaleLog2 = 8.f;
constexpr int kQSplitRows = 64;   // query tiles of at most this many rows are double-buffered inside their slot
constexpr float kLazySumLimit = 1.8446744e19f;   // 2^64: see the kLazy form of the softmax loop
constexpr int kPolyEvery = 6;     // every 6th pair of exponentials goes to the FMA pipe (0: none); swept 2, 3, 4, 6, 8

// kWide: one CTA per SM with two S buffers per stream and an issuing warp per stream (below): the form
// 128 channels use.  64 channels use the two-CTA form (the wide form is instantiable for them, but lost
// wherever it was measured).
// kDen: the launch also accumulates the attention density (below): two CTAs per SM then run with three
// key/value stages, the fourth stage's 16 KB holding the per-row sums.
template <int D, bool kWide, bool kDen = false>
struct Cfg {
    static_assert(D == 64 || kWide, "128 channels always use the wide form");
    static constexpr int kHalves = D / 64;                      // 128-byte swizzle atoms per row
    static constexpr int kStages = (kDen && !kWide) ? 3 : 4;
    static constexpr uint32_t kQBytes = kQRows * D * 2;         // one query tile
    static constexpr uint32_t kQHalfBytes = kQRows * 128;
    static constexpr uint32_t kKVBytes = kKT * D * 2;           // one K (or V) tile
    static constexpr uint32_t kKVHalfBytes = kKT * 128;
    static constexpr uint32_t kStageBytes = 2 * kKVBytes;
    static constexpr uint32_t kDenBytes = kDen ? 2u * kMaxDenRuns * kQRows * 4u : 0u;   // [stream][run][row] fp32
    static constexpr uint32_t kTileBytes = 2 * kQBytes + kStages * kStageBytes + kDenBytes;
    static constexpr uint32_t kSmemBytes = 4096 + kTileBytes;   // barriers, tile table and alignment slack in front
    // Score buffers per stream.  With 64 channels two CTAs share the SM's 512 tensor-memory columns and a
    // stream has one S buffer (S and O of two streams: 256 columns).  With 128 channels one CTA has all
    // 512 columns and a stream has two S buffers used alternately, so that S of the next tile is computed
    // while the softmax of the current one runs (2 x 2 x 64 for S, 2 x 128 for O).
    static constexpr int kSBufs = kWide ? 2 : 1;
    // MMA-issuing warps.  One thread issuing for both streams is enough with 64 channels (two CTAs per SM
    // share the tensor pipe).  With 128 channels a stream's tile is 12 instructions of 50-65 clocks of issue
    // each plus three barrier waits, and a single issuer for both streams was what bound the kernel: each
    // stream gets its own issuing warp (one CTA per SM, so the registers are there).
    static constexpr int kMmaWarps = kWide ? 2 : 1;
    static constexpr int kThreads = (kMmaWarp + kMmaWarps) * 32;
    static constexpr uint32_t kTmemCols = kWide ? 512 : 256;
    static constexpr uint32_t kSCol = 0, kOCol = 2 * kSBufs * kKT;
    static constexpr int kCtasPerSm = kWide ? 1 : 2;
    // Extents every address in the kernel is derived from, checked at compile time:
    //  - tensor memory: S buffers of both streams, then O of both streams, inside the allocation, and the
    //    allocations of all CTAs of an SM inside its 512 columns (otherwise tcgen05.alloc would block);
    //  - shared memory: the CTAs of an SM (each with 1 KB reserved by the system) inside 228 KB;
    //  - matrix descriptors: a start address is 14 bits of 16-byte units (256 KB), so adding a stage, half
    //    or K-step offset to the low descriptor word can never carry into the field above it.
    static_assert(kOCol + 2 * D <= kTmemCols, "S and O of both streams must fit the tensor-memory allocation");
    static_assert((kTmemCols & (kTmemCols - 1)) == 0 && kTmemCols >= 32 && kCtasPerSm * kTmemCols <= 512,
                  "tensor-memory allocations of an SM's CTAs");
    static_assert(kCtasPerSm * (kSmemBytes + 1024) <= 228 * 1024, "shared memory of an SM's CTAs");
    static_assert(kKVHalfBytes % 1024 == 0 && kQHalfBytes % 1024 == 0 && kStageBytes % 1024 == 0 && kQBytes % 1024 == 0,
                  "swizzle atoms must stay 1024-byte aligned");
    static_assert(228 * 1024 <= (1 << 18), "descriptor start-address field covers all of shared memory");
    static_assert(kStages <= kMaxStages, "barrier arrays");
};

constexpr int kTileTab = 256;     // tiles whose (first token, valid tokens) are tabulated in shared memory

struct Barriers {
    uint64_t q_full[2][2];     // [stream][half]: see kQSplitRows
    uint64_t kv_full[kMaxStages], kv_empty[kMaxStages];
    uint64_t s_full[2][2], p_full[2][2];   // [stream][S buffer]
    uint64_t o_full[2], pv_done[2];
    uint32_t tmem_base;
    int abort_flag;
    int2 tile_tab[kTileTab];
};

static_assert(sizeof(Barriers) + 1024 <= 4096, "barrier block must fit in front of the 1024-byte aligned tiles");

// How the pairs (units of two streams) of one launch are formed; shared by every role.  The first
// n_shared pairs are two consecutive query tiles of one item, which share every key/value tile in
// shared memory; an item with an odd number of query tiles has one tile left over, and the left-over
// tiles of two consecutive items form a pair whose streams fetch their own key/value tiles (with one
// query tile per item every pair is of that kind).
struct PairPlan {
    int32_t nqt;          // query tiles per item
    int32_t npi;          // shared pairs per item = nqt / 2
    int32_t n_items;
    int32_t n_shared;     // = n_items * npi
    int32_t n_pairs;      // n_shared + ceil(n_items * (nqt & 1) / 2)
    int32_t kind;         // 0: no pair is shared, 1: every pair is, 2: both kinds (so that the common cases test a launch constant)
};

// The current scale read from the caller's K/V tensors instead of the cache: the last entry of the
// range list stands for it (start 0, len T).  With `store` every tile fetched that way is also written
// to the scale's place in the cache (the append fused into attention).
constexpr int32_t kExtFlag = 1 << 30;   // marks such a tile's first token in the tile table
struct ExtArgs {
    CUtensorMap k64, v64, k16, v16;   // rank-4 maps of the caller's K and V (64- and 16-token boxes)
    CUtensorMap k_store, v_store;     // the layer's region, clipped at the end of the scale's place (64-token boxes)
    int32_t range;                    // index of the range that stands for the current scale
    int32_t store;
    int32_t dst;                      // first position of the scale in the per-item region
    int3 pos;                         // coordinate slots of token, head and row in the rank-4 maps
    int32_t rider_tok, rider_valid;   // older cache tokens that ride in the spare box of the scale's last tile
};

// Attention density as a by-product (Sec. 4.1): the range list of such a launch has one entry per piece of a
// run of attended tokens (never merged across runs), so every key tile belongs to one run and a row's
// un-normalised probability mass per run is a running sum of the tile sums the softmax computes anyway.
struct DenArgs {
    double* out;                       // [heads][n_runs], accumulated with atomic adds
    int32_t n_runs;
    float weight[kMaxDenRuns];         // 1 / (rows * tokens of the run)
    int8_t run_of_range[kMaxRanges];
};

struct Stream {
    int32_t item;
    int32_t qt;
    bool valid;
};

__device__ __forceinline__ bool pair_is_shared(const PairPlan& pp, int32_t pair)
{
    return pp.kind == 2 ? pair < pp.n_shared : pp.kind == 1;
}

__device__ __forceinline__ Stream stream_of(const PairPlan& pp, int32_t pair, int g)
{
    Stream s;
    if (pair_is_shared(pp, pair)) {
        s.item = pp.npi == 1 ? pair : pair / pp.npi;
        s.qt = 2 * (pair - s.item * pp.npi) + g;
        s.valid = true;
    } else {
        s.item = 2 * (pair - pp.n_shared) + g;
        s.qt = pp.nqt - 1;
        s.valid = s.item < pp.n_items;
    }
    return s;
}

using namespace ptx;


// Tile j of the resident ranges: first token and number of valid tokens (<= 64).
// A tile of range `ext_range` (the current scale in the caller's tensors) carries kExtFlag in t0.
__device__ __forceinline__ void tile_at(const RangeList& rl, int j, int32_t& t0, int32_t& valid, int ext_range = -1,
                                        int* range_index = nullptr)
{
    int r = 0;
    for (; r < rl.n - 1; ++r) {
        const int nt = (rl.r[r].len + kKT - 1) / kKT;
        if (j < nt) break;
        j -= nt;
    }
    t0 = rl.r[r].start + j * kKT;
    valid = min(kKT, rl.r[r].start + rl.r[r].len - t0);
    if (r == ext_range) t0 |= kExtFlag;
    if (range_index) *range_index = r;
}

// ---------------------------------------------------------------- kernel
template <int D, bool kExt, bool kWide, bool kDen, bool kLazy, bool kShort>
__global__ void __launch_bounds__(Cfg<D, kWide, kDen>::kThreads, Cfg<D, kWide, kDen>::kCtasPerSm)
attend_pair_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                   const __grid_constant__ CUtensorMap v_map, const __grid_constant__ CUtensorMap k_map64,
                   const __grid_constant__ CUtensorMap v_map64, const __grid_constant__ ExtArgs ext,
                   __nv_bfloat16* __restrict__ O, int64_t o_row,
                   int64_t o_head, int64_t o_tok, const RangeList ranges, int32_t T, int32_t heads,
                   const PairPlan pp, int32_t n_tiles, int3 qpos, float scale_log2, int* __restrict__ status,
                   const __grid_constant__ DenArgs den)
{
    static_assert(!(kDen && kExt), "the density form serves the plain attend call");
    const int ext_range = kExt ? ext.range : -1;
    using C = Cfg<D, kWide, kDen>;
    extern __shared__ uint8_t smem_raw[];
    Barriers* bars = reinterpret_cast<Barriers*>(smem_raw);
    volatile int* abort_flag = &bars->abort_flag;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + (uint32_t)sizeof(Barriers) + 1023u) & ~1023u;
    const uint32_t q_smem = tiles;
    const uint32_t kv_smem = q_smem + 2 * C::kQBytes;
    // the warp index is taken through a shuffle so that the compiler knows it to be the same in every
    // lane: role branches are then uniform branches and the issuing warps keep their operands uniform
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;

    const bool layout_ok = (tiles + C::kTileBytes) <= (raw + C::kSmemBytes);
    if (threadIdx.x == 0) {
        bars->abort_flag = 0;
        for (int g = 0; g < 2; ++g) {
            mbar_init(smem_u32(&bars->q_full[g][0]), 1);
            mbar_init(smem_u32(&bars->q_full[g][1]), 1);
            for (int b = 0; b < 2; ++b) {
                mbar_init(smem_u32(&bars->s_full[g][b]), 1);
                mbar_init(smem_u32(&bars->p_full[g][b]), kGroupWarps);
            }
            mbar_init(smem_u32(&bars->pv_done[g]), 1);
            mbar_init(smem_u32(&bars->o_full[g]), 1);
        }
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(smem_u32(&bars->kv_full[s]), 1);
            mbar_init(smem_u32(&bars->kv_empty[s]), C::kMmaWarps);   // one arrival per issuing warp
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!layout_ok) report(status, kStatusSyncTimeout, abort_flag);
    }
    for (int j = threadIdx.x; j < n_tiles && j < kTileTab; j += C::kThreads) {
        int32_t t0, valid;
        int ri = 0;
        tile_at(ranges, j, t0, valid, ext_range, &ri);
        bars->tile_tab[j] = make_int2(t0, kDen ? (valid | ((int32_t)den.run_of_range[ri] << 8)) : valid);
    }
    if (layout_ok) {
        // query rows a tile does not cover keep whatever the slot held before; start them at zero
        uint4* qz = reinterpret_cast<uint4*>(smem_raw + (q_smem - raw));
        for (uint32_t i = threadIdx.x; i < 2 * C::kQBytes / 16; i += C::kThreads) qz[i] = make_uint4(0, 0, 0, 0);
        if constexpr (kDen) {
            uint4* dz = reinterpret_cast<uint4*>(smem_raw + (kv_smem - raw) + C::kStages * C::kStageBytes);
            for (uint32_t i = threadIdx.x; i < C::kDenBytes / 16; i += C::kThreads) dz[i] = make_uint4(0, 0, 0, 0);
        }
        fence_async_smem();
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
    const uint32_t tmem = __shfl_sync(0xffffffffu, bars->tmem_base, 0);
    // (in a density launch `valid` carries the tile's run in its bits 8..15; tile_run() strips it)
    auto tile_of = [&](int j, int32_t& t0, int32_t& valid) {
        if (j < kTileTab) {
            const int2 e = bars->tile_tab[j];
            t0 = e.x;
            valid = e.y;
        } else {
            int ri = 0;
            tile_at(ranges, j, t0, valid, ext_range, &ri);
            if (kDen) valid |= (int32_t)den.run_of_range[ri] << 8;
        }
    };
    auto tile_run = [](int32_t& valid) -> int {
        const int run = kDen ? (valid >> 8) : 0;
        if (kDen) valid &= 0xff;
        return run;
    };

    const uint32_t q_full0 = smem_u32(&bars->q_full[0][0]);   // [g][half] at + 16 * g + 8 * half
    // With at most 64 query tokens a query tile fills half of its slot, so the slot holds the tiles of two
    // consecutive units and the next unit's queries are fetched a whole unit ahead.  The MMA reads 128
    // rows from wherever the tile starts; what it reads past the tile only reaches dead rows of S.
    const bool q_split = T <= kQSplitRows;
    constexpr uint32_t kQHalfSlot = kQSplitRows * 128;   // bytes from the first to the second tile of a slot
    const uint32_t s_full0 = smem_u32(&bars->s_full[0][0]), p_full0 = smem_u32(&bars->p_full[0][0]);   // + 16 g + 8 buffer
    const uint32_t pv_done0 = smem_u32(&bars->pv_done[0]);
    // S buffer and barrier phase of a stream's flat tile index: with two buffers they alternate, and each
    // buffer's barriers see every other tile
    auto buf_of = [](uint32_t t) -> uint32_t { return C::kSBufs == 2 ? (t & 1u) : 0u; };
    auto par_of = [](uint32_t t) -> uint32_t { return C::kSBufs == 2 ? ((t >> 1) & 1u) : (t & 1u); };
    const uint32_t o_full0 = smem_u32(&bars->o_full[0]);
    const uint32_t kv_full0 = smem_u32(&bars->kv_full[0]), kv_empty0 = smem_u32(&bars->kv_empty[0]);

    // pairs of this CTA: p = blockIdx.x + n * gridDim.x, n = 0 .. my_pairs-1
    const uint32_t my_pairs = (int32_t)blockIdx.x < pp.n_pairs ? ((uint32_t)pp.n_pairs - 1u - blockIdx.x) / gridDim.x + 1u : 0u;

    // The producer and the MMA issuer run their loops with the whole warp converged and let one
    // elected lane issue: addresses, descriptors and coordinates then stay warp-uniform values,
    // which keeps the per-instruction issue cost of the TMA and tcgen05 instructions low.
    if (layout_ok && warp == kProducerWarp) {
        // ------------------------------------------------------------ TMA producer of K/V tiles
        uint32_t sq = 0;  // stages issued so far
        bool ok = true;
        // Fused append: a tile of the current scale is written to the cache two stages after it was
        // requested (it has landed by then, so the wait costs nothing), by lane 0, as one bulk group per
        // stage; before a stage is refilled, every group but the two newest has finished reading it.
        const bool storing = kExt && ext.store != 0;
        if (kShort && lane == 0) {
            prefetch_tensormap(&k_map);
            prefetch_tensormap(&v_map);
            prefetch_tensormap(&k_map64);
            prefetch_tensormap(&v_map64);
            if (kExt) {
                prefetch_tensormap(&ext.k64);
                prefetch_tensormap(&ext.v64);
                prefetch_tensormap(&ext.k16);
                prefetch_tensormap(&ext.v16);
                if (storing) {
                    prefetch_tensormap(&ext.k_store);
                    prefetch_tensormap(&ext.v_store);
                }
            }
        }
        uint32_t st_sq[2] = {0, 0};
        int32_t st_tok[2] = {0, 0}, st_item[2] = {0, 0};
        int st_n = 0;
        auto store_front = [&]() -> bool {
            const uint32_t stage = st_sq[0] % C::kStages, use = st_sq[0] / C::kStages;
            if (!warp_wait(kv_full0 + 8 * stage, use & 1u, abort_flag)) return false;
            if (lane == 0) {
                const uint32_t k_src = kv_smem + stage * C::kStageBytes, v_src = k_src + C::kKVBytes;
#pragma unroll
                for (int h = 0; h < C::kHalves; ++h) {
                    tma_store_3d(&ext.k_store, k_src + h * C::kKVHalfBytes, h * 64, ext.dst + st_tok[0], st_item[0]);
                    tma_store_3d(&ext.v_store, v_src + h * C::kKVHalfBytes, h * 64, ext.dst + st_tok[0], st_item[0]);
                }
            }
            st_sq[0] = st_sq[1];
            st_tok[0] = st_tok[1];
            st_item[0] = st_item[1];
            --st_n;
            return true;
        };
        for (uint32_t n = 0; ok && n < my_pairs; ++n) {
            const int32_t pair = (int32_t)(blockIdx.x + n * gridDim.x);
            const Stream sa = stream_of(pp, pair, 0), sb = stream_of(pp, pair, 1);
            const bool shared = pair_is_shared(pp, pair);
            const int per_tile = (!shared && sb.valid) ? 2 : 1;
            // one unit per item writes the item's tiles: the unit of its first query tiles
            const bool unit_stores = storing && (shared ? sa.qt == 0 : pp.nqt == 1);
            for (int j = 0; ok && j < n_tiles; ++j) {
                int32_t t0, valid;
                tile_of(j, t0, valid);
                (void)tile_run(valid);
                const bool from_ext = kExt && (t0 & kExtFlag) != 0;
                t0 &= ~kExtFlag;
                const int nch = (valid + 15) >> 4;
                const bool rider = kExt && ext.rider_valid > 0 && j == n_tiles - 1;   // one more box, from the cache
                for (int g = 0; g < per_tile; ++g, ++sq) {
                    const int item = g == 0 ? sa.item : sb.item;
                    const uint32_t stage = sq % C::kStages, use = sq / C::kStages;
                    if (storing) {
                        if (st_n > 0 && st_sq[0] + 2 <= sq && !store_front()) {
                            ok = false;
                            break;
                        }
                        if (lane == 0) {
                            bulk_commit();
                            bulk_wait_read<2>();
                        }
                        __syncwarp();
                    }
                    if (!warp_wait(kv_empty0 + 8 * stage, (use & 1u) ^ 1u, abort_flag)) {
                        ok = false;
                        break;
                    }
                    const uint32_t full = kv_full0 + 8 * stage;
                    const uint32_t k_dst = kv_smem + stage * C::kStageBytes, v_dst = k_dst + C::kKVBytes;
                    // A tile of the caller's tensors that no rider shares its stage with is one 64-token box whatever
                    // its length: the tokens past the end of the scale are outside the tensor, cost no traffic and
                    // arrive as zeros (the products never read their rows, the fused write is clipped at the scale's end).
                    const bool whole_box = nch == kKT / kKVBoxRows || (kShort && from_ext && !rider);
                    if (whole_box) {
                        if (elect_one()) {
                            mbar_expect_tx(full, (uint32_t)kKT * D * 2 * 2);
                            if (from_ext) {
                                const int32_t row = item / heads, head = item - row * heads;
                                int c[4] = {0, 0, 0, 0};
                                c[ext.pos.y] = head;
                                c[ext.pos.z] = row;
                                c[ext.pos.x] = t0;
#pragma unroll
                                for (int h = 0; h < C::kHalves; ++h) {
                                    tma_load_4d(k_dst + h * C::kKVHalfBytes, &ext.k64, full, h * 64, c[1], c[2], c[3]);
                                    tma_load_4d(v_dst + h * C::kKVHalfBytes, &ext.v64, full, h * 64, c[1], c[2], c[3]);
                                }
                            } else {
#pragma unroll
                                for (int h = 0; h < C::kHalves; ++h) {
                                    tma_load_3d(k_dst + h * C::kKVHalfBytes, &k_map64, full, h * 64, t0, item);
                                    tma_load_3d(v_dst + h * C::kKVHalfBytes, &v_map64, full, h * 64, t0, item);
                                }
                            }
                        }
                    } else if (!kShort) {
                        // 16-token boxes (and the rider's box), issued by one lane
                        if (elect_one()) {
                            mbar_expect_tx(full, (uint32_t)(nch + (rider ? 1 : 0)) * kKVBoxRows * D * 2 * 2);
                            if (rider) {
#pragma unroll
                                for (int h = 0; h < C::kHalves; ++h) {
                                    tma_load_3d(k_dst + h * C::kKVHalfBytes + nch * kKVBoxRows * 128, &k_map, full, h * 64,
                                                ext.rider_tok, item);
                                    tma_load_3d(v_dst + h * C::kKVHalfBytes + nch * kKVBoxRows * 128, &v_map, full, h * 64,
                                                ext.rider_tok, item);
                                }
                            }
                            if (from_ext) {
                                const int32_t row = item / heads, head = item - row * heads;
                                int c[4] = {0, 0, 0, 0};
                                c[ext.pos.y] = head;
                                c[ext.pos.z] = row;
                                for (int bx = 0; bx < nch; ++bx) {
                                    c[ext.pos.x] = t0 + bx * kKVBoxRows;
#pragma unroll
                                    for (int h = 0; h < C::kHalves; ++h) {
                                        tma_load_4d(k_dst + h * C::kKVHalfBytes + bx * kKVBoxRows * 128, &ext.k16, full, h * 64,
                                                    c[1], c[2], c[3]);
                                        tma_load_4d(v_dst + h * C::kKVHalfBytes + bx * kKVBoxRows * 128, &ext.v16, full, h * 64,
                                                    c[1], c[2], c[3]);
                                    }
                                }
                            } else {
                                for (int bx = 0; bx < nch; ++bx) {
#pragma unroll
                                    for (int h = 0; h < C::kHalves; ++h) {
                                        tma_load_3d(k_dst + h * C::kKVHalfBytes + bx * kKVBoxRows * 128, &k_map, full, h * 64,
                                                    t0 + bx * kKVBoxRows, item);
                                        tma_load_3d(v_dst + h * C::kKVHalfBytes + bx * kKVBoxRows * 128, &v_map, full, h * 64,
                                                    t0 + bx * kKVBoxRows, item);
                                    }
                                }
                            }
                        }
                    } else {
                        // Short units (at most four key tiles): one lane per bulk copy, all issued by one instruction.  A
                        // lane issuing six or eight copies one after the other is what such units wait for (the issuing
                        // warp of a 36-token scale spent half its time waiting for tiles).
                        if (lane == 0) mbar_expect_tx(full, (uint32_t)(nch + (rider ? 1 : 0)) * kKVBoxRows * D * 2 * 2);
                        __syncwarp();
                        const int n_main = 2 * C::kHalves * nch, n_ops = n_main + (rider ? 2 * C::kHalves : 0);
                        if (lane < n_ops) {
                            const bool is_rider = lane >= n_main;
                            const int o = is_rider ? lane - n_main : lane;
                            const int h = o % C::kHalves, kv = (o / C::kHalves) & 1, bx = is_rider ? nch : o / (2 * C::kHalves);
                            const uint32_t dst = (kv ? v_dst : k_dst) + h * C::kKVHalfBytes + bx * kKVBoxRows * 128;
                            if (from_ext && !is_rider) {
                                const int32_t row = item / heads, head = item - row * heads;
                                int c[4] = {0, 0, 0, 0};
                                c[ext.pos.y] = head;
                                c[ext.pos.z] = row;
                                c[ext.pos.x] = t0 + bx * kKVBoxRows;
                                tma_load_4d(dst, kv ? &ext.v16 : &ext.k16, full, h * 64, c[1], c[2], c[3]);
                            } else {
                                tma_load_3d(dst, kv ? &v_map : &k_map, full, h * 64, is_rider ? ext.rider_tok : t0 + bx * kKVBoxRows, item);
                            }
                        }
                    }
                    __syncwarp();
                    if (from_ext && unit_stores) {
                        st_sq[st_n] = sq;
                        st_tok[st_n] = t0;
                        st_item[st_n] = item;
                        ++st_n;
                    }
                }
            }
        }
        if (storing) {
            while (ok && st_n > 0) ok = store_front();
            if (lane == 0) {
                bulk_commit();
                bulk_wait_all();   // the writes are complete, and the stages no longer read, before the CTA ends
            }
            __syncwarp();
        }
        if (!ok) {
            if (lane == 0) report(status, kStatusTmaTimeout, abort_flag);
            // wind down: let the copies that were issued land before the CTA gives its shared memory back
            const uint32_t first = sq > (uint32_t)C::kStages ? sq - C::kStages : 0u;
            for (uint32_t q = first; q < sq; ++q) {
                const uint32_t stage = q % C::kStages, use = q / C::kStages;
                for (uint32_t i = 0; i < kSpinLimit; ++i)
                    if (mbar_try_wait(kv_full0 + 8 * stage, use & 1u)) break;
            }
        }
    } else if (layout_ok && warp >= kMmaWarp) {
        // ------------------------------------------------------------ MMA issuer(s)
        // With two issuing warps, warp kMmaWarp + g issues for stream g only; both walk the same loop, so the
        // stage counter advances alike in both.  A commit covers the issuing thread's own instructions only,
        // hence a key/value stage is released by one arrival per issuing warp: each commits its own P V on a
        // shared tile, and the one stream that uses a tile of its own commits twice.
        const int my_g = C::kMmaWarps == 2 ? warp - kMmaWarp : -1;   // -1: this warp issues for both streams
        if (my_pairs > 0) {
            bool ok = true;
            const uint32_t idesc_pv = make_idesc(kQRows, D, 1);
            const uint32_t k_lo0 = desc_lo(kv_smem, 16);                             // K tile of stage 0, K-major
            const uint32_t v_lo0 = desc_lo(kv_smem + C::kKVBytes, C::kKVHalfBytes);  // V tile of stage 0, MN-major
            const uint32_t q_lo0 = desc_lo(q_smem, 16);
            constexpr uint32_t kStageLo = C::kStageBytes >> 4, kQLo = C::kQBytes >> 4;
            // per stream: the tile whose S was issued last and whose P V is still to be issued
            uint32_t pv_stage[2] = {0, 0}, pv_nch[2] = {0, 0}, pv_t[2] = {0, 0};
            bool pv_live[2] = {false, false}, pv_first[2] = {false, false}, pv_release[2] = {false, false},
                 pv_last[2] = {false, false}, pv_twice[2] = {false, false};
            uint32_t tcount[2] = {0, 0};   // tiles issued per stream
            uint32_t ucount[2] = {0, 0};   // units started per stream
            uint32_t q_half[2] = {0, 0};   // half of the query slot the current unit of each stream uses
            uint32_t sq = 0;

            // O (+)= P V : M = 128, N = D channels, K = 16 * nch tokens; P from TMEM (packed over S),
            // V read MN-major from its stage
            auto issue_pv = [&](const int g) -> bool {
                const uint32_t t = pv_t[g];  // flat tile index of this stream
                if (!warp_wait(p_full0 + 16 * g + 8 * buf_of(t), par_of(t), abort_flag)) return false;
                // (a unit's first P V overwrites O: every warp of the group arrives on p_full for that tile
                // only after its epilogue of the previous unit, so O has been read by then)
                tc_fence_after();
                const uint32_t v_lo = v_lo0 + pv_stage[g] * kStageLo;
                const uint32_t p_tmem = tmem + C::kSCol + (g * C::kSBufs + buf_of(t)) * kKT;
                const uint32_t o_tmem = tmem + C::kOCol + g * D;
                const uint32_t nch = pv_nch[g];
                if (elect_one()) {
                    umma_ts(o_tmem, p_tmem, v_lo, kDescHi, idesc_pv, pv_first[g] ? 0u : 1u);
                    if (nch > 1) umma_ts(o_tmem, p_tmem + 8, v_lo + (2048 >> 4), kDescHi, idesc_pv, 1u);
                    if (nch > 2) umma_ts(o_tmem, p_tmem + 16, v_lo + (4096 >> 4), kDescHi, idesc_pv, 1u);
                    if (nch > 3) umma_ts(o_tmem, p_tmem + 24, v_lo + (6144 >> 4), kDescHi, idesc_pv, 1u);
                    if (pv_release[g]) umma_commit(kv_empty0 + 8 * pv_stage[g]);
                    if (C::kMmaWarps == 2 && pv_twice[g]) umma_commit(kv_empty0 + 8 * pv_stage[g]);
                    if (pv_last[g]) umma_commit(o_full0 + 8 * g);
                    if (C::kSBufs == 2) umma_commit(pv_done0 + 8 * g);   // read by the (rare) rescale of O only
                }
                __syncwarp();
                return true;
            };

            for (uint32_t n = 0; ok && n < my_pairs; ++n) {
                const int32_t pair = (int32_t)(blockIdx.x + n * gridDim.x);
                const int ng = stream_of(pp, pair, 1).valid ? 2 : 1;
                const bool shared = pair_is_shared(pp, pair);
                for (int j = 0; ok && j < n_tiles; ++j) {
                    int32_t t0, valid;
                    tile_of(j, t0, valid);
                    (void)tile_run(valid);
                    const uint32_t nch = ((uint32_t)(valid + 15) >> 4) +
                                         ((kExt && ext.rider_valid > 0 && j == n_tiles - 1) ? 1u : 0u);
                    const uint32_t idesc_s = make_idesc(kQRows, nch * 16, 0);
#pragma unroll
                    for (int g = 0; g < 2; ++g) {
                        if (!ok) continue;
                        if (my_g >= 0 && g != my_g) continue;
                        if (g >= ng) {
                            // the stream is absent from this pair: its last P V of the previous pair must not
                            // wait for a next S that is not coming soon (it also holds a key/value stage)
                            if (pv_live[g]) {
                                if (!issue_pv(g)) ok = false;
                                pv_live[g] = false;
                            }
                            continue;
                        }
                        // S = Q K^T for (stream g, tile j).  Its operands are waited for first: they have
                        // almost always landed, and this keeps the two waits out of the P -> P V -> S chain.
                        const uint32_t seq = shared ? sq : sq + g;
                        const uint32_t stage = seq % C::kStages, use = seq / C::kStages;
                        if (j == 0) {
                            const uint32_t u = ucount[g];
                            q_half[g] = q_split ? (u & 1u) : 0u;
                            const uint32_t parity = q_split ? ((u >> 1) & 1u) : (u & 1u);
                            if (!warp_wait(q_full0 + 16 * g + 8 * q_half[g], parity, abort_flag)) { ok = false; continue; }
                            ++ucount[g];
                        }
                        if (!(shared && g == 1 && my_g < 0)) {  // one issuer: the second stream of a shared tile finds it landed
                            if (!warp_wait(kv_full0 + 8 * stage, use & 1u, abort_flag)) { ok = false; continue; }
                        }
                        // One S buffer: the pending P V of the previous tile goes first, because this S
                        // overwrites its P.  Two buffers: this S goes first and runs on the tensor pipe while
                        // the softmax of the previous tile finishes (streams with tiles of their own keep the
                        // first order: they need their key/value stages back sooner).
                        const bool s_first = C::kSBufs == 2 && shared;
                        if (!s_first && pv_live[g] && !issue_pv(g)) { ok = false; continue; }
                        tc_fence_after();
                        const uint32_t t_now = tcount[g];
                        const uint32_t q_lo = q_lo0 + g * kQLo + q_half[g] * (kQHalfSlot >> 4);
                        const uint32_t k_lo = k_lo0 + stage * kStageLo;
                        const uint32_t d = tmem + C::kSCol + (g * C::kSBufs + buf_of(t_now)) * kKT;
                        if (elect_one()) {
                            umma_ss<false>(d, q_lo, k_lo, kDescHi, idesc_s);
#pragma unroll
                            for (int ks = 1; ks < D / 16; ++ks) {
                                constexpr uint32_t kQH = C::kQHalfBytes >> 4, kKH = C::kKVHalfBytes >> 4;
                                umma_ss<true>(d, q_lo + (ks >> 2) * kQH + (ks & 3) * 2,
                                              k_lo + (ks >> 2) * kKH + (ks & 3) * 2, kDescHi, idesc_s);
                            }
                            umma_commit(s_full0 + 16 * g + 8 * buf_of(t_now));
                        }
                        __syncwarp();
                        if (s_first && pv_live[g] && !issue_pv(g)) { ok = false; continue; }
                        pv_live[g] = true;
                        pv_stage[g] = stage;
                        pv_nch[g] = nch;
                        pv_t[g] = t_now;
                        pv_first[g] = (j == 0);
                        pv_last[g] = (j == n_tiles - 1);
                        pv_release[g] = (shared && my_g < 0) ? (g == ng - 1) : true;
                        pv_twice[g] = !shared;
                        ++tcount[g];
                    }
                    sq += shared ? 1 : ng;
                }
            }
#pragma unroll
            for (int g = 0; g < 2; ++g)
                if (ok && (my_g < 0 || g == my_g) && pv_live[g] && !issue_pv(g)) ok = false;
            if (!ok && lane == 0) report(status, kStatusMmaTimeout, abort_flag);
        }
    } else if (layout_ok) {
        // ------------------------------------------------------------ softmax + epilogue (warps 0-7)
        const int g = warp >> 2, wq = warp & 3;
        const uint32_t lane_base = ((uint32_t)(wq * 32)) << 16;
        const int r = wq * 32 + lane;  // query row inside the tile = TMEM lane
        const uint32_t s_tmem0 = tmem + C::kSCol + g * C::kSBufs * kKT + lane_base;   // + kKT per S buffer
        const uint32_t o_tmem = tmem + C::kOCol + g * D + lane_base;
        const uint32_t o_full = o_full0 + 8 * g;
        const bool q_loader = (wq == 0 && lane == 0);
        // the output rows start on 32-byte boundaries (the interface only promises 16)
        const bool o_sectors = ((reinterpret_cast<uintptr_t>(O) | (uintptr_t)(2 * o_row) | (uintptr_t)(2 * o_head) | (uintptr_t)(2 * o_tok)) & 31u) == 0;
        // density: [run][row] sums of this stream, in the shared memory the fourth key/value stage would take
        // (every thread only ever touches the entries of its own row; they were zeroed before the roles split)
        float* den_rows = reinterpret_cast<float*>(smem_raw + (kv_smem - raw) + C::kStages * C::kStageBytes) + g * kMaxDenRuns * kQRows;
        uint32_t q_armed = 0;     // query tiles requested so far
        uint32_t q_next_n = 0;    // first pair index not yet searched for a query tile

        // request the query tile of this stream's next unit not yet requested (first lane of the group only)
        if (kShort && q_loader) prefetch_tensormap(&q_map);
        auto load_next_q = [&]() {
            for (; q_next_n < my_pairs; ++q_next_n) {
                const int32_t pair = (int32_t)(blockIdx.x + q_next_n * gridDim.x);
                const Stream s = stream_of(pp, pair, g);
                if (!s.valid) continue;
                const int32_t row = s.item / heads, head = s.item - row * heads;
                const int32_t valid_rows = min(kQRows, T - s.qt * kQRows);
                const int qboxes = (valid_rows + kQBoxRows - 1) / kQBoxRows;
                const uint32_t half = q_split ? (q_armed & 1u) : 0u;
                const uint32_t bar = q_full0 + 16 * g + 8 * half;
                const uint32_t dst = q_smem + g * C::kQBytes + half * kQHalfSlot;
                mbar_expect_tx(bar, (uint32_t)qboxes * kQBoxRows * D * 2);
                int c[4] = {0, 0, 0, 0};
                c[qpos.y] = head;
                c[qpos.z] = row;
                for (int bx = 0; bx < qboxes; ++bx) {
                    c[qpos.x] = s.qt * kQRows + bx * kQBoxRows;
#pragma unroll
                    for (int h = 0; h < C::kHalves; ++h)
                        tma_load_4d(dst + h * C::kQHalfBytes + bx * kQBoxRows * 128, &q_map, bar, h * 64, c[1], c[2], c[3]);
                }
                ++q_armed;
                ++q_next_n;
                return;
            }
        };
        if (q_loader) {
            load_next_q();
            if (q_split) load_next_q();
        }

        uint32_t t = 0;   // flat tile counter of this stream
        uint32_t un = 0;  // units done by this stream
        bool ok = true;
        for (uint32_t n = 0; ok && n < my_pairs; ++n) {
            const int32_t pair = (int32_t)(blockIdx.x + n * gridDim.x);
            const Stream st = stream_of(pp, pair, g);
            if (!st.valid) continue;
            const int32_t valid_rows = min(kQRows, T - st.qt * kQRows);
            const bool warp_live = wq * 32 < valid_rows;
            float m_ref = 0.f, nb = 0.f, l = 0.f;
            float run_mass = 0.f;   // density: this row's un-normalised mass on the run the tiles are in
            int cur_run = -1;
            for (int j = 0; j < n_tiles; ++j, ++t) {
                int32_t t0, valid;
                tile_of(j, t0, valid);
                const int run = tile_run(valid);
                if (kDen && run != cur_run) {
                    // (the same for every thread: tiles and their runs are launch constants)
                    if (cur_run >= 0 && warp_live) den_rows[cur_run * kQRows + r] += run_mass;
                    run_mass = 0.f;
                    cur_run = run;
                }
                const uint32_t s_tmem = s_tmem0 + buf_of(t) * kKT;
                const uint32_t s_full = s_full0 + 16 * g + 8 * buf_of(t), p_full = p_full0 + 16 * g + 8 * buf_of(t);
                if (!__all_sync(0xffffffffu, mbar_wait(s_full, par_of(t), abort_flag))) {
                    report(status, kStatusSyncTimeout, abort_flag);
                    ok = false;
                    break;
                }
                tc_fence_after();
                // the last S of this unit has landed, so its query tile is no longer read
                if (j == n_tiles - 1 && q_loader) load_next_q();
                if (warp_live) {
                    uint32_t sr[kKT];
                    tmem_ld64(s_tmem, sr);
                    if (valid < kKT) {
                        // (a rider occupies the box behind the tile's own: its tokens stay, the gap before them goes)
                        // as a bit per column, so that each column costs one test of a constant bit
                        uint64_t keep = (1ull << valid) - 1ull;
                        if (kExt && ext.rider_valid > 0 && j == n_tiles - 1)
                            keep |= ((1ull << ext.rider_valid) - 1ull) << ((valid + 15) & ~15);
                        const uint32_t keep_lo = (uint32_t)keep, keep_hi = (uint32_t)(keep >> 32);
#pragma unroll
                        for (int i = 0; i < kKT; ++i)
                            if ((((i < 32 ? keep_lo : keep_hi) >> (i & 31)) & 1u) == 0u) sr[i] = 0xff800000u;  // -inf
                    }
                    // row maximum with four independent chains
                    auto row_max = [&]() -> float {
                        float mx[4];
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            mx[c] = max3(__uint_as_float(sr[c]), __uint_as_float(sr[4 + c]), __uint_as_float(sr[8 + c]));
#pragma unroll
                        for (int i = 12; i < kKT - 4; i += 8) {
#pragma unroll
                            for (int c = 0; c < 4; ++c)
                                mx[c] = max3(mx[c], __uint_as_float(sr[i + c]), __uint_as_float(sr[i + 4 + c]));
                        }
#pragma unroll
                        for (int c = 0; c < 4; ++c) mx[c] = fmaxf(mx[c], __uint_as_float(sr[kKT - 4 + c]));
                        return fmaxf(max3(mx[0], mx[1], mx[2]), mx[3]);
                    };
                    // rare: bring O and the row sum to a new reference (rows with `grow`).  The previous P V must
                    // be done.  One S buffer: it was issued before this tile's S, whose arrival covers every
                    // earlier product.  Two buffers: this S may have been issued first, so wait for the
                    // product's own completion (one arrival per P V; at most one phase can be ahead,
                    // because the next P V needs the P this tile has not written yet).
                    auto rescale = [&](const bool grow, const float mt) -> bool {
                        if (C::kSBufs == 2 && !__all_sync(0xffffffffu, mbar_wait(pv_done0 + 8 * g, (t - 1u) & 1u, abort_flag))) {
                            report(status, kStatusSyncTimeout, abort_flag);
                            return false;
                        }
                        if (C::kSBufs == 2) tc_fence_after();
                        float alpha = 1.f;
                        if (grow) {
                            alpha = fast_exp2((m_ref - mt) * scale_log2);
                            m_ref = mt;
                            nb = -mt * scale_log2;
                            l *= alpha;
                            if (kDen) {
                                run_mass *= alpha;
                                for (int rn = 0; rn < den.n_runs; ++rn) den_rows[rn * kQRows + r] *= alpha;
                            }
                        }
#pragma unroll 1
                        for (int cblk = 0; cblk < D / 8; ++cblk) {
                            uint32_t o[8];
                            tmem_ld8(o_tmem + cblk * 8, o);
#pragma unroll
                            for (int i = 0; i < 8; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                            tmem_st8(o_tmem + cblk * 8, o);
                        }
                        return true;
                    };
                    if (j == 0) {
                        const float mt = row_max();
                        m_ref = mt;
                        nb = -mt * scale_log2;
                    } else if (!kLazy) {
                        const float mt = row_max();
                        const bool grow = fmaf(mt, scale_log2, nb) > kRescaleLog2;
                        if (__any_sync(0xffffffffu, grow) && !rescale(grow, mt)) {
                            ok = false;
                            break;
                        }
                    }
                    // P over S: columns 0..31 receive the 64 probabilities as bf16 pairs, 16 tokens per store.
                    // A partly filled tile only exponentiates the 16-token groups the products will read (the
                    // P V is issued for as many 16-token steps): the columns behind them keep stale bits.
                    int groups = kKT / 16;
                    if (valid < kKT) groups = ((valid + 15) >> 4) + ((kExt && ext.rider_valid > 0 && j == n_tiles - 1) ? 1 : 0);
                    auto exp_tile = [&]() -> float {
                        float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
                        for (int grp = 0; grp < kKT / 16; ++grp) {
                            if (grp < groups) {   // (the same for the whole warp)
                                uint32_t pk[8];
#pragma unroll
                                for (int ii = 0; ii < 8; ++ii) {
                                    const int i = (grp & 1) * 8 + ii;   // pair index within its 32-token half, as before
                                    const int c = grp * 16 + 2 * ii;
                                    // every kPolyEvery-th pair takes its exponentials from a polynomial on the FMA pipe:
                                    // the special-function unit (16 results per clock per SM) is the narrowest resource
                                    float x0, x1, p0, p1;
                                    fma2(x0, x1, __uint_as_float(sr[c]), __uint_as_float(sr[c + 1]), scale_log2, scale_log2, nb, nb);
                                    if (kPolyEvery > 0 && (i % (kPolyEvery > 0 ? kPolyEvery : 1)) == 0) {
                                        exp2_poly2(p0, p1, x0, x1);
                                    } else {
                                        p0 = fast_exp2(x0);
                                        p1 = fast_exp2(x1);
                                    }
                                    add2(sum0, sum1, sum0, sum1, p0, p1);
                                    const __nv_bfloat162 h = __floats2bfloat162_rn(p0, p1);
                                    pk[ii] = *reinterpret_cast<const uint32_t*>(&h);
                                }
                                tmem_st8_nowait(s_tmem + grp * 8, pk);
                            }
                        }
                        return sum0 + sum1;
                    };
                    float tile_sum = exp_tile();
                    if (kLazy && j > 0) {
                        // No maximum was taken for this tile: its exponentials were formed against the row's reference
                        // as it stood (the maximum of the unit's first tile, or of the last tile that was redone).
                        // That is exact as long as nothing overflows.  A row whose tile sum is beyond the limit (or
                        // not a number) has outgrown its reference by more than 2^58; the warp then takes the tile's
                        // true maxima, rescales and forms the tile again before it announces P.  The polynomial
                        // saturates at 2^126, so it cannot hide such a row.
                        const bool over = !(tile_sum <= kLazySumLimit);
                        if (__any_sync(0xffffffffu, over)) {
                            tmem_wait_st();
                            const float mt = row_max();
                            const bool grow = over || fmaf(mt, scale_log2, nb) > kRescaleLog2;
                            if (!rescale(grow, mt)) {
                                ok = false;
                                break;
                            }
                            tile_sum = exp_tile();
                        }
                    }
                    l += tile_sum;
                    if (kDen) run_mass += tile_sum;
                    tmem_wait_st();
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full);
            }
            if (!ok) break;
            // epilogue: out = O / l once the last P V of the unit is done
            if (!__all_sync(0xffffffffu, mbar_wait(o_full, un & 1u, abort_flag))) {
                report(status, kStatusSyncTimeout, abort_flag);
                ok = false;
                break;
            }
            tc_fence_after();
            if (warp_live) {
                const float inv = 1.f / l;
                const int32_t row = st.item / heads, head = st.item - row * heads;
                __nv_bfloat16* dst = O + row * o_row + head * o_head + (int64_t)(st.qt * kQRows + r) * o_tok;
#pragma unroll
                for (int cblk = 0; cblk < D / 32; ++cblk) {
                    uint32_t o[32];
                    tmem_ld32(o_tmem + cblk * 32, o);
                    if (r < valid_rows) {
                        uint32_t w[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(o[2 * i]) * inv, __uint_as_float(o[2 * i + 1]) * inv);
                            w[i] = *reinterpret_cast<const uint32_t*>(&h);
                        }
                        if (o_sectors) {
                            // whole 32-byte sectors per thread: half the store instructions, no partly written sector
                            st_global_32B(dst + cblk * 32, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
                            st_global_32B(dst + cblk * 32 + 16, w[8], w[9], w[10], w[11], w[12], w[13], w[14], w[15]);
                        } else {
#pragma unroll
                            for (int c = 0; c < 4; ++c)
                                reinterpret_cast<uint4*>(dst + cblk * 32)[c] = make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
                        }
                    }
                }
            }
            if (kDen && warp_live) {
                // the row's share of every run, normalised by its row sum, added up over the warp's rows and
                // then, weighted by 1 / (rows * tokens of the run), into the head's entry of the result
                if (cur_run >= 0) den_rows[cur_run * kQRows + r] += run_mass;
                const float inv = (r < valid_rows) ? 1.f / l : 0.f;
                const int32_t head = st.item % heads;
                for (int rn = 0; rn < den.n_runs; ++rn) {
                    float v = den_rows[rn * kQRows + r] * inv;
                    den_rows[rn * kQRows + r] = 0.f;   // the next unit starts from zero
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
                    if (lane == 0) atomicAdd(den.out + (int64_t)head * den.n_runs + rn, (double)v * (double)den.weight[rn]);
                }
            }
            tc_fence_before();   // orders the reads of O before the arrival on p_full for the next unit's first tile
            ++un;
        }
        // wind down: query tiles requested but never consumed must land before the CTA exits
        if (q_loader) {
            for (uint32_t q = un; q < q_armed; ++q) {
                const uint32_t half = q_split ? (q & 1u) : 0u;
                const uint32_t parity = q_split ? ((q >> 1) & 1u) : (q & 1u);
                for (uint32_t i = 0; i < kSpinLimit; ++i)
                    if (mbar_try_wait(q_full0 + 16 * g + 8 * half, parity)) break;
            }
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
template <int D, bool kExt, bool kWide, bool kDen, bool kLazy, bool kShort>
cudaError_t launch(const CUtensorMap& qm, const CUtensorMap& km, const CUtensorMap& vm, const CUtensorMap& km64,
                   const CUtensorMap& vm64, const ExtArgs& ext, const Strided& O,
                   const RangeList& ranges, int32_t T, int32_t heads, const PairPlan& pp, int32_t n_tiles, int3 qpos,
                   float scale_log2, int* status, int sm_count, cudaStream_t stream, const DenArgs& den)
{
    using C = Cfg<D, kWide, kDen>;
    static SharedMemoryOptIn opt_in;
    const cudaError_t oe = opt_in.ensure(attend_pair_kernel<D, kExt, kWide, kDen, kLazy, kShort>, (int)C::kSmemBytes);
    if (oe != cudaSuccess) return oe;
    int64_t grid = (int64_t)sm_count * C::kCtasPerSm;
    if (grid > pp.n_pairs) grid = pp.n_pairs;
    attend_pair_kernel<D, kExt, kWide, kDen, kLazy, kShort><<<(unsigned)grid, C::kThreads, C::kSmemBytes, stream>>>(
        qm, km, vm, km64, vm64, ext, (__nv_bfloat16*)O.ptr, O.row, O.head, O.token, ranges, T, heads, pp, n_tiles, qpos,
        scale_log2, status, den);
    count_launch();
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_attend_pair(const Strided& Q, const Strided& O, const void* k_map, const void* v_map,
                               const void* k_map64, const void* v_map64, const RangeList& ranges, int32_t T, int32_t rows, int32_t heads, int32_t D,
                               float softmax_scale, int* status, int sm_count, cudaStream_t stream,
                               const CurrentScaleSource* cur, const PairDensity* density)
{
    if (ranges.n < 1 || ranges.total < 1 || T < 1) return cudaErrorInvalidValue;
    DenArgs den;
    memset(&den, 0, sizeof(den));
    if (density) {
        static_assert(kPairMaxDensityRuns == kMaxDenRuns, "interface and kernel disagree");
        if (cur || density->n_runs < 1 || density->n_runs > kMaxDenRuns || !density->out) return cudaErrorInvalidValue;
        den.out = density->out;
        den.n_runs = density->n_runs;
        for (int i = 0; i < density->n_runs; ++i) den.weight[i] = density->weight[i];
        for (int i = 0; i < ranges.n; ++i) {
            if (density->run_of_range[i] < 0 || density->run_of_range[i] >= density->n_runs) return cudaErrorInvalidValue;
            den.run_of_range[i] = density->run_of_range[i];
        }
    }
    ExtArgs ext;
    memset(&ext, 0, sizeof(ext));
    ext.range = -1;
    if (cur) {
        // the last range stands for the current scale, whose tokens come from the caller's tensors
        if (ranges.r[ranges.n - 1].start != 0 || ranges.r[ranges.n - 1].len != T) return cudaErrorInvalidValue;
        int kp[3], vp[3];
        if (!tc_encode_q_map(cur->K, T, rows, heads, D, kKT, &ext.k64, kp) ||
            !tc_encode_q_map(cur->V, T, rows, heads, D, kKT, &ext.v64, vp) ||
            !tc_encode_q_map(cur->K, T, rows, heads, D, kKVBoxRows, &ext.k16, kp) ||
            !tc_encode_q_map(cur->V, T, rows, heads, D, kKVBoxRows, &ext.v16, vp))
            return cudaErrorNotSupported;
        if (kp[0] != vp[0] || kp[1] != vp[1] || kp[2] != vp[2]) return cudaErrorNotSupported;
        ext.pos = make_int3(kp[0], kp[1], kp[2]);
        ext.range = ranges.n - 1;
        ext.store = cur->store ? 1 : 0;
        ext.dst = cur->dst;
        if (cur->rider_valid > 0) {
            const int32_t tail = T % kKT;
            if (cur->rider_valid > kKVBoxRows || tail < 1 || tail > kKT - kKVBoxRows) return cudaErrorInvalidValue;
            ext.rider_tok = cur->rider_tok;
            ext.rider_valid = cur->rider_valid;
        }
        if (cur->store &&
            !tc_encode_kv_store_maps(cur->region, (int64_t)rows * heads, D, kKT, cur->dst + T, &ext.k_store, &ext.v_store))
            return cudaErrorNotSupported;
    }
    CUtensorMap qm;
    int pos[3];
    if (!tc_encode_q_map(Q, T, rows, heads, D, kQBoxRows, &qm, pos)) return cudaErrorNotSupported;
    CUtensorMap km, vm, km64, vm64;
    memcpy(&km, k_map, sizeof(km));
    memcpy(&vm, v_map, sizeof(vm));
    memcpy(&km64, k_map64, sizeof(km64));
    memcpy(&vm64, v_map64, sizeof(vm64));
    PairPlan pp;
    pp.nqt = (T + kQRows - 1) / kQRows;
    pp.npi = pp.nqt / 2;
    if ((int64_t)rows * heads > 0x3fffffffll) return cudaErrorInvalidValue;
    pp.n_items = rows * heads;
    const int64_t n_shared = (int64_t)pp.n_items * pp.npi;
    const int64_t n_pairs = n_shared + ((pp.nqt & 1) ? ((int64_t)pp.n_items + 1) / 2 : 0);
    if (n_pairs > 0x7fffffffll) return cudaErrorInvalidValue;
    pp.n_shared = (int32_t)n_shared;
    pp.n_pairs = (int32_t)n_pairs;
    pp.kind = pp.npi == 0 ? 0 : ((pp.nqt & 1) ? 2 : 1);
    int32_t n_tiles = 0;
    for (int i = 0; i < ranges.n; ++i) n_tiles += (ranges.r[i].len + kKT - 1) / kKT;
    const int3 qpos = make_int3(pos[0], pos[1], pos[2]);
    const float scale_log2 = softmax_scale * 1.4426950408889634f;
    // 64 channels always take the two-CTA form: the wide form was measured on the tensor-bound launches of a
    // 2 240-token schedule (T = 576 and 1 024, 36 heads) and lost there too (26.3 vs 20.8 and 64.2 vs 53.9 ms):
    // two streams per SM do not keep the tensor pipe as busy as four, even with the chain broken.
#define AMSKV_PAIR_LAUNCH(DD, EXT, WIDE, DEN, LAZY, SHORT)                                                          \
    return launch<DD, EXT, WIDE, DEN, LAZY, SHORT>(qm, km, vm, km64, vm64, ext, O, ranges, T, heads, pp, n_tiles, qpos,  \
                                                   scale_log2, status, sm_count, stream, den)
    // Launches of three key tiles or more take the row maximum of a unit's first tile only (the kLazy form of the
    // softmax loop: 1.7 % of a 256x256-shaped pass, 6 % of a 1024x1024-shaped one); with fewer tiles there is next
    // to nothing to skip and the plain form is the faster code.  Launches of at most four key tiles (kShort, 64
    // channels) have a producer that issues a tile's bulk copies from several lanes at once and fetches a partly
    // filled tile of the caller's tensors as one box; the long launches keep the one-lane producer (its smaller code
    // measured 2 % faster there).
    constexpr int lazy_min = 3, lazy128_min = 3, short_max = 4;
    if (D == 128) {
        if (density) AMSKV_PAIR_LAUNCH(128, false, true, true, false, false);
        if (n_tiles >= lazy128_min) {
            if (cur) AMSKV_PAIR_LAUNCH(128, true, true, false, true, false);
            AMSKV_PAIR_LAUNCH(128, false, true, false, true, false);
        }
        if (cur) AMSKV_PAIR_LAUNCH(128, true, true, false, false, false);
        AMSKV_PAIR_LAUNCH(128, false, true, false, false, false);
    }
    if (density) AMSKV_PAIR_LAUNCH(64, false, false, true, false, false);
    if (n_tiles > short_max) {
        if (cur) AMSKV_PAIR_LAUNCH(64, true, false, false, true, false);
        AMSKV_PAIR_LAUNCH(64, false, false, false, true, false);
    }
    if (n_tiles >= lazy_min) {
        if (cur) AMSKV_PAIR_LAUNCH(64, true, false, false, true, true);
        AMSKV_PAIR_LAUNCH(64, false, false, false, true, true);
    }
    if (cur) AMSKV_PAIR_LAUNCH(64, true, false, false, false, true);
    AMSKV_PAIR_LAUNCH(64, false, false, false, false, true);
#undef AMSKV_PAIR_LAUNCH
}

}  // namespace amskv
