// C ABI of the AMS-KV library: argument checking, the segment table and kernel launches.
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <numeric>
#include <vector>

#include <nvtx3/nvToolsExt.h>   // header-only; ranges cost nothing measurable unless a profiler is attached

#include "../../include/amskv.h"
#include "kernels.cuh"

namespace amskv {

static std::atomic<int64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

constexpr size_t kAlign = 256;
constexpr size_t kStatusBytes = 256;

static size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct alignas(64) TensorMapBlob {
    unsigned char bytes[128];
};

}  // namespace amskv

using namespace amskv;

struct amskv_cache {
    int32_t layers = 0, heads = 0, head_dim = 0, rows = 0, n_scales = 0;
    uint32_t flags = 0;
    float softmax_scale = 0.f;
    int path = AMSKV_PATH_AUTO;
    int sm_count = 0;
    std::vector<int32_t> sides, tokens;
    std::vector<LayerLayout> layout;
    std::vector<LayerLayout> layout0;   // as created: amskv_cache_reset undoes promotions
    std::vector<uint8_t> promotable, promoted;
    std::vector<size_t> layer_offset;  // bytes from the arena start
    std::vector<int32_t> last_appended;
    std::vector<TensorMapBlob> k_maps, v_maps;      // 16-token boxes
    std::vector<TensorMapBlob> k_maps64, v_maps64;  // 64-token boxes (whole tiles)
    bool tc_ready = false;
    char* arena = nullptr;
    size_t arena_bytes = 0;
    bool owns_arena = false;
    size_t resident_now = 0, peak = 0;

    bool plan_only() const { return (flags & AMSKV_FLAG_PLAN_ONLY) != 0; }
    // the scale is the last one of a cache that never stores its last scale
    bool transient(int scale) const { return (flags & AMSKV_FLAG_TRANSIENT_LAST_SCALE) != 0 && scale == n_scales - 1; }
    int64_t items() const { return (int64_t)rows * heads; }
    size_t token_bytes() const { return (size_t)items() * head_dim * 2 /*bf16*/ * 2 /*K and V*/; }
    LayerRegion region(int layer) const
    {
        return LayerRegion{reinterpret_cast<__nv_bfloat16*>(arena + layer_offset[layer]), layout[layer].capacity};
    }
    int* status_word() const { return reinterpret_cast<int*>(arena); }
};

namespace {

// A named range around one call's enqueueing, for timeline tools (cache flag AMSKV_FLAG_NVTX).
struct CallRange {
    bool on;
    CallRange(const amskv_cache* c, const char* what, int layer, int scale) : on(c && (c->flags & AMSKV_FLAG_NVTX) != 0)
    {
        if (!on) return;
        char name[64];
        snprintf(name, sizeof(name), "%s L%d s%d", what, layer, scale);
        nvtxRangePushA(name);
    }
    ~CallRange()
    {
        if (on) nvtxRangePop();
    }
};

int check_desc(const amskv_desc* d)
{
    if (!d || !d->scale_sides || !d->policy) return AMSKV_ERR_INVALID;
    if (d->layers < 1 || d->heads < 1 || d->rows < 1) return AMSKV_ERR_INVALID;
    if (d->n_scales < 1 || d->n_scales > AMSKV_MAX_SCALES) return AMSKV_ERR_INVALID;
    if (d->head_dim != 64 && d->head_dim != 128) return AMSKV_ERR_UNSUPPORTED;
    for (int i = 0; i < d->n_scales; ++i)
        if (d->scale_sides[i] < 1 || d->scale_sides[i] > 4096) return AMSKV_ERR_INVALID;
    for (int l = 0; l < d->layers; ++l) {
        if (d->token_budget && d->token_budget[l].budget_tokens != 0) {
            const amskv_token_budget& b = d->token_budget[l];
            if (b.budget_tokens < 0 || b.condensed_tokens < 0) return AMSKV_ERR_INVALID;
            if (b.promoted_budget_tokens != 0 && b.promoted_budget_tokens < b.budget_tokens) return AMSKV_ERR_INVALID;
            continue;  // the layer's scale-granular fields are not used
        }
        if (d->policy[l].n_condensed < 0 || d->policy[l].n_local < 1) return AMSKV_ERR_INVALID;
        if (d->policy[l].cache_demanding < 0 || d->policy[l].cache_demanding > AMSKV_LAYER_PROMOTABLE) return AMSKV_ERR_INVALID;
    }
    if ((d->flags & ~(AMSKV_FLAG_PLAN_ONLY | AMSKV_FLAG_BULK_APPEND | AMSKV_FLAG_TRANSIENT_LAST_SCALE | AMSKV_FLAG_NVTX)) != 0)
        return AMSKV_ERR_INVALID;
    if (!(d->softmax_scale == d->softmax_scale)) return AMSKV_ERR_INVALID;  // NaN
    return AMSKV_OK;
}

// Fills everything that depends only on the descriptor.
int plan(const amskv_desc* d, amskv_cache* c)
{
    c->layers = d->layers;
    c->heads = d->heads;
    c->head_dim = d->head_dim;
    c->rows = d->rows;
    c->n_scales = d->n_scales;
    c->flags = d->flags;
    c->softmax_scale = d->softmax_scale > 0.f ? d->softmax_scale : 1.0f / std::sqrt((float)d->head_dim);
    c->sides.assign(d->scale_sides, d->scale_sides + d->n_scales);
    c->tokens.resize(d->n_scales);
    for (int i = 0; i < d->n_scales; ++i) {
        const int64_t t = (int64_t)c->sides[i] * c->sides[i];
        if (t > (1 << 24)) return AMSKV_ERR_INVALID;
        c->tokens[i] = (int32_t)t;
    }
    c->layout.resize(d->layers);
    c->promotable.assign(d->layers, 0);
    c->promoted.assign(d->layers, 0);
    c->layer_offset.resize(d->layers);
    size_t at = kStatusBytes;
    for (int l = 0; l < d->layers; ++l) {
        const bool transient_last = (d->flags & AMSKV_FLAG_TRANSIENT_LAST_SCALE) != 0;
        if (d->token_budget && d->token_budget[l].budget_tokens > 0) {
            c->layout[l].build_tokens(c->tokens, d->token_budget[l].budget_tokens, d->token_budget[l].condensed_tokens,
                                      transient_last, d->token_budget[l].promoted_budget_tokens);
            c->promotable[l] = c->layout[l].c_promoted > 0;
        } else {
            const bool may_promote = d->policy[l].cache_demanding == AMSKV_LAYER_PROMOTABLE;
            c->layout[l].build(c->tokens, d->policy[l].n_condensed, d->policy[l].n_local,
                               d->policy[l].cache_demanding == AMSKV_LAYER_DEMANDING, transient_last, may_promote);
            c->promotable[l] = may_promote && !c->layout[l].full;
        }
        if ((int64_t)c->layout[l].capacity > (1ll << 30)) return AMSKV_ERR_INVALID;
        c->layer_offset[l] = at;
        at += align_up((size_t)c->layout[l].capacity * c->token_bytes());
    }
    c->arena_bytes = at;
    c->layout0 = c->layout;
    c->last_appended.assign(d->layers, -1);
    return AMSKV_OK;
}

bool bad_layer_scale(const amskv_cache* c, int layer, int scale)
{
    return !c || layer < 0 || layer >= c->layers || scale < 0 || scale >= c->n_scales;
}

bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

// `is_output`: the tensor is written.  A zero row or head stride repeats one slice along that dimension
// (a broadcast view); the TMA paths cannot express that, and a written tensor must not alias itself, so
// it is refused wherever the dimension has more than one entry, and for outputs always.
int make_strided(const void* ptr, const int64_t* strides, int32_t rows, int32_t heads, int32_t T, int32_t D, Strided* out,
                 bool is_output = false)
{
    if (!ptr || misaligned(ptr)) return AMSKV_ERR_INVALID;
    out->ptr = ptr;
    if (strides) {
        out->row = strides[0];
        out->head = strides[1];
        out->token = strides[2];
        if (out->row < 0 || out->head < 0 || out->token < D) return AMSKV_ERR_INVALID;
        if ((out->row % 8) || (out->head % 8) || (out->token % 8)) return AMSKV_ERR_INVALID;
        if ((out->row == 0 && (rows > 1 || is_output)) || (out->head == 0 && (heads > 1 || is_output)))
            return AMSKV_ERR_INVALID;
    } else {
        out->token = D;
        out->head = (int64_t)T * D;
        out->row = (int64_t)heads * T * D;
    }
    return AMSKV_OK;
}

// host-side state after scale `scale` of `layer` was stored
void note_appended(amskv_cache* cache, int layer, int scale)
{
    const LayerLayout& lay = cache->layout[layer];
    const int64_t before = scale > 0 ? lay.resident_tokens(cache->tokens, scale - 1) : 0;
    const int64_t after = lay.resident_tokens(cache->tokens, scale);
    cache->resident_now = (size_t)((int64_t)cache->resident_now + (after - before) * (int64_t)cache->token_bytes());
    cache->peak = std::max(cache->peak, cache->resident_now);
    cache->last_appended[layer] = scale;
}

// which kernel amskv_attend uses for T query tokens over `total` keys
enum class AttendKernel { Small, Simt, Pair, Tensor };
AttendKernel choose_kernel(const amskv_cache* cache, int32_t T, int32_t total)
{
    // AUTO: the warp-per-item kernel wherever a scale's retained keys fit its register tile, the paired
    // tcgen05 kernel elsewhere (the CUDA-core kernel only where tensor maps are unavailable)
    // (a single query token per item is fastest on the CUDA-core kernel: measured)
    if ((cache->path == AMSKV_PATH_SMALL || (cache->path == AMSKV_PATH_AUTO && T > 1)) && small_supported(T, total))
        return AttendKernel::Small;
    if (cache->path == AMSKV_PATH_SIMT || (cache->path == AMSKV_PATH_AUTO && T == 1) || !cache->tc_ready)
        return AttendKernel::Simt;
    return cache->path == AMSKV_PATH_TENSOR ? AttendKernel::Tensor : AttendKernel::Pair;
}

}  // namespace

extern "C" {

int amskv_cache_required_bytes(const amskv_desc* desc, size_t* bytes)
{
    if (!bytes) return AMSKV_ERR_INVALID;
    int rc = check_desc(desc);
    if (rc != AMSKV_OK) return rc;
    amskv_cache tmp;
    rc = plan(desc, &tmp);
    if (rc != AMSKV_OK) return rc;
    *bytes = tmp.arena_bytes;
    return AMSKV_OK;
}

int amskv_cache_create(const amskv_desc* desc, void* dev_mem, size_t dev_bytes, amskv_cache** out)
{
    if (!out) return AMSKV_ERR_INVALID;
    *out = nullptr;
    int rc = check_desc(desc);
    if (rc != AMSKV_OK) return rc;
    amskv_cache* c = new (std::nothrow) amskv_cache();
    if (!c) return AMSKV_ERR_NOMEM;
    rc = plan(desc, c);
    if (rc != AMSKV_OK) { delete c; return rc; }
    if (c->plan_only()) { *out = c; return AMSKV_OK; }

    int dev = 0;
    cudaDeviceProp prop;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) {
        (void)cudaGetLastError();
        delete c;
        return AMSKV_ERR_CUDA;
    }
    c->sm_count = prop.multiProcessorCount;
    if (dev_mem) {
        if ((reinterpret_cast<uintptr_t>(dev_mem) % kAlign) != 0) { delete c; return AMSKV_ERR_INVALID; }
        if (dev_bytes < c->arena_bytes) { delete c; return AMSKV_ERR_NOMEM; }
        c->arena = static_cast<char*>(dev_mem);
    } else {
        size_t free_b = 0, total_b = 0;
        if (cudaMemGetInfo(&free_b, &total_b) != cudaSuccess) { (void)cudaGetLastError(); delete c; return AMSKV_ERR_CUDA; }
        if (free_b < c->arena_bytes) { delete c; return AMSKV_ERR_NOMEM; }
        void* p = nullptr;
        if (cudaMalloc(&p, c->arena_bytes) != cudaSuccess) { (void)cudaGetLastError(); delete c; return AMSKV_ERR_NOMEM; }
        c->arena = static_cast<char*>(p);
        c->owns_arena = true;
    }
    // Tiles may extend past a range's end into tokens nobody attends; zero-filling once keeps
    // those bytes finite so that a zero probability times such a value is zero.
    cudaError_t e = cudaMemsetAsync(c->arena, 0, c->arena_bytes, 0);
    if (e == cudaSuccess) e = cudaStreamSynchronize(0);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        if (c->owns_arena) cudaFree(c->arena);
        delete c;
        return AMSKV_ERR_CUDA;
    }
    c->tc_ready = false;
    if (tc_supported(c->head_dim) && prop.major == 10) {
        c->k_maps.resize(c->layers);
        c->v_maps.resize(c->layers);
        c->k_maps64.resize(c->layers);
        c->v_maps64.resize(c->layers);
        bool ok = true;
        for (int l = 0; l < c->layers && ok; ++l)
            ok = tc_encode_kv_maps(c->region(l), c->items(), c->head_dim, 16, c->k_maps[l].bytes, c->v_maps[l].bytes) &&
                 tc_encode_kv_maps(c->region(l), c->items(), c->head_dim, 64, c->k_maps64[l].bytes, c->v_maps64[l].bytes);
        c->tc_ready = ok;
    }
    *out = c;
    return AMSKV_OK;
}

int amskv_cache_destroy(amskv_cache* cache)
{
    if (!cache) return AMSKV_ERR_INVALID;
    int rc = AMSKV_OK;
    if (cache->owns_arena && cache->arena) {
        if (cudaFree(cache->arena) != cudaSuccess) { (void)cudaGetLastError(); rc = AMSKV_ERR_CUDA; }
    }
    delete cache;
    return rc;
}

int amskv_cache_reset(amskv_cache* cache)
{
    if (!cache) return AMSKV_ERR_INVALID;
    std::fill(cache->last_appended.begin(), cache->last_appended.end(), -1);
    // every layer starts a new batch in the class it was created with (Algorithm 1 starts at C_min)
    for (int l = 0; l < cache->layers; ++l)
        if (cache->promoted[l]) { cache->layout[l] = cache->layout0[l]; cache->promoted[l] = 0; }
    cache->resident_now = 0;
    cache->peak = 0;
    return AMSKV_OK;
}

int amskv_append(amskv_cache* cache, int layer, int scale, const void* K, const void* V, const int64_t strides[3],
                 void* stream)
{
    if (bad_layer_scale(cache, layer, scale)) return AMSKV_ERR_INVALID;
    const CallRange range(cache, "amskv_append", layer, scale);
    if (scale != cache->last_appended[layer] + 1) return AMSKV_ERR_ORDER;
    if (cache->transient(scale)) return AMSKV_ERR_UNSUPPORTED;   // it has no place in the arena: amskv_append_attend
    const int32_t T = cache->tokens[scale];
    const LayerLayout& lay = cache->layout[layer];
    if (!cache->plan_only()) {
        Strided ks, vs;
        int rc = make_strided(K, strides, cache->rows, cache->heads, T, cache->head_dim, &ks);
        if (rc != AMSKV_OK) return rc;
        rc = make_strided(V, strides, cache->rows, cache->heads, T, cache->head_dim, &vs);
        if (rc != AMSKV_OK) return rc;
        Piece piece[LayerLayout::kMaxPieces];
        const int32_t n_pieces = lay.pieces(cache->tokens, scale, piece);
        for (int32_t i = 0; i < n_pieces; ++i) {
            Strided kp = ks, vp = vs;
            kp.ptr = static_cast<const __nv_bfloat16*>(ks.ptr) + (int64_t)piece[i].src * ks.token;
            vp.ptr = static_cast<const __nv_bfloat16*>(vs.ptr) + (int64_t)piece[i].src * vs.token;
            cudaError_t e = launch_append(kp, vp, cache->region(layer), piece[i].dst, piece[i].len, cache->rows,
                                          cache->heads, cache->head_dim, (cache->flags & AMSKV_FLAG_BULK_APPEND) != 0,
                                          cache->status_word(), cache->sm_count, static_cast<cudaStream_t>(stream));
            if (e != cudaSuccess) { (void)cudaGetLastError(); return AMSKV_ERR_CUDA; }
        }
    }
    note_appended(cache, layer, scale);
    return AMSKV_OK;
}

int amskv_first_overflow_scale(const amskv_cache* cache, int layer, int* scale)
{
    if (!cache || layer < 0 || layer >= cache->layers || !scale) return AMSKV_ERR_INVALID;
    *scale = cache->layout[layer].first_overflow(cache->tokens);
    return AMSKV_OK;
}

int amskv_promote_layer(amskv_cache* cache, int layer)
{
    if (!cache || layer < 0 || layer >= cache->layers) return AMSKV_ERR_INVALID;
    if (!cache->promotable[layer]) return AMSKV_ERR_UNSUPPORTED;
    if (cache->promoted[layer]) return AMSKV_OK;
    // legal until the append that overflows the budget: nothing has been evicted, and every cached token sits
    // where the larger layout expects it
    if (cache->last_appended[layer] >= cache->layout[layer].first_overflow(cache->tokens)) return AMSKV_ERR_ORDER;
    cache->layout[layer].promote(cache->tokens);
    cache->promoted[layer] = 1;
    return AMSKV_OK;
}

int amskv_set_attend_path(amskv_cache* cache, int path)
{
    if (!cache || path < AMSKV_PATH_AUTO || path > AMSKV_PATH_SMALL) return AMSKV_ERR_INVALID;
    if ((path == AMSKV_PATH_TENSOR || path == AMSKV_PATH_TENSOR_PAIR) && !cache->tc_ready) return AMSKV_ERR_UNSUPPORTED;
    cache->path = path;
    return AMSKV_OK;
}

int amskv_attend(amskv_cache* cache, int layer, int scale, const void* Q, void* out, const int64_t q_strides[3],
                 const int64_t o_strides[3], void* stream)
{
    if (bad_layer_scale(cache, layer, scale)) return AMSKV_ERR_INVALID;
    const CallRange range(cache, "amskv_attend", layer, scale);
    if (cache->plan_only()) return AMSKV_ERR_UNSUPPORTED;
    if (scale != cache->last_appended[layer]) return AMSKV_ERR_ORDER;
    const int32_t T = cache->tokens[scale];
    Strided q, o;
    int rc = make_strided(Q, q_strides, cache->rows, cache->heads, T, cache->head_dim, &q);
    if (rc != AMSKV_OK) return rc;
    rc = make_strided(out, o_strides, cache->rows, cache->heads, T, cache->head_dim, &o, true);
    if (rc != AMSKV_OK) return rc;
    RangeList ranges;
    ranges.n = cache->layout[layer].ranges(cache->tokens, scale, ranges.r);
    ranges.total = 0;
    for (int i = 0; i < ranges.n; ++i) ranges.total += ranges.r[i].len;
    const AttendKernel kernel = choose_kernel(cache, T, ranges.total);
    cudaError_t e;
    if (kernel == AttendKernel::Small) {
        e = launch_attend_small(q, o, cache->region(layer), ranges, T, cache->rows, cache->heads, cache->head_dim,
                                cache->softmax_scale, static_cast<cudaStream_t>(stream));
    } else if (kernel == AttendKernel::Pair) {
        e = launch_attend_pair(q, o, cache->k_maps[layer].bytes, cache->v_maps[layer].bytes,
                               cache->k_maps64[layer].bytes, cache->v_maps64[layer].bytes, ranges, T, cache->rows,
                               cache->heads, cache->head_dim, cache->softmax_scale, cache->status_word(),
                               cache->sm_count, static_cast<cudaStream_t>(stream));
    } else if (kernel == AttendKernel::Tensor) {
        e = launch_attend_tc(q, o, cache->region(layer), cache->k_maps[layer].bytes, cache->v_maps[layer].bytes, ranges,
                             T, cache->rows, cache->heads, cache->head_dim, cache->softmax_scale, cache->status_word(),
                             cache->sm_count, static_cast<cudaStream_t>(stream));
    } else {
        e = launch_attend_simt(q, o, cache->region(layer), ranges, T, cache->rows, cache->heads, cache->head_dim,
                               cache->softmax_scale, static_cast<cudaStream_t>(stream));
    }
    if (e != cudaSuccess) { (void)cudaGetLastError(); return AMSKV_ERR_CUDA; }
    return AMSKV_OK;
}

int amskv_append_attend(amskv_cache* cache, int layer, int scale, const void* K, const void* V,
                        const int64_t kv_strides[3], const void* Q, void* out, const int64_t q_strides[3],
                        const int64_t o_strides[3], void* stream)
{
    if (bad_layer_scale(cache, layer, scale)) return AMSKV_ERR_INVALID;
    const CallRange range(cache, "amskv_append_attend", layer, scale);
    if (scale != cache->last_appended[layer] + 1) return AMSKV_ERR_ORDER;
    if (cache->plan_only()) {   // bookkeeping only
        note_appended(cache, layer, scale);
        return AMSKV_OK;
    }
    const int32_t T = cache->tokens[scale];
    const LayerLayout& lay = cache->layout[layer];
    Strided ks, vs, q, o;
    int rc = make_strided(K, kv_strides, cache->rows, cache->heads, T, cache->head_dim, &ks);
    if (rc == AMSKV_OK) rc = make_strided(V, kv_strides, cache->rows, cache->heads, T, cache->head_dim, &vs);
    if (rc == AMSKV_OK) rc = make_strided(Q, q_strides, cache->rows, cache->heads, T, cache->head_dim, &q);
    if (rc == AMSKV_OK) rc = make_strided(out, o_strides, cache->rows, cache->heads, T, cache->head_dim, &o, true);
    if (rc != AMSKV_OK) return rc;
    if (cache->transient(scale)) {
        // Never stored: the queries attend to the older retained tokens in the cache and to the scale's own
        // K and V straight from the caller's tensors (paired kernel, else the CUDA-core kernel).
        RangeList rl;
        rl.n = lay.ranges_before(cache->tokens, scale, rl.r);
        if (rl.n >= kMaxRanges) return AMSKV_ERR_UNSUPPORTED;
        rl.r[rl.n++] = Range{0, T};
        rl.total = 0;
        for (int i = 0; i < rl.n; ++i) rl.total += rl.r[i].len;
        CurrentScaleSource src{ks, vs, false, 0, cache->region(layer)};
        cudaError_t e;
        if (cache->tc_ready && cache->path != AMSKV_PATH_SIMT && !(cache->path == AMSKV_PATH_AUTO && T == 1))
            e = launch_attend_pair(q, o, cache->k_maps[layer].bytes, cache->v_maps[layer].bytes, cache->k_maps64[layer].bytes,
                                   cache->v_maps64[layer].bytes, rl, T, cache->rows, cache->heads, cache->head_dim,
                                   cache->softmax_scale, cache->status_word(), cache->sm_count,
                                   static_cast<cudaStream_t>(stream), &src);
        else
            e = launch_attend_simt(q, o, cache->region(layer), rl, T, cache->rows, cache->heads, cache->head_dim,
                                   cache->softmax_scale, static_cast<cudaStream_t>(stream), &src);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return AMSKV_ERR_CUDA; }
        note_appended(cache, layer, scale);
        return AMSKV_OK;
    }
    // One launch where the paired kernel serves this scale and the append is a single copy: the kernel
    // reads the scale from K and V, attends to it together with the older retained tokens, and writes
    // it to its place in the cache on the way.  Elsewhere: the two calls, one after the other.
    RangeList after;
    after.n = lay.ranges(cache->tokens, scale, after.r);
    after.total = 0;
    for (int i = 0; i < after.n; ++i) after.total += after.r[i].len;
    Piece piece[LayerLayout::kMaxPieces];
    const int32_t n_pieces = lay.pieces(cache->tokens, scale, piece);
    const bool one_copy = n_pieces == 1 && piece[0].src == 0 && piece[0].len == T;
    AttendKernel kernel = choose_kernel(cache, T, after.total);
    // a single-token scale that is its own only key (the first scale): out = V, one copy kernel does both calls
    if (cache->path == AMSKV_PATH_AUTO && T == 1 && after.total == 1) kernel = AttendKernel::Small;
    if (kernel == AttendKernel::Small && one_copy) {
        // the warp-per-item kernel reads the scale from K and V and stores it on the way
        RangeList before;
        before.n = lay.ranges_before(cache->tokens, scale, before.r);
        before.total = 0;
        for (int i = 0; i < before.n; ++i) before.total += before.r[i].len;
        if (before.total + T == after.total) {
            CurrentScaleSource cur{ks, vs, true, piece[0].dst, cache->region(layer)};
            cudaError_t e = launch_attend_small(q, o, cache->region(layer), before, T, cache->rows, cache->heads, cache->head_dim,
                                                cache->softmax_scale, static_cast<cudaStream_t>(stream), &cur);
            if (e != cudaSuccess) { (void)cudaGetLastError(); return AMSKV_ERR_CUDA; }
            note_appended(cache, layer, scale);
            return AMSKV_OK;
        }
    }
    bool fused = cache->tc_ready && kernel == AttendKernel::Pair && one_copy;
    RangeList ranges;
    if (fused) {
        ranges.n = lay.ranges_before(cache->tokens, scale, ranges.r);
        if (ranges.n >= kMaxRanges) fused = false;
    }
    int32_t rider_tok = 0, rider_valid = 0;
    if (fused) {
        // The kernel works in 64-token key tiles per range.  Up to 16 tokens left over at the end of a cache
        // range (the condensed scales behind a 64-token scale, say) would cost a tile of their own; when the
        // current scale's last tile has a 16-token box to spare they ride there instead.
        const int32_t tail = T % 64;
        if (tail >= 1 && tail <= 48) {
            for (int i = ranges.n - 1; i >= 0 && rider_valid == 0; --i) {
                const int32_t left = ranges.r[i].len % 64;
                if (left >= 1 && left <= 16) {
                    rider_valid = left;
                    rider_tok = ranges.r[i].start + ranges.r[i].len - left;
                    ranges.r[i].len -= left;
                    if (ranges.r[i].len == 0) {
                        for (int m = i; m + 1 < ranges.n; ++m) ranges.r[m] = ranges.r[m + 1];
                        --ranges.n;
                    }
                }
            }
        }
    }
    if (fused && cache->path == AMSKV_PATH_AUTO) {
        // Taking the scale from the caller's tensors splits it off the range it would be part of in the
        // cache; where that adds a tile, attention loses more than the saved copy is worth (measured), so
        // such scales run as the two calls (AMSKV_PATH_TENSOR_PAIR fuses wherever it can).
        auto tiles = [](const RangeList& rl) {
            int32_t n = 0;
            for (int i = 0; i < rl.n; ++i) n += (rl.r[i].len + 63) / 64;
            return n;
        };
        if (tiles(ranges) + (T + 63) / 64 > tiles(after)) fused = false;
        // Well below a full key tile per scale the units are so short that the kernel is bound by the latency of
        // its loads; holding a stage until it has been written out costs as much there as the copy (measured:
        // equal at T = 36, where fusing at least saves the launch and the second read; a loss at T = 25).
        if (T < 32) fused = false;
    }
    if (!fused) {
        rc = amskv_append(cache, layer, scale, K, V, kv_strides, stream);
        if (rc != AMSKV_OK) return rc;
        return amskv_attend(cache, layer, scale, Q, out, q_strides, o_strides, stream);
    }
    ranges.r[ranges.n++] = Range{0, T};   // the current scale, in the caller's tensors
    ranges.total = 0;
    for (int i = 0; i < ranges.n; ++i) ranges.total += ranges.r[i].len;
    CurrentScaleSource cur{ks, vs, true, piece[0].dst, cache->region(layer)};
    cur.rider_tok = rider_tok;
    cur.rider_valid = rider_valid;
    cudaError_t e = launch_attend_pair(q, o, cache->k_maps[layer].bytes, cache->v_maps[layer].bytes,
                                       cache->k_maps64[layer].bytes, cache->v_maps64[layer].bytes, ranges, T, cache->rows,
                                       cache->heads, cache->head_dim, cache->softmax_scale, cache->status_word(),
                                       cache->sm_count, static_cast<cudaStream_t>(stream), &cur);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return AMSKV_ERR_CUDA; }
    note_appended(cache, layer, scale);
    return AMSKV_OK;
}

int amskv_attention_density(amskv_cache* cache, int layer, int scale, const void* Q, const int64_t q_strides[3],
                            double* out, size_t out_entries, void* stream)
{
    if (bad_layer_scale(cache, layer, scale) || !out || (reinterpret_cast<uintptr_t>(out) & 7u)) return AMSKV_ERR_INVALID;
    if (cache->plan_only()) return AMSKV_ERR_UNSUPPORTED;
    if (scale != cache->last_appended[layer]) return AMSKV_ERR_ORDER;
    const int32_t T = cache->tokens[scale];
    Strided q;
    int rc = make_strided(Q, q_strides, cache->rows, cache->heads, T, cache->head_dim, &q);
    if (rc != AMSKV_OK) return rc;
    const LayerLayout& lay = cache->layout[layer];
    TokenRun runs[2 * AMSKV_MAX_SCALES];
    const int32_t n_runs = lay.attended(cache->tokens, scale, runs);
    if (out_entries < (size_t)cache->heads * (size_t)n_runs) return AMSKV_ERR_NOMEM;
    LayerLayout::RunPiece rp[kMaxDensityPieces];
    const int32_t n = lay.attended_pieces(cache->tokens, scale, rp, kMaxDensityPieces);
    if (n < 0) return AMSKV_ERR_UNSUPPORTED;   // the scale's own keys are not in the cache (never-stored last scale)
    DensityPieces pieces;
    pieces.n = n;
    pieces.n_runs = n_runs;
    for (int32_t i = 0; i < n; ++i) {
        pieces.start[i] = rp[i].start;
        pieces.len[i] = rp[i].len;
        pieces.run[i] = rp[i].run;
        pieces.weight[i] = 1.0 / (double)runs[rp[i].run].count;
    }
    cudaError_t e = launch_density(q, cache->region(layer), pieces, T, cache->rows, cache->heads, cache->head_dim,
                                   cache->softmax_scale, out, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { (void)cudaGetLastError(); return AMSKV_ERR_CUDA; }
    return AMSKV_OK;
}

int amskv_attend_density(amskv_cache* cache, int layer, int scale, const void* Q, void* out, const int64_t q_strides[3],
                         const int64_t o_strides[3], double* density, size_t density_entries, void* stream)
{
    if (bad_layer_scale(cache, layer, scale) || !density || (reinterpret_cast<uintptr_t>(density) & 7u)) return AMSKV_ERR_INVALID;
    if (cache->plan_only()) return AMSKV_ERR_UNSUPPORTED;
    if (scale != cache->last_appended[layer]) return AMSKV_ERR_ORDER;
    const int32_t T = cache->tokens[scale];
    Strided q, o;
    int rc = make_strided(Q, q_strides, cache->rows, cache->heads, T, cache->head_dim, &q);
    if (rc == AMSKV_OK) rc = make_strided(out, o_strides, cache->rows, cache->heads, T, cache->head_dim, &o, true);
    if (rc != AMSKV_OK) return rc;
    const LayerLayout& lay = cache->layout[layer];
    TokenRun runs[2 * AMSKV_MAX_SCALES];
    const int32_t n_runs = lay.attended(cache->tokens, scale, runs);
    if (density_entries < (size_t)cache->heads * (size_t)n_runs) return AMSKV_ERR_NOMEM;
    LayerLayout::RunPiece rp[kMaxDensityPieces];
    const int32_t n = lay.attended_pieces(cache->tokens, scale, rp, kMaxDensityPieces);
    if (n < 0) return AMSKV_ERR_UNSUPPORTED;   // the scale's own keys are not in the cache (never-stored last scale)
    int32_t total = 0;
    for (int32_t i = 0; i < n; ++i) total += rp[i].len;
    // One launch where the paired kernel serves the scale: its key tiles are cut at the boundaries of the runs
    // (one range per piece of a run), and each row's mass per run falls out of the softmax loop.
    if (cache->tc_ready && choose_kernel(cache, T, total) == AttendKernel::Pair && n_runs <= kPairMaxDensityRuns && n <= kMaxRanges) {
        RangeList ranges;
        PairDensity den;
        den.out = density;
        den.n_runs = n_runs;
        for (int32_t r = 0; r < n_runs; ++r) den.weight[r] = (float)(1.0 / ((double)cache->rows * (double)runs[r].count));
        ranges.n = n;
        ranges.total = total;
        for (int32_t i = 0; i < n; ++i) {
            ranges.r[i] = Range{rp[i].start, rp[i].len};
            den.run_of_range[i] = (int8_t)rp[i].run;
        }
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        cudaError_t e = cudaMemsetAsync(density, 0, sizeof(double) * (size_t)cache->heads * n_runs, st);
        if (e == cudaSuccess)
            e = launch_attend_pair(q, o, cache->k_maps[layer].bytes, cache->v_maps[layer].bytes, cache->k_maps64[layer].bytes,
                                   cache->v_maps64[layer].bytes, ranges, T, cache->rows, cache->heads, cache->head_dim,
                                   cache->softmax_scale, cache->status_word(), cache->sm_count, st, nullptr, &den);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return AMSKV_ERR_CUDA; }
        return AMSKV_OK;
    }
    // elsewhere (the coarse scales, more runs than the kernel tells apart): the two calls
    rc = amskv_attend(cache, layer, scale, Q, out, q_strides, o_strides, stream);
    if (rc != AMSKV_OK) return rc;
    return amskv_attention_density(cache, layer, scale, Q, q_strides, density, density_entries, stream);
}

int amskv_step_staging_bytes(const amskv_cache* cache, size_t* bytes)
{
    if (!cache || !bytes) return AMSKV_ERR_INVALID;
    const int32_t tmax = *std::max_element(cache->tokens.begin(), cache->tokens.end());
    const size_t one = align_up((size_t)cache->items() * tmax * cache->head_dim * 2);
    *bytes = 4 * one;  // K, V, Q, out
    return AMSKV_OK;
}

int amskv_step_host(amskv_cache* cache, int layer, int scale, const void* K_host, const void* V_host,
                    const void* Q_host, void* out_host, void* staging, size_t staging_bytes, void* stream)
{
    if (bad_layer_scale(cache, layer, scale)) return AMSKV_ERR_INVALID;
    if (cache->plan_only()) return AMSKV_ERR_UNSUPPORTED;
    if (!K_host || !V_host || !Q_host || !out_host || !staging) return AMSKV_ERR_INVALID;
    if ((reinterpret_cast<uintptr_t>(staging) % kAlign) != 0) return AMSKV_ERR_INVALID;
    size_t need = 0;
    amskv_step_staging_bytes(cache, &need);
    if (staging_bytes < need) return AMSKV_ERR_NOMEM;
    if (scale != cache->last_appended[layer] + 1) return AMSKV_ERR_ORDER;
    const size_t one = need / 4;
    const size_t bytes = (size_t)cache->items() * cache->tokens[scale] * cache->head_dim * 2;
    char* s = static_cast<char*>(staging);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(s, K_host, bytes, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(s + one, V_host, bytes, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(s + 2 * one, Q_host, bytes, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return AMSKV_ERR_CUDA; }
    int rc = amskv_append_attend(cache, layer, scale, s, s + one, nullptr, s + 2 * one, s + 3 * one, nullptr, nullptr, stream);
    if (rc != AMSKV_OK) return rc;
    e = cudaMemcpyAsync(out_host, s + 3 * one, bytes, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return AMSKV_ERR_CUDA; }
    return AMSKV_OK;
}

size_t amskv_similarity_workspace_bytes(void) { return align_up(sizeof(double) * kSimilarityMaxBlocks); }

int amskv_layer_similarity(const void* K_prev, int side_prev, const void* K_cur, int side_cur, int rows, int heads,
                           int head_dim, double* out_ss, void* workspace, size_t workspace_bytes, void* stream)
{
    if (!K_prev || !K_cur || !out_ss || !workspace) return AMSKV_ERR_INVALID;
    if (misaligned(K_prev) || misaligned(K_cur) || (reinterpret_cast<uintptr_t>(out_ss) & 7u)) return AMSKV_ERR_INVALID;
    if ((reinterpret_cast<uintptr_t>(workspace) % kAlign) != 0) return AMSKV_ERR_INVALID;
    if (side_prev < 1 || side_cur < 1 || side_prev > 4096 || side_cur > 4096 || rows < 1 || heads < 1)
        return AMSKV_ERR_INVALID;
    if (head_dim != 64 && head_dim != 128) return AMSKV_ERR_UNSUPPORTED;
    if (workspace_bytes < amskv_similarity_workspace_bytes()) return AMSKV_ERR_NOMEM;
    cudaError_t e = launch_similarity((const __nv_bfloat16*)K_prev, side_prev, (const __nv_bfloat16*)K_cur, side_cur,
                                      (int64_t)rows * heads, head_dim, out_ss, static_cast<double*>(workspace),
                                      static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { (void)cudaGetLastError(); return AMSKV_ERR_CUDA; }
    return AMSKV_OK;
}

int amskv_classify_by_threshold(const double* scores, int layers, double theta, int32_t* demanding)
{
    if (!scores || !demanding || layers < 1) return AMSKV_ERR_INVALID;
    for (int l = 0; l < layers; ++l) demanding[l] = scores[l] < theta ? 1 : 0;
    return AMSKV_OK;
}

int amskv_classify_lowest(const double* scores, int layers, int n_demanding, int32_t* demanding)
{
    if (!scores || !demanding || layers < 1 || n_demanding < 0 || n_demanding > layers) return AMSKV_ERR_INVALID;
    std::vector<int> order(layers);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return scores[a] < scores[b]; });
    for (int l = 0; l < layers; ++l) demanding[l] = 0;
    for (int i = 0; i < n_demanding; ++i) demanding[order[i]] = 1;
    return AMSKV_OK;
}

int amskv_kept_segments(const amskv_cache* cache, int layer, int scale, int32_t* ids, int32_t* n)
{
    if (bad_layer_scale(cache, layer, scale) || !ids || !n) return AMSKV_ERR_INVALID;
    *n = cache->layout[layer].kept(scale, ids);
    return AMSKV_OK;
}

int amskv_evicted_at(const amskv_cache* cache, int layer, int scale, int32_t* ids, int32_t* n)
{
    if (bad_layer_scale(cache, layer, scale) || !ids || !n) return AMSKV_ERR_INVALID;
    *n = cache->layout[layer].evicted(scale, ids);
    return AMSKV_OK;
}

int amskv_resident_ranges(const amskv_cache* cache, int layer, int scale, int32_t* ranges, int32_t* n)
{
    if (bad_layer_scale(cache, layer, scale) || !ranges || !n) return AMSKV_ERR_INVALID;
    Range r[kMaxRanges];
    *n = cache->layout[layer].ranges(cache->tokens, scale, r);
    for (int i = 0; i < *n; ++i) {
        ranges[2 * i] = r[i].start;
        ranges[2 * i + 1] = r[i].len;
    }
    return AMSKV_OK;
}

int amskv_attended_tokens(const amskv_cache* cache, int layer, int scale, int32_t* runs, int32_t* n)
{
    if (bad_layer_scale(cache, layer, scale) || !runs || !n) return AMSKV_ERR_INVALID;
    TokenRun r[2 * AMSKV_MAX_SCALES];
    *n = cache->layout[layer].attended(cache->tokens, scale, r);
    for (int i = 0; i < *n; ++i) {
        runs[3 * i] = r[i].segment;
        runs[3 * i + 1] = r[i].first;
        runs[3 * i + 2] = r[i].count;
    }
    return AMSKV_OK;
}

int amskv_append_copies(const amskv_cache* cache, int layer, int scale, int32_t* copies, int32_t* n)
{
    if (bad_layer_scale(cache, layer, scale) || !copies || !n) return AMSKV_ERR_INVALID;
    static_assert(LayerLayout::kMaxPieces == AMSKV_MAX_APPEND_COPIES, "header and layout disagree");
    Piece p[LayerLayout::kMaxPieces];
    *n = cache->layout[layer].pieces(cache->tokens, scale, p);
    for (int i = 0; i < *n; ++i) {
        copies[3 * i] = p[i].src;
        copies[3 * i + 1] = p[i].dst;
        copies[3 * i + 2] = p[i].len;
    }
    return AMSKV_OK;
}

int amskv_cache_bytes(const amskv_cache* cache, size_t* allocated, size_t* resident_now, size_t* peak)
{
    if (!cache) return AMSKV_ERR_INVALID;
    if (allocated) *allocated = cache->arena_bytes;
    if (resident_now) *resident_now = cache->resident_now;
    if (peak) *peak = cache->peak;
    return AMSKV_OK;
}

int amskv_status(amskv_cache* cache, int* device_status)
{
    if (!cache || !device_status) return AMSKV_ERR_INVALID;
    if (cache->plan_only()) { *device_status = 0; return AMSKV_OK; }
    int word = 0;
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(&word, cache->status_word(), sizeof(int), cudaMemcpyDeviceToHost);
    // read and clear: one report must not mark every later call of this cache as failed
    if (e == cudaSuccess && word != 0) e = cudaMemset(cache->status_word(), 0, sizeof(int));
    if (e != cudaSuccess) { (void)cudaGetLastError(); return AMSKV_ERR_CUDA; }
    *device_status = word;
    return word == 0 ? AMSKV_OK : AMSKV_ERR_DEVICE_TIMEOUT;
}

int amskv_selftest_wait_timeout(amskv_cache* cache, uint32_t iterations, void* stream)
{
    if (!cache) return AMSKV_ERR_INVALID;
    if (cache->plan_only()) return AMSKV_ERR_UNSUPPORTED;
    if (iterations < 1 || iterations > (1u << 20)) return AMSKV_ERR_INVALID;
    cudaError_t e = launch_wait_gives_up(iterations, cache->status_word(), static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { (void)cudaGetLastError(); return AMSKV_ERR_CUDA; }
    return AMSKV_OK;
}

int64_t amskv_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* amskv_strerror(int code)
{
    switch (code) {
        case AMSKV_OK: return "ok";
        case AMSKV_ERR_INVALID: return "invalid argument";
        case AMSKV_ERR_ORDER: return "call out of order";
        case AMSKV_ERR_NOMEM: return "not enough device memory";
        case AMSKV_ERR_UNSUPPORTED: return "unsupported shape or mode";
        case AMSKV_ERR_CUDA: return "CUDA call failed";
        case AMSKV_ERR_DEVICE_TIMEOUT: return "a device-side wait gave up";
        default: return "unknown error";
    }
}

}  // extern "C"
