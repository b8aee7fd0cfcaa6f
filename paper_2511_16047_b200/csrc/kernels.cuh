// Internal interface between the C ABI (api.cu) and the kernels.  Not installed.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>

#include "policy.hpp"

namespace amskv {

constexpr int kMaxRanges = 32;

// Token ranges of one layer's per-item region that an attention call reads; passed by value.
struct RangeList {
    int32_t n;
    int32_t total;  // sum of len
    Range r[kMaxRanges];
};

// A [rows, heads, tokens, D] bf16 tensor described by element strides (D contiguous).
struct Strided {
    const void* ptr;
    int64_t row, head, token;
};

// One layer's KV region: item i (= row * heads + head) owns 2 * capacity * D bf16 values,
// keys first ([capacity][D]) and values right behind them.
struct LayerRegion {
    __nv_bfloat16* base;
    int32_t capacity;  // tokens per item
};

// Device status codes written (first one wins) when a bounded wait gives up.
enum DeviceStatus : int {
    kStatusOk = 0,
    kStatusTmaTimeout = 1,
    kStatusMmaTimeout = 2,
    kStatusSyncTimeout = 3,
};

cudaError_t launch_append(const Strided& K, const Strided& V, const LayerRegion& region, int32_t token_offset,
                          int32_t T, int32_t rows, int32_t heads, int32_t D, bool bulk, int* status, int sm_count,
                          cudaStream_t stream);

// The current scale taken from the caller's K/V tensors instead of the cache: the last entry of the
// range list given with it stands for that scale (start 0, len T).  With `store`, the kernel also
// writes the scale to position `dst` of every item's part of `region` (the append fused into attention).
// `rider`: up to 16 older tokens of the cache (positions rider_tok .. rider_tok + rider_valid - 1) that are
// not in the range list but ride in the free 16-token box of the scale's last, partly filled key tile, so
// that they do not cost a tile of their own (rider_valid = 0: none; the scale's last tile must then have
// a box to spare: (T mod 64) in 1..48).
struct CurrentScaleSource {
    Strided K, V;
    bool store;
    int32_t dst;
    LayerRegion region;
    int32_t rider_tok = 0, rider_valid = 0;
};

// (the CUDA-core kernel takes a current-scale source without `store` only)
cudaError_t launch_attend_simt(const Strided& Q, const Strided& O, const LayerRegion& region, const RangeList& ranges,
                               int32_t T, int32_t rows, int32_t heads, int32_t D, float softmax_scale,
                               cudaStream_t stream, const CurrentScaleSource* cur = nullptr);

constexpr int kSimilarityMaxBlocks = 2048;
cudaError_t launch_similarity(const __nv_bfloat16* K_prev, int32_t side_prev, const __nv_bfloat16* K_cur,
                              int32_t side_cur, int64_t items, int32_t D, double* out_ss, double* partials,
                              cudaStream_t stream);

// Tensor-core path.  The tensor maps are built on the host by the caller of launch_attend_tc.
struct TcMaps;  // defined in attend_tc.cu
bool tc_supported(int32_t D);
// Encodes the tensor maps a layer needs for its K and V streams; returns false on failure.
// (box = 64 channels x box_rows tokens of one item)
bool tc_encode_kv_maps(const LayerRegion& region, int64_t items, int32_t D, int box_rows, void* k_map_out,
                       void* v_map_out);
cudaError_t launch_attend_tc(const Strided& Q, const Strided& O, const LayerRegion& region, const void* k_map,
                             const void* v_map, const RangeList& ranges, int32_t T, int32_t rows, int32_t heads,
                             int32_t D, float softmax_scale, int* status, int sm_count, cudaStream_t stream);

// Encodes the rank-4 tensor map of a strided Q tensor (box = 64 channels x box_rows tokens).
bool tc_encode_q_map(const Strided& Q, int32_t T, int32_t rows, int32_t heads, int32_t D, int box_rows, void* map_out,
                     int pos[3]);
// The layer's region as store targets (box = 64 channels x box_rows tokens) whose token extent ends at
// `token_extent`, so that a box reaching past it is clipped by the copy engine.
bool tc_encode_kv_store_maps(const LayerRegion& region, int64_t items, int32_t D, int box_rows, int32_t token_extent,
                             void* k_map_out, void* v_map_out);

// Attention density as a by-product of a paired-kernel launch: `ranges` then has one entry per piece of a run
// of attended tokens (run_of_range[i] = the run of entry i; entries are never merged across runs), and the
// launch adds weight[r] * (sum over the item's queries of the normalised probability mass on run r) to
// out[head * n_runs + r] with atomic adds (out is zeroed by the caller, on the same stream).
constexpr int kPairMaxDensityRuns = 16;
struct PairDensity {
    double* out;
    int32_t n_runs;
    float weight[kPairMaxDensityRuns];
    int8_t run_of_range[kMaxRanges];
};

// Paired tensor-core kernel: two softmax groups per CTA, probabilities kept in tensor memory.
cudaError_t launch_attend_pair(const Strided& Q, const Strided& O, const void* k_map16, const void* v_map16,
                               const void* k_map64, const void* v_map64, const RangeList& ranges, int32_t T, int32_t rows, int32_t heads, int32_t D,
                               float softmax_scale, int* status, int sm_count, cudaStream_t stream,
                               const CurrentScaleSource* cur = nullptr, const PairDensity* density = nullptr);

// Warp-per-item kernel for the coarse scales: every retained key in one register tile.
constexpr int kSmallMaxKeys = 32;
constexpr int kSmallMaxQueries = 16;
bool small_supported(int32_t T, int32_t total_keys);
// With `cur`, `ranges` lists the cached keys only and the current scale's T tokens come from the caller's
// tensors (and are written to position cur->dst of the region when cur->store is set): T plus the cached
// keys must fit the limits.  A single-token scale that is its own only key is served by a copy kernel.
cudaError_t launch_attend_small(const Strided& Q, const Strided& O, const LayerRegion& region, const RangeList& ranges,
                                int32_t T, int32_t rows, int32_t heads, int32_t D, float softmax_scale,
                                cudaStream_t stream, const CurrentScaleSource* cur = nullptr);

// Attention density: the pieces of the per-item region that hold the attended tokens, each with the run
// (of the attended-token list) it belongs to and the weight 1 / (tokens of that run).
constexpr int kMaxDensityPieces = 96;
struct DensityPieces {
    int32_t n, n_runs;
    int32_t start[kMaxDensityPieces], len[kMaxDensityPieces], run[kMaxDensityPieces];
    double weight[kMaxDensityPieces];
};
cudaError_t launch_density(const Strided& Q, const LayerRegion& region, const DensityPieces& pieces, int32_t T,
                           int32_t rows, int32_t heads, int32_t D, float softmax_scale, double* out, cudaStream_t stream);

// One warp whose bounded wait runs out after `limit` iterations (nothing ever arrives): records
// kStatusSyncTimeout in *status and returns normally.
cudaError_t launch_wait_gives_up(uint32_t limit, int* status, cudaStream_t stream);

void count_launch(int n = 1);

// A kernel's dynamic shared-memory limit is a per-device setting: raised once per device and kernel,
// from whichever host thread gets there first (setting it twice is harmless).
struct SharedMemoryOptIn {
    std::atomic<uint64_t> done{0};   // bit d: set on device d
    template <typename Kernel>
    cudaError_t ensure(Kernel* kernel, int bytes)
    {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64 && ((done.load(std::memory_order_acquire) >> dev) & 1u)) return cudaSuccess;
        e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        if (e == cudaSuccess && dev >= 0 && dev < 64) done.fetch_or(1ull << dev, std::memory_order_release);
        return e;
    }
};

}  // namespace amskv
