/*
 * amskv.h -- C ABI of the AMS-KV hot path on one NVIDIA B200 (sm_100a).
 *
 * What the library does (AMS-KV, "Adaptive Multi-Scale KV Caching", Sec. 4.3):
 * a next-scale-prediction transformer generates an image scale by scale; the keys and
 * values of every finished scale are cached per layer.  This library owns that cache as
 * one segment per scale, keeps only the segments the policy retains (the condensed,
 * coarsest scales plus the most recent, local scales in cache-efficient layers; every
 * scale in cache-demanding layers), and computes exact softmax attention of the current
 * scale's queries over exactly the retained segments.
 *
 * Conventions
 *  - Scales are numbered from 0.  A scale of side s has s*s tokens in row-major raster
 *    order (token = y*s + x).  rows = 2 * batch when classifier-free guidance doubles it.
 *  - Every function returns AMSKV_OK (0) or a negative AMSKV_ERR_* code.  Nothing throws,
 *    aborts or prints.
 *  - "device pointer" = memory of the current CUDA device, owned by the caller, bf16 unless
 *    said otherwise, innermost (channel) dimension contiguous, 16-byte aligned, and valid
 *    until the stream has executed the call.  "host pointer" = ordinary host memory.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *  - amskv_append / amskv_attend / amskv_layer_similarity only enqueue work on `stream`:
 *    they allocate nothing, copy nothing between host and device and do not synchronise.
 *  - Device-side ordering is the caller's when it uses more than one stream.  On one stream the
 *    calls run in the order made.  With several streams two orders must be kept per layer
 *    (with events): append(layer, k) before attend(layer, k), and attend(layer, k) before
 *    append(layer, k + 1), which may overwrite a segment that attend(layer, k) still reads.
 *    Appends of different layers are independent of each other and of other layers' attends,
 *    so they can run on a side stream underneath the attention kernels.
 *  - A cache object may be used by one host thread at a time.
 *  - There is no CPU implementation behind any entry point: without a CUDA device the
 *    compute calls fail with AMSKV_ERR_CUDA.
 */
#ifndef AMSKV_H_
#define AMSKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define AMSKV_API __attribute__((visibility("default")))
#else
#define AMSKV_API
#endif

#define AMSKV_OK 0
#define AMSKV_ERR_INVALID (-1)        /* bad argument (null, out of range, misaligned)      */
#define AMSKV_ERR_ORDER (-2)          /* call out of the append/attend order contract       */
#define AMSKV_ERR_NOMEM (-3)          /* arena too small or device allocation failed         */
#define AMSKV_ERR_UNSUPPORTED (-4)    /* shape or mode this build does not handle            */
#define AMSKV_ERR_CUDA (-5)           /* a CUDA runtime / driver call failed                 */
#define AMSKV_ERR_DEVICE_TIMEOUT (-6) /* a bounded device-side wait gave up (see amskv_status) */

#define AMSKV_MAX_SCALES 32

/* amskv_desc.flags */
#define AMSKV_FLAG_PLAN_ONLY 1u /* host bookkeeping only: no device memory is touched and
                                   attend / similarity are refused; append takes NULL K, V
                                   (append_attend does the bookkeeping of append, whatever its pointers).
                                   For sizing and for inspecting the policy without a GPU. */

#define AMSKV_FLAG_BULK_APPEND 2u /* amskv_append moves token-contiguous inputs with bulk asynchronous
                                    copies from 32-thread CTAs that need 24 KB of shared memory and
                                    few registers, so that they fit on an SM beside the attention
                                    kernel's CTAs.  Meant for callers that enqueue appends on a side
                                    stream underneath attention; on its own it is a little slower
                                    than the default copy kernel. */

#define AMSKV_FLAG_TRANSIENT_LAST_SCALE 4u /* The last scale of the schedule is never stored: no later scale
                                    reads it (Algorithm 1 would append it all the same).  The arena reserves no
                                    room for it -- a cache-demanding layer of the 680-token schedule holds 424
                                    tokens instead of 680, a cache-efficient one (2 condensed, 2 local scales) 274
                                    instead of 430 -- and its step must be made through amskv_append_attend
                                    (or amskv_step_host), which reads the scale's K and V from the caller's
                                    tensors; amskv_append refuses it with AMSKV_ERR_UNSUPPORTED.  The attention
                                    result is the same as without the flag.  The policy queries report the
                                    scale as not retained (amskv_kept_segments) and as dropped at its own step
                                    (amskv_evicted_at). */

#define AMSKV_FLAG_NVTX 8u /* amskv_append, amskv_attend and amskv_append_attend wrap their work in an NVTX range
                              named after the call, layer and scale (timeline tools show which kernels belong to
                              which step); no effect on results */

/* amskv_set_attend_path */
#define AMSKV_PATH_AUTO 0   /* warp-per-item kernel for the coarse scales (at most 16 queries and 32
                               retained keys; CUDA-core kernel for a single query token with several
                               keys), paired tcgen05 kernel otherwise                               */
#define AMSKV_PATH_SIMT 1   /* always the CUDA-core kernel                                     */
#define AMSKV_PATH_TENSOR 2 /* always the single-stream tcgen05 kernel                         */
#define AMSKV_PATH_TENSOR_PAIR 3 /* always the paired tcgen05 kernel (two query tiles per CTA)  */
#define AMSKV_PATH_SMALL 4  /* the warp-per-item kernel wherever it applies (paired kernel elsewhere) */

typedef struct amskv_cache amskv_cache; /* opaque; owned by the library */

/*
 * Per-layer policy (Sec. 4.1 scale groups, Sec. 4.2 layer classes).
 *   n_condensed      c >= 0: the first c scales are pinned (the paper's C_cds, counted in
 *                    scales; the ablation in Appendix A uses 0, 1 and 2).
 *   n_local          w >= 1: the w most recent scales are kept, the just-appended one
 *                    included (Algorithm 2 keeps the tail of the cache after the append).
 *   cache_demanding  AMSKV_LAYER_EFFICIENT (0), AMSKV_LAYER_DEMANDING (1): the layer keeps every scale
 *                    (full retention), or AMSKV_LAYER_PROMOTABLE (2): the layer starts cache-efficient
 *                    and amskv_promote_layer may make it cache-demanding until its first eviction
 *                    (Algorithm 1 decides at the first overflow).  A promotable layer's region is sized
 *                    and laid out like a cache-demanding layer's, whether or not it is promoted.
 * A cache-efficient layer keeps scale s at step k iff s < c or s > k - w.
 */
#define AMSKV_LAYER_EFFICIENT 0
#define AMSKV_LAYER_DEMANDING 1
#define AMSKV_LAYER_PROMOTABLE 2
typedef struct {
    int32_t n_condensed;
    int32_t n_local;
    int32_t cache_demanding;
} amskv_layer_policy;

/*
 * Per-layer token budget: Algorithm 1 with Algorithm 2 (Appendix F) as its roll, taken literally,
 * with capacities counted in tokens (Sec. 5 sets C_max to the condensed scales plus the last two
 * scales and C_min to the condensed scales plus the penultimate one).
 *   budget_tokens     C_bgt > 0: the layer holds at most this many tokens per (row, head).  Pass
 *                     C_max for a cache-demanding layer and C_min for a cache-efficient one:
 *                     nothing is evicted before a layer's first overflow, so starting at C_max
 *                     equals Algorithm 1's promotion at that overflow.  0 = this layer follows
 *                     its amskv_layer_policy (whole scales) instead.
 *   condensed_tokens  C_cds >= 0 in tokens (clamped to the budget): the first C_cds cached
 *                     tokens are pinned.
 *   promoted_budget_tokens  0, or C_max >= budget_tokens: the layer starts with budget_tokens (C_min)
 *                     and amskv_promote_layer may raise its budget to this value until its first
 *                     overflow, as Algorithm 1 does when S < theta there.  The region is sized for
 *                     the larger of the two layouts.
 * After the append of a scale the cache holds every cached token while their number is within
 * the budget, else the first C_cds of them and the most recent C_bgt - C_cds: the tail may end
 * inside a scale.  A scale with more tokens than the budget is never cached (Algorithm 1 skips
 * it).  The queries of a scale always attend to that whole scale besides the cache (the paper
 * leaves this open; without it the skipped scale would not see itself): a scale that is not
 * resident in full after its own append is kept in a transient slot until the next append.
 */
typedef struct {
    int32_t budget_tokens;
    int32_t condensed_tokens;
    int32_t promoted_budget_tokens;
} amskv_token_budget;

typedef struct {
    int32_t layers;
    int32_t heads;
    int32_t head_dim;            /* 64 or 128                                              */
    int32_t rows;                /* sequences held at once (2 * batch under guidance)      */
    int32_t n_scales;            /* 1 .. AMSKV_MAX_SCALES                                  */
    const int32_t* scale_sides;  /* [n_scales] side lengths, each >= 1; copied             */
    const amskv_layer_policy* policy; /* [layers]; copied                                  */
    float softmax_scale;         /* <= 0 selects 1/sqrt(head_dim)                          */
    uint32_t flags;              /* AMSKV_FLAG_*                                           */
    const amskv_token_budget* token_budget; /* [layers] or NULL (no layer uses token budgets); copied */
} amskv_desc;

/* Bytes of device memory a cache for `desc` needs (its KV arena; Appendix D, Eq. 5 counts
 * the same tokens).  Host-only. */
AMSKV_API int amskv_cache_required_bytes(const amskv_desc* desc, size_t* bytes);

/*
 * Create a cache (one independent cache per layer, Sec. 4.3).
 *   dev_mem    device pointer to an arena of dev_bytes bytes, 256-byte aligned, owned by the
 *              caller and kept alive until destroy; or NULL, in which case the library
 *              allocates (and later frees) the arena itself.
 * The arena is zero-filled on the default stream and the call synchronises once.
 * Errors: INVALID (descriptor), NOMEM (dev_bytes too small, allocation failed), CUDA.
 */
AMSKV_API int amskv_cache_create(const amskv_desc* desc, void* dev_mem, size_t dev_bytes, amskv_cache** out);

/* Free the object, and the arena only if the library allocated it. */
AMSKV_API int amskv_cache_destroy(amskv_cache* cache);

/* Forget all appended scales (start a new batch of images) and undo promotions.  Metadata only. */
AMSKV_API int amskv_cache_reset(amskv_cache* cache);

/*
 * Append scale `scale` of `layer` and evict in place (Algorithm 1 "append", then
 * Algorithm 2 "rolling", at scale granularity).
 *   K, V      device pointers, logical shape [rows, heads, T, head_dim], T = side^2.
 *   strides   element strides of the (row, head, token) dimensions, or NULL for a
 *             contiguous tensor; all three must be multiples of 8, the token stride at least
 *             head_dim.  A zero row (head) stride -- one slice repeated, as an expanded view has --
 *             is refused with INVALID when there is more than one row (head), and always for a
 *             tensor the call writes (`out`).
 * The segment that leaves the local window is dropped by bookkeeping alone; its slot is
 * the one the new segment is written to.  Scales must be appended in order 0, 1, 2, ...
 * per layer (ORDER otherwise).  Non-finite K/V values give unspecified results.
 */
AMSKV_API int amskv_append(amskv_cache* cache, int layer, int scale, const void* K, const void* V,
                 const int64_t strides[3], void* stream);

/*
 * Attention of the queries of `scale` over the segments `layer` retains at that step
 * (Sec. 3.1, Eq. 2: a whole scale is conditioned on whole earlier scales, so there is no
 * mask inside the retained set):  out = softmax(softmax_scale * Q K^T) V.
 *   Q, out    device pointers, [rows, heads, T, head_dim] bf16; strides as in append.
 * `scale` must be the scale most recently appended to `layer` (ORDER otherwise).  out must not
 * overlap Q.
 * Arithmetic: bf16 inputs, fp32 accumulation, probabilities rounded to bf16 before the
 * second product on the tensor-core path, bf16 output.
 */
AMSKV_API int amskv_attend(amskv_cache* cache, int layer, int scale, const void* Q, void* out,
                 const int64_t q_strides[3], const int64_t o_strides[3], void* stream);

/*
 * amskv_append(layer, scale, K, V) followed by amskv_attend(layer, scale, Q, out), with the same
 * results, cache state and order contract (scale must be the layer's next scale), in one kernel
 * launch where possible: Algorithm 1 appends a scale right before that scale attends, so the
 * paired tensor-core kernel can read the scale's K and V from the caller's tensors, use them as
 * keys and values beside the older retained tokens it reads from the cache, and write them to
 * the scale's place in the cache on the way -- the separate copy and its second read of K and V
 * disappear.  The warp-per-item kernel of the coarse scales does the same (it reads the scale's K and V
 * from the caller's tensors and stores the registers that feed its products), and a single-token scale
 * that is its own only key is one copy kernel (out = V).  Appends that are more than one contiguous copy
 * (a token budget whose ring wraps inside the scale), scales served by the CUDA-core or the single-stream
 * kernel and, under AMSKV_PATH_AUTO, paired-kernel scales of fewer than 32 tokens and scales where
 * splitting the current scale off its cache range would add a 64-token key tile, run as the two calls.
 *   K, V: as for amskv_append (one stride triple kv_strides for both); Q, out: as for
 *   amskv_attend.  out must not overlap Q, K or V.
 * Stream ordering: as for the two calls -- this call must come after attend(layer, scale - 1)
 * has finished reading (same stream, or an event).
 */
AMSKV_API int amskv_append_attend(amskv_cache* cache, int layer, int scale, const void* K, const void* V,
                                  const int64_t kv_strides[3], const void* Q, void* out, const int64_t q_strides[3],
                                  const int64_t o_strides[3], void* stream);

/*
 * Attention density (Sec. 4.1): d = (1 / T_i) * sum over the queries of `scale` and over the keys of a
 * retained scale i of the attention probabilities -- the attention a retained scale receives per key
 * token, the quantity behind the choice of the condensed and local scales.  An analysis call, not part
 * of the generation step; it recomputes the softmax of amskv_attend(layer, scale, Q) on the CUDA cores
 * (fp32, no rounding of the probabilities).
 *   out          device pointer to heads * n doubles, n = the number of runs amskv_attended_tokens
 *                reports for (layer, scale); out[h * n + r] receives the density of run r for head h,
 *                averaged over the rows.  For a run that is part of a segment (token budgets) the
 *                divisor is the run's own token count.  Zeroed and filled by the call, on `stream`.
 *   out_entries  doubles `out` can hold (NOMEM if too few).
 * `scale` must be the scale most recently appended to `layer` (ORDER otherwise); a never-stored last
 * scale is refused (UNSUPPORTED: its keys are not in the cache).  The sums are accumulated with
 * floating-point atomic adds, so results agree to rounding only between calls.
 * Identity: sum over r of count_r * out[h * n + r] = T of `scale` (every query's probabilities sum to 1).
 */
AMSKV_API int amskv_attention_density(amskv_cache* cache, int layer, int scale, const void* Q,
                                      const int64_t q_strides[3], double* out, size_t out_entries, void* stream);

/*
 * amskv_attend(layer, scale, Q, out) that also returns the attention density of the same queries (Sec. 4.1,
 * the definition of d), as a by-product of the attention launch: where the paired tensor-core kernel serves
 * the scale, its key tiles are cut at the boundaries of the runs of attended tokens, and the un-normalised
 * probability mass of a query row on a run is a running sum of the per-tile sums the softmax computes anyway;
 * the rows are normalised by their row sums in the epilogue and added up per (head, run).  One launch, no
 * second pass over the keys; the cut tiles make the launch somewhat longer than a plain amskv_attend (more,
 * partly filled key tiles).  `out` is the same as amskv_attend's.  `density`, `density_entries` and the
 * meaning of the numbers are those of amskv_attention_density (probabilities after their rounding to bf16,
 * where that call uses them unrounded: they agree to about 1e-4 relative).  Scales the other kernels serve,
 * and layers with more than 16 runs, run as amskv_attend followed by amskv_attention_density.
 * Errors: as for the two calls.
 */
AMSKV_API int amskv_attend_density(amskv_cache* cache, int layer, int scale, const void* Q, void* out,
                                   const int64_t q_strides[3], const int64_t o_strides[3], double* density,
                                   size_t density_entries, void* stream);

/*
 * On-line promotion (Sec. 4.3, Algorithm 1: when the cache first exceeds the budget C_min and the
 * similarity S(k_i, resized k_{i-1}) of the arriving scale is below theta, the budget becomes C_max).
 * amskv_first_overflow_scale reports the scale i whose append is the first to exceed the layer's budget
 * (n_scales if none does): the caller computes S for that scale with amskv_layer_similarity (it holds
 * K_i, and K_{i-1} from the previous step), compares it with theta (amskv_classify_by_threshold) and, if
 * the layer is cache-demanding, calls amskv_promote_layer BEFORE appending scale i.  A layer created
 * AMSKV_LAYER_PROMOTABLE then keeps every scale; a token-budget layer with promoted_budget_tokens gets
 * that budget.  Host-only, metadata only: nothing has been evicted yet and every cached token already
 * sits where the larger layout expects it.
 * Scope: Algorithm 1 repeats the test at every later overflow while the budget is still C_min; this
 * library takes the decision at the first overflow only -- after an eviction the call is refused.
 * Errors: UNSUPPORTED (the layer was not created promotable), ORDER (the overflowing scale has already
 * been appended); promoting twice is harmless.  amskv_cache_reset returns every layer to the class it
 * was created with.
 */
AMSKV_API int amskv_first_overflow_scale(const amskv_cache* cache, int layer, int* scale);
AMSKV_API int amskv_promote_layer(amskv_cache* cache, int layer);

/* Choose the kernel used by amskv_attend (AMSKV_PATH_*).  The default is AUTO. */
AMSKV_API int amskv_set_attend_path(amskv_cache* cache, int path);

/*
 * One generation step from HOST buffers: copies K, V, Q of `scale` (contiguous
 * [rows, heads, T, head_dim] bf16 host arrays; pinned memory makes the copies asynchronous)
 * into `staging`, appends, attends and copies the result to the host array `out`.
 *   staging        device pointer, at least amskv_step_staging_bytes() bytes, 256-byte aligned.
 * Everything is enqueued on `stream`; the host arrays must stay valid until it has run.
 */
AMSKV_API int amskv_step_host(amskv_cache* cache, int layer, int scale, const void* K_host, const void* V_host,
                    const void* Q_host, void* out_host, void* staging, size_t staging_bytes,
                    void* stream);

/* Bytes of staging amskv_step_host needs for the largest scale of this cache. */
AMSKV_API int amskv_step_staging_bytes(const amskv_cache* cache, size_t* bytes);

/*
 * Inter-scale key similarity (Sec. 4.3, Eq. 4): resizes the keys of the previous scale to
 * the current scale's side by 2-D bilinear interpolation (half-pixel centres, edge clamp)
 * and returns the sum over every (row, head, token, channel) of the squared difference,
 *   ss = || k_i - resize(k_{i-1}) ||_2^2,   so that S = -sqrt(ss).
 *   K_prev, K_cur   device pointers, contiguous [rows, heads, side^2, head_dim] bf16.
 *   out_ss          device pointer to one double (written by the kernel).
 *   workspace       device pointer, amskv_similarity_workspace_bytes() bytes, 256-byte
 *                   aligned; scratch for per-block partial sums, overwritten by every call,
 *                   so calls sharing a workspace must not overlap on the device.
 * The reduction order is fixed, so equal inputs give bit-equal results.
 */
AMSKV_API int amskv_layer_similarity(const void* K_prev, int side_prev, const void* K_cur, int side_cur,
                           int rows, int heads, int head_dim, double* out_ss, void* workspace,
                           size_t workspace_bytes, void* stream);

/* Bytes of workspace amskv_layer_similarity needs (independent of the problem size). */
AMSKV_API size_t amskv_similarity_workspace_bytes(void);

/*
 * amskv_layer_similarity for callers that cannot provide a workspace because they cannot
 * allocate device memory at the point of the call: code running inside a memory pool whose
 * budget is fixed, a plug-in that is handed its tensors and nothing else, a real-time or
 * latency-critical loop in which cudaMalloc (which may synchronise the whole device) is
 * forbidden.  (The paper has no counterpart of this call; it exists for those callers.)
 * Same arguments, arithmetic, reduction order and result as amskv_layer_similarity, but the
 * per-block partial sums go to a 16 KB array that lives inside the library image on every
 * device that loads it, until the process exits.  The call allocates and frees nothing.
 *   Limit       rows * heads * side_cur^2 * head_dim / 8 <= 2^30 (16 GiB of current-scale
 *               keys); larger problems are refused with AMSKV_ERR_UNSUPPORTED, and devices
 *               with an ordinal of 64 or more likewise.
 *   First call  on each device looks up the array's device address (with that device
 *               current); make that first call outside any stream capture.
 *   Sharing     all calls on a device use the one array.  It keeps whatever the last call
 *               left there; nothing in it has to start at zero because every slot that is read
 *               is rewritten by the same call first.  Two calls that overlap on the device (on
 *               different streams, or from different threads) race on it: serialise them.
 * Errors: INVALID (null or misaligned pointer, bad side / rows / heads), UNSUPPORTED
 * (head_dim, size limit, device ordinal), CUDA.
 */
AMSKV_API int amskv_layer_similarity_static(const void* K_prev, int side_prev, const void* K_cur, int side_cur,
                                  int rows, int heads, int head_dim, double* out_ss, void* stream);

/*
 * Layer classification from similarity scores (host-only).
 *   by threshold: demanding[l] = scores[l] < theta (strict; Algorithm 1).
 *   by rank:      the n_demanding lowest-scoring layers are demanding, ties to the lower
 *                 layer index (the similarity-aware allocation S2 of Sec. 4.2).
 */
AMSKV_API int amskv_classify_by_threshold(const double* scores, int layers, double theta, int32_t* demanding);
AMSKV_API int amskv_classify_lowest(const double* scores, int layers, int n_demanding, int32_t* demanding);

/* Segment ids `layer` retains right after scale `scale` was appended, ascending (host-only;
 * a pure function of the policy).  ids must hold AMSKV_MAX_SCALES entries.  Under a token budget a
 * segment counts as retained while the cache holds at least one of its tokens. */
AMSKV_API int amskv_kept_segments(const amskv_cache* cache, int layer, int scale, int32_t* ids, int32_t* n);

/* Segment ids the append of `scale` drops from `layer` (host-only).  Under a token budget: the
 * segments that lose their last cached token; a scale too large to be cached is reported at its own
 * step. */
AMSKV_API int amskv_evicted_at(const amskv_cache* cache, int layer, int scale, int32_t* ids, int32_t* n);

/* Token ranges (start, length) of the layer's per-(row, head) arena region that attend
 * reads at `scale`, merged where adjacent (host-only).  ranges must hold
 * 2 * AMSKV_MAX_SCALES entries. */
AMSKV_API int amskv_resident_ranges(const amskv_cache* cache, int layer, int scale, int32_t* ranges, int32_t* n);

/* The keys the queries of `scale` attend to in `layer`, as runs (segment, first token, count) in
 * ascending segment order (host-only; a pure function of the policy).  Whole segments under the
 * scale-granular policy; under a token budget a segment may appear with part of its tokens, as up to
 * two runs (its share of the pinned head and of the tail).  runs must hold 3 * 2 * AMSKV_MAX_SCALES
 * entries; *n receives the number of runs. */
AMSKV_API int amskv_attended_tokens(const amskv_cache* cache, int layer, int scale, int32_t* runs, int32_t* n);

/* The copies amskv_append(layer, scale) performs, as triples (first source token, destination
 * position in the per-(row, head) region, tokens) (host-only).  One copy under the scale-granular
 * policy; up to AMSKV_MAX_APPEND_COPIES under a token budget (pinned head, the ring's two sides of
 * its wrap point, transient slot).  copies must hold 3 * AMSKV_MAX_APPEND_COPIES entries. */
#define AMSKV_MAX_APPEND_COPIES 4
AMSKV_API int amskv_append_copies(const amskv_cache* cache, int layer, int scale, int32_t* copies, int32_t* n);

/* Bytes: the arena, the KV bytes resident now, and the largest residency seen since the
 * last reset. */
AMSKV_API int amskv_cache_bytes(const amskv_cache* cache, size_t* allocated, size_t* resident_now, size_t* peak);

/* Reads the device status word (synchronises the device) and clears it.  *device_status is 0 when no
 * kernel reported a problem since the last call; otherwise it is the code of the first bounded wait that
 * gave up (1: a key/value or query copy did not arrive, 2: the MMA-issuing warp gave up, 3: a softmax
 * group or another role gave up) and the return value is AMSKV_ERR_DEVICE_TIMEOUT.  A kernel that gives
 * up still returns normally (its roles wind down, copies in flight are awaited, tensor memory is freed),
 * so the context stays usable, but the outputs of that launch are undefined: the calls that enqueue work
 * return AMSKV_OK regardless, and only this call tells.  amskv_cache_reset does not touch the word. */
AMSKV_API int amskv_status(amskv_cache* cache, int* device_status);

/* Diagnostic (the paper has no counterpart): enqueues one 32-thread kernel whose bounded wait -- the same
 * helper every attention kernel waits with -- runs out after `iterations` polls (1 .. 2^20) of a barrier
 * that nothing arrives at.  The kernel records code 3 in the cache's status word and returns normally;
 * nothing faults or hangs.  Lets a caller (and the tests) check the whole reporting chain:
 * amskv_status must then return AMSKV_ERR_DEVICE_TIMEOUT once, and AMSKV_OK afterwards. */
AMSKV_API int amskv_selftest_wait_timeout(amskv_cache* cache, uint32_t iterations, void* stream);

/* Number of kernels this library has launched since it was loaded. */
AMSKV_API int64_t amskv_launch_count(void);

AMSKV_API const char* amskv_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* AMSKV_H_ */
