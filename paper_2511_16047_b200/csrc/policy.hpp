// Host-side bookkeeping of the segmented KV cache: which segments a layer keeps, where each
// segment lives inside the layer's per-(row, head) region, and which token ranges an
// attention call reads.  Integers only; no CUDA here.
#pragma once

#include <algorithm>
#include <cstdint>
#include <vector>

namespace amskv {

struct Range {
    int32_t start;  // first token of the range inside the per-item region
    int32_t len;    // tokens
};

// One contiguous copy of an append: `len` tokens of the incoming scale, from its token `src`,
// to position `dst` of the per-item region.
struct Piece {
    int32_t src, dst, len;
};

// `count` tokens of segment `segment`, from its token `first`.
struct TokenRun {
    int32_t segment, first, count;
};

// Layout of one layer.  A cache-demanding layer (or one whose pinned prefix plus window
// already covers the whole schedule) stores its segments back to back in scale order.
// A cache-efficient layer has a pinned region for the condensed scales and n_local slots
// that the later scales rotate through: scale s >= c uses slot (s - c) mod w, so the segment
// that leaves the window (s - w) is the previous tenant of the slot the new segment takes and
// is evicted by being overwritten.  Slot 0 sits below the pinned region with its tenant
// right-aligned and slot 1 directly above the pinned region, which makes the resident
// tokens one contiguous run whenever w <= 2.
struct LayerLayout {
    static constexpr int32_t kMinCapacity = 16;   // with a never-stored last scale a region could be empty; its tensor maps need an extent
    int32_t c = 0;          // pinned scales (clamped to the schedule length)
    int32_t w = 1;          // window, in scales (clamped)
    bool full = false;      // nothing is ever evicted
    bool skip_last = false; // the last scale of the schedule is never stored (no later scale reads it)
    int32_t n_scales = 0;
    int32_t capacity = 0;   // tokens per item
    std::vector<int32_t> offset;  // [n_scales] token offset of each segment's home

    // Token-budget form (Algorithm 1 with Algorithm 2 as its roll, budgets counted in tokens).
    // The cached scales form one token stream; stream index g lives at position g while g < c_cds
    // (the pinned head) and at c_cds + (g - c_cds) mod (c_bgt - c_cds) otherwise, so the region
    // [0, c_bgt) is a pinned head followed by a ring whose newest tokens overwrite its oldest:
    // exactly "the first C_cds entries and the last C_bgt - C_cds entries".  A scale that is not
    // resident in full after its own append (larger than the budget, or larger than the ring once
    // the ring rolls) is also written to a transient slot behind the ring, from which its own
    // queries read it.
    bool token_mode = false;
    int32_t c_bgt = 0, c_cds = 0;
    int32_t c_promoted = 0;     // budget the layer may be promoted to (0: none)
    int32_t used = 0;           // positions [0, used) hold cached tokens; the transient slot starts at `used`
    std::vector<uint8_t> cached;      // [n_scales] scale enters the stream (its size fits the budget)
    std::vector<uint8_t> transient;   // [n_scales] scale is read from the transient slot at its own step
    std::vector<int64_t> stream_end;  // [n_scales] stream length after the scale

    // `linear`: the segments sit back to back in scale order whatever the class (the layout of a
    // cache-demanding layer), so that a cache-efficient layer can be promoted later without moving data: until
    // then it reads the pinned scales and the window out of that layout and reuses no slot.
    void build(const std::vector<int32_t>& tokens, int32_t n_condensed, int32_t n_local, bool demanding,
               bool transient_last = false, bool linear = false)
    {
        const int32_t K = (int32_t)tokens.size();
        n_scales = K;
        skip_last = transient_last;
        const int32_t stored = skip_last ? K - 1 : K;   // scales that get a home
        c = std::min(std::max(n_condensed, 0), K);
        w = std::min(std::max(n_local, 1), K);
        full = demanding || (c + w >= K);
        offset.assign(K, 0);
        if (full || linear) {
            int32_t at = 0;
            for (int32_t s = 0; s < stored; ++s) { offset[s] = at; at += tokens[s]; }
            capacity = skip_last ? std::max(at, kMinCapacity) : at;
            return;
        }
        std::vector<int32_t> slot_size(w, 0);
        for (int32_t s = c; s < stored; ++s) slot_size[(s - c) % w] = std::max(slot_size[(s - c) % w], tokens[s]);
        int32_t pinned = 0;
        for (int32_t s = 0; s < c; ++s) pinned += tokens[s];
        const int32_t pinned_at = slot_size[0];
        std::vector<int32_t> slot_at(w, 0);
        int32_t at = pinned_at + pinned;
        for (int32_t j = 1; j < w; ++j) { slot_at[j] = at; at += slot_size[j]; }
        capacity = skip_last ? std::max(at, kMinCapacity) : at;
        int32_t p = pinned_at;
        for (int32_t s = 0; s < c; ++s) { offset[s] = p; p += tokens[s]; }
        for (int32_t s = c; s < stored; ++s) {
            const int32_t j = (s - c) % w;
            offset[s] = (j == 0) ? (slot_size[0] - tokens[s]) : slot_at[j];
        }
    }

    // Token-budget form: `budget` = C_bgt (C_max for a cache-demanding layer, C_min otherwise) and
    // `condensed` = C_cds, both in tokens.  Starting a cache-demanding layer at C_max is the same as
    // promoting it at its first overflow, because nothing is evicted before that overflow.
    // `promoted_budget` > budget: the layer may later be given that budget (Algorithm 1's C_max); the region is
    // sized for whichever of the two layouts needs more.  Before the first overflow both layouts put stream
    // index g at position g, so switching budgets then moves no data.
    void build_tokens(const std::vector<int32_t>& tokens, int32_t budget, int32_t condensed, bool transient_last = false,
                      int32_t promoted_budget = 0)
    {
        build_tokens_one(tokens, budget, condensed, transient_last);
        c_promoted = 0;
        if (promoted_budget > budget) {
            LayerLayout alt;
            alt.build_tokens_one(tokens, promoted_budget, condensed, transient_last);
            capacity = std::max(capacity, alt.capacity);
            c_promoted = promoted_budget;
        }
    }

    void build_tokens_one(const std::vector<int32_t>& tokens, int32_t budget, int32_t condensed, bool transient_last)
    {
        const int32_t K = (int32_t)tokens.size();
        n_scales = K;
        skip_last = transient_last;
        token_mode = true;
        full = false;
        c = 0;
        w = 1;
        c_bgt = budget;
        c_cds = std::min(std::max(condensed, 0), budget);
        offset.assign(K, 0);
        cached.assign(K, 0);
        transient.assign(K, 0);
        stream_end.assign(K, 0);
        int64_t g = 0;
        int32_t slot = 0;
        for (int32_t s = 0; s < K; ++s) {
            const int32_t T = tokens[s];
            if (T <= c_bgt) {
                cached[s] = 1;
                const int64_t g0 = g;
                g += T;
                // the roll cuts into the scale itself when more of it lies behind the pinned head than the ring holds
                const int64_t behind_head = g - std::max<int64_t>(g0, c_cds);
                if (g > c_bgt && behind_head > c_bgt - c_cds) transient[s] = 1;
            } else {
                transient[s] = 1;  // never cached (Algorithm 1 skips it); attended from the transient slot
            }
            if (transient[s] && !(skip_last && s == K - 1)) slot = std::max(slot, T);
            stream_end[s] = g;
        }
        // (a last scale that is never stored takes no room: neither in the ring nor in the transient slot)
        const int64_t stored_stream = skip_last ? (K > 1 ? stream_end[K - 2] : 0) : g;
        used = (int32_t)std::min<int64_t>(stored_stream, c_bgt);
        capacity = skip_last ? std::max(used + slot, kMinCapacity) : used + slot;
    }

    // Scale whose append is the first to push the cache over its budget (Algorithm 1 takes the promotion
    // decision there); n_scales if the cache never overflows.
    int32_t first_overflow(const std::vector<int32_t>& tokens) const
    {
        if (!token_mode) return full ? n_scales : std::min(c + w, n_scales);
        const int32_t top = std::max(c_bgt, c_promoted);
        int64_t g = 0;
        for (int32_t s = 0; s < n_scales; ++s) {
            if (tokens[s] > top) continue;   // never cached under either budget: no overflow test
            if (g + tokens[s] > c_bgt) return s;
            g += tokens[s];
        }
        return n_scales;
    }

    // Promotion to the cache-demanding class; legal while nothing has been evicted (the caller checks).
    void promote(const std::vector<int32_t>& tokens)
    {
        if (!token_mode) {
            full = true;
            return;
        }
        const int32_t cap = capacity;
        build_tokens_one(tokens, c_promoted, c_cds, skip_last);
        capacity = std::max(capacity, cap);
        c_promoted = 0;
    }

    int32_t position(int64_t g) const
    {
        return g < c_cds ? (int32_t)g : c_cds + (int32_t)((g - c_cds) % (c_bgt - c_cds));
    }

    // first stream index of the surviving tail after scale k (the pinned head survives besides)
    int64_t tail_begin(int32_t k) const
    {
        const int64_t G = stream_end[k];
        return G > c_bgt ? std::max<int64_t>(G - (c_bgt - c_cds), c_cds) : 0;
    }

    // does the cache hold any token of segment s right after scale k was appended
    bool keeps(int32_t s, int32_t k) const
    {
        if (s > k) return false;
        if (skip_last && s == n_scales - 1) return false;   // attended at its own step, never held
        if (!token_mode) return full || s < c || s > k - w;
        if (!cached[s]) return false;
        const int64_t e = stream_end[s], b = s > 0 ? stream_end[s - 1] : 0;
        if (stream_end[k] <= c_bgt) return true;
        return b < c_cds || e > tail_begin(k);
    }

    // ascending segment ids resident right after scale k was appended
    int32_t kept(int32_t k, int32_t* ids) const
    {
        int32_t n = 0;
        for (int32_t s = 0; s <= k; ++s)
            if (keeps(s, k)) ids[n++] = s;
        return n;
    }

    // segments dropped by the append of scale k (a scale too large to be cached is reported at its own step)
    int32_t evicted(int32_t k, int32_t* ids) const
    {
        int32_t n = 0;
        for (int32_t s = 0; s <= k; ++s) {
            const bool before = (s == k) || keeps(s, k - 1);
            if (before && !keeps(s, k)) ids[n++] = s;
        }
        return n;
    }

    // the copies that append scale k; at most kMaxPieces
    static constexpr int kMaxPieces = 4;
    int32_t pieces(const std::vector<int32_t>& tokens, int32_t k, Piece* out) const
    {
        const int32_t T = tokens[k];
        if (skip_last && k == n_scales - 1) return 0;
        if (!token_mode) {
            out[0] = Piece{0, offset[k], T};
            return 1;
        }
        int32_t n = 0;
        auto push = [&](int32_t src, int32_t dst, int32_t len) {
            if (n > 0 && out[n - 1].src + out[n - 1].len == src && out[n - 1].dst + out[n - 1].len == dst) out[n - 1].len += len;
            else out[n++] = Piece{src, dst, len};
        };
        if (cached[k]) {
            const int64_t g1 = stream_end[k], g0 = g1 - T;
            if (g0 < c_cds) push(0, (int32_t)g0, (int32_t)(std::min<int64_t>(g1, c_cds) - g0));
            // behind the head only the tokens that survive the scale's own roll are written, so no two copies overlap
            int64_t g = std::max<int64_t>(std::max<int64_t>(g0, c_cds), tail_begin(k));
            while (g < g1) {
                const int32_t p = position(g);
                const int32_t run = (int32_t)std::min<int64_t>(g1 - g, c_bgt - p);
                push((int32_t)(g - g0), p, run);
                g += run;
            }
        }
        if (transient[k]) push(0, used, T);
        return n;
    }

    // token ranges read at scale k, sorted by position and merged where they touch
    int32_t ranges(const std::vector<int32_t>& tokens, int32_t k, Range* out) const
    {
        if (skip_last && k == n_scales - 1) return ranges_before(tokens, k, out);   // the scale itself is not in the cache
        if (token_mode) {
            int32_t n = 0;
            int32_t res = (int32_t)std::min<int64_t>(stream_end[k], c_bgt);
            // a scale cut by its own roll owns every resident token except the head that was there before it
            if (transient[k] && cached[k]) res = (int32_t)std::min<int64_t>(stream_end[k] - tokens[k], c_cds);
            if (res > 0) out[n++] = Range{0, res};
            if (transient[k]) {
                if (n > 0 && res == used) out[0].len += tokens[k];
                else out[n++] = Range{used, tokens[k]};
            }
            return n;
        }
        std::vector<Range> r;
        for (int32_t s = 0; s <= k; ++s)
            if (keeps(s, k)) r.push_back(Range{offset[s], tokens[s]});
        std::sort(r.begin(), r.end(), [](const Range& a, const Range& b) { return a.start < b.start; });
        int32_t n = 0;
        for (const Range& x : r) {
            if (n > 0 && out[n - 1].start + out[n - 1].len == x.start) out[n - 1].len += x.len;
            else out[n++] = x;
        }
        return n;
    }

    // which tokens of which segments the queries of scale k attend to (ascending segments; at most two
    // runs per segment: its part of the pinned head and its part of the tail)
    int32_t attended(const std::vector<int32_t>& tokens, int32_t k, TokenRun* out) const
    {
        int32_t n = 0;
        if (!token_mode) {
            for (int32_t s = 0; s <= k; ++s)
                if (s == k || keeps(s, k)) out[n++] = TokenRun{s, 0, tokens[s]};
            return n;
        }
        const bool rolled = stream_end[k] > c_bgt;
        const int64_t lo = tail_begin(k);
        for (int32_t s = 0; s <= k; ++s) {
            if (!cached[s] || (s == k && (transient[k] || (skip_last && k == n_scales - 1)))) continue;
            const int64_t e = stream_end[s], b = e - tokens[s];
            if (!rolled) {
                out[n++] = TokenRun{s, 0, tokens[s]};
                continue;
            }
            const int64_t head_end = std::min<int64_t>(e, c_cds);
            if (b < head_end) out[n++] = TokenRun{s, 0, (int32_t)(head_end - b)};
            const int64_t t0 = std::max<int64_t>(b, lo);
            if (t0 < e) {
                if (n > 0 && out[n - 1].segment == s && out[n - 1].first + out[n - 1].count == t0 - b) out[n - 1].count += (int32_t)(e - t0);
                else out[n++] = TokenRun{s, (int32_t)(t0 - b), (int32_t)(e - t0)};
            }
        }
        if (transient[k] || (skip_last && k == n_scales - 1)) out[n++] = TokenRun{k, 0, tokens[k]};
        return n;
    }

    // token ranges of the segments other than k that the queries of scale k attend to (sorted, merged):
    // what attention reads from the cache when scale k itself comes from the caller's tensors.  These
    // positions are not touched by the append of scale k, so they may be read while it is written.
    int32_t ranges_before(const std::vector<int32_t>& tokens, int32_t k, Range* out) const
    {
        TokenRun runs[2 * 32];
        const int32_t n_runs = attended(tokens, k, runs);
        std::vector<Range> r;
        for (int32_t i = 0; i < n_runs; ++i) {
            const int32_t s = runs[i].segment;
            if (s == k) continue;
            if (!token_mode) {
                r.push_back(Range{offset[s] + runs[i].first, runs[i].count});
                continue;
            }
            int64_t g = (s > 0 ? stream_end[s - 1] : 0) + runs[i].first;
            int32_t left = runs[i].count;
            while (left > 0) {
                const int32_t p = g < c_cds ? (int32_t)g : position(g);
                const int32_t run = std::min<int32_t>(left, (g < c_cds ? c_cds : c_bgt) - p);
                r.push_back(Range{p, run});
                g += run;
                left -= run;
            }
        }
        std::sort(r.begin(), r.end(), [](const Range& a, const Range& b) { return a.start < b.start; });
        int32_t n = 0;
        for (const Range& x : r) {
            if (n > 0 && out[n - 1].start + out[n - 1].len == x.start) out[n - 1].len += x.len;
            else out[n++] = x;
        }
        return n;
    }

    // Where the runs of attended(k) sit in the per-item region right after the append of scale k: pieces
    // (start, len) tagged with the index of their run; a run of a token-budget layer is two pieces where
    // the ring wraps inside it.  Returns the number of pieces, or -1 if a run has no place in the region
    // (a never-stored last scale) or `cap` is too small.
    struct RunPiece {
        int32_t start, len, run;
    };
    int32_t attended_pieces(const std::vector<int32_t>& tokens, int32_t k, RunPiece* out, int32_t cap) const
    {
        TokenRun runs[2 * 32];
        const int32_t n_runs = attended(tokens, k, runs);
        int32_t n = 0;
        for (int32_t i = 0; i < n_runs; ++i) {
            const int32_t s = runs[i].segment;
            if (skip_last && s == n_scales - 1) return -1;
            if (!token_mode || (s == k && transient[k])) {
                if (n >= cap) return -1;
                out[n++] = RunPiece{(token_mode ? used : offset[s]) + runs[i].first, runs[i].count, i};
                continue;
            }
            int64_t g = (s > 0 ? stream_end[s - 1] : 0) + runs[i].first;
            int32_t left = runs[i].count;
            while (left > 0) {
                const int32_t p = g < c_cds ? (int32_t)g : position(g);
                const int32_t run = std::min<int32_t>(left, (g < c_cds ? c_cds : c_bgt) - p);
                if (n >= cap) return -1;
                out[n++] = RunPiece{p, run, i};
                g += run;
                left -= run;
            }
        }
        return n;
    }

    int64_t resident_tokens(const std::vector<int32_t>& tokens, int32_t k) const
    {
        if (skip_last && k == n_scales - 1) {
            // what the step leaves in the cache: the older tokens its queries attended to
            TokenRun runs[2 * 32];
            const int32_t n_runs = attended(tokens, k, runs);
            int64_t t = 0;
            for (int32_t i = 0; i < n_runs; ++i)
                if (runs[i].segment != k) t += runs[i].count;
            return t;
        }
        if (token_mode) return std::min<int64_t>(stream_end[k], c_bgt);
        int64_t t = 0;
        for (int32_t s = 0; s <= k; ++s)
            if (keeps(s, k)) t += tokens[s];
        return t;
    }
};

}  // namespace amskv
