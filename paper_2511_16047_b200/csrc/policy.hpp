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

// Layout of one layer.  A cache-demanding layer (or one whose pinned prefix plus window
// already covers the whole schedule) stores its segments back to back in scale order.
// A cache-efficient layer has a pinned region for the condensed scales and n_local slots
// that the later scales rotate through: scale s >= c uses slot (s - c) mod w, so the segment
// that leaves the window (s - w) is the previous tenant of the slot the new segment takes and
// is evicted by being overwritten.  Slot 0 sits below the pinned region with its tenant
// right-aligned and slot 1 directly above the pinned region, which makes the resident
// tokens one contiguous run whenever w <= 2.
struct LayerLayout {
    int32_t c = 0;          // pinned scales (clamped to the schedule length)
    int32_t w = 1;          // window, in scales (clamped)
    bool full = false;      // nothing is ever evicted
    int32_t capacity = 0;   // tokens per item
    std::vector<int32_t> offset;  // [n_scales] token offset of each segment's home

    void build(const std::vector<int32_t>& tokens, int32_t n_condensed, int32_t n_local, bool demanding)
    {
        const int32_t K = (int32_t)tokens.size();
        c = std::min(std::max(n_condensed, 0), K);
        w = std::min(std::max(n_local, 1), K);
        full = demanding || (c + w >= K);
        offset.assign(K, 0);
        if (full) {
            int32_t at = 0;
            for (int32_t s = 0; s < K; ++s) { offset[s] = at; at += tokens[s]; }
            capacity = at;
            return;
        }
        std::vector<int32_t> slot_size(w, 0);
        for (int32_t s = c; s < K; ++s) slot_size[(s - c) % w] = std::max(slot_size[(s - c) % w], tokens[s]);
        int32_t pinned = 0;
        for (int32_t s = 0; s < c; ++s) pinned += tokens[s];
        const int32_t pinned_at = slot_size[0];
        std::vector<int32_t> slot_at(w, 0);
        int32_t at = pinned_at + pinned;
        for (int32_t j = 1; j < w; ++j) { slot_at[j] = at; at += slot_size[j]; }
        capacity = at;
        int32_t p = pinned_at;
        for (int32_t s = 0; s < c; ++s) { offset[s] = p; p += tokens[s]; }
        for (int32_t s = c; s < K; ++s) {
            const int32_t j = (s - c) % w;
            offset[s] = (j == 0) ? (slot_size[0] - tokens[s]) : slot_at[j];
        }
    }

    bool keeps(int32_t s, int32_t k) const { return s <= k && (full || s < c || s > k - w); }

    // ascending segment ids resident right after scale k was appended
    int32_t kept(int32_t k, int32_t* ids) const
    {
        int32_t n = 0;
        for (int32_t s = 0; s <= k; ++s)
            if (keeps(s, k)) ids[n++] = s;
        return n;
    }

    // segments dropped by the append of scale k
    int32_t evicted(int32_t k, int32_t* ids) const
    {
        int32_t n = 0;
        for (int32_t s = 0; s <= k; ++s) {
            const bool before = (s == k) || keeps(s, k - 1);
            if (before && !keeps(s, k)) ids[n++] = s;
        }
        return n;
    }

    // token ranges read at scale k, sorted by position and merged where they touch
    int32_t ranges(const std::vector<int32_t>& tokens, int32_t k, Range* out) const
    {
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

    int64_t resident_tokens(const std::vector<int32_t>& tokens, int32_t k) const
    {
        int64_t t = 0;
        for (int32_t s = 0; s <= k; ++s)
            if (keeps(s, k)) t += tokens[s];
        return t;
    }
};

}  // namespace amskv
