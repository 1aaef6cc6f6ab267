// Work decomposition shared by every phase of the attention kernel.
//
// Every (sequence b, KV head g) pair is a *segment* of tiles_b = ceil(keys_b / kTileKeys) tiles;
// segments are laid end to end on one line of n tiles in (b, g) order. CTA c of C owns the tile
// range [c*n/C, (c+1)*n/C). A consumer group emits one partial result per segment it enters; a
// segment's partials live in its own run of slots (handed out by an atomic counter in the order of
// entry). Everything is computed from the device-resident lengths in O(B) per CTA; nothing is O(S)
// and nothing comes from the host.
#pragma once

#include "wmtp_internal.h"

namespace wmtp {

// Ring slot of logical position p (Appendix A, RING): the sink is fixed, the window region circular.
__device__ __forceinline__ int ring_slot(int64_t p, int n_sink, int cap) {
    if (p < n_sink) return (int)p;
    const int64_t w = p - n_sink;
    // 64-bit division is a long dependent instruction chain on the GPU: take the 32-bit path when it is exact
    return n_sink + (w < 0x7fffffffLL ? (int)((uint32_t)w % (uint32_t)cap) : (int)(w % cap));
}

// Does this launch append a token to sequence b before attending (fused draft step)? (Only with one query per sequence.)
__device__ __forceinline__ bool appends_to(const AttnParams& p, int b) {
    return p.k_new != nullptr && (p.mode == kRing || p.len[b] < p.S_cap);
}

// The batch index b of the kernel counts *queries*: with q_len queries per sequence (draft-extend: the last q_len
// tokens of a sequence re-processed in one launch, each attending causally up to itself), query b belongs to
// sequence b / q_len and is its (b % q_len)-th new token.
__device__ __forceinline__ int kv_seq(const AttnParams& p, int b) { return p.q_len > 1 ? b / p.q_len : b; }

// Sequence length the attention of query b sees: the stored length, plus the token appended by this launch; for
// draft-extend, the length at which that query's own token was the newest.
__device__ __forceinline__ int64_t eff_len(const AttnParams& p, int b) {
    if (p.q_len > 1) {
        const int64_t S = p.len[b / p.q_len] - (p.q_len - 1 - b % p.q_len);
        return S > 0 ? S : 0;
    }
    return p.len[b] + (appends_to(p, b) ? 1 : 0);
}

// Key slots the kernel scans for sequence b: the live part of the ring, or all S positions.
__device__ __forceinline__ int64_t scan_keys(const AttnParams& p, int b) {
    const int64_t S = eff_len(p, b);
    if (p.mode == kRing) {
        const int64_t slots = (int64_t)p.n_sink + p.cap;
        return S < slots ? S : slots;
    }
    return S;
}

// How the tiles of one sequence map onto its K/V rows. A sequence contributes `tiles` tiles per KV head: first
// `sink_tiles` tiles covering rows [0, ns) (source tile j = j), then tiles covering rows [lo, S) (source tile
// win_first + j - sink_tiles). Without a window view everything is the first kind: ns = keys scanned, no second part.
// With a window view (the paper's own mechanism, Section 4: the draft's block table is reduced to the sink blocks and
// the blocks of the last W tokens) the rows are those of the full KV store and ns = min(S, n_sink),
// lo = max(ns, S - W); a 64-row tile that straddles lo, ns or S is masked row by row, so the ends are token-granular
// whatever the page size.
struct SeqView {
    int64_t S, nk, ns, lo, sink_tiles, win_first, tiles;
};
__device__ __forceinline__ SeqView seq_view(const AttnParams& p, int b) {
    SeqView v;
    v.S = eff_len(p, b);
    v.nk = scan_keys(p, b);
    if (!p.window_view) {
        v.ns = v.nk; v.lo = v.nk;
        v.sink_tiles = (v.nk + kTileKeys - 1) / kTileKeys;
        v.win_first = 0;
        v.tiles = v.sink_tiles;
    } else {
        v.ns = v.S < p.n_sink ? v.S : p.n_sink;
        v.lo = v.S - p.W > v.ns ? v.S - p.W : v.ns;
        v.sink_tiles = (v.ns + kTileKeys - 1) / kTileKeys;
        v.win_first = v.lo / kTileKeys;
        v.tiles = v.sink_tiles + (v.S > v.ns ? (v.S - 1) / kTileKeys - v.win_first + 1 : 0);
    }
    return v;
}

// Is ring slot s (< scan_keys) inside sink + last-W? Always true when cap == W.
__device__ __forceinline__ bool ring_slot_live(int s, int64_t S, int n_sink, int W, int cap) {
    if (s < n_sink) return true;
    const int64_t last = S - 1 - n_sink;
    const int cur = last < 0x7fffffffLL ? (int)((uint32_t)last % (uint32_t)cap) : (int)(last % cap);
    int age = cur - (s - n_sink);
    if (age < 0) age += cap;
    return age < W;
}

// CTAs that take part: never more than there are tiles, so every participating CTA owns >= 1 tile.
__device__ __forceinline__ int effective_ctas(int launched, int64_t n) {
    return n < (int64_t)launched ? (int)n : launched;
}

// (Tile counts below 2^23 keep c * n and (t + 1) * C inside 32 bits for C <= kMaxCtas; 64-bit division
// costs hundreds of dependent cycles on one thread, which the short windowed launches would feel.)
__device__ __forceinline__ int64_t cta_range_start(int c, int64_t n, int C) {
    if (n < (1 << 23)) return (int64_t)(((uint32_t)c * (uint32_t)n) / (uint32_t)C);
    return ((int64_t)c * n) / C;   // c <= kMaxCtas and n < 2^40: no overflow
}

// In-place inclusive running sum of a[0 .. n) in shared memory by one warp: every lane sums a contiguous chunk, the
// lanes' totals are scanned with shuffles, the offsets are added back. n <= kMaxBatch: at most 32 elements per lane.
template <typename T>
__device__ __forceinline__ void warp_inclusive_scan(T* a, int n) {
    const int lane = threadIdx.x & 31;
    const int per = (n + 31) >> 5, lo = lane * per, hi = lo + per < n ? lo + per : n;
    T sum = 0;
    for (int i = lo; i < hi; ++i) { sum += a[i]; a[i] = sum; }
    T incl = sum;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const T up = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += up;
    }
    const T before = incl - sum;
    for (int i = lo; i < hi; ++i) a[i] += before;
}

// Sequence whose segment group contains global tile t (Hkv segments per sequence).
__device__ __forceinline__ int find_seq(const int64_t* tile_prefix, int B, int Hkv, int64_t t) {
    int lo = 0, hi = B - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if ((int64_t)Hkv * tile_prefix[mid] <= t) lo = mid; else hi = mid - 1;
    }
    return lo;
}

}  // namespace wmtp
