// Split-KV decode attention for the draft head: one TMA-fed kernel per draft step that appends the
// step's K/V, computes split-KV partials and merges them by log-sum-exp.
//
// The operation is softmax attention of one query per head over a key set (Section 4
// "Mechanism"; Appendix D: o = sum_j p_j v_j): the ring's live slots for the windowed draft,
// all S positions for the full-context (native) draft of Section 3. The work is bound by the
// HBM read of K and V, so the kernel is organised around keeping bytes in flight:
//
//   * at most one persistent CTA per SM (the launcher takes seven eighths of the SMs for long bf16 streams:
//     the memory system delivers more to fewer requesters); the tile line (attn_plan.cuh) is split into one
//     contiguous range per CTA, and the tail of every range can be taken over by CTAs that finish early
//     (SMs do not all stream at the same rate);
//   * a producer warp streams K and V tiles into a ring of shared-memory stages with TMA
//     (cp.async.bulk.tensor, 128-byte swizzle, completion on mbarriers) and tells the consumers
//     which tile each stage holds;
//   * consumer groups of four warps take whole tiles in turn (one group when a stage holds 64 KB, two
//     when it holds less -- head_dim 128 or an fp8 store -- where a tile carries fewer bytes for the same
//     softmax work, and the producer's warpgroup then hands registers to the consumers'); each warp of a
//     group takes 16 keys of the tile. Scores are computed as S^T[key, head] = K[key, :] . Q^T (keys on the
//     MMA M dimension, the G <= 8 query heads of the GQA group exactly on N = 8), the online softmax runs
//     in fp32, and O^T[d, head] += V^T[d, key] . P^T[key, head] accumulates in registers. The 8-row problem
//     is far too small for tcgen05 (M >= 64); mma.sync.m16n8k16 needs a few percent of tensor peak here.
//     The codes of an fp8 store are widened to f16 after ldmatrix and take the f16 MMA. The smallest tiles (8 KB:
//     head_dim 128, fp8) are streamed and consumed two at a time -- a stage holds two consecutive tiles of a segment and
//     a warp works on its 16 keys of both, one softmax update over the 32 keys;
//   * every K/V byte is read once from HBM and once from shared memory, shared by all heads
//     of the group;
//   * long launches (the full-context draft) are cooperative (all CTAs co-resident): after publishing its partial a
//     group waits, with a bounded spin, for the other contributors of its segment and reduces its slice of the output,
//     so the merge needs no second launch and no single CTA serialises it; short launches (the windowed draft: a few
//     thousand keys per sequence, out of L2) run as one thread-block cluster per segment and merge through distributed
//     shared memory instead (see the kernel's two forms below);
//   * a draft step's append (Appendix A, RING; the KV write of a draft forward) is fused: the warp
//     that owns the new token's row patches the tile in shared memory from k_new / v_new and stores
//     the row to the KV store; the group that completes the launch's last segment advances len[].
#include <cuda.h>
#include <cuda_bf16.h>

#include <mutex>
#include <type_traits>

#include "attn_plan.cuh"
#include "fp8_util.cuh"
#include "ptx_util.cuh"

namespace wmtp {

namespace {

constexpr float kLn2 = 0.6931471805599453f;
constexpr int kGroupWarps = 4;                  // warps per consumer group: 4 x 16 keys = one tile
constexpr int kGroupThreads = kGroupWarps * 32;
constexpr int kMaxParts = kMaxGroups * kMaxCtas; // partials one segment can receive
// Per-group scratch, used for two things in turn:
//   the warp merge of a flush: [4 warps][8 heads][pass columns + 4] floats, `pass columns` of d at a time;
//   the combine: weights [heads of this contributor's slice][np], inverses [8], a reduction buffer [128] float4 and the
//   visiting order [np] (16-bit entries). A contributor's slice of the (head, d) columns spans at most two heads once there are at least
//   G contributors, and fewer than G * G (head, partial) pairs otherwise: 2 * kMaxParts weights always suffice.
constexpr int kCombineWeights = 2 * kMaxParts;
constexpr int kCombineFloats = kCombineWeights + 8 + 4 * kGroupThreads + kMaxParts / 2;
static_assert(kMaxParts < 65536 && kMaxParts % 2 == 0, "visiting order held in 16-bit entries");
static_assert(kMaxGroup * kMaxGroup <= kCombineWeights, "weights of a slice must fit");
constexpr int kMaxContrib = 32;     // segments a group may have outstanding before it combines them
constexpr int kStealChunkBytes = 262144;        // bytes of K/V handed out per cursor step
// per-group bookkeeping in shared memory (ints): [0] launch-last flag, [1] broadcast word, then
// contrib[kMaxContrib][4] = {seg, b, g, slot}, reg_k[kMaxContrib] (slot of the group's i-th contribution, producer -> group)
constexpr int kGroupInts = 4 + 5 * kMaxContrib;

// D: head_dim; F8: the store holds e4m3 codes (one byte per entry) instead of bf16; CL: the cluster form of the kernel;
// ONE (cluster form only): one consumer group whatever the tile size -- for launches that leave a CTA a handful of tiles.
template <int D, bool F8, bool CL = false, bool ONE = false>
struct Cfg {
    static_assert(CL || !ONE, "the one-group variant exists in the cluster form only");
    static constexpr int kElemBytes = F8 ? 1 : 2;
    static constexpr int kChunks = D * kElemBytes / 128;      // 128-byte column chunks per row
    static constexpr int kChunkBytes = kTileKeys * 128;       // one TMA box: 64 rows x 128 B
    static constexpr int kTileBytes = kChunks * kChunkBytes;  // K (or V) tile
    // Tiles per stage. The smallest tiles (8 KB: head_dim 128, fp8) travel and are consumed in pairs of consecutive tiles
    // of a segment in the streaming form: a warp then works on two independent 16-key slabs at once (its dependent
    // chain per tile, not any unit of the SM, limits the rate), and the producer's per-stage work is halved.
    static constexpr int kPair = (F8 && D == 128 && !CL) ? 2 : 1;
    static constexpr int kStageBytes = kPair * 2 * kTileBytes;
    // consumer groups: a tile of fewer bytes brings the same softmax work, so the smaller tiles get two groups
    static constexpr int kGroups = ((D == 256 && !F8) || ONE) ? 1 : 2;
    // Stages of the shared-memory ring. What counts for the streaming rate is the bytes a CTA keeps in flight (about
    // 190 KB per SM saturate HBM at the loaded latency of ~4 us): the host takes as many stages as fit beside the
    // batch-dependent tables, up to kMaxStages, in multiples of the group count (a stage then always serves one group).
    static constexpr int kMaxStages = (kStageBytes >= 65536) ? 3 : (kStageBytes >= 32768 ? 6 : 12);
    // Tiles handed out per cursor step. A step costs a global atomic (about 1.5 us) that is fetched one chunk ahead: the
    // chunk must take longer than that to stream, so it is sized in bytes (256 KB), not in tiles.
    static constexpr int kStealChunk = kStealChunkBytes / (2 * kTileBytes);
    static_assert(kStealChunk % kPair == 0, "a cursor step hands out whole stages");
    static constexpr int kStealMinTiles = 8 * kStealChunk;   // ranges shorter than this are streamed statically
    // columns of d merged per pass of a flush: the two-group configurations trade a second pass for shared memory
    // (A group of a cluster-form CTA is done with its own stages when it flushes: the warp merge then runs in the group's
    // first stage, all of d in one pass with one group, 128 columns at a time with two; 16 KB stages are too small.)
    static constexpr bool kFlushInStages = CL && (kGroups == 1 || kStageBytes >= 32768);
    static constexpr int kPassCols = kFlushInStages ? (kGroups == 1 ? D : 128) : ((kGroups == 2) ? 64 : 128);
    static constexpr int kScratchRow = kPassCols + 4;
    static constexpr int kMergeFloats = kFlushInStages ? 0 : kGroupWarps * kMaxGroup * kScratchRow;
    static_assert(!kFlushInStages || kGroupWarps * kMaxGroup * kScratchRow * 4 <= kStageBytes, "the warp merge fits one stage");
    static constexpr int kScratchFloats = kMergeFloats > kCombineFloats ? kMergeFloats : kCombineFloats;
    // With two groups the CTA has 9 warps and a thread at most 168 registers: the query fragments (the same in all four
    // warps of a group) then live in shared memory, one copy per group, instead of D / 8 registers per thread.
    static constexpr bool kQShared = (kGroups >= 2);
    static constexpr int kQBytes = kQShared ? kGroups * (D / 16) * 32 * 8 : 0;
    static constexpr int kConsumerWarps = kGroups * kGroupWarps;
    // With two consumer groups the CTA would have 9 warps and every thread at most 168 registers (three warps share
    // one scheduler's register file); the consumers want more and the producer needs about 56. So after the common
    // prologue the producer's warpgroup hands registers to the consumers' warpgroups (setmaxnreg). The instruction is
    // warpgroup-wide: the producer's warpgroup is filled up with three warps that execute it and exit.
    static constexpr bool kRebalance = (kGroups >= 2);
    static constexpr int kPadWarps = kRebalance ? 3 : 0;
    static constexpr int kThreads = (kConsumerWarps + 1 + kPadWarps) * 32;
    static constexpr int kRegsProducer = 56, kRegsConsumer = 224;
    // the 8 consumer warps and the 4 warps of the producer's warpgroup share what the 12 warps were launched with
    static_assert(!kRebalance || (kGroups == 2 && 8 * kRegsConsumer + 4 * kRegsProducer <= 12 * 168), "register trade must balance");
    static constexpr int kKSteps = D / 16;
    static constexpr int kBarriers = (1 + 2 * kGroups) * kMaxStages;
    // bytes of the fixed-size part of shared memory (scratch, softmax statistics, query fragments, barriers, stage tags,
    // contribution lists, per-group words, flags), rounded up to the stage ring's alignment
    static constexpr int kFixedRaw = 4 * kGroups * (kScratchFloats + 3 * kGroupWarps * kMaxGroup) + kQBytes + 8 * kBarriers +
                                     8 * kMaxStages + 8 * kGroups * 2 * kMaxContrib + 4 * kGroups * kGroupInts + 16;
    static constexpr int kFixedBytes = (kFixedRaw + 1023) / 1024 * 1024;
    static_assert(kMaxStages % kGroups == 0, "a stage must always serve the same group");
    static_assert(kGroups <= kMaxGroups, "partial slots are reserved for kMaxGroups groups per CTA");
};

// Bounded spin on a global word written by other CTAs of this (cooperative) launch: waits until
// (value - base) >= target in wrap-around arithmetic.
__device__ __forceinline__ uint32_t wait_word(const void* word, uint32_t base, uint32_t target, uint32_t limit, volatile int* abort_flag,
                                              int* status) {
    uint32_t v = 0;
    for (uint32_t i = 0; i < limit; ++i) {
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(word) : "memory");
        if (v - base >= target) return v;
        if ((i & 255u) == 255u && *abort_flag) return v;
        __nanosleep(32);
    }
    if (*abort_flag == 0) *abort_flag = kAbortWord;
    atomicCAS(status, 0, kErrTimeout);
    return v;
}

// Bounded spin on a segment's arrival word until its tile count (low half) reaches `tiles`; returns the number of
// published partials (high half).
__device__ __forceinline__ int wait_tiles(const unsigned long long* word, uint32_t tiles, uint32_t limit, volatile int* abort_flag, int* status) {
    unsigned long long v = 0;
    for (uint32_t i = 0; i < limit; ++i) {
        asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(word) : "memory");
        if ((uint32_t)v >= tiles) return (int)(v >> 32);
        if ((i & 255u) == 255u && *abort_flag) return 0;
        __nanosleep(32);
    }
    if (*abort_flag == 0) *abort_flag = kAbortWord;
    atomicCAS(status, 0, kErrTimeout);
    return 0;
}
__device__ __forceinline__ int kMaxSegmentsPadded(const AttnParams& p) { return p.seg_stride; }

// One (sequence, KV head) segment as seen by a CTA.
struct Segment {
    int b, g, seg;
    // Tile indices and row counts fit 32 bits: the K/V tensors are limited to 2^31 - 1 rows (TMA coordinates), so the
    // tile line has fewer than 2^25 tiles. Only the logical length of a ring can be larger.
    int seg_start, tiles, nk;
    int ns, lo, hi, sink_tiles, win_first;   // tile -> row mapping of the sequence (SeqView); hi = rows end of the second part
    int slot_base;              // first partial slot of the segment
    int64_t S;
    int cap;                    // partial slots the segment has
};
__device__ __forceinline__ Segment locate_segment(const AttnParams& p, const int64_t* tile_prefix, const int* cap_prefix, int64_t t) {
    Segment s;
    s.b = find_seq(tile_prefix, p.B, p.Hkv, t);
    s.tiles = (int)(tile_prefix[s.b + 1] - tile_prefix[s.b]);
    const int seq_start = p.Hkv * (int)tile_prefix[s.b];
    const int in_seq = (int)t - seq_start;
    s.g = (int)((uint32_t)in_seq / (uint32_t)s.tiles);
    s.seg_start = seq_start + s.g * s.tiles;
    const SeqView v = seq_view(p, s.b);
    s.S = v.S; s.nk = (int)v.nk; s.ns = (int)v.ns; s.lo = (int)v.lo; s.sink_tiles = (int)v.sink_tiles; s.win_first = (int)v.win_first;
    s.hi = (int)(v.S < 0x7fffffffLL ? v.S : 0x7fffffffLL);
    s.seg = s.b * p.Hkv + s.g;
    s.cap = cap_prefix[s.b + 1] - cap_prefix[s.b];
    s.slot_base = p.Hkv * cap_prefix[s.b] + s.g * s.cap;
    return s;
}

// The segment (b, g) by itself, tiles numbered from 0 (cluster launches: one cluster per segment, no tile line).
__device__ __forceinline__ Segment make_segment(const AttnParams& p, int b, int g) {
    Segment s;
    s.b = b; s.g = g; s.seg = b * p.Hkv + g;
    const SeqView v = seq_view(p, b);
    s.seg_start = 0; s.tiles = (int)v.tiles;
    s.S = v.S; s.nk = (int)v.nk; s.ns = (int)v.ns; s.lo = (int)v.lo; s.sink_tiles = (int)v.sink_tiles; s.win_first = (int)v.win_first;
    s.hi = (int)(v.S < 0x7fffffffLL ? v.S : 0x7fffffffLL);
    s.cap = 0; s.slot_base = 0;
    return s;
}
// Barrier over all threads of the cluster that have not exited: what was written to shared memory before it is visible
// to the other CTAs' distributed-shared-memory reads after it.
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Element offset of row `key` of (b, g) in the K / V tensor; *ok = false on a bad page id.
__device__ __forceinline__ int64_t kv_row_offset(const AttnParams& p, int b, int g, int64_t key, bool* ok) {
    if (p.mode == kPaged) {
        const int page = p.page_table[(int64_t)b * p.max_pages + key / p.page_size];
        if (page < 0 || page >= p.num_pages) { *ok = false; return 0; }
        return (((int64_t)page * p.Hkv + g) * p.page_size + key % p.page_size) * p.D;
    }
    return (((int64_t)b * p.Hkv + g) * p.rows_per_head + key) * p.D;
}

// ---------------------------------------------------------------------------------------------
// Distributed combine of one segment (split-KV algebra): lse = logsumexp_s(lse_s),
// out = sum_s exp(lse_s - lse) * o_s. Called by the 128 threads of every consumer group that contributed
// a partial to the segment. Contributor number j of the np contributors reduces the j-th slice of the
// (head, d) columns, so the merge is spread over all SMs that worked on the segment.
// With the fixed partition the partials are visited in the order of their keys (CTA, group), which makes
// the result independent of the order in which the slots were handed out: bit-reproducible.
// ---------------------------------------------------------------------------------------------
__device__ __noinline__ void combine_segment(const AttnParams& p, int b, int g, int64_t pbase, int np, int j, float* scratch,
                                             int tid, int grp) {
    const int G = p.G, D = p.D;
    float* w_sm = scratch;                                                  // [heads of the slice][np]
    float* inv_sm = scratch + kCombineWeights;                              // [8], indexed by head - first head of the slice
    float4* red = reinterpret_cast<float4*>(inv_sm + 8);                    // [128]
    uint16_t* perm = reinterpret_cast<uint16_t*>(inv_sm + 8 + 4 * kGroupThreads);   // [np] visiting order

    // ---- visiting order: the fixed partition ranks the partials by their keys; with stealing on they are taken as stored
    const bool ranked = !p.steal_slots_enabled;
    if (ranked) {
        int* keys = reinterpret_cast<int*>(red);                            // borrowed until the barrier below
        for (int i = tid; i < np; i += kGroupThreads) keys[i] = __ldcg(p.part_key + pbase + i);
        group_barrier(grp);
        for (int i = tid; i < np; i += kGroupThreads) {
            const int ki = keys[i];
            int r = 0;
            for (int q = 0; q < np; ++q) r += keys[q] < ki;
            perm[r] = (uint16_t)i;
        }
        group_barrier(grp);
    }
    auto part = [&](int i) { return ranked ? (int)perm[i] : i; };

    // ---- this group's slice of the (head, d) columns; the first rows are requested before the weights exist
    constexpr int kPre = 6;
    const int vec = D / 4, cols = G * vec;
    // columns per contributor: the smallest power of two that covers all columns (this runs once per launch on the
    // critical path of the tail: shifts and masks instead of integer divisions)
    int csh = 0;
    while ((np << csh) < cols) ++csh;
    const int cpc = 1 << csh;
    const int bsh = csh < 7 ? csh : 7, cb = 1 << bsh;                       // columns handled per pass: min(cpc, 128)
    const int R = kGroupThreads >> bsh, cl = tid & (cb - 1), rg = tid >> bsh;   // R rows of partials in flight per column
    const int col_lo = j * cpc, col_hi = col_lo + cpc < cols ? col_lo + cpc : cols;
    const int vsh = D == 256 ? 6 : 5;                                       // vec = D / 4 is a power of two: log2(vec)
    const int h_lo = col_lo < cols ? col_lo >> vsh : 0;                     // heads the slice touches: [h_lo, h_lo + nh)
    const int nh = col_lo < col_hi ? ((col_hi - 1) >> vsh) - h_lo + 1 : 0;
    const float4* rows = reinterpret_cast<const float4*>(p.part_o);
    float4 pre[kPre];
#pragma unroll
    for (int u = 0; u < kPre; ++u) {
        const int i = rg + u * R;
        pre[u] = (col_lo + cl < col_hi && i < np) ? __ldcg(rows + (pbase + part(i)) * cols + col_lo + cl) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    // ---- weights of the slice's heads, all at once: 16 threads per head, the partial lse values taken 128 at a time
    //      with a running maximum (weights already stored are rescaled when it moves; one chunk is the common case).
    //      The contributor whose slice holds a head's first column also writes the head's lse.
    {
        const int hh = tid >> 4, h = h_lo + hh, li = tid & 15;
        const bool act = hh < nh;
        constexpr int kPer = 8;
        float M = -INFINITY, sum = 0.f;
        for (int c0 = 0; c0 < np; c0 += 16 * kPer) {
            float x[kPer];
            float mc = -INFINITY;
#pragma unroll
            for (int u = 0; u < kPer; ++u) {
                const int i = c0 + li + 16 * u;
                x[u] = (act && i < np) ? __ldcg(p.part_lse + (pbase + part(i)) * G + h) : -INFINITY;
                mc = fmaxf(mc, x[u]);
            }
#pragma unroll
            for (int off = 8; off > 0; off >>= 1) mc = fmaxf(mc, __shfl_xor_sync(0xffffffffu, mc, off));
                    if (mc > M) {
                if (c0 > 0 && act) {
                    const float r = __expf(M - mc);                    // 0 when nothing finite was seen before
                    for (int i = li; i < c0; i += 16) w_sm[hh * np + i] *= r;
                    sum *= r;
                }
                M = mc;
            }
#pragma unroll
            for (int u = 0; u < kPer; ++u) {
                const int i = c0 + li + 16 * u;
                if (act && i < np) {
                    const float w = (M > -INFINITY) ? __expf(x[u] - M) : 0.f;
                    w_sm[hh * np + i] = w;
                    sum += w;
                }
            }
        }
#pragma unroll
        for (int off = 8; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
            if (li == 0 && act) {
            inv_sm[hh] = sum > 0.f ? 1.f / sum : 0.f;
            if (p.lse && col_lo <= (h << vsh)) p.lse[(int64_t)b * p.Hq + g * G + h] = sum > 0.f ? M + __logf(sum) : -INFINITY;
        }
    }
    group_barrier(grp);
    __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.out) + ((int64_t)b * p.Hq + g * G) * D;
    for (int c0 = col_lo; c0 < col_hi; c0 += kGroupThreads) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c0 + cl < col_hi) {
            const int col = c0 + cl, h = (col >> vsh) - h_lo;
            int i = rg;
            if (c0 == col_lo) {
#pragma unroll
                for (int u = 0; u < kPre; ++u, i += R) {
                    if (i < np) {
                        const float w = w_sm[h * np + i];
                        acc.x = fmaf(w, pre[u].x, acc.x); acc.y = fmaf(w, pre[u].y, acc.y);
                        acc.z = fmaf(w, pre[u].z, acc.z); acc.w = fmaf(w, pre[u].w, acc.w);
                    }
                }
            }
#pragma unroll 4
            for (; i < np; i += R) {
                const float w = w_sm[h * np + i];
                const float4 x = __ldcg(rows + (pbase + part(i)) * cols + col);
                acc.x = fmaf(w, x.x, acc.x); acc.y = fmaf(w, x.y, acc.y); acc.z = fmaf(w, x.z, acc.z); acc.w = fmaf(w, x.w, acc.w);
            }
        }
        red[tid] = acc;
        group_barrier(grp);
        if (tid < cb && c0 + tid < col_hi) {
            float4 o = red[tid];
            for (int r = 1; r < R; ++r) {
                const float4 x = red[r * cb + tid];
                o.x += x.x; o.y += x.y; o.z += x.z; o.w += x.w;
            }
            const int col = c0 + tid;
            const float inv = inv_sm[(col >> vsh) - h_lo];
            uint2 packed;
            packed.x = pack_bf16x2(o.x * inv, o.y * inv);
            packed.y = pack_bf16x2(o.z * inv, o.w * inv);
            *reinterpret_cast<uint2*>(out + (int64_t)col * 4) = packed;
        }
        group_barrier(grp);
    }
}

// Fused append, one tensor (K or V): the row TMA brought for the new token's slot may be stale, so the warp that owns
// it takes the row from the step's input (quantised for an fp8 store), writes it into the landed tile in shared memory
// (`tile`: shared-memory address of the K or V tile, 128-byte swizzle) and into the store (`dst_row`, or nullptr when
// the row has no valid place there). Kept out of line: it runs once per launch and sequence, and inside the tile loop
// its code (the fp8 quantiser above all) would sit in the middle of every iteration's instruction stream.
template <int D, bool F8>
__device__ __noinline__ void patch_new_row(const void* new_rows, int64_t row_index, const float* scale, int g, uint32_t tile,
                                           int new_row, void* dst_row, int lane) {
    using C = Cfg<D, F8>;
    constexpr int kRowVecs = D * C::kElemBytes / 16;        // 16-byte vectors per stored row
    if (lane >= kRowVecs) return;
    const uint4* src = reinterpret_cast<const uint4*>(new_rows) + row_index * (D / 8);
    uint4 x;
    if constexpr (F8) x = quant16_e4m3(__ldg(src + 2 * lane), __ldg(src + 2 * lane + 1), __ldg(scale + g));
    else x = __ldg(src + lane);
    const uint32_t addr = tile + (lane >> 3) * C::kChunkBytes + new_row * 128 + (((lane & 7) ^ (new_row & 7)) << 4);
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(x.x), "r"(x.y), "r"(x.z), "r"(x.w) : "memory");
    if (dst_row) reinterpret_cast<uint4*>(dst_row)[lane] = x;
}

// Launch-level bookkeeping (workspace header and per-segment words), with no reset pass and no grid barrier.
// The per-segment words exist twice; a launch uses the copy selected by the parity of the launch epoch and,
// at its very end, clears the other copy for the next launch (nobody can be using that one).
//   cur[c]       tiles of CTA c's dynamic part already handed out (to the owner or to thieves);
//   nparts[s]    partial slots handed out for segment s (a consumer group takes one whenever it enters s);
//   nthief[s]    CTAs admitted into s from another segment;
//   arrive[s]    64 bits: (published partials << 32) | tiles covered by them. Contributors add to it after their
//                partial is visible and then poll it: when the tile count equals the segment's tiles, the high
//                half is the number of partials to combine. One hop, no "ready" flag;
//   segs_done    completed segments; the group that completes the last one advances the epoch and, after every
//                CTA has stopped taking tiles (grab_done, which also means it has read len[] for the last
//                time), resets the cursors, clears the other copy and advances the lengths of a fused append;
//   dirty[2]     (header) segments whose words each copy may hold non-zero: launches on one workspace may differ in
//                their segment count (a draft-extend between decode steps), so the other copy is cleared over the
//                count of the launch that used it last, not over this launch's.

// ---------------------------------------------------------------------------------------------
// The attention kernel (one launch per draft step), in two forms.
//   CL = false: the cooperative launch described above -- one tile line over all segments, work stealing, partials in the
//     workspace, distributed combine. Made for long streams, where its fixed cost (about 13 us of plan, flush, arrival
//     and combine round trips through L2) does not matter.
//   CL = true: a thread-block cluster per segment, for launches whose segments are short (the windowed draft: a ring
//     or a window view of a few thousand keys per sequence). CTA r of the cluster's n takes tiles [r T / n, (r + 1) T / n)
//     of its segment; every consumer group leaves its partial in its own shared memory, and after one cluster barrier
//     CTA r reduces the r-th slice of the output columns over all partials of the cluster through distributed shared
//     memory (log-sum-exp weights from the partials' lse values). No workspace traffic, no atomics, no polling; the
//     launch is an ordinary one (no CTA waits for another cluster), and the cluster that finishes last -- a ticket in
//     the workspace header -- advances the lengths of a fused append. Tile processing is the same code in both forms.
// ---------------------------------------------------------------------------------------------
template <int D, bool F8, bool ONE, bool CL>
__global__ void __launch_bounds__(Cfg<D, F8, CL, ONE>::kThreads, 1)
attn_fused_tma(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV,
               const __grid_constant__ AttnParams p) {
    using C = Cfg<D, F8, CL, ONE>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    // Shared memory: the fixed-size part first (compile-time offsets), then the stage ring (1024-byte aligned for the
    // 128-byte swizzle, as many stages as the launcher found room for), then the batch-sized tables.
    float* scratch_all = reinterpret_cast<float*>(smem);                                  // [kGroups][kScratchFloats]
    float* sm_stats = scratch_all + C::kGroups * C::kScratchFloats;                       // [kGroups][3][4][8]: m, l, le per warp and head
    uint2* q_sm_all = reinterpret_cast<uint2*>(sm_stats + C::kGroups * 3 * kGroupWarps * kMaxGroup);   // [kGroups][kKSteps][32] (kQShared)
    // Barriers: empty[stage] (the producer observes every use of a stage) and, per consumer group, fullK / fullV[stage].
    // A group only sees the uses of a stage that are its own, and a parity wait can only tell consecutive phases
    // apart, so the "full" barriers must not be shared between groups.
    uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<unsigned char*>(q_sm_all) + C::kQBytes);
    int64_t* stage_tile = reinterpret_cast<int64_t*>(bars + C::kBarriers);                // [kMaxStages] global tile index, -1 = end
    int64_t* contrib_base_all = stage_tile + C::kMaxStages;                               // [kGroups][2][kMaxContrib]
    int* group_ints = reinterpret_cast<int*>(contrib_base_all + C::kGroups * 2 * kMaxContrib);   // [kGroups][kGroupInts]
    int* cta_flags = group_ints + C::kGroups * kGroupInts;                                // [0] abort
    unsigned char* stages = smem + C::kFixedBytes;                                        // nst x (K tile, V tile)
    const uint32_t nst = (uint32_t)p.stages;                                              // stages in use (<= kMaxStages)
    int64_t* tile_prefix = reinterpret_cast<int64_t*>(stages + nst * C::kStageBytes);     // [B + 1]       (CL = false)
    int* cap_prefix = reinterpret_cast<int*>(tile_prefix + (p.B + 1));                    // [B + 1]
    float* part_sm = reinterpret_cast<float*>(stages + nst * C::kStageBytes);             // [kGroups][8 D + 8] (CL = true): o, lse
    volatile int* abort_flag = cta_flags;

    if (threadIdx.x == C::kConsumerWarps * 32) {            // descriptor fetch overlaps the len[] round trip
        asm volatile("prefetch.tensormap [%0];" ::"l"(&mapK) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&mapV) : "memory");
    }
    const int lane = threadIdx.x & 31;
    const uint32_t bar_empty = smem_u32(bars), bar_fullK0 = smem_u32(bars + C::kMaxStages), bar_fullV0 = smem_u32(bars + (1 + C::kGroups) * C::kMaxStages);
    if (threadIdx.x == 0) {                                  // under the shadow of the len[] round trip
        for (int s = 0; s < C::kMaxStages; ++s) {
            mbar_init(bar_empty + 8 * s, kGroupWarps);
            for (int q = 0; q < C::kGroups; ++q) {
                mbar_init(bar_fullK0 + 8 * (q * C::kMaxStages + s), 1);
                mbar_init(bar_fullV0 + 8 * (q * C::kMaxStages + s), 1);
            }
        }
        cta_flags[0] = 0;
        cta_flags[1] = 0;                                    // segments that hold at least one tile (counted below)
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if constexpr (CL) {
        // Programmatic dependent launch: the cluster form is launched so that it may start while the kernel before it on
        // the stream (normally the previous draft step) is still finishing on other SMs. Everything above touches only
        // shared memory and the kernel's parameters; from here on global memory is read and written, which has to wait
        // until that kernel has completed and its writes (lengths, the appended row, the ticket word) are visible. The
        // next kernel on the stream may be set up from now on.
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        asm volatile("griddepcontrol.wait;" ::: "memory");
    }
    // ---- cluster form: this cluster's segment and this CTA's share of its tiles (one length to read, no tables)
    Segment csg;
    csg.seg = -1; csg.seg_start = 0; csg.tiles = 0; csg.b = 0; csg.g = 0; csg.nk = 0; csg.S = 0; csg.slot_base = 0; csg.cap = 0;
    csg.ns = 0; csg.lo = 0; csg.hi = 0; csg.sink_tiles = 0; csg.win_first = 0;
    int c_lo = 0, c_hi = 0;
    uint32_t crank = 0, csize = 1;
    if constexpr (CL) {
        asm("mov.u32 %0, %%cluster_ctarank;" : "=r"(crank));
        asm("mov.u32 %0, %%cluster_nctarank;" : "=r"(csize));
        const int cseg = (int)(blockIdx.x / csize);
        csg = make_segment(p, cseg / p.Hkv, cseg % p.Hkv);
        c_lo = (int)(crank * (uint32_t)csg.tiles / csize);
        c_hi = (int)((crank + 1) * (uint32_t)csg.tiles / csize);
        // a group that gets no tile contributes an empty partial
        if (threadIdx.x < C::kGroups * kMaxGroup)
            part_sm[(threadIdx.x / kMaxGroup) * (kMaxGroup * D + kMaxGroup) + kMaxGroup * D + threadIdx.x % kMaxGroup] = -INFINITY;
        __syncthreads();
    }
    const uint32_t epoch = CL ? 0u : *reinterpret_cast<const volatile uint32_t*>(p.epoch);
    const int par_off = (epoch & 1u) ? kMaxSegmentsPadded(p) : 0;        // which copy of the per-segment words this launch uses

    if constexpr (!CL) {
    // ---- plan: tiles per sequence and partial-slot capacity per sequence (all from len[]; O(B / 32) steps: the
    //      per-sequence values are computed by all threads, the two running sums by one warp)
    for (int b = threadIdx.x; b < p.B; b += blockDim.x)
        tile_prefix[b + 1] = seq_view(p, b).tiles;
    if (threadIdx.x == 0) { tile_prefix[0] = 0; cap_prefix[0] = 0; }
    __syncthreads();
    if (threadIdx.x < 32) warp_inclusive_scan(tile_prefix + 1, p.B);
    __syncthreads();
    {
        const int64_t n_ = tile_prefix[p.B] * p.Hkv;
        const int cn_ = effective_ctas(gridDim.x, n_);
        for (int b = threadIdx.x; b < p.B; b += blockDim.x) {
            // contributors of a segment: per CTA whose static range meets it (<= T * Cn / n + 2 of them), per thief
            // admitted from another segment (<= steal_slots) and per chunk straddling into it, one partial per group
            const int64_t tb = tile_prefix[b + 1] - tile_prefix[b];
            int64_t own = tb == 0 ? 0 : (n_ < (1 << 23) ? (int64_t)(((uint32_t)tb * (uint32_t)cn_) / (uint32_t)n_) : tb * cn_ / n_) + 2;
            if (own > tb) own = tb;
            cap_prefix[b + 1] = tb == 0 ? 0 : kMaxGroups * ((int)own + p.steal_slots + 1);
            if (tb != 0) atomicAdd(cta_flags + 1, p.Hkv);
        }
    }
    __syncthreads();
    if (threadIdx.x < 32) warp_inclusive_scan(cap_prefix + 1, p.B);
    __syncthreads();
    }
    const int G = p.G;
    const int nseg = p.B * p.Hkv;
    const int64_t n = CL ? (int64_t)csg.tiles : (int64_t)p.Hkv * tile_prefix[p.B];
    const int Cg = gridDim.x;
    const int Cn = CL ? Cg : effective_ctas(Cg, n);
    // ---- sequences that hold no token: out = 0, lse = -inf (no CTA owns a tile of theirs)
    for (int seg = blockIdx.x; !CL && seg < nseg; seg += gridDim.x) {
        const int b = seg / p.Hkv, g = seg % p.Hkv;
        if (tile_prefix[b + 1] != tile_prefix[b]) continue;
        __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(p.out) + ((int64_t)b * p.Hq + g * G) * D;
        for (int idx = threadIdx.x; idx < G * D; idx += blockDim.x) o[idx] = __float2bfloat16(0.f);
        if (p.lse && threadIdx.x < G) p.lse[(int64_t)b * p.Hq + g * G + threadIdx.x] = -INFINITY;
    }
    if (!CL && n == 0) {                                     // nothing to attend over at all
        if (threadIdx.x == 0 && atomicAdd(p.grab_done, 1) + 1 == Cg) {
            *p.grab_done = 0;
            if (p.k_new) atomicCAS(p.status, 0, kErrBounds);
        }
        return;
    }
    const bool slack = (p.mode == kRing) && (p.cap != p.W);

    if ((int)(threadIdx.x >> 5) >= C::kConsumerWarps) {
        if constexpr (C::kRebalance) {
            asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(C::kRegsProducer));
            if ((int)(threadIdx.x >> 5) > C::kConsumerWarps) {                // filler warps of the producer's warpgroup
                if constexpr (CL) { cluster_sync_all(); cluster_sync_all(); }   // every thread of the cluster joins its two barriers
                return;
            }
        }
        // =================================== producer warp ===================================
        // CTA c < Cn owns the tile range [c n / Cn, (c+1) n / Cn). It streams the first part of it without any
        // bookkeeping; the rest is handed out in small chunks through the per-CTA cursor cur[c], to the owner
        // and, once they run dry, to other CTAs: SMs do not all stream at the same rate, and the slowest one
        // would otherwise set the launch time. A thief prefers a victim inside the segment it is already in
        // (no new partial); moving into another segment is admitted steal_slots times per segment.
        // Tile number `it` of this CTA goes to stage it % nst (kept incrementally: ps, with the parity pph of the
        // stage's use count) and to consumer group it % kGroups.
        const uint32_t stage0 = smem_u32(stages);
        uint32_t it = 0, ps = 0, pph = 0;
        if constexpr (CL) {
            // ---- cluster form: tiles [c_lo, c_hi) of the cluster's segment, in order; page ids fetched 32 at a time
            const int ntiles = c_hi - c_lo;
            for (int base = 0; base < ntiles; base += 32) {
                int page = 0;
                if (p.mode == kPaged) {
                    const int64_t tj = c_lo + base + lane;
                    const int64_t ti = tj < csg.sink_tiles ? tj : csg.win_first + tj - csg.sink_tiles;   // source tile = page index
                    if (base + lane < ntiles) {
                        page = p.page_table[(int64_t)kv_seq(p, csg.b) * p.max_pages + ti];
                        if (page < 0 || page >= p.num_pages) { atomicCAS(p.status, 0, kErrBounds); page = 0; }
                    }
                }
                const int cnt = ntiles - base < 32 ? ntiles - base : 32;
                for (int j = 0; j < cnt; ++j, ++it, ps = (ps + 1 == nst ? 0 : ps + 1), pph ^= (ps == 0)) {
                    const int pg = __shfl_sync(0xffffffffu, page, j);
                    if (lane == 0) {
                        const uint32_t s = ps, ph = pph, gq = it % C::kGroups;
                        const uint32_t bar_fullK = bar_fullK0 + 8 * (gq * C::kMaxStages), bar_fullV = bar_fullV0 + 8 * (gq * C::kMaxStages);
                        if (mbar_wait(bar_empty + 8 * s, ph ^ 1u, abort_flag, p.status)) {
                            int64_t row;
                            if (p.mode == kPaged) row = ((int64_t)pg * p.Hkv + csg.g) * kTileKeys;
                            else {
                                const int64_t tj = c_lo + base + j;
                                const int64_t src = tj < csg.sink_tiles ? tj : csg.win_first + tj - csg.sink_tiles;
                                row = ((int64_t)kv_seq(p, csg.b) * p.Hkv + csg.g) * p.rows_per_head + src * kTileKeys;
                            }
                            const uint32_t dstK = stage0 + s * C::kStageBytes, dstV = dstK + C::kTileBytes;
                            // One barrier for both tensors: the data comes from L2 well ahead of its use, and the consumers
                            // know their tiles by number (group q takes c_lo + q, c_lo + q + kGroups, ... in order), so
                            // this form has neither a second wait per tile nor tags nor end markers.
                            mbar_expect_tx(bar_fullK + 8 * s, 2 * C::kTileBytes);
                            tma_load_3d(dstK, &mapK, (int)row, bar_fullK + 8 * s);
                            tma_load_3d(dstV, &mapV, (int)row, bar_fullK + 8 * s);
                        }
                    }
                }
            }
            (void)bar_fullV0;
            __syncwarp();
            cluster_sync_all();                  // the two barriers of the cluster's merge (the consumers' work lies between them)
            cluster_sync_all();
            return;
        }
        int cur_seg = -1;                    // segment of the last issued tile
        int64_t cur_lo = 0, cur_hi = 0;      // its tile range
        int grp_seg[kMaxGroups], grp_ord[kMaxGroups], pend_k[kMaxGroups];
        bool pend[kMaxGroups];
#pragma unroll
        for (int q = 0; q < kMaxGroups; ++q) { grp_seg[q] = -1; grp_ord[q] = 0; pend_k[q] = 0; pend[q] = false; }
        const bool is_owner = (int)blockIdx.x < Cn;

        // hand the slot number of group gq's latest segment entry over (the group reads it at its flush of that
        // segment, which follows a later arrive of ours on one of its stages)
        auto settle = [&](int gq) {
            if (pend[gq]) {
                if (lane == 0) group_ints[gq * kGroupInts + 4 + 4 * kMaxContrib + (grp_ord[gq] - 1) % kMaxContrib] = pend_k[gq];
                pend[gq] = false;
            }
        };
        // tiles [a, e) of the global line (may cross segment boundaries); page ids fetched 32 at a time
        auto issue_range = [&](int64_t a, int64_t e) {
            int64_t t = a;
            while (t < e) {
                const Segment sg = locate_segment(p, tile_prefix, cap_prefix, t);
                const int64_t seg_end = sg.seg_start + sg.tiles;
                const int64_t t_end = seg_end < e ? seg_end : e;
                const int64_t first_tile = t - sg.seg_start;
                const int ntiles = (int)(t_end - t);
                for (int base = 0; base < ntiles; base += 32) {
                    int page = 0;
                    if (p.mode == kPaged) {
                        const int64_t tj = first_tile + base + lane;
                        const int64_t ti = tj < sg.sink_tiles ? tj : sg.win_first + tj - sg.sink_tiles;   // source tile = page index
                        if (base + lane < ntiles) {
                            page = p.page_table[(int64_t)kv_seq(p, sg.b) * p.max_pages + ti];
                            if (page < 0 || page >= p.num_pages) { atomicCAS(p.status, 0, kErrBounds); page = 0; }
                        }
                    }
                    const int cnt = ntiles - base < 32 ? ntiles - base : 32;
                    // one stage per step: kPair consecutive tiles of the segment (a single one at an odd end)
                    for (int j = 0; j < cnt; j += C::kPair, ++it, ps = (ps + 1 == nst ? 0 : ps + 1), pph ^= (ps == 0)) {
                        const int c2 = cnt - j < C::kPair ? cnt - j : C::kPair;       // tiles in this stage
                        int pg[C::kPair];
#pragma unroll
                        for (int h = 0; h < C::kPair; ++h) pg[h] = __shfl_sync(0xffffffffu, page, (j + h) & 31);
                        const int gq = (int)(it % C::kGroups);
                        settle(gq);
                        if (grp_seg[gq] != sg.seg) {
                            // group gq enters the segment: it needs a partial slot there (result used at the next settle)
                            if (lane == 0) pend_k[gq] = atomicAdd(p.nparts + par_off + sg.seg, 1);
                            pend[gq] = true;
                            grp_seg[gq] = sg.seg;
                            ++grp_ord[gq];
                        }
                        if (lane == 0) {
                            const uint32_t s = ps, ph = pph;
                            const uint32_t bar_fullK = bar_fullK0 + 8 * (gq * C::kMaxStages), bar_fullV = bar_fullV0 + 8 * (gq * C::kMaxStages);
                            if (mbar_wait(bar_empty + 8 * s, ph ^ 1u, abort_flag, p.status)) {
                                const uint32_t dstK = stage0 + s * C::kStageBytes, dstV = dstK + C::kPair * C::kTileBytes;
                                // ordered before the consumers' wait by the arrive below
                                stage_tile[s] = C::kPair == 1 ? t + base + j : (((t + base + j) << 1) | (int64_t)(c2 - 1));
                                int64_t row[C::kPair];
#pragma unroll
                                for (int h = 0; h < C::kPair; ++h) {
                                    if (p.mode == kPaged) row[h] = ((int64_t)pg[h] * p.Hkv + sg.g) * kTileKeys;
                                    else {
                                        const int64_t tj = first_tile + base + j + h;
                                        const int64_t src = tj < sg.sink_tiles ? tj : sg.win_first + tj - sg.sink_tiles;
                                        row[h] = ((int64_t)kv_seq(p, sg.b) * p.Hkv + sg.g) * p.rows_per_head + src * kTileKeys;
                                    }
                                }
                                mbar_expect_tx(bar_fullK + 8 * s, c2 * C::kTileBytes);
#pragma unroll
                                for (int h = 0; h < C::kPair; ++h)
                                    if (h < c2) tma_load_3d(dstK + h * C::kTileBytes, &mapK, (int)row[h], bar_fullK + 8 * s);
                                mbar_expect_tx(bar_fullV + 8 * s, c2 * C::kTileBytes);
#pragma unroll
                                for (int h = 0; h < C::kPair; ++h)
                                    if (h < c2) tma_load_3d(dstV + h * C::kTileBytes, &mapV, (int)row[h], bar_fullV + 8 * s);
                            }
                        }
                    }
                }
                cur_seg = sg.seg; cur_lo = sg.seg_start; cur_hi = seg_end;
                t = t_end;
            }
        };
        auto range_of = [&](int c, int64_t* lo, int64_t* len, int64_t* first) {
            *lo = cta_range_start(c, n, Cn);
            *len = cta_range_start(c + 1, n, Cn) - *lo;
            *first = (!p.steal_slots_enabled || *len < C::kStealMinTiles) ? *len : *len - *len / 4;
        };

        // One loop, three sources of work in turn: the static part of the own range, the rest of the own range chunk
        // by chunk through the cursor (thieves may be taking from it too), then other CTAs' cursors.
        const bool may_steal = p.steal_slots_enabled && n >= (int64_t)C::kStealMinTiles * Cn;
        int phase = is_owner ? 0 : 2;
        int64_t own_lo = 0, own_len = 0, own_first = 0;
        int k_own = 0;                       // own cursor value for the next chunk (phase 1), fetched one chunk ahead
        int64_t adm_lo = 0, adm_hi = 0;      // lane 0: tile range of the segment this CTA was last admitted to as a thief
        if (is_owner) range_of(blockIdx.x, &own_lo, &own_len, &own_first);
        for (int round = 0; round < (1 << 20); ++round) {
            int64_t a = 0, e = 0;            // next tiles to issue
            if (phase == 0) {
                a = own_lo; e = own_lo + own_first;
                phase = 1;
                if (own_len > own_first) {
                    if (lane == 0) k_own = atomicAdd(p.cur + blockIdx.x, C::kStealChunk);
                } else {
                    k_own = 0x7fffffff;
                }
            } else if (phase == 1) {
                const int k = __shfl_sync(0xffffffffu, k_own, 0);
                if (k >= own_len - own_first) { phase = 2; continue; }
                if (lane == 0) k_own = atomicAdd(p.cur + blockIdx.x, C::kStealChunk);     // overlaps the issue below
                a = own_lo + own_first + k;
                e = a + C::kStealChunk < own_lo + own_len ? a + C::kStealChunk : own_lo + own_len;
            } else {
                if (!may_steal || *abort_flag) break;
                // ---- steal: look at every cursor, take from the range with the most left
                int64_t best_rem = 0;
                int best_v = -1, best_used = 0;
                for (int v = lane; v < Cn; v += 32) {
                    if (v == (int)blockIdx.x) continue;
                    int64_t lo, len, first;
                    range_of(v, &lo, &len, &first);
                    const int64_t used = __ldcg(p.cur + v);
                    int64_t rem = len - first - used;
                    if (rem <= 0) continue;
                    const int64_t tv = lo + first + used;
                    if (cur_seg >= 0 && tv >= cur_lo && tv < cur_hi) rem += (int64_t)1 << 40;     // same segment: preferred
                    if (rem > best_rem) { best_rem = rem; best_v = v; best_used = (int)used; }
                }
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) {
                    const int64_t r2 = __shfl_xor_sync(0xffffffffu, best_rem, off);
                    const int v2 = __shfl_xor_sync(0xffffffffu, best_v, off);
                    const int u2 = __shfl_xor_sync(0xffffffffu, best_used, off);
                    if (r2 > best_rem || (r2 == best_rem && v2 > best_v)) { best_rem = r2; best_v = v2; best_used = u2; }
                }
                if (best_v < 0) break;
                int64_t lo, len, first;
                range_of(best_v, &lo, &len, &first);
                // Take tiles from the victim's cursor with a compare-and-swap, clipped to the segment we are in or have
                // been admitted to: a thief never lands in a segment where it holds no right to a partial slot, and a
                // stolen chunk never straddles a segment boundary.
                int got = 0;                       // 1: tiles [a, e) are ours; 0: look again; -1: stop stealing
                if (lane == 0) {
                    int used = best_used;          // cursor value seen by the scan; a failed swap returns the current one
                    for (int tries = 0; tries < 8 && got == 0; ++tries) {
                        const int64_t rem = len - first - used;
                        if (rem <= 0) break;
                        const int64_t tv = lo + first + used;
                        int64_t alo = cur_lo, ahi = cur_hi;
                        if (!(cur_seg >= 0 && tv >= cur_lo && tv < cur_hi)) {
                            if (tv >= adm_lo && tv < adm_hi) {
                                alo = adm_lo; ahi = adm_hi;
                            } else {
                                // another segment: needs partial slots there, admitted steal_slots times per segment
                                const Segment vs = locate_segment(p, tile_prefix, cap_prefix, tv);
                                if (atomicAdd(p.nthief + par_off + vs.seg, 1) >= p.steal_slots) { got = -1; break; }
                                adm_lo = alo = vs.seg_start; adm_hi = ahi = vs.seg_start + vs.tiles;
                            }
                        }
                        int64_t take = rem / 8;            // larger bites while much is left: a steal costs two round trips
                        if (take < C::kStealChunk) take = C::kStealChunk;
                        if (take > 4 * C::kStealChunk) take = 4 * C::kStealChunk;
                        if (take > rem) take = rem;
                        if (tv + take > ahi) take = ahi - tv;
                        const int prev = atomicCAS(p.cur + best_v, used, used + (int)take);
                        if (prev == used) { a = tv; e = tv + take; got = 1; }
                        else used = prev;
                    }
                }
                got = __shfl_sync(0xffffffffu, got, 0);
                if (got < 0) break;                // no slot for us elsewhere: stop stealing
                if (got == 0) continue;            // somebody else got there first: look again
                a = __shfl_sync(0xffffffffu, a, 0);
                e = __shfl_sync(0xffffffffu, e, 0);
            }
            issue_range(a, e);
        }
#pragma unroll
        for (int q = 0; q < C::kGroups; ++q) settle(q);
        if (lane == 0) {
            // one end marker per consumer group, then: this CTA takes no more tiles
            for (int q = 0; q < C::kGroups; ++q, ++it, ps = (ps + 1 == nst ? 0 : ps + 1), pph ^= (ps == 0)) {
                const uint32_t s = ps, ph = pph;
                const uint32_t gq = it % C::kGroups;
                mbar_wait(bar_empty + 8 * s, ph ^ 1u, abort_flag, p.status);
                stage_tile[s] = -1;
                mbar_arrive(bar_fullK0 + 8 * (gq * C::kMaxStages + s));
                mbar_arrive(bar_fullV0 + 8 * (gq * C::kMaxStages + s));
            }
            atomicAdd(p.grab_done, 1);
        }
        return;
    }

    if constexpr (C::kRebalance) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(C::kRegsConsumer));
    // ===================================== consumer groups =====================================
    const int grp = threadIdx.x / kGroupThreads, tid = threadIdx.x % kGroupThreads;   // group, thread within the group
    const int warp = tid >> 5;                           // warp within the group: owns keys [16 warp, 16 warp + 16) of a tile
    float* scratch = scratch_all + grp * C::kScratchFloats;
    // where a flush merges the four warps' accumulators: the group's scratch, or the first stage (see kFlushInStages)
    float* fscratch = C::kFlushInStages ? reinterpret_cast<float*>(stages + grp * C::kStageBytes) : scratch;
    float* sm_m = sm_stats + grp * 3 * kGroupWarps * kMaxGroup;
    float* sm_l = sm_m + kGroupWarps * kMaxGroup;
    float* sm_le = sm_l + kGroupWarps * kMaxGroup;
    int* gints = group_ints + grp * kGroupInts;          // [0] launch-last, [1] broadcast
    int* contrib = gints + 4;                            // [kMaxContrib][4]
    volatile int* reg_k = gints + 4 + 4 * kMaxContrib;   // [kMaxContrib]
    int64_t* contrib_base = contrib_base_all + grp * 2 * kMaxContrib;       // [kMaxContrib] slot base, then [kMaxContrib] segment tiles
    int64_t* contrib_tiles = contrib_base + kMaxContrib;
    const int g8 = lane >> 2, t4 = lane & 3;            // MMA fragment coordinates
    const float scale = p.scale_log2;
    // ldmatrix lane addressing (byte offsets inside a 64-row x 128-byte swizzled chunk)
    const int mi = lane >> 3, rr = lane & 7;
    const int rowK = warp * 16 + (mi & 1) * 8 + rr, halfK = mi >> 1;       // K as A operand (non-transposed)
    const int rowV = warp * 16 + (mi >> 1) * 8 + rr, halfV = mi & 1;       // V as A operand (transposed load)
    const uint32_t offK = rowK * 128, offV = rowV * 128;
    const uint32_t stage0 = smem_u32(stages);
    const uint32_t bar_fullK = bar_fullK0 + 8 * (grp * C::kMaxStages), bar_fullV = bar_fullV0 + 8 * (grp * C::kMaxStages);

    const int nonempty_segs = cta_flags[1];
    bool launch_last = false;                            // group thread 0: did this group complete the launch's last segment?
    int ncontrib = 0;                                    // uniform across the group
    int ord = 0;                                         // segment entries so far (mirrors the producer's count for this group)

    Segment sg;
    sg.seg = -1; sg.seg_start = 0; sg.tiles = 0; sg.b = 0; sg.g = 0; sg.nk = 0; sg.S = 0; sg.slot_base = 0; sg.cap = 0;
    sg.ns = 0; sg.lo = 0; sg.hi = 0; sg.sink_tiles = 0; sg.win_first = 0;
    int new_tile = -1;                                   // tile (within the segment) whose row this warp must patch (fused append)
    int new_row = 0;
    int seg_tiles_done = 0;                              // tiles of the current segment this group has processed
    uint32_t qb[C::kQShared ? 1 : C::kKSteps][2];      // query fragments (registers), or ...
    uint2* q_sm = q_sm_all + grp * C::kKSteps * 32 + lane;   // ... this lane's column of the group's shared copy
    float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f}, le[2] = {0.f, 0.f};   // l: rounded weights (normaliser), le: exact (lse)
    float o[C::kKSteps][4];
    // multiplier of the raw scores of heads 2*t4 and 2*t4+1: the softmax scale in log2 units; for an fp8 store also
    // the key scale of the KV head and the power of two the head's query was normalised by
    float smul[2] = {scale, scale};
    float vscale = 1.f;                                  // fp8: dequantisation scale of V, applied to the normalised partial

    // Combine every segment this group has contributed to (waits for their last partial), then forget them.
    auto combine_outstanding = [&]() {
        for (int i = 0; !CL && i < ncontrib; ++i) {
            const int seg = contrib[4 * i], b = contrib[4 * i + 1], g = contrib[4 * i + 2], k = contrib[4 * i + 3];
            if (tid == 0) {
                gints[1] = wait_tiles(p.arrive + par_off + seg, (uint32_t)contrib_tiles[i], p.spin_limit, abort_flag, p.status);
            }
            group_barrier(grp);
            const int np = gints[1];
            if (np >= 1 && np <= kMaxParts && k < np) combine_segment(p, b, g, contrib_base[i], np, k, scratch, tid, grp);
            group_barrier(grp);
        }
        ncontrib = 0;
    };

    // Merge the four warps' states, publish the partial of (this group, current segment), note the contribution.
    auto flush_segment = [&]() {
#pragma unroll
        for (int off = 4; off <= 16; off <<= 1) {
            l[0] += __shfl_xor_sync(0xffffffffu, l[0], off);
            l[1] += __shfl_xor_sync(0xffffffffu, l[1], off);
            le[0] += __shfl_xor_sync(0xffffffffu, le[0], off);
            le[1] += __shfl_xor_sync(0xffffffffu, le[1], off);
        }
        group_barrier(grp);                                   // scratch / sm_m free
        if (g8 == 0) {
            sm_m[warp * kMaxGroup + 2 * t4] = m[0]; sm_m[warp * kMaxGroup + 2 * t4 + 1] = m[1];
            sm_l[warp * kMaxGroup + 2 * t4] = l[0]; sm_l[warp * kMaxGroup + 2 * t4 + 1] = l[1];
            sm_le[warp * kMaxGroup + 2 * t4] = le[0]; sm_le[warp * kMaxGroup + 2 * t4 + 1] = le[1];
        }
        group_barrier(grp);
        int k = CL ? 0 : reg_k[ord % kMaxContrib];            // slot the producer took when this group entered the segment
        if (!CL && (k < 0 || k >= sg.cap)) {
            // cannot happen while the admission rules hold; never write outside the segment's slots
            if (tid == 0) {
                atomicCAS(p.status, 0, kErrBounds);
                int* dbg = p.status + 8;                       // header bytes [32, 64): diagnostic record
                dbg[0] = k; dbg[1] = sg.cap; dbg[2] = sg.seg; dbg[3] = (int)blockIdx.x * kMaxGroups + grp; dbg[4] = ord; dbg[5] = seg_tiles_done;
            }
            k = sg.cap - 1;
        }
        if (!CL && tid == 0) {
            contrib[4 * ncontrib + 3] = k;
            p.part_key[sg.slot_base + k] = (int)blockIdx.x * kMaxGroups + grp;
        }
        ++ord;
        const int64_t pidx = (int64_t)sg.slot_base + k;
        // where the partial goes: the workspace, or (cluster form) this group's buffer in shared memory, rows of D floats
        float* const dst_o = CL ? part_sm + grp * (kMaxGroup * D + kMaxGroup) : p.part_o + pidx * G * D;
        float* const dst_lse = CL ? part_sm + grp * (kMaxGroup * D + kMaxGroup) + kMaxGroup * D : p.part_lse + pidx * G;
        float f[2];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int h = 2 * t4 + i;
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < kGroupWarps; ++w) M = fmaxf(M, sm_m[w * kMaxGroup + h]);
            float L = 0.f, Le = 0.f;
            if (M > -INFINITY) {
#pragma unroll
                for (int w = 0; w < kGroupWarps; ++w) {
                    const float e = ex2(sm_m[w * kMaxGroup + h] - M);
                    L += sm_l[w * kMaxGroup + h] * e;
                    Le += sm_le[w * kMaxGroup + h] * e;
                }
            }
            f[i] = (L > 0.f && m[i] > -INFINITY) ? ex2(m[i] - M) / L * vscale : 0.f;
            if (warp == 0 && g8 == 0 && h < G) dst_lse[h] = Le > 0.f ? (M + lg2(Le)) * kLn2 : -INFINITY;
        }
        constexpr int kPasses = D / C::kPassCols;               // kPassCols columns of d per pass through the scratch
        constexpr int kScratchRow = C::kScratchRow;
#pragma unroll
        for (int pass = 0; pass < kPasses; ++pass) {
            if (pass > 0) group_barrier(grp);
#pragma unroll
            for (int mbl = 0; mbl < C::kPassCols / 16; ++mbl) {
                const int mb = pass * (C::kPassCols / 16) + mbl;
                // accumulator rows g8 and g8 + 8 of block mb hold d = 16 mb + g8 and + 8 (bf16 store), or, for an fp8
                // store whose V fragments come out of the transposed load with d pairs interleaved, d = 16 mb + 2 g8 and + 1
                float* row0 = fscratch + (warp * kMaxGroup + 2 * t4) * kScratchRow + mbl * 16 + (F8 ? 2 * g8 : g8);
                float* row1 = row0 + kScratchRow;
                constexpr int kSecond = F8 ? 1 : 8;
                row0[0] = o[mb][0] * f[0]; row1[0] = o[mb][1] * f[1];
                row0[kSecond] = o[mb][2] * f[0]; row1[kSecond] = o[mb][3] * f[1];
            }
            group_barrier(grp);
            for (int idx = tid; idx < G * C::kPassCols; idx += kGroupThreads) {
                const int h = idx / C::kPassCols, dd = idx % C::kPassCols;
                float acc = 0.f;
#pragma unroll
                for (int w = 0; w < kGroupWarps; ++w) acc += fscratch[(w * kMaxGroup + h) * kScratchRow + dd];
                dst_o[h * D + pass * C::kPassCols + dd] = acc;
            }
        }
        group_barrier(grp);
        if (!CL && tid == 0) {
            __threadfence();                                   // the group's partial is visible device-wide before the arrival
            const unsigned long long old = atomicAdd(p.arrive + par_off + sg.seg, (1ull << 32) | (unsigned long long)seg_tiles_done);
            if ((int)(uint32_t)old + seg_tiles_done == sg.tiles) {        // this contribution completes the segment
                if (atomicAdd(p.segs_done, 1) + 1 == nonempty_segs) {
                    *p.segs_done = 0;
                    *p.epoch = epoch + 1u;
                    launch_last = true;
                }
            }
        }
        ++ncontrib;
    };

    // Start work on the segment that holds tile tt: partial bookkeeping, append target, query fragments, fresh state.
    auto enter_segment = [&](int64_t tt) {
        if constexpr (CL) sg = csg;
        else sg = locate_segment(p, tile_prefix, cap_prefix, tt);
        if (!CL && tid == 0) {
            contrib[4 * ncontrib] = sg.seg; contrib[4 * ncontrib + 1] = sg.b; contrib[4 * ncontrib + 2] = sg.g;
            contrib_base[ncontrib] = sg.slot_base;
            contrib_tiles[ncontrib] = sg.tiles;
        }
        seg_tiles_done = 0;
        // fused append (Appendix A, RING / the KV write of a draft forward): where does the new token go?
        new_tile = -1;
        if (appends_to(p, sg.b)) {
            const int64_t pos = sg.S - 1;
            const int64_t key = p.mode == kRing ? ring_slot(pos, p.n_sink, p.cap) : pos;
            new_row = (int)(key % kTileKeys);
            // tile of the segment that holds the row: with a window view, the last tile unless the token is a sink token
            if ((new_row >> 4) == warp) new_tile = (p.window_view && sg.S > sg.ns) ? sg.tiles - 1 : (int)(key / kTileKeys);
        }
        // Q^T fragments (B operand: k = d, n = head); heads >= G read as zero
        const uint32_t* qrow = reinterpret_cast<const uint32_t*>(
            reinterpret_cast<const __nv_bfloat16*>(p.q) + ((int64_t)sg.b * p.Hq + sg.g * G + g8) * D);
        // Words of the query row that make up this lane's fragment of 16-column step ks: ks * 8 + w0 and ks * 8 + w1.
        // For an fp8 store the MMA k-slot order within 16 columns of d follows the byte order ldmatrix delivers the
        // codes in: lane t4 holds d = 4 t4 .. 4 t4 + 3 of each 16.
        const int w0 = F8 ? 2 * t4 : t4, w1 = F8 ? 2 * t4 + 1 : 4 + t4;
        float down = 1.f;
        if constexpr (F8) {
            // The e4m3 codes are widened to f16 (exact), so the query goes through the f16 MMA too. Its range is made
            // safe by a per-head power of two (exact both ways): q' = q * 2^-e with 2^e <= max|q| < 2^(e+1), and 2^e goes
            // into the score multiplier together with the key scale.
            float amax = 0.f;
#pragma unroll
            for (int ks = 0; ks < C::kKSteps; ++ks) {
                const uint32_t a = g8 < G ? __ldg(qrow + ks * 8 + w0) : 0u, b = g8 < G ? __ldg(qrow + ks * 8 + w1) : 0u;
                amax = fmaxf(fmaxf(amax, fmaxf(fabsf(bf16lo(a)), fabsf(bf16hi(a)))), fmaxf(fabsf(bf16lo(b)), fabsf(bf16hi(b))));
            }
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
            amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
            uint32_t eb = (__float_as_uint(amax) >> 23) & 0xffu;
            eb = eb < 1u ? 1u : (eb > 253u ? 253u : eb);
            down = __uint_as_float((254u - eb) << 23);
            const float hmul = g8 < G ? scale * __uint_as_float(eb << 23) * __ldg(p.k_scale + sg.g) : 0.f;
            smul[0] = __shfl_sync(0xffffffffu, hmul, 8 * t4);
            smul[1] = __shfl_sync(0xffffffffu, hmul, 8 * t4 + 4);
            vscale = __ldg(p.v_scale + sg.g);
        }
        auto fragment = [&](int ks) {
            uint2 f;
            f.x = g8 < G ? __ldg(qrow + ks * 8 + w0) : 0u;
            f.y = g8 < G ? __ldg(qrow + ks * 8 + w1) : 0u;
            if constexpr (F8) {
                f.x = pack_f16x2(bf16lo(f.x) * down, bf16hi(f.x) * down);
                f.y = pack_f16x2(bf16lo(f.y) * down, bf16hi(f.y) * down);
            }
            return f;
        };
        if constexpr (C::kQShared) {
            group_barrier(grp);                          // no warp of the group still reads the previous segment's fragments
            for (int ks = warp; ks < C::kKSteps; ks += kGroupWarps) q_sm[ks * 32] = fragment(ks);
            group_barrier(grp);
        } else {
#pragma unroll
            for (int ks = 0; ks < C::kKSteps; ++ks) {
                const uint2 f = fragment(ks);
                qb[ks][0] = f.x; qb[ks][1] = f.y;
            }
        }
        m[0] = m[1] = -INFINITY; l[0] = l[1] = 0.f; le[0] = le[1] = 0.f;
#pragma unroll
        for (int mb = 0; mb < C::kKSteps; ++mb) { o[mb][0] = o[mb][1] = o[mb][2] = o[mb][3] = 0.f; }
    };
    // One stage: NH consecutive tiles of the current segment (tiles tj0 .. tj0 + NH - 1 of it) in stage s, this warp's 16
    // keys of each. With NH = 2 the two slabs are independent until the softmax, which takes them as one block of 32 keys.
    auto process_stage = [&](auto nh_tag, uint32_t s, uint32_t ph, int tj0) {
        constexpr int NH = decltype(nh_tag)::value;
        const uint32_t sK = stage0 + s * C::kStageBytes, sV = sK + C::kPair * C::kTileBytes;
        int key0[NH], vlo[NH], vhi[NH], wkey0[NH];
        bool has_new[NH];
        bool any_valid = false, all_full = true, any_new = false, any_tail = false;
#pragma unroll
        for (int h = 0; h < NH; ++h) {
            const int tj = tj0 + h;                                    // tile within the segment
            const bool sink_part = tj < sg.sink_tiles;
            key0[h] = (sink_part ? tj : sg.win_first + tj - sg.sink_tiles) * kTileKeys;      // first row of the tile
            vlo[h] = sink_part ? 0 : sg.lo; vhi[h] = sink_part ? sg.ns : sg.hi;              // rows of it that count
            wkey0[h] = key0[h] + warp * 16;
            all_full = all_full && key0[h] >= vlo[h] && key0[h] + kTileKeys <= vhi[h] && !slack;
            any_valid = any_valid || (wkey0[h] < vhi[h] && wkey0[h] + 16 > vlo[h]);
            has_new[h] = tj == new_tile;                               // this warp owns the appended row in this tile
            any_new = any_new || has_new[h];
            any_tail = any_tail || wkey0[h] + 16 > vhi[h];
        }
        int64_t new_off = 0;
        bool new_ok = true;
        if (__builtin_expect(any_new, 0)) {
#pragma unroll
            for (int h = 0; h < NH; ++h) {
                if (!has_new[h]) continue;
                new_off = kv_row_offset(p, sg.b, sg.g, key0[h] + new_row, &new_ok);
                if (!new_ok && lane == 0) atomicCAS(p.status, 0, kErrBounds);
                patch_new_row<D, F8>(p.k_new, (int64_t)sg.b * p.Hkv + sg.g, p.k_scale, sg.g, sK + h * C::kTileBytes, new_row,
                                     new_ok ? reinterpret_cast<unsigned char*>(p.k) + new_off * C::kElemBytes : nullptr, lane);
                if (p.mode == kRing && sg.g == 0 && lane == 0)
                    p.slot_pos[(int64_t)sg.b * p.rows_per_head + key0[h] + new_row] = (int32_t)(sg.S - 1);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
        }
        uint32_t pb[NH][2];
#pragma unroll
        for (int h = 0; h < NH; ++h) pb[h][0] = pb[h][1] = 0;
        if (any_valid) {
            // ---- S^T = K . Q^T for this warp's 16 keys of every tile (two accumulator chains per tile)
            float sa[NH][4], sb[NH][4];
#pragma unroll
            for (int h = 0; h < NH; ++h) { sa[h][0] = sa[h][1] = sa[h][2] = sa[h][3] = 0.f; sb[h][0] = sb[h][1] = sb[h][2] = sb[h][3] = 0.f; }
            if constexpr (!F8) {
#pragma unroll
                for (int ks = 0; ks < C::kKSteps; ++ks) {
                    uint32_t q0, q1;
                    if constexpr (C::kQShared) { const uint2 f = q_sm[ks * 32]; q0 = f.x; q1 = f.y; }
                    else { q0 = qb[ks][0]; q1 = qb[ks][1]; }
                    const uint32_t c16 = (uint32_t)((ks & 3) * 2 + halfK);
#pragma unroll
                    for (int h = 0; h < NH; ++h) {
                        uint32_t a[4];
                        ldmatrix_x4(a, sK + h * C::kTileBytes + (ks >> 2) * C::kChunkBytes + offK + ((c16 ^ (uint32_t)rr) << 4));
                        if (ks & 1) mma_bf16(sb[h], a, q0, q1);
                        else mma_bf16(sa[h], a, q0, q1);
                    }
                }
            } else {
                // one ldmatrix brings 32 columns of d for the warp's 16 keys: matrices {keys 0-7, 8-15} x {16 d, next 16 d};
                // a thread's word holds 4 consecutive codes of one key, which become the k-slots (2 t4, 2 t4 + 1) and
                // (2 t4 + 8, 2 t4 + 9) of that 16-column step (the query fragments use the same order)
#pragma unroll
                for (int j = 0; j < C::kKSteps / 2; ++j) {
                    uint2 qa, qc;
                    if constexpr (C::kQShared) { qa = q_sm[(2 * j) * 32]; qc = q_sm[(2 * j + 1) * 32]; }
                    else { qa = make_uint2(qb[2 * j][0], qb[2 * j][1]); qc = make_uint2(qb[2 * j + 1][0], qb[2 * j + 1][1]); }
                    const uint32_t c16 = (uint32_t)((j & 3) * 2 + halfK);
#pragma unroll
                    for (int h = 0; h < NH; ++h) {
                        uint32_t r[4], a[4];
                        ldmatrix_x4(r, sK + h * C::kTileBytes + (j >> 2) * C::kChunkBytes + offK + ((c16 ^ (uint32_t)rr) << 4));
                        e4m3x4_to_f16x2x2(r[0], a[0], a[2]);
                        e4m3x4_to_f16x2x2(r[1], a[1], a[3]);
                        mma_f16(sa[h], a, qa.x, qa.y);
                        e4m3x4_to_f16x2x2(r[2], a[0], a[2]);
                        e4m3x4_to_f16x2x2(r[3], a[1], a[3]);
                        mma_f16(sb[h], a, qc.x, qc.y);
                    }
                }
            }
            // raw scores; the multipliers smul (softmax scale in log2 units, for an fp8 store also the key scale and the
            // query's power of two: all positive) are applied to the maxima and inside the exponentials
            float sc[NH][4];
#pragma unroll
            for (int h = 0; h < NH; ++h) {
#pragma unroll
                for (int i = 0; i < 4; ++i) sc[h][i] = sa[h][i] + sb[h][i];
            }
            if (__builtin_expect(!all_full, 0)) {
#pragma unroll
                for (int h = 0; h < NH; ++h) {
                    const int ka = wkey0[h] + g8, kb = ka + 8;
                    bool va = ka >= vlo[h] && ka < vhi[h], vb = kb >= vlo[h] && kb < vhi[h];
                    if (slack) {
                        va = va && ring_slot_live(ka, sg.S, p.n_sink, p.W, p.cap);
                        vb = vb && ring_slot_live(kb, sg.S, p.n_sink, p.W, p.cap);
                    }
                    if (!va) { sc[h][0] = -INFINITY; sc[h][1] = -INFINITY; }
                    if (!vb) { sc[h][2] = -INFINITY; sc[h][3] = -INFINITY; }
                }
            }
            // ---- online softmax; this thread holds heads 2*t4, 2*t4+1 for keys g8 and g8+8 of every tile
            float mx0 = fmaxf(sc[0][0], sc[0][2]), mx1 = fmaxf(sc[0][1], sc[0][3]);
#pragma unroll
            for (int h = 1; h < NH; ++h) {
                mx0 = fmaxf(mx0, fmaxf(sc[h][0], sc[h][2]));
                mx1 = fmaxf(mx1, fmaxf(sc[h][1], sc[h][3]));
            }
#pragma unroll
            for (int off = 4; off <= 16; off <<= 1) {
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
            }
            const float mn0 = fmaxf(m[0], mx0 * smul[0]), mn1 = fmaxf(m[1], mx1 * smul[1]);
            // the running maxima rarely move after the first tiles of a segment: rescale only when some lane's did
            if (__builtin_expect(__any_sync(0xffffffffu, mn0 != m[0] || mn1 != m[1]), 0)) {
                const float corr0 = mn0 == -INFINITY ? 1.f : ex2(m[0] - mn0), corr1 = mn1 == -INFINITY ? 1.f : ex2(m[1] - mn1);
                le[0] *= corr0; le[1] *= corr1;
                l[0] *= corr0; l[1] *= corr1;
#pragma unroll
                for (int mb = 0; mb < C::kKSteps; ++mb) {
                    o[mb][0] *= corr0; o[mb][1] *= corr1; o[mb][2] *= corr0; o[mb][3] *= corr1;
                }
                m[0] = mn0; m[1] = mn1;
            }
            const float nu0 = mn0 == -INFINITY ? 0.f : -mn0, nu1 = mn1 == -INFINITY ? 0.f : -mn1;
#pragma unroll
            for (int h = 0; h < NH; ++h) {
                const float p0 = ex2(fmaf(sc[h][0], smul[0], nu0)), p1 = ex2(fmaf(sc[h][1], smul[1], nu1));
                const float p2 = ex2(fmaf(sc[h][2], smul[0], nu0)), p3 = ex2(fmaf(sc[h][3], smul[1], nu1));
                const uint32_t pa = F8 ? pack_f16x2(p0, p1) : pack_bf16x2(p0, p1);             // key g8   : heads 2t4, 2t4+1
                const uint32_t pc = F8 ? pack_f16x2(p2, p3) : pack_bf16x2(p2, p3);             // key g8+8
                le[0] += p0 + p2;
                le[1] += p1 + p3;
                if constexpr (F8) {
                    l[0] += f16lo(pa) + f16lo(pc);
                    l[1] += f16hi(pa) + f16hi(pc);
                } else {
                    l[0] += bf16lo(pa) + bf16lo(pc);      // sums of the rounded weights the MMA will use
                    l[1] += bf16hi(pa) + bf16hi(pc);
                }
                pb[h][0] = movmatrix_trans(pa);                      // P^T as B operand: k = key, n = head
                pb[h][1] = movmatrix_trans(pc);
            }
        }
        if constexpr (!CL) mbar_wait(bar_fullV + 8 * s, ph, abort_flag, p.status);      // (cluster form: K and V share a barrier)
        if (__builtin_expect(any_new, 0)) {
#pragma unroll
            for (int h = 0; h < NH; ++h)
                if (has_new[h])
                    patch_new_row<D, F8>(p.v_new, (int64_t)sg.b * p.Hkv + sg.g, p.v_scale, sg.g, sV + h * C::kTileBytes, new_row,
                                         new_ok ? reinterpret_cast<unsigned char*>(p.v) + new_off * C::kElemBytes : nullptr, lane);
        }
        if (any_valid) {
            if (__builtin_expect(any_tail, 0)) {
                // rows past the end were never written (or, in a sink tile of a window view, may be): they can hold
                // NaN/Inf bit patterns, and 0 * NaN would poison the accumulators. Zero them in shared memory.
#pragma unroll
                for (int h = 0; h < NH; ++h) {
                    if (wkey0[h] + 16 <= vhi[h]) continue;
                    const int first_bad = vhi[h] > wkey0[h] ? vhi[h] - wkey0[h] : 0;
                    for (int idx = lane; idx < (16 - first_bad) * C::kChunks * 8; idx += 32) {
                        const int r = first_bad + idx / (C::kChunks * 8), rem = idx % (C::kChunks * 8);
                        const uint32_t addr = sV + h * C::kTileBytes + (rem >> 3) * C::kChunkBytes + (warp * 16 + r) * 128 + ((rem & 7) << 4);
                        asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(addr), "r"(0u) : "memory");
                    }
                }
            }
            if (__builtin_expect(any_new || any_tail, 0)) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
            }
            // ---- O^T += V^T . P^T
            if constexpr (!F8) {
#pragma unroll
                for (int mb = 0; mb < C::kKSteps; ++mb) {
                    const uint32_t c16 = (uint32_t)((mb & 3) * 2 + halfV);
#pragma unroll
                    for (int h = 0; h < NH; ++h) {
                        uint32_t a[4];
                        ldmatrix_x4_trans(a, sV + h * C::kTileBytes + (mb >> 2) * C::kChunkBytes + offV + ((c16 ^ (uint32_t)rr) << 4));
                        mma_bf16(o[mb], a, pb[h][0], pb[h][1]);
                    }
                }
            } else {
                // the transposed load hands a thread, per matrix, the codes of keys (2 t4, 2 t4 + 1) for d = 2 g8 and
                // 2 g8 + 1 of a 16-column unit: accumulator row g8 of the block is d = 2 g8, row g8 + 8 is d = 2 g8 + 1
#pragma unroll
                for (int j = 0; j < C::kKSteps / 2; ++j) {
                    const uint32_t c16 = (uint32_t)((j & 3) * 2 + halfK);
#pragma unroll
                    for (int h = 0; h < NH; ++h) {
                        uint32_t r[4], a[4];
                        ldmatrix_x4_trans(r, sV + h * C::kTileBytes + (j >> 2) * C::kChunkBytes + offK + ((c16 ^ (uint32_t)rr) << 4));
                        e4m3x4_to_f16x2x2(__byte_perm(r[0], 0, 0x3120), a[0], a[1]);
                        e4m3x4_to_f16x2x2(__byte_perm(r[1], 0, 0x3120), a[2], a[3]);
                        mma_f16(o[2 * j], a, pb[h][0], pb[h][1]);
                        e4m3x4_to_f16x2x2(__byte_perm(r[2], 0, 0x3120), a[0], a[1]);
                        e4m3x4_to_f16x2x2(__byte_perm(r[3], 0, 0x3120), a[2], a[3]);
                        mma_f16(o[2 * j + 1], a, pb[h][0], pb[h][1]);
                    }
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_empty + 8 * s);
    };
    // The loop is written so that enter / flush / tile processing each appear once in the code (the kernel's
    // tail runs once per launch, from a cold instruction cache: code size is latency there).
    int64_t tt = -1;                                     // (first) tile in hand
    int tcnt = 1;                                        // tiles in the stage in hand
    bool have_tile = false, need_enter = false;
    if constexpr (CL) {
        if (c_lo + grp < c_hi) { tt = c_lo + grp; need_enter = true; }
    } else if ((int)blockIdx.x < Cn) {
        // an owner knows its first tiles: fetch the query while they are still in flight
        const int64_t first = cta_range_start(blockIdx.x, n, Cn) + grp * C::kPair;
        if (first < cta_range_start(blockIdx.x + 1, n, Cn)) { tt = first; need_enter = true; }
    }
    uint32_t it = grp, cs = grp, cph = 0;
    for (;;) {
        if (__builtin_expect(need_enter, 0)) { enter_segment(tt); need_enter = false; }
        const uint32_t s = cs, ph = cph;             // stage of tile `it` and the parity of this group's use count of it
        if (!have_tile) {
            bool end, outside;
            if constexpr (CL) {
                tt = c_lo + (int)it;                                   // this CTA's tiles in order: nothing to look up
                end = tt >= c_hi || !mbar_wait(bar_fullK + 8 * s, ph, abort_flag, p.status);
                outside = false;                                       // one segment per cluster
            } else {
                const bool landed = mbar_wait(bar_fullK + 8 * s, ph, abort_flag, p.status);
                tt = *reinterpret_cast<volatile int64_t*>(stage_tile + s);
                if (C::kPair == 2 && tt >= 0) { tcnt = (int)(tt & 1) + 1; tt >>= 1; }      // (first tile << 1) | (tiles - 1)
                end = tt < 0 || !landed;
                outside = sg.seg < 0 || tt < sg.seg_start || tt >= sg.seg_start + sg.tiles;
            }
            if (__builtin_expect((end || outside) && sg.seg >= 0 && seg_tiles_done > 0, 0)) flush_segment();
            if (__builtin_expect(end || ncontrib == kMaxContrib, 0)) {
                combine_outstanding();           // every segment this group contributed to (normally: once, at the end)
                if (end) break;
            }
            have_tile = true;
            if (__builtin_expect(outside, 0)) { need_enter = true; continue; }
        }
        have_tile = false;
        seg_tiles_done += tcnt;
        if (C::kPair == 2 && tcnt == 2) process_stage(std::integral_constant<int, C::kPair>{}, s, ph, (int)tt - sg.seg_start);
        else process_stage(std::integral_constant<int, 1>{}, s, ph, (int)tt - sg.seg_start);
        it += C::kGroups;
        cs += C::kGroups;                            // nst is a multiple of kGroups: the stage stays with this group
        if (cs >= nst) { cs -= nst; cph ^= 1u; }
    }

    // ---- a CTA that gave up on a barrier must not leave while copies into its shared memory may still land:
    //      wait (bounded) for this group's next use of each of its stages; a stage nothing was issued for just runs
    //      the short limit out. If even that expires the copy is lost with the CTA: the launch's results were
    //      already invalid, the memory written is still this kernel's own.
    if (*abort_flag == kAbortBarrier && tid == 0) {
        for (uint32_t s2 = grp; s2 < nst; s2 += C::kGroups) {
            const uint32_t par = s2 >= cs ? cph : cph ^ 1u;
            for (uint32_t i = 0; i < kDrainLimit && !mbar_test_wait(bar_fullK + 8 * s2, par); ++i) { }
            for (uint32_t i = 0; i < kDrainLimit && !mbar_test_wait(bar_fullV + 8 * s2, par); ++i) { }
        }
    }
    if constexpr (CL) {
        // ---- cluster form: merge the cluster's partials through distributed shared memory. CTA r reduces the r-th slice
        //      of the (head, d) columns: weights exp(lse_s - lse) from all partials' lse values, then the weighted sum.
        cluster_sync_all();                                   // every group of every CTA has left its partial (or none)
        if (grp == 0) {
            constexpr int kVec = D / 4;                       // float4 columns per head
            constexpr int kPart = kMaxGroup * D + kMaxGroup;  // floats per partial: o [8][D], lse [8]
            const int cols = G * kVec, np = (int)csize * C::kGroups;
            const int per = (cols + (int)csize - 1) / (int)csize;
            const int col_lo = (int)crank * per, col_hi = col_lo + per < cols ? col_lo + per : cols;
            const uint32_t part_local = smem_u32(part_sm);
            float4* red = reinterpret_cast<float4*>(scratch);  // [4 warps][32]
            __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.out) + ((int64_t)csg.b * p.Hq + csg.g * G) * D;
            auto remote = [&](int s_, int off_floats) {       // shared::cluster address of float `off` of partial s_
                uint32_t a;
                asm volatile("mapa.shared::cluster.u32 %0, %1, %2;"
                             : "=r"(a) : "r"(part_local + 4u * (uint32_t)((s_ % C::kGroups) * kPart + off_floats)), "r"((uint32_t)(s_ / C::kGroups)));
                return a;
            };
            constexpr int kMaxNp = kMaxCluster * C::kGroups;           // partials of the largest cluster
            constexpr int kMaxOwn = kMaxNp / kGroupWarps;     // ... of which a warp sums every fourth
            float* lse_all = scratch + 4 * kGroupThreads;     // [np][8], behind the reduction buffer
            // one round trip through the cluster: the lse values of all partials (staged in shared memory for everybody)
            // and, for the first pass of columns, the rows of the partials this warp sums
            for (int i = tid; i < np * kMaxGroup; i += kGroupThreads) {
                float x;
                asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(x) : "r"(remote(i / kMaxGroup, kMaxGroup * D + i % kMaxGroup)));
                lse_all[i] = x;
            }
            for (int c0 = col_lo; c0 < col_hi; c0 += 32) {
                const int col = c0 + lane;
                const bool act = col < col_hi;
                const int h = act ? col / kVec : 0;
                float4 v[kMaxOwn];
#pragma unroll
                for (int u = 0; u < kMaxOwn; ++u) {
                    const int s_ = warp + kGroupWarps * u;
                    v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (s_ < np && act)
                        asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];"
                                     : "=f"(v[u].x), "=f"(v[u].y), "=f"(v[u].z), "=f"(v[u].w) : "r"(remote(s_, col * 4)));
                }
                if (c0 == col_lo) group_barrier(grp);       // lse_all is in place
                // weights of head h: every thread computes them for its own column
                float M = -INFINITY, sum = 0.f;
                for (int s_ = 0; s_ < np; ++s_) M = fmaxf(M, lse_all[s_ * kMaxGroup + h]);
                for (int s_ = 0; s_ < np; ++s_) sum += M > -INFINITY ? __expf(lse_all[s_ * kMaxGroup + h] - M) : 0.f;
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int u = 0; u < kMaxOwn; ++u) {
                    const int s_ = warp + kGroupWarps * u;
                    const float w = (s_ < np && M > -INFINITY) ? __expf(lse_all[s_ * kMaxGroup + h] - M) : 0.f;
                    if (w > 0.f) {                           // an empty partial's rows were never written
                        acc.x = fmaf(w, v[u].x, acc.x); acc.y = fmaf(w, v[u].y, acc.y);
                        acc.z = fmaf(w, v[u].z, acc.z); acc.w = fmaf(w, v[u].w, acc.w);
                    }
                }
                red[warp * 32 + lane] = acc;
                group_barrier(grp);
                if (warp == 0 && act) {
                    float4 o4 = red[lane];
#pragma unroll
                    for (int w2 = 1; w2 < kGroupWarps; ++w2) {
                        const float4 y = red[w2 * 32 + lane];
                        o4.x += y.x; o4.y += y.y; o4.z += y.z; o4.w += y.w;
                    }
                    const float inv = sum > 0.f ? 1.f / sum : 0.f;
                    uint2 packed;
                    packed.x = pack_bf16x2(o4.x * inv, o4.y * inv);
                    packed.y = pack_bf16x2(o4.z * inv, o4.w * inv);
                    *reinterpret_cast<uint2*>(out + (int64_t)col * 4) = packed;
                    if (p.lse && col % kVec == 0) p.lse[(int64_t)csg.b * p.Hq + csg.g * G + h] = sum > 0.f ? M + __logf(sum) : -INFINITY;
                }
                group_barrier(grp);
            }
        }
        cluster_sync_all();                                   // nobody's shared memory goes away while it is being read
        // ---- the cluster that finishes last closes the launch (all others have read len[] for the last time)
        if (grp == 0) {
            if (tid == 0) {
                gints[0] = 0;
                if (crank == 0 && atomicAdd(p.segs_done, 1) + 1 == (int)(gridDim.x / csize)) {
                    *p.segs_done = 0;
                    gints[0] = 1;
                }
            }
            group_barrier(grp);
            if (gints[0] && p.k_new) {
                for (int b = tid; b < p.B; b += kGroupThreads) {
                    if (appends_to(p, b)) p.len[b] += 1;
                    else atomicCAS(p.status, 0, kErrBounds);      // append past S_cap: skipped and flagged
                }
            }
        }
        return;
    }
    // ---- the group that completed the launch's last segment closes the launch
    if (tid == 0) gints[0] = launch_last ? 1 : 0;
    group_barrier(grp);
    if (gints[0]) {
        if (tid == 0) {
            wait_word(p.grab_done, 0u, (uint32_t)Cg, p.spin_limit, abort_flag, p.status);   // nobody takes tiles or reads len[] any more
            *p.grab_done = 0;
        }
        group_barrier(grp);
        for (int c = tid; c < Cg; c += kGroupThreads) p.cur[c] = 0;
        const int other = (epoch & 1u) ? 0 : kMaxSegmentsPadded(p);
        int* dirty = p.status + 4;                                             // header ints [4], [5]
        const int nclear = dirty[(epoch & 1u) ^ 1u];                           // segments the other copy's last user touched
        group_barrier(grp);
        for (int sgi = tid; sgi < nclear; sgi += kGroupThreads) {              // the next launch's copy
            p.arrive[other + sgi] = 0ull; p.nparts[other + sgi] = 0; p.nthief[other + sgi] = 0;
        }
        if (tid == 0) { dirty[(epoch & 1u) ^ 1u] = 0; dirty[epoch & 1u] = nseg; }
        if (p.k_new) {
            for (int b = tid; b < p.B; b += kGroupThreads) {
                if (appends_to(p, b)) p.len[b] += 1;
                else atomicCAS(p.status, 0, kErrBounds);      // append past S_cap: skipped and flagged
            }
        }
    }
}

// ---- host side: launch ------------------------------------------------------------------------
template <int D, bool F8>
size_t partial_smem_bytes(int B, int stages) {
    using C = Cfg<D, F8>;
    return 1024 + (size_t)C::kFixedBytes + (size_t)stages * C::kStageBytes + (sizeof(int64_t) + sizeof(int)) * (B + 1) + 16;
}

template <int D, bool F8>
cudaError_t launch_fused(CUtensorMap& mk, CUtensorMap& mv, AttnParams& p, cudaStream_t st) {
    using C = Cfg<D, F8>;
    int stages = C::kMaxStages;                                  // as many as fit beside the batch-dependent tables
    while (stages > C::kGroups && partial_smem_bytes<D, F8>(p.B, stages) > 227 * 1024) stages -= C::kGroups;
    p.stages = stages;
    const size_t smem = partial_smem_bytes<D, F8>(p.B, stages);
    {
        static std::mutex mu;
        static bool attr_set[64] = {};      // per device: the opt-in to > 48 KB of dynamic shared memory
        int dev = 0;
        cudaGetDevice(&dev);
        std::lock_guard<std::mutex> lock(mu);
        if (dev < 0 || dev >= 64 || !attr_set[dev]) {
            cudaError_t e = cudaFuncSetAttribute(attn_fused_tma<D, F8, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
            if (e != cudaSuccess) return e;
            if (dev >= 0 && dev < 64) attr_set[dev] = true;
        }
    }
    void* args[] = {&mk, &mv, &p};
    // cooperative: the CTAs wait on one another in the combine, so they must all be resident
    return cudaLaunchCooperativeKernel(reinterpret_cast<void*>(attn_fused_tma<D, F8, false, false>), dim3(p.num_ctas), dim3(Cfg<D, F8>::kThreads), args, smem, st);
}

// ---- cluster form ----
// Stages of the cluster form: as many as fit beside the groups' partial buffers (the data comes from L2: depth matters less
// than in the streaming form).
template <int D, bool F8, bool ONE>
constexpr int cluster_stages() {
    using C = Cfg<D, F8, true, ONE>;
    int stages = C::kMaxStages;
    while (stages > C::kGroups &&
           1024 + C::kFixedBytes + stages * C::kStageBytes + (int)sizeof(float) * C::kGroups * (kMaxGroup * D + kMaxGroup) + 16 > 227 * 1024)
        stages -= C::kGroups;
    return stages;
}
template <int D, bool F8, bool ONE>
size_t cluster_smem_bytes() {
    using C = Cfg<D, F8, true, ONE>;
    return 1024 + (size_t)C::kFixedBytes + (size_t)cluster_stages<D, F8, ONE>() * C::kStageBytes +
           sizeof(float) * C::kGroups * (kMaxGroup * D + kMaxGroup) + 16;
}
static_assert(cluster_stages<256, false, false>() == 3 && cluster_stages<256, true, false>() >= 4 && cluster_stages<128, false, false>() >= 4 &&
              cluster_stages<128, true, false>() >= 4 && cluster_stages<128, false, true>() >= 4, "cluster form: stages that fit shared memory");

// One-time set-up per device: shared-memory opt-in, non-portable cluster sizes, and how many clusters of each size the
// device holds at once (index: log2 of the cluster size).
struct ClusterInfo { bool ready; int sms; int active[kMaxCluster + 1]; };   // active[c]: resident clusters of c CTAs
template <int D, bool F8, bool ONE>
cudaError_t cluster_info(const ClusterInfo** out) {
    static std::mutex mu;
    static ClusterInfo info[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (!info[dev].ready) {
        auto* fn = attn_fused_tma<D, F8, ONE, true>;
        cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (e != cudaSuccess) return e;
        if (cudaDeviceGetAttribute(&info[dev].sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) info[dev].sms = 0;
        for (int cl = 1; cl <= kMaxCluster; ++cl) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(cl); cfg.blockDim = dim3(Cfg<D, F8, true, ONE>::kThreads); cfg.dynamicSmemBytes = cluster_smem_bytes<D, F8, ONE>();
            cudaLaunchAttribute at[1];
            at[0].id = cudaLaunchAttributeClusterDimension;
            at[0].val.clusterDim.x = (unsigned)cl; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
            cfg.attrs = at; cfg.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, fn, &cfg) != cudaSuccess) { n = 0; (void)cudaGetLastError(); }
            info[dev].active[cl] = n;
        }
        info[dev].ready = true;
    }
    *out = &info[dev];
    return cudaSuccess;
}

template <int D, bool F8, bool ONE>
cudaError_t launch_cluster(CUtensorMap& mk, CUtensorMap& mv, AttnParams& p, cudaStream_t st) {
    using C = Cfg<D, F8, true, ONE>;
    if constexpr (ONE) {
        // this variant's own one-time set-up (the shared-memory and cluster-size opt-ins); its CTAs use no more shared
        // memory than the two-group variant's, whose resident-cluster counts chose the cluster size
        const ClusterInfo* unused = nullptr;
        if (cudaError_t e = cluster_info<D, F8, ONE>(&unused); e != cudaSuccess) return e;
    }
    p.stages = cluster_stages<D, F8, ONE>();
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.num_ctas); cfg.blockDim = dim3(C::kThreads); cfg.dynamicSmemBytes = cluster_smem_bytes<D, F8, ONE>(); cfg.stream = st;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)p.cluster; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    // may be set up while the previous kernel on the stream drains (the kernel waits before it touches global memory)
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, attn_fused_tma<D, F8, ONE, true>, mk, mv, p);
}

}  // namespace

int64_t attention_rows(const AttnParams& p) {
    if (p.mode == kPaged) return (int64_t)p.num_pages * p.Hkv * p.page_size;
    // p.B counts queries; the store holds p.B / q_len sequences. The extent must be exact: rows of the last tile that
    // lie beyond it are filled by TMA instead of being read from memory the caller may not own.
    return (int64_t)(p.B / (p.q_len > 1 ? p.q_len : 1)) * p.Hkv * p.rows_per_head;
}

cudaError_t make_attention_maps(const AttnParams& p, AttnMaps* maps) {
    const int64_t rows = attention_rows(p);
    const int esz = p.f8 ? 1 : 2;
    if (!make_map(&maps->k, p.k, rows, p.D, esz) || !make_map(&maps->v, p.v, rows, p.D, esz)) return cudaErrorInvalidValue;
    return cudaSuccess;
}

cudaError_t launch_attention(const AttnParams& p_in, const AttnMaps& maps, cudaStream_t st) {
    AttnParams p = p_in;
    CUtensorMap mk = maps.k, mv = maps.v;
    cudaError_t e;
    if (p.cluster > 0) {
        if (p.f8) e = p.D == 128 ? launch_cluster<128, true, false>(mk, mv, p, st) : launch_cluster<256, true, false>(mk, mv, p, st);
        else if (p.D == 256) e = launch_cluster<256, false, false>(mk, mv, p, st);
        else e = p.one_group ? launch_cluster<128, false, true>(mk, mv, p, st) : launch_cluster<128, false, false>(mk, mv, p, st);
    } else {
        if (p.f8) e = p.D == 128 ? launch_fused<128, true>(mk, mv, p, st) : launch_fused<256, true>(mk, mv, p, st);
        else e = p.D == 128 ? launch_fused<128, false>(mk, mv, p, st) : launch_fused<256, false>(mk, mv, p, st);
    }
    count_launch(1);
    return e;
}

// CTAs per cluster for a launch of `nseg` segments of at most `tiles` tiles each through the cluster form of the kernel,
// or 0 when the cooperative form should serve it: the largest power of two (at most 16, at most `max_ctas` CTAs in all
// when that is positive) whose clusters are all resident at once, as long as that leaves a CTA a handful of tiles.
int pick_cluster(int D, int f8, int nseg, int64_t tiles, int max_ctas, int* one_group) {
    *one_group = 0;
    const ClusterInfo* info = nullptr;
    cudaError_t e;
    if (f8) e = D == 128 ? cluster_info<128, true, false>(&info) : cluster_info<256, true, false>(&info);
    else e = D == 128 ? cluster_info<128, false, false>(&info) : cluster_info<256, false, false>(&info);
    if (e != cudaSuccess) { (void)cudaGetLastError(); return 0; }
    // the largest cluster all of whose copies are resident at once (a second wave of clusters would double the time)
    int best = 0;
    for (int cl = 1; cl <= kMaxCluster; ++cl) {
        if (info->active[cl] <= 0 || (cl > 1 && nseg > info->active[cl])) continue;
        if (cl > 1 && cl > tiles) break;
        if (max_ctas > 0 && (int64_t)nseg * cl > max_ctas && cl > 1) break;
        best = cl;
    }
    if (best == 0) return 0;
    // Which form is faster: a cluster CTA streams ceil(tiles / best) tiles of its segment, the cooperative form spreads
    // all tiles over every SM but pays a longer launch, a grid-wide combine and no overlap with the launch before it.
    // Measured per-tile times of one CTA reading through L2 and the difference of the fixed costs decide.
    const int64_t per_cta = (tiles + best - 1) / best;
    const int coop_ctas = max_ctas > 0 && max_ctas < info->sms ? max_ctas : info->sms;
    const int64_t per_coop = (tiles * nseg + coop_ctas - 1) / (coop_ctas > 0 ? coop_ctas : 1);
    const int tile_ns = f8 ? (D == 256 ? kTileNsF8D256 : kTileNsF8D128) : (D == 256 ? kTileNsD256 : kTileNsD128);
    if ((per_cta - per_coop) * tile_ns > kClusterFixedGainNs) return 0;
    // With a handful of tiles per CTA one consumer group is the faster arrangement for the 32 KB tiles of a bf16
    // head_dim-128 store too (one flush pass, half as many partials to merge); from six tiles on two groups win (measured on 1 to 16 rings of W = 2048 to 16384).
    *one_group = !f8 && D == 128 && per_cta <= kOneGroupMaxTiles;
    return best;
}

}  // namespace wmtp
