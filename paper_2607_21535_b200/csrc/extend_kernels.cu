// Shared-tile multi-query attention for the full-context draft-extend.
//
// After a verify step the draft re-processes the accepted tokens in one pass: q_len new tokens per sequence, each
// attending causally up to itself (Section 5, "The backend is not the confound"; Appendix B, per-kernel table: this
// is the step that costs the native draft a second full read of its KV). Query j of a sequence sees the keys below
// len - (q_len - 1 - j), so the q_len queries read the same K/V rows except for the last few. Here every K/V tile is
// brought from HBM once and consumed by all queries of a chunk of kQC = 4:
//
//   * a *stream* is (sequence, KV head, query chunk); streams are laid end to end as a line of 64-key tiles and
//     CTA c of C takes the range [c n / C, (c + 1) n / C) -- a fixed partition, no CTA waits for another, so the
//     launch is an ordinary one;
//   * a producer warp streams K tiles and V tiles through two rings of shared-memory slots with TMA (128-byte
//     swizzle, completion on mbarriers); the rings are released separately, K after the scores, V after the read-out;
//   * eight consumer warps in two groups share every tile: warp w takes the 16 keys (w mod 4) of the tile and the
//     two queries of its group (w / 4). Scores S^T[key, head] = K . Q^T go through mma.sync with keys on M and the
//     G <= 8 heads of one query on N = 8, one MMA per query for each K fragment loaded; the online softmax runs per
//     query in fp32; O^T += V^T . P^T likewise loads each V fragment once for both queries. G * q_len = 32 columns is
//     a real MMA tile, but still an order of magnitude below what tcgen05 is built for (M >= 64 rows of queries):
//     the bound stays HBM;
//   * a warp's work on consecutive tiles is software-pipelined: the score MMAs of tile t + 1, the softmax weights of
//     tile t + 1 and the read-out MMAs of tile t form one branch-free block (independent chains: the shuffles,
//     exponentials and transposes of the softmax overlap with the issue of the read-out MMAs), and the rescaling of the
//     accumulators, rare after the first tiles of a stream, is the only branch between blocks. With the three phases of
//     a tile back to back every warp spent most of a tile's time in its own dependent chain (measured per phase with
//     clock64: 790 cycles of softmax, 1800 of MMA blocks, 650 of waits and hand-over per 64-key tile, against 2730
//     cycles of HBM time per tile);
//   * the causal limit differs per query only in the last tile(s) of a stream, where rows are masked one by one;
//   * a CTA leaving a stream writes one normalised fp32 partial (+ lse) per query, at slot (CTA + stream): that
//     index is injective along the tile line and makes a stream's partials contiguous, so nothing is allocated by
//     an atomic; a second small kernel merges the partials by log-sum-exp (lse = logsumexp_s lse_s,
//     out = sum_s e^{lse_s - lse} o_s -> bf16).
//
// Sequences with more than kQC new tokens take ceil(q_len / kQC) passes over their K/V.
#include <mutex>
#include <type_traits>

#include "attn_plan.cuh"
#include "fp8_util.cuh"
#include "ptx_util.cuh"

namespace wmtp {

namespace {

constexpr float kLn2f = 0.6931471805599453f;
constexpr int kQC = kExtendChunk;          // queries that share one pass over the K/V of a sequence
constexpr int kMqGroups = 2;               // consumer groups: each takes half of the chunk's queries, on every tile
constexpr int kQW = kQC / kMqGroups;       // queries per consumer warp
constexpr int kMqWarps = 4;                // warps per group: 4 x 16 keys = one tile
constexpr int kMqGroupThreads = kMqWarps * 32;
constexpr int kCombineRows = 8;            // partials in flight per output column in the merge kernel

// D: head_dim; F8: the store holds e4m3 codes (one byte per entry) instead of bf16.
template <int D, bool F8>
struct MqCfg {
    static constexpr int kElemBytes = F8 ? 1 : 2;
    static constexpr int kChunks = D * kElemBytes / 128;       // 128-byte column chunks per row
    static constexpr int kChunkBytes = kTileKeys * 128;        // one TMA box: 64 rows x 128 B
    static constexpr int kTileBytes = kChunks * kChunkBytes;   // K (or V) tile
    static constexpr int kStageBytes = 2 * kTileBytes;
    static constexpr int kStages = 196608 / kStageBytes;       // 192 KB of tiles in flight per SM
    static constexpr int kKSteps = D / 16;
    static constexpr int kQRegs = D <= 128 ? kQW : 0;          // queries of a warp whose fragments live in registers
    static constexpr int kPassCols = 32;                       // columns of d merged per pass of a flush
    static constexpr int kScratchRow = kPassCols + 4;
    static constexpr int kScratchFloats = kMqWarps * kMaxGroup * kScratchRow;
    static constexpr int kStatFloats = kQW * 3 * kMqWarps * kMaxGroup;   // m, l, le per query, warp and head
    static constexpr int kQBytes = kQC * kKSteps * 32 * 8;     // query fragments, one uint2 per (query, k-step, lane)
    static constexpr int kBarriers = 4 * kStages;              // emptyK, emptyV, fullK, fullV
    // Nine warps would leave every thread 168 registers (three warps share one scheduler's register file) and the
    // consumers, with two queries' accumulators, need more. So the producer's warpgroup is filled up with three warps
    // that exit at once, drops to kRegsProducer registers and the consumers' two warpgroups rise to kRegsConsumer
    // (setmaxnreg is warpgroup-wide; 8 * 224 + 4 * 56 = 12 * 168, what the CTA was launched with).
    static constexpr int kPadWarps = 3;
    static constexpr int kRegsProducer = 56, kRegsConsumer = 224;
    static constexpr int kThreads = (kMqGroups * kMqWarps + 1 + kPadWarps) * 32;
    static constexpr int kFixedRaw = 4 * kMqGroups * (kScratchFloats + kStatFloats) + kQBytes + 8 * kBarriers + 8 * kStages + 16;
    static constexpr int kFixedBytes = (kFixedRaw + 1023) / 1024 * 1024;
};

// ---- the plan: streams and their tiles, from the device-resident lengths ------------------------------------
__device__ __forceinline__ int mq_chunks(const AttnParams& p) { return (p.q_len + kQC - 1) / kQC; }
// partial rows per (CTA, stream) slot
__device__ __forceinline__ int mq_slot_rows(const AttnParams& p) { return p.q_len < kQC ? p.q_len : kQC; }
// queries in chunk ch
__device__ __forceinline__ int mq_chunk_queries(const AttnParams& p, int ch) {
    const int left = p.q_len - ch * kQC;
    return left < kQC ? left : kQC;
}
// keys the last query of chunk ch of sequence b sees (the chunk's stream covers exactly these)
__device__ __forceinline__ int64_t mq_chunk_keys(const AttnParams& p, int b, int ch) {
    const int last = ch * kQC + mq_chunk_queries(p, ch) - 1;
    const int64_t S = p.len[b] - (p.q_len - 1 - last);
    return S > 0 ? S : 0;
}
__device__ __forceinline__ int64_t mq_chunk_tiles(const AttnParams& p, int b, int ch) {
    return (mq_chunk_keys(p, b, ch) + kTileKeys - 1) / kTileKeys;
}
// tiles of all chunks of sequence b, per KV head
__device__ __forceinline__ int64_t mq_seq_tiles(const AttnParams& p, int b) {
    int64_t t = 0;
    for (int ch = 0; ch < mq_chunks(p); ++ch) t += mq_chunk_tiles(p, b, ch);
    return t;
}
// CTA owning tile t under the fixed partition: the largest c with c n / C <= t
__device__ __forceinline__ int mq_owner(int64_t t, int64_t n, int C) { return (int)(((t + 1) * (int64_t)C - 1) / n); }

struct MqStream {
    int b, g, ch, nq, sidx;
    int64_t start, tiles, S_last;
};
// stream that holds global tile t; tile_prefix[b] = tiles (per KV head) of the sequences before b
__device__ __forceinline__ MqStream mq_locate(const AttnParams& p, const int64_t* tile_prefix, int64_t t) {
    MqStream s;
    s.b = find_seq(tile_prefix, p.B, p.Hkv, t);
    const int64_t Tb = tile_prefix[s.b + 1] - tile_prefix[s.b];
    const int64_t in_seq = t - (int64_t)p.Hkv * tile_prefix[s.b];
    s.g = (int)(in_seq / Tb);
    int64_t r = in_seq - (int64_t)s.g * Tb;
    int64_t start = (int64_t)p.Hkv * tile_prefix[s.b] + (int64_t)s.g * Tb;
    const int nch = mq_chunks(p);
    int ch = 0;
    int64_t tc = mq_chunk_tiles(p, s.b, 0);
    while (ch + 1 < nch && r >= tc) { r -= tc; start += tc; ++ch; tc = mq_chunk_tiles(p, s.b, ch); }
    s.ch = ch; s.tiles = tc; s.start = start;
    s.nq = mq_chunk_queries(p, ch);
    s.S_last = mq_chunk_keys(p, s.b, ch);
    s.sidx = (s.b * p.Hkv + s.g) * nch + ch;
    return s;
}

__device__ __forceinline__ void mq_group_barrier(int grp) { asm volatile("bar.sync %0, 128;" ::"r"(grp + 1) : "memory"); }

// ---------------------------------------------------------------------------------------------
// Partials: one launch, fixed partition, no inter-CTA wait
// ---------------------------------------------------------------------------------------------
template <int D, bool F8>
__global__ void __launch_bounds__(MqCfg<D, F8>::kThreads, 1)
attn_extend_mq(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV,
               const __grid_constant__ AttnParams p) {
    using C = MqCfg<D, F8>;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    float* scratch_all = reinterpret_cast<float*>(smem);                                   // [groups][kScratchFloats]
    float* stats_all = scratch_all + kMqGroups * C::kScratchFloats;                        // [groups][kQW][3][4][8]
    uint2* q_sm_all = reinterpret_cast<uint2*>(stats_all + kMqGroups * C::kStatFloats);    // [kQC][kKSteps][32]
    uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<unsigned char*>(q_sm_all) + C::kQBytes);
    int64_t* stage_tile = reinterpret_cast<int64_t*>(bars + C::kBarriers);                 // [kStages] global tile, -1 = end
    int* cta_flags = reinterpret_cast<int*>(stage_tile + C::kStages);                      // [0] abort
    unsigned char* stages = smem + C::kFixedBytes;
    int64_t* tile_prefix = reinterpret_cast<int64_t*>(stages + C::kStages * C::kStageBytes);   // [B + 1]
    volatile int* abort_flag = cta_flags;

    const int lane = threadIdx.x & 31, warp_id = threadIdx.x >> 5;
    const uint32_t bar_emptyK = smem_u32(bars), bar_emptyV = smem_u32(bars + C::kStages);
    const uint32_t bar_fullK = smem_u32(bars + 2 * C::kStages), bar_fullV = smem_u32(bars + 3 * C::kStages);
    if (threadIdx.x == kMqGroups * kMqGroupThreads) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&mapK) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&mapV) : "memory");
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < C::kStages; ++s) {
            mbar_init(bar_emptyK + 8 * s, kMqGroups * kMqWarps);      // every consumer warp releases every slot
            mbar_init(bar_emptyV + 8 * s, kMqGroups * kMqWarps);
            mbar_init(bar_fullK + 8 * s, 1);
            mbar_init(bar_fullV + 8 * s, 1);
        }
        cta_flags[0] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // the merge kernel that follows on the stream may be set up from now on (it waits for this grid before it reads)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    for (int b = threadIdx.x; b < p.B; b += blockDim.x) tile_prefix[b + 1] = mq_seq_tiles(p, b);
    if (threadIdx.x == 0) tile_prefix[0] = 0;
    __syncthreads();
    if (threadIdx.x < 32) warp_inclusive_scan(tile_prefix + 1, p.B);
    __syncthreads();
    const int64_t n = (int64_t)p.Hkv * tile_prefix[p.B];
    const int Cn = effective_ctas(gridDim.x, n);
    if ((int)blockIdx.x >= Cn) return;                       // no tile for this CTA (streams without tiles are the merge kernel's)
    const int64_t t_lo = cta_range_start(blockIdx.x, n, Cn), t_hi = cta_range_start(blockIdx.x + 1, n, Cn);
    const int G = p.G;

    if (warp_id >= kMqGroups * kMqWarps) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(C::kRegsProducer));
        if (warp_id > kMqGroups * kMqWarps) return;          // filler warps of the producer's warpgroup
        // =================================== producer warp ===================================
        const uint32_t stage0 = smem_u32(stages);
        uint32_t ps = 0, pph = 0;
        int64_t t = t_lo;
        while (t < t_hi) {
            const MqStream sg = mq_locate(p, tile_prefix, t);
            const int64_t s_end = sg.start + sg.tiles;
            const int64_t t_end = s_end < t_hi ? s_end : t_hi;
            const int64_t first_tile = t - sg.start;
            const int ntiles = (int)(t_end - t);
            for (int base = 0; base < ntiles; base += 32) {
                int page = 0;
                if (p.mode == kPaged && base + lane < ntiles) {
                    page = p.page_table[(int64_t)sg.b * p.max_pages + first_tile + base + lane];   // 64-key tile = page
                    if (page < 0 || page >= p.num_pages) { atomicCAS(p.status, 0, kErrBounds); page = 0; }
                }
                const int cnt = ntiles - base < 32 ? ntiles - base : 32;
                for (int j = 0; j < cnt; ++j, ps = (ps + 1 == (uint32_t)C::kStages ? 0 : ps + 1), pph ^= (ps == 0)) {
                    const int pg = __shfl_sync(0xffffffffu, page, j);
                    if (lane == 0) {
                        const uint32_t s = ps, ph = pph;
                        int64_t row;
                        if (p.mode == kPaged) row = ((int64_t)pg * p.Hkv + sg.g) * kTileKeys;
                        else row = ((int64_t)sg.b * p.Hkv + sg.g) * p.rows_per_head + (first_tile + base + j) * kTileKeys;
                        const uint32_t dstK = stage0 + s * C::kStageBytes, dstV = dstK + C::kTileBytes;
                        if (mbar_wait(bar_emptyK + 8 * s, ph ^ 1u, abort_flag, p.status)) {
                            stage_tile[s] = t + base + j;          // ordered before the consumers' wait by the arrive below
                            mbar_expect_tx(bar_fullK + 8 * s, C::kTileBytes);
                            tma_load_3d(dstK, &mapK, (int)row, bar_fullK + 8 * s);
                        }
                        if (mbar_wait(bar_emptyV + 8 * s, ph ^ 1u, abort_flag, p.status)) {
                            mbar_expect_tx(bar_fullV + 8 * s, C::kTileBytes);
                            tma_load_3d(dstV, &mapV, (int)row, bar_fullV + 8 * s);
                        }
                    }
                }
            }
            t = t_end;
        }
        if (lane == 0) {                                     // end marker (a K slot without a tile)
            mbar_wait(bar_emptyK + 8 * ps, pph ^ 1u, abort_flag, p.status);
            stage_tile[ps] = -1;
            mbar_arrive(bar_fullK + 8 * ps);
        }
        return;
    }

    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(C::kRegsConsumer));
    // ===================================== consumer warps =====================================
    const int grp = warp_id / kMqWarps, warp = warp_id % kMqWarps, tid = threadIdx.x % kMqGroupThreads;
    float* scratch = scratch_all + grp * C::kScratchFloats;
    float* stats = stats_all + grp * C::kStatFloats;                  // [kQW][3][4][8]
    uint2* q_sm = q_sm_all + (grp * kQW) * C::kKSteps * 32 + lane;    // this lane's column of the group's first query
    const int g8 = lane >> 2, t4 = lane & 3;
    const float scale = p.scale_log2;
    const int mi = lane >> 3, rr = lane & 7;
    const int rowK = warp * 16 + (mi & 1) * 8 + rr, halfK = mi >> 1;
    const int rowV = warp * 16 + (mi >> 1) * 8 + rr, halfV = mi & 1;
    // byte offset of this lane's ldmatrix row inside a tile, per 32-byte column pair i of a 128-byte chunk (128-byte swizzle)
    uint32_t koff[4], voff[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        koff[i] = rowK * 128 + (((uint32_t)(2 * i + halfK) ^ (uint32_t)rr) << 4);
        voff[i] = rowV * 128 + (((uint32_t)(2 * i + halfV) ^ (uint32_t)rr) << 4);
    }
    const uint32_t stage0 = smem_u32(stages);

    MqStream sg;
    sg.sidx = -1; sg.start = 0; sg.tiles = 0; sg.b = 0; sg.g = 0; sg.ch = 0; sg.nq = 0; sg.S_last = 0;
    int64_t Sq[kQW];                         // keys each of this warp's queries sees (0: no such query in the chunk)
    float m[kQW][2], le[kQW][2];          // running maxima (log2 units) and exact sums of weights
    float lacc[kQW][4];                   // sums of the rounded weights: [0], [1] = heads 2 t4, 2 t4 + 1 (the same in every lane group)
    float o[kQW][C::kKSteps][4];
    // Query fragments: in registers where they fit beside the accumulators (head_dim 128), else in shared memory, one
    // copy per group (head_dim 256: 64 registers of fragments next to 128 of accumulators spill, and keeping only one
    // query's fragments in registers measured no faster).
    uint32_t qreg[C::kQRegs > 0 ? C::kQRegs : 1][C::kKSteps][2];
    // multipliers of the raw scores of heads 2 t4 and 2 t4 + 1 of each query: the softmax scale in log2 units; for an fp8
    // store also the key scale of the KV head and the power of two the head's query was normalised by (all positive)
    float smul[kQW][2];
    float vscale = 1.f;                      // fp8: dequantisation scale of V, applied to the normalised partial
#pragma unroll
    for (int j = 0; j < kQW; ++j) { Sq[j] = 0; smul[j][0] = smul[j][1] = scale; }

    // Merge the four warps' states per query, write the partial of (this CTA, current stream, query).
    auto flush = [&]() {
        const int64_t slot = (int64_t)blockIdx.x + sg.sidx;
#pragma unroll
        for (int j = 0; j < kQW; ++j) {
            const int qi = grp * kQW + j;
            float* sm_m = stats + j * 3 * kMqWarps * kMaxGroup;
            float* sm_l = sm_m + kMqWarps * kMaxGroup;
            float* sm_le = sm_l + kMqWarps * kMaxGroup;
#pragma unroll
            for (int off = 4; off <= 16; off <<= 1) {
                le[j][0] += __shfl_xor_sync(0xffffffffu, le[j][0], off);
                le[j][1] += __shfl_xor_sync(0xffffffffu, le[j][1], off);
            }
            mq_group_barrier(grp);                             // scratch and statistics free
            if (g8 == 0) {
                sm_m[warp * kMaxGroup + 2 * t4] = m[j][0]; sm_m[warp * kMaxGroup + 2 * t4 + 1] = m[j][1];
                sm_l[warp * kMaxGroup + 2 * t4] = lacc[j][0]; sm_l[warp * kMaxGroup + 2 * t4 + 1] = lacc[j][1];
                sm_le[warp * kMaxGroup + 2 * t4] = le[j][0]; sm_le[warp * kMaxGroup + 2 * t4 + 1] = le[j][1];
            }
            mq_group_barrier(grp);
            if (qi >= sg.nq) continue;                         // uniform across the group: no such query in this chunk
            const int64_t prow = slot * mq_slot_rows(p) + qi;
            float f[2];
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                const int h = 2 * t4 + i;
                float M = -INFINITY;
#pragma unroll
                for (int w = 0; w < kMqWarps; ++w) M = fmaxf(M, sm_m[w * kMaxGroup + h]);
                float L = 0.f, Le = 0.f;
                if (M > -INFINITY) {
#pragma unroll
                    for (int w = 0; w < kMqWarps; ++w) {
                        const float e = ex2(sm_m[w * kMaxGroup + h] - M);
                        L += sm_l[w * kMaxGroup + h] * e;
                        Le += sm_le[w * kMaxGroup + h] * e;
                    }
                }
                f[i] = (L > 0.f && m[j][i] > -INFINITY) ? ex2(m[j][i] - M) / L * vscale : 0.f;
                if (warp == 0 && g8 == 0 && h < G) p.part_lse[prow * G + h] = Le > 0.f ? (M + lg2(Le)) * kLn2f : -INFINITY;
            }
            constexpr int kPasses = D / C::kPassCols;
#pragma unroll
            for (int pass = 0; pass < kPasses; ++pass) {
                if (pass > 0) mq_group_barrier(grp);
#pragma unroll
                for (int mbl = 0; mbl < C::kPassCols / 16; ++mbl) {
                    const int mb = pass * (C::kPassCols / 16) + mbl;
                    // accumulator rows g8 and g8 + 8 of block mb hold d = 16 mb + g8 and + 8 (bf16 store), or, for an fp8
                    // store whose V fragments come out of the transposed load with d pairs interleaved, d = 16 mb + 2 g8 and + 1
                    float* row0 = scratch + (warp * kMaxGroup + 2 * t4) * C::kScratchRow + mbl * 16 + (F8 ? 2 * g8 : g8);
                    float* row1 = row0 + C::kScratchRow;
                    constexpr int kSecond = F8 ? 1 : 8;
                    row0[0] = o[j][mb][0] * f[0]; row1[0] = o[j][mb][1] * f[1];
                    row0[kSecond] = o[j][mb][2] * f[0]; row1[kSecond] = o[j][mb][3] * f[1];
                }
                mq_group_barrier(grp);
                for (int idx = tid; idx < G * C::kPassCols; idx += kMqGroupThreads) {
                    const int h = idx / C::kPassCols, dd = idx % C::kPassCols;
                    float acc = 0.f;
#pragma unroll
                    for (int w = 0; w < kMqWarps; ++w) acc += scratch[(w * kMaxGroup + h) * C::kScratchRow + dd];
                    p.part_o[(prow * G + h) * D + pass * C::kPassCols + dd] = acc;
                }
            }
        }
    };

    // Start work on the stream that holds tile tt: per-query limits, query fragments, fresh state.
    auto enter = [&](int64_t tt) {
        sg = mq_locate(p, tile_prefix, tt);
        mq_group_barrier(grp);                                 // no warp of the group still reads the previous fragments
#pragma unroll
        for (int j = 0; j < kQW; ++j) {
            const int qi = grp * kQW + j;
            Sq[j] = qi < sg.nq ? sg.S_last - (sg.nq - 1 - qi) : 0;
            if (Sq[j] < 0) Sq[j] = 0;
            // Q^T fragments (B operand: k = d, n = head) of query ch * kQC + qi; heads >= G and absent queries read as zero
            const bool have = qi < sg.nq && g8 < G;
            const uint32_t* qrow = reinterpret_cast<const uint32_t*>(
                reinterpret_cast<const __nv_bfloat16*>(p.q) +
                ((((int64_t)sg.b * p.q_len + sg.ch * kQC + (qi < sg.nq ? qi : 0)) * p.Hq) + sg.g * G + (g8 < G ? g8 : 0)) * D);
            // Words of the query row that make up this lane's fragment of 16-column step ks: ks * 8 + w0 and ks * 8 + w1.
            // For an fp8 store the MMA k-slot order within 16 columns of d follows the byte order ldmatrix delivers the
            // codes in: lane t4 holds d = 4 t4 .. 4 t4 + 3 of each 16.
            const int w0 = F8 ? 2 * t4 : t4, w1 = F8 ? 2 * t4 + 1 : 4 + t4;
            float down = 1.f;
            if constexpr (F8) {
                // The e4m3 codes are widened to f16 (exact), so the query goes through the f16 MMA too. Its range is made
                // safe by a per-head power of two (exact both ways): q' = q * 2^-e with 2^e <= max|q| < 2^(e+1), and 2^e
                // goes into the score multiplier together with the key scale.
                float amax = 0.f;
#pragma unroll
                for (int ks = 0; ks < C::kKSteps; ++ks) {
                    const uint32_t a = have ? __ldg(qrow + ks * 8 + w0) : 0u, b = have ? __ldg(qrow + ks * 8 + w1) : 0u;
                    amax = fmaxf(fmaxf(amax, fmaxf(fabsf(bf16lo(a)), fabsf(bf16hi(a)))), fmaxf(fabsf(bf16lo(b)), fabsf(bf16hi(b))));
                }
                amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
                amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
                uint32_t eb = (__float_as_uint(amax) >> 23) & 0xffu;
                eb = eb < 1u ? 1u : (eb > 253u ? 253u : eb);
                down = __uint_as_float((254u - eb) << 23);
                const float hmul = g8 < G ? scale * __uint_as_float(eb << 23) * __ldg(p.k_scale + sg.g) : 0.f;
                smul[j][0] = __shfl_sync(0xffffffffu, hmul, 8 * t4);
                smul[j][1] = __shfl_sync(0xffffffffu, hmul, 8 * t4 + 4);
                vscale = __ldg(p.v_scale + sg.g);
            }
            auto fragment = [&](int ks) {
                uint2 f;
                f.x = have ? __ldg(qrow + ks * 8 + w0) : 0u;
                f.y = have ? __ldg(qrow + ks * 8 + w1) : 0u;
                if constexpr (F8) {
                    f.x = pack_f16x2(bf16lo(f.x) * down, bf16hi(f.x) * down);
                    f.y = pack_f16x2(bf16lo(f.y) * down, bf16hi(f.y) * down);
                }
                return f;
            };
            if (j < C::kQRegs) {
#pragma unroll
                for (int ks = 0; ks < C::kKSteps; ++ks) {
                    const uint2 f = fragment(ks);
                    qreg[j < C::kQRegs ? j : 0][ks][0] = f.x;
                    qreg[j < C::kQRegs ? j : 0][ks][1] = f.y;
                }
            } else {
                for (int ks = warp; ks < C::kKSteps; ks += kMqWarps) q_sm[(j * C::kKSteps + ks) * 32] = fragment(ks);
            }
            m[j][0] = m[j][1] = -INFINITY; le[j][0] = le[j][1] = 0.f;
            lacc[j][0] = lacc[j][1] = lacc[j][2] = lacc[j][3] = 0.f;
#pragma unroll
            for (int mb = 0; mb < C::kKSteps; ++mb) { o[j][mb][0] = o[j][mb][1] = o[j][mb][2] = o[j][mb][3] = 0.f; }
        }
        mq_group_barrier(grp);
    };

    // Scores of the tile in K slot sK for this warp's 16 keys (scaled, not yet masked) and / or the read-out product of
    // the tile in V slot sV with the weights pb: S^T = K . Q^T and O^T += V^T . P^T, every fragment used for both
    // queries. Both at once is the steady state: two independent instruction streams, interleaved step by step.
    auto qk_pv = [&](auto do_qk, uint32_t sK, float (&scn)[kQW][4], auto do_pv, uint32_t sV, const uint32_t (&pb)[kQW][2]) {
        constexpr bool kQK = decltype(do_qk)::value, kPV = decltype(do_pv)::value;
        float sd[kQW][4];                    // second accumulator chain per query: a dependent MMA costs its full latency
        if constexpr (kQK) {
#pragma unroll
            for (int j = 0; j < kQW; ++j) {
                scn[j][0] = scn[j][1] = scn[j][2] = scn[j][3] = 0.f;
                sd[j][0] = sd[j][1] = sd[j][2] = sd[j][3] = 0.f;
            }
        }
        auto qfrag = [&](int j, int ks, uint32_t& q0, uint32_t& q1) {
            if (j < C::kQRegs) { q0 = qreg[j < C::kQRegs ? j : 0][ks][0]; q1 = qreg[j < C::kQRegs ? j : 0][ks][1]; }
            else { const uint2 f = q_sm[(j * C::kKSteps + ks) * 32]; q0 = f.x; q1 = f.y; }
        };
        if constexpr (!F8) {
#pragma unroll
            for (int ks = 0; ks < C::kKSteps; ++ks) {
                if constexpr (kQK) {
                    uint32_t a[4];
                    ldmatrix_x4(a, sK + (ks >> 2) * C::kChunkBytes + koff[ks & 3]);
#pragma unroll
                    for (int j = 0; j < kQW; ++j) {
                        uint32_t q0, q1;
                        qfrag(j, ks, q0, q1);
                        if (ks & 1) mma_bf16(sd[j], a, q0, q1);
                        else mma_bf16(scn[j], a, q0, q1);
                    }
                }
                if constexpr (kPV) {
                    uint32_t a[4];
                    ldmatrix_x4_trans(a, sV + (ks >> 2) * C::kChunkBytes + voff[ks & 3]);
#pragma unroll
                    for (int j = 0; j < kQW; ++j) mma_bf16(o[j][ks], a, pb[j][0], pb[j][1]);
                }
            }
        } else {
            // e4m3 codes: one ldmatrix brings 32 columns of d for the warp's 16 keys; a thread's word holds 4 consecutive
            // codes of one key (K) or, from the transposed load, the codes of two keys for two consecutive d (V, after one
            // byte permute). They are widened to f16 (exact) four at a time and take the f16 MMA; the query fragments are
            // stored in the matching k-slot order, the accumulator rows of the read-out come out with d pairs interleaved.
#pragma unroll
            for (int jj = 0; jj < C::kKSteps / 2; ++jj) {
                if constexpr (kQK) {
                    uint32_t r[4], a[4];
                    ldmatrix_x4(r, sK + (jj >> 2) * C::kChunkBytes + koff[jj & 3]);
                    e4m3x4_to_f16x2x2(r[0], a[0], a[2]);
                    e4m3x4_to_f16x2x2(r[1], a[1], a[3]);
#pragma unroll
                    for (int j = 0; j < kQW; ++j) {
                        uint32_t q0, q1;
                        qfrag(j, 2 * jj, q0, q1);
                        mma_f16(scn[j], a, q0, q1);
                    }
                    e4m3x4_to_f16x2x2(r[2], a[0], a[2]);
                    e4m3x4_to_f16x2x2(r[3], a[1], a[3]);
#pragma unroll
                    for (int j = 0; j < kQW; ++j) {
                        uint32_t q0, q1;
                        qfrag(j, 2 * jj + 1, q0, q1);
                        mma_f16(sd[j], a, q0, q1);
                    }
                }
                if constexpr (kPV) {
                    uint32_t r[4], a[4];
                    ldmatrix_x4_trans(r, sV + (jj >> 2) * C::kChunkBytes + koff[jj & 3]);
                    e4m3x4_to_f16x2x2(__byte_perm(r[0], 0, 0x3120), a[0], a[1]);
                    e4m3x4_to_f16x2x2(__byte_perm(r[1], 0, 0x3120), a[2], a[3]);
#pragma unroll
                    for (int j = 0; j < kQW; ++j) mma_f16(o[j][2 * jj], a, pb[j][0], pb[j][1]);
                    e4m3x4_to_f16x2x2(__byte_perm(r[2], 0, 0x3120), a[0], a[1]);
                    e4m3x4_to_f16x2x2(__byte_perm(r[3], 0, 0x3120), a[2], a[3]);
#pragma unroll
                    for (int j = 0; j < kQW; ++j) mma_f16(o[j][2 * jj + 1], a, pb[j][0], pb[j][1]);
                }
            }
        }
        if constexpr (kPV) {
            // the normaliser: sums of the rounded weights, as one more row block of the product (V^T = all ones)
            constexpr uint32_t kOne = F8 ? 0x3c003c00u : 0x3f803f80u;      // 1.0 twice, in the weights' format
            const uint32_t ones[4] = {kOne, kOne, kOne, kOne};
#pragma unroll
            for (int j = 0; j < kQW; ++j) {
                if constexpr (F8) mma_f16(lacc[j], ones, pb[j][0], pb[j][1]);
                else mma_bf16(lacc[j], ones, pb[j][0], pb[j][1]);
            }
        }
        if constexpr (kQK) {
#pragma unroll
            for (int j = 0; j < kQW; ++j) {
#pragma unroll
                for (int i = 0; i < 4; ++i) scn[j][i] += sd[j][i];     // raw scores: the softmax scale is applied in the exponent
            }
        }
    };
    using Yes = std::true_type;
    using No = std::false_type;

    // Online softmax of the tile whose scores are in sc (first row key0): masks, running maxima and sums, rescaled
    // accumulators, and the weights as B operand of the read-out product.
    // Online softmax of a tile, in two parts. weights(): from the raw scores sc of the tile whose first row is key0, the
    // candidate maxima mn, the weights as B operand of the read-out product (pbn) and their exact sums (psum); it reads
    // nothing the read-out MMAs write and has no branch, so it can sit in one block with them and its dependent chains
    // (shuffles, exponentials, transposes) overlap with their issue. settle(): adopts the maxima, rescaling the
    // accumulators when some maximum moved (rare after the first tiles of a stream), and adds the sums.
    float mn[kQW][2], psum[kQW][2];
    auto weights = [&](float (&sc)[kQW][4], int key0, uint32_t (&pbn)[kQW][2]) {
        const int ka = key0 + warp * 16 + g8, kb = ka + 8;
        // this thread holds heads 2*t4, 2*t4+1 for keys g8 and g8+8; sc are raw scores, m is kept in scaled (log2) units
#pragma unroll
        for (int j = 0; j < kQW; ++j) {
            // the causal limit of query j: only the last tile(s) of a stream have rows beyond it
            if (ka >= Sq[j]) { sc[j][0] = -INFINITY; sc[j][1] = -INFINITY; }
            if (kb >= Sq[j]) { sc[j][2] = -INFINITY; sc[j][3] = -INFINITY; }
            float mx0 = fmaxf(sc[j][0], sc[j][2]), mx1 = fmaxf(sc[j][1], sc[j][3]);
#pragma unroll
            for (int off = 4; off <= 16; off <<= 1) {
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
            }
            mn[j][0] = fmaxf(m[j][0], mx0 * smul[j][0]); mn[j][1] = fmaxf(m[j][1], mx1 * smul[j][1]);
            const float nu0 = mn[j][0] == -INFINITY ? 0.f : -mn[j][0], nu1 = mn[j][1] == -INFINITY ? 0.f : -mn[j][1];
            const float p0 = ex2(fmaf(sc[j][0], smul[j][0], nu0)), p1 = ex2(fmaf(sc[j][1], smul[j][1], nu1));
            const float p2 = ex2(fmaf(sc[j][2], smul[j][0], nu0)), p3 = ex2(fmaf(sc[j][3], smul[j][1], nu1));
            const uint32_t pa = F8 ? pack_f16x2(p0, p1) : pack_bf16x2(p0, p1);             // key g8   : heads 2t4, 2t4+1
            const uint32_t pc = F8 ? pack_f16x2(p2, p3) : pack_bf16x2(p2, p3);             // key g8+8
            psum[j][0] = p0 + p2;                                  // exact weights: the lse
            psum[j][1] = p1 + p3;
            pbn[j][0] = movmatrix_trans(pa);                       // P^T as B operand: k = key, n = head
            pbn[j][1] = movmatrix_trans(pc);
        }
    };
    auto settle = [&]() {
        bool moved = false;
#pragma unroll
        for (int j = 0; j < kQW; ++j) moved = moved || mn[j][0] != m[j][0] || mn[j][1] != m[j][1];
        if (__builtin_expect(__any_sync(0xffffffffu, moved), 0)) {
#pragma unroll
            for (int j = 0; j < kQW; ++j) {
                const float corr0 = mn[j][0] == -INFINITY ? 1.f : ex2(m[j][0] - mn[j][0]);
                const float corr1 = mn[j][1] == -INFINITY ? 1.f : ex2(m[j][1] - mn[j][1]);
                le[j][0] *= corr0; le[j][1] *= corr1;
                lacc[j][0] *= corr0; lacc[j][1] *= corr1; lacc[j][2] *= corr0; lacc[j][3] *= corr1;
#pragma unroll
                for (int mb = 0; mb < C::kKSteps; ++mb) {
                    o[j][mb][0] *= corr0; o[j][mb][1] *= corr1; o[j][mb][2] *= corr0; o[j][mb][3] *= corr1;
                }
                m[j][0] = mn[j][0]; m[j][1] = mn[j][1];
            }
        }
#pragma unroll
        for (int j = 0; j < kQW; ++j) { le[j][0] += psum[j][0]; le[j][1] += psum[j][1]; }
    };
    // does this warp's slab of the tile hold a key that counts for one of its queries?
    auto slab_valid = [&](int64_t t) {
        const int64_t Smax = Sq[kQW - 1] > Sq[0] ? Sq[kQW - 1] : Sq[0];       // later queries see more keys
        return (t - sg.start) * kTileKeys + warp * 16 < Smax;
    };

    // Tile number i of this CTA uses slot i mod kStages of both rings; (cs, cph) is the slot and use parity of the tile
    // in hand, whose weights are already in pb. One iteration: the scores and weights of the next tile together with the
    // read-out of the tile in hand.
    uint32_t cs = 0, cph = 0;
    float scn[kQW][4];
    uint32_t pb[kQW][2], pbn[kQW][2];
#pragma unroll
    for (int j = 0; j < kQW; ++j) { pb[j][0] = pb[j][1] = 0u; pbn[j][0] = pbn[j][1] = 0u; }
    const bool first_landed = mbar_wait(bar_fullK, 0u, abort_flag, p.status);
    int64_t tt = *reinterpret_cast<volatile int64_t*>(stage_tile);
    if (tt >= 0 && first_landed) {
        enter(tt);
        bool valid_c = slab_valid(tt);
        if (valid_c) {
            qk_pv(Yes{}, stage0, scn, No{}, 0u, pb);
            weights(scn, (int)(tt - sg.start) * kTileKeys, pb);
            settle();
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_emptyK);
        for (;;) {
            const int key0 = (int)(tt - sg.start) * kTileKeys;           // first row of the tile in hand within the sequence
            // ---- the next tile's K slot: same stream?
            const uint32_t ns = cs + 1 == (uint32_t)C::kStages ? 0u : cs + 1, nph = ns == 0 ? cph ^ 1u : cph;
            const bool landed = mbar_wait(bar_fullK + 8 * ns, nph, abort_flag, p.status);
            const int64_t tn = *reinterpret_cast<volatile int64_t*>(stage_tile + ns);
            const bool end = tn < 0 || !landed;
            const bool same = !end && tn >= sg.start && tn < sg.start + sg.tiles;
            bool valid_n = same && slab_valid(tn);
            const int key0n = (int)(tn - sg.start) * kTileKeys;
            const uint32_t sKn = stage0 + ns * C::kStageBytes, sV = stage0 + cs * C::kStageBytes + C::kTileBytes;
            mbar_wait(bar_fullV + 8 * cs, cph, abort_flag, p.status);
            if (__builtin_expect(valid_c && key0 + warp * 16 + 16 > sg.S_last, 0)) {
                // rows past the end of the sequence were never written: they can hold NaN/Inf bit patterns, and 0 * NaN
                // would poison the accumulators. Zero them in shared memory (the other group's warp on the same keys
                // writes the same zeros).
                const int wkey0 = key0 + warp * 16;
                const int first_bad = sg.S_last > wkey0 ? (int)(sg.S_last - wkey0) : 0;
                for (int idx = lane; idx < (16 - first_bad) * C::kChunks * 8; idx += 32) {
                    const int r = first_bad + idx / (C::kChunks * 8), rem = idx % (C::kChunks * 8);
                    const uint32_t addr = sV + (rem >> 3) * C::kChunkBytes + (warp * 16 + r) * 128 + ((rem & 7) << 4);
                    asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(addr), "r"(0u) : "memory");
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
            }
            if (__builtin_expect(valid_c && valid_n, 1)) { qk_pv(Yes{}, sKn, scn, Yes{}, sV, pb); weights(scn, key0n, pbn); }
            else if (valid_c) qk_pv(No{}, 0u, scn, Yes{}, sV, pb);
            else if (valid_n) { qk_pv(Yes{}, sKn, scn, No{}, 0u, pb); weights(scn, key0n, pbn); }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_emptyV + 8 * cs);
            if (__builtin_expect(!same, 0)) {
                flush();
                if (end) break;
                enter(tn);
                valid_n = slab_valid(tn);
                if (valid_n) { qk_pv(Yes{}, sKn, scn, No{}, 0u, pb); weights(scn, (int)(tn - sg.start) * kTileKeys, pbn); }
                __syncwarp();
            }
            if (lane == 0) mbar_arrive(bar_emptyK + 8 * ns);
            if (valid_n) settle();
#pragma unroll
            for (int j = 0; j < kQW; ++j) { pb[j][0] = pbn[j][0]; pb[j][1] = pbn[j][1]; }
            tt = tn; valid_c = valid_n; cs = ns; cph = nph;
        }
    }
    // a CTA that gave up on a barrier waits (bounded) for the copies that may still be in flight into its slots
    if (*abort_flag == kAbortBarrier && threadIdx.x == 0) {
        for (uint32_t s2 = 0; s2 < (uint32_t)C::kStages; ++s2) {
            for (uint32_t par = 0; par < 2; ++par) {
                for (uint32_t i = 0; i < kDrainLimit && !mbar_test_wait(bar_fullK + 8 * s2, par); ++i) { }
                for (uint32_t i = 0; i < kDrainLimit && !mbar_test_wait(bar_fullV + 8 * s2, par); ++i) { }
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Merge: one block per output row (sequence, new token, query head); D / 4 columns x kCombineRows partials in flight
// ---------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(D / 4 * kCombineRows)
extend_mq_combine(const AttnParams p) {
    constexpr int kCols = D / 4;
    __shared__ float w_sm[kMaxCtas];
    __shared__ float4 red[kCols * kCombineRows];
    __shared__ long long sums[2];                           // tiles (per KV head) before this sequence, and of all sequences
    __shared__ float inv_sm;
    const int tid = threadIdx.x;
    const int row = blockIdx.x;
    const int hq = row % p.Hq, jq = (row / p.Hq) % p.q_len, b = row / (p.Hq * p.q_len);
    const int G = p.G, g = hq / G, h = hq % G;
    const int ch = jq / kQC, qi = jq % kQC, nch = mq_chunks(p);
    if (tid < 2) sums[tid] = 0;
    // launched as a programmatic dependent of the partials kernel: nothing of global memory is read before that grid
    // has completed and its partials are visible
    asm volatile("griddepcontrol.wait;" ::: "memory");
    __syncthreads();
    {
        long long before = 0, all = 0;
        for (int b2 = tid; b2 < p.B; b2 += blockDim.x) {
            const long long t = mq_seq_tiles(p, b2);
            all += t;
            if (b2 < b) before += t;
        }
        if (before) atomicAdd(reinterpret_cast<unsigned long long*>(&sums[0]), (unsigned long long)before);
        if (all) atomicAdd(reinterpret_cast<unsigned long long*>(&sums[1]), (unsigned long long)all);
    }
    __syncthreads();
    const int64_t n = (int64_t)p.Hkv * sums[1];
    int64_t start = (int64_t)p.Hkv * sums[0] + (int64_t)g * mq_seq_tiles(p, b);
    for (int c2 = 0; c2 < ch; ++c2) start += mq_chunk_tiles(p, b, c2);
    const int64_t tiles = mq_chunk_tiles(p, b, ch);
    __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.out) + (int64_t)row * D;
    if (tiles == 0) {                                        // the query sees no key: out = 0, lse = -inf
        if (tid < kCols) *reinterpret_cast<uint2*>(out + 4 * tid) = make_uint2(0u, 0u);
        if (tid == 0 && p.lse) p.lse[row] = -INFINITY;
        return;
    }
    const int Cn = effective_ctas(p.num_ctas, n);
    const int c0 = mq_owner(start, n, Cn), c1 = mq_owner(start + tiles - 1, n, Cn);
    const int np = c1 - c0 + 1;
    const int sidx = (b * p.Hkv + g) * nch + ch;
    const int kq = mq_slot_rows(p);
    const int64_t prow0 = ((int64_t)c0 + sidx) * kq + qi;    // partial i of this row: prow0 + i * kq
    // ---- weights: exp(lse_i - max), by the first warp
    if (tid < 32) {
        float M = -INFINITY;
        for (int i = tid; i < np; i += 32) {
            const float x = __ldcg(p.part_lse + (prow0 + (int64_t)i * kq) * G + h);
            w_sm[i] = x;
            M = fmaxf(M, x);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
        float sum = 0.f;
        for (int i = tid; i < np; i += 32) {
            const float w = M > -INFINITY ? __expf(w_sm[i] - M) : 0.f;
            w_sm[i] = w;
            sum += w;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
        if (tid == 0) {
            inv_sm = sum > 0.f ? 1.f / sum : 0.f;
            if (p.lse) p.lse[row] = sum > 0.f ? M + __logf(sum) : -INFINITY;
        }
    }
    __syncthreads();
    const int col = tid % kCols, r = tid / kCols;
    const float4* rows = reinterpret_cast<const float4*>(p.part_o);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
    for (int i = r; i < np; i += kCombineRows) {
        const float w = w_sm[i];
        const float4 x = __ldcg(rows + ((prow0 + (int64_t)i * kq) * G + h) * kCols + col);
        acc.x = fmaf(w, x.x, acc.x); acc.y = fmaf(w, x.y, acc.y); acc.z = fmaf(w, x.z, acc.z); acc.w = fmaf(w, x.w, acc.w);
    }
    red[tid] = acc;
    __syncthreads();
    if (tid < kCols) {
        float4 o = red[tid];
#pragma unroll
        for (int r2 = 1; r2 < kCombineRows; ++r2) {
            const float4 x = red[r2 * kCols + tid];
            o.x += x.x; o.y += x.y; o.z += x.z; o.w += x.w;
        }
        const float inv = inv_sm;
        uint2 packed;
        packed.x = pack_bf16x2(o.x * inv, o.y * inv);
        packed.y = pack_bf16x2(o.z * inv, o.w * inv);
        *reinterpret_cast<uint2*>(out + 4 * tid) = packed;
    }
}

template <int D, bool F8>
size_t mq_smem_bytes(int B) {
    using C = MqCfg<D, F8>;
    return 1024 + (size_t)C::kFixedBytes + (size_t)C::kStages * C::kStageBytes + sizeof(int64_t) * (B + 1) + 16;
}

template <int D, bool F8>
cudaError_t launch_mq(CUtensorMap& mk, CUtensorMap& mv, AttnParams& p, cudaStream_t st) {
    const size_t smem = mq_smem_bytes<D, F8>(p.B);
    {
        static std::mutex mu;
        static bool attr_set[64] = {};      // per device: the opt-in to > 48 KB of dynamic shared memory
        int dev = 0;
        cudaGetDevice(&dev);
        std::lock_guard<std::mutex> lock(mu);
        if (dev < 0 || dev >= 64 || !attr_set[dev]) {
            cudaError_t e = cudaFuncSetAttribute(attn_extend_mq<D, F8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
            if (e != cudaSuccess) return e;
            if (dev >= 0 && dev < 64) attr_set[dev] = true;
        }
    }
    attn_extend_mq<D, F8><<<p.num_ctas, MqCfg<D, F8>::kThreads, smem, st>>>(mk, mv, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.B * p.q_len * p.Hq); cfg.blockDim = dim3(D / 4 * kCombineRows); cfg.dynamicSmemBytes = 0; cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, extend_mq_combine<D>, p);
}

}  // namespace

bool extend_mq_fits(int B, int D, int f8) {
    const size_t need = f8 ? (D == 128 ? mq_smem_bytes<128, true>(B) : mq_smem_bytes<256, true>(B))
                           : (D == 128 ? mq_smem_bytes<128, false>(B) : mq_smem_bytes<256, false>(B));
    return need <= 227 * 1024;
}

cudaError_t launch_extend_mq(const AttnParams& p_in, cudaStream_t st) {
    AttnParams p = p_in;
    const int64_t rows = p.mode == kPaged ? (int64_t)p.num_pages * p.Hkv * p.page_size : (int64_t)p.B * p.Hkv * p.rows_per_head;
    CUtensorMap mk, mv;
    const int esz = p.f8 ? 1 : 2;
    if (!make_map(&mk, p.k, rows, p.D, esz) || !make_map(&mv, p.v, rows, p.D, esz)) return cudaErrorInvalidValue;
    cudaError_t e;
    if (p.f8) e = p.D == 128 ? launch_mq<128, true>(mk, mv, p, st) : launch_mq<256, true>(mk, mv, p, st);
    else e = p.D == 128 ? launch_mq<128, false>(mk, mv, p, st) : launch_mq<256, false>(mk, mv, p, st);
    count_launch(2);
    return e;
}

}  // namespace wmtp
