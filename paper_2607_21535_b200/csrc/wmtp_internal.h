// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/wmtp.h"

namespace wmtp {

constexpr int kTileKeys = 64;       // keys per K/V tile; equals the page size of the paged layout
constexpr int kMaxCtas = 160;       // upper bound on attention CTAs (one per SM; a B200 has 148)
constexpr int kStealSlotsMax = 16;   // thieves a segment admits from other segments (fewer when there are many segments)
constexpr int kMaxGroups = 2;        // consumer groups per CTA (each contributes its own partial)
constexpr int kMaxBatch = 1024;     // sequences per call (prefix table lives in shared memory)
constexpr int kMaxGroup = 8;        // query heads per KV head
constexpr int kMaxSegments = 16384; // batch * Hkv per call
constexpr int kMaxCluster = 16;                                  // CTAs in a thread-block cluster (the non-portable limit)
// Choice between the cluster form and the cooperative form of a windowed launch: time one CTA takes per 64-key tile (ns,
// measured with the ring in L2) and what the cluster form saves in fixed cost (launch overlap, no grid-wide combine).
constexpr int kTileNsD256 = 1000, kTileNsD128 = 500, kTileNsF8D256 = 800, kTileNsF8D128 = 450;
constexpr int kClusterFixedGainNs = 5500;
constexpr int kOneGroupMaxTiles = 5;   // tiles per CTA up to which the one-group cluster variant is used (bf16, head_dim 128)
constexpr int kExtendChunk = 4;     // new tokens of a sequence whose queries share one pass over its K/V (draft-extend)
constexpr size_t kCursorBytes = 1024;                                          // int cur[kMaxCtas], padded
constexpr size_t kWorkspaceZeroBytes = 256 + kCursorBytes + 2 * (8 + 4 + 4) * kMaxSegments;   // header + cursors + two copies of the per-segment words

enum KvMode : int { kContiguous = 0, kPaged = 1, kRing = 2 };

// Workspace layout (all offsets from a 256-byte aligned base):
//   [0, 256)            header: int status @0, uint epoch @4, int segs_done @8, int grab_done @12, int dirty[2] @16
//                       (segments whose per-segment words each copy may hold non-zero), diagnostic record @32
//   [256, 1280)         int cur[kMaxCtas]: per-CTA cursors of the work-stealing scheme
//   counters            u64 arrive[2][kMaxSegments], int nparts[2][..], int nthief[2][..]
//                       (fixed size: initialisation needs no shape)
//   part_key            int   [slots]           slots = pool_slots(batch * Hkv)
//   part_lse            float [slots][G]
//   part_o              float [slots][G][D]
struct WorkspaceLayout {
    size_t counters_off, part_key_off, part_lse_off, part_o_off, total;
};
WorkspaceLayout workspace_layout(int batch, int Hq, int Hkv, int D);
// kStealSlotsMax for few segments, fewer as batch * Hkv grows
__host__ __device__ inline int steal_slots_for(int nseg) {
    const int x = 512 / (nseg < 1 ? 1 : nseg);
    return x > kStealSlotsMax ? kStealSlotsMax : x;
}
// Partial slots the workspace holds: per CTA or admitted thief or straddling chunk, one per consumer group.
__host__ __device__ inline size_t pool_slots(int nseg) {
    return (size_t)kMaxGroups * ((size_t)kMaxCtas + (size_t)(steal_slots_for(nseg) + 3) * (size_t)nseg);
}

// Everything the attention kernel needs; passed by value.
struct AttnParams {
    const void* q;            // bf16 [B][Hq][D]
    void* k;                  // bf16 (or e4m3 codes when f8), layout per mode (written only by a fused append)
    void* v;
    const float* k_scale;     // f8 only: [Hkv] dequantisation scales (value = code value * scale)
    const float* v_scale;
    int f8;                   // 1: the store holds e4m3 codes
    const int32_t* page_table;
    int64_t* len;             // [B]; advanced at the end of a launch that appends
    const void* k_new;        // bf16 [B][Hkv][D], or nullptr: attention only, no append
    const void* v_new;
    int32_t* slot_pos;        // ring only: [B][n_sink + cap]
    float* part_o;
    float* part_lse;
    int* part_key;            // [slots]: (CTA, group) that wrote the partial; orders the fixed-partition combine
    unsigned long long* arrive;   // [2][seg_stride]: (published partials << 32) | tiles covered by them
    int* nparts;              // [2][seg_stride]: partial slots handed out
    int seg_stride;           // elements between the two copies of the per-segment words (selected by epoch parity)
    uint32_t* epoch;          // launch counter (header)
    int* segs_done;           // completed segments (header)
    int* grab_done;           // CTAs that take no more tickets (header)
    int* cur;                 // [CTAs]: tiles of each CTA's dynamic part handed out so far
    int* nthief;              // [2][seg_stride]: CTAs admitted from other segments
    int steal_slots;          // thieves a segment admits from other segments
    int steal_slots_enabled;  // 0: purely static partition (deterministic, smallest partial pool)
    int* status;
    void* out;                // bf16 [B][Hq][D]
    float* lse;               // [B][Hq] or nullptr
    int64_t rows_per_head;    // contiguous: S_cap; ring: n_sink + cap; paged: page_size
    int64_t S_cap;            // tokens a sequence can hold (contiguous / paged); unused for the ring
    int B, Hq, Hkv, D, G;
    int mode;
    int page_size, max_pages, num_pages;
    int n_sink, W, cap;
    int q_len;                // queries per sequence (1: decode; > 1: draft-extend, B then counts queries)
    int window_view;          // contiguous / paged only: attend over the first n_sink and the last W positions of the KV store
    float scale_log2;         // sm_scale * log2(e)
    int num_ctas;
    int stages;               // stages of the kernel's shared-memory ring (set by the launcher)
    uint32_t spin_limit;      // polls a CTA spends waiting for another CTA's global word before it gives up
    int cluster;              // > 0: the cluster form of the kernel, one cluster of this many CTAs per segment (num_ctas = segments * cluster)
    int one_group;            // cluster form, bf16 head_dim 128: the variant with one consumer group (few tiles per CTA)
};

struct RingParams {
    void* k; void* v; int32_t* slot_pos; int64_t* len;
    int B, Hkv, D, n_sink, W, cap;
    int f8; const float* k_scale; const float* v_scale;    // f8: e4m3 codes, per-KV-head scales
};

struct KvParams {
    void* k; void* v; const int32_t* page_table; int64_t* len;
    int64_t S_cap;
    int B, Hkv, D, page_size, max_pages, num_pages;
    int f8; const float* k_scale; const float* v_scale;
};

// Launchers (defined in the .cu files). Each returns the cudaError_t of its launch.
cudaError_t launch_ring_reset(const RingParams& r, cudaStream_t st);
cudaError_t launch_ring_append(const RingParams& r, const void* k_new, const void* v_new, cudaStream_t st);
cudaError_t launch_ring_init_from_kv(const RingParams& r, const KvParams& kv, cudaStream_t st);
cudaError_t launch_kv_append(const KvParams& kv, const void* k_new, const void* v_new, int* status, cudaStream_t st);
cudaError_t launch_ring_append_many(const RingParams& r, int n_tok, const void* k_new, const void* v_new, cudaStream_t st);
cudaError_t launch_kv_append_many(const KvParams& kv, int n_tok, const void* k_new, const void* v_new, int* status, cudaStream_t st);
cudaError_t launch_ring_rewind(const RingParams& r, const int32_t* n_drop, int* status, cudaStream_t st);
cudaError_t launch_ring_replace_tail(const RingParams& r, const int32_t* n_drop, int n_tok, const void* k_new, const void* v_new,
                                     int* status, cudaStream_t st);
cudaError_t launch_reduced_block_table(const KvParams& kv, int n_sink, int W, int32_t* table, int stride, int32_t* meta, int* status,
                                       cudaStream_t st);
cudaError_t launch_full_token_index(const KvParams& kv, int32_t* index, int64_t stride, int* status, cudaStream_t st);
// The TMA descriptors of a store's K and V tensors. They depend on the store only (base pointers, rows, head_dim, entry
// size), so a chain of launches on one store encodes them once.
struct AttnMaps { CUtensorMap k, v; };
cudaError_t make_attention_maps(const AttnParams& p, AttnMaps* maps);
// One launch: optional append of (k_new, v_new), split-KV partials, LSE combine (cooperative or cluster form: p.cluster).
cudaError_t launch_attention(const AttnParams& p, const AttnMaps& maps, cudaStream_t st);
int pick_cluster(int D, int f8, int nseg, int64_t tiles_per_segment, int max_ctas, int* one_group);

// Full-context draft-extend with shared K/V tiles: p.B counts sequences, p.q_len their new tokens;
// partial results go to p.part_lse / p.part_o, (p.num_ctas + streams) * min(q_len, kExtendChunk) rows of G (x D) floats.
cudaError_t launch_extend_mq(const AttnParams& p, cudaStream_t st);
bool extend_mq_fits(int B, int D, int f8);     // does the kernel's shared memory hold the tables of B sequences?

cudaError_t launch_mass_diagnostics(const void* o_win, const float* lse_win, const void* o_full, const float* lse_full, int rows,
                                    int D, float* mass, float* perturb, float* tail, cudaStream_t st);

void count_launch(int n);
int  sm_count();   // multiprocessors of the current device (cached per device), 0 on failure

}  // namespace wmtp
