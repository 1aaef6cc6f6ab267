// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/wmtp.h"

namespace wmtp {

constexpr int kTileKeys = 64;       // keys per K/V tile; equals the page size of the paged layout
constexpr int kMaxCtas = 256;       // upper bound on attention CTAs (one per SM), sizes the partial buffers
constexpr int kMaxBatch = 1024;     // sequences per call (prefix table lives in shared memory)
constexpr int kMaxGroup = 8;        // query heads per KV head
constexpr int kMaxSegments = 16384; // batch * Hkv per call
constexpr size_t kWorkspaceZeroBytes = 256 + sizeof(int) * kMaxSegments;   // header + arrival counters

enum KvMode : int { kContiguous = 0, kPaged = 1, kRing = 2 };

// Workspace layout (all offsets from a 256-byte aligned base):
//   [0, 256)            header: int status @0, uint epoch @4, int segs_done @8, int checkin @12
//   counters            int arrive[kMaxSegments] (fixed size: initialisation needs no shape)
//   part_lse            float [kMaxCtas + batch * Hkv][G]
//   part_o              float [kMaxCtas + batch * Hkv][G][D]
struct WorkspaceLayout {
    size_t counters_off, part_lse_off, part_o_off, total;
};
WorkspaceLayout workspace_layout(int batch, int Hq, int Hkv, int D);

// Everything the attention kernel needs; passed by value.
struct AttnParams {
    const void* q;            // bf16 [B][Hq][D]
    void* k;                  // bf16, layout per mode (written only by a fused append)
    void* v;
    const int32_t* page_table;
    int64_t* len;             // [B]; advanced at the end of a launch that appends
    const void* k_new;        // bf16 [B][Hkv][D], or nullptr: attention only, no append
    const void* v_new;
    int32_t* slot_pos;        // ring only: [B][n_sink + cap]
    float* part_o;
    float* part_lse;
    int* arrive;              // [segments]: CTAs that have published their partial of the segment
    uint32_t* epoch;          // launch counter (header); arrival counters count from epoch * stride
    int* segs_done;           // segments whose last partial has arrived (header)
    int* checkin;             // CTAs of this launch that have read len[] (header)
    int* status;
    void* out;                // bf16 [B][Hq][D]
    float* lse;               // [B][Hq] or nullptr
    int64_t rows_per_head;    // contiguous: S_cap; ring: n_sink + cap; paged: page_size
    int64_t S_cap;            // tokens a sequence can hold (contiguous / paged); unused for the ring
    int B, Hq, Hkv, D, G;
    int mode;
    int page_size, max_pages, num_pages;
    int n_sink, W, cap;
    float scale_log2;         // sm_scale * log2(e)
    int num_ctas;
};

struct RingParams {
    void* k; void* v; int32_t* slot_pos; int64_t* len;
    int B, Hkv, D, n_sink, W, cap;
};

struct KvParams {
    void* k; void* v; const int32_t* page_table; int64_t* len;
    int64_t S_cap;
    int B, Hkv, D, page_size, max_pages, num_pages;
};

// Launchers (defined in the .cu files). Each returns the cudaError_t of its launch.
cudaError_t launch_ring_reset(const RingParams& r, cudaStream_t st);
cudaError_t launch_ring_append(const RingParams& r, const void* k_new, const void* v_new, cudaStream_t st);
cudaError_t launch_ring_init_from_kv(const RingParams& r, const KvParams& kv, cudaStream_t st);
cudaError_t launch_kv_append(const KvParams& kv, const void* k_new, const void* v_new, int* status, cudaStream_t st);
// One cooperative launch: optional append of (k_new, v_new), split-KV partials, distributed LSE combine.
cudaError_t launch_attention(const AttnParams& p, cudaStream_t st);

void count_launch(int n);
int  sm_count();   // multiprocessors of the current device (cached), 0 on failure

}  // namespace wmtp
