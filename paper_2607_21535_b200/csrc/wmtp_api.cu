// C ABI of the library: argument validation, workspace layout, launches. No device allocation.
#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <climits>
#include <cstring>
#include <mutex>

#include "wmtp_internal.h"

namespace wmtp {

namespace {
thread_local char g_err[512] = "";
std::atomic<int64_t> g_launches{0};
std::atomic<int> g_max_ctas{0};
std::atomic<int> g_stealing{1};
std::atomic<uint32_t> g_wait_limit{0};          // 0: the default below
constexpr uint32_t kDefaultWaitLimit = 1u << 22;

wmtp_status fail(wmtp_status s, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
    return s;
}

wmtp_status cuda_fail(cudaError_t e, const char* what) {
    return fail(WMTP_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

wmtp_status check_shape(int batch, int Hkv, int D) {
    if (batch < 1 || Hkv < 1) return fail(WMTP_ERR_INVALID_ARG, "batch=%d, Hkv=%d must be positive", batch, Hkv);
    if (batch > kMaxBatch) return fail(WMTP_ERR_UNSUPPORTED, "batch=%d exceeds %d", batch, kMaxBatch);
    if ((int64_t)batch * Hkv > kMaxSegments) return fail(WMTP_ERR_UNSUPPORTED, "batch*Hkv=%lld exceeds %d", (long long)batch * Hkv, kMaxSegments);
    if (D != 128 && D != 256) return fail(WMTP_ERR_UNSUPPORTED, "head_dim=%d (supported: 128, 256)", D);
    return WMTP_OK;
}

wmtp_status check_dtype(int kv_dtype, const float* k_scale, const float* v_scale) {
    if (kv_dtype != WMTP_KV_BF16 && kv_dtype != WMTP_KV_FP8_E4M3) return fail(WMTP_ERR_UNSUPPORTED, "kv_dtype=%d (supported: bf16, fp8 e4m3)", kv_dtype);
    if (kv_dtype == WMTP_KV_FP8_E4M3 && (!k_scale || !v_scale || !aligned(k_scale, 4) || !aligned(v_scale, 4)))
        return fail(WMTP_ERR_INVALID_ARG, "an fp8 store needs k_scale and v_scale (device fp32 [Hkv])");
    return WMTP_OK;
}

wmtp_status check_ring(const wmtp_ring* r) {
    if (!r) return fail(WMTP_ERR_INVALID_ARG, "ring descriptor is NULL");
    if (wmtp_status s = check_shape(r->batch, r->Hkv, r->D)) return s;
    if (wmtp_status s = check_dtype(r->kv_dtype, r->k_scale, r->v_scale)) return s;
    if (r->n_sink < 0 || r->W < 1 || r->cap < r->W)
        return fail(WMTP_ERR_INVALID_ARG, "ring needs n_sink >= 0, W >= 1, cap >= W (n_sink=%d W=%d cap=%d)", r->n_sink, r->W, r->cap);
    if ((int64_t)r->n_sink + r->cap > (1 << 30)) return fail(WMTP_ERR_INVALID_ARG, "ring of %lld slots is too large", (long long)r->n_sink + r->cap);
    if ((int64_t)r->batch * r->Hkv * ((int64_t)r->n_sink + r->cap) > INT32_MAX)
        return fail(WMTP_ERR_UNSUPPORTED, "ring has more than 2^31 - 1 rows in total");
    if (!r->k || !r->v || !r->slot_pos || !r->len) return fail(WMTP_ERR_INVALID_ARG, "ring has a NULL pointer");
    if (!aligned(r->k, 16) || !aligned(r->v, 16) || !aligned(r->slot_pos, 4) || !aligned(r->len, 8))
        return fail(WMTP_ERR_INVALID_ARG, "ring pointers must be 16-byte (k, v), 4-byte (slot_pos), 8-byte (len) aligned");
    return WMTP_OK;
}

wmtp_status check_kv(const wmtp_kv* kv) {
    if (!kv) return fail(WMTP_ERR_INVALID_ARG, "kv descriptor is NULL");
    if (wmtp_status s = check_shape(kv->batch, kv->Hkv, kv->D)) return s;
    if (wmtp_status s = check_dtype(kv->kv_dtype, kv->k_scale, kv->v_scale)) return s;
    if (!kv->k || !kv->v || !kv->len) return fail(WMTP_ERR_INVALID_ARG, "kv has a NULL pointer");
    if (!aligned(kv->k, 16) || !aligned(kv->v, 16) || !aligned(kv->len, 8))
        return fail(WMTP_ERR_INVALID_ARG, "kv pointers must be 16-byte (k, v), 8-byte (len) aligned");
    if (kv->S_cap < 1) return fail(WMTP_ERR_INVALID_ARG, "S_cap=%lld must be positive", (long long)kv->S_cap);
    const int64_t kv_rows = kv->page_table ? (int64_t)kv->num_pages * kv->Hkv * kv->page_size : (int64_t)kv->batch * kv->Hkv * kv->S_cap;
    if (kv_rows > INT32_MAX) return fail(WMTP_ERR_UNSUPPORTED, "kv has more than 2^31 - 1 rows in total");
    if (kv->page_table) {
        if (kv->page_size != kTileKeys) return fail(WMTP_ERR_UNSUPPORTED, "page_size=%d (supported: %d)", kv->page_size, kTileKeys);
        if (kv->max_pages < 1 || kv->num_pages < 1) return fail(WMTP_ERR_INVALID_ARG, "max_pages, num_pages must be positive");
        if (!aligned(kv->page_table, 4)) return fail(WMTP_ERR_INVALID_ARG, "page_table must be 4-byte aligned");
        if (kv->S_cap > (int64_t)kv->max_pages * kv->page_size)
            return fail(WMTP_ERR_CAPACITY, "S_cap=%lld exceeds the page table's %lld tokens", (long long)kv->S_cap,
                        (long long)kv->max_pages * kv->page_size);
    }
    return WMTP_OK;
}

RingParams ring_params(const wmtp_ring* r) {
    return RingParams{r->k, r->v, r->slot_pos, r->len, r->batch, r->Hkv, r->D, r->n_sink, r->W, r->cap,
                      r->kv_dtype == WMTP_KV_FP8_E4M3 ? 1 : 0, r->k_scale, r->v_scale};
}
KvParams kv_params(const wmtp_kv* kv) {
    return KvParams{kv->k, kv->v, kv->page_table, kv->len, kv->S_cap, kv->batch, kv->Hkv, kv->D,
                    kv->page_table ? kv->page_size : 0, kv->max_pages, kv->num_pages,
                    kv->kv_dtype == WMTP_KV_FP8_E4M3 ? 1 : 0, kv->k_scale, kv->v_scale};
}

wmtp_status check_attn_common(const void* q, int Hq, int Hkv, int batch, int D, const void* out, const float* lse,
                              const void* ws, size_t ws_bytes) {
    if (!q || !out) return fail(WMTP_ERR_INVALID_ARG, "q or out is NULL");
    if (!aligned(q, 16) || !aligned(out, 16)) return fail(WMTP_ERR_INVALID_ARG, "q and out must be 16-byte aligned");
    if (lse && !aligned(lse, 4)) return fail(WMTP_ERR_INVALID_ARG, "lse must be 4-byte aligned");
    if (Hq < 1 || Hq % Hkv != 0) return fail(WMTP_ERR_INVALID_ARG, "Hq=%d must be a positive multiple of Hkv=%d", Hq, Hkv);
    if (Hq / Hkv > kMaxGroup) return fail(WMTP_ERR_UNSUPPORTED, "Hq/Hkv=%d exceeds %d", Hq / Hkv, kMaxGroup);
    if (!ws || !aligned(ws, 256)) return fail(WMTP_ERR_WORKSPACE, "workspace is NULL or not 256-byte aligned");
    const size_t need = wmtp_workspace_bytes(batch, Hq, Hkv, D);
    if (ws_bytes < need) return fail(WMTP_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", ws_bytes, need);
    return WMTP_OK;
}

// `streaming`: a long HBM-bound launch over a bf16 store. Those run faster on 7/8 of the SMs than on all of them
// (S = 1M: 321 us on 148 CTAs, 310-312 us on 116 to 132; S = 256K: 98 -> 94 us): the memory system delivers more to
// fewer requesters. The fp8 kernels are bound by arithmetic and keep every SM. An explicit cap is honoured as given.
int pick_ctas(int64_t max_tiles, bool streaming = false) {
    int c = g_max_ctas.load();
    const int sms = sm_count();
    if (sms <= 0) return 0;
    if (c <= 0 && streaming && max_tiles >= 16 * (int64_t)sms) c = (sms * 7 / 8) & ~7;
    if (c <= 0 || c > sms) c = sms;          // one CTA per SM: the cooperative launch needs all CTAs resident
    if (c > kMaxCtas) c = kMaxCtas;
    if (max_tiles < c) c = (int)(max_tiles < 1 ? 1 : max_tiles);
    return c;
}

// Launches whose segments all have (about) the same number of tiles -- rings and window views in steady state: a CTA
// count that is a multiple of the segment count puts the CTAs' range boundaries on the segment boundaries, so no CTA
// works in two segments, which would cost it a second flush and a second merge (about 5 us on these short launches).
// Worth up to a fifth of the SMs idle (measured at 16 and 32 sequences: 13 % idle SMs, 8-11 % faster).
int align_ctas_to_segments(int ctas, int nseg, int64_t tiles) {
    if (nseg > 1 && nseg < ctas && tiles > ctas) {
        const int aligned_ctas = ctas / nseg * nseg;
        if ((ctas - aligned_ctas) * 5 <= ctas) return aligned_ctas;
    }
    return ctas;
}

// Where the kernel's scratch lives: the header at `base`, the cursors behind it, two copies of the per-segment words
// `seg_stride` elements apart, then the partial results. Both the caller's workspace and the library's built-in
// scratch array are described this way.
struct ScratchLayout {
    size_t counters_off;
    int seg_stride;
    size_t part_key_off, part_lse_off, part_o_off;
};

// Everything of AttnParams that does not depend on the kind of store.
void fill_attn(AttnParams& p, const void* q, int Hq, int Hkv, int batch, int D, float sm_scale, void* out, float* lse,
               void* scratch, const ScratchLayout& L, bool stealing) {
    char* base = static_cast<char*>(scratch);
    p.q = q; p.out = out; p.lse = lse;
    p.status = reinterpret_cast<int*>(base);
    p.epoch = reinterpret_cast<uint32_t*>(base + 4);
    p.segs_done = reinterpret_cast<int*>(base + 8);
    p.grab_done = reinterpret_cast<int*>(base + 12);
    p.cur = reinterpret_cast<int*>(base + 256);
    p.arrive = reinterpret_cast<unsigned long long*>(base + L.counters_off);
    p.nparts = reinterpret_cast<int*>(p.arrive + 2 * L.seg_stride);
    p.nthief = p.nparts + 2 * L.seg_stride;
    p.seg_stride = L.seg_stride;
    p.steal_slots_enabled = stealing ? 1 : 0;
    p.steal_slots = stealing ? steal_slots_for(batch * Hkv) : 0;
    p.part_key = reinterpret_cast<int*>(base + L.part_key_off);
    p.part_lse = reinterpret_cast<float*>(base + L.part_lse_off);
    p.part_o = reinterpret_cast<float*>(base + L.part_o_off);
    p.B = batch; p.Hq = Hq; p.Hkv = Hkv; p.D = D; p.G = Hq / Hkv;
    p.q_len = 1;
    const float s = sm_scale > 0.f ? sm_scale : 1.0f / std::sqrt((float)D);
    p.scale_log2 = s * 1.4426950408889634f;
    const uint32_t wl = g_wait_limit.load();
    p.spin_limit = wl ? wl : kDefaultWaitLimit;
}

void fill_attn(AttnParams& p, const void* q, int Hq, int Hkv, int batch, int D, float sm_scale, void* out, float* lse,
               void* ws) {
    const WorkspaceLayout W = workspace_layout(batch, Hq, Hkv, D);
    fill_attn(p, q, Hq, Hkv, batch, D, sm_scale, out, lse, ws,
              ScratchLayout{W.counters_off, kMaxSegments, W.part_key_off, W.part_lse_off, W.part_o_off}, g_stealing.load() != 0);
}

// The ring as the attention kernel sees it.
void bind_ring(AttnParams& p, const wmtp_ring* ring, const void* k_new, const void* v_new) {
    p.k = ring->k; p.v = ring->v; p.page_table = nullptr; p.len = ring->len;
    p.f8 = ring->kv_dtype == WMTP_KV_FP8_E4M3 ? 1 : 0; p.k_scale = ring->k_scale; p.v_scale = ring->v_scale;
    p.k_new = k_new; p.v_new = v_new; p.slot_pos = ring->slot_pos;
    p.mode = kRing;
    p.rows_per_head = (int64_t)ring->n_sink + ring->cap;
    p.n_sink = ring->n_sink; p.W = ring->W; p.cap = ring->cap;
}

// k_new / v_new non-NULL: a fused draft step (append, then attend) in one launch.
// A chain of launches on one store encodes the store's TMA descriptors once.
struct MapCache { AttnMaps maps; bool ready = false; };
cudaError_t launch_with(const AttnParams& p, MapCache* cache, cudaStream_t st) {
    MapCache local;
    if (!cache) cache = &local;
    if (!cache->ready) {
        cudaError_t e = make_attention_maps(p, &cache->maps);
        if (e != cudaSuccess) return e;
        cache->ready = true;
    }
    return launch_attention(p, cache->maps, st);
}

wmtp_status attn_windowed(const void* q, int Hq, const wmtp_ring* ring, float sm_scale, void* out, float* lse,
                          void* ws, size_t ws_bytes, cudaStream_t st, bool validate, const void* k_new = nullptr,
                          const void* v_new = nullptr, int q_len = 1, MapCache* cache = nullptr) {
    if (validate) {
        if (wmtp_status s = check_ring(ring)) return s;
        if (wmtp_status s = check_attn_common(q, Hq, ring->Hkv, ring->batch * q_len, ring->D, out, lse, ws, ws_bytes)) return s;
    }
    AttnParams p{};
    fill_attn(p, q, Hq, ring->Hkv, ring->batch * q_len, ring->D, sm_scale, out, lse, ws);
    p.q_len = q_len;
    bind_ring(p, ring, k_new, v_new);
    const int nseg = ring->batch * q_len * ring->Hkv;
    const int64_t tiles_per_seg = (p.rows_per_head + kTileKeys - 1) / kTileKeys, tiles = tiles_per_seg * nseg;
    p.cluster = pick_cluster(p.D, p.f8, nseg, tiles_per_seg, g_max_ctas.load(), &p.one_group);
    if (p.cluster > 0) {
        p.num_ctas = nseg * p.cluster;
    } else {
        p.num_ctas = pick_ctas(tiles);
        p.num_ctas = align_ctas_to_segments(p.num_ctas, nseg, tiles);
    }
    if (p.num_ctas <= 0) return fail(WMTP_ERR_CUDA, "no CUDA device available");
    cudaError_t e = launch_with(p, cache, st);
    if (e != cudaSuccess) return cuda_fail(e, "windowed attention launch");
    return WMTP_OK;
}

// W > 0: window view (attend over the first n_sink and the last W positions of the KV store); W == 0: all positions.
wmtp_status attn_full(const void* q, int Hq, const wmtp_kv* kv, float sm_scale, void* out, float* lse, void* ws,
                      size_t ws_bytes, cudaStream_t st, bool validate, const void* k_new = nullptr,
                      const void* v_new = nullptr, int n_sink = 0, int W = 0, int q_len = 1, MapCache* cache = nullptr) {
    if (validate) {
        if (wmtp_status s = check_kv(kv)) return s;
        if (wmtp_status s = check_attn_common(q, Hq, kv->Hkv, kv->batch * q_len, kv->D, out, lse, ws, ws_bytes)) return s;
    }
    AttnParams p{};
    fill_attn(p, q, Hq, kv->Hkv, kv->batch * q_len, kv->D, sm_scale, out, lse, ws);
    p.q_len = q_len;
    p.k = kv->k; p.v = kv->v; p.page_table = kv->page_table; p.len = kv->len;
    p.f8 = kv->kv_dtype == WMTP_KV_FP8_E4M3 ? 1 : 0; p.k_scale = kv->k_scale; p.v_scale = kv->v_scale;
    p.k_new = k_new; p.v_new = v_new; p.slot_pos = nullptr; p.S_cap = kv->S_cap;
    p.mode = kv->page_table ? kPaged : kContiguous;
    p.rows_per_head = kv->page_table ? kv->page_size : kv->S_cap;
    p.page_size = kv->page_size; p.max_pages = kv->max_pages; p.num_pages = kv->num_pages;
    int64_t tiles_per_seg = (kv->S_cap + kTileKeys - 1) / kTileKeys;
    if (W > 0) {
        p.window_view = 1; p.n_sink = n_sink; p.W = W;
        const int64_t view_tiles = ((int64_t)n_sink + kTileKeys - 1) / kTileKeys + ((int64_t)W + kTileKeys - 1) / kTileKeys + 1;
        if (view_tiles < tiles_per_seg) tiles_per_seg = view_tiles;
    }
    // few long segments of a bf16 store, one query each: see pick_ctas (a ragged 32-sequence batch and the multi-query
    // extend, which re-reads rows through L2, measured slower on fewer SMs)
    const bool streaming = W == 0 && !p.f8 && q_len == 1 && kv->batch * kv->Hkv <= 8;
    const int nseg = kv->batch * q_len * kv->Hkv;
    if (W > 0) p.cluster = pick_cluster(p.D, p.f8, nseg, tiles_per_seg, g_max_ctas.load(), &p.one_group);
    if (p.cluster > 0) {
        p.num_ctas = nseg * p.cluster;
    } else {
        p.num_ctas = pick_ctas(tiles_per_seg * nseg, streaming);
        if (W > 0) p.num_ctas = align_ctas_to_segments(p.num_ctas, nseg, tiles_per_seg * nseg);
    }
    if (p.num_ctas <= 0) return fail(WMTP_ERR_CUDA, "no CUDA device available");
    cudaError_t e = launch_with(p, cache, st);
    if (e != cudaSuccess) return cuda_fail(e, W > 0 ? "windowed (KV view) attention launch" : "full attention launch");
    return WMTP_OK;
}

wmtp_status check_loop(int gamma, const void* k_new, const void* v_new) {
    if (gamma < 1) return fail(WMTP_ERR_INVALID_ARG, "gamma=%d must be positive", gamma);
    if (!k_new || !v_new) return fail(WMTP_ERR_INVALID_ARG, "k_new or v_new is NULL");
    if (!aligned(k_new, 16) || !aligned(v_new, 16)) return fail(WMTP_ERR_INVALID_ARG, "k_new and v_new must be 16-byte aligned");
    return WMTP_OK;
}

struct StagePlan { size_t q, k, v, out, lse, total; };
StagePlan stage_plan(int gamma, int batch, int Hq, int Hkv, int D) {
    StagePlan s;
    const size_t qb = (size_t)gamma * batch * Hq * D * 2, kb = (size_t)gamma * batch * Hkv * D * 2;
    s.q = 0;
    s.k = round_up(qb, 256);
    s.v = s.k + round_up(kb, 256);
    s.out = s.v + round_up(kb, 256);
    s.lse = s.out + round_up(qb, 256);
    s.total = s.lse + round_up((size_t)gamma * batch * Hq * 4, 256);
    return s;
}

}  // namespace

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }


int sm_count() {
    static std::atomic<int> cached[64];     // per device ordinal; zero-initialised
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    const bool slot = dev >= 0 && dev < 64;
    if (slot) {
        const int c = cached[dev].load();
        if (c > 0) return c;
    }
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    if (slot) cached[dev].store(n);
    return n;
}

WorkspaceLayout workspace_layout(int batch, int Hq, int Hkv, int D) {
    WorkspaceLayout L;
    const size_t G = (size_t)(Hq / Hkv), nseg = (size_t)batch * Hkv, np = pool_slots((int)nseg);
    L.counters_off = 256 + kCursorBytes;
    L.part_key_off = kWorkspaceZeroBytes;
    L.part_lse_off = L.part_key_off + round_up(np * sizeof(int), 256);
    L.part_o_off = L.part_lse_off + round_up(np * G * sizeof(float), 256);
    L.total = L.part_o_off + round_up(np * G * D * sizeof(float), 256);
    return L;
}

}  // namespace wmtp

using namespace wmtp;

extern "C" {

const char* wmtp_status_string(wmtp_status s) {
    switch (s) {
        case WMTP_OK: return "ok";
        case WMTP_ERR_INVALID_ARG: return "invalid argument";
        case WMTP_ERR_UNSUPPORTED: return "unsupported shape";
        case WMTP_ERR_CAPACITY: return "capacity exceeded";
        case WMTP_ERR_WORKSPACE: return "bad workspace";
        case WMTP_ERR_CUDA: return "CUDA error";
        case WMTP_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        case WMTP_ERR_DEVICE_BOUNDS: return "device-side bounds check failed";
    }
    return "unknown status";
}

const char* wmtp_last_error(void) { return g_err; }

size_t wmtp_kv_elem_bytes(int kv_dtype) { return kv_dtype == WMTP_KV_BF16 ? 2 : (kv_dtype == WMTP_KV_FP8_E4M3 ? 1 : 0); }

size_t wmtp_ring_bytes(int batch, int Hkv, int D, int n_sink, int cap, size_t* pos_bytes) {
    if (batch < 1 || Hkv < 1 || D < 1 || n_sink < 0 || cap < 1) { if (pos_bytes) *pos_bytes = 0; return 0; }
    const size_t slots = (size_t)n_sink + cap;
    if (pos_bytes) *pos_bytes = (size_t)batch * slots * sizeof(int32_t);
    return (size_t)batch * Hkv * slots * D * 2;
}

size_t wmtp_workspace_bytes(int batch, int Hq, int Hkv, int D) {
    if (batch < 1 || Hq < 1 || Hkv < 1 || D < 1 || Hq % Hkv != 0) return 0;
    return workspace_layout(batch, Hq, Hkv, D).total;
}

wmtp_status wmtp_workspace_init(void* workspace, size_t ws_bytes, void* stream) {
    if (!workspace || !aligned(workspace, 256)) return fail(WMTP_ERR_WORKSPACE, "workspace is NULL or not 256-byte aligned");
    if (ws_bytes < kWorkspaceZeroBytes) return fail(WMTP_ERR_WORKSPACE, "workspace of %zu bytes is too small", ws_bytes);
    // only the status word and the completion counters must start at zero; partials are always written before read
    cudaError_t e = cudaMemsetAsync(workspace, 0, kWorkspaceZeroBytes, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e, "workspace memset");
    return WMTP_OK;
}

wmtp_status wmtp_device_status(void* workspace, void* stream) {
    if (!workspace) return fail(WMTP_ERR_WORKSPACE, "workspace is NULL");
    int word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, workspace, sizeof word, cudaMemcpyDeviceToHost, (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(e, "reading the device status");
    if (word != 0) {
        e = cudaMemsetAsync(workspace, 0, sizeof word, (cudaStream_t)stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
        if (e != cudaSuccess) return cuda_fail(e, "clearing the device status");
        if (word == WMTP_ERR_DEVICE_TIMEOUT) return fail(WMTP_ERR_DEVICE_TIMEOUT, "a device-side wait expired");
        return fail(WMTP_ERR_DEVICE_BOUNDS, "a device-side bounds check failed (status word %d)", word);
    }
    return WMTP_OK;
}

wmtp_status wmtp_ring_reset(const wmtp_ring* ring, void* stream) {
    if (wmtp_status s = check_ring(ring)) return s;
    cudaError_t e = launch_ring_reset(ring_params(ring), (cudaStream_t)stream);
    return e == cudaSuccess ? WMTP_OK : cuda_fail(e, "ring reset launch");
}

// ---- snapshot / restore of a ring: four plain copies, each part on a 256-byte boundary of the blob
namespace {
struct RingState { size_t kv_bytes, pos_bytes, len_bytes, off_v, off_pos, off_len, total; };
RingState ring_state(const wmtp_ring* r) {
    RingState s;
    const size_t slots = (size_t)r->n_sink + (size_t)r->cap;
    s.kv_bytes = (size_t)r->batch * r->Hkv * slots * r->D * (r->kv_dtype == WMTP_KV_FP8_E4M3 ? 1 : 2);
    s.pos_bytes = (size_t)r->batch * slots * sizeof(int32_t);
    s.len_bytes = (size_t)r->batch * sizeof(int64_t);
    s.off_v = round_up(s.kv_bytes, 256);
    s.off_pos = s.off_v + round_up(s.kv_bytes, 256);
    s.off_len = s.off_pos + round_up(s.pos_bytes, 256);
    s.total = s.off_len + round_up(s.len_bytes, 256);
    return s;
}
wmtp_status ring_copy(const wmtp_ring* ring, void* blob, size_t blob_bytes, cudaStream_t st, bool to_blob) {
    if (wmtp_status s = check_ring(ring)) return s;
    if (!blob || !aligned(blob, 16)) return fail(WMTP_ERR_INVALID_ARG, "blob is NULL or not 16-byte aligned");
    const RingState rs = ring_state(ring);
    if (blob_bytes < rs.total) return fail(WMTP_ERR_CAPACITY, "blob of %zu bytes, the ring's state takes %zu", blob_bytes, rs.total);
    char* b = static_cast<char*>(blob);
    struct Part { void* ring_ptr; size_t off, bytes; };
    const Part parts[4] = {{ring->k, 0, rs.kv_bytes}, {ring->v, rs.off_v, rs.kv_bytes}, {ring->slot_pos, rs.off_pos, rs.pos_bytes},
                           {ring->len, rs.off_len, rs.len_bytes}};
    for (const Part& pt : parts) {
        const cudaError_t e = to_blob ? cudaMemcpyAsync(b + pt.off, pt.ring_ptr, pt.bytes, cudaMemcpyDefault, st)
                                      : cudaMemcpyAsync(pt.ring_ptr, b + pt.off, pt.bytes, cudaMemcpyDefault, st);
        if (e != cudaSuccess) return cuda_fail(e, to_blob ? "ring export copy" : "ring import copy");
    }
    return WMTP_OK;
}
}  // namespace

size_t wmtp_ring_state_bytes(const wmtp_ring* ring) {
    if (check_ring(ring) != WMTP_OK) return 0;
    return ring_state(ring).total;
}

wmtp_status wmtp_ring_export(const wmtp_ring* ring, void* blob, size_t blob_bytes, void* stream) {
    return ring_copy(ring, blob, blob_bytes, (cudaStream_t)stream, true);
}

wmtp_status wmtp_ring_import(const wmtp_ring* ring, const void* blob, size_t blob_bytes, void* stream) {
    return ring_copy(ring, const_cast<void*>(blob), blob_bytes, (cudaStream_t)stream, false);
}

wmtp_status wmtp_ring_init_from_kv(const wmtp_ring* ring, const wmtp_kv* kv, void* stream) {
    if (wmtp_status s = check_ring(ring)) return s;
    if (wmtp_status s = check_kv(kv)) return s;
    if (ring->batch != kv->batch || ring->Hkv != kv->Hkv || ring->D != kv->D)
        return fail(WMTP_ERR_INVALID_ARG, "ring and kv disagree on batch / Hkv / D");
    if (ring->kv_dtype != kv->kv_dtype) return fail(WMTP_ERR_INVALID_ARG, "ring and kv disagree on kv_dtype (rows are copied as stored)");
    cudaError_t e = launch_ring_init_from_kv(ring_params(ring), kv_params(kv), (cudaStream_t)stream);
    return e == cudaSuccess ? WMTP_OK : cuda_fail(e, "ring init launch");
}

wmtp_status wmtp_ring_append(const wmtp_ring* ring, const void* k_new, const void* v_new, void* stream) {
    if (wmtp_status s = check_ring(ring)) return s;
    if (wmtp_status s = check_loop(1, k_new, v_new)) return s;
    cudaError_t e = launch_ring_append(ring_params(ring), k_new, v_new, (cudaStream_t)stream);
    return e == cudaSuccess ? WMTP_OK : cuda_fail(e, "ring append launch");
}

wmtp_status wmtp_kv_append(const wmtp_kv* kv, const void* k_new, const void* v_new, void* workspace, void* stream) {
    if (wmtp_status s = check_kv(kv)) return s;
    if (wmtp_status s = check_loop(1, k_new, v_new)) return s;
    if (workspace && !aligned(workspace, 256)) return fail(WMTP_ERR_WORKSPACE, "workspace is not 256-byte aligned");
    cudaError_t e = launch_kv_append(kv_params(kv), k_new, v_new, static_cast<int*>(workspace), (cudaStream_t)stream);
    return e == cudaSuccess ? WMTP_OK : cuda_fail(e, "kv append launch");
}

wmtp_status wmtp_draft_attn_windowed(const void* q, int Hq, const wmtp_ring* ring, float sm_scale, void* out,
                                     float* lse, void* workspace, size_t ws_bytes, void* stream) {
    return attn_windowed(q, Hq, ring, sm_scale, out, lse, workspace, ws_bytes, (cudaStream_t)stream, true);
}

wmtp_status wmtp_draft_attn_full(const void* q, int Hq, const wmtp_kv* kv, float sm_scale, void* out, float* lse,
                                 void* workspace, size_t ws_bytes, void* stream) {
    return attn_full(q, Hq, kv, sm_scale, out, lse, workspace, ws_bytes, (cudaStream_t)stream, true);
}

wmtp_status wmtp_draft_loop_windowed(const wmtp_ring* ring, int gamma, const void* q, int Hq, const void* k_new,
                                     const void* v_new, float sm_scale, void* out, float* lse, void* workspace,
                                     size_t ws_bytes, void* stream) {
    if (wmtp_status s = check_ring(ring)) return s;
    if (wmtp_status s = check_loop(gamma, k_new, v_new)) return s;
    if (wmtp_status s = check_attn_common(q, Hq, ring->Hkv, ring->batch, ring->D, out, lse, workspace, ws_bytes)) return s;
    const size_t q_step = (size_t)ring->batch * Hq * ring->D * 2, kv_step = (size_t)ring->batch * ring->Hkv * ring->D * 2;
    MapCache cache;
    for (int i = 0; i < gamma; ++i) {
        // one launch per draft step: the kernel appends step i's K/V row, then attends
        if (wmtp_status s = attn_windowed((const char*)q + i * q_step, Hq, ring, sm_scale, (char*)out + i * q_step,
                                          lse ? lse + (size_t)i * ring->batch * Hq : nullptr, workspace, ws_bytes,
                                          (cudaStream_t)stream, false, (const char*)k_new + i * kv_step,
                                          (const char*)v_new + i * kv_step, 1, &cache))
            return s;
    }
    return WMTP_OK;
}

wmtp_status wmtp_draft_loop_full(const wmtp_kv* kv, int gamma, const void* q, int Hq, const void* k_new,
                                 const void* v_new, float sm_scale, void* out, float* lse, void* workspace,
                                 size_t ws_bytes, void* stream) {
    if (wmtp_status s = check_kv(kv)) return s;
    if (wmtp_status s = check_loop(gamma, k_new, v_new)) return s;
    if (wmtp_status s = check_attn_common(q, Hq, kv->Hkv, kv->batch, kv->D, out, lse, workspace, ws_bytes)) return s;
    const size_t q_step = (size_t)kv->batch * Hq * kv->D * 2, kv_step = (size_t)kv->batch * kv->Hkv * kv->D * 2;
    MapCache cache;
    for (int i = 0; i < gamma; ++i) {
        if (wmtp_status s = attn_full((const char*)q + i * q_step, Hq, kv, sm_scale, (char*)out + i * q_step,
                                      lse ? lse + (size_t)i * kv->batch * Hq : nullptr, workspace, ws_bytes,
                                      (cudaStream_t)stream, false, (const char*)k_new + i * kv_step,
                                      (const char*)v_new + i * kv_step, 0, 0, 1, &cache))
            return s;
    }
    return WMTP_OK;
}

/* ---- draft-extend: several new tokens per sequence in one launch ---- */

static wmtp_status check_extend(int q_len, int batch) {
    if (q_len < 1 || q_len > 64) return fail(WMTP_ERR_INVALID_ARG, "q_len=%d must be in [1, 64]", q_len);
    if ((int64_t)batch * q_len > kMaxBatch) return fail(WMTP_ERR_UNSUPPORTED, "batch*q_len=%lld exceeds %d", (long long)batch * q_len, kMaxBatch);
    return WMTP_OK;
}

wmtp_status wmtp_ring_append_many(const wmtp_ring* ring, int n_tok, const void* k_new, const void* v_new, void* stream) {
    if (wmtp_status s = check_ring(ring)) return s;
    if (wmtp_status s = check_loop(n_tok, k_new, v_new)) return s;
    if (n_tok > ring->cap) return fail(WMTP_ERR_CAPACITY, "n_tok=%d exceeds the ring's %d window slots", n_tok, ring->cap);
    cudaError_t e = launch_ring_append_many(ring_params(ring), n_tok, k_new, v_new, (cudaStream_t)stream);
    return e == cudaSuccess ? WMTP_OK : cuda_fail(e, "ring append launch");
}

wmtp_status wmtp_kv_append_many(const wmtp_kv* kv, int n_tok, const void* k_new, const void* v_new, void* workspace, void* stream) {
    if (wmtp_status s = check_kv(kv)) return s;
    if (wmtp_status s = check_loop(n_tok, k_new, v_new)) return s;
    if (workspace && !aligned(workspace, 256)) return fail(WMTP_ERR_WORKSPACE, "workspace is not 256-byte aligned");
    cudaError_t e = launch_kv_append_many(kv_params(kv), n_tok, k_new, v_new, static_cast<int*>(workspace), (cudaStream_t)stream);
    return e == cudaSuccess ? WMTP_OK : cuda_fail(e, "kv append launch");
}

wmtp_status wmtp_ring_rewind(const wmtp_ring* ring, const int32_t* n_drop, void* workspace, void* stream) {
    if (wmtp_status s = check_ring(ring)) return s;
    if (!n_drop || !aligned(n_drop, 4)) return fail(WMTP_ERR_INVALID_ARG, "n_drop is NULL or misaligned");
    if (workspace && !aligned(workspace, 256)) return fail(WMTP_ERR_WORKSPACE, "workspace is not 256-byte aligned");
    cudaError_t e = launch_ring_rewind(ring_params(ring), n_drop, static_cast<int*>(workspace), (cudaStream_t)stream);
    return e == cudaSuccess ? WMTP_OK : cuda_fail(e, "ring rewind launch");
}

wmtp_status wmtp_ring_replace_tail(const wmtp_ring* ring, const int32_t* n_drop, int n_tok, const void* k_new, const void* v_new,
                                   void* workspace, void* stream) {
    if (wmtp_status s = check_ring(ring)) return s;
    if (n_drop && !aligned(n_drop, 4)) return fail(WMTP_ERR_INVALID_ARG, "n_drop is misaligned");
    if (wmtp_status s = check_loop(n_tok, k_new, v_new)) return s;
    if (n_tok > ring->cap) return fail(WMTP_ERR_CAPACITY, "n_tok=%d exceeds the ring's %d window slots", n_tok, ring->cap);
    if (workspace && !aligned(workspace, 256)) return fail(WMTP_ERR_WORKSPACE, "workspace is not 256-byte aligned");
    cudaError_t e = launch_ring_replace_tail(ring_params(ring), n_drop, n_tok, k_new, v_new, static_cast<int*>(workspace),
                                             (cudaStream_t)stream);
    return e == cudaSuccess ? WMTP_OK : cuda_fail(e, "ring replace-tail launch");
}

wmtp_status wmtp_draft_extend_windowed(const void* q, int q_len, int Hq, const wmtp_ring* ring, float sm_scale, void* out,
                                       float* lse, void* workspace, size_t ws_bytes, void* stream) {
    if (wmtp_status s = check_ring(ring)) return s;
    if (wmtp_status s = check_extend(q_len, ring->batch)) return s;
    if (ring->cap < ring->W + q_len - 1)
        return fail(WMTP_ERR_CAPACITY, "draft-extend of %d tokens needs cap >= W + %d slots (cap=%d, W=%d): the oldest query's "
                    "window would already be overwritten", q_len, q_len - 1, ring->cap, ring->W);
    return attn_windowed(q, Hq, ring, sm_scale, out, lse, workspace, ws_bytes, (cudaStream_t)stream, true, nullptr, nullptr, q_len);
}

// The shared-tile multi-query kernel (extend_kernels.cu): every K/V tile is read once for up to kExtendChunk queries of
// a sequence. Returns false when the launch does not fit it (the per-query path then serves the call).
static bool extend_full_shared_tiles(const void* q, int q_len, int Hq, const wmtp_kv* kv, float sm_scale, void* out, float* lse,
                                     void* ws, cudaStream_t st, wmtp_status* result) {
    if (q_len < 2 || !extend_mq_fits(kv->batch, kv->D, kv->kv_dtype == WMTP_KV_FP8_E4M3)) return false;
    const int nch = (q_len + kExtendChunk - 1) / kExtendChunk, nstreams = kv->batch * kv->Hkv * nch;
    const int slot_rows = q_len < kExtendChunk ? q_len : kExtendChunk;
    // the partial pool of a workspace sized for batch * q_len sequences holds pool_slots rows of G x (D + 1) floats
    const int64_t max_ctas = (int64_t)pool_slots(kv->batch * q_len * kv->Hkv) / slot_rows - nstreams;
    if (max_ctas < 1) return false;
    AttnParams p{};
    fill_attn(p, q, Hq, kv->Hkv, kv->batch * q_len, kv->D, sm_scale, out, lse, ws);
    p.B = kv->batch;                        // this kernel counts sequences, not queries
    p.q_len = q_len;
    p.k = kv->k; p.v = kv->v; p.page_table = kv->page_table; p.len = kv->len;
    p.f8 = kv->kv_dtype == WMTP_KV_FP8_E4M3 ? 1 : 0; p.k_scale = kv->k_scale; p.v_scale = kv->v_scale;
    p.S_cap = kv->S_cap;
    p.mode = kv->page_table ? kPaged : kContiguous;
    p.rows_per_head = kv->page_table ? kv->page_size : kv->S_cap;
    p.page_size = kv->page_size; p.max_pages = kv->max_pages; p.num_pages = kv->num_pages;
    const int64_t tiles = (kv->S_cap + kTileKeys - 1) / kTileKeys * nstreams;
    p.num_ctas = pick_ctas(tiles);
    if (p.num_ctas <= 0) { *result = fail(WMTP_ERR_CUDA, "no CUDA device available"); return true; }
    if (p.num_ctas > max_ctas) p.num_ctas = (int)max_ctas;
    const cudaError_t e = launch_extend_mq(p, st);
    *result = e == cudaSuccess ? WMTP_OK : cuda_fail(e, "multi-query draft-extend launch");
    return true;
}

wmtp_status wmtp_draft_extend_full(const void* q, int q_len, int Hq, const wmtp_kv* kv, float sm_scale, void* out, float* lse,
                                   void* workspace, size_t ws_bytes, void* stream) {
    if (wmtp_status s = check_kv(kv)) return s;
    if (wmtp_status s = check_extend(q_len, kv->batch)) return s;
    if (wmtp_status s = check_attn_common(q, Hq, kv->Hkv, kv->batch * q_len, kv->D, out, lse, workspace, ws_bytes)) return s;
    wmtp_status r = WMTP_OK;
    if (extend_full_shared_tiles(q, q_len, Hq, kv, sm_scale, out, lse, workspace, (cudaStream_t)stream, &r)) return r;
    return attn_full(q, Hq, kv, sm_scale, out, lse, workspace, ws_bytes, (cudaStream_t)stream, true, nullptr, nullptr, 0, 0, q_len);
}

static wmtp_status check_window(int n_sink, int W) {
    if (n_sink < 0 || W < 1) return fail(WMTP_ERR_INVALID_ARG, "window view needs n_sink >= 0 and W >= 1 (n_sink=%d W=%d)", n_sink, W);
    return WMTP_OK;
}

wmtp_status wmtp_draft_attn_windowed_kv(const void* q, int Hq, const wmtp_kv* kv, int n_sink, int W, float sm_scale,
                                        void* out, float* lse, void* workspace, size_t ws_bytes, void* stream) {
    if (wmtp_status s = check_window(n_sink, W)) return s;
    return attn_full(q, Hq, kv, sm_scale, out, lse, workspace, ws_bytes, (cudaStream_t)stream, true, nullptr, nullptr, n_sink, W);
}

int wmtp_reduced_block_table_width(int n_sink, int W, int page_size) {
    if (n_sink < 0 || W < 1 || page_size < 1) return 0;
    return (n_sink + page_size - 1) / page_size + (W + page_size - 1) / page_size + 1;
}

wmtp_status wmtp_reduced_block_table(const wmtp_kv* kv, int n_sink, int W, int32_t* table, int table_stride, int32_t* meta,
                                     void* workspace, void* stream) {
    if (wmtp_status s = check_window(n_sink, W)) return s;
    if (wmtp_status s = check_kv(kv)) return s;
    if (!kv->page_table) return fail(WMTP_ERR_INVALID_ARG, "a reduced block table needs a paged store");
    if (!table || !meta || !aligned(table, 4) || !aligned(meta, 4)) return fail(WMTP_ERR_INVALID_ARG, "table or meta is NULL or misaligned");
    if (table_stride < wmtp_reduced_block_table_width(n_sink, W, kv->page_size))
        return fail(WMTP_ERR_CAPACITY, "table_stride=%d, %d entries per sequence needed", table_stride,
                    wmtp_reduced_block_table_width(n_sink, W, kv->page_size));
    cudaError_t e = launch_reduced_block_table(kv_params(kv), n_sink, W, table, table_stride, meta, static_cast<int*>(workspace),
                                               (cudaStream_t)stream);
    return e == cudaSuccess ? WMTP_OK : cuda_fail(e, "reduced block table launch");
}

wmtp_status wmtp_full_token_index(const wmtp_kv* kv, int32_t* index, int64_t index_stride, void* workspace, void* stream) {
    if (wmtp_status s = check_kv(kv)) return s;
    if (!kv->page_table) return fail(WMTP_ERR_INVALID_ARG, "a token index needs a paged store");
    if (!index || !aligned(index, 4)) return fail(WMTP_ERR_INVALID_ARG, "index is NULL or misaligned");
    if (index_stride < 1) return fail(WMTP_ERR_INVALID_ARG, "index_stride=%lld must be positive", (long long)index_stride);
    if ((int64_t)kv->num_pages * kv->page_size > INT32_MAX)
        return fail(WMTP_ERR_UNSUPPORTED, "pool rows do not fit the 32-bit index");
    cudaError_t e = launch_full_token_index(kv_params(kv), index, index_stride, static_cast<int*>(workspace), (cudaStream_t)stream);
    return e == cudaSuccess ? WMTP_OK : cuda_fail(e, "token index launch");
}

wmtp_status wmtp_draft_loop_windowed_kv(const wmtp_kv* kv, int n_sink, int W, int gamma, const void* q, int Hq,
                                        const void* k_new, const void* v_new, float sm_scale, void* out, float* lse,
                                        void* workspace, size_t ws_bytes, void* stream) {
    if (wmtp_status s = check_window(n_sink, W)) return s;
    if (wmtp_status s = check_kv(kv)) return s;
    if (wmtp_status s = check_loop(gamma, k_new, v_new)) return s;
    if (wmtp_status s = check_attn_common(q, Hq, kv->Hkv, kv->batch, kv->D, out, lse, workspace, ws_bytes)) return s;
    const size_t q_step = (size_t)kv->batch * Hq * kv->D * 2, kv_step = (size_t)kv->batch * kv->Hkv * kv->D * 2;
    MapCache cache;
    for (int i = 0; i < gamma; ++i) {
        if (wmtp_status s = attn_full((const char*)q + i * q_step, Hq, kv, sm_scale, (char*)out + i * q_step,
                                      lse ? lse + (size_t)i * kv->batch * Hq : nullptr, workspace, ws_bytes,
                                      (cudaStream_t)stream, false, (const char*)k_new + i * kv_step,
                                      (const char*)v_new + i * kv_step, n_sink, W, 1, &cache))
            return s;
    }
    return WMTP_OK;
}

size_t wmtp_stage_bytes(int gamma, int batch, int Hq, int Hkv, int D) {
    if (gamma < 1 || batch < 1 || Hq < 1 || Hkv < 1 || D < 1) return 0;
    return stage_plan(gamma, batch, Hq, Hkv, D).total;
}

static wmtp_status loop_host(const wmtp_ring* ring, const wmtp_kv* kv, int gamma, const void* qh, int Hq, const void* kh,
                             const void* vh, float sm_scale, void* outh, float* lseh, void* stage, void* ws,
                             size_t ws_bytes, void* stream) {
    const int batch = ring ? ring->batch : kv->batch, Hkv = ring ? ring->Hkv : kv->Hkv, D = ring ? ring->D : kv->D;
    if (!qh || !kh || !vh || !outh) return fail(WMTP_ERR_INVALID_ARG, "a host pointer is NULL");
    if (!stage || !aligned(stage, 256)) return fail(WMTP_ERR_INVALID_ARG, "stage is NULL or not 256-byte aligned");
    if (gamma < 1 || Hq < 1) return fail(WMTP_ERR_INVALID_ARG, "gamma and Hq must be positive");
    const StagePlan sp = stage_plan(gamma, batch, Hq, Hkv, D);
    const size_t qb = (size_t)gamma * batch * Hq * D * 2, kb = (size_t)gamma * batch * Hkv * D * 2;
    char* sb = static_cast<char*>(stage);
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e;
    if ((e = cudaMemcpyAsync(sb + sp.q, qh, qb, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_fail(e, "H2D q");
    if ((e = cudaMemcpyAsync(sb + sp.k, kh, kb, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_fail(e, "H2D k_new");
    if ((e = cudaMemcpyAsync(sb + sp.v, vh, kb, cudaMemcpyHostToDevice, st)) != cudaSuccess) return cuda_fail(e, "H2D v_new");
    float* lse_d = lseh ? reinterpret_cast<float*>(sb + sp.lse) : nullptr;
    wmtp_status s = ring ? wmtp_draft_loop_windowed(ring, gamma, sb + sp.q, Hq, sb + sp.k, sb + sp.v, sm_scale, sb + sp.out,
                                                    lse_d, ws, ws_bytes, stream)
                         : wmtp_draft_loop_full(kv, gamma, sb + sp.q, Hq, sb + sp.k, sb + sp.v, sm_scale, sb + sp.out, lse_d,
                                                ws, ws_bytes, stream);
    if (s != WMTP_OK) return s;
    if ((e = cudaMemcpyAsync(outh, sb + sp.out, qb, cudaMemcpyDeviceToHost, st)) != cudaSuccess) return cuda_fail(e, "D2H out");
    if (lseh && (e = cudaMemcpyAsync(lseh, lse_d, (size_t)gamma * batch * Hq * 4, cudaMemcpyDeviceToHost, st)) != cudaSuccess)
        return cuda_fail(e, "D2H lse");
    if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return cuda_fail(e, "stream synchronize");
    return WMTP_OK;
}

wmtp_status wmtp_draft_loop_windowed_host(const wmtp_ring* ring, int gamma, const void* q_host, int Hq,
                                          const void* k_new_host, const void* v_new_host, float sm_scale, void* out_host,
                                          float* lse_host, void* stage, void* workspace, size_t ws_bytes, void* stream) {
    if (wmtp_status s = check_ring(ring)) return s;
    return loop_host(ring, nullptr, gamma, q_host, Hq, k_new_host, v_new_host, sm_scale, out_host, lse_host, stage,
                     workspace, ws_bytes, stream);
}

wmtp_status wmtp_draft_loop_full_host(const wmtp_kv* kv, int gamma, const void* q_host, int Hq, const void* k_new_host,
                                      const void* v_new_host, float sm_scale, void* out_host, float* lse_host, void* stage,
                                      void* workspace, size_t ws_bytes, void* stream) {
    if (wmtp_status s = check_kv(kv)) return s;
    return loop_host(nullptr, kv, gamma, q_host, Hq, k_new_host, v_new_host, sm_scale, out_host, lse_host, stage, workspace,
                     ws_bytes, stream);
}

wmtp_status wmtp_attn_mass_diagnostics(const void* out_win, const float* lse_win, const void* out_full, const float* lse_full,
                                       int rows, int D, float* mass, float* perturb, float* tail, void* stream) {
    if (!out_win || !lse_win || !out_full || !lse_full) return fail(WMTP_ERR_INVALID_ARG, "an input pointer is NULL");
    if (!mass && !perturb && !tail) return fail(WMTP_ERR_INVALID_ARG, "no output requested");
    if (rows < 1 || D < 2 || D % 2 != 0) return fail(WMTP_ERR_INVALID_ARG, "rows=%d must be positive and D=%d even", rows, D);
    if (!aligned(out_win, 4) || !aligned(out_full, 4)) return fail(WMTP_ERR_INVALID_ARG, "outputs of attention must be 4-byte aligned");
    cudaError_t e = launch_mass_diagnostics(out_win, lse_win, out_full, lse_full, rows, D, mass, perturb, tail, (cudaStream_t)stream);
    return e == cudaSuccess ? WMTP_OK : cuda_fail(e, "mass diagnostics launch");
}

void wmtp_set_max_ctas(int max_ctas) { g_max_ctas.store(max_ctas < 0 ? 0 : max_ctas); }

void wmtp_set_work_stealing(int enabled) { g_stealing.store(enabled ? 1 : 0); }

void wmtp_set_wait_limit(int polls) { g_wait_limit.store(polls > 0 ? (uint32_t)polls : 0u); }

int64_t wmtp_launch_count(void) { return g_launches.load(); }

// ---- allocation-free windowed attention ---------------------------------------------------------
// Some callers cannot hand the library a workspace because they cannot call cudaMalloc at all: code
// running inside a framework that owns the device allocator, a process whose memory budget is fixed
// before start-up, a real-time loop where an allocation is forbidden after initialisation. For them
// the split-KV scratch of the windowed attention lives in this file-scope device array instead of a
// caller buffer. Every GPU that loads the library holds it until the process exits.
namespace {
constexpr int kStaticMaxCtas = kMaxCtas;   // CTAs (KV splits) the static scratch has room for
constexpr int kStaticMaxSegments = 32;     // batch * Hkv
constexpr size_t kStaticCountersOff = 256 + kCursorBytes;
constexpr size_t kStaticZeroBytes = kStaticCountersOff + 2 * (8 + 4 + 4) * kStaticMaxSegments;   // header, cursors, two copies of the per-segment words
// Partial slots: with the fixed partition a segment receives at most one partial per consumer group of every CTA whose
// range meets it; the kernel reserves kMaxGroups * (own + 1) slots per segment with own <= CTAs * tiles_b / tiles + 2,
// which sums to at most kMaxGroups * (CTAs + 3 * segments) over a launch.
constexpr size_t kStaticSlots = (size_t)kMaxGroups * (kStaticMaxCtas + 3 * kStaticMaxSegments);
constexpr size_t kStaticPartKeyOff = kStaticZeroBytes;                        // int [kStaticSlots]
constexpr size_t kStaticPartLseOff = kStaticPartKeyOff + kStaticSlots * sizeof(int);
constexpr size_t kStaticPartOOff = kStaticPartLseOff + kStaticSlots * kMaxGroup * sizeof(float);
constexpr size_t kStaticBytes = kStaticPartOOff + kStaticSlots * kMaxGroup * 256 * sizeof(float);
static_assert(kStaticMaxCtas >= kMaxCtas, "the launcher may use up to kMaxCtas CTAs");
static_assert(kStaticSlots >= (size_t)kMaxGroups * (kMaxCtas + 3 * kStaticMaxSegments), "partial slots of the largest accepted launch");
static_assert(kStaticPartKeyOff % 256 == 0 && kStaticPartLseOff % 256 == 0 && kStaticPartOOff % 256 == 0,
              "static scratch regions must stay 256-byte aligned");
static_assert(kStaticMaxSegments <= kMaxSegments, "per-segment words");

static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];   // ~4 MiB

// In host code the array's name is only a handle; the device address must be asked for, once per device.
std::mutex g_static_mu;
void* g_static_ptr[64] = {};

wmtp_status static_scratch(void** ptr) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= 64) return fail(WMTP_ERR_UNSUPPORTED, "device ordinal %d is outside [0, 64)", dev);
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_ptr[dev]) {
        void* a = nullptr;
        e = cudaGetSymbolAddress(&a, g_static_scratch);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(static scratch)");
        g_static_ptr[dev] = a;
    }
    *ptr = g_static_ptr[dev];
    return WMTP_OK;
}
}  // namespace

wmtp_status wmtp_draft_attn_windowed_noalloc(const void* q, int Hq, const wmtp_ring* ring, float sm_scale, void* out,
                                             float* lse, void* stream) {
    if (wmtp_status s = check_ring(ring)) return s;
    if (!q || !out) return fail(WMTP_ERR_INVALID_ARG, "q or out is NULL");
    if (!aligned(q, 16) || !aligned(out, 16)) return fail(WMTP_ERR_INVALID_ARG, "q and out must be 16-byte aligned");
    if (lse && !aligned(lse, 4)) return fail(WMTP_ERR_INVALID_ARG, "lse must be 4-byte aligned");
    if (Hq < 1 || Hq % ring->Hkv != 0) return fail(WMTP_ERR_INVALID_ARG, "Hq=%d must be a positive multiple of Hkv=%d", Hq, ring->Hkv);
    if (Hq / ring->Hkv > kMaxGroup) return fail(WMTP_ERR_UNSUPPORTED, "Hq/Hkv=%d exceeds %d", Hq / ring->Hkv, kMaxGroup);
    const int nseg = ring->batch * ring->Hkv;
    if (nseg > kStaticMaxSegments)
        return fail(WMTP_ERR_CAPACITY, "batch*Hkv=%d exceeds the %d (sequence, KV head) pairs the built-in scratch holds; "
                    "use wmtp_draft_attn_windowed with a workspace", nseg, kStaticMaxSegments);
    void* base_v = nullptr;
    if (wmtp_status s = static_scratch(&base_v)) return s;
    char* base = static_cast<char*>(base_v);
    cudaStream_t st = (cudaStream_t)stream;
    // status word and this call's counters must start at zero; the array keeps the previous call's contents
    cudaError_t e = cudaMemsetAsync(base, 0, kStaticZeroBytes, st);
    if (e != cudaSuccess) return cuda_fail(e, "clearing the static scratch header");

    AttnParams p{};
    // static partition: deterministic and the smallest partial pool
    fill_attn(p, q, Hq, ring->Hkv, ring->batch, ring->D, sm_scale, out, lse, base,
              ScratchLayout{kStaticCountersOff, kStaticMaxSegments, kStaticPartKeyOff, kStaticPartLseOff, kStaticPartOOff}, false);
    bind_ring(p, ring, nullptr, nullptr);
    const int64_t tiles = (p.rows_per_head + kTileKeys - 1) / kTileKeys * ring->batch * ring->Hkv;
    p.num_ctas = pick_ctas(tiles);
    if (p.num_ctas <= 0) return fail(WMTP_ERR_CUDA, "no CUDA device available");
    if (p.num_ctas > kStaticMaxCtas) p.num_ctas = kStaticMaxCtas;
    e = launch_with(p, nullptr, st);
    if (e != cudaSuccess) return cuda_fail(e, "windowed attention launch (static scratch)");
    return WMTP_OK;
}

}  // extern "C"
