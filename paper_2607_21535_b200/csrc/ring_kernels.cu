// Ring-buffer draft KV store and full-context KV append kernels.
//
// Slot rule (Section 4 "Memory"; Appendix A, RING comment, read with the sink kept fixed):
// position p lives in slot p when p < n_sink, else in n_sink + ((p - n_sink) mod cap).
// All of this is integer work and copies -- bit-exact by construction -- except the quantisation of new rows for an
// fp8 store, which is defined to the bit (fp32 division, round to nearest even, saturation; fp8_util.cuh).
#include "wmtp_internal.h"
#include "fp8_util.cuh"

namespace wmtp {

namespace {

constexpr int kErrBounds = WMTP_ERR_DEVICE_BOUNDS;

// 16-byte vectors of one stored row of head_dim D: 8 bf16 or 16 e4m3 codes each.
__device__ __forceinline__ int store_vecs(int D, int f8) { return f8 ? D / 16 : D / 8; }
// Vector c of the stored form of a bf16 source row (`src`: its D / 8 vectors): a copy, or its e4m3 codes.
__device__ __forceinline__ uint4 stored_vec(const uint4* __restrict__ src, int c, int f8, float scale) {
    if (!f8) return src[c];
    return quant16_e4m3(src[2 * c], src[2 * c + 1], scale);
}

__device__ __forceinline__ int ring_slot(int64_t p, int n_sink, int cap) {
    return p < n_sink ? (int)p : n_sink + (int)((p - n_sink) % cap);
}

// Position held by window slot `s` (s >= n_sink) of a ring of logical length S, or -1.
__device__ __forceinline__ int64_t ring_slot_position(int s, int64_t S, int n_sink, int cap) {
    if (s < n_sink) return s < S ? (int64_t)s : -1;
    if (S <= n_sink) return -1;
    const int64_t last = S - 1 - n_sink;          // window-relative index of the newest token
    const int cur = (int)(last % cap);
    int age = cur - (s - n_sink);
    if (age < 0) age += cap;
    return (int64_t)age <= last ? S - 1 - age : -1;
}

__global__ void ring_reset_kernel(RingParams r) {
    const int slots = r.n_sink + r.cap;
    const int64_t n = (int64_t)r.B * slots;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        r.slot_pos[i] = -1;
    if (blockIdx.x == 0)
        for (int b = threadIdx.x; b < r.B; b += blockDim.x) r.len[b] = 0;
}

// One block per sequence; thread t writes 16 bytes of the token's [Hkv][D] K row and V row (copied, or quantised to
// e4m3 codes for an fp8 store).
__global__ void ring_append_kernel(RingParams r, const uint4* __restrict__ k_new, const uint4* __restrict__ v_new) {
    const int b = blockIdx.x;
    const int64_t p = r.len[b];
    const int slots = r.n_sink + r.cap;
    const int slot = ring_slot(p, r.n_sink, r.cap);
    const int vec_per_row = store_vecs(r.D, r.f8), src_vecs = r.D / 8;
    const int n_vec = r.Hkv * vec_per_row;
    uint4* K = reinterpret_cast<uint4*>(r.k);
    uint4* V = reinterpret_cast<uint4*>(r.v);
    for (int i = threadIdx.x; i < n_vec; i += blockDim.x) {
        const int g = i / vec_per_row, c = i % vec_per_row;
        const int64_t dst = (((int64_t)b * r.Hkv + g) * slots + slot) * vec_per_row + c;
        const int64_t src = ((int64_t)b * r.Hkv + g) * src_vecs;
        K[dst] = stored_vec(k_new + src, c, r.f8, r.f8 ? r.k_scale[g] : 1.f);
        V[dst] = stored_vec(v_new + src, c, r.f8, r.f8 ? r.v_scale[g] : 1.f);
    }
    __syncthreads();   // every thread has read len[b] before it moves
    if (threadIdx.x == 0) {
        r.slot_pos[(int64_t)b * slots + slot] = (int32_t)p;
        r.len[b] = p + 1;
    }
}

__device__ __forceinline__ int64_t kv_row_vec(const KvParams& kv, int b, int g, int64_t p, int vec_per_row, bool* ok) {
    if (kv.page_table == nullptr) return (((int64_t)b * kv.Hkv + g) * kv.S_cap + p) * vec_per_row;
    const int page = kv.page_table[(int64_t)b * kv.max_pages + p / kv.page_size];
    if (page < 0 || page >= kv.num_pages) { *ok = false; return 0; }
    return (((int64_t)page * kv.Hkv + g) * kv.page_size + p % kv.page_size) * vec_per_row;
}

__global__ void kv_append_kernel(KvParams kv, const uint4* __restrict__ k_new, const uint4* __restrict__ v_new, int* status) {
    const int b = blockIdx.x;
    const int64_t p = kv.len[b];
    const int vec_per_row = store_vecs(kv.D, kv.f8), src_vecs = kv.D / 8;
    const int n_vec = kv.Hkv * vec_per_row;
    __shared__ int bad;
    if (threadIdx.x == 0) bad = 0;
    __syncthreads();
    if (p >= kv.S_cap) {
        if (threadIdx.x == 0 && status) atomicCAS(status, 0, kErrBounds);
        return;
    }
    uint4* K = reinterpret_cast<uint4*>(kv.k);
    uint4* V = reinterpret_cast<uint4*>(kv.v);
    for (int i = threadIdx.x; i < n_vec; i += blockDim.x) {
        const int g = i / vec_per_row, c = i % vec_per_row;
        bool ok = true;
        const int64_t dst = kv_row_vec(kv, b, g, p, vec_per_row, &ok) + c;
        if (!ok) { bad = 1; continue; }
        const int64_t src = ((int64_t)b * kv.Hkv + g) * src_vecs;
        K[dst] = stored_vec(k_new + src, c, kv.f8, kv.f8 ? kv.k_scale[g] : 1.f);
        V[dst] = stored_vec(v_new + src, c, kv.f8, kv.f8 ? kv.v_scale[g] : 1.f);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        if (bad) { if (status) atomicCAS(status, 0, kErrBounds); }
        else kv.len[b] = p + 1;
    }
}

// grid (ceil(slots / slots_per_block), B); each warp copies whole slots.
__global__ void ring_init_kernel(RingParams r, KvParams kv) {
    const int b = blockIdx.y;
    const int slots = r.n_sink + r.cap;
    const int64_t S = kv.len[b];
    const int vec_per_row = store_vecs(r.D, r.f8);           // rows are copied as stored (same dtype and scales on both sides)
    const int warps = blockDim.x / 32, warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const uint4* Ksrc = reinterpret_cast<const uint4*>(kv.k);
    const uint4* Vsrc = reinterpret_cast<const uint4*>(kv.v);
    uint4* K = reinterpret_cast<uint4*>(r.k);
    uint4* V = reinterpret_cast<uint4*>(r.v);
    for (int s = blockIdx.x * warps + warp; s < slots; s += gridDim.x * warps) {
        const int64_t p = ring_slot_position(s, S, r.n_sink, r.cap);
        bool page_ok = true;
        if (p >= 0) kv_row_vec(kv, b, 0, p, vec_per_row, &page_ok);
        // a position whose page id is out of range cannot be copied: the slot is marked empty rather than claimed
        if (lane == 0) r.slot_pos[(int64_t)b * slots + s] = page_ok ? (int32_t)p : -1;
        if (p < 0 || !page_ok) continue;
        for (int g = 0; g < r.Hkv; ++g) {
            bool ok = true;
            const int64_t src = kv_row_vec(kv, b, g, p, vec_per_row, &ok);
            if (!ok) continue;
            const int64_t dst = (((int64_t)b * r.Hkv + g) * slots + s) * vec_per_row;
            for (int c = lane; c < vec_per_row; c += 32) {
                K[dst + c] = Ksrc[src + c];
                V[dst + c] = Vsrc[src + c];
            }
        }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) r.len[b] = S;
}


// n_tok tokens per sequence in one launch (the accepted tokens of a decode step, re-processed by the draft):
// token j goes to position len + j. One block per sequence; k_new / v_new are [B][n_tok][Hkv][D].
__global__ void ring_append_many_kernel(RingParams r, int n_tok, const uint4* __restrict__ k_new, const uint4* __restrict__ v_new) {
    const int b = blockIdx.x;
    const int64_t p0 = r.len[b];
    const int slots = r.n_sink + r.cap;
    const int vec_per_row = store_vecs(r.D, r.f8), src_vecs = r.D / 8;
    const int n_vec = r.Hkv * vec_per_row;
    uint4* K = reinterpret_cast<uint4*>(r.k);
    uint4* V = reinterpret_cast<uint4*>(r.v);
    for (int idx = threadIdx.x; idx < n_tok * n_vec; idx += blockDim.x) {
        const int j = idx / n_vec, i = idx % n_vec;
        const int g = i / vec_per_row, c = i % vec_per_row;
        const int slot = ring_slot(p0 + j, r.n_sink, r.cap);
        const int64_t dst = (((int64_t)b * r.Hkv + g) * slots + slot) * vec_per_row + c;
        const int64_t src = (((int64_t)b * n_tok + j) * r.Hkv + g) * src_vecs;
        K[dst] = stored_vec(k_new + src, c, r.f8, r.f8 ? r.k_scale[g] : 1.f);
        V[dst] = stored_vec(v_new + src, c, r.f8, r.f8 ? r.v_scale[g] : 1.f);
    }
    __syncthreads();   // every thread has read len[b] before it moves
    for (int j = threadIdx.x; j < n_tok; j += blockDim.x)
        r.slot_pos[(int64_t)b * slots + ring_slot(p0 + j, r.n_sink, r.cap)] = (int32_t)(p0 + j);
    if (threadIdx.x == 0) r.len[b] = p0 + n_tok;
}

__global__ void kv_append_many_kernel(KvParams kv, int n_tok, const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                                      int* status) {
    const int b = blockIdx.x;
    const int64_t p0 = kv.len[b];
    const int vec_per_row = store_vecs(kv.D, kv.f8), src_vecs = kv.D / 8;
    const int n_vec = kv.Hkv * vec_per_row;
    __shared__ int bad;
    if (threadIdx.x == 0) bad = 0;
    __syncthreads();
    if (p0 + n_tok > kv.S_cap) {                     // all or nothing: a partial append would leave len ambiguous
        if (threadIdx.x == 0 && status) atomicCAS(status, 0, kErrBounds);
        return;
    }
    uint4* K = reinterpret_cast<uint4*>(kv.k);
    uint4* V = reinterpret_cast<uint4*>(kv.v);
    for (int idx = threadIdx.x; idx < n_tok * n_vec; idx += blockDim.x) {
        const int j = idx / n_vec, i = idx % n_vec;
        const int g = i / vec_per_row, c = i % vec_per_row;
        bool ok = true;
        const int64_t dst = kv_row_vec(kv, b, g, p0 + j, vec_per_row, &ok) + c;
        if (!ok) { bad = 1; continue; }
        const int64_t src = (((int64_t)b * n_tok + j) * kv.Hkv + g) * src_vecs;
        K[dst] = stored_vec(k_new + src, c, kv.f8, kv.f8 ? kv.k_scale[g] : 1.f);
        V[dst] = stored_vec(v_new + src, c, kv.f8, kv.f8 ? kv.v_scale[g] : 1.f);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        if (bad) { if (status) atomicCAS(status, 0, kErrBounds); }
        else kv.len[b] = p0 + n_tok;
    }
}

// Discards the last n_drop[b] tokens of every sequence (speculative tokens the target rejected; Section 4 "Memory" and
// Section 6: the ring reserves d extra slots for them). Only the bookkeeping moves: len shrinks and the slots of the
// dropped positions are marked empty; the rows they overwrote lie outside every future window as long as no more than
// cap - W tokens are dropped, which is checked.
__global__ void ring_rewind_kernel(RingParams r, const int32_t* __restrict__ n_drop, int* status) {
    const int b = blockIdx.x;
    const int64_t S = r.len[b];
    const int slots = r.n_sink + r.cap;
    const int n = n_drop[b];
    if (n < 0 || n > S || n > r.cap - r.W) {
        if (threadIdx.x == 0 && status) atomicCAS(status, 0, kErrBounds);
        return;
    }
    for (int j = threadIdx.x; j < n; j += blockDim.x)
        r.slot_pos[(int64_t)b * slots + ring_slot(S - 1 - j, r.n_sink, r.cap)] = -1;
    __syncthreads();
    if (threadIdx.x == 0) r.len[b] = S - n;
}

// The windowed draft's block table over a paged store (Section 4 "Mechanism": the per-request table reduced to
// [sink blocks] || [recent-W blocks]): O((n_sink + W) / page_size) entries per sequence from the device-resident length,
// plus the row bounds that keep the ends token-granular. One block per sequence.
__global__ void reduced_block_table_kernel(KvParams kv, int n_sink, int W, int32_t* __restrict__ table, int stride,
                                           int32_t* __restrict__ meta, int* status) {
    const int b = blockIdx.x, ps = kv.page_size;
    const int64_t S = kv.len[b];
    const int64_t ns = S < n_sink ? S : n_sink;                 // sink positions [0, ns)
    const int64_t lo = S - W > ns ? S - W : ns;                 // window positions [lo, S)
    const int n_s = (int)((ns + ps - 1) / ps);
    const int first_w = (int)(lo / ps);
    const int n_w = S > ns ? (int)((S - 1) / ps) - first_w + 1 : 0;
    const bool fits = n_s + n_w <= stride && (n_w == 0 || first_w + n_w <= kv.max_pages) && n_s <= kv.max_pages;
    if (!fits && threadIdx.x == 0 && status) atomicCAS(status, 0, kErrBounds);
    const int n = fits ? n_s + n_w : 0;
    for (int i = threadIdx.x; i < stride; i += blockDim.x) {
        int page = -1;
        if (i < n) {
            page = kv.page_table[(int64_t)b * kv.max_pages + (i < n_s ? i : first_w + i - n_s)];
            if (page < 0 || page >= kv.num_pages) { if (status) atomicCAS(status, 0, kErrBounds); page = -1; }
        }
        table[(int64_t)b * stride + i] = page;
    }
    if (threadIdx.x == 0) {
        int32_t* m = meta + (int64_t)b * 5;
        m[0] = fits ? n_s : 0;
        m[1] = fits ? n_w : 0;
        m[2] = (fits && ns > 0) ? (int)((ns - 1) % ps) + 1 : 0;         // rows used in the last sink page
        m[3] = (fits && n_w > 0) ? (int)(lo % ps) : 0;                  // first row used in the first window page
        m[4] = (fits && n_w > 0) ? (int)((S - 1) % ps) + 1 : 0;         // rows used in the last window page
    }
}

// The structure a full-context draft over a paged store rebuilds before every attention call (Appendix B, per-kernel
// table: the draft's KV index build, O(S) per step): the pool row of every token, index[b][s] = page * page_size +
// s mod page_size for s < len[b], -1 beyond. Built here to be measured against the O(W) table above; the attention
// kernels of this library walk the page table directly and need neither.
__global__ void full_token_index_kernel(KvParams kv, int32_t* __restrict__ index, int64_t stride, int vec4, int* status) {
    const int b = blockIdx.y, ps = kv.page_size;
    const int64_t S = kv.len[b];
    if (S > stride && blockIdx.x == 0 && threadIdx.x == 0 && status) atomicCAS(status, 0, kErrBounds);
    const int32_t* pt = kv.page_table + (int64_t)b * kv.max_pages;
    auto row_of = [&](int64_t s, int page) { return page * ps + (int32_t)(s % ps); };
    auto page_of = [&](int64_t s) {
        const int page = pt[s / ps];
        if (page < 0 || page >= kv.num_pages) { if (status) atomicCAS(status, 0, kErrBounds); return -1; }
        return page;
    };
    const int64_t t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x, dt = (int64_t)gridDim.x * blockDim.x;
    if (vec4) {
        // four consecutive tokens lie in one page (page_size and stride are multiples of 4): one lookup, one 16-byte store
        int4* out = reinterpret_cast<int4*>(index + (int64_t)b * stride);
        for (int64_t i = t0; i < stride / 4; i += dt) {
            const int64_t s = 4 * i;
            int4 r = make_int4(-1, -1, -1, -1);
            if (s < S) {
                const int page = page_of(s);
                if (page >= 0) {
                    const int32_t r0 = row_of(s, page);
                    r.x = r0;
                    if (s + 1 < S) r.y = r0 + 1;
                    if (s + 2 < S) r.z = r0 + 2;
                    if (s + 3 < S) r.w = r0 + 3;
                }
            }
            out[i] = r;
        }
    } else {
        for (int64_t s = t0; s < stride; s += dt) {
            int32_t row = -1;
            if (s < S) {
                const int page = page_of(s);
                if (page >= 0) row = row_of(s, page);
            }
            index[(int64_t)b * stride + s] = row;
        }
    }
}

// Rollback and append in one launch (the draft's state update after a verify step): drop the last n_drop[b] tokens, then
// append n_tok new ones at the positions that follow. Slots of dropped positions that are not rewritten are marked
// empty. Same conditions as ring_rewind_kernel; a violation leaves the sequence unchanged and is flagged.
__global__ void ring_replace_tail_kernel(RingParams r, const int32_t* __restrict__ n_drop, int n_tok, const uint4* __restrict__ k_new,
                                         const uint4* __restrict__ v_new, int* status) {
    const int b = blockIdx.x;
    const int64_t S = r.len[b];
    const int slots = r.n_sink + r.cap;
    const int n = n_drop ? n_drop[b] : 0;
    if (n < 0 || n > S || n > r.cap - r.W) {
        if (threadIdx.x == 0 && status) atomicCAS(status, 0, kErrBounds);
        return;
    }
    const int64_t p0 = S - n;
    const int vec_per_row = store_vecs(r.D, r.f8), src_vecs = r.D / 8;
    const int n_vec = r.Hkv * vec_per_row;
    uint4* K = reinterpret_cast<uint4*>(r.k);
    uint4* V = reinterpret_cast<uint4*>(r.v);
    for (int idx = threadIdx.x; idx < n_tok * n_vec; idx += blockDim.x) {
        const int j = idx / n_vec, i = idx % n_vec;
        const int g = i / vec_per_row, c = i % vec_per_row;
        const int slot = ring_slot(p0 + j, r.n_sink, r.cap);
        const int64_t dst = (((int64_t)b * r.Hkv + g) * slots + slot) * vec_per_row + c;
        const int64_t src = (((int64_t)b * n_tok + j) * r.Hkv + g) * src_vecs;
        K[dst] = stored_vec(k_new + src, c, r.f8, r.f8 ? r.k_scale[g] : 1.f);
        V[dst] = stored_vec(v_new + src, c, r.f8, r.f8 ? r.v_scale[g] : 1.f);
    }
    __syncthreads();   // every thread has read len[b] before it moves
    const int m = n > n_tok ? n : n_tok;
    for (int j = threadIdx.x; j < m; j += blockDim.x)
        r.slot_pos[(int64_t)b * slots + ring_slot(p0 + j, r.n_sink, r.cap)] = j < n_tok ? (int32_t)(p0 + j) : -1;
    if (threadIdx.x == 0) r.len[b] = p0 + n_tok;
}

__device__ __forceinline__ float bf16_bits_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_bits_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// One warp per (sequence, query head) row: attention-mass diagnostics of a windowed against a full read-out
// (Appendix D): mu = exp(lse_win - lse_full), ||o_full - o_win|| / ||o_full||, ||o_full - mu o_win|| / ||o_full||.
__global__ void mass_diagnostics_kernel(const uint32_t* __restrict__ o_win, const float* __restrict__ lse_win,
                                        const uint32_t* __restrict__ o_full, const float* __restrict__ lse_full, int rows,
                                        int D, float* __restrict__ mass, float* __restrict__ perturb, float* __restrict__ tail) {
    const int row = blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32, lane = threadIdx.x % 32;
    if (row >= rows) return;
    const float lw = lse_win[row], lf = lse_full[row];
    const float mu = (lf == -INFINITY) ? 0.f : __expf(lw - lf);
    float n_full = 0.f, n_diff = 0.f, n_far = 0.f;
    for (int w = lane; w < D / 2; w += 32) {
        const uint32_t a = o_win[(int64_t)row * (D / 2) + w], b = o_full[(int64_t)row * (D / 2) + w];
        const float w0 = bf16_bits_lo(a), w1 = bf16_bits_hi(a), f0 = bf16_bits_lo(b), f1 = bf16_bits_hi(b);
        n_full += f0 * f0 + f1 * f1;
        n_diff += (f0 - w0) * (f0 - w0) + (f1 - w1) * (f1 - w1);
        n_far += (f0 - mu * w0) * (f0 - mu * w0) + (f1 - mu * w1) * (f1 - mu * w1);
    }
    for (int off = 16; off > 0; off >>= 1) {
        n_full += __shfl_xor_sync(0xffffffffu, n_full, off);
        n_diff += __shfl_xor_sync(0xffffffffu, n_diff, off);
        n_far += __shfl_xor_sync(0xffffffffu, n_far, off);
    }
    if (lane == 0) {
        const float inv = n_full > 0.f ? rsqrtf(n_full) : 0.f;
        if (mass) mass[row] = mu;
        if (perturb) perturb[row] = sqrtf(n_diff) * inv;
        if (tail) tail[row] = sqrtf(n_far) * inv;
    }
}

}  // namespace

cudaError_t launch_ring_reset(const RingParams& r, cudaStream_t st) {
    const int64_t n = (int64_t)r.B * (r.n_sink + r.cap);
    const int blocks = (int)((n + 255) / 256 < 1 ? 1 : ((n + 255) / 256 > 1184 ? 1184 : (n + 255) / 256));
    ring_reset_kernel<<<blocks, 256, 0, st>>>(r);
    count_launch(1);
    return cudaGetLastError();
}

cudaError_t launch_ring_append(const RingParams& r, const void* k_new, const void* v_new, cudaStream_t st) {
    const int n_vec = r.Hkv * r.D / (r.f8 ? 16 : 8);
    const int threads = n_vec < 32 ? 32 : (n_vec > 256 ? 256 : (n_vec + 31) / 32 * 32);
    ring_append_kernel<<<r.B, threads, 0, st>>>(r, (const uint4*)k_new, (const uint4*)v_new);
    count_launch(1);
    return cudaGetLastError();
}

cudaError_t launch_kv_append(const KvParams& kv, const void* k_new, const void* v_new, int* status, cudaStream_t st) {
    const int n_vec = kv.Hkv * kv.D / (kv.f8 ? 16 : 8);
    const int threads = n_vec < 32 ? 32 : (n_vec > 256 ? 256 : (n_vec + 31) / 32 * 32);
    kv_append_kernel<<<kv.B, threads, 0, st>>>(kv, (const uint4*)k_new, (const uint4*)v_new, status);
    count_launch(1);
    return cudaGetLastError();
}

cudaError_t launch_ring_init_from_kv(const RingParams& r, const KvParams& kv, cudaStream_t st) {
    const int slots = r.n_sink + r.cap;
    const int warps = 8;
    int bx = (slots + warps - 1) / warps;
    if (bx > 592) bx = 592;
    dim3 grid(bx, r.B);
    ring_init_kernel<<<grid, warps * 32, 0, st>>>(r, kv);
    count_launch(1);
    return cudaGetLastError();
}

cudaError_t launch_mass_diagnostics(const void* o_win, const float* lse_win, const void* o_full, const float* lse_full, int rows,
                                    int D, float* mass, float* perturb, float* tail, cudaStream_t st) {
    const int warps = 4;
    mass_diagnostics_kernel<<<(rows + warps - 1) / warps, warps * 32, 0, st>>>((const uint32_t*)o_win, lse_win, (const uint32_t*)o_full,
                                                                             lse_full, rows, D, mass, perturb, tail);
    count_launch(1);
    return cudaGetLastError();
}

cudaError_t launch_ring_append_many(const RingParams& r, int n_tok, const void* k_new, const void* v_new, cudaStream_t st) {
    ring_append_many_kernel<<<r.B, 256, 0, st>>>(r, n_tok, (const uint4*)k_new, (const uint4*)v_new);
    count_launch(1);
    return cudaGetLastError();
}

cudaError_t launch_kv_append_many(const KvParams& kv, int n_tok, const void* k_new, const void* v_new, int* status, cudaStream_t st) {
    kv_append_many_kernel<<<kv.B, 256, 0, st>>>(kv, n_tok, (const uint4*)k_new, (const uint4*)v_new, status);
    count_launch(1);
    return cudaGetLastError();
}

cudaError_t launch_reduced_block_table(const KvParams& kv, int n_sink, int W, int32_t* table, int stride, int32_t* meta, int* status,
                                       cudaStream_t st) {
    reduced_block_table_kernel<<<kv.B, 128, 0, st>>>(kv, n_sink, W, table, stride, meta, status);
    count_launch(1);
    return cudaGetLastError();
}

cudaError_t launch_full_token_index(const KvParams& kv, int32_t* index, int64_t stride, int* status, cudaStream_t st) {
    const int vec4 = kv.page_size % 4 == 0 && stride % 4 == 0 && reinterpret_cast<uintptr_t>(index) % 16 == 0;
    const int64_t per_seq = ((vec4 ? stride / 4 : stride) + 255) / 256;
    const unsigned gx = (unsigned)(per_seq < 1 ? 1 : (per_seq > 1024 ? 1024 : per_seq));
    full_token_index_kernel<<<dim3(gx, kv.B), 256, 0, st>>>(kv, index, stride, vec4, status);
    count_launch(1);
    return cudaGetLastError();
}

cudaError_t launch_ring_replace_tail(const RingParams& r, const int32_t* n_drop, int n_tok, const void* k_new, const void* v_new,
                                     int* status, cudaStream_t st) {
    ring_replace_tail_kernel<<<r.B, 256, 0, st>>>(r, n_drop, n_tok, (const uint4*)k_new, (const uint4*)v_new, status);
    count_launch(1);
    return cudaGetLastError();
}

cudaError_t launch_ring_rewind(const RingParams& r, const int32_t* n_drop, int* status, cudaStream_t st) {
    ring_rewind_kernel<<<r.B, 32, 0, st>>>(r, n_drop, status);
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace wmtp
