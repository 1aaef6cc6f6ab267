// Split-KV decode attention for the draft head: partial kernel + log-sum-exp combine.
//
// The operation is softmax attention of one query per head over a key set (Section 4
// "Mechanism"; Appendix D: o = sum_j p_j v_j): the ring's live slots for the windowed draft,
// all S positions for the full-context (native) draft of Section 3.
#include <cuda_bf16.h>

#include "attn_plan.cuh"

namespace wmtp {

namespace {

constexpr int kErrBounds = WMTP_ERR_DEVICE_BOUNDS;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ float bf16lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// ---------------------------------------------------------------------------------------------
// Partial kernel, CUDA-core version: one warp per key row, lanes split head_dim, all G query
// heads of the group share every K/V row that is loaded.
// ---------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(128) attn_partial_simple(AttnParams p) {
    constexpr int EPL = D / 32;             // elements per lane (4 or 8)
    constexpr int WPL = EPL / 2;            // 32-bit words per lane
    constexpr int NW = 4;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    int64_t* tile_prefix = reinterpret_cast<int64_t*>(smem_raw);                 // [B + 1]
    float* sm_m = reinterpret_cast<float*>(tile_prefix + (p.B + 1));             // [NW][8]
    float* sm_l = sm_m + NW * kMaxGroup;                                         // [NW][8]
    float* sm_acc = sm_l + NW * kMaxGroup;                                       // [NW][8][D]

    build_tile_prefix(p, tile_prefix);
    const int C = gridDim.x;
    const int64_t n = (int64_t)p.Hkv * tile_prefix[p.B];
    if (n == 0) return;
    const int64_t t0 = cta_range_start(blockIdx.x, n, C), t1 = cta_range_start(blockIdx.x + 1, n, C);
    if (t0 >= t1) return;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = p.G;
    const __nv_bfloat16* Q = reinterpret_cast<const __nv_bfloat16*>(p.q);

    int64_t t = t0;
    while (t < t1) {
        // ---- locate the segment (b, g) of tile t and the end of this CTA's share of it
        const int b = find_seq(tile_prefix, p.B, p.Hkv, t);
        const int64_t tiles_b = tile_prefix[b + 1] - tile_prefix[b];
        const int64_t seq_start = (int64_t)p.Hkv * tile_prefix[b];
        const int g = (int)((t - seq_start) / tiles_b);
        const int64_t seg_start = seq_start + (int64_t)g * tiles_b;
        const int64_t seg_end = seg_start + tiles_b;
        const int64_t t_end = seg_end < t1 ? seg_end : t1;
        const int64_t S = p.len[b];
        const int64_t nk = scan_keys(p, b);
        const int seg = b * p.Hkv + g;

        // ---- query rows of this group, pre-scaled to the exp2 domain
        float qf[kMaxGroup][EPL];
#pragma unroll
        for (int hh = 0; hh < kMaxGroup; ++hh) {
            if (hh < G) {
                const __nv_bfloat16* qrow = Q + ((int64_t)b * p.Hq + g * G + hh) * D + lane * EPL;
#pragma unroll
                for (int e = 0; e < EPL; ++e) qf[hh][e] = __bfloat162float(qrow[e]) * p.scale_log2;
            } else {
#pragma unroll
                for (int e = 0; e < EPL; ++e) qf[hh][e] = 0.f;
            }
        }
        float m[kMaxGroup], l[kMaxGroup], acc[kMaxGroup][EPL];
#pragma unroll
        for (int hh = 0; hh < kMaxGroup; ++hh) {
            m[hh] = -INFINITY; l[hh] = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) acc[hh][e] = 0.f;
        }

        for (int64_t tt = t; tt < t_end; ++tt) {
            const int64_t key0 = (tt - seg_start) * kTileKeys;
            int64_t row_base;     // element offset of the tile's first row for this KV head
            if (p.mode == kPaged) {
                const int page = p.page_table[(int64_t)b * p.max_pages + key0 / p.page_size];
                if (page < 0 || page >= p.num_pages) {
                    if (threadIdx.x == 0) atomicCAS(p.status, 0, kErrBounds);
                    continue;
                }
                row_base = ((int64_t)page * p.Hkv + g) * p.page_size * D;
            } else {
                row_base = (((int64_t)b * p.Hkv + g) * p.rows_per_head + key0) * D;
            }
            for (int kk = warp; kk < kTileKeys; kk += NW) {
                const int64_t key = key0 + kk;
                if (key >= nk) break;
                if (p.mode == kRing && p.cap != p.W && !ring_slot_live((int)key, S, p.n_sink, p.W, p.cap)) continue;
                const uint32_t* krow = reinterpret_cast<const uint32_t*>(
                    reinterpret_cast<const __nv_bfloat16*>(p.k) + row_base + (int64_t)kk * D) + lane * WPL;
                const uint32_t* vrow = reinterpret_cast<const uint32_t*>(
                    reinterpret_cast<const __nv_bfloat16*>(p.v) + row_base + (int64_t)kk * D) + lane * WPL;
                uint32_t kw[WPL], vw[WPL];
#pragma unroll
                for (int w = 0; w < WPL; ++w) { kw[w] = __ldg(krow + w); vw[w] = __ldg(vrow + w); }
                float s[kMaxGroup];
#pragma unroll
                for (int hh = 0; hh < kMaxGroup; ++hh) {
                    float a = 0.f;
#pragma unroll
                    for (int w = 0; w < WPL; ++w) {
                        a = fmaf(qf[hh][2 * w], bf16lo(kw[w]), a);
                        a = fmaf(qf[hh][2 * w + 1], bf16hi(kw[w]), a);
                    }
                    s[hh] = a;
                }
#pragma unroll
                for (int off = 16; off > 0; off >>= 1)
#pragma unroll
                    for (int hh = 0; hh < kMaxGroup; ++hh) s[hh] += __shfl_xor_sync(0xffffffffu, s[hh], off);
#pragma unroll
                for (int hh = 0; hh < kMaxGroup; ++hh) {
                    const float mn = fmaxf(m[hh], s[hh]);
                    const float corr = exp2f(m[hh] - mn);      // exp2(-inf) = 0 on the first key
                    const float pj = exp2f(s[hh] - mn);
                    m[hh] = mn;
                    l[hh] = l[hh] * corr + pj;
#pragma unroll
                    for (int w = 0; w < WPL; ++w) {
                        acc[hh][2 * w] = fmaf(pj, bf16lo(vw[w]), acc[hh][2 * w] * corr);
                        acc[hh][2 * w + 1] = fmaf(pj, bf16hi(vw[w]), acc[hh][2 * w + 1] * corr);
                    }
                }
            }
        }

        // ---- merge the four warps' states and emit the partial of (this CTA, this segment)
        __syncthreads();
#pragma unroll
        for (int hh = 0; hh < kMaxGroup; ++hh) {
            if (lane == 0) { sm_m[warp * kMaxGroup + hh] = m[hh]; sm_l[warp * kMaxGroup + hh] = l[hh]; }
#pragma unroll
            for (int e = 0; e < EPL; ++e) sm_acc[(warp * kMaxGroup + hh) * D + lane * EPL + e] = acc[hh][e];
        }
        __syncthreads();
        const int64_t pidx = (int64_t)blockIdx.x + seg;
        for (int idx = threadIdx.x; idx < G * D; idx += blockDim.x) {
            const int hh = idx / D, d = idx % D;
            float M = -INFINITY;
#pragma unroll
            for (int w = 0; w < NW; ++w) M = fmaxf(M, sm_m[w * kMaxGroup + hh]);
            float L = 0.f, o = 0.f;
            if (M > -INFINITY) {
#pragma unroll
                for (int w = 0; w < NW; ++w) {
                    const float sc = exp2f(sm_m[w * kMaxGroup + hh] - M);
                    L += sm_l[w * kMaxGroup + hh] * sc;
                    o += sm_acc[(w * kMaxGroup + hh) * D + d] * sc;
                }
            }
            p.part_o[(pidx * G + hh) * D + d] = L > 0.f ? o / L : 0.f;
            if (d == 0) p.part_lse[pidx * G + hh] = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
        }
        t = t_end;
    }
}

// ---------------------------------------------------------------------------------------------
// Combine: one block per segment (b, g); merges the segment's partials by log-sum-exp.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128) attn_combine(AttnParams p, int C) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    int64_t* tile_prefix = reinterpret_cast<int64_t*>(smem_raw);     // [B + 1]
    float* w_sm = reinterpret_cast<float*>(tile_prefix + (p.B + 1)); // [kMaxGroup][np]  (np <= C)
    __shared__ float inv_sum[kMaxGroup], lse_sm[kMaxGroup];

    build_tile_prefix(p, tile_prefix);
    const int seg = blockIdx.x, b = seg / p.Hkv, g = seg % p.Hkv;
    const int G = p.G, D = p.D;
    const int64_t n = (int64_t)p.Hkv * tile_prefix[p.B];
    const int64_t tiles_b = tile_prefix[b + 1] - tile_prefix[b];
    __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.out) + ((int64_t)b * p.Hq + g * G) * D;
    if (tiles_b == 0) {                       // empty sequence: out = 0, lse = -inf
        for (int idx = threadIdx.x; idx < G * D; idx += blockDim.x) out[idx] = __float2bfloat16(0.f);
        if (p.lse && threadIdx.x < G) p.lse[(int64_t)b * p.Hq + g * G + threadIdx.x] = -INFINITY;
        return;
    }
    const int64_t seg_start = (int64_t)p.Hkv * tile_prefix[b] + (int64_t)g * tiles_b;
    const int c_first = tile_owner(seg_start, n, C), c_last = tile_owner(seg_start + tiles_b - 1, n, C);
    const int np = c_last - c_first + 1;
    const int64_t pbase = (int64_t)c_first + seg;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    for (int hh = warp; hh < G; hh += 4) {
        float M = -INFINITY;
        for (int i = lane; i < np; i += 32) M = fmaxf(M, p.part_lse[(pbase + i) * G + hh]);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
        float sum = 0.f;
        for (int i = lane; i < np; i += 32) {
            const float x = p.part_lse[(pbase + i) * G + hh];
            const float w = (M > -INFINITY) ? __expf(x - M) : 0.f;
            w_sm[hh * np + i] = w;
            sum += w;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
        if (lane == 0) {
            inv_sum[hh] = sum > 0.f ? 1.f / sum : 0.f;
            lse_sm[hh] = sum > 0.f ? M + __logf(sum) : -INFINITY;
        }
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < G * D; idx += blockDim.x) {
        const int hh = idx / D, d = idx % D;
        float o = 0.f;
        for (int i = 0; i < np; ++i) o = fmaf(w_sm[hh * np + i], p.part_o[((pbase + i) * G + hh) * D + d], o);
        out[idx] = __float2bfloat16(o * inv_sum[hh]);
    }
    if (p.lse && threadIdx.x < G) p.lse[(int64_t)b * p.Hq + g * G + threadIdx.x] = lse_sm[threadIdx.x];
}

}  // namespace

cudaError_t launch_attention(const AttnParams& p, cudaStream_t st) {
    const int C = p.num_ctas;
    const size_t prefix_bytes = sizeof(int64_t) * (p.B + 1);
    const size_t sm_partial = prefix_bytes + sizeof(float) * (4 * kMaxGroup * 2 + 4 * kMaxGroup * p.D);
    cudaError_t e;
    if (p.D == 128) {
        attn_partial_simple<128><<<C, 128, sm_partial, st>>>(p);
    } else {
        attn_partial_simple<256><<<C, 128, sm_partial, st>>>(p);
    }
    count_launch(1);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    const size_t sm_combine = prefix_bytes + sizeof(float) * kMaxGroup * C;
    attn_combine<<<p.B * p.Hkv, 128, sm_combine, st>>>(p, C);
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace wmtp
