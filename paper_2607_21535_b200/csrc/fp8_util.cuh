// e4m3 helpers of the fp8-KV variant (Section 6, "Robustness to KV-cache quantization": the KV dtype only
// sets the bytes per entry). A store entry of KV head g has the value code_value * scale[g]; rows are
// quantised when they are appended: code = e4m3(x / scale[g]), the division in fp32, round to nearest even,
// magnitudes beyond 448 saturate (the format has no infinities).
#pragma once

#include <cuda_fp8.h>
#include <stdint.h>

namespace wmtp {

// Four bf16 values (two packed words) -> four e4m3 codes, lowest address first.
__device__ __forceinline__ uint32_t quant4_e4m3(uint32_t w0, uint32_t w1, float scale) {
    const float x0 = __uint_as_float(w0 << 16), x1 = __uint_as_float(w0 & 0xffff0000u);
    const float x2 = __uint_as_float(w1 << 16), x3 = __uint_as_float(w1 & 0xffff0000u);
    const uint32_t lo = __nv_cvt_float2_to_fp8x2(make_float2(__fdiv_rn(x0, scale), __fdiv_rn(x1, scale)), __NV_SATFINITE, __NV_E4M3);
    const uint32_t hi = __nv_cvt_float2_to_fp8x2(make_float2(__fdiv_rn(x2, scale), __fdiv_rn(x3, scale)), __NV_SATFINITE, __NV_E4M3);
    return lo | (hi << 16);
}

// Sixteen bf16 values (two 16-byte vectors) -> sixteen e4m3 codes (one 16-byte vector).
__device__ __forceinline__ uint4 quant16_e4m3(const uint4& a, const uint4& b, float scale) {
    uint4 r;
    r.x = quant4_e4m3(a.x, a.y, scale);
    r.y = quant4_e4m3(a.z, a.w, scale);
    r.z = quant4_e4m3(b.x, b.y, scale);
    r.w = quant4_e4m3(b.z, b.w, scale);
    return r;
}

}  // namespace wmtp
