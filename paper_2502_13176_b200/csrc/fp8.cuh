// FP8 E4M3 conversions for quantised K/V slabs (device side): the hardware's own converters.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

namespace fp8 {

// two fp32 values -> two E4M3 codes (round to nearest even, saturating at +-448); `lo` lands in the low byte
__device__ __forceinline__ uint32_t e4m3x2_from_f32(float lo, float hi) {
    uint16_t d;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(d) : "f"(hi), "f"(lo));
    return d;
}
// two E4M3 codes (low 16 bits of `pair`) -> two fp16 values, exactly
__device__ __forceinline__ uint32_t f16x2_from_e4m3x2(uint32_t pair) {
    uint32_t d;
    const uint16_t h = (uint16_t)pair;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(d) : "h"(h));
    return d;
}
// four E4M3 codes (one register) -> fp16 pairs of the low and of the high half, exactly
__device__ __forceinline__ void f16x4_from_e4m3x4(uint32_t four, uint32_t& lo, uint32_t& hi) {
    asm("{\n\t.reg .b16 l, h;\n\t"
        "mov.b32 {l, h}, %2;\n\t"
        "cvt.rn.f16x2.e4m3x2 %0, l;\n\t"
        "cvt.rn.f16x2.e4m3x2 %1, h;\n\t}"
        : "=r"(lo), "=r"(hi) : "r"(four));
}
// eight bf16 values (16 bytes) times `inv_scale` -> eight codes (8 bytes)
__device__ __forceinline__ uint2 quantise8(uint4 raw, float inv_scale) {
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
    uint32_t c[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[i]));
        c[i] = e4m3x2_from_f32(f.x * inv_scale, f.y * inv_scale);
    }
    return make_uint2(c[0] | (c[1] << 16), c[2] | (c[3] << 16));
}

}  // namespace fp8
