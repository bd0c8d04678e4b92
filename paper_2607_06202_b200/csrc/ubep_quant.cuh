// FP8 e4m3 quantisation of bf16 rows with one fp32 scale per 128 channels (device side).
#pragma once

#include <cuda_fp8.h>

#include "ubep_common.cuh"

namespace ubep {

// ------------------------------------------------------------------ FP8 quantisation
// 8 consecutive bf16 channels per thread, 16 threads per 128-channel group.  All steps in
// fp32 without contraction: amax -> max(amax, 1e-4) -> scale = a / 448, inv = 448 / a,
// q = e4m3_rne_satfinite(x * inv).
__device__ __forceinline__ void quantize8(const uint4 in, bool valid, uint2& out, float& scale) {
    const uint32_t w[4] = {in.x, in.y, in.z, in.w};
    float f[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
    float a = 0.0f;
    if (valid) {
#pragma unroll
        for (int i = 0; i < 8; ++i) a = fmaxf(a, fabsf(f[i]));
    }
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
    a = fmaxf(a, 1e-4f);
    scale = __fdiv_rn(a, 448.0f);
    const float inv = __fdiv_rn(448.0f, a);
    uint32_t q[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 v = make_float2(__fmul_rn(f[2 * i], inv), __fmul_rn(f[2 * i + 1], inv));
        q[i] = (uint32_t)__nv_cvt_float2_to_fp8x2(v, __NV_SATFINITE, __NV_E4M3);
    }
    out.x = q[0] | (q[1] << 16);
    out.y = q[2] | (q[3] << 16);
}

}  // namespace ubep
