// bf16 -> e4m3 quantisation of cache rows, shared by the fp8 cache update and the decode kernels that append the
// step's newest token to an fp8 cache themselves: value / scale in fp32 (IEEE division), then round to e4m3,
// nearest even, saturating at +-448. Every caller must take this decision in this precision: the stored codes
// are compared bit for bit.
#pragma once

#include <cuda_fp8.h>

#include "l4l_ptx.cuh"

namespace l4l {

// 8 bf16 values / scale -> 8 e4m3 bytes (two 32-bit words). The quotient is an IEEE fp32 division, so
// the stored code is RN_e4m3(RN_fp32(x / scale)) exactly.
__device__ __forceinline__ uint2 quantise8(const uint4 &v, float scale)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t out[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        uint32_t packed = 0;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const uint32_t word = w[2 * i + j];
            const float lo = __fdiv_rn(__uint_as_float(word << 16), scale);
            const float hi = __fdiv_rn(__uint_as_float(word & 0xffff0000u), scale);
            const uint32_t two = __nv_cvt_float2_to_fp8x2(make_float2(lo, hi), __NV_SATFINITE, __NV_E4M3);
            packed |= (two & 0xffffu) << (16 * j);
        }
        out[i] = packed;
    }
    return make_uint2(out[0], out[1]);
}

// 16 bf16 values (two 16-byte pieces) -> 16 e4m3 bytes
__device__ __forceinline__ uint4 quantise16(const uint4 &a, const uint4 &b, float scale)
{
    const uint2 lo = quantise8(a, scale), hi = quantise8(b, scale);
    return make_uint4(lo.x, lo.y, hi.x, hi.y);
}

}  // namespace l4l
