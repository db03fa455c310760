// An fp32 value as the exact sum of three bf16 terms (each the bf16 rounding of what the previous
// ones left: 3 x 8 significand bits cover fp32's 24).  Used by everything that produces an operand
// of the fp32 models' tensor-core projections.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace ebrl {

__device__ __forceinline__ void split3(float a, __nv_bfloat16 &t0, __nv_bfloat16 &t1, __nv_bfloat16 &t2)
{
    t0 = __float2bfloat16_rn(a);
    const float r1 = a - __bfloat162float(t0);      // exact
    t1 = __float2bfloat16_rn(r1);
    const float r2 = r1 - __bfloat162float(t1);     // exact
    t2 = __float2bfloat16_rn(r2);
}

// Four consecutive values to the same offset of the three term planes (8 bytes each).
__device__ __forceinline__ void store_split4(void *p0, void *p1, void *p2, size_t off, float a, float b, float c, float d)
{
    __nv_bfloat16 t0[4], t1[4], t2[4];
    split3(a, t0[0], t1[0], t2[0]);
    split3(b, t0[1], t1[1], t2[1]);
    split3(c, t0[2], t1[2], t2[2]);
    split3(d, t0[3], t1[3], t2[3]);
    *reinterpret_cast<uint2 *>((__nv_bfloat16 *)p0 + off) = *reinterpret_cast<const uint2 *>(t0);
    *reinterpret_cast<uint2 *>((__nv_bfloat16 *)p1 + off) = *reinterpret_cast<const uint2 *>(t1);
    *reinterpret_cast<uint2 *>((__nv_bfloat16 *)p2 + off) = *reinterpret_cast<const uint2 *>(t2);
}

}  // namespace ebrl
