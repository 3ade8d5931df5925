// Two fp32 fused multiply-adds in one instruction (fma.rn.f32x2): each half is an ordinary
// round-to-nearest FMA, so results are those of two scalar fmaf calls; what changes is that one
// instruction issue does the work of two.
#pragma once
#include <cuda_runtime.h>

namespace evo {

__device__ __forceinline__ void ffma2(float2& acc, float2 a, float2 b)
{
    asm("fma.rn.f32x2 %0, %1, %2, %0;"
        : "+l"(*reinterpret_cast<unsigned long long*>(&acc))
        : "l"(*reinterpret_cast<const unsigned long long*>(&a)), "l"(*reinterpret_cast<const unsigned long long*>(&b)));
}

}  // namespace evo
