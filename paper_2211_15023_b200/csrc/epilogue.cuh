// The fixed per-element arithmetic of the path, shared by every kernel of the library:
// input quantisation, the epilogue float and the requantisation.  Explicit round-to-nearest
// intrinsics keep the compiler from contracting or approximating anything.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace accerl {

// q = clamp(rintf(t), -128, 127) for a float that is already y / s
__device__ __forceinline__ int clamp_round_i8(float t)
{
    t = rintf(t);
    t = fminf(fmaxf(t, -128.f), 127.f);
    return (int)t;
}

// vector observation -> int8
__device__ __forceinline__ int8_t quantise_input(float x, float s_input)
{
    return (int8_t)clamp_round_i8(__fdiv_rn(x, s_input));
}

// y = fmaf((float)acc, k, b), ReLU if asked
__device__ __forceinline__ float epilogue_float(int acc, float k, float b, bool relu)
{
    float y = __fmaf_rn(__int2float_rn(acc), k, b);
    return relu ? fmaxf(y, 0.f) : y;
}

// q = clamp(rintf(y / s_out), -128, 127) with the IEEE divide
__device__ __forceinline__ int8_t requant(float y, float s_out)
{
    return (int8_t)clamp_round_i8(__fdiv_rn(y, s_out));
}

}  // namespace accerl
