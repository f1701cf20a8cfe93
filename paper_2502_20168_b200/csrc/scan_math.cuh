// Arithmetic shared by the scan kernels: the recurrence step with a multiplier carried as an
// fp32 pair, and powers of that multiplier.
#pragma once

#include "common.cuh"

namespace ssm {

// (a + alo) * x + b with the small product added first: a step of the recurrence whose multiplier
// is carried as an fp32 pair (hi, lo), i.e. to about 48 bits.
__device__ __forceinline__ float2 cfma2(float2 a, float2 alo, float2 x, float2 b) {
    return cfma(a, x, cfma(alo, x, b));
}
// (a + alo)^n for n a power of two, evaluated in double and returned as an fp32 pair.
template <int N>
__device__ __forceinline__ void cpow2_pair(float2 a, float2 alo, float2& hi, float2& lo) {
    double re = (double)a.x + (double)alo.x, im = (double)a.y + (double)alo.y;
#pragma unroll
    for (int n = 1; n < N; n *= 2) {
        const double r2 = re * re - im * im, i2 = 2.0 * re * im;
        re = r2;
        im = i2;
    }
    hi = make_float2((float)re, (float)im);
    lo = make_float2((float)(re - (double)hi.x), (float)(im - (double)hi.y));
}

}  // namespace ssm
