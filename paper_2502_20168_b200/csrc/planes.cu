// fp32 tensors as bf16 planes, for fp32-accurate projections on the bf16 tensor cores.
//
// A value v is carried as three bf16 numbers, hi = bf16(v), mid = bf16(v - hi), lo = bf16(v - hi - mid):
// 3 x 8 mantissa bits, so hi + mid + lo = v exactly (up to underflow).  A matrix [M, K] becomes
// [M, 3K] with the planes side by side along K; the product of two such matrices is the sum of the
// six plane products whose terms are not below 2^-24 of the result (hi hi, hi mid, mid hi, mid mid,
// hi lo, lo hi), which the GEMM kernels accumulate in one fp32 accumulator (see GemmTcTN / GemmTcNT).
#include <algorithm>

#include "kernels.h"

namespace ssm {

__device__ __forceinline__ void split3(float v, __nv_bfloat16& hi, __nv_bfloat16& mid, __nv_bfloat16& lo) {
    hi = __float2bfloat16_rn(v);
    const float r1 = v - __bfloat162float(hi);
    mid = __float2bfloat16_rn(r1);
    lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
}

// in [M, K] fp32 -> out [M, 3K] bf16 (planes side by side).  One thread per 4 neighbouring elements.
__global__ void __launch_bounds__(256)
split_planes_kernel(const float* __restrict__ in, size_t M, int K, __nv_bfloat16* __restrict__ out) {
    const size_t quads = M * (size_t)(K / 4);
    for (size_t q = (size_t)blockIdx.x * blockDim.x + threadIdx.x; q < quads; q += (size_t)gridDim.x * blockDim.x) {
        const size_t m = q / (K / 4);
        const int k = (int)(q - m * (K / 4)) * 4;
        const float4 v = *reinterpret_cast<const float4*>(in + m * K + k);
        const float vv[4] = {v.x, v.y, v.z, v.w};
        __nv_bfloat16 h[4], d[4], l[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) split3(vv[i], h[i], d[i], l[i]);
        __nv_bfloat16* row = out + m * 3 * (size_t)K + k;
        *reinterpret_cast<uint2*>(row) = *reinterpret_cast<const uint2*>(h);
        *reinterpret_cast<uint2*>(row + K) = *reinterpret_cast<const uint2*>(d);
        *reinterpret_cast<uint2*>(row + 2 * (size_t)K) = *reinterpret_cast<const uint2*>(l);
    }
}

void launch_split_planes(const float* in, size_t M, int K, void* out, cudaStream_t st) {
    const size_t quads = M * (size_t)(K / 4);
    const int blocks = (int)std::min<size_t>((quads + 255) / 256, 148 * 16);
    count_launch();
    split_planes_kernel<<<blocks, 256, 0, st>>>(in, M, K, (__nv_bfloat16*)out);
}

// out[m, n] = acc[m, n] + diag[n] * skip[m, n] (+ add[m, n]): what follows a projection whose fp32 result
// came out of the tensor cores without an epilogue.  TS / TO: types of skip and out; add is fp32 or NULL.
template <typename TS, typename TO>
__global__ void __launch_bounds__(256)
diag_skip_kernel(const float* __restrict__ acc, const float* __restrict__ diag, const TS* __restrict__ skip,
                 const float* __restrict__ add, size_t M, int N, TO* __restrict__ out) {
    const size_t n = M * (size_t)N;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        float v = fmaf(diag[e % N], to_f32<TS>(skip[e]), acc[e]);
        if (add) v += add[e];
        out[e] = from_f32<TO>(v);
    }
}

void launch_diag_skip(const float* acc, const float* diag, const void* skip, bool skip_bf16, const float* add, size_t M,
                      int N, void* out, bool out_bf16, cudaStream_t st) {
    using bf = __nv_bfloat16;
    const size_t n = M * (size_t)N;
    const int blocks = (int)std::min<size_t>((n + 255) / 256, 148 * 16);
    count_launch();
    if (skip_bf16 && out_bf16)
        diag_skip_kernel<bf, bf><<<blocks, 256, 0, st>>>(acc, diag, (const bf*)skip, add, M, N, (bf*)out);
    else if (skip_bf16)
        diag_skip_kernel<bf, float><<<blocks, 256, 0, st>>>(acc, diag, (const bf*)skip, add, M, N, (float*)out);
    else if (out_bf16)
        diag_skip_kernel<float, bf><<<blocks, 256, 0, st>>>(acc, diag, (const float*)skip, add, M, N, (bf*)out);
    else
        diag_skip_kernel<float, float><<<blocks, 256, 0, st>>>(acc, diag, (const float*)skip, add, M, N, (float*)out);
}

}  // namespace ssm
