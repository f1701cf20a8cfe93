// Half-GLU gate of the S5 sequence layer (Appendix "S5 Sequence Layer"):
//   x1 = GELU(v),  z = W^T x1 (row by row: z[m, j] = sum_i x1[m, i] W[i, j]),  out = v * sigmoid(z)
// and its backward.  The two H x H contractions per direction and the weight gradient run on the
// projection GEMMs of this library; this file holds what surrounds them: operand packing and
// the elementwise passes (each streams [B*T, H] arrays once: HBM-bound).
#include "kernels.h"

namespace ssm {
namespace {

__device__ __forceinline__ float gelu_f(float v) { return 0.5f * v * (1.f + erff(v * 0.70710678118654752f)); }
__device__ __forceinline__ float gelu_grad_f(float v) {
    return 0.5f * (1.f + erff(v * 0.70710678118654752f)) + v * 0.3989422804014327f * expf(-0.5f * v * v);
}
__device__ __forceinline__ float sigmoid_f(float z) { return 1.f / (1.f + expf(-z)); }

constexpr int kThreads = 256;
inline int blocks_for(size_t n) {
    const size_t b = (n + kThreads - 1) / kThreads;
    return (int)(b < 148 * 16 ? b : 148 * 16);
}

// Weight operands.  tc: hi/lo bf16 halves stacked as the TN kernel wants them (rows
// (n/128)*256 + n%128 hold the high halves of output column n, 128 rows further the low halves).
//   Wt*: output column j, reduction index i (for z = x1 W);  Wn*: output column i, reduction j
//   (for g_x1 = gz W^T).  Both are H x H reads of W[i, j].
__global__ void glu_pack_kernel(int H, const float* __restrict__ W, __nv_bfloat16* __restrict__ Wt_split,
                                __nv_bfloat16* __restrict__ Wn_split, float* __restrict__ Wt_f32) {
    const size_t n = (size_t)H * H;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        const int i = (int)(e / H), j = (int)(e % H);
        const float w = W[e];
        if (Wt_f32) Wt_f32[(size_t)j * H + i] = w;
        if (Wt_split) {
            const __nv_bfloat16 hi = __float2bfloat16_rn(w);
            const __nv_bfloat16 lo = __float2bfloat16_rn(w - __bfloat162float(hi));
            const size_t rt = (size_t)(j / 128) * 256 + (j % 128), rn = (size_t)(i / 128) * 256 + (i % 128);
            Wt_split[rt * H + i] = hi;
            Wt_split[(rt + 128) * H + i] = lo;
            Wn_split[rn * H + j] = hi;
            Wn_split[(rn + 128) * H + j] = lo;
        }
    }
}

// x1 = GELU(v): fp32, or two bf16 planes hi / lo n elements apart (hi alone feeds the gate's GEMM,
// hi + lo the weight-gradient sum over all rows, where a single bf16 rounding is not enough)
template <typename IO, bool kPlanes>
__global__ void glu_gelu_kernel(size_t n, const IO* __restrict__ v, void* __restrict__ x1) {
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        const float g = gelu_f(to_f32<IO>(v[e]));
        if (kPlanes) {
            __nv_bfloat16* p = reinterpret_cast<__nv_bfloat16*>(x1);
            const __nv_bfloat16 hi = __float2bfloat16_rn(g);
            p[e] = hi;
            p[n + e] = __float2bfloat16_rn(g - __bfloat162float(hi));
        } else {
            reinterpret_cast<float*>(x1)[e] = g;
        }
    }
}

// out = v * sigmoid(z); with z2 (the product with the low half of x1) z becomes z + z2 first
template <typename IO>
__global__ void glu_out_kernel(size_t n, const IO* __restrict__ v, float* __restrict__ z, const float* __restrict__ z2,
                               IO* __restrict__ out) {
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        float zz = z[e];
        if (z2) {
            zz += z2[e];
            z[e] = zz;
        }
        out[e] = from_f32<IO>(to_f32<IO>(v[e]) * sigmoid_f(zz));
    }
}

// gz = gout * v * s (1 - s), s = sigmoid(z): fp32, or two bf16 planes hi / lo `plane` elements apart
template <typename IO, bool kPlanes>
__global__ void glu_gz_kernel(size_t n, const IO* __restrict__ v, const IO* __restrict__ gout,
                              const float* __restrict__ z, void* __restrict__ gz, size_t plane) {
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        const float s = sigmoid_f(z[e]);
        const float g = to_f32<IO>(gout[e]) * to_f32<IO>(v[e]) * s * (1.f - s);
        if (kPlanes) {
            __nv_bfloat16* p = reinterpret_cast<__nv_bfloat16*>(gz);
            const __nv_bfloat16 hi = __float2bfloat16_rn(g);
            p[e] = hi;
            p[plane + e] = __float2bfloat16_rn(g - __bfloat162float(hi));
        } else {
            reinterpret_cast<float*>(gz)[e] = g;
        }
    }
}

template <typename IO>
__global__ void glu_gv_kernel(size_t n, const IO* __restrict__ v, const IO* __restrict__ gout,
                              const float* __restrict__ z, const float* __restrict__ gx1, IO* __restrict__ gv) {
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        const float vv = to_f32<IO>(v[e]);
        gv[e] = from_f32<IO>(to_f32<IO>(gout[e]) * sigmoid_f(z[e]) + gx1[e] * gelu_grad_f(vv));
    }
}

__global__ void glu_reduce_kernel(const float* __restrict__ part, int splits, size_t n, float* __restrict__ out) {
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        float acc = 0.f;
        for (int s = 0; s < splits; ++s) acc += part[(size_t)s * n + e];
        out[e] = acc;
    }
}

}  // namespace

void launch_glu_pack(int H, const float* W, void* Wt_split, void* Wn_split, float* Wt_f32, cudaStream_t st) {
    count_launch();
    glu_pack_kernel<<<blocks_for((size_t)H * H), kThreads, 0, st>>>(H, W, (__nv_bfloat16*)Wt_split,
                                                                    (__nv_bfloat16*)Wn_split, Wt_f32);
}

void launch_glu_gelu(bool io_bf16, bool planes, size_t n, const void* v, void* x1, cudaStream_t st) {
    count_launch();
    const int b = blocks_for(n);
    if (io_bf16 && planes)
        glu_gelu_kernel<__nv_bfloat16, true><<<b, kThreads, 0, st>>>(n, (const __nv_bfloat16*)v, x1);
    else if (io_bf16)
        glu_gelu_kernel<__nv_bfloat16, false><<<b, kThreads, 0, st>>>(n, (const __nv_bfloat16*)v, x1);
    else
        glu_gelu_kernel<float, false><<<b, kThreads, 0, st>>>(n, (const float*)v, x1);
}

void launch_glu_out(bool io_bf16, size_t n, const void* v, float* z, const float* z2, void* out, cudaStream_t st) {
    count_launch();
    const int b = blocks_for(n);
    if (io_bf16) glu_out_kernel<<<b, kThreads, 0, st>>>(n, (const __nv_bfloat16*)v, z, z2, (__nv_bfloat16*)out);
    else glu_out_kernel<<<b, kThreads, 0, st>>>(n, (const float*)v, z, z2, (float*)out);
}

void launch_glu_gz(bool io_bf16, bool planes, size_t n, const void* v, const void* gout, const float* z, void* gz,
                   cudaStream_t st) {
    count_launch();
    const int b = blocks_for(n);
    if (io_bf16 && planes)
        glu_gz_kernel<__nv_bfloat16, true><<<b, kThreads, 0, st>>>(n, (const __nv_bfloat16*)v, (const __nv_bfloat16*)gout, z, gz, n);
    else if (io_bf16)
        glu_gz_kernel<__nv_bfloat16, false><<<b, kThreads, 0, st>>>(n, (const __nv_bfloat16*)v, (const __nv_bfloat16*)gout, z, gz, n);
    else
        glu_gz_kernel<float, false><<<b, kThreads, 0, st>>>(n, (const float*)v, (const float*)gout, z, gz, n);
}

void launch_glu_gv(bool io_bf16, size_t n, const void* v, const void* gout, const float* z, const float* gx1, void* gv,
                   cudaStream_t st) {
    count_launch();
    const int b = blocks_for(n);
    if (io_bf16)
        glu_gv_kernel<<<b, kThreads, 0, st>>>(n, (const __nv_bfloat16*)v, (const __nv_bfloat16*)gout, z, gx1, (__nv_bfloat16*)gv);
    else
        glu_gv_kernel<<<b, kThreads, 0, st>>>(n, (const float*)v, (const float*)gout, z, gx1, (float*)gv);
}

void launch_glu_reduce(const float* part, int splits, size_t n, float* out, cudaStream_t st) {
    count_launch();
    glu_reduce_kernel<<<blocks_for(n), kThreads, 0, st>>>(part, splits, n, out);
}

}  // namespace ssm
