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
    return (int)(b < 148 * 32 ? b : 148 * 32);
}

// Weight operands.  tc: hi/lo bf16 halves stacked as the TN kernel wants them (rows
// (n/128)*256 + n%128 hold the high halves of output column n, 128 rows further the low halves).
//   Wt2: for z = [x1_hi | x1_lo] W (the two planes of x1 side by side along K): output column j,
//        reduction index k < H -> W[k, j] (hi, lo rows), k >= H -> W[k - H, j] (hi rows only;
//        the product of two low halves is dropped);  [2H rows, 2H columns].
//   Wn:  for g_x1 = gz W^T: output column i, reduction index j;  [2H rows, H columns].
__global__ void glu_pack_kernel(int H, const float* __restrict__ W, __nv_bfloat16* __restrict__ Wt2,
                                __nv_bfloat16* __restrict__ Wn_split, float* __restrict__ Wt_f32) {
    const size_t n = (size_t)H * H;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        const int i = (int)(e / H), j = (int)(e % H);
        const float w = W[e];
        if (Wt_f32) Wt_f32[(size_t)j * H + i] = w;
        if (Wt2) {
            const __nv_bfloat16 hi = __float2bfloat16_rn(w);
            const __nv_bfloat16 lo = __float2bfloat16_rn(w - __bfloat162float(hi));
            const size_t rt = (size_t)(j / 128) * 256 + (j % 128), rn = (size_t)(i / 128) * 256 + (i % 128);
            const size_t K2 = 2 * (size_t)H;
            Wt2[rt * K2 + i] = hi;
            Wt2[rt * K2 + H + i] = hi;
            Wt2[(rt + 128) * K2 + i] = lo;
            Wt2[(rt + 128) * K2 + H + i] = __float2bfloat16_rn(0.f);
            Wn_split[rn * H + j] = hi;
            Wn_split[(rn + 128) * H + j] = lo;
        }
    }
}

// The elementwise passes work on groups of 8 consecutive elements (H is a multiple of 8): 16- or
// 32-byte accesses per array and thread.
struct F8 {
    float x[8];
};
template <typename T> __device__ __forceinline__ F8 load8(const T* p);
template <> __device__ __forceinline__ F8 load8<float>(const float* p) {
    const float4 a = __ldcs(reinterpret_cast<const float4*>(p)), b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
    return F8{{a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w}};
}
template <> __device__ __forceinline__ F8 load8<__nv_bfloat16>(const __nv_bfloat16* p) {
    const uint4 r = __ldcs(reinterpret_cast<const uint4*>(p));
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&r);
    F8 o;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 f = __bfloat1622float2(h[i]);
        o.x[2 * i] = f.x;
        o.x[2 * i + 1] = f.y;
    }
    return o;
}
template <typename T> __device__ __forceinline__ void store8(T* p, const F8& v);
template <> __device__ __forceinline__ void store8<float>(float* p, const F8& v) {
    reinterpret_cast<float4*>(p)[0] = make_float4(v.x[0], v.x[1], v.x[2], v.x[3]);
    reinterpret_cast<float4*>(p)[1] = make_float4(v.x[4], v.x[5], v.x[6], v.x[7]);
}
template <> __device__ __forceinline__ void store8<__nv_bfloat16>(__nv_bfloat16* p, const F8& v) {
    uint4 r;
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&r);
#pragma unroll
    for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(v.x[2 * i], v.x[2 * i + 1]);
    *reinterpret_cast<uint4*>(p) = r;
}
// hi = bf16(v), lo = bf16(v - hi) into two planes `plane` elements apart
__device__ __forceinline__ void store8_planes(__nv_bfloat16* p, size_t plane, const F8& v) {
    F8 hi_f, lo;
    uint4 r;
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&r);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        h[i] = __floats2bfloat162_rn(v.x[2 * i], v.x[2 * i + 1]);
        const float2 f = __bfloat1622float2(h[i]);
        hi_f.x[2 * i] = f.x;
        hi_f.x[2 * i + 1] = f.y;
    }
    *reinterpret_cast<uint4*>(p) = r;
#pragma unroll
    for (int i = 0; i < 8; ++i) lo.x[i] = v.x[i] - hi_f.x[i];
    store8<__nv_bfloat16>(p + plane, lo);
}

// x1 = GELU(v): fp32 [M, H], or bf16 [M, 2H] with the high halves in columns [0, H) and the low
// halves (bf16(x1 - hi)) in [H, 2H): one operand for the gate's GEMM with both planes along K, two
// column blocks for the weight-gradient products.  A single bf16 rounding of x1 is not enough there.
template <typename IO, bool kPlanes>
__global__ void glu_gelu_kernel(size_t n, int H, const IO* __restrict__ v, void* __restrict__ x1) {
    for (size_t e = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 8; e < n; e += (size_t)gridDim.x * blockDim.x * 8) {
        F8 a = load8<IO>(v + e);
#pragma unroll
        for (int i = 0; i < 8; ++i) a.x[i] = gelu_f(a.x[i]);
        if (kPlanes) {
            const size_t m = e / H, h = e % H;   // a group of 8 stays inside one row (H % 8 == 0)
            store8_planes(reinterpret_cast<__nv_bfloat16*>(x1) + m * 2 * H + h, (size_t)H, a);
        } else {
            store8<float>(reinterpret_cast<float*>(x1) + e, a);
        }
    }
}

template <typename IO>
__global__ void glu_out_kernel(size_t n, const IO* __restrict__ v, const float* __restrict__ z, IO* __restrict__ out) {
    for (size_t e = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 8; e < n; e += (size_t)gridDim.x * blockDim.x * 8) {
        const F8 a = load8<IO>(v + e), zz = load8<float>(z + e);
        F8 o;
#pragma unroll
        for (int i = 0; i < 8; ++i) o.x[i] = a.x[i] * sigmoid_f(zz.x[i]);
        store8<IO>(out + e, o);
    }
}

// gz = gout * v * s (1 - s), s = sigmoid(z): fp32, or two bf16 planes hi / lo `plane` elements apart
template <typename IO, bool kPlanes>
__global__ void glu_gz_kernel(size_t n, const IO* __restrict__ v, const IO* __restrict__ gout,
                              const float* __restrict__ z, void* __restrict__ gz, size_t plane) {
    for (size_t e = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 8; e < n; e += (size_t)gridDim.x * blockDim.x * 8) {
        const F8 a = load8<IO>(v + e), g = load8<IO>(gout + e), zz = load8<float>(z + e);
        F8 o;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float s = sigmoid_f(zz.x[i]);
            o.x[i] = g.x[i] * a.x[i] * s * (1.f - s);
        }
        if (kPlanes) store8_planes(reinterpret_cast<__nv_bfloat16*>(gz) + e, plane, o);
        else store8<float>(reinterpret_cast<float*>(gz) + e, o);
    }
}

template <typename IO>
__global__ void glu_gv_kernel(size_t n, const IO* __restrict__ v, const IO* __restrict__ gout,
                              const float* __restrict__ z, const float* __restrict__ gx1, IO* __restrict__ gv) {
    for (size_t e = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 8; e < n; e += (size_t)gridDim.x * blockDim.x * 8) {
        const F8 a = load8<IO>(v + e), g = load8<IO>(gout + e), zz = load8<float>(z + e), x = load8<float>(gx1 + e);
        F8 o;
#pragma unroll
        for (int i = 0; i < 8; ++i) o.x[i] = g.x[i] * sigmoid_f(zz.x[i]) + x.x[i] * gelu_grad_f(a.x[i]);
        store8<IO>(gv + e, o);
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

void launch_glu_pack(int H, const float* W, void* Wt2, void* Wn_split, float* Wt_f32, cudaStream_t st) {
    count_launch();
    glu_pack_kernel<<<blocks_for((size_t)H * H), kThreads, 0, st>>>(H, W, (__nv_bfloat16*)Wt2,
                                                                    (__nv_bfloat16*)Wn_split, Wt_f32);
}

void launch_glu_gelu(bool io_bf16, bool planes, size_t n, int H, const void* v, void* x1, cudaStream_t st) {
    count_launch();
    const int b = blocks_for(n / 8);
    if (io_bf16 && planes)
        glu_gelu_kernel<__nv_bfloat16, true><<<b, kThreads, 0, st>>>(n, H, (const __nv_bfloat16*)v, x1);
    else if (io_bf16)
        glu_gelu_kernel<__nv_bfloat16, false><<<b, kThreads, 0, st>>>(n, H, (const __nv_bfloat16*)v, x1);
    else
        glu_gelu_kernel<float, false><<<b, kThreads, 0, st>>>(n, H, (const float*)v, x1);
}

void launch_glu_out(bool io_bf16, size_t n, const void* v, const float* z, void* out, cudaStream_t st) {
    count_launch();
    const int b = blocks_for(n / 8);
    if (io_bf16) glu_out_kernel<<<b, kThreads, 0, st>>>(n, (const __nv_bfloat16*)v, z, (__nv_bfloat16*)out);
    else glu_out_kernel<<<b, kThreads, 0, st>>>(n, (const float*)v, z, (float*)out);
}

void launch_glu_gz(bool io_bf16, bool planes, size_t n, const void* v, const void* gout, const float* z, void* gz,
                   cudaStream_t st) {
    count_launch();
    const int b = blocks_for(n / 8);
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
    const int b = blocks_for(n / 8);
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
