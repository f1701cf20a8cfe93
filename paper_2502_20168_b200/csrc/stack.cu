// Wrapper of the stacked sequence model: out = LayerNorm(u + GELU(v)) * w + b with v = SSM(u),
// forward and backward.  One CTA per row of H features; arithmetic in fp32, storage in the I/O type.
#include "kernels.h"

namespace ssm {

constexpr int kRowThreads = 128;
constexpr float kLnEps = 1e-5f;

__device__ __forceinline__ float gelu_f(float v) { return 0.5f * v * (1.f + erff(v * 0.70710678118654752f)); }
__device__ __forceinline__ float gelu_grad_f(float v) {
    return 0.5f * (1.f + erff(v * 0.70710678118654752f)) + v * 0.3989422804014327f * expf(-0.5f * v * v);
}

// Sum over the CTA; every thread gets the result.
__device__ __forceinline__ float block_sum(float v, float* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < kRowThreads / 32; ++w) t += red[w];
    return t;
}

template <typename T>
__global__ void __launch_bounds__(kRowThreads)
stack_fwd_kernel(int H, const T* __restrict__ u, const T* __restrict__ v, const float* __restrict__ w,
                 const float* __restrict__ b, T* __restrict__ out, float* __restrict__ mu_out,
                 float* __restrict__ rstd_out) {
    __shared__ float red[kRowThreads / 32];
    const size_t row = blockIdx.x;
    const T* ur = u + row * H;
    const T* vr = v + row * H;
    float sum = 0.f;
    for (int h = threadIdx.x; h < H; h += kRowThreads) sum += to_f32<T>(ur[h]) + gelu_f(to_f32<T>(vr[h]));
    const float mu = block_sum(sum, red) / (float)H;
    float sq = 0.f;
    for (int h = threadIdx.x; h < H; h += kRowThreads) {
        const float z = to_f32<T>(ur[h]) + gelu_f(to_f32<T>(vr[h])) - mu;
        sq = fmaf(z, z, sq);
    }
    const float rstd = rsqrtf(block_sum(sq, red) / (float)H + kLnEps);
    for (int h = threadIdx.x; h < H; h += kRowThreads) {
        const float z = to_f32<T>(ur[h]) + gelu_f(to_f32<T>(vr[h]));
        out[row * H + h] = from_f32<T>(fmaf((z - mu) * rstd, w[h], b[h]));
    }
    if (threadIdx.x == 0) {
        mu_out[row] = mu;
        rstd_out[row] = rstd;
    }
}

// gz = LayerNorm'(g);  gzr = round(gz);  gv = round(gz * GELU'(v)).
template <typename T>
__global__ void __launch_bounds__(kRowThreads)
stack_bwd_kernel(int H, const T* __restrict__ g, const T* __restrict__ u, const T* __restrict__ v,
                 const float* __restrict__ w, const float* __restrict__ mu_in, const float* __restrict__ rstd_in,
                 T* __restrict__ gzr, T* __restrict__ gv) {
    __shared__ float red[kRowThreads / 32];
    const size_t row = blockIdx.x;
    const T* gr = g + row * H;
    const T* ur = u + row * H;
    const T* vr = v + row * H;
    const float mu = mu_in[row], rstd = rstd_in[row];
    float s1 = 0.f, s2 = 0.f;
    for (int h = threadIdx.x; h < H; h += kRowThreads) {
        const float zhat = (to_f32<T>(ur[h]) + gelu_f(to_f32<T>(vr[h])) - mu) * rstd;
        const float gh = to_f32<T>(gr[h]) * w[h];
        s1 += gh;
        s2 = fmaf(gh, zhat, s2);
    }
    const float m1 = block_sum(s1, red) / (float)H;
    const float m2 = block_sum(s2, red) / (float)H;
    for (int h = threadIdx.x; h < H; h += kRowThreads) {
        const float vv = to_f32<T>(vr[h]);
        const float zhat = (to_f32<T>(ur[h]) + gelu_f(vv) - mu) * rstd;
        const float gz = rstd * (to_f32<T>(gr[h]) * w[h] - m1 - zhat * m2);
        gzr[row * H + h] = from_f32<T>(gz);
        gv[row * H + h] = from_f32<T>(gz * gelu_grad_f(vv));
    }
}

// part_w[grp, h] = sum over the group's rows of g * zhat;  part_b[grp, h] = sum of g.
constexpr int kLnGradRows = 64;
template <typename T>
__global__ void __launch_bounds__(256)
ln_param_grad_kernel(int M, int H, const T* __restrict__ g, const T* __restrict__ u, const T* __restrict__ v,
                     const float* __restrict__ mu_in, const float* __restrict__ rstd_in,
                     float* __restrict__ part_w, float* __restrict__ part_b) {
    __shared__ float sw[8][33], sb[8][33];
    const int h = blockIdx.x * 32 + threadIdx.x;
    const int r0 = blockIdx.y * kLnGradRows, r1 = min(M, r0 + kLnGradRows);
    float aw = 0.f, ab = 0.f;
    if (h < H)
        for (int r = r0 + threadIdx.y; r < r1; r += 8) {
            const size_t i = (size_t)r * H + h;
            const float zhat = (to_f32<T>(u[i]) + gelu_f(to_f32<T>(v[i])) - mu_in[r]) * rstd_in[r];
            const float gg = to_f32<T>(g[i]);
            aw = fmaf(gg, zhat, aw);
            ab += gg;
        }
    sw[threadIdx.y][threadIdx.x] = aw;
    sb[threadIdx.y][threadIdx.x] = ab;
    __syncthreads();
    if (threadIdx.y == 0 && h < H) {
        float tw = 0.f, tb = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            tw += sw[i][threadIdx.x];
            tb += sb[i][threadIdx.x];
        }
        part_w[(size_t)blockIdx.y * H + h] = tw;
        part_b[(size_t)blockIdx.y * H + h] = tb;
    }
}

static inline int ln_groups(int M) { return (M + kLnGradRows - 1) / kLnGradRows; }

size_t stack_tmp_floats(int M, int H) {
    const int g = ln_groups(M);
    return 2 * (size_t)g * H + colsum_tmp_floats(g, H);
}

void launch_stack_fwd(bool bf16, int M, int H, const void* u, const void* v, const float* w, const float* b, void* out,
                      float* mu, float* rstd, cudaStream_t st) {
    count_launch();
    if (bf16)
        stack_fwd_kernel<__nv_bfloat16><<<M, kRowThreads, 0, st>>>(H, (const __nv_bfloat16*)u, (const __nv_bfloat16*)v,
                                                                   w, b, (__nv_bfloat16*)out, mu, rstd);
    else
        stack_fwd_kernel<float><<<M, kRowThreads, 0, st>>>(H, (const float*)u, (const float*)v, w, b, (float*)out, mu,
                                                           rstd);
}

void launch_stack_bwd(bool bf16, int M, int H, const void* g, const void* u, const void* v, const float* w,
                      const float* mu, const float* rstd, void* gzr, void* gv, float* dw, float* db, float* tmp,
                      cudaStream_t st) {
    const int grp = ln_groups(M);
    float* part_w = tmp;
    float* part_b = tmp + (size_t)grp * H;
    float* ctmp = part_b + (size_t)grp * H;
    dim3 blk(32, 8), grid((H + 31) / 32, grp);
    count_launch(2);
    if (bf16) {
        stack_bwd_kernel<__nv_bfloat16><<<M, kRowThreads, 0, st>>>(
            H, (const __nv_bfloat16*)g, (const __nv_bfloat16*)u, (const __nv_bfloat16*)v, w, mu, rstd,
            (__nv_bfloat16*)gzr, (__nv_bfloat16*)gv);
        ln_param_grad_kernel<__nv_bfloat16><<<grid, blk, 0, st>>>(M, H, (const __nv_bfloat16*)g, (const __nv_bfloat16*)u,
                                                                  (const __nv_bfloat16*)v, mu, rstd, part_w, part_b);
    } else {
        stack_bwd_kernel<float><<<M, kRowThreads, 0, st>>>(H, (const float*)g, (const float*)u, (const float*)v, w, mu,
                                                           rstd, (float*)gzr, (float*)gv);
        ln_param_grad_kernel<float><<<grid, blk, 0, st>>>(M, H, (const float*)g, (const float*)u, (const float*)v, mu,
                                                          rstd, part_w, part_b);
    }
    launch_colsum(part_w, grp, H, dw, ctmp, st);
    launch_colsum(part_b, grp, H, db, ctmp, st);
}

}  // namespace ssm
