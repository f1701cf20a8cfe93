// Wrapper of the stacked sequence model: out = LayerNorm(u + GELU(v)) * w + b with v = SSM(u),
// forward and backward.  One CTA per row of H features; arithmetic in fp32.  Only the stack's own
// input, output and their gradients are in the I/O type; what passes between the layers (v, the
// layer inputs, the gradients handed down) is fp32, hence the separate element types below.
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

// TI: type of the layer input u; TO: type of out.
template <typename TI, typename TO>
__global__ void __launch_bounds__(kRowThreads)
stack_fwd_kernel(int H, const TI* __restrict__ u, const float* __restrict__ v, const float* __restrict__ w,
                 const float* __restrict__ b, TO* __restrict__ out, float* __restrict__ mu_out,
                 float* __restrict__ rstd_out) {
    __shared__ float red[kRowThreads / 32];
    const size_t row = blockIdx.x;
    const TI* ur = u + row * H;
    const float* vr = v + row * H;
    float sum = 0.f;
    for (int h = threadIdx.x; h < H; h += kRowThreads) sum += to_f32<TI>(ur[h]) + gelu_f(vr[h]);
    const float mu = block_sum(sum, red) / (float)H;
    float sq = 0.f;
    for (int h = threadIdx.x; h < H; h += kRowThreads) {
        const float z = to_f32<TI>(ur[h]) + gelu_f(vr[h]) - mu;
        sq = fmaf(z, z, sq);
    }
    const float rstd = rsqrtf(block_sum(sq, red) / (float)H + kLnEps);
    for (int h = threadIdx.x; h < H; h += kRowThreads) {
        const float z = to_f32<TI>(ur[h]) + gelu_f(vr[h]);
        out[row * H + h] = from_f32<TO>(fmaf((z - mu) * rstd, w[h], b[h]));
    }
    if (threadIdx.x == 0) {
        mu_out[row] = mu;
        rstd_out[row] = rstd;
    }
}

// gz = LayerNorm'(g) (the gradient of the residual branch);  gv = gz * GELU'(v) (what the SSM
// backward takes).  TG: type of the incoming gradient g; TI: type of the layer input u.
template <typename TG, typename TI>
__global__ void __launch_bounds__(kRowThreads)
stack_bwd_kernel(int H, const TG* __restrict__ g, const TI* __restrict__ u, const float* __restrict__ v,
                 const float* __restrict__ w, const float* __restrict__ mu_in, const float* __restrict__ rstd_in,
                 float* __restrict__ gz_out, float* __restrict__ gv) {
    __shared__ float red[kRowThreads / 32];
    const size_t row = blockIdx.x;
    const TG* gr = g + row * H;
    const TI* ur = u + row * H;
    const float* vr = v + row * H;
    const float mu = mu_in[row], rstd = rstd_in[row];
    float s1 = 0.f, s2 = 0.f;
    for (int h = threadIdx.x; h < H; h += kRowThreads) {
        const float zhat = (to_f32<TI>(ur[h]) + gelu_f(vr[h]) - mu) * rstd;
        const float gh = to_f32<TG>(gr[h]) * w[h];
        s1 += gh;
        s2 = fmaf(gh, zhat, s2);
    }
    const float m1 = block_sum(s1, red) / (float)H;
    const float m2 = block_sum(s2, red) / (float)H;
    for (int h = threadIdx.x; h < H; h += kRowThreads) {
        const float vv = vr[h];
        const float zhat = (to_f32<TI>(ur[h]) + gelu_f(vv) - mu) * rstd;
        const float gz = rstd * (to_f32<TG>(gr[h]) * w[h] - m1 - zhat * m2);
        gz_out[row * H + h] = gz;
        gv[row * H + h] = gz * gelu_grad_f(vv);
    }
}

// part_w[grp, h] = sum over the group's rows of g * zhat;  part_b[grp, h] = sum of g.
constexpr int kLnGradRows = 64;
template <typename TG, typename TI>
__global__ void __launch_bounds__(256)
ln_param_grad_kernel(int M, int H, const TG* __restrict__ g, const TI* __restrict__ u, const float* __restrict__ v,
                     const float* __restrict__ mu_in, const float* __restrict__ rstd_in,
                     float* __restrict__ part_w, float* __restrict__ part_b) {
    __shared__ float sw[8][33], sb[8][33];
    const int h = blockIdx.y * 32 + threadIdx.x;
    const int r0 = blockIdx.x * kLnGradRows, r1 = min(M, r0 + kLnGradRows);   // row groups along x (no 65535 limit)
    float aw = 0.f, ab = 0.f;
    if (h < H)
        for (int r = r0 + threadIdx.y; r < r1; r += 8) {
            const size_t i = (size_t)r * H + h;
            const float zhat = (to_f32<TI>(u[i]) + gelu_f(v[i]) - mu_in[r]) * rstd_in[r];
            const float gg = to_f32<TG>(g[i]);
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
        part_w[(size_t)blockIdx.x * H + h] = tw;
        part_b[(size_t)blockIdx.x * H + h] = tb;
    }
}

static inline int ln_groups(int M) { return (M + kLnGradRows - 1) / kLnGradRows; }

size_t stack_tmp_floats(int M, int H) {
    const int g = ln_groups(M);
    return 2 * (size_t)g * H + colsum_tmp_floats(g, H);
}

void launch_stack_fwd(bool u_bf16, bool out_bf16, int M, int H, const void* u, const float* v, const float* w,
                      const float* b, void* out, float* mu, float* rstd, cudaStream_t st) {
    using bf = __nv_bfloat16;
    count_launch();
    if (u_bf16 && out_bf16)
        stack_fwd_kernel<bf, bf><<<M, kRowThreads, 0, st>>>(H, (const bf*)u, v, w, b, (bf*)out, mu, rstd);
    else if (u_bf16)
        stack_fwd_kernel<bf, float><<<M, kRowThreads, 0, st>>>(H, (const bf*)u, v, w, b, (float*)out, mu, rstd);
    else if (out_bf16)
        stack_fwd_kernel<float, bf><<<M, kRowThreads, 0, st>>>(H, (const float*)u, v, w, b, (bf*)out, mu, rstd);
    else
        stack_fwd_kernel<float, float><<<M, kRowThreads, 0, st>>>(H, (const float*)u, v, w, b, (float*)out, mu, rstd);
}

template <typename TG, typename TI>
static void stack_bwd_launch(int M, int H, const void* g, const void* u, const float* v, const float* w, const float* mu,
                             const float* rstd, float* gz, float* gv, float* part_w, float* part_b, cudaStream_t st) {
    dim3 blk(32, 8), grid(ln_groups(M), (H + 31) / 32);
    stack_bwd_kernel<TG, TI><<<M, kRowThreads, 0, st>>>(H, (const TG*)g, (const TI*)u, v, w, mu, rstd, gz, gv);
    ln_param_grad_kernel<TG, TI><<<grid, blk, 0, st>>>(M, H, (const TG*)g, (const TI*)u, v, mu, rstd, part_w, part_b);
}

void launch_stack_bwd(bool g_bf16, bool u_bf16, int M, int H, const void* g, const void* u, const float* v,
                      const float* w, const float* mu, const float* rstd, float* gz, float* gv, float* dw, float* db,
                      float* tmp, cudaStream_t st) {
    using bf = __nv_bfloat16;
    const int grp = ln_groups(M);
    float* part_w = tmp;
    float* part_b = tmp + (size_t)grp * H;
    float* ctmp = part_b + (size_t)grp * H;
    count_launch(2);
    if (g_bf16 && u_bf16) stack_bwd_launch<bf, bf>(M, H, g, u, v, w, mu, rstd, gz, gv, part_w, part_b, st);
    else if (g_bf16) stack_bwd_launch<bf, float>(M, H, g, u, v, w, mu, rstd, gz, gv, part_w, part_b, st);
    else if (u_bf16) stack_bwd_launch<float, bf>(M, H, g, u, v, w, mu, rstd, gz, gv, part_w, part_b, st);
    else stack_bwd_launch<float, float>(M, H, g, u, v, w, mu, rstd, gz, gv, part_w, part_b, st);
    launch_colsum(part_w, grp, H, dw, ctmp, st);
    launch_colsum(part_b, grp, H, db, ctmp, st);
}

}  // namespace ssm
