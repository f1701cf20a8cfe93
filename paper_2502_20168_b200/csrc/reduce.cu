// Deterministic column reductions (parameter-gradient sums over all B*T rows).
#include "kernels.h"

namespace ssm {

constexpr int kRowsPerBlock = 64;

// block = 32 columns x 8 row lanes; grid.x = row groups (the dimension that grows with B*T), grid.y = ceil(C/32).
// out[g, c] = sum of in[r, c] for r in group g.
__global__ void colsum_kernel(const float* __restrict__ in, int R, int C, int rows_per_group,
                              float* __restrict__ out) {
    __shared__ float sm[8][33];
    const int c = blockIdx.y * 32 + threadIdx.x;
    const int r0 = blockIdx.x * rows_per_group;
    const int r1 = min(R, r0 + rows_per_group);
    float acc = 0.f;
    if (c < C)
        for (int r = r0 + threadIdx.y; r < r1; r += 8) acc += in[(size_t)r * C + c];
    sm[threadIdx.y][threadIdx.x] = acc;
    __syncthreads();
    if (threadIdx.y == 0 && c < C) {
        float t = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) t += sm[i][threadIdx.x];
        out[(size_t)blockIdx.x * C + c] = t;
    }
}

size_t colsum_tmp_floats(int R, int C) { return (size_t)((R + kRowsPerBlock - 1) / kRowsPerBlock) * C; }

void launch_colsum(const float* in, int R, int C, float* out, float* tmp, cudaStream_t st) {
    dim3 blk(32, 8);
    const int gx = (C + 31) / 32;
    if (R <= kRowsPerBlock * 2) {
        count_launch();
        colsum_kernel<<<dim3(1, gx), blk, 0, st>>>(in, R, C, R, out);
        return;
    }
    const int groups = (R + kRowsPerBlock - 1) / kRowsPerBlock;
    count_launch(2);
    colsum_kernel<<<dim3(groups, gx), blk, 0, st>>>(in, R, C, kRowsPerBlock, tmp);
    colsum_kernel<<<dim3(1, gx), blk, 0, st>>>(tmp, groups, C, groups, out);
}

// Brings a [R, C] array of partial sums down to at most `limit` rows by summing groups of kRowsPerBlock rows
// (fixed order), alternating between `in` and `tmp` (colsum_tmp_floats(R, C) floats); both are overwritten.
// Returns where the remaining rows are and how many.
const float* launch_reduce_rows(float* in, int R, int C, float* tmp, int limit, int* rows_out, cudaStream_t st) {
    dim3 blk(32, 8);
    const int gx = (C + 31) / 32;
    float* cur = in;
    float* other = tmp;
    while (R > limit) {
        const int groups = (R + kRowsPerBlock - 1) / kRowsPerBlock;
        count_launch();
        colsum_kernel<<<dim3(groups, gx), blk, 0, st>>>(cur, R, C, kRowsPerBlock, other);
        float* t = cur;
        cur = other;
        other = t;
        R = groups;
    }
    *rows_out = R;
    return cur;
}

// part[g, c] = sum_{m in group g} a[m, c] * b[m, c].  A thread owns 4 neighbouring columns
// (16 bytes of fp32, 8 bytes of bf16 per load); block = 32 column quads x 8 row lanes.
constexpr int kDotRows = 128;
template <typename T>
__device__ __forceinline__ void load_quad(const T* p, float (&v)[4]);
template <>
__device__ __forceinline__ void load_quad<float>(const float* p, float (&v)[4]) {
    const float4 t = __ldcs(reinterpret_cast<const float4*>(p));
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
template <>
__device__ __forceinline__ void load_quad<__nv_bfloat16>(const __nv_bfloat16* p, float (&v)[4]) {
    const uint2 t = __ldcs(reinterpret_cast<const uint2*>(p));
    const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&t.x));
    const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&t.y));
    v[0] = lo.x; v[1] = lo.y; v[2] = hi.x; v[3] = hi.y;
}

template <typename TA, typename TB>
__global__ void __launch_bounds__(256)
dot_columns_kernel(const TA* __restrict__ a, const TB* __restrict__ b, int M, int C, float* __restrict__ part) {
    __shared__ float4 sm[8][33];
    const int c = (blockIdx.y * 32 + threadIdx.x) * 4;
    const int r0 = blockIdx.x * kDotRows;
    const int r1 = min(M, r0 + kDotRows);
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    if (c < C) {
#pragma unroll 4
        for (int r = r0 + threadIdx.y; r < r1; r += 8) {
            float va[4], vb[4];
            load_quad<TA>(a + (size_t)r * C + c, va);
            load_quad<TB>(b + (size_t)r * C + c, vb);
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[i] = fmaf(va[i], vb[i], acc[i]);
        }
    }
    sm[threadIdx.y][threadIdx.x] = make_float4(acc[0], acc[1], acc[2], acc[3]);
    __syncthreads();
    if (threadIdx.y == 0 && c < C) {
        float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float4 v = sm[i][threadIdx.x];
            t.x += v.x; t.y += v.y; t.z += v.z; t.w += v.w;
        }
        *reinterpret_cast<float4*>(part + (size_t)blockIdx.x * C + c) = t;
    }
}

static inline int dot_groups(int M) { return (M + kDotRows - 1) / kDotRows; }

size_t dot_columns_tmp_floats(int M, int C) {
    const int g = dot_groups(M);
    return (size_t)g * C + colsum_tmp_floats(g, C);
}

// The group sums stay in tmp[0 .. groups * C) (the caller adds them); returns the number of groups.
int launch_dot_columns_partial(bool a_bf16, const void* a, bool b_bf16, const void* b, int M, int C, float* tmp,
                               cudaStream_t st) {
    using bf = __nv_bfloat16;
    const int g = dot_groups(M);
    dim3 blk(32, 8), grid(g, (C + 127) / 128);
    count_launch();
    if (a_bf16 && b_bf16)
        dot_columns_kernel<bf, bf><<<grid, blk, 0, st>>>((const bf*)a, (const bf*)b, M, C, tmp);
    else if (a_bf16)
        dot_columns_kernel<bf, float><<<grid, blk, 0, st>>>((const bf*)a, (const float*)b, M, C, tmp);
    else if (b_bf16)
        dot_columns_kernel<float, bf><<<grid, blk, 0, st>>>((const float*)a, (const bf*)b, M, C, tmp);
    else
        dot_columns_kernel<float, float><<<grid, blk, 0, st>>>((const float*)a, (const float*)b, M, C, tmp);
    return g;
}

}  // namespace ssm
