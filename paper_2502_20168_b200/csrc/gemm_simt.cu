// fp32-accumulate CUDA-core GEMMs.  They serve the fp32 workloads (whose 1e-4 tolerance a
// single-pass reduced-precision tensor-core product cannot meet; those shapes are tiny) and
// any shape the tensor-core path does not take.
#include "kernels.h"

namespace ssm {

constexpr int TM = 64, TN = 64, TK = 16;
constexpr int kGemmThreads = 256;

template <typename T>
__device__ __forceinline__ void load4(const T* p, float (&v)[4]);
template <>
__device__ __forceinline__ void load4<float>(const float* p, float (&v)[4]) {
    const float4 t = *reinterpret_cast<const float4*>(p);
    v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
template <>
__device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16* p, float (&v)[4]) {
    const uint2 t = *reinterpret_cast<const uint2*>(p);
    const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162*>(&t.x);
    const __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162*>(&t.y);
    v[0] = __low2float(lo); v[1] = __high2float(lo); v[2] = __low2float(hi); v[3] = __high2float(hi);
}

struct EpiArgs {
    void* out;
    const float* diag;
    const void* skip;
    const void* add;
    int ldo;
};

// out[m,n] = sum_k A[m,k] Bm[n,k]; both operands K-contiguous.  K % 4 == 0.
// TO: type of out; TS: type of the skip operand; the addend, where there is one, is fp32.
template <typename TA, typename TB, typename TO, typename TS, bool kAddDiag>
__global__ void __launch_bounds__(kGemmThreads)
gemm_tn_kernel(const TA* __restrict__ A, int lda, const TB* __restrict__ Bm, int ldb, int M, int N, int K,
               EpiArgs e) {
    __shared__ __align__(16) float As[TK][TM + 4];
    __shared__ __align__(16) float Bs[TK][TN + 4];
    const int m0 = blockIdx.x * TM, n0 = blockIdx.y * TN;   // rows along x: grid.y is limited to 65535
    const int tid = threadIdx.x;
    const int lr = tid >> 2;         // 0..63: row of the tile this thread loads
    const int lk = (tid & 3) * 4;    // 0,4,8,12: k offset
    const int tx = tid & 15, ty = tid >> 4;  // 16 x 16 threads, 4 x 4 outputs each
    float acc[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += TK) {
        float va[4] = {0.f, 0.f, 0.f, 0.f}, vb[4] = {0.f, 0.f, 0.f, 0.f};
        if (m0 + lr < M && k0 + lk < K) load4<TA>(A + (size_t)(m0 + lr) * lda + k0 + lk, va);
        if (n0 + lr < N && k0 + lk < K) load4<TB>(Bm + (size_t)(n0 + lr) * ldb + k0 + lk, vb);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            As[lk + i][lr] = va[i];
            Bs[lk + i][lr] = vb[i];
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < TK; ++k) {
            const float4 a = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            const float4 b = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
            const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
    TO* out = reinterpret_cast<TO*>(e.out);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int m = m0 + ty * 4 + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n >= N) continue;
            float v = acc[i][j];
            if (kAddDiag) {
                const TS* skip = reinterpret_cast<const TS*>(e.skip);
                v = fmaf(e.diag[n], to_f32<TS>(skip[(size_t)m * e.ldo + n]), v);
                if (e.add) v += reinterpret_cast<const float*>(e.add)[(size_t)m * e.ldo + n];
            }
            out[(size_t)m * e.ldo + n] = from_f32<TO>(v);
        }
    }
}

template <typename TA, typename TB>
static void dispatch_tn(const GemmTN& g, cudaStream_t st) {
    dim3 grid((g.M + TM - 1) / TM, (g.N + TN - 1) / TN);
    count_launch();
    EpiArgs e{g.out, g.diag, g.skip, g.add, g.N};
    const TA* A = (const TA*)g.A;
    const TB* Bm = (const TB*)g.Bm;
    using bf = __nv_bfloat16;
    if (g.epi == Epi::StoreF32)
        gemm_tn_kernel<TA, TB, float, float, false><<<grid, kGemmThreads, 0, st>>>(A, g.lda, Bm, g.ldb, g.M, g.N, g.K, e);
    else if (g.out_bf16 && g.skip_bf16)
        gemm_tn_kernel<TA, TB, bf, bf, true><<<grid, kGemmThreads, 0, st>>>(A, g.lda, Bm, g.ldb, g.M, g.N, g.K, e);
    else if (g.out_bf16)
        gemm_tn_kernel<TA, TB, bf, float, true><<<grid, kGemmThreads, 0, st>>>(A, g.lda, Bm, g.ldb, g.M, g.N, g.K, e);
    else if (g.skip_bf16)
        gemm_tn_kernel<TA, TB, float, bf, true><<<grid, kGemmThreads, 0, st>>>(A, g.lda, Bm, g.ldb, g.M, g.N, g.K, e);
    else
        gemm_tn_kernel<TA, TB, float, float, true><<<grid, kGemmThreads, 0, st>>>(A, g.lda, Bm, g.ldb, g.M, g.N, g.K, e);
}

void launch_gemm_tn(const GemmTN& g, cudaStream_t st) {
    if (g.a_bf16 && g.b_bf16) dispatch_tn<__nv_bfloat16, __nv_bfloat16>(g, st);
    else if (g.a_bf16) dispatch_tn<__nv_bfloat16, float>(g, st);
    else if (g.b_bf16) dispatch_tn<float, __nv_bfloat16>(g, st);
    else dispatch_tn<float, float>(g, st);
}

// part[s,i,j] = sum_{k in slice s} A[k,i] Bm[k,j]; both operands contiguous in i / j.
template <typename TA, typename TB>
__global__ void __launch_bounds__(kGemmThreads)
gemm_nt_kernel(const TA* __restrict__ A, int I, const TB* __restrict__ Bm, int J, int K, int k_per_split,
               float* __restrict__ part) {
    __shared__ __align__(16) float As[TK][TM + 4];
    __shared__ __align__(16) float Bs[TK][TN + 4];
    const int i0 = blockIdx.y * TM, j0 = blockIdx.x * TN;
    const int kb = blockIdx.z * k_per_split, ke = min(K, kb + k_per_split);
    const int tid = threadIdx.x;
    const int lk = tid >> 4;          // 0..15
    const int lc = (tid & 15) * 4;    // 0..60
    const int tx = tid & 15, ty = tid >> 4;
    float acc[4][4] = {};
    for (int k0 = kb; k0 < ke; k0 += TK) {
        float va[4] = {0.f, 0.f, 0.f, 0.f}, vb[4] = {0.f, 0.f, 0.f, 0.f};
        if (k0 + lk < ke) {
            if (i0 + lc < I) load4<TA>(A + (size_t)(k0 + lk) * I + i0 + lc, va);
            if (j0 + lc < J) load4<TB>(Bm + (size_t)(k0 + lk) * J + j0 + lc, vb);
        }
        *reinterpret_cast<float4*>(&As[lk][lc]) = make_float4(va[0], va[1], va[2], va[3]);
        *reinterpret_cast<float4*>(&Bs[lk][lc]) = make_float4(vb[0], vb[1], vb[2], vb[3]);
        __syncthreads();
#pragma unroll
        for (int k = 0; k < TK; ++k) {
            const float4 a = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            const float4 b = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
            const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
    float* out = part + (size_t)blockIdx.z * I * J;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int ii = i0 + ty * 4 + i;
        if (ii >= I) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int jj = j0 + tx * 4 + j;
            if (jj < J) out[(size_t)ii * J + jj] = acc[i][j];
        }
    }
}

int gemm_nt_splits(int K) {
    int s = (K + 511) / 512;
    return s < 1 ? 1 : (s > 64 ? 64 : s);
}

void launch_gemm_nt(const GemmNT& g, cudaStream_t st) {
    int kps = (g.K + g.splits - 1) / g.splits;
    kps = (kps + TK - 1) / TK * TK;
    dim3 grid((g.J + TN - 1) / TN, (g.I + TM - 1) / TM, g.splits);
    count_launch();
    if (g.a_bf16 && g.b_bf16)
        gemm_nt_kernel<__nv_bfloat16, __nv_bfloat16><<<grid, kGemmThreads, 0, st>>>((const __nv_bfloat16*)g.A, g.I, (const __nv_bfloat16*)g.Bm, g.J, g.K, kps, g.part);
    else if (g.a_bf16)
        gemm_nt_kernel<__nv_bfloat16, float><<<grid, kGemmThreads, 0, st>>>((const __nv_bfloat16*)g.A, g.I, (const float*)g.Bm, g.J, g.K, kps, g.part);
    else if (g.b_bf16)
        gemm_nt_kernel<float, __nv_bfloat16><<<grid, kGemmThreads, 0, st>>>((const float*)g.A, g.I, (const __nv_bfloat16*)g.Bm, g.J, g.K, kps, g.part);
    else
        gemm_nt_kernel<float, float><<<grid, kGemmThreads, 0, st>>>((const float*)g.A, g.I, (const float*)g.Bm, g.J, g.K, kps, g.part);
}

// Both weight-gradient reductions of a layer in one launch: blockIdx.y = 0 sums part0 into out0 in mode 0,
// blockIdx.y = 1 sums part1 into out1 in mode 1.
// mode 0: complex out[J/2, I]: out[j/2, i].(re if j even else im) = sum_s part[s,i,j]
// mode 1: complex out[I, J/2]: out[i, j/2] likewise, with the imaginary part negated
__global__ void splitk_reduce2_kernel(const float* __restrict__ part0, const float* __restrict__ part1, int splits,
                                      int I, int J, float* __restrict__ out0, float* __restrict__ out1) {
    const size_t n = (size_t)I * J;
    const int mode = blockIdx.y;
    const float* part = mode ? part1 : part0;
    float* out = mode ? out1 : out0;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        float acc = 0.f;
        for (int s = 0; s < splits; ++s) acc += part[(size_t)s * n + e];
        const int i = (int)(e / J), j = (int)(e % J);
        if (mode == 0)
            out[((size_t)(j >> 1) * I + i) * 2 + (j & 1)] = acc;
        else
            out[((size_t)i * (J >> 1) + (j >> 1)) * 2 + (j & 1)] = (j & 1) ? -acc : acc;
    }
}

void launch_splitk_reduce2(const float* part0, const float* part1, int splits, int I, int J, float2* out0, float2* out1,
                           cudaStream_t st) {
    const int threads = 256;
    const int blocks = (int)(((size_t)I * J + threads - 1) / threads);
    count_launch();
    splitk_reduce2_kernel<<<dim3(blocks, 2), threads, 0, st>>>(part0, part1, splits, I, J, (float*)out0, (float*)out1);
}

}  // namespace ssm
