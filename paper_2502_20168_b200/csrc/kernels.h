// Internal launcher interface between the C-ABI layer (api.cu) and the kernel files.
#pragma once

#include "common.cuh"

namespace ssm {

// discretize.cu
void launch_discretize(int H, int P, const float2* Lambda, const float* Delta, const float2* Bc, float2* Abar,
                       float2* Bbar, cudaStream_t st);
void launch_discretize_bwd(int H, int P, const float2* Lambda, const float* Delta, const float2* Bc,
                           const float2* gAbar, const float2* gBbar, float2* dLambda, float* dDelta, float2* dB,
                           cudaStream_t st);
void launch_pack_operands(int H, int P, bool bf16, const float2* Bbar, const float2* Cc, void* Bp, void* Bq,
                          void* Cp, void* Cq, cudaStream_t st);

// scan.cu
// Scratch the scans need for a [B,T,P] problem: look-back records and the partial sums of gAbar.
size_t scan_scratch_bytes(int B, int T, int P);
int launch_scan_fwd(int B, int T, int P, const float2* Abar, const float2* Bu, const uint8_t* done,
                    const float2* x0, float2* x, float2* xT, WsHeader* hdr, void* scratch, cudaStream_t st);
int launch_scan_bwd(int B, int T, int P, const float2* Abar, const uint8_t* done, const float2* x0,
                    const float2* x, const float2* gx, const float2* gxT, float2* gBu, float2* gAbar,
                    float2* gx0, WsHeader* hdr, void* scratch, cudaStream_t st);

// reduce.cu
// out[c] = sum_r in[r, c]; `tmp` must hold colsum_tmp_floats(R, C) floats.  Deterministic.
void launch_colsum(const float* in, int R, int C, float* out, float* tmp, cudaStream_t st);
size_t colsum_tmp_floats(int R, int C);
// out[c] = sum_m a[m,c]*b[m,c] (a, b in io dtype).
void launch_dot_columns(bool bf16, const void* a, const void* b, int M, int C, float* out, float* tmp,
                        cudaStream_t st);
size_t dot_columns_tmp_floats(int M, int C);

// gemm_simt.cu: fp32-accumulate CUDA-core GEMMs (exact enough for the fp32 workloads and the
// fallback for shapes the tensor-core path does not take).
enum class Epi { StoreF32, AddDiagIo };
struct GemmTN {
    // out[m, n] = sum_k A[m, k] * Bm[n, k]   (+ diag[n] * skip[m, n] (+ add[m, n]) for AddDiagIo)
    const void* A; bool a_bf16; int lda;
    const void* Bm; bool b_bf16; int ldb;
    int M, N, K;
    Epi epi;
    void* out; bool out_bf16;            // StoreF32 ignores out_bf16
    const float* diag; const void* skip; // io dtype = out dtype
    const void* add;                     // optional, io dtype
};
void launch_gemm_tn(const GemmTN& g, cudaStream_t st);

struct GemmNT {
    // part[s, i, j] = sum_{k in slice s} A[k, i] * Bm[k, j]
    const void* A; bool a_bf16; int I;
    const void* Bm; bool b_bf16; int J;
    int K; int splits;
    float* part;
};
int gemm_nt_splits(int K);
void launch_gemm_nt(const GemmNT& g, cudaStream_t st);
// mode 0: complex out[J/2, I]: out[j/2, i].(re if j even else im) = sum_s part[s,i,j]
// mode 1: complex out[I, J/2]: out[i, j/2] likewise, with the imaginary part negated
void launch_splitk_reduce(const float* part, int splits, int I, int J, int mode, float2* out, cudaStream_t st);

}  // namespace ssm
