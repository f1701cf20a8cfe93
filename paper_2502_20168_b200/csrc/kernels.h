// Internal launcher interface between the C-ABI layer (api.cu) and the kernel files.
#pragma once

#include "common.cuh"

namespace ssm {

// discretize.cu
// Abar_lo (may be NULL): Abar's rounding residual, exp(Lambda Delta) - Abar, as fp32.
void launch_discretize(int H, int P, const float2* Lambda, const float* Delta, const float2* Bc, float2* Abar,
                       float2* Abar_lo, float2* Bbar, cudaStream_t st);
void launch_discretize_bwd(int H, int P, const float2* Lambda, const float* Delta, const float2* Bc,
                           const float2* gAbar, const float2* gBbar, float2* dLambda, float* dDelta, float2* dB,
                           cudaStream_t st);
// The adjoint of the discretisation with the last sums of the layer's backward pass folded in: gAbar comes
// as gA_rows rows of partial sums [gA_rows, P] (one row: the finished gradient), and dD, if dD_part is given,
// as dD_rows rows [dD_rows, H]; both are summed here in a fixed order.
void launch_layer_finalize(int H, int P, const float2* Lambda, const float* Delta, const float2* Bc,
                           const float2* gA_part, int gA_rows, const float2* gBbar, float2* dLambda, float* dDelta,
                           float2* dB, const float* dD_part, int dD_rows, float* dD, cudaStream_t st);
void launch_pack_operands(int H, int P, bool bf16, const float2* Bbar, const float2* Cc, void* Bp, void* Bq,
                          void* Cp, void* Cq, cudaStream_t st);

// scan.cu
// Scratch the scans need for a [B,T,P] problem: a work counter and the partial sums of gAbar.
size_t scan_scratch_bytes(int B, int T, int P, int rows_per_seq = 1);   // rows_per_seq = 2: room for launch_gemm_scan_bwd_part
// Alo (may be NULL): low part of Abar, so that Abar + Alo carries the multiplier to ~48 bits.
int launch_scan_fwd(int B, int T, int P, const float2* Abar, const float2* Alo, const float2* Bu, const uint8_t* done,
                    const float2* x0, void* x, bool x_bf16, float2* xT, WsHeader* hdr, void* scratch,
                    cudaStream_t st);
// x and gBu are stored both as fp32 pairs or both as bf16 pairs (x_bf16 == s_bf16).
// With gA_part / gA_rows (both or neither) the sum over the sequences is left to the caller: *gA_part points
// at *gA_rows <= kMaxPartialRows rows of P partial sums inside `scratch`, and gAbar is not written.
constexpr int kMaxPartialRows = 512;
int launch_scan_bwd(int B, int T, int P, const float2* Abar, const float2* Alo, const uint8_t* done, const float2* x0,
                    const void* x, bool x_bf16, const float2* gx, const float2* gxT, void* gBu, bool s_bf16,
                    float2* gAbar, float2* gx0, WsHeader* hdr, void* scratch, cudaStream_t st,
                    const float2** gA_part = nullptr, int* gA_rows = nullptr);

// scan_stream.cu: the scans as TMA-fed streaming kernels (a CTA walks whole sequences; all
// parallelism over time is inside the CTA).  `ticket`: one int of scratch.  The backward pass
// leaves B rows of P partial gAbar sums in `part`.
bool scan_stream_supported(int B, int T, int P);
int launch_scan_fwd_stream(int B, int T, int P, const float2* Abar, const float2* Alo, const float2* Bu,
                           const uint8_t* done, const float2* x0, void* x, bool x_bf16, float2* xT, WsHeader* hdr,
                           int* ticket, cudaStream_t st);
int launch_scan_bwd_stream(int B, int T, int P, const float2* Abar, const float2* Alo, const uint8_t* done,
                           const float2* x0, const void* x, bool x_bf16, const float2* gx, const float2* gxT,
                           void* gBu, float2* gx0, float2* part, WsHeader* hdr, int* ticket, cudaStream_t st);

// reduce.cu
// out[c] = sum_r in[r, c]; `tmp` must hold colsum_tmp_floats(R, C) floats.  Deterministic.
void launch_colsum(const float* in, int R, int C, float* out, float* tmp, cudaStream_t st);
size_t colsum_tmp_floats(int R, int C);
// Reduces [R, C] partial sums to at most `limit` rows (groups of rows summed in a fixed order; `in` and `tmp`,
// colsum_tmp_floats(R, C) floats, are both overwritten); returns where the rows are, *rows_out how many.
const float* launch_reduce_rows(float* in, int R, int C, float* tmp, int limit, int* rows_out, cudaStream_t st);
// part[g, c] = sum over the rows m of group g of a[m,c]*b[m,c]; a and b each fp32 or bf16.
size_t dot_columns_tmp_floats(int M, int C);
// The group sums only: tmp[g, c] for g < the returned number of groups.
int launch_dot_columns_partial(bool a_bf16, const void* a, bool b_bf16, const void* b, int M, int C, float* tmp,
                               cudaStream_t st);

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
    const float* diag; const void* skip; bool skip_bf16;
    const float* add;                    // optional, fp32 [M, N]
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
// part0 in mode 0 into out0 and part1 in mode 1 into out1, one launch
void launch_splitk_reduce2(const float* part0, const float* part1, int splits, int I, int J, float2* out0, float2* out1,
                           cudaStream_t st);

// gemm_tc.cu: bf16 projections on tcgen05 tensor cores (operands by TMA, accumulators in TMEM).
struct GemmTcTN {
    // out[m, n] = sum_k A[m, k] * W[n, k];  A bf16 [M, K];  W bf16 packed by discretize_pack_tc_kernel:
    // [N_out, K], or with split_w [2 * N_out, K] where each group of 256 rows holds the high
    // halves of 128 output columns followed by their low halves.
    const void* A; const void* W;
    int M, N_out, K;
    bool split_w;
    bool store_f32;                      // true: out fp32 [M, N_out]; false: out bf16 with the epilogue below
    void* out;
    const float* diag; const void* skip;   // bf16 result: out = acc + diag[n] * skip[m, n]
    WsHeader* hdr;
    // Gate (with store_f32, split_w and skip): besides the fp32 result also gate_out[m, n] =
    // bf16(skip[m, n] * sigmoid(acc)).  Only where tc_tn_gate_supported says so.
    void* gate_out = nullptr;
    // Column sums (with the bf16 epilogue, where tc_tn_dot_supported says so): dot_part[c, n] = sum over the
    // rows m that CTA c drained of skip[m, n] * dot[m, n]; *dot_rows receives the number of rows c written
    // (at most tc_tn_dot_max_rows()).  dot: bf16 [M, N_out].
    const void* dot = nullptr;
    float* dot_part = nullptr;
    int* dot_rows = nullptr;
    // Sum of n_products products in one accumulator (fp32-accurate results from bf16 tensor-core products):
    // A is planes_a bf16 planes of K columns side by side ([M, planes_a * K]), W likewise ([N_out, planes_w * K]);
    // product j multiplies plane (prod_a >> 4 j) & 15 of A by plane (prod_w >> 4 j) & 15 of W.  fp32 result only.
    int n_products = 0, planes_a = 1, planes_w = 1;
    uint32_t prod_a = 0, prod_w = 0;
};
bool tc_tn_supported(int M, int N_out, int K, bool split_w);
int tc_max_n();   // widest output of the tensor-core projections
bool tc_tn_dot_supported(int M, int N_out, int K);
int tc_tn_dot_max_rows();
bool tc_tn_gate_supported(int M, int N_out, int K);
int launch_gemm_tc_tn(const GemmTcTN& g, cudaStream_t st);

// Input projection and forward scan fused (gemm_tc.cu): x = scan(u Bbar^T) written as the two bf16
// planes of x; Bu never reaches memory.  T must be a multiple of 128 and there must be enough
// (sequence, 64 states) chains for every pair of CTAs (tc_gemm_scan_fwd_supported).
struct GemmScanFwd {
    const void* u;          // bf16 [B*T, H]
    const void* Wsplit;     // hi/lo stacked Bbar operand [4P, H] (as for GemmTcTN with split_w)
    int B, T, H, P;
    const float2* Abar;     // [P]
    const uint8_t* done;    // [B*T] or NULL
    const float2* x0;       // [B, P] or NULL
    void* x_planes;         // out: bf16 hi plane [B*T, 2P], then the lo plane
    float2* xT;             // out [B, P] or NULL
    WsHeader* hdr;
};
bool tc_gemm_scan_fwd_supported(int B, int T, int H, int P);
// States per chain these kernels (forward and backward alike) use for a problem: 64 or 32; 0: not taken.  The
// hi/lo stacked operands they read are packed for that group size (launch_discretize_pack_tc).
int tc_gemm_scan_group(int B, int T, int H, int P);
// Whether these kernels put both CTAs of a pair on one sequence for a problem (few long sequences).
bool tc_gemm_scan_time_pairs(int B, int T, int H, int P);
int launch_gemm_scan_fwd(const GemmScanFwd& g, cudaStream_t st);

// g_x projection and reverse scan fused (gemm_tc.cu): s = reverse scan(gy conj(C)) written as the two
// bf16 planes of s, the sums s_t conj(x_{t-1}) per (sequence, state) in gA_part; g_x never reaches
// memory.  T must be a multiple of 128, or 16, 32 or 64 (a 128-row tile then holds whole sequences), with
// enough chains (tc_gemm_scan_bwd_supported).
struct GemmScanBwd {
    const void* gy;         // bf16 [B*T, H]
    const void* Wsplit;     // hi/lo stacked conj(C) operand [4P, H], rows in the pair_cols order
    int B, T, H, P;
    const float2* Abar;     // [P]
    const uint8_t* done;    // [B*T] or NULL
    const float2* x0;       // [B, P] or NULL
    const float2* gxT;      // [B, P] or NULL
    const void* x_planes;   // bf16 hi plane [B*T, 2P], then the lo plane
    void* s_planes;         // out: the same layout
    float2* gA_part;        // out [tc_gemm_scan_bwd_part_rows(B, T, H, P), P]
    float2* gx0;            // out [B, P] or NULL
    WsHeader* hdr;
};
bool tc_gemm_scan_bwd_supported(int B, int T, int H, int P);
int tc_gemm_scan_bwd_part_rows(int B, int T, int H, int P);   // rows of gA_part the kernel writes (at most 2 B)
int launch_gemm_scan_bwd(const GemmScanBwd& g, cudaStream_t st);
// scan.cu: the same with gA_part placed in `scratch` (as for launch_scan_bwd) and brought down to
// *gA_rows <= kMaxPartialRows rows at *gA_part_out; the caller sums those.
int launch_gemm_scan_bwd_part(GemmScanBwd g, void* scratch, const float2** gA_part_out, int* gA_rows, cudaStream_t st);

struct GemmTcNT {
    // part[s, i, j] = sum_{m in slice s} A[m, i] * (Bm_hi[m, j] + Bm_lo[m, j]);  A bf16 [K, I],
    // Bm_hi / Bm_lo bf16 [K, J]: the two planes of a state tensor
    const void* A; int I;
    const void* Bm_hi; const void* Bm_lo; int J;
    int K; int splits;
    float* part;
    WsHeader* hdr;
    int lda = 0;   // elements between rows of A when A is a column block of a wider matrix (0: I)
    // Product schedule (see GemmTcTN): A = planes_a planes of I columns, Bm_hi = planes_b planes of J columns
    // (Bm_lo unused), J a multiple of 256; splits from tc_nt_multi_splits.
    int n_products = 0, planes_a = 1, planes_b = 1;
    uint32_t prod_a = 0, prod_b = 0;
};
int tc_nt_multi_splits(int K, int I, int J);
bool tc_nt_supported(int I, int J);
int tc_nt_splits(int K, int I, int J);
int launch_gemm_tc_nt(const GemmTcNT& g, cudaStream_t st);

// discretize.cu: operands of the tensor-core path (bf16).  Wsplit_B / Wsplit_C: [4P, H] hi/lo
// stacked forms of Bp / Cq (see GemmTcTN);  Cp, Bq: [H, 2P] single bf16.
// Discretisation and packing of the four bf16 operands in one kernel.
// group_B / group_C: 0 = rows in the plain order (2p + c, hi/lo stacked per 128 rows: GemmTcTN with split_w), or the
// states per chain (64, 32) of the kernels that scan in their epilogue: rows of two neighbouring states interleaved
// as (re, re, im, im) inside groups of that many states, hi/lo stacked per group.
void launch_discretize_pack_tc(int H, int P, int group_B, int group_C, const float2* Lambda, const float* Delta,
                               const float2* Bc, const float2* Cc, float2* Abar, float2* Abar_lo, float2* Bbar,
                               void* Wsplit_B, void* Wsplit_C, void* Cp, void* Bq, cudaStream_t st);

// planes.cu / discretize.cu: fp32 tensors as three bf16 planes side by side ([M, K] -> [M, 3K]) so that a
// projection with fp32 inputs runs on the bf16 tensor cores as a sum of plane products (GemmTcTN / GemmTcNT
// with a product schedule), and what follows such a projection: out = acc + diag * skip (+ add).
void launch_split_planes(const float* in, size_t M, int K, void* out, cudaStream_t st);
void launch_diag_skip(const float* acc, const float* diag, const void* skip, bool skip_bf16, const float* add, size_t M,
                      int N, void* out, bool out_bf16, cudaStream_t st);
// Discretisation and the four projection operands as planes: Wb3, Cq3 [2P, 3H]; Cp3, Bq3 [H, 3 * 2P].
void launch_discretize_pack_planes(int H, int P, const float2* Lambda, const float* Delta, const float2* Bc,
                                   const float2* Cc, float2* Abar, float2* Abar_lo, float2* Bbar, void* Wb3, void* Cq3,
                                   void* Cp3, void* Bq3, cudaStream_t st);

// glu.cu: what surrounds the GEMMs of the half-GLU gate out = v * sigmoid(GELU(v) W).
// Tensor-core path (may be NULL): Wt2 [2H, 2H], the hi/lo stacked operand of z = [x1_hi | x1_lo] W, and
// Wn_split [2H, H], that of g_x1 = gz W^T;  Wt_f32 (CUDA-core path, may be NULL): W transposed.
void launch_glu_pack(int H, const float* W, void* Wt2, void* Wn_split, float* Wt_f32, cudaStream_t st);
// x1 = GELU(v); planes: bf16 [M, 2H], high halves in columns [0, H), low halves in [H, 2H); else fp32 [M, H]
void launch_glu_gelu(bool io_bf16, bool planes, size_t n, int H, const void* v, void* x1, cudaStream_t st);
void launch_glu_out(bool io_bf16, size_t n, const void* v, const float* z, void* out, cudaStream_t st);
// gz = gout * v * s (1 - s), s = sigmoid(z); planes: two bf16 planes (hi, lo) n elements apart, else fp32
void launch_glu_gz(bool io_bf16, bool planes, size_t n, const void* v, const void* gout, const float* z, void* gz,
                   cudaStream_t st);
void launch_glu_gv(bool io_bf16, size_t n, const void* v, const void* gout, const float* z, const float* gx1, void* gv,
                   cudaStream_t st);
void launch_glu_reduce(const float* part, int splits, size_t n, float* out, cudaStream_t st);

// stack.cu: out = LayerNorm(u + GELU(v)) * w + b per row of H features, and its backward
// (gz = LN'(g), gv = gz * GELU'(v), dw, db).  v, gz, gv are fp32; u, out and g are fp32 or bf16 as
// flagged (only the stack's own input, output and output gradient are in the I/O type).
// tmp: stack_tmp_floats(M, H) floats.
size_t stack_tmp_floats(int M, int H);
void launch_stack_fwd(bool u_bf16, bool out_bf16, int M, int H, const void* u, const float* v, const float* w,
                      const float* b, void* out, float* mu, float* rstd, cudaStream_t st);
void launch_stack_bwd(bool g_bf16, bool u_bf16, int M, int H, const void* g, const void* u, const float* v,
                      const float* w, const float* mu, const float* rstd, float* gz, float* gv, float* dw, float* db,
                      float* tmp, cudaStream_t st);

}  // namespace ssm
