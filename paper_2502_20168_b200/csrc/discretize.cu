// Zero-order-hold discretisation of the diagonal SSM (Sec. III-B, Eq. 3) and its adjoint,
// plus the packing of the discretised parameters into real GEMM operands.
#include "kernels.h"

namespace ssm {

// exp(z) - 1 for z = a + ib without cancellation near z = 0.
__device__ __forceinline__ void expm1_complex(double a, double b, double& re, double& im) {
    double sb, cb;
    sincos(b, &sb, &cb);
    double sh = sin(0.5 * b);
    re = expm1(a) * cb - 2.0 * sh * sh;
    im = exp(a) * sb;
}

struct ZohTerms {
    double ar, ai;  // Abar = exp(Lambda Delta)
    double gr, gi;  // gamma = (Abar - 1) / Lambda
};

__device__ __forceinline__ ZohTerms zoh_terms(float2 lam, float dt) {
    double lr = lam.x, li = lam.y, d = dt;
    double er, ei;
    expm1_complex(lr * d, li * d, er, ei);
    double n = lr * lr + li * li;
    ZohTerms z;
    z.ar = er + 1.0;
    z.ai = ei;
    z.gr = (er * lr + ei * li) / n;
    z.gi = (ei * lr - er * li) / n;
    return z;
}

// One block per state p: Abar[p], Bbar[p, :] = gamma_p * B[p, :].
__global__ void discretize_kernel(int H, const float2* __restrict__ Lambda, const float* __restrict__ Delta,
                                  const float2* __restrict__ Bc, float2* __restrict__ Abar,
                                  float2* __restrict__ Abar_lo, float2* __restrict__ Bbar) {
    __shared__ float2 gamma_s;
    const int p = blockIdx.x;
    if (threadIdx.x == 0) {
        ZohTerms z = zoh_terms(Lambda[p], Delta[p]);
        const float2 ah = make_float2((float)z.ar, (float)z.ai);
        Abar[p] = ah;
        if (Abar_lo) Abar_lo[p] = make_float2((float)(z.ar - (double)ah.x), (float)(z.ai - (double)ah.y));
        gamma_s = make_float2((float)z.gr, (float)z.gi);
    }
    __syncthreads();
    const float2 g = gamma_s;
    for (int h = threadIdx.x; h < H; h += blockDim.x) Bbar[(size_t)p * H + h] = cmul(g, Bc[(size_t)p * H + h]);
}

// Adjoint.  One block per state p.  gAbar arrives as gA_rows rows of partial sums ([gA_rows, P], summed here
// in a fixed order; one row = the finished gradient).  Blocks past the P states (if any) finish dD the same
// way: dD[h] = sum of the dD_rows rows of dD_part ([dD_rows, H]).
__global__ void discretize_bwd_kernel(int H, int P, const float2* __restrict__ Lambda, const float* __restrict__ Delta,
                                      const float2* __restrict__ Bc, const float2* __restrict__ gAbar, int gA_rows,
                                      const float2* __restrict__ gBbar, float2* __restrict__ dLambda,
                                      float* __restrict__ dDelta, float2* __restrict__ dB,
                                      const float* __restrict__ dD_part, int dD_rows, float* __restrict__ dD) {
    __shared__ float2 gamma_s;
    __shared__ float red[2][32];
    __shared__ double redA[2][32];
    if ((int)blockIdx.x >= P) {   // columns of dD
        const int h = ((int)blockIdx.x - P) * blockDim.x + threadIdx.x;
        if (h < H) {
            float acc = 0.f;
            for (int r = 0; r < dD_rows; ++r) acc += dD_part[(size_t)r * H + h];
            dD[h] = acc;
        }
        return;
    }
    const int p = blockIdx.x;
    double gar_t = 0.0, gai_t = 0.0;   // this thread's rows of the partial sums of gAbar[p]
    for (int r = threadIdx.x; r < gA_rows; r += blockDim.x) {
        const float2 v = gAbar[(size_t)r * P + p];
        gar_t += (double)v.x;
        gai_t += (double)v.y;
    }
    for (int o = 16; o > 0; o >>= 1) {
        gar_t += __shfl_xor_sync(0xffffffffu, gar_t, o);
        gai_t += __shfl_xor_sync(0xffffffffu, gai_t, o);
    }
    if ((threadIdx.x & 31) == 0) {
        redA[0][threadIdx.x >> 5] = gar_t;
        redA[1][threadIdx.x >> 5] = gai_t;
    }
    const float2 lam = Lambda[p];
    const float dt = Delta[p];
    ZohTerms z = {};
    if (threadIdx.x == 0) {
        z = zoh_terms(lam, dt);
        gamma_s = make_float2((float)z.gr, (float)z.gi);
    }
    __syncthreads();
    const float2 gc = cconj(gamma_s);
    float sr = 0.f, si = 0.f;  // g_gamma = sum_h conj(B) gBbar
    for (int h = threadIdx.x; h < H; h += blockDim.x) {
        float2 gb = gBbar[(size_t)p * H + h];
        float2 b = Bc[(size_t)p * H + h];
        dB[(size_t)p * H + h] = cmul(gc, gb);
        float2 t = cmul(cconj(b), gb);
        sr += t.x;
        si += t.y;
    }
    for (int o = 16; o > 0; o >>= 1) {
        sr += __shfl_xor_sync(0xffffffffu, sr, o);
        si += __shfl_xor_sync(0xffffffffu, si, o);
    }
    if ((threadIdx.x & 31) == 0) {
        red[0][threadIdx.x >> 5] = sr;
        red[1][threadIdx.x >> 5] = si;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double ggr = 0.0, ggi = 0.0;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) {
            ggr += red[0][w];
            ggi += red[1][w];
        }
        const double lr = lam.x, li = lam.y, d = dt;
        double gar = 0.0, gai = 0.0;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) {
            gar += redA[0][w];
            gai += redA[1][w];
        }
        // dgamma/dLambda = (Delta Abar - gamma) / Lambda     (= (Delta Abar Lambda - (Abar-1)) / Lambda^2)
        const double nr = d * z.ar - z.gr, ni = d * z.ai - z.gi;
        const double n = lr * lr + li * li;
        const double qr = (nr * lr + ni * li) / n, qi = (ni * lr - nr * li) / n;
        // dLambda = conj(Delta Abar) gAbar + conj(dgamma/dLambda) g_gamma
        double outr = d * (z.ar * gar + z.ai * gai) + (qr * ggr + qi * ggi);
        double outi = d * (z.ar * gai - z.ai * gar) + (qr * ggi - qi * ggr);
        dLambda[p] = make_float2((float)outr, (float)outi);
        // dDelta = Re(conj(Lambda Abar) gAbar) + Re(conj(Abar) g_gamma)
        const double lar = lr * z.ar - li * z.ai, lai = lr * z.ai + li * z.ar;
        dDelta[p] = (float)((lar * gar + lai * gai) + (z.ar * ggr + z.ai * ggi));
    }
}

// Real GEMM operands from the complex parameters (W = float or bf16):
//   Bp[2p+c, h] = Bq[h, 2p+c] = c ? Im Bbar[p,h] : Re Bbar[p,h]
//   Cp[h, 2p+c] = Cq[2p+c, h] = c ? -Im C[h,p]   : Re C[h,p]
template <typename W>
__global__ void pack_operands_kernel(int H, int P, const float2* __restrict__ Bbar, const float2* __restrict__ Cc,
                                     W* __restrict__ Bp, W* __restrict__ Bq, W* __restrict__ Cp,
                                     W* __restrict__ Cq) {
    const size_t n = (size_t)P * H;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        {   // i indexes Bbar[p, h]
            const int p = (int)(i / H), h = (int)(i % H);
            const float2 v = Bbar[i];
            Bp[(size_t)(2 * p) * H + h] = from_f32<W>(v.x);
            Bp[(size_t)(2 * p + 1) * H + h] = from_f32<W>(v.y);
            Bq[(size_t)h * 2 * P + 2 * p] = from_f32<W>(v.x);
            Bq[(size_t)h * 2 * P + 2 * p + 1] = from_f32<W>(v.y);
        }
        {   // i indexes C[h, p]
            const int h = (int)(i / P), p = (int)(i % P);
            const float2 v = Cc[i];
            Cp[(size_t)h * 2 * P + 2 * p] = from_f32<W>(v.x);
            Cp[(size_t)h * 2 * P + 2 * p + 1] = from_f32<W>(-v.y);
            Cq[(size_t)(2 * p) * H + h] = from_f32<W>(v.x);
            Cq[(size_t)(2 * p + 1) * H + h] = from_f32<W>(-v.y);
        }
    }
}

// Operands of the tensor-core path.  A weight w is carried as hi = bf16(w), lo = bf16(w - hi)
// in the two projections that feed the states (Bu and g_x), so that the states see ~16
// mantissa bits of the parameters.  Logical row n of the [2P, H] operand goes to rows
// (n/128)*256 + n%128 (hi) and (n/128)*256 + 128 + n%128 (lo) of the stacked [4P, H] matrix.
// `stack`: rows per hi (and per lo) block, 128 for the plain projections, twice the states per chain otherwise.
__device__ __forceinline__ void store_split(__nv_bfloat16* W, int H, int n, int h, float w, int stack = 128) {
    const __nv_bfloat16 hi = __float2bfloat16_rn(w);
    const __nv_bfloat16 lo = __float2bfloat16_rn(w - __bfloat162float(hi));
    const size_t r = (size_t)(n / stack) * (2 * stack) + (n % stack);
    W[r * H + h] = hi;
    W[(r + stack) * H + h] = lo;
}

// Discretisation and operand packing of the tensor-core path in one kernel: block p computes Abar_p and
// gamma_p (double precision, one thread), then the row p of Bbar with its packed forms and the packed forms
// of column p of C.
__global__ void __launch_bounds__(128)
discretize_pack_tc_kernel(int H, int P, int group_B, int group_C, const float2* __restrict__ Lambda,
                          const float* __restrict__ Delta, const float2* __restrict__ Bc, const float2* __restrict__ Cc,
                          float2* __restrict__ Abar, float2* __restrict__ Abar_lo, float2* __restrict__ Bbar,
                          __nv_bfloat16* __restrict__ WsB, __nv_bfloat16* __restrict__ WsC,
                          __nv_bfloat16* __restrict__ Cp, __nv_bfloat16* __restrict__ Bq) {
    __shared__ float2 gamma_s;
    const int p = blockIdx.x;
    if (threadIdx.x == 0) {
        ZohTerms z = zoh_terms(Lambda[p], Delta[p]);
        const float2 ah = make_float2((float)z.ar, (float)z.ai);
        Abar[p] = ah;
        if (Abar_lo) Abar_lo[p] = make_float2((float)(z.ar - (double)ah.x), (float)(z.ai - (double)ah.y));
        gamma_s = make_float2((float)z.gr, (float)z.gi);
    }
    __syncthreads();
    const float2 g = gamma_s;
    // state p, component c -> row (p / G) 2G + 4 ((p % G) / 2) + 2 c + p % 2 inside groups of G states
    auto row_of = [&](int G) { return G ? (p / G) * 2 * G + 4 * ((p % G) >> 1) + (p & 1) : 2 * p; };
    const int nB = row_of(group_B), nC = row_of(group_C);
    const int sB = group_B ? 2 * group_B : 128, sC = group_C ? 2 * group_C : 128;
    for (int h = threadIdx.x; h < H; h += blockDim.x) {
        const float2 v = cmul(g, Bc[(size_t)p * H + h]);
        Bbar[(size_t)p * H + h] = v;
        store_split(WsB, H, nB, h, v.x, sB);
        store_split(WsB, H, nB + (group_B ? 2 : 1), h, v.y, sB);
        *reinterpret_cast<__nv_bfloat162*>(Bq + (size_t)h * 2 * P + 2 * p) = __floats2bfloat162_rn(v.x, v.y);
        const float2 c = Cc[(size_t)h * P + p];
        *reinterpret_cast<__nv_bfloat162*>(Cp + (size_t)h * 2 * P + 2 * p) = __floats2bfloat162_rn(c.x, -c.y);
        store_split(WsC, H, nC, h, c.x, sC);
        store_split(WsC, H, nC + (group_C ? 2 : 1), h, -c.y, sC);
    }
}

// The same for the projections that run as sums of bf16 plane products (fp32 inputs and outputs): every
// operand as three planes side by side along its K.
//   Wb3[2p+c, a H + h] = plane a of (c ? Im : Re) Bbar[p,h]       [2P, 3H]   (Bu = u Wb3^T)
//   Cq3[2p+c, a H + h] = plane a of (c ? -Im : Re) C[h,p]         [2P, 3H]   (g_x = gy Cq3^T)
//   Cp3[h, a 2P + 2p+c] = plane a of (c ? -Im : Re) C[h,p]        [H, 3 2P]  (y = x Cp3^T)
//   Bq3[h, a 2P + 2p+c] = plane a of (c ? Im : Re) Bbar[p,h]      [H, 3 2P]  (du = s Bq3^T)
__device__ __forceinline__ void store3(__nv_bfloat16* base, size_t plane_stride, float v) {
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    const float r1 = v - __bfloat162float(hi);
    const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
    base[0] = hi;
    base[plane_stride] = mid;
    base[2 * plane_stride] = __float2bfloat16_rn(r1 - __bfloat162float(mid));
}

__global__ void __launch_bounds__(128)
discretize_pack_planes_kernel(int H, int P, const float2* __restrict__ Lambda, const float* __restrict__ Delta,
                              const float2* __restrict__ Bc, const float2* __restrict__ Cc, float2* __restrict__ Abar,
                              float2* __restrict__ Abar_lo, float2* __restrict__ Bbar, __nv_bfloat16* __restrict__ Wb3,
                              __nv_bfloat16* __restrict__ Cq3, __nv_bfloat16* __restrict__ Cp3,
                              __nv_bfloat16* __restrict__ Bq3) {
    __shared__ float2 gamma_s;
    const int p = blockIdx.x;
    if (threadIdx.x == 0) {
        ZohTerms z = zoh_terms(Lambda[p], Delta[p]);
        const float2 ah = make_float2((float)z.ar, (float)z.ai);
        Abar[p] = ah;
        if (Abar_lo) Abar_lo[p] = make_float2((float)(z.ar - (double)ah.x), (float)(z.ai - (double)ah.y));
        gamma_s = make_float2((float)z.gr, (float)z.gi);
    }
    __syncthreads();
    const float2 g = gamma_s;
    const size_t H3 = 3 * (size_t)H, P6 = 6 * (size_t)P;
    for (int h = threadIdx.x; h < H; h += blockDim.x) {
        const float2 v = cmul(g, Bc[(size_t)p * H + h]);
        Bbar[(size_t)p * H + h] = v;
        store3(Wb3 + (size_t)(2 * p) * H3 + h, H, v.x);
        store3(Wb3 + (size_t)(2 * p + 1) * H3 + h, H, v.y);
        store3(Bq3 + (size_t)h * P6 + 2 * p, 2 * (size_t)P, v.x);
        store3(Bq3 + (size_t)h * P6 + 2 * p + 1, 2 * (size_t)P, v.y);
        const float2 c = Cc[(size_t)h * P + p];
        store3(Cq3 + (size_t)(2 * p) * H3 + h, H, c.x);
        store3(Cq3 + (size_t)(2 * p + 1) * H3 + h, H, -c.y);
        store3(Cp3 + (size_t)h * P6 + 2 * p, 2 * (size_t)P, c.x);
        store3(Cp3 + (size_t)h * P6 + 2 * p + 1, 2 * (size_t)P, -c.y);
    }
}

void launch_discretize_pack_planes(int H, int P, const float2* Lambda, const float* Delta, const float2* Bc,
                                   const float2* Cc, float2* Abar, float2* Abar_lo, float2* Bbar, void* Wb3, void* Cq3,
                                   void* Cp3, void* Bq3, cudaStream_t st) {
    count_launch();
    discretize_pack_planes_kernel<<<P, 128, 0, st>>>(H, P, Lambda, Delta, Bc, Cc, Abar, Abar_lo, Bbar, (__nv_bfloat16*)Wb3,
                                                     (__nv_bfloat16*)Cq3, (__nv_bfloat16*)Cp3, (__nv_bfloat16*)Bq3);
}

void launch_discretize_pack_tc(int H, int P, int group_B, int group_C, const float2* Lambda, const float* Delta,
                               const float2* Bc, const float2* Cc, float2* Abar, float2* Abar_lo, float2* Bbar,
                               void* Wsplit_B, void* Wsplit_C, void* Cp, void* Bq, cudaStream_t st) {
    count_launch();
    discretize_pack_tc_kernel<<<P, 128, 0, st>>>(H, P, group_B, group_C, Lambda, Delta, Bc, Cc, Abar, Abar_lo, Bbar,
                                                 (__nv_bfloat16*)Wsplit_B, (__nv_bfloat16*)Wsplit_C, (__nv_bfloat16*)Cp,
                                                 (__nv_bfloat16*)Bq);
}

void launch_discretize(int H, int P, const float2* Lambda, const float* Delta, const float2* Bc, float2* Abar,
                       float2* Abar_lo, float2* Bbar, cudaStream_t st) {
    count_launch();
    discretize_kernel<<<P, 128, 0, st>>>(H, Lambda, Delta, Bc, Abar, Abar_lo, Bbar);
}

void launch_discretize_bwd(int H, int P, const float2* Lambda, const float* Delta, const float2* Bc,
                           const float2* gAbar, const float2* gBbar, float2* dLambda, float* dDelta, float2* dB,
                           cudaStream_t st) {
    count_launch();
    discretize_bwd_kernel<<<P, 128, 0, st>>>(H, P, Lambda, Delta, Bc, gAbar, 1, gBbar, dLambda, dDelta, dB, nullptr, 0,
                                             nullptr);
}

void launch_layer_finalize(int H, int P, const float2* Lambda, const float* Delta, const float2* Bc,
                           const float2* gA_part, int gA_rows, const float2* gBbar, float2* dLambda, float* dDelta,
                           float2* dB, const float* dD_part, int dD_rows, float* dD, cudaStream_t st) {
    count_launch();
    const int extra = dD_part ? (H + 127) / 128 : 0;
    discretize_bwd_kernel<<<P + extra, 128, 0, st>>>(H, P, Lambda, Delta, Bc, gA_part, gA_rows, gBbar, dLambda, dDelta, dB,
                                                     dD_part, dD_rows, dD);
}

void launch_pack_operands(int H, int P, bool bf16, const float2* Bbar, const float2* Cc, void* Bp, void* Bq,
                          void* Cp, void* Cq, cudaStream_t st) {
    const int threads = 256;
    const int blocks = (int)(((size_t)P * H + threads - 1) / threads);
    count_launch();
    if (bf16)
        pack_operands_kernel<__nv_bfloat16><<<blocks, threads, 0, st>>>(
            H, P, Bbar, Cc, (__nv_bfloat16*)Bp, (__nv_bfloat16*)Bq, (__nv_bfloat16*)Cp, (__nv_bfloat16*)Cq);
    else
        pack_operands_kernel<float><<<blocks, threads, 0, st>>>(H, P, Bbar, Cc, (float*)Bp, (float*)Bq,
                                                                 (float*)Cp, (float*)Cq);
}

}  // namespace ssm
