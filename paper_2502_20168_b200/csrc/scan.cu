// The scan over the sequence (Sec. III-B Eq. "scan".."full_scan"; resets Sec. IV-A) and its
// adjoint.  Because Abar is diagonal and the same at every step, one state is one
// independent first-order recurrence; a thread owns two neighbouring states (one 16-byte
// access per step, coalesced across the warp) and walks a stretch of time steps.
#include "kernels.h"

namespace ssm {

constexpr int kUnroll = 8;     // time steps whose loads are in flight per thread
constexpr int kScanThreads = 128;

__device__ __forceinline__ float4 ld_stream(const float4* p) { return __ldcs(p); }

// ---- forward, whole sequence per thread ------------------------------------------------
// grid: ceil(B * P/2 / kScanThreads); thread -> (b, pair of states).  x may alias Bu.
__global__ void __launch_bounds__(kScanThreads)
scan_fwd_seq_kernel(int B, int T, int P2, const float4* __restrict__ Abar, const float4* Bu,
                    const uint8_t* __restrict__ done, const float4* __restrict__ x0, float4* x,
                    float4* __restrict__ xT) {
    const int idx = blockIdx.x * kScanThreads + threadIdx.x;
    if (idx >= B * P2) return;
    const int b = idx / P2, pp = idx - b * P2;
    const float4 a = Abar[pp];
    const float2 a0 = make_float2(a.x, a.y), a1 = make_float2(a.z, a.w);
    float2 s0 = make_float2(0.f, 0.f), s1 = s0;
    if (x0) {
        const float4 v = x0[(size_t)b * P2 + pp];
        s0 = make_float2(v.x, v.y);
        s1 = make_float2(v.z, v.w);
    }
    const float4* src = Bu + (size_t)b * T * P2 + pp;
    float4* dst = x + (size_t)b * T * P2 + pp;
    const uint8_t* dn = done ? done + (size_t)b * T : nullptr;
    for (int t0 = 0; t0 < T; t0 += kUnroll) {
        float4 v[kUnroll];
        bool d[kUnroll];
#pragma unroll
        for (int i = 0; i < kUnroll; ++i) {
            const int t = t0 + i;
            if (t < T) {
                v[i] = ld_stream(src + (size_t)t * P2);
                d[i] = dn ? (dn[t] != 0) : false;
            }
        }
#pragma unroll
        for (int i = 0; i < kUnroll; ++i) {
            const int t = t0 + i;
            if (t < T) {
                if (d[i]) {
                    s0 = make_float2(0.f, 0.f);
                    s1 = s0;
                }
                s0 = cfma(a0, s0, make_float2(v[i].x, v[i].y));
                s1 = cfma(a1, s1, make_float2(v[i].z, v[i].w));
                dst[(size_t)t * P2] = make_float4(s0.x, s0.y, s1.x, s1.y);
            }
        }
    }
    if (xT) xT[(size_t)b * P2 + pp] = make_float4(s0.x, s0.y, s1.x, s1.y);
}

// ---- backward, whole sequence per thread ------------------------------------------------
// s_t = gx_t + keep_{t+1} conj(Abar) s_{t+1};  gAbar partial = sum_t keep_t s_t conj(x_{t-1}).
// gBu may alias gx.
__global__ void __launch_bounds__(kScanThreads)
scan_bwd_seq_kernel(int B, int T, int P2, const float4* __restrict__ Abar, const uint8_t* __restrict__ done,
                    const float4* __restrict__ x0, const float4* __restrict__ x, const float4* gx,
                    const float4* __restrict__ gxT, float4* gBu, float4* __restrict__ gA_part,
                    float4* __restrict__ gx0) {
    const int idx = blockIdx.x * kScanThreads + threadIdx.x;
    if (idx >= B * P2) return;
    const int b = idx / P2, pp = idx - b * P2;
    const float4 a = Abar[pp];
    const float2 ac0 = make_float2(a.x, -a.y), ac1 = make_float2(a.z, -a.w);
    float2 c0 = make_float2(0.f, 0.f), c1 = c0;  // keep_{t+1} conj(Abar) s_{t+1}
    if (gxT) {
        const float4 v = gxT[(size_t)b * P2 + pp];
        c0 = make_float2(v.x, v.y);
        c1 = make_float2(v.z, v.w);
    }
    float2 g0 = make_float2(0.f, 0.f), g1 = g0;
    const float4* gsrc = gx + (size_t)b * T * P2 + pp;
    const float4* xsrc = x + (size_t)b * T * P2 + pp;
    float4* dst = gBu + (size_t)b * T * P2 + pp;
    const uint8_t* dn = done ? done + (size_t)b * T : nullptr;
    float4 xinit = make_float4(0.f, 0.f, 0.f, 0.f);
    if (x0) xinit = x0[(size_t)b * P2 + pp];
    for (int t0 = T - 1; t0 >= 0; t0 -= kUnroll) {
        float4 v[kUnroll], xp[kUnroll];
        bool d[kUnroll];
#pragma unroll
        for (int i = 0; i < kUnroll; ++i) {
            const int t = t0 - i;
            if (t >= 0) {
                v[i] = ld_stream(gsrc + (size_t)t * P2);
                xp[i] = (t > 0) ? ld_stream(xsrc + (size_t)(t - 1) * P2) : xinit;
                d[i] = dn ? (dn[t] != 0) : false;
            }
        }
#pragma unroll
        for (int i = 0; i < kUnroll; ++i) {
            const int t = t0 - i;
            if (t >= 0) {
                const float2 s0 = make_float2(v[i].x + c0.x, v[i].y + c0.y);
                const float2 s1 = make_float2(v[i].z + c1.x, v[i].w + c1.y);
                dst[(size_t)t * P2] = make_float4(s0.x, s0.y, s1.x, s1.y);
                if (d[i]) {
                    c0 = make_float2(0.f, 0.f);
                    c1 = c0;
                } else {
                    g0 = cfma(s0, make_float2(xp[i].x, -xp[i].y), g0);
                    g1 = cfma(s1, make_float2(xp[i].z, -xp[i].w), g1);
                    c0 = cmul(ac0, s0);
                    c1 = cmul(ac1, s1);
                }
            }
        }
    }
    gA_part[(size_t)b * P2 + pp] = make_float4(g0.x, g0.y, g1.x, g1.y);
    if (gx0) gx0[(size_t)b * P2 + pp] = make_float4(c0.x, c0.y, c1.x, c1.y);
}

size_t scan_scratch_bytes(int B, int T, int P) {
    (void)T;
    const size_t part = (size_t)B * P * 2;  // floats
    return align_up((part + colsum_tmp_floats(B, 2 * P)) * sizeof(float), 256);
}

int launch_scan_fwd(int B, int T, int P, const float2* Abar, const float2* Bu, const uint8_t* done,
                    const float2* x0, float2* x, float2* xT, WsHeader* hdr, void* scratch, cudaStream_t st) {
    (void)hdr;
    (void)scratch;
    const int P2 = P / 2;
    const int blocks = (int)(((size_t)B * P2 + kScanThreads - 1) / kScanThreads);
    count_launch();
    scan_fwd_seq_kernel<<<blocks, kScanThreads, 0, st>>>(B, T, P2, (const float4*)Abar, (const float4*)Bu, done,
                                                         (const float4*)x0, (float4*)x, (float4*)xT);
    return SSM_OK;
}

int launch_scan_bwd(int B, int T, int P, const float2* Abar, const uint8_t* done, const float2* x0,
                    const float2* x, const float2* gx, const float2* gxT, float2* gBu, float2* gAbar,
                    float2* gx0, WsHeader* hdr, void* scratch, cudaStream_t st) {
    (void)hdr;
    const int P2 = P / 2;
    float* part = (float*)scratch;
    float* tmp = part + (size_t)B * P * 2;
    const int blocks = (int)(((size_t)B * P2 + kScanThreads - 1) / kScanThreads);
    count_launch();
    scan_bwd_seq_kernel<<<blocks, kScanThreads, 0, st>>>(B, T, P2, (const float4*)Abar, done, (const float4*)x0,
                                                         (const float4*)x, (const float4*)gx, (const float4*)gxT,
                                                         (float4*)gBu, (float4*)part, (float4*)gx0);
    launch_colsum(part, B, 2 * P, (float*)gAbar, tmp, st);
    return SSM_OK;
}

}  // namespace ssm
