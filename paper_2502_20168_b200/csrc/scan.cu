// The scan over the sequence (Sec. III-B Eq. "scan".."full_scan"; resets Sec. IV-A) and its
// adjoint: entry points of the scan stage and the plain kernels.
//
// Abar is diagonal and the same at every step, so one state is one independent first-order
// recurrence x_t = m_t x_{t-1} + v_t with m_t = Abar or 0 (flagged step).  The work is 8 flop
// per 16 bytes: HBM-bound, so every element is read once and written once.
//
// The scans normally run as the TMA-fed streaming kernels of scan_stream.cu.  The kernels
// here walk a whole sequence per thread with plain loads and stores; they serve the shapes
// the streaming kernels do not take (fewer than 16 states) or are wasted on (fewer than 8
// steps: single-step mode), and need no tensor maps.
//
// States are stored as fp32 pairs, or as bf16 pairs when they only feed bf16 tensor-core
// operands (the arithmetic and the carried state stay fp32).
#include "kernels.h"
#include "scan_math.cuh"

namespace ssm {

constexpr int kUnrollFwd = 16;    // time steps whose loads are in flight per thread (seq kernels)
constexpr int kSeqThreads = 64;   // small blocks spread a few hundred thousand threads evenly over the SMs

// ---- two complex states as stored in memory ----------------------------------------------
struct C2 {
    float2 a, b;
};
__device__ __forceinline__ C2 c2_zero() { return C2{make_float2(0.f, 0.f), make_float2(0.f, 0.f)}; }

// Storage of a state tensor [B*T, P]:
//  float4: fp32 pairs (re, im, re, im);
//  uint2:  two bf16 planes, `plane` elements apart: hi = bf16(v) and lo = bf16(v - hi), each as
//          (re, im, re, im).  hi alone is a tensor-core operand; hi + lo carries ~16 mantissa
//          bits for the contractions whose results are sums over all B*T rows.
template <typename ST> struct StateIO;
template <> struct StateIO<float4> {
    static __device__ __forceinline__ C2 load(const float4* p, size_t) {
        const float4 v = __ldcs(p);
        return C2{make_float2(v.x, v.y), make_float2(v.z, v.w)};
    }
    static __device__ __forceinline__ void store(float4* p, const C2& v, size_t) {
        *p = make_float4(v.a.x, v.a.y, v.b.x, v.b.y);
    }
};
__device__ __forceinline__ C2 unpack_bf16x4(uint2 v) {
    return C2{__bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v.x)),
              __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v.y))};
}
__device__ __forceinline__ uint2 pack_bf16x4(const C2& v) {
    const __nv_bfloat162 a = __floats2bfloat162_rn(v.a.x, v.a.y), b = __floats2bfloat162_rn(v.b.x, v.b.y);
    uint2 o;
    o.x = *reinterpret_cast<const uint32_t*>(&a);
    o.y = *reinterpret_cast<const uint32_t*>(&b);
    return o;
}
template <> struct StateIO<uint2> {
    static __device__ __forceinline__ C2 load(const uint2* p, size_t plane) {
        const C2 h = unpack_bf16x4(__ldcs(p)), l = unpack_bf16x4(__ldcs(p + plane));
        return C2{cadd(h.a, l.a), cadd(h.b, l.b)};
    }
    static __device__ __forceinline__ void store(uint2* p, const C2& v, size_t plane) {
        const uint2 hi = pack_bf16x4(v);
        const C2 h = unpack_bf16x4(hi);
        const C2 r{make_float2(v.a.x - h.a.x, v.a.y - h.a.y), make_float2(v.b.x - h.b.x, v.b.y - h.b.y)};
        p[0] = hi;
        p[plane] = pack_bf16x4(r);
    }
};
__device__ __forceinline__ C2 c2_from(const float4 v) { return C2{make_float2(v.x, v.y), make_float2(v.z, v.w)}; }
__device__ __forceinline__ float4 c2_pack(const C2& v) { return make_float4(v.a.x, v.a.y, v.b.x, v.b.y); }

// =============================================================================================
// Whole sequence per thread
// =============================================================================================
// grid: ceil(B * P/2 / kSeqThreads); thread -> (b, pair of states).  x may alias Bu.
template <typename XT>
__global__ void __launch_bounds__(kSeqThreads)
scan_fwd_seq_kernel(int B, int T, int P2, const float4* __restrict__ Abar, const float4* __restrict__ Alo,
                    const float4* Bu,
                    const uint8_t* __restrict__ done, const float4* __restrict__ x0, XT* x,
                    float4* __restrict__ xT) {
    const int idx = blockIdx.x * kSeqThreads + threadIdx.x;
    if (idx >= B * P2) return;
    const int b = idx / P2, pp = idx - b * P2;
    const size_t plane = (size_t)B * T * P2;
    const C2 a = c2_from(Abar[pp]);
    const C2 al = Alo ? c2_from(Alo[pp]) : c2_zero();
    C2 s = x0 ? c2_from(x0[(size_t)b * P2 + pp]) : c2_zero();
    const float4* src = Bu + (size_t)b * T * P2 + pp;
    XT* dst = x + (size_t)b * T * P2 + pp;
    const uint8_t* dn = done ? done + (size_t)b * T : nullptr;
    for (int t0 = 0; t0 < T; t0 += kUnrollFwd) {
        C2 v[kUnrollFwd];
        bool d[kUnrollFwd];
#pragma unroll
        for (int i = 0; i < kUnrollFwd; ++i) {
            const int t = t0 + i;
            if (t < T) {
                v[i] = StateIO<float4>::load(src + (size_t)t * P2, 0);
                d[i] = dn ? (dn[t] != 0) : false;
            }
        }
#pragma unroll
        for (int i = 0; i < kUnrollFwd; ++i) {
            const int t = t0 + i;
            if (t < T) {
                if (d[i]) s = c2_zero();
                s.a = cfma2(a.a, al.a, s.a, v[i].a);
                s.b = cfma2(a.b, al.b, s.b, v[i].b);
                StateIO<XT>::store(dst + (size_t)t * P2, s, plane);
            }
        }
    }
    if (xT) xT[(size_t)b * P2 + pp] = c2_pack(s);
}

// Storage of one state: float2 (fp32 pair) or uint32_t (bf16 pair) in two planes hi / lo.
template <typename XS> struct Raw1;
template <> struct Raw1<float2> {
    float2 v;
    __device__ __forceinline__ void load(const float2* p, size_t) { v = __ldcs(p); }
    __device__ __forceinline__ float2 get() const { return v; }
    static __device__ __forceinline__ void store(float2* p, float2 s, size_t) { *p = s; }
};
template <> struct Raw1<uint32_t> {
    uint32_t hi, lo;
    __device__ __forceinline__ void load(const uint32_t* p, size_t plane) {
        hi = __ldcs(p);
        lo = __ldcs(p + plane);
    }
    __device__ __forceinline__ float2 get() const {
        const float2 h = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&hi));
        const float2 l = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&lo));
        return cadd(h, l);
    }
    static __device__ __forceinline__ void store(uint32_t* p, float2 s, size_t plane) {
        const __nv_bfloat162 h = __floats2bfloat162_rn(s.x, s.y);
        const float2 hf = __bfloat1622float2(h);
        const __nv_bfloat162 l = __floats2bfloat162_rn(s.x - hf.x, s.y - hf.y);
        p[0] = *reinterpret_cast<const uint32_t*>(&h);
        p[plane] = *reinterpret_cast<const uint32_t*>(&l);
    }
};

// Whole-sequence backward scan, ONE state per thread (8-byte accesses): the backward step carries
// about twice the instructions of the forward one, and with two states per thread the SMs ran
// short of warps to hide their latency.
//   s_t = gx_t + c_t,  c_{t-1} = keep_t conj(Abar) s_t  (c_{T-1} = gxT);
//   gAbar partial = sum_t keep_t s_t conj(x_{t-1}).  gBu may alias gx.
// Two register batches of kUnroll1 steps alternate (the loads of one are issued before the other
// is processed); pointers advance by a constant and a guard-free main loop handles full batches.
constexpr int kUnroll1 = 8;
template <typename XS>
__global__ void __launch_bounds__(kSeqThreads)
scan_bwd_seq1_kernel(int B, int T, int P, const float2* __restrict__ Abar, const float2* __restrict__ Alo,
                     const uint8_t* __restrict__ done, const float2* __restrict__ x0, const XS* __restrict__ x,
                     const float2* gx, const float2* __restrict__ gxT, XS* gBu, float2* __restrict__ gA_part,
                     float2* __restrict__ gx0) {
    const int idx = blockIdx.x * kSeqThreads + threadIdx.x;
    if (idx >= B * P) return;
    const int b = idx / P, p = idx - b * P;
    const size_t plane = (size_t)B * T * P;
    const float2 ac = cconj(Abar[p]);
    const float2 acl = Alo ? cconj(Alo[p]) : make_float2(0.f, 0.f);
    const float2 zero2 = make_float2(0.f, 0.f);
    float2 c = gxT ? gxT[(size_t)b * P + p] : zero2;
    float2 g = zero2;
    const uint8_t* dn = done ? done + (size_t)b * T : nullptr;
    const float2 xinit = x0 ? x0[(size_t)b * P + p] : zero2;
    // pointers at step t = T-1; every step back moves them by -P
    const float2* gp = gx + ((size_t)b * T + (T - 1)) * P + p;
    const XS* xp = x + ((size_t)b * T + (T - 1)) * P + p - P;   // x_{t-1}
    XS* sp = gBu + ((size_t)b * T + (T - 1)) * P + p;

    struct Batch {
        float2 v[kUnroll1];
        Raw1<XS> xr[kUnroll1];
        uint32_t flags;
    };
    // steps t0 .. t0-kUnroll1+1, all known to exist and t0-kUnroll1+1 >= 1 (so x_{t-1} exists)
    auto fetch_full = [&](int t0, Batch& q) {
        q.flags = 0u;
#pragma unroll
        for (int i = 0; i < kUnroll1; ++i) {
            q.v[i] = __ldcs(gp - (ptrdiff_t)i * P);
            q.xr[i].load(xp - (ptrdiff_t)i * P, plane);
            if (dn && dn[t0 - i] != 0) q.flags |= 1u << i;
        }
        gp -= (ptrdiff_t)kUnroll1 * P;
        xp -= (ptrdiff_t)kUnroll1 * P;
    };
    auto step = [&](float2 v, float2 xprev, bool flagged, XS* dst) {
        const float2 s = cadd(v, c);
        Raw1<XS>::store(dst, s, plane);
        if (flagged) {
            c = zero2;
        } else {
            g = cfma(s, cconj(xprev), g);
            c = cfma2(ac, acl, s, zero2);
        }
    };
    auto process_full = [&](const Batch& q) {
#pragma unroll
        for (int i = 0; i < kUnroll1; ++i) step(q.v[i], q.xr[i].get(), (q.flags >> i) & 1u, sp - (ptrdiff_t)i * P);
        sp -= (ptrdiff_t)kUnroll1 * P;
    };
    // Full batches cover steps T-1 .. r where every step has t >= 1; the rest goes one by one.
    int t = T - 1;
    const int nfull = (T - 1) / kUnroll1;     // batches whose lowest step is >= 1
    if (nfull > 0) {
        Batch q0, q1;
        fetch_full(t, q0);
        int left = nfull - 1;
        while (true) {
            if (left > 0) fetch_full(t - kUnroll1, q1);
            process_full(q0);
            t -= kUnroll1;
            if (left-- == 0) break;
            if (left > 0) fetch_full(t - kUnroll1, q0);
            process_full(q1);
            t -= kUnroll1;
            if (left-- == 0) break;
        }
    }
    for (; t >= 0; --t) {
        const float2 v = __ldcs(gp);
        float2 xprev = xinit;
        if (t > 0) {
            Raw1<XS> r;
            r.load(xp, plane);
            xprev = r.get();
        }
        step(v, xprev, dn && dn[t] != 0, sp);
        gp -= P;
        xp -= P;
        sp -= P;
    }
    gA_part[(size_t)b * P + p] = g;
    if (gx0) gx0[(size_t)b * P + p] = c;
}

// =============================================================================================
// One step (T = 1): x = keep Abar x0 + Bu, the recurrence of single-step mode
// =============================================================================================
// grid: ceil(B * P/2 / 256); thread -> (b, pair of states).  x is written in the layout the next
// kernel wants and, if asked for, as the fp32 final state xT (which may be the array x0 came from:
// a thread reads its entry before it writes it).
template <typename XT>
__global__ void __launch_bounds__(256)
scan_fwd_step_kernel(int B, int P2, const float4* __restrict__ Abar, const float4* __restrict__ Alo,
                     const float4* Bu /* may be the array x is written to */, const uint8_t* __restrict__ done,
                     const float4* x0, XT* x, float4* xT) {
    const int idx = blockIdx.x * 256 + threadIdx.x;
    if (idx >= B * P2) return;
    const int b = idx / P2, pp = idx - b * P2;
    const size_t plane = (size_t)B * P2;
    C2 s = c2_from(Bu[idx]);
    if (x0 && !(done && done[b] != 0)) {
        const C2 a = c2_from(Abar[pp]);
        const C2 al = Alo ? c2_from(Alo[pp]) : c2_zero();
        const C2 prev = c2_from(x0[idx]);
        s.a = cfma2(a.a, al.a, prev.a, s.a);
        s.b = cfma2(a.b, al.b, prev.b, s.b);
    }
    StateIO<XT>::store(x + idx, s, plane);
    if (xT) xT[idx] = c2_pack(s);
}

// =============================================================================================
// Host side
// =============================================================================================
// Scratch layout: [counter of the streaming kernels (256 B)][gAbar partials: B rows of P float2]
// [column-sum scratch].
namespace {

struct ScanCounters {
    int ticket;
    int pad[63];
};

struct ScanPlan {
    size_t off_part, off_tmp, total;
};

// rows_per_seq: rows of partial sums per sequence (2 for the kernel that puts both CTAs of a pair on one sequence)
ScanPlan plan_scan(int B, int P, int rows_per_seq = 1) {
    ScanPlan s{};
    size_t off = sizeof(ScanCounters);
    s.off_part = off;
    off += align_up((size_t)rows_per_seq * B * P * 8, 256);
    s.off_tmp = off;
    off += align_up(colsum_tmp_floats(rows_per_seq * B, 2 * P) * 4, 256);
    s.total = off;
    return s;
}

}  // namespace

// Sequences of a few steps (single-step mode above all) are not worth a tile pipeline: one
// thread per state walks them.
static bool use_stream(int B, int T, int P) { return T >= 8 && scan_stream_supported(B, T, P); }

size_t scan_scratch_bytes(int B, int T, int P, int rows_per_seq) {
    (void)T;
    return align_up(plan_scan(B, P, rows_per_seq).total, 256);
}

int launch_scan_fwd(int B, int T, int P, const float2* Abar, const float2* Alo, const float2* Bu, const uint8_t* done,
                    const float2* x0, void* x, bool x_bf16, float2* xT, WsHeader* hdr, void* scratch,
                    cudaStream_t st) {
    if (T == 1) {
        const int n = B * (P / 2);
        count_launch();
        if (x_bf16)
            scan_fwd_step_kernel<uint2><<<(n + 255) / 256, 256, 0, st>>>(B, P / 2, (const float4*)Abar, (const float4*)Alo,
                                                                         (const float4*)Bu, done, (const float4*)x0,
                                                                         (uint2*)x, (float4*)xT);
        else
            scan_fwd_step_kernel<float4><<<(n + 255) / 256, 256, 0, st>>>(B, P / 2, (const float4*)Abar, (const float4*)Alo,
                                                                          (const float4*)Bu, done, (const float4*)x0,
                                                                          (float4*)x, (float4*)xT);
        return SSM_OK;
    }
    if (use_stream(B, T, P))
        return launch_scan_fwd_stream(B, T, P, Abar, Alo, Bu, done, x0, x, x_bf16, xT, hdr,
                                      &reinterpret_cast<ScanCounters*>(scratch)->ticket, st);
    const int P2 = P / 2;
    const int blocks = (int)(((size_t)B * P2 + kSeqThreads - 1) / kSeqThreads);
    count_launch();
    if (x_bf16)
        scan_fwd_seq_kernel<uint2><<<blocks, kSeqThreads, 0, st>>>(B, T, P2, (const float4*)Abar, (const float4*)Alo, (const float4*)Bu,
                                                                   done, (const float4*)x0, (uint2*)x, (float4*)xT);
    else
        scan_fwd_seq_kernel<float4><<<blocks, kSeqThreads, 0, st>>>(B, T, P2, (const float4*)Abar, (const float4*)Alo, (const float4*)Bu,
                                                                    done, (const float4*)x0, (float4*)x, (float4*)xT);
    return SSM_OK;
}

int launch_scan_bwd(int B, int T, int P, const float2* Abar, const float2* Alo, const uint8_t* done, const float2* x0,
                    const void* x, bool x_bf16, const float2* gx, const float2* gxT, void* gBu, bool s_bf16,
                    float2* gAbar, float2* gx0, WsHeader* hdr, void* scratch, cudaStream_t st,
                    const float2** gA_part, int* gA_rows) {
    const ScanPlan s = plan_scan(B, P);
    char* base = (char*)scratch;
    float* part = reinterpret_cast<float*>(base + s.off_part);
    float* tmp = reinterpret_cast<float*>(base + s.off_tmp);
    if (x_bf16 != s_bf16) return SSM_ERR_DTYPE;
    if (use_stream(B, T, P)) {
        const int err = launch_scan_bwd_stream(B, T, P, Abar, Alo, done, x0, x, x_bf16, gx, gxT, gBu, gx0, (float2*)part,
                                               hdr, &reinterpret_cast<ScanCounters*>(scratch)->ticket, st);
        if (err != SSM_OK) return err;
    } else {
        count_launch();
        const int blocks1 = (int)(((size_t)B * P + kSeqThreads - 1) / kSeqThreads);
        if (x_bf16)
            scan_bwd_seq1_kernel<uint32_t><<<blocks1, kSeqThreads, 0, st>>>(
                B, T, P, Abar, Alo, done, x0, (const uint32_t*)x, gx, gxT, (uint32_t*)gBu, (float2*)part, gx0);
        else
            scan_bwd_seq1_kernel<float2><<<blocks1, kSeqThreads, 0, st>>>(
                B, T, P, Abar, Alo, done, x0, (const float2*)x, gx, gxT, (float2*)gBu, (float2*)part, gx0);
    }
    if (gA_part && gA_rows)
        *gA_part = reinterpret_cast<const float2*>(launch_reduce_rows(part, B, 2 * P, tmp, kMaxPartialRows, gA_rows, st));
    else
        launch_colsum(part, B, 2 * P, (float*)gAbar, tmp, st);
    return SSM_OK;
}

int launch_gemm_scan_bwd_part(GemmScanBwd g, void* scratch, const float2** gA_part_out, int* gA_rows, cudaStream_t st) {
    const ScanPlan s = plan_scan(g.B, g.P, 2);
    char* base = (char*)scratch;
    float* part = reinterpret_cast<float*>(base + s.off_part);
    float* tmp = reinterpret_cast<float*>(base + s.off_tmp);
    g.gA_part = reinterpret_cast<float2*>(part);
    if (int rc = launch_gemm_scan_bwd(g, st)) return rc;
    *gA_part_out = reinterpret_cast<const float2*>(
        launch_reduce_rows(part, tc_gemm_scan_bwd_part_rows(g.B, g.T, g.H, g.P), 2 * g.P, tmp, kMaxPartialRows, gA_rows, st));
    return SSM_OK;
}

}  // namespace ssm
