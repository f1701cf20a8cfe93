// The scan over the sequence (Sec. III-B Eq. "scan".."full_scan"; resets Sec. IV-A) and its
// adjoint.
//
// Abar is diagonal and the same at every step, so one state is one independent first-order
// recurrence x_t = m_t x_{t-1} + v_t with m_t = Abar or 0 (flagged step).  The work is 8 flop
// per 16 bytes: HBM-bound, so every element is read once and written once.  A thread owns two
// neighbouring states (one 16-byte access per step, coalesced across the warp over p) and
// walks a stretch of time steps sequentially.
//
//  * "seq" kernels: one thread walks a whole sequence (enough parallelism when B*P is large).
//  * "chunk" kernels: a sequence is cut into chunks of L steps that different CTAs scan
//    concurrently.  A CTA keeps its chunk in registers, folds it once from a zero state to get
//    the chunk's aggregate (the second component of the paper's scan tuple; the first, Abar^L,
//    is a constant), publishes it, obtains the state entering the chunk by looking back over
//    its predecessors' aggregates / inclusive states (decoupled look-back; associativity of the
//    operator is what allows it), and folds the chunk again from that state.  A chunk that
//    contains a flagged step publishes an inclusive state at once, because nothing before the
//    flag can pass it.  Chunk ids come from an atomic ticket, so a predecessor has always
//    started; the polls are bounded and give up into the workspace status word.
//
// States are stored as fp32 pairs, or as bf16 pairs when they only feed bf16 tensor-core
// operands (the arithmetic and the carried state stay fp32).
#include <atomic>
#include <chrono>

#include "kernels.h"

namespace ssm {

constexpr int kUnrollFwd = 16;    // time steps whose loads are in flight per thread (seq kernels)
constexpr int kSeqThreads = 64;   // small blocks spread a few hundred thousand threads evenly over the SMs
constexpr int kScanThreads = 128;
constexpr int kFwdChunk = 32;     // steps per chunk, forward
constexpr int kBwdChunk = 16;     // steps per chunk, backward (its buffers also hold x)
constexpr uint32_t kPollLimit = 1u << 22;

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
// (a + alo) * x + b with the small product added first: a step of the recurrence whose multiplier
// is carried as an fp32 pair (hi, lo), i.e. to about 48 bits.
__device__ __forceinline__ float2 cfma2(float2 a, float2 alo, float2 x, float2 b) {
    return cfma(a, x, cfma(alo, x, b));
}
// (a + alo)^n for n a power of two, evaluated in double and returned as an fp32 pair.
template <int N>
__device__ __forceinline__ void cpow2_pair(float2 a, float2 alo, float2& hi, float2& lo) {
    double re = (double)a.x + (double)alo.x, im = (double)a.y + (double)alo.y;
#pragma unroll
    for (int n = 1; n < N; n *= 2) {
        const double r2 = re * re - im * im, i2 = 2.0 * re * im;
        re = r2;
        im = i2;
    }
    hi = make_float2((float)re, (float)im);
    lo = make_float2((float)(re - (double)hi.x), (float)(im - (double)hi.y));
}
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

// =============================================================================================
// Chunked, with decoupled look-back
// =============================================================================================
// Here a thread owns ONE state (8-byte accesses; twice the threads of the whole-sequence
// kernels, half the registers per buffered step) and a CTA of 128 threads is persistent: it
// takes chunk ids from an atomic ticket and always has the loads of its next chunk in flight
// while it folds, publishes, looks back and stores the current one.
//
// Items are numbered chunk-major (item = chunk * nchains + chain, a chain being one
// (sequence, group of 128 states)), so the chunks in flight at any moment are spread over all
// chains and the carry of every chain advances at the same time.
//
// A chunk's record for one state is a single 16-byte word {value, launch tag, state}: it is
// written and read with one 16-byte access, so no fence has to order a value against its flag
// (a fence would also wait for the prefetched loads).  The 62-bit tag is unique to the launch;
// whatever an earlier launch or nobody left in the scratch memory does not match it, so the
// records need no clearing.  state: 1 = aggregate of the chunk alone, 2 = inclusive.
//
// Scratch layout: [ScanCounters (256 B), zeroed before each launch][records: items*128 x 16 B]
// [gA partials (backward): grid rows of P float2][column-sum scratch].
struct ScanCounters {
    int ticket;
    int pad[63];
};

struct ChunkArgs {
    int B, T, P, nchunks, npg, nchains, items;
    const float2* Abar;
    const float2* Alo;     // low part of Abar as an fp32 pair, or NULL
    const uint8_t* done;
    int* ticket;
    uint4* rec;
    uint32_t tag_hi, tag_lo;   // tag_lo has its two low bits clear
    WsHeader* hdr;
};

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

__device__ __forceinline__ void publish(const ChunkArgs& k, int item, float2 v, uint32_t state) {
    uint4 r;
    r.x = __float_as_uint(v.x);
    r.y = __float_as_uint(v.y);
    r.z = k.tag_hi;
    r.w = k.tag_lo | state;
    __stcg(k.rec + (size_t)item * kScanThreads + threadIdx.x, r);
}

// State entering chunk `ci` of a chain, from the records of the chain's earlier chunks (items
// item - nchains, item - 2 nchains, ...).  `mult` is the per-chunk multiplier (Abar^L or its
// conjugate) as an fp32 pair.  A window of kWindow predecessors is fetched with independent
// loads, so a long run of aggregates costs a few round trips instead of one per chunk.
// Bounded: gives up into hdr->status.
constexpr int kWindow = 8;
__device__ __forceinline__ float2 look_back(const ChunkArgs& k, int item, int ci, float2 mult, float2 mult_lo) {
    float2 carry = make_float2(0.f, 0.f);
    float2 m = make_float2(1.f, 0.f);
    int back = 1;             // next predecessor to absorb: chunk ci - back
    uint32_t polls = 0;
    for (;;) {
        uint4 r[kWindow];
#pragma unroll
        for (int i = 0; i < kWindow; ++i) {
            const int d = back + i;
            r[i] = d <= ci ? __ldcv(k.rec + (size_t)(item - d * k.nchains) * kScanThreads + threadIdx.x)
                           : make_uint4(0u, 0u, 0u, 0u);
        }
        int n = 0;            // predecessors usable now: a ready prefix, cut after the first inclusive one
        bool closed = false;
#pragma unroll
        for (int i = 0; i < kWindow; ++i) {
            const bool ready = r[i].z == k.tag_hi && (r[i].w & ~3u) == k.tag_lo && (r[i].w & 3u) != 0u && back + i <= ci;
            if (n == i && !closed && ready) {
                n = i + 1;
                closed = (r[i].w & 3u) == 2u;
            }
        }
        if (n == 0) {
            if (++polls > kPollLimit) {
                k.hdr->status = SSM_ERR_TIMEOUT;
                return carry;
            }
            __nanosleep(20);
            continue;
        }
#pragma unroll
        for (int i = 0; i < kWindow; ++i)
            if (i < n) {
                carry = cfma(m, make_float2(__uint_as_float(r[i].x), __uint_as_float(r[i].y)), carry);
                m = cfma2(mult, mult_lo, m, make_float2(0.f, 0.f));
            }
        if (closed) return carry;
        back += n;
    }
}

// One ticket for the CTA.  All threads call it.
__device__ __forceinline__ int take_ticket(const ChunkArgs& k) {
    __shared__ int s_item;
    __syncthreads();   // everybody has read the previous ticket
    if (threadIdx.x == 0) s_item = atomicAdd(k.ticket, 1);
    __syncthreads();
    return s_item;
}

struct Where {
    int item, ci, c, b, p, len;   // ci: position in processing order; c: chunk index in time
    size_t row0;       // (b * T + t0)
    uint32_t mask;     // bit i: step t0 + i carries a done flag
    bool active;       // this thread's state exists
};

// `from_end`: items count chunks from the end of the sequence (backward pass).
template <int L>
__device__ __forceinline__ Where locate(const ChunkArgs& k, int item, bool from_end) {
    Where w;
    w.item = item;
    const int ci = item / k.nchains;      // position in processing order
    const int chain = item - ci * k.nchains;
    const int pg = chain % k.npg;
    w.b = chain / k.npg;
    w.ci = ci;
    w.c = from_end ? k.nchunks - 1 - ci : ci;
    w.p = pg * kScanThreads + threadIdx.x;
    w.active = w.p < k.P;
    const int t0 = w.c * L;
    w.len = min(L, k.T - t0);
    w.row0 = (size_t)w.b * k.T + t0;
    w.mask = 0u;
    if (k.done) {
        const int lane = threadIdx.x & 31;
        const bool f = lane < w.len && k.done[w.row0 + lane] != 0;
        w.mask = __ballot_sync(0xffffffffu, f);
    }
    return w;
}

template <int L, typename XS>
__global__ void __launch_bounds__(kScanThreads, 4)
scan_fwd_chunk_kernel(ChunkArgs k, const float2* Bu, const float2* __restrict__ x0, XS* x,
                      float2* __restrict__ xT) {
    static_assert(L <= 32 && (L & (L - 1)) == 0, "chunk length: power of two, at most 32");
    const size_t plane = (size_t)k.B * k.T * k.P;
    struct Buf {
        Where w;
        float2 v[L];
    };
    auto fetch = [&](int item, Buf& q) {
        q.w = locate<L>(k, item, false);
        if (!q.w.active) return;
        const float2* src = Bu + q.w.row0 * k.P + q.w.p;
#pragma unroll
        for (int i = 0; i < L; ++i)
            if (i < q.w.len) q.v[i] = __ldcs(src + (size_t)i * k.P);
    };
    auto process = [&](const Buf& q) {
        const Where& w = q.w;
        const float2 a = w.active ? k.Abar[w.p] : make_float2(0.f, 0.f);
        const float2 al = (w.active && k.Alo) ? k.Alo[w.p] : make_float2(0.f, 0.f);
        // fold from a zero state: the chunk's aggregate
        float2 e = make_float2(0.f, 0.f);
        if (w.active) {
#pragma unroll
            for (int i = 0; i < L; ++i)
                if (i < w.len) {
                    if ((w.mask >> i) & 1u) e = make_float2(0.f, 0.f);
                    e = cfma2(a, al, e, q.v[i]);
                }
        }
        const bool has_reset = w.mask != 0u;
        const bool last = w.c == k.nchunks - 1;
        float2 aL, aLlo;
        cpow2_pair<L>(a, al, aL, aLlo);
        float2 carry;
        if (w.c == 0) {
            carry = (x0 && w.active) ? x0[(size_t)w.b * k.P + w.p] : make_float2(0.f, 0.f);
        } else {
            if (!last && w.active) publish(k, w.item, e, has_reset ? 2u : 1u);
            if (w.active) carry = look_back(k, w.item, w.ci, aL, aLlo);
            else carry = make_float2(0.f, 0.f);
        }
        if (!w.active) return;
        if (!last && (w.c == 0 || !has_reset)) publish(k, w.item, has_reset ? e : cfma2(aL, aLlo, carry, e), 2u);
        // fold again from the true entering state and store
        float2 s = carry;
        XS* dst = x + w.row0 * k.P + w.p;
#pragma unroll
        for (int i = 0; i < L; ++i)
            if (i < w.len) {
                if ((w.mask >> i) & 1u) s = make_float2(0.f, 0.f);
                s = cfma2(a, al, s, q.v[i]);
                Raw1<XS>::store(dst + (size_t)i * k.P, s, plane);
            }
        if (last && xT) xT[(size_t)w.b * k.P + w.p] = s;
    };
    Buf q;
    for (int item = take_ticket(k); item < k.items; item = take_ticket(k)) {
        fetch(item, q);
        process(q);
    }
}

// Backward: chunks are taken from the end of the sequence; the carried quantity is
// c_{t-1} = keep_t conj(Abar) (gx_t + c_t), a recurrence of the same form run in reverse.
// gAbar: each CTA keeps one row of partial sums (one entry per state), zeroed by itself first.
template <int L, typename XS>
__global__ void __launch_bounds__(kScanThreads, 4)
scan_bwd_chunk_kernel(ChunkArgs k, const float2* __restrict__ x0, const XS* __restrict__ x, const float2* gx,
                      const float2* __restrict__ gxT, XS* gBu, float2* __restrict__ gA_part,
                      float2* __restrict__ gx0) {
    static_assert(L <= 32 && (L & (L - 1)) == 0, "chunk length: power of two, at most 32");
    const int tid = threadIdx.x;
    const size_t plane = (size_t)k.B * k.T * k.P;
    float2* my_part = gA_part + (size_t)blockIdx.x * k.P;
    for (int p = tid; p < k.P; p += kScanThreads) my_part[p] = make_float2(0.f, 0.f);
    struct Buf {
        Where w;
        float2 v[L];
        Raw1<XS> xp[L];
    };
    auto fetch = [&](int item, Buf& q) {
        q.w = locate<L>(k, item, true);
        if (!q.w.active) return;
        const float2* gsrc = gx + q.w.row0 * k.P + q.w.p;
        const XS* xsrc = x + q.w.row0 * k.P + q.w.p;
        const bool at_start = q.w.c == 0;
#pragma unroll
        for (int i = 0; i < L; ++i)
            if (i < q.w.len) {
                q.v[i] = __ldcs(gsrc + (size_t)i * k.P);
                if (!(at_start && i == 0)) q.xp[i].load(xsrc + ((ptrdiff_t)i - 1) * k.P, plane);
            }
    };
    auto process = [&](const Buf& q) {
        const Where& w = q.w;
        const float2 ac = w.active ? cconj(k.Abar[w.p]) : make_float2(0.f, 0.f);
        const float2 acl = (w.active && k.Alo) ? cconj(k.Alo[w.p]) : make_float2(0.f, 0.f);
        const float2 zero2 = make_float2(0.f, 0.f);
        // fold from a zero carry: aggregate = c_{t0-1} given c_{t1-1} = 0
        float2 e = make_float2(0.f, 0.f);
        if (w.active) {
#pragma unroll
            for (int i = L - 1; i >= 0; --i)
                if (i < w.len) e = ((w.mask >> i) & 1u) ? zero2 : cfma2(ac, acl, cadd(q.v[i], e), zero2);
        }
        const bool has_reset = w.mask != 0u;
        const bool first_item = w.c == k.nchunks - 1;   // the chunk at the end of the sequence
        const bool final_item = w.c == 0;               // the chunk at t = 0: nobody looks at it
        float2 aL, aLlo;
        cpow2_pair<L>(ac, acl, aL, aLlo);
        float2 carry;
        if (first_item) {
            carry = (gxT && w.active) ? gxT[(size_t)w.b * k.P + w.p] : make_float2(0.f, 0.f);
        } else {
            if (!final_item && w.active) publish(k, w.item, e, has_reset ? 2u : 1u);
            if (w.active) carry = look_back(k, w.item, w.ci, aL, aLlo);
            else carry = zero2;
        }
        if (!w.active) return;
        if (!final_item && (first_item || !has_reset)) {
            float2 inc = e;
            if (!has_reset) {
                float2 pw = aL, pwl = aLlo;   // a short chunk at the end multiplies by conj(Abar)^len
                if (w.len != L) {
                    pw = make_float2(1.f, 0.f);
                    pwl = zero2;
                    for (int i = 0; i < w.len; ++i) pw = cfma2(ac, acl, pw, zero2);
                }
                inc = cfma2(pw, pwl, carry, e);
            }
            publish(k, w.item, inc, 2u);
        }
        // true pass
        float2 cc = carry, g = make_float2(0.f, 0.f);
        XS* dst = gBu + w.row0 * k.P + w.p;
        const float2 xinit = (final_item && x0) ? x0[(size_t)w.b * k.P + w.p] : make_float2(0.f, 0.f);
#pragma unroll
        for (int i = L - 1; i >= 0; --i)
            if (i < w.len) {
                const float2 s = cadd(q.v[i], cc);
                Raw1<XS>::store(dst + (size_t)i * k.P, s, plane);
                if ((w.mask >> i) & 1u) {
                    cc = make_float2(0.f, 0.f);
                } else {
                    const float2 xprev = (final_item && i == 0) ? xinit : q.xp[i].get();
                    g = cfma(s, cconj(xprev), g);
                    cc = cfma2(ac, acl, s, zero2);
                }
            }
        my_part[w.p] = cadd(my_part[w.p], g);   // only this thread touches this entry of this row
        if (final_item && gx0) gx0[(size_t)w.b * k.P + w.p] = cc;
    };
    Buf q;
    for (int item = take_ticket(k); item < k.items; item = take_ticket(k)) {
        fetch(item, q);
        process(q);
    }
}

// =============================================================================================
// Host side
// =============================================================================================
namespace {

constexpr int kChunkCtasPerSm = 8;

struct ScanPlan {
    bool chunked;
    int L, nchunks, npg, items, grid;
    size_t off_rec, off_part, off_tmp, zero_bytes, total;
    int part_rows;
};

int scan_sm_count() {
    static int n = 0;
    if (!n) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
            (void)cudaGetLastError();
            n = 148;
        }
    }
    return n;
}

// A different 62-bit value for every launch of this process (splitmix64 over a counter that
// starts from the clock).
uint64_t next_launch_tag() {
    static std::atomic<uint64_t> counter{(uint64_t)std::chrono::steady_clock::now().time_since_epoch().count()};
    uint64_t z = counter.fetch_add(0x9E3779B97F4A7C15ull) + 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

ScanPlan plan_scan(int B, int T, int P, int L) {
    ScanPlan s{};
    const int P2 = P / 2;
    // Whole-sequence threads suffice when there are enough of them to keep HBM busy.
    s.chunked = T >= 2 * L && (size_t)B * P2 < (size_t)16 * 1024;
    s.L = L;
    s.nchunks = s.chunked ? (T + L - 1) / L : 1;
    s.npg = (P + kScanThreads - 1) / kScanThreads;
    s.items = B * s.npg * s.nchunks;
    const int max_grid = scan_sm_count() * kChunkCtasPerSm;
    s.grid = s.items < max_grid ? s.items : max_grid;
    size_t off = sizeof(ScanCounters);
    s.zero_bytes = off;
    s.off_rec = off;
    off += s.chunked ? (size_t)s.items * kScanThreads * 16 : 0;
    s.part_rows = s.chunked ? 148 * 2 * kChunkCtasPerSm : B;   // upper bound on the grid, any device
    s.off_part = off;
    off += align_up((size_t)s.part_rows * P * 8, 256);
    s.off_tmp = off;
    off += align_up(colsum_tmp_floats(s.part_rows, 2 * P) * 4, 256);
    s.total = off;
    return s;
}

ChunkArgs chunk_args(const ScanPlan& s, int B, int T, int P, const float2* Abar, const float2* Alo, const uint8_t* done,
                     WsHeader* hdr, char* scratch) {
    ChunkArgs k;
    k.B = B;
    k.T = T;
    k.P = P;
    k.nchunks = s.nchunks;
    k.npg = s.npg;
    k.nchains = B * s.npg;
    k.items = s.items;
    k.Abar = Abar;
    k.Alo = Alo;
    k.done = done;
    k.ticket = &reinterpret_cast<ScanCounters*>(scratch)->ticket;
    k.rec = reinterpret_cast<uint4*>(scratch + s.off_rec);
    const uint64_t tag = next_launch_tag();
    k.tag_hi = (uint32_t)(tag >> 32);
    k.tag_lo = (uint32_t)tag & ~3u;
    k.hdr = hdr;
    return k;
}

}  // namespace

size_t scan_scratch_bytes(int B, int T, int P) {
    const size_t f = plan_scan(B, T, P, kFwdChunk).total, b = plan_scan(B, T, P, kBwdChunk).total;
    return align_up(f > b ? f : b, 256);
}

int launch_scan_fwd(int B, int T, int P, const float2* Abar, const float2* Alo, const float2* Bu, const uint8_t* done,
                    const float2* x0, void* x, bool x_bf16, float2* xT, WsHeader* hdr, void* scratch,
                    cudaStream_t st) {
    const int P2 = P / 2;
    const ScanPlan s = plan_scan(B, T, P, kFwdChunk);
    if (!s.chunked) {
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
    if (cudaMemsetAsync(scratch, 0, s.zero_bytes, st) != cudaSuccess) return SSM_ERR_CUDA;
    const ChunkArgs k = chunk_args(s, B, T, P, Abar, Alo, done, hdr, (char*)scratch);
    count_launch();
    if (x_bf16)
        scan_fwd_chunk_kernel<kFwdChunk, uint32_t><<<s.grid, kScanThreads, 0, st>>>(k, Bu, x0, (uint32_t*)x, xT);
    else
        scan_fwd_chunk_kernel<kFwdChunk, float2><<<s.grid, kScanThreads, 0, st>>>(k, Bu, x0, (float2*)x, xT);
    return SSM_OK;
}

int launch_scan_bwd(int B, int T, int P, const float2* Abar, const float2* Alo, const uint8_t* done, const float2* x0,
                    const void* x, bool x_bf16, const float2* gx, const float2* gxT, void* gBu, bool s_bf16,
                    float2* gAbar, float2* gx0, WsHeader* hdr, void* scratch, cudaStream_t st) {
    const ScanPlan s = plan_scan(B, T, P, kBwdChunk);
    char* base = (char*)scratch;
    float* part = reinterpret_cast<float*>(base + s.off_part);
    float* tmp = reinterpret_cast<float*>(base + s.off_tmp);
    if (x_bf16 != s_bf16) return SSM_ERR_DTYPE;
    int rows = B;
    if (!s.chunked) {
        count_launch();
        const int blocks1 = (int)(((size_t)B * P + kSeqThreads - 1) / kSeqThreads);
        if (x_bf16)
            scan_bwd_seq1_kernel<uint32_t><<<blocks1, kSeqThreads, 0, st>>>(
                B, T, P, Abar, Alo, done, x0, (const uint32_t*)x, gx, gxT, (uint32_t*)gBu, (float2*)part, gx0);
        else
            scan_bwd_seq1_kernel<float2><<<blocks1, kSeqThreads, 0, st>>>(
                B, T, P, Abar, Alo, done, x0, (const float2*)x, gx, gxT, (float2*)gBu, (float2*)part, gx0);
    } else {
        if (cudaMemsetAsync(scratch, 0, s.zero_bytes, st) != cudaSuccess) return SSM_ERR_CUDA;
        const ChunkArgs k = chunk_args(s, B, T, P, Abar, Alo, done, hdr, base);
        rows = s.grid < s.part_rows ? s.grid : s.part_rows;
        count_launch();
        if (x_bf16)
            scan_bwd_chunk_kernel<kBwdChunk, uint32_t><<<rows, kScanThreads, 0, st>>>(
                k, x0, (const uint32_t*)x, gx, gxT, (uint32_t*)gBu, (float2*)part, gx0);
        else
            scan_bwd_chunk_kernel<kBwdChunk, float2><<<rows, kScanThreads, 0, st>>>(
                k, x0, (const float2*)x, gx, gxT, (float2*)gBu, (float2*)part, gx0);
    }
    launch_colsum(part, rows, 2 * P, (float*)gAbar, tmp, st);
    return SSM_OK;
}

}  // namespace ssm
