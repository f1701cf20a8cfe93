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
#include "kernels.h"

namespace ssm {

constexpr int kUnrollFwd = 16;    // time steps whose loads are in flight per thread (seq kernels)
constexpr int kUnrollBwd = 8;
constexpr int kSeqThreads = 64;   // small blocks spread a few hundred thousand threads evenly over the SMs
constexpr int kScanThreads = 128;
constexpr int kFwdChunk = 32;     // steps per chunk, forward
constexpr int kBwdChunk = 16;     // steps per chunk, backward (it also holds x)
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
__device__ __forceinline__ C2 c2_from(const float4 v) { return C2{make_float2(v.x, v.y), make_float2(v.z, v.w)}; }
__device__ __forceinline__ float4 c2_pack(const C2& v) { return make_float4(v.a.x, v.a.y, v.b.x, v.b.y); }

// =============================================================================================
// Whole sequence per thread
// =============================================================================================
// grid: ceil(B * P/2 / kSeqThreads); thread -> (b, pair of states).  x may alias Bu.
template <typename XT>
__global__ void __launch_bounds__(kSeqThreads)
scan_fwd_seq_kernel(int B, int T, int P2, const float4* __restrict__ Abar, const float4* Bu,
                    const uint8_t* __restrict__ done, const float4* __restrict__ x0, XT* x,
                    float4* __restrict__ xT) {
    const int idx = blockIdx.x * kSeqThreads + threadIdx.x;
    if (idx >= B * P2) return;
    const int b = idx / P2, pp = idx - b * P2;
    const size_t plane = (size_t)B * T * P2;
    const C2 a = c2_from(Abar[pp]);
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
                s.a = cfma(a.a, s.a, v[i].a);
                s.b = cfma(a.b, s.b, v[i].b);
                StateIO<XT>::store(dst + (size_t)t * P2, s, plane);
            }
        }
    }
    if (xT) xT[(size_t)b * P2 + pp] = c2_pack(s);
}

// Undecoded state loads, so that a whole batch of them can be in flight while the previous
// batch is being processed.
template <typename ST> struct RawState;
template <> struct RawState<float4> {
    float4 v;
    __device__ __forceinline__ void load(const float4* p, size_t) { v = __ldcs(p); }
    __device__ __forceinline__ C2 get() const { return c2_from(v); }
};
template <> struct RawState<uint2> {
    uint2 hi, lo;
    __device__ __forceinline__ void load(const uint2* p, size_t plane) {
        hi = __ldcs(p);
        lo = __ldcs(p + plane);
    }
    __device__ __forceinline__ C2 get() const {
        const C2 h = unpack_bf16x4(hi), l = unpack_bf16x4(lo);
        return C2{cadd(h.a, l.a), cadd(h.b, l.b)};
    }
};

// s_t = gx_t + c_t,  c_{t-1} = keep_t conj(Abar) s_t  (c_{T-1} = gxT);
// gAbar partial = sum_t keep_t s_t conj(x_{t-1}).  gBu may alias gx.
// Two register batches of kUnrollBwd steps alternate: the loads of one are issued before the
// other is processed.
template <typename XT, typename ST>
__global__ void __launch_bounds__(kSeqThreads)
scan_bwd_seq_kernel(int B, int T, int P2, const float4* __restrict__ Abar, const uint8_t* __restrict__ done,
                    const float4* __restrict__ x0, const XT* __restrict__ x, const float4* gx,
                    const float4* __restrict__ gxT, ST* gBu, float4* __restrict__ gA_part,
                    float4* __restrict__ gx0) {
    const int idx = blockIdx.x * kSeqThreads + threadIdx.x;
    if (idx >= B * P2) return;
    const int b = idx / P2, pp = idx - b * P2;
    const size_t plane = (size_t)B * T * P2;
    const C2 a = c2_from(Abar[pp]);
    const float2 ac0 = cconj(a.a), ac1 = cconj(a.b);
    C2 c = gxT ? c2_from(gxT[(size_t)b * P2 + pp]) : c2_zero();
    C2 g = c2_zero();
    const float4* gsrc = gx + (size_t)b * T * P2 + pp;
    const XT* xsrc = x + (size_t)b * T * P2 + pp;
    ST* dst = gBu + (size_t)b * T * P2 + pp;
    const uint8_t* dn = done ? done + (size_t)b * T : nullptr;
    const C2 xinit = x0 ? c2_from(x0[(size_t)b * P2 + pp]) : c2_zero();

    struct Batch {
        float4 v[kUnrollBwd];
        RawState<XT> xp[kUnrollBwd];
        uint32_t flags;
    };
    // steps t0, t0-1, ..., t0-kUnrollBwd+1 (those that exist)
    auto fetch = [&](int t0, Batch& q) {
        q.flags = 0u;
#pragma unroll
        for (int i = 0; i < kUnrollBwd; ++i) {
            const int t = t0 - i;
            if (t >= 0) {
                q.v[i] = __ldcs(gsrc + (size_t)t * P2);
                if (t > 0) q.xp[i].load(xsrc + (size_t)(t - 1) * P2, plane);
                if (dn && dn[t] != 0) q.flags |= 1u << i;
            }
        }
    };
    auto process = [&](int t0, const Batch& q) {
#pragma unroll
        for (int i = 0; i < kUnrollBwd; ++i) {
            const int t = t0 - i;
            if (t >= 0) {
                const C2 vi = c2_from(q.v[i]);
                const C2 s{cadd(vi.a, c.a), cadd(vi.b, c.b)};
                StateIO<ST>::store(dst + (size_t)t * P2, s, plane);
                if ((q.flags >> i) & 1u) {
                    c = c2_zero();
                } else {
                    const C2 xprev = t > 0 ? q.xp[i].get() : xinit;
                    g.a = cfma(s.a, cconj(xprev.a), g.a);
                    g.b = cfma(s.b, cconj(xprev.b), g.b);
                    c.a = cmul(ac0, s.a);
                    c.b = cmul(ac1, s.b);
                }
            }
        }
    };
    Batch q0, q1;
    fetch(T - 1, q0);
    for (int t0 = T - 1; t0 >= 0; t0 -= 2 * kUnrollBwd) {
        fetch(t0 - kUnrollBwd, q1);
        process(t0, q0);
        fetch(t0 - 2 * kUnrollBwd, q0);
        process(t0 - kUnrollBwd, q1);
    }
    gA_part[(size_t)b * P2 + pp] = c2_pack(g);
    if (gx0) gx0[(size_t)b * P2 + pp] = c2_pack(c);
}

// =============================================================================================
// Chunked, with decoupled look-back
// =============================================================================================
// Scratch layout: [ScanCounters (256 B)][status: items*128 int][agg: items*128 float4]
// [incl: items*128 float4][gA partials (backward): items * P2 float4][column-sum scratch].
// Everything up to the end of `status` is zeroed before each launch.
struct ScanCounters {
    int ticket;
    int pad[63];
};

struct ChunkArgs {
    int B, T, P2, nchunks, npg;
    const float4* Abar;
    const uint8_t* done;
    int* ticket;
    int* status;
    float4* agg;
    float4* incl;
    WsHeader* hdr;
};

// m^n for n a power of two
template <int N>
__device__ __forceinline__ float2 cpow2(float2 m) {
#pragma unroll
    for (int n = 1; n < N; n *= 2) m = cmul(m, m);
    return m;
}

__device__ __forceinline__ void publish(float4* slot, int* status, const C2& v, int state) {
    *slot = c2_pack(v);
    __threadfence();
    *reinterpret_cast<volatile int*>(status) = state;
}

// State entering this chunk, from the records of the chunks processed before it (items
// item-1, item-2, ... in ticket order).  `mult` is the per-chunk multiplier (Abar^L or its
// conjugate).  Bounded: gives up into hdr->status.
__device__ __forceinline__ C2 look_back(const ChunkArgs& k, int item, int tid, float2 mult_a, float2 mult_b) {
    C2 carry = c2_zero();
    float2 ma = make_float2(1.f, 0.f), mb = ma;
    for (int j = item - 1;; --j) {
        const size_t r = (size_t)j * kScanThreads + tid;
        volatile int* st = k.status + r;
        int state = *st;
        uint32_t polls = 0;
        while (state == 0) {
            if (++polls > kPollLimit) {
                k.hdr->status = SSM_ERR_TIMEOUT;
                return carry;
            }
            __nanosleep(40);
            state = *st;
        }
        __threadfence();
        const C2 v = c2_from(__ldcg((state == 2 ? k.incl : k.agg) + r));
        carry.a = cfma(ma, v.a, carry.a);
        carry.b = cfma(mb, v.b, carry.b);
        if (state == 2) return carry;
        ma = cmul(ma, mult_a);
        mb = cmul(mb, mult_b);
    }
}

// Decodes the ticket: chunks of one (sequence, state group) are consecutive items.
struct Item {
    int item, c, pg, b;
};
__device__ __forceinline__ Item take_item(const ChunkArgs& k) {
    __shared__ int s_item;
    if (threadIdx.x == 0) s_item = atomicAdd(k.ticket, 1);
    __syncthreads();
    Item it;
    it.item = s_item;
    it.c = it.item % k.nchunks;
    const int rest = it.item / k.nchunks;
    it.pg = rest % k.npg;
    it.b = rest / k.npg;
    return it;
}

// Bit i of the result: step t0 + i carries a done flag (i < len <= 32).
__device__ __forceinline__ uint32_t done_mask(const uint8_t* done, size_t row0, int len) {
    if (!done) return 0u;
    const int lane = threadIdx.x & 31;
    const bool f = lane < len && done[row0 + lane] != 0;
    return __ballot_sync(0xffffffffu, f);
}

template <int L, typename XT>
__global__ void __launch_bounds__(kScanThreads)
scan_fwd_chunk_kernel(ChunkArgs k, const float4* Bu, const float4* __restrict__ x0, XT* x,
                      float4* __restrict__ xT) {
    static_assert(L <= 32 && (L & (L - 1)) == 0, "chunk length: power of two, at most 32");
    const Item it = take_item(k);
    const int tid = threadIdx.x;
    const int pp = it.pg * kScanThreads + tid;
    const size_t plane = (size_t)k.B * k.T * k.P2;
    const int t0 = it.c * L;
    const int len = min(L, k.T - t0);
    const size_t row0 = (size_t)it.b * k.T + t0;
    const uint32_t mask = done_mask(k.done, row0, len);
    if (pp >= k.P2) return;
    const C2 a = c2_from(k.Abar[pp]);
    const float4* src = Bu + row0 * k.P2 + pp;
    C2 v[L];
#pragma unroll
    for (int i = 0; i < L; ++i)
        if (i < len) v[i] = StateIO<float4>::load(src + (size_t)i * k.P2, 0);
    // fold from a zero state: the chunk's aggregate
    C2 e = c2_zero();
#pragma unroll
    for (int i = 0; i < L; ++i)
        if (i < len) {
            if ((mask >> i) & 1u) e = c2_zero();
            e.a = cfma(a.a, e.a, v[i].a);
            e.b = cfma(a.b, e.b, v[i].b);
        }
    const bool has_reset = mask != 0u;
    const bool last = it.c == k.nchunks - 1;
    const float2 aLa = cpow2<L>(a.a), aLb = cpow2<L>(a.b);
    const size_t rec = (size_t)it.item * kScanThreads + tid;
    C2 carry;
    if (it.c == 0) {
        carry = x0 ? c2_from(x0[(size_t)it.b * k.P2 + pp]) : c2_zero();
    } else {
        if (!last) {
            if (has_reset) publish(k.incl + rec, k.status + rec, e, 2);
            else publish(k.agg + rec, k.status + rec, e, 1);
        }
        carry = look_back(k, it.item, tid, aLa, aLb);
    }
    if (!last && (it.c == 0 || !has_reset)) {
        C2 inc = e;
        if (!has_reset) {
            inc.a = cfma(aLa, carry.a, e.a);
            inc.b = cfma(aLb, carry.b, e.b);
        }
        publish(k.incl + rec, k.status + rec, inc, 2);
    }
    // fold again from the true entering state and store
    C2 s = carry;
    XT* dst = x + row0 * k.P2 + pp;
#pragma unroll
    for (int i = 0; i < L; ++i)
        if (i < len) {
            if ((mask >> i) & 1u) s = c2_zero();
            s.a = cfma(a.a, s.a, v[i].a);
            s.b = cfma(a.b, s.b, v[i].b);
            StateIO<XT>::store(dst + (size_t)i * k.P2, s, plane);
        }
    if (last && xT) xT[(size_t)it.b * k.P2 + pp] = c2_pack(s);
}

// Backward: chunks are taken from the end of the sequence; the carried quantity is
// c_{t-1} = keep_t conj(Abar) (gx_t + c_t), a recurrence of the same form run in reverse.
template <int L, typename XT, typename ST>
__global__ void __launch_bounds__(kScanThreads)
scan_bwd_chunk_kernel(ChunkArgs k, const float4* __restrict__ x0, const XT* __restrict__ x, const float4* gx,
                      const float4* __restrict__ gxT, ST* gBu, float4* __restrict__ gA_part,
                      float4* __restrict__ gx0) {
    static_assert(L <= 32 && (L & (L - 1)) == 0, "chunk length: power of two, at most 32");
    const Item it = take_item(k);
    const int tid = threadIdx.x;
    const int pp = it.pg * kScanThreads + tid;
    const size_t plane = (size_t)k.B * k.T * k.P2;
    const int c = k.nchunks - 1 - it.c;          // chunk index in time; it.c counts from the end
    const int t0 = c * L;
    const int len = min(L, k.T - t0);
    const size_t row0 = (size_t)it.b * k.T + t0;
    const uint32_t mask = done_mask(k.done, row0, len);
    if (pp >= k.P2) return;
    const C2 a = c2_from(k.Abar[pp]);
    const float2 ac0 = cconj(a.a), ac1 = cconj(a.b);
    const float4* gsrc = gx + row0 * k.P2 + pp;
    const XT* xsrc = x + row0 * k.P2 + pp;
    C2 v[L], xp[L];
#pragma unroll
    for (int i = 0; i < L; ++i)
        if (i < len) {
            v[i] = StateIO<float4>::load(gsrc + (size_t)i * k.P2, 0);
            if (t0 + i > 0) xp[i] = StateIO<XT>::load(xsrc + ((ptrdiff_t)i - 1) * k.P2, plane);
            else xp[i] = x0 ? c2_from(x0[(size_t)it.b * k.P2 + pp]) : c2_zero();
        }
    // fold from a zero carry: aggregate = c_{t0-1} given c_{t1-1} = 0
    C2 e = c2_zero();
#pragma unroll
    for (int i = L - 1; i >= 0; --i)
        if (i < len) {
            if ((mask >> i) & 1u) {
                e = c2_zero();
            } else {
                e.a = cmul(ac0, cadd(v[i].a, e.a));
                e.b = cmul(ac1, cadd(v[i].b, e.b));
            }
        }
    const bool has_reset = mask != 0u;
    const bool first_item = it.c == 0;           // the chunk at the end of the sequence
    const bool final_item = it.c == k.nchunks - 1;  // the chunk at t = 0: nobody looks at it
    const float2 aLa = cpow2<L>(ac0), aLb = cpow2<L>(ac1);
    const size_t rec = (size_t)it.item * kScanThreads + tid;
    C2 carry;
    if (first_item) {
        carry = gxT ? c2_from(gxT[(size_t)it.b * k.P2 + pp]) : c2_zero();
    } else {
        if (!final_item) {
            if (has_reset) publish(k.incl + rec, k.status + rec, e, 2);
            else publish(k.agg + rec, k.status + rec, e, 1);
        }
        carry = look_back(k, it.item, tid, aLa, aLb);
    }
    if (!final_item && (first_item || !has_reset)) {
        C2 inc = e;
        if (!has_reset) {
            // a short chunk at the end of the sequence multiplies by conj(Abar)^len
            float2 pa = aLa, pb = aLb;
            if (len != L) {
                pa = make_float2(1.f, 0.f);
                pb = pa;
                for (int i = 0; i < len; ++i) {
                    pa = cmul(pa, ac0);
                    pb = cmul(pb, ac1);
                }
            }
            inc.a = cfma(pa, carry.a, e.a);
            inc.b = cfma(pb, carry.b, e.b);
        }
        publish(k.incl + rec, k.status + rec, inc, 2);
    }
    // true pass
    C2 cc = carry, g = c2_zero();
    ST* dst = gBu + row0 * k.P2 + pp;
#pragma unroll
    for (int i = L - 1; i >= 0; --i)
        if (i < len) {
            const C2 s{cadd(v[i].a, cc.a), cadd(v[i].b, cc.b)};
            StateIO<ST>::store(dst + (size_t)i * k.P2, s, plane);
            if ((mask >> i) & 1u) {
                cc = c2_zero();
            } else {
                g.a = cfma(s.a, cconj(xp[i].a), g.a);
                g.b = cfma(s.b, cconj(xp[i].b), g.b);
                cc.a = cmul(ac0, s.a);
                cc.b = cmul(ac1, s.b);
            }
        }
    gA_part[((size_t)it.b * k.nchunks + c) * k.P2 + pp] = c2_pack(g);
    if (final_item && gx0) gx0[(size_t)it.b * k.P2 + pp] = c2_pack(cc);
}

// =============================================================================================
// Host side
// =============================================================================================
namespace {

struct ScanPlan {
    bool chunked;
    int L, nchunks, npg, items;
    size_t off_status, off_agg, off_incl, off_part, off_tmp, zero_bytes, total;
    int part_rows;
};

ScanPlan plan_scan(int B, int T, int P, int L) {
    ScanPlan s{};
    const int P2 = P / 2;
    // Whole-sequence threads suffice when there are enough of them to keep HBM busy.
    s.chunked = T >= 2 * L && (size_t)B * P2 < (size_t)16 * 1024;
    s.L = L;
    s.nchunks = s.chunked ? (T + L - 1) / L : 1;
    s.npg = (P2 + kScanThreads - 1) / kScanThreads;
    s.items = B * s.npg * s.nchunks;
    size_t off = sizeof(ScanCounters);
    s.off_status = off;
    off += s.chunked ? align_up((size_t)s.items * kScanThreads * 4, 256) : 0;
    s.zero_bytes = off;
    s.off_agg = off;
    off += s.chunked ? (size_t)s.items * kScanThreads * 16 : 0;
    s.off_incl = off;
    off += s.chunked ? (size_t)s.items * kScanThreads * 16 : 0;
    s.part_rows = B * s.nchunks;
    s.off_part = off;
    off += align_up((size_t)s.part_rows * P2 * 16, 256);
    s.off_tmp = off;
    off += align_up(colsum_tmp_floats(s.part_rows, 2 * P) * 4, 256);
    s.total = off;
    return s;
}

ChunkArgs chunk_args(const ScanPlan& s, int B, int T, int P, const float2* Abar, const uint8_t* done,
                     WsHeader* hdr, char* scratch) {
    ChunkArgs k;
    k.B = B;
    k.T = T;
    k.P2 = P / 2;
    k.nchunks = s.nchunks;
    k.npg = s.npg;
    k.Abar = (const float4*)Abar;
    k.done = done;
    k.ticket = &reinterpret_cast<ScanCounters*>(scratch)->ticket;
    k.status = reinterpret_cast<int*>(scratch + s.off_status);
    k.agg = reinterpret_cast<float4*>(scratch + s.off_agg);
    k.incl = reinterpret_cast<float4*>(scratch + s.off_incl);
    k.hdr = hdr;
    return k;
}

}  // namespace

size_t scan_scratch_bytes(int B, int T, int P) {
    const size_t f = plan_scan(B, T, P, kFwdChunk).total, b = plan_scan(B, T, P, kBwdChunk).total;
    return align_up(f > b ? f : b, 256);
}

int launch_scan_fwd(int B, int T, int P, const float2* Abar, const float2* Bu, const uint8_t* done,
                    const float2* x0, void* x, bool x_bf16, float2* xT, WsHeader* hdr, void* scratch,
                    cudaStream_t st) {
    const int P2 = P / 2;
    const ScanPlan s = plan_scan(B, T, P, kFwdChunk);
    if (!s.chunked) {
        const int blocks = (int)(((size_t)B * P2 + kSeqThreads - 1) / kSeqThreads);
        count_launch();
        if (x_bf16)
            scan_fwd_seq_kernel<uint2><<<blocks, kSeqThreads, 0, st>>>(B, T, P2, (const float4*)Abar, (const float4*)Bu,
                                                                       done, (const float4*)x0, (uint2*)x, (float4*)xT);
        else
            scan_fwd_seq_kernel<float4><<<blocks, kSeqThreads, 0, st>>>(B, T, P2, (const float4*)Abar, (const float4*)Bu,
                                                                        done, (const float4*)x0, (float4*)x, (float4*)xT);
        return SSM_OK;
    }
    if (cudaMemsetAsync(scratch, 0, s.zero_bytes, st) != cudaSuccess) return SSM_ERR_CUDA;
    const ChunkArgs k = chunk_args(s, B, T, P, Abar, done, hdr, (char*)scratch);
    count_launch();
    if (x_bf16)
        scan_fwd_chunk_kernel<kFwdChunk, uint2><<<s.items, kScanThreads, 0, st>>>(k, (const float4*)Bu, (const float4*)x0,
                                                                                 (uint2*)x, (float4*)xT);
    else
        scan_fwd_chunk_kernel<kFwdChunk, float4><<<s.items, kScanThreads, 0, st>>>(k, (const float4*)Bu, (const float4*)x0,
                                                                                  (float4*)x, (float4*)xT);
    return SSM_OK;
}

int launch_scan_bwd(int B, int T, int P, const float2* Abar, const uint8_t* done, const float2* x0,
                    const void* x, bool x_bf16, const float2* gx, const float2* gxT, void* gBu, bool s_bf16,
                    float2* gAbar, float2* gx0, WsHeader* hdr, void* scratch, cudaStream_t st) {
    const int P2 = P / 2;
    const ScanPlan s = plan_scan(B, T, P, kBwdChunk);
    char* base = (char*)scratch;
    float4* part = reinterpret_cast<float4*>(base + s.off_part);
    float* tmp = reinterpret_cast<float*>(base + s.off_tmp);
    if (x_bf16 != s_bf16) return SSM_ERR_DTYPE;
    if (!s.chunked) {
        const int blocks = (int)(((size_t)B * P2 + kSeqThreads - 1) / kSeqThreads);
        count_launch();
        if (x_bf16)
            scan_bwd_seq_kernel<uint2, uint2><<<blocks, kSeqThreads, 0, st>>>(
                B, T, P2, (const float4*)Abar, done, (const float4*)x0, (const uint2*)x, (const float4*)gx,
                (const float4*)gxT, (uint2*)gBu, part, (float4*)gx0);
        else
            scan_bwd_seq_kernel<float4, float4><<<blocks, kSeqThreads, 0, st>>>(
                B, T, P2, (const float4*)Abar, done, (const float4*)x0, (const float4*)x, (const float4*)gx,
                (const float4*)gxT, (float4*)gBu, part, (float4*)gx0);
    } else {
        if (cudaMemsetAsync(scratch, 0, s.zero_bytes, st) != cudaSuccess) return SSM_ERR_CUDA;
        const ChunkArgs k = chunk_args(s, B, T, P, Abar, done, hdr, base);
        count_launch();
        if (x_bf16)
            scan_bwd_chunk_kernel<kBwdChunk, uint2, uint2><<<s.items, kScanThreads, 0, st>>>(
                k, (const float4*)x0, (const uint2*)x, (const float4*)gx, (const float4*)gxT, (uint2*)gBu, part,
                (float4*)gx0);
        else
            scan_bwd_chunk_kernel<kBwdChunk, float4, float4><<<s.items, kScanThreads, 0, st>>>(
                k, (const float4*)x0, (const float4*)x, (const float4*)gx, (const float4*)gxT, (float4*)gBu, part,
                (float4*)gx0);
    }
    launch_colsum((const float*)part, s.part_rows, 2 * P, (float*)gAbar, tmp, st);
    return SSM_OK;
}

}  // namespace ssm
