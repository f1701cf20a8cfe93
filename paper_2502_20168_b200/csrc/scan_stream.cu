// The scan over the sequence (Sec. III-B Eq. "scan".."full_scan"; resets Sec. IV-A) and its
// adjoint as streaming kernels: tiles move between HBM and shared memory by TMA, and all the
// parallelism over time stays inside one CTA.
//
// A chain is one sequence b and a group of G neighbouring states (G = 16..128, chosen so that
// there are enough chains to fill the machine).  A persistent CTA takes chains from an atomic
// counter and walks each one from its first step to its last (the adjoint: last to first) in
// tiles of R rows x G states.  The 256 scanning threads of the CTA are `slices` = 256 / G
// groups of G; group q owns rows [q r, (q + 1) r) of the tile (r = kRows) and one thread owns
// one state there.  Per tile:
//   1. every thread folds its r rows from a zero state (the second component of the paper's
//      scan element; the first is Abar^r, or 0 after a flagged row) and leaves the pair in
//      shared memory;
//   2. after one barrier it combines the pairs of the groups before it, starting from the state
//      that entered the tile (kept in shared memory from the previous tile), which is the
//      associative operator of Eq. "associative" / "associative_reset" applied in order;
//   3. it folds its rows again from that state and writes the results over the tile, in the
//      layout of the output; one thread hands the tile to the TMA unit.
// No CTA ever waits for another one, the result does not depend on scheduling, and a producer
// warp keeps the next tiles in flight through a ring of three or four shared-memory stages.
//
// The tensor maps are three-dimensional (2P, T, B): rows past the end of a sequence read as
// zero and are dropped on store; the adjoint's tile of x_{t-1} starts one row early, and row -1
// reads as zero.  Every barrier wait is bounded and gives up into the workspace status word.
#include "kernels.h"
#include "scan_math.cuh"
#include "tma.cuh"

namespace ssm {
namespace stream {

using namespace tma;

constexpr int kConsumers = 256;
constexpr int kThreads = kConsumers + 32;
constexpr int kMaxStages = 4;   // stages of the ring: Args::stages of them are used (3, or 4 for the forward scan of narrow chains)
constexpr int kMaxRows = 256;   // rows of the tallest tile (limit of a TMA box)
constexpr int kMaxG = 128;
constexpr int kFwdRows = 8;     // rows per thread and tile, forward (16 measured 6 % slower on few long sequences, equal elsewhere)
constexpr int kBwdRows = 8;     // backward: its stages also hold x
constexpr int kBwdRowsLong = 16;   // backward, sequences of kBwdLongT steps or more: one CTA per SM with tiles twice as tall
constexpr int kBwdLongT = 2048;    // (16 x 16384: 5.15 -> 5.5 TB/s, 64 x 4096: 5.7 -> 6.2; T = 1024 equal; T = 64 9 % slower, T = 16 2.7 x)

struct Args {
    int B, T, P;
    int G, g_shift;      // states per chain (power of two) and its log2
    int slices, R;       // groups of threads along time; rows per tile
    int ntiles, npg, nchains;
    int stages;          // stages of the shared-memory ring in use (<= kMaxStages)
    const float2* Abar;
    const float2* Alo;   // low part of Abar as an fp32 pair, or NULL
    const uint8_t* done;
    int* ticket;
    WsHeader* hdr;
};

struct Meta {
    int chain;   // -1: no more work
    int tile;    // position in processing order
};

struct Shared {
    uint64_t full[kMaxStages], empty[kMaxStages];
    Meta meta[kMaxStages];
    int abort_flag;       // raised by a scanning thread whose wait gave up; read by all after a barrier
    int producer_abort;   // the producer warp's own
    uint8_t flags[kMaxStages][kMaxRows];
    float2 agg_e[kConsumers], agg_m[kConsumers], agg_ml[kConsumers];
    float2 carry[2][kMaxG];
    float2 gsum[kConsumers];
};

template <bool kPair>
__device__ __forceinline__ float2 rstep(float2 a, float2 al, float2 x, float2 b) {
    if (kPair) return cfma2(a, al, x, b);
    return cfma(a, x, b);
}

__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory"); }

// (a + alo)^n for any small n, in double, as an fp32 pair.
__device__ __forceinline__ void cpow_n_pair(float2 a, float2 alo, int n, float2& hi, float2& lo) {
    const double ar = (double)a.x + (double)alo.x, ai = (double)a.y + (double)alo.y;
    double re = 1.0, im = 0.0;
    for (int i = 0; i < n; ++i) {
        const double r2 = re * ar - im * ai, i2 = re * ai + im * ar;
        re = r2;
        im = i2;
    }
    hi = make_float2((float)re, (float)im);
    lo = make_float2((float)(re - (double)hi.x), (float)(im - (double)hi.y));
}

// Result tile written over the input tile.  fp32 pairs: same layout.  bf16: a tile of high
// halves (rows of G 32-bit words) followed by a tile of low halves.
template <typename XS> struct TileIO;
template <> struct TileIO<float2> {
    static __device__ __forceinline__ void put(uint8_t* tile, int R, int G, int row, int col, float2 s) {
        reinterpret_cast<float2*>(tile)[row * G + col] = s;
    }
    static __device__ __forceinline__ float2 get(const uint8_t* tile, int R, int G, int row, int col) {
        return reinterpret_cast<const float2*>(tile)[row * G + col];
    }
};
template <> struct TileIO<uint32_t> {
    static __device__ __forceinline__ void put(uint8_t* tile, int R, int G, int row, int col, float2 s) {
        const __nv_bfloat162 h = __floats2bfloat162_rn(s.x, s.y);
        const float2 hf = __bfloat1622float2(h);
        const __nv_bfloat162 l = __floats2bfloat162_rn(s.x - hf.x, s.y - hf.y);
        uint32_t* t = reinterpret_cast<uint32_t*>(tile);
        t[row * G + col] = *reinterpret_cast<const uint32_t*>(&h);
        t[(R + row) * G + col] = *reinterpret_cast<const uint32_t*>(&l);
    }
    static __device__ __forceinline__ float2 get(const uint8_t* tile, int R, int G, int row, int col) {
        const uint32_t* t = reinterpret_cast<const uint32_t*>(tile);
        const uint32_t hi = t[row * G + col], lo = t[(R + row) * G + col];
        return cadd(__bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&hi)),
                    __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&lo)));
    }
};

__device__ __forceinline__ void init_shared(Shared& sm) {
    if (threadIdx.x == 0) {
        for (int i = 0; i < kMaxStages; ++i) {
            mbar_init(smem_u32(&sm.full[i]), 1);
            mbar_init(smem_u32(&sm.empty[i]), 1);
        }
        sm.abort_flag = 0;
        sm.producer_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
}

// Producer warp: chains from the counter; per tile the done flags and up to three TMA loads
// (m1 / m2, the states of the adjoint, start one row earlier).
template <bool kBwd>
__device__ __forceinline__ void producer(const Args& k, Shared& sm, uint8_t* stages, uint32_t stage_bytes,
                                         const CUtensorMap* m0, const CUtensorMap* m1, const CUtensorMap* m2,
                                         uint32_t bytes0, uint32_t bytes1, uint32_t bytes2) {
    const int lane = threadIdx.x & 31;
    int s = 0, round = 0;   // stage of the next tile; how many times the ring has wrapped
    for (;;) {
        int chain = 0;
        if (lane == 0) chain = atomicAdd(k.ticket, 1);
        chain = __shfl_sync(0xffffffffu, chain, 0);
        const bool end = chain >= k.nchains;
        const int tiles = end ? 1 : k.ntiles;
        for (int j = 0; j < tiles; ++j, s = (s + 1 == k.stages) ? 0 : s + 1, round += (s == 0)) {
            if (round > 0 && !mbar_wait(smem_u32(&sm.empty[s]), (round - 1) & 1, &sm.producer_abort)) return;
            if (end) {
                if (lane == 0) {
                    sm.meta[s].chain = -1;
                    mbar_arrive(smem_u32(&sm.full[s]));
                }
                return;
            }
            const int pg = chain % k.npg, b = chain / k.npg;
            const int c = kBwd ? k.ntiles - 1 - j : j;
            const int t0 = c * k.R;
            if (k.done) {
                const int len = min(k.R, k.T - t0);
                const uint8_t* dn = k.done + (size_t)b * k.T + t0;
                for (int i = lane; i < k.R; i += 32) sm.flags[s][i] = (i < len && dn[i] != 0) ? 1 : 0;
                __syncwarp();
            }
            if (lane == 0) {
                sm.meta[s].chain = chain;
                sm.meta[s].tile = j;
                const uint32_t bar = smem_u32(&sm.full[s]);
                const uint32_t dst = smem_u32(stages + (size_t)s * stage_bytes);
                const int c0 = pg * 2 * k.G;
                mbar_expect_tx(bar, bytes0 + bytes1 + bytes2);
                tma_load_3d(dst, m0, bar, c0, t0, b);
                if (bytes1) tma_load_3d(dst + bytes0, m1, bar, c0, t0 - 1, b);
                if (bytes2) tma_load_3d(dst + bytes0 + bytes1, m2, bar, c0, t0 - 1, b);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Forward:  x_t = keep_t Abar x_{t-1} + Bu_t
// ---------------------------------------------------------------------------------------------
// The first group of a tile knows its entering state already (it left the previous tile), so
// it folds once, from that state, and publishes its final state with multiplier 0; only the
// other groups fold twice.  Rows are processed without per-row tests when the thread's rows
// are all present and carry no flag (`plain`).
template <int G, typename XS, bool kPair>
__global__ void __launch_bounds__(kThreads, 2)
scan_fwd_stream_kernel(Args k, const __grid_constant__ CUtensorMap tm_in, const __grid_constant__ CUtensorMap tm_o0,
                       const __grid_constant__ CUtensorMap tm_o1, const float2* __restrict__ x0,
                       float2* __restrict__ xT) {
    constexpr int r = kFwdRows, slices = kConsumers / G, R = slices * r;
    constexpr uint32_t stage_bytes = (uint32_t)R * G * 8;
    extern __shared__ uint8_t stream_raw[];
    __shared__ Shared sm;
    uint8_t* stages = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(stream_raw) + 127) & ~(uintptr_t)127);
    const int tid = threadIdx.x;
    init_shared(sm);
    if (tid >= kConsumers) {
        producer<false>(k, sm, stages, stage_bytes, &tm_in, nullptr, nullptr, stage_bytes, 0, 0);
        return;
    }
    const int col = tid % G, sl = tid / G, row0 = sl * r;
    const float2 zero2 = make_float2(0.f, 0.f);
    float2 a = zero2, al = zero2, aR = zero2, aRl = zero2, xin = zero2;
    int s = 0, round = 0, s_prev = 0;
    for (int n = 0;; ++n, s_prev = s, s = (s + 1 == k.stages) ? 0 : s + 1, round += (s == 0)) {
        if (!mbar_wait(smem_u32(&sm.full[s]), round & 1, &sm.abort_flag)) k.hdr->status = SSM_ERR_TIMEOUT;
        consumer_sync();   // the scanning warps leave together or not at all
        if (sm.abort_flag) break;
        const int chain = sm.meta[s].chain;
        if (chain < 0) break;
        const int j = sm.meta[s].tile;
        const int pg = chain % k.npg, b = chain / k.npg;
        const int p = pg * G + col;
        const bool active = p < k.P;
        const int t0 = j * R;
        const int len = min(R, k.T - t0);
        if (j == 0) {
            a = active ? k.Abar[p] : zero2;
            al = (kPair && active) ? k.Alo[p] : zero2;
            cpow2_pair<r>(a, al, aR, aRl);
            xin = (x0 && active) ? x0[(size_t)b * k.P + p] : zero2;
        }
        uint8_t* stage = stages + (size_t)s * stage_bytes;
        const int valid = max(0, min(r, len - row0));
        uint32_t mask = 0u;
        if (k.done) {
#pragma unroll
            for (int i = 0; i < r; ++i) mask |= (uint32_t)sm.flags[s][row0 + i] << i;
        }
        const bool plain = valid == r && mask == 0u;
        float2 v[r];
        const float2* in = reinterpret_cast<const float2*>(stage) + row0 * G + col;
#pragma unroll
        for (int i = 0; i < r; ++i) v[i] = in[i * G];
        float2 e, m = aR, ml = aRl;
        if (sl == 0) {
            // the true pass at once; v becomes the results
            float2 st = (j == 0) ? xin : sm.carry[n & 1][col];
            if (plain) {
#pragma unroll
                for (int i = 0; i < r; ++i) v[i] = st = rstep<kPair>(a, al, st, v[i]);
            } else {
#pragma unroll
                for (int i = 0; i < r; ++i)
                    if (i < valid) {
                        if ((mask >> i) & 1u) st = zero2;
                        v[i] = st = rstep<kPair>(a, al, st, v[i]);
                    }
            }
            e = st;
            m = zero2;
            ml = zero2;
        } else if (plain) {
            e = v[0];
#pragma unroll
            for (int i = 1; i < r; ++i) e = rstep<kPair>(a, al, e, v[i]);
        } else {
            e = zero2;
#pragma unroll
            for (int i = 0; i < r; ++i)
                if (i < valid) {
                    if ((mask >> i) & 1u) e = zero2;
                    e = rstep<kPair>(a, al, e, v[i]);
                }
            if (mask != 0u) {
                m = zero2;
                ml = zero2;
            } else {
                cpow_n_pair(a, al, valid, m, ml);
            }
        }
        sm.agg_e[tid] = e;
        sm.agg_m[tid] = m;
        sm.agg_ml[tid] = ml;
        if (tid == 0 && n > 0) {   // the store of the previous tile has read its stage by now: recycle it
            tma_store_wait_read_n<0>();
            mbar_arrive(smem_u32(&sm.empty[s_prev]));
        }
        consumer_sync();   // pairs visible; every thread has its rows in registers
        float2 st = e;
        if (sl == 0) {
#pragma unroll
            for (int i = 0; i < r; ++i)
                if (i < valid) TileIO<XS>::put(stage, R, G, row0 + i, col, v[i]);
        } else {
            st = sm.agg_e[col];   // group 0 left its final state
            for (int q = 1; q < sl; ++q) {
                const int o = q * G + col;
                // the group multiplier Abar^r always as an fp32 pair: its rounding error is the same at every
                // join of a chain, so with a single fp32 it grows linearly with the sequence length
                st = cfma2(sm.agg_m[o], sm.agg_ml[o], st, sm.agg_e[o]);
            }
            if (plain) {
#pragma unroll
                for (int i = 0; i < r; ++i) {
                    st = rstep<kPair>(a, al, st, v[i]);
                    TileIO<XS>::put(stage, R, G, row0 + i, col, st);
                }
            } else {
#pragma unroll
                for (int i = 0; i < r; ++i)
                    if (i < valid) {
                        if ((mask >> i) & 1u) st = zero2;
                        st = rstep<kPair>(a, al, st, v[i]);
                        TileIO<XS>::put(stage, R, G, row0 + i, col, st);
                    }
            }
        }
        if (sl == slices - 1) sm.carry[(n + 1) & 1][col] = st;
        if (xT && active && j == k.ntiles - 1 && valid > 0 && row0 + valid == len) xT[(size_t)b * k.P + p] = st;
        fence_async_smem();
        consumer_sync();
        if (tid == 0) {
            const uint32_t src = smem_u32(stage);
            tma_store_3d_nocommit(&tm_o0, src, pg * 2 * G, t0, b);
            if (sizeof(XS) == 4) tma_store_3d_nocommit(&tm_o1, src + stage_bytes / 2, pg * 2 * G, t0, b);
            tma_commit_group();
        }
    }
    if (tid == 0) tma_store_wait_all();
}

// ---------------------------------------------------------------------------------------------
// Backward:  s_t = gx_t + c_t,  c_{t-1} = keep_t conj(Abar) s_t  (c_{T-1} = gxT);
//            gAbar partial = sum_t keep_t s_t conj(x_{t-1}).
// Stage = [gx tile][x tile one row earlier]; the s tile overwrites the gx tile.  Tiles, groups
// and rows are all taken from the end, and it is the last group that passes only once.
// gA_part: one row of P sums per sequence, each entry written once (so the sum over rows that
// follows does not depend on which CTA ran what).
// ---------------------------------------------------------------------------------------------
template <int G, typename XS, bool kPair, int kRowsPerThread>
__global__ void __launch_bounds__(kThreads, 2)
scan_bwd_stream_kernel(Args k, const __grid_constant__ CUtensorMap tm_g, const __grid_constant__ CUtensorMap tm_x0,
                       const __grid_constant__ CUtensorMap tm_x1, const __grid_constant__ CUtensorMap tm_o0,
                       const __grid_constant__ CUtensorMap tm_o1, const float2* __restrict__ x0,
                       const float2* __restrict__ gxT, float2* __restrict__ gA_part, float2* __restrict__ gx0) {
    constexpr int r = kRowsPerThread, slices = kConsumers / G, R = slices * r;
    constexpr uint32_t tile_bytes = (uint32_t)R * G * 8, stage_bytes = 2 * tile_bytes;
    extern __shared__ uint8_t stream_raw[];
    __shared__ Shared sm;
    uint8_t* stages = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(stream_raw) + 127) & ~(uintptr_t)127);
    const int tid = threadIdx.x;
    init_shared(sm);
    if (tid >= kConsumers) {
        if (sizeof(XS) == 4)
            producer<true>(k, sm, stages, stage_bytes, &tm_g, &tm_x0, &tm_x1, tile_bytes, tile_bytes / 2, tile_bytes / 2);
        else
            producer<true>(k, sm, stages, stage_bytes, &tm_g, &tm_x0, nullptr, tile_bytes, tile_bytes, 0);
        return;
    }
    const int col = tid % G, sl = tid / G, row0 = sl * r;
    const bool first = sl == slices - 1;
    const float2 zero2 = make_float2(0.f, 0.f);
    float2 ac = zero2, acl = zero2, aR = zero2, aRl = zero2, cin = zero2, xinit = zero2, g = zero2;
    int s = 0, round = 0, s_prev = 0;
    for (int n = 0;; ++n, s_prev = s, s = (s + 1 == k.stages) ? 0 : s + 1, round += (s == 0)) {
        if (!mbar_wait(smem_u32(&sm.full[s]), round & 1, &sm.abort_flag)) k.hdr->status = SSM_ERR_TIMEOUT;
        consumer_sync();
        if (sm.abort_flag) break;
        const int chain = sm.meta[s].chain;
        if (chain < 0) break;
        const int j = sm.meta[s].tile;
        const int pg = chain % k.npg, b = chain / k.npg;
        const int p = pg * G + col;
        const bool active = p < k.P;
        const int c = k.ntiles - 1 - j;       // tile index in time
        const int t0 = c * R;
        const int len = min(R, k.T - t0);
        if (j == 0) {
            ac = active ? cconj(k.Abar[p]) : zero2;
            acl = (kPair && active) ? cconj(k.Alo[p]) : zero2;
            cpow2_pair<r>(ac, acl, aR, aRl);
            cin = (gxT && active) ? gxT[(size_t)b * k.P + p] : zero2;
            xinit = (x0 && active) ? x0[(size_t)b * k.P + p] : zero2;
            g = zero2;
        }
        uint8_t* stage = stages + (size_t)s * stage_bytes;
        const uint8_t* xtile = stage + tile_bytes;
        const int valid = max(0, min(r, len - row0));
        uint32_t mask = 0u;
        if (k.done) {
#pragma unroll
            for (int i = 0; i < r; ++i) mask |= (uint32_t)sm.flags[s][row0 + i] << i;
        }
        const bool plain = valid == r && mask == 0u && !(c == 0 && sl == 0);
        float2 v[r];
        const float2* in = reinterpret_cast<const float2*>(stage) + row0 * G + col;
#pragma unroll
        for (int i = 0; i < r; ++i) v[i] = in[i * G];
        // One true pass over this thread's rows from carry `cc` (= keep conj(Abar) s of the row after the
        // thread's last); results to `out(i, s_i)`.  Inside the thread's rows the recurrence is one fused
        // multiply-add per step, s_i = conj(Abar) s_{i+1} + gx_i (one rounding, as in the forward scan); the
        // carry form conj(Abar) s is only taken at the thread's two ends.
        auto true_pass = [&](float2 cc, auto&& out) -> float2 {
            if (plain) {
                float2 sv = cadd(v[r - 1], cc);
#pragma unroll
                for (int i = r - 1; i >= 0; --i) {
                    if (i < r - 1) sv = rstep<kPair>(ac, acl, sv, v[i]);
                    out(i, sv);
                    g = cfma(sv, cconj(TileIO<XS>::get(xtile, R, G, row0 + i, col)), g);
                }
                return rstep<kPair>(ac, acl, sv, zero2);
            }
            float2 sv = zero2;
            bool have = false, cut = false;   // have: sv is s of the row after row i; cut: that row carries a flag
#pragma unroll
            for (int i = r - 1; i >= 0; --i)
                if (i < valid) {
                    sv = !have ? cadd(v[i], cc) : (cut ? v[i] : rstep<kPair>(ac, acl, sv, v[i]));
                    have = true;
                    out(i, sv);
                    cut = (mask >> i) & 1u;
                    if (!cut) {
                        const float2 xprev =
                            (c == 0 && row0 + i == 0) ? xinit : TileIO<XS>::get(xtile, R, G, row0 + i, col);
                        g = cfma(sv, cconj(xprev), g);
                    }
                }
            if (!have) return cc;   // no row of this thread lies inside the sequence
            return cut ? zero2 : rstep<kPair>(ac, acl, sv, zero2);
        };
        float2 e, m = aR, ml = aRl;
        if (first) {
            e = true_pass((j == 0) ? cin : sm.carry[n & 1][col], [&](int i, float2 sv) { v[i] = sv; });
            m = zero2;
            ml = zero2;
        } else if (plain) {
            float2 sv = v[r - 1];
#pragma unroll
            for (int i = r - 2; i >= 0; --i) sv = rstep<kPair>(ac, acl, sv, v[i]);
            e = rstep<kPair>(ac, acl, sv, zero2);
        } else {
            float2 sv = zero2;
            bool cut = true;   // nothing enters from beyond the thread's rows in this pass
#pragma unroll
            for (int i = r - 1; i >= 0; --i)
                if (i < valid) {
                    sv = cut ? v[i] : rstep<kPair>(ac, acl, sv, v[i]);
                    cut = (mask >> i) & 1u;
                }
            e = (valid == 0 || cut) ? zero2 : rstep<kPair>(ac, acl, sv, zero2);
            if (mask != 0u) {
                m = zero2;
                ml = zero2;
            } else {
                cpow_n_pair(ac, acl, valid, m, ml);
            }
        }
        sm.agg_e[tid] = e;
        sm.agg_m[tid] = m;
        sm.agg_ml[tid] = ml;
        if (tid == 0 && n > 0) {   // the store of the previous tile has read its stage by now: recycle it
            tma_store_wait_read_n<0>();
            mbar_arrive(smem_u32(&sm.empty[s_prev]));
        }
        consumer_sync();
        float2 cc = e;
        if (first) {
#pragma unroll
            for (int i = 0; i < r; ++i)
                if (i < valid) TileIO<XS>::put(stage, R, G, row0 + i, col, v[i]);
        } else {
            cc = sm.agg_e[(slices - 1) * G + col];   // the last group left its final carry
            for (int q = slices - 2; q > sl; --q) {
                const int o = q * G + col;
                cc = cfma2(sm.agg_m[o], sm.agg_ml[o], cc, sm.agg_e[o]);   // (multiplier as an fp32 pair, as in the forward scan)
            }
            cc = true_pass(cc, [&](int i, float2 sv) { TileIO<XS>::put(stage, R, G, row0 + i, col, sv); });
        }
        if (sl == 0) sm.carry[(n + 1) & 1][col] = cc;
        const bool chain_end = j == k.ntiles - 1;
        if (chain_end) {
            if (gx0 && active && sl == 0) gx0[(size_t)b * k.P + p] = cc;
            sm.gsum[tid] = g;
            g = zero2;
        }
        fence_async_smem();
        consumer_sync();
        if (tid == 0) {
            const uint32_t src = smem_u32(stage);
            tma_store_3d_nocommit(&tm_o0, src, pg * 2 * G, t0, b);
            if (sizeof(XS) == 4) tma_store_3d_nocommit(&tm_o1, src + tile_bytes / 2, pg * 2 * G, t0, b);
            tma_commit_group();
        }
        if (chain_end && sl == 0 && active) {
            float2 sum = zero2;
#pragma unroll
            for (int q = 0; q < slices; ++q) sum = cadd(sum, sm.gsum[q * G + col]);
            gA_part[(size_t)b * k.P + p] = sum;   // every (sequence, state) belongs to exactly one chain
        }
    }
    if (tid == 0) tma_store_wait_all();
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
namespace {

int sm_count() { return device_sm_count(); }

constexpr int kCtasPerSm = 2;

// Tensor map over a [B, T, 2P] array (fp32 or bf16 elements) with boxes of 2G x R x 1.
bool make_map3(CUtensorMap* map, const void* base, bool bf16, int B, int T, int P, int G, int R) {
    PFN_cuTensorMapEncodeTiled fn = encode_fn();
    if (!fn) return false;
    const uint64_t es = bf16 ? 2 : 4;
    cuuint64_t dims[3] = {(cuuint64_t)2 * P, (cuuint64_t)T, (cuuint64_t)B};
    cuuint64_t strides[2] = {(cuuint64_t)2 * P * es, (cuuint64_t)T * 2 * P * es};
    cuuint32_t box[3] = {(cuuint32_t)2 * G, (cuuint32_t)R, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    // L2 fetch granularity no wider than a row of the box: wider would pull in neighbouring chains
    const uint64_t row_bytes = 2 * (uint64_t)G * es;
    const CUtensorMapL2promotion promo = row_bytes >= 256   ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B
                                         : row_bytes >= 128 ? CU_TENSOR_MAP_L2_PROMOTION_L2_128B
                                                            : CU_TENSOR_MAP_L2_PROMOTION_L2_64B;
    return fn(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3,
              const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_NONE, promo,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

Args make_args(int B, int T, int P, int rows, bool forward, const float2* Abar, const float2* Alo, const uint8_t* done, int* ticket,
               WsHeader* hdr) {
    Args k{};
    k.B = B;
    k.T = T;
    k.P = P;
    // Group width: the chains are dealt to kCtasPerSm * SMs resident CTAs, so the last round of
    // chains should be nearly full; tiles should not be much taller than the sequence; among the
    // widths within 5 % of the best, the widest (longest contiguous rows in memory).
    const int slots = kCtasPerSm * sm_count();
    int G = 16;
    double best = 0.0;
    for (int pass = 0; pass < 2; ++pass)
        for (int g = kMaxG; g >= 16; g /= 2) {
            if (g > P && g > 16) continue;
            const long long chains = (long long)B * ((P + g - 1) / g);
            const long long rounds = (chains + slots - 1) / slots;
            const int R = (kConsumers / g) * rows;
            const int tiles = (T + R - 1) / R;
            const double eff = (double)chains / (double)(rounds * slots) * (double)T / (double)((long long)tiles * R);
            if (pass == 0) {
                if (eff > best) best = eff;
            } else if (eff >= 0.95 * best) {
                G = g;
                pass = 2;
                break;
            }
        }
    k.G = G;
    k.g_shift = 0;
    while ((1 << k.g_shift) < G) ++k.g_shift;
    k.slices = kConsumers / G;
    k.R = k.slices * rows;
    k.ntiles = (T + k.R - 1) / k.R;
    k.npg = (P + G - 1) / G;
    k.nchains = B * k.npg;
    // Narrow chains (128-byte rows: few long sequences) keep one more tile in flight in the forward scan:
    // 4.8 -> 5.4 TB/s at 16 x 16384, P = 256; with wider chains a fourth stage costs 1 %, and the adjoint, whose
    // stages also hold x, loses 8 % with four.
    k.stages = (forward && G <= 16) ? 4 : 3;
    k.Abar = Abar;
    k.Alo = Alo;
    k.done = done;
    k.ticket = ticket;
    k.hdr = hdr;
    return k;
}

template <typename K>
bool set_smem(K kernel, size_t bytes) {
    return set_max_dynamic_smem(reinterpret_cast<const void*>(kernel), bytes);
}

}  // namespace
}  // namespace stream

bool scan_stream_supported(int B, int T, int P) {
    (void)B;
    (void)T;
    return P >= 16 && stream::encode_fn() != nullptr;
}

int launch_scan_fwd_stream(int B, int T, int P, const float2* Abar, const float2* Alo, const float2* Bu,
                           const uint8_t* done, const float2* x0, void* x, bool x_bf16, float2* xT, WsHeader* hdr,
                           int* ticket, cudaStream_t st) {
    using namespace stream;
    const Args k = make_args(B, T, P, kFwdRows, true, Abar, Alo, done, ticket, hdr);
    const size_t smem = (size_t)k.stages * k.R * k.G * 8 + 128;
    const int grid = k.nchains < kCtasPerSm * sm_count() ? k.nchains : kCtasPerSm * sm_count();
    const size_t plane_bytes = (size_t)B * T * P * 4;
    CUtensorMap mi, o0, o1;
    if (!make_map3(&mi, Bu, false, B, T, P, k.G, k.R)) return SSM_ERR_CUDA;
    if (!make_map3(&o0, x, x_bf16, B, T, P, k.G, k.R)) return SSM_ERR_CUDA;
    o1 = o0;
    if (x_bf16 && !make_map3(&o1, (const char*)x + plane_bytes, true, B, T, P, k.G, k.R)) return SSM_ERR_CUDA;
    if (cudaMemsetAsync(ticket, 0, sizeof(int), st) != cudaSuccess) return SSM_ERR_CUDA;
    count_launch();
#define SSM_LAUNCH_G(GG, XS, PAIR)                                                      \
    do {                                                                                \
        auto kern = scan_fwd_stream_kernel<GG, XS, PAIR>;                               \
        if (!set_smem(kern, smem)) return SSM_ERR_CUDA;                                 \
        kern<<<grid, kThreads, smem, st>>>(k, mi, o0, o1, x0, xT);                      \
    } while (0)
#define SSM_LAUNCH(XS, PAIR)                                                            \
    do {                                                                                \
        if (k.G == 128) SSM_LAUNCH_G(128, XS, PAIR);                                    \
        else if (k.G == 64) SSM_LAUNCH_G(64, XS, PAIR);                                 \
        else if (k.G == 32) SSM_LAUNCH_G(32, XS, PAIR);                                 \
        else SSM_LAUNCH_G(16, XS, PAIR);                                                \
    } while (0)
    if (x_bf16) {
        SSM_LAUNCH(uint32_t, false);   // bf16 storage: Abar as one fp32 is accurate enough
    } else {
        if (Alo) SSM_LAUNCH(float2, true);
        else SSM_LAUNCH(float2, false);
    }
#undef SSM_LAUNCH_G
#undef SSM_LAUNCH
    return SSM_OK;
}

int launch_scan_bwd_stream(int B, int T, int P, const float2* Abar, const float2* Alo, const uint8_t* done,
                           const float2* x0, const void* x, bool x_bf16, const float2* gx, const float2* gxT,
                           void* gBu, float2* gx0, float2* part, WsHeader* hdr, int* ticket, cudaStream_t st) {
    using namespace stream;
    const bool tall = T >= kBwdLongT;
    const Args k = make_args(B, T, P, tall ? kBwdRowsLong : kBwdRows, false, Abar, Alo, done, ticket, hdr);
    const size_t smem = (size_t)k.stages * 2 * k.R * k.G * 8 + 128;
    const int grid = k.nchains < kCtasPerSm * sm_count() ? k.nchains : kCtasPerSm * sm_count();
    const size_t plane_bytes = (size_t)B * T * P * 4;
    CUtensorMap mg, x0m, x1m, o0, o1;
    if (!make_map3(&mg, gx, false, B, T, P, k.G, k.R)) return SSM_ERR_CUDA;
    if (!make_map3(&x0m, x, x_bf16, B, T, P, k.G, k.R)) return SSM_ERR_CUDA;
    if (!make_map3(&o0, gBu, x_bf16, B, T, P, k.G, k.R)) return SSM_ERR_CUDA;
    x1m = x0m;
    o1 = o0;
    if (x_bf16) {
        if (!make_map3(&x1m, (const char*)x + plane_bytes, true, B, T, P, k.G, k.R)) return SSM_ERR_CUDA;
        if (!make_map3(&o1, (const char*)gBu + plane_bytes, true, B, T, P, k.G, k.R)) return SSM_ERR_CUDA;
    }
    if (cudaMemsetAsync(ticket, 0, sizeof(int), st) != cudaSuccess) return SSM_ERR_CUDA;
    count_launch();
#define SSM_LAUNCH_G(GG, XS, PAIR)                                                                 \
    do {                                                                                           \
        if (tall) {                                                                                \
            auto kern = scan_bwd_stream_kernel<GG, XS, PAIR, kBwdRowsLong>;                        \
            if (!set_smem(kern, smem)) return SSM_ERR_CUDA;                                        \
            kern<<<grid, kThreads, smem, st>>>(k, mg, x0m, x1m, o0, o1, x0, gxT, part, gx0);       \
        } else {                                                                                   \
            auto kern = scan_bwd_stream_kernel<GG, XS, PAIR, kBwdRows>;                            \
            if (!set_smem(kern, smem)) return SSM_ERR_CUDA;                                        \
            kern<<<grid, kThreads, smem, st>>>(k, mg, x0m, x1m, o0, o1, x0, gxT, part, gx0);       \
        }                                                                                          \
    } while (0)
#define SSM_LAUNCH(XS, PAIR)                                                                       \
    do {                                                                                           \
        if (k.G == 128) SSM_LAUNCH_G(128, XS, PAIR);                                               \
        else if (k.G == 64) SSM_LAUNCH_G(64, XS, PAIR);                                            \
        else if (k.G == 32) SSM_LAUNCH_G(32, XS, PAIR);                                            \
        else SSM_LAUNCH_G(16, XS, PAIR);                                                           \
    } while (0)
    if (x_bf16) {
        SSM_LAUNCH(uint32_t, false);   // bf16 storage: Abar as one fp32 is accurate enough
    } else {
        if (Alo) SSM_LAUNCH(float2, true);
        else SSM_LAUNCH(float2, false);
    }
#undef SSM_LAUNCH_G
#undef SSM_LAUNCH
    return SSM_OK;
}

}  // namespace ssm
