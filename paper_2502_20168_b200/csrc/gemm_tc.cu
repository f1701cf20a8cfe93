#include <type_traits>
// bf16 projections on the 5th-generation tensor cores (tcgen05.mma, accumulators in tensor
// memory, operands staged in shared memory by TMA).  The kernels:
//
//  * gemm_tc_tn_kernel / gemm_tc_tn_pair_kernel: out[m, n] = sum_k A[m, k] * W[n, k]  (both operands
//    K-contiguous).  Persistent; one CTA per SM walking 128 x 256 accumulator tiles, or clusters of two
//    CTAs on 256 x 256 tiles.  A = activations or states [B*T, K]; W = packed parameters.  With kSplitW
//    the 256 accumulator columns of a tile hold the products with the high and the low bf16 halves of 128
//    weight rows, summed in the epilogue (weights then carry ~16 mantissa bits; see
//    discretize_pack_tc_kernel).  With a product schedule the accumulator sums several products of bf16
//    planes of both operands (fp32-accurate results, see planes.cu).  Epilogues: fp32 store; bf16
//    acc + diag * skip; the same with column sums of skip * dot; fp32 store with a gated bf16 result.
//  * gemm_scan_fwd_kernel / gemm_scan_bwd_kernel: the pair kernel with the scan of Sec. III-B (and its
//    adjoint) in the epilogue, so that Bu and g_x never reach memory.  The CTAs of a pair take two
//    sequences, or (kTPair) alternate tiles of one.
//  * gemm_tc_nt_kernel / gemm_tc_nt_pair_kernel: part[s, i, j] = sum_{m in slice s} A[m, i] * Bm[m, j]
//    (both operands contiguous in the output index, i.e. MN-major), split over the B*T rows: the weight
//    gradients.
//
// Warp roles in all: warp 0 issues TMA loads, warp 1 owns tensor memory and issues the MMAs, the other
// warps drain accumulators (each may read one TMEM lane quarter).  Every mbarrier wait is bounded; a wait
// that gives up raises a CTA-wide abort flag, the status word of the workspace header is set, tensor
// memory is released and the kernel returns.
#include <map>
#include <mutex>
#include <utility>

#include "kernels.h"
#include "tma.cuh"

namespace ssm {
namespace tc {
using namespace tma;

constexpr int BM = 128;   // accumulator rows per tile = TMEM lanes
constexpr int BN = 256;   // accumulator columns per tile
constexpr int BK = 64;    // bf16 elements per shared-memory row: 128 bytes, one swizzle span
constexpr int UK = 16;    // K extent of one tcgen05.mma of kind::f16
constexpr int kStages = 4;      // shared-memory stages of the NT kernel (and size of the barrier arrays)
constexpr int kTnStages = 3;    // the TN kernel gives one stage up for its epilogue buffers
constexpr int kABytes = BM * BK * 2;
constexpr int kBBytes = BN * BK * 2;
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kThreads = 192;      // NT kernel: producer, MMA, 4 epilogue warps
constexpr int kTnEpiWarps = 8;     // TN kernel: two epilogue warps per TMEM lane quarter
constexpr int kTnThreads = 64 + 32 * kTnEpiWarps;
constexpr int kTmemCols = 512;  // two accumulator buffers of BN columns
constexpr int kStagingBytes = kTnEpiWarps * 32 * 32 * 4;  // per epilogue warp: 32 rows x 32 fp32 columns
constexpr int kMaxDiag = 4096;                  // widest output whose diagonal fits the shared copy
constexpr int kSkipBytes = kTnEpiWarps * 2 * 32 * 32 * 2;   // two 32 x 32 bf16 skip tiles per epilogue warp
// Epilogues of the TN kernels: 0 = fp32 result; 1 = bf16(acc + diag * skip); 2 = fp32 result AND
// a gated bf16 result skip * sigmoid(acc) (needs a staging buffer for each); 3 = epilogue 1 AND the
// column sums of skip * dot over the rows this CTA drains (a second operand tile beside every skip
// tile, per-warp sums in shared memory): CTA pairs only, outputs of at most kDotMaxN columns.
constexpr int kDotMaxN = 1024;
__host__ __device__ constexpr int tn_skip_bytes(int epi) { return epi == 0 ? 0 : (epi == 3 ? 2 * kSkipBytes : kSkipBytes); }
__host__ __device__ constexpr int tn_diag_bytes(int epi) {
    return epi == 1 ? kMaxDiag * 4 : (epi == 3 ? kDotMaxN * 4 + kTnEpiWarps * (kDotMaxN / 2) * 4 : 0);
}
__host__ __device__ constexpr int tn_staging_bytes(int epi) { return epi == 2 ? kStagingBytes + kStagingBytes / 2 : kStagingBytes; }
constexpr size_t tn_smem_bytes(int epi) {
    return (size_t)kTnStages * kStageBytes + tn_staging_bytes(epi) + tn_skip_bytes(epi) + tn_diag_bytes(epi) +
           1024 /*alignment slack*/ + 256 /*barriers*/;
}
constexpr size_t kNtSmemBytes = (size_t)kStages * kStageBytes + 1024 + 256;

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrives on the mbarrier once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// ---- CTA pairs (cta_group::2): one MMA spans the tensor cores and tensor memory of two CTAs
// of a cluster; each CTA holds its 128 rows of A and its half of the B rows in shared memory at
// the same offsets.  Allocation and release of tensor memory are issued by one warp of each CTA.
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// For data handed from one CTA of the cluster to the other through shared memory: the sender stores into the
// peer's memory and arrives (release, cluster scope) on the peer's barrier, the receiver waits with acquire.
__device__ __forceinline__ void mbar_arrive_release_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_acquire_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_acquire_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try_wait_acquire_cluster(bar, parity)) return true;
        if ((i & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void st_cluster_f4(uint32_t cluster_addr, float4 v) {
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
                 : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// Asks L2 to fetch a contiguous range (a multiple of 16 bytes from a 16-byte aligned address).
__device__ __forceinline__ void l2_prefetch_bulk(const void* ptr, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(ptr), "r"(bytes) : "memory");
}
// Tile load whose completion is counted on a barrier of either CTA of the pair (cluster address).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrives on the barrier at this offset in both CTAs once every MMA issued so far has completed.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}

// 32 lanes x 32 consecutive 32-bit columns: thread i of the warp gets lane (base lane + i).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptors (128-byte swizzle).  Fields: start address >> 4 in bits
// [0,14), leading byte offset >> 4 in [16,30), stride byte offset >> 4 in [32,46), descriptor
// version 1 in [46,48), swizzle mode 2 (128 B) in [61,64).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// K-major tile: rows of 128 bytes, groups of 8 rows 1024 bytes apart (leading offset unused).
__device__ __forceinline__ uint64_t smem_desc_kmajor(uint32_t addr) { return smem_desc(addr, 16, 1024); }
// MN-major tile made of [BK rows][64 elements] blocks: 64-element blocks 8192 bytes apart,
// groups of 8 k-rows 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_mnmajor(uint32_t addr) { return smem_desc(addr, BK * 128, 1024); }

// Instruction descriptor: D = f32 (bits [4,6) = 1), A = B = bf16 (bits [7,10), [10,13) = 1),
// operand majors in bits 15 / 16 (0 = K), N >> 3 in [17,23), M >> 4 in [24,29).
__host__ __device__ constexpr uint32_t instr_desc(int m, int n, int a_mn, int b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
           ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

struct Smem {
    uint8_t* tiles;       // 1024-byte aligned
    uint8_t* staging;     // epilogue transpose buffers
    float* diag;          // copy of the epilogue's diagonal
    uint8_t* skipbuf;     // bf16 epilogue: per epilogue warp two 32 x 32 bf16 tiles of the skip operand
    // mbarriers of a kind sit 8 bytes apart: their addresses are computed, so that no array is indexed at
    // run time (that would put this struct into local memory)
    uint32_t full0, empty0, tmem_full0, tmem_empty0, skip_full0;
    __device__ __forceinline__ uint32_t full(int i) const { return full0 + 8u * (uint32_t)i; }
    __device__ __forceinline__ uint32_t empty(int i) const { return empty0 + 8u * (uint32_t)i; }
    __device__ __forceinline__ uint32_t tmem_full(int i) const { return tmem_full0 + 8u * (uint32_t)i; }
    __device__ __forceinline__ uint32_t tmem_empty(int i) const { return tmem_empty0 + 8u * (uint32_t)i; }
    __device__ __forceinline__ uint32_t skip_full(int i) const { return skip_full0 + 8u * (uint32_t)i; }
    uint32_t tmem_slot;   // where tcgen05.alloc writes the base address
    volatile int* abort_flag;
    volatile uint32_t* tmem_slot_ptr;
};

// Layout: [stages][epilogue staging][skip tiles][diag copy][barriers]; the NT kernel has none of the
// epilogue buffers.
__device__ __forceinline__ Smem carve_smem(uint8_t* raw, int stages, int staging_bytes, int diag_bytes,
                                           int stage_bytes = kStageBytes, int skip_bytes = 0) {
    Smem s;
    uintptr_t base = (reinterpret_cast<uintptr_t>(raw) + 1023) & ~(uintptr_t)1023;
    s.tiles = reinterpret_cast<uint8_t*>(base);
    s.staging = s.tiles + (size_t)stages * stage_bytes;
    s.skipbuf = s.staging + staging_bytes;
    s.diag = reinterpret_cast<float*>(s.skipbuf + skip_bytes);
    uint8_t* bars = s.skipbuf + skip_bytes + diag_bytes;
    s.full0 = smem_u32(bars);
    s.empty0 = smem_u32(bars + 8 * kStages);
    s.tmem_full0 = smem_u32(bars + 8 * (2 * kStages));
    s.tmem_empty0 = smem_u32(bars + 8 * (2 * kStages + 2));
    s.tmem_slot_ptr = reinterpret_cast<volatile uint32_t*>(bars + 8 * (2 * kStages + 4));
    s.tmem_slot = smem_u32(bars + 8 * (2 * kStages + 4));
    s.abort_flag = reinterpret_cast<volatile int*>(bars + 8 * (2 * kStages + 4) + 4);
    s.skip_full0 = smem_u32(bars + 8 * (2 * kStages + 5));
    return s;
}

// Common prologue: barriers, tensor memory.  Returns the TMEM base address.
__device__ __forceinline__ uint32_t prologue(const Smem& s, int warp, int lane, int epilogue_threads) {
    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(s.full(i), 1);
            mbar_init(s.empty(i), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(s.tmem_full(i), 1);
            mbar_init(s.tmem_empty(i), epilogue_threads);
        }
        for (int i = 0; i < 2 * kTnEpiWarps; ++i) mbar_init(s.skip_full(i), 1);
        *s.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(s.tmem_slot, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    (void)lane;
    return *s.tmem_slot_ptr;
}

__device__ __forceinline__ void epilogue_exit(const Smem& s, int warp, uint32_t tmem_base, WsHeader* hdr) {
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0 && *s.abort_flag && hdr) hdr->status = SSM_ERR_TIMEOUT;
}

// ---------------------------------------------------------------------------------------------
// TN kernel
// ---------------------------------------------------------------------------------------------
struct TnParams {
    int M;            // rows of A / out
    int n_tiles;      // accumulator tiles along N (each BN columns of W rows)
    int k_blocks;     // K / BK
    int ldo;          // leading dimension of out (and skip): the number of output columns
    const float* diag;
    WsHeader* hdr;
    const char* a_base;   // A as bytes; rows are K * 2 bytes apart and contiguous
    int a_row_bytes;
    float* dot_part;      // epilogue 3: [CTAs, ldo] column sums of skip * dot, one row per CTA
    // Sum of several products in one accumulator (operands split into bf16 planes laid side by side along K:
    // plane a of A in columns [a Kp, (a + 1) Kp), likewise W): k-block kb belongs to product kb / kpp, which
    // takes plane (pa >> 4 j) & 15 of A and plane (pb >> 4 j) & 15 of W.  kpp = 0: one product, planes 0.
    int kpp;              // k-blocks per product (Kp / BK)
    uint32_t pa, pb;
    __device__ __forceinline__ int a_col(int kb) const {
        if (kpp == 0) return kb * BK;
        const int j = kb / kpp;
        return (int)((pa >> (4 * j)) & 15u) * kpp * BK + (kb - j * kpp) * BK;
    }
    __device__ __forceinline__ int w_col(int kb) const {
        if (kpp == 0) return kb * BK;
        const int j = kb / kpp;
        return (int)((pb >> (4 * j)) & 15u) * kpp * BK + (kb - j * kpp) * BK;
    }
};

// One epilogue warp's share of a finished accumulator tile: rows m0 + 32 (warp % 4) .. + 31, one half
// of the tile's output columns (from n_out0), in slabs of 32 columns; a lane holds one row of a slab.
// Waits for the tile's MMAs; false when aborting.
//  kEpi 0: fp32 results.  The slab goes through a 128-byte-swizzled staging buffer and leaves as
//          one TMA store of a 32 x 32 box (rows past M are clipped by the unit).
//  kEpi 1: out = bf16(acc + diag[n] * skip[m, n]).  The skip slab arrives by TMA (two buffers per
//          warp, fetched two slabs ahead, the first ones while the tile's MMAs still run) and the
//          bf16 slab leaves by TMA, both as 32 x 32 boxes with the 64-byte swizzle, so a lane reads
//          and writes its own 64-byte row without bank conflicts and nothing passes through the
//          load/store path to global memory.  `skip_phase`: the warp's barrier parities (bit b).
//          With next_m0 >= 0 (the tile this warp drains next) a buffer that has been read is refilled with the next
//          tile's first slabs, so that they have arrived when that tile starts; *skip_ahead says whether the
//          tile now starting found its first slabs requested already.
template <int kEpi, bool kSplitW>
__device__ __forceinline__ bool tn_drain_tile(const Smem& s, const TnParams& p, const CUtensorMap* tmOut,
                                              const CUtensorMap* tmSkip, const CUtensorMap* tmGate, int warp, int lane,
                                              int m0, int n_out0, int acc, uint32_t acc_phase, uint32_t tmem_base,
                                              uint32_t& skip_phase, int next_m0 = -1, int next_n_out0 = 0,
                                              bool* skip_ahead = nullptr) {
    constexpr int kOutCols = kSplitW ? BN / 2 : BN;
    const int q = warp & 3;             // TMEM lane quarter this warp may read
    const int half = (warp - 2) >> 2;   // which half of the tile's columns this warp drains
    const int row0 = m0 + q * 32;       // first of this warp's 32 rows
    constexpr int kSlabs = kOutCols / 32 / 2;
    const int slab0 = half * kSlabs;    // this warp's slabs: slab0 .. slab0 + kSlabs - 1
    const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BN);
    uint8_t* stg_bytes = s.staging + (size_t)(warp - 2) * (tn_staging_bytes(kEpi) / kTnEpiWarps);

    if (kEpi == 0) {
        if (!mbar_wait(s.tmem_full(acc), acc_phase, s.abort_flag)) return false;
        tc_fence_after();
        float4* stg = reinterpret_cast<float4*>(stg_bytes);
#pragma unroll
        for (int sl = 0; sl < kSlabs; ++sl) {
            const int c = (slab0 + sl) * 32;
            uint32_t r[32], r2[32];
            tmem_ld32(t_row + (uint32_t)c, r);
            if (kSplitW) tmem_ld32(t_row + (uint32_t)(BN / 2 + c), r2);
            tmem_ld_wait();
            if (lane == 0) tma_store_wait_read();   // the previous slab has left the staging buffer
            __syncwarp();
            // 16-byte chunk j of row `lane` sits at chunk j ^ (lane & 7): the 128-byte swizzle
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                float4 v = make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                                       __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
                if (kSplitW) {
                    v.x += __uint_as_float(r2[4 * j]);
                    v.y += __uint_as_float(r2[4 * j + 1]);
                    v.z += __uint_as_float(r2[4 * j + 2]);
                    v.w += __uint_as_float(r2[4 * j + 3]);
                }
                stg[lane * 8 + (j ^ (lane & 7))] = v;
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0 && row0 < p.M && n_out0 + c < p.ldo) tma_store_2d(tmOut, smem_u32(stg), n_out0 + c, row0);
        }
        return true;
    }

    // ---- kEpi == 1, 2, 3: the skip operand arrives by TMA (kEpi 3: and the dot operand beside it)
    constexpr bool kDot = kEpi == 3;
    const int w = warp - 2;
    uint8_t* skb = s.skipbuf + (size_t)w * (kDot ? 8192 : 4096);   // two 2 KB skip tiles (then two dot tiles)
    const uint32_t sbar[2] = {s.skip_full(2 * w), s.skip_full(2 * w + 1)};
    const int swz = (lane >> 1) & 3;               // 64-byte swizzle: chunk c of row `lane` sits at chunk c ^ swz
    auto fetch_skip_at = [&](int sl, int n_first, int row_first) {
        const int b = sl & 1;
        mbar_expect_tx(sbar[b], kDot ? 4096 : 2048);
        tma_load_2d(smem_u32(skb + b * 2048), tmSkip, sbar[b], n_first + (slab0 + sl) * 32, row_first);
        if (kDot) tma_load_2d(smem_u32(skb + 4096 + b * 2048), tmGate, sbar[b], n_first + (slab0 + sl) * 32, row_first);
    };
    auto fetch_skip = [&](int sl) { fetch_skip_at(sl, n_out0, row0); };
    static_assert(kSlabs % 2 == 0, "slab s of the next tile takes the buffer of slab s of this one");
    const bool ahead = skip_ahead && *skip_ahead;   // this tile's first two slabs were requested while the last one was drained
    const bool prefetch_next = kEpi != 2 && skip_ahead && next_m0 >= 0;
    if (skip_ahead) *skip_ahead = prefetch_next;
    if (lane == 0 && !ahead) {
        fence_async_smem();   // (the lanes' reads of the previous tile's last slabs: fenced and joined there)
        fetch_skip(0);
        if (kSlabs > 1) fetch_skip(1);
    }
    if (!mbar_wait(s.tmem_full(acc), acc_phase, s.abort_flag)) return false;
    tc_fence_after();
    if (kEpi == 2) {
        // z = acc (hi + lo columns) goes out in fp32, skip * sigmoid(z) in bf16; one staging buffer each
        float4* stg = reinterpret_cast<float4*>(stg_bytes);
        uint8_t* ob = stg_bytes + 4096;
#pragma unroll
        for (int sl = 0; sl < kSlabs; ++sl) {
            const int c = (slab0 + sl) * 32, b = sl & 1;
            uint32_t r[32], r2[32];
            tmem_ld32(t_row + (uint32_t)c, r);
            tmem_ld32(t_row + (uint32_t)(BN / 2 + c), r2);
            if (!mbar_wait(sbar[b], (skip_phase >> b) & 1u, s.abort_flag)) return false;
            skip_phase ^= 1u << b;
            uint4 sk[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) sk[j] = *reinterpret_cast<const uint4*>(skb + b * 2048 + lane * 64 + ((j ^ swz) << 4));
            tmem_ld_wait();
            // The refill below is a write of the async proxy over what these lanes have just read through the
            // generic proxy: without the proxy fences it can land before a lane's read has been served.
            fence_async_smem();
            __syncwarp();
            if (lane == 0 && sl + 2 < kSlabs) {
                fence_async_smem();
                fetch_skip(sl + 2);
            }
            if (lane == 0) tma_store_wait_read();   // the previous slab has left both staging buffers
            __syncwarp();
            uint4 o[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const __nv_bfloat162* s2 = reinterpret_cast<const __nv_bfloat162*>(&sk[j]);
                __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&o[j]);
                float z[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) z[e] = __uint_as_float(r[8 * j + e]) + __uint_as_float(r2[8 * j + e]);
                stg[lane * 8 + ((2 * j) ^ (lane & 7))] = make_float4(z[0], z[1], z[2], z[3]);
                stg[lane * 8 + ((2 * j + 1) ^ (lane & 7))] = make_float4(z[4], z[5], z[6], z[7]);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 sf = __bfloat1622float2(s2[e]);
                    o2[e] = __floats2bfloat162_rn(sf.x / (1.f + __expf(-z[2 * e])), sf.y / (1.f + __expf(-z[2 * e + 1])));
                }
                *reinterpret_cast<uint4*>(ob + lane * 64 + ((j ^ swz) << 4)) = o[j];
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0 && row0 < p.M && n_out0 + c < p.ldo) {
                tma_store_2d(tmOut, smem_u32(stg), n_out0 + c, row0);
                tma_store_2d(tmGate, smem_u32(ob), n_out0 + c, row0);
            }
        }
        return true;
    }
#pragma unroll
    for (int sl = 0; sl < kSlabs; ++sl) {
        const int c = (slab0 + sl) * 32, b = sl & 1;
        uint32_t r[32];
        tmem_ld32(t_row + (uint32_t)c, r);
        if (!mbar_wait(sbar[b], (skip_phase >> b) & 1u, s.abort_flag)) return false;
        skip_phase ^= 1u << b;
        uint4 sk[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) sk[j] = *reinterpret_cast<const uint4*>(skb + b * 2048 + lane * 64 + ((j ^ swz) << 4));
        float prod[kDot ? 32 : 1];
        if (kDot) {   // skip * dot for this lane's row of the slab
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint4 dt = *reinterpret_cast<const uint4*>(skb + 4096 + b * 2048 + lane * 64 + ((j ^ swz) << 4));
                const __nv_bfloat162* s2 = reinterpret_cast<const __nv_bfloat162*>(&sk[j]);
                const __nv_bfloat162* d2 = reinterpret_cast<const __nv_bfloat162*>(&dt);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 a = __bfloat1622float2(s2[e]), c2 = __bfloat1622float2(d2[e]);
                    prod[8 * j + 2 * e] = a.x * c2.x;
                    prod[8 * j + 2 * e + 1] = a.y * c2.y;
                }
            }
        }
        tmem_ld_wait();
        // Every lane has asked for its skip row; the buffer takes the slab after next.  That refill is a
        // write of the async proxy over data just read through the generic proxy: the proxy fences order the
        // two (without them the refill was seen to land before a lane's read had been served, when another
        // kernel shared the SMs and the skip rows came from L2).
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
            if (sl + 2 < kSlabs) {
                fence_async_smem();
                fetch_skip(sl + 2);
            } else if (prefetch_next) {   // the next tile's slab sl + 2 - kSlabs (0 or 1) into the buffer just read
                fence_async_smem();
                fetch_skip_at(sl + 2 - kSlabs, next_n_out0, next_m0 + q * 32);
            }
        }
        uint4 o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float4 d0 = *reinterpret_cast<const float4*>(s.diag + n_out0 + c + 8 * j);
            const float4 d1 = *reinterpret_cast<const float4*>(s.diag + n_out0 + c + 8 * j + 4);
            const float dd[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
            const __nv_bfloat162* s2 = reinterpret_cast<const __nv_bfloat162*>(&sk[j]);
            __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&o[j]);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 sf = __bfloat1622float2(s2[e]);
                o2[e] = __floats2bfloat162_rn(fmaf(dd[2 * e], sf.x, __uint_as_float(r[8 * j + 2 * e])),
                                              fmaf(dd[2 * e + 1], sf.y, __uint_as_float(r[8 * j + 2 * e + 1])));
            }
        }
        uint8_t* ob = stg_bytes + b * 2048;
        if (lane == 0) tma_store_wait_read_n<1>();   // the store from this buffer two slabs ago has read it
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 4; ++j) *reinterpret_cast<uint4*>(ob + lane * 64 + ((j ^ swz) << 4)) = o[j];
        fence_async_smem();
        __syncwarp();
        if (lane == 0 && row0 < p.M && n_out0 + c < p.ldo) tma_store_2d(tmOut, smem_u32(ob), n_out0 + c, row0);
        if (kDot) {
            // Column sums over the warp's 32 rows: at every halving step a lane keeps the half of its values
            // that its lane bit selects and adds the other lane's; lane l ends with the sum of column l.
#pragma unroll
            for (int h = 16; h >= 1; h >>= 1) {
                const bool upper = (lane & h) != 0;
#pragma unroll
                for (int j = 0; j < h; ++j) {
                    const float send = upper ? prod[j] : prod[j + h];
                    const float keep = upper ? prod[j + h] : prod[j];
                    prod[j] = keep + __shfl_xor_sync(0xffffffffu, send, h);
                }
            }
            // this warp's own sums (it always drains the same half of a tile's columns): rows outside M were
            // read as zero
            float* acc_col = s.diag + kDotMaxN + (size_t)w * (kDotMaxN / 2) + (n_out0 / BN) * (BN / 2) + sl * 32 + lane;
            *acc_col += prod[0];
        }
    }
    return true;
}

// kEpi 0: store fp32;  kEpi 1: out = bf16(acc + diag[n] * skip[m, n]).
// kSplitW: columns [0,128) and [128,256) of the accumulator tile are the hi and lo weight
// halves of the same 128 output columns.
template <int kEpi, bool kSplitW>
__global__ void __launch_bounds__(kTnThreads, 1)
gemm_tc_tn_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW,
                  const __grid_constant__ CUtensorMap tmOut, const __grid_constant__ CUtensorMap tmSkip,
                  const __grid_constant__ CUtensorMap tmGate, TnParams p) {
    extern __shared__ uint8_t smem_raw[];
    const Smem s = carve_smem(smem_raw, kTnStages, tn_staging_bytes(kEpi), tn_diag_bytes(kEpi), kStageBytes, tn_skip_bytes(kEpi));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (kEpi == 1)   // (zero where the last tile reaches past the output's columns)
        for (int i = threadIdx.x; i < p.n_tiles * BN; i += kTnThreads) s.diag[i] = i < p.ldo ? p.diag[i] : 0.f;
    const uint32_t tmem_base = prologue(s, warp, lane, 32 * kTnEpiWarps);
    const int m_tiles = (p.M + BM - 1) / BM;
    const int total = m_tiles * p.n_tiles;
    constexpr int kOutCols = kSplitW ? BN / 2 : BN;

    if (warp == 0) {
        if (lane == 0) {
            prefetch_tmap(&tmA);
            prefetch_tmap(&tmW);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x) {
                const int m0 = (tile / p.n_tiles) * BM, n0 = (tile % p.n_tiles) * BN;
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!(ok = mbar_wait(s.empty(stage), phase ^ 1u, s.abort_flag))) break;
                    mbar_expect_tx(s.full(stage), kStageBytes);
                    const uint32_t a_dst = smem_u32(s.tiles + (size_t)stage * kStageBytes);
                    tma_load_2d(a_dst, &tmA, s.full(stage), p.a_col(kb), m0);
                    tma_load_2d(a_dst + kABytes, &tmW, s.full(stage), p.w_col(kb), n0);
                    if (++stage == kTnStages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(BM, BN, 0, 0);
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x) {
                if (!(ok = mbar_wait(s.tmem_empty(acc), acc_phase ^ 1u, s.abort_flag))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!(ok = mbar_wait(s.full(stage), phase, s.abort_flag))) break;
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(s.tiles + (size_t)stage * kStageBytes);
                    const uint64_t adesc = smem_desc_kmajor(a_addr);
                    const uint64_t bdesc = smem_desc_kmajor(a_addr + kABytes);
#pragma unroll
                    for (int k = 0; k < BK / UK; ++k) {
                        // 16 bf16 = 32 bytes further along the 128-byte row: +2 in the address field
                        umma_bf16(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc,
                                  (uint32_t)((kb | k) != 0));
                    }
                    umma_commit(s.empty(stage));
                    if (++stage == kTnStages) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (!ok) break;
                umma_commit(s.tmem_full(acc));
                if ((acc ^= 1) == 0) acc_phase ^= 1u;
            }
        }
    } else {
        int acc = 0;
        uint32_t acc_phase = 0, skip_phase = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < total && ok; tile += gridDim.x) {
            const int m0 = (tile / p.n_tiles) * BM, n_out0 = (tile % p.n_tiles) * kOutCols;
            if (!(ok = tn_drain_tile<kEpi, kSplitW>(s, p, &tmOut, &tmSkip, &tmGate, warp, lane, m0, n_out0, acc, acc_phase, tmem_base,
                                                    skip_phase)))
                break;
            tc_fence_before();
            mbar_arrive(s.tmem_empty(acc));
            if ((acc ^= 1) == 0) acc_phase ^= 1u;
        }
        if (lane == 0) tma_store_wait_all();
    }
    epilogue_exit(s, warp, tmem_base, p.hdr);
}

// ---------------------------------------------------------------------------------------------
// TN kernel on CTA pairs
// ---------------------------------------------------------------------------------------------
// Same product, same epilogue, but a cluster of two CTAs works on a 256 x 256 accumulator tile:
// CTA r holds rows m0 + 128 r .. of A and rows n0 + 128 r .. of the W tile, so every CTA brings
// in 32 KB per k-block instead of 48 KB for the same number of tensor-core cycles (operand
// delivery into the SM, not the tensor pipe, bounds the single-CTA kernel).  The leader (CTA 0)
// issues the MMAs; its `full` barriers count the bytes of both CTAs' loads; its commits arrive
// on the `empty` / `tmem_full` barriers of both CTAs; both CTAs' epilogue warps arrive on the
// leader's `tmem_empty` barriers.
constexpr int kPairStages = 4;
constexpr int kPairStageBytes = kABytes + kBBytes / 2;
// (the epilogue with the column sums gives one operand stage up for its second operand tiles and its sums)
#ifndef SSM_PAIR_STAGES_BF16_EPILOGUE
#define SSM_PAIR_STAGES_BF16_EPILOGUE 4
#endif
__host__ __device__ constexpr int pair_stages(int epi) { return epi == 3 ? 3 : (epi == 1 ? SSM_PAIR_STAGES_BF16_EPILOGUE : kPairStages); }
constexpr size_t pair_smem_bytes(int epi) {
    return (size_t)pair_stages(epi) * kPairStageBytes + tn_staging_bytes(epi) + tn_skip_bytes(epi) + tn_diag_bytes(epi) + 1024 +
           256;
}

template <int kEpi, bool kSplitW>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kTnThreads, 1)
gemm_tc_tn_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmWh,
                       const __grid_constant__ CUtensorMap tmOut, const __grid_constant__ CUtensorMap tmSkip,
                       const __grid_constant__ CUtensorMap tmGate, TnParams p) {
    extern __shared__ uint8_t smem_raw[];
    constexpr int kSt = pair_stages(kEpi);
    const Smem s = carve_smem(smem_raw, kSt, tn_staging_bytes(kEpi), tn_diag_bytes(kEpi), kPairStageBytes,
                              tn_skip_bytes(kEpi));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    if (kEpi == 1 || kEpi == 3)   // (zero where the last tile reaches past the output's columns)
        for (int i = threadIdx.x; i < p.n_tiles * BN; i += kTnThreads) s.diag[i] = i < p.ldo ? p.diag[i] : 0.f;
    if (kEpi == 3)   // the epilogue warps' column sums start at zero
        for (int i = threadIdx.x; i < kTnEpiWarps * (kDotMaxN / 2); i += kTnThreads) s.diag[kDotMaxN + i] = 0.f;
    // barriers and tensor memory (both CTAs), then the whole pair meets
    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(s.full(i), 1);
            mbar_init(s.empty(i), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(s.tmem_full(i), 1);
            mbar_init(s.tmem_empty(i), 2 * 32 * kTnEpiWarps);
        }
        for (int i = 0; i < 2 * kTnEpiWarps; ++i) mbar_init(s.skip_full(i), 1);
        *s.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();
    if (warp == 1) tmem_alloc_pair(s.tmem_slot, kTmemCols);
    tc_fence_before();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *s.tmem_slot_ptr;

    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    const int m_pairs = (p.M + 2 * BM - 1) / (2 * BM);
    const int total = m_pairs * p.n_tiles;
    constexpr int kOutCols = kSplitW ? BN / 2 : BN;

    if (warp == 0) {
        if (lane == 0) {
            prefetch_tmap(&tmA);
            prefetch_tmap(&tmWh);
            const uint32_t leader_full0 = map_to_cta(s.full(0), 0);   // (the leader's barriers are 8 bytes apart there too)
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            // The 128 rows of A a tile needs are one contiguous range: have L2 fetch the next tile's
            // range in one piece, so that DRAM sees long bursts instead of 128-byte row pieces.
            auto prefetch_a = [&](int tile) {
                if (tile >= total) return;
                const int m0 = (tile / p.n_tiles) * (2 * BM) + (int)rank * BM;
                const int rows = min(BM, p.M - m0);
                if (rows > 0) l2_prefetch_bulk(p.a_base + (size_t)m0 * p.a_row_bytes, (uint32_t)rows * p.a_row_bytes);
                // (asking L2 for the epilogue's operand rows as well made the bf16-epilogue kernels 15 - 30 % slower)
            };
            prefetch_a(pair);
            for (int tile = pair; tile < total && ok; tile += npairs) {
                const int m0 = (tile / p.n_tiles) * (2 * BM) + (int)rank * BM;
                const int n0 = (tile % p.n_tiles) * BN + (int)rank * (BN / 2);
                prefetch_a(tile + npairs);
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!(ok = mbar_wait(s.empty(stage), phase ^ 1u, s.abort_flag))) break;
                    if (rank == 0) mbar_expect_tx(s.full(stage), 2 * kPairStageBytes);
                    const uint32_t a_dst = smem_u32(s.tiles + (size_t)stage * kPairStageBytes);
                    tma_load_2d_pair(a_dst, &tmA, leader_full0 + 8u * stage, p.a_col(kb), m0);
                    tma_load_2d_pair(a_dst + kABytes, &tmWh, leader_full0 + 8u * stage, p.w_col(kb), n0);
                    if (++stage == kSt) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = instr_desc(2 * BM, BN, 0, 0);
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int tile = pair; tile < total && ok; tile += npairs) {
                if (!(ok = mbar_wait(s.tmem_empty(acc), acc_phase ^ 1u, s.abort_flag))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                for (int kb = 0; kb < p.k_blocks; ++kb) {
                    if (!(ok = mbar_wait(s.full(stage), phase, s.abort_flag))) break;
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(s.tiles + (size_t)stage * kPairStageBytes);
                    const uint64_t adesc = smem_desc_kmajor(a_addr);
                    const uint64_t bdesc = smem_desc_kmajor(a_addr + kABytes);
#pragma unroll
                    for (int k = 0; k < BK / UK; ++k)
                        umma_bf16_pair(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc,
                                       (uint32_t)((kb | k) != 0));
                    umma_commit_pair(s.empty(stage));
                    if (++stage == kSt) {
                        stage = 0;
                        phase ^= 1u;
                    }
                }
                if (!ok) break;
                umma_commit_pair(s.tmem_full(acc));
                if ((acc ^= 1) == 0) acc_phase ^= 1u;
            }
        }
    } else {
        const uint32_t leader_empty0 = map_to_cta(s.tmem_empty(0), 0);
        int acc = 0;
        uint32_t acc_phase = 0, skip_phase = 0;
        bool ok = true;
        bool skip_ahead = false;
        for (int tile = pair; tile < total && ok; tile += npairs) {
            const int m0 = (tile / p.n_tiles) * (2 * BM) + (int)rank * BM, n_out0 = (tile % p.n_tiles) * kOutCols;
            const int nxt = tile + npairs;
            const int next_m0 = nxt < total ? (nxt / p.n_tiles) * (2 * BM) + (int)rank * BM : -1;
            if (!(ok = tn_drain_tile<kEpi, kSplitW>(s, p, &tmOut, &tmSkip, &tmGate, warp, lane, m0, n_out0, acc, acc_phase, tmem_base,
                                                    skip_phase, next_m0, nxt < total ? (nxt % p.n_tiles) * kOutCols : 0, &skip_ahead)))
                break;
            tc_fence_before();
            mbar_arrive_cluster(leader_empty0 + 8u * acc);
            if ((acc ^= 1) == 0) acc_phase ^= 1u;
        }
        if (lane == 0) tma_store_wait_all();
        if (kEpi == 3) {
            // this CTA's column sums: the four warps that drain a column half added in a fixed order, one row
            // of p.dot_part per CTA (the sum over the CTAs follows in another kernel)
            asm volatile("bar.sync 1, %0;" ::"n"(32 * kTnEpiWarps) : "memory");
            const float* sums = s.diag + kDotMaxN;
            for (int n = threadIdx.x - 64; n < p.ldo; n += 32 * kTnEpiWarps) {
                const int half = (n % BN) / (BN / 2), idx = (n / BN) * (BN / 2) + n % (BN / 2);
                float t = 0.f;
#pragma unroll
                for (int q = 0; q < 4; ++q) t += sums[(size_t)(4 * half + q) * (kDotMaxN / 2) + idx];
                p.dot_part[(size_t)blockIdx.x * p.ldo + n] = t;
            }
        }
    }
    // nobody leaves (or frees tensor memory) while the other CTA may still signal or compute
    tc_fence_before();
    __syncwarp();
    cluster_sync_all();
    tc_fence_after();
    if (warp == 1) tmem_dealloc_pair(tmem_base, kTmemCols);
    if (threadIdx.x == 0 && *s.abort_flag && p.hdr) p.hdr->status = SSM_ERR_TIMEOUT;
}

// ---------------------------------------------------------------------------------------------
// Input projection and forward scan in one kernel (CTA pairs)
// ---------------------------------------------------------------------------------------------
// x_t = keep_t Abar x_{t-1} + Bbar u_t without Bu ever reaching HBM: the accumulator tile of the
// projection (128 consecutive steps of one sequence x 64 states, weights hi + lo) is scanned by
// the epilogue and leaves as the two bf16 planes of x.  To make that possible a CTA walks the
// tiles of one (sequence, 64 states) chain in time order and keeps the state between tiles; the
// two CTAs of a pair take different sequences (the rows of an MMA need not be neighbours) and the
// same weight tile.  Epilogue per tile, 256 threads: (1) accumulators (hi + lo) into a
// 128 x 128 fp32 tile in shared memory, 128-byte swizzled; the weight rows are packed so that the
// columns of two neighbouring states come out as (re, re, im, im); (2) thread (pair of states,
// eighth of the rows) reads its 16 rows into registers and folds them with packed fp32x2
// multiply-adds - the first group from the carried state, the others from zero - and the groups
// are joined as in the streaming scan kernels; (3) it folds again and writes the hi and lo bf16
// halves of its results into its row group's part of the tile (everybody has read the tile by
// then), which one lane per row group hands to the TMA unit (8-byte global stores from the
// threads themselves measured 5 % slower).
// T is a multiple of 128, or 16, 32 or 64: then a tile holds 128 / T whole sequences, a chain is one
// tile, and every row group that begins a sequence starts from that sequence's initial state.
// kTPair (few long sequences, T a multiple of 256): both CTAs of a pair walk ONE sequence, CTA 0 its
// even tiles and CTA 1 its odd ones, which gives twice the chains at the full tile size.  Every row
// group then folds from zero; the last row group joins the groups' results into the tile's own
// contribution, waits for the state that enters the tile (written into this CTA's shared memory by
// the peer, two slots and two barriers in turn), adds Abar^128 times that state unless a flag cuts
// it off, and stores the result into the peer's shared memory: one multiply-add per tile and CTA
// lies between receiving a state and passing it on.
struct FsParams {
    int B, T, P;
    int n_tiles;      // state groups: P / kS
    int k_blocks;     // H / 64
    int tblocks;      // tiles a CTA walks per chain: T / 128, or 1; kTPair: T / 256
    int unit_rows;    // rows of a chain: T, or 128 when T < 128
    int n_units;      // chains per state group: B, or ceil(B * T / 128)
    int gps;          // row groups per sequence inside a tile: 8, or T / 16
    int nchains;      // n_tiles * ceil(n_units / 2); kTPair: n_tiles * B
    const float2* Abar;
    const uint8_t* done;
    const float2* x0;
    float2* xT;
    uint32_t* x_hi;   // plane of high halves, one 32-bit word (re, im as bf16) per state: [B*T, P]
    size_t plane;     // words from the hi plane to the lo plane
    WsHeader* hdr;
};

// Sizes of the kernels that scan in their epilogue, for chains of kS states (64, or 32 where 64-state
// chains would leave CTA pairs without work): the MMA tile is 256 rows x 4 kS columns (re / im of kS states,
// hi | lo weight halves), a CTA holds 2 kS weight rows, the fp32 tile it scans is 128 rows x 2 kS columns,
// and kS / 2 scanning threads (two states each) share a group of 16 rows.
constexpr int kFsRows = 16;                  // rows per scanning thread; 8 row groups per tile
template <int kS>
struct FsCfg {
    static_assert(kS == 64 || kS == 32, "chains of 64 or 32 states");
    static constexpr int kPairs = kS / 2;              // state pairs of a tile = scanning threads per row group
    static constexpr int kN = 4 * kS;                  // accumulator columns of a tile
    static constexpr int kCols = 2 * kS;               // fp32 columns after hi + lo
    static constexpr int kChunks = kCols / 4;          // 16-byte chunks per row of the fp32 tile
    static constexpr int kWRows = 2 * kS;              // weight rows per CTA
    static constexpr int kEpiWarps = kS / 8;           // 8 (two per TMEM lane quarter; 16 measured slower) or 4
    static constexpr int kEpiThreads = 32 * kEpiWarps;
    static constexpr int kThreads = 64 + kEpiThreads;
    static constexpr int kTileBytes = BM * kCols * 4;
    static constexpr int kStageBytes = kABytes + kWRows * BK * 2;
    static constexpr int kGroupBytes = 2 * kFsRows * kPairs * 8;   // both planes of one row group's results
    static constexpr size_t kSmemBytes = (size_t)kPairStages * kStageBytes + kTileBytes + 1024 + 256;
};

// Two fp32 values in one 64-bit register pair, and the packed multiply-add on them: the scan of
// the epilogue advances two states per instruction.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
struct C2 {
    f32x2 re, im;   // two complex numbers: (re, re), (im, im)
};
// a * x + b for two states at once (nai = -Im a)
__device__ __forceinline__ C2 cstep2(f32x2 ar, f32x2 ai, f32x2 nai, C2 x, C2 b) {
    C2 r;
    r.re = fma2(ar, x.re, fma2(nai, x.im, b.re));
    r.im = fma2(ar, x.im, fma2(ai, x.re, b.im));
    return r;
}

template <int kThreadsN>
__device__ __forceinline__ void epi_sync_n() { asm volatile("bar.sync 1, %0;" ::"n"(kThreadsN) : "memory"); }

template <int kS, bool kTPair>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(FsCfg<kS>::kThreads, 1)
gemm_scan_fwd_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmWh,
                     const __grid_constant__ CUtensorMap tmX, FsParams p) {
    using Cfg = FsCfg<kS>;
    constexpr int kPairs = Cfg::kPairs, kChunks = Cfg::kChunks, kFsEpiThreads = Cfg::kEpiThreads, kFsEpiWarps = Cfg::kEpiWarps;
    constexpr int kStageB = Cfg::kStageBytes;
    auto epi_sync = [] { epi_sync_n<Cfg::kEpiThreads>(); };
    extern __shared__ uint8_t smem_raw[];
    __shared__ float4 agg_e[kFsEpiThreads], carry_s[kPairs];   // (re, re, im, im) of two neighbouring states
    __shared__ uint32_t masks[4];
    __shared__ float4 carry_ring[2][kTPair ? kPairs : 1];   // kTPair: the state handed over by the peer CTA, two slots in turn
    __shared__ __align__(8) uint64_t carry_bar[2];           // kTPair: slot i has arrived (one arrival per sending thread)
    static_assert(!kTPair || kPairs == 32, "the last row group of a tile is one warp");
    const Smem s = carve_smem(smem_raw, kPairStages, Cfg::kTileBytes, 0, kStageB, 0);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(s.full(i), 1);
            mbar_init(s.empty(i), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(s.tmem_full(i), 1);
            mbar_init(s.tmem_empty(i), 2 * kFsEpiThreads);
            mbar_init(smem_u32(&carry_bar[i]), kPairs);
        }
        *s.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (threadIdx.x < 4) masks[threadIdx.x] = 0u;
    __syncwarp();
    if (warp == 1) tmem_alloc_pair(s.tmem_slot, kTmemCols);
    tc_fence_before();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *s.tmem_slot_ptr;

    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    const int M = p.B * p.T;
    // chain -> (64 states, this CTA's sequence or, for short sequences, tile of rows); tile tb of a chain -> first row
    // kTPair: both CTAs of the pair walk ONE sequence, tile 2 tb on CTA 0 and tile 2 tb + 1 on CTA 1.
    auto seq_of = [&](int chain) { return kTPair ? chain / p.n_tiles : 2 * (chain / p.n_tiles) + (int)rank; };
    auto row_of = [&](int chain, int tb) {
        const int b = seq_of(chain);
        if (kTPair) return b * p.unit_rows + (2 * tb + (int)rank) * BM;
        return b < p.n_units ? b * p.unit_rows + tb * BM : M;   // nothing left for this CTA: rows past the end read as zero
    };

    if (warp == 0) {
        if (lane == 0) {
            prefetch_tmap(&tmA);
            prefetch_tmap(&tmWh);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int chain = pair; chain < p.nchains && ok; chain += npairs) {
                const int n0 = (chain % p.n_tiles) * Cfg::kN + (int)rank * Cfg::kWRows;
                for (int tb = 0; tb < p.tblocks && ok; ++tb) {
                    const int m0 = row_of(chain, tb);
                    // (no L2 prefetch of the next tile's rows here: with it the kernel ran 7 % slower)
                    for (int kb = 0; kb < p.k_blocks; ++kb) {
                        if (!(ok = mbar_wait(s.empty(stage), phase ^ 1u, s.abort_flag))) break;
                        const uint32_t leader_full = map_to_cta(s.full(stage), 0);
                        if (rank == 0) mbar_expect_tx(s.full(stage), 2 * kStageB);
                        const uint32_t a_dst = smem_u32(s.tiles + (size_t)stage * kStageB);
                        tma_load_2d_pair(a_dst, &tmA, leader_full, kb * BK, m0);
                        tma_load_2d_pair(a_dst + kABytes, &tmWh, leader_full, kb * BK, n0);
                        if (++stage == kPairStages) {
                            stage = 0;
                            phase ^= 1u;
                        }
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = instr_desc(2 * BM, Cfg::kN, 0, 0);
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int chain = pair; chain < p.nchains && ok; chain += npairs) {
                for (int tb = 0; tb < p.tblocks && ok; ++tb) {
                    if (!(ok = mbar_wait(s.tmem_empty(acc), acc_phase ^ 1u, s.abort_flag))) break;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + (uint32_t)(acc * Cfg::kN);
                    for (int kb = 0; kb < p.k_blocks; ++kb) {
                        if (!(ok = mbar_wait(s.full(stage), phase, s.abort_flag))) break;
                        tc_fence_after();
                        const uint32_t a_addr = smem_u32(s.tiles + (size_t)stage * kStageB);
                        const uint64_t adesc = smem_desc_kmajor(a_addr);
                        const uint64_t bdesc = smem_desc_kmajor(a_addr + kABytes);
#pragma unroll
                        for (int k = 0; k < BK / UK; ++k)
                            umma_bf16_pair(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc,
                                           (uint32_t)((kb | k) != 0));
                        umma_commit_pair(s.empty(stage));
                        if (++stage == kPairStages) {
                            stage = 0;
                            phase ^= 1u;
                        }
                    }
                    if (!ok) break;
                    umma_commit_pair(s.tmem_full(acc));
                    if ((acc ^= 1) == 0) acc_phase ^= 1u;
                }
            }
        }
    } else {
        const uint32_t leader_empty0 = map_to_cta(s.tmem_empty(0), 0);
        constexpr int R = kFsRows, nsl = BM / kFsRows;   // rows per thread; groups of rows
        const int te = threadIdx.x - 64;            // 0 .. kFsEpiThreads - 1
        const int q = warp & 3, grp = (warp - 2) >> 2;   // drain role: TMEM lane quarter, 32-column group
        const int sp = te % kPairs, sl = te / kPairs;   // scan role: pair of states of the tile, group of its rows
        const bool group_leader = lane % kPairs == 0;   // the lane that talks to the TMA unit for its row group
        const int prow = q * 32 + lane;             // drain role: row of the tile
        float4* T4 = reinterpret_cast<float4*>(s.staging);
        const C2 zero = {0ull, 0ull};
        int acc = 0;
        uint32_t acc_phase = 0;
        uint32_t n_recv = 0, n_send = 0;            // kTPair: states received from / handed to the peer so far
        const uint32_t peer_ring = map_to_cta(smem_u32(&carry_ring[0][0]), rank ^ 1u);
        const uint32_t peer_bar = map_to_cta(smem_u32(&carry_bar[0]), rank ^ 1u);
        bool ok = true;
        // The flag of this thread's row, loaded one tile ahead (the load's latency would otherwise stand at the
        // head of every tile).
        auto flag_of = [&](int chain, int tb) {
            if (!p.done || te >= BM || chain >= p.nchains) return false;
            const int m = row_of(chain, tb) + te;
            return seq_of(chain) < p.n_units && m < M && p.done[(size_t)m] != 0;
        };
        bool flag_next = flag_of(pair, 0);
        // The chain's multipliers are loaded one chain ahead as well (a chain is a single tile when the sequences are short).
        auto abar_of = [&](int chain, int k) {
            return chain < p.nchains ? p.Abar[(chain % p.n_tiles) * kS + 2 * sp + k] : make_float2(0.f, 0.f);
        };
        float2 a0_next = abar_of(pair, 0), a1_next = abar_of(pair, 1);
        for (int chain = pair; chain < p.nchains && ok; chain += npairs) {
            const int n_tile = chain % p.n_tiles, b = seq_of(chain);
            const bool has_seq = b < p.n_units;
            const bool short_seq = !kTPair && p.T < BM;        // then b counts tiles of rows, not sequences
            const int g0 = sl - sl % p.gps;         // the first row group of this group's sequence in the tile
            const bool from_carry = !kTPair && sl == g0;   // (kTPair: the carried state arrives late; every group joins)
            const int pg = n_tile * kS + 2 * sp;    // the first of this thread's two states
            const float2 a0 = a0_next, a1 = a1_next;
            a0_next = abar_of(chain + npairs, 0);
            a1_next = abar_of(chain + npairs, 1);
            const f32x2 ar = pack2(a0.x, a1.x), ai = pack2(a0.y, a1.y), nai = pack2(-a0.y, -a1.y);
            f32x2 pr, pi, npi;   // Abar^R by squaring in fp32 (a few 1e-7 relative: the results leave as bf16 pairs)
            f32x2 tr = 0ull, ti = 0ull, nti = 0ull;
            {
                float re0 = a0.x, im0 = a0.y, re1 = a1.x, im1 = a1.y;
#pragma unroll
                for (int n = 1; n < R; n *= 2) {
                    const float r0 = fmaf(re0, re0, -im0 * im0), i0 = 2.f * re0 * im0;
                    const float r1 = fmaf(re1, re1, -im1 * im1), i1 = 2.f * re1 * im1;
                    re0 = r0, im0 = i0, re1 = r1, im1 = i1;
                }
                pr = pack2(re0, re1);
                pi = pack2(im0, im1);
                npi = pack2(-im0, -im1);
                if (kTPair) {   // Abar^128: what a tile without flags does to the state that enters it
#pragma unroll
                    for (int n = R; n < BM; n *= 2) {
                        const float r0 = fmaf(re0, re0, -im0 * im0), i0 = 2.f * re0 * im0;
                        const float r1 = fmaf(re1, re1, -im1 * im1), i1 = 2.f * re1 * im1;
                        re0 = r0, im0 = i0, re1 = r1, im1 = i1;
                    }
                    tr = pack2(re0, re1);
                    ti = pack2(im0, im1);
                    nti = pack2(-im0, -im1);
                }
            }
            C2 cin = zero;      // kTPair: the state that enters this CTA's tile
            if (kTPair && rank == 0 && p.x0) {
                const float2 c0 = p.x0[(size_t)b * p.P + pg], c1 = p.x0[(size_t)b * p.P + pg + 1];
                cin.re = pack2(c0.x, c1.x);
                cin.im = pack2(c0.y, c1.y);
            }
            if (sl == 0 && !short_seq && !kTPair) {   // the carried state, as (re, re, im, im) of the two states
                float2 c0 = make_float2(0.f, 0.f), c1 = c0;
                if (p.x0 && has_seq) {
                    c0 = p.x0[(size_t)b * p.P + pg];
                    c1 = p.x0[(size_t)b * p.P + pg + 1];
                }
                carry_s[sp] = make_float4(c0.x, c1.x, c0.y, c1.y);
            }
            for (int tb = 0; tb < p.tblocks; ++tb) {
                const int m0 = row_of(chain, tb);
                if (p.done && te < BM) {
                    const uint32_t mk = __ballot_sync(0xffffffffu, flag_next);
                    if (lane == 0) masks[te >> 5] = mk;
                }
                flag_next = tb + 1 < p.tblocks ? flag_of(chain, tb + 1) : flag_of(chain + npairs, 0);
                (void)mbar_wait(s.tmem_full(acc), acc_phase, s.abort_flag);
                if (group_leader) tma_store_wait_read();   // this row group's results of the previous tile have left shared memory
                epi_sync();   // flags visible, tile free (nobody reads the previous one any more); also:
                              // the 256 threads leave together or not at all
                if (*s.abort_flag) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                // (1) accumulators -> shared-memory tile: 16-byte chunk j of a 128-byte group sits at j ^ (row & 7)
                const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * Cfg::kN);
#pragma unroll
                for (int g = grp; g < Cfg::kCols / 32; g += kFsEpiWarps / 4) {   // 32 columns = one 128-byte group of the row
                    uint32_t r[32], r2[32];
                    tmem_ld32(t_row + (uint32_t)(g * 32), r);
                    tmem_ld32(t_row + (uint32_t)(Cfg::kCols + g * 32), r2);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        T4[prow * kChunks + g * 8 + (j ^ (prow & 7))] =
                            make_float4(__uint_as_float(r[4 * j]) + __uint_as_float(r2[4 * j]),
                                        __uint_as_float(r[4 * j + 1]) + __uint_as_float(r2[4 * j + 1]),
                                        __uint_as_float(r[4 * j + 2]) + __uint_as_float(r2[4 * j + 2]),
                                        __uint_as_float(r[4 * j + 3]) + __uint_as_float(r2[4 * j + 3]));
                }
                tc_fence_before();
                mbar_arrive_cluster(leader_empty0 + 8u * acc);
                if ((acc ^= 1) == 0) acc_phase ^= 1u;
                epi_sync();
                // (2) scan: this thread's two states over its R rows.  The flags of a row group are the
                // same for the whole warp: a group without flags takes loops without the tests.
                const int r0 = sl * R;
                const bool grp_valid = has_seq && m0 + r0 < M;           // (short sequences: the last tile may be ragged)
                const int b_grp = short_seq ? (m0 + r0) / p.T : b;      // this group's sequence
                uint32_t gflags = 0;   // bit g: row group g has a flag
                if (p.done) {
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        const uint32_t mk = masks[w];
#pragma unroll
                        for (int h = 0; h < 32 / R; ++h)
                            if ((mk >> (h * R)) & ((1u << R) - 1u)) gflags |= 1u << (w * (32 / R) + h);
                    }
                }
                const uint32_t mask = p.done ? (masks[r0 >> 5] >> (r0 & 31)) & ((1u << R) - 1u) : 0u;
                C2 v[R];
#pragma unroll
                for (int i = 0; i < R; ++i) {
                    const int row = r0 + i;
                    const float4 t = T4[row * kChunks + ((sp & ~7) | ((sp & 7) ^ (row & 7)))];   // (re, re, im, im)
                    v[i].re = pack2(t.x, t.y);
                    v[i].im = pack2(t.z, t.w);
                }
                C2 e = zero;
                if (from_carry) {   // from the carried or the initial state: these results are final
                    float4 c;
                    if (!short_seq) {
                        c = carry_s[sp];
                    } else if (p.x0 && grp_valid) {
                        const float2 c0 = p.x0[(size_t)b_grp * p.P + pg], c1 = p.x0[(size_t)b_grp * p.P + pg + 1];
                        c = make_float4(c0.x, c1.x, c0.y, c1.y);
                    } else {
                        c = make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                    C2 x = {pack2(c.x, c.y), pack2(c.z, c.w)};
                    if (mask == 0u) {
#pragma unroll
                        for (int i = 0; i < R; ++i) v[i] = x = cstep2(ar, ai, nai, x, v[i]);
                    } else {
#pragma unroll
                        for (int i = 0; i < R; ++i) {
                            if ((mask >> i) & 1u) x = zero;
                            v[i] = x = cstep2(ar, ai, nai, x, v[i]);
                        }
                    }
                    e = x;
                } else if (mask == 0u) {
#pragma unroll
                    for (int i = 0; i < R; ++i) e = cstep2(ar, ai, nai, e, v[i]);
                } else {
#pragma unroll
                    for (int i = 0; i < R; ++i) {
                        if ((mask >> i) & 1u) e = zero;
                        e = cstep2(ar, ai, nai, e, v[i]);
                    }
                }
                {
                    float e0, e1, e2, e3;
                    unpack2(e.re, e0, e1);
                    unpack2(e.im, e2, e3);
                    agg_e[te] = make_float4(e0, e1, e2, e3);
                }
                epi_sync();   // group results visible; every thread has its rows in registers
                C2 x = e;
                if (kTPair) {
                    // The state that enters the tile comes from the peer CTA (the tile before this one), except for
                    // the sequence's first tile.  The last row group passes the tile's end state on as soon as it
                    // can: the tile's own contribution (the groups' results joined from zero) is ready before the
                    // peer's state arrives, so the hand-over costs one multiply-add per tile and CTA.
                    const bool first = rank == 0 && tb == 0, last = rank == 1 && tb == p.tblocks - 1;
                    C2 tile = zero;
                    if (sl == nsl - 1 && !last) {
#pragma unroll
                        for (int g = 0; g < nsl - 1; ++g) {
                            const float4 c = agg_e[g * kPairs + sp];
                            const C2 eg = {pack2(c.x, c.y), pack2(c.z, c.w)};
                            tile = (g == 0 || ((gflags >> g) & 1u)) ? eg : cstep2(pr, pi, npi, tile, eg);
                        }
                        tile = ((gflags >> (nsl - 1)) & 1u) ? e : cstep2(pr, pi, npi, tile, e);
                    }
                    if (!first) {
                        (void)mbar_wait_acquire_cluster(smem_u32(&carry_bar[n_recv & 1u]), (n_recv >> 1) & 1u, s.abort_flag);
                        const float4 c = carry_ring[n_recv & 1u][sp];
                        cin.re = pack2(c.x, c.y);
                        cin.im = pack2(c.z, c.w);
                        ++n_recv;
                    }
                    if (sl == nsl - 1 && !last) {
                        const C2 out = gflags == 0u ? cstep2(tr, ti, nti, cin, tile) : tile;
                        float o0, o1, o2, o3;
                        unpack2(out.re, o0, o1);
                        unpack2(out.im, o2, o3);
                        st_cluster_f4(peer_ring + (uint32_t)(((n_send & 1u) * kPairs + sp) * sizeof(float4)), make_float4(o0, o1, o2, o3));
                        mbar_arrive_release_cluster(peer_bar + 8u * (n_send & 1u));
                        ++n_send;
                    }
                    x = cin;
#pragma unroll
                    for (int g = 0; g < nsl - 1; ++g) {
                        if (g < sl) {
                            const float4 c = agg_e[g * kPairs + sp];
                            const C2 eg = {pack2(c.x, c.y), pack2(c.z, c.w)};
                            x = ((gflags >> g) & 1u) ? eg : cstep2(pr, pi, npi, x, eg);
                        }
                    }
                } else if (!from_carry) {   // state before this group's first row
                    {
                        const float4 c = agg_e[g0 * kPairs + sp];
                        x.re = pack2(c.x, c.y);
                        x.im = pack2(c.z, c.w);
                    }
#pragma unroll
                    for (int g = 1; g < nsl - 1; ++g) {
                        if (g > g0 && g < sl) {
                            const float4 c = agg_e[g * kPairs + sp];
                            const C2 eg = {pack2(c.x, c.y), pack2(c.z, c.w)};
                            x = ((gflags >> g) & 1u) ? eg : cstep2(pr, pi, npi, x, eg);
                        }
                    }
                }
                // (3) fold again; results as hi / lo bf16 halves into this warp's part of the tile (everybody
                // has its rows in registers by now): [plane][row][64 states], which the warp hands to the TMA unit
                uint8_t* warp_out = s.staging + sl * Cfg::kGroupBytes;
                uint2* out = reinterpret_cast<uint2*>(warp_out) + sp;
                auto emit = [&](int i, C2 xv) {
                    float re0, re1, im0, im1;
                    unpack2(xv.re, re0, re1);
                    unpack2(xv.im, im0, im1);
                    const __nv_bfloat162 h0 = __floats2bfloat162_rn(re0, im0), h1 = __floats2bfloat162_rn(re1, im1);
                    const float2 f0 = __bfloat1622float2(h0), f1 = __bfloat1622float2(h1);
                    const __nv_bfloat162 l0 = __floats2bfloat162_rn(re0 - f0.x, im0 - f0.y);
                    const __nv_bfloat162 l1 = __floats2bfloat162_rn(re1 - f1.x, im1 - f1.y);
                    out[i * kPairs] = make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1));
                    out[(R + i) * kPairs] = make_uint2(*reinterpret_cast<const uint32_t*>(&l0), *reinterpret_cast<const uint32_t*>(&l1));
                };
                if (from_carry) {
#pragma unroll
                    for (int i = 0; i < R; ++i) emit(i, v[i]);
                } else if (mask == 0u) {
#pragma unroll
                    for (int i = 0; i < R; ++i) emit(i, x = cstep2(ar, ai, nai, x, v[i]));
                } else {
#pragma unroll
                    for (int i = 0; i < R; ++i) {
                        if ((mask >> i) & 1u) x = zero;
                        emit(i, x = cstep2(ar, ai, nai, x, v[i]));
                    }
                }
                fence_async_smem();
                __syncwarp();
                if (group_leader && grp_valid) {
                    tma_store_3d_nocommit(&tmX, smem_u32(warp_out), n_tile * kS, m0 + r0, 0);
                    tma_commit_group();
                }
                if (short_seq ? (sl - g0 == p.gps - 1) : (sl == nsl - 1)) {   // the group that ends a sequence or the tile
                    float x0r, x1r, x0i, x1i;
                    unpack2(x.re, x0r, x1r);
                    unpack2(x.im, x0i, x1i);
                    // (not after the chain's last tile: by then the first group may already have set up the next chain)
                    if (kTPair) {
                        if (rank == 1 && tb == p.tblocks - 1 && p.xT) {
                            p.xT[(size_t)b * p.P + pg] = make_float2(x0r, x0i);
                            p.xT[(size_t)b * p.P + pg + 1] = make_float2(x1r, x1i);
                        }
                    } else if (!short_seq && tb < p.tblocks - 1) {
                        carry_s[sp] = make_float4(x0r, x1r, x0i, x1i);
                    } else if (p.xT && grp_valid) {
                        p.xT[(size_t)b_grp * p.P + pg] = make_float2(x0r, x0i);
                        p.xT[(size_t)b_grp * p.P + pg + 1] = make_float2(x1r, x1i);
                    }
                }
            }
        }
        if (group_leader) tma_store_wait_all();
    }
    tc_fence_before();
    __syncwarp();
    cluster_sync_all();
    tc_fence_after();
    if (warp == 1) tmem_dealloc_pair(tmem_base, kTmemCols);
    if (threadIdx.x == 0 && *s.abort_flag && p.hdr) p.hdr->status = SSM_ERR_TIMEOUT;
}

// ---------------------------------------------------------------------------------------------
// g_x projection and reverse scan in one kernel (CTA pairs)
// ---------------------------------------------------------------------------------------------
// s_t = g_x,t + keep_{t+1} conj(Abar) s_{t+1} without g_x ever reaching HBM, and the sums
// gAbar = sum_t keep_t s_t conj(x_{t-1}).  The kernel is gemm_scan_fwd_kernel run backwards: a CTA
// walks the tiles of a chain from the last to the first, the last row group starts from the carried
// value, rows are folded from the last to the first, and the reset that acts between rows i and
// i + 1 is the flag of row i + 1.  What is new is x_{t-1}: once a warp has its 16 rows of g_x in
// registers, its part of the shared-memory tile is free, and one lane has the TMA unit copy the
// rows m - 1 ... m + 14 of both planes of x there (one row early; the row before a sequence's first
// is replaced by x0).  In the second pass a thread reads its two states' x_{t-1}, adds
// s_t conj(x_{t-1}) to its sums and writes the hi / lo halves of s_t to the same place, which
// then leaves through the TMA unit as in the forward kernel.  The sums stay in registers for the
// whole chain and are added over the row groups at its end: one entry of gA_part per (sequence,
// state), each written once.  T as for the forward kernel.  kTPair as there, run backwards: CTA 1
// holds the later tile of a pair of tiles, the first row group passes s of the tile's first row
// on, and each CTA writes its own row of gA_part (two per sequence).
struct FbParams {
    int B, T, P;
    int n_tiles;      // state groups: P / kS
    int k_blocks;     // H / 64
    int tblocks;      // tiles a CTA walks per chain: T / 128, or 1; kTPair: T / 256
    int unit_rows;    // rows of a chain: T, or 128 when T < 128 (a tile then holds 128 / T whole sequences)
    int n_units;      // chains per state group: B, or ceil(B * T / 128)
    int gps;          // row groups per sequence inside a tile: 8, or T / 16
    int nchains;      // n_tiles * ceil(n_units / 2); kTPair: n_tiles * B
    const float2* Abar;
    const uint8_t* done;
    const float2* x0;     // [B, P] or NULL
    const float2* gxT;    // [B, P] or NULL
    float2* gA_part;      // [n_units, P]: one row of sums per chain; kTPair: [2 B, P], row 2 b + CTA rank
    float2* gx0;          // [B, P] or NULL
    WsHeader* hdr;
};

template <int kS, bool kTPair>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(FsCfg<kS>::kThreads, 1)
gemm_scan_bwd_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmWh,
                     const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmS, FbParams p) {
    using Cfg = FsCfg<kS>;
    constexpr int kPairs = Cfg::kPairs, kChunks = Cfg::kChunks, kFsEpiThreads = Cfg::kEpiThreads, kFsEpiWarps = Cfg::kEpiWarps;
    constexpr int kStageB = Cfg::kStageBytes;
    auto epi_sync = [] { epi_sync_n<Cfg::kEpiThreads>(); };
    extern __shared__ uint8_t smem_raw[];
    __shared__ float4 agg_e[kFsEpiThreads], carry_s[kPairs];   // (re, re, im, im) of two neighbouring states
    __shared__ uint32_t masks[8];   // [0, 4): flags of the rows one later (the resets of the reverse scan); [4, 8): of the rows
    __shared__ __align__(8) uint64_t xbar[BM / kFsRows];   // one per row group: its rows of x have arrived
    __shared__ float4 carry_ring[2][kTPair ? kPairs : 1];   // kTPair: the value handed over by the peer CTA, two slots in turn
    __shared__ __align__(8) uint64_t carry_bar[2];           // kTPair: slot i has arrived (one arrival per sending thread)
    static_assert(!kTPair || kPairs == 32, "the first row group of a tile is one warp");
    const Smem s = carve_smem(smem_raw, kPairStages, Cfg::kTileBytes, 0, kStageB, 0);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(s.full(i), 1);
            mbar_init(s.empty(i), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(s.tmem_full(i), 1);
            mbar_init(s.tmem_empty(i), 2 * kFsEpiThreads);
            mbar_init(smem_u32(&carry_bar[i]), kPairs);
        }
        for (int i = 0; i < BM / kFsRows; ++i) mbar_init(smem_u32(&xbar[i]), 1);
        *s.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (threadIdx.x < 8) masks[threadIdx.x] = 0u;
    __syncwarp();
    if (warp == 1) tmem_alloc_pair(s.tmem_slot, kTmemCols);
    tc_fence_before();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *s.tmem_slot_ptr;

    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    const int M = p.B * p.T;
    // kTPair: both CTAs of the pair walk ONE sequence, tile 2 tb on CTA 0 and tile 2 tb + 1 on CTA 1.
    auto seq_of = [&](int chain) { return kTPair ? chain / p.n_tiles : 2 * (chain / p.n_tiles) + (int)rank; };
    auto row_of = [&](int chain, int tb) {
        const int b = seq_of(chain);
        if (kTPair) return b * p.unit_rows + (2 * tb + (int)rank) * BM;
        return b < p.n_units ? b * p.unit_rows + tb * BM : M;   // nothing for this CTA: rows past the end read as zero
    };

    if (warp == 0) {
        if (lane == 0) {
            prefetch_tmap(&tmA);
            prefetch_tmap(&tmWh);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int chain = pair; chain < p.nchains && ok; chain += npairs) {
                const int n0 = (chain % p.n_tiles) * Cfg::kN + (int)rank * Cfg::kWRows;
                for (int tb = p.tblocks - 1; tb >= 0 && ok; --tb) {
                    const int m0 = row_of(chain, tb);
                    for (int kb = 0; kb < p.k_blocks; ++kb) {
                        if (!(ok = mbar_wait(s.empty(stage), phase ^ 1u, s.abort_flag))) break;
                        const uint32_t leader_full = map_to_cta(s.full(stage), 0);
                        if (rank == 0) mbar_expect_tx(s.full(stage), 2 * kStageB);
                        const uint32_t a_dst = smem_u32(s.tiles + (size_t)stage * kStageB);
                        tma_load_2d_pair(a_dst, &tmA, leader_full, kb * BK, m0);
                        tma_load_2d_pair(a_dst + kABytes, &tmWh, leader_full, kb * BK, n0);
                        if (++stage == kPairStages) {
                            stage = 0;
                            phase ^= 1u;
                        }
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = instr_desc(2 * BM, Cfg::kN, 0, 0);
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int chain = pair; chain < p.nchains && ok; chain += npairs) {
                for (int tb = 0; tb < p.tblocks && ok; ++tb) {
                    if (!(ok = mbar_wait(s.tmem_empty(acc), acc_phase ^ 1u, s.abort_flag))) break;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + (uint32_t)(acc * Cfg::kN);
                    for (int kb = 0; kb < p.k_blocks; ++kb) {
                        if (!(ok = mbar_wait(s.full(stage), phase, s.abort_flag))) break;
                        tc_fence_after();
                        const uint32_t a_addr = smem_u32(s.tiles + (size_t)stage * kStageB);
                        const uint64_t adesc = smem_desc_kmajor(a_addr);
                        const uint64_t bdesc = smem_desc_kmajor(a_addr + kABytes);
#pragma unroll
                        for (int k = 0; k < BK / UK; ++k)
                            umma_bf16_pair(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc,
                                           (uint32_t)((kb | k) != 0));
                        umma_commit_pair(s.empty(stage));
                        if (++stage == kPairStages) {
                            stage = 0;
                            phase ^= 1u;
                        }
                    }
                    if (!ok) break;
                    umma_commit_pair(s.tmem_full(acc));
                    if ((acc ^= 1) == 0) acc_phase ^= 1u;
                }
            }
        }
    } else {
        const uint32_t leader_empty0 = map_to_cta(s.tmem_empty(0), 0);
        constexpr int R = kFsRows, nsl = BM / kFsRows;   // rows per thread; groups of rows
        const int te = threadIdx.x - 64;            // 0 .. kFsEpiThreads - 1
        const int q = warp & 3, grp = (warp - 2) >> 2;   // drain role: TMEM lane quarter, 32-column group
        const int sp = te % kPairs, sl = te / kPairs;   // scan role: pair of states of the tile, group of its rows
        const bool group_leader = lane % kPairs == 0;   // the lane that talks to the TMA unit for its row group
        const int prow = q * 32 + lane;             // drain role: row of the tile
        const bool short_seq = !kTPair && p.T < BM;            // then a chain is one tile of 128 / T whole sequences
        const int g0 = sl - sl % p.gps;             // first and last row group of this group's sequence in the tile
        const int gl = g0 + p.gps - 1;
        const bool from_carry = !kTPair && sl == gl;           // the last rows come first (kTPair: the carried value arrives late; every group joins)
        uint32_t n_recv = 0, n_send = 0;            // kTPair: values received from / handed to the peer so far
        const uint32_t peer_ring = map_to_cta(smem_u32(&carry_ring[0][0]), rank ^ 1u);
        const uint32_t peer_bar = map_to_cta(smem_u32(&carry_bar[0]), rank ^ 1u);
        float4* T4 = reinterpret_cast<float4*>(s.staging);
        uint8_t* warp_buf = s.staging + sl * Cfg::kGroupBytes;   // this row group's rows of the tile; later x_{t-1}, then s
        uint2* xs = reinterpret_cast<uint2*>(warp_buf) + sp;
        const uint32_t xb = smem_u32(&xbar[sl]);
        uint32_t xphase = 0;
        const C2 zero = {0ull, 0ull};
        int acc = 0;
        uint32_t acc_phase = 0;
        bool ok = true;
        // The chain's multipliers are loaded one chain ahead (a chain is a single tile when the sequences are short).
        auto abar_of = [&](int chain, int k) {
            return chain < p.nchains ? p.Abar[(chain % p.n_tiles) * kS + 2 * sp + k] : make_float2(0.f, 0.f);
        };
        float2 a0_next = abar_of(pair, 0), a1_next = abar_of(pair, 1);
        for (int chain = pair; chain < p.nchains && ok; chain += npairs) {
            const int n_tile = chain % p.n_tiles, b = seq_of(chain);
            const bool has_seq = b < p.n_units;
            const int pg = n_tile * kS + 2 * sp;    // the first of this thread's two states
            const float2 a0 = cconj(a0_next), a1 = cconj(a1_next);
            a0_next = abar_of(chain + npairs, 0);
            a1_next = abar_of(chain + npairs, 1);
            const f32x2 ar = pack2(a0.x, a1.x), ai = pack2(a0.y, a1.y), nai = pack2(-a0.y, -a1.y);
            f32x2 pr, pi, npi;   // conj(Abar)^R by squaring in fp32
            f32x2 tr = 0ull, ti = 0ull, nti = 0ull;
            {
                float re0 = a0.x, im0 = a0.y, re1 = a1.x, im1 = a1.y;
#pragma unroll
                for (int n = 1; n < R; n *= 2) {
                    const float r0 = fmaf(re0, re0, -im0 * im0), i0 = 2.f * re0 * im0;
                    const float r1 = fmaf(re1, re1, -im1 * im1), i1 = 2.f * re1 * im1;
                    re0 = r0, im0 = i0, re1 = r1, im1 = i1;
                }
                pr = pack2(re0, re1);
                pi = pack2(im0, im1);
                npi = pack2(-im0, -im1);
                if (kTPair) {   // conj(Abar)^128: what a tile without flags does to the value that enters it
#pragma unroll
                    for (int n = R; n < BM; n *= 2) {
                        const float r0 = fmaf(re0, re0, -im0 * im0), i0 = 2.f * re0 * im0;
                        const float r1 = fmaf(re1, re1, -im1 * im1), i1 = 2.f * re1 * im1;
                        re0 = r0, im0 = i0, re1 = r1, im1 = i1;
                    }
                    tr = pack2(re0, re1);
                    ti = pack2(im0, im1);
                    nti = pack2(-im0, -im1);
                }
            }
            C2 cin = zero;      // kTPair: s of the row after this CTA's tile (nothing after the sequence's last row)
            C2 g = zero;        // this thread's part of the chain's sums s_t conj(x_{t-1})
            f32x2 gim_neg = 0ull;   // the part of Im g that enters with a minus sign, summed apart
            C2 xinit = zero;    // x0: what stands before the sequence's first row
            if (!short_seq && sl == 0 && p.x0 && has_seq && (!kTPair || rank == 0)) {
                const float2 c0 = p.x0[(size_t)b * p.P + pg], c1 = p.x0[(size_t)b * p.P + pg + 1];
                xinit.re = pack2(c0.x, c1.x);
                xinit.im = pack2(c0.y, c1.y);
            }
            if (from_carry) carry_s[sp] = make_float4(0.f, 0.f, 0.f, 0.f);   // nothing follows the last row
            for (int tb = p.tblocks - 1; tb >= 0; --tb) {
                const int m0 = row_of(chain, tb);
                if (p.done && te < BM) {
                    // a row's own flag, and the flag of the row after it if that row belongs to the same sequence
                    const int tix = kTPair ? 2 * tb + (int)rank : tb;   // this tile's place in its sequence
                    const bool next_in_seq = short_seq ? ((te + 1) % p.T != 0 && m0 + te + 1 < M) : (tix * BM + te + 1 < p.T);
                    const bool f0 = has_seq && m0 + te < M && p.done[(size_t)m0 + te] != 0;
                    const bool f1 = has_seq && next_in_seq && p.done[(size_t)m0 + te + 1] != 0;
                    const uint32_t mk0 = __ballot_sync(0xffffffffu, f0), mk1 = __ballot_sync(0xffffffffu, f1);
                    if (lane == 0) {
                        masks[te >> 5] = mk1;
                        masks[4 + (te >> 5)] = mk0;
                    }
                }
                (void)mbar_wait(s.tmem_full(acc), acc_phase, s.abort_flag);
                tc_fence_after();
                // (1) accumulators -> shared-memory tile: 16-byte chunk j of a 128-byte group sits at j ^ (row & 7).
                // A warp drains two groups of 32 columns (hi + lo halves each): the first group's loads are in
                // flight while it waits for the tile to be free, the second group's while it stores the first.
                constexpr int kGrpStep = kFsEpiWarps / 4;   // a warp drains the 32-column groups grp and grp + kGrpStep
                static_assert(Cfg::kCols / 32 == 2 * kGrpStep, "two 32-column groups per warp");
                const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * Cfg::kN);
                uint32_t ra[32], ra2[32], rb[32], rb2[32];
                tmem_ld32(t_row + (uint32_t)(grp * 32), ra);
                tmem_ld32(t_row + (uint32_t)(Cfg::kCols + grp * 32), ra2);
                if (group_leader) tma_store_wait_read();   // this row group's results of the previous tile have left shared memory
                epi_sync();   // flags visible, tile free (nobody reads the previous one any more); also:
                              // the 256 threads leave together or not at all
                tmem_ld_wait();
                if (*s.abort_flag) {
                    ok = false;
                    break;
                }
                tmem_ld32(t_row + (uint32_t)((grp + kGrpStep) * 32), rb);
                tmem_ld32(t_row + (uint32_t)(Cfg::kCols + (grp + kGrpStep) * 32), rb2);
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    T4[prow * kChunks + grp * 8 + (j ^ (prow & 7))] =
                        make_float4(__uint_as_float(ra[4 * j]) + __uint_as_float(ra2[4 * j]),
                                    __uint_as_float(ra[4 * j + 1]) + __uint_as_float(ra2[4 * j + 1]),
                                    __uint_as_float(ra[4 * j + 2]) + __uint_as_float(ra2[4 * j + 2]),
                                    __uint_as_float(ra[4 * j + 3]) + __uint_as_float(ra2[4 * j + 3]));
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    T4[prow * kChunks + (grp + kGrpStep) * 8 + (j ^ (prow & 7))] =
                        make_float4(__uint_as_float(rb[4 * j]) + __uint_as_float(rb2[4 * j]),
                                    __uint_as_float(rb[4 * j + 1]) + __uint_as_float(rb2[4 * j + 1]),
                                    __uint_as_float(rb[4 * j + 2]) + __uint_as_float(rb2[4 * j + 2]),
                                    __uint_as_float(rb[4 * j + 3]) + __uint_as_float(rb2[4 * j + 3]));
                tc_fence_before();
                mbar_arrive_cluster(leader_empty0 + 8u * acc);
                if ((acc ^= 1) == 0) acc_phase ^= 1u;
                epi_sync();
                // (2) this thread's two states over its R rows, last row first
                const int r0 = sl * R;
                const bool grp_valid = has_seq && m0 + r0 < M;           // (short sequences: the last tile may be ragged)
                const int b_grp = short_seq ? (m0 + r0) / p.T : b;      // this group's sequence
                uint32_t gflags = 0;   // bit g: a reset acts inside or right after row group g
                uint32_t mask = 0u, mask0 = 0u;
                if (p.done) {
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        const uint32_t mk = masks[w];
#pragma unroll
                        for (int h = 0; h < 32 / R; ++h)
                            if ((mk >> (h * R)) & ((1u << R) - 1u)) gflags |= 1u << (w * (32 / R) + h);
                    }
                    mask = (masks[r0 >> 5] >> (r0 & 31)) & ((1u << R) - 1u);
                    mask0 = (masks[4 + (r0 >> 5)] >> (r0 & 31)) & ((1u << R) - 1u);
                }
                C2 v[R];
#pragma unroll
                for (int i = 0; i < R; ++i) {
                    const int row = r0 + i;
                    const float4 t = T4[row * kChunks + ((sp & ~7) | ((sp & 7) ^ (row & 7)))];   // (re, re, im, im)
                    v[i].re = pack2(t.x, t.y);
                    v[i].im = pack2(t.z, t.w);
                }
                if (sl == gl && tb == p.tblocks - 1 && (!kTPair || rank == 1) && p.gxT && grp_valid) {   // the gradient of the final state
                    const float2 c0 = p.gxT[(size_t)b_grp * p.P + pg], c1 = p.gxT[(size_t)b_grp * p.P + pg + 1];
                    float v0, v1, v2, v3;
                    unpack2(v[R - 1].re, v0, v1);
                    unpack2(v[R - 1].im, v2, v3);
                    v[R - 1].re = pack2(v0 + c0.x, v1 + c1.x);
                    v[R - 1].im = pack2(v2 + c0.y, v3 + c1.y);
                }
                // the warp has its rows: rows m - 1 ... m + R - 2 of x (both planes) into its part of the tile
                fence_async_smem();
                __syncwarp();
                if (group_leader) {
                    mbar_expect_tx(xb, Cfg::kGroupBytes);
                    tma_load_3d(smem_u32(warp_buf), &tmX, xb, n_tile * kS, m0 + r0 - 1, 0);
                    // and the same rows of the tile before this one into L2, where the next load will find them
                    if (tb > 0) tma_prefetch_3d(&tmX, n_tile * kS, m0 - (kTPair ? 2 : 1) * BM + r0 - 1, 0);
                }
                C2 e = zero;
                if (from_carry) {   // from the carried value (nothing, for a sequence inside the tile): these results are final
                    const float4 c = short_seq ? make_float4(0.f, 0.f, 0.f, 0.f) : carry_s[sp];
                    C2 x = {pack2(c.x, c.y), pack2(c.z, c.w)};
                    if (mask == 0u) {
#pragma unroll
                        for (int i = R - 1; i >= 0; --i) v[i] = x = cstep2(ar, ai, nai, x, v[i]);
                    } else {
#pragma unroll
                        for (int i = R - 1; i >= 0; --i) {
                            if ((mask >> i) & 1u) x = zero;
                            v[i] = x = cstep2(ar, ai, nai, x, v[i]);
                        }
                    }
                    e = x;
                } else if (mask == 0u) {
#pragma unroll
                    for (int i = R - 1; i >= 0; --i) e = cstep2(ar, ai, nai, e, v[i]);
                } else {
#pragma unroll
                    for (int i = R - 1; i >= 0; --i) {
                        if ((mask >> i) & 1u) e = zero;
                        e = cstep2(ar, ai, nai, e, v[i]);
                    }
                }
                {
                    float e0, e1, e2, e3;
                    unpack2(e.re, e0, e1);
                    unpack2(e.im, e2, e3);
                    agg_e[te] = make_float4(e0, e1, e2, e3);
                }
                epi_sync();   // group results visible
                C2 x = e;
                if (kTPair) {
                    // The value that enters the tile (s of the row after it) comes from the peer CTA, which holds the
                    // tile after this one, except for the sequence's last tile.  The first row group passes s of the
                    // tile's first row on as soon as it can: the tile's own contribution (the groups' results joined
                    // from zero) is ready before the peer's value arrives.
                    const bool first = rank == 1 && tb == p.tblocks - 1, last = rank == 0 && tb == 0;
                    C2 tile = zero;
                    if (sl == 0 && !last) {
#pragma unroll
                        for (int gq = nsl - 1; gq >= 1; --gq) {
                            const float4 c = agg_e[gq * kPairs + sp];
                            const C2 eg = {pack2(c.x, c.y), pack2(c.z, c.w)};
                            tile = (gq == nsl - 1 || ((gflags >> gq) & 1u)) ? eg : cstep2(pr, pi, npi, tile, eg);
                        }
                        tile = (gflags & 1u) ? e : cstep2(pr, pi, npi, tile, e);
                    }
                    if (!first) {
                        (void)mbar_wait_acquire_cluster(smem_u32(&carry_bar[n_recv & 1u]), (n_recv >> 1) & 1u, s.abort_flag);
                        const float4 c = carry_ring[n_recv & 1u][sp];
                        cin.re = pack2(c.x, c.y);
                        cin.im = pack2(c.z, c.w);
                        ++n_recv;
                    } else {
                        cin = zero;
                    }
                    if (sl == 0 && !last) {
                        const C2 out = gflags == 0u ? cstep2(tr, ti, nti, cin, tile) : tile;
                        float o0, o1, o2, o3;
                        unpack2(out.re, o0, o1);
                        unpack2(out.im, o2, o3);
                        st_cluster_f4(peer_ring + (uint32_t)(((n_send & 1u) * kPairs + sp) * sizeof(float4)), make_float4(o0, o1, o2, o3));
                        mbar_arrive_release_cluster(peer_bar + 8u * (n_send & 1u));
                        ++n_send;
                    }
                    x = cin;
#pragma unroll
                    for (int gq = nsl - 1; gq >= 1; --gq) {
                        if (gq > sl) {
                            const float4 c = agg_e[gq * kPairs + sp];
                            const C2 eg = {pack2(c.x, c.y), pack2(c.z, c.w)};
                            x = ((gflags >> gq) & 1u) ? eg : cstep2(pr, pi, npi, x, eg);
                        }
                    }
                } else if (!from_carry) {   // s of the row after this group's last
                    {
                        const float4 c = agg_e[gl * kPairs + sp];
                        x.re = pack2(c.x, c.y);
                        x.im = pack2(c.z, c.w);
                    }
#pragma unroll
                    for (int gq = nsl - 2; gq >= 1; --gq) {
                        if (gq > sl && gq < gl) {
                            const float4 c = agg_e[gq * kPairs + sp];
                            const C2 eg = {pack2(c.x, c.y), pack2(c.z, c.w)};
                            x = ((gflags >> gq) & 1u) ? eg : cstep2(pr, pi, npi, x, eg);
                        }
                    }
                }
                // (3) fold again, with x_{t-1} at hand: sums for gAbar, s as hi / lo bf16 halves in place of x
                if (!mbar_wait(xb, xphase, s.abort_flag)) {
                    // (the wait gave up: the flag is set, everybody leaves at the next barrier)
                }
                xphase ^= 1u;
                const bool seq_start = tb == 0 && sl == g0 && (!kTPair || rank == 0);   // row 0 of this group is the sequence's first row
                if (short_seq && seq_start) {                // the state before that row: this sequence's x0
                    xinit = zero;
                    if (p.x0 && grp_valid) {
                        const float2 c0 = p.x0[(size_t)b_grp * p.P + pg], c1 = p.x0[(size_t)b_grp * p.P + pg + 1];
                        xinit.re = pack2(c0.x, c1.x);
                        xinit.im = pack2(c0.y, c1.y);
                    }
                }
                // A tile without flags (the common case) takes the loop without the per-row tests.
                auto fold_rows = [&](auto with_flags) {
                    constexpr bool kFlags = decltype(with_flags)::value;
#pragma unroll
                    for (int i = R - 1; i >= 0; --i) {
                        C2 sv = v[i];
                        if (!from_carry) {
                            if (kFlags && ((mask >> i) & 1u)) x = zero;
                            sv = x = cstep2(ar, ai, nai, x, v[i]);
                        }
                        if (!kFlags || !((mask0 >> i) & 1u)) {
                            C2 xp;
                            if (seq_start && i == 0) {
                                xp = xinit;
                            } else {
                                const uint2 xh = xs[i * kPairs], xl = xs[(R + i) * kPairs];
                                xp.re = add2(pack2(__uint_as_float(xh.x << 16), __uint_as_float(xh.y << 16)),
                                             pack2(__uint_as_float(xl.x << 16), __uint_as_float(xl.y << 16)));
                                xp.im = add2(pack2(__uint_as_float(xh.x & 0xffff0000u), __uint_as_float(xh.y & 0xffff0000u)),
                                             pack2(__uint_as_float(xl.x & 0xffff0000u), __uint_as_float(xl.y & 0xffff0000u)));
                            }
                            // g += s conj(x):  re += s.re x.re + s.im x.im,  im += s.im x.re - s.re x.im (two sums)
                            g.re = fma2(sv.re, xp.re, fma2(sv.im, xp.im, g.re));
                            g.im = fma2(sv.im, xp.re, g.im);
                            gim_neg = fma2(sv.re, xp.im, gim_neg);
                        }
                        float re0, re1, im0, im1;
                        unpack2(sv.re, re0, re1);
                        unpack2(sv.im, im0, im1);
                        const __nv_bfloat162 h0 = __floats2bfloat162_rn(re0, im0), h1 = __floats2bfloat162_rn(re1, im1);
                        const uint32_t hb0 = *reinterpret_cast<const uint32_t*>(&h0), hb1 = *reinterpret_cast<const uint32_t*>(&h1);
                        const f32x2 lre = sub2(sv.re, pack2(__uint_as_float(hb0 << 16), __uint_as_float(hb1 << 16)));
                        const f32x2 lim = sub2(sv.im, pack2(__uint_as_float(hb0 & 0xffff0000u), __uint_as_float(hb1 & 0xffff0000u)));
                        float lr0, lr1, li0, li1;
                        unpack2(lre, lr0, lr1);
                        unpack2(lim, li0, li1);
                        const __nv_bfloat162 l0 = __floats2bfloat162_rn(lr0, li0), l1 = __floats2bfloat162_rn(lr1, li1);
                        xs[i * kPairs] = make_uint2(hb0, hb1);
                        xs[(R + i) * kPairs] = make_uint2(*reinterpret_cast<const uint32_t*>(&l0), *reinterpret_cast<const uint32_t*>(&l1));
                    }
                };
                if ((mask | mask0) == 0u)
                    fold_rows(std::false_type{});
                else
                    fold_rows(std::true_type{});
                fence_async_smem();
                __syncwarp();
                if (group_leader && grp_valid) {
                    tma_store_3d_nocommit(&tmS, smem_u32(warp_buf), n_tile * kS, m0 + r0, 0);
                    tma_commit_group();
                }
                if (sl == g0) {   // x is s of the first row of the tile (of the sequence, when it lies inside the tile)
                    float x0r, x1r, x0i, x1i;
                    unpack2(x.re, x0r, x1r);
                    unpack2(x.im, x0i, x1i);
                    if (kTPair && !(rank == 0 && tb == 0)) {
                        // (handed to the peer above)
                    } else if (tb > 0) {
                        carry_s[sp] = make_float4(x0r, x1r, x0i, x1i);
                    } else if (p.gx0 && grp_valid) {   // what reaches the initial state: keep_0 conj(Abar) s_0
                        const bool cut = (mask0 & 1u) != 0u;
                        const float2 z = make_float2(0.f, 0.f);
                        p.gx0[(size_t)b_grp * p.P + pg] = cut ? z : cfma(a0, make_float2(x0r, x0i), z);
                        p.gx0[(size_t)b_grp * p.P + pg + 1] = cut ? z : cfma(a1, make_float2(x1r, x1i), z);
                    }
                }
            }
            if (!ok) break;
            // the chain's sums over the row groups (agg_e is free: everybody is past the last tile's join)
            epi_sync();
            {
                float g0, g1, g2, g3;
                unpack2(g.re, g0, g1);
                unpack2(sub2(g.im, gim_neg), g2, g3);
                agg_e[te] = make_float4(g0, g1, g2, g3);
            }
            epi_sync();
            if (sl == 0 && has_seq) {
                float4 sum = agg_e[sp];
#pragma unroll
                for (int gq = 1; gq < nsl; ++gq) {
                    const float4 c = agg_e[gq * kPairs + sp];
                    sum.x += c.x, sum.y += c.y, sum.z += c.z, sum.w += c.w;
                }
                const size_t part_row = kTPair ? 2 * (size_t)b + rank : (size_t)b;   // kTPair: each CTA has half of the sequence's rows
                p.gA_part[part_row * p.P + pg] = make_float2(sum.x, sum.z);
                p.gA_part[part_row * p.P + pg + 1] = make_float2(sum.y, sum.w);
            }
        }
        if (group_leader) tma_store_wait_all();
    }
    tc_fence_before();
    __syncwarp();
    cluster_sync_all();
    tc_fence_after();
    if (warp == 1) tmem_dealloc_pair(tmem_base, kTmemCols);
    if (threadIdx.x == 0 && *s.abort_flag && p.hdr) p.hdr->status = SSM_ERR_TIMEOUT;
}

// ---------------------------------------------------------------------------------------------
// NT kernel (weight gradients): one 128 x 256 output tile and one slice of the rows per CTA
// ---------------------------------------------------------------------------------------------
struct NtParams {
    int K;              // rows of A and Bm (the reduction index)
    int J;              // columns of Bm = leading dimension of a partial
    int I;              // columns of A
    int j_tiles;        // J / BN
    int blocks_per_split;  // k-blocks (of BK rows) per slice
    float* part;        // [splits, I, J]
    WsHeader* hdr;
    // kMulti: n_prod products of bf16 planes in one accumulator; product j takes plane (pa >> 4 j) & 15 of A
    // (columns [a I, (a + 1) I) of its matrix) and plane (pb >> 4 j) & 15 of Bm (columns [b J, (b + 1) J)).
    int n_prod;
    uint32_t pa, pb;
};

// kMulti = false: the 256 accumulator columns are 128 output columns times the two planes (hi, lo) of Bm, added
// in the epilogue.  kMulti = true: 256 output columns, every product of the schedule accumulated in place.
template <bool kMulti>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_nt_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmBhi,
                  const __grid_constant__ CUtensorMap tmBlo, NtParams p) {
    extern __shared__ uint8_t smem_raw[];
    const Smem s = carve_smem(smem_raw, kStages, 0, 0);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t tmem_base = prologue(s, warp, lane, 128);
    const int tile = blockIdx.x, split = blockIdx.y;
    constexpr int kOutCols = kMulti ? BN : BN / 2;   // (not kMulti) accumulator columns [0,128): hi plane, [128,256): lo plane
    const int i0 = (tile / p.j_tiles) * BM, j0 = (tile % p.j_tiles) * kOutCols;
    const int total_blocks = (p.K + BK - 1) / BK;
    const int kb0 = split * p.blocks_per_split;
    const int kb1 = min(total_blocks, kb0 + p.blocks_per_split);
    const int nkb = max(0, kb1 - kb0);

    if (warp == 0) {
        if (lane == 0) {
            prefetch_tmap(&tmA);
            prefetch_tmap(&tmBhi);
            prefetch_tmap(&tmBlo);
            int stage = 0;
            uint32_t phase = 0;
            for (int kq = 0; kq < (kMulti ? p.n_prod : 1) * nkb; ++kq) {
                if (!mbar_wait(s.empty(stage), phase ^ 1u, s.abort_flag)) break;
                mbar_expect_tx(s.full(stage), kStageBytes);
                const uint32_t a_dst = smem_u32(s.tiles + (size_t)stage * kStageBytes);
                const int j = kq / max(nkb, 1), kb = kq - j * nkb;   // product of the schedule, k-block of the slice
                const int row = (kb0 + kb) * BK;
                const int ia = kMulti ? (int)((p.pa >> (4 * j)) & 15u) * p.I + i0 : i0;
                const int jb = kMulti ? (int)((p.pb >> (4 * j)) & 15u) * p.J + j0 : j0;
#pragma unroll
                for (int h = 0; h < BM / 64; ++h) tma_load_2d(a_dst + h * (BK * 128), &tmA, s.full(stage), ia + 64 * h, row);
                if (kMulti) {
#pragma unroll
                    for (int h = 0; h < BN / 64; ++h)
                        tma_load_2d(a_dst + kABytes + h * (BK * 128), &tmBhi, s.full(stage), jb + 64 * h, row);
                } else {
#pragma unroll
                    for (int h = 0; h < BN / 128; ++h) {
                        tma_load_2d(a_dst + kABytes + h * (BK * 128), &tmBhi, s.full(stage), j0 + 64 * h, row);
                        tma_load_2d(a_dst + kABytes + (BN / 128 + h) * (BK * 128), &tmBlo, s.full(stage), j0 + 64 * h, row);
                    }
                }
                if (++stage == kStages) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && nkb > 0) {
            constexpr uint32_t idesc = instr_desc(BM, BN, 1, 1);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int kb = 0; kb < (kMulti ? p.n_prod : 1) * nkb; ++kb) {
                if (!(ok = mbar_wait(s.full(stage), phase, s.abort_flag))) break;
                tc_fence_after();
                const uint32_t a_addr = smem_u32(s.tiles + (size_t)stage * kStageBytes);
                const uint64_t adesc = smem_desc_mnmajor(a_addr);
                const uint64_t bdesc = smem_desc_mnmajor(a_addr + kABytes);
#pragma unroll
                for (int k = 0; k < BK / UK; ++k) {
                    // 16 k-rows of 128 bytes further: +2048 bytes = +128 in the address field
                    umma_bf16(tmem_base, adesc + (uint64_t)(128 * k), bdesc + (uint64_t)(128 * k), idesc,
                              (uint32_t)((kb | k) != 0));
                }
                umma_commit(s.empty(stage));
                if (++stage == kStages) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
            if (ok) umma_commit(s.tmem_full(0));
        }
    } else {
        const int q = warp & 3;
        const int row = i0 + q * 32 + lane;
        float* dst_row = p.part + ((size_t)split * p.I + row) * p.J + j0;
        bool ok = true;
        if (nkb > 0) {
            ok = mbar_wait(s.tmem_full(0), 0, s.abort_flag);
            tc_fence_after();
        }
        if (ok) {
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
            for (int c = 0; c < kOutCols; c += 32) {
                float v[32];
                if (nkb > 0) {
                    uint32_t r[32];
                    tmem_ld32(t_row + (uint32_t)c, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
                    if (!kMulti) {
                        tmem_ld32(t_row + (uint32_t)(kOutCols + c), r);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] += __uint_as_float(r[i]);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = 0.f;
                }
                if (row < p.I) {
                    float4* dst = reinterpret_cast<float4*>(dst_row + c);
#pragma unroll
                    for (int i = 0; i < 8; ++i) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                }
            }
        }
    }
    epilogue_exit(s, warp, tmem_base, p.hdr);
}

// ---------------------------------------------------------------------------------------------
// NT kernel on CTA pairs
// ---------------------------------------------------------------------------------------------
// The same product on clusters of two CTAs: one MMA spans a 256 x 256 accumulator tile, CTA r holding
// output rows i0 + 128 r .. (its 128 columns of A) and one plane of Bm (r = 0: the high halves, r = 1: the low
// halves; the MMA takes half of its B columns from each CTA).  Every CTA then brings in 32 KB per k-block
// instead of 48 KB for the same tensor-core cycles, which is what bounds the single-CTA kernel (96 KB through
// shared memory per 512 tensor-core cycles).  Barriers as in the TN pair kernel: the leader's `full` barriers
// count both CTAs' bytes, its commits arrive in both CTAs.  One tile and one slice of the rows per pair.
constexpr int kNtPairStages = 6;
constexpr int kNtPairStageBytes = kABytes + kBBytes / 2;   // 32 KB
constexpr size_t kNtPairSmemBytes = (size_t)kNtPairStages * kNtPairStageBytes + 1024 + 256;

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_tc_nt_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmBhi,
                       const __grid_constant__ CUtensorMap tmBlo, NtParams p) {
    extern __shared__ uint8_t smem_raw[];
    const Smem s = carve_smem(smem_raw, kNtPairStages, 0, 0, kNtPairStageBytes, 0);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    // barriers of the ring: more stages than the common layout has slots for, so they take the skip slots
    auto rfull = [&](int i) { return s.skip_full(i); };
    auto rempty = [&](int i) { return s.skip_full(kNtPairStages + i); };
    if (threadIdx.x == 0) {
        for (int i = 0; i < kNtPairStages; ++i) {
            mbar_init(rfull(i), 1);
            mbar_init(rempty(i), 1);
        }
        mbar_init(s.tmem_full(0), 1);
        *s.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();
    if (warp == 1) tmem_alloc_pair(s.tmem_slot, BN);
    tc_fence_before();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *s.tmem_slot_ptr;

    const int tile = blockIdx.x >> 1, split = blockIdx.y;
    constexpr int kOutCols = BN / 2;
    const int i0 = (tile / p.j_tiles) * (2 * BM) + (int)rank * BM, j0 = (tile % p.j_tiles) * kOutCols;
    const int total_blocks = (p.K + BK - 1) / BK;
    const int kb0 = split * p.blocks_per_split;
    const int nkb = max(0, min(total_blocks, kb0 + p.blocks_per_split) - kb0);

    if (warp == 0) {
        if (lane == 0) {
            prefetch_tmap(&tmA);
            prefetch_tmap(rank == 0 ? &tmBhi : &tmBlo);
            const CUtensorMap* tmB = rank == 0 ? &tmBhi : &tmBlo;
            int stage = 0;
            uint32_t phase = 0;
            for (int kb = 0; kb < nkb; ++kb) {
                if (!mbar_wait(rempty(stage), phase ^ 1u, s.abort_flag)) break;
                const uint32_t leader_full = map_to_cta(rfull(stage), 0);
                if (rank == 0) mbar_expect_tx(rfull(stage), 2 * kNtPairStageBytes);
                const uint32_t a_dst = smem_u32(s.tiles + (size_t)stage * kNtPairStageBytes);
                const int row = (kb0 + kb) * BK;
#pragma unroll
                for (int h = 0; h < BM / 64; ++h) tma_load_2d_pair(a_dst + h * (BK * 128), &tmA, leader_full, i0 + 64 * h, row);
#pragma unroll
                for (int h = 0; h < kOutCols / 64; ++h)
                    tma_load_2d_pair(a_dst + kABytes + h * (BK * 128), tmB, leader_full, j0 + 64 * h, row);
                if (++stage == kNtPairStages) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0 && nkb > 0) {
            constexpr uint32_t idesc = instr_desc(2 * BM, BN, 1, 1);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int kb = 0; kb < nkb; ++kb) {
                if (!(ok = mbar_wait(rfull(stage), phase, s.abort_flag))) break;
                tc_fence_after();
                const uint32_t a_addr = smem_u32(s.tiles + (size_t)stage * kNtPairStageBytes);
                const uint64_t adesc = smem_desc_mnmajor(a_addr);
                const uint64_t bdesc = smem_desc_mnmajor(a_addr + kABytes);
#pragma unroll
                for (int k = 0; k < BK / UK; ++k)
                    umma_bf16_pair(tmem_base, adesc + (uint64_t)(128 * k), bdesc + (uint64_t)(128 * k), idesc,
                                   (uint32_t)((kb | k) != 0));
                umma_commit_pair(rempty(stage));
                if (++stage == kNtPairStages) {
                    stage = 0;
                    phase ^= 1u;
                }
            }
            if (ok) umma_commit_pair(s.tmem_full(0));
        }
    } else {
        const int q = warp & 3;
        const int row = i0 + q * 32 + lane;
        float* dst_row = p.part + ((size_t)split * p.I + row) * p.J + j0;
        bool ok = true;
        if (nkb > 0) {
            ok = mbar_wait(s.tmem_full(0), 0, s.abort_flag);
            tc_fence_after();
        }
        if (ok) {
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
            for (int c = 0; c < kOutCols; c += 32) {
                float v[32];
                if (nkb > 0) {
                    uint32_t r[32], r2[32];
                    tmem_ld32(t_row + (uint32_t)c, r);
                    tmem_ld32(t_row + (uint32_t)(kOutCols + c), r2);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]) + __uint_as_float(r2[i]);
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = 0.f;
                }
                if (row < p.I) {
                    float4* dst = reinterpret_cast<float4*>(dst_row + c);
#pragma unroll
                    for (int i = 0; i < 8; ++i) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                }
            }
        }
    }
    // nobody leaves (or frees tensor memory) while the other CTA may still signal or compute
    tc_fence_before();
    __syncwarp();
    cluster_sync_all();
    tc_fence_after();
    if (warp == 1) tmem_dealloc_pair(tmem_base, BN);
    if (threadIdx.x == 0 && *s.abort_flag && p.hdr) p.hdr->status = SSM_ERR_TIMEOUT;
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
// Row-major bf16 matrix [rows, cols] (cols contiguous), boxes of box_cols x box_rows, 128-byte swizzle.
static bool make_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_cols,
                     uint32_t box_rows, bool f32 = false, CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B,
                     uint64_t pitch_elems = 0) {
    PFN_cuTensorMapEncodeTiled fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {(pitch_elems ? pitch_elems : cols) * (f32 ? 4u : 2u)};   // rows may be wider than the view
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static int sm_count() { return device_sm_count(); }

// How many clusters of two CTAs of `kernel` the current device runs at the same time (cached per
// kernel and device).
static int resident_pairs(const void* kernel, size_t smem_bytes, int threads = kTnThreads) {
    static std::mutex mu;
    static std::map<std::pair<const void*, int>, int> cache;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    std::lock_guard<std::mutex> lock(mu);
    auto it = cache.find({kernel, dev});
    if (it != cache.end()) return it->second;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (unsigned)sm_count(), 1, 1);
    cfg.blockDim = dim3((unsigned)threads, 1, 1);
    cfg.dynamicSmemBytes = smem_bytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess) {
        (void)cudaGetLastError();
        n = 0;
    }
    cache[{kernel, dev}] = n;
    return n;
}

template <typename K>
static bool set_smem(K kernel, size_t bytes) {
    return set_max_dynamic_smem(reinterpret_cast<const void*>(kernel), bytes);
}

}  // namespace tc

int tc_max_n() { return tc::kMaxDiag; }

bool tc_tn_supported(int M, int N_out, int K, bool split_w) {
    const int out_cols = split_w ? tc::BN / 2 : tc::BN;
    // Outputs are a multiple of 128 columns wide; a last tile of the 256-column kind may be half empty (its
    // weight rows past N_out read as zero and its results past N_out are clipped by the TMA stores).
    (void)out_cols;
    return M >= 1 && K >= tc::BK && (K % tc::BK) == 0 && (N_out % (tc::BN / 2)) == 0 && N_out <= tc::kMaxDiag;
}

static int pair_tiles_of(int M, int n_tiles) { return ((M + 2 * tc::BM - 1) / (2 * tc::BM)) * n_tiles; }

// The bf16 epilogue can also sum skip * dot over the rows (one partial row per CTA) where the pair kernel
// runs and the output is at most kDotMaxN wide.
bool tc_tn_dot_supported(int M, int N_out, int K) {
    return tc_tn_supported(M, N_out, K, false) && N_out <= tc::kDotMaxN && pair_tiles_of(M, (N_out + tc::BN - 1) / tc::BN) >= tc::sm_count() / 2;
}
int tc_tn_dot_max_rows() { return 2 * tc::sm_count(); }

bool tc_tn_gate_supported(int M, int N_out, int K) {
    return tc_tn_supported(M, N_out, K, true) && pair_tiles_of(M, N_out / (tc::BN / 2)) >= tc::sm_count() / 2;
}

int launch_gemm_tc_tn(const GemmTcTN& g, cudaStream_t st) {
    using namespace tc;
    const int out_cols = g.split_w ? BN / 2 : BN;
    const int n_tiles = (g.N_out + out_cols - 1) / out_cols;
    const int epi = g.gate_out ? 2 : (g.store_f32 ? 0 : (g.dot ? 3 : 1));
    if ((epi == 1 || epi == 3) && (g.split_w || !g.diag || !g.skip)) return SSM_ERR_SHAPE;
    if (epi == 3 && (!g.dot_part || !g.dot_rows || !tc_tn_dot_supported(g.M, g.N_out, g.K))) return SSM_ERR_SHAPE;
    if (epi == 2 && (!g.split_w || !g.store_f32 || !g.skip || !tc_tn_gate_supported(g.M, g.N_out, g.K))) return SSM_ERR_SHAPE;
    CUtensorMap ma, mw, mo, ms, mg;
    // with a product schedule the operands are planes_a / planes_w bf16 planes of K columns each, side by side
    const int n_prod = g.n_products > 0 ? g.n_products : 1;
    const uint64_t a_cols = (uint64_t)g.K * (g.n_products > 0 ? g.planes_a : 1);
    const uint64_t w_cols = (uint64_t)g.K * (g.n_products > 0 ? g.planes_w : 1);
    if (g.n_products > 8) return SSM_ERR_SHAPE;
    if (!make_map(&ma, g.A, (uint64_t)g.M, a_cols, BK, BM)) return SSM_ERR_CUDA;
    if (g.store_f32) {   // fp32 result, stored by the TMA unit in boxes of 32 rows x 32 columns
        if (!make_map(&mo, g.out, (uint64_t)g.M, (uint64_t)g.N_out, 32, 32, true)) return SSM_ERR_CUDA;
    } else {             // bf16 result: 32 x 32 boxes, 64-byte rows
        if (!make_map(&mo, g.out, (uint64_t)g.M, (uint64_t)g.N_out, 32, 32, false, CU_TENSOR_MAP_SWIZZLE_64B)) return SSM_ERR_CUDA;
    }
    ms = mo;             // unused unless there is a skip operand
    mg = mo;             // unused unless there is a gated result
    if (epi != 0 && !make_map(&ms, g.skip, (uint64_t)g.M, (uint64_t)g.N_out, 32, 32, false, CU_TENSOR_MAP_SWIZZLE_64B))
        return SSM_ERR_CUDA;
    if (epi == 2 && !make_map(&mg, g.gate_out, (uint64_t)g.M, (uint64_t)g.N_out, 32, 32, false, CU_TENSOR_MAP_SWIZZLE_64B))
        return SSM_ERR_CUDA;
    if (epi == 3 && !make_map(&mg, g.dot, (uint64_t)g.M, (uint64_t)g.N_out, 32, 32, false, CU_TENSOR_MAP_SWIZZLE_64B))
        return SSM_ERR_CUDA;   // (the dot operand travels in the map slot of the gated result)
    TnParams p{g.M, n_tiles, n_prod * (g.K / BK), g.N_out, g.diag, g.hdr, (const char*)g.A, (int)a_cols * 2, g.dot_part,
               g.n_products > 0 ? g.K / BK : 0, g.prod_a, g.prod_w};
    const int m_tiles = (g.M + BM - 1) / BM;
    const int pair_tiles = pair_tiles_of(g.M, n_tiles);
    // rows of the packed weight matrix that exist (tiles may reach past them: those rows read as zero)
    const uint64_t w_rows = g.split_w ? (uint64_t)2 * g.N_out : (uint64_t)g.N_out;
    bool ok = true;
    if (pair_tiles >= sm_count() / 2) {   // enough 256-row tiles to give every CTA pair one
        if (!make_map(&mw, g.W, w_rows, w_cols, BK, BN / 2)) return SSM_ERR_CUDA;
        count_launch();
        // The kernel is persistent: its grid is the number of CTA pairs the device can hold at once
        // (not every SM has a partner that a cluster may use).
#define SSM_LAUNCH_PAIR(EPI, SPLIT)                                                                        \
    do {                                                                                                   \
        auto kern = gemm_tc_tn_pair_kernel<EPI, SPLIT>;                                                    \
        constexpr size_t smem = pair_smem_bytes(EPI);                                                      \
        ok = set_smem(kern, smem);                                                                         \
        const int pairs = ok ? resident_pairs(reinterpret_cast<const void*>(kern), smem) : 0;              \
        ok = ok && pairs > 0;                                                                              \
        if (ok) kern<<<2 * min(pairs, pair_tiles), kTnThreads, smem, st>>>(ma, mw, mo, ms, mg, p);         \
        if (ok && g.dot_rows) *g.dot_rows = 2 * min(pairs, pair_tiles);                                    \
    } while (0)
        if (epi == 3) SSM_LAUNCH_PAIR(3, false);
        else if (epi == 2) SSM_LAUNCH_PAIR(2, true);
        else if (epi == 1) SSM_LAUNCH_PAIR(1, false);
        else if (g.split_w) SSM_LAUNCH_PAIR(0, true);
        else SSM_LAUNCH_PAIR(0, false);
#undef SSM_LAUNCH_PAIR
        return ok ? SSM_OK : SSM_ERR_CUDA;
    }
    if (!make_map(&mw, g.W, w_rows, w_cols, BK, BN)) return SSM_ERR_CUDA;
    const int grid = min(sm_count(), m_tiles * n_tiles);
    count_launch();
#define SSM_LAUNCH_TN(EPI, SPLIT)                                                                          \
    do {                                                                                                   \
        auto kern = gemm_tc_tn_kernel<EPI, SPLIT>;                                                         \
        ok = set_smem(kern, tn_smem_bytes(EPI));                                                           \
        if (ok) kern<<<grid, kTnThreads, tn_smem_bytes(EPI), st>>>(ma, mw, mo, ms, mg, p);                 \
    } while (0)
    if (epi == 1) SSM_LAUNCH_TN(1, false);
    else if (g.split_w) SSM_LAUNCH_TN(0, true);
    else SSM_LAUNCH_TN(0, false);
#undef SSM_LAUNCH_TN
    return ok ? SSM_OK : SSM_ERR_CUDA;
}

// The two bf16 planes of a state tensor as [2, B*T, P] 32-bit words, in boxes of `states` states x kFsRows rows x both planes.
static bool make_plane_map(CUtensorMap* map, const void* planes, int M, int P, int states) {
    PFN_cuTensorMapEncodeTiled fn = tc::encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)P, (cuuint64_t)M, 2};
    cuuint64_t strides[2] = {(cuuint64_t)P * 4, (cuuint64_t)M * P * 4};
    cuuint32_t box[3] = {(cuuint32_t)states, (cuuint32_t)tc::kFsRows, 2};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 3, const_cast<void*>(planes), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Fewest (sequence, state group) chain pairs for which the kernels that scan in the epilogue of a projection
// are taken: below it too many CTA pairs would idle while a few walk their chains tile by tile.
#ifndef SSM_FUSED_MIN_PAIRS
#define SSM_FUSED_MIN_PAIRS 32   // measured: 32 pairs (16 sequences of 256 states) still beat the separate kernels
#endif
#ifndef SSM_FUSED_NARROW_BELOW
#define SSM_FUSED_NARROW_BELOW 0   // 0: chains of 32 states where chains of 64 would occupy at most half of the CTA pairs
#endif

// Chains per state group: the sequences, or, when a 128-row tile holds several whole sequences, the tiles.
static int fs_units(int B, int T) { return T >= tc::BM ? B : (B * T + tc::BM - 1) / tc::BM; }

// How the kernels that scan in their epilogue take a problem: chains of 64 states, of 32 (few sequences: twice
// the chains, half the tile), or not at all (group 0); and, for few long sequences, both CTAs of a pair on one
// sequence (time pairs: CTA 0 has the even tiles, CTA 1 the odd ones, the state passes from one to the other
// through shared memory), which doubles the chains without halving the tile.
#ifndef SSM_FUSED_TIME_PAIRS
#define SSM_FUSED_TIME_PAIRS 1
#endif
struct FusedMode {
    int group;
    bool time_pairs;
};
static FusedMode fused_mode(int B, int T, int H, int P) {
    const bool t_ok = T % tc::BM == 0 || T == 16 || T == 32 || T == 64;
    if (!t_ok || H % tc::BK != 0 || P % 64 != 0) return {0, false};
    const int pairs64 = (P / 64) * ((fs_units(B, T) + 1) / 2);
    // A tile of 32 states takes about 0.8 of the time of a tile of 64 (measured), so halving the chains pays only
    // where the second half of the CTA pairs would otherwise idle: 16 x 16384 at P = 256 1.88 -> 1.78 ms per step,
    // 16 x 1024 0.242 -> 0.229; with 64 of 74 pairs busy (32 sequences) it costs 30 - 50 % in these kernels.
    // Time pairs double the chains at the full tile: 16 x 16384 1.76 -> 1.48 ms, 16 x 1024 0.228 -> 0.212.
    const int narrow_below = SSM_FUSED_NARROW_BELOW > 0 ? SSM_FUSED_NARROW_BELOW : tc::sm_count() / 4 + 1;
    const bool tp_ok = SSM_FUSED_TIME_PAIRS && T % (2 * tc::BM) == 0;
    if (pairs64 >= narrow_below) {
        // Enough chains either way.  Time pairs give twice the chains at half the length, which fills the last
        // round of chains better when there are only a few rounds (48 sequences at P = 256: 96 chains take two
        // rounds on 74 CTA pairs, 192 half-length chains three half-rounds).
        const int np = tc::sm_count() / 2;
        const int rounds = (pairs64 + np - 1) / np, half_rounds = (2 * pairs64 + np - 1) / np;
        return {64, tp_ok && half_rounds < 2 * rounds};
    }
    if (tp_ok && (P / 64) * B >= SSM_FUSED_MIN_PAIRS) return {64, true};
    if (pairs64 < SSM_FUSED_MIN_PAIRS) return {0, false};
    return {32, false};
}
int tc_gemm_scan_group(int B, int T, int H, int P) { return fused_mode(B, T, H, P).group; }
bool tc_gemm_scan_time_pairs(int B, int T, int H, int P) { return fused_mode(B, T, H, P).time_pairs; }
bool tc_gemm_scan_fwd_supported(int B, int T, int H, int P) { return tc_gemm_scan_group(B, T, H, P) != 0; }
bool tc_gemm_scan_bwd_supported(int B, int T, int H, int P) { return tc_gemm_scan_group(B, T, H, P) != 0; }

template <int kS, bool kTPair>
static int launch_gemm_scan_fwd_s(const GemmScanFwd& g, cudaStream_t st) {
    using namespace tc;
    using Cfg = FsCfg<kS>;
    const int M = g.B * g.T;
    CUtensorMap ma, mw, mx;
    if (!make_map(&ma, g.u, (uint64_t)M, (uint64_t)g.H, BK, BM)) return SSM_ERR_CUDA;
    if (!make_map(&mw, g.Wsplit, (uint64_t)4 * g.P, (uint64_t)g.H, BK, Cfg::kWRows)) return SSM_ERR_CUDA;
    if (!make_plane_map(&mx, g.x_planes, M, g.P, kS)) return SSM_ERR_CUDA;
    const int units = fs_units(g.B, g.T), n_tiles = g.P / kS;
    FsParams p{g.B, g.T, g.P, n_tiles, g.H / BK, g.T >= BM ? g.T / BM : 1, g.T >= BM ? g.T : BM, units,
               g.T >= BM ? BM / kFsRows : g.T / kFsRows, n_tiles * ((units + 1) / 2),
               g.Abar, g.done, g.x0, g.xT, (uint32_t*)g.x_planes, (size_t)M * g.P, g.hdr};
    if (kTPair) {   // a chain is one sequence; each CTA has every other tile
        p.tblocks = g.T / (2 * BM);
        p.nchains = n_tiles * g.B;
    }
    count_launch();
    auto kern = gemm_scan_fwd_kernel<kS, kTPair>;
    if (!set_smem(kern, Cfg::kSmemBytes)) return SSM_ERR_CUDA;
    const int pairs = resident_pairs(reinterpret_cast<const void*>(kern), Cfg::kSmemBytes, Cfg::kThreads);
    if (pairs <= 0) return SSM_ERR_CUDA;
    kern<<<2 * min(pairs, p.nchains), Cfg::kThreads, Cfg::kSmemBytes, st>>>(ma, mw, mx, p);
    return SSM_OK;
}

int launch_gemm_scan_fwd(const GemmScanFwd& g, cudaStream_t st) {
    const FusedMode m = fused_mode(g.B, g.T, g.H, g.P);
    if (m.group == 64) return m.time_pairs ? launch_gemm_scan_fwd_s<64, true>(g, st) : launch_gemm_scan_fwd_s<64, false>(g, st);
    if (m.group == 32) return launch_gemm_scan_fwd_s<32, false>(g, st);
    return SSM_ERR_SHAPE;
}

// Rows of gA_part that launch_gemm_scan_bwd writes: one per chain of a state group (two per sequence where both
// CTAs of a pair share a sequence).
int tc_gemm_scan_bwd_part_rows(int B, int T, int H, int P) {
    return fused_mode(B, T, H, P).time_pairs ? 2 * B : fs_units(B, T);
}

template <int kS, bool kTPair>
static int launch_gemm_scan_bwd_s(const GemmScanBwd& g, cudaStream_t st) {
    using namespace tc;
    using Cfg = FsCfg<kS>;
    const int M = g.B * g.T;
    CUtensorMap ma, mw, mx, ms;
    if (!make_map(&ma, g.gy, (uint64_t)M, (uint64_t)g.H, BK, BM)) return SSM_ERR_CUDA;
    if (!make_map(&mw, g.Wsplit, (uint64_t)4 * g.P, (uint64_t)g.H, BK, Cfg::kWRows)) return SSM_ERR_CUDA;
    if (!make_plane_map(&mx, g.x_planes, M, g.P, kS) || !make_plane_map(&ms, g.s_planes, M, g.P, kS)) return SSM_ERR_CUDA;
    const int units = fs_units(g.B, g.T), n_tiles = g.P / kS;
    FbParams p{g.B, g.T, g.P, n_tiles, g.H / BK, g.T >= BM ? g.T / BM : 1, g.T >= BM ? g.T : BM, units,
               g.T >= BM ? BM / kFsRows : g.T / kFsRows, n_tiles * ((units + 1) / 2),
               g.Abar, g.done, g.x0, g.gxT, g.gA_part, g.gx0, g.hdr};
    if (kTPair) {
        p.tblocks = g.T / (2 * BM);
        p.nchains = n_tiles * g.B;
    }
    count_launch();
    auto kern = gemm_scan_bwd_kernel<kS, kTPair>;
    if (!set_smem(kern, Cfg::kSmemBytes)) return SSM_ERR_CUDA;
    const int pairs = resident_pairs(reinterpret_cast<const void*>(kern), Cfg::kSmemBytes, Cfg::kThreads);
    if (pairs <= 0) return SSM_ERR_CUDA;
    kern<<<2 * min(pairs, p.nchains), Cfg::kThreads, Cfg::kSmemBytes, st>>>(ma, mw, mx, ms, p);
    return SSM_OK;
}

int launch_gemm_scan_bwd(const GemmScanBwd& g, cudaStream_t st) {
    const FusedMode m = fused_mode(g.B, g.T, g.H, g.P);
    if (m.group == 64) return m.time_pairs ? launch_gemm_scan_bwd_s<64, true>(g, st) : launch_gemm_scan_bwd_s<64, false>(g, st);
    if (m.group == 32) return launch_gemm_scan_bwd_s<32, false>(g, st);
    return SSM_ERR_SHAPE;
}

bool tc_nt_supported(int I, int J) { return (I % tc::BM) == 0 && (J % (tc::BN / 2)) == 0; }

int tc_nt_splits(int K, int I, int J) {
    const int tiles = (I / tc::BM) * (J / (tc::BN / 2));
    const int blocks = (K + tc::BK - 1) / tc::BK;
    int s = tc::sm_count() / (tiles > 0 ? tiles : 1);
    if (s < 1) s = 1;
    if (s > blocks) s = blocks;
    if (s > 64) s = 64;
    return s;
}

#ifndef SSM_NT_PAIRS
#define SSM_NT_PAIRS 1   // weight-gradient products on CTA pairs where the output has a multiple of 256 rows
#endif
int launch_gemm_tc_nt(const GemmTcNT& g, cudaStream_t st) {
    using namespace tc;
    CUtensorMap ma, mbh, mbl;
    const int blocks = (g.K + BK - 1) / BK;
    const int bps = (blocks + g.splits - 1) / g.splits;
    if (g.n_products > 0) {   // planes side by side: A [K, planes_a * I], Bm [K, planes_b * J]
        if (g.n_products > 8 || g.J % BN != 0) return SSM_ERR_SHAPE;
        if (!make_map(&ma, g.A, (uint64_t)g.K, (uint64_t)g.I * g.planes_a, 64, BK)) return SSM_ERR_CUDA;
        if (!make_map(&mbh, g.Bm_hi, (uint64_t)g.K, (uint64_t)g.J * g.planes_b, 64, BK)) return SSM_ERR_CUDA;
        const int j_tiles = g.J / BN;
        NtParams p{g.K, g.J, g.I, j_tiles, bps, g.part, g.hdr, g.n_products, g.prod_a, g.prod_b};
        dim3 grid((g.I / BM) * j_tiles, g.splits);
        count_launch();
        const bool ok = set_smem(gemm_tc_nt_kernel<true>, kNtSmemBytes);
        gemm_tc_nt_kernel<true><<<grid, kThreads, kNtSmemBytes, st>>>(ma, mbh, mbh, p);
        return ok ? SSM_OK : SSM_ERR_CUDA;
    }
    if (!make_map(&ma, g.A, (uint64_t)g.K, (uint64_t)g.I, 64, BK, false, CU_TENSOR_MAP_SWIZZLE_128B, (uint64_t)g.lda))
        return SSM_ERR_CUDA;
    if (!make_map(&mbh, g.Bm_hi, (uint64_t)g.K, (uint64_t)g.J, 64, BK)) return SSM_ERR_CUDA;
    if (!make_map(&mbl, g.Bm_lo, (uint64_t)g.K, (uint64_t)g.J, 64, BK)) return SSM_ERR_CUDA;
    const int j_tiles = g.J / (BN / 2);
    NtParams p{g.K, g.J, g.I, j_tiles, bps, g.part, g.hdr, 0, 0u, 0u};
    if (SSM_NT_PAIRS && g.I % (2 * BM) == 0) {   // 256 x 256 tiles on CTA pairs
        dim3 grid(2 * (g.I / (2 * BM)) * j_tiles, g.splits);
        count_launch();
        const bool ok = set_smem(gemm_tc_nt_pair_kernel, kNtPairSmemBytes);
        gemm_tc_nt_pair_kernel<<<grid, kThreads, kNtPairSmemBytes, st>>>(ma, mbh, mbl, p);
        return ok ? SSM_OK : SSM_ERR_CUDA;
    }
    dim3 grid((g.I / BM) * j_tiles, g.splits);
    count_launch();
    const bool ok = set_smem(gemm_tc_nt_kernel<false>, kNtSmemBytes);
    gemm_tc_nt_kernel<false><<<grid, kThreads, kNtSmemBytes, st>>>(ma, mbh, mbl, p);
    return ok ? SSM_OK : SSM_ERR_CUDA;
}

// Split-K factor of the product-schedule variant (tiles of 128 x 256 outputs).
int tc_nt_multi_splits(int K, int I, int J) {
    const int tiles = (I / tc::BM) * (J / tc::BN);
    const int blocks = (K + tc::BK - 1) / tc::BK;
    int s = tc::sm_count() / (tiles > 0 ? tiles : 1);
    if (s < 1) s = 1;
    if (s > blocks) s = blocks;
    if (s > 64) s = 64;
    return s;
}

}  // namespace ssm
