// C-ABI entry points (see include/ssm.h): argument checks, workspace layout, launch order.
#include <cstdio>
#include <algorithm>

#include "kernels.h"

using namespace ssm;

#define SSM_API extern "C" __attribute__((visibility("default")))

namespace {

// Workspace of one layer.  Two paths:
//  * tensor-core path (bf16 I/O and tile-sized H, P): projections on tcgen05, states Bu / g_x
//    in one fp32 buffer, x and s kept as bf16 pairs;
//  * CUDA-core path (fp32 I/O, or odd shapes): fp32 weights and states throughout.
//  * plane path (fp32 I/O and tile-sized H, P with enough rows): the same projections on tcgen05 as sums
//    of products of bf16 planes (three planes per fp32 value: exact), fp32 states, scans as on the
//    CUDA-core path.
struct LayerPlan {
    bool tc;
    bool planes;
    int splits;
    size_t hdr, Abar, Alo, Bbar, W0, W1, W2, W3, f32buf, xs, gs, gAbar, gBbar, scan, part, dot, total;
    size_t u3, gy3, x3, s3, acc;   // plane path: planes of u, gy, x, s and the fp32 result of a projection
};

#ifndef SSM_PLANES_MIN_ROWS
#define SSM_PLANES_MIN_ROWS 1   // fewest B*T rows for which fp32 layers take the plane path
#endif
bool planes_supported(const ssm_shape& s) {
    const long long BT = (long long)s.B * s.T;
    return s.H % 256 == 0 && s.P % 128 == 0 && s.H <= tc_max_n() && 2 * s.P <= tc_max_n() && BT >= SSM_PLANES_MIN_ROWS;
}
// Product schedules (plane of the first operand, plane of the second, four bits each, smallest terms first):
// fp32 x fp32 = lo hi, hi lo, mid mid, mid hi, hi mid, hi hi;  bf16 x fp32 = hi lo, hi mid, hi hi.
constexpr uint32_t kProd6A = 0x001102u, kProd6B = 0x010120u;
constexpr uint32_t kProd3A = 0x000u, kProd3B = 0x012u;

size_t take(size_t& off, size_t bytes) {
    const size_t at = off;
    off = align_up(off + bytes, 256);
    return at;
}

LayerPlan plan_layer(const ssm_shape& s, bool allow_tc = true) {
    LayerPlan p{};
    size_t off = 0;
    const size_t BT = (size_t)s.B * s.T, PH = (size_t)s.P * s.H;
    const int P2 = 2 * s.P;
    p.tc = allow_tc && s.io_dtype == SSM_BF16 && tc_tn_supported((int)BT, P2, s.H, true) &&
           tc_tn_supported((int)BT, s.H, P2, false) && tc_nt_supported(s.H, P2);
    p.planes = !p.tc && s.io_dtype == SSM_F32 && planes_supported(s);
    p.splits = p.tc ? tc_nt_splits((int)BT, s.H, P2) : (p.planes ? tc_nt_multi_splits((int)BT, s.H, P2) : gemm_nt_splits((int)BT));
    p.hdr = take(off, sizeof(WsHeader));
    p.Abar = take(off, (size_t)s.P * 8);
    p.Alo = take(off, (size_t)s.P * 8);
    p.Bbar = take(off, PH * 8);
    if (p.tc) {
        p.W0 = take(off, 4 * PH * 2);   // hi/lo stacked Bbar operand  [4P, H] bf16
        p.W1 = take(off, 4 * PH * 2);   // hi/lo stacked conj(C) operand [4P, H] bf16
        p.W2 = take(off, 2 * PH * 2);   // Cp [H, 2P] bf16
        p.W3 = take(off, 2 * PH * 2);   // Bq [H, 2P] bf16
        p.f32buf = take(off, BT * s.P * 8);   // Bu (forward), then g_x (backward)
        p.xs = take(off, BT * s.P * 8);       // x as two bf16 planes (hi, lo)
        p.gs = take(off, BT * s.P * 8);       // s as two bf16 planes (hi, lo)
    } else {
        // CUDA-core path: fp32 operands.  Plane path: three bf16 planes of each (6 PH values, 2 bytes each).
        p.W0 = take(off, p.planes ? 6 * PH * 2 : 2 * PH * 4);   // Bp [2P, H]   | Wb3 [2P, 3H]
        p.W1 = take(off, p.planes ? 6 * PH * 2 : 2 * PH * 4);   // Cq [2P, H]   | Cq3 [2P, 3H]
        p.W2 = take(off, p.planes ? 6 * PH * 2 : 2 * PH * 4);   // Cp [H, 2P]   | Cp3 [H, 3 * 2P]
        p.W3 = take(off, p.planes ? 6 * PH * 2 : 2 * PH * 4);   // Bq [H, 2P]   | Bq3 [H, 3 * 2P]
        p.f32buf = off;                 // unused
        p.xs = take(off, BT * s.P * 8); // Bu, overwritten in place by x
        p.gs = take(off, BT * s.P * 8); // g_x, overwritten in place by s
        if (p.planes) {
            p.u3 = take(off, BT * 3 * s.H * 2);
            p.gy3 = take(off, BT * 3 * s.H * 2);
            p.x3 = take(off, BT * 6 * s.P * 2);
            p.s3 = take(off, BT * 6 * s.P * 2);
            p.acc = take(off, BT * s.H * 4);
        }
    }
    p.gAbar = take(off, (size_t)s.P * 8);
    p.gBbar = take(off, PH * 8);
    p.scan = take(off, scan_scratch_bytes(s.B, s.T, s.P, 2));
    p.part = take(off, (size_t)2 * p.splits * 2 * PH * 4);   // split-K partials of gBbar, then those of dC
    {   // dD: partial column sums of gy * u, from the stand-alone kernel or from the epilogue of the du projection
        const size_t rows = (size_t)tc_tn_dot_max_rows();
        const size_t fused = rows * s.H + colsum_tmp_floats((int)rows, s.H);
        p.dot = take(off, std::max(dot_columns_tmp_floats((int)BT, s.H), fused) * 4);
    }
    p.total = off;
    return p;
}

template <typename T>
T* at(void* ws, size_t off) { return reinterpret_cast<T*>(reinterpret_cast<char*>(ws) + off); }

int check_ws(const void* ws, size_t have, size_t need) {
    if (!ws) return SSM_ERR_WORKSPACE;
    if (misaligned(ws, 256)) return SSM_ERR_ALIGN;
    if (have < need) return SSM_ERR_WORKSPACE;
    return SSM_OK;
}

}  // namespace

SSM_API const char* ssm_status_string(int status) {
    switch (status) {
        case SSM_OK: return "ok";
        case SSM_ERR_NULL: return "a required pointer is NULL";
        case SSM_ERR_SHAPE: return "bad shape (B,T >= 1; H,P positive multiples of 8; reserved == 0)";
        case SSM_ERR_ALIGN: return "a pointer is not aligned as required";
        case SSM_ERR_DTYPE: return "io_dtype must be SSM_F32 or SSM_BF16";
        case SSM_ERR_WORKSPACE: return "workspace missing or too small";
        case SSM_ERR_CUDA: return "a CUDA call or kernel launch failed";
        case SSM_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        case SSM_ERR_TOO_LARGE: return "problem needs more scratch than the library's built-in static buffer holds";
        default: return "unknown status";
    }
}

SSM_API int ssm_check(const void* ws, void* stream) {
    if (!ws) return SSM_ERR_NULL;
    int status = 0;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemcpyAsync(&status, ws, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return SSM_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return SSM_ERR_CUDA;
    return status == 0 ? SSM_OK : SSM_ERR_TIMEOUT;
}

SSM_API int ssm_discretize(const ssm_shape* shape, const ssm_c64* Lambda, const float* Delta, const ssm_c64* Bc,
                           ssm_c64* Abar, ssm_c64* Bbar, void* stream) {
    if (int rc = check_shape(shape)) return rc;
    if (!Lambda || !Delta || !Bc || !Abar || !Bbar) return SSM_ERR_NULL;
    if (misaligned(Lambda) || misaligned(Delta) || misaligned(Bc) || misaligned(Abar) || misaligned(Bbar))
        return SSM_ERR_ALIGN;
    launch_discretize(shape->H, shape->P, (const float2*)Lambda, Delta, (const float2*)Bc, (float2*)Abar, nullptr,
                      (float2*)Bbar, (cudaStream_t)stream);
    SSM_RETURN_IF_CUDA_ERROR();
    return SSM_OK;
}

SSM_API int ssm_discretize_bwd(const ssm_shape* shape, const ssm_c64* Lambda, const float* Delta,
                               const ssm_c64* Bc, const ssm_c64* gAbar, const ssm_c64* gBbar, ssm_c64* dLambda,
                               float* dDelta, ssm_c64* dB, void* stream) {
    if (int rc = check_shape(shape)) return rc;
    if (!Lambda || !Delta || !Bc || !gAbar || !gBbar || !dLambda || !dDelta || !dB) return SSM_ERR_NULL;
    if (misaligned(Lambda) || misaligned(Delta) || misaligned(Bc) || misaligned(gAbar) || misaligned(gBbar) ||
        misaligned(dLambda) || misaligned(dDelta) || misaligned(dB))
        return SSM_ERR_ALIGN;
    launch_discretize_bwd(shape->H, shape->P, (const float2*)Lambda, Delta, (const float2*)Bc,
                          (const float2*)gAbar, (const float2*)gBbar, (float2*)dLambda, dDelta, (float2*)dB,
                          (cudaStream_t)stream);
    SSM_RETURN_IF_CUDA_ERROR();
    return SSM_OK;
}

SSM_API size_t ssm_scan_workspace_bytes(const ssm_shape* shape) {
    if (check_shape(shape) != SSM_OK) return 0;
    return sizeof(WsHeader) + scan_scratch_bytes(shape->B, shape->T, shape->P);
}

SSM_API int ssm_scan_fwd(const ssm_shape* shape, const ssm_c64* Abar, const ssm_c64* Bu, const uint8_t* done,
                         const ssm_c64* x0, ssm_c64* x, ssm_c64* xT, void* ws, size_t ws_bytes, void* stream) {
    if (int rc = check_shape(shape)) return rc;
    if (!Abar || !Bu || !x) return SSM_ERR_NULL;
    if (misaligned(Abar) || misaligned(Bu) || misaligned(x) || misaligned(x0) || misaligned(xT)) return SSM_ERR_ALIGN;
    if (int rc = check_ws(ws, ws_bytes, ssm_scan_workspace_bytes(shape))) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(ws, 0, sizeof(WsHeader), st) != cudaSuccess) return SSM_ERR_CUDA;
    StageTimer tm("scan_fwd", st);
    int rc = launch_scan_fwd(shape->B, shape->T, shape->P, (const float2*)Abar, nullptr, (const float2*)Bu, done,
                             (const float2*)x0, x, false, (float2*)xT, at<WsHeader>(ws, 0),
                             at<char>(ws, sizeof(WsHeader)), st);
    if (rc) return rc;
    SSM_RETURN_IF_CUDA_ERROR();
    return SSM_OK;
}

SSM_API int ssm_scan_bwd(const ssm_shape* shape, const ssm_c64* Abar, const uint8_t* done, const ssm_c64* x0,
                         const ssm_c64* x, const ssm_c64* gx, const ssm_c64* gxT, ssm_c64* gBu, ssm_c64* gAbar,
                         ssm_c64* gx0, void* ws, size_t ws_bytes, void* stream) {
    if (int rc = check_shape(shape)) return rc;
    if (!Abar || !x || !gx || !gBu || !gAbar) return SSM_ERR_NULL;
    if (misaligned(Abar) || misaligned(x) || misaligned(gx) || misaligned(gBu) || misaligned(gAbar) ||
        misaligned(x0) || misaligned(gxT) || misaligned(gx0))
        return SSM_ERR_ALIGN;
    if (int rc = check_ws(ws, ws_bytes, ssm_scan_workspace_bytes(shape))) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(ws, 0, sizeof(WsHeader), st) != cudaSuccess) return SSM_ERR_CUDA;
    StageTimer tm("scan_bwd", st);
    int rc = launch_scan_bwd(shape->B, shape->T, shape->P, (const float2*)Abar, nullptr, done, (const float2*)x0, x, false,
                             (const float2*)gx, (const float2*)gxT, gBu, false, (float2*)gAbar, (float2*)gx0,
                             at<WsHeader>(ws, 0), at<char>(ws, sizeof(WsHeader)), st);
    if (rc) return rc;
    SSM_RETURN_IF_CUDA_ERROR();
    return SSM_OK;
}

SSM_API size_t ssm_layer_workspace_bytes(const ssm_shape* shape) {
    if (check_shape(shape) != SSM_OK) return 0;
    return plan_layer(*shape).total;
}

SSM_API int ssm_layer_plan_string(const ssm_shape* shape, char* buf, size_t len) {
    if (!buf || len == 0) return SSM_ERR_NULL;
    buf[0] = 0;
    if (int rc = check_shape(shape)) return rc;
    const ssm_shape& s = *shape;
    const LayerPlan p = plan_layer(s);
    const int group = p.tc ? tc_gemm_scan_group(s.B, s.T, s.H, s.P) : 0;
    const char* proj = p.tc ? "tensor-cores" : (p.planes ? "tensor-cores-planes" : "cuda-cores");
    if (group)
        snprintf(buf, len, "projections=%s scans=fused chain_states=%d time_pairs=%d", proj, group,
                 tc_gemm_scan_time_pairs(s.B, s.T, s.H, s.P) ? 1 : 0);
    else
        snprintf(buf, len, "projections=%s scans=separate", proj);
    return SSM_OK;
}

// Discretised parameters and packed projection operands into the workspace.
static void layer_prepare(const ssm_shape& s, const LayerPlan& p, const ssm_c64* Lambda, const float* Delta,
                          const ssm_c64* Bc, const ssm_c64* Cc, void* ws, cudaStream_t st) {
    StageTimer tm("discretize_pack", st);
    if (p.tc) {
        // one kernel (the kernels that scan in the epilogue of a projection want their own column order)
        const int group = tc_gemm_scan_group(s.B, s.T, s.H, s.P);
        launch_discretize_pack_tc(s.H, s.P, group, group, (const float2*)Lambda, Delta,
                                  (const float2*)Bc, (const float2*)Cc, at<float2>(ws, p.Abar), at<float2>(ws, p.Alo),
                                  at<float2>(ws, p.Bbar), at<void>(ws, p.W0), at<void>(ws, p.W1), at<void>(ws, p.W2),
                                  at<void>(ws, p.W3), st);
        return;
    }
    if (p.planes) {
        launch_discretize_pack_planes(s.H, s.P, (const float2*)Lambda, Delta, (const float2*)Bc, (const float2*)Cc,
                                      at<float2>(ws, p.Abar), at<float2>(ws, p.Alo), at<float2>(ws, p.Bbar),
                                      at<void>(ws, p.W0), at<void>(ws, p.W1), at<void>(ws, p.W2), at<void>(ws, p.W3), st);
        return;
    }
    launch_discretize(s.H, s.P, (const float2*)Lambda, Delta, (const float2*)Bc, at<float2>(ws, p.Abar),
                      at<float2>(ws, p.Alo), at<float2>(ws, p.Bbar), st);
    launch_pack_operands(s.H, s.P, false, at<float2>(ws, p.Bbar), (const float2*)Cc, at<void>(ws, p.W0),
                         at<void>(ws, p.W3), at<void>(ws, p.W2), at<void>(ws, p.W1), st);
}

// Launch sequence of one layer's forward pass from a prepared workspace.  `hdr` receives the
// status of bounded waits.
// Storage types of the tensors a layer reads and writes.  For the entry points of a single layer all
// of them are shape->io_dtype; inside a stack only the stack's own input and outputs are.
struct LayerIo {
    bool u_bf16, y_bf16;      // forward: u in, y out
    bool gy_bf16, du_bf16;    // backward: gy in, du out
};
static LayerIo layer_io(const ssm_shape& s) {
    const bool b = s.io_dtype == SSM_BF16;
    return {b, b, b, b};
}

static int layer_fwd_run(const ssm_shape& s, const LayerPlan& p, const LayerIo& io, const float* D, const void* u,
                         const uint8_t* done, const ssm_c64* x0, void* y, ssm_c64* xT, void* ws, WsHeader* hdr,
                         cudaStream_t st) {
    const int BT = s.B * s.T, P2 = 2 * s.P;
    if (p.tc && !(io.u_bf16 && io.y_bf16)) return SSM_ERR_DTYPE;   // the tensor-core path reads and writes bf16
    int rc = SSM_OK;
    if (p.tc && tc_gemm_scan_fwd_supported(s.B, s.T, s.H, s.P)) {
        {   // projection and scan in one kernel: x = scan(u Bbar^T), Bu stays on chip
            StageTimer tm("gemm_Bu_scan_fwd", st);
            GemmScanFwd g{u, at<void>(ws, p.W0), s.B, s.T, s.H, s.P, at<float2>(ws, p.Abar), done, (const float2*)x0,
                          at<void>(ws, p.xs), (float2*)xT, hdr};
            if ((rc = launch_gemm_scan_fwd(g, st))) return rc;
        }
        {   // y[m,h] = sum_k x[m,k] Cp[h,k] + D[h] u[m,h]
            StageTimer tm("gemm_y", st);
            GemmTcTN g{at<void>(ws, p.xs), at<void>(ws, p.W2), BT, s.H, P2, false, false, y, D, u, hdr};
            if ((rc = launch_gemm_tc_tn(g, st))) return rc;
        }
    } else if (p.tc) {
        {   // Bu[m, 2p+c] = sum_h u[m,h] Bbar_c[p,h]     (weights as hi + lo bf16)
            StageTimer tm("gemm_Bu", st);
            GemmTcTN g{u, at<void>(ws, p.W0), BT, P2, s.H, true, true, at<void>(ws, p.f32buf), nullptr, nullptr, hdr};
            if ((rc = launch_gemm_tc_tn(g, st))) return rc;
        }
        {
            StageTimer tm("scan_fwd", st);
            rc = launch_scan_fwd(s.B, s.T, s.P, at<float2>(ws, p.Abar), at<float2>(ws, p.Alo), at<float2>(ws, p.f32buf), done,
                                 (const float2*)x0, at<void>(ws, p.xs), true, (float2*)xT, hdr,
                                 at<char>(ws, p.scan), st);
            if (rc) return rc;
        }
        {   // y[m,h] = sum_k x[m,k] Cp[h,k] + D[h] u[m,h]
            StageTimer tm("gemm_y", st);
            GemmTcTN g{at<void>(ws, p.xs), at<void>(ws, p.W2), BT, s.H, P2, false, false, y, D, u, hdr};
            if ((rc = launch_gemm_tc_tn(g, st))) return rc;
        }
    } else if (p.planes) {
        {   // Bu = u Bbar^T as a sum of plane products (u: three planes of an fp32 input, or the bf16 input itself)
            StageTimer tm("gemm_Bu", st);
            if (!io.u_bf16) launch_split_planes((const float*)u, (size_t)BT, s.H, at<void>(ws, p.u3), st);
            GemmTcTN g{io.u_bf16 ? u : at<void>(ws, p.u3), at<void>(ws, p.W0), BT, P2, s.H, false, true, at<void>(ws, p.xs),
                       nullptr, nullptr, hdr};
            g.n_products = io.u_bf16 ? 3 : 6;
            g.planes_a = io.u_bf16 ? 1 : 3;
            g.planes_w = 3;
            g.prod_a = io.u_bf16 ? kProd3A : kProd6A;
            g.prod_w = io.u_bf16 ? kProd3B : kProd6B;
            if ((rc = launch_gemm_tc_tn(g, st))) return rc;
        }
        {
            StageTimer tm("scan_fwd", st);
            rc = launch_scan_fwd(s.B, s.T, s.P, at<float2>(ws, p.Abar), at<float2>(ws, p.Alo), at<float2>(ws, p.xs), done,
                                 (const float2*)x0, at<void>(ws, p.xs), false, (float2*)xT, hdr,
                                 at<char>(ws, p.scan), st);
            if (rc) return rc;
        }
        {   // y = x Cp^T + D u: planes of x, six products, then the skip term
            StageTimer tm("gemm_y", st);
            launch_split_planes(at<float>(ws, p.xs), (size_t)BT, P2, at<void>(ws, p.x3), st);
            GemmTcTN g{at<void>(ws, p.x3), at<void>(ws, p.W2), BT, s.H, P2, false, true, at<void>(ws, p.acc), nullptr,
                       nullptr, hdr};
            g.n_products = 6;
            g.planes_a = 3;
            g.planes_w = 3;
            g.prod_a = kProd6A;
            g.prod_w = kProd6B;
            if ((rc = launch_gemm_tc_tn(g, st))) return rc;
            launch_diag_skip(at<float>(ws, p.acc), D, u, io.u_bf16, nullptr, (size_t)BT, s.H, y, io.y_bf16, st);
        }
    } else {
        {
            StageTimer tm("gemm_Bu", st);
            GemmTN g1{u, io.u_bf16, s.H, at<void>(ws, p.W0), false, s.H, BT, P2, s.H, Epi::StoreF32,
                      at<void>(ws, p.xs), false, nullptr, nullptr, false, nullptr};
            launch_gemm_tn(g1, st);
        }
        {
            StageTimer tm("scan_fwd", st);
            rc = launch_scan_fwd(s.B, s.T, s.P, at<float2>(ws, p.Abar), at<float2>(ws, p.Alo), at<float2>(ws, p.xs), done,
                                 (const float2*)x0, at<void>(ws, p.xs), false, (float2*)xT, hdr,
                                 at<char>(ws, p.scan), st);
            if (rc) return rc;
        }
        {
            StageTimer tm("gemm_y", st);
            GemmTN g2{at<void>(ws, p.xs), false, P2, at<void>(ws, p.W2), false, P2, BT, s.H, P2, Epi::AddDiagIo,
                      y, io.y_bf16, D, u, io.u_bf16, nullptr};
            launch_gemm_tn(g2, st);
        }
    }
    SSM_RETURN_IF_CUDA_ERROR();
    return SSM_OK;
}

static int layer_fwd_impl(const ssm_shape& s, const LayerPlan& p, const LayerIo& io, const ssm_c64* Lambda,
                          const float* Delta, const ssm_c64* Bc, const ssm_c64* Cc, const float* D, const void* u,
                          const uint8_t* done, const ssm_c64* x0, void* y, ssm_c64* xT, void* ws, WsHeader* hdr,
                          cudaStream_t st) {
    layer_prepare(s, p, Lambda, Delta, Bc, Cc, ws, st);
    return layer_fwd_run(s, p, io, D, u, done, x0, y, xT, ws, hdr, st);
}

SSM_API int ssm_layer_fwd(const ssm_shape* shape, const ssm_c64* Lambda, const float* Delta, const ssm_c64* Bc,
                          const ssm_c64* Cc, const float* D, const void* u, const uint8_t* done,
                          const ssm_c64* x0, void* y, ssm_c64* xT, void* ws, size_t ws_bytes, void* stream) {
    if (int rc = check_shape(shape)) return rc;
    if (!Lambda || !Delta || !Bc || !Cc || !D || !u || !y) return SSM_ERR_NULL;
    if (misaligned(Lambda) || misaligned(Delta) || misaligned(Bc) || misaligned(Cc) || misaligned(D) ||
        misaligned(u) || misaligned(y) || misaligned(x0) || misaligned(xT))
        return SSM_ERR_ALIGN;
    const ssm_shape& s = *shape;
    const LayerPlan p = plan_layer(s);
    if (int rc = check_ws(ws, ws_bytes, p.total)) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    WsHeader* hdr = at<WsHeader>(ws, p.hdr);
    if (cudaMemsetAsync(ws, 0, sizeof(WsHeader), st) != cudaSuccess) return SSM_ERR_CUDA;
    return layer_fwd_impl(s, p, layer_io(s), Lambda, Delta, Bc, Cc, D, u, done, x0, y, xT, ws, hdr, st);
}

// Single-step mode: the layer's forward launch sequence for T = 1 from operands prepared once.
static ssm_shape step_shape(const ssm_shape& s) {
    ssm_shape t = s;
    t.T = 1;
    return t;
}

SSM_API size_t ssm_step_workspace_bytes(const ssm_shape* shape) {
    if (check_shape(shape) != SSM_OK) return 0;
    return plan_layer(step_shape(*shape)).total;
}

SSM_API int ssm_step_prepare(const ssm_shape* shape, const ssm_c64* Lambda, const float* Delta, const ssm_c64* Bc,
                             const ssm_c64* Cc, void* ws, size_t ws_bytes, void* stream) {
    if (int rc = check_shape(shape)) return rc;
    if (!Lambda || !Delta || !Bc || !Cc) return SSM_ERR_NULL;
    if (misaligned(Lambda) || misaligned(Delta) || misaligned(Bc) || misaligned(Cc)) return SSM_ERR_ALIGN;
    const ssm_shape s = step_shape(*shape);
    const LayerPlan p = plan_layer(s);
    if (int rc = check_ws(ws, ws_bytes, p.total)) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(ws, 0, sizeof(WsHeader), st) != cudaSuccess) return SSM_ERR_CUDA;
    layer_prepare(s, p, Lambda, Delta, Bc, Cc, ws, st);
    SSM_RETURN_IF_CUDA_ERROR();
    return SSM_OK;
}

SSM_API int ssm_step(const ssm_shape* shape, const float* D, const void* u, const uint8_t* done,
                     const ssm_c64* x_prev, ssm_c64* x_next, void* y, void* ws, size_t ws_bytes, void* stream) {
    if (int rc = check_shape(shape)) return rc;
    if (!D || !u || !x_prev || !x_next || !y) return SSM_ERR_NULL;
    if (misaligned(D) || misaligned(u) || misaligned(x_prev) || misaligned(x_next) || misaligned(y))
        return SSM_ERR_ALIGN;
    const ssm_shape s = step_shape(*shape);
    const LayerPlan p = plan_layer(s);
    if (int rc = check_ws(ws, ws_bytes, p.total)) return rc;
    // each (trajectory, state) is read as x0 and written as xT by the same thread, so x_next may be x_prev
    return layer_fwd_run(s, p, layer_io(s), D, u, done, x_prev, y, x_next, ws, at<WsHeader>(ws, p.hdr),
                         (cudaStream_t)stream);
}

// ---- half-GLU gate -----------------------------------------------------------------------
namespace {

struct GluPlan {
    bool tc;
    int splits;
    size_t hdr, Wt, Wn, x1, z, gz, gx1, part, total;
};

GluPlan plan_glu(const ssm_shape& s) {
    GluPlan p{};
    size_t off = 0;
    const size_t M = (size_t)s.B * s.T, HH = (size_t)s.H * s.H;
    p.tc = s.io_dtype == SSM_BF16 && tc_tn_supported((int)M, s.H, 2 * s.H, true) &&
           tc_tn_supported((int)M, s.H, s.H, true) && tc_nt_supported(s.H, s.H);
    p.splits = p.tc ? tc_nt_splits((int)M, s.H, s.H) : gemm_nt_splits((int)M);
    p.hdr = take(off, sizeof(WsHeader));
    p.Wt = take(off, p.tc ? 4 * HH * 2 : HH * 4);   // tc: hi/lo stacked bf16 [2H, 2H]; else W^T fp32
    p.Wn = take(off, p.tc ? 2 * HH * 2 : 0);
    p.x1 = take(off, M * s.H * 4);                  // GELU(v): fp32, or two bf16 planes
    p.z = take(off, M * s.H * 4);                   // the gate's argument
    p.gz = take(off, M * s.H * 4);                  // fp32, or two bf16 planes
    p.gx1 = take(off, M * s.H * 4);
    p.part = take(off, (size_t)2 * p.splits * HH * 4);
    p.total = off;
    return p;
}

}  // namespace

SSM_API size_t ssm_glu_workspace_bytes(const ssm_shape* shape) {
    if (check_shape(shape) != SSM_OK) return 0;
    return plan_glu(*shape).total;
}

SSM_API int ssm_glu_fwd(const ssm_shape* shape, const float* W, const void* v, void* out, void* ws, size_t ws_bytes,
                        void* stream) {
    if (int rc = check_shape(shape)) return rc;
    if (!W || !v || !out) return SSM_ERR_NULL;
    if (misaligned(W) || misaligned(v) || misaligned(out)) return SSM_ERR_ALIGN;
    const ssm_shape& s = *shape;
    const GluPlan p = plan_glu(s);
    if (int rc = check_ws(ws, ws_bytes, p.total)) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    const bool bf16 = s.io_dtype == SSM_BF16;
    const int M = s.B * s.T;
    const size_t n = (size_t)M * s.H;
    WsHeader* hdr = at<WsHeader>(ws, p.hdr);
    const bool fused_gate = p.tc && tc_tn_gate_supported(M, s.H, 2 * s.H);
    if (cudaMemsetAsync(ws, 0, sizeof(WsHeader), st) != cudaSuccess) return SSM_ERR_CUDA;
    {
        StageTimer tm("glu_pack_gelu", st);
        launch_glu_pack(s.H, W, p.tc ? at<void>(ws, p.Wt) : nullptr, p.tc ? at<void>(ws, p.Wn) : nullptr,
                        p.tc ? nullptr : at<float>(ws, p.Wt), st);
        launch_glu_gelu(bf16, p.tc, n, s.H, v, at<void>(ws, p.x1), st);
    }
    {   // z[m, j] = sum_i x1[m, i] W[i, j]
        StageTimer tm("glu_gemm_z", st);
        if (p.tc) {
            // both planes of x1 along K: a single bf16 rounding of x1 here costs 2e-2 on dW
            GemmTcTN g{at<void>(ws, p.x1), at<void>(ws, p.Wt), M, s.H, 2 * s.H, true, true, at<void>(ws, p.z), nullptr, nullptr, hdr};
            if (fused_gate) {   // out = v * sigmoid(z) leaves from the same epilogue
                g.skip = v;
                g.gate_out = out;
            }
            if (int rc = launch_gemm_tc_tn(g, st)) return rc;
        } else {
            GemmTN g{at<void>(ws, p.x1), false, s.H, at<void>(ws, p.Wt), false, s.H, M, s.H, s.H, Epi::StoreF32,
                     at<void>(ws, p.z), false, nullptr, nullptr, false, nullptr};
            launch_gemm_tn(g, st);
        }
    }
    if (!fused_gate) {
        StageTimer tm("glu_out", st);
        launch_glu_out(bf16, n, v, at<float>(ws, p.z), out, st);
    }
    SSM_RETURN_IF_CUDA_ERROR();
    return SSM_OK;
}

SSM_API int ssm_glu_bwd(const ssm_shape* shape, const float* W, const void* v, const void* gout, void* ws,
                        size_t ws_bytes, void* gv, float* dW, void* stream) {
    if (int rc = check_shape(shape)) return rc;
    if (!W || !v || !gout || !gv || !dW) return SSM_ERR_NULL;
    if (misaligned(W) || misaligned(v) || misaligned(gout) || misaligned(gv) || misaligned(dW)) return SSM_ERR_ALIGN;
    const ssm_shape& s = *shape;
    const GluPlan p = plan_glu(s);
    if (int rc = check_ws(ws, ws_bytes, p.total)) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    const bool bf16 = s.io_dtype == SSM_BF16;
    const int M = s.B * s.T;
    const size_t n = (size_t)M * s.H, HH = (size_t)s.H * s.H;
    WsHeader* hdr = at<WsHeader>(ws, p.hdr);
    {
        StageTimer tm("glu_gz", st);
        launch_glu_gz(bf16, p.tc, n, v, gout, at<float>(ws, p.z), at<void>(ws, p.gz), st);
    }
    {   // g_x1[m, i] = sum_j gz[m, j] W[i, j]
        StageTimer tm("glu_gemm_gx1", st);
        if (p.tc) {
            GemmTcTN g{at<void>(ws, p.gz), at<void>(ws, p.Wn), M, s.H, s.H, true, true, at<void>(ws, p.gx1), nullptr, nullptr, hdr};
            if (int rc = launch_gemm_tc_tn(g, st)) return rc;
        } else {
            GemmTN g{at<void>(ws, p.gz), false, s.H, W, false, s.H, M, s.H, s.H, Epi::StoreF32,
                     at<void>(ws, p.gx1), false, nullptr, nullptr, false, nullptr};
            launch_gemm_tn(g, st);
        }
    }
    {   // dW[i, j] = sum_m x1[m, i] gz[m, j]
        StageTimer tm("glu_gemm_dW", st);
        if (p.tc) {
            // (x1_hi + x1_lo)^T (gz_hi + gz_lo) as two products, one per plane of x1
            GemmTcNT g{at<void>(ws, p.x1), s.H, at<void>(ws, p.gz), at<void>(ws, p.gz + n * 2), s.H, M, p.splits,
                       at<float>(ws, p.part), hdr, 2 * s.H};
            if (int rc = launch_gemm_tc_nt(g, st)) return rc;
            g.A = at<void>(ws, p.x1 + (size_t)s.H * 2);   // the low halves: columns [H, 2H) of x1
            g.part = at<float>(ws, p.part) + (size_t)p.splits * HH;
            if (int rc = launch_gemm_tc_nt(g, st)) return rc;
            launch_glu_reduce(at<float>(ws, p.part), 2 * p.splits, HH, dW, st);
        } else {
            GemmNT g{at<void>(ws, p.x1), false, s.H, at<void>(ws, p.gz), false, s.H, M, p.splits, at<float>(ws, p.part)};
            launch_gemm_nt(g, st);
            launch_glu_reduce(at<float>(ws, p.part), p.splits, HH, dW, st);
        }
    }
    {
        StageTimer tm("glu_gv", st);
        launch_glu_gv(bf16, n, v, gout, at<float>(ws, p.z), at<float>(ws, p.gx1), gv, st);
    }
    SSM_RETURN_IF_CUDA_ERROR();
    return SSM_OK;
}

// Launch sequence of one layer's backward pass.  du_add (fp32 [B,T,H], may be NULL) is added to du
// before it is stored (the gradient of the residual branch of a stacked model).
static int layer_bwd_impl(const ssm_shape& s, const LayerPlan& p, const LayerIo& io, const ssm_c64* Lambda,
                          const float* Delta, const ssm_c64* Bc, const float* D, const void* u, const uint8_t* done,
                          const ssm_c64* x0, const void* gy, const ssm_c64* gxT, const float* du_add, void* ws,
                          WsHeader* hdr, void* du, ssm_c64* dLambda, float* dDelta, ssm_c64* dB, ssm_c64* dC, float* dD,
                          ssm_c64* dx0, cudaStream_t st) {
    const int BT = s.B * s.T, P2 = 2 * s.P;
    if (p.tc && !(io.u_bf16 && io.gy_bf16 && io.du_bf16)) return SSM_ERR_DTYPE;
    float* part = at<float>(ws, p.part);                       // split-K partials of gBbar ...
    float* part_c = part + (size_t)p.splits * 2 * s.P * s.H;   // ... and of dC
    const size_t plane = (size_t)BT * s.P * 4;   // bytes of one bf16 plane of a state tensor
    int rc = SSM_OK;
    // The last sums (gAbar over the sequences, dD over row groups, the two split-K sums) are left to the two
    // kernels at the end of the pass: what the stages leave are rows of partial sums.
    const float2* gA_part = nullptr;
    const float* dD_part = nullptr;
    int gA_rows = 0, dD_rows = 0;

    if (p.tc) {
        if (tc_gemm_scan_bwd_supported(s.B, s.T, s.H, s.P)) {
            // projection and reverse scan in one kernel: s = reverse scan(gy conj(C)), g_x stays on chip
            StageTimer tm("gemm_gx_scan_bwd", st);
            GemmScanBwd g{gy, at<void>(ws, p.W1), s.B, s.T, s.H, s.P, at<float2>(ws, p.Abar), done, (const float2*)x0,
                          (const float2*)gxT, at<void>(ws, p.xs), at<void>(ws, p.gs), nullptr, (float2*)dx0, hdr};
            if ((rc = launch_gemm_scan_bwd_part(g, at<char>(ws, p.scan), &gA_part, &gA_rows, st))) return rc;
        } else {
            {   // gx[m, 2p+c] = sum_h gy[m,h] conj(C)_c[h,p]   (weights as hi + lo bf16)
                StageTimer tm("gemm_gx", st);
                GemmTcTN g{gy, at<void>(ws, p.W1), BT, P2, s.H, true, true, at<void>(ws, p.f32buf), nullptr, nullptr, hdr};
                if ((rc = launch_gemm_tc_tn(g, st))) return rc;
            }
            {
                StageTimer tm("scan_bwd", st);
                rc = launch_scan_bwd(s.B, s.T, s.P, at<float2>(ws, p.Abar), at<float2>(ws, p.Alo), done,
                                     (const float2*)x0, at<void>(ws, p.xs), true, at<float2>(ws, p.f32buf),
                                     (const float2*)gxT, at<void>(ws, p.gs), true, at<float2>(ws, p.gAbar), (float2*)dx0,
                                     hdr, at<char>(ws, p.scan), st, &gA_part, &gA_rows);
                if (rc) return rc;
            }
        }
        {   // du[m,h] = sum_k s[m,k] Bq[h,k] + D[h] gy[m,h];  where the kernel can, also dD[h] = sum_m gy[m,h] u[m,h]
            // from the tiles of gy its epilogue holds anyway (one more operand tile, u, beside each)
            StageTimer tm("gemm_du", st);
            if (du_add) return SSM_ERR_SHAPE;   // the residual addend exists only on the CUDA-core path (stacks)
            GemmTcTN g{at<void>(ws, p.gs), at<void>(ws, p.W3), BT, s.H, P2, false, false, du, D, gy, hdr};
            int rows = 0;
            if (tc_tn_dot_supported(BT, s.H, P2)) {
                g.dot = u;
                g.dot_part = at<float>(ws, p.dot);
                g.dot_rows = &rows;
            }
            if ((rc = launch_gemm_tc_tn(g, st))) return rc;
            if (g.dot) {
                dD_part = at<float>(ws, p.dot);
                dD_rows = rows;
            }
        }
        {   // gBbar[p,h] = sum_m s[m,p] u[m,h]
            StageTimer tm("gemm_gBbar", st);
            GemmTcNT g{u, s.H, at<void>(ws, p.gs), at<void>(ws, p.gs + plane), P2, BT, p.splits, part, hdr};
            if ((rc = launch_gemm_tc_nt(g, st))) return rc;
        }
        {   // dC[h,p] = sum_m gy[m,h] conj(x[m,p])
            StageTimer tm("gemm_gC", st);
            GemmTcNT g{gy, s.H, at<void>(ws, p.xs), at<void>(ws, p.xs + plane), P2, BT, p.splits, part_c, hdr};
            if ((rc = launch_gemm_tc_nt(g, st))) return rc;
        }
    } else if (p.planes) {
        const bool gyb = io.gy_bf16, ub = io.u_bf16;
        {   // g_x = gy conj(C)
            StageTimer tm("gemm_gx", st);
            if (!gyb) launch_split_planes((const float*)gy, (size_t)BT, s.H, at<void>(ws, p.gy3), st);
            GemmTcTN g{gyb ? gy : at<void>(ws, p.gy3), at<void>(ws, p.W1), BT, P2, s.H, false, true, at<void>(ws, p.gs),
                       nullptr, nullptr, hdr};
            g.n_products = gyb ? 3 : 6;
            g.planes_a = gyb ? 1 : 3;
            g.planes_w = 3;
            g.prod_a = gyb ? kProd3A : kProd6A;
            g.prod_w = gyb ? kProd3B : kProd6B;
            if ((rc = launch_gemm_tc_tn(g, st))) return rc;
        }
        {
            StageTimer tm("scan_bwd", st);
            rc = launch_scan_bwd(s.B, s.T, s.P, at<float2>(ws, p.Abar), at<float2>(ws, p.Alo), done, (const float2*)x0,
                                 at<void>(ws, p.xs), false, at<float2>(ws, p.gs), (const float2*)gxT,
                                 at<void>(ws, p.gs), false, at<float2>(ws, p.gAbar), (float2*)dx0, hdr,
                                 at<char>(ws, p.scan), st, &gA_part, &gA_rows);
            if (rc) return rc;
        }
        {   // du = s Bq^T + D gy (+ the residual branch's gradient)
            StageTimer tm("gemm_du", st);
            launch_split_planes(at<float>(ws, p.gs), (size_t)BT, P2, at<void>(ws, p.s3), st);
            GemmTcTN g{at<void>(ws, p.s3), at<void>(ws, p.W3), BT, s.H, P2, false, true, at<void>(ws, p.acc), nullptr,
                       nullptr, hdr};
            g.n_products = 6;
            g.planes_a = 3;
            g.planes_w = 3;
            g.prod_a = kProd6A;
            g.prod_w = kProd6B;
            if ((rc = launch_gemm_tc_tn(g, st))) return rc;
            launch_diag_skip(at<float>(ws, p.acc), D, gy, gyb, du_add, (size_t)BT, s.H, du, io.du_bf16, st);
        }
        {   // gBbar = s^T u
            StageTimer tm("gemm_gBbar", st);
            GemmTcNT g{ub ? u : at<void>(ws, p.u3), s.H, at<void>(ws, p.s3), nullptr, P2, BT, p.splits, part, hdr};
            g.n_products = ub ? 3 : 6;
            g.planes_a = ub ? 1 : 3;
            g.planes_b = 3;
            g.prod_a = ub ? kProd3A : kProd6A;
            g.prod_b = ub ? kProd3B : kProd6B;
            if ((rc = launch_gemm_tc_nt(g, st))) return rc;
        }
        {   // dC = gy^T conj(x)
            StageTimer tm("gemm_gC", st);
            GemmTcNT g{gyb ? gy : at<void>(ws, p.gy3), s.H, at<void>(ws, p.x3), nullptr, P2, BT, p.splits, part_c, hdr};
            g.n_products = gyb ? 3 : 6;
            g.planes_a = gyb ? 1 : 3;
            g.planes_b = 3;
            g.prod_a = gyb ? kProd3A : kProd6A;
            g.prod_b = gyb ? kProd3B : kProd6B;
            if ((rc = launch_gemm_tc_nt(g, st))) return rc;
        }
    } else {
        {
            StageTimer tm("gemm_gx", st);
            GemmTN g3{gy, io.gy_bf16, s.H, at<void>(ws, p.W1), false, s.H, BT, P2, s.H, Epi::StoreF32,
                      at<void>(ws, p.gs), false, nullptr, nullptr, false, nullptr};
            launch_gemm_tn(g3, st);
        }
        {
            StageTimer tm("scan_bwd", st);
            rc = launch_scan_bwd(s.B, s.T, s.P, at<float2>(ws, p.Abar), at<float2>(ws, p.Alo), done, (const float2*)x0,
                                 at<void>(ws, p.xs), false, at<float2>(ws, p.gs), (const float2*)gxT,
                                 at<void>(ws, p.gs), false, at<float2>(ws, p.gAbar), (float2*)dx0, hdr,
                                 at<char>(ws, p.scan), st, &gA_part, &gA_rows);
            if (rc) return rc;
        }
        {
            StageTimer tm("gemm_du", st);
            GemmTN g4{at<void>(ws, p.gs), false, P2, at<void>(ws, p.W3), false, P2, BT, s.H, P2, Epi::AddDiagIo,
                      du, io.du_bf16, D, gy, io.gy_bf16, du_add};
            launch_gemm_tn(g4, st);
        }
        {
            StageTimer tm("gemm_gBbar", st);
            GemmNT g5{u, io.u_bf16, s.H, at<void>(ws, p.gs), false, P2, BT, p.splits, part};
            launch_gemm_nt(g5, st);
        }
        {
            StageTimer tm("gemm_gC", st);
            GemmNT g6{gy, io.gy_bf16, s.H, at<void>(ws, p.xs), false, P2, BT, p.splits, part_c};
            launch_gemm_nt(g6, st);
        }
    }
    {   // dD[h] = sum_m gy[m,h] u[m,h] (unless the du projection left its partial sums already), the two split-K
        // sums, then the adjoint of the discretisation with the sums of gAbar and dD folded in
        StageTimer tm("gD_and_discretize_bwd", st);
        if (!dD_part) {
            float* tmp = at<float>(ws, p.dot);
            int groups = launch_dot_columns_partial(io.gy_bf16, gy, io.u_bf16, u, BT, s.H, tmp, st);
            dD_part = launch_reduce_rows(tmp, groups, s.H, tmp + (size_t)groups * s.H, kMaxPartialRows, &dD_rows, st);
        }
        launch_splitk_reduce2(part, part_c, p.splits, s.H, P2, at<float2>(ws, p.gBbar), (float2*)dC, st);
        launch_layer_finalize(s.H, s.P, (const float2*)Lambda, Delta, (const float2*)Bc, gA_part, gA_rows,
                              at<float2>(ws, p.gBbar), (float2*)dLambda, dDelta, (float2*)dB, dD_part, dD_rows, dD, st);
    }
    SSM_RETURN_IF_CUDA_ERROR();
    return SSM_OK;
}

SSM_API int ssm_layer_bwd(const ssm_shape* shape, const ssm_c64* Lambda, const float* Delta, const ssm_c64* Bc,
                          const ssm_c64* Cc, const float* D, const void* u, const uint8_t* done,
                          const ssm_c64* x0, const void* gy, const ssm_c64* gxT, void* ws, size_t ws_bytes,
                          void* du, ssm_c64* dLambda, float* dDelta, ssm_c64* dB, ssm_c64* dC, float* dD,
                          ssm_c64* dx0, void* stream) {
    if (int rc = check_shape(shape)) return rc;
    if (!Lambda || !Delta || !Bc || !Cc || !D || !u || !gy || !du || !dLambda || !dDelta || !dB || !dC || !dD)
        return SSM_ERR_NULL;
    if (misaligned(Lambda) || misaligned(Delta) || misaligned(Bc) || misaligned(Cc) || misaligned(D) ||
        misaligned(u) || misaligned(gy) || misaligned(du) || misaligned(dLambda) || misaligned(dDelta) ||
        misaligned(dB) || misaligned(dC) || misaligned(dD) || misaligned(x0) || misaligned(gxT) || misaligned(dx0))
        return SSM_ERR_ALIGN;
    const ssm_shape& s = *shape;
    const LayerPlan p = plan_layer(s);
    if (int rc = check_ws(ws, ws_bytes, p.total)) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    WsHeader* hdr = at<WsHeader>(ws, p.hdr);
    return layer_bwd_impl(s, p, layer_io(s), Lambda, Delta, Bc, D, u, done, x0, gy, gxT, nullptr, ws, hdr, du, dLambda,
                          dDelta, dB, dC, dD, dx0, st);
}

// ---- stacked model -----------------------------------------------------------------------------
namespace {

// Storage inside a stack.  Only the stack's input u, its output, gout and du are in the I/O type.
// Everything that passes between the layers (the SSM outputs v, the layer inputs, the gradients
// handed from a layer to the one below) is fp32: stored in bf16, a value that rounds to the other
// neighbour than in an exact evaluation is a legitimate difference between two correct runs, and the
// layers that follow amplify such differences in the parameter-gradient sums beyond the tolerance of
// the I/O type.  The layers therefore run with fp32 inputs and outputs (except for the first layer's
// input and the last gradient), on the fp32 path of the layer.
struct StackPlan {
    size_t layer_ws;   // bytes of one layer workspace
    size_t act;        // bytes of one fp32 [B,T,H] tensor
    size_t hdr, layers, acts, vs, stats, gz, gv, g0, g1, tmp, total;
};

ssm_shape stack_layer_shape(const ssm_shape& s) {
    ssm_shape t = s;
    t.io_dtype = SSM_F32;
    return t;
}

StackPlan plan_stack(const ssm_shape& s, int L) {
    StackPlan p{};
    size_t off = 0;
    const size_t BT = (size_t)s.B * s.T;
    p.layer_ws = align_up(plan_layer(stack_layer_shape(s), false).total, 256);
    p.act = align_up(BT * s.H * 4, 256);
    p.hdr = take(off, sizeof(WsHeader));
    p.layers = take(off, p.layer_ws * L);
    p.acts = take(off, p.act * (L > 1 ? L - 1 : 0));   // inputs of layers 1 .. L-1
    p.vs = take(off, p.act * L);                       // SSM outputs
    p.stats = take(off, align_up(BT * 4, 256) * 2 * L);   // mean and 1/std of every row, per layer
    p.gz = take(off, p.act);
    p.gv = take(off, p.act);
    p.g0 = take(off, p.act);
    p.g1 = take(off, p.act);
    p.tmp = take(off, stack_tmp_floats((int)BT, s.H) * 4);
    p.total = off;
    return p;
}

int check_stack_args(const ssm_shape* shape, int n_layers, const ssm_stack_params* params) {
    if (int rc = check_shape(shape)) return rc;
    if (n_layers < 1 || n_layers > 64) return SSM_ERR_SHAPE;
    if (!params) return SSM_ERR_NULL;
    for (int l = 0; l < n_layers; ++l) {
        const ssm_stack_params& q = params[l];
        if (!q.Lambda || !q.Delta || !q.Bc || !q.Cc || !q.D || !q.ln_weight || !q.ln_bias) return SSM_ERR_NULL;
        if (misaligned(q.Lambda) || misaligned(q.Delta) || misaligned(q.Bc) || misaligned(q.Cc) || misaligned(q.D) ||
            misaligned(q.ln_weight) || misaligned(q.ln_bias))
            return SSM_ERR_ALIGN;
    }
    return SSM_OK;
}

}  // namespace

SSM_API size_t ssm_stack_workspace_bytes(const ssm_shape* shape, int n_layers) {
    if (check_shape(shape) != SSM_OK || n_layers < 1 || n_layers > 64) return 0;
    return plan_stack(*shape, n_layers).total;
}

SSM_API int ssm_stack_fwd(const ssm_shape* shape, int n_layers, const ssm_stack_params* params, const void* u,
                          const uint8_t* done, void* out, void* ws, size_t ws_bytes, void* stream) {
    if (int rc = check_stack_args(shape, n_layers, params)) return rc;
    if (!u || !out) return SSM_ERR_NULL;
    if (misaligned(u) || misaligned(out)) return SSM_ERR_ALIGN;
    const ssm_shape& s = *shape;
    const StackPlan sp = plan_stack(s, n_layers);
    if (int rc = check_ws(ws, ws_bytes, sp.total)) return rc;
    const ssm_shape ls = stack_layer_shape(s);
    const LayerPlan lp = plan_layer(ls, false);
    cudaStream_t st = (cudaStream_t)stream;
    const bool bf16 = s.io_dtype == SSM_BF16;
    const int BT = s.B * s.T;
    const size_t stat = align_up((size_t)BT * 4, 256);
    WsHeader* hdr = at<WsHeader>(ws, sp.hdr);
    if (cudaMemsetAsync(ws, 0, sizeof(WsHeader), st) != cudaSuccess) return SSM_ERR_CUDA;
    const void* in = u;
    for (int l = 0; l < n_layers; ++l) {
        const ssm_stack_params& q = params[l];
        const bool first = l == 0, last = l == n_layers - 1;
        void* lws = at<void>(ws, sp.layers + sp.layer_ws * l);
        float* v = at<float>(ws, sp.vs + sp.act * l);
        void* o = last ? out : at<void>(ws, sp.acts + sp.act * l);
        const LayerIo io{first && bf16, false, false, false};
        if (int rc = layer_fwd_impl(ls, lp, io, q.Lambda, q.Delta, q.Bc, q.Cc, q.D, in, done, nullptr, v, nullptr, lws, hdr, st))
            return rc;
        StageTimer tm("stack_gelu_ln_fwd", st);
        launch_stack_fwd(first && bf16, last && bf16, BT, s.H, in, v, q.ln_weight, q.ln_bias, o,
                         at<float>(ws, sp.stats + stat * (2 * l)), at<float>(ws, sp.stats + stat * (2 * l + 1)), st);
        in = o;
    }
    SSM_RETURN_IF_CUDA_ERROR();
    return SSM_OK;
}

SSM_API int ssm_stack_bwd(const ssm_shape* shape, int n_layers, const ssm_stack_params* params, const void* u,
                          const uint8_t* done, const void* gout, void* ws, size_t ws_bytes, void* du,
                          const ssm_stack_grads* grads, void* stream) {
    if (int rc = check_stack_args(shape, n_layers, params)) return rc;
    if (!u || !gout || !du || !grads) return SSM_ERR_NULL;
    if (misaligned(u) || misaligned(gout) || misaligned(du)) return SSM_ERR_ALIGN;
    for (int l = 0; l < n_layers; ++l) {
        const ssm_stack_grads& g = grads[l];
        if (!g.dLambda || !g.dDelta || !g.dB || !g.dC || !g.dD || !g.dln_weight || !g.dln_bias) return SSM_ERR_NULL;
        if (misaligned(g.dLambda) || misaligned(g.dDelta) || misaligned(g.dB) || misaligned(g.dC) || misaligned(g.dD) ||
            misaligned(g.dln_weight) || misaligned(g.dln_bias))
            return SSM_ERR_ALIGN;
    }
    const ssm_shape& s = *shape;
    const StackPlan sp = plan_stack(s, n_layers);
    if (int rc = check_ws(ws, ws_bytes, sp.total)) return rc;
    const ssm_shape ls = stack_layer_shape(s);
    const LayerPlan lp = plan_layer(ls, false);
    cudaStream_t st = (cudaStream_t)stream;
    const bool bf16 = s.io_dtype == SSM_BF16;
    const int BT = s.B * s.T;
    const size_t stat = align_up((size_t)BT * 4, 256);
    WsHeader* hdr = at<WsHeader>(ws, sp.hdr);
    const void* g = gout;
    for (int l = n_layers - 1; l >= 0; --l) {
        const ssm_stack_params& q = params[l];
        const ssm_stack_grads& gr = grads[l];
        const bool first = l == 0, top = l == n_layers - 1;
        void* lws = at<void>(ws, sp.layers + sp.layer_ws * l);
        const void* in = first ? u : at<void>(ws, sp.acts + sp.act * (l - 1));
        const float* v = at<float>(ws, sp.vs + sp.act * l);
        void* gnext = first ? du : at<void>(ws, (l & 1) ? sp.g1 : sp.g0);
        {
            StageTimer tm("stack_gelu_ln_bwd", st);
            launch_stack_bwd(top && bf16, first && bf16, BT, s.H, g, in, v, q.ln_weight,
                             at<float>(ws, sp.stats + stat * (2 * l)), at<float>(ws, sp.stats + stat * (2 * l + 1)),
                             at<float>(ws, sp.gz), at<float>(ws, sp.gv), gr.dln_weight, gr.dln_bias, at<float>(ws, sp.tmp), st);
        }
        // the gradient handed down: gz (residual branch) + du of the SSM, summed in fp32 in the du epilogue
        const LayerIo io{first && bf16, false, false, first && bf16};
        if (int rc = layer_bwd_impl(ls, lp, io, q.Lambda, q.Delta, q.Bc, q.D, in, done, nullptr, at<void>(ws, sp.gv), nullptr,
                                    at<float>(ws, sp.gz), lws, hdr, gnext, gr.dLambda, gr.dDelta, gr.dB, gr.dC, gr.dD,
                                    nullptr, st))
            return rc;
        g = gnext;
    }
    SSM_RETURN_IF_CUDA_ERROR();
    return SSM_OK;
}
