// ssm_scan_bwd_static: the reverse scan for callers that cannot hand the library a scratch
// buffer because they are not allowed to allocate device memory at that point (see ssm.h).
// It is ssm_scan_bwd with its scratch taken from a fixed array that lives in this library's
// device image instead of from a caller-provided workspace.  The kernels are the same.
#include <mutex>

#include "kernels.h"

using namespace ssm;

#define SSM_API extern "C" __attribute__((visibility("default")))

namespace {

// Scratch shared by every ssm_scan_bwd_static call on a device.  Each GPU that loads the
// library carries this array until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[SSM_STATIC_SCRATCH_BYTES];

// In host code `g_static_scratch` is only a handle for the runtime, not a device address; the
// address a kernel may use comes from cudaGetSymbolAddress, asked once per device with that
// device current.
constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_ptr[kMaxDevices] = {};

int static_scratch_for_current_device(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SSM_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return SSM_ERR_CUDA;
        }
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return SSM_OK;
}

}  // namespace

// The status word of ssm_scan_bwd_static's kernels sits at the start of the static array, which
// the caller has no pointer to: this reads it back (and synchronises `stream`, like ssm_check).
SSM_API int ssm_check_static(void* stream) {
    void* base = nullptr;
    if (int rc = static_scratch_for_current_device(&base)) return rc;
    int status = 0;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemcpyAsync(&status, base, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return SSM_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return SSM_ERR_CUDA;
    return status == 0 ? SSM_OK : SSM_ERR_TIMEOUT;
}

SSM_API int ssm_scan_bwd_static(const ssm_shape* shape, const ssm_c64* Abar, const uint8_t* done,
                                const ssm_c64* x0, const ssm_c64* x, const ssm_c64* gx, const ssm_c64* gxT,
                                ssm_c64* gBu, ssm_c64* gAbar, ssm_c64* gx0, void* stream) {
    if (int rc = check_shape(shape)) return rc;
    if (!Abar || !x || !gx || !gBu || !gAbar) return SSM_ERR_NULL;
    if (misaligned(Abar) || misaligned(x) || misaligned(gx) || misaligned(gBu) || misaligned(gAbar) ||
        misaligned(x0) || misaligned(gxT) || misaligned(gx0))
        return SSM_ERR_ALIGN;
    const size_t need = sizeof(WsHeader) + scan_scratch_bytes(shape->B, shape->T, shape->P);
    if (need > (size_t)SSM_STATIC_SCRATCH_BYTES) return SSM_ERR_TOO_LARGE;
    void* base = nullptr;
    if (int rc = static_scratch_for_current_device(&base)) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    // The array keeps whatever the previous call left; the header (status word) is the part
    // that has to start at zero (the scan zeroes its own work counter).
    if (cudaMemsetAsync(base, 0, sizeof(WsHeader), st) != cudaSuccess) return SSM_ERR_CUDA;
    int rc = launch_scan_bwd(shape->B, shape->T, shape->P, (const float2*)Abar, nullptr, done, (const float2*)x0,
                             (const float2*)x, false, (const float2*)gx, (const float2*)gxT, (float2*)gBu, false,
                             (float2*)gAbar, (float2*)gx0, reinterpret_cast<WsHeader*>(base),
                             reinterpret_cast<char*>(base) + sizeof(WsHeader), st);
    if (rc) return rc;
    SSM_RETURN_IF_CUDA_ERROR();
    return SSM_OK;
}
