// Shared device/host helpers of the S5 SSM library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/ssm.h"

namespace ssm {

// ---- complex arithmetic on float2 ---------------------------------------------------
__device__ __forceinline__ float2 cmul(float2 a, float2 b) {
    return make_float2(a.x * b.x - a.y * b.y, a.x * b.y + a.y * b.x);
}
// a * x + b
__device__ __forceinline__ float2 cfma(float2 a, float2 x, float2 b) {
    return make_float2(fmaf(a.x, x.x, fmaf(-a.y, x.y, b.x)), fmaf(a.x, x.y, fmaf(a.y, x.x, b.y)));
}
__device__ __forceinline__ float2 cconj(float2 a) { return make_float2(a.x, -a.y); }
__device__ __forceinline__ float2 cadd(float2 a, float2 b) { return make_float2(a.x + b.x, a.y + b.y); }

// ---- io element access ----------------------------------------------------------------
template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// ---- workspace header -------------------------------------------------------------------
// First 256 bytes of every workspace.  `status` is written by kernels whose bounded waits
// give up.
struct WsHeader {
    int status;
    int pad[63];
};
static_assert(sizeof(WsHeader) == 256, "header is one 256-byte line group");

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

inline int check_shape(const ssm_shape* s) {
    if (!s) return SSM_ERR_NULL;
    if (s->B < 1 || s->T < 1 || s->H < 8 || s->P < 8 || (s->H % 8) || (s->P % 8)) return SSM_ERR_SHAPE;
    if ((int64_t)s->B * s->T >= (int64_t)1 << 31) return SSM_ERR_SHAPE;
    if (s->io_dtype != SSM_F32 && s->io_dtype != SSM_BF16) return SSM_ERR_DTYPE;
    if (s->reserved != 0) return SSM_ERR_SHAPE;
    return SSM_OK;
}
inline bool misaligned(const void* p, size_t a = 16) { return (reinterpret_cast<uintptr_t>(p) % a) != 0; }

// Measurement hooks (profile.cu): launch counter and optional per-stage event timing.
void count_launch(int n = 1);
// Number of SMs of the current device, cached per device ordinal (148 where no device answers).
int device_sm_count();
// Raises a kernel's dynamic shared-memory limit, once per (kernel, device) (device_setup.cu).
bool set_max_dynamic_smem(const void* kernel, size_t bytes);
class StageTimer {
  public:
    StageTimer(const char* name, cudaStream_t st);
    ~StageTimer();
  private:
    cudaStream_t st_;
    int idx_;
};

#define SSM_RETURN_IF_CUDA_ERROR()                              \
    do {                                                        \
        if (cudaPeekAtLastError() != cudaSuccess) {             \
            (void)cudaGetLastError();                           \
            return SSM_ERR_CUDA;                                \
        }                                                       \
    } while (0)

}  // namespace ssm
