/*
 * ssm.h - C ABI of the B200 (sm_100a) S5 state-space layer library.
 *
 * The library evaluates, forward and backward, the diagonal complex linear
 * state-space layer that the paper's world model uses as its sequence model
 * (Sec. III-B "State-Space Models", Sec. IV-A "State-Space World Model"):
 *
 *     Abar = exp(Lambda Delta),  Bbar = Lambda^-1 (Abar - 1) B      (zero-order hold)
 *     x_t  = (done_t ? 0 : Abar * x_{t-1}) + Bbar u_t ,   x_0 given or 0
 *     y_t  = Re(C x_t) + D * u_t
 *
 * evaluated in parallel over the sequence with the associative scan of Sec. III-B
 * (Eq. "scan".."full_scan") and its reset-aware form of Sec. IV-A
 * (Eq. "sequence_scan_reset", "associative_reset").
 *
 * Conventions shared by every entry point
 *  - All data pointers are DEVICE pointers owned by the caller; `shape` is a HOST
 *    pointer.  The entry points allocate no device memory and never synchronise the host
 *    (except ssm_check, ssm_check_static and ssm_profile_end).  Work is enqueued on `stream`
 *    (a cudaStream_t passed as void*; NULL = the legacy default stream).
 *  - What the library keeps per process: small host-side caches filled on first use per
 *    device (SM count, kernel attributes, the tensor-map encoder's address), the launch
 *    counter and the event pool of the measurement helpers, and one fixed device array of
 *    SSM_STATIC_SCRATCH_BYTES per GPU for ssm_scan_bwd_static.  Results never depend on them.
 *  - Tensors are dense, row-major, last index fastest.  Complex numbers are
 *    interleaved (re, im) float pairs, bit-compatible with float2 / complex64.
 *  - Parameters, states and their gradients are always fp32.  Only u, y, gy, du follow
 *    shape->io_dtype (SSM_F32 or SSM_BF16).
 *  - done[B,T] is uint8; nonzero at (b,t) means the episode ended before step t:
 *    x_{t-1} is dropped (also x0 when t is the first step) and u_t still enters.
 *  - Requirements: B,T >= 1; H and P positive multiples of 8; every pointer 16-byte
 *    aligned.  Violations are detected on the host before any launch.
 *  - Gradient convention for complex values under a real loss L:
 *    g_z = dL/dRe(z) + i dL/dIm(z).  Gradient outputs are overwritten, not accumulated.
 *  - Return value: SSM_OK (0) or a negative SSM_ERR_* code.  Nothing throws, aborts or
 *    traps.  Device-side waits (shared-memory barriers of the pipelines) are bounded; if one gives
 *    up it records SSM_ERR_TIMEOUT in the workspace header, which ssm_check reads back.
 *  - Workspaces: the *_workspace_bytes functions give the size for a shape; the caller
 *    passes a 256-byte aligned device buffer of at least that size.  A layer workspace
 *    written by ssm_layer_fwd holds the residuals that ssm_layer_bwd reads, so it must
 *    stay untouched between the two calls.  Calls sharing a workspace must not overlap.
 */
#ifndef SSM_B200_H
#define SSM_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct { float re, im; } ssm_c64;

enum { SSM_F32 = 0, SSM_BF16 = 1 };

enum {
    SSM_OK = 0,
    SSM_ERR_NULL = -1,       /* a required pointer is NULL                        */
    SSM_ERR_SHAPE = -2,      /* B,T < 1, or H,P not positive multiples of 8        */
    SSM_ERR_ALIGN = -3,      /* a pointer is not aligned as required               */
    SSM_ERR_DTYPE = -4,      /* io_dtype is neither SSM_F32 nor SSM_BF16           */
    SSM_ERR_WORKSPACE = -5,  /* workspace missing or too small                     */
    SSM_ERR_CUDA = -6,       /* a CUDA runtime call or launch reported an error    */
    SSM_ERR_TIMEOUT = -7,    /* a bounded device-side wait gave up                 */
    SSM_ERR_TOO_LARGE = -8   /* problem exceeds a built-in fixed-size buffer       */
};

typedef struct {
    int32_t B;         /* sequences in the batch                                   */
    int32_t T;         /* steps per sequence (the paper's L)                       */
    int32_t H;         /* width of u and y                                         */
    int32_t P;         /* number of complex diagonal states                        */
    int32_t io_dtype;  /* SSM_F32 or SSM_BF16: storage type of u, y, gy, du        */
    int32_t reserved;  /* must be 0                                                */
} ssm_shape;

/* Human-readable name of a status code (static storage, never NULL). */
const char* ssm_status_string(int status);

/* Reads the workspace header back to the host (synchronises `stream`) and returns
 * SSM_OK, or SSM_ERR_TIMEOUT if a kernel that used this workspace gave up a wait. */
int ssm_check(const void* ws, void* stream);

/* ---- discretisation: Sec. III-B, Eq. 3 (rule: zero-order hold) --------------------
 * Abar[P] = exp(Lambda Delta);  Bbar[P,H] = ((Abar - 1)/Lambda) * B.  Lambda must be
 * nonzero.  The P-sized part is evaluated in double precision and rounded once.
 * Uses shape->H, shape->P. */
int ssm_discretize(const ssm_shape* shape, const ssm_c64* Lambda /*[P]*/,
                   const float* Delta /*[P]*/, const ssm_c64* Bc /*[P,H]*/,
                   ssm_c64* Abar /*[P] out*/, ssm_c64* Bbar /*[P,H] out*/, void* stream);

/* Adjoint of ssm_discretize: from gAbar[P], gBbar[P,H] to dLambda[P], dDelta[P], dB[P,H]. */
int ssm_discretize_bwd(const ssm_shape* shape, const ssm_c64* Lambda, const float* Delta,
                       const ssm_c64* Bc, const ssm_c64* gAbar, const ssm_c64* gBbar,
                       ssm_c64* dLambda, float* dDelta, ssm_c64* dB, void* stream);

/* ---- the scan: Sec. III-B Eq. "scan".."full_scan"; resets Sec. IV-A ---------------
 * x[b,t,p] = (done[b,t] ? 0 : Abar[p] x[b,t-1,p]) + Bu[b,t,p],  x[b,-1,:] = x0[b,:] or 0.
 * A sequence is scanned tile by tile; inside a tile groups of threads scan stretches of
 * rows concurrently and are joined with the operator's associativity, so the result does
 * not depend on scheduling.  done, x0, xT may be NULL.
 * x may alias Bu (in-place).  Uses shape->B, T, P. */
size_t ssm_scan_workspace_bytes(const ssm_shape* shape);
int ssm_scan_fwd(const ssm_shape* shape, const ssm_c64* Abar /*[P]*/,
                 const ssm_c64* Bu /*[B,T,P]*/, const uint8_t* done /*[B,T] or NULL*/,
                 const ssm_c64* x0 /*[B,P] or NULL*/, ssm_c64* x /*[B,T,P] out*/,
                 ssm_c64* xT /*[B,P] out or NULL*/, void* ws, size_t ws_bytes, void* stream);

/* Adjoint of ssm_scan_fwd (the same scan run backwards in time):
 *   s_t = gx_t + (done_{t+1} ? 0 : conj(Abar) s_{t+1}),   s_{T+1} = gxT or 0
 *   gBu = s;  gAbar[p] = sum_{b,t} (done_t ? 0 : s_t conj(x_{t-1}));
 *   gx0 = done_1 ? 0 : conj(Abar) s_1.
 * gxT, x0, done, gx0 may be NULL.  gBu may alias gx. */
int ssm_scan_bwd(const ssm_shape* shape, const ssm_c64* Abar, const uint8_t* done,
                 const ssm_c64* x0, const ssm_c64* x /*[B,T,P] from the forward*/,
                 const ssm_c64* gx /*[B,T,P]*/, const ssm_c64* gxT /*[B,P] or NULL*/,
                 ssm_c64* gBu /*[B,T,P] out*/, ssm_c64* gAbar /*[P] out*/,
                 ssm_c64* gx0 /*[B,P] out or NULL*/, void* ws, size_t ws_bytes, void* stream);

/* ---- reverse scan without a caller workspace (the paper has no counterpart) ---------
 * Same result as ssm_scan_bwd, for callers that have no scratch buffer to pass and are
 * not in a position to get one: code running where device allocation is off limits, for
 * example a plug-in inside a host framework that owns all device memory through its own
 * pool and forbids cudaMalloc (which also stalls the whole device while it runs), a
 * real-time loop with a memory budget fixed at start-up, or a callback that may not call
 * allocating CUDA routines.  The scratch lives in a fixed array of
 * SSM_STATIC_SCRATCH_BYTES inside the library's device image, so every GPU that loads the
 * library gives up that much memory until the process ends.  The call allocates nothing.
 *  - Limit: problems whose scan scratch (ssm_scan_workspace_bytes(shape)) exceeds
 *    SSM_STATIC_SCRATCH_BYTES are refused with SSM_ERR_TOO_LARGE before anything runs.
 *  - The first call on each device looks up the array's device address (with that device
 *    current); make that first call outside any stream capture.
 *  - All calls on a device share the one array.  The library clears what has to start at
 *    zero on every call, but two calls whose GPU work overlaps (different streams) race on
 *    it: issue them on one stream or order them yourself.
 *  - A bounded device-side wait that gives up records SSM_ERR_TIMEOUT in the array's first word;
 *    ssm_check_static(stream) reads it back (it synchronises `stream`, allocates nothing, and
 *    reports the most recent call on the current device, since every call clears the word).
 * Arguments are those of ssm_scan_bwd minus the workspace. */
#define SSM_STATIC_SCRATCH_BYTES (8u << 20)
int ssm_scan_bwd_static(const ssm_shape* shape, const ssm_c64* Abar, const uint8_t* done,
                        const ssm_c64* x0, const ssm_c64* x, const ssm_c64* gx,
                        const ssm_c64* gxT, ssm_c64* gBu, ssm_c64* gAbar, ssm_c64* gx0,
                        void* stream);
int ssm_check_static(void* stream);

/* ---- the whole layer: Sec. III-B Eq. 3 with the resets of Sec. IV-A ----------------
 * Forward: discretise, Bu = Bbar u, scan, y = Re(C x) + D u.  u, y are [B,T,H] in
 * io_dtype.  ws keeps the residuals (discretised parameters, states) for the backward. */
size_t ssm_layer_workspace_bytes(const ssm_shape* shape);
/* Which kernels ssm_layer_fwd / ssm_layer_bwd take for a shape on the current device, as text in buf
 * (host only, nothing is launched; at most len - 1 characters and a terminating 0).  The text is
 * "projections=<tensor-cores|tensor-cores-planes|cuda-cores> scans=<fused|separate>", and for fused scans
 * " chain_states=<64|32> time_pairs=<0|1>": the states a CTA pair scans together, and whether its two CTAs
 * share one sequence (few long sequences) or take two.  Returns SSM_OK, SSM_ERR_NULL (buf NULL or len 0)
 * or the shape's error. */
int ssm_layer_plan_string(const ssm_shape* shape, char* buf, size_t len);
int ssm_layer_fwd(const ssm_shape* shape, const ssm_c64* Lambda /*[P]*/, const float* Delta /*[P]*/,
                  const ssm_c64* Bc /*[P,H]*/, const ssm_c64* Cc /*[H,P]*/, const float* D /*[H]*/,
                  const void* u /*[B,T,H] io*/, const uint8_t* done /*[B,T] or NULL*/,
                  const ssm_c64* x0 /*[B,P] or NULL*/, void* y /*[B,T,H] io, out*/,
                  ssm_c64* xT /*[B,P] out or NULL*/, void* ws, size_t ws_bytes, void* stream);

/* Backward of L = sum(gy*y) + Re sum(conj(gxT) xT): needs the workspace ssm_layer_fwd
 * filled for the same arguments.  Outputs: du[B,T,H] (io_dtype), dLambda[P], dDelta[P],
 * dB[P,H], dC[H,P], dD[H], dx0[B,P] (or NULL).  gxT may be NULL. */
int ssm_layer_bwd(const ssm_shape* shape, const ssm_c64* Lambda, const float* Delta,
                  const ssm_c64* Bc, const ssm_c64* Cc, const float* D, const void* u,
                  const uint8_t* done, const ssm_c64* x0, const void* gy /*[B,T,H] io*/,
                  const ssm_c64* gxT, void* ws, size_t ws_bytes, void* du,
                  ssm_c64* dLambda, float* dDelta, ssm_c64* dB, ssm_c64* dC, float* dD,
                  ssm_c64* dx0, void* stream);

/* ---- single-step mode: Sec. IV-A Eq. "wm", x_t, y_t = SSM(u_t, done_t, x_{t-1}) ------
 * The form the world model is called in when a policy sits between two steps (imagination
 * rollouts, Sec. IV-B; context warm-up followed by a rollout): one time step for B
 * trajectories, the state handed from call to call by the caller.
 *   x_next[b,p] = (done[b] ? 0 : Abar[p] x_prev[b,p]) + sum_h Bbar[p,h] u[b,h]
 *   y[b,h]      = Re sum_p C[h,p] x_next[b,p] + D[h] u[b,h]
 * ssm_step_prepare discretises the parameters and packs the projection operands into ws
 * once (again after every parameter update); ssm_step then runs the step from that
 * workspace and may be called any number of times.  shape->T is ignored (taken as 1);
 * u, y are [B,H] in io_dtype; done is [B] or NULL; x_next may alias x_prev.  The state
 * entering the first step is the xT of ssm_layer_fwd over the context, or zero. */
size_t ssm_step_workspace_bytes(const ssm_shape* shape);
int ssm_step_prepare(const ssm_shape* shape, const ssm_c64* Lambda /*[P]*/, const float* Delta /*[P]*/,
                     const ssm_c64* Bc /*[P,H]*/, const ssm_c64* Cc /*[H,P]*/, void* ws,
                     size_t ws_bytes, void* stream);
int ssm_step(const ssm_shape* shape, const float* D /*[H]*/, const void* u /*[B,H] io*/,
             const uint8_t* done /*[B] or NULL*/, const ssm_c64* x_prev /*[B,P]*/,
             ssm_c64* x_next /*[B,P] out*/, void* y /*[B,H] io, out*/, void* ws, size_t ws_bytes,
             void* stream);

/* ---- half-GLU gate of the S5 sequence layer: Appendix "S5 Sequence Layer" -----------
 * The gate the paper's block applies to the SSM output v:
 *   x1 = GELU(v);   out[m,j] = v[m,j] * sigmoid( sum_i W[i,j] x1[m,i] )      (exact erf GELU, no bias)
 * over the B*T rows m of [B,T,H] tensors in io_dtype; W is [H,H] fp32, row i = input feature.
 * ssm_glu_fwd leaves GELU(v) and the gate's argument in ws; ssm_glu_bwd needs that workspace
 * and returns, for L = sum(gout * out), gv[B,T,H] (io_dtype) and dW[H,H] (overwritten).
 * A block of the paper is ssm_layer_fwd followed by ssm_glu_fwd on its y (and the reverse order
 * backward, the gate's gv being the layer's gy).  Uses shape->B, T, H. */
size_t ssm_glu_workspace_bytes(const ssm_shape* shape);
int ssm_glu_fwd(const ssm_shape* shape, const float* W /*[H,H]*/, const void* v /*[B,T,H] io*/,
                void* out /*[B,T,H] io*/, void* ws, size_t ws_bytes, void* stream);
int ssm_glu_bwd(const ssm_shape* shape, const float* W, const void* v, const void* gout /*[B,T,H] io*/,
                void* ws, size_t ws_bytes, void* gv /*[B,T,H] io, out*/, float* dW /*[H,H] out*/,
                void* stream);

/* ---- stacked sequence model --------------------------------------------------------
 * n_layers layers of   v = SSM_l(u_l);  u_{l+1} = LayerNorm(u_l + GELU(v)) * ln_weight + ln_bias
 * (exact erf GELU, LayerNorm over the H features with eps 1e-5), the same done flags in every
 * layer and a zero initial state.  The paper wraps its S5 SSM in a block of nonlinearity and
 * gating (Appendix "S5 Sequence Layer", whose schematic is a half-GLU); this post-norm
 * residual block is the stacked configuration the benchmark defines.  u, out, gout and du are in
 * io_dtype; what passes between the layers stays in fp32 inside the workspace (rounded to bf16
 * there, two correct evaluations differ by more than the bf16 tolerance in the parameter
 * gradients of the layers below).
 * `params` / `grads` are HOST arrays of n_layers structs holding DEVICE pointers.  The
 * workspace filled by ssm_stack_fwd is read by ssm_stack_bwd.  Backward: from gout[B,T,H] to
 * du[B,T,H] and every layer's parameter gradients (overwritten). */
typedef struct {
    const ssm_c64* Lambda; const float* Delta; const ssm_c64* Bc; const ssm_c64* Cc; const float* D;
    const float* ln_weight; const float* ln_bias;   /* [H] each */
} ssm_stack_params;
typedef struct {
    ssm_c64* dLambda; float* dDelta; ssm_c64* dB; ssm_c64* dC; float* dD;
    float* dln_weight; float* dln_bias;
} ssm_stack_grads;
size_t ssm_stack_workspace_bytes(const ssm_shape* shape, int n_layers);
int ssm_stack_fwd(const ssm_shape* shape, int n_layers, const ssm_stack_params* params,
                  const void* u /*[B,T,H] io*/, const uint8_t* done /*[B,T] or NULL*/,
                  void* out /*[B,T,H] io*/, void* ws, size_t ws_bytes, void* stream);
int ssm_stack_bwd(const ssm_shape* shape, int n_layers, const ssm_stack_params* params,
                  const void* u, const uint8_t* done, const void* gout /*[B,T,H] io*/,
                  void* ws, size_t ws_bytes, void* du /*[B,T,H] io*/,
                  const ssm_stack_grads* grads, void* stream);

/* ---- measurement helpers (no counterpart in the paper; they never change results) ----
 * ssm_launch_count: kernels this library has launched in this process so far.
 * ssm_profile_begin / ssm_profile_end: between the two, every internal stage of the
 * entry points above is bracketed by CUDA events on its stream.  ssm_profile_end
 * synchronises the device and writes one line per stage, "name launches total_ms\n",
 * into the HOST buffer `buf` (truncated to buf_bytes, NUL-terminated).  Process-wide,
 * not thread-safe; creates CUDA events, allocates no device memory. */
long long ssm_launch_count(void);
int ssm_profile_begin(void);
int ssm_profile_end(char* buf, size_t buf_bytes);

#ifdef __cplusplus
}
#endif
#endif /* SSM_B200_H */
