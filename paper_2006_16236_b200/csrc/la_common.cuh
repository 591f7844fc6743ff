// Shared device/host helpers of the linear-attention library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "la.h"

namespace la {

// ---- host-side error plumbing (defined in la_api.cu) -----------------------
int fail(int status, const char* fmt, ...);
int cuda_fail(cudaError_t e, const char* what);

// After a <<<...>>> launch: count it and surface a launch error.
#define LA_LAUNCHED()                          \
    do {                                       \
        ::la::note_launch();                   \
        LA_CUDA_TRY(cudaGetLastError());       \
    } while (0)

#define LA_CUDA_TRY(expr)                                          \
    do {                                                           \
        cudaError_t e__ = (expr);                                  \
        if (e__ != cudaSuccess) return ::la::cuda_fail(e__, #expr); \
    } while (0)

// Argument checks shared by every entry point (defined in la_api.cu): sizes, enums and limits of a
// problem descriptor (need_n: N is used and must be >= 0 and not too long); 16-byte alignment;
// compute capability 10.x of the current device (cached per device and thread).
int check_problem(const la_problem* p, bool need_n);
bool aligned16(const void* p);
int check_arch();

// Device status word: kernels that give up on a bounded wait OR a code into it.
// Returns its device address for the current device (NULL on failure).
int* device_status_ptr();

// Every kernel launch of the library is counted (see la_kernel_launches()).
void note_launch();

// Optional per-kernel timing with CUDA events on the launch stream (see la_profile_enable()).
// Indices are part of the C ABI (la_profile_read); no-ops unless profiling is switched on.
enum ProfKernel {
    kProfCausalFwd = 0, kProfCausalBwdDq = 1, kProfCausalBwdDkv = 2, kProfSegmentSum = 3, kProfProjection = 4,
    kProfLinearSum = 5, kProfLinearApply = 6, kProfRecurrent = 7, kProfCount = 8
};
void prof_begin(int kernel, cudaStream_t st);
void prof_end(int kernel, cudaStream_t st);

// ---- element access in the I/O type ----------------------------------------
template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) {
    return __bfloat162float(x);
}
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) {
    return __float2bfloat16_rn(x);
}

// ---- feature map, Eq. 7 ------------------------------------------------------
// phi(x) = x + 1 for x > 0, exp(x) otherwise; identity mode passes x through.
__device__ __forceinline__ float phi_apply(float x, int phi) {
    if (phi == LA_PHI_IDENTITY) return x;
    return x > 0.f ? x + 1.f : expf(x);
}
// Slope of phi recovered from its value y = phi(x): x > 0 <=> y > 1, where the
// slope is 1; otherwise the slope equals the value exp(x).
__device__ __forceinline__ float phi_slope_from_value(float y, int phi) {
    if (phi == LA_PHI_IDENTITY) return 1.f;
    return y > 1.f ? 1.f : y;
}

// ---- launchers implemented in the kernel files -------------------------------
int launch_feature_map(const void* x, void* y, int64_t n, int dtype, int deriv, cudaStream_t st);
int launch_poly2_map(const void* x, void* y, int64_t rows, int D, int C, int dtype, cudaStream_t st);
int launch_poly2_map_backward(const void* x, const void* dy, void* dx, int64_t rows, int D, int C, int dtype,
                              cudaStream_t st);

int launch_recurrent_steps(const la_problem& p, const void* q, const void* k, const void* v,
                           float* S, float* Z, void* out, cudaStream_t st);
// chained: launch as a programmatic dependent of the kernel before it in the stream (its launch overlaps that
// kernel's tail; it waits for that kernel before it reads anything).  early_state (with chained, D = M = 64):
// the state is read before that wait; only for a caller whose kernel in front belongs to the same call, leaves
// the state alone, and itself waits before it lets this one be scheduled.
int launch_recurrent_step(const la_problem& p, const void* q, const void* k, const void* v,
                          float* S, float* Z, void* out, cudaStream_t st, bool chained = false, bool early_state = false);

// Decode step of a whole attention sublayer (projections + recurrent step + output projection), bf16, D = M = 64
bool decode_layer_supported(const la_problem& p);
size_t decode_layer_workspace(const la_problem& p);
int decode_layer_step(const la_problem& p, const void* x, const void* Wqkv, const void* Wo, float* S, float* Z,
                      void* y, void* ws, cudaStream_t st);

// State arguments of the causal backward pass (device, fp32, any of them may be null): the state the
// forward started from, the upstream gradient of the final state, and where the gradient of the
// initial state goes.  S: [B,H,D,M], Z: [B,H,D].
struct StateArgs {
    const float* S_in = nullptr;
    const float* Z_in = nullptr;
    const float* dS_out = nullptr;
    const float* dZ_out = nullptr;
    float* dS_in = nullptr;
    float* dZ_in = nullptr;
};

// General (any D, M multiple of 8 up to 128, any N) fp32-arithmetic kernels.
size_t general_workspace_bytes(const la_problem& p, int op);
// lengths ([B] int32, device, or null): real positions per batch element of a right-padded ragged batch
int general_causal_forward(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths,
                           const float* S_in, const float* Z_in,
                           void* O, float* den, float* S_out, float* Z_out, cudaStream_t st);
int general_causal_backward(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths,
                            const void* G, const StateArgs& sa, void* dQ, void* dK, void* dV, void* ws,
                            cudaStream_t st);
// lengths ([B] int32, device, or null): real positions per batch element (the rest is padding);
// saved (or null): where the forward leaves its per-split sums and the backward finds them
int general_linear_forward(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths,
                           void* O, float* den, float* KV, float* Zs, void* saved, void* ws, cudaStream_t st);
int general_linear_backward(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths,
                            const void* saved, const void* G, void* dQ, void* dK, void* dV, void* ws, cudaStream_t st);

}  // namespace la
