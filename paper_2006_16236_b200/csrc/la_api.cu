// C ABI of the linear-attention library: argument validation, dispatch between
// the tensor-core and the general kernels, status reporting.  Nothing here
// allocates device memory or synchronises (except la_last_device_status).
#include <cuda.h>
#include <atomic>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include "la_common.cuh"
#include "la_tc.cuh"

namespace la {

static thread_local char g_error[512] = "";

int fail(int status, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_error, sizeof(g_error), fmt, ap);
    va_end(ap);
    return status;
}

int cuda_fail(cudaError_t e, const char* what) {
    return fail(LA_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

static std::atomic<long long> g_launches{0};
void note_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

// ---- optional per-kernel event timing --------------------------------------
static constexpr int kProfSamples = 512;
static bool g_prof_on = false;
static cudaEvent_t g_prof_ev[kProfCount][2][kProfSamples];
static bool g_prof_created = false;
static int g_prof_n[kProfCount];

void prof_begin(int kernel, cudaStream_t st) {
    if (!g_prof_on || g_prof_n[kernel] >= kProfSamples) return;
    cudaEventRecord(g_prof_ev[kernel][0][g_prof_n[kernel]], st);
}
void prof_end(int kernel, cudaStream_t st) {
    if (!g_prof_on || g_prof_n[kernel] >= kProfSamples) return;
    cudaEventRecord(g_prof_ev[kernel][1][g_prof_n[kernel]], st);
    ++g_prof_n[kernel];
}

__device__ int g_device_status_word = 0;

int* device_status_ptr() {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_device_status_word) != cudaSuccess) return nullptr;
    return (int*)p;
}

int check_arch() {
    static thread_local int cached_dev = -1, cached_rc = 0;
    int dev = 0;
    LA_CUDA_TRY(cudaGetDevice(&dev));
    if (dev == cached_dev) return cached_rc;
    int major = 0;
    LA_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    cached_dev = dev;
    cached_rc = major == 10 ? LA_OK : LA_ERR_ARCH;
    if (cached_rc) return fail(LA_ERR_ARCH, "device %d has compute capability %d.x; this library is built for sm_100a only", dev, major);
    return LA_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_problem(const la_problem* p, bool need_n) {
    if (!p) return fail(LA_ERR_INVALID_ARG, "problem descriptor is NULL");
    if (p->B < 1 || p->H < 1 || p->D < 1 || p->M < 1 || (need_n && p->N < 0))
        return fail(LA_ERR_INVALID_ARG, "sizes must be B,H,D,M >= 1 and N >= 0 (got B=%lld H=%lld N=%lld D=%lld M=%lld)",
                    (long long)p->B, (long long)p->H, (long long)p->N, (long long)p->D, (long long)p->M);
    if (p->dtype != LA_F32 && p->dtype != LA_BF16) return fail(LA_ERR_INVALID_ARG, "dtype %d is not a la_dtype", p->dtype);
    if (p->phi != LA_PHI_ELU1 && p->phi != LA_PHI_IDENTITY) return fail(LA_ERR_INVALID_ARG, "phi %d is not a la_phi", p->phi);
    if (!(p->eps >= 0.f)) return fail(LA_ERR_INVALID_ARG, "eps must be >= 0");
    if (p->D % 8 || p->M % 8 || p->D > 128 || p->M > 128)
        return fail(LA_ERR_UNSUPPORTED, "D and M must be multiples of 8 in [8,128] (got D=%lld M=%lld)",
                    (long long)p->D, (long long)p->M);
    if (p->B * p->H > 0x7fffffffLL) return fail(LA_ERR_UNSUPPORTED, "B*H exceeds 2^31-1");
    if (need_n && p->N > (1LL << 40) / (p->D > p->M ? p->D : p->M))
        return fail(LA_ERR_UNSUPPORTED, "sequence too long");
    return LA_OK;
}

// ---------------------------------------------------------------------------------------------------------
// Checked mode (environment variable LA_DEBUG=1, read once): before anything is enqueued every tensor argument
// is looked up with the driver (device memory of the current device? does the allocation that holds it reach
// as far as the call will read or write?), and after the call the stream is synchronised and the device
// status word and the CUDA error state are read, so that a failure is reported by the call that caused it.
// It turns an out-of-bounds access on a shared GPU into an error code on the host.  Off by default: the
// look-ups and the synchronisation cost tens of microseconds per call.
static bool debug_mode() {
    static const bool on = [] {
        const char* v = getenv("LA_DEBUG");
        return v && atoi(v) != 0;
    }();
    return on;
}

static int debug_span(const void* ptr, size_t bytes, const char* name) {
    if (!debug_mode() || !ptr || !bytes) return LA_OK;
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, ptr) != cudaSuccess) {
        cudaGetLastError();
        return fail(LA_ERR_INVALID_ARG, "checked mode: %s (%p) is not a pointer CUDA knows", name, ptr);
    }
    if (at.type != cudaMemoryTypeDevice && at.type != cudaMemoryTypeManaged)
        return fail(LA_ERR_INVALID_ARG, "checked mode: %s (%p) is not device memory", name, ptr);
    int dev = 0;
    LA_CUDA_TRY(cudaGetDevice(&dev));
    if (at.type == cudaMemoryTypeDevice && at.device != dev)
        return fail(LA_ERR_INVALID_ARG, "checked mode: %s lives on device %d, the current device is %d", name, at.device, dev);
    typedef CUresult (*range_fn)(CUdeviceptr*, size_t*, CUdeviceptr);
    static range_fn range = [] {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuMemGetAddressRange", &fn, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            fn = nullptr;
        return reinterpret_cast<range_fn>(fn);
    }();
    if (!range) return LA_OK;
    CUdeviceptr base = 0;
    size_t size = 0;
    if (range(&base, &size, (CUdeviceptr)(uintptr_t)ptr) != CUDA_SUCCESS) return LA_OK;      // not a plain allocation: no range to check
    const uintptr_t end = (uintptr_t)ptr + bytes, alloc_end = (uintptr_t)base + size;
    if (end > alloc_end)
        return fail(LA_ERR_INVALID_ARG, "checked mode: %s needs %zu bytes at %p, its allocation ends %zu bytes earlier", name,
                    bytes, ptr, (size_t)(end - alloc_end));
    return LA_OK;
}
#define LA_DEBUG_SPAN(ptr, bytes)                                   \
    do {                                                            \
        if (int rc_ = debug_span(ptr, bytes, #ptr)) return rc_;     \
    } while (0)

extern "C" int la_last_device_status(void* stream);
// the tail of every compute entry point: in checked mode the call's own failures surface here
static int debug_finish(int rc, void* stream) {
    if (rc != LA_OK || !debug_mode()) return rc;
    if (int st = la_last_device_status(stream)) return st;
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(LA_ERR_CUDA, "checked mode: %s after the call", cudaGetErrorString(e));
    return LA_OK;
}

struct TensorBytes {        // sizes of the tensors of a problem, for the span checks
    size_t qk, vo, den, s, z;
    explicit TensorBytes(const la_problem& p) {
        const size_t e = p.dtype == LA_BF16 ? 2 : 4, bh = (size_t)(p.B * p.H);
        qk = bh * (size_t)p.N * (size_t)p.D * e;
        vo = bh * (size_t)p.N * (size_t)p.M * e;
        den = bh * (size_t)p.N * sizeof(float);
        s = bh * (size_t)(p.D * p.M) * sizeof(float);
        z = bh * (size_t)p.D * sizeof(float);
    }
};

#define LA_REQUIRE_PTR(ptr)                                                                \
    do {                                                                                   \
        if (!(ptr)) return fail(LA_ERR_INVALID_ARG, #ptr " is NULL");                      \
        if (!aligned16(ptr)) return fail(LA_ERR_INVALID_ARG, #ptr " is not 16-byte aligned"); \
    } while (0)
#define LA_OPTIONAL_PTR(ptr)                                                               \
    do {                                                                                   \
        if ((ptr) && !aligned16(ptr)) return fail(LA_ERR_INVALID_ARG, #ptr " is not 16-byte aligned"); \
    } while (0)

static int check_ws(const la_problem* p, int op, const void* ws, size_t ws_bytes) {
    const size_t need = la_workspace_bytes(p, op);
    if (need == 0) return LA_OK;
    if (!ws) return fail(LA_ERR_WORKSPACE, "workspace is NULL but %zu bytes are needed", need);
    if (!aligned16(ws)) return fail(LA_ERR_INVALID_ARG, "workspace is not 16-byte aligned");
    if (ws_bytes < need) return fail(LA_ERR_WORKSPACE, "workspace has %zu bytes, %zu are needed", ws_bytes, need);
    return LA_OK;
}

// `saved` is optional; when given it must hold la_workspace_bytes(p, LA_OP_CAUSAL_SAVED) bytes.
static int check_saved(const la_problem* p, const void* saved, size_t saved_bytes) {
    if (!saved) return LA_OK;
    const size_t need = la_workspace_bytes(p, LA_OP_CAUSAL_SAVED);
    if (!aligned16(saved) || ((uintptr_t)saved & 127)) return fail(LA_ERR_INVALID_ARG, "saved buffer is not 128-byte aligned");
    if (saved_bytes < need) return fail(LA_ERR_WORKSPACE, "saved buffer has %zu bytes, %zu are needed", saved_bytes, need);
    return LA_OK;
}

}  // namespace la

using namespace la;

extern "C" {

const char* la_version(void) { return "0.1"; }

const char* la_status_string(int status) {
    switch (status) {
        case LA_OK: return "LA_OK";
        case LA_ERR_INVALID_ARG: return "LA_ERR_INVALID_ARG";
        case LA_ERR_UNSUPPORTED: return "LA_ERR_UNSUPPORTED";
        case LA_ERR_WORKSPACE: return "LA_ERR_WORKSPACE";
        case LA_ERR_CUDA: return "LA_ERR_CUDA";
        case LA_ERR_ARCH: return "LA_ERR_ARCH";
        case LA_ERR_DEVICE_TIMEOUT: return "LA_ERR_DEVICE_TIMEOUT";
        default: return "LA_ERR_UNKNOWN";
    }
}

const char* la_last_error(void) { return g_error; }

long long la_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

int la_profile_enable(int on) {
    if (on && !g_prof_created) {
        for (int k = 0; k < kProfCount; ++k)
            for (int e = 0; e < 2; ++e)
                for (int i = 0; i < kProfSamples; ++i) LA_CUDA_TRY(cudaEventCreate(&g_prof_ev[k][e][i]));
        g_prof_created = true;
    }
    for (int k = 0; k < kProfCount; ++k) g_prof_n[k] = 0;
    g_prof_on = on != 0;
    return LA_OK;
}

int la_profile_read(int kernel, double* mean_ms, int* launches) {
    if (kernel < 0 || kernel >= kProfCount || !mean_ms || !launches) return fail(LA_ERR_INVALID_ARG, "bad profile query");
    double total = 0.0;
    const int n = g_prof_n[kernel];
    for (int i = 0; i < n; ++i) {
        LA_CUDA_TRY(cudaEventSynchronize(g_prof_ev[kernel][1][i]));
        float ms = 0.f;
        LA_CUDA_TRY(cudaEventElapsedTime(&ms, g_prof_ev[kernel][0][i], g_prof_ev[kernel][1][i]));
        total += ms;
    }
    *launches = n;
    *mean_ms = n ? total / n : 0.0;
    return LA_OK;
}

const char* la_profile_kernel_name(int kernel) {
    static const char* names[kProfCount] = {"causal_fwd_kernel", "causal_bwd_dq_kernel", "causal_bwd_dkv_kernel",
                                            "segment_sum_kernel", "projection_gemm_kernel", "linear_sum_kernel",
                                            "linear_apply_kernel", "recurrent_step_kernel"};
    return kernel >= 0 && kernel < kProfCount ? names[kernel] : "";
}

size_t la_workspace_bytes(const la_problem* p, int32_t op) {
    if (!p || p->B < 1 || p->H < 1 || p->N < 0 || p->D < 1 || p->M < 1 || p->D > 128 || p->M > 128) return 0;
    if (op < LA_OP_LINEAR_FORWARD || op > LA_OP_CAUSAL_VARLEN_BACKWARD) return 0;
    if (op == LA_OP_CAUSAL_VARLEN_FORWARD) op = LA_OP_CAUSAL_FORWARD;         // the ragged calls run the same kernels
    if (op == LA_OP_CAUSAL_VARLEN_BACKWARD) op = LA_OP_CAUSAL_BACKWARD;
    if (op == LA_OP_DECODE_LAYER) return decode_layer_supported(*p) ? decode_layer_workspace(*p) : 0;
    if (p->N == 0) return 0;
    if (op == LA_OP_LINEAR_SAVED) op = LA_OP_LINEAR_FORWARD;          // the saved buffer holds what the forward's workspace holds
    if (op == LA_OP_CAUSAL_SAVED) return tc_supported(*p, LA_OP_CAUSAL_BACKWARD) ? tc::causal_saved_bytes(*p) : 0;
    if (op == LA_OP_LINEAR_VARLEN_FORWARD || op == LA_OP_LINEAR_VARLEN_BACKWARD) {
        const int full = op == LA_OP_LINEAR_VARLEN_FORWARD ? LA_OP_LINEAR_FORWARD : LA_OP_LINEAR_BACKWARD;
        return tc_supported(*p, full) ? tc_workspace_bytes(*p, full) : general_workspace_bytes(*p, op);
    }
    if (tc_supported(*p, op)) return tc_workspace_bytes(*p, op);
    return general_workspace_bytes(*p, op);
}

int la_causal_plan(const la_problem* p, int32_t* out, int capacity) {
    if (int rc = check_problem(p, true)) return rc;
    if (capacity < 0 || (capacity > 0 && !out)) return fail(LA_ERR_INVALID_ARG, "out is NULL or capacity is negative");
    if (p->N == 0 || !tc_supported(*p, LA_OP_CAUSAL_FORWARD)) return 0;
    return tc_causal_plan(*p, out, capacity);
}

int la_plan_override(int32_t causal_pieces, int32_t causal_short, int32_t linear_splits) {
    if (causal_pieces < -1 || causal_pieces == 0 || causal_short < -1 || linear_splits < -1 || linear_splits == 0)
        return fail(LA_ERR_INVALID_ARG, "overrides are -1 (automatic) or positive counts (causal_short may be 0: no short piece)");
    tc::set_plan_override(causal_pieces, causal_short, linear_splits);
    return LA_OK;
}

int la_feature_map(const void* x, void* y, int64_t n, int32_t dtype, int32_t deriv, void* stream) {
    if (n < 0) return fail(LA_ERR_INVALID_ARG, "n must be >= 0");
    if (dtype != LA_F32 && dtype != LA_BF16) return fail(LA_ERR_INVALID_ARG, "dtype %d is not a la_dtype", dtype);
    if (n == 0) return LA_OK;
    LA_REQUIRE_PTR(x);
    LA_REQUIRE_PTR(y);
    if (int rc = check_arch()) return rc;
    return launch_feature_map(x, y, n, dtype, deriv != 0, (cudaStream_t)stream);
}

static int check_poly2(int64_t rows, int64_t D, int64_t C, int32_t dtype) {
    if (rows < 0) return fail(LA_ERR_INVALID_ARG, "rows must be >= 0");
    if (dtype != LA_F32 && dtype != LA_BF16) return fail(LA_ERR_INVALID_ARG, "dtype %d is not a la_dtype", dtype);
    if (D < 1 || D > 11) return fail(LA_ERR_INVALID_ARG, "D=%lld: the feature dimension D*D must fit 128 columns", (long long)D);
    if (C < D * D || C > 128 || C % 8) return fail(LA_ERR_INVALID_ARG, "C=%lld must be a multiple of 8 in [D*D, 128]", (long long)C);
    return LA_OK;
}

int la_feature_map_poly2(const void* x, void* y, int64_t rows, int64_t D, int64_t C, int32_t dtype, void* stream) {
    if (int rc = check_poly2(rows, D, C, dtype)) return rc;
    if (rows == 0) return LA_OK;
    LA_REQUIRE_PTR(x);          // rows of eight bf16 are read with 16-byte loads
    LA_REQUIRE_PTR(y);
    if (int rc = check_arch()) return rc;
    return launch_poly2_map(x, y, rows, (int)D, (int)C, dtype, (cudaStream_t)stream);
}

int la_feature_map_poly2_backward(const void* x, const void* dy, void* dx, int64_t rows, int64_t D, int64_t C,
                                  int32_t dtype, void* stream) {
    if (int rc = check_poly2(rows, D, C, dtype)) return rc;
    if (rows == 0) return LA_OK;
    LA_REQUIRE_PTR(x);
    LA_REQUIRE_PTR(dy);
    LA_REQUIRE_PTR(dx);
    if (dx == x) return fail(LA_ERR_INVALID_ARG, "dx must not alias x");
    if (int rc = check_arch()) return rc;
    return launch_poly2_map_backward(x, dy, dx, rows, (int)D, (int)C, dtype, (cudaStream_t)stream);
}

// The optional buffer in which the non-causal forward keeps its per-split sums for the backward pass.
static int check_rff(int64_t rows, int64_t D, int64_t C, int32_t dtype) {
    if (rows < 0 || D < 1 || C < 2) return fail(LA_ERR_INVALID_ARG, "rows >= 0, D >= 1 and C >= 2 are required");
    if (dtype != LA_F32 && dtype != LA_BF16) return fail(LA_ERR_INVALID_ARG, "dtype %d is not a la_dtype", dtype);
    if (rows > 0 && !tc::rff_supported(rows, D, C, dtype))
        return fail(LA_ERR_UNSUPPORTED, "random Fourier features take bf16, D a multiple of 8 in [8, 64], C = 64 or 128, rows < 2^31 "
                                        "(got dtype %d, D=%lld, C=%lld, rows=%lld)", dtype, (long long)D, (long long)C, (long long)rows);
    return LA_OK;
}

int la_feature_map_rff(const void* x, const void* W, void* y, int64_t rows, int64_t D, int64_t C, int32_t dtype, void* stream) {
    if (int rc = check_rff(rows, D, C, dtype)) return rc;
    if (rows == 0) return LA_OK;
    LA_REQUIRE_PTR(x); LA_REQUIRE_PTR(W); LA_REQUIRE_PTR(y);
    if (int rc = check_arch()) return rc;
    LA_DEBUG_SPAN(x, (size_t)(rows * D) * 2); LA_DEBUG_SPAN(W, (size_t)(C / 2 * D) * 2); LA_DEBUG_SPAN(y, (size_t)(rows * C) * 2);
    return debug_finish(tc::rff_forward(x, W, y, rows, (int)D, (int)C, (cudaStream_t)stream), stream);
}

int la_feature_map_rff_backward(const void* x, const void* W, const void* dy, void* dx, int64_t rows, int64_t D, int64_t C,
                                int32_t dtype, void* stream) {
    if (int rc = check_rff(rows, D, C, dtype)) return rc;
    if (rows == 0) return LA_OK;
    LA_REQUIRE_PTR(x); LA_REQUIRE_PTR(W); LA_REQUIRE_PTR(dy); LA_REQUIRE_PTR(dx);
    if (dx == x) return fail(LA_ERR_INVALID_ARG, "dx must not alias x");
    if (int rc = check_arch()) return rc;
    LA_DEBUG_SPAN(x, (size_t)(rows * D) * 2); LA_DEBUG_SPAN(W, (size_t)(C / 2 * D) * 2); LA_DEBUG_SPAN(dy, (size_t)(rows * C) * 2);
    LA_DEBUG_SPAN(dx, (size_t)(rows * D) * 2);
    return debug_finish(tc::rff_backward(x, W, dy, dx, rows, (int)D, (int)C, (cudaStream_t)stream), stream);
}

static int check_linear_saved(const la_problem* p, const void* saved, size_t saved_bytes) {
    if (!saved) return LA_OK;
    if (!aligned16(saved)) return fail(LA_ERR_INVALID_ARG, "saved is not 16-byte aligned");
    const size_t need = la_workspace_bytes(p, LA_OP_LINEAR_SAVED);
    if (saved_bytes < need)
        return fail(LA_ERR_WORKSPACE, "saved buffer too small: %zu bytes given, %zu needed", saved_bytes, need);
    return LA_OK;
}

// All non-causal forward entry points: `lengths` given (ragged batch) or not, `saved` given or not.
static int linear_forward_common(const la_problem* p, const void* Q, const void* K, const void* V, const int32_t* lengths,
                                 bool ragged, void* O, float* den, float* KV, float* Zs, void* saved, size_t saved_bytes,
                                 void* ws, size_t ws_bytes, void* stream) {
    if (int rc = check_problem(p, true)) return rc;
    if (p->N == 0) return LA_OK;
    LA_REQUIRE_PTR(Q); LA_REQUIRE_PTR(K); LA_REQUIRE_PTR(V); LA_REQUIRE_PTR(O);
    if (ragged && !lengths) return fail(LA_ERR_INVALID_ARG, "lengths is NULL");
    if (reinterpret_cast<uintptr_t>(lengths) & 3u) return fail(LA_ERR_INVALID_ARG, "lengths is not 4-byte aligned");
    LA_OPTIONAL_PTR(den); LA_OPTIONAL_PTR(KV); LA_OPTIONAL_PTR(Zs);
    if (int rc = check_linear_saved(p, saved, saved_bytes)) return rc;
    if (!saved)         // with a saved buffer the sums go there and the workspace is not touched
        if (int rc = check_ws(p, lengths ? LA_OP_LINEAR_VARLEN_FORWARD : LA_OP_LINEAR_FORWARD, ws, ws_bytes)) return rc;
    if (int rc = check_arch()) return rc;
    const TensorBytes tb(*p);
    LA_DEBUG_SPAN(Q, tb.qk); LA_DEBUG_SPAN(K, tb.qk); LA_DEBUG_SPAN(V, tb.vo); LA_DEBUG_SPAN(O, tb.vo);
    LA_DEBUG_SPAN(den, tb.den); LA_DEBUG_SPAN(KV, tb.s); LA_DEBUG_SPAN(Zs, tb.z);
    LA_DEBUG_SPAN(lengths, (size_t)p->B * 4); LA_DEBUG_SPAN(ws, ws_bytes); LA_DEBUG_SPAN(saved, saved_bytes);
    cudaStream_t st = (cudaStream_t)stream;
    if (tc_supported(*p, LA_OP_LINEAR_FORWARD))
        return debug_finish(tc::linear_forward(*p, Q, K, V, lengths, O, den, KV, Zs, saved, ws, st), stream);
    return debug_finish(general_linear_forward(*p, Q, K, V, lengths, O, den, KV, Zs, saved, ws, st), stream);
}

static int linear_backward_common(const la_problem* p, const void* Q, const void* K, const void* V, const int32_t* lengths,
                                  bool ragged, const void* saved, size_t saved_bytes, const void* O, const float* den,
                                  const void* G, void* dQ, void* dK, void* dV, void* ws, size_t ws_bytes, void* stream) {
    if (int rc = check_problem(p, true)) return rc;
    if (p->N == 0) return LA_OK;
    LA_REQUIRE_PTR(Q); LA_REQUIRE_PTR(K); LA_REQUIRE_PTR(V); LA_REQUIRE_PTR(G);
    LA_REQUIRE_PTR(dQ); LA_REQUIRE_PTR(dK); LA_REQUIRE_PTR(dV);
    if (ragged && !lengths) return fail(LA_ERR_INVALID_ARG, "lengths is NULL");
    if (reinterpret_cast<uintptr_t>(lengths) & 3u) return fail(LA_ERR_INVALID_ARG, "lengths is not 4-byte aligned");
    LA_OPTIONAL_PTR(O); LA_OPTIONAL_PTR(den);
    if (int rc = check_linear_saved(p, saved, saved_bytes)) return rc;
    if (int rc = check_ws(p, lengths ? LA_OP_LINEAR_VARLEN_BACKWARD : LA_OP_LINEAR_BACKWARD, ws, ws_bytes)) return rc;
    if (int rc = check_arch()) return rc;
    const TensorBytes tb(*p);
    LA_DEBUG_SPAN(Q, tb.qk); LA_DEBUG_SPAN(K, tb.qk); LA_DEBUG_SPAN(V, tb.vo); LA_DEBUG_SPAN(G, tb.vo);
    LA_DEBUG_SPAN(dQ, tb.qk); LA_DEBUG_SPAN(dK, tb.qk); LA_DEBUG_SPAN(dV, tb.vo);
    LA_DEBUG_SPAN(lengths, (size_t)p->B * 4); LA_DEBUG_SPAN(ws, ws_bytes); LA_DEBUG_SPAN(saved, saved_bytes);
    cudaStream_t st = (cudaStream_t)stream;
    if (tc_supported(*p, LA_OP_LINEAR_BACKWARD))
        return debug_finish(tc::linear_backward(*p, Q, K, V, lengths, saved, G, dQ, dK, dV, ws, st), stream);
    return debug_finish(general_linear_backward(*p, Q, K, V, lengths, saved, G, dQ, dK, dV, ws, st), stream);
}

int la_linear_attention(const la_problem* p, const void* Q, const void* K, const void* V,
                        void* O, float* den, float* KV, float* Zs,
                        void* ws, size_t ws_bytes, void* stream) {
    return linear_forward_common(p, Q, K, V, nullptr, false, O, den, KV, Zs, nullptr, 0, ws, ws_bytes, stream);
}

int la_linear_attention_varlen(const la_problem* p, const void* Q, const void* K, const void* V,
                               const int32_t* lengths,
                               void* O, float* den, float* KV, float* Zs,
                               void* ws, size_t ws_bytes, void* stream) {
    return linear_forward_common(p, Q, K, V, lengths, true, O, den, KV, Zs, nullptr, 0, ws, ws_bytes, stream);
}

int la_linear_attention_keep(const la_problem* p, const void* Q, const void* K, const void* V,
                             const int32_t* lengths,
                             void* O, float* den, float* KV, float* Zs,
                             void* saved, size_t saved_bytes,
                             void* ws, size_t ws_bytes, void* stream) {
    return linear_forward_common(p, Q, K, V, lengths, false, O, den, KV, Zs, saved, saved_bytes, ws, ws_bytes, stream);
}

int la_linear_attention_backward(const la_problem* p, const void* Q, const void* K, const void* V,
                                 const void* O, const float* den, const void* G,
                                 void* dQ, void* dK, void* dV,
                                 void* ws, size_t ws_bytes, void* stream) {
    return linear_backward_common(p, Q, K, V, nullptr, false, nullptr, 0, O, den, G, dQ, dK, dV, ws, ws_bytes, stream);
}

int la_linear_attention_varlen_backward(const la_problem* p, const void* Q, const void* K, const void* V,
                                        const int32_t* lengths,
                                        const void* O, const float* den, const void* G,
                                        void* dQ, void* dK, void* dV,
                                        void* ws, size_t ws_bytes, void* stream) {
    return linear_backward_common(p, Q, K, V, lengths, true, nullptr, 0, O, den, G, dQ, dK, dV, ws, ws_bytes, stream);
}

int la_linear_attention_backward_kept(const la_problem* p, const void* Q, const void* K, const void* V,
                                      const int32_t* lengths,
                                      const void* saved, size_t saved_bytes,
                                      const void* O, const float* den, const void* G,
                                      void* dQ, void* dK, void* dV,
                                      void* ws, size_t ws_bytes, void* stream) {
    return linear_backward_common(p, Q, K, V, lengths, false, saved, saved_bytes, O, den, G, dQ, dK, dV, ws, ws_bytes, stream);
}

static bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
    const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
    return a && b && x < y + nb && y < x + na;
}

}  // extern "C"

// All causal forward entry points: from a state or from zero, `lengths` given (ragged batch) or not.
static int causal_forward_common(const la_problem* p, const void* Q, const void* K, const void* V, const int32_t* lengths,
                                 bool ragged, const float* S_in, const float* Z_in,
                                 void* O, float* den, float* S_out, float* Z_out,
                                 void* saved, size_t saved_bytes,
                                 void* ws, size_t ws_bytes, void* stream) {
    if (int rc = check_problem(p, true)) return rc;
    if (ragged && !lengths) return fail(LA_ERR_INVALID_ARG, "lengths is NULL");
    if (reinterpret_cast<uintptr_t>(lengths) & 3u) return fail(LA_ERR_INVALID_ARG, "lengths is not 4-byte aligned");
    if ((S_in == nullptr) != (Z_in == nullptr)) return fail(LA_ERR_INVALID_ARG, "S_in and Z_in must both be given or both be NULL");
    LA_OPTIONAL_PTR(S_in); LA_OPTIONAL_PTR(Z_in);
    LA_OPTIONAL_PTR(den); LA_OPTIONAL_PTR(S_out); LA_OPTIONAL_PTR(Z_out);
    const size_t s_bytes = (size_t)(p->B * p->H * p->D * p->M) * sizeof(float), z_bytes = (size_t)(p->B * p->H * p->D) * sizeof(float);
    if (overlaps(S_in, s_bytes, S_out, s_bytes) || overlaps(S_in, s_bytes, Z_out, z_bytes) ||
        overlaps(Z_in, z_bytes, S_out, s_bytes) || overlaps(Z_in, z_bytes, Z_out, z_bytes))
        return fail(LA_ERR_INVALID_ARG, "S_in / Z_in overlap S_out / Z_out");
    cudaStream_t st = (cudaStream_t)stream;
    if (p->N == 0) {
        if (S_in && S_out) LA_CUDA_TRY(cudaMemcpyAsync(S_out, S_in, s_bytes, cudaMemcpyDeviceToDevice, st));
        if (Z_in && Z_out) LA_CUDA_TRY(cudaMemcpyAsync(Z_out, Z_in, z_bytes, cudaMemcpyDeviceToDevice, st));
        return LA_OK;
    }
    LA_REQUIRE_PTR(Q); LA_REQUIRE_PTR(K); LA_REQUIRE_PTR(V); LA_REQUIRE_PTR(O);
    LA_OPTIONAL_PTR(saved);
    if (int rc = check_ws(p, lengths ? LA_OP_CAUSAL_VARLEN_FORWARD : LA_OP_CAUSAL_FORWARD, ws, ws_bytes)) return rc;
    if (int rc = check_saved(p, saved, saved_bytes)) return rc;
    if (int rc = check_arch()) return rc;
    const TensorBytes tb(*p);
    LA_DEBUG_SPAN(Q, tb.qk); LA_DEBUG_SPAN(K, tb.qk); LA_DEBUG_SPAN(V, tb.vo); LA_DEBUG_SPAN(O, tb.vo);
    LA_DEBUG_SPAN(den, tb.den); LA_DEBUG_SPAN(S_in, tb.s); LA_DEBUG_SPAN(Z_in, tb.z); LA_DEBUG_SPAN(S_out, tb.s);
    LA_DEBUG_SPAN(Z_out, tb.z); LA_DEBUG_SPAN(lengths, (size_t)p->B * 4); LA_DEBUG_SPAN(ws, ws_bytes);
    LA_DEBUG_SPAN(saved, saved_bytes);
    if (tc_supported(*p, LA_OP_CAUSAL_FORWARD))
        return debug_finish(tc::causal_forward(*p, Q, K, V, lengths, S_in, Z_in, O, den, S_out, Z_out, saved, ws, st), stream);
    return debug_finish(general_causal_forward(*p, Q, K, V, lengths, S_in, Z_in, O, den, S_out, Z_out, st), stream);
}

extern "C" {

int la_causal_forward_from(const la_problem* p, const void* Q, const void* K, const void* V,
                           const float* S_in, const float* Z_in,
                           void* O, float* den, float* S_out, float* Z_out,
                           void* saved, size_t saved_bytes,
                           void* ws, size_t ws_bytes, void* stream) {
    return causal_forward_common(p, Q, K, V, nullptr, false, S_in, Z_in, O, den, S_out, Z_out, saved, saved_bytes, ws, ws_bytes, stream);
}

int la_causal_forward_varlen(const la_problem* p, const void* Q, const void* K, const void* V, const int32_t* lengths,
                             const float* S_in, const float* Z_in,
                             void* O, float* den, float* S_out, float* Z_out,
                             void* saved, size_t saved_bytes,
                             void* ws, size_t ws_bytes, void* stream) {
    return causal_forward_common(p, Q, K, V, lengths, true, S_in, Z_in, O, den, S_out, Z_out, saved, saved_bytes, ws, ws_bytes, stream);
}

int la_causal_forward(const la_problem* p, const void* Q, const void* K, const void* V,
                      void* O, float* den, float* S_out, float* Z_out,
                      void* saved, size_t saved_bytes,
                      void* ws, size_t ws_bytes, void* stream) {
    return la_causal_forward_from(p, Q, K, V, nullptr, nullptr, O, den, S_out, Z_out, saved, saved_bytes, ws, ws_bytes, stream);
}

}  // extern "C"

static int causal_backward_common(const la_problem* p, const void* Q, const void* K, const void* V, const int32_t* lengths,
                                  bool ragged, const float* S_in, const float* Z_in,
                                  const void* O, const float* den, const void* G,
                                  const float* dS_out, const float* dZ_out,
                                  const void* saved, size_t saved_bytes,
                                  void* dQ, void* dK, void* dV, float* dS_in, float* dZ_in,
                                  void* ws, size_t ws_bytes, void* stream) {
    if (int rc = check_problem(p, true)) return rc;
    if (ragged && !lengths) return fail(LA_ERR_INVALID_ARG, "lengths is NULL");
    if (reinterpret_cast<uintptr_t>(lengths) & 3u) return fail(LA_ERR_INVALID_ARG, "lengths is not 4-byte aligned");
    if ((S_in == nullptr) != (Z_in == nullptr)) return fail(LA_ERR_INVALID_ARG, "S_in and Z_in must both be given or both be NULL");
    LA_OPTIONAL_PTR(S_in); LA_OPTIONAL_PTR(Z_in); LA_OPTIONAL_PTR(dS_out); LA_OPTIONAL_PTR(dZ_out);
    LA_OPTIONAL_PTR(dS_in); LA_OPTIONAL_PTR(dZ_in);
    const size_t s_bytes = (size_t)(p->B * p->H * p->D * p->M) * sizeof(float), z_bytes = (size_t)(p->B * p->H * p->D) * sizeof(float);
    if (overlaps(dS_out, s_bytes, dS_in, s_bytes) || overlaps(dS_out, s_bytes, dZ_in, z_bytes) ||
        overlaps(dZ_out, z_bytes, dS_in, s_bytes) || overlaps(dZ_out, z_bytes, dZ_in, z_bytes))
        return fail(LA_ERR_INVALID_ARG, "dS_in / dZ_in overlap dS_out / dZ_out");
    cudaStream_t st = (cudaStream_t)stream;
    if (p->N == 0) {            // nothing between the two states: the gradient passes through
        if (dS_in) {
            if (dS_out) LA_CUDA_TRY(cudaMemcpyAsync(dS_in, dS_out, s_bytes, cudaMemcpyDeviceToDevice, st));
            else LA_CUDA_TRY(cudaMemsetAsync(dS_in, 0, s_bytes, st));
        }
        if (dZ_in) {
            if (dZ_out) LA_CUDA_TRY(cudaMemcpyAsync(dZ_in, dZ_out, z_bytes, cudaMemcpyDeviceToDevice, st));
            else LA_CUDA_TRY(cudaMemsetAsync(dZ_in, 0, z_bytes, st));
        }
        return LA_OK;
    }
    LA_REQUIRE_PTR(Q); LA_REQUIRE_PTR(K); LA_REQUIRE_PTR(V); LA_REQUIRE_PTR(G);
    LA_REQUIRE_PTR(dQ); LA_REQUIRE_PTR(dK); LA_REQUIRE_PTR(dV);
    LA_OPTIONAL_PTR(O); LA_OPTIONAL_PTR(den); LA_OPTIONAL_PTR(saved);
    if (int rc = check_ws(p, lengths ? LA_OP_CAUSAL_VARLEN_BACKWARD : LA_OP_CAUSAL_BACKWARD, ws, ws_bytes)) return rc;
    if (int rc = check_saved(p, saved, saved_bytes)) return rc;
    if (int rc = check_arch()) return rc;
    StateArgs sa;
    sa.S_in = S_in; sa.Z_in = Z_in; sa.dS_out = dS_out; sa.dZ_out = dZ_out; sa.dS_in = dS_in; sa.dZ_in = dZ_in;
    const TensorBytes tb(*p);
    LA_DEBUG_SPAN(Q, tb.qk); LA_DEBUG_SPAN(K, tb.qk); LA_DEBUG_SPAN(V, tb.vo); LA_DEBUG_SPAN(G, tb.vo);
    LA_DEBUG_SPAN(dQ, tb.qk); LA_DEBUG_SPAN(dK, tb.qk); LA_DEBUG_SPAN(dV, tb.vo);
    LA_DEBUG_SPAN(S_in, tb.s); LA_DEBUG_SPAN(Z_in, tb.z); LA_DEBUG_SPAN(dS_out, tb.s); LA_DEBUG_SPAN(dZ_out, tb.z);
    LA_DEBUG_SPAN(dS_in, tb.s); LA_DEBUG_SPAN(dZ_in, tb.z); LA_DEBUG_SPAN(lengths, (size_t)p->B * 4);
    LA_DEBUG_SPAN(ws, ws_bytes); LA_DEBUG_SPAN(saved, saved_bytes);
    if (tc_supported(*p, LA_OP_CAUSAL_BACKWARD))
        return debug_finish(tc::causal_backward(*p, Q, K, V, lengths, G, sa, saved, dQ, dK, dV, ws, st), stream);
    return debug_finish(general_causal_backward(*p, Q, K, V, lengths, G, sa, dQ, dK, dV, ws, st), stream);
}

extern "C" {

int la_causal_backward_from(const la_problem* p, const void* Q, const void* K, const void* V,
                            const float* S_in, const float* Z_in,
                            const void* O, const float* den, const void* G,
                            const float* dS_out, const float* dZ_out,
                            const void* saved, size_t saved_bytes,
                            void* dQ, void* dK, void* dV, float* dS_in, float* dZ_in,
                            void* ws, size_t ws_bytes, void* stream) {
    return causal_backward_common(p, Q, K, V, nullptr, false, S_in, Z_in, O, den, G, dS_out, dZ_out, saved, saved_bytes,
                                  dQ, dK, dV, dS_in, dZ_in, ws, ws_bytes, stream);
}

int la_causal_backward_varlen(const la_problem* p, const void* Q, const void* K, const void* V, const int32_t* lengths,
                              const float* S_in, const float* Z_in,
                              const void* O, const float* den, const void* G,
                              const float* dS_out, const float* dZ_out,
                              const void* saved, size_t saved_bytes,
                              void* dQ, void* dK, void* dV, float* dS_in, float* dZ_in,
                              void* ws, size_t ws_bytes, void* stream) {
    return causal_backward_common(p, Q, K, V, lengths, true, S_in, Z_in, O, den, G, dS_out, dZ_out, saved, saved_bytes,
                                  dQ, dK, dV, dS_in, dZ_in, ws, ws_bytes, stream);
}

int la_causal_backward(const la_problem* p, const void* Q, const void* K, const void* V,
                       const void* O, const float* den, const void* G,
                       const void* saved, size_t saved_bytes,
                       void* dQ, void* dK, void* dV,
                       void* ws, size_t ws_bytes, void* stream) {
    return la_causal_backward_from(p, Q, K, V, nullptr, nullptr, O, den, G, nullptr, nullptr, saved, saved_bytes,
                                   dQ, dK, dV, nullptr, nullptr, ws, ws_bytes, stream);
}

int la_recurrent_step(const la_problem* p, const void* q, const void* k, const void* v,
                      float* S, float* Z, void* out, void* stream) {
    if (int rc = check_problem(p, false)) return rc;
    LA_REQUIRE_PTR(q); LA_REQUIRE_PTR(k); LA_REQUIRE_PTR(v);
    LA_REQUIRE_PTR(S); LA_REQUIRE_PTR(Z); LA_REQUIRE_PTR(out);
    if (int rc = check_arch()) return rc;
    {
        la_problem one = *p;
        one.N = 1;
        const TensorBytes tb(one);
        LA_DEBUG_SPAN(q, tb.qk); LA_DEBUG_SPAN(k, tb.qk); LA_DEBUG_SPAN(v, tb.vo); LA_DEBUG_SPAN(out, tb.vo);
        LA_DEBUG_SPAN(S, tb.s); LA_DEBUG_SPAN(Z, tb.z);
    }
    // launched as a programmatic dependent: a decode loop's next step is scheduled while this one runs (the kernel
    // waits for its predecessor in the stream before it touches memory)
    return debug_finish(launch_recurrent_step(*p, q, k, v, S, Z, out, (cudaStream_t)stream, /*chained=*/true), stream);
}

int la_decode_layer_step(const la_problem* p, const void* x, const void* Wqkv, const void* Wo,
                         float* S, float* Z, void* y, void* ws, size_t ws_bytes, void* stream) {
    if (int rc = check_problem(p, false)) return rc;
    if (!decode_layer_supported(*p))
        return fail(LA_ERR_UNSUPPORTED, "the fused decode layer takes bf16 with D = M = 64 (got dtype %d, D=%lld, M=%lld)",
                    p->dtype, (long long)p->D, (long long)p->M);
    if (p->B * p->H * p->D >= (1LL << 31) || p->H * p->D > 65536)
        return fail(LA_ERR_UNSUPPORTED, "B * H * D must be below 2^31 and the model width H * D at most 65536");
    LA_REQUIRE_PTR(x); LA_REQUIRE_PTR(Wqkv); LA_REQUIRE_PTR(Wo);
    LA_REQUIRE_PTR(S); LA_REQUIRE_PTR(Z); LA_REQUIRE_PTR(y);
    if (y == x) return fail(LA_ERR_INVALID_ARG, "y must not alias x (x is read again for the residual while y is written)");
    if (int rc = check_ws(p, LA_OP_DECODE_LAYER, ws, ws_bytes)) return rc;
    if (int rc = check_arch()) return rc;
    {
        const size_t F = (size_t)(p->H * p->D), xb = (size_t)p->B * F * 2;
        const TensorBytes tb(*p);
        LA_DEBUG_SPAN(x, xb); LA_DEBUG_SPAN(y, xb); LA_DEBUG_SPAN(Wqkv, 3 * F * F * 2); LA_DEBUG_SPAN(Wo, F * F * 2);
        LA_DEBUG_SPAN(S, tb.s); LA_DEBUG_SPAN(Z, tb.z); LA_DEBUG_SPAN(ws, ws_bytes);
    }
    return debug_finish(decode_layer_step(*p, x, Wqkv, Wo, S, Z, y, ws, (cudaStream_t)stream), stream);
}

int la_recurrent_steps(const la_problem* p, const void* q, const void* k, const void* v,
                       float* S, float* Z, void* out, void* stream) {
    if (int rc = check_problem(p, true)) return rc;
    if (p->N == 0) return LA_OK;
    LA_REQUIRE_PTR(q); LA_REQUIRE_PTR(k); LA_REQUIRE_PTR(v);
    LA_REQUIRE_PTR(S); LA_REQUIRE_PTR(Z); LA_REQUIRE_PTR(out);
    if (int rc = check_arch()) return rc;
    {
        const TensorBytes tb(*p);
        LA_DEBUG_SPAN(q, tb.qk); LA_DEBUG_SPAN(k, tb.qk); LA_DEBUG_SPAN(v, tb.vo); LA_DEBUG_SPAN(out, tb.vo);
        LA_DEBUG_SPAN(S, tb.s); LA_DEBUG_SPAN(Z, tb.z);
    }
    return debug_finish(launch_recurrent_steps(*p, q, k, v, S, Z, out, (cudaStream_t)stream), stream);
}

int la_last_device_status(void* stream) {
    LA_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    int word = 0;
    LA_CUDA_TRY(cudaMemcpyFromSymbol(&word, g_device_status_word, sizeof(int)));
    if (word == 0) return LA_OK;
    int zero = 0;
    LA_CUDA_TRY(cudaMemcpyToSymbol(g_device_status_word, &zero, sizeof(int)));
    if (word & 8)
        return fail(LA_ERR_INVALID_ARG, "a saved buffer was written by a forward pass with another piece plan (another "
                                        "la_plan_override() setting or device): the backward pass computed nothing (device status 0x%x)", word);
    return fail(LA_ERR_DEVICE_TIMEOUT, "a kernel gave up on a bounded wait (device status 0x%x)", word);
}

}  // extern "C"
