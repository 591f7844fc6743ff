// la_linear_attention_noalloc: the non-causal forward for callers that cannot allocate.
//
// The general non-causal kernels split every (batch, head) sequence over several CTAs
// and need scratch memory for the per-split partial sums of phi(K)^T [V | 1].  The
// regular entry point takes that scratch from the caller.  Some callers have no way to
// provide it: code running inside a framework's memory-planning phase or under a memory
// budget that forbids new device allocations, plugin interfaces that hand over input and
// output buffers only, and real-time loops where a cudaMalloc (which may synchronise the
// device) is not acceptable.  For them the scratch lives in a fixed array in the
// library's device image: every GPU that loads the library holds
// LA_NOALLOC_SCRATCH_BYTES until the process exits, whether the entry point is used or not.
#include <mutex>

#include "la_common.cuh"

namespace la {
namespace {

// File-scope device array: in HOST code this name is only a stand-in for the symbol, not
// a device address; the address is looked up once per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_noalloc_scratch[LA_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the scratch array on the CURRENT device (set-up on first use).
int scratch_for_current_device(void** out) {
    int dev = 0;
    LA_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return fail(LA_ERR_UNSUPPORTED, "device ordinal %d is out of range", dev);
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(scratch)");
        if (!p) return fail(LA_ERR_CUDA, "the scratch symbol has no device address");
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return LA_OK;
}

}  // namespace
}  // namespace la

using namespace la;

extern "C" int la_linear_attention_noalloc(const la_problem* p, const void* Q, const void* K, const void* V,
                                           void* O, float* den, float* KV, float* Zs, void* stream) {
    if (int rc = check_problem(p, true)) return rc;        // the same checks as la_linear_attention()
    if (p->N == 0) return LA_OK;
    const void* required[4] = {Q, K, V, O};
    for (const void* ptr : required) {
        if (!ptr) return fail(LA_ERR_INVALID_ARG, "Q, K, V and O must not be NULL");
        if (!aligned16(ptr)) return fail(LA_ERR_INVALID_ARG, "Q, K, V and O must be 16-byte aligned");
    }
    if ((den && !aligned16(den)) || (KV && !aligned16(KV)) || (Zs && !aligned16(Zs)))
        return fail(LA_ERR_INVALID_ARG, "den, KV and Zs must be 16-byte aligned");

    const size_t need = general_workspace_bytes(*p, LA_OP_LINEAR_FORWARD);
    if (need > (size_t)LA_NOALLOC_SCRATCH_BYTES)
        return fail(LA_ERR_WORKSPACE,
                    "this problem needs %zu bytes of scratch but the built-in array holds %zu: use "
                    "la_linear_attention with a caller-provided workspace",
                    need, (size_t)LA_NOALLOC_SCRATCH_BYTES);
    if (int rc = check_arch()) return rc;

    void* scratch = nullptr;
    if (int rc = scratch_for_current_device(&scratch)) return rc;
    // Every partial sum the second kernel reads is written by the first one in the same call,
    // so nothing in the array has to start at zero.
    return general_linear_forward(*p, Q, K, V, nullptr, O, den, KV, Zs, nullptr, scratch, (cudaStream_t)stream);
}
