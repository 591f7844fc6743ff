// Tensor-core kernels: dispatch (kernels are added per operation).
#include "la_tc.cuh"

namespace la {

bool tc_supported(const la_problem&, int) { return false; }
size_t tc_workspace_bytes(const la_problem&, int) { return 0; }

int tc_causal_forward(const la_problem&, const void*, const void*, const void*, void*, float*, float*,
                      float*, void*, cudaStream_t) {
    return fail(LA_ERR_UNSUPPORTED, "tensor-core causal forward not available");
}
int tc_causal_backward(const la_problem&, const void*, const void*, const void*, const void*, void*, void*,
                       void*, void*, cudaStream_t) {
    return fail(LA_ERR_UNSUPPORTED, "tensor-core causal backward not available");
}
int tc_linear_forward(const la_problem&, const void*, const void*, const void*, void*, float*, float*,
                      float*, void*, cudaStream_t) {
    return fail(LA_ERR_UNSUPPORTED, "tensor-core linear forward not available");
}
int tc_linear_backward(const la_problem&, const void*, const void*, const void*, const void*, void*, void*,
                       void*, void*, cudaStream_t) {
    return fail(LA_ERR_UNSUPPORTED, "tensor-core linear backward not available");
}

}  // namespace la
