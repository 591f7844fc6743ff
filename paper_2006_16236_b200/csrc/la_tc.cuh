// Tensor-core (tcgen05 / TMA) kernels for bf16 problems: interface to the API layer.
#pragma once
#include "la_common.cuh"

namespace la {

// True when problem p / operation op runs on the tensor-core kernels.
bool tc_supported(const la_problem& p, int op);
size_t tc_workspace_bytes(const la_problem& p, int op);

// pieces, parts, piece_begin[], piece_first_part[], part_begin[], launch_order[] (see la_causal_plan)
int tc_causal_plan(const la_problem& p, int32_t* out, int capacity);

namespace tc {
// process-wide overrides of the automatic plans (see la_plan_override)
void set_plan_override(int causal_pieces, int causal_short, int linear_splits);
// In all of these: lengths ([B] int32, device, or null) = real positions per batch element of a right-padded
// ragged batch; saved (or null) = where the forward leaves what the backward pass can reuse.
size_t causal_forward_workspace(const la_problem& p);
size_t causal_saved_bytes(const la_problem& p);
int causal_forward(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths, const float* S_in,
                   const float* Z_in, void* O, float* den, float* S_out, float* Z_out, void* saved, void* ws,
                   cudaStream_t st);
size_t causal_backward_workspace(const la_problem& p);
int causal_backward(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths, const void* G,
                    const StateArgs& sa, const void* saved, void* dQ, void* dK, void* dV, void* ws, cudaStream_t st);
size_t linear_forward_workspace(const la_problem& p);
size_t linear_backward_workspace(const la_problem& p);
int linear_forward(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths, void* O,
                   float* den, float* KV, float* Zs, void* saved, void* ws, cudaStream_t st);
int linear_backward(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths,
                    const void* saved, const void* G, void* dQ, void* dK, void* dV, void* ws, cudaStream_t st);
// random Fourier features (la_rff.cu)
bool rff_supported(int64_t rows, int64_t D, int64_t C, int dtype);
int rff_forward(const void* x, const void* W, void* y, int64_t rows, int D, int C, cudaStream_t st);
int rff_backward(const void* x, const void* W, const void* dy, void* dx, int64_t rows, int D, int C, cudaStream_t st);
}  // namespace tc

}  // namespace la
