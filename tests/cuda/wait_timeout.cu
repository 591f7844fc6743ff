// Test-only translation unit (built by tests/test_gpu_bounded_wait.py, never part of libla.so): one CTA
// runs the library's bounded mbarrier wait, from the same header as the product kernels, on a barrier
// that nobody arrives at.  The wait has to give up after its poll limit (built here with a limit of a
// thousand polls: a few milliseconds), OR its code into the status word and return false, after which
// the kernel leaves normally.  Nothing traps, faults or spins beyond that limit.
#include <cuda_runtime.h>

#include "la_sm100.cuh"

using namespace la::sm100;

// out[0]: what the wait on the silent barrier returned (1 = completed, 0 = gave up); out[1]: what a wait
// on a barrier that a second thread does arrive at returned; out[2]: polls-limit the unit was built with.
__global__ void wait_kernel(int* status, int* out) {
    __shared__ uint64_t silent, served;
    if (threadIdx.x == 0) {
        mbar_init(&silent, 1);
        mbar_init(&served, 1);
        fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        out[1] = mbar_wait(&served, 0, status, kStatusMmaTimeout) ? 1 : 0;
        out[0] = mbar_wait(&silent, 0, status, kStatusPipeTimeout) ? 1 : 0;
        out[2] = (int)kWaitLimit;
    } else if (threadIdx.x == 32) {
        mbar_arrive(&served);
    }
}

// Host entry for ctypes: runs the kernel once on the current device; status_and_out = {status word, out[0..2]}.
// Returns the CUDA error code of the run (0: the context is intact).
extern "C" int run_wait_timeout(int* status_and_out) {
    int* dev = nullptr;
    cudaError_t e = cudaMalloc(&dev, 4 * sizeof(int));
    if (e != cudaSuccess) return (int)e;
    cudaMemset(dev, 0, 4 * sizeof(int));
    wait_kernel<<<1, 64>>>(dev, dev + 1);
    e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(status_and_out, dev, 4 * sizeof(int), cudaMemcpyDeviceToHost);
    cudaFree(dev);
    return (int)e;
}
