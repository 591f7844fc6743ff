// Feature map (Eq. 7) as a stand-alone elementwise kernel, and the one-token
// recurrent step (Eq. 16-20, attention part).
#include "la_common.cuh"

namespace la {

// ---------------------------------------------------------------------------
// Feature map: y = phi(x) or phi'(x).  Bandwidth-bound; 16-byte accesses on the
// aligned body, four of them in flight per thread (a thread with one load outstanding
// leaves the memory system short of requests: 0.74 of the copy bandwidth against 0.9),
// scalar accesses on the ragged tail.  exp through ex2.approx (relative error 2^-22).
// ---------------------------------------------------------------------------
__device__ __forceinline__ float fm(float x, int deriv) {
    if (x > 0.f) return deriv ? 1.f : x + 1.f;
    return __expf(x);
}

template <typename T>
__global__ void __launch_bounds__(256)
feature_map_kernel(const T* __restrict__ x, T* __restrict__ y, int64_t n, int deriv) {
    constexpr int V = 16 / sizeof(T);
    constexpr int U = 4;                        // 16-byte vectors per thread and iteration
    const int64_t nvec = n / V;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    int64_t i = t0;
    for (; i + (U - 1) * stride < nvec; i += U * stride) {
        uint4 raw[U];
#pragma unroll
        for (int u = 0; u < U; ++u) raw[u] = __ldcs(reinterpret_cast<const uint4*>(x) + i + u * stride);
#pragma unroll
        for (int u = 0; u < U; ++u) {
            T* e = reinterpret_cast<T*>(&raw[u]);
#pragma unroll
            for (int j = 0; j < V; ++j) e[j] = from_f32<T>(fm(to_f32<T>(e[j]), deriv));
            __stcs(reinterpret_cast<uint4*>(y) + i + u * stride, raw[u]);
        }
    }
    for (; i < nvec; i += stride) {
        uint4 raw = reinterpret_cast<const uint4*>(x)[i];
        T* e = reinterpret_cast<T*>(&raw);
#pragma unroll
        for (int j = 0; j < V; ++j) e[j] = from_f32<T>(fm(to_f32<T>(e[j]), deriv));
        reinterpret_cast<uint4*>(y)[i] = raw;
    }
    for (int64_t k = nvec * V + t0; k < n; k += stride) y[k] = from_f32<T>(fm(to_f32<T>(x[k]), deriv));
}

int launch_feature_map(const void* x, void* y, int64_t n, int dtype, int deriv, cudaStream_t st) {
    if (n == 0) return LA_OK;
    const int threads = 256;
    const int64_t vec = dtype == LA_F32 ? 4 : 8;
    int64_t blocks = (n / vec + threads - 1) / threads;
    if (blocks < 1) blocks = 1;
    if (blocks > 148 * 8) blocks = 148 * 8;            // one resident wave: 8 blocks of 256 threads per SM
    if (dtype == LA_F32)
        feature_map_kernel<float><<<(unsigned)blocks, threads, 0, st>>>((const float*)x, (float*)y, n, deriv);
    else
        feature_map_kernel<__nv_bfloat16><<<(unsigned)blocks, threads, 0, st>>>(
            (const __nv_bfloat16*)x, (__nv_bfloat16*)y, n, deriv);
    LA_LAUNCHED();
    return LA_OK;
}

// ---------------------------------------------------------------------------
// Degree-2 polynomial kernel (Section 3.2.1): the exact feature map of sim(a, b) = (a . b)^2 is
// phi(x) = vec(x x^T), y[r][i*D + j] = x[r][i] x[r][j]; columns D*D .. C-1 are zero padding, so that
// the attention kernels (feature map = identity) can take C as their query/key dimension.
// Bandwidth-bound on the C-wide side: a thread writes (forward) eight consecutive columns with
// 16-byte stores; the D-wide row of x is re-read through L1.
// ---------------------------------------------------------------------------
// Thread layout of both kernels: threadIdx.x = position inside a row (group of eight columns / component i),
// threadIdx.y = row inside the block; no division by a run-time number per element.
template <typename T>
__global__ void __launch_bounds__(256)
poly2_map_kernel(const T* __restrict__ x, T* __restrict__ y, int64_t rows, int D, int C) {
    const int c0 = threadIdx.x << 3, DD = D * D;
    const int i0 = c0 / D, j0 = c0 - i0 * D;
    const int64_t stride = (int64_t)gridDim.x * blockDim.y;
    for (int64_t r = (int64_t)blockIdx.x * blockDim.y + threadIdx.y; r < rows; r += stride) {
        const T* xr = x + r * D;
        T out[8];
        if (sizeof(T) == 2 && D == 8) {          // a group is row i0 of x x^T: x_i0 times the 16-byte row of x
            const uint4 raw = __ldg(reinterpret_cast<const uint4*>(xr));
            const T* xe = reinterpret_cast<const T*>(&raw);
            const float xi = to_f32<T>(__ldg(xr + (i0 & 7)));     // (a group of padding columns has no row)
#pragma unroll
            for (int e = 0; e < 8; ++e) out[e] = from_f32<T>(c0 < DD ? xi * to_f32<T>(xe[e]) : 0.f);
        } else {
            int i = i0, j = j0;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                out[e] = from_f32<T>(c0 + e < DD ? to_f32<T>(__ldg(xr + i)) * to_f32<T>(__ldg(xr + j)) : 0.f);
                if (++j == D) { j = 0; ++i; }
            }
        }
        T* dst = y + r * C + c0;
        if (sizeof(T) == 2) {
            *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(out);
        } else {
            reinterpret_cast<uint4*>(dst)[0] = reinterpret_cast<const uint4*>(out)[0];
            reinterpret_cast<uint4*>(dst)[1] = reinterpret_cast<const uint4*>(out)[1];
        }
    }
}

// dx[r][i] = sum_j (dy[r][i*D + j] + dy[r][j*D + i]) x[r][j]; one thread per (r, i), fp32 sums.
template <typename T>
__global__ void __launch_bounds__(256)
poly2_map_backward_kernel(const T* __restrict__ x, const T* __restrict__ dy, T* __restrict__ dx,
                          int64_t rows, int D, int C) {
    const int i = threadIdx.x;
    const int64_t stride = (int64_t)gridDim.x * blockDim.y;
    for (int64_t r = (int64_t)blockIdx.x * blockDim.y + threadIdx.y; r < rows; r += stride) {
        const T* xr = x + r * D;
        const T* gr = dy + r * C;
        float s = 0.f;
        if (sizeof(T) == 2 && D == 8) {          // row i of dy and the row of x in one 16-byte load each
            const uint4 rawg = __ldg(reinterpret_cast<const uint4*>(gr + i * 8));
            const uint4 rawx = __ldg(reinterpret_cast<const uint4*>(xr));
            const T* ge = reinterpret_cast<const T*>(&rawg);
            const T* xe = reinterpret_cast<const T*>(&rawx);
#pragma unroll
            for (int j = 0; j < 8; ++j)
                s = fmaf(to_f32<T>(ge[j]) + to_f32<T>(__ldg(gr + j * 8 + i)), to_f32<T>(xe[j]), s);
        } else {
            for (int j = 0; j < D; ++j)
                s = fmaf(to_f32<T>(__ldg(gr + i * D + j)) + to_f32<T>(__ldg(gr + j * D + i)), to_f32<T>(__ldg(xr + j)), s);
        }
        dx[r * D + i] = from_f32<T>(s);
    }
}

// D = 8, C = 64, bf16 (the shape the tensor-core attention kernels take).  Forward: eight threads per row, one
// 16-byte group of columns each (thread i writes x_i times the row), four rows per thread in flight.  Backward:
// one thread per row with the whole 8x8 gradient block in registers, the rows staged through shared memory.
__global__ void __launch_bounds__(256)
poly2_map_d8_kernel(const __nv_bfloat16* __restrict__ x, __nv_bfloat16* __restrict__ y, int64_t rows) {
    constexpr int U = 4;
    const int i = threadIdx.x & 7;
    const int64_t stride = (int64_t)gridDim.x * 32;                     // rows per step of the whole grid
    int64_t r = (int64_t)blockIdx.x * 32 + (threadIdx.x >> 3);
    for (; r < rows; r += U * stride) {
        uint4 raw[U];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (r + u * stride < rows) raw[u] = __ldg(reinterpret_cast<const uint4*>(x + (r + u * stride) * 8));
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (r + u * stride >= rows) break;
            const __nv_bfloat16* xe = reinterpret_cast<const __nv_bfloat16*>(&raw[u]);
            float xi = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) xi = e == i ? __bfloat162float(xe[e]) : xi;
            uint32_t o[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const __nv_bfloat162 pr = __floats2bfloat162_rn(xi * __bfloat162float(xe[2 * e]), xi * __bfloat162float(xe[2 * e + 1]));
                o[e] = *reinterpret_cast<const uint32_t*>(&pr);
            }
            __stcs(reinterpret_cast<uint4*>(y + (r + u * stride) * 64 + i * 8), make_uint4(o[0], o[1], o[2], o[3]));
        }
    }
}

__global__ void __launch_bounds__(256)
poly2_map_backward_d8_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ dy,
                             __nv_bfloat16* __restrict__ dx, int64_t rows) {
    // 256 rows per step of a block: their gradient rows (128 bytes each) come in as one contiguous 32 KB run,
    // eight 16-byte loads per thread in flight, and are parked in shared memory with a row pitch of 144 bytes
    // (a quarter-warp's 16-byte reads of eight consecutive rows then fall into different banks); after the
    // barrier every thread takes one row with its whole 8x8 block in registers.
    constexpr int kPitch = 144;
    __shared__ __align__(16) uint8_t tile[256 * kPitch];
    const int tid = threadIdx.x;
    for (int64_t r0 = (int64_t)blockIdx.x * 256; r0 < rows; r0 += (int64_t)gridDim.x * 256) {
        const int64_t nrows = rows - r0 < 256 ? rows - r0 : 256;
        const uint4* src = reinterpret_cast<const uint4*>(dy + r0 * 64);
        uint4 raw[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int v = k * 256 + tid;                        // 16-byte vector of the run: row v / 8, group v % 8
            raw[k] = (v >> 3) < nrows ? __ldcs(src + v) : make_uint4(0u, 0u, 0u, 0u);
        }
        uint4 rawx = make_uint4(0u, 0u, 0u, 0u);
        if (tid < nrows) rawx = __ldg(reinterpret_cast<const uint4*>(x + (r0 + tid) * 8));
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int v = k * 256 + tid;
            *reinterpret_cast<uint4*>(tile + (v >> 3) * kPitch + (v & 7) * 16) = raw[k];
        }
        __syncthreads();
        const __nv_bfloat16* xe = reinterpret_cast<const __nv_bfloat16*>(&rawx);
        float xv[8], s[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) { xv[j] = __bfloat162float(xe[j]); s[j] = 0.f; }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint4 g4 = *reinterpret_cast<const uint4*>(tile + tid * kPitch + i * 16);
            const __nv_bfloat16* ge = reinterpret_cast<const __nv_bfloat16*>(&g4);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float g = __bfloat162float(ge[j]);        // g_ij: a term of dx_i (with x_j) and of dx_j (with x_i)
                s[i] = fmaf(g, xv[j], s[i]);
                s[j] = fmaf(g, xv[i], s[j]);
            }
        }
        if (tid < nrows) {
            uint32_t o[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const __nv_bfloat162 pr = __floats2bfloat162_rn(s[2 * e], s[2 * e + 1]);
                o[e] = *reinterpret_cast<const uint32_t*>(&pr);
            }
            *reinterpret_cast<uint4*>(dx + (r0 + tid) * 8) = make_uint4(o[0], o[1], o[2], o[3]);
        }
        __syncthreads();                                        // the tile is rewritten by the next step
    }
}

// blocks of (width, 256 / width) threads over the rows, at most 16 blocks per SM
static void poly2_launch_shape(int64_t rows, int width, dim3* grid, dim3* block) {
    const int rpb = 256 / width;
    int64_t blocks = (rows + rpb - 1) / rpb;
    if (blocks > 148 * 16) blocks = 148 * 16;
    *grid = dim3((unsigned)blocks);
    *block = dim3((unsigned)width, (unsigned)rpb);
}

int launch_poly2_map(const void* x, void* y, int64_t rows, int D, int C, int dtype, cudaStream_t st) {
    if (rows == 0) return LA_OK;
    if (dtype == LA_BF16 && D == 8 && C == 64) {
        int64_t blocks = (rows + 31) / 32;
        if (blocks > 148 * 8) blocks = 148 * 8;
        poly2_map_d8_kernel<<<(unsigned)blocks, 256, 0, st>>>((const __nv_bfloat16*)x, (__nv_bfloat16*)y, rows);
        LA_LAUNCHED();
        return LA_OK;
    }
    dim3 grid, block;
    poly2_launch_shape(rows, C >> 3, &grid, &block);
    if (dtype == LA_F32)
        poly2_map_kernel<float><<<grid, block, 0, st>>>((const float*)x, (float*)y, rows, D, C);
    else
        poly2_map_kernel<__nv_bfloat16><<<grid, block, 0, st>>>((const __nv_bfloat16*)x, (__nv_bfloat16*)y, rows, D, C);
    LA_LAUNCHED();
    return LA_OK;
}

int launch_poly2_map_backward(const void* x, const void* dy, void* dx, int64_t rows, int D, int C, int dtype,
                              cudaStream_t st) {
    if (rows == 0) return LA_OK;
    if (dtype == LA_BF16 && D == 8 && C == 64) {
        int64_t blocks = (rows + 255) / 256;
        if (blocks > 148 * 6) blocks = 148 * 6;             // 36 KB of shared memory each
        poly2_map_backward_d8_kernel<<<(unsigned)blocks, 256, 0, st>>>((const __nv_bfloat16*)x, (const __nv_bfloat16*)dy,
                                                                      (__nv_bfloat16*)dx, rows);
        LA_LAUNCHED();
        return LA_OK;
    }
    dim3 grid, block;
    poly2_launch_shape(rows, D, &grid, &block);
    if (dtype == LA_F32)
        poly2_map_backward_kernel<float><<<grid, block, 0, st>>>((const float*)x, (const float*)dy, (float*)dx, rows, D, C);
    else
        poly2_map_backward_kernel<__nv_bfloat16><<<grid, block, 0, st>>>(
            (const __nv_bfloat16*)x, (const __nv_bfloat16*)dy, (__nv_bfloat16*)dx, rows, D, C);
    LA_LAUNCHED();
    return LA_OK;
}

// ---------------------------------------------------------------------------
// Recurrent step.  One CTA of 128 threads per (batch, head) state.  The D x M
// fp32 state is streamed HBM -> registers -> HBM exactly once with 16-byte
// accesses: a thread owns four consecutive columns of every RPP-th row, so a
// warp covers whole 128-byte lines.  All state loads are issued before anything
// else is waited on.  phi(q)^T S is reduced with warp shuffles and one shared
// memory hop across the four warps; phi(q)^T Z likewise.
// ---------------------------------------------------------------------------
// kEarlyState (the decode layer's use only): the state is read BEFORE the dependency wait.  The kernel in
// front is then the projection of the same call, which never touches the state, waited for everything before it
// and only then let this kernel be scheduled, so the last writer of the state has completed: the state, which
// is all the traffic of this kernel, streams in while that projection runs.
template <typename T, int D, int M, bool kEarlyState = false>
__global__ void __launch_bounds__(128)
recurrent_step_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                      float* __restrict__ S, float* __restrict__ Z, T* __restrict__ out,
                      float eps, int phi) {
    constexpr int TPR = M / 4;        // threads per state row (one float4 each)
    constexpr int RPP = 128 / TPR;    // rows covered per pass of the CTA
    constexpr int PASSES = D / RPP;
    static_assert(D % RPP == 0 && PASSES >= 1, "unsupported state shape");

    __shared__ float sq[D], sk[D];
    __shared__ __align__(16) float sv[M];
    __shared__ __align__(16) float spart[4][M];
    __shared__ float sden[4];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t bh = blockIdx.x;
    const int c4 = tid % TPR, r0 = tid / TPR;

    // When launched as a programmatic dependent of the kernel before it in the stream (the decode layer does
    // that), this is where that kernel's results become visible; in an ordinary launch both are no-ops.
    float4* Sp = reinterpret_cast<float4*>(S + bh * (int64_t)(D * M));
    float4 s[PASSES];
    if (kEarlyState) {
#pragma unroll
        for (int p = 0; p < PASSES; ++p) s[p] = Sp[(r0 + p * RPP) * TPR + c4];
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (!kEarlyState) {
#pragma unroll
        for (int p = 0; p < PASSES; ++p) s[p] = Sp[(r0 + p * RPP) * TPR + c4];
    }

    float zq = 0.f;
    if (tid < D) {
        float kd = phi_apply(to_f32<T>(k[bh * D + tid]), phi);
        float qd = phi_apply(to_f32<T>(q[bh * D + tid]), phi);
        float z = Z[bh * D + tid] + kd;
        Z[bh * D + tid] = z;
        sk[tid] = kd;
        sq[tid] = qd;
        zq = qd * z;
    }
    if (tid < M) sv[tid] = to_f32<T>(v[bh * M + tid]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) zq += __shfl_xor_sync(0xffffffffu, zq, off);
    if (lane == 0) sden[warp] = zq;
    __syncthreads();

    const float4 vv = reinterpret_cast<const float4*>(sv)[c4];
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int p = 0; p < PASSES; ++p) {
        const int d = r0 + p * RPP;
        const float kd = sk[d], qd = sq[d];
        s[p].x = fmaf(kd, vv.x, s[p].x);
        s[p].y = fmaf(kd, vv.y, s[p].y);
        s[p].z = fmaf(kd, vv.z, s[p].z);
        s[p].w = fmaf(kd, vv.w, s[p].w);
        Sp[d * TPR + c4] = s[p];
        acc.x = fmaf(qd, s[p].x, acc.x);
        acc.y = fmaf(qd, s[p].y, acc.y);
        acc.z = fmaf(qd, s[p].z, acc.z);
        acc.w = fmaf(qd, s[p].w, acc.w);
    }
#pragma unroll
    for (int off = 16; off >= TPR; off >>= 1) {
        acc.x += __shfl_xor_sync(0xffffffffu, acc.x, off);
        acc.y += __shfl_xor_sync(0xffffffffu, acc.y, off);
        acc.z += __shfl_xor_sync(0xffffffffu, acc.z, off);
        acc.w += __shfl_xor_sync(0xffffffffu, acc.w, off);
    }
    if (lane < TPR) reinterpret_cast<float4*>(spart[warp])[lane] = acc;
    __syncthreads();
    if (tid < M) {
        const float den = sden[0] + sden[1] + sden[2] + sden[3] + eps;
        const float num = spart[0][tid] + spart[1][tid] + spart[2][tid] + spart[3][tid];
        out[bh * M + tid] = from_f32<T>(num / den);
    }
}

// Any D, M (multiples of 8 up to 128): thread m owns column m of the state.
template <typename T>
__global__ void __launch_bounds__(128)
recurrent_step_general_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                              float* __restrict__ S, float* __restrict__ Z, T* __restrict__ out,
                              int D, int M, float eps, int phi) {
    __shared__ float sq[128], sk[128], sden[4];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t bh = blockIdx.x;
    float zq = 0.f;
    if (tid < D) {
        float kd = phi_apply(to_f32<T>(k[bh * D + tid]), phi);
        float qd = phi_apply(to_f32<T>(q[bh * D + tid]), phi);
        float z = Z[bh * D + tid] + kd;
        Z[bh * D + tid] = z;
        sk[tid] = kd;
        sq[tid] = qd;
        zq = qd * z;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) zq += __shfl_xor_sync(0xffffffffu, zq, off);
    if (lane == 0) sden[warp] = zq;
    __syncthreads();
    if (tid < M) {
        const float vm = to_f32<T>(v[bh * M + tid]);
        float* Sp = S + bh * (int64_t)D * M + tid;
        float num = 0.f;
        for (int d = 0; d < D; ++d) {
            float s = fmaf(sk[d], vm, Sp[(int64_t)d * M]);
            Sp[(int64_t)d * M] = s;
            num = fmaf(sq[d], s, num);
        }
        out[bh * M + tid] = from_f32<T>(num / (sden[0] + sden[1] + sden[2] + sden[3] + eps));
    }
}

// ---------------------------------------------------------------------------
// Several recurrent steps in one launch (Eq. 18-20 for t = 1..N with the inputs of all steps
// given): the state is read from HBM once, kept in registers across the steps (Z by the first D
// threads) and written back once; per step only q_t, k_t, v_t come in and out_t goes out.  The
// arithmetic of a step is that of recurrent_step_kernel, in the same order: the results are
// bit-identical to N single-step launches.  Shared buffers alternate between steps, so two
// barriers per step suffice.
// q, k: [B,H,N,D]; v, out: [B,H,N,M].
// ---------------------------------------------------------------------------
template <typename T, int D, int M>
__global__ void __launch_bounds__(128)
recurrent_steps_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                       float* __restrict__ S, float* __restrict__ Z, T* __restrict__ out,
                       int64_t N, float eps, int phi) {
    constexpr int TPR = M / 4;
    constexpr int RPP = 128 / TPR;
    constexpr int PASSES = D / RPP;
    static_assert(D % RPP == 0 && PASSES >= 1, "unsupported state shape");

    __shared__ float sq[2][D], sk[2][D];
    __shared__ __align__(16) float sv[2][M];
    __shared__ __align__(16) float spart[2][4][M];
    __shared__ float sden[2][4];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t bh = blockIdx.x;
    const int c4 = tid % TPR, r0 = tid / TPR;

    float4* Sp = reinterpret_cast<float4*>(S + bh * (int64_t)(D * M));
    float4 s[PASSES];
#pragma unroll
    for (int p = 0; p < PASSES; ++p) s[p] = Sp[(r0 + p * RPP) * TPR + c4];
    float z = tid < D ? Z[bh * D + tid] : 0.f;

    const T* qb = q + bh * N * D;
    const T* kb = k + bh * N * D;
    const T* vb = v + bh * N * M;
    T* ob = out + bh * N * M;
    #pragma unroll 1
    for (int64_t t = 0; t < N; ++t) {
        const int b = (int)(t & 1);
        float zq = 0.f;
        if (tid < D) {
            const float kd = phi_apply(to_f32<T>(kb[t * D + tid]), phi);
            const float qd = phi_apply(to_f32<T>(qb[t * D + tid]), phi);
            z += kd;
            sk[b][tid] = kd;
            sq[b][tid] = qd;
            zq = qd * z;
        }
        if (tid < M) sv[b][tid] = to_f32<T>(vb[t * M + tid]);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) zq += __shfl_xor_sync(0xffffffffu, zq, off);
        if (lane == 0) sden[b][warp] = zq;
        __syncthreads();

        const float4 vv = reinterpret_cast<const float4*>(sv[b])[c4];
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int p = 0; p < PASSES; ++p) {
            const int d = r0 + p * RPP;
            const float kd = sk[b][d], qd = sq[b][d];
            s[p].x = fmaf(kd, vv.x, s[p].x);
            s[p].y = fmaf(kd, vv.y, s[p].y);
            s[p].z = fmaf(kd, vv.z, s[p].z);
            s[p].w = fmaf(kd, vv.w, s[p].w);
            acc.x = fmaf(qd, s[p].x, acc.x);
            acc.y = fmaf(qd, s[p].y, acc.y);
            acc.z = fmaf(qd, s[p].z, acc.z);
            acc.w = fmaf(qd, s[p].w, acc.w);
        }
#pragma unroll
        for (int off = 16; off >= TPR; off >>= 1) {
            acc.x += __shfl_xor_sync(0xffffffffu, acc.x, off);
            acc.y += __shfl_xor_sync(0xffffffffu, acc.y, off);
            acc.z += __shfl_xor_sync(0xffffffffu, acc.z, off);
            acc.w += __shfl_xor_sync(0xffffffffu, acc.w, off);
        }
        if (lane < TPR) reinterpret_cast<float4*>(spart[b][warp])[lane] = acc;
        __syncthreads();
        if (tid < M) {
            const float den = sden[b][0] + sden[b][1] + sden[b][2] + sden[b][3] + eps;
            const float num = spart[b][0][tid] + spart[b][1][tid] + spart[b][2][tid] + spart[b][3][tid];
            ob[t * M + tid] = from_f32<T>(num / den);
        }
    }
#pragma unroll
    for (int p = 0; p < PASSES; ++p) Sp[(r0 + p * RPP) * TPR + c4] = s[p];
    if (tid < D) Z[bh * D + tid] = z;
}

// Any D, M (multiples of 8 up to 128): the single-step arithmetic of recurrent_step_general_kernel looped
// over the steps; the state stays in global memory (cached) between them.
template <typename T>
__global__ void __launch_bounds__(128)
recurrent_steps_general_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                               float* __restrict__ S, float* __restrict__ Z, T* __restrict__ out,
                               int64_t N, int D, int M, float eps, int phi) {
    __shared__ float sq[2][128], sk[2][128], sden[2][4];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t bh = blockIdx.x;
    float z = tid < D ? Z[bh * D + tid] : 0.f;
    #pragma unroll 1
    for (int64_t t = 0; t < N; ++t) {
        const int b = (int)(t & 1);
        float zq = 0.f;
        if (tid < D) {
            const float kd = phi_apply(to_f32<T>(k[(bh * N + t) * D + tid]), phi);
            const float qd = phi_apply(to_f32<T>(q[(bh * N + t) * D + tid]), phi);
            z += kd;
            sk[b][tid] = kd;
            sq[b][tid] = qd;
            zq = qd * z;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) zq += __shfl_xor_sync(0xffffffffu, zq, off);
        if (lane == 0) sden[b][warp] = zq;
        __syncthreads();
        if (tid < M) {
            const float vm = to_f32<T>(v[(bh * N + t) * M + tid]);
            float* Sp = S + bh * (int64_t)D * M + tid;
            float num = 0.f;
            for (int d = 0; d < D; ++d) {
                float sv = fmaf(sk[b][d], vm, Sp[(int64_t)d * M]);
                Sp[(int64_t)d * M] = sv;
                num = fmaf(sq[b][d], sv, num);
            }
            out[(bh * N + t) * M + tid] = from_f32<T>(num / (sden[b][0] + sden[b][1] + sden[b][2] + sden[b][3] + eps));
        }
    }
    if (tid < D) Z[bh * D + tid] = z;
}

template <typename T>
static int recurrent_steps_dispatch(const la_problem& p, const void* q, const void* k, const void* v,
                                    float* S, float* Z, void* out, cudaStream_t st) {
    const unsigned grid = (unsigned)(p.B * p.H);
    const T *qq = (const T*)q, *kk = (const T*)k, *vv = (const T*)v;
    T* oo = (T*)out;
#define LA_RS_CASE(DD, MM)                                                                     \
    if (p.D == DD && p.M == MM) {                                                              \
        recurrent_steps_kernel<T, DD, MM><<<grid, 128, 0, st>>>(qq, kk, vv, S, Z, oo, p.N, p.eps, p.phi); \
        LA_LAUNCHED();                                                       \
        return LA_OK;                                                                          \
    }
    LA_RS_CASE(32, 32) LA_RS_CASE(32, 64) LA_RS_CASE(64, 32) LA_RS_CASE(64, 64)
    LA_RS_CASE(64, 128) LA_RS_CASE(128, 64) LA_RS_CASE(128, 128)
#undef LA_RS_CASE
    recurrent_steps_general_kernel<T><<<grid, 128, 0, st>>>(qq, kk, vv, S, Z, oo, p.N, (int)p.D, (int)p.M,
                                                            p.eps, p.phi);
    LA_LAUNCHED();
    return LA_OK;
}

int launch_recurrent_steps(const la_problem& p, const void* q, const void* k, const void* v,
                           float* S, float* Z, void* out, cudaStream_t st) {
    prof_begin(kProfRecurrent, st);
    const int rc = p.dtype == LA_F32 ? recurrent_steps_dispatch<float>(p, q, k, v, S, Z, out, st)
                                     : recurrent_steps_dispatch<__nv_bfloat16>(p, q, k, v, S, Z, out, st);
    prof_end(kProfRecurrent, st);
    return rc;
}

template <typename T>
static int recurrent_dispatch(const la_problem& p, const void* q, const void* k, const void* v,
                              float* S, float* Z, void* out, cudaStream_t st, bool chained, bool early_state) {
    const unsigned grid = (unsigned)(p.B * p.H);
    const T *qq = (const T*)q, *kk = (const T*)k, *vv = (const T*)v;
    T* oo = (T*)out;
    if (chained && p.D == 64 && p.M == 64) {        // a programmatic dependent of the kernel before it: see the kernel
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr.val.programmaticStreamSerializationAllowed = 1;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3(128);
        cfg.stream = st;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        if (early_state) LA_CUDA_TRY(cudaLaunchKernelEx(&cfg, recurrent_step_kernel<T, 64, 64, true>, qq, kk, vv, S, Z, oo, p.eps, p.phi));
        else LA_CUDA_TRY(cudaLaunchKernelEx(&cfg, recurrent_step_kernel<T, 64, 64>, qq, kk, vv, S, Z, oo, p.eps, p.phi));
        note_launch();
        return LA_OK;
    }
#define LA_RS_CASE(DD, MM)                                                                     \
    if (p.D == DD && p.M == MM) {                                                              \
        recurrent_step_kernel<T, DD, MM><<<grid, 128, 0, st>>>(qq, kk, vv, S, Z, oo, p.eps, p.phi); \
        LA_LAUNCHED();                                                       \
        return LA_OK;                                                                          \
    }
    LA_RS_CASE(32, 32) LA_RS_CASE(32, 64) LA_RS_CASE(64, 32) LA_RS_CASE(64, 64)
    LA_RS_CASE(64, 128) LA_RS_CASE(128, 64) LA_RS_CASE(128, 128)
#undef LA_RS_CASE
    recurrent_step_general_kernel<T><<<grid, 128, 0, st>>>(qq, kk, vv, S, Z, oo, (int)p.D, (int)p.M,
                                                           p.eps, p.phi);
    LA_LAUNCHED();
    return LA_OK;
}

int launch_recurrent_step(const la_problem& p, const void* q, const void* k, const void* v,
                          float* S, float* Z, void* out, cudaStream_t st, bool chained, bool early_state) {
    prof_begin(kProfRecurrent, st);
    const int rc = p.dtype == LA_F32 ? recurrent_dispatch<float>(p, q, k, v, S, Z, out, st, chained, early_state)
                                     : recurrent_dispatch<__nv_bfloat16>(p, q, k, v, S, Z, out, st, chained, early_state);
    prof_end(kProfRecurrent, st);
    return rc;
}

}  // namespace la
