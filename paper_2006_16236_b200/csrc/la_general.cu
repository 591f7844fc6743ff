// General kernels: any D, M (multiples of 8 up to 128), any N, fp32 or bf16 I/O,
// fp32 arithmetic on the CUDA cores.  They serve fp32 problems (bf16 tensor-core
// products cannot hold the fp32 tolerance) and every shape the tensor-core
// kernels do not cover.  All four are chunked restatements of Algorithm 1 on the
// values extended by a ones column:
//     Vt_j = [V_j, 1],   St = [S | Z]  (D x (M+1)),   [num_i | den_i] = phi(Q_i)^T St_i.
// For a chunk c of T consecutive positions with L the lower-triangular mask,
//     [num|den]_c = ((q_c k_c^T) o L) Vt_c + q_c St_{c-1},   St_c = St_{c-1} + k_c^T Vt_c,
// which is Eq. 9-12 with the sum over j <= i split at the chunk boundary.
#include "la_common.cuh"

namespace la {

namespace {

constexpr int T = 32;          // positions per chunk
constexpr int THREADS = 256;

struct Dims {
    int D, M;      // feature / value dims
    int DS;        // row stride of q/k tiles (D + 1: conflict-free column walks)
    int MS;        // row stride of extended value tiles and states (M + 1)
};

__device__ __forceinline__ Dims make_dims(int D, int M) { return Dims{D, M, D + 1, M + 1}; }

// Register-blocked product of small shared-memory matrices:
//   out(i, j) = sum_{k < K1} A1(i, k) B1(k, j) + sum_{k < K2} A2(i, k) B2(k, j),   i < I, j < J,
// with X(i, k) = x[i * xi + k * xk] (any strides; I a multiple of RI, J of RJ; K2 = 0: one product).  A thread
// owns RI x RJ outputs spread over the matrix (i = il + r I/RI, j = jl + s J/RJ), so that the lanes of a
// warp read consecutive j of B (consecutive or padded-stride addresses) and broadcast A: RI + RJ loads feed
// RI * RJ multiply-adds.  `store(i, j, value)` consumes the results.
struct Mat { const float* p; int s0, s1; };      // element (a, b) at p[a * s0 + b * s1]

template <int RI, int RJ, typename Store>
__device__ __forceinline__ void block_product(int I, int J, Mat A1, Mat B1, int K1, Mat A2, Mat B2, int K2, Store store) {
    const int ni = I / RI, nj = J / RJ;
    for (int tile = threadIdx.x; tile < ni * nj; tile += THREADS) {
        const int il = tile / nj, jl = tile - il * nj;
        float acc[RI][RJ];
#pragma unroll
        for (int r = 0; r < RI; ++r)
#pragma unroll
            for (int c = 0; c < RJ; ++c) acc[r][c] = 0.f;
        for (int pass = 0; pass < 2; ++pass) {
            const Mat A = pass ? A2 : A1, B = pass ? B2 : B1;
            const int K = pass ? K2 : K1;
            const float* a0 = A.p + il * A.s0;
            const float* b0 = B.p + jl * B.s1;
#pragma unroll 4
            for (int k = 0; k < K; ++k) {
                float a[RI], b[RJ];
#pragma unroll
                for (int r = 0; r < RI; ++r) a[r] = a0[r * ni * A.s0 + k * A.s1];
#pragma unroll
                for (int c = 0; c < RJ; ++c) b[c] = b0[k * B.s0 + c * nj * B.s1];
#pragma unroll
                for (int r = 0; r < RI; ++r)
#pragma unroll
                    for (int c = 0; c < RJ; ++c) acc[r][c] = fmaf(a[r], b[c], acc[r][c]);
            }
        }
#pragma unroll
        for (int r = 0; r < RI; ++r)
#pragma unroll
            for (int c = 0; c < RJ; ++c) store(il + r * ni, jl + c * nj, acc[r][c]);
    }
}

// A chunk of rows ([cn][cols] of IO, contiguous in global memory, 16-byte aligned: chunks start at multiples
// of T rows and cols is a multiple of 8) travels as up to FETCH 16-byte groups per thread, all requested
// before any is used; rows cn..T-1 (beyond the sequence) read as zero bits.
constexpr int FETCH = 4;       // T * 128 columns * 4 bytes / 16 bytes / THREADS

template <typename IO>
__device__ __forceinline__ void fetch_rows(uint4 (&r)[FETCH], const IO* src, int cn, int cols) {
    constexpr int VEC = 16 / (int)sizeof(IO);
    const int total = cn * (cols / VEC);
#pragma unroll
    for (int u = 0; u < FETCH; ++u) {
        const int g = threadIdx.x + u * THREADS;
        r[u] = g < total ? __ldg(reinterpret_cast<const uint4*>(src) + g) : make_uint4(0u, 0u, 0u, 0u);
    }
}

// dst[i][c] = f(i, value) for the fetched rows (i < cn), 0 for the padded rows (zero in feature space: a
// padded key contributes nothing to any sum).
template <typename IO, typename F>
__device__ __forceinline__ void store_rows(float* dst, const uint4 (&r)[FETCH], int cn, int cols, int stride, F f) {
    constexpr int VEC = 16 / (int)sizeof(IO);
    const int gpr = cols / VEC, all = T * gpr;
#pragma unroll
    for (int u = 0; u < FETCH; ++u) {
        const int g = threadIdx.x + u * THREADS;
        if (g < all) {
            const int i = g / gpr, c0 = (g - i * gpr) * VEC;
            const IO* e = reinterpret_cast<const IO*>(&r[u]);
#pragma unroll
            for (int j = 0; j < VEC; ++j) dst[i * stride + c0 + j] = i < cn ? f(i, to_f32<IO>(e[j])) : 0.f;
        }
    }
}

// dst[i][d] = phi(x[i][d])
template <typename IO>
__device__ __forceinline__ void store_mapped(float* dst, const uint4 (&r)[FETCH], int cn, int D, int DS, int phi) {
    store_rows<IO>(dst, r, cn, D, DS, [phi](int, float x) { return phi_apply(x, phi); });
}

// dst[i][0..M) = x[i][:], dst[i][M] = 1 (the ones column); padded rows are 0.
template <typename IO>
__device__ __forceinline__ void store_values_ext(float* dst, const uint4 (&r)[FETCH], int cn, int M, int MS) {
    store_rows<IO>(dst, r, cn, M, MS, [](int, float x) { return x; });
    for (int i = threadIdx.x; i < T; i += THREADS) dst[i * MS + M] = i < cn ? 1.f : 0.f;
}

// P[i][j] = q_i . k_j for j <= i (causal) else 0.
__device__ void masked_scores(float* P, const float* q, const float* k, int D, int DS) {
    block_product<2, 2>(T, T, Mat{q, DS, 1}, Mat{k, 1, DS}, D, Mat{q, 0, 0}, Mat{k, 0, 0}, 0,
                        [&](int i, int j, float v) { P[i * (T + 1) + j] = j <= i ? v : 0.f; });
}

// nd[i][e] = sum_{j<=i} P[i][j] vt[j][e] + sum_d q[i][d] St[d][e]   (e in [0, M])
__device__ void numerator_denominator(float* nd, const float* P, const float* vt, const float* q,
                                      const float* St, const Dims& dm, bool causal_part) {
    // (P is zero right of the diagonal: the sum over all j of the chunk is the causal one)
    block_product<4, 4>(T, dm.M, Mat{q, dm.DS, 1}, Mat{St, dm.MS, 1}, dm.D, Mat{P, T + 1, 1}, Mat{vt, dm.MS, 1},
                        causal_part ? T : 0, [&](int i, int e, float v) { nd[i * dm.MS + e] = v; });
    for (int i = threadIdx.x; i < T; i += THREADS) {            // the normaliser column e = M
        float s = 0.f;
        if (causal_part)
            for (int j = 0; j <= i; ++j) s = fmaf(P[i * (T + 1) + j], vt[j * dm.MS + dm.M], s);
        for (int d = 0; d < dm.D; ++d) s = fmaf(q[i * dm.DS + d], St[d * dm.MS + dm.M], s);
        nd[i * dm.MS + dm.M] = s;
    }
}

// St[d][e] += sum_i x[i][d] y[i][e]   (rank-T update of a D x (M+1) state)
__device__ void state_update(float* St, const float* x, const float* y, const Dims& dm) {
    block_product<4, 4>(dm.D, dm.M, Mat{x, 1, dm.DS}, Mat{y, dm.MS, 1}, T, Mat{x, 0, 0}, Mat{y, 0, 0}, 0,
                        [&](int d, int e, float v) { St[d * dm.MS + e] += v; });
    for (int d = threadIdx.x; d < dm.D; d += THREADS) {         // column e = M
        float s = St[d * dm.MS + dm.M];
        for (int i = 0; i < T; ++i) s = fmaf(x[i * dm.DS + d], y[i * dm.MS + dm.M], s);
        St[d * dm.MS + dm.M] = s;
    }
}

__device__ void zero_fill(float* p, int n) {
    for (int idx = threadIdx.x; idx < n; idx += THREADS) p[idx] = 0.f;
}

// Turn the raw upstream gradient tile g (values in [0,M), anything in column M)
// into Gt_i = [G_i / dn_i, -(G_i . O_i) / dn_i] with dn_i = den_i + eps and
// O_i = num_i / dn_i taken from nd.  One warp handles rows i = warp, warp+8, ...
__device__ void extend_upstream(float* g, const float* nd, const Dims& dm, float eps, int cn,
                                float* dn_out, float* delta_out) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = warp; i < T; i += THREADS / 32) {
        const float dn = nd[i * dm.MS + dm.M] + eps;
        const float inv = i < cn ? 1.f / dn : 0.f;
        float go = 0.f;
        for (int e = lane; e < dm.M; e += 32) {
            const float gi = g[i * dm.MS + e];
            go = fmaf(gi, nd[i * dm.MS + e] * inv, go);
            g[i * dm.MS + e] = gi * inv;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) go += __shfl_xor_sync(0xffffffffu, go, off);
        if (lane == 0) {
            const float delta = -go * inv;
            g[i * dm.MS + dm.M] = delta;
            if (dn_out && i < cn) { dn_out[i] = dn; delta_out[i] = delta; }
        }
    }
}

// dP[i][j] = Gt_i . Vt_j for j <= i (causal) else 0.
__device__ void masked_dscores(float* dP, const float* gt, const float* vt, const Dims& dm) {
    block_product<2, 2>(T, T, Mat{gt, dm.MS, 1}, Mat{vt, 1, dm.MS}, dm.MS, Mat{gt, 0, 0}, Mat{vt, 0, 0}, 0,
                        [&](int i, int j, float v) { dP[i * (T + 1) + j] = j <= i ? v : 0.f; });
}

size_t smem_floats_forward(int D, int M) {
    return (size_t)2 * T * (D + 1) + (size_t)2 * T * (M + 1) + (size_t)D * (M + 1) + (size_t)T * (T + 1);
}
size_t smem_floats_backward(int D, int M) {
    return (size_t)2 * T * (D + 1) + (size_t)3 * T * (M + 1) + (size_t)D * (M + 1) + (size_t)2 * T * (T + 1);
}

// ---------------------------------------------------------------------------
// Causal forward: one CTA walks one (batch, head) sequence chunk by chunk.
// ---------------------------------------------------------------------------
// KD: D = M = KD known at compile time (all tile strides become constants), or 0: any D, M.
template <typename IO, int KD>
__global__ void __launch_bounds__(THREADS)
general_causal_forward_kernel(const IO* __restrict__ Q, const IO* __restrict__ K, const IO* __restrict__ V,
                              const float* __restrict__ S_in, const float* __restrict__ Z_in,
                              IO* __restrict__ O, float* __restrict__ den, float* __restrict__ S_out,
                              float* __restrict__ Z_out, int64_t Nfull, int D_arg, int M_arg, float eps, int phi,
                              const int* __restrict__ lengths, int heads) {
    extern __shared__ float smem[];
    const int D = KD ? KD : D_arg, M = KD ? KD : M_arg;
    const Dims dm = make_dims(D, M);
    float* sq = smem;
    float* sk = sq + T * dm.DS;
    float* sv = sk + T * dm.DS;
    float* snd = sv + T * dm.MS;
    float* sSt = snd + T * dm.MS;
    float* sP = sSt + D * dm.MS;

    const int64_t bh = blockIdx.x;
    // a right-padded ragged batch: only the first N positions of this sequence are real, the rest of its
    // Nfull rows is padding that is neither read nor summed and receives zeros
    int64_t N = Nfull;
    if (lengths) {
        const int64_t len = lengths[bh / heads];
        N = len < 0 ? 0 : (len < Nfull ? len : Nfull);
    }
    Q += bh * Nfull * D; K += bh * Nfull * D; V += bh * Nfull * M; O += bh * Nfull * M;
    zero_fill(sSt, D * dm.MS);
    if (S_in) {                 // continue from a given state (Eq. 16-20 started from S_in, Z_in)
        __syncthreads();
        for (int idx = threadIdx.x; idx < D * M; idx += THREADS)
            sSt[(idx / M) * dm.MS + idx % M] = S_in[bh * D * M + idx];
        for (int d = threadIdx.x; d < D; d += THREADS) sSt[d * dm.MS + M] = Z_in[bh * D + d];
    }

    // the rows of a chunk are requested one chunk ahead and wait in registers while the chunk before is worked on
    uint4 rq[FETCH], rk[FETCH], rv[FETCH];
    auto fetch = [&](int64_t n0) {
        const int cn = (int)((N - n0) < T ? (N - n0) : T);
        fetch_rows<IO>(rq, Q + n0 * D, cn, D);
        fetch_rows<IO>(rk, K + n0 * D, cn, D);
        fetch_rows<IO>(rv, V + n0 * M, cn, M);
    };
    if (N > 0) fetch(0);
    for (int64_t n0 = 0; n0 < N; n0 += T) {
        const int cn = (int)((N - n0) < T ? (N - n0) : T);
        __syncthreads();
        store_mapped<IO>(sq, rq, cn, D, dm.DS, phi);
        store_mapped<IO>(sk, rk, cn, D, dm.DS, phi);
        store_values_ext<IO>(sv, rv, cn, M, dm.MS);
        if (n0 + T < N) fetch(n0 + T);
        __syncthreads();
        masked_scores(sP, sq, sk, D, dm.DS);
        __syncthreads();
        numerator_denominator(snd, sP, sv, sq, sSt, dm, true);
        __syncthreads();
        for (int idx = threadIdx.x; idx < cn * M; idx += THREADS) {
            const int i = idx / M, e = idx - i * M;
            O[(n0 + i) * M + e] = from_f32<IO>(snd[i * dm.MS + e] / (snd[i * dm.MS + M] + eps));
        }
        if (den)
            for (int i = threadIdx.x; i < cn; i += THREADS) den[bh * Nfull + n0 + i] = snd[i * dm.MS + M];
        state_update(sSt, sk, sv, dm);
    }
    __syncthreads();
    for (int64_t idx = N * M + threadIdx.x; idx < Nfull * M; idx += THREADS) O[idx] = from_f32<IO>(0.f);
    if (den)
        for (int64_t i = N + threadIdx.x; i < Nfull; i += THREADS) den[bh * Nfull + i] = 0.f;
    if (S_out)
        for (int idx = threadIdx.x; idx < D * M; idx += THREADS)
            S_out[bh * D * M + idx] = sSt[(idx / M) * dm.MS + idx % M];
    if (Z_out)
        for (int d = threadIdx.x; d < D; d += THREADS) Z_out[bh * D + d] = sSt[d * dm.MS + M];
}

// ---------------------------------------------------------------------------
// Causal backward: forward sweep (grad Q, Eq. 13) then reverse sweep (grad K,
// grad V, Eq. 14-15) by the same CTA.  The per-position scalars dn_i and
// delta_i found in the forward sweep are parked in `aux` ([B,H,N,2] fp32) for
// the reverse sweep; no per-position state is stored.
// ---------------------------------------------------------------------------
template <typename IO, int KD>
__global__ void __launch_bounds__(THREADS)
general_causal_backward_kernel(const IO* __restrict__ Q, const IO* __restrict__ K, const IO* __restrict__ V,
                               const IO* __restrict__ G, const StateArgs sa, IO* __restrict__ dQ,
                               IO* __restrict__ dK, IO* __restrict__ dV, float* __restrict__ aux,
                               int64_t Nfull, int D_arg, int M_arg, float eps, int phi,
                               const int* __restrict__ lengths, int heads) {
    extern __shared__ float smem[];
    const int D = KD ? KD : D_arg, M = KD ? KD : M_arg;
    const Dims dm = make_dims(D, M);
    float* sq = smem;
    float* sk = sq + T * dm.DS;
    float* sv = sk + T * dm.DS;
    float* sg = sv + T * dm.MS;
    float* snd = sg + T * dm.MS;
    float* sSt = snd + T * dm.MS;
    float* sP = sSt + D * dm.MS;
    float* sdP = sP + T * (T + 1);

    const int64_t bh = blockIdx.x;
    int64_t N = Nfull;          // real positions of this sequence (see the forward kernel)
    if (lengths) {
        const int64_t len = lengths[bh / heads];
        N = len < 0 ? 0 : (len < Nfull ? len : Nfull);
    }
    Q += bh * Nfull * D; K += bh * Nfull * D; V += bh * Nfull * M; G += bh * Nfull * M;
    dQ += bh * Nfull * D; dK += bh * Nfull * D; dV += bh * Nfull * M;
    float* dn_all = aux + bh * Nfull * 2;
    float* delta_all = dn_all + Nfull;
    for (int64_t idx = N * D + threadIdx.x; idx < Nfull * D; idx += THREADS) {
        dQ[idx] = from_f32<IO>(0.f);
        dK[idx] = from_f32<IO>(0.f);
    }
    for (int64_t idx = N * M + threadIdx.x; idx < Nfull * M; idx += THREADS) dV[idx] = from_f32<IO>(0.f);

    // ---- forward sweep: St = running sum of phi(K_j) Vt_j^T (from the given state, if any) ----
    zero_fill(sSt, D * dm.MS);
    if (sa.S_in) {
        __syncthreads();
        for (int idx = threadIdx.x; idx < D * M; idx += THREADS)
            sSt[(idx / M) * dm.MS + idx % M] = sa.S_in[bh * D * M + idx];
        for (int d = threadIdx.x; d < D; d += THREADS) sSt[d * dm.MS + M] = sa.Z_in[bh * D + d];
    }
    // the rows of a chunk are requested one chunk ahead and wait in registers while the chunk before is worked on
    uint4 rq[FETCH], rk[FETCH], rv[FETCH], rg[FETCH];
    auto fetch = [&](int64_t n0) {
        const int cn = (int)((N - n0) < T ? (N - n0) : T);
        fetch_rows<IO>(rq, Q + n0 * D, cn, D);
        fetch_rows<IO>(rk, K + n0 * D, cn, D);
        fetch_rows<IO>(rv, V + n0 * M, cn, M);
        fetch_rows<IO>(rg, G + n0 * M, cn, M);
    };
    if (N > 0) fetch(0);
    for (int64_t n0 = 0; n0 < N; n0 += T) {
        const int cn = (int)((N - n0) < T ? (N - n0) : T);
        __syncthreads();
        store_mapped<IO>(sq, rq, cn, D, dm.DS, phi);
        store_mapped<IO>(sk, rk, cn, D, dm.DS, phi);
        store_values_ext<IO>(sv, rv, cn, M, dm.MS);
        store_values_ext<IO>(sg, rg, cn, M, dm.MS);
        if (n0 + T < N) fetch(n0 + T);
        __syncthreads();
        masked_scores(sP, sq, sk, D, dm.DS);
        __syncthreads();
        numerator_denominator(snd, sP, sv, sq, sSt, dm, true);
        __syncthreads();
        extend_upstream(sg, snd, dm, eps, cn, dn_all + n0, delta_all + n0);
        __syncthreads();
        masked_dscores(sdP, sg, sv, dm);
        __syncthreads();
        // grad phi(Q_i) = sum_{j<=i} dP_ij k_j + St_{c-1} Gt_i
        // (dP is zero right of the diagonal)
        block_product<4, 4>(T, D, Mat{sdP, T + 1, 1}, Mat{sk, dm.DS, 1}, T, Mat{sg, dm.MS, 1}, Mat{sSt, 1, dm.MS}, dm.MS,
                            [&](int i, int d, float v) {
                                if (i < cn) dQ[(n0 + i) * D + d] = from_f32<IO>(v * phi_slope_from_value(sq[i * dm.DS + d], phi));
                            });
        __syncthreads();
        state_update(sSt, sk, sv, dm);
    }

    // ---- reverse sweep: Rt = running sum (from the end) of phi(Q_j) Gt_j^T, started from the upstream
    // ---- gradient of the final state, if any ----
    __syncthreads();
    zero_fill(sSt, D * dm.MS);
    if (sa.dS_out || sa.dZ_out) {
        __syncthreads();
        if (sa.dS_out)
            for (int idx = threadIdx.x; idx < D * M; idx += THREADS)
                sSt[(idx / M) * dm.MS + idx % M] = sa.dS_out[bh * D * M + idx];
        if (sa.dZ_out)
            for (int d = threadIdx.x; d < D; d += THREADS) sSt[d * dm.MS + M] = sa.dZ_out[bh * D + d];
    }
    const int64_t nchunks = (N + T - 1) / T;
    float r_dn = 1.f, r_delta = 0.f;          // dn_i, delta_i of row threadIdx.x of the fetched chunk
    auto fetch_back = [&](int64_t n0) {
        const int cn = (int)((N - n0) < T ? (N - n0) : T);
        fetch(n0);
        if ((int)threadIdx.x < cn) {
            r_dn = dn_all[n0 + threadIdx.x];
            r_delta = delta_all[n0 + threadIdx.x];
        }
    };
    if (nchunks > 0) fetch_back((nchunks - 1) * T);
    float* s_dn = snd;                        // [T] dn_i of the chunk (snd is free in this sweep)
    for (int64_t c = nchunks - 1; c >= 0; --c) {
        const int64_t n0 = c * T;
        const int cn = (int)((N - n0) < T ? (N - n0) : T);
        __syncthreads();
        if ((int)threadIdx.x < T) s_dn[threadIdx.x] = (int)threadIdx.x < cn ? r_dn : 1.f;
        store_mapped<IO>(sq, rq, cn, D, dm.DS, phi);
        store_mapped<IO>(sk, rk, cn, D, dm.DS, phi);
        store_values_ext<IO>(sv, rv, cn, M, dm.MS);
        __syncthreads();
        // Gt_i = [G_i / dn_i, delta_i]
        store_rows<IO>(sg, rg, cn, M, dm.MS, [&](int i, float x) { return x / s_dn[i]; });
        if ((int)threadIdx.x < T) sg[threadIdx.x * dm.MS + M] = (int)threadIdx.x < cn ? r_delta : 0.f;
        if (c > 0) fetch_back(n0 - T);
        __syncthreads();
        masked_scores(sP, sq, sk, D, dm.DS);
        masked_dscores(sdP, sg, sv, dm);
        __syncthreads();
        // grad phi(K_j) = sum_{i>=j} dP_ij q_i + Rt_{c+1} Vt_j          (Eq. 14)
        // (dP and P are zero right of the diagonal: summing over all i of the chunk keeps i >= j)
        block_product<4, 4>(T, D, Mat{sdP, 1, T + 1}, Mat{sq, dm.DS, 1}, T, Mat{sv, dm.MS, 1}, Mat{sSt, 1, dm.MS}, dm.MS,
                            [&](int j, int d, float v) {
                                if (j < cn) dK[(n0 + j) * D + d] = from_f32<IO>(v * phi_slope_from_value(sk[j * dm.DS + d], phi));
                            });
        // grad V_j = sum_{i>=j} P_ij Gt_i[0:M] + Rt_{c+1}^T k_j          (Eq. 15)
        block_product<4, 4>(T, M, Mat{sP, 1, T + 1}, Mat{sg, dm.MS, 1}, T, Mat{sk, dm.DS, 1}, Mat{sSt, dm.MS, 1}, D,
                            [&](int j, int e, float v) {
                                if (j < cn) dV[(n0 + j) * M + e] = from_f32<IO>(v);
                            });
        __syncthreads();
        state_update(sSt, sq, sg, dm);
    }
    // what is left in the reverse sum is the gradient of the state the sequence started from
    __syncthreads();
    if (sa.dS_in)
        for (int idx = threadIdx.x; idx < D * M; idx += THREADS)
            sa.dS_in[bh * D * M + idx] = sSt[(idx / M) * dm.MS + idx % M];
    if (sa.dZ_in)
        for (int d = threadIdx.x; d < D; d += THREADS) sa.dZ_in[bh * D + d] = sSt[d * dm.MS + M];
}

// ---------------------------------------------------------------------------
// Non-causal pieces (Eq. 5-6): a split-parallel sum of x_i yt_i^T and per-token
// apply kernels that read the reduced sums.
// ---------------------------------------------------------------------------
struct Split { int nsplit; int64_t len; };

Split choose_split(const la_problem& p) {
    int64_t bh = p.B * p.H;
    int64_t want = (2 * 148 + bh - 1) / bh;                // about two CTAs per SM in total
    int64_t maxs = (p.N + 4 * T - 1) / (4 * T);            // at least four chunks per split
    if (maxs < 1) maxs = 1;
    if (want > maxs) want = maxs;
    if (want < 1) want = 1;
    if (want > 64) want = 64;
    int64_t len = (p.N + want - 1) / want;
    len = (len + T - 1) / T * T;
    int64_t ns = len > 0 ? (p.N + len - 1) / len : 1;
    if (ns < 1) ns = 1;
    return Split{(int)ns, len};
}

// Ragged batches (non-causal form): lengths[b] positions of batch element b are real, the rest is padding
// that takes no part in any sum and receives zeros.  `real_end` clips a split's range to the sequence.
__device__ __forceinline__ int64_t real_end(const int* lengths, int heads, int64_t bh, int64_t hi) {
    if (!lengths) return hi;
    const int64_t len = lengths[bh / heads];
    return len < hi ? len : hi;
}

// part[bh][split] = sum over the split's positions of phi(X_i) [Y_i, 1]^T.
template <typename IO, int KD>
__global__ void __launch_bounds__(THREADS)
general_kv_sum_kernel(const IO* __restrict__ X, const IO* __restrict__ Y, float* __restrict__ part,
                      int64_t N, int64_t split_len, int D_arg, int M_arg, int phi, const int* __restrict__ lengths, int heads) {
    extern __shared__ float smem[];
    const int D = KD ? KD : D_arg, M = KD ? KD : M_arg;
    const Dims dm = make_dims(D, M);
    float* sx = smem;
    float* sy = sx + T * dm.DS;
    float* sSt = sy + T * dm.MS;
    const int64_t bh = blockIdx.x, sp = blockIdx.y;
    const int64_t lo = sp * split_len, hi = real_end(lengths, heads, bh, (lo + split_len) < N ? (lo + split_len) : N);
    X += bh * N * D; Y += bh * N * M;
    zero_fill(sSt, D * dm.MS);
    uint4 rx[FETCH], ry[FETCH];               // the rows of the chunk after the one being worked on
    auto fetch = [&](int64_t n0) {
        const int cn = (int)((hi - n0) < T ? (hi - n0) : T);
        fetch_rows<IO>(rx, X + n0 * D, cn, D);
        fetch_rows<IO>(ry, Y + n0 * M, cn, M);
    };
    if (lo < hi) fetch(lo);
    for (int64_t n0 = lo; n0 < hi; n0 += T) {
        const int cn = (int)((hi - n0) < T ? (hi - n0) : T);
        __syncthreads();
        store_mapped<IO>(sx, rx, cn, D, dm.DS, phi);
        store_values_ext<IO>(sy, ry, cn, M, dm.MS);
        if (n0 + T < hi) fetch(n0 + T);
        __syncthreads();
        state_update(sSt, sx, sy, dm);
    }
    __syncthreads();
    float* dst = part + (bh * gridDim.y + sp) * (int64_t)(D * dm.MS);
    for (int idx = threadIdx.x; idx < D * dm.MS; idx += THREADS) dst[idx] = sSt[idx];
}

__device__ void load_reduced_state(float* sSt, const float* part, int nsplit, int n) {
    for (int idx = threadIdx.x; idx < n; idx += THREADS) {
        float s = 0.f;
        for (int sp = 0; sp < nsplit; ++sp) s += part[(int64_t)sp * n + idx];
        sSt[idx] = s;
    }
}

template <typename IO, int KD>
__global__ void __launch_bounds__(THREADS)
general_linear_apply_kernel(const IO* __restrict__ Q, const float* __restrict__ part, IO* __restrict__ O,
                            float* __restrict__ den, float* __restrict__ KV, float* __restrict__ Zs,
                            int nsplit, int64_t N, int64_t split_len, int D_arg, int M_arg, float eps, int phi,
                            const int* __restrict__ lengths, int heads) {
    extern __shared__ float smem[];
    const int D = KD ? KD : D_arg, M = KD ? KD : M_arg;
    const Dims dm = make_dims(D, M);
    float* sq = smem;
    float* snd = sq + T * dm.DS;
    float* sSt = snd + T * dm.MS;
    const int64_t bh = blockIdx.x, sp = blockIdx.y;
    const int64_t lo = sp * split_len, hi_all = (lo + split_len) < N ? (lo + split_len) : N;
    const int64_t hi = real_end(lengths, heads, bh, hi_all);
    Q += bh * N * D; O += bh * N * M;
    for (int64_t idx = (lo > hi ? lo : hi) * M + threadIdx.x; idx < hi_all * M; idx += THREADS) O[idx] = from_f32<IO>(0.f);
    if (den)
        for (int64_t i = (lo > hi ? lo : hi) + threadIdx.x; i < hi_all; i += THREADS) den[bh * N + i] = 0.f;
    load_reduced_state(sSt, part + bh * nsplit * (int64_t)(D * dm.MS), nsplit, D * dm.MS);
    __syncthreads();
    if (sp == 0) {
        if (KV)
            for (int idx = threadIdx.x; idx < D * M; idx += THREADS)
                KV[bh * D * M + idx] = sSt[(idx / M) * dm.MS + idx % M];
        if (Zs)
            for (int d = threadIdx.x; d < D; d += THREADS) Zs[bh * D + d] = sSt[d * dm.MS + M];
    }
    uint4 rx[FETCH];                          // the rows of the chunk after the one being worked on
    auto fetch = [&](int64_t n0) {
        const int cn = (int)((hi - n0) < T ? (hi - n0) : T);
        fetch_rows<IO>(rx, Q + n0 * D, cn, D);
    };
    if (lo < hi) fetch(lo);
    for (int64_t n0 = lo; n0 < hi; n0 += T) {
        const int cn = (int)((hi - n0) < T ? (hi - n0) : T);
        __syncthreads();
        store_mapped<IO>(sq, rx, cn, D, dm.DS, phi);
        if (n0 + T < hi) fetch(n0 + T);
        __syncthreads();
        numerator_denominator(snd, nullptr, nullptr, sq, sSt, dm, false);
        __syncthreads();
        for (int idx = threadIdx.x; idx < cn * M; idx += THREADS) {
            const int i = idx / M, e = idx - i * M;
            O[(n0 + i) * M + e] = from_f32<IO>(snd[i * dm.MS + e] / (snd[i * dm.MS + M] + eps));
        }
        if (den)
            for (int i = threadIdx.x; i < cn; i += THREADS) den[bh * N + n0 + i] = snd[i * dm.MS + M];
    }
}

// Backward, query side: with St = full sum, form Gt_i, write
// grad phi(Q_i) = St Gt_i (Eq. 13 with the full sum) and accumulate this split's
// part of Rt = sum_i phi(Q_i) Gt_i^T.
template <typename IO, int KD>
__global__ void __launch_bounds__(THREADS)
general_linear_bwd_q_kernel(const IO* __restrict__ Q, const IO* __restrict__ G,
                            const float* __restrict__ part_s, IO* __restrict__ dQ,
                            float* __restrict__ part_r, int nsplit, int64_t N, int64_t split_len,
                            int D_arg, int M_arg, float eps, int phi, const int* __restrict__ lengths, int heads) {
    extern __shared__ float smem[];
    const int D = KD ? KD : D_arg, M = KD ? KD : M_arg;
    const Dims dm = make_dims(D, M);
    float* sq = smem;
    float* sg = sq + T * dm.DS;
    float* snd = sg + T * dm.MS;
    float* sSt = snd + T * dm.MS;
    float* sRt = sSt + D * dm.MS;
    const int64_t bh = blockIdx.x, sp = blockIdx.y;
    const int64_t lo = sp * split_len, hi_all = (lo + split_len) < N ? (lo + split_len) : N;
    const int64_t hi = real_end(lengths, heads, bh, hi_all);
    Q += bh * N * D; G += bh * N * M; dQ += bh * N * D;
    for (int64_t idx = (lo > hi ? lo : hi) * D + threadIdx.x; idx < hi_all * D; idx += THREADS) dQ[idx] = from_f32<IO>(0.f);
    load_reduced_state(sSt, part_s + bh * nsplit * (int64_t)(D * dm.MS), nsplit, D * dm.MS);
    zero_fill(sRt, D * dm.MS);
    uint4 rx[FETCH], ry[FETCH];               // the rows of the chunk after the one being worked on
    auto fetch = [&](int64_t n0) {
        const int cn = (int)((hi - n0) < T ? (hi - n0) : T);
        fetch_rows<IO>(rx, Q + n0 * D, cn, D);
        fetch_rows<IO>(ry, G + n0 * M, cn, M);
    };
    if (lo < hi) fetch(lo);
    for (int64_t n0 = lo; n0 < hi; n0 += T) {
        const int cn = (int)((hi - n0) < T ? (hi - n0) : T);
        __syncthreads();
        store_mapped<IO>(sq, rx, cn, D, dm.DS, phi);
        store_values_ext<IO>(sg, ry, cn, M, dm.MS);
        if (n0 + T < hi) fetch(n0 + T);
        __syncthreads();
        numerator_denominator(snd, nullptr, nullptr, sq, sSt, dm, false);
        __syncthreads();
        extend_upstream(sg, snd, dm, eps, cn, nullptr, nullptr);
        __syncthreads();
        block_product<4, 4>(T, D, Mat{sg, dm.MS, 1}, Mat{sSt, 1, dm.MS}, dm.MS, Mat{sg, 0, 0}, Mat{sSt, 0, 0}, 0,
                            [&](int i, int d, float v) {
                                if (i < cn) dQ[(n0 + i) * D + d] = from_f32<IO>(v * phi_slope_from_value(sq[i * dm.DS + d], phi));
                            });
        state_update(sRt, sq, sg, dm);
    }
    __syncthreads();
    float* dst = part_r + (bh * gridDim.y + sp) * (int64_t)(D * dm.MS);
    for (int idx = threadIdx.x; idx < D * dm.MS; idx += THREADS) dst[idx] = sRt[idx];
}

// Backward, key/value side: grad phi(K_j) = Rt Vt_j (Eq. 14), grad V_j = (Rt^T phi(K_j))[0:M] (Eq. 15).
template <typename IO, int KD>
__global__ void __launch_bounds__(THREADS)
general_linear_bwd_kv_kernel(const IO* __restrict__ K, const IO* __restrict__ V,
                             const float* __restrict__ part_r, IO* __restrict__ dK, IO* __restrict__ dV,
                             int nsplit, int64_t N, int64_t split_len, int D_arg, int M_arg, int phi,
                             const int* __restrict__ lengths, int heads) {
    extern __shared__ float smem[];
    const int D = KD ? KD : D_arg, M = KD ? KD : M_arg;
    const Dims dm = make_dims(D, M);
    float* sk = smem;
    float* sv = sk + T * dm.DS;
    float* sRt = sv + T * dm.MS;
    const int64_t bh = blockIdx.x, sp = blockIdx.y;
    const int64_t lo = sp * split_len, hi_all = (lo + split_len) < N ? (lo + split_len) : N;
    const int64_t hi = real_end(lengths, heads, bh, hi_all);
    K += bh * N * D; V += bh * N * M; dK += bh * N * D; dV += bh * N * M;
    for (int64_t idx = (lo > hi ? lo : hi) * D + threadIdx.x; idx < hi_all * D; idx += THREADS) dK[idx] = from_f32<IO>(0.f);
    for (int64_t idx = (lo > hi ? lo : hi) * M + threadIdx.x; idx < hi_all * M; idx += THREADS) dV[idx] = from_f32<IO>(0.f);
    load_reduced_state(sRt, part_r + bh * nsplit * (int64_t)(D * dm.MS), nsplit, D * dm.MS);
    uint4 rx[FETCH], ry[FETCH];               // the rows of the chunk after the one being worked on
    auto fetch = [&](int64_t n0) {
        const int cn = (int)((hi - n0) < T ? (hi - n0) : T);
        fetch_rows<IO>(rx, K + n0 * D, cn, D);
        fetch_rows<IO>(ry, V + n0 * M, cn, M);
    };
    if (lo < hi) fetch(lo);
    for (int64_t n0 = lo; n0 < hi; n0 += T) {
        const int cn = (int)((hi - n0) < T ? (hi - n0) : T);
        __syncthreads();
        store_mapped<IO>(sk, rx, cn, D, dm.DS, phi);
        store_values_ext<IO>(sv, ry, cn, M, dm.MS);
        if (n0 + T < hi) fetch(n0 + T);
        __syncthreads();
        block_product<4, 4>(T, D, Mat{sv, dm.MS, 1}, Mat{sRt, 1, dm.MS}, dm.MS, Mat{sv, 0, 0}, Mat{sRt, 0, 0}, 0,
                            [&](int j, int d, float v) {
                                if (j < cn) dK[(n0 + j) * D + d] = from_f32<IO>(v * phi_slope_from_value(sk[j * dm.DS + d], phi));
                            });
        block_product<4, 4>(T, M, Mat{sk, dm.DS, 1}, Mat{sRt, dm.MS, 1}, D, Mat{sk, 0, 0}, Mat{sRt, 0, 0}, 0,
                            [&](int j, int e, float v) {
                                if (j < cn) dV[(n0 + j) * M + e] = from_f32<IO>(v);
                            });
    }
}

template <typename Kern>
int opt_in_smem(Kern kern, size_t bytes) {
    if (bytes > 48 * 1024)
        LA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
    return LA_OK;
}

size_t state_floats(const la_problem& p) { return (size_t)p.D * (p.M + 1); }

}  // namespace

size_t general_workspace_bytes(const la_problem& p, int op) {
    const size_t bh = (size_t)(p.B * p.H);
    switch (op) {
        case LA_OP_CAUSAL_FORWARD: return 0;
        case LA_OP_CAUSAL_BACKWARD: return bh * (size_t)p.N * 2 * sizeof(float);
        case LA_OP_LINEAR_FORWARD:
        case LA_OP_LINEAR_VARLEN_FORWARD: return bh * choose_split(p).nsplit * state_floats(p) * sizeof(float);
        case LA_OP_LINEAR_BACKWARD:
        case LA_OP_LINEAR_VARLEN_BACKWARD: return 2 * bh * choose_split(p).nsplit * state_floats(p) * sizeof(float);
        default: return 0;
    }
}

template <typename IO>
static int causal_forward_t(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths, const float* S_in,
                            const float* Z_in, void* O, float* den, float* S_out, float* Z_out, cudaStream_t st) {
    const size_t smem = smem_floats_forward((int)p.D, (int)p.M) * sizeof(float);
    auto kern = p.D == 64 && p.M == 64 ? general_causal_forward_kernel<IO, 64> : general_causal_forward_kernel<IO, 0>;
    if (int rc = opt_in_smem(kern, smem)) return rc;
    kern<<<(unsigned)(p.B * p.H), THREADS, smem, st>>>((const IO*)Q, (const IO*)K, (const IO*)V, S_in, Z_in, (IO*)O, den,
                                                       S_out, Z_out, p.N, (int)p.D, (int)p.M, p.eps, p.phi, lengths, (int)p.H);
    LA_LAUNCHED();
    return LA_OK;
}

int general_causal_forward(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths, const float* S_in,
                           const float* Z_in, void* O, float* den, float* S_out, float* Z_out, cudaStream_t st) {
    return p.dtype == LA_F32 ? causal_forward_t<float>(p, Q, K, V, lengths, S_in, Z_in, O, den, S_out, Z_out, st)
                             : causal_forward_t<__nv_bfloat16>(p, Q, K, V, lengths, S_in, Z_in, O, den, S_out, Z_out, st);
}

template <typename IO>
static int causal_backward_t(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths,
                             const void* G, const StateArgs& sa, void* dQ, void* dK, void* dV, void* ws,
                             cudaStream_t st) {
    const size_t smem = smem_floats_backward((int)p.D, (int)p.M) * sizeof(float);
    auto kern = p.D == 64 && p.M == 64 ? general_causal_backward_kernel<IO, 64> : general_causal_backward_kernel<IO, 0>;
    if (int rc = opt_in_smem(kern, smem)) return rc;
    kern<<<(unsigned)(p.B * p.H), THREADS, smem, st>>>((const IO*)Q, (const IO*)K, (const IO*)V, (const IO*)G, sa,
                                                       (IO*)dQ, (IO*)dK, (IO*)dV, (float*)ws, p.N, (int)p.D,
                                                       (int)p.M, p.eps, p.phi, lengths, (int)p.H);
    LA_LAUNCHED();
    return LA_OK;
}

int general_causal_backward(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths, const void* G,
                            const StateArgs& sa, void* dQ, void* dK, void* dV, void* ws, cudaStream_t st) {
    return p.dtype == LA_F32 ? causal_backward_t<float>(p, Q, K, V, lengths, G, sa, dQ, dK, dV, ws, st)
                             : causal_backward_t<__nv_bfloat16>(p, Q, K, V, lengths, G, sa, dQ, dK, dV, ws, st);
}

template <typename IO>
static int linear_forward_t(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths,
                            void* O, float* den, float* KV, float* Zs, void* saved, void* ws, cudaStream_t st) {
    const int D = (int)p.D, M = (int)p.M;
    const Split sp = choose_split(p);
    const dim3 grid((unsigned)(p.B * p.H), (unsigned)sp.nsplit);
    float* part = saved ? (float*)saved : (float*)ws;        // the per-split sums, kept for the backward pass if asked
    {
        const size_t smem = ((size_t)T * (D + 1) + (size_t)T * (M + 1) + state_floats(p)) * sizeof(float);
        auto kern = D == 64 && M == 64 ? general_kv_sum_kernel<IO, 64> : general_kv_sum_kernel<IO, 0>;
        if (int rc = opt_in_smem(kern, smem)) return rc;
        kern<<<grid, THREADS, smem, st>>>((const IO*)K, (const IO*)V, part, p.N, sp.len, D, M, p.phi, lengths, (int)p.H);
        LA_LAUNCHED();
    }
    {
        const size_t smem = ((size_t)T * (D + 1) + (size_t)T * (M + 1) + state_floats(p)) * sizeof(float);
        auto kern = D == 64 && M == 64 ? general_linear_apply_kernel<IO, 64> : general_linear_apply_kernel<IO, 0>;
        if (int rc = opt_in_smem(kern, smem)) return rc;
        kern<<<grid, THREADS, smem, st>>>((const IO*)Q, part, (IO*)O, den, KV, Zs, sp.nsplit, p.N, sp.len, D, M,
                                          p.eps, p.phi, lengths, (int)p.H);
        LA_LAUNCHED();
    }
    return LA_OK;
}

int general_linear_forward(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths,
                           void* O, float* den, float* KV, float* Zs, void* saved, void* ws, cudaStream_t st) {
    return p.dtype == LA_F32 ? linear_forward_t<float>(p, Q, K, V, lengths, O, den, KV, Zs, saved, ws, st)
                             : linear_forward_t<__nv_bfloat16>(p, Q, K, V, lengths, O, den, KV, Zs, saved, ws, st);
}

template <typename IO>
static int linear_backward_t(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths,
                             const void* saved, const void* G, void* dQ, void* dK, void* dV, void* ws, cudaStream_t st) {
    const int D = (int)p.D, M = (int)p.M;
    const Split sp = choose_split(p);
    const dim3 grid((unsigned)(p.B * p.H), (unsigned)sp.nsplit);
    float* part_s = (float*)ws;
    float* part_r = part_s + (size_t)(p.B * p.H) * sp.nsplit * state_floats(p);
    if (saved) {
        part_s = (float*)saved;           // the forward's own sums: nothing to recompute
    } else {
        const size_t smem = ((size_t)T * (D + 1) + (size_t)T * (M + 1) + state_floats(p)) * sizeof(float);
        auto kern = D == 64 && M == 64 ? general_kv_sum_kernel<IO, 64> : general_kv_sum_kernel<IO, 0>;
        if (int rc = opt_in_smem(kern, smem)) return rc;
        kern<<<grid, THREADS, smem, st>>>((const IO*)K, (const IO*)V, part_s, p.N, sp.len, D, M, p.phi, lengths, (int)p.H);
        LA_LAUNCHED();
    }
    {
        const size_t smem = ((size_t)T * (D + 1) + (size_t)2 * T * (M + 1) + 2 * state_floats(p)) * sizeof(float);
        auto kern = D == 64 && M == 64 ? general_linear_bwd_q_kernel<IO, 64> : general_linear_bwd_q_kernel<IO, 0>;
        if (int rc = opt_in_smem(kern, smem)) return rc;
        kern<<<grid, THREADS, smem, st>>>((const IO*)Q, (const IO*)G, part_s, (IO*)dQ, part_r, sp.nsplit, p.N,
                                          sp.len, D, M, p.eps, p.phi, lengths, (int)p.H);
        LA_LAUNCHED();
    }
    {
        const size_t smem = ((size_t)T * (D + 1) + (size_t)T * (M + 1) + state_floats(p)) * sizeof(float);
        auto kern = D == 64 && M == 64 ? general_linear_bwd_kv_kernel<IO, 64> : general_linear_bwd_kv_kernel<IO, 0>;
        if (int rc = opt_in_smem(kern, smem)) return rc;
        kern<<<grid, THREADS, smem, st>>>((const IO*)K, (const IO*)V, part_r, (IO*)dK, (IO*)dV, sp.nsplit, p.N,
                                          sp.len, D, M, p.phi, lengths, (int)p.H);
        LA_LAUNCHED();
    }
    return LA_OK;
}

int general_linear_backward(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths,
                            const void* saved, const void* G, void* dQ, void* dK, void* dV, void* ws, cudaStream_t st) {
    return p.dtype == LA_F32 ? linear_backward_t<float>(p, Q, K, V, lengths, saved, G, dQ, dK, dV, ws, st)
                             : linear_backward_t<__nv_bfloat16>(p, Q, K, V, lengths, saved, G, dQ, dK, dV, ws, st);
}

}  // namespace la
