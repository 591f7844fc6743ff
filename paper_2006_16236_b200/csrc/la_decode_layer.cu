// One decode step of a whole attention sublayer (Eq. 16-20 with the projections of Eq. 2 written out):
//     [q | k | v] = x [W_Q | W_K | W_V]          projection GEMM on the tensor cores (this file)
//     S += phi(k) v^T, Z += phi(k), a = phi(q)^T S / (phi(q)^T Z + eps)     the recurrent step kernel
//     y = a W_O + x                              projection GEMM with the residual added in its epilogue
// Three launches per token.  The two projections are the same kernel: C[rows][n] = A[rows][K] . W[n][K]^T
// (+ R), bf16 operands staged by TMA as 128-byte-swizzled tiles, fp32 accumulation in TMEM (tcgen05, M = 128,
// N = 64, K = 16 per instruction), one CTA per 128 x 64 tile of C.  At decode sizes (a few hundred streams, a
// model width of a few hundred) a projection is a few microseconds of latency, not a throughput problem: the
// tiles are small on purpose, so that the QKV projection fills 48 SMs instead of 12.
// Warps 0-3: epilogue (thread t owns row t of the tile = TMEM lane t); warp 4: TMA; warp 5: MMA issue.
#include "la_tc.cuh"
#include "la_tc_common.cuh"

namespace la {
namespace tc {

using namespace sm100;

namespace {

constexpr int kGemmThreads = 192;
constexpr int kGemmStages = 8;      // a model width of 512 is eight K blocks: all loads of a tile are in flight at once
constexpr int kGemmTileN = 64;
constexpr uint32_t kGemmStageBytes = kTileBytes + kGemmTileN * 128;        // A [128][64] + W [64][64]
constexpr uint32_t kGemmOffBar = kGemmStages * kGemmStageBytes;
constexpr uint32_t kGemmSmemBytes = kGemmOffBar + 128 + 1024;              // + slack for the 1 KB alignment of the base

struct GemmBarriers {
    uint64_t full[kGemmStages], empty[kGemmStages], done;
    uint32_t tmem_base;
    int abort_flag;
};

struct GemmParams {
    __nv_bfloat16* out[3];      // column tile n0 goes to out[n0 / out_cols] at column n0 % out_cols (row stride out_cols)
    const __nv_bfloat16* res;   // residual [rows][out_cols] added in the epilogue, or null
    int* status;
    int rows, kblocks, out_cols;
    int early_w;                // the weight tiles of the first ring are requested before the dependency wait
};

__global__ void __launch_bounds__(kGemmThreads, 1)
projection_gemm_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapW, const GemmParams prm) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    GemmBarriers* bars = reinterpret_cast<GemmBarriers*>(smem + kGemmOffBar);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int row0 = blockIdx.y * kChunk, n0 = blockIdx.x * kGemmTileN;

    if (tid == 0) {
        for (int s = 0; s < kGemmStages; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], 1);
        }
        mbar_init(&bars->done, 1);
        bars->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 5) {
        __syncwarp();
        tmem_alloc(&bars->tmem_base, 64);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    // Everything above is private to the CTA; from here on memory of the kernel before this one is touched.
    // Every thread waits for that kernel and only then lets the next one be scheduled (a kernel behind this one
    // may read, before its own wait, what no kernel of the call writes: by then everything older is complete).
    // With early_w (the output projection: its weights are written by no kernel of the call and the kernels in
    // front of it kept that order) the producer requests the weight tiles of the first ring before it waits.
    const bool early_w = prm.early_w != 0 && warp == 4 && lane == 0;
    const int ring = min(prm.kblocks, kGemmStages);
    if (early_w) {
        prefetch_tensormap(&mapW);
        for (int kb = 0; kb < ring; ++kb) {
            mbar_arrive_expect_tx(&bars->full[kb], kGemmStageBytes);
            tma_load_2d(smem + kb * kGemmStageBytes + kTileBytes, &mapW, kb * kDim, n0, &bars->full[kb]);
        }
    }
    grid_dependency_wait();
    allow_dependent_launch();
    const uint32_t tmem = bars->tmem_base;
    volatile int* abort_flag = &bars->abort_flag;

    if (warp == 4) {
        if (lane == 0) {
            prefetch_tensormap(&mapA);
            if (!early_w) prefetch_tensormap(&mapW);
            #pragma unroll 1
            for (int kb = 0; kb < prm.kblocks; ++kb) {
                const int s = kb % kGemmStages;
                if (kb >= kGemmStages && !mbar_wait(&bars->empty[s], ((kb / kGemmStages) - 1) & 1, prm.status, kStatusPipeTimeout)) {
                    *abort_flag = 1;
                    break;
                }
                uint8_t* st = smem + s * kGemmStageBytes;
                const bool w_requested = early_w && kb < ring;
                if (!w_requested) mbar_arrive_expect_tx(&bars->full[s], kGemmStageBytes);
                tma_load_2d(st, &mapA, kb * kDim, row0, &bars->full[s]);               // rows past the end read as zeros
                if (!w_requested) tma_load_2d(st + kTileBytes, &mapW, kb * kDim, n0, &bars->full[s]);
            }
        }
    } else if (warp == 5) {
        // all 32 lanes run the loop and an elected one issues: addresses and descriptors stay in uniform registers
        const bool leader = elect_one();
        const uint32_t idesc = umma_idesc_bf16(128, kGemmTileN, 0, 0);
        bool ok = true;
        #pragma unroll 1
        for (int kb = 0; kb < prm.kblocks && ok; ++kb) {
            const int s = kb % kGemmStages;
            ok = mbar_wait_warp(&bars->full[s], (kb / kGemmStages) & 1, prm.status, kStatusTmaTimeout);
            if (!ok || __any_sync(0xFFFFFFFFu, *abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t aA = sbase + s * kGemmStageBytes, aW = aA + kTileBytes;
#pragma unroll
            for (int k = 0; k < 4; ++k)
                umma_bf16(leader, tmem, desc_k(aA + 32 * k), desc_k(aW + 32 * k), idesc, (kb | k) != 0);
            umma_commit(leader, &bars->empty[s]);
        }
        if (!ok) *abort_flag = 1;
        umma_commit(leader, &bars->done);
    } else {
        // epilogue: row t of the tile, 64 columns
        const int t = tid;
        const int row = row0 + t;
        const bool ok = mbar_wait(&bars->done, 0, prm.status, kStatusMmaTimeout) && !*abort_flag;
        tc_fence_after_sync();
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        __nv_bfloat16* dst = prm.out[n0 / prm.out_cols] + (int64_t)row * prm.out_cols + n0 % prm.out_cols;
        const __nv_bfloat16* res = prm.res ? prm.res + (int64_t)row * prm.out_cols + n0 % prm.out_cols : nullptr;
        #pragma unroll 1
        for (int h = 0; h < 2; ++h) {
            uint32_t v[32];
            tmem_ld32(tmem + lane_base + h * 32, v);
            tmem_ld_wait();
            if (ok && row < prm.rows) {
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    float add[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                    if (res) {
                        const uint4 r = __ldg(reinterpret_cast<const uint4*>(res + h * 32 + cc * 8));
                        const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) { add[2 * j] = bf16_lo(rw[j]); add[2 * j + 1] = bf16_hi(rw[j]); }
                    }
                    stg128(dst + h * 32 + cc * 8,
                           pack_bf16x2(__uint_as_float(v[cc * 8 + 0]) + add[0], __uint_as_float(v[cc * 8 + 1]) + add[1]),
                           pack_bf16x2(__uint_as_float(v[cc * 8 + 2]) + add[2], __uint_as_float(v[cc * 8 + 3]) + add[3]),
                           pack_bf16x2(__uint_as_float(v[cc * 8 + 4]) + add[4], __uint_as_float(v[cc * 8 + 5]) + add[5]),
                           pack_bf16x2(__uint_as_float(v[cc * 8 + 6]) + add[6], __uint_as_float(v[cc * 8 + 7]) + add[7]));
                }
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 5) {
        __syncwarp();
        tmem_dealloc(tmem, 64);
    }
}

// C[rows][n] = A[rows][K] W[n][K]^T (+ res): n = n_out * out_cols columns in all, written to out[0..n_out-1]
int projection_gemm(const void* A, const void* W, int rows, int K, int n_out, int out_cols, __nv_bfloat16* const* out,
                    const void* res, bool early_w, cudaStream_t st) {
    CUtensorMap mA, mW;
    if (int rc = encode_tile_map(&mA, A, (uint64_t)rows, kChunk, K)) return rc;
    if (int rc = encode_tile_map(&mW, W, (uint64_t)n_out * out_cols, kGemmTileN, K)) return rc;
    static std::atomic<uint64_t> attr_done{0};
    if (int rc = opt_in_smem_once(projection_gemm_kernel, kGemmSmemBytes, attr_done)) return rc;
    GemmParams prm;
    for (int i = 0; i < 3; ++i) prm.out[i] = i < n_out ? out[i] : nullptr;
    prm.res = (const __nv_bfloat16*)res;
    prm.status = device_status_ptr();
    if (!prm.status) return fail(LA_ERR_CUDA, "device status word unavailable");
    prm.rows = rows;
    prm.kblocks = K / kDim;
    prm.out_cols = out_cols;
    prm.early_w = early_w ? 1 : 0;
    prof_begin(kProfProjection, st);
    cudaLaunchAttribute attr;
    cudaLaunchConfig_t cfg = chained_launch((unsigned)(n_out * out_cols / kGemmTileN), kGemmThreads, kGemmSmemBytes, st, &attr);
    cfg.gridDim = dim3((unsigned)(n_out * out_cols / kGemmTileN), (unsigned)((rows + kChunk - 1) / kChunk));
    LA_CUDA_TRY(cudaLaunchKernelEx(&cfg, projection_gemm_kernel, mA, mW, prm));
    note_launch();
    prof_end(kProfProjection, st);
    return LA_OK;
}

}  // namespace

}  // namespace tc

size_t decode_layer_workspace(const la_problem& p) {
    return (size_t)(4 * p.B * p.H * p.D) * sizeof(__nv_bfloat16);       // q, k, v, a: [B][H*D] each
}

bool decode_layer_supported(const la_problem& p) { return p.dtype == LA_BF16 && p.D == 64 && p.M == 64; }

int decode_layer_step(const la_problem& p, const void* x, const void* Wqkv, const void* Wo, float* S, float* Z,
                      void* y, void* ws, cudaStream_t st) {
    const int B = (int)p.B, F = (int)(p.H * p.D);
    __nv_bfloat16* q = (__nv_bfloat16*)ws;
    __nv_bfloat16* qkv[3] = {q, q + (size_t)B * F, q + 2 * (size_t)B * F};
    __nv_bfloat16* a = q + 3 * (size_t)B * F;
    // The first kernel of the call waits for everything before it; the two behind it start on what no kernel of
    // the call writes (the state, the output weights) while the kernel in front of them still runs.
    if (int rc = tc::projection_gemm(x, Wqkv, B, F, 3, F, qkv, nullptr, /*early_w=*/false, st)) return rc;
    if (int rc = launch_recurrent_step(p, qkv[0], qkv[1], qkv[2], S, Z, a, st, /*chained=*/true, /*early_state=*/true)) return rc;
    __nv_bfloat16* yy[1] = {(__nv_bfloat16*)y};
    return tc::projection_gemm(a, Wo, B, F, 1, F, yy, x, /*early_w=*/true, st);
}

}  // namespace la
