// Non-causal linear attention on the tensor cores (bf16, D = M = 64), Eq. 5-6 and the
// gradient of Eq. 13-15 with full (unmasked) sums.
//
// The per-head sums are formed once (pre-pass: every sequence is cut into splits, each
// split's sums go to a record; consumers add the records) and reused for every position
// by three "apply" passes that share one kernel:
//   forward        O_i  = q_i S / (q_i . Z + eps)                        X = Q
//   backward, Q    h_i  = G_i S^T,  dn_i = q_i . Z + eps,  dl_i = -(q_i . h_i) / dn_i,
//                  gq_i = (h_i + dl_i Z) / dn_i,  dQ = gq o phi'(Q)      X = Q, Y = G
//   backward, K/V  gk_j = V_j R^T + r,  dK = gk o phi'(K),  dV_j = k_j R  X = K, Y = V
// with St = [S | Z] = sum_j k_j [V_j | 1]^T and Rt = [R | r] = sum_i (q_i / dn_i) [G_i | dl_i]^T.
// As in the causal kernels, -(G_i . O_i) is taken from the same rounded products as h_i
// (projection form), never from a stored output.
//
// Centred operands.  phi = elu + 1 is positive, so phi(X) ~ 1 + (something small) whenever
// the inputs are small, and every sum above is dominated by a rank-one part that carries
// none of the Q / K gradient.  Rounding phi(X) or the sums to bf16 as they stand would
// spend the 8 mantissa bits on that part.  The tensor cores therefore only see centred
// operands, and every rank-one part is carried in fp32:
//   x' = elu(X) = phi(X) - 1                     (tile operand; full bf16 relative precision)
//   S  = 1 (ysum + mu)^T + S'',  S'' = sum_j k'_j V_j^T - 1 mu^T  (mu = column means), Z = N 1 + Z'
//   R  = 1 (gsum + rho)^T + R'', R'' = sum_i qh'_i G_i^T - 1 rho^T,  r = rho0 1 + r'
// with ysum = sum_j V_j, gsum = sum_i G_i / dn_i, rho0 = sum_i dl_i / dn_i, qh' = q' / dn.
// The column sums of S'' and R'' vanish, so (1 + x')^T S'' = x'^T S''.
//
// Sum kernel: 10 warps (0-7 apply elu to the X tile in place, half a row per thread; 8 TMA; 9 MMA issue).
// Apply kernel: 14 warps (0-7 epilogue, two per TMEM quadrant, half a chunk row each; 8-11 apply elu to the
// X tile in place; 12 TMA; 13 MMA issue).
#include "la_tc.cuh"
#include "la_tc_common.cuh"

namespace la {
namespace tc {

using namespace sm100;

LA_TRACE_DECL(g_trace_lin)

namespace {

// Record of one split: [A' (64x64) | a' (64) | ysum (64) | w0 (1) | pad]:
//   forward sums (sum kernel)            : A' = sum k'_j V_j^T, a' = sum k'_j, ysum = sum V_j,        w0 unused
//   reverse sums (backward-Q apply pass) : A' = sum qh'_i G_i^T, a' = sum qh'_i dl_i, ysum = sum G_i / dn_i, w0 = sum dl_i / dn_i
constexpr int kRecFloats = kDim * kDim + kDim + kDim + 8;

__device__ __forceinline__ float elu_fast(float x) {      // elu(x) = phi(x) - 1
    float e;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(x * 1.4426950408889634f));
    return x > 0.f ? x : e - 1.f;
}

// elu (optionally scaled) on one row of a swizzled tile, in place; returns nothing.
template <bool kElu>
__device__ __forceinline__ void elu_row_inplace(uint8_t* row, uint32_t r7, float scale, int nch) {
    uint32_t v[8][4];
    load_row(row, r7, v);
#pragma unroll
    for (int c = 0; c < 8; ++c)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float x0 = bf16_lo(v[c][j]), x1 = bf16_hi(v[c][j]);
            v[c][j] = pack_bf16x2((kElu ? elu_fast(x0) : x0 - 1.f) * scale, (kElu ? elu_fast(x1) : x1 - 1.f) * scale);
        }
    store_row(row, r7, v, nch);          // the zero padding of a 32-column row stays zero
}

// elu on logical chunks [4 hf, 4 hf + 4) of a row (those below nch).
template <bool kElu>
__device__ __forceinline__ void elu_half_row_inplace(uint8_t* row, uint32_t r7, float scale, int hf, int nch) {
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
        const int c = hf * 4 + cc;
        if (c < nch) {
            uint32_t v[4];
            lds128(row + ((c ^ r7) << 4), v);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float x0 = bf16_lo(v[j]), x1 = bf16_hi(v[j]);
                v[j] = pack_bf16x2((kElu ? elu_fast(x0) : x0 - 1.f) * scale, (kElu ? elu_fast(x1) : x1 - 1.f) * scale);
            }
            sts128(row + ((c ^ r7) << 4), v[0], v[1], v[2], v[3]);
        }
    }
}

// ===========================================================================
// Pre-pass: per-split sums.  Warps 0-7: elu on X (scaled by w_i; two threads per row, half a row
// each), aux tile, final read-out (warps 0-2); warp 8: TMA; warp 9: MMA.
// ===========================================================================
constexpr int kLsThreads = 320;
// Six stages of {X, Y}: a tile arrives 2400-4000 cycles after its load is issued, against about 1000 cycles of
// mapping and 600 of MMA issue per chunk, so the ring has to hold the loads of several chunks ahead.  One aux
// tile (constant ones) serves every stage.
constexpr int kLsStages = 6;
constexpr uint32_t kLsStageBytes = 2 * kTileBytes;                  // X, Y
constexpr uint32_t kLsOffAux = kLsStages * kLsStageBytes;           // [128][64] ones: second block of both operands
constexpr uint32_t kLsOffBar = kLsOffAux + kTileBytes;
constexpr uint32_t kLsSmemBytes = kLsOffBar + 256 + 1024;

struct LsBarriers {
    uint64_t full[kLsStages], empty[kLsStages], mapped[kLsStages];
    uint64_t done;
    uint32_t tmem_base;
    int abort_flag;
};

struct LsParams {
    float* records;        // [BH][nseg][kRecFloats]
    const int* lengths;    // [B] real positions per batch element (right-padded ragged batch), or null
    int heads;
    int* status;
    int64_t N;
    int chunks, chunks_per_seg, nseg;
    int phi;
    int dim;
};

template <bool k3d>         // N is not a multiple of the chunk: the tiles are 3-D boxes that end with their sequence
__global__ void __launch_bounds__(kLsThreads, 1)
linear_sum_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapY,
                  const LsParams prm) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    LsBarriers* bars = reinterpret_cast<LsBarriers*>(smem + kLsOffBar);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int seg = blockIdx.x % prm.nseg;
    const int64_t bh = blockIdx.x / prm.nseg;
    const int c_begin = seg * prm.chunks_per_seg;
    const int L_all = min(prm.chunks, c_begin + prm.chunks_per_seg) - c_begin;
    LA_TRACE_CTA(g_trace_lin, 0);

    if (tid == 0) {
        for (int s = 0; s < kLsStages; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], 1);
            mbar_init(&bars->mapped[s], 256);
        }
        mbar_init(&bars->done, 1);
        bars->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 9) {
        __syncwarp();
        tmem_alloc(&bars->tmem_base, 256);
        tmem_relinquish();
    }
    // The aux tile is the second 64-column block of both operands: of B = [Y | aux] (N = 80: its columns 0..15
    // are read) and of A = [X | aux] (M = 128: accumulator row 64 + m is the sum weighted by column m; row 80 is
    // the one read out).  It is constant ones: [A' | a'] = x'^T [Y | 1] and [ysum | count] = 1^T [Y | 1].
    for (int i = tid; i < kTileBytes / 4; i += kLsThreads) reinterpret_cast<uint32_t*>(smem + kLsOffAux)[i] = 0x3F803F80u;
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = bars->tmem_base;
    volatile int* abort_flag = &bars->abort_flag;
    // everything above is private to the CTA; from here on memory of the kernel before this one is touched.
    // (Wait first, then let the next kernel be scheduled: an apply kernel behind this one requests its first
    // tiles before it waits in turn, which is safe only if everything before this kernel is complete by then.)
    grid_dependency_wait();
    allow_dependent_launch();
    LA_TRACE_CTA(g_trace_lin, 1);
    // Ragged batch: only `real` rows of this split exist; chunks behind them are skipped and the rows behind
    // them in the last chunk are zeroed after the load (at least one chunk runs, so that the record is written
    // from an accumulator that holds zeros and not from one that was never started).
    // (Without lengths every sequence has N positions, and N need not be a multiple of the chunk: rows of the last
    // chunk at positions >= N are not in memory; the 3-D tile loads read zeros there.)
    int64_t real = (int64_t)L_all * kChunk;
    {
        const int64_t len = prm.lengths ? min((int64_t)max(prm.lengths[bh / prm.heads], 0), prm.N) : prm.N;
        real = min(max(len - (int64_t)c_begin * kChunk, (int64_t)0), real);
    }
    const int L = max(1, (int)((real + kChunk - 1) / kChunk));

    if (warp == 8) {
        if (lane == 0) {
            prefetch_tensormap(&mapX); prefetch_tensormap(&mapY);
            #pragma unroll 1
            for (int c = 0; c < L; ++c) {
                const int s = c % kLsStages;
                if (c >= kLsStages && !mbar_wait(&bars->empty[s], ((c / kLsStages) - 1) & 1, prm.status, kStatusPipeTimeout)) {
                    *abort_flag = 1;
                    break;
                }
                if (*abort_flag) break;
                uint8_t* st = smem + s * kLsStageBytes;
                const int y = (c_begin + c) * kChunk, z = (int)bh;      // position in the sequence; sequence
                LA_TRACE(g_trace_lin, c, 2);
                mbar_arrive_expect_tx(&bars->full[s], 2 * kTileBytes);
                tile_load<k3d>(st, &mapX, y, z, prm.N, &bars->full[s]);
                tile_load<k3d>(st + kTileBytes, &mapY, y, z, prm.N, &bars->full[s]);
            }
        }
    } else if (warp == 9) {
        {
            const bool leader = elect_one();
            // one M = 128, N = 80 product per K group: A = [X | aux], B = [Y | aux], the second 64-column block
            // of either operand addressed through the leading-offset field.
            // Accumulator rows 0..63: [A' | a'] = x'^T [Y | 1];  row 80: [ysum | count] = 1^T [Y | 1].
            const uint32_t idesc = umma_idesc_bf16(128, 80, 1, 1);
            bool ok = true;
            #pragma unroll 1
            for (int c = 0; c < L && ok; ++c) {
                const int s = c % kLsStages;
                const uint32_t aX = sbase + s * kLsStageBytes, aY = aX + kTileBytes, aA = sbase + kLsOffAux;
                ok = mbar_wait_warp(&bars->mapped[s], (c / kLsStages) & 1, prm.status, kStatusPipeTimeout);
                if (!ok || __any_sync(0xFFFFFFFFu, *abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                if (leader) LA_TRACE(g_trace_lin, c, 0);
                const uint32_t acc = (c != 0);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    umma_bf16(leader, tmem, desc_mn(aX + k * 2048, aA - aX), desc_mn(aY + k * 2048, aA - aY), idesc, acc | (k != 0));
                }
                umma_commit(leader, &bars->empty[s]);
                if (leader) LA_TRACE(g_trace_lin, c, 1);
            }
            if (!ok) *abort_flag = 1;
            umma_commit(leader, &bars->done);
        }
    } else {
        const int t = tid & 127, hf = tid >> 7;
        const uint32_t r7 = t & 7;
        const bool elu = prm.phi == LA_PHI_ELU1;
        const int nch = prm.dim >> 3;
        #pragma unroll 1
        for (int c = 0; c < L; ++c) {
            const int s = c % kLsStages;
            const bool padded = (int64_t)c * kChunk + t >= real;      // whatever the tensors hold there is not read as numbers
            if (!mbar_wait(&bars->full[s], (c / kLsStages) & 1, prm.status, kStatusTmaTimeout)) { *abort_flag = 1; break; }
            if (*abort_flag) break;
            if (tid == 0) LA_TRACE(g_trace_lin, c, 5);
            uint8_t* rowX = smem + s * kLsStageBytes + t * 128;
            if (padded) {
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    sts128(rowX + ((hf * 4 + cc) << 4), 0u, 0u, 0u, 0u);
                    sts128(rowX + kTileBytes + ((hf * 4 + cc) << 4), 0u, 0u, 0u, 0u);
                }
            } else if (elu) {
                elu_half_row_inplace<true>(rowX, r7, 1.f, hf, nch);
            } else {
                elu_half_row_inplace<false>(rowX, r7, 1.f, hf, nch);
            }
            fence_proxy_async_smem();
            mbar_arrive(&bars->mapped[s]);
            if (tid == 0) LA_TRACE(g_trace_lin, c, 6);
        }
        // read-out of this split's record
        const bool ok = mbar_wait(&bars->done, 0, prm.status, kStatusMmaTimeout) && !*abort_flag;
        LA_TRACE_CTA(g_trace_lin, 2);
        tc_fence_after_sync();
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        float* rec = prm.records + (bh * prm.nseg + seg) * (int64_t)kRecFloats;
        if (warp < 3) {             // warps 0, 1: accumulator rows 0..63; warp 2, lane 16: row 80, the w-weighted sums
            const int d_row = warp * 32 + lane;
            const bool mine = ok && (warp < 2 || lane == 16);
            float* dst = warp < 2 ? rec + d_row * kDim : rec + kDim * kDim + kDim;
            for (int h = 0; h < 2; ++h) {
                uint32_t v[32];
                tmem_ld32(tmem + lane_base + h * 32, v);
                tmem_ld_wait();
                if (mine)
#pragma unroll
                    for (int j = 0; j < 32; ++j) dst[h * 32 + j] = __uint_as_float(v[j]);
            }
            const float z = __uint_as_float(tmem_ld1(tmem + lane_base + 64));
            tmem_ld_wait();
            if (mine) {
                if (warp < 2) rec[kDim * kDim + d_row] = z;
                else rec[kDim * kDim + 2 * kDim] = 0.f;        // (the count: unused)
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    LA_TRACE_CTA(g_trace_lin, 3);
    if (warp == 9) {
        __syncwarp();
        tmem_dealloc(tmem, 256);
    }
}

// ===========================================================================
// Apply passes.
// ===========================================================================
enum ApplyMode { kApplyForward = 0, kApplyBackwardQ = 1, kApplyBackwardKV = 2 };

constexpr int kApStages = 4;
constexpr int kApThreads = 448;
constexpr uint32_t kApOffStage = 0;                                   // kApStages x {X, Y}
constexpr uint32_t kApOffState = kApOffStage + kApStages * 2 * kTileBytes;   // bf16 centred state tile [64][64]
constexpr uint32_t kApOffVec = kApOffState + kDim * 128;              // fp32 [3][64]: a' (Z' or r'), nu, scratch
constexpr uint32_t kApOffBar = kApOffVec + 1024;
constexpr uint32_t kApOffOut = (kApOffBar + 256 + 1023) & ~1023u;      // two result tiles on their way out
constexpr uint32_t kApOffX = kApOffOut + 2 * kTileBytes;               // fp32 [2 halves][128 rows][8]: partial sums exchanged
// backward Q only: the chunk's weighted queries x' / dn and its aux tile (columns 0..15: dl_i, 16..23: 1 / dn_i),
// operands of the reverse sums that this pass forms on the side (see the sum kernel for the product)
constexpr uint32_t kApOffXS = kApOffX + 2 * 128 * 8 * 4;
constexpr uint32_t kApOffAux = kApOffXS + kTileBytes;
constexpr uint32_t kApSmemBytes = kApOffAux + kTileBytes + 1024;       // + slack for the 1 KB alignment of the base
constexpr uint32_t kApColSums = 256;                                   // TMEM columns of the reverse sums (80)

struct ApBarriers {
    uint64_t full[kApStages], empty[kApStages], mapped[kApStages];
    uint64_t acc_full[2], acc_free[2];
    uint64_t xs_ready, xs_free, sums_done;      // backward Q: hand-offs of the weighted tile and the end of the reverse sums
    uint32_t tmem_base;
    int abort_flag;
};

struct ApParams {
    const float* records;       // [BH][nseg][kRecFloats]: summed by every CTA
    __nv_bfloat16* out0;        // forward: O;  backward Q: dQ;  backward K/V: dK
    __nv_bfloat16* out1;        // backward K/V: dV
    float* den;                 // forward: q.Z (optional)
    float* rec_out;             // backward Q: [BH][nseg][kRecFloats] reverse sums of this pass's rows (out)
    float* state_out;           // forward: KV [BH][64][64] (optional)
    float* vec_out;             // forward: Zs [BH][64] (optional)
    const int* lengths;         // [B] real positions per batch element (right-padded ragged batch), or null
    int heads;
    int* status;
    int64_t N;
    int chunks, chunks_per_seg, nseg;
    float eps;
    int phi;
    int dim;                    // D = M: 64, or 32 (tiles zero-padded to 64 columns)
    int early;                  // a kernel of the same call runs in front: the first tiles are requested before the wait
};

template <int kMode, bool k3d>
__global__ void __launch_bounds__(kApThreads, 1)
linear_apply_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapY,
                    const __grid_constant__ CUtensorMap mapOut0, const __grid_constant__ CUtensorMap mapOut1,
                    const ApParams prm) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    ApBarriers* bars = reinterpret_cast<ApBarriers*>(smem + kApOffBar);
    float* sA = reinterpret_cast<float*>(smem + kApOffVec);      // a': Z' (forward, backward Q) or r' (backward K/V)
    float* sNu = sA + 64;                                        // rank-one part along 1: ysum + mu  /  gsum + rho
    float* sScal = sA + 128;                                     // [0] = sum_d a'_d, [1] = w0
    constexpr bool kHasY = kMode != kApplyForward;
    constexpr uint32_t kTiles = kHasY ? 2 : 1;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int seg = blockIdx.x % prm.nseg;
    const int64_t bh = blockIdx.x / prm.nseg;
    const int c_begin = seg * prm.chunks_per_seg;
    const int L_all = min(prm.chunks, c_begin + prm.chunks_per_seg) - c_begin;
    const int64_t row0 = bh * prm.N + (int64_t)c_begin * kChunk;
    LA_TRACE_CTA(g_trace_lin, 4);

    if (tid == 0) {
        for (int s = 0; s < kApStages; ++s) {
            mbar_init(&bars->full[s], 1);
            // MMA commit + epilogue threads (they read the X and Y rows) (+ the commit of the reverse sums, which read Y)
            mbar_init(&bars->empty[s], 1 + 256 + (kMode == kApplyBackwardQ ? 1 : 0));
            mbar_init(&bars->mapped[s], 128);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&bars->acc_full[b], 1);
            mbar_init(&bars->acc_free[b], 256);
        }
        mbar_init(&bars->xs_ready, 256);
        mbar_init(&bars->xs_free, 1);
        mbar_init(&bars->sums_done, 1);
        bars->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 9) {
        __syncwarp();
        tmem_alloc(&bars->tmem_base, 512);
        tmem_relinquish();
    }
    __syncthreads();            // the barriers are initialised for the loads issued before the prologue below
    // (set-up above is private to the CTA; the records below come from the kernel before this one)
    // The tiles of this pass are inputs of the call.  Behind another kernel of the same call (which waited for
    // everything before it and only then let this one be scheduled) the first of them are requested before the
    // wait and arrive while that kernel drains; as the first kernel of a call everything waits first.
    const bool early = prm.early != 0;
    if (!early) {
        grid_dependency_wait();
        allow_dependent_launch();
    }
    // Ragged batch: `len` positions of this sequence exist, `real` of them in this split.  Only the chunks that
    // hold real rows go through the pipeline; the padding behind them is filled with zeros at the end.
    // (Without lengths len = N, which need not be a multiple of the chunk: rows at positions >= N are not in memory;
    // the tile loads read zeros there, the tile stores clip them and the plain stores below skip them.)
    int64_t len = prm.N, real = (int64_t)L_all * kChunk;
    if (prm.lengths) len = min((int64_t)max(prm.lengths[bh / prm.heads], 0), prm.N);
    real = min(max(len - (int64_t)c_begin * kChunk, (int64_t)0), real);
    const int L = (int)((real + kChunk - 1) / kChunk);
    // the loads of the first chunks travel while the state is put together below
    auto issue_load = [&](int c) {
        const int s = c % kApStages;
        uint8_t* st = smem + kApOffStage + s * 2 * kTileBytes;
        const int y = (c_begin + c) * kChunk, z = (int)bh;          // position in the sequence; sequence
        mbar_arrive_expect_tx(&bars->full[s], kTiles * kTileBytes);
        tile_load<k3d>(st, &mapX, y, z, prm.N, &bars->full[s]);
        if (kHasY) tile_load<k3d>(st + kTileBytes, &mapY, y, z, prm.N, &bars->full[s]);
    };
    if (warp == 8 && lane == 0) {
        prefetch_tensormap(&mapX);
        if (kHasY) prefetch_tensormap(&mapY);
        for (int c = 0; c < min(L, kApStages); ++c) issue_load(c);
    }
    if (early) {
        grid_dependency_wait();
        allow_dependent_launch();
    }
    // state of this head: add the split records (fp32), remove the column means, round the
    // centred remainder to a bf16 operand tile.  Scratch: the output staging tiles, free until the first epilogue.
    {
        const float* rec = prm.records + bh * prm.nseg * (int64_t)kRecFloats;
        float* sF = reinterpret_cast<float*>(smem + kApOffOut);                   // fp32 [64][64] scratch (+ 64 means)
        {
            constexpr int kPer = (kDim * kDim / 4 + kApThreads - 1) / kApThreads;     // float4 slots per thread
            float4 acc[kPer];
#pragma unroll
            for (int u = 0; u < kPer; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 2
            for (int n = 0; n < prm.nseg; ++n) {
                const float4* src = reinterpret_cast<const float4*>(rec + (int64_t)n * kRecFloats);
#pragma unroll
                for (int u = 0; u < kPer; ++u) {        // independent loads: all in flight together
                    const int idx = tid + u * kApThreads;
                    if (idx < kDim * kDim / 4) {
                        const float4 a = __ldg(src + idx);
                        acc[u].x += a.x; acc[u].y += a.y; acc[u].z += a.z; acc[u].w += a.w;
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < kPer; ++u) {
                const int idx = tid + u * kApThreads;
                if (idx < kDim * kDim / 4) reinterpret_cast<float4*>(sF)[idx] = acc[u];
            }
        }
        if (tid < 2 * kDim + 1) {       // a' (64), ysum (64), w0 (1)
            float z = 0.f;
            for (int n = 0; n < prm.nseg; ++n) z += __ldg(rec + (int64_t)n * kRecFloats + kDim * kDim + tid);
            if (tid < kDim) sA[tid] = z;
            else if (tid < 2 * kDim) sNu[tid - kDim] = z;
            else sScal[1] = z;
        }
        __syncthreads();
        const int dim = prm.dim;
        // column sums in two steps (a thread alone would walk its column for a microsecond): four threads per column
        // take every fourth row, in a fixed order, and leave their partial sums behind the matrix
        float* sPartial = sF + kDim * kDim + kDim;                                // fp32 [4][64]
        if (tid < 4 * kDim) {
            const int col = tid & (kDim - 1), part = tid >> 6;
            float m = 0.f;
            for (int d = part; d < dim; d += 4) m += sF[d * kDim + col];
            sPartial[part * kDim + col] = m;
        }
        __syncthreads();
        if (tid < kDim) {               // column tid: mean over the dim real rows; nu = ysum + mu
            float m = (sPartial[tid] + sPartial[kDim + tid]) + (sPartial[2 * kDim + tid] + sPartial[3 * kDim + tid]);
            m *= 1.f / dim;
            const float ysum = sNu[tid];
            sNu[tid] = ysum + m;
            sF[kDim * kDim + tid] = m;                                            // mu, just past the matrix
            if (kMode == kApplyForward && seg == 0 && tid < dim) {
                // true sums for the caller: S = 1 ysum^T + A', Z = N 1 + a'
                if (prm.vec_out) prm.vec_out[bh * dim + tid] = (float)len + sA[tid];
                if (prm.state_out)
                    for (int d = 0; d < dim; ++d)
                        prm.state_out[bh * (int64_t)(dim * dim) + d * dim + tid] = sF[d * kDim + tid] + ysum;
            }
        }
        if (warp == 2) {                // sum of a' (64 values, two per lane, then a butterfly: the same order in every CTA)
            float z = sA[lane] + sA[lane + 32];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) z += __shfl_xor_sync(0xffffffffu, z, off);
            if (lane == 0) sScal[0] = z;
        }
        __syncthreads();
        for (int idx = tid; idx < kDim * kDim / 8; idx += kApThreads) {       // 8 consecutive columns of one row
            const int d = idx >> 3, c8 = idx & 7;
            float v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = d < dim ? sF[d * kDim + c8 * 8 + j] - sF[kDim * kDim + c8 * 8 + j] : 0.f;
            sts128(smem + kApOffState + d * 128 + ((c8 ^ (d & 7)) << 4), pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]),
                   pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
        }
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = bars->tmem_base;
    volatile int* abort_flag = &bars->abort_flag;
    LA_TRACE_CTA(g_trace_lin, 5);

    if (warp == 8) {
        if (lane == 0) {
            #pragma unroll 1
            for (int c = kApStages; c < L; ++c) {
                if (!mbar_wait(&bars->empty[c % kApStages], ((c / kApStages) - 1) & 1, prm.status, kStatusPipeTimeout)) {
                    *abort_flag = 1;
                    break;
                }
                if (*abort_flag) break;
                issue_load(c);
            }
        }
    } else if (warp == 9) {
        {
            const bool leader = elect_one();
            const uint32_t idesc_kk = umma_idesc_bf16(128, 64, 0, 0);
            const uint32_t idesc_kmn = umma_idesc_bf16(128, 64, 0, 1);
            const uint32_t aSt = sbase + kApOffState;
            bool ok = true;
            // backward Q: the reverse sums of chunk c, [A' | a'] += (x' / dn)^T [G | dl] and (row 80) the sums weighted by
            // 1 / dn, once the epilogue threads have written the weighted tile: one M = 128, N = 80 product per K
            // group, A = [XS | aux], B = [G | aux] (second blocks through the leading-offset field)
            auto issue_sums = [&](int c) -> bool {
                if (!mbar_wait_warp(&bars->xs_ready, c & 1, prm.status, kStatusPipeTimeout) || __any_sync(0xFFFFFFFFu, *abort_flag)) return false;
                tc_fence_after_sync();
                const uint32_t idesc = umma_idesc_bf16(128, 80, 1, 1);
                const uint32_t aXS = sbase + kApOffXS, aAux = sbase + kApOffAux;
                const uint32_t aG = sbase + kApOffStage + (c % kApStages) * 2 * kTileBytes + kTileBytes;
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    umma_bf16(leader, tmem + kApColSums, desc_mn(aXS + k * 2048, aAux - aXS), desc_mn(aG + k * 2048, aAux - aG), idesc,
                              (c | k) != 0);
                umma_commit(leader, &bars->empty[c % kApStages]);
                umma_commit(leader, &bars->xs_free);
                return true;
            };
            #pragma unroll 1
            for (int c = 0; c < L && ok; ++c) {
                const int s = c % kApStages, b = c & 1;
                const uint32_t aX = sbase + kApOffStage + s * 2 * kTileBytes, aY = aX + kTileBytes;
                ok = mbar_wait_warp(&bars->mapped[s], (c / kApStages) & 1, prm.status, kStatusPipeTimeout);
                if (ok && c >= 2) ok = mbar_wait_warp(&bars->acc_free[b], ((c >> 1) - 1) & 1, prm.status, kStatusPipeTimeout);
                if (!ok || __any_sync(0xFFFFFFFFu, *abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d0 = tmem + b * 128, d1 = d0 + 64;
                if (kMode == kApplyForward) {
                    for (int k = 0; k < 4; ++k)      // q' S''
                        umma_bf16(leader, d0, desc_k(aX + k * 32), desc_mn(aSt + k * 2048), idesc_kmn, k > 0);
                } else if (kMode == kApplyBackwardQ) {
                    for (int k = 0; k < 4; ++k)      // h'' = G S''^T
                        umma_bf16(leader, d0, desc_k(aY + k * 32), desc_k(aSt + k * 32), idesc_kk, k > 0);
                } else {
                    for (int k = 0; k < 4; ++k)      // V R''^T
                        umma_bf16(leader, d0, desc_k(aY + k * 32), desc_k(aSt + k * 32), idesc_kk, k > 0);
                    for (int k = 0; k < 4; ++k)      // k' R''
                        umma_bf16(leader, d1, desc_k(aX + k * 32), desc_mn(aSt + k * 2048), idesc_kmn, k > 0);
                }
                umma_commit(leader, &bars->acc_full[b]);
                umma_commit(leader, &bars->empty[s]);
                if (kMode == kApplyBackwardQ && c >= 1) ok = issue_sums(c - 1);
            }
            if (kMode == kApplyBackwardQ && ok && L >= 1) ok = issue_sums(L - 1);
            if (kMode == kApplyBackwardQ) umma_commit(leader, &bars->sums_done);
            if (!ok) *abort_flag = 1;
        }
    } else if (warp >= 4 && warp < 8) {
        const int t = tid - 128;
        const uint32_t r7 = t & 7;
        const bool elu = prm.phi == LA_PHI_ELU1;
        #pragma unroll 1
        for (int c = 0; c < L; ++c) {
            const int s = c % kApStages;
            if (!mbar_wait(&bars->full[s], (c / kApStages) & 1, prm.status, kStatusTmaTimeout)) { *abort_flag = 1; break; }
            if (*abort_flag) break;
            if (t == 0) LA_TRACE(g_trace_lin, c, 14);
            uint8_t* rowX = smem + kApOffStage + s * 2 * kTileBytes + t * 128;
            if (elu) elu_row_inplace<true>(rowX, r7, 1.f, prm.dim >> 3); else elu_row_inplace<false>(rowX, r7, 1.f, prm.dim >> 3);
            fence_proxy_async_smem();
            mbar_arrive(&bars->mapped[s]);
            if (t == 0) LA_TRACE(g_trace_lin, c, 15);
        }
    } else {
        // Epilogue: two warps per TMEM quadrant (warps 0-3: columns 0..31 of a row, warps 10-13: columns 32..63;
        // one thread per row and half).  The sums that run over a whole row (x'.1, x'.a', Y.nu, 1.h'', q'.h'') are
        // formed per half and exchanged through shared memory inside the pair.
        const int hf = warp >= 10 ? 1 : 0;
        const int quad = warp & 3;
        const int t = quad * 32 + lane;
        const uint32_t r7 = t & 7;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        const bool elu = prm.phi == LA_PHI_ELU1;
        const float fD = (float)prm.dim, fN = (float)len;
        // (columns beyond a 32-wide problem are zero padding: they add nothing to the sums, and the store clips them)
        float* sX = reinterpret_cast<float*>(smem + kApOffX);
        float* mine = sX + (hf * 128 + t) * 8;
        const float* other = sX + ((hf ^ 1) * 128 + t) * 8;
        const float* aH = sA + hf * 32;
        const float* nuH = sNu + hf * 32;
        #pragma unroll 1
        for (int c = 0; c < L; ++c) {
            const int s = c % kApStages, b = c & 1;
            const int64_t row = row0 + (int64_t)c * kChunk + t;
            const bool padded = (int64_t)c * kChunk + t >= real;      // a row behind the sequence's end: zeros go out
            if (!mbar_wait(&bars->mapped[s], (c / kApStages) & 1, prm.status, kStatusPipeTimeout)) { *abort_flag = 1; break; }
            if (*abort_flag) break;
            if (tid == 0) LA_TRACE(g_trace_lin, c, 8);
            uint32_t xv[4][4];                       // this half of the x' = elu(X) row
            const uint8_t* rowX = smem + kApOffStage + s * 2 * kTileBytes + t * 128;
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) lds128(rowX + (((hf * 4 + cc) ^ r7) << 4), xv[cc]);
            float ynu_h = 0.f;                       // this half of Y_i . nu (backward)
            if (kHasY) {
                uint32_t yv[4][4];
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) lds128(rowX + kTileBytes + (((hf * 4 + cc) ^ r7) << 4), yv[cc]);
                // (two columns per instruction from here on: the epilogue is bound by instruction issue)
                f32x2 p4[4] = {0, 0, 0, 0};
#pragma unroll
                for (int cc = 0; cc < 4; ++cc)
#pragma unroll
                    for (int j = 0; j < 4; ++j) p4[j] = fma2(pair_bf16(yv[cc][j]), pair_ld(nuH + cc * 8 + 2 * j), p4[j]);
                ynu_h = pair_sum(add2(add2(p4[0], p4[1]), add2(p4[2], p4[3])));
            }
            mbar_arrive(&bars->empty[s]);
            f32x2 sx4[4] = {0, 0, 0, 0}, xa4[4] = {0, 0, 0, 0};
#pragma unroll
            for (int cc = 0; cc < 4; ++cc)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const f32x2 x2 = pair_bf16(xv[cc][j]);
                    sx4[j] = add2(sx4[j], x2);
                    xa4[j] = fma2(x2, pair_ld(aH + cc * 8 + 2 * j), xa4[j]);
                }
            if (!mbar_wait(&bars->acc_full[b], (c >> 1) & 1, prm.status, kStatusMmaTimeout)) { *abort_flag = 1; break; }
            tc_fence_after_sync();
            if (tid == 0) LA_TRACE(g_trace_lin, c, 9);
            uint32_t acc[32];
            tmem_ld32(tmem + lane_base + b * 128 + hf * 32, acc);
            tmem_ld_wait();
            float sh_h = 0.f, qh_h = 0.f;
            if (kMode == kApplyBackwardQ) {
                f32x2 sh4[4] = {0, 0, 0, 0}, qh4[4] = {0, 0, 0, 0};
#pragma unroll
                for (int cc = 0; cc < 4; ++cc)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const f32x2 h2 = pair(acc[cc * 8 + 2 * j], acc[cc * 8 + 2 * j + 1]);
                        sh4[j] = add2(sh4[j], h2);
                        qh4[j] = fma2(pair_bf16(xv[cc][j]), h2, qh4[j]);
                    }
                sh_h = pair_sum(add2(add2(sh4[0], sh4[1]), add2(sh4[2], sh4[3])));
                qh_h = pair_sum(add2(add2(qh4[0], qh4[1]), add2(qh4[2], qh4[3])));
            }
            // the pair's previous slab must have left the staging tile before either warp rewrites it below
            if (hf == 0 && lane == 0) tma_store_wait_read<0>();
            if (tid == 0) LA_TRACE(g_trace_lin, c, 10);
            mine[0] = pair_sum(add2(add2(sx4[0], sx4[1]), add2(sx4[2], sx4[3])));
            mine[1] = pair_sum(add2(add2(xa4[0], xa4[1]), add2(xa4[2], xa4[3])));
            mine[2] = ynu_h;
            mine[3] = sh_h;
            mine[4] = qh_h;
            named_barrier(2 + quad, 64);
            // both threads of a row add the halves in the same order (half 0 first): identical totals
            const float* lo = hf ? other : mine;
            const float* hi = hf ? mine : other;
            const float sx = lo[0] + hi[0], xa = lo[1] + hi[1], ynu = lo[2] + hi[2], sh = lo[3] + hi[3], qh = lo[4] + hi[4];
            named_barrier(2 + quad, 64);            // the exchange slots may be rewritten after this
            if (tid == 0) LA_TRACE(g_trace_lin, c, 11);
            const float x1sum = fD + sx;             // (1 + x') . 1
            uint8_t* out_row = smem + kApOffOut + t * 128;
            if (kMode == kApplyForward) {
                // den = (1 + q') . (N 1 + Z');  num = (1 + q').1 nu + q' S''
                const float den = fN * x1sum + sScal[0] + xa;
                const float inv = 1.f / (den + prm.eps);
                const float w = x1sum * inv;
                if (hf == 0 && prm.den && (!k3d || (int64_t)(c_begin + c) * kChunk + t < prm.N)) prm.den[row] = padded ? 0.f : den;
                const f32x2 inv2 = pair(inv, inv), w2 = pair(w, w);
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    uint32_t outp[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j)     // acc * inv + w * nu
                        outp[j] = pack_bf16x2(fma2(pair(acc[cc * 8 + 2 * j], acc[cc * 8 + 2 * j + 1]), inv2,
                                                   mul2(w2, pair_ld(nuH + cc * 8 + 2 * j))));
                    sts128(out_row + (((hf * 4 + cc) ^ r7) << 4), outp[0], outp[1], outp[2], outp[3]);
                }
            } else {
                // backward Q:  h = (G.nu) 1 + h'',  Z = N 1 + Z',  gq = (h - (q.h / dn) Z) / dn
                // backward KV: gk = (V.nu_R + w0) 1 + V R''^T + r'
                float c1 = 0.f, cz = 0.f, scale = 1.f;          // out_d = scale * (acc_d + c1 + cz * a'_d)
                if (kMode == kApplyBackwardQ) {
                    const float den = fN * x1sum + sScal[0] + xa;
                    const float dn = den + prm.eps;
                    scale = 1.f / dn;
                    const float q_h = ynu * x1sum + sh + qh;                      // q . h
                    const float dl = -q_h * scale;                                // dl_i = -(G_i . O_i)
                    c1 = fmaf(dl, fN, ynu);                                       // (G.nu) + dl N
                    cz = dl;
                    // operands of the reverse sums: the weighted queries x' / dn, and [dl_i | 1 / dn_i] in the aux tile
                    // (rows behind the sequence's end: zeros, also in the G tile, whatever it holds there)
                    if (c > 0 && !mbar_wait(&bars->xs_free, (c - 1) & 1, prm.status, kStatusMmaTimeout)) { *abort_flag = 1; break; }
                    const float wq = padded ? 0.f : scale, dq = padded ? 0.f : dl;
                    uint8_t* xs_row = smem + kApOffXS + t * 128;
                    const f32x2 wq2 = pair(wq, wq);
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc)
                        sts128(xs_row + (((hf * 4 + cc) ^ r7) << 4),
                               pack_bf16x2(mul2(pair_bf16(xv[cc][0]), wq2)), pack_bf16x2(mul2(pair_bf16(xv[cc][1]), wq2)),
                               pack_bf16x2(mul2(pair_bf16(xv[cc][2]), wq2)), pack_bf16x2(mul2(pair_bf16(xv[cc][3]), wq2)));
                    if (hf == 0) {
                        uint8_t* aux_row = smem + kApOffAux + t * 128;
                        const uint32_t dd = pack_bf16x2(dq, dq), ww = pack_bf16x2(wq, wq);
                        sts128(aux_row + ((0 ^ r7) << 4), dd, dd, dd, dd);
                        sts128(aux_row + ((1 ^ r7) << 4), dd, dd, dd, dd);
                        sts128(aux_row + ((2 ^ r7) << 4), ww, ww, ww, ww);
                    }
                    if (padded) {
                        uint8_t* g_row = smem + kApOffStage + s * 2 * kTileBytes + kTileBytes + t * 128;
#pragma unroll
                        for (int cc = 0; cc < 4; ++cc) sts128(g_row + ((hf * 4 + cc) << 4), 0u, 0u, 0u, 0u);
                    }
                    fence_proxy_async_smem();
                    mbar_arrive(&bars->xs_ready);
                } else {
                    c1 = ynu + sScal[1];
                    cz = 1.f;
                }
                const f32x2 scale2 = pair(scale, scale), cz2 = pair(cz, cz), c12 = pair(c1, c1), one2 = pair(1.f, 1.f);
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    uint32_t outp[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int e = cc * 8 + 2 * j;
                        f32x2 g2 = mul2(scale2, add2(fma2(cz2, pair_ld(aH + e), pair(acc[e], acc[e + 1])), c12));
                        // phi'(x) from x' = elu(x): 1 where x' > 0, else 1 + x', i.e. 1 + min(x', 0)
                        if (elu) g2 = mul2(g2, add2(pair_bf16(min_bf16x2(xv[cc][j], 0u)), one2));
                        outp[j] = pack_bf16x2(g2);
                    }
                    sts128(out_row + (((hf * 4 + cc) ^ r7) << 4), outp[0], outp[1], outp[2], outp[3]);
                }
                if (kMode == kApplyBackwardKV) {
                    tmem_ld32(tmem + lane_base + b * 128 + 64 + hf * 32, acc);
                    tmem_ld_wait();
                    const f32x2 xs2 = pair(x1sum, x1sum);
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {       // gV = (1 + k').1 nu_R + k' R''
                        uint32_t outp[4];
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            outp[j] = pack_bf16x2(fma2(xs2, pair_ld(nuH + cc * 8 + 2 * j), pair(acc[cc * 8 + 2 * j], acc[cc * 8 + 2 * j + 1])));
                        sts128(out_row + kTileBytes + (((hf * 4 + cc) ^ r7) << 4), outp[0], outp[1], outp[2], outp[3]);
                    }
                }
            }
            if (padded) {
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    sts128(out_row + (((hf * 4 + cc) ^ r7) << 4), 0u, 0u, 0u, 0u);
                    if (kMode == kApplyBackwardKV) sts128(out_row + kTileBytes + (((hf * 4 + cc) ^ r7) << 4), 0u, 0u, 0u, 0u);
                }
            }
            if (tid == 0) LA_TRACE(g_trace_lin, c, 12);
            tc_fence_before_sync();
            mbar_arrive(&bars->acc_free[b]);
            fence_proxy_async_smem();
            named_barrier(2 + quad, 64);            // both halves of the 32 rows are in the slab
            if (hf == 0 && lane == 0) {
                const int y = (c_begin + c) * kChunk + quad * 32;       // rows at positions >= N are clipped by the store
                if (!k3d || y < prm.N) {
                    tile_store<k3d>(&mapOut0, smem + kApOffOut + quad * 32 * 128, y, (int)bh, prm.N);
                    if (kMode == kApplyBackwardKV) tile_store<k3d>(&mapOut1, smem + kApOffOut + kTileBytes + quad * 32 * 128, y, (int)bh, prm.N);
                }
                tma_store_commit();
            }
            if (tid == 0) LA_TRACE(g_trace_lin, c, 13);
        }
        if (hf == 0 && lane == 0) tma_store_wait_all<0>();
        LA_TRACE_CTA(g_trace_lin, 6);
        if (kMode == kApplyBackwardQ && warp < 3) {
            // this split's record of the reverse sums: accumulator rows 0..63 (warps 0, 1) and row 80 (warp 2, lane 16),
            // zeros if the split holds no real row
            const bool ok = mbar_wait(&bars->sums_done, 0, prm.status, kStatusMmaTimeout) && !*abort_flag;
            tc_fence_after_sync();
            float* rec = prm.rec_out + (bh * prm.nseg + seg) * (int64_t)kRecFloats;
            const int d_row = warp * 32 + lane;
            const bool mine = ok && (warp < 2 || lane == 16);
            float* dst = warp < 2 ? rec + d_row * kDim : rec + kDim * kDim + kDim;
            for (int h = 0; h < 2; ++h) {
                uint32_t v[32];
                tmem_ld32(tmem + lane_base + kApColSums + h * 32, v);
                tmem_ld_wait();
                if (mine)
#pragma unroll
                    for (int j = 0; j < 32; ++j) dst[h * 32 + j] = L > 0 ? __uint_as_float(v[j]) : 0.f;
            }
            const float z = __uint_as_float(tmem_ld1(tmem + lane_base + kApColSums + 64));
            tmem_ld_wait();
            if (mine) {
                if (warp < 2) rec[kDim * kDim + d_row] = L > 0 ? z : 0.f;
                else rec[kDim * kDim + 2 * kDim] = L > 0 ? z : 0.f;
            }
        }
        if (L < L_all) {            // whole chunks of padding: zeros, written directly
            const int e = hf * 128 + t;
            const int64_t r_lo = row0 + (int64_t)L * kChunk;
            const int64_t nrows = max((int64_t)0, min((int64_t)(L_all - L) * kChunk, prm.N - (int64_t)(c_begin + L) * kChunk));
            const int64_t n16 = nrows * prm.dim * 2 / 16;
            uint4* o0 = reinterpret_cast<uint4*>(prm.out0 + r_lo * prm.dim);
            for (int64_t i = e; i < n16; i += 256) o0[i] = make_uint4(0u, 0u, 0u, 0u);
            if (kMode == kApplyBackwardKV) {
                uint4* o1 = reinterpret_cast<uint4*>(prm.out1 + r_lo * prm.dim);
                for (int64_t i = e; i < n16; i += 256) o1[i] = make_uint4(0u, 0u, 0u, 0u);
            }
            if (kMode == kApplyForward && prm.den)
                for (int64_t i = e; i < nrows; i += 256) prm.den[r_lo + i] = 0.f;
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    LA_TRACE_CTA(g_trace_lin, 7);
    if (warp == 9) {
        __syncwarp();
        tmem_dealloc(tmem, 512);
    }
}

// Splits per sequence: at most one CTA per SM over all heads (measured at B*H = 64, N = 4096: two splits of
// 16 chunks take 0.24 ms per forward + backward, five splits of 6-7 chunks 0.33 ms: a CTA's start-up costs
// several chunk times, and more CTAs than resident slots run in waves), at least two chunks each.
Segmentation choose_splits(const la_problem& p) {
    const int chunks = chunks_of(p.N);
    const int64_t bh = p.B * p.H;
    int nseg = (int)(sm_count() / bh);
    if (plan_override().linear_splits > 0) nseg = plan_override().linear_splits;        // A/B checks
    if (nseg > chunks / 2) nseg = chunks / 2;
    if (nseg < 1) nseg = 1;
    const int cps = (chunks + nseg - 1) / nseg;
    nseg = (chunks + cps - 1) / cps;
    return Segmentation{nseg, cps};
}

template <bool k3d>
int launch_sums_as(const la_problem& p, const Segmentation& sg, const CUtensorMap& mX, const CUtensorMap& mY,
                   const int* lengths, float* records, cudaStream_t st) {
    static std::atomic<uint64_t> attr_done{0};          // one per instantiation
    if (int rc = opt_in_smem_once(linear_sum_kernel<k3d>, kLsSmemBytes, attr_done)) return rc;
    LsParams prm;
    prm.records = records;
    prm.lengths = lengths;
    prm.heads = (int)p.H;
    prm.status = device_status_ptr();
    if (!prm.status) return fail(LA_ERR_CUDA, "device status word unavailable");
    prm.N = p.N;
    prm.chunks = chunks_of(p.N);
    prm.chunks_per_seg = sg.chunks_per_seg;
    prm.nseg = sg.nseg;
    prm.phi = p.phi;
    prm.dim = (int)p.D;
    prof_begin(kProfLinearSum, st);
    cudaLaunchAttribute attr;
    const cudaLaunchConfig_t cfg = chained_launch((unsigned)(sg.nseg * p.B * p.H), kLsThreads, kLsSmemBytes, st, &attr);
    LA_CUDA_TRY(cudaLaunchKernelEx(&cfg, linear_sum_kernel<k3d>, mX, mY, prm));
    note_launch();
    prof_end(kProfLinearSum, st);
    return LA_OK;
}

int launch_sums(const la_problem& p, const Segmentation& sg, const CUtensorMap& mX, const CUtensorMap& mY,
                const int* lengths, float* records, cudaStream_t st) {
    return p.N % kChunk ? launch_sums_as<true>(p, sg, mX, mY, lengths, records, st)
                        : launch_sums_as<false>(p, sg, mX, mY, lengths, records, st);
}

template <int kMode, bool k3d>
int launch_apply_as(const la_problem& p, const Segmentation& sg, const CUtensorMap& mX, const CUtensorMap& mY,
                    ApParams prm, cudaStream_t st) {
    static std::atomic<uint64_t> attr_done{0};          // one per instantiation
    if (int rc = opt_in_smem_once(linear_apply_kernel<kMode, k3d>, kApSmemBytes, attr_done)) return rc;
    prm.status = device_status_ptr();
    if (!prm.status) return fail(LA_ERR_CUDA, "device status word unavailable");
    prm.heads = (int)p.H;
    prm.N = p.N;
    prm.chunks = chunks_of(p.N);
    prm.chunks_per_seg = sg.chunks_per_seg;
    prm.nseg = sg.nseg;
    prm.eps = p.eps;
    prm.phi = p.phi;
    prm.dim = (int)p.D;
    const uint64_t seqs = (uint64_t)(p.B * p.H), n = (uint64_t)p.N;
    CUtensorMap mO0, mO1;                   // one warp's 32 rows per store
    if (int rc = encode_attention_map(&mO0, prm.out0, p.N % kChunk != 0, seqs, n, 32, (int)p.D)) return rc;
    if (int rc = encode_attention_map(&mO1, prm.out1 ? prm.out1 : prm.out0, p.N % kChunk != 0, seqs, n, 32, (int)p.D)) return rc;
    prof_begin(kProfLinearApply, st);
    cudaLaunchAttribute attr;
    const cudaLaunchConfig_t cfg = chained_launch((unsigned)(sg.nseg * p.B * p.H), kApThreads, kApSmemBytes, st, &attr);
    LA_CUDA_TRY(cudaLaunchKernelEx(&cfg, linear_apply_kernel<kMode, k3d>, mX, mY, mO0, mO1, prm));
    note_launch();
    prof_end(kProfLinearApply, st);
    return LA_OK;
}

template <int kMode>
int launch_apply(const la_problem& p, const Segmentation& sg, const CUtensorMap& mX, const CUtensorMap& mY,
                 const ApParams& prm, cudaStream_t st) {
    return p.N % kChunk ? launch_apply_as<kMode, true>(p, sg, mX, mY, prm, st)
                        : launch_apply_as<kMode, false>(p, sg, mX, mY, prm, st);
}

}  // namespace

size_t linear_forward_workspace(const la_problem& p) {
    return (size_t)(p.B * p.H) * choose_splits(p).nseg * kRecFloats * sizeof(float);
}

size_t linear_backward_workspace(const la_problem& p) {
    return 2 * linear_forward_workspace(p);
}

int linear_forward(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths, void* O,
                   float* den, float* KV, float* Zs, void* saved, void* ws, cudaStream_t st) {
    const Segmentation sg = choose_splits(p);
    const uint64_t seqs = (uint64_t)(p.B * p.H), n = (uint64_t)p.N;
    CUtensorMap mQ, mK, mV;
    if (int rc = encode_attention_map(&mQ, Q, p.N % kChunk != 0, seqs, n, kChunk, (int)p.D)) return rc;
    if (int rc = encode_attention_map(&mK, K, p.N % kChunk != 0, seqs, n, kChunk, (int)p.D)) return rc;
    if (int rc = encode_attention_map(&mV, V, p.N % kChunk != 0, seqs, n, kChunk, (int)p.D)) return rc;
    float* rec = saved ? (float*)saved : (float*)ws;      // the split records, kept for the backward pass if asked
    if (int rc = launch_sums(p, sg, mK, mV, lengths, rec, st)) return rc;
    ApParams a = {};
    a.lengths = lengths;
    a.records = rec;
    a.out0 = (__nv_bfloat16*)O;
    a.den = den;
    a.state_out = KV;
    a.vec_out = Zs;
    a.early = 1;                // behind the sum kernel
    return launch_apply<kApplyForward>(p, sg, mQ, mQ, a, st);
}

int linear_backward(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths,
                    const void* saved, const void* G, void* dQ, void* dK, void* dV, void* ws, cudaStream_t st) {
    const Segmentation sg = choose_splits(p);
    const size_t bh = (size_t)(p.B * p.H);
    const uint64_t n = (uint64_t)p.N;
    CUtensorMap mQ, mK, mV, mG;
    if (int rc = encode_attention_map(&mQ, Q, p.N % kChunk != 0, bh, n, kChunk, (int)p.D)) return rc;
    if (int rc = encode_attention_map(&mK, K, p.N % kChunk != 0, bh, n, kChunk, (int)p.D)) return rc;
    if (int rc = encode_attention_map(&mV, V, p.N % kChunk != 0, bh, n, kChunk, (int)p.D)) return rc;
    if (int rc = encode_attention_map(&mG, G, p.N % kChunk != 0, bh, n, kChunk, (int)p.D)) return rc;
    uint8_t* w = (uint8_t*)ws;
    float* rec_s = (float*)w;   w += bh * sg.nseg * kRecFloats * sizeof(float);
    float* rec_r = (float*)w;   w += bh * sg.nseg * kRecFloats * sizeof(float);

    if (saved) rec_s = (float*)saved;         // the forward's own records: nothing to recompute
    else if (int rc = launch_sums(p, sg, mK, mV, lengths, rec_s, st)) return rc;
    ApParams a = {};
    a.early = saved ? 0 : 1;    // the first kernel of the call with saved records, else behind the sum kernel
    a.lengths = lengths;
    a.records = rec_s;
    a.out0 = (__nv_bfloat16*)dQ;
    a.rec_out = rec_r;          // the reverse sums of Q / dn and G are formed by the same pass
    if (int rc = launch_apply<kApplyBackwardQ>(p, sg, mQ, mG, a, st)) return rc;
    ApParams b = {};
    b.lengths = lengths;
    b.records = rec_r;
    b.out0 = (__nv_bfloat16*)dK;
    b.out1 = (__nv_bfloat16*)dV;
    b.early = 1;                // behind the dQ pass
    return launch_apply<kApplyBackwardKV>(p, sg, mK, mV, b, st);
}

}  // namespace tc
}  // namespace la

#ifdef LA_TC_TRACE
extern "C" int la_debug_read_trace_lin(long long* out, int n) {
    return (int)cudaMemcpyFromSymbol(out, la::tc::g_trace_lin, n * sizeof(long long));
}
#endif
