// Causal linear attention forward on the tensor cores (bf16, D = M = 64).
//
// Chunked form of Eq. 9-12.  For a chunk c of 128 positions, with q = phi(Q_c),
// k = phi(K_c), L the lower-triangular mask and St = [S | Z] the running state:
//     P    = (q k^T) o L                        tcgen05, 128x128x64, fp32 in TMEM
//     num  = P V_c + q S_{c-1}                  tcgen05, 128x64x(128+64)
//     den  = rowsum(P) + q . Z_{c-1}            CUDA cores, fp32
//     O_c  = num / (den + eps)
//     St_c = St_{c-1} + k^T [V_c | 1]           tcgen05, M=64, accumulated in TMEM (fp32)
// A sequence is cut into segments that run on different SMs; a segment starts from
// the exclusive prefix of the per-segment sums of k^T [V | 1], produced by a
// pre-pass over K and V and a scan.
//
// CTA = 10 warps: warps 0-3 post-process P and write O and the state (thread t owns
// chunk row t = TMEM lane t), warps 4-7 apply phi to the Q and K tiles in place,
// warp 8 issues TMA loads, warp 9 issues the MMAs and owns the TMEM allocation.
#include "la_tc.cuh"
#include "la_tc_common.cuh"

namespace la {
namespace tc {

using namespace sm100;

namespace {

constexpr int kStages = 3;
constexpr int kThreads = 320;
constexpr uint32_t kTmemCols = 512;
// TMEM columns
constexpr uint32_t kColP = 0;        // 2 x 128: P of even / odd chunks
constexpr uint32_t kColNum = 256;    // 2 x 64 : numerators of even / odd chunks
constexpr uint32_t kColS = 384;      // 64 + 16: state S (M=64 layout) and Z replicated in 16 columns

// shared memory map (bytes from a 1024-aligned base)
constexpr uint32_t kOffStage = 0;                                    // kStages x {Q, K, V}
constexpr uint32_t kOffP = kOffStage + kStages * 3 * kTileBytes;     // 2 tiles: P[:, 0:64], P[:, 64:128]
constexpr uint32_t kOffO = kOffP + 2 * kTileBytes;                   // output tile
constexpr uint32_t kOffS = kOffO + kTileBytes;                       // bf16 copy of S, [64][64]
constexpr uint32_t kOffOnes = kOffS + kDim * 128;                    // 8 rows of ones (1 KB)
constexpr uint32_t kOffZ = kOffOnes + 1024;                          // fp32 Z[64]
constexpr uint32_t kOffBar = kOffZ + 256;
constexpr uint32_t kSmemBytes = kOffBar + 256 + 1024;                // + alignment slack

struct Barriers {
    uint64_t full[kStages], empty[kStages], mapped[kStages];
    uint64_t p_full[2], o_full[2];
    uint64_t p_ready, state_ready, done;
    uint32_t tmem_base;
    int abort_flag;
};

struct FwdParams {
    float* den;            // [BH, N] or null
    const float* init;     // per (bh, seg) initial [S|Z] records, or null (zero start)
    float* S_out;          // [BH, 64, 64] or null
    float* Z_out;          // [BH, 64] or null
    int* status;
    int64_t N;
    int chunks;            // chunks per sequence
    int chunks_per_seg;
    int nseg;
    float eps;
    int phi;
    int dim;               // D = M: 64, or 32 (tiles zero-padded to 64 columns)
};

// ---------------------------------------------------------------------------
// Main kernel.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 1)
causal_fwd_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                  const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapO,
                  const FwdParams prm) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    Barriers* bars = reinterpret_cast<Barriers*>(smem + kOffBar);
    float* sZ = reinterpret_cast<float*>(smem + kOffZ);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int seg = blockIdx.x % prm.nseg;
    const int64_t bh = blockIdx.x / prm.nseg;
    const int c_begin = seg * prm.chunks_per_seg;
    const int c_end = min(prm.chunks, c_begin + prm.chunks_per_seg);
    const int L = c_end - c_begin;
    const int64_t row0 = bh * prm.N + (int64_t)c_begin * kChunk;      // first global row of this segment

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], 1);
            mbar_init(&bars->mapped[s], 128);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&bars->p_full[b], 1);
            mbar_init(&bars->o_full[b], 1);
        }
        mbar_init(&bars->p_ready, 128);
        mbar_init(&bars->state_ready, 128);
        mbar_init(&bars->done, 1);
        bars->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 9) {
        __syncwarp();
        tmem_alloc(&bars->tmem_base, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = bars->tmem_base;
    volatile int* abort_flag = &bars->abort_flag;

    if (warp == 8) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tensormap(&mapQ); prefetch_tensormap(&mapK); prefetch_tensormap(&mapV);
            for (int c = 0; c < L; ++c) {
                const int s = c % kStages;
                if (c >= kStages && !mbar_wait(&bars->empty[s], ((c / kStages) - 1) & 1, prm.status, kStatusPipeTimeout)) {
                    *abort_flag = 1;
                    break;
                }
                if (*abort_flag) break;
                uint8_t* st = smem + kOffStage + s * 3 * kTileBytes;
                const int y = (int)(row0 + (int64_t)c * kChunk);
                mbar_arrive_expect_tx(&bars->full[s], 3 * kTileBytes);
                tma_load_2d(st, &mapQ, 0, y, &bars->full[s]);
                tma_load_2d(st + kTileBytes, &mapK, 0, y, &bars->full[s]);
                tma_load_2d(st + 2 * kTileBytes, &mapV, 0, y, &bars->full[s]);
            }
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            const uint32_t idesc_p = umma_idesc_bf16(128, 128, 0, 0);
            const uint32_t idesc_num = umma_idesc_bf16(128, 64, 0, 1);
            const uint32_t idesc_s = umma_idesc_bf16(64, 64, 1, 1);
            const uint32_t idesc_z = umma_idesc_bf16(64, 16, 1, 1);
            const uint32_t aS = sbase + kOffS, aP = sbase + kOffP, aOnes = sbase + kOffOnes;
            bool ok = true;
            for (int c = 0; c < L && ok; ++c) {
                const int s = c % kStages, b = c & 1;
                const uint32_t aQ = sbase + kOffStage + s * 3 * kTileBytes, aK = aQ + kTileBytes, aV = aK + kTileBytes;
                ok = mbar_wait(&bars->mapped[s], (c / kStages) & 1, prm.status, kStatusPipeTimeout);
                if (!ok || *abort_flag) { ok = false; break; }
                tc_fence_after_sync();
                for (int k = 0; k < 4; ++k)      // P = q k^T
                    umma_bf16(tmem + kColP + b * 128, desc_k(aQ + k * 32), desc_k(aK + k * 32), idesc_p, k > 0);
                umma_commit(&bars->p_full[b]);
                ok = mbar_wait(&bars->state_ready, c & 1, prm.status, kStatusPipeTimeout);
                if (!ok) break;
                tc_fence_after_sync();
                for (int k = 0; k < 4; ++k)      // num = q S_{c-1}
                    umma_bf16(tmem + kColNum + b * 64, desc_k(aQ + k * 32), desc_mn(aS + k * 2048), idesc_num, k > 0);
                ok = mbar_wait(&bars->p_ready, c & 1, prm.status, kStatusPipeTimeout);
                if (!ok) break;
                tc_fence_after_sync();
                for (int k = 0; k < 8; ++k)      // num += P V
                    umma_bf16(tmem + kColNum + b * 64, desc_k(aP + (k >> 2) * kTileBytes + (k & 3) * 32),
                              desc_mn(aV + k * 2048), idesc_num, 1);
                for (int k = 0; k < 8; ++k)      // S += k^T V
                    umma_bf16(tmem + kColS, desc_mn(aK + k * 2048), desc_mn(aV + k * 2048), idesc_s, 1);
                for (int k = 0; k < 8; ++k)      // Z += k^T 1
                    umma_bf16(tmem + kColS + 64, desc_mn(aK + k * 2048), umma_desc_sw128(aOnes, 16, 0), idesc_z, 1);
                umma_commit(&bars->o_full[b]);
                umma_commit(&bars->empty[s]);
            }
            if (!ok) *abort_flag = 1;
            umma_commit(&bars->done);
            mbar_wait(&bars->done, 0, prm.status, kStatusMmaTimeout);
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------ feature-map warps
        const int t = tid - 128;                 // chunk row owned by this thread
        const uint32_t r7 = t & 7;
        for (int c = 0; c < L; ++c) {
            const int s = c % kStages;
            if (!mbar_wait(&bars->full[s], (c / kStages) & 1, prm.status, kStatusTmaTimeout)) { *abort_flag = 1; break; }
            if (*abort_flag) break;
            if (prm.phi == LA_PHI_ELU1) {
                uint8_t* rowQ = smem + kOffStage + s * 3 * kTileBytes + t * 128;
                phi_row_inplace(rowQ, r7, prm.dim >> 3);
                phi_row_inplace(rowQ + kTileBytes, r7, prm.dim >> 3);
                fence_proxy_async_smem();
            }
            mbar_arrive(&bars->mapped[s]);
        }
    } else {
        // ---------------------------------------- P / output / state warps (0-3)
        const int t = tid;                        // chunk row = TMEM lane
        const uint32_t r7 = t & 7;
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        const bool owns_state_row = lane < 16;    // M=64 accumulators use lanes 0-15 of each quadrant
        const int d_row = warp * 16 + lane;       // state row held by this thread (if owns_state_row)

        // ---- prologue: ones tile, initial state into TMEM / smem
        for (int i = tid; i < 256; i += 128) reinterpret_cast<uint32_t*>(smem + kOffOnes)[i] = 0x3F803F80u;
        {
            const float* init = prm.init ? prm.init + (bh * prm.nseg + seg) * (int64_t)kStateFloats : nullptr;
            state_init(tmem + kColS, warp, lane, smem + kOffS, sZ, init);
        }
        fence_proxy_async_smem();
        tc_fence_before_sync();
        named_barrier(1, 128);
        mbar_arrive(&bars->state_ready);

        for (int c = 0; c < L; ++c) {
            const int s = c % kStages, b = c & 1;
            const uint8_t* rowQ = smem + kOffStage + s * 3 * kTileBytes + t * 128;
            if (!mbar_wait(&bars->mapped[s], (c / kStages) & 1, prm.status, kStatusPipeTimeout) ||
                !mbar_wait(&bars->p_full[b], (c >> 1) & 1, prm.status, kStatusMmaTimeout)) { *abort_flag = 1; break; }
            if (*abort_flag) break;
            tc_fence_after_sync();

            // q . Z_{c-1} on the rounded features the MMA consumed
            float qz = 0.f;
            {
                uint32_t qv[8][4];
                load_row(rowQ, r7, qv);
                float part[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int cc = 0; cc < 8; ++cc)
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        part[j] = fmaf(bf16_lo(qv[cc][j]), sZ[cc * 8 + 2 * j], fmaf(bf16_hi(qv[cc][j]), sZ[cc * 8 + 2 * j + 1], part[j]));
                qz = (part[0] + part[1]) + (part[2] + part[3]);
            }

            // P: TMEM -> mask -> bf16 -> swizzled smem (K-major A operand of P V), row sums
            float rowsum = 0.f;
#pragma unroll
            for (int blk = 0; blk < 4; ++blk) {
                uint32_t packed[16];
                if (blk <= warp) {                       // warp-uniform: blocks right of the diagonal are zero
                    uint32_t v[32];
                    tmem_ld32(tmem + lane_base + kColP + b * 128 + blk * 32, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        float x0 = __uint_as_float(v[2 * j]), x1 = __uint_as_float(v[2 * j + 1]);
                        if (blk == warp) {
                            if (2 * j > lane) x0 = 0.f;
                            if (2 * j + 1 > lane) x1 = 0.f;
                        }
                        const uint32_t pk = pack_bf16x2(x0, x1);
                        rowsum += bf16_lo(pk) + bf16_hi(pk);
                        packed[j] = pk;
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j) packed[j] = 0u;
                }
                uint8_t* tile = smem + kOffP + (blk >> 1) * kTileBytes + t * 128;
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    const int chunk = (blk & 1) * 4 + cc;
                    sts128(tile + ((chunk ^ r7) << 4), packed[cc * 4], packed[cc * 4 + 1], packed[cc * 4 + 2],
                           packed[cc * 4 + 3]);
                }
            }
            fence_proxy_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&bars->p_ready);

            const float den = rowsum + qz;
            const float inv = 1.f / (den + prm.eps);
            if (prm.den) prm.den[row0 + (int64_t)c * kChunk + t] = den;

            if (!mbar_wait(&bars->o_full[b], (c >> 1) & 1, prm.status, kStatusMmaTimeout)) { *abort_flag = 1; break; }
            tc_fence_after_sync();

            // previous output tile must have left shared memory before it is overwritten
            if (tid == 0) tma_store_wait_read<0>();
            named_barrier(1, 128);

#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint32_t v[32];
                tmem_ld32(tmem + lane_base + kColNum + b * 64 + h * 32, v);
                tmem_ld_wait();
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    const int chunk = h * 4 + cc;
                    sts128(smem + kOffO + t * 128 + ((chunk ^ r7) << 4),
                           pack_bf16x2(__uint_as_float(v[cc * 8 + 0]) * inv, __uint_as_float(v[cc * 8 + 1]) * inv),
                           pack_bf16x2(__uint_as_float(v[cc * 8 + 2]) * inv, __uint_as_float(v[cc * 8 + 3]) * inv),
                           pack_bf16x2(__uint_as_float(v[cc * 8 + 4]) * inv, __uint_as_float(v[cc * 8 + 5]) * inv),
                           pack_bf16x2(__uint_as_float(v[cc * 8 + 6]) * inv, __uint_as_float(v[cc * 8 + 7]) * inv));
                }
            }

            // state S_c, Z_c: TMEM (fp32) -> bf16 B operand for the next chunk, fp32 Z for q.Z
            {
                const bool fin = (c == L - 1) && (seg == prm.nseg - 1);
                state_to_smem(tmem + kColS, warp, lane, smem + kOffS, sZ,
                              fin && prm.S_out ? prm.S_out + bh * (int64_t)(prm.dim * prm.dim) : nullptr,
                              fin && prm.Z_out ? prm.Z_out + bh * prm.dim : nullptr, prm.dim);
            }
            fence_proxy_async_smem();
            tc_fence_before_sync();
            named_barrier(1, 128);
            if (tid == 0) {
                tma_store_2d(&mapO, smem + kOffO, 0, (int)(row0 + (int64_t)c * kChunk));
                tma_store_commit();
            }
            mbar_arrive(&bars->state_ready);
        }
        if (tid == 0) tma_store_wait_all<0>();
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 9) {
        __syncwarp();
        tmem_dealloc(tmem, kTmemCols);
    }
}

}  // namespace

Segmentation choose_segments(const la_problem& p) {
    const int chunks = (int)(p.N / kChunk);
    const int64_t bh = p.B * p.H;
    int nseg = 1;
    if (const char* e = getenv("LA_TC_NSEG")) {
        nseg = atoi(e);
    } else if (bh < 120) {
        nseg = (int)((120 + bh - 1) / bh);
    }
    if (nseg > chunks / 2) nseg = chunks / 2;
    if (nseg < 1) nseg = 1;
    const int cps = (chunks + nseg - 1) / nseg;
    nseg = (chunks + cps - 1) / cps;
    return Segmentation{nseg, cps};
}

size_t causal_forward_workspace(const la_problem& p) {
    const Segmentation sg = choose_segments(p);
    if (sg.nseg <= 1) return 0;
    return (size_t)(p.B * p.H) * sg.nseg * kStateFloats * sizeof(float);
}

int causal_forward(const la_problem& p, const void* Q, const void* K, const void* V, void* O, float* den,
                   float* S_out, float* Z_out, void* ws, cudaStream_t st) {
    const Segmentation sg = choose_segments(p);
    const int chunks = (int)(p.N / kChunk);
    const uint64_t rows = (uint64_t)(p.B * p.H * p.N);
    CUtensorMap mQ, mK, mV, mO;
    if (int rc = encode_tile_map(&mQ, Q, rows, kChunk, (int)p.D)) return rc;
    if (int rc = encode_tile_map(&mK, K, rows, kChunk, (int)p.D)) return rc;
    if (int rc = encode_tile_map(&mV, V, rows, kChunk, (int)p.D)) return rc;
    if (int rc = encode_tile_map(&mO, O, rows, kChunk, (int)p.D)) return rc;
    int* status = device_status_ptr();
    if (!status) return fail(LA_ERR_CUDA, "device status word unavailable");

    static bool attr_done = false;
    if (!attr_done) {
        LA_CUDA_TRY(cudaFuncSetAttribute(causal_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes));
        attr_done = true;
    }
    float* records = (float*)ws;
    if (sg.nseg > 1) {
        if (int rc = segment_states(p, sg, mK, mV, nullptr, nullptr, records, /*reverse=*/false, st)) return rc;
    }
    FwdParams prm;
    prm.den = den;
    prm.init = sg.nseg > 1 ? records : nullptr;
    prm.S_out = S_out;
    prm.Z_out = Z_out;
    prm.status = status;
    prm.N = p.N;
    prm.chunks = chunks;
    prm.chunks_per_seg = sg.chunks_per_seg;
    prm.nseg = sg.nseg;
    prm.eps = p.eps;
    prm.phi = p.phi;
    prm.dim = (int)p.D;
    prof_begin(kProfCausalFwd, st);
    causal_fwd_kernel<<<(unsigned)(sg.nseg * p.B * p.H), kThreads, kSmemBytes, st>>>(mQ, mK, mV, mO, prm);
    LA_LAUNCHED();
    prof_end(kProfCausalFwd, st);
    return LA_OK;
}

}  // namespace tc
}  // namespace la
