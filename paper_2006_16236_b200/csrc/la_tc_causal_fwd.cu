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
// the sum of the pre-pass records of the parts before it (k^T [V | 1] per part).
//
// CTA = 18 warps.  Warps 0-7 ("score/epilogue" warps, two per TMEM quadrant: the pair
// shares the 32 rows of the quadrant, one warp per 32-column half of the outputs): mask and
// round P of chunk c+1, then the output epilogue of chunk c.  Warps 8-11: phi(K) in place and
// the state conversion.  Warps 12-15: phi(Q) in place.  Warp 16: TMA.  Warp 17: MMA issue and
// TMEM allocation.
#include "la_tc.cuh"
#include "la_tc_common.cuh"

namespace la {
namespace tc {

using namespace sm100;

LA_TRACE_DECL(g_trace_fwd)

namespace {

constexpr int kStages = 3;
constexpr int kThreads = 576;
constexpr uint32_t kTmemCols = 512;
// TMEM columns
constexpr uint32_t kColP = 0;        // 128
constexpr uint32_t kColNum = 128;    // 2 x 64 : numerators of even / odd chunks
constexpr uint32_t kColS = 256;      // 64 + 16: state S (M=64 layout) and Z replicated in 16 columns

// shared memory map (bytes from a 1024-aligned base)
constexpr uint32_t kOffStage = 0;                                    // kStages x {Q, K, V}
constexpr uint32_t kOffP = kOffStage + kStages * 3 * kTileBytes;     // 2 tiles: P[:, 0:64], P[:, 64:128]
constexpr uint32_t kOffS = kOffP + 2 * kTileBytes;                   // bf16 copy of S, [64][64]
constexpr uint32_t kOffOnes = kOffS + kDim * 128;                    // 8 rows of ones (1 KB)
constexpr uint32_t kOffZ = kOffOnes + 1024;                          // fp32 Z[3][64]
constexpr uint32_t kOffX = kOffZ + 768;                              // fp32 [2 halves][128][2]: row-pair exchange
constexpr uint32_t kOffBar = kOffX + 2048;
constexpr uint32_t kSmemBytes = kOffBar + 256 + 1024;                // + alignment slack

struct Barriers {
    uint64_t full[kStages], empty[kStages], mapped[kStages];
    uint64_t o_full[2], o_drained[2];
    uint64_t p_full, p_ready, s_full, state_ready;
    uint32_t tmem_base;
    int abort_flag;
};

struct FwdParams {
    __nv_bfloat16* O;
    float* den;            // [BH, N] or null
    const float* init;     // per (bh, part) [S|Z] records of the pre-pass, or null (single segment)
    int sub;               // parts per segment
    float* S_out;          // [BH, D, M] or null
    float* Z_out;          // [BH, D] or null
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
                  const __grid_constant__ CUtensorMap mapV, const FwdParams prm) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    Barriers* bars = reinterpret_cast<Barriers*>(smem + kOffBar);
    float* sZ = reinterpret_cast<float*>(smem + kOffZ);
    float* sX = reinterpret_cast<float*>(smem + kOffX);

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
            mbar_init(&bars->empty[s], 1 + 256);      // MMA commit + the epilogue warps (they read phi(Q) rows)
            mbar_init(&bars->mapped[s], 256);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&bars->o_full[b], 1);
            mbar_init(&bars->o_drained[b], 256);
        }
        mbar_init(&bars->p_full, 1);
        mbar_init(&bars->p_ready, 256);
        mbar_init(&bars->s_full, 1);
        mbar_init(&bars->state_ready, 128);
        bars->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 17) {
        __syncwarp();
        tmem_alloc(&bars->tmem_base, kTmemCols);
        tmem_relinquish();
    }
    // the score tile is zero right of the diagonal for ever: clear it once
    for (uint32_t i = tid; i < 2 * kTileBytes / 16; i += kThreads) sts128(smem + kOffP + i * 16, 0u, 0u, 0u, 0u);
    for (int i = tid; i < 256; i += kThreads) reinterpret_cast<uint32_t*>(smem + kOffOnes)[i] = 0x3F803F80u;
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = bars->tmem_base;
    volatile int* abort_flag = &bars->abort_flag;

    if (warp == 16) {
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
    } else if (warp == 17) {
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
                LA_TRACE(g_trace_fwd, c, 0);
                for (int k = 0; k < 4; ++k)      // P = q k^T (the P tile in TMEM is free: p_ready(c-1) was awaited)
                    umma_bf16(tmem + kColP, desc_k(aQ + k * 32), desc_k(aK + k * 32), idesc_p, k > 0);
                umma_commit(&bars->p_full);
                ok = mbar_wait(&bars->state_ready, c & 1, prm.status, kStatusPipeTimeout);
                if (ok && c >= 2) ok = mbar_wait(&bars->o_drained[b], ((c >> 1) - 1) & 1, prm.status, kStatusPipeTimeout);
                if (!ok) break;
                tc_fence_after_sync();
                LA_TRACE(g_trace_fwd, c, 1);
                for (int k = 0; k < 4; ++k)      // num = q S_{c-1}
                    umma_bf16(tmem + kColNum + b * 64, desc_k(aQ + k * 32), desc_mn(aS + k * 2048), idesc_num, k > 0);
                for (int k = 0; k < 8; ++k)      // S += k^T V
                    umma_bf16(tmem + kColS, desc_mn(aK + k * 2048), desc_mn(aV + k * 2048), idesc_s, 1);
                for (int k = 0; k < 8; ++k)      // Z += k^T 1
                    umma_bf16(tmem + kColS + 64, desc_mn(aK + k * 2048), desc_ones(aOnes), idesc_z, 1);
                umma_commit(&bars->s_full);
                LA_TRACE(g_trace_fwd, c, 2);
                ok = mbar_wait(&bars->p_ready, c & 1, prm.status, kStatusPipeTimeout);
                if (!ok) break;
                tc_fence_after_sync();
                LA_TRACE(g_trace_fwd, c, 3);
                for (int k = 0; k < 8; ++k)      // num += P V
                    umma_bf16(tmem + kColNum + b * 64, desc_k(aP + (k >> 2) * kTileBytes + (k & 3) * 32),
                              desc_mn(aV + k * 2048), idesc_num, 1);
                umma_commit(&bars->o_full[b]);
                umma_commit(&bars->empty[s]);
                LA_TRACE(g_trace_fwd, c, 4);
            }
            if (!ok) *abort_flag = 1;
        }
    } else if (warp >= 12) {
        // ------------------------------------------------ operand warps: phi(Q) in place
        const int t = tid - 12 * 32;
        const uint32_t r7 = t & 7;
        for (int c = 0; c < L; ++c) {
            const int s = c % kStages;
            if (!mbar_wait(&bars->full[s], (c / kStages) & 1, prm.status, kStatusTmaTimeout)) { *abort_flag = 1; break; }
            if (*abort_flag) break;
            if (prm.phi == LA_PHI_ELU1) {
                phi_row_inplace(smem + kOffStage + s * 3 * kTileBytes + t * 128, r7, prm.dim >> 3);
                fence_proxy_async_smem();
            }
            mbar_arrive(&bars->mapped[s]);
        }
    } else if (warp >= 8) {
        // ---------------- operand warps: phi(K) in place, then the state conversion
        const int quad = warp - 8;
        const int t = tid - 8 * 32;
        const uint32_t r7 = t & 7;
        const float* rec = prm.init ? prm.init + bh * (int64_t)(prm.nseg * prm.sub) * kStateFloats : nullptr;
        state_init(tmem + kColS, quad, lane, smem + kOffS, sZ + 2 * 64, rec, 0, rec ? seg * prm.sub : 0);   // "chunk -1"
        fence_proxy_async_smem();
        tc_fence_before_sync();
        mbar_arrive(&bars->state_ready);
        auto map_chunk = [&](int c) -> bool {
            const int s = c % kStages;
            if (!mbar_wait(&bars->full[s], (c / kStages) & 1, prm.status, kStatusTmaTimeout)) return false;
            if (t == 0) LA_TRACE(g_trace_fwd, c, 5);
            if (prm.phi == LA_PHI_ELU1) {
                phi_row_inplace(smem + kOffStage + s * 3 * kTileBytes + kTileBytes + t * 128, r7, prm.dim >> 3);
                fence_proxy_async_smem();
            }
            mbar_arrive(&bars->mapped[s]);
            if (t == 0) LA_TRACE(g_trace_fwd, c, 6);
            return true;
        };
        bool ok = map_chunk(0);
        for (int c = 0; c < L && ok; ++c) {
            if (c + 1 < L) ok = map_chunk(c + 1);
            if (!ok || *abort_flag) { ok = false; break; }
            if (!mbar_wait(&bars->s_full, c & 1, prm.status, kStatusMmaTimeout)) { ok = false; break; }
            tc_fence_after_sync();
            if (t == 0) LA_TRACE(g_trace_fwd, c, 7);
            // Z_c goes to buffer c % 3: the epilogue of chunk c still reads Z_{c-1}, and Z_{c-2}'s
            // readers are done (the MMA warp waited for that epilogue before issuing chunk c)
            const bool fin = (c == L - 1) && (seg == prm.nseg - 1);
            state_to_smem(tmem + kColS, quad, lane, smem + kOffS, sZ + (c % 3) * 64,
                          fin && prm.S_out ? prm.S_out + bh * (int64_t)(prm.dim * prm.dim) : nullptr,
                          fin && prm.Z_out ? prm.Z_out + bh * prm.dim : nullptr, prm.dim);
            fence_proxy_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&bars->state_ready);
            if (t == 0) LA_TRACE(g_trace_fwd, c, 8);
        }
        if (!ok) *abort_flag = 1;
    } else {
        // ------------------------------------------------ score / epilogue warps
        const int quad = warp & 3, half = warp >> 2;
        const int t = quad * 32 + lane;                     // chunk row = TMEM lane
        const uint32_t r7 = t & 7;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        // score blocks of this warp: half 0 -> {0, 2}, half 1 -> {1, 3}, restricted to blk <= quad
        const int blk0 = half, blk1 = half + 2;
        const bool has0 = blk0 <= quad, has1 = blk1 <= quad;
        uint8_t* tile_row = smem + kOffP + t * 128;
        const uint32_t src = tmem + lane_base + kColP;
        float rs_prev = 0.f;                                // this thread's part of rowsum(P) of the pending chunk

        auto score_block = [&](int blk) -> float {          // one 32-column block: mask, round, store, row sum
            uint32_t v[32];
            tmem_ld32(src + blk * 32, v);
            tmem_ld_wait();
            uint32_t packed[16];
            float rs = 0.f;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                float x0 = __uint_as_float(v[2 * j]), x1 = __uint_as_float(v[2 * j + 1]);
                if (blk == quad) {
                    if (2 * j > lane) x0 = 0.f;
                    if (2 * j + 1 > lane) x1 = 0.f;
                }
                const uint32_t pk = pack_bf16x2(x0, x1);
                rs += bf16_lo(pk) + bf16_hi(pk);            // the sum of what the MMA will see
                packed[j] = pk;
            }
            uint8_t* base = tile_row + (blk >> 1) * kTileBytes;
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                const uint32_t chunk = (blk & 1) * 4 + cc;
                sts128(base + ((chunk ^ r7) << 4), packed[cc * 4], packed[cc * 4 + 1], packed[cc * 4 + 2], packed[cc * 4 + 3]);
            }
            return rs;
        };
        auto process_scores = [&]() -> float {
            float rs = 0.f;
            if (has0) rs += score_block(blk0);
            if (has1) rs += score_block(blk1);
            fence_proxy_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&bars->p_ready);
            return rs;
        };

        bool ok = mbar_wait(&bars->p_full, 0, prm.status, kStatusMmaTimeout) && !*abort_flag;
        if (ok) {
            tc_fence_after_sync();
            rs_prev = process_scores();
        }
        for (int c = 0; c < L && ok; ++c) {
            const int s = c % kStages, b = c & 1;
            float rs_next = 0.f;
            if (c + 1 < L) {            // scores of the next chunk first: its MMAs then overlap this chunk's epilogue
                if (!mbar_wait(&bars->p_full, (c + 1) & 1, prm.status, kStatusMmaTimeout)) { ok = false; break; }
                tc_fence_after_sync();
                if (warp == 3 && lane == 0) LA_TRACE(g_trace_fwd, c + 1, 11);
                rs_next = process_scores();
                if (warp == 3 && lane == 0) LA_TRACE(g_trace_fwd, c + 1, 12);
            }
            // ---- epilogue of chunk c: this thread owns output columns [32 half, 32 half + 32) of row t
            if (!mbar_wait(&bars->mapped[s], (c / kStages) & 1, prm.status, kStatusPipeTimeout)) { ok = false; break; }
            float qz = 0.f;             // this half's part of q . Z_{c-1}, on the rounded features the MMA consumed
            {
                const uint8_t* rowQ = smem + kOffStage + s * 3 * kTileBytes + t * 128;
                const float* zprev = sZ + ((c + 2) % 3) * 64 + half * 32;
                float part[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    uint32_t qv[4];
                    lds128(rowQ + (((half * 4 + cc) ^ r7) << 4), qv);
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        part[j] = fmaf(bf16_lo(qv[j]), zprev[cc * 8 + 2 * j], fmaf(bf16_hi(qv[j]), zprev[cc * 8 + 2 * j + 1], part[j]));
                }
                qz = (part[0] + part[1]) + (part[2] + part[3]);
            }
            mbar_arrive(&bars->empty[s]);
            // combine the two halves of the row: den = rowsum(P) + q . Z
            float* xch = sX + (half * 128 + t) * 2;
            xch[0] = rs_prev + qz;
            named_barrier(2 + quad, 64);
            const float den = xch[0] + sX[((half ^ 1) * 128 + t) * 2];
            named_barrier(2 + quad, 64);                    // the exchange slots may be rewritten after this
            const float inv = 1.f / (den + prm.eps);
            const int64_t row = row0 + (int64_t)c * kChunk + t;
            if (half == 0 && prm.den) prm.den[row] = den;
            if (!mbar_wait(&bars->o_full[b], (c >> 1) & 1, prm.status, kStatusMmaTimeout)) { ok = false; break; }
            if (*abort_flag) { ok = false; break; }
            tc_fence_after_sync();
            if (tid == 0) LA_TRACE(g_trace_fwd, c, 9);
            uint32_t v[32];
            tmem_ld32(tmem + lane_base + kColNum + b * 64 + half * 32, v);
            tmem_ld_wait();
            tc_fence_before_sync();
            mbar_arrive(&bars->o_drained[b]);
            if (half * 32 < prm.dim) {                      // columns beyond a 32-wide problem are padding
                __nv_bfloat16* dst = prm.O + row * prm.dim + half * 32;
#pragma unroll
                for (int cc = 0; cc < 4; ++cc)
                    stg128(dst + cc * 8,
                           pack_bf16x2(__uint_as_float(v[cc * 8 + 0]) * inv, __uint_as_float(v[cc * 8 + 1]) * inv),
                           pack_bf16x2(__uint_as_float(v[cc * 8 + 2]) * inv, __uint_as_float(v[cc * 8 + 3]) * inv),
                           pack_bf16x2(__uint_as_float(v[cc * 8 + 4]) * inv, __uint_as_float(v[cc * 8 + 5]) * inv),
                           pack_bf16x2(__uint_as_float(v[cc * 8 + 6]) * inv, __uint_as_float(v[cc * 8 + 7]) * inv));
            }
            if (tid == 0) LA_TRACE(g_trace_fwd, c, 10);
            rs_prev = rs_next;
        }
        if (!ok) *abort_flag = 1;
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 17) {
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
    // pre-pass parts: about two CTAs per SM in total, each part a whole number of chunks that divides a segment
    int sub = 1;
    if (nseg > 1) {
        const int64_t want = (2 * 148 + bh * (nseg - 1) - 1) / (bh * (nseg - 1));
        for (int d = 1; d <= cps; ++d)
            if (cps % d == 0 && d <= want && cps / d >= 2) sub = d;
    }
    return Segmentation{nseg, cps, sub, cps / sub};
}

size_t causal_forward_workspace(const la_problem& p) {
    const Segmentation sg = choose_segments(p);
    if (sg.nseg <= 1) return 0;
    return (size_t)(p.B * p.H) * sg.parts() * kStateFloats * sizeof(float);
}

int causal_forward(const la_problem& p, const void* Q, const void* K, const void* V, void* O, float* den,
                   float* S_out, float* Z_out, void* ws, cudaStream_t st) {
    const Segmentation sg = choose_segments(p);
    const int chunks = (int)(p.N / kChunk);
    const uint64_t rows = (uint64_t)(p.B * p.H * p.N);
    CUtensorMap mQ, mK, mV;
    if (int rc = encode_tile_map(&mQ, Q, rows, kChunk, (int)p.D)) return rc;
    if (int rc = encode_tile_map(&mK, K, rows, kChunk, (int)p.D)) return rc;
    if (int rc = encode_tile_map(&mV, V, rows, kChunk, (int)p.D)) return rc;
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
    prm.O = (__nv_bfloat16*)O;
    prm.den = den;
    prm.init = sg.nseg > 1 ? records : nullptr;
    prm.S_out = S_out;
    prm.Z_out = Z_out;
    prm.status = status;
    prm.N = p.N;
    prm.chunks = chunks;
    prm.chunks_per_seg = sg.chunks_per_seg;
    prm.nseg = sg.nseg;
    prm.sub = sg.sub;
    prm.eps = p.eps;
    prm.phi = p.phi;
    prm.dim = (int)p.D;
    prof_begin(kProfCausalFwd, st);
    causal_fwd_kernel<<<(unsigned)(sg.nseg * p.B * p.H), kThreads, kSmemBytes, st>>>(mQ, mK, mV, prm);
    LA_LAUNCHED();
    prof_end(kProfCausalFwd, st);
    return LA_OK;
}

}  // namespace tc
}  // namespace la

#ifdef LA_TC_TRACE
extern "C" int la_debug_read_trace_fwd(long long* out, int n) {
    return (int)cudaMemcpyFromSymbol(out, la::tc::g_trace_fwd, n * sizeof(long long));
}
#endif
