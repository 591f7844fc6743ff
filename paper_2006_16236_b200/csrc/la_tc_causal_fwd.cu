// Causal linear attention forward on the tensor cores (bf16, D = M = 64 or 32).
//
// Chunked form of Eq. 9-12.  For a chunk c of 128 positions, with q = phi(Q_c),
// k = phi(K_c), L the lower-triangular mask and St = [S | Z] the running state:
//     P        = (q k^T) o L                       tcgen05 128x128x64, fp32 in TMEM; masked and
//                                                  rounded to bf16 in place (TMEM) by the score warps
//     [num|den] = P [V_c | 1] + q [S | Z]_{c-1}    tcgen05 128x80x(128+64); P is read from TMEM, the
//                                                  ones column makes den = rowsum(P) + q . Z
//     O_c      = num / (den + eps)
//     St_c     = St_{c-1} + k^T [V_c | 1]          tcgen05, M = 64, N = 80, accumulated in TMEM (fp32)
// A sequence is cut into segments that run on different SMs; a segment starts from
// the sum of the pre-pass records of the parts before it (k^T [V | 1] per part).
//
// Nothing in a chunk's score path depends on the previous chunk: the fp32 score tile is
// double-buffered in TMEM, so the MMA warp issues P of chunk c+1 before it waits for the
// rounded P of chunk c, and the score warps never wait for a round trip through the MMA warp.
// The only chain between chunks is the state (S update -> bf16 copy -> q S of the next chunk),
// which runs one chunk ahead of its use.
//
// CTA = 19 warps.  Warps 0-7 ("score/epilogue" warps, two per TMEM quadrant: the pair
// shares the 32 rows of the quadrant; one takes score columns 0-63 and output columns 0-31,
// the other 64-127 and 32-63): mask and round P of chunk c, then the output epilogue of chunk
// c-1.  Warps 8-11: phi(K) in place (two chunks ahead) and the state conversion.  Warps 12-15:
// phi(Q) in place.  Warp 16: TMA.  Warps 17, 18: MMA issue (17 also allocates TMEM).
#include "la_tc.cuh"
#include "la_tc_common.cuh"

namespace la {
namespace tc {

using namespace sm100;

LA_TRACE_DECL(g_trace_fwd)

namespace {

constexpr int kStages = 4;
constexpr int kThreads = 608;
constexpr uint32_t kTmemCols = 512;
// TMEM columns
constexpr uint32_t kColP = 0;        // 2 x 128: scores of even / odd chunks (fp32, then bf16 pairs in place)
constexpr uint32_t kColNum = 256;    // 2 x 80 : [numerator | denominator x 16] of even / odd chunks
constexpr uint32_t kColS = 416;      // 64 + 16: state S (M = 64 layout) and Z replicated in 16 columns
constexpr uint32_t kNumStride = 80;

// shared memory map (bytes from the 1024-aligned base of dynamic shared memory)
constexpr uint32_t kOffStage = 0;                                    // kStages x {Q, K, V}
constexpr uint32_t kStageBytes = 3 * kTileBytes;
constexpr uint32_t kOffS = kOffStage + kStages * kStageBytes;        // 2 x {bf16 S [64][64], bf16 Z tile}
constexpr uint32_t kStateTileBytes = 2 * kDim * 128;
constexpr uint32_t kOffOnes = kOffS + 2 * kStateTileBytes;           // 16 rows of ones (2 KB)
constexpr uint32_t kOffBar = kOffOnes + 2048;
constexpr uint32_t kSmemBytes = kOffBar + 256;
static_assert(kSmemBytes <= 232448, "shared memory budget of one CTA");

struct Barriers {
    uint64_t full[kStages], empty[kStages], mapped[kStages];
    uint64_t p_full[2], p_ready[2], o_full[2], o_drained[2], state_ready[2], qs_full[2];
    uint64_t s_full, s_drained;
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(Barriers) <= 256, "barrier block");

struct FwdParams {
    __nv_bfloat16* O;
    float* den;            // [BH, N] or null
    const float* init;     // per (bh, part) [S|Z] records of the pre-pass, or null (single piece)
    const float* S_in;     // [BH, D, M] state the sequence continues from, or null (zero)
    const float* Z_in;     // [BH, D]
    CausalPlan plan;       // pieces of a sequence and their pre-pass parts
    float* S_out;          // [BH, D, M] or null
    float* Z_out;          // [BH, D] or null
    int* status;
    int64_t N;
    float eps;
    int phi;
    int dim;               // D = M: 64, or 32 (tiles zero-padded to 64 columns)
    int save;              // store the mapped phi(Q), phi(K) tiles for the backward pass
    int* stamp;            // where the plan is recorded for the backward pass (in the saved buffer), or null
    const int* lengths;    // [B] real positions per batch element of a right-padded ragged batch (kVarlen only)
    int heads;
};

// ---------------------------------------------------------------------------
// Main kernel.
// ---------------------------------------------------------------------------
// kVarlen: a right-padded ragged batch (prm.lengths): chunks behind a sequence's end are skipped and their
// outputs zeroed, the padded rows of the chunk that holds the end are zeroed in shared memory.  The other
// instantiation carries none of that code.
template <bool kVarlen>
__global__ void __launch_bounds__(kThreads, 1)
causal_fwd_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                  const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapPQ,
                  const __grid_constant__ CUtensorMap mapPK, const FwdParams prm) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    Barriers* bars = reinterpret_cast<Barriers*>(smem + kOffBar);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const CausalPlan& plan = prm.plan;
    const int64_t bh = blockIdx.x % plan.bh;                        // long pieces first: see CausalPlan
    const int piece = plan.piece_of_slot(blockIdx.x / plan.bh);
    const bool last_piece = piece == plan.npieces() - 1;
    const int c_begin = plan.piece_begin(piece);
    const int L_full = plan.piece_begin(piece + 1) - c_begin;
    RaggedSpan span{L_full, kChunk, last_piece};
    if (kVarlen) span = ragged_span(prm.lengths, prm.heads, bh, prm.N, c_begin, L_full);
    const int L = span.chunks;                                        // chunks this CTA processes
    const int tail_rows = span.tail_rows;                             // real rows of the last of them
    const bool ends_here = span.has_end;                              // the final state is this CTA's to write
    const int64_t row0 = bh * prm.N + (int64_t)c_begin * kChunk;      // first global row of this segment

    LA_TRACE_CTA(g_trace_fwd, 0);
#ifdef LA_TC_TRACE
    if (threadIdx.x == 0) { uint32_t sm_; asm volatile("mov.u32 %0, %%smid;" : "=r"(sm_)); g_trace_fwd[(512 + (blockIdx.x & 1023)) * 32 + 2] = sm_; }
#endif
    if (sbase & 1023u) {            // the swizzled tiles need a 1 KB aligned base: report, touch nothing
        if (tid == 0) atomicOr(prm.status, kStatusPipeTimeout);
        return;
    }
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], prm.save ? 3 : 1);      // MMA commit (+ the two threads that store mapped tiles)
            mbar_init(&bars->mapped[s], 256);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&bars->p_full[b], 1);
            mbar_init(&bars->p_ready[b], 256);
            mbar_init(&bars->o_full[b], 1);
            mbar_init(&bars->o_drained[b], 256);
            mbar_init(&bars->state_ready[b], 256);
            mbar_init(&bars->qs_full[b], 1);
        }
        mbar_init(&bars->s_full, 1);
        mbar_init(&bars->s_drained, 256);
        bars->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 17) {
        __syncwarp();
        tmem_alloc(&bars->tmem_base, kTmemCols);
        tmem_relinquish();
    }
    for (int i = tid; i < 512; i += kThreads) reinterpret_cast<uint32_t*>(smem + kOffOnes)[i] = 0x3F803F80u;
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    // everything above is private to the CTA; from here on memory of the kernel before this one is touched
    // With a pre-pass of the same call before this kernel (it waits for everything before it, then lets this kernel
    // be scheduled, and writes records only) the TMA producer requests its first tiles, which are inputs of the
    // call, before it waits: they arrive while the pre-pass drains.  Without one this may be the first kernel of
    // the call, and everybody waits first.
    allow_dependent_launch();
    const bool early_loads = prm.init != nullptr && warp == 16;
    if (!early_loads) grid_dependency_wait();
    const uint32_t tmem = bars->tmem_base;
    volatile int* abort_flag = &bars->abort_flag;

    if (warp == 16) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            if (prm.stamp && blockIdx.x == 0) {
                grid_dependency_wait();         // a write to global memory: after the wait
                int st[kPlanStampInts];
                plan_stamp(plan, prm.dim, st);
#pragma unroll
                for (int i = 0; i < kPlanStampInts; ++i) prm.stamp[i] = st[i];
            }
            prefetch_tensormap(&mapQ); prefetch_tensormap(&mapK); prefetch_tensormap(&mapV);
            #pragma unroll 1
            for (int c = 0; c < L; ++c) {
                const int s = c % kStages;
                if (c >= kStages && !mbar_wait(&bars->empty[s], ((c / kStages) - 1) & 1, prm.status, kStatusPipeTimeout)) {
                    *abort_flag = 1;
                    break;
                }
                if (*abort_flag) break;
                if (early_loads && c == kStages) grid_dependency_wait();    // (nothing this thread does depends on it)
                uint8_t* st = smem + kOffStage + s * kStageBytes;
                const int y = (c_begin + c) * kChunk, z = (int)bh;      // position in the sequence; sequence
                mbar_arrive_expect_tx(&bars->full[s], kStageBytes);
                tile_load<kVarlen>(st, &mapQ, y, z, prm.N, &bars->full[s]);
                tile_load<kVarlen>(st + kTileBytes, &mapK, y, z, prm.N, &bars->full[s]);
                tile_load<kVarlen>(st + 2 * kTileBytes, &mapV, y, z, prm.N, &bars->full[s]);
            }
        }
    } else if (warp >= 17) {
        // ------------------------------------------------------------- MMA issuers
        // Two warps share the issue work (the waits of one stream of products would otherwise hold up the
        // other): warp 17 issues the score products P and P [V | 1], warp 18 the state update and
        // q [S | Z].  Each runs its loop with all 32 lanes and issues through an elected lane, which keeps
        // addresses and descriptors in uniform registers.  MMAs of one thread execute in order; the two
        // accumulations into the same numerator are ordered through qs_full.
        {
            const bool leader = elect_one();
            const uint32_t idesc_p = umma_idesc_bf16(128, 128, 0, 0);
            const uint32_t idesc_num = umma_idesc_bf16(128, 80, 0, 1);
            const uint32_t idesc_s = umma_idesc_bf16(64, 80, 1, 1);
            const uint32_t aOnes = sbase + kOffOnes;
            // Descriptors are (low word: start address and leading offset, high word: constant), so a
            // step along K is one 32-bit add on the low word: +2 (32 bytes, K-major) or +128 (2048
            // bytes, MN-major).  For B = [V | 1] the second 64-column block of every 16-row K group is
            // the ones region: its leading offset shrinks as the start address grows (+128 - (128 << 16)).
            const uint32_t hi = (uint32_t)(desc_k(0) >> 32);
            auto mk = [&](uint32_t lo) { return ((uint64_t)hi << 32) | lo; };
            auto lo_k = [&](uint32_t a) { return (uint32_t)desc_k(a); };
            auto lo_mn = [&](uint32_t a, uint32_t lbo) { return (uint32_t)desc_mn(a, lbo); };
            auto stage_addr = [&](int c) { return sbase + kOffStage + (uint32_t)(c % kStages) * kStageBytes; };
            constexpr uint32_t kStepV1 = 128u - (128u << 16);
            bool ok = true;
            if (warp == 17) {
                #pragma unroll 1
                for (int c = -1; c < L && ok; ++c) {        // step c: P of chunk c + 1, then P [V | 1] of chunk c
                    const int b = c & 1;
                    if (c + 1 < L) {
                        // the buffer's previous readers are done: p_ready(c-1) was awaited before
                        // P [V | 1] of chunk c-1 was issued, and this thread's MMAs run in order
                        ok = mbar_wait_warp(&bars->mapped[(c + 1) % kStages], ((c + 1) / kStages) & 1, prm.status, kStatusPipeTimeout);
                        if (!ok || __any_sync(0xFFFFFFFFu, *abort_flag)) { ok = false; break; }
                        tc_fence_after_sync();
                        const uint32_t nQ = lo_k(stage_addr(c + 1)), nK = lo_k(stage_addr(c + 1) + kTileBytes);
#pragma unroll 1
                        for (int k = 0; k < 4; ++k)
                            umma_bf16(leader, tmem + kColP + (b ^ 1) * 128, mk(nQ + 2 * k), mk(nK + 2 * k), idesc_p, k > 0);
                        umma_commit(leader, &bars->p_full[b ^ 1]);
                    }
                    if (c < 0) continue;
                    if (leader) LA_TRACE(g_trace_fwd, c, 2);
                    // += P [V | 1] with the rounded, masked P read from TMEM, on top of q [S | Z]
                    ok = mbar_wait_warp(&bars->p_ready[b], (c >> 1) & 1, prm.status, kStatusPipeTimeout) &&
                         mbar_wait_warp(&bars->qs_full[b], (c >> 1) & 1, prm.status, kStatusMmaTimeout);
                    if (!ok) break;
                    tc_fence_after_sync();
                    if (leader) LA_TRACE(g_trace_fwd, c, 3);
                    const uint32_t aV = stage_addr(c) + 2 * kTileBytes;
                    const uint32_t dV1 = lo_mn(aV, aOnes - aV);
#pragma unroll 1
                    for (int k = 0; k < 8; ++k)
                        umma_bf16_ta(leader, tmem + kColNum + b * kNumStride, tmem + kColP + b * 128 + (k >> 2) * 64 + (k & 3) * 8,
                                     mk(dV1 + kStepV1 * k), idesc_num, 1);
                    umma_commit(leader, &bars->o_full[b]);
                    // qs_full(c) was awaited: every MMA of either thread that reads this stage is covered
                    umma_commit(leader, &bars->empty[c % kStages]);
                    if (leader) LA_TRACE(g_trace_fwd, c, 4);
                }
            } else {
                #pragma unroll 1
                for (int c = 0; c < L && ok; ++c) {
                    const int s = c % kStages, b = c & 1;
                    const uint32_t aQ = stage_addr(c), aK = aQ + kTileBytes, aV = aK + kTileBytes;
                    const uint32_t dQ = lo_k(aQ), dKmn = lo_mn(aK, kTileBytes), dV1 = lo_mn(aV, aOnes - aV);
                    if (leader) LA_TRACE(g_trace_fwd, c, 0);
                    // St_c = St_{c-1} + k^T [V | 1]: the accumulator must have been read out (or initialised)
                    ok = mbar_wait_warp(&bars->mapped[s], (c / kStages) & 1, prm.status, kStatusPipeTimeout) &&
                         (c == 0 ? mbar_wait_warp(&bars->state_ready[1], 0, prm.status, kStatusPipeTimeout)
                                 : mbar_wait_warp(&bars->s_drained, (c - 1) & 1, prm.status, kStatusPipeTimeout));
                    if (!ok || __any_sync(0xFFFFFFFFu, *abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
#pragma unroll 1
                    for (int k = 0; k < 8; ++k)
                        umma_bf16(leader, tmem + kColS, mk(dKmn + 128 * k), mk(dV1 + kStepV1 * k), idesc_s, 1);
                    umma_commit(leader, &bars->s_full);
                    if (leader) LA_TRACE(g_trace_fwd, c, 1);
                    // [num | den] = q [S | Z]_{c-1}: tile (c-1) & 1 holds the state before this chunk
                    ok = mbar_wait_warp(&bars->state_ready[b ^ 1], (c >> 1) & 1, prm.status, kStatusPipeTimeout);
                    if (ok && c >= 2) ok = mbar_wait_warp(&bars->o_drained[b], ((c >> 1) - 1) & 1, prm.status, kStatusPipeTimeout);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t dS = lo_mn(sbase + kOffS + (b ^ 1) * kStateTileBytes, kDim * 128);
#pragma unroll 1
                    for (int k = 0; k < 4; ++k)
                        umma_bf16(leader, tmem + kColNum + b * kNumStride, mk(dQ + 2 * k), mk(dS + 128 * k), idesc_num, k > 0);
                    umma_commit(leader, &bars->qs_full[b]);
                }
            }
            if (!ok) *abort_flag = 1;
        }
    } else if (warp >= 12) {
        // ------- operand warps: phi(Q) in place, and the upper half (columns 32..63) of the state conversion
        const int quad = warp - 12;
        const int t = tid - 12 * 32;
        const uint32_t r7 = t & 7;
        mbar_arrive(&bars->state_ready[1]);         // the initial state is written by the other group alone
        auto map_chunk = [&](int c) -> bool {
            const int s = c % kStages;
            if (!mbar_wait(&bars->full[s], (c / kStages) & 1, prm.status, kStatusTmaTimeout)) return false;
            uint8_t* tile = smem + kOffStage + s * kStageBytes;
            if (prm.phi == LA_PHI_ELU1) {
                phi_row_inplace(tile + t * 128, r7, prm.dim >> 3);
                fence_proxy_async_smem();
            }
            if (kVarlen && c == L - 1 && t >= tail_rows) {      // padding: its values take no part in any product
                zero_row(tile + 2 * kTileBytes + t * 128);
                fence_proxy_async_smem();
            }
            if (prm.save) {         // the whole mapped tile goes out with one bulk store
                named_barrier(3, 128);
                if (t == 0) {
                    if (c > 0) {    // the previous chunk's store has long read its tile: release that stage
                        tma_store_wait_read<0>();
                        mbar_arrive(&bars->empty[(c - 1) % kStages]);
                    }
                    tile_store<kVarlen>(&mapPQ, tile, (c_begin + c) * kChunk, (int)bh, prm.N);
                    tma_store_commit();
                }
            }
            mbar_arrive(&bars->mapped[s]);
            return true;
        };
        bool ok = true;
        #pragma unroll 1
        for (int i = 0; i < L + 2 && ok; ++i) {         // step i: state conversion of chunk i - 2, then phi(Q) of chunk i
            const int c = i - 2;
            if (c >= 0) {
                if (*abort_flag) { ok = false; break; }
                if (!mbar_wait(&bars->s_full, c & 1, prm.status, kStatusMmaTimeout)) { ok = false; break; }
                tc_fence_after_sync();
                const bool fin = (c == L - 1) && ends_here;
                uint8_t* tile = smem + kOffS + (c & 1) * kStateTileBytes;
                state_half_to_tiles(tmem + kColS, quad, lane, 1, tile, nullptr, &bars->s_drained,
                                    fin && prm.S_out ? prm.S_out + bh * (int64_t)(prm.dim * prm.dim) : nullptr, nullptr, prm.dim);
                fence_proxy_async_smem();
                mbar_arrive(&bars->state_ready[c & 1]);
            }
            if (i < L) ok = map_chunk(i);
        }
        if (prm.save && t == 0) {
            tma_store_wait_all<0>();
            if (ok) mbar_arrive(&bars->empty[(L - 1) % kStages]);
        }
        if (!ok) *abort_flag = 1;
    } else if (warp >= 8) {
        // ---- operand warps: phi(K) in place (two chunks ahead), then the lower half (columns 0..31 and Z)
        // ---- of the state conversion
        const int quad = warp - 8;
        const int t = tid - 8 * 32;
        const uint32_t r7 = t & 7;
        const float* rec = prm.init ? prm.init + bh * (int64_t)plan.nparts() * kStateFloats : nullptr;
        uint8_t* tile1 = smem + kOffS + kStateTileBytes;            // the state before chunk 0 lives in tile 1
        state_init_tiles(tmem + kColS, quad, lane, tile1, tile1 + kDim * 128, rec, 0, rec ? plan.piece_first_part(piece) : 0);
        if (prm.S_in)           // the sequence continues from a given state: every piece starts from it
            state_add_given<true>(tmem + kColS, quad, lane, tile1, tile1 + kDim * 128, nullptr,
                                  prm.S_in + bh * (int64_t)(prm.dim * prm.dim), prm.Z_in + bh * prm.dim, prm.dim);
        fence_proxy_async_smem();
        tc_fence_before_sync();
        mbar_arrive(&bars->state_ready[1]);
        auto map_chunk = [&](int c) -> bool {
            const int s = c % kStages;
            if (!mbar_wait(&bars->full[s], (c / kStages) & 1, prm.status, kStatusTmaTimeout)) return false;
            if (t == 0) LA_TRACE(g_trace_fwd, c, 5);
            uint8_t* tile = smem + kOffStage + s * kStageBytes + kTileBytes;
            if (prm.phi == LA_PHI_ELU1) {
                phi_row_inplace(tile + t * 128, r7, prm.dim >> 3);
                fence_proxy_async_smem();
            }
            if (kVarlen && c == L - 1 && t >= tail_rows) {      // padding: no feature, so no score and no state update
                zero_row(tile + t * 128);
                fence_proxy_async_smem();
            }
            if (prm.save) {
                named_barrier(4, 128);
                if (t == 0) {
                    if (c > 0) {
                        tma_store_wait_read<0>();
                        mbar_arrive(&bars->empty[(c - 1) % kStages]);
                    }
                    tile_store<kVarlen>(&mapPK, tile, (c_begin + c) * kChunk, (int)bh, prm.N);
                    tma_store_commit();
                }
            }
            mbar_arrive(&bars->mapped[s]);
            if (t == 0) LA_TRACE(g_trace_fwd, c, 6);
            return true;
        };
        bool ok = true;
        #pragma unroll 1
        for (int i = 0; i < L + 2 && ok; ++i) {         // step i: state conversion of chunk i - 2, then phi(K) of chunk i
            const int c = i - 2;
            if (c >= 0) {
                if (*abort_flag) { ok = false; break; }
                if (!mbar_wait(&bars->s_full, c & 1, prm.status, kStatusMmaTimeout)) { ok = false; break; }
                tc_fence_after_sync();
                if (t == 0) LA_TRACE(g_trace_fwd, c, 7);
                const bool fin = (c == L - 1) && ends_here;
                uint8_t* tile = smem + kOffS + (c & 1) * kStateTileBytes;
                state_half_to_tiles(tmem + kColS, quad, lane, 0, tile, tile + kDim * 128, &bars->s_drained,
                                    fin && prm.S_out ? prm.S_out + bh * (int64_t)(prm.dim * prm.dim) : nullptr,
                                    fin && prm.Z_out ? prm.Z_out + bh * prm.dim : nullptr, prm.dim);
                fence_proxy_async_smem();
                mbar_arrive(&bars->state_ready[c & 1]);
                if (t == 0) LA_TRACE(g_trace_fwd, c, 8);
            }
            if (i < L) ok = map_chunk(i);
        }
        if (prm.save && t == 0) {
            tma_store_wait_all<0>();
            if (ok) mbar_arrive(&bars->empty[(L - 1) % kStages]);
        }
        if (!ok) *abort_flag = 1;
    } else {
        // ------------------------------------------------ score / epilogue warps
        const int quad = warp & 3, half = warp >> 2;
        const int t = quad * 32 + lane;                     // chunk row = TMEM lane
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        // this warp's score blocks (32 columns each): 2 half and 2 half + 1; blocks above the
        // diagonal block `quad` are zeros
        const int blkA = 2 * half, blkB = 2 * half + 1;
        const bool hasA = blkA <= quad, hasB = blkB <= quad;

        auto scores = [&](int c) {          // fp32 P of chunk c -> masked bf16 pairs, in place
            const int b = c & 1;
            const uint32_t pb = tmem + lane_base + kColP + b * 128;
            // bf16 block j of this warp goes to columns 64 half + 16 j .. + 15: inside the fp32
            // columns of block 2 half, which this thread has read before its first store, so nothing
            // another thread still needs is overwritten
            uint32_t v[32], pk[16];
            if (hasA) tmem_ld32(pb + blkA * 32, v);
            tmem_ld_wait();
            score_block_round<false>(v, hasA, blkA == quad, lane, pk);
            if (hasB) tmem_ld32(pb + blkB * 32, v);
            tmem_st16(pb + half * 64, pk);
            tmem_ld_wait();
            score_block_round<false>(v, hasB, blkB == quad, lane, pk);
            tmem_st16(pb + half * 64 + 16, pk);
            tmem_st_wait();
            tc_fence_before_sync();
            mbar_arrive(&bars->p_ready[b]);
        };
        auto epilogue = [&](int c) -> bool {    // output columns [32 half, 32 half + 32) of row t of chunk c
            const int b = c & 1;
            if (!mbar_wait(&bars->o_full[b], (c >> 1) & 1, prm.status, kStatusMmaTimeout)) return false;
            if (*abort_flag) return false;
            tc_fence_after_sync();
            if (tid == 0) LA_TRACE(g_trace_fwd, c, 9);
            const uint32_t nb = tmem + lane_base + kColNum + b * kNumStride;
            uint32_t v[32];
            tmem_ld32(nb + half * 32, v);
            const float den = __uint_as_float(tmem_ld1(nb + 64));
            tmem_ld_wait();
            tc_fence_before_sync();
            mbar_arrive(&bars->o_drained[b]);
            const float inv = 1.f / (den + prm.eps);
            const f32x2 inv2 = pair(inv, inv);
            const int64_t row = row0 + (int64_t)c * kChunk + t;
            if (kVarlen && c == L - 1 && t >= tail_rows) {  // a padded row of the chunk that holds the sequence's end
                if ((int64_t)(c_begin + c) * kChunk + t >= prm.N) return true;      // past the sequence: not in memory
                if (half == 0 && prm.den) prm.den[row] = 0.f;
                if (half * 32 < prm.dim) {
                    __nv_bfloat16* dst = prm.O + row * prm.dim + half * 32;
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) stg128(dst + cc * 8, 0u, 0u, 0u, 0u);
                }
                return true;
            }
            if (half == 0 && prm.den) prm.den[row] = den;
            if (half * 32 < prm.dim) {                      // columns beyond a 32-wide problem are padding
                __nv_bfloat16* dst = prm.O + row * prm.dim + half * 32;
#pragma unroll
                for (int cc = 0; cc < 4; ++cc)              // two columns per multiply
                    stg128(dst + cc * 8,
                           pack_bf16x2(mul2(pair(v[cc * 8 + 0], v[cc * 8 + 1]), inv2)),
                           pack_bf16x2(mul2(pair(v[cc * 8 + 2], v[cc * 8 + 3]), inv2)),
                           pack_bf16x2(mul2(pair(v[cc * 8 + 4], v[cc * 8 + 5]), inv2)),
                           pack_bf16x2(mul2(pair(v[cc * 8 + 6], v[cc * 8 + 7]), inv2)));
            }
            if (tid == 0) LA_TRACE(g_trace_fwd, c, 10);
            return true;
        };

        bool ok = true;
        #pragma unroll 1
        for (int c = 0; c <= L && ok; ++c) {            // step c: scores of chunk c, then the epilogue of chunk c - 1
            if (c < L) {
                if (!mbar_wait(&bars->p_full[c & 1], (c >> 1) & 1, prm.status, kStatusMmaTimeout) || *abort_flag) { ok = false; break; }
                tc_fence_after_sync();
                if (warp == 3 && lane == 0) LA_TRACE(g_trace_fwd, c, 11);
                scores(c);
                if (warp == 3 && lane == 0) LA_TRACE(g_trace_fwd, c, 12);
            }
            if (c >= 1) ok = epilogue(c - 1);
        }
        if (!ok) *abort_flag = 1;
        if (kVarlen) {          // chunks of this piece behind the sequence's end: zeros
            #pragma unroll 1
            for (int c = L; c < L_full; ++c) {
                const int64_t row = row0 + (int64_t)c * kChunk + t;
                if ((int64_t)(c_begin + c) * kChunk + t >= prm.N) continue;         // past the sequence: not in memory
                if (half == 0 && prm.den) prm.den[row] = 0.f;
                if (half * 32 < prm.dim) {
                    __nv_bfloat16* dst = prm.O + row * prm.dim + half * 32;
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) stg128(dst + cc * 8, 0u, 0u, 0u, 0u);
                }
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    LA_TRACE_CTA(g_trace_fwd, 1);
    if (warp == 17) {
        __syncwarp();
        tmem_dealloc(tmem, kTmemCols);
    }
}

}  // namespace

CausalPlan choose_plan(const la_problem& p) {
    const int kSms = sm_count();
    const PlanOverride ov = plan_override();        // A/B checks: a fixed number of equal pieces, a fixed short length
    CausalPlan pl;
    pl.chunks = chunks_of(p.N);
    pl.bh = (int)(p.B * p.H);
    pl.nlong = 1;
    pl.m = 0;
    pl.spos = 0;
    pl.sub = 1;
    const bool forced = ov.causal_pieces > 0;
    int nlong = forced ? ov.causal_pieces : (pl.bh < 120 ? kSms / pl.bh : 1);
    if (nlong > pl.chunks / 2) nlong = pl.chunks / 2;   // a piece is at least two chunks
    if (nlong < 1) nlong = 1;
    pl.nlong = nlong;
    // With B*H*nlong CTAs on 148 SMs, `rest` SMs would idle.  They take one short piece per sequence, several
    // in a row each (`rounds` at most): the short length m balances a long piece against `rounds` short ones,
    // each CTA costing about three chunk times to start up and drain (measured: records summed, pipeline
    // filled, last stores out).  The short piece sits in the middle of the sequence, so that the pre-passes (which skip
    // the last piece forward, the first one backward) skip a long one.
    const int rest = kSms - pl.bh * nlong;
    if (!forced && nlong >= 2 && rest >= 8) {
        const int rounds = (pl.bh + rest - 1) / rest;
        const double startup = 3.0;
        int m = (int)(((double)pl.chunks / nlong - (rounds - 1) * startup) / (rounds + 1.0 / nlong));
        if (ov.causal_short >= 0) m = ov.causal_short;
        if (m >= 4 && (pl.chunks - m) / nlong >= 2) {
            pl.m = m;
            pl.spos = nlong / 2;
        }
    }
    // pre-pass parts: about two CTAs per SM over the parts one pre-pass computes (all but one long piece)
    if (pl.npieces() > 1) {
        const int covered = nlong > 1 ? nlong - 1 : 1;
        int sub = (2 * kSms / pl.bh - pl.has_short()) / covered;
        const int shortest = (pl.chunks - pl.m) / nlong;
        if (sub > shortest / 2) sub = shortest / 2;
        if (sub < 1) sub = 1;
        pl.sub = sub;
    }
    return pl;
}

size_t causal_forward_workspace(const la_problem& p) {
    const CausalPlan pl = choose_plan(p);
    if (pl.npieces() <= 1) return 0;
    return (size_t)(p.B * p.H) * pl.nparts() * kStateFloats * sizeof(float);
}

size_t causal_saved_bytes(const la_problem& p) { return saved_layout(p, choose_plan(p)).bytes; }

int causal_forward(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths, const float* S_in,
                   const float* Z_in, void* O, float* den, float* S_out, float* Z_out, void* saved, void* ws,
                   cudaStream_t st) {
    const CausalPlan pl = choose_plan(p);
    const uint64_t seqs = (uint64_t)(p.B * p.H), n = (uint64_t)p.N;
    const bool ragged = ragged_problem(p, lengths);
    const SavedLayout sl = saved_layout(p, pl);
    uint8_t* sv = (uint8_t*)saved;
    const bool save = sv != nullptr && p.phi == LA_PHI_ELU1;     // with identity features Q, K are the mapped tensors
    CUtensorMap mQ, mK, mV, mPQ, mPK;
    if (int rc = encode_attention_map(&mQ, Q, ragged, seqs, n, kChunk, (int)p.D)) return rc;
    if (int rc = encode_attention_map(&mK, K, ragged, seqs, n, kChunk, (int)p.D)) return rc;
    if (int rc = encode_attention_map(&mV, V, ragged, seqs, n, kChunk, (int)p.D)) return rc;
    if (int rc = encode_attention_map(&mPQ, save ? sv + sl.phiq : Q, ragged, seqs, n, kChunk, (int)p.D)) return rc;
    if (int rc = encode_attention_map(&mPK, save ? sv + sl.phik : K, ragged, seqs, n, kChunk, (int)p.D)) return rc;
    int* status = device_status_ptr();
    if (!status) return fail(LA_ERR_CUDA, "device status word unavailable");

    static std::atomic<uint64_t> attr_done{0}, attr_done_ragged{0};
    if (int rc = ragged ? opt_in_smem_once(causal_fwd_kernel<true>, kSmemBytes, attr_done_ragged)
                         : opt_in_smem_once(causal_fwd_kernel<false>, kSmemBytes, attr_done)) return rc;
    // the pre-pass records go straight into the saved buffer when there is one
    float* records = sv ? (float*)(sv + sl.records) : (float*)ws;
    if (pl.npieces() > 1) {
        if (int rc = segment_states(p, pl, mK, mV, nullptr, nullptr, records, /*reverse=*/false, p.phi == LA_PHI_ELU1, st, lengths)) return rc;
    }
    if (lengths) {
        // the final state is written by the CTA that holds a sequence's last real chunk; a sequence without any
        // keeps the state it started from
        const size_t s_bytes = (size_t)(p.B * p.H * p.D * p.M) * sizeof(float), z_bytes = (size_t)(p.B * p.H * p.D) * sizeof(float);
        if (S_out) {
            if (S_in) LA_CUDA_TRY(cudaMemcpyAsync(S_out, S_in, s_bytes, cudaMemcpyDeviceToDevice, st));
            else LA_CUDA_TRY(cudaMemsetAsync(S_out, 0, s_bytes, st));
        }
        if (Z_out) {
            if (Z_in) LA_CUDA_TRY(cudaMemcpyAsync(Z_out, Z_in, z_bytes, cudaMemcpyDeviceToDevice, st));
            else LA_CUDA_TRY(cudaMemsetAsync(Z_out, 0, z_bytes, st));
        }
    }
    FwdParams prm;
    prm.O = (__nv_bfloat16*)O;
    prm.den = den;
    prm.init = pl.npieces() > 1 ? records : nullptr;
    prm.plan = pl;
    prm.S_in = S_in;
    prm.Z_in = Z_in;
    prm.S_out = S_out;
    prm.Z_out = Z_out;
    prm.status = status;
    prm.N = p.N;
    prm.eps = p.eps;
    prm.phi = p.phi;
    prm.dim = (int)p.D;
    prm.save = save ? 1 : 0;
    prm.stamp = sv ? (int*)(sv + sl.stamp) : nullptr;
    prm.lengths = lengths;
    prm.heads = (int)p.H;
    prof_begin(kProfCausalFwd, st);
    cudaLaunchAttribute attr;
    const cudaLaunchConfig_t cfg = chained_launch((unsigned)(pl.npieces() * pl.bh), kThreads, kSmemBytes, st, &attr);
    if (ragged) LA_CUDA_TRY(cudaLaunchKernelEx(&cfg, causal_fwd_kernel<true>, mQ, mK, mV, mPQ, mPK, prm));
    else LA_CUDA_TRY(cudaLaunchKernelEx(&cfg, causal_fwd_kernel<false>, mQ, mK, mV, mPQ, mPK, prm));
    note_launch();
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
