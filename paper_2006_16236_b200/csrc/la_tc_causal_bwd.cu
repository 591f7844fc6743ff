// Causal linear attention backward on the tensor cores (bf16, D = M = 64).
//
// Eq. 13-15 / Algorithm 1 "backward" on the ones-extended values, chunked.  With
// q = phi(Q_c), k = phi(K_c), dn_i = q_i . Z_i + eps, qh_i = q_i / dn_i,
// dl_i = -(G_i . O_i) (so that the extended upstream gradient of the numerator is
// [G_i, dl_i] / dn_i), L the lower-triangular mask, St = [S | Z] the forward running
// state and Rt = [R | r] the reverse running sum of qh_j [G_j | dl_j]^T:
//
//   forward sweep  (kernel "dq"):   h   = ((G V^T) o L) k + G S_{c-1}^T
//                                   gq  = (h - (q . h / dn) Z_i) / dn                 (Eq. 13)
//                                   dl  = -(q . h) / dn,   St_c = St_{c-1} + k^T [V | 1]
//   reverse sweep  (kernel "dkv"):  Ph  = (qh k^T) o L,   dP = (G V^T + dl 1^T) o L
//                                   gk  = dP^T qh + V R_{c+1}^T + 1 r_{c+1}^T         (Eq. 14)
//                                   gV  = Ph^T G + k R_{c+1}                          (Eq. 15)
//                                   Rt_c = Rt_{c+1} + qh^T [G | dl]
//   dQ = gq o phi'(Q),  dK = gk o phi'(K).
// G and V enter every product exactly as given (no re-rounding); the division by dn
// is carried by the query side, in fp32 or in the rounded qh.
//
// Every product runs on tcgen05 with fp32 accumulators in TMEM; the running states
// stay in TMEM in fp32 and are re-rounded to a bf16 operand tile once per chunk.  No
// per-position state is ever stored.  Sequences are cut into segments that run on
// different SMs; a segment starts from the sum of the pre-pass records of the parts before it
// (forward sweep) or after it (reverse sweep), which it adds up itself.
#include "la_tc.cuh"
#include "la_tc_common.cuh"

namespace la {
namespace tc {

using namespace sm100;

LA_TRACE_DECL(g_trace_dq)
LA_TRACE_DECL(g_trace_dkv)

namespace {

// ===========================================================================
// Forward sweep: dQ and delta.
//
// G_i . O_i is NOT taken from the stored (rounded) output.  With
//     h_i = sum_{j<=i} (G_i . V_j) k_j        (intra-chunk MMA plus G_i S_{c-1}^T)
// one has  G_i . O_i = (q_i . h_i) / dn_i  with  dn_i = q_i . Z_i + eps,  hence
//     gq_i = (h_i - (q_i . h_i / dn_i) Z_i) / dn_i :
// h_i projected so that q_i . gq_i = 0 (O is homogeneous of degree 0 in phi(Q_i)).
// Taking the projection from the same rounded products as h keeps that cancellation
// exact; a delta from the bf16 output loses several digits in the first rows, where
// the two terms nearly cancel.  The per-row prefix Z_i = Z_{c-1} + sum_{j<=i in chunk} k_j
// comes from one more MMA, T = L k with L the lower-triangular matrix of ones.  The
// kernel needs neither the forward output nor its denominators, and hands dn_i and
// dl_i = -(G_i . O_i) to the reverse sweep.
// In the first chunk of a sequence a row has few keys and h_i is a difference of nearly
// equal terms; there the scores are centred before rounding, dP_ij - m_i with
// m_i = dP_i0, and m_i T_i is added back in fp32 (a row constant times the prefix sum).
//
// Warps 0-7 ("score/epilogue" warps, two per TMEM quadrant: the pair shares the 128 rows
// of the quadrant, one warp per 32-column half): mask + round dP of chunk c+1, then the dQ
// epilogue of chunk c.  Warps 8-11: phi(K), phi(Q) in place and the state conversion.
// Warp 12: TMA.  Warps 13, 14, 15: MMA issue (13 also allocates TMEM).
// ===========================================================================
constexpr int kDqStages = 2;
constexpr int kDqThreads = 512;
constexpr uint32_t kDqColDP = 0;       // 128
constexpr uint32_t kDqColGt = 128;     // 2 x 64: h of even / odd chunks
constexpr uint32_t kDqColT = 256;      // 2 x 64: T = L k of even / odd chunks
constexpr uint32_t kDqColS = 384;      // 64 + 16

constexpr uint32_t kDqOffStage = 0;                                        // kDqStages x {K, V, G, Q}
constexpr uint32_t kDqOffDP = kDqOffStage + kDqStages * 4 * kTileBytes;    // 2 tiles
constexpr uint32_t kDqOffL = kDqOffDP + 2 * kTileBytes;                    // 2 tiles: lower-triangular ones
constexpr uint32_t kDqOffS = kDqOffL + 2 * kTileBytes;                     // bf16 S tile
constexpr uint32_t kDqOffOnes = kDqOffS + kDim * 128;
constexpr uint32_t kDqOffZ = kDqOffOnes + 2048;                            // fp32 [3][64]
constexpr uint32_t kDqOffX = kDqOffZ + 768;                                // fp32 [2 halves][128][2]: row-pair exchange
constexpr uint32_t kDqOffBar = kDqOffX + 2048;
constexpr uint32_t kDqOffOut = (kDqOffBar + 256 + 1023) & ~1023u;          // dQ tile on its way out
constexpr uint32_t kDqSmemBytes = kDqOffOut + kTileBytes + 1024;           // + slack for the 1 KB alignment of the base
static_assert(kDqSmemBytes <= 232448, "shared memory budget of one CTA");

struct DqBarriers {
    uint64_t full[kDqStages], empty[kDqStages], mapped[kDqStages];
    uint64_t dq_full[2], dq_drained[2], gst_full[2];
    uint64_t dp_full, dp_ready, s_full, state_ready;
    uint32_t tmem_base;
    int abort_flag;
};

struct DqParams {
    float* dn;                  // out: dn_i = q_i . Z_i + eps per row, for the reverse sweep
    float* dl;                  // out: dl_i = -(G_i . O_i) per row, for the reverse sweep
    const float* init;          // per (bh, part) [S|Z] records of the pre-pass, or null (single piece)
    const float* S_in;          // [BH, D, M] / [BH, D] state the sequence started from, or null (zero)
    const float* Z_in;
    CausalPlan plan;            // pieces of a sequence and their pre-pass parts
    int* status;
    int64_t N;
    float eps;
    int phi;
    int dim;                    // D = M: 64, or 32 (tiles zero-padded to 64 columns)
    int map;                    // apply the feature map on load (0: the inputs are already phi(Q), phi(K))
    const int* stamp;           // the plan the forward recorded in the saved buffer, or null (no saved buffer)
    const int* lengths;         // [B] real positions per batch element of a right-padded ragged batch (kVarlen only)
    int heads;
    __nv_bfloat16* dQ;          // for the rows of padding, which are zeroed with plain stores (kVarlen only)
};

// kVarlen: a right-padded ragged batch (see the forward kernel): chunks behind a sequence's end are skipped and
// their dQ rows zeroed, the padded rows of the chunk that holds the end are zeroed in shared memory.
template <bool kVarlen>
__global__ void __launch_bounds__(kDqThreads, 1)
causal_bwd_dq_kernel(const __grid_constant__ CUtensorMap mapK, const __grid_constant__ CUtensorMap mapV,
                     const __grid_constant__ CUtensorMap mapG, const __grid_constant__ CUtensorMap mapQ,
                     const __grid_constant__ CUtensorMap mapDQ, const DqParams prm) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    DqBarriers* bars = reinterpret_cast<DqBarriers*>(smem + kDqOffBar);
    float* sZ = reinterpret_cast<float*>(smem + kDqOffZ);
    float* sX = reinterpret_cast<float*>(smem + kDqOffX);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const CausalPlan& plan = prm.plan;
    const int64_t bh = blockIdx.x % plan.bh;                        // long pieces first: see CausalPlan
    const int piece = plan.piece_of_slot(blockIdx.x / plan.bh);
    const int c_begin = plan.piece_begin(piece);
    const int L_full = plan.piece_begin(piece + 1) - c_begin;
    RaggedSpan span{L_full, kChunk, false};
    if (kVarlen) span = ragged_span(prm.lengths, prm.heads, bh, prm.N, c_begin, L_full);
    const int L = span.chunks;                  // chunks this CTA processes
    const int tail_rows = span.tail_rows;       // real rows of the last of them
    const int64_t row0 = bh * prm.N + (int64_t)c_begin * kChunk;

    if (tid == 0) {
        for (int s = 0; s < kDqStages; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], 1 + 256);      // MMA commit + the epilogue warps (they read phi(Q) rows)
            mbar_init(&bars->mapped[s], 128);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&bars->dq_full[b], 1);
            mbar_init(&bars->dq_drained[b], 256);
            mbar_init(&bars->gst_full[b], 1);
        }
        mbar_init(&bars->dp_full, 1);
        mbar_init(&bars->dp_ready, 256);
        mbar_init(&bars->s_full, 1);
        mbar_init(&bars->state_ready, 128);
        bars->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 13) {
        __syncwarp();
        tmem_alloc(&bars->tmem_base, 512);
        tmem_relinquish();
    }
    // the score tile is zero right of the diagonal for ever: clear it once
    for (uint32_t i = tid; i < 2 * kTileBytes / 16; i += kDqThreads) sts128(smem + kDqOffDP + i * 16, 0u, 0u, 0u, 0u);
    for (int i = tid; i < 512; i += kDqThreads) reinterpret_cast<uint32_t*>(smem + kDqOffOnes)[i] = 0x3F803F80u;
    if (tid < 128) {        // L[i][j] = 1 for j <= i
        const uint32_t r7 = tid & 7;
        for (int cc = 0; cc < 16; ++cc) {
            uint32_t w[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int col = cc * 8 + 2 * j;
                w[j] = (col <= tid ? 0x3F80u : 0u) | (col + 1 <= tid ? 0x3F800000u : 0u);
            }
            sts128(smem + kDqOffL + (cc >> 3) * kTileBytes + tid * 128 + (((cc & 7) ^ r7) << 4), w[0], w[1], w[2], w[3]);
        }
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    // everything above is private to the CTA; from here on memory of the kernel before this one is touched
    // (wait first, then let the next kernel be scheduled: the reverse pre-pass fetches its first tiles before it
    // waits in turn, which is safe only if everything before this kernel is complete by then)
    grid_dependency_wait();
    allow_dependent_launch();
    const uint32_t tmem = bars->tmem_base;
    volatile int* abort_flag = &bars->abort_flag;
    bool mismatch = false;      // the saved buffer must come from a forward pass with this very plan
    if (prm.stamp) {
        int want[kPlanStampInts];
        plan_stamp(plan, prm.dim, want);
#pragma unroll
        for (int i = 0; i < kPlanStampInts; ++i) mismatch = mismatch || __ldg(prm.stamp + i) != want[i];
    }

    if (mismatch) {             // the same for every thread: nothing is started, the CTA leaves through the common exit
        if (tid == 0) atomicOr(prm.status, kStatusPlanMismatch);
    } else if (kVarlen && L == 0) {
        // this piece is all padding: nothing to sweep (its dQ rows are zeroed below)
    } else if (warp == 12) {
        // ------------------------------------------------------------ TMA producer
        // warp-wide loop, the elected lane issues (as in the MMA warps: the time from a stage's release to the
        // requests for its next tiles is part of the longest chain of this two-stage kernel)
        const bool leader = elect_one();
        const uint64_t pol_keep = l2_policy_evict_last(), pol_stream = l2_policy_evict_first();
        if (lane == 0) {
            prefetch_tensormap(&mapK); prefetch_tensormap(&mapV); prefetch_tensormap(&mapG); prefetch_tensormap(&mapQ);
            prefetch_tensormap(&mapDQ);
        }
        __syncwarp();
        #pragma unroll 1
        for (int c = 0; c < L; ++c) {
            const int s = c % kDqStages;
            if (c >= kDqStages && !mbar_wait_warp(&bars->empty[s], ((c / kDqStages) - 1) & 1, prm.status, kStatusPipeTimeout)) {
                *abort_flag = 1;
                break;
            }
            if (__any_sync(0xFFFFFFFFu, *abort_flag)) break;
            uint8_t* st = smem + kDqOffStage + s * 4 * kTileBytes;
            const int y = (c_begin + c) * kChunk, z = (int)bh;      // position in the sequence; sequence
            if (leader) LA_TRACE(g_trace_dq, c, 13);
            // the reverse sweep starts where this piece ends: its last chunks are asked to stay in L2, the rest,
            // which will be long gone by then, to leave first
            const uint64_t pol = c >= L_full - kKeepTailChunks ? pol_keep : pol_stream;
            mbar_arrive_expect_tx(leader, &bars->full[s], 4 * kTileBytes);
            tile_load<kVarlen>(leader, st + kTileBytes, &mapV, y, z, prm.N, &bars->full[s], pol);
            tile_load<kVarlen>(leader, st + 2 * kTileBytes, &mapG, y, z, prm.N, &bars->full[s], pol);
            tile_load<kVarlen>(leader, st, &mapK, y, z, prm.N, &bars->full[s], pol);
            tile_load<kVarlen>(leader, st + 3 * kTileBytes, &mapQ, y, z, prm.N, &bars->full[s], pol);
        }
    } else if (warp >= 13) {
        // ------------------------------------------------------------- MMA issuers
        // Three warps share the issue work, each running its loop with all lanes and issuing through an
        // elected one: addresses and descriptors then live in uniform registers (about 40 cycles per
        // tcgen05.mma; a loop under `if (lane == 0)` moves them there for every instruction and needs 100).
        // Warp 15: the score tile dP = G V^T of the next chunk, as soon as the score warps have taken the
        // previous one out of TMEM.  Warp 13: the product that consumes the rounded copy, h += dP k.  Warp 14:
        // everything that involves the running state (h = G S^T, St += k^T [V | 1]) and T = L k.  MMAs of one
        // thread execute in order; gst_full orders the two threads' writes to the h accumulator and tells
        // warp 13 that warp 14 is done with a stage; the score warps wait for dq_full(c) before they overwrite
        // the shared-memory score tile that h += dP k of chunk c reads.
        {
            const bool leader = elect_one();
            const uint32_t idesc_dp = umma_idesc_bf16(128, 128, 0, 0);
            const uint32_t idesc_kk = umma_idesc_bf16(128, 64, 0, 0);
            const uint32_t idesc_kmn = umma_idesc_bf16(128, 64, 0, 1);
            const uint32_t idesc_s = umma_idesc_bf16(64, 80, 1, 1);
            const uint32_t aS = sbase + kDqOffS, aOnes = sbase + kDqOffOnes, aL = sbase + kDqOffL,
                           aDP = sbase + kDqOffDP;
            const uint32_t hi = (uint32_t)(desc_k(0) >> 32);
            auto mk = [&](uint32_t lo) { return ((uint64_t)hi << 32) | lo; };
            auto lo_k = [&](uint32_t a) { return (uint32_t)desc_k(a); };
            auto lo_mn = [&](uint32_t a, uint32_t lbo) { return (uint32_t)desc_mn(a, lbo); };
            auto stage_k = [&](int c) { return sbase + kDqOffStage + (uint32_t)(c % kDqStages) * 4 * kTileBytes; };
            bool ok = true;
            if (warp == 15) {
                #pragma unroll 1
                for (int c = 0; c < L && ok; ++c) {     // dP = G V^T needs only the raw tiles
                    ok = mbar_wait_warp(&bars->full[c % kDqStages], (c / kDqStages) & 1, prm.status, kStatusTmaTimeout);
                    if (ok && c >= 1) ok = mbar_wait_warp(&bars->dp_ready, (c - 1) & 1, prm.status, kStatusPipeTimeout);
                    if (!ok || __any_sync(0xFFFFFFFFu, *abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t dV = lo_k(stage_k(c) + kTileBytes), dG = lo_k(stage_k(c) + 2 * kTileBytes);
#pragma unroll
                    for (int k = 0; k < 4; ++k) umma_bf16(leader, tmem + kDqColDP, mk(dG + 2 * k), mk(dV + 2 * k), idesc_dp, k > 0);
                    umma_commit(leader, &bars->dp_full);
                }
            } else if (warp == 13) {
                #pragma unroll 1
                for (int c = 0; c < L && ok; ++c) {
                    const int b = c & 1;
                    if (leader) LA_TRACE(g_trace_dq, c, 0);
                    ok = mbar_wait_warp(&bars->dp_ready, c & 1, prm.status, kStatusPipeTimeout) &&
                         mbar_wait_warp(&bars->gst_full[b], (c >> 1) & 1, prm.status, kStatusMmaTimeout);
                    if (!ok || __any_sync(0xFFFFFFFFu, *abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
                    if (leader) LA_TRACE(g_trace_dq, c, 3);
                    const uint32_t dDP = lo_k(aDP), dKmn = lo_mn(stage_k(c), kTileBytes);
#pragma unroll
                    for (int k = 0; k < 8; ++k)      // h += dP k
                        umma_bf16(leader, tmem + kDqColGt + b * 64, mk(dDP + (k >> 2) * (kTileBytes >> 4) + (k & 3) * 2), mk(dKmn + 128 * k),
                                  idesc_kmn, 1);
                    umma_commit(leader, &bars->dq_full[b]);
                    // gst_full(c) and dp_ready(c) were awaited: they cover the other threads' products on this stage
                    umma_commit(leader, &bars->empty[c % kDqStages]);
                    if (leader) LA_TRACE(g_trace_dq, c, 4);
                }
            } else {
                #pragma unroll 1
                for (int c = 0; c < L && ok; ++c) {
                    const int s = c % kDqStages, b = c & 1;
                    const uint32_t aK = stage_k(c), aV = aK + kTileBytes, aG = aV + kTileBytes;
                    const uint32_t dKmn = lo_mn(aK, kTileBytes), dV1 = lo_mn(aV, aOnes - aV), dG = lo_k(aG), dS = lo_k(aS), dL = lo_k(aL);
                    constexpr uint32_t kStepV1 = 128u - (128u << 16);
                    ok = mbar_wait_warp(&bars->mapped[s], (c / kDqStages) & 1, prm.status, kStatusPipeTimeout) &&
                         mbar_wait_warp(&bars->state_ready, c & 1, prm.status, kStatusPipeTimeout);
                    if (ok && c >= 2) ok = mbar_wait_warp(&bars->dq_drained[b], ((c >> 1) - 1) & 1, prm.status, kStatusPipeTimeout);
                    if (!ok || __any_sync(0xFFFFFFFFu, *abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
                    if (leader) LA_TRACE(g_trace_dq, c, 1);
#pragma unroll
                    for (int k = 0; k < 4; ++k)      // h = G S_{c-1}^T (before the state tile is rewritten)
                        umma_bf16(leader, tmem + kDqColGt + b * 64, mk(dG + 2 * k), mk(dS + 2 * k), idesc_kk, k > 0);
#pragma unroll
                    for (int k = 0; k < 8; ++k)      // [S | Z] += k^T [V | 1]: the ones region is the second 64-column block
                        umma_bf16(leader, tmem + kDqColS, mk(dKmn + 128 * k), mk(dV1 + kStepV1 * k), idesc_s, 1);
                    umma_commit(leader, &bars->s_full);
#pragma unroll
                    for (int k = 0; k < 8; ++k)      // T = L k  (row-wise prefix sums of k inside the chunk)
                        umma_bf16(leader, tmem + kDqColT + b * 64, mk(dL + (k >> 2) * (kTileBytes >> 4) + (k & 3) * 2), mk(dKmn + 128 * k),
                                  idesc_kmn, k > 0);
                    umma_commit(leader, &bars->gst_full[b]);
                    if (leader) LA_TRACE(g_trace_dq, c, 2);
                }
            }
            if (!ok) *abort_flag = 1;
        }
    } else if (warp >= 8) {
        // ---------------- operand warps: phi(K), phi(Q) in place, then the state conversion
        const int quad = warp - 8;
        const int t = tid - 8 * 32;
        const uint32_t r7 = t & 7;
        const float* rec = prm.init ? prm.init + bh * (int64_t)plan.nparts() * kStateFloats : nullptr;
        state_init(tmem + kDqColS, quad, lane, smem + kDqOffS, sZ + 2 * 64, rec, 0, rec ? plan.piece_first_part(piece) : 0,
                   prm.S_in ? prm.S_in + bh * (int64_t)(prm.dim * prm.dim) : nullptr,
                   prm.Z_in ? prm.Z_in + bh * prm.dim : nullptr, prm.dim);   // "chunk -1" -> Z buffer 2
        fence_proxy_async_smem();
        tc_fence_before_sync();
        mbar_arrive(&bars->state_ready);
        auto map_chunk = [&](int c) -> bool {
            const int s = c % kDqStages;
            if (!mbar_wait(&bars->full[s], (c / kDqStages) & 1, prm.status, kStatusTmaTimeout)) return false;
            if (t == 0) LA_TRACE(g_trace_dq, c, 5);
            if (prm.map) {
                uint8_t* rowK = smem + kDqOffStage + s * 4 * kTileBytes + t * 128;
                phi_row_inplace(rowK, r7, prm.dim >> 3);
                phi_row_inplace(rowK + 3 * kTileBytes, r7, prm.dim >> 3);
                fence_proxy_async_smem();
            }
            if (kVarlen && c == L - 1 && t >= tail_rows) {      // padding: no key feature, no value, no upstream gradient
                uint8_t* rowK = smem + kDqOffStage + s * 4 * kTileBytes + t * 128;
                zero_row(rowK);
                zero_row(rowK + kTileBytes);
                zero_row(rowK + 2 * kTileBytes);
                fence_proxy_async_smem();
            }
            mbar_arrive(&bars->mapped[s]);
            if (t == 0) LA_TRACE(g_trace_dq, c, 6);
            return true;
        };
        bool ok = map_chunk(0);
        #pragma unroll 1
        for (int c = 0; c < L && ok; ++c) {
            if (*abort_flag) { ok = false; break; }
            if (!mbar_wait(&bars->s_full, c & 1, prm.status, kStatusMmaTimeout)) { ok = false; break; }
            tc_fence_after_sync();
            if (t == 0) LA_TRACE(g_trace_dq, c, 7);
            // Z_c goes to buffer c % 3: the epilogue of chunk c still reads Z_{c-1}, and Z_{c-2}'s
            // readers are done (the MMA warp waited for that epilogue before issuing chunk c)
            state_to_smem(tmem + kDqColS, quad, lane, smem + kDqOffS, sZ + (c % 3) * 64, nullptr, nullptr);
            fence_proxy_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&bars->state_ready);
            if (t == 0) LA_TRACE(g_trace_dq, c, 8);
            // the state conversion first (the state chain waits for it), then the next chunk's operands
            // (which may still be in flight)
            if (c + 1 < L) ok = map_chunk(c + 1);
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
        uint8_t* tile_row = smem + kDqOffDP + t * 128;
        const uint32_t src = tmem + lane_base + kDqColDP;
        const bool elu = prm.phi == LA_PHI_ELU1;
        float m_prev = 0.f;                                 // centring offset of the chunk whose epilogue is pending

        bool scores_ok = true;
        auto process_scores = [&](int c) -> float {         // chunk c: TMEM dP -> masked bf16 tile
            float m = 0.f;
            if (c_begin + c == 0) {                          // first chunk of the sequence: centre on dP_i0
                m = __uint_as_float(tmem_ld1(src));
                tmem_ld_wait();
            }
            // the shared-memory tile is still the A operand of h += dP k of the chunk before, which another
            // thread issues: it must have completed before the tile is overwritten
            if (c >= 1 && !mbar_wait(&bars->dq_full[(c - 1) & 1], ((c - 1) >> 1) & 1, prm.status, kStatusMmaTimeout))
                scores_ok = false;
            if (has0) {
                uint32_t v[32];
                tmem_ld32(src + blk0 * 32, v);
                tmem_ld_wait();
                score_block_store(v, tile_row, r7, blk0, blk0 == quad, lane, -m);
            }
            if (has1) {
                uint32_t v[32];
                tmem_ld32(src + blk1 * 32, v);
                tmem_ld_wait();
                score_block_store(v, tile_row, r7, blk1, blk1 == quad, lane, -m);
            }
            fence_proxy_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&bars->dp_ready);
            return m;
        };

        // This thread's part of the phi(Q) row of a chunk (logical 16-byte chunks 4 half .. 4 half + 3) is taken
        // into registers at the end of the previous chunk's epilogue, ahead of its own, so that the stage goes
        // back to the TMA producer early.
        uint32_t qv[4][4];
        auto load_q = [&](int c) -> bool {
            const int s = c % kDqStages;
            if (!mbar_wait(&bars->mapped[s], (c / kDqStages) & 1, prm.status, kStatusPipeTimeout)) return false;
            const uint8_t* rowQ = smem + kDqOffStage + s * 4 * kTileBytes + 3 * kTileBytes + t * 128;
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) lds128(rowQ + (((half * 4 + cc) ^ r7) << 4), qv[cc]);
            mbar_arrive(&bars->empty[s]);
            return true;
        };
        bool ok = mbar_wait(&bars->dp_full, 0, prm.status, kStatusMmaTimeout) && !*abort_flag;
        if (ok) {
            tc_fence_after_sync();
            m_prev = process_scores(0);
            ok = load_q(0);
        }
        #pragma unroll 1
        for (int c = 0; c < L && ok; ++c) {
            const int b = c & 1;
            float m_next = 0.f;
            if (c + 1 < L) {            // scores of the next chunk first: its MMAs then overlap this chunk's epilogue
                if (!mbar_wait(&bars->dp_full, (c + 1) & 1, prm.status, kStatusMmaTimeout)) { ok = false; break; }
                tc_fence_after_sync();
                if (warp == 3 && lane == 0) LA_TRACE(g_trace_dq, c + 1, 11);
                m_next = process_scores(c + 1);
                if (!scores_ok) { ok = false; break; }
                if (warp == 3 && lane == 0) LA_TRACE(g_trace_dq, c + 1, 12);
            }
            // ---- epilogue of chunk c: this thread owns columns [32 half, 32 half + 32) of row t
            if (!mbar_wait(&bars->dq_full[b], (c >> 1) & 1, prm.status, kStatusMmaTimeout)) { ok = false; break; }
            if (*abort_flag) { ok = false; break; }
            tc_fence_after_sync();
            if (tid == 0) LA_TRACE(g_trace_dq, c, 9);
            const float* zprev = sZ + ((c + 2) % 3) * 64 + half * 32;           // Z_{c-1}
            uint32_t g[32], tt[32];
            tmem_ld32(tmem + lane_base + kDqColGt + b * 64 + half * 32, g);
            tmem_ld32(tmem + lane_base + kDqColT + b * 64 + half * 32, tt);
            tmem_ld_wait();
            tc_fence_before_sync();
            // (two columns per instruction from here on: the kernel is bound by instruction issue, and this
            // epilogue is a fifth of a chunk's instructions)
            const f32x2 m2 = pair(m_prev, m_prev);
            f32x2 h2[16], z2[16];
            f32x2 qg2[4] = {0, 0, 0, 0}, qz2[4] = {0, 0, 0, 0};
#pragma unroll
            for (int cc = 0; cc < 4; ++cc)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int e = cc * 8 + 2 * j, p2 = cc * 4 + j;
                    const f32x2 q2 = pair_bf16(qv[cc][j]);
                    const f32x2 t2 = pair(tt[e], tt[e + 1]);
                    h2[p2] = fma2(m2, t2, pair(g[e], g[e + 1]));
                    z2[p2] = add2(pair_ld(zprev + e), t2);
                    qg2[j] = fma2(q2, h2[p2], qg2[j]);
                    qz2[j] = fma2(q2, z2[p2], qz2[j]);
                }
            // both accumulators are in registers and Z_{c-1} has been consumed: the MMA warp may reuse
            // this accumulator pair, and the state warps the Z buffer (only after this arrival)
            mbar_arrive(&bars->dq_drained[b]);
            // combine the two halves of the row
            // the quadrant's previous dQ slab must have left the staging tile before it is rewritten below
            if (half == 0 && lane == 0) tma_store_wait_read<0>();
            float* xch = sX + (half * 128 + t) * 2;
            xch[0] = pair_sum(add2(add2(qg2[0], qg2[1]), add2(qg2[2], qg2[3])));
            xch[1] = pair_sum(add2(add2(qz2[0], qz2[1]), add2(qz2[2], qz2[3])));
            named_barrier(2 + quad, 64);
            const float* other = sX + ((half ^ 1) * 128 + t) * 2;
            const float qg = xch[0] + other[0], qz = xch[1] + other[1];
            named_barrier(2 + quad, 64);                    // the exchange slots may be rewritten after this
            const float dn = qz + prm.eps;
            const float inv = 1.f / dn;
            const float delta = -qg * inv;                  // = -(G_i . O_i)
            const int64_t row = row0 + (int64_t)c * kChunk + t;
            const bool pad = kVarlen && c == L - 1 && t >= tail_rows;     // a padded row of the chunk that holds the sequence's end
            if (half == 0 && !(pad && (int64_t)(c_begin + c) * kChunk + t >= prm.N)) {     // (a padded row may lie past the sequence's N)
                prm.dn[row] = pad ? 1.f : dn;
                prm.dl[row] = pad ? 0.f : delta;
            }
            // dQ leaves through a staging tile: each quadrant (two warps, 32 rows) fills its 4 KB slab and one
            // of its threads stores it with TMA: full 128-byte rows per request instead of 32 rows per store
            // instruction.  Columns beyond a 32-wide problem are padding: the store clips them.
            uint8_t* out_row = smem + kDqOffOut + t * 128;
            const f32x2 inv2 = pair(inv, inv), delta2 = pair(delta, delta);
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                uint32_t outp[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int p2 = cc * 4 + j;
                    f32x2 gq = mul2(inv2, fma2(delta2, z2[p2], h2[p2]));
                    // phi'(x) from phi(x): 1 where x > 0 (phi > 1), else phi(x), i.e. min(phi, 1)
                    if (elu) gq = mul2(gq, pair_bf16(min_bf16x2(qv[cc][j], 0x3F803F80u)));
                    outp[j] = pad ? 0u : pack_bf16x2(gq);
                }
                sts128(out_row + (((half * 4 + cc) ^ r7) << 4), outp[0], outp[1], outp[2], outp[3]);
            }
            fence_proxy_async_smem();
            named_barrier(2 + quad, 64);
            if (half == 0 && lane == 0) {
                const int y = (c_begin + c) * kChunk + quad * 32;       // rows past the sequence's N are clipped by the store
                if (!kVarlen || y < prm.N) tile_store<kVarlen>(&mapDQ, smem + kDqOffOut + quad * 32 * 128, y, (int)bh, prm.N);
                tma_store_commit();
            }
            if (tid == 0) LA_TRACE(g_trace_dq, c, 10);
            m_prev = m_next;
            if (c + 1 < L) ok = load_q(c + 1);
        }
        if (half == 0 && lane == 0) tma_store_wait_all<0>();
        if (!ok) *abort_flag = 1;
    }
    if (kVarlen && warp < 8 && !mismatch) {      // chunks of this piece behind the sequence's end: zero gradient
        const int t = (warp & 3) * 32 + lane, half = warp >> 2;
        #pragma unroll 1
        for (int c = L; c < L_full; ++c) {
            if (half * 32 < prm.dim && (int64_t)(c_begin + c) * kChunk + t < prm.N) {
                __nv_bfloat16* dst = prm.dQ + (row0 + (int64_t)c * kChunk + t) * prm.dim + half * 32;
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) stg128(dst + cc * 8, 0u, 0u, 0u, 0u);
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 13) {
        __syncwarp();
        tmem_dealloc(tmem, 512);
    }
}

// ===========================================================================
// Reverse sweep: dK, dV.  Chunks are visited from the last to the first.
// Warps 0-7: P and dP post-processing, 8-11: state conversion and dK/dV
// epilogue, 12-15: qh = phi(Q) / dn, phi(K), dl column, 16: TMA, 17-19: MMA.
// ===========================================================================
constexpr int kKvStages = 3;
constexpr int kKvThreads = 640;
constexpr uint32_t kKvColP = 0;        // 128: Ph^T (fp32, then bf16 pairs in place)
constexpr uint32_t kKvColDP = 128;     // 128: dP^T
constexpr uint32_t kKvColDk = 256;     // 64
constexpr uint32_t kKvColDv = 320;     // 64
constexpr uint32_t kKvColR = 384;      // 64 + 16

constexpr uint32_t kKvStageBytes = 4 * kTileBytes;                         // {Q, K, V, G}
constexpr uint32_t kKvOffStage = 0;
constexpr uint32_t kKvOffAux = kKvOffStage + kKvStages * kKvStageBytes;    // dl column tile: (hi, lo) in columns 0, 1
constexpr uint32_t kKvOffR = kKvOffAux + kTileBytes;                       // 2 bf16 R tiles (iteration i reads tile i & 1)
constexpr uint32_t kKvOffOnes = kKvOffR + 2 * kDim * 128;                  // 1 KB group: ones in columns 0, 1 (A operand)
constexpr uint32_t kKvOffRv = kKvOffOnes + 1024;                           // fp32 r[2][64]
constexpr uint32_t kKvOffBar = kKvOffRv + 512;
constexpr uint32_t kKvSmemBytes = kKvOffBar + 256;
static_assert(kKvSmemBytes <= 232448, "shared memory budget of one CTA");

struct KvBarriers {
    uint64_t full[kKvStages], empty[kKvStages], mapped[kKvStages];
    uint64_t p_full, dp_full, p_ready, dp_ready, r_full, state_ready, dkv_full, dv_full, dk_drained, dv_drained, kr_full, vr_full;
    uint32_t tmem_base;
    int abort_flag;
};

struct KvParams {
    const float* dn;            // dn_i from the forward sweep
    const float* dl;            // dl_i = -(G_i . O_i) from the forward sweep
    const float* init;          // per (bh, part) [R | r] records of the pre-pass, or null (single piece)
    const float* dS_out;        // [BH, D, M] / [BH, D] upstream gradient of the final state, or null (zero)
    const float* dZ_out;
    float* dS_in;               // [BH, D, M] / [BH, D] gradient of the state the sequence started from, or null
    float* dZ_in;
    CausalPlan plan;            // pieces of a sequence and their pre-pass parts
    int* status;
    int64_t N;
    float eps;
    int phi;
    int dim;
    int map;                    // apply the feature map on load (0: the inputs are already phi(Q), phi(K))
    const int* lengths;         // [B] real positions per batch element of a right-padded ragged batch (kVarlen only)
    int heads;
    __nv_bfloat16* dK;          // for the rows of padding, which are zeroed with plain stores (kVarlen only)
    __nv_bfloat16* dV;
};

// kVarlen: a right-padded ragged batch (see the forward kernel): the sweep starts at the sequence's last real
// chunk, whose padded rows are zeroed in shared memory; the dK, dV rows of the skipped chunks are zeroed.
template <bool kVarlen>
__global__ void __launch_bounds__(kKvThreads, 1)
causal_bwd_dkv_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                      const __grid_constant__ CUtensorMap mapV, const __grid_constant__ CUtensorMap mapG,
                      const __grid_constant__ CUtensorMap mapDK, const __grid_constant__ CUtensorMap mapDV,
                      const KvParams prm) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    KvBarriers* bars = reinterpret_cast<KvBarriers*>(smem + kKvOffBar);
    float* sRv = reinterpret_cast<float*>(smem + kKvOffRv);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const CausalPlan& plan = prm.plan;
    const int64_t bh = blockIdx.x % plan.bh;                        // long pieces first: see CausalPlan
    const int piece = plan.piece_of_slot(blockIdx.x / plan.bh);
    const int c_begin = plan.piece_begin(piece);
    const int L_full = plan.piece_begin(piece + 1) - c_begin;
    RaggedSpan span{L_full, kChunk, false};
    if (kVarlen) span = ragged_span(prm.lengths, prm.heads, bh, prm.N, c_begin, L_full);
    const int L = span.chunks;                  // chunks this CTA processes
    const int tail_rows = span.tail_rows;       // real rows of the first one it visits (the sequence's last)
    const int c_end = c_begin + L;
    const bool idle = kVarlen && L == 0;        // all padding: only the state gradient passes through (warps 8-11)
    // iteration i visits chunk c_end - 1 - i
    auto chunk_pos = [&](int i) { return (c_end - 1 - i) * kChunk; };               // position of its first row in the sequence
    auto chunk_row = [&](int i) { return bh * prm.N + (int64_t)chunk_pos(i); };     // the same as a row of the whole tensor

    LA_TRACE_CTA(g_trace_dkv, 0);
    if (sbase & 1023u) {            // the swizzled tiles need a 1 KB aligned base: report, touch nothing
        if (tid == 0) atomicOr(prm.status, kStatusPipeTimeout);
        return;
    }
    if (tid == 0) {
        for (int s = 0; s < kKvStages; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], 2 + 1);        // two MMA commits + the epilogue (its stores leave from the stage)
            mbar_init(&bars->mapped[s], 128);
        }
        mbar_init(&bars->p_full, 1);
        mbar_init(&bars->dp_full, 1);
        mbar_init(&bars->p_ready, 256);
        mbar_init(&bars->dp_ready, 256);
        mbar_init(&bars->r_full, 1);
        mbar_init(&bars->state_ready, 128);
        mbar_init(&bars->dkv_full, 1);
        mbar_init(&bars->dv_full, 1);
        mbar_init(&bars->dk_drained, 128);
        mbar_init(&bars->dv_drained, 128);
        mbar_init(&bars->kr_full, 1);
        mbar_init(&bars->vr_full, 1);
        bars->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 17) {
        __syncwarp();
        tmem_alloc(&bars->tmem_base, 512);
        tmem_relinquish();
    }
    // the dl column tile keeps zeros outside its first two columns; the ones group (8 rows, re-read for
    // every row group through a zero stride) has ones in columns 0 and 1: together they add dl_i to dP_ij
    for (uint32_t i = tid; i < kTileBytes / 16; i += kKvThreads) sts128(smem + kKvOffAux + i * 16, 0u, 0u, 0u, 0u);
    if (tid < 64) {
        const uint32_t row = tid >> 3, chunk = tid & 7;
        const uint32_t w0 = chunk == 0 ? 0x3F803F80u : 0u;
        sts128(smem + kKvOffOnes + row * 128 + ((chunk ^ row) << 4), w0, 0u, 0u, 0u);
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    // everything above is private to the CTA; from here on memory of the kernel before this one is touched.  The
    // kernel before this one (the reverse pre-pass) writes records only, and everything before IT is complete
    // when this kernel is scheduled (it waits before it lets its successor go): the TMA producer may request
    // the first tiles, which are inputs of the call, before it waits, so that they arrive while the pre-pass
    // is still draining.
    allow_dependent_launch();
    if (warp != 16) grid_dependency_wait();
    const uint32_t tmem = bars->tmem_base;
    volatile int* abort_flag = &bars->abort_flag;

    if (idle && (warp < 8 || warp >= 12)) {
        // nothing to sweep
    } else if (warp == 16) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tensormap(&mapQ); prefetch_tensormap(&mapK); prefetch_tensormap(&mapV); prefetch_tensormap(&mapG);
            prefetch_tensormap(&mapDK); prefetch_tensormap(&mapDV);
            const uint64_t pol_stream = l2_policy_evict_first();
            #pragma unroll 1
            for (int i = 0; i < L; ++i) {
                const int s = i % kKvStages;
                if (i >= kKvStages && !mbar_wait(&bars->empty[s], ((i / kKvStages) - 1) & 1, prm.status, kStatusPipeTimeout)) {
                    *abort_flag = 1;
                    break;
                }
                if (*abort_flag) break;
                if (i == kKvStages) grid_dependency_wait();     // (nothing this thread does depends on it: for symmetry)
                uint8_t* st = smem + kKvOffStage + s * kKvStageBytes;
                const int y = chunk_pos(i), z = (int)bh;
                mbar_arrive_expect_tx(&bars->full[s], kKvStageBytes);
                // read once, and nothing of it is wanted again: asked to leave L2 first, so that the tiles kept for the
                // pieces that start later are not pushed out by this stream
                tile_load<kVarlen>(true, st, &mapQ, y, z, prm.N, &bars->full[s], pol_stream);
                tile_load<kVarlen>(true, st + kTileBytes, &mapK, y, z, prm.N, &bars->full[s], pol_stream);
                tile_load<kVarlen>(true, st + 2 * kTileBytes, &mapV, y, z, prm.N, &bars->full[s], pol_stream);
                tile_load<kVarlen>(true, st + 3 * kTileBytes, &mapG, y, z, prm.N, &bars->full[s], pol_stream);
            }
        }
    } else if (warp >= 17) {
        // ------------------------------------------------------------- MMA issuers
        // Three warps share the issue work; each runs its loop with all 32 lanes and issues through an elected
        // lane (operands stay in uniform registers: about 40 cycles per tcgen05.mma instead of 100 to 140).  Warps 17 and 19: one score tile each and the product that
        // consumes it (transposed tiles, rows = keys: Ph^T = k qh^T, then gV += Ph^T G; dP^T = [V | 1] [G | dl]^T,
        // whose fifth K step is (ones in two columns) x (dl_i split into a bf16 high and low part), then
        // gk += dP^T qh; the rounded tiles are read from TMEM).  Warp 18: everything that involves the running
        // state ([R | r] += qh^T [G | dl]; gV = k R, gk = V R^T, which start the two accumulators).  MMAs of
        // one thread execute in order; kr_full / vr_full order two threads' writes to one accumulator.
        {
            const bool leader = elect_one();
            const uint32_t idesc_pp = umma_idesc_bf16(128, 128, 0, 0);
            const uint32_t idesc_kk = umma_idesc_bf16(128, 64, 0, 0);
            const uint32_t idesc_kmn = umma_idesc_bf16(128, 64, 0, 1);     // also: A from TMEM, B MN-major
            const uint32_t idesc_r = umma_idesc_bf16(64, 80, 1, 1);
            const uint32_t aAux = sbase + kKvOffAux, aOnes = sbase + kKvOffOnes;
            auto lo_k = [&](uint32_t a) { return (uint32_t)desc_k(a); };
            auto lo_mn = [&](uint32_t a, uint32_t lbo) { return (uint32_t)desc_mn(a, lbo); };
            auto stage_q = [&](int i) { return sbase + kKvOffStage + (uint32_t)(i % kKvStages) * kKvStageBytes; };
            bool ok = true;
            if (warp != 18) {
                // The two score tiles are two independent pipelines, each with its own issuing thread, so that
                // the score warps always have a tile to work on: Ph^T of chunk i+1 is issued as soon as the
                // rounded Ph^T of chunk i has been consumed, and likewise dP^T.  The next tile overwrites the
                // rounded copy only after the product that reads it (in-order execution within a thread).  Both
                // threads run this one loop on their own tile, accumulator, operands and barriers (one copy of
                // the code in the instruction cache).
                const bool dp = warp == 19;                                // the dP^T pipeline (else Ph^T)
                const uint32_t col = dp ? kKvColDP : kKvColP;              // score tile
                const uint32_t acc = dp ? kKvColDk : kKvColDv;             // what it is contracted into
                const uint32_t offA = (dp ? 2u : 1u) * kTileBytes;         // tile = A B^T: [V | 1] [G | dl]^T  or  k qh^T
                const uint32_t offB = (dp ? 3u : 0u) * kTileBytes;
                const uint32_t offC = (dp ? 0u : 3u) * kTileBytes;         // acc += tile x C: qh  or  G
                uint64_t* tile_full = dp ? &bars->dp_full : &bars->p_full;
                uint64_t* tile_ready = dp ? &bars->dp_ready : &bars->p_ready;
                uint64_t* acc_started = dp ? &bars->vr_full : &bars->kr_full;      // the state thread's first product
                uint64_t* acc_full = dp ? &bars->dkv_full : &bars->dv_full;
                auto issue_tile = [&](int i) {
                    umma_group4(leader, tmem + col, lo_k(stage_q(i) + offA), 2, lo_k(stage_q(i) + offB), 2, idesc_pp, 0);
                    if (dp) umma_bf16(leader, tmem + col, desc_ones(aOnes), desc_k(aAux), idesc_pp, 1);    // + dl_i (fifth K step)
                    umma_commit(leader, tile_full);
                };
                ok = mbar_wait_warp(&bars->mapped[0], 0, prm.status, kStatusPipeTimeout) && !__any_sync(0xFFFFFFFFu, *abort_flag);
                if (ok) {
                    tc_fence_after_sync();
                    issue_tile(0);
                }
                #pragma unroll 1
                for (int i = 0; i < L && ok; ++i) {
                    const uint32_t dC = lo_mn(stage_q(i) + offC, kTileBytes);
                    if (leader && !dp) LA_TRACE(g_trace_dkv, i, 0);
                    ok = mbar_wait_warp(tile_ready, i & 1, prm.status, kStatusPipeTimeout) &&
                         mbar_wait_warp(acc_started, i & 1, prm.status, kStatusMmaTimeout);
                    if (!ok || __any_sync(0xFFFFFFFFu, *abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
                    if (leader) LA_TRACE(g_trace_dkv, i, dp ? 3 : 1);
                    umma_group4_ta(leader, tmem + acc, tmem + col, dC, 128, idesc_kmn, 1);                 // gV += Ph^T G / gk += dP^T qh
                    umma_group4_ta(leader, tmem + acc, tmem + col + 64, dC + 512, 128, idesc_kmn, 1);
                    umma_commit(leader, acc_full);      // gV is complete first: its epilogue overlaps gk
                    // this thread's reads of the stage; the awaited vr_full(i) covers the state thread's products on it
                    umma_commit(leader, &bars->empty[i % kKvStages]);
                    if (i + 1 < L) {
                        // mapped(i+1) also says that the dl column tile holds chunk i+1
                        ok = mbar_wait_warp(&bars->mapped[(i + 1) % kKvStages], ((i + 1) / kKvStages) & 1, prm.status, kStatusPipeTimeout);
                        if (!ok) break;
                        tc_fence_after_sync();
                        issue_tile(i + 1);
                    }
                    if (leader) LA_TRACE(g_trace_dkv, i, dp ? 4 : 2);
                }
            } else {
                #pragma unroll 1
                for (int i = 0; i < L && ok; ++i) {
                    const uint32_t aQ = stage_q(i), aK = aQ + kTileBytes, aV = aK + kTileBytes, aG = aV + kTileBytes;
                    const uint32_t aR = sbase + kKvOffR + (i & 1) * kDim * 128;      // R_{c+1}: the state before this chunk
                    const uint32_t dQmn = lo_mn(aQ, kTileBytes), dG1 = lo_mn(aG, aAux - aG);
                    // gV = k R_{c+1} starts its accumulator as soon as the epilogue of the previous chunk has taken the
                    // old values out of TMEM (the score thread waits for it before gV += Ph^T G)
                    ok = mbar_wait_warp(&bars->mapped[i % kKvStages], (i / kKvStages) & 1, prm.status, kStatusPipeTimeout) &&
                         mbar_wait_warp(&bars->state_ready, i & 1, prm.status, kStatusPipeTimeout);
                    if (ok && i >= 1) ok = mbar_wait_warp(&bars->dv_drained, (i - 1) & 1, prm.status, kStatusPipeTimeout);
                    if (!ok || __any_sync(0xFFFFFFFFu, *abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
                    umma_group4(leader, tmem + kKvColDv, lo_k(aK), 2, lo_mn(aR, kTileBytes), 128, idesc_kmn, 0);
                    umma_commit(leader, &bars->kr_full);
                    // [R | r] += qh^T [G | dl], the dl column tile being the second 64-column block of B.  The
                    // previous state has been converted (state_ready), and dP^T of this chunk, which reads the same
                    // column tile, must be done (dp_full): the operand warps take r_full as the signal that the tile
                    // may be rewritten.
                    ok = mbar_wait_warp(&bars->dp_full, i & 1, prm.status, kStatusMmaTimeout);
                    if (!ok) break;
                    tc_fence_after_sync();
                    umma_group4(leader, tmem + kKvColR, dQmn, 128, dG1, 128, idesc_r, 1);
                    umma_group4(leader, tmem + kKvColR, dQmn + 512, 128, dG1 + 512, 128, idesc_r, 1);
                    umma_commit(leader, &bars->r_full);
                    // gk = V R_{c+1}^T likewise, once the previous gk has been taken out
                    if (i >= 1) ok = mbar_wait_warp(&bars->dk_drained, (i - 1) & 1, prm.status, kStatusPipeTimeout);
                    if (!ok) break;
                    tc_fence_after_sync();
                    umma_group4(leader, tmem + kKvColDk, lo_k(aV), 2, lo_k(aR), 2, idesc_kk, 0);
                    umma_commit(leader, &bars->vr_full);
                }
            }
            if (!ok) *abort_flag = 1;
        }
    } else if (warp >= 12) {
        // ---------------------- prep warps: qh = phi(Q) / dn, phi(K), dl column
        const int t = tid - 12 * 32;
        const uint32_t r7 = t & 7;
        const bool elu = prm.map != 0;
        #pragma unroll 1
        for (int i = 0; i < L; ++i) {
            const int s = i % kKvStages;
            const int64_t row = chunk_row(i) + t;
            const bool pad = kVarlen && i == 0 && t >= tail_rows;       // (a padded row may lie past the sequence's N)
            const float inv = pad ? 1.f : 1.f / __ldg(prm.dn + row);
            const float delta = pad ? 0.f : __ldg(prm.dl + row);
            if (!mbar_wait(&bars->full[s], (i / kKvStages) & 1, prm.status, kStatusTmaTimeout)) { *abort_flag = 1; break; }
            if (*abort_flag) break;
            if (t == 0) LA_TRACE(g_trace_dkv, i, 5);
            uint8_t* rowQ = smem + kKvOffStage + s * kKvStageBytes + t * 128;
            if (elu) map_row_inplace<true>(rowQ, r7, inv, prm.dim >> 3); else map_row_inplace<false>(rowQ, r7, inv, prm.dim >> 3);
            if (t == 0) LA_TRACE(g_trace_dkv, i, 13);
            if (elu) phi_row_inplace(rowQ + kTileBytes, r7, prm.dim >> 3);
            if (t == 0) LA_TRACE(g_trace_dkv, i, 14);
            // the single dl column tile is an operand of the previous chunk's dP^T and state MMAs
            if (i >= 1 && !mbar_wait(&bars->r_full, (i - 1) & 1, prm.status, kStatusMmaTimeout)) { *abort_flag = 1; break; }
            if (t == 0) LA_TRACE(g_trace_dkv, i, 15);
            // dl_i as a bf16 high and low part in columns 0 and 1 (the rest of the row stays zero)
            if (pad) {                                          // padding: the row takes no part in any product
                zero_row(rowQ);
                zero_row(rowQ + kTileBytes);
                zero_row(rowQ + 2 * kTileBytes);
                zero_row(rowQ + 3 * kTileBytes);
            }
            const float dl_hi = bf16_lo(pack_bf16x2(delta, 0.f));
            sts128(smem + kKvOffAux + t * 128 + ((0 ^ r7) << 4), pack_bf16x2(dl_hi, delta - dl_hi), 0u, 0u, 0u);
            fence_proxy_async_smem();
            mbar_arrive(&bars->mapped[s]);
            if (t == 0) LA_TRACE(g_trace_dkv, i, 6);
        }
    } else if (warp >= 8) {
        // ------------------------------ state conversion and dK / dV epilogue warps
        const int quad = warp - 8;
        const int t = quad * 32 + lane;
        const uint32_t r7 = t & 7;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        const float* rec = prm.init ? prm.init + bh * (int64_t)plan.nparts() * kStateFloats : nullptr;
        const uint32_t floor2 = prm.phi == LA_PHI_ELU1 ? 0u : 0x3F803F80u;     // slope >= 0 (elu + 1) or = 1 (identity), as a bf16 pair
        rstate_init(tmem + kKvColR, quad, lane, smem + kKvOffR, sRv + 64, rec, rec ? plan.piece_first_part(piece + 1) : 0,
                   rec ? plan.nparts() : 0);
        if (prm.dS_out || prm.dZ_out)       // upstream gradient of the final state: every piece's reverse sum starts from it
            state_add_given<false>(tmem + kKvColR, quad, lane, smem + kKvOffR, nullptr, sRv + 64,
                                   prm.dS_out ? prm.dS_out + bh * (int64_t)(prm.dim * prm.dim) : nullptr,
                                   prm.dZ_out ? prm.dZ_out + bh * prm.dim : nullptr, prm.dim);                                     // "iteration -1" -> buffer 1
        fence_proxy_async_smem();
        tc_fence_before_sync();
        named_barrier(1, 128);
        mbar_arrive(&bars->state_ready);

        #pragma unroll 1
        for (int i = 0; i < L; ++i) {
            const int s = i % kKvStages;
            if (!mbar_wait(&bars->mapped[s], (i / kKvStages) & 1, prm.status, kStatusPipeTimeout)) { *abort_flag = 1; break; }
            if (*abort_flag) break;
            const uint8_t* rowK = smem + kKvOffStage + s * kKvStageBytes + kTileBytes + t * 128;     // phi(K) row, for phi'

            if (!mbar_wait(&bars->r_full, i & 1, prm.status, kStatusMmaTimeout)) { *abort_flag = 1; break; }
            tc_fence_after_sync();
            if (t == 0) LA_TRACE(g_trace_dkv, i, 7);
            rstate_to_smem(tmem + kKvColR, quad, lane, smem + kKvOffR + ((i + 1) & 1) * kDim * 128, sRv + (i & 1) * 64);
            fence_proxy_async_smem();
            tc_fence_before_sync();
            mbar_arrive(&bars->state_ready);
            if (t == 0) LA_TRACE(g_trace_dkv, i, 8);

            if (!mbar_wait(&bars->dv_full, i & 1, prm.status, kStatusMmaTimeout)) { *abort_flag = 1; break; }
            tc_fence_after_sync();
            if (t == 0) LA_TRACE(g_trace_dkv, i, 9);
            const float* rprev = sRv + ((i + 1) & 1) * 64;               // r_{c+1}
            // The results leave through the stage: dV rows overwrite this chunk's G tile and dK rows its phi(K)
            // tile (every product that reads them is complete by then, and a thread reads its phi(K) row before
            // it writes there), and one thread stores each tile with TMA: full 128-byte rows per request instead
            // of 32 rows per store instruction.
            uint8_t* rowG = smem + kKvOffStage + s * kKvStageBytes + 3 * kTileBytes + t * 128;
            // gV first (plain rounding), so that the next chunk's k R can start early; then gk
            #pragma unroll 1
            for (int h = 0; h < 2; ++h) {
                uint32_t v[32];
                tmem_ld32(tmem + lane_base + kKvColDv + h * 32, v);
                tmem_ld_wait();
                if (h == 1) {
                    tc_fence_before_sync();
                    mbar_arrive(&bars->dv_drained);
                }
                if (h * 32 < prm.dim) {                   // columns beyond a 32-wide problem are padding
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc)
                        sts128(rowG + (((h * 4 + cc) ^ r7) << 4),
                               pack_bf16x2(__uint_as_float(v[cc * 8 + 0]), __uint_as_float(v[cc * 8 + 1])),
                               pack_bf16x2(__uint_as_float(v[cc * 8 + 2]), __uint_as_float(v[cc * 8 + 3])),
                               pack_bf16x2(__uint_as_float(v[cc * 8 + 4]), __uint_as_float(v[cc * 8 + 5])),
                               pack_bf16x2(__uint_as_float(v[cc * 8 + 6]), __uint_as_float(v[cc * 8 + 7])));
                }
            }
            fence_proxy_async_smem();
            named_barrier(1, 128);
            if (t == 0) {
                tile_store<kVarlen>(&mapDV, smem + kKvOffStage + s * kKvStageBytes + 3 * kTileBytes, chunk_pos(i), (int)bh, prm.N);
                tma_store_commit();
            }
            if (!mbar_wait(&bars->dkv_full, i & 1, prm.status, kStatusMmaTimeout)) { *abort_flag = 1; break; }
            tc_fence_after_sync();
            // gk + r_{c+1}, times phi'(K) = min(phi(K), 1) for elu + 1 (phi > 1 exactly where the slope is 1;
            // elsewhere the slope equals phi), times 1 for the identity map.  Rolled over the two halves:
            // the role loops of this kernel together have to fit the instruction cache.
            #pragma unroll 1
            for (int h = 0; h < 2; ++h) {
                uint32_t v[32];
                tmem_ld32(tmem + lane_base + kKvColDk + h * 32, v);
                tmem_ld_wait();
                if (h == 1) {
                    tc_fence_before_sync();
                    mbar_arrive(&bars->dk_drained);
                }
                if (h * 32 < prm.dim) {
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        uint32_t outp[4], kf[4];
                        lds128(rowK + (((h * 4 + cc) ^ r7) << 4), kf);
                        const float4 ra = *reinterpret_cast<const float4*>(rprev + h * 32 + cc * 8);
                        const float4 rb = *reinterpret_cast<const float4*>(rprev + h * 32 + cc * 8 + 4);
                        const float rr[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {       // two columns per instruction: issue-bound
                            const f32x2 g2 = add2(pair(v[cc * 8 + 2 * j], v[cc * 8 + 2 * j + 1]), pair(rr[2 * j], rr[2 * j + 1]));
                            const uint32_t slope = max_bf16x2(min_bf16x2(kf[j], 0x3F803F80u), floor2);
                            outp[j] = (kVarlen && i == 0 && t >= tail_rows) ? 0u : pack_bf16x2(mul2(g2, pair_bf16(slope)));
                        }
                        sts128(const_cast<uint8_t*>(rowK) + (((h * 4 + cc) ^ r7) << 4), outp[0], outp[1], outp[2], outp[3]);
                    }
                }
            }
            fence_proxy_async_smem();
            named_barrier(1, 128);          // all dK rows are in the tile; also orders the r double buffer
            if (t == 0) {
                tile_store<kVarlen>(&mapDK, smem + kKvOffStage + s * kKvStageBytes + kTileBytes, chunk_pos(i), (int)bh, prm.N);
                tma_store_commit();
                tma_store_wait_read<0>();           // both tiles have been read: the stage may be refilled
                mbar_arrive(&bars->empty[s]);
            }
            if (t == 0) LA_TRACE(g_trace_dkv, i, 10);
        }
        // after the first chunk of the sequence the reverse sum is the gradient of the state the sequence started
        // from (the last conversion above waited for its final update)
        if (piece == 0 && (prm.dS_in || prm.dZ_in))
            rstate_write(tmem + kKvColR, quad, lane, prm.dS_in ? prm.dS_in + bh * (int64_t)(prm.dim * prm.dim) : nullptr,
                         prm.dZ_in ? prm.dZ_in + bh * prm.dim : nullptr, prm.dim);
        if (t == 0) tma_store_wait_all<0>();
        if (kVarlen) {          // chunks of this piece behind the sequence's end: zero gradient
            #pragma unroll 1
            for (int c = c_end; c < c_begin + L_full; ++c) {
                const int64_t row = bh * prm.N + (int64_t)c * kChunk + t;
                if ((int64_t)c * kChunk + t >= prm.N) continue;             // past the sequence: not in memory
                for (int cc = 0; cc < prm.dim / 8; ++cc) {
                    stg128(prm.dK + row * prm.dim + cc * 8, 0u, 0u, 0u, 0u);
                    stg128(prm.dV + row * prm.dim + cc * 8, 0u, 0u, 0u, 0u);
                }
            }
        }
    } else {
        // ------------------------------------------- score warps: Ph^T and dP^T, masked and rounded in place
        const int quad = warp & 3, half = warp >> 2;
        const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
        #pragma unroll 1
        for (int i = 0; i < L; ++i) {
            if (warp == 3 && lane == 0) LA_TRACE(g_trace_dkv, i, 11);
            if (*abort_flag ||
                !round_score_tile<true>(tmem + lane_base + kKvColP, &bars->p_full, &bars->p_ready, i & 1, quad, half, lane, prm.status) ||
                !round_score_tile<true>(tmem + lane_base + kKvColDP, &bars->dp_full, &bars->dp_ready, i & 1, quad, half, lane, prm.status)) {
                *abort_flag = 1;
                break;
            }
            if (warp == 3 && lane == 0) LA_TRACE(g_trace_dkv, i, 12);
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    LA_TRACE_CTA(g_trace_dkv, 1);
    if (warp == 17) {
        __syncwarp();
        tmem_dealloc(tmem, 512);
    }
}

}  // namespace

size_t causal_backward_workspace(const la_problem& p) {
    const CausalPlan pl = choose_plan(p);
    const size_t bh = (size_t)(p.B * p.H);
    size_t bytes = 2 * bh * pl.nparts() * kStateFloats * sizeof(float);    // forward and reverse pre-pass records
    bytes += 2 * bh * (size_t)p.N * sizeof(float);                       // dn_i and dl_i per row
    return bytes;
}

int causal_backward(const la_problem& p, const void* Q, const void* K, const void* V, const int* lengths, const void* G,
                    const StateArgs& sa, const void* saved, void* dQ, void* dK, void* dV, void* ws, cudaStream_t st) {
    const CausalPlan pl = choose_plan(p);
    // With what the forward saved, phi(Q) and phi(K) are read as tensors (no feature map on load)
    // and the forward pre-pass records are the forward's own.
    const SavedLayout sl = saved_layout(p, pl);
    const uint8_t* sv = (const uint8_t*)saved;
    const bool premapped = sv != nullptr && p.phi == LA_PHI_ELU1;
    const bool map = !premapped && p.phi == LA_PHI_ELU1;
    if (premapped) {
        Q = sv + sl.phiq;
        K = sv + sl.phik;
    }
    const size_t bh = (size_t)(p.B * p.H);
    const uint64_t n = (uint64_t)p.N;
    const bool ragged = ragged_problem(p, lengths);

    // workspace carve-up (see causal_backward_workspace)
    uint8_t* w = (uint8_t*)ws;
    float* rec_s = (float*)w;            w += bh * pl.nparts() * kStateFloats * sizeof(float);
    float* rec_r = (float*)w;            w += bh * pl.nparts() * kStateFloats * sizeof(float);
    float* dn = (float*)w;               w += bh * (size_t)p.N * sizeof(float);
    float* dl = (float*)w;

    CUtensorMap mQ, mK, mV, mG;
    if (int rc = encode_attention_map(&mQ, Q, ragged, bh, n, kChunk, (int)p.D)) return rc;
    if (int rc = encode_attention_map(&mK, K, ragged, bh, n, kChunk, (int)p.D)) return rc;
    if (int rc = encode_attention_map(&mV, V, ragged, bh, n, kChunk, (int)p.D)) return rc;
    if (int rc = encode_attention_map(&mG, G, ragged, bh, n, kChunk, (int)p.D)) return rc;
    int* status = device_status_ptr();
    if (!status) return fail(LA_ERR_CUDA, "device status word unavailable");

    static std::atomic<uint64_t> attr_dq{0}, attr_dkv{0}, attr_dq_ragged{0}, attr_dkv_ragged{0};
    if (ragged) {
        if (int rc = opt_in_smem_once(causal_bwd_dq_kernel<true>, kDqSmemBytes, attr_dq_ragged)) return rc;
        if (int rc = opt_in_smem_once(causal_bwd_dkv_kernel<true>, kKvSmemBytes, attr_dkv_ragged)) return rc;
    } else {
        if (int rc = opt_in_smem_once(causal_bwd_dq_kernel<false>, kDqSmemBytes, attr_dq)) return rc;
        if (int rc = opt_in_smem_once(causal_bwd_dkv_kernel<false>, kKvSmemBytes, attr_dkv)) return rc;
    }
    const unsigned grid = (unsigned)(pl.npieces() * bh);

    // forward sweep: dQ, and dn_i, dl_i for the reverse sweep
    if (sv) rec_s = (float*)(sv + sl.records);
    else if (int rc = segment_states(p, pl, mK, mV, nullptr, nullptr, rec_s, /*reverse=*/false, map, st, lengths)) return rc;
    DqParams a;
    a.dn = dn;
    a.dl = dl;
    a.init = pl.npieces() > 1 ? rec_s : nullptr;
    a.S_in = sa.S_in;
    a.Z_in = sa.Z_in;
    a.plan = pl;
    a.status = status;
    a.N = p.N;
    a.eps = p.eps;
    a.phi = p.phi;
    a.dim = (int)p.D;
    a.map = map ? 1 : 0;
    a.stamp = sv ? (const int*)(sv + sl.stamp) : nullptr;
    a.lengths = lengths;
    a.heads = (int)p.H;
    a.dQ = (__nv_bfloat16*)dQ;
    prof_begin(kProfCausalBwdDq, st);
    CUtensorMap mDQ;
    if (int rc = encode_attention_map(&mDQ, dQ, ragged, bh, n, 32, (int)p.D)) return rc;      // one quadrant's rows per store
    cudaLaunchAttribute attr;
    const cudaLaunchConfig_t cfg_q = chained_launch(grid, kDqThreads, kDqSmemBytes, st, &attr);
    if (ragged) LA_CUDA_TRY(cudaLaunchKernelEx(&cfg_q, causal_bwd_dq_kernel<true>, mK, mV, mG, mQ, mDQ, a));
    else LA_CUDA_TRY(cudaLaunchKernelEx(&cfg_q, causal_bwd_dq_kernel<false>, mK, mV, mG, mQ, mDQ, a));
    note_launch();
    prof_end(kProfCausalBwdDq, st);

    // reverse sweep: dK, dV
    if (int rc = segment_states(p, pl, mQ, mG, dn, dl, rec_r, /*reverse=*/true, map, st, lengths)) return rc;
    KvParams b;
    b.dn = dn;
    b.dl = dl;
    b.init = pl.npieces() > 1 ? rec_r : nullptr;
    b.dS_out = sa.dS_out;
    b.dZ_out = sa.dZ_out;
    b.dS_in = sa.dS_in;
    b.dZ_in = sa.dZ_in;
    b.plan = pl;
    b.status = status;
    b.N = p.N;
    b.eps = p.eps;
    b.phi = p.phi;
    b.dim = (int)p.D;
    b.map = map ? 1 : 0;
    b.lengths = lengths;
    b.heads = (int)p.H;
    b.dK = (__nv_bfloat16*)dK;
    b.dV = (__nv_bfloat16*)dV;
    prof_begin(kProfCausalBwdDkv, st);
    CUtensorMap mDK, mDV;
    if (int rc = encode_attention_map(&mDK, dK, ragged, bh, n, kChunk, (int)p.D)) return rc;
    if (int rc = encode_attention_map(&mDV, dV, ragged, bh, n, kChunk, (int)p.D)) return rc;
    const cudaLaunchConfig_t cfg_kv = chained_launch(grid, kKvThreads, kKvSmemBytes, st, &attr);
    if (ragged) LA_CUDA_TRY(cudaLaunchKernelEx(&cfg_kv, causal_bwd_dkv_kernel<true>, mQ, mK, mV, mG, mDK, mDV, b));
    else LA_CUDA_TRY(cudaLaunchKernelEx(&cfg_kv, causal_bwd_dkv_kernel<false>, mQ, mK, mV, mG, mDK, mDV, b));
    note_launch();
    prof_end(kProfCausalBwdDkv, st);
    return LA_OK;
}

}  // namespace tc
}  // namespace la

#ifdef LA_TC_TRACE
extern "C" int la_debug_read_trace_dq(long long* out, int n) {
    return (int)cudaMemcpyFromSymbol(out, la::tc::g_trace_dq, n * sizeof(long long));
}
extern "C" int la_debug_read_trace_dkv(long long* out, int n) {
    return (int)cudaMemcpyFromSymbol(out, la::tc::g_trace_dkv, n * sizeof(long long));
}
#endif
