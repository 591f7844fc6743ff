// Segment pre-pass of the tensor-core causal kernels: per-segment sums of
//     phi(X_i) [Y_i | a_i]^T        (64 x 65 per segment, fp32)
// over parts of a sequence (a segment of the main kernels is one or several parts).
//   forward state  St: X = K, Y = V,            a_i = 1        (Eq. 10-11)
//   reverse state  Rt: X = Q (rows / dn_i), Y = G, a_i = dl_i  (the cumulative sum of Eq. 14-15)
// A segment of the main kernels starts from the sum of the records before it (forward sweep)
// or after it (reverse sweep): the state the sequential recurrence would have reached.  Warps 0-3: phi on X, scaling of Y and the final read-out; warp 4: TMA;
// warp 5: MMA (M = 64 accumulators in TMEM).
#include "la_tc.cuh"
#include "la_tc_common.cuh"

namespace la {
namespace tc {

using namespace sm100;

LA_TRACE_DECL(g_trace_seg)

namespace {

constexpr int kSumThreads = 192;
// Three stages of {X, Y} and one shared column tile (the ones, or the dl column of the chunk in
// flight): the loads have to run about two chunks ahead to cover the TMA latency, and two CTAs
// share an SM (2 x (112.25 KB + 1 KB reserved) fits the 228 KB of an SM).
constexpr int kSumStages = 3;
constexpr uint32_t kSumStageBytes = 2 * kTileBytes;                  // X, Y
constexpr uint32_t kSumOffAux = kSumStages * kSumStageBytes;         // [128][64] column tile: B operand block [64, 80)
constexpr uint32_t kSumOffBar = kSumOffAux + kTileBytes;
constexpr uint32_t kSumSmemBytes = kSumOffBar + 256;
static_assert(2 * (kSumSmemBytes + 1024) <= 233472, "two CTAs per SM");

struct SumBarriers {
    uint64_t full[kSumStages], empty[kSumStages], mapped[kSumStages];
    uint64_t done;
    uint32_t tmem_base;
    int abort_flag;
};

struct SumParams {
    float* records;        // [BH][parts][kStateFloats]
    const float* dn;       // null: phi(X) is used as is and a_i = 1; else phi(X_i) is divided by dn_i
    const float* dl;       // with dn: a_i = dl_i
    int* status;
    int64_t N;
    CausalPlan plan;
    int first_part;        // parts first_part .. first_part + parts_per_seq - 1 of every sequence are summed
    int parts_per_seq;
    float eps;
    int map;               // apply the feature map to X on load
    int dim;
    const int* lengths;    // [B] real positions per batch element of a right-padded ragged batch (kVarlen only)
    int heads;
};

// kVarlen: a right-padded ragged batch: only the chunks of the part that hold real positions are summed, the
// padded rows of the chunk that holds a sequence's end are zeroed, a part that is all padding gives a zero record.
template <bool kVarlen>
__global__ void __launch_bounds__(kSumThreads, 2)
segment_sum_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapY,
                   const SumParams prm) {
    extern __shared__ __align__(1024) uint8_t smem[];
    const uint32_t sbase = smem_u32(smem);
    SumBarriers* bars = reinterpret_cast<SumBarriers*>(smem + kSumOffBar);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    LA_TRACE_CTA(g_trace_seg, 0);
    const int seg = prm.first_part + blockIdx.x % prm.parts_per_seq;       // index of this part
    const int64_t bh = blockIdx.x / prm.parts_per_seq;
    const int c_begin = prm.plan.part_begin(seg);
    const int L_full = prm.plan.part_begin(seg + 1) - c_begin;
    RaggedSpan span{L_full, kChunk, false};
    if (kVarlen) span = ragged_span(prm.lengths, prm.heads, bh, prm.N, c_begin, L_full);
    const int L = span.chunks;
    const int64_t row0 = bh * prm.N + (int64_t)c_begin * kChunk;
    const bool scaled = prm.dn != nullptr;

    if (sbase & 1023u) {            // the swizzled tiles need a 1 KB aligned base: report, touch nothing
        if (tid == 0) atomicOr(prm.status, kStatusPipeTimeout);
        return;
    }
    if (tid == 0) {
        for (int s = 0; s < kSumStages; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], 1);
            mbar_init(&bars->mapped[s], 128);
        }
        mbar_init(&bars->done, 1);
        bars->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 5) {
        __syncwarp();
        tmem_alloc(&bars->tmem_base, 128);
        tmem_relinquish();
    }
    // the column tile: ones (a_i = 1) unless the mapping threads write dl there chunk by chunk
    for (int i = tid; i < kTileBytes / 4; i += kSumThreads)
        reinterpret_cast<uint32_t*>(smem + kSumOffAux)[i] = scaled ? 0u : 0x3F803F80u;
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    // everything above is private to the CTA; from here on memory of the kernel before this one is touched
    // wait first, then let the next kernel be scheduled: a kernel that follows this one may then fetch its own
    // inputs before it waits in turn, knowing that everything before this kernel is complete
    // The reverse pre-pass follows the dQ sweep of the same call and reads, as tiles, only inputs of that call and
    // the saved tiles of an earlier one: its TMA producer requests the first tiles before it waits (they arrive
    // while the sweep before it drains); the per-row scalars of that sweep are read by the other warps, after
    // their wait.  (The forward pre-pass may be the first kernel of a call: everybody waits first.)
    const bool early_loads = scaled && warp == 4;
    if (!early_loads) {
        grid_dependency_wait();
        allow_dependent_launch();
    }
    LA_TRACE_CTA(g_trace_seg, 2);
    const uint32_t tmem = bars->tmem_base;
    volatile int* abort_flag = &bars->abort_flag;

    if (warp == 4) {
        if (lane == 0) {
            prefetch_tensormap(&mapX); prefetch_tensormap(&mapY);
            // a pre-pass reads what a sweep reads next: the tiles that sweep starts with (the end of every piece for the
            // reverse sweep, the beginning for a forward sweep) are asked to stay in L2, everything else, read once
            // here, to leave first
            const uint64_t pol_stream = l2_policy_evict_first(), pol_keep = l2_policy_evict_last();
            #pragma unroll 1
            for (int c = 0; c < L; ++c) {
                const int s = c % kSumStages;
                if (c >= kSumStages && !mbar_wait(&bars->empty[s], ((c / kSumStages) - 1) & 1, prm.status, kStatusPipeTimeout)) {
                    *abort_flag = 1;
                    break;
                }
                if (*abort_flag) break;
                if (early_loads && c == kSumStages) {
                    grid_dependency_wait();
                    allow_dependent_launch();
                }
                uint8_t* st = smem + s * kSumStageBytes;
                const int y = (c_begin + c) * kChunk, z = (int)bh;      // position in the sequence; sequence
                LA_TRACE(g_trace_seg, c, 2);
                mbar_arrive_expect_tx(&bars->full[s], 2 * kTileBytes);
                const bool wanted_soon = scaled ? prm.plan.in_piece_tail(c_begin + c, kKeepTailChunks)
                                                : prm.plan.in_piece_head(c_begin + c, kKeepTailChunks);
                const uint64_t pol = wanted_soon ? pol_keep : pol_stream;
                tile_load<kVarlen>(true, st, &mapX, y, z, prm.N, &bars->full[s], pol);
                tile_load<kVarlen>(true, st + kTileBytes, &mapY, y, z, prm.N, &bars->full[s], pol);
            }
        }
        if (early_loads && L <= kSumStages) {        // a part of at most three chunks: the loop never got there
            grid_dependency_wait();
            allow_dependent_launch();
        }
    } else if (warp == 5) {
        {
            const bool leader = elect_one();
            // one M = 64, N = 80 product per K group: B = [Y | a], the second 64-column block being the
            // column tile (same K group)
            const uint32_t idesc = umma_idesc_bf16(64, 80, 1, 1);
            const uint32_t aAux = sbase + kSumOffAux;
            bool ok = true;
            #pragma unroll 1
            for (int c = 0; c < L && ok; ++c) {
                const int s = c % kSumStages;
                const uint32_t aX = sbase + s * kSumStageBytes, aY = aX + kTileBytes;
                ok = mbar_wait_warp(&bars->mapped[s], (c / kSumStages) & 1, prm.status, kStatusPipeTimeout);
                if (!ok || __any_sync(0xFFFFFFFFu, *abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                if (leader) LA_TRACE(g_trace_seg, c, 0);
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    umma_bf16(leader, tmem, desc_mn(aX + k * 2048), desc_mn(aY + k * 2048, aAux - aY), idesc, (c | k) != 0);
                umma_commit(leader, &bars->empty[s]);
                if (leader) LA_TRACE(g_trace_seg, c, 1);
            }
            if (!ok) *abort_flag = 1;
            umma_commit(leader, &bars->done);
        }
    } else {
        const int t = tid;
        const uint32_t r7 = t & 7;
        #pragma unroll 1
        for (int c = 0; c < L; ++c) {
            const int s = c % kSumStages;
            const int64_t row = row0 + (int64_t)c * kChunk + t;
            const bool pad = kVarlen && c == L - 1 && t >= span.tail_rows;      // (a padded row may lie past the sequence's N)
            float inv = 1.f, delta = 0.f;
            if (scaled && !pad) {
                inv = 1.f / __ldg(prm.dn + row);
                delta = __ldg(prm.dl + row);
            }
            if (!mbar_wait(&bars->full[s], (c / kSumStages) & 1, prm.status, kStatusTmaTimeout)) { *abort_flag = 1; break; }
            if (*abort_flag) break;
            if (t == 0) LA_TRACE(g_trace_seg, c, 5);
            uint8_t* rowX = smem + s * kSumStageBytes + t * 128;
            if (prm.map) {
                if (scaled) map_row_inplace<true>(rowX, r7, inv, prm.dim >> 3);
                else phi_row_inplace(rowX, r7, prm.dim >> 3);
            }
            else if (scaled) map_row_inplace<false>(rowX, r7, inv, prm.dim >> 3);
            if (pad) {                                              // padding: no feature, no value, no dl
                zero_row(rowX);
                zero_row(rowX + kTileBytes);
                delta = 0.f;
            }
            if (scaled) {
                // the single column tile is still an operand of the previous chunk's products
                if (c >= 1 && !mbar_wait(&bars->empty[(c - 1) % kSumStages], ((c - 1) / kSumStages) & 1, prm.status,
                                         kStatusMmaTimeout)) { *abort_flag = 1; break; }
                uint8_t* rowA = smem + kSumOffAux + t * 128;
                const uint32_t dd = pack_bf16x2(delta, delta);      // columns 0..15 of the column tile
                sts128(rowA + ((0 ^ r7) << 4), dd, dd, dd, dd);
                sts128(rowA + ((1 ^ r7) << 4), dd, dd, dd, dd);
            }
            fence_proxy_async_smem();
            mbar_arrive(&bars->mapped[s]);
            if (t == 0) LA_TRACE(g_trace_seg, c, 6);
        }
        if (t == 0) LA_TRACE(g_trace_seg, 100, 7);
        // read-out: the [S | Z]-shaped record of this (bh, seg)
        const bool empty = kVarlen && L == 0;           // nothing was summed: the accumulator holds no result
        const bool ok = mbar_wait(&bars->done, 0, prm.status, kStatusMmaTimeout) && !*abort_flag;
        tc_fence_after_sync();
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        float* rec = prm.records + (bh * prm.plan.nparts() + seg) * (int64_t)kStateFloats;
        const int d_row = warp * 16 + lane;
        for (int h = 0; h < 2; ++h) {
            uint32_t v[32];
            tmem_ld32(tmem + lane_base + h * 32, v);
            tmem_ld_wait();
            if (ok && lane < 16)
#pragma unroll
                for (int j = 0; j < 32; ++j) rec[d_row * kDim + h * 32 + j] = empty ? 0.f : __uint_as_float(v[j]);
        }
        const float z = __uint_as_float(tmem_ld1(tmem + lane_base + 64));
        tmem_ld_wait();
        if (ok && lane < 16) rec[kDim * kDim + d_row] = empty ? 0.f : z;
    }
    tc_fence_before_sync();
    __syncthreads();
    LA_TRACE_CTA(g_trace_seg, 1);
    if (warp == 5) {
        __syncwarp();
        tmem_dealloc(tmem, 128);
    }
}

}  // namespace

int segment_states(const la_problem& p, const CausalPlan& pl, const CUtensorMap& mapX, const CUtensorMap& mapY,
                   const float* dn, const float* dl, float* records, bool reverse, bool map, cudaStream_t st,
                   const int* lengths) {
    if (pl.npieces() <= 1) return LA_OK;
    static std::atomic<uint64_t> attr_done{0}, attr_done_ragged{0};
    const bool ragged = ragged_problem(p, lengths);
    if (int rc = ragged ? opt_in_smem_once(segment_sum_kernel<true>, kSumSmemBytes, attr_done_ragged)
                         : opt_in_smem_once(segment_sum_kernel<false>, kSumSmemBytes, attr_done)) return rc;
    SumParams prm;
    prm.records = records;
    prm.dn = dn;
    prm.dl = dl;
    prm.status = device_status_ptr();
    if (!prm.status) return fail(LA_ERR_CUDA, "device status word unavailable");
    prm.N = p.N;
    prm.plan = pl;
    // the sums of the piece at the open end of a sweep are never needed
    prm.first_part = reverse ? pl.piece_first_part(1) : 0;
    prm.parts_per_seq = reverse ? pl.nparts() - prm.first_part : pl.piece_first_part(pl.npieces() - 1);
    prm.eps = p.eps;
    prm.map = map ? 1 : 0;
    prm.dim = (int)p.D;
    prm.lengths = lengths;
    prm.heads = (int)p.H;
    prof_begin(kProfSegmentSum, st);
    cudaLaunchAttribute attr;
    const cudaLaunchConfig_t cfg = chained_launch((unsigned)(prm.parts_per_seq * p.B * p.H), kSumThreads, kSumSmemBytes, st, &attr);
    if (ragged) LA_CUDA_TRY(cudaLaunchKernelEx(&cfg, segment_sum_kernel<true>, mapX, mapY, prm));
    else LA_CUDA_TRY(cudaLaunchKernelEx(&cfg, segment_sum_kernel<false>, mapX, mapY, prm));
    note_launch();
    prof_end(kProfSegmentSum, st);
    return LA_OK;
}

}  // namespace tc
}  // namespace la

#ifdef LA_TC_TRACE
extern "C" int la_debug_read_trace_seg(long long* out, int n) {
    return (int)cudaMemcpyFromSymbol(out, la::tc::g_trace_seg, n * sizeof(long long));
}
#endif
