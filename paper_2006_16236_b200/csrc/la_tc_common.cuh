// Pieces shared by the tensor-core kernels: chunk geometry, host-side tensor-map
// encoding, the per-segment state records in the workspace, and the device helpers
// for the feature map on a swizzled tile row.
#pragma once

#include <atomic>

#include <cudaTypedefs.h>

#include "la_common.cuh"
#include "la_sm100.cuh"

namespace la {
namespace tc {

// Optional pipeline trace (compile with -DLA_TC_TRACE): CTA 0 stamps clock64() per chunk and
// event into a per-file buffer that la_debug_read_trace_*() copies out.  Compiled out otherwise.
#ifdef LA_TC_TRACE
#define LA_TRACE_DECL(name) __device__ long long name[1536 * 32];
#define LA_TRACE(buf, c, slot) do { if (blockIdx.x == 0 && (c) < 512) buf[(c) * 32 + (slot)] = clock64(); } while (0)
#define LA_TRACE_CTA(buf, slot) do { if (threadIdx.x == 0) { unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); buf[(512 + (blockIdx.x & 1023)) * 32 + (slot)] = (long long)t_; } } while (0)
#else
#define LA_TRACE_DECL(name)
#define LA_TRACE(buf, c, slot) do { } while (0)
#define LA_TRACE_CTA(buf, slot) do { } while (0)
#endif

// Launch configuration of a kernel that may start while the kernel before it in the stream drains (its set-up
// overlaps that kernel's tail; it waits on the grid dependency before touching global memory).
inline cudaLaunchConfig_t chained_launch(unsigned grid, unsigned block, size_t smem, cudaStream_t st,
                                         cudaLaunchAttribute* attr) {
    attr->id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr->val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cfg;
}

// cudaFuncAttributeMaxDynamicSharedMemorySize belongs to a (function, device) pair: it is set the first
// time a kernel is launched on each device (`done`: one bit per device ordinal, one word per kernel).
template <typename Kernel>
inline int opt_in_smem_once(Kernel kernel, size_t bytes, std::atomic<uint64_t>& done) {
    int dev = 0;
    LA_CUDA_TRY(cudaGetDevice(&dev));
    const uint64_t bit = dev >= 0 && dev < 64 ? 1ull << dev : 0;
    if (bit && (done.load(std::memory_order_acquire) & bit)) return LA_OK;
    LA_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
    done.fetch_or(bit, std::memory_order_release);
    return LA_OK;
}

// SMs of the current device (148 on a B200; also the answer when no device can be asked, so that the
// host-only plan and workspace queries work without one).
int sm_count();

// Overrides of the automatic piece / split plans, set through la_plan_override() (-1: automatic).
struct PlanOverride {
    int causal_pieces, causal_short, linear_splits;
};
PlanOverride plan_override();

constexpr int kChunk = 128;                  // positions per chunk = MMA M
constexpr int kDim = 64;                     // D = M = 64: one 128-byte swizzle row
constexpr int kTileBytes = kChunk * kDim * 2;  // one [128][64] bf16 tile
constexpr int kStateFloats = kDim * (kDim + 1);  // [S (64x64) | Z (64)] per record

// How a (batch, head) sequence of the non-causal kernels is cut into segments that run concurrently.
struct Segmentation {
    int nseg;             // segments per sequence (one CTA of the main kernels each)
    int chunks_per_seg;   // chunks in every segment but possibly the last
};

// How the causal kernels cut a sequence into pieces (one CTA of a main kernel each) and the pieces
// into pre-pass parts (one CTA of the pre-pass and one [S | Z]-shaped record each).
//   `nlong` long pieces of near-equal length and, if m > 0, one short piece of m chunks at position
//   `spos` of the sequence.  The CTAs of the long pieces have the lowest block indices and start first;
//   when B*H*nlong is less than the SM count, the SMs left over take the short pieces, several each, one
//   after the other, so that every SM is busy for about the same time although B*H does not divide 148.
//   Every long piece has `sub` parts of near-equal length, the short piece is one part.  A piece starts
//   from the sum of the records of the parts before it (forward sweep) or after it (reverse sweep).
// All fields are small integers: the struct is passed to the kernels by value.
struct CausalPlan {
    int chunks, bh;       // chunks per sequence; sequences (batch x head pairs)
    int nlong, m, spos, sub;

    __host__ __device__ int has_short() const { return m > 0 ? 1 : 0; }
    __host__ __device__ int npieces() const { return nlong + has_short(); }
    __host__ __device__ int nparts() const { return nlong * sub + has_short(); }
    // first chunk of the j-th long piece, counted without the short piece
    __host__ __device__ int long_start(int j) const {
        const int lt = chunks - m;
        return j * (lt / nlong) + (j < lt % nlong ? j : lt % nlong);
    }
    // piece k of the sequence: first chunk, and first part; k = npieces() gives the end
    __host__ __device__ int piece_begin(int k) const {
        if (!has_short() || k <= spos) return long_start(k);
        return long_start(k - 1) + m;
    }
    __host__ __device__ int piece_first_part(int k) const {
        if (!has_short() || k <= spos) return k * sub;
        return (k - 1) * sub + 1;
    }
    // launch slot (blockIdx.x / bh) -> piece: long pieces first, the short one last
    __host__ __device__ int piece_of_slot(int slot) const {
        if (!has_short()) return slot;
        if (slot == nlong) return spos;
        return slot < spos ? slot : slot + 1;
    }
    // part q of the sequence: first chunk; q = nparts() gives the end
    __host__ __device__ int part_begin(int q) const {
        int k, i;                               // piece and index of the part inside it
        if (has_short() && q >= spos * sub + 1) {
            k = (q - 1) / sub + 1;
            i = (q - 1) % sub;
        } else if (has_short() && q == spos * sub) {
            return piece_begin(spos);
        } else {
            k = q / sub;
            i = q % sub;
        }
        if (k >= npieces()) return chunks;
        const int b = piece_begin(k), len = piece_begin(k + 1) - b;
        return b + i * (len / sub) + (i < len % sub ? i : len % sub);
    }
    // is chunk g of the sequence among the last `keep` chunks of its piece?  (the reverse sweep starts there: those
    // tiles are asked to stay in L2 by the kernels that read them shortly before it)
    __host__ __device__ bool in_piece_tail(int g, int keep) const {
        for (int k = 1; k <= npieces(); ++k) {
            const int e = piece_begin(k);
            if (g < e) return g >= e - keep;
        }
        return false;
    }
    // ... or among its first `keep` chunks (where the forward sweeps start)?
    __host__ __device__ bool in_piece_head(int g, int keep) const {
        for (int k = 0; k < npieces(); ++k) {
            const int b = piece_begin(k);
            if (g >= b && g < b + keep) return true;
        }
        return false;
    }
};

// Chunks at the end of every piece whose tiles the forward sweep of the backward pass and the reverse pre-pass ask
// L2 to keep for the reverse sweep (192 pieces x 7 chunks x 64 KB = 86 MB of the 126 MB L2 at the benchmark
// shape); every other tile of those kernels is read once and asked to leave first.
constexpr int kKeepTailChunks = 7;

CausalPlan choose_plan(const la_problem& p);
// chunks of a sequence of N positions (the last one may be partial); the ragged variants of the kernels run when
// a batch carries lengths or N is not a multiple of the chunk
inline int chunks_of(int64_t N) { return (int)((N + kChunk - 1) / kChunk); }
inline bool ragged_problem(const la_problem& p, const int* lengths) { return lengths != nullptr || p.N % kChunk != 0; }

// Per-part sums of phi(X)^T [Y | a] into `records` (forward: the parts before the last piece; reverse:
// the parts after the first piece)
// lengths ([B] int32, device, or null): real positions per batch element of a right-padded ragged batch
int segment_states(const la_problem& p, const CausalPlan& pl, const CUtensorMap& mapX, const CUtensorMap& mapY,
                   const float* dn, const float* dl, float* records, bool reverse, bool map, cudaStream_t st,
                   const int* lengths = nullptr);

// What the causal forward leaves for the causal backward when the caller passes a `saved`
// buffer: the mapped phi(Q) and phi(K) ([B*H*N, D] bf16 each, exactly the operands the
// forward's tensor-core products consumed) and the forward pre-pass records.  The backward
// then reads the mapped tensors in place of Q and K, evaluates no exponential and skips its
// own forward pre-pass; its results are the same bit for bit.
struct SavedLayout {
    size_t phiq, phik, records, stamp, bytes;      // byte offsets of the four parts; total size
};
// The forward also stamps the buffer with the plan it used (kPlanStampInts integers); a backward pass whose
// own plan differs (an override changed in between, another device) reports kStatusPlanMismatch and
// computes nothing, instead of reading records at offsets they were not written at.
constexpr int kPlanStampInts = 8;
__host__ __device__ inline void plan_stamp(const CausalPlan& pl, int dim, int (&out)[kPlanStampInts]) {
    out[0] = 0x4c41504c;    // "LAPL"
    out[1] = pl.chunks; out[2] = pl.bh; out[3] = pl.nlong; out[4] = pl.m; out[5] = pl.spos; out[6] = pl.sub; out[7] = dim;
}
inline SavedLayout saved_layout(const la_problem& p, const CausalPlan& pl) {
    const size_t rows = (size_t)(p.B * p.H * p.N);
    const size_t tensor = (rows * (size_t)p.D * 2 + 1023) & ~(size_t)1023;
    SavedLayout l;
    l.phiq = 0;
    l.phik = tensor;
    l.stamp = 2 * tensor;            // at an offset that does not depend on the plan
    l.records = l.stamp + 1024;
    l.bytes = l.records + (pl.npieces() > 1 ? (size_t)(p.B * p.H) * pl.nparts() * kStateFloats * sizeof(float) : 0);
    return l;
}

// 2-D view of a [rows][cols] bf16 tensor (cols = 32 or 64) with a [box_rows][64] box and the
// 128-byte swizzle.  With cols = 32 the upper half of every 128-byte tile row is out of bounds:
// loads fill it with zeros (zero features and zero values contribute nothing to any product),
// stores clip it.  The kernels then run as for 64 and only touch `cols` columns in global memory.
int encode_tile_map(CUtensorMap* map, const void* base, uint64_t rows, uint32_t box_rows, int cols = kDim);
// The same over [seqs][n][cols] with boxes of one sequence's rows: coordinates (column, position, sequence)
int encode_seq_tile_map(CUtensorMap* map, const void* base, uint64_t seqs, uint64_t n, uint32_t box_rows, int cols = kDim);

// ---------------------------------------------------------------------------
// Feature map on one 128-byte row of a swizzled tile, in place: thread-per-row.
// `row_base` is the shared-memory address of the row; r7 = row & 7 (swizzle key).
// ---------------------------------------------------------------------------
__device__ __forceinline__ float phi_fast(float x) {
    // elu(x) + 1 with the hardware exponential: exp(x) = 2^(x * log2 e)
    float e;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(x * 1.4426950408889634f));
    return x > 0.f ? x + 1.f : e;
}

// elu(x) + 1 on a packed pair of bf16 values, nine instructions per pair instead of thirteen:
// x + 1 is one packed bf16 add (a single rounding of the exact sum, as the fp32 add followed by a
// conversion gives), the two products with log2 e are one packed fp32 multiply, and each half
// takes the exponential where its sign bit is set (a byte permute that replicates the sign
// bits builds the mask; -0 takes 2^0 = 1 = 0 + 1).  Bit-identical to phi_fast per element.
__device__ __forceinline__ uint32_t phi_pair(uint32_t w) {
    uint32_t lin, mask, ex, res;
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(lin) : "r"(w), "r"(0x3F803F80u));
    uint64_t xx, tt, cc;
    asm("mov.b64 %0, {%1, %2};" : "=l"(xx) : "r"(w << 16), "r"(w & 0xFFFF0000u));
    asm("mov.b64 %0, {%1, %1};" : "=l"(cc) : "f"(1.4426950408889634f));
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(tt) : "l"(xx), "l"(cc));
    float t0, t1, e0, e1;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(t0), "=f"(t1) : "l"(tt));
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(t0));
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(t1));
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(ex) : "f"(e1), "f"(e0));
    asm("prmt.b32 %0, %1, %1, 0xBB99;" : "=r"(mask) : "r"(w));
    asm("lop3.b32 %0, %1, %2, %3, 0xCA;" : "=r"(res) : "r"(mask), "r"(ex), "r"(lin));    // mask ? ex : lin
    return res;
}

// Shared-memory accesses of the CUDA-core roles are plain C++ vector accesses on pointers
// derived from the dynamic shared-memory base, so that the compiler can batch and schedule
// them (the waits and fences around them are asm statements with memory clobbers).
__device__ __forceinline__ void lds128(const uint8_t* p, uint32_t (&v)[4]) {
    const uint4 x = *reinterpret_cast<const uint4*>(p);
    v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
}
__device__ __forceinline__ void sts128(uint8_t* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    *reinterpret_cast<uint4*>(p) = make_uint4(a, b, c, d);
}

// One 128-byte row (64 bf16) of a swizzled tile into registers / back, in LOGICAL chunk order
// (chunk c of row r lives at physical chunk c ^ (r & 7); visiting it that way also keeps the
// eight rows of a quarter-warp on eight different bank groups).
__device__ __forceinline__ void load_row(const uint8_t* row, uint32_t r7, uint32_t (&v)[8][4]) {
#pragma unroll
    for (int c = 0; c < 8; ++c) lds128(row + ((c ^ r7) << 4), v[c]);
}
// first `nch` logical chunks only (nch = 4 when the row holds 32 real columns)
__device__ __forceinline__ void store_row(uint8_t* row, uint32_t r7, const uint32_t (&v)[8][4], int nch = 8) {
#pragma unroll
    for (int c = 0; c < 8; ++c)
        if (c < nch) sts128(row + ((c ^ r7) << 4), v[c][0], v[c][1], v[c][2], v[c][3]);
}

// Feature map on one row in place (optionally scaled), two 16-byte chunks per iteration of a
// rolled loop: the loop body stays small enough to live in the instruction cache next to the
// other roles' loops (a fully unrolled row is 8 KB of code per call site).
template <bool kElu, bool kScale = true>
__device__ __forceinline__ void map_row_inplace(uint8_t* row, uint32_t r7, float scale, int nch = 8) {
#pragma unroll 1
    for (int c = 0; c < nch; c += 2) {
        uint32_t v[2][4];
        lds128(row + ((c ^ r7) << 4), v[0]);
        lds128(row + (((c + 1) ^ r7) << 4), v[1]);
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (kElu && !kScale) {
                    v[i][j] = phi_pair(v[i][j]);
                } else if (!kElu && kScale) {           // one multiply for the pair
                    v[i][j] = sm100::pack_bf16x2(sm100::mul2(sm100::pair_bf16(v[i][j]), sm100::pair(scale, scale)));
                } else {
                    const float x0 = sm100::bf16_lo(v[i][j]), x1 = sm100::bf16_hi(v[i][j]);
                    const float y0 = kElu ? phi_fast(x0) : x0, y1 = kElu ? phi_fast(x1) : x1;
                    v[i][j] = kScale ? sm100::pack_bf16x2(y0 * scale, y1 * scale) : sm100::pack_bf16x2(y0, y1);
                }
            }
        sts128(row + ((c ^ r7) << 4), v[0][0], v[0][1], v[0][2], v[0][3]);
        sts128(row + (((c + 1) ^ r7) << 4), v[1][0], v[1][1], v[1][2], v[1][3]);
    }
}
__device__ __forceinline__ void phi_row_inplace(uint8_t* row, uint32_t r7, int nch = 8) {
    map_row_inplace<true, false>(row, r7, 1.f, nch);
}

// Right-padded ragged batches, and sequences whose length N is not a multiple of the chunk (lengths == nullptr:
// every sequence has N positions).  Of the chunks [c_begin, c_begin + n_full) a CTA is responsible for, only those
// that hold real positions of the sequence are processed; the last of them may be partly padding.  Rows of a
// chunk at positions >= N do not exist in memory (they would be the next sequence's): the 3-D tile loads read
// zeros there and the tile stores clip them; plain loads and stores skip them.
struct RaggedSpan {
    int chunks;         // chunks of the span to process (0: the span is all padding)
    int tail_rows;      // real rows of the last processed chunk (kChunk unless the sequence ends inside it)
    bool has_end;       // the sequence's last real chunk lies in this span
};
__device__ __forceinline__ RaggedSpan ragged_span(const int* lengths, int heads, int64_t bh, int64_t N, int c_begin, int n_full) {
    int64_t len = lengths ? lengths[bh / heads] : N;
    len = len < 0 ? 0 : (len < N ? len : N);
    const int nc = (int)((len + kChunk - 1) / kChunk);              // chunks of the sequence with real rows
    RaggedSpan r;
    r.chunks = nc - c_begin < 0 ? 0 : (nc - c_begin < n_full ? nc - c_begin : n_full);
    r.has_end = r.chunks > 0 && c_begin + r.chunks == nc;
    r.tail_rows = r.has_end ? (int)(len - (int64_t)(nc - 1) * kChunk) : kChunk;
    return r;
}
// Tile transfers of the attention kernels: position `pos` of sequence `seq` (N positions each).  Whole chunks only
// (k3d false): the tensor is one [seqs * N][cols] matrix and the tile a 2-D box, which the TMA unit handles a little
// faster (0.3 % of the benchmark step); otherwise a 3-D box over [seqs][N][cols] that ends with its sequence.
template <bool k3d>
__device__ __forceinline__ void tile_load(void* dst, const CUtensorMap* map, int pos, int seq, int64_t N, uint64_t* bar) {
    if (k3d) sm100::tma_load_3d(dst, map, 0, pos, seq, bar);
    else sm100::tma_load_2d(dst, map, 0, (int)(seq * N + pos), bar);
}
template <bool k3d>
__device__ __forceinline__ void tile_load(bool leader, void* dst, const CUtensorMap* map, int pos, int seq, int64_t N, uint64_t* bar,
                                          uint64_t policy) {
    if (k3d) sm100::tma_load_3d(leader, dst, map, 0, pos, seq, bar, policy);
    else sm100::tma_load_2d(leader, dst, map, 0, (int)(seq * N + pos), bar, policy);
}
template <bool k3d>
__device__ __forceinline__ void tile_store(const CUtensorMap* map, const void* src, int pos, int seq, int64_t N) {
    if (k3d) sm100::tma_store_3d(map, src, 0, pos, seq);
    else sm100::tma_store_2d(map, src, 0, (int)(seq * N + pos));
}
// the map that goes with them
inline int encode_attention_map(CUtensorMap* map, const void* base, bool three_d, uint64_t seqs, uint64_t n, uint32_t box_rows, int cols) {
    return three_d ? encode_seq_tile_map(map, base, seqs, n, box_rows, cols) : encode_tile_map(map, base, seqs * n, box_rows, cols);
}

// A whole 128-byte tile row of zeros (padding rows of a ragged batch: whatever they held, they contribute nothing).
__device__ __forceinline__ void zero_row(uint8_t* row) {
#pragma unroll
    for (int c = 0; c < 8; ++c) sts128(row + (c << 4), 0u, 0u, 0u, 0u);
}

__device__ __forceinline__ uint64_t desc_k(uint32_t addr) { return sm100::umma_desc_sw128(addr, 16, 1024); }
__device__ __forceinline__ uint64_t desc_mn(uint32_t addr, uint32_t lbo = kTileBytes) {
    return sm100::umma_desc_sw128(addr, lbo, 1024);
}
// B operand whose every entry is 1: one 1 KB group of ones re-read for every K group (SBO = 0).
__device__ __forceinline__ uint64_t desc_ones(uint32_t addr) { return sm100::umma_desc_sw128(addr, 16, 0); }

__device__ __forceinline__ void stg128(void* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    *reinterpret_cast<uint4*>(p) = make_uint4(a, b, c, d);
}

// One 32-column block of a 128x128 fp32 score matrix (already loaded from TMEM into v)
// -> + `add` -> causal mask on the diagonal block -> bf16 -> this row's 64 bytes of the
// swizzled [128][64] tile pair.  tile_row = shared address of row t in tile 0 of the pair.
__device__ __forceinline__ void score_block_store(const uint32_t (&v)[32], uint8_t* tile_row, uint32_t r7, int blk,
                                                  bool diagonal, int lane, float add) {
    uint32_t packed[16];
    const sm100::f32x2 add2 = sm100::pair(add, add);
    if (!diagonal) {            // (one warp-uniform branch per block instead of a select per element)
#pragma unroll
        for (int j = 0; j < 16; ++j) packed[j] = sm100::pack_bf16x2(sm100::add2(sm100::pair(v[2 * j], v[2 * j + 1]), add2));
    } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            float x0, x1;
            sm100::unpair(sm100::add2(sm100::pair(v[2 * j], v[2 * j + 1]), add2), x0, x1);      // one add for two columns
            if (2 * j > lane) x0 = 0.f;
            if (2 * j + 1 > lane) x1 = 0.f;
            packed[j] = sm100::pack_bf16x2(x0, x1);
        }
    }
    uint8_t* base = tile_row + (blk >> 1) * kTileBytes;
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
        const uint32_t chunk = (blk & 1) * 4 + cc;
        sts128(base + ((chunk ^ r7) << 4), packed[cc * 4], packed[cc * 4 + 1], packed[cc * 4 + 2], packed[cc * 4 + 3]);
    }
}

// State accumulator (M = 64 layout: lanes 0-15 of quadrant w hold rows 16w..16w+15; 64 columns
// of S followed by Z) -> bf16 [64][64] swizzled tile + fp32 Z; optionally the fp32 values to
// global memory.  Executed by the four warps of one warpgroup; `quad` = warp % 4.
__device__ __forceinline__ void state_to_smem(uint32_t tmem_state, int quad, int lane, uint8_t* s_tile, float* z_out,
                                              float* g_S, float* g_Z, int dim = kDim) {
    const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
    const int d_row = quad * 16 + lane;
    const bool owner = lane < 16;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        uint32_t v[32];
        sm100::tmem_ld32(tmem_state + lane_base + h * 32, v);
        sm100::tmem_ld_wait();
        if (owner) {
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                const uint32_t chunk = h * 4 + cc;
                sts128(s_tile + d_row * 128 + ((chunk ^ (d_row & 7)) << 4),
                       sm100::pack_bf16x2(__uint_as_float(v[cc * 8 + 0]), __uint_as_float(v[cc * 8 + 1])),
                       sm100::pack_bf16x2(__uint_as_float(v[cc * 8 + 2]), __uint_as_float(v[cc * 8 + 3])),
                       sm100::pack_bf16x2(__uint_as_float(v[cc * 8 + 4]), __uint_as_float(v[cc * 8 + 5])),
                       sm100::pack_bf16x2(__uint_as_float(v[cc * 8 + 6]), __uint_as_float(v[cc * 8 + 7])));
            }
            if (g_S && d_row < dim && h * 32 < dim) {
#pragma unroll
                for (int j = 0; j < 32; ++j) g_S[d_row * dim + h * 32 + j] = __uint_as_float(v[j]);
            }
        }
    }
    const float z = __uint_as_float(sm100::tmem_ld1(tmem_state + lane_base + 64));
    sm100::tmem_ld_wait();
    if (owner) {
        z_out[d_row] = z;
        if (g_Z && d_row < dim) g_Z[d_row] = z;
    }
}

// Sum over the records of parts [part_lo, part_hi) of sixteen consecutive floats (at `offset` inside a
// record), in part order, with the loads of four records in flight: a piece late in a sequence starts
// from several records, and one round trip to L2 per record and column group would cost microseconds
// on the critical start-up of its CTA.
__device__ __forceinline__ void sum_records16(const float* rec, int part_lo, int part_hi, int offset, float (&acc)[16],
                                              const float* base = nullptr) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {      // `base` (16 floats, 16-byte aligned, or null): the value the sum starts from
        const float4 b = base ? __ldg(reinterpret_cast<const float4*>(base) + j) : make_float4(0.f, 0.f, 0.f, 0.f);
        acc[4 * j] = b.x; acc[4 * j + 1] = b.y; acc[4 * j + 2] = b.z; acc[4 * j + 3] = b.w;
    }
#pragma unroll 1
    for (int p = part_lo; p < part_hi; p += 4) {
        float4 a[4][4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const bool on = p + u < part_hi;
            const float4* src = reinterpret_cast<const float4*>(rec + (int64_t)(on ? p + u : p) * kStateFloats + offset);
#pragma unroll
            for (int j = 0; j < 4; ++j) a[u][j] = on ? __ldg(src + j) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                acc[4 * j] += a[u][j].x; acc[4 * j + 1] += a[u][j].y; acc[4 * j + 2] += a[u][j].z; acc[4 * j + 3] += a[u][j].w;
            }
    }
}
// The same for one float per record.
__device__ __forceinline__ float sum_records1(const float* rec, int part_lo, int part_hi, int offset) {
    float z = 0.f;
#pragma unroll 1
    for (int p = part_lo; p < part_hi; p += 4) {
        float a[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) a[u] = p + u < part_hi ? __ldg(rec + (int64_t)(p + u) * kStateFloats + offset) : 0.f;
#pragma unroll
        for (int u = 0; u < 4; ++u) z += a[u];
    }
    return z;
}

// Initial state of a segment: the sum of the records of parts [part_lo, part_hi) of this
// (batch, head) (none: zeros) goes into the TMEM state accumulator, its bf16 tile and z_out.
// s_in / z_in (or null): the [dim][dim] / [dim] fp32 state of this (batch, head) the sequence continues from.
__device__ __forceinline__ void state_init(uint32_t tmem_state, int quad, int lane, uint8_t* s_tile, float* z_out,
                                           const float* rec, int part_lo, int part_hi,
                                           const float* s_in = nullptr, const float* z_in = nullptr, int dim = kDim) {
    const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
    const int d_row = quad * 16 + lane;
    const bool owner = lane < 16;
    const bool in_row = owner && s_in && d_row < dim;
#pragma unroll 1
    for (int g = 0; g < 4; ++g) {
        float acc[16];
        sum_records16(rec, owner ? part_lo : 0, owner ? part_hi : 0, d_row * kDim + g * 16, acc,
                      in_row && g * 16 < dim ? s_in + d_row * dim + g * 16 : nullptr);
        uint32_t v[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] = __float_as_uint(acc[j]);
        sm100::tmem_st16(tmem_state + lane_base + g * 16, v);
        if (owner) {
#pragma unroll
            for (int cc = 0; cc < 2; ++cc)
                sts128(s_tile + d_row * 128 + (((2 * g + cc) ^ (d_row & 7)) << 4),
                       sm100::pack_bf16x2(acc[cc * 8 + 0], acc[cc * 8 + 1]), sm100::pack_bf16x2(acc[cc * 8 + 2], acc[cc * 8 + 3]),
                       sm100::pack_bf16x2(acc[cc * 8 + 4], acc[cc * 8 + 5]), sm100::pack_bf16x2(acc[cc * 8 + 6], acc[cc * 8 + 7]));
        }
    }
    const float z = (owner ? sum_records1(rec, part_lo, part_hi, kDim * kDim + d_row) : 0.f) + (in_row ? __ldg(z_in + d_row) : 0.f);
    uint32_t zz[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) zz[j] = __float_as_uint(z);
    sm100::tmem_st16(tmem_state + lane_base + 64, zz);
    sm100::tmem_st_wait();
    if (owner) z_out[d_row] = z;
}

// ---------------------------------------------------------------------------
// Variants that keep Z as a bf16 MMA operand next to S: the 8 KB tile `z_tile` ([64][64]
// swizzled, row d = Z_d in its first 16 columns) is the second 64-column block of an MN-major
// B operand [S | Z] of width 80, so that q [S | Z] yields the numerator and q . Z in one MMA.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void z_row_store(uint8_t* z_tile, int d_row, float z) {
    const uint32_t zz = sm100::pack_bf16x2(z, z);
    uint8_t* row = z_tile + d_row * 128;
    const uint32_t r7 = d_row & 7;
    sts128(row + ((0 ^ r7) << 4), zz, zz, zz, zz);
    sts128(row + ((1 ^ r7) << 4), zz, zz, zz, zz);
}

__device__ __forceinline__ void state_row_store(uint8_t* s_tile, int d_row, int h, const uint32_t (&v)[32]) {
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
        const uint32_t chunk = h * 4 + cc;
        sts128(s_tile + d_row * 128 + ((chunk ^ (d_row & 7)) << 4),
               sm100::pack_bf16x2(__uint_as_float(v[cc * 8 + 0]), __uint_as_float(v[cc * 8 + 1])),
               sm100::pack_bf16x2(__uint_as_float(v[cc * 8 + 2]), __uint_as_float(v[cc * 8 + 3])),
               sm100::pack_bf16x2(__uint_as_float(v[cc * 8 + 4]), __uint_as_float(v[cc * 8 + 5])),
               sm100::pack_bf16x2(__uint_as_float(v[cc * 8 + 6]), __uint_as_float(v[cc * 8 + 7])));
    }
}

// One half (columns 32 h .. 32 h + 31; h = 0 also carries Z) of the state accumulator -> registers,
// `drained` is signalled at once (the accumulator may be updated again: the update of the next chunk
// waits for exactly this), then the bf16 tiles are written; optionally the fp32 values go to global
// memory.  Two groups of four warps convert one half each.
__device__ __forceinline__ void state_half_to_tiles(uint32_t tmem_state, int quad, int lane, int h, uint8_t* s_tile,
                                                    uint8_t* z_tile, uint64_t* drained, float* g_S, float* g_Z, int dim) {
    const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
    const int d_row = quad * 16 + lane;
    const bool owner = lane < 16;
    uint32_t v[32];
    sm100::tmem_ld32(tmem_state + lane_base + h * 32, v);
    float z = 0.f;
    if (h == 0) z = __uint_as_float(sm100::tmem_ld1(tmem_state + lane_base + 64));
    sm100::tmem_ld_wait();
    sm100::tc_fence_before_sync();
    if (drained) sm100::mbar_arrive(drained);
    if (owner) {
        state_row_store(s_tile, d_row, h, v);
        if (h == 0) z_row_store(z_tile, d_row, z);
        if (g_S && d_row < dim && h * 32 < dim) {
#pragma unroll
            for (int j = 0; j < 32; ++j) g_S[d_row * dim + h * 32 + j] = __uint_as_float(v[j]);
        }
        if (h == 0 && g_Z && d_row < dim) g_Z[d_row] = z;
    }
}

// Initial state of a segment (sum of the records of parts [part_lo, part_hi), or zeros) into
// the TMEM accumulator (S in 64 columns, Z replicated in 16) and the bf16 tiles.
__device__ __forceinline__ void state_init_tiles(uint32_t tmem_state, int quad, int lane, uint8_t* s_tile, uint8_t* z_tile,
                                                 const float* rec, int part_lo, int part_hi) {
    const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
    const int d_row = quad * 16 + lane;
    const bool owner = lane < 16;
#pragma unroll 1
    for (int g = 0; g < 4; ++g) {
        float acc[16];
        sum_records16(rec, owner ? part_lo : 0, owner ? part_hi : 0, d_row * kDim + g * 16, acc);
        uint32_t v[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] = __float_as_uint(acc[j]);
        sm100::tmem_st16(tmem_state + lane_base + g * 16, v);
        if (owner) {
#pragma unroll
            for (int cc = 0; cc < 2; ++cc)
                sts128(s_tile + d_row * 128 + (((2 * g + cc) ^ (d_row & 7)) << 4),
                       sm100::pack_bf16x2(acc[cc * 8 + 0], acc[cc * 8 + 1]), sm100::pack_bf16x2(acc[cc * 8 + 2], acc[cc * 8 + 3]),
                       sm100::pack_bf16x2(acc[cc * 8 + 4], acc[cc * 8 + 5]), sm100::pack_bf16x2(acc[cc * 8 + 6], acc[cc * 8 + 7]));
        }
    }
    const float z = owner ? sum_records1(rec, part_lo, part_hi, kDim * kDim + d_row) : 0.f;
    uint32_t zz[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) zz[j] = __float_as_uint(z);
    sm100::tmem_st16(tmem_state + lane_base + 64, zz);
    sm100::tmem_st_wait();
    if (owner) z_row_store(z_tile, d_row, z);
}

// A state given by the caller ([dim][dim] and [dim] fp32 of this (batch, head): the state a sequence continues
// from, or the upstream gradient of its final state) added to a freshly initialised accumulator and its
// bf16 tile.  Out of line and only called when such a state is given: the kernels' own code keeps its shape.
// kForward: the 65th column is replicated over 16 columns and mirrored in `z_tile`; else it lives in column 64
// alone and is mirrored in `r_out`.
template <bool kForward>
__device__ __noinline__ void state_add_given(uint32_t tmem_state, int quad, int lane, uint8_t* s_tile, uint8_t* z_tile,
                                             float* r_out, const float* s_in, const float* z_in, int dim) {
    const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
    const int d_row = quad * 16 + lane;
    const bool owner = lane < 16;
    const bool in_row = owner && d_row < dim;
    sm100::tc_fence_after_sync();
    // the whole row of the given state is requested at once: one round trip to memory, not one per column group
    float4 given[16];
#pragma unroll
    for (int j = 0; j < 16; ++j)
        given[j] = (in_row && s_in && j * 4 < dim) ? __ldg(reinterpret_cast<const float4*>(s_in + d_row * dim) + j)
                                                    : make_float4(0.f, 0.f, 0.f, 0.f);
    const float z_given = (in_row && z_in) ? __ldg(z_in + d_row) : 0.f;
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        uint32_t v[16];
        sm100::tmem_ld16(tmem_state + lane_base + g * 16, v);
        sm100::tmem_ld_wait();
        float acc[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) acc[j] = __uint_as_float(v[j]);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float4 b = given[4 * g + j];
            acc[4 * j] += b.x; acc[4 * j + 1] += b.y; acc[4 * j + 2] += b.z; acc[4 * j + 3] += b.w;
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] = __float_as_uint(acc[j]);
        sm100::tmem_st16(tmem_state + lane_base + g * 16, v);
        if (owner) {
#pragma unroll
            for (int cc = 0; cc < 2; ++cc)
                sts128(s_tile + d_row * 128 + (((2 * g + cc) ^ (d_row & 7)) << 4),
                       sm100::pack_bf16x2(acc[cc * 8 + 0], acc[cc * 8 + 1]), sm100::pack_bf16x2(acc[cc * 8 + 2], acc[cc * 8 + 3]),
                       sm100::pack_bf16x2(acc[cc * 8 + 4], acc[cc * 8 + 5]), sm100::pack_bf16x2(acc[cc * 8 + 6], acc[cc * 8 + 7]));
        }
    }
    float z = __uint_as_float(sm100::tmem_ld1(tmem_state + lane_base + 64));
    sm100::tmem_ld_wait();
    z += z_given;
    uint32_t zz[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) zz[j] = (kForward || j == 0) ? __float_as_uint(z) : 0u;
    sm100::tmem_st16(tmem_state + lane_base + 64, zz);
    sm100::tmem_st_wait();
    if (owner) {
        if (kForward) z_row_store(z_tile, d_row, z); else r_out[d_row] = z;
    }
}

// The reverse-sweep state [R | r] of the accumulator to global memory ([dim][dim] and [dim] fp32): after the
// first chunk of a sequence it is the gradient of the state the sequence started from.  Out of line, called once.
static __device__ __noinline__ void rstate_write(uint32_t tmem_state, int quad, int lane, float* g_R, float* g_r, int dim) {
    const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
    const int d_row = quad * 16 + lane;
    const bool in_row = lane < 16 && d_row < dim;
    sm100::tc_fence_after_sync();
#pragma unroll 1
    for (int g = 0; g < 4; ++g) {
        uint32_t v[16];
        sm100::tmem_ld16(tmem_state + lane_base + g * 16, v);
        sm100::tmem_ld_wait();
        if (g_R && in_row && g * 16 < dim) {
#pragma unroll
            for (int j = 0; j < 16; ++j) g_R[d_row * dim + g * 16 + j] = __uint_as_float(v[j]);
        }
    }
    const float r0 = __uint_as_float(sm100::tmem_ld1(tmem_state + lane_base + 64));
    const float r1 = __uint_as_float(sm100::tmem_ld1(tmem_state + lane_base + 65));
    sm100::tmem_ld_wait();
    if (g_r && in_row) g_r[d_row] = r0 + r1;
}

// One 32-column block of fp32 scores -> 16 packed bf16 pairs (pair j = columns 2j, 2j+1), with
// the causal mask on the diagonal block; a block above the diagonal (`present` false) is zeros.
// One warp-uniform branch per block instead of per-element selects: a block off the
// diagonal costs sixteen conversions, an absent block none.  (The score warps of the quadrant with
// four present blocks set the pace of a chunk, and most of their blocks are off the diagonal.)
template <bool kTransposed>
__device__ __forceinline__ void score_block_round(const uint32_t (&v)[32], bool present, bool diagonal, int lane,
                                                  uint32_t (&packed)[16]) {
    if (!present) {
#pragma unroll
        for (int j = 0; j < 16; ++j) packed[j] = 0u;
    } else if (!diagonal) {
#pragma unroll
        for (int j = 0; j < 16; ++j) packed[j] = sm100::pack_bf16x2(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]));
    } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const bool drop0 = kTransposed ? 2 * j < lane : 2 * j > lane;
            const bool drop1 = kTransposed ? 2 * j + 1 < lane : 2 * j + 1 > lane;
            packed[j] = sm100::pack_bf16x2(drop0 ? 0.f : __uint_as_float(v[2 * j]), drop1 ? 0.f : __uint_as_float(v[2 * j + 1]));
        }
    }
}

// Reverse-sweep state [R | r]: r is carried as two columns (the dl column tile holds a bf16
// high and low part of dl_i in its columns 0 and 1), so r = column 64 + column 65.
// Accumulator (M = 64 layout) -> bf16 R tile + fp32 r.
__device__ __forceinline__ void rstate_to_smem(uint32_t tmem_state, int quad, int lane, uint8_t* s_tile, float* r_out) {
    const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
    const int d_row = quad * 16 + lane;
    const bool owner = lane < 16;
#pragma unroll 1
    for (int h = 0; h < 2; ++h) {
        uint32_t v[32];
        sm100::tmem_ld32(tmem_state + lane_base + h * 32, v);
        sm100::tmem_ld_wait();
        if (owner) state_row_store(s_tile, d_row, h, v);
    }
    const float r0 = __uint_as_float(sm100::tmem_ld1(tmem_state + lane_base + 64));
    const float r1 = __uint_as_float(sm100::tmem_ld1(tmem_state + lane_base + 65));
    sm100::tmem_ld_wait();
    if (owner) r_out[d_row] = r0 + r1;
}
// Initial [R | r] of a segment: the sum of the records of parts [part_lo, part_hi), or zeros.
// Sixteen columns at a time (rolled): this runs once per CTA and must not raise the register
// pressure of the role that calls it.
__device__ __forceinline__ void rstate_init(uint32_t tmem_state, int quad, int lane, uint8_t* s_tile, float* r_out,
                                            const float* rec, int part_lo, int part_hi) {
    const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
    const int d_row = quad * 16 + lane;
    const bool owner = lane < 16;
#pragma unroll 1
    for (int g = 0; g < 4; ++g) {
        float acc[16];
        sum_records16(rec, owner ? part_lo : 0, owner ? part_hi : 0, d_row * kDim + g * 16, acc);
        uint32_t v[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) v[j] = __float_as_uint(acc[j]);
        sm100::tmem_st16(tmem_state + lane_base + g * 16, v);
        if (owner) {
#pragma unroll
            for (int cc = 0; cc < 2; ++cc)
                sts128(s_tile + d_row * 128 + (((2 * g + cc) ^ (d_row & 7)) << 4),
                       sm100::pack_bf16x2(acc[cc * 8 + 0], acc[cc * 8 + 1]), sm100::pack_bf16x2(acc[cc * 8 + 2], acc[cc * 8 + 3]),
                       sm100::pack_bf16x2(acc[cc * 8 + 4], acc[cc * 8 + 5]), sm100::pack_bf16x2(acc[cc * 8 + 6], acc[cc * 8 + 7]));
        }
    }
    const float r = owner ? sum_records1(rec, part_lo, part_hi, kDim * kDim + d_row) : 0.f;
    uint32_t rr[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) rr[j] = j == 0 ? __float_as_uint(r) : 0u;      // all of r in column 64
    sm100::tmem_st16(tmem_state + lane_base + 64, rr);
    sm100::tmem_st_wait();
    if (owner) r_out[d_row] = r;
}

// One 128 x 128 score tile (fp32 in TMEM at `pb`, this thread's lane): wait for it, apply the
// causal mask, round to bf16 pairs in place, signal `ready`.  kTransposed: rows are keys and
// columns queries (keep query >= key), else rows are queries (keep key <= query).  The warp
// (quad, half) owns the 32-column blocks 2 half and 2 half + 1 of the quadrant's 32 rows; the bf16
// block j of a warp goes to columns 64 half + 16 j .. + 15, inside fp32 columns this thread has
// already read, so nothing another thread still needs is overwritten.
// Deliberately not inlined: every caller shares one copy, whose shape does not depend on what the
// compiler makes of the surrounding role loops (inlined, the same source ran up to 1.5x slower
// depending on unrelated statements nearby).
template <bool kTransposed>
__device__ __noinline__ bool round_score_tile(uint32_t pb, uint64_t* full, uint64_t* ready, uint32_t parity, int quad,
                                              int half, int lane, int* status) {
    if (!sm100::mbar_wait(full, parity, status, sm100::kStatusMmaTimeout)) return false;
    sm100::tc_fence_after_sync();
    // rolled over the warp's two blocks: this routine is on the critical path of a chunk and has to stay
    // resident in the instruction cache next to every other role's loop
#pragma unroll 1
    for (int b = 0; b < 2; ++b) {
        const int blk = 2 * half + b;
        const bool has = kTransposed ? blk >= quad : blk <= quad;
        uint32_t v[32], pk[16];
        if (has) {
            sm100::tmem_ld32(pb + blk * 32, v);
            sm100::tmem_ld_wait();
        }
        score_block_round<kTransposed>(v, has, blk == quad, lane, pk);
        sm100::tmem_st16(pb + half * 64 + b * 16, pk);
    }
    sm100::tmem_st_wait();
    sm100::tc_fence_before_sync();
    sm100::mbar_arrive(ready);
    return true;
}

// tcgen05.mma with the A operand read from TMEM (bf16 pairs: column j of lane i = A[i][2j], A[i][2j+1]).
__device__ __forceinline__ void umma_bf16_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// the same issued from a warp-wide loop by its elected lane (see umma_bf16(leader, ...))
__device__ __forceinline__ void umma_bf16_ta(bool leader, uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p, e;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "setp.ne.b32 e, %5, 0;\n\t"
        "@e tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"((uint32_t)leader)
        : "memory");
}

// Four tcgen05.mma over consecutive K groups of one product, issued from a warp-wide loop through its elected
// lane (see umma_bf16(leader, ...)): the low descriptor words advance by a_step / b_step per K group (2 for a
// K-major operand inside a 128-byte swizzle row, 128 for an MN-major operand whose K groups are 2 KB apart);
// the first one accumulates only if `acc_first`.  Inline: with the operands in uniform registers a product is a
// handful of instructions, and a call would move them back into vector registers (issued from a one-lane
// loop these groups were out of line, a dozen instructions per product).
__device__ __forceinline__ void umma_group4(bool leader, uint32_t d_tmem, uint32_t a_lo, uint32_t a_step, uint32_t b_lo,
                                            uint32_t b_step, uint32_t idesc, uint32_t acc_first) {
    const uint64_t hi = desc_k(0) & 0xFFFFFFFF00000000ull;
#pragma unroll
    for (uint32_t k = 0; k < 4; ++k)
        sm100::umma_bf16(leader, d_tmem, hi | (a_lo + k * a_step), hi | (b_lo + k * b_step), idesc, k > 0 ? 1u : acc_first);
}
__device__ __forceinline__ void umma_group4_ta(bool leader, uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_step,
                                               uint32_t idesc, uint32_t acc_first) {
    const uint64_t hi = desc_k(0) & 0xFFFFFFFF00000000ull;
#pragma unroll
    for (uint32_t k = 0; k < 4; ++k)
        umma_bf16_ta(leader, d_tmem, a_tmem + k * 8, hi | (b_lo + k * b_step), idesc, k > 0 ? 1u : acc_first);
}

}  // namespace tc
}  // namespace la
