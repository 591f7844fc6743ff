// Tensor-core kernels: which problems they take, workspace sizes, tensor-map encoding.
#include <stdlib.h>

#include "la_tc.cuh"
#include "la_tc_common.cuh"

namespace la {

namespace tc {

static std::atomic<int> g_override_pieces{-1}, g_override_short{-1}, g_override_splits{-1};

PlanOverride plan_override() {
    return PlanOverride{g_override_pieces.load(std::memory_order_relaxed), g_override_short.load(std::memory_order_relaxed),
                        g_override_splits.load(std::memory_order_relaxed)};
}
void set_plan_override(int pieces, int short_len, int splits) {
    g_override_pieces.store(pieces, std::memory_order_relaxed);
    g_override_short.store(short_len, std::memory_order_relaxed);
    g_override_splits.store(splits, std::memory_order_relaxed);
}

int sm_count() {
    static thread_local int cached_dev = -1, cached_sms = 148;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();         // no device: not an error of the caller's
        return 148;
    }
    if (dev != cached_dev) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
            cudaGetLastError();
            return 148;
        }
        cached_dev = dev;
        cached_sms = n;
    }
    return cached_sms;
}

// Encoding a tensor map is a driver call of a microsecond or two and a training loop passes the same few
// tensors again and again: the last maps of the calling thread are kept, keyed by everything that goes in.
namespace {
struct MapKey {
    const void* base;
    uint64_t rows;          // 2-D map: rows in all; 3-D map: positions per sequence
    uint64_t seqs;          // 3-D map: sequences; 0 for a 2-D map
    uint32_t box_rows;
    int cols, dev;
    bool operator==(const MapKey& o) const {
        return base == o.base && rows == o.rows && seqs == o.seqs && box_rows == o.box_rows && cols == o.cols && dev == o.dev;
    }
};
constexpr int kMapCache = 32;
struct MapCache {
    MapKey key[kMapCache];
    CUtensorMap map[kMapCache];
    bool used[kMapCache];
    int next;
};
thread_local MapCache g_maps = {};
}  // namespace

static int encode_tile_map_uncached(CUtensorMap* map, const void* base, uint64_t seqs, uint64_t rows, uint32_t box_rows, int cols);

static int encode_cached(CUtensorMap* map, const void* base, uint64_t seqs, uint64_t rows, uint32_t box_rows, int cols) {
    int dev = 0;
    LA_CUDA_TRY(cudaGetDevice(&dev));
    const MapKey key{base, rows, seqs, box_rows, cols, dev};
    for (int i = 0; i < kMapCache; ++i)
        if (g_maps.used[i] && g_maps.key[i] == key) {
            *map = g_maps.map[i];
            return LA_OK;
        }
    if (int rc = encode_tile_map_uncached(map, base, seqs, rows, box_rows, cols)) return rc;
    const int slot = g_maps.next;
    g_maps.next = (slot + 1) % kMapCache;
    g_maps.key[slot] = key;
    g_maps.map[slot] = *map;
    g_maps.used[slot] = true;
    return LA_OK;
}

int encode_tile_map(CUtensorMap* map, const void* base, uint64_t rows, uint32_t box_rows, int cols) {
    return encode_cached(map, base, 0, rows, box_rows, cols);
}
int encode_seq_tile_map(CUtensorMap* map, const void* base, uint64_t seqs, uint64_t n, uint32_t box_rows, int cols) {
    return encode_cached(map, base, seqs, n, box_rows, cols);
}

// seqs == 0: a 2-D map over [rows][cols]; otherwise a 3-D map over [seqs][rows][cols] whose boxes hold rows of one
// sequence only (a box that reaches past a sequence's end is filled with zeros on a load and clipped on a store)
static int encode_tile_map_uncached(CUtensorMap* map, const void* base, uint64_t seqs, uint64_t rows, uint32_t box_rows, int cols) {
    static PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        LA_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
        if (qres != cudaDriverEntryPointSuccess || !fn)
            return fail(LA_ERR_CUDA, "the driver does not export cuTensorMapEncodeTiled");
        encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
    }
    const cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)seqs};
    const cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)cols * 2 * rows};
    const cuuint32_t box[3] = {(cuuint32_t)kDim, box_rows, 1};
    const cuuint32_t elem_strides[3] = {1, 1, 1};
    const CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, seqs ? 3 : 2, const_cast<void*>(base), dims, strides, box,
                              elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(LA_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
    return LA_OK;
}

}  // namespace tc

bool tc_supported(const la_problem& p, int op) {
    static const bool disabled = getenv("LA_DISABLE_TC") != nullptr;
    if (disabled) return false;
    if (p.dtype != LA_BF16 || p.D != p.M || (p.D != 32 && p.D != 64)) return false;
    if (p.N < 1) return false;      // any length: a last chunk that is not full is handled as padding
    if (p.B * p.H * p.N >= (1LL << 31)) return false;          // TMA coordinates are 32-bit
    return op >= LA_OP_LINEAR_FORWARD && op <= LA_OP_CAUSAL_BACKWARD;
}

size_t tc_workspace_bytes(const la_problem& p, int op) {
    switch (op) {
        case LA_OP_LINEAR_FORWARD: return tc::linear_forward_workspace(p);
        case LA_OP_LINEAR_BACKWARD: return tc::linear_backward_workspace(p);
        case LA_OP_CAUSAL_FORWARD: return tc::causal_forward_workspace(p);
        case LA_OP_CAUSAL_BACKWARD: return tc::causal_backward_workspace(p);
        default: return 0;
    }
}

int tc_causal_plan(const la_problem& p, int32_t* out, int capacity) {
    const tc::CausalPlan pl = tc::choose_plan(p);
    const int np = pl.npieces(), nq = pl.nparts();
    int n = 0;
    auto put = [&](int v) {
        if (out && n < capacity) out[n] = v;
        ++n;
    };
    put(np);
    put(nq);
    for (int k = 0; k <= np; ++k) put(pl.piece_begin(k));
    for (int k = 0; k <= np; ++k) put(pl.piece_first_part(k));
    for (int q = 0; q <= nq; ++q) put(pl.part_begin(q));
    for (int s = 0; s < np; ++s) put(pl.piece_of_slot(s));
    return n;
}
}  // namespace la
