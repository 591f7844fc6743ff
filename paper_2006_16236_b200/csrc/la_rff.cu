// Random Fourier features for the Gaussian kernel (the feature map the paper's conclusion proposes to explore;
// its Section 3.2.1 counts the cost of a feature map of dimension C as O(N C M)), in the paired form
//     phi(x) = sqrt(2 / C) [cos(W x), sin(W x)],   W [C/2, D] given by the caller,
// and the gradient with respect to x.  Both are a projection followed by an element-wise map, so both run on
// the tensor cores: per tile of 128 rows, z = x W^T is one tcgen05 product (A = the x tile, B = W, K-major,
// N = C/2, fp32 in TMEM); the forward pass turns z into cos / sin rows and stores the tile with TMA; the
// backward pass forms t = sqrt(2 / C) (-sin z * dy_cos + cos z * dy_sin) as a bf16 operand tile and issues a
// second product dx = t W, which reads the SAME W tile as an MN-major B operand (rows = the contraction).
// Persistent CTAs walk the row tiles; x (and dy) tiles arrive through a two-stage TMA ring, z is double
// buffered in TMEM, so the loads and the product of the next tile overlap the sin / cos of this one.
// Warps 0-3: per-row work (thread t = row t = TMEM lane t); warp 4: TMA; warp 5: MMA issue.
// Bound: HBM ((D + C) e bytes per row forward, (2 D + C) e backward); sin / cos go through the MUFU after a
// range reduction to [-pi, pi].
#include "la_tc.cuh"
#include "la_tc_common.cuh"

namespace la {
namespace tc {

using namespace sm100;

namespace {

constexpr int kRffThreads = 192;
template <bool kBackward, int kYTiles>            // kYTiles = C / 64: 64-column tiles of y / dy
struct RffLayout {
    static constexpr uint32_t kStageBytes = (kBackward ? 1 + kYTiles : 1) * kTileBytes;     // x tile (+ the dy tiles)
    static constexpr uint32_t kOffX = 0;                                        // 2 stages
    static constexpr uint32_t kOffW = kOffX + 2 * kStageBytes;                  // W tile [C/2 <= 64][64]
    static constexpr uint32_t kOffOut = kOffW + kDim * 128;                     // forward: the y tiles; backward: t, then dx
    static constexpr uint32_t kOffBar = kOffOut + (kBackward ? 1 : kYTiles) * kTileBytes;
    static constexpr uint32_t kSmemBytes = kOffBar + 256 + 1024;                // + slack for the 1 KB alignment of the base
};
constexpr uint32_t kRffColZ = 0, kRffColDx = 128;                   // TMEM: z double-buffered (2 x 64), dx 64

struct RffBarriers {
    uint64_t w_full, x_full[2], x_empty[2], z_full[2], z_free[2], t_ready, dx_full, dx_free;
    uint32_t tmem_base;
    int abort_flag;
};

struct RffParams {
    int* status;
    int ntiles;
    int half;           // C / 2: 32 or 64
    int dim;            // D
    float scale;        // sqrt(2 / C)
};

// sin and cos of z through the special-function unit after reducing z to [-pi, pi] (the fast instructions lose
// accuracy with |z|; the reduction costs one multiply-add and one rounding)
__device__ __forceinline__ void sincos_reduced(float z, float& s, float& c) {
    const float k = rintf(z * 0.15915494309189535f);
    float r = fmaf(k, -6.2831854820251465f, z);
    r = fmaf(k, 1.7484555e-7f, r);                                  // 2 pi = 6.2831854820251465 - 1.7484555e-7
    __sincosf(r, &s, &c);
}

template <bool kBackward, int kYTiles>
__global__ void __launch_bounds__(kRffThreads)
rff_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapW,
           const __grid_constant__ CUtensorMap mapY, const __grid_constant__ CUtensorMap mapDx, const RffParams prm) {
    using Lay = RffLayout<kBackward, kYTiles>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    RffBarriers* bars = reinterpret_cast<RffBarriers*>(smem + Lay::kOffBar);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr int half = 32 * kYTiles, ytiles = kYTiles;            // frequencies; 64-column tiles of y / dy
    const int mine = (prm.ntiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;      // tiles of this CTA
    constexpr uint32_t kTmemCols = kBackward ? 256 : 128;

    if (tid == 0) {
        mbar_init(&bars->w_full, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bars->x_full[s], 1);
            mbar_init(&bars->x_empty[s], kBackward ? 1 + 128 : 1);  // the product's commit (+ the rows that read dy)
            mbar_init(&bars->z_full[s], 1);
            mbar_init(&bars->z_free[s], 128);
        }
        mbar_init(&bars->t_ready, 128);
        mbar_init(&bars->dx_full, 1);
        mbar_init(&bars->dx_free, 128);
        bars->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 5) {
        __syncwarp();
        tmem_alloc(&bars->tmem_base, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = bars->tmem_base;
    volatile int* abort_flag = &bars->abort_flag;

    if (warp == 4) {
        if (lane == 0) {
            prefetch_tensormap(&mapX); prefetch_tensormap(&mapW); prefetch_tensormap(&mapY);
            if (kBackward) prefetch_tensormap(&mapDx);
            mbar_arrive_expect_tx(&bars->w_full, (uint32_t)half * 128);
            tma_load_2d(smem + Lay::kOffW, &mapW, 0, 0, &bars->w_full);          // columns past D read as zeros
            #pragma unroll 1
            for (int it = 0; it < mine; ++it) {
                const int s = it & 1;
                if (it >= 2 && !mbar_wait(&bars->x_empty[s], ((it >> 1) - 1) & 1, prm.status, kStatusPipeTimeout)) {
                    *abort_flag = 1;
                    break;
                }
                const int row = ((int)blockIdx.x + it * (int)gridDim.x) * kChunk;
                uint8_t* st = smem + Lay::kOffX + s * Lay::kStageBytes;
                mbar_arrive_expect_tx(&bars->x_full[s], kTileBytes * (kBackward ? 1 + ytiles : 1));
                tma_load_2d(st, &mapX, 0, row, &bars->x_full[s]);               // rows past the end read as zeros
                if (kBackward)
                    for (int j = 0; j < ytiles; ++j) tma_load_2d(st + (1 + j) * kTileBytes, &mapY, j * kDim, row, &bars->x_full[s]);
            }
        }
    } else if (warp == 5) {
        const bool leader = elect_one();
        const uint32_t idesc_z = umma_idesc_bf16(128, half, 0, 0);
        const uint32_t idesc_dx = umma_idesc_bf16(128, kDim, 0, 1);            // B = W, MN-major
        const uint32_t aW = sbase + Lay::kOffW, aT = sbase + Lay::kOffOut;
        bool ok = mbar_wait_warp(&bars->w_full, 0, prm.status, kStatusTmaTimeout);
        #pragma unroll 1
        for (int it = 0; it < mine && ok; ++it) {
            const int s = it & 1;
            ok = mbar_wait_warp(&bars->x_full[s], (it >> 1) & 1, prm.status, kStatusTmaTimeout);
            if (ok && it >= 2) ok = mbar_wait_warp(&bars->z_free[s], ((it >> 1) - 1) & 1, prm.status, kStatusPipeTimeout);
            if (!ok || __any_sync(0xFFFFFFFFu, *abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t aX = sbase + Lay::kOffX + s * Lay::kStageBytes;
#pragma unroll
            for (int k = 0; k < 4; ++k)         // z = x W^T (the K steps past D multiply zeros)
                umma_bf16(leader, tmem + kRffColZ + s * 64, desc_k(aX + 32 * k), desc_k(aW + 32 * k), idesc_z, k != 0);
            umma_commit(leader, &bars->z_full[s]);
            umma_commit(leader, &bars->x_empty[s]);
            if (kBackward) {
                ok = mbar_wait_warp(&bars->t_ready, it & 1, prm.status, kStatusPipeTimeout);
                if (ok && it >= 1) ok = mbar_wait_warp(&bars->dx_free, (it - 1) & 1, prm.status, kStatusPipeTimeout);
                if (!ok) break;
                tc_fence_after_sync();
                for (int k = 0; k < half / 16; ++k)         // dx = t W: 16 frequencies (rows of W) per step
                    umma_bf16(leader, tmem + kRffColDx, desc_k(aT + 32 * k), desc_mn(aW + 2048 * k), idesc_dx, k != 0);
                umma_commit(leader, &bars->dx_full);
            }
        }
        if (!ok) *abort_flag = 1;
    } else {
        // ---------------------------------------------------------------- rows: thread t owns row t of the tile
        const uint32_t r7 = tid & 7;
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        uint8_t* out = smem + Lay::kOffOut;
        bool ok = true;
        #pragma unroll 1
        for (int it = 0; it < mine && ok; ++it) {
            const int s = it & 1;
            const int row0 = ((int)blockIdx.x + it * (int)gridDim.x) * kChunk;
            if (!mbar_wait(&bars->z_full[s], (it >> 1) & 1, prm.status, kStatusMmaTimeout) ||
                (kBackward && !mbar_wait(&bars->x_full[s], (it >> 1) & 1, prm.status, kStatusTmaTimeout)) || *abort_flag) {
                ok = false;
                break;
            }
            tc_fence_after_sync();
            // the staging tiles still belong to the store of the tile before until it has been read
            if (tid == 0) tma_store_wait_read<0>();
            named_barrier(1, 128);
            const uint8_t* dy_row = smem + Lay::kOffX + s * Lay::kStageBytes + kTileBytes + tid * 128;
            #pragma unroll 1
            for (int g = 0; g < half / 32; ++g) {           // 32 frequencies at a time
                uint32_t v[32];
                tmem_ld32(tmem + lane_base + kRffColZ + s * 64 + g * 32, v);
                tmem_ld_wait();
                if (g == half / 32 - 1) {
                    tc_fence_before_sync();
                    mbar_arrive(&bars->z_free[s]);
                }
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {            // 8 frequencies = one 16-byte chunk of a bf16 row
                    float sn[8], cs[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) sincos_reduced(__uint_as_float(v[cc * 8 + j]), sn[j], cs[j]);
                    const int f0 = g * 32 + cc * 8;         // first frequency of the chunk
                    if (!kBackward) {
                        // cos at column f0, sin at column half + f0 of y
                        const int cc_cos = f0 >> 3, cc_sin = (half + f0) >> 3;
                        sts128(out + (cc_cos >> 3) * kTileBytes + tid * 128 + (((cc_cos & 7) ^ r7) << 4),
                               pack_bf16x2(prm.scale * cs[0], prm.scale * cs[1]), pack_bf16x2(prm.scale * cs[2], prm.scale * cs[3]),
                               pack_bf16x2(prm.scale * cs[4], prm.scale * cs[5]), pack_bf16x2(prm.scale * cs[6], prm.scale * cs[7]));
                        sts128(out + (cc_sin >> 3) * kTileBytes + tid * 128 + (((cc_sin & 7) ^ r7) << 4),
                               pack_bf16x2(prm.scale * sn[0], prm.scale * sn[1]), pack_bf16x2(prm.scale * sn[2], prm.scale * sn[3]),
                               pack_bf16x2(prm.scale * sn[4], prm.scale * sn[5]), pack_bf16x2(prm.scale * sn[6], prm.scale * sn[7]));
                    } else {
                        const int cc_cos = f0 >> 3, cc_sin = (half + f0) >> 3;
                        uint32_t dc[4], ds[4], t[4];
                        lds128(dy_row + (cc_cos >> 3) * kTileBytes + (((cc_cos & 7) ^ r7) << 4), dc);
                        lds128(dy_row + (cc_sin >> 3) * kTileBytes + (((cc_sin & 7) ^ r7) << 4), ds);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float t0 = prm.scale * fmaf(cs[2 * j], bf16_lo(ds[j]), -sn[2 * j] * bf16_lo(dc[j]));
                            const float t1 = prm.scale * fmaf(cs[2 * j + 1], bf16_hi(ds[j]), -sn[2 * j + 1] * bf16_hi(dc[j]));
                            t[j] = pack_bf16x2(t0, t1);
                        }
                        sts128(out + tid * 128 + (((f0 >> 3) ^ r7) << 4), t[0], t[1], t[2], t[3]);
                    }
                }
            }
            fence_proxy_async_smem();
            if (!kBackward) {
                named_barrier(1, 128);
                if (tid == 0) {
                    for (int j = 0; j < ytiles; ++j) tma_store_2d(&mapY, out + j * kTileBytes, j * kDim, row0);   // rows past the end are clipped
                    tma_store_commit();
                }
            } else {
                mbar_arrive(&bars->x_empty[s]);             // dy has been read
                tc_fence_before_sync();
                mbar_arrive(&bars->t_ready);
                if (!mbar_wait(&bars->dx_full, it & 1, prm.status, kStatusMmaTimeout)) { ok = false; break; }
                tc_fence_after_sync();
                // dx rows leave through the tile t came in (the product that read it is complete)
                #pragma unroll 1
                for (int g = 0; g < 2; ++g) {
                    uint32_t v[32];
                    tmem_ld32(tmem + lane_base + kRffColDx + g * 32, v);
                    tmem_ld_wait();
                    if (g == 1) {
                        tc_fence_before_sync();
                        mbar_arrive(&bars->dx_free);
                    }
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc)
                        sts128(out + tid * 128 + (((g * 4 + cc) ^ r7) << 4),
                               pack_bf16x2(__uint_as_float(v[cc * 8 + 0]), __uint_as_float(v[cc * 8 + 1])),
                               pack_bf16x2(__uint_as_float(v[cc * 8 + 2]), __uint_as_float(v[cc * 8 + 3])),
                               pack_bf16x2(__uint_as_float(v[cc * 8 + 4]), __uint_as_float(v[cc * 8 + 5])),
                               pack_bf16x2(__uint_as_float(v[cc * 8 + 6]), __uint_as_float(v[cc * 8 + 7])));
                }
                fence_proxy_async_smem();
                named_barrier(1, 128);
                if (tid == 0) {
                    tma_store_2d(&mapDx, out, 0, row0);     // columns past D and rows past the end are clipped
                    tma_store_commit();
                }
            }
        }
        if (tid == 0) tma_store_wait_all<0>();
        if (!ok) *abort_flag = 1;
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 5) {
        __syncwarp();
        tmem_dealloc(tmem, kTmemCols);
    }
}

template <bool kBackward, int kYTiles>
int launch_rff(const void* x, const void* W, const void* y, void* dx, int64_t rows, int D, int C, cudaStream_t st) {
    const int half = C / 2;
    CUtensorMap mX, mW, mY, mDx;
    if (int rc = encode_tile_map(&mX, x, (uint64_t)rows, kChunk, D)) return rc;
    if (int rc = encode_tile_map(&mW, W, (uint64_t)half, (uint32_t)half, D)) return rc;
    if (int rc = encode_tile_map(&mY, y, (uint64_t)rows, kChunk, C)) return rc;
    if (int rc = encode_tile_map(&mDx, kBackward ? dx : y, (uint64_t)rows, kChunk, kBackward ? D : C)) return rc;
    static std::atomic<uint64_t> attr_done{0};
    constexpr uint32_t kSmem = RffLayout<kBackward, kYTiles>::kSmemBytes;
    if (int rc = opt_in_smem_once(rff_kernel<kBackward, kYTiles>, kSmem, attr_done)) return rc;
    RffParams prm;
    prm.status = device_status_ptr();
    if (!prm.status) return fail(LA_ERR_CUDA, "device status word unavailable");
    prm.ntiles = (int)((rows + kChunk - 1) / kChunk);
    prm.half = half;
    prm.dim = D;
    prm.scale = sqrtf(2.0f / (float)C);
    // several CTAs share an SM where shared memory and TMEM (128 columns forward, 256 backward) allow it; inside
    // a CTA the two-stage ring and the double-buffered accumulator overlap the loads and the product of the
    // next tile with the per-row work of this one
    constexpr int kPerSm = kBackward ? (kSmem <= 100 * 1024 ? 2 : 1) : (kSmem <= 74 * 1024 ? 3 : 2);
    const int slots = sm_count() * kPerSm;
    const int grid = prm.ntiles < slots ? prm.ntiles : slots;
    rff_kernel<kBackward, kYTiles><<<grid, kRffThreads, kSmem, st>>>(mX, mW, mY, mDx, prm);
    LA_CUDA_TRY(cudaGetLastError());
    note_launch();
    return LA_OK;
}

}  // namespace

bool rff_supported(int64_t rows, int64_t D, int64_t C, int dtype) {
    return dtype == LA_BF16 && D >= 8 && D <= 64 && D % 8 == 0 && (C == 64 || C == 128) && rows >= 1 && rows < (1LL << 31);
}

int rff_forward(const void* x, const void* W, void* y, int64_t rows, int D, int C, cudaStream_t st) {
    return C == 64 ? launch_rff<false, 1>(x, W, y, nullptr, rows, D, C, st) : launch_rff<false, 2>(x, W, y, nullptr, rows, D, C, st);
}

int rff_backward(const void* x, const void* W, const void* dy, void* dx, int64_t rows, int D, int C, cudaStream_t st) {
    return C == 64 ? launch_rff<true, 1>(x, W, dy, dx, rows, D, C, st) : launch_rff<true, 2>(x, W, dy, dx, rows, D, C, st);
}

}  // namespace tc
}  // namespace la
