// Split-precision tensor-core form of tensor times matrix with packed input and output (opt-in, its
// own entry point).
//
// A(i,j,k) = sum_l B(i,j,l) C(k,l) over a structure whose trailing index is dense (the running example
// of Section 3 over the upper half cube): the ranking polynomial keeps the trailing index contiguous,
// so in packed form the rule is the dense product Y[p][k] = sum_l X[p][l] C[k][l] of the packed
// input, viewed as a [rows][Q] matrix, with C (ttm.cu).  Here it runs on the tensor cores in TF32
// with both operands split into a high and a low part (tf32_mma.cuh):
//     X C^T ~ Xhi Chi^T + Xhi Clo^T + Xlo Chi^T,   fp32 accumulation in tensor memory.
// A row of X is its own K-major operand row: a block of 128 rows x 32 l arrives by one bulk tensor copy
// in the 128-byte swizzle and serves as Xhi as it is (the tensor core reads only the upper 19 bits of
// a value); producer warps write Xlo = X - trunc(X) beside it.
//
// Tile = 128 packed rows x 32 output columns, l in blocks of 32.
//   loader thread    waits for a free stage and starts the copy of the next block of X
//   producer warps   three groups of four, taking the blocks in turn: wait for the copy, write Xlo
//   MMA threads      four, taking the tiles in turn (one accumulator each: issuing the eight small MMAs
//                    of a tile costs a thread more than a thousand cycles); per block and k-step of 8: tcgen05.mma kind::tf32 M128 N64 K8 with A = X,
//                    B = [Chi ; Clo] (columns 0..31 get Xhi Chi, 32..63 get Xhi Clo), and M128 N32 K8
//                    with A = Xlo, B = Chi into columns 0..31
//   epilogue warps   two sets of four, one per accumulator (the proxy fence before a bulk store
//                    costs about a thousand cycles): tcgen05.ld of both halves, their sum leaves as a 32 x 32 chunk through shared
//                    memory by a bulk tensor store (reduce-add when accumulating; plain stores when
//                    the rows of Y are not 16-byte aligned)
// C is staged once per CTA as hi / lo K-major tiles (8 KiB per block of l, Q <= 256).  Four
// accumulators of 64 columns in tensor memory, one per MMA issuer.  Every wait is bounded.
#include <cuda.h>

#include <cstring>

#include "common.cuh"
#include "tf32_mma.cuh"
#include "waits.cuh"

namespace dastac {
namespace {

constexpr int kTtRows = 128;                 // packed rows per tile
constexpr int kTtCols = 32;                  // output columns per tile
constexpr int kTtTile = kTtRows * 128;       // 16 KiB: 128 x 32 fp32
constexpr int kTtStageBytes = 2 * kTtTile;   // X (= Xhi), Xlo
constexpr int kTtCBlock = 2 * kTtCols * 128; // 8 KiB: [Chi ; Clo] of one block of l
constexpr int kTtMaxQBlocks = 8;
constexpr int kTtMaxStages = 6;
// warps 0-7 epilogue (two sets of four: set e drains accumulator e, i.e. every second tile), 8-9 MMA
// (issuer e fills accumulator e: the eight small MMAs of a tile cost one thread more than a thousand
// cycles to issue), 10 loader, 11.. low parts (three groups of four, taking the blocks in turn)
constexpr int kTtEpiSets = 2, kTtEpiWarps = 4 * kTtEpiSets, kTtWarpMma = 8, kTtMmaWarps = 4, kTtWarpLoad = 12, kTtWarpLo0 = 13;
constexpr int kTtLoWarps = 4, kTtLoGroups = 3;
constexpr int kTtThreads = (kTtWarpLo0 + kTtLoWarps * kTtLoGroups) * 32;
constexpr int kTtAccs = kTtMmaWarps;         // accumulators of 64 columns, one per issuer
constexpr int kTtTmemCols = 64 * kTtAccs;
constexpr int kTtEpiBufBytes = 32 * 128;
constexpr int kTtEpiBytes = kTtEpiWarps * kTtEpiBufBytes;  // one buffer per epilogue warp
constexpr long long kTtWaitBudget = 2000000000LL;
constexpr int32_t kErrWordTtmTc = 0x5454;    // "TT"

struct TtParams {
    const float* C;
    float* Y;
    int64_t P, Q, K, ldc;
    int32_t q_blocks, stages, row_tiles, col_tiles;
    int64_t tiles;
    int32_t accumulate, tma_y, vec_y;
    int32_t* err_word;
};

// `site` (1..5) is added to the code so that the word tells which wait ran out
__device__ __forceinline__ bool tt_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* err_word, int site = 0) {
    return tc_wait_coded(bar, parity, abort_flag, err_word, kErrWordTtmTc + (site << 16), kTtWaitBudget);
}

__global__ void __launch_bounds__(kTtThreads, 1)
ttm_tc_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_y, const TtParams p) {
    extern __shared__ uint8_t tt_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(tt_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int S = p.stages;
    uint8_t* const Cb = smem;                                         // q_blocks x [Chi ; Clo]
    uint8_t* const stage0 = Cb + (size_t)p.q_blocks * kTtCBlock;      // S x (X, Xlo)
    uint8_t* const epi0 = stage0 + (size_t)S * kTtStageBytes;
    uint64_t* const bars = reinterpret_cast<uint64_t*>(epi0 + kTtEpiBytes);
    auto raw = [&](int s) { return tc_smem(&bars[s]); };
    auto full = [&](int s) { return tc_smem(&bars[kTtMaxStages + s]); };
    auto empty = [&](int s) { return tc_smem(&bars[2 * kTtMaxStages + s]); };
    auto tmem_full = [&](int a) { return tc_smem(&bars[3 * kTtMaxStages + a]); };
    auto tmem_empty = [&](int a) { return tc_smem(&bars[3 * kTtMaxStages + kTtAccs + a]); };
    uint32_t* const tmem_slot = reinterpret_cast<uint32_t*>(&bars[3 * kTtMaxStages + 2 * kTtAccs]);
    volatile int* const abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            tc_mbar_init(raw(s), 1);
            tc_mbar_init(full(s), kTtLoWarps);
            tc_mbar_init(empty(s), 1);
        }
        for (int a = 0; a < kTtAccs; ++a) {
            tc_mbar_init(tmem_full(a), 1);
            tc_mbar_init(tmem_empty(a), 4);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc_smem(tmem_slot)),
                     "r"((uint32_t)kTtTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // C(k0 .. k0+31, :) as hi / lo K-major tiles: element (k, l) -> block l / 32, rows k (hi) and 32 + k (lo)
    const int64_t k0 = (int64_t)blockIdx.y * kTtCols;
    for (int idx = threadIdx.x; idx < p.q_blocks * 32 * 32; idx += blockDim.x) {
        const int l = idx & 31, k = (idx >> 5) & 31, qb = idx >> 10;
        const int64_t lg = 32 * (int64_t)qb + l;
        const float v = (k0 + k < p.K && lg < p.Q) ? __ldg(p.C + (k0 + k) * p.ldc + lg) : 0.f;
        float hi, lo;
        tc_split(v, hi, lo);
        uint8_t* const blk = Cb + (size_t)qb * kTtCBlock;
        *reinterpret_cast<float*>(blk + tc_tile_offset(k, l >> 2) + (l & 3) * 4) = hi;
        *reinterpret_cast<float*>(blk + tc_tile_offset(32 + k, l >> 2) + (l & 3) * 4) = lo;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    // this CTA's row tiles: blockIdx.x, blockIdx.x + gridDim.x, ...; one item per (row tile, block of l)
    const int G = gridDim.x;
    const int64_t my_tiles = p.row_tiles > (int64_t)blockIdx.x ? (p.row_tiles - blockIdx.x + G - 1) / G : 0;
    const int64_t items = my_tiles * p.q_blocks;

    if (warp == kTtWarpLoad) {
        // ---- loader: one thread ----
        if (lane == 0) {
            for (int64_t it = 0; it < items; ++it) {
                const int s = (int)(it % S);
                if (it >= S && !tt_wait(empty(s), (uint32_t)(((it / S) - 1) & 1), abort_flag, p.err_word, 1)) break;
                const int64_t tile = blockIdx.x + (it / p.q_blocks) * G;
                const int qb = (int)(it % p.q_blocks);
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(raw(s)), "r"((uint32_t)kTtTile) : "memory");
                asm volatile(
                    "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                    ::"r"(tc_smem(stage0 + (size_t)s * kTtStageBytes)), "l"(&tmap_x), "r"(32 * qb), "r"((int)(tile * kTtRows)),
                      "r"(raw(s))
                    : "memory");
            }
        }
    } else if (warp >= kTtWarpLo0) {
        // ---- low parts: group g takes the items g, g + 2, ...; thread = four 16-byte pieces of the block ----
        const int grp = (warp - kTtWarpLo0) / kTtLoWarps, t = ((warp - kTtWarpLo0) % kTtLoWarps) * 32 + lane;
        for (int64_t it = grp; it < items; it += kTtLoGroups) {
            const int s = (int)(it % S);
            bool ok = true;
            if (lane == 0) ok = tt_wait(raw(s), (uint32_t)((it / S) & 1), abort_flag, p.err_word, 2);
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            uint8_t* const x = stage0 + (size_t)s * kTtStageBytes;
            constexpr int kPer = kTtTile / (16 * kTtLoWarps * 32);
            float4 v[kPer];
#pragma unroll
            for (int u = 0; u < kPer; ++u) v[u] = *reinterpret_cast<const float4*>(x + (size_t)(u * kTtLoWarps * 32 + t) * 16);
#pragma unroll
            for (int u = 0; u < kPer; ++u) {
                float4 h, l;
                tc_split(v[u].x, h.x, l.x), tc_split(v[u].y, h.y, l.y), tc_split(v[u].z, h.z, l.z), tc_split(v[u].w, h.w, l.w);
                *reinterpret_cast<float4*>(x + kTtTile + (size_t)(u * kTtLoWarps * 32 + t) * 16) = l;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) tc_mbar_arrive(full(s));
        }
    }
    else if (warp >= kTtWarpMma && warp < kTtWarpMma + kTtMmaWarps) {
        // ---- MMA issuers: one thread per accumulator, taking the tiles in turn ----
        if (lane == 0) {
            constexpr uint32_t kIdesc64 = tc_idesc_mn(kTtRows, 64), kIdesc32 = tc_idesc_mn(kTtRows, 32);
            const int me = warp - kTtWarpMma;
            bool ok = true;
            for (int64_t tile_n = me; tile_n < my_tiles && ok; tile_n += kTtMmaWarps) {
                int64_t it = tile_n * p.q_blocks;
                const int acc = me;
                const int64_t use = tile_n / kTtMmaWarps;  // earlier uses of this accumulator
                if (use >= 1 && !tt_wait(tmem_empty(acc), (uint32_t)((use - 1) & 1), abort_flag, p.err_word, 3)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem_base + acc * 64;
                for (int qb = 0; qb < p.q_blocks; ++qb, ++it) {
                    const int s = (int)(it % S);
                    if (!tt_wait(full(s), (uint32_t)((it / S) & 1), abort_flag, p.err_word, 4)) {
                        ok = false;
                        break;
                    }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t x_hi = tc_smem(stage0 + (size_t)s * kTtStageBytes), x_lo = x_hi + kTtTile;
                    const uint32_t c_blk = tc_smem(Cb + (size_t)qb * kTtCBlock);
#pragma unroll
                    for (int k8 = 0; k8 < 4; ++k8)  // X [Chi ; Clo] -> columns 0..63
                        tc_mma_tf32(d_tmem, tc_desc(x_hi + k8 * 32), tc_desc(c_blk + k8 * 32), kIdesc64, (qb > 0 || k8 > 0) ? 1u : 0u);
#pragma unroll
                    for (int k8 = 0; k8 < 4; ++k8)  // Xlo Chi -> columns 0..31
                        tc_mma_tf32(d_tmem, tc_desc(x_lo + k8 * 32), tc_desc(c_blk + k8 * 32), kIdesc32, 1u);
                    tc_commit(empty(s));
                }
                if (ok) tc_commit(tmem_full(acc));
            }
        }
    } else if (warp < kTtEpiWarps) {
        // ---- epilogue: warp = lane quarter of tensor memory, thread = packed row ----
        const int set = warp >> 2, quarter = warp & 3;
        for (int64_t tile_n = set; tile_n < my_tiles; tile_n += kTtEpiSets) {
            const int64_t p0 = (blockIdx.x + tile_n * G) * kTtRows + quarter * 32;
            const int acc = (int)(tile_n % kTtAccs);
            const int64_t use = tile_n / kTtAccs;
            int got = 1;
            if (lane == 0) got = tt_wait(tmem_full(acc), (uint32_t)(use & 1), abort_flag, p.err_word, 5) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (!got) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * 64;
            uint32_t d0[32], d1[32];
            tc_ld32(taddr, d0);
            tc_ld32(taddr + 32, d1);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) tc_mbar_arrive(tmem_empty(acc));  // the accumulator may be overwritten
            float o[32];
#pragma unroll
            for (int v = 0; v < 32; ++v) o[v] = __uint_as_float(d0[v]) + __uint_as_float(d1[v]);
            if (p.tma_y) {
                uint8_t* const buf = epi0 + (size_t)warp * kTtEpiBufBytes;
                if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // its last store has read it
                __syncwarp();
#pragma unroll
                for (int v = 0; v < 8; ++v)
                    *reinterpret_cast<float4*>(buf + lane * 128 + ((v ^ (lane & 7)) << 4)) =
                        make_float4(o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3]);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0 && p0 < p.P) {
                    if (p.accumulate)
                        asm volatile(
                            "cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
                            ::"l"(&tmap_y), "r"((int)k0), "r"((int)p0), "r"(tc_smem(buf))
                            : "memory");
                    else
                        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
                                     ::"l"(&tmap_y), "r"((int)k0), "r"((int)p0), "r"(tc_smem(buf))
                                     : "memory");
                }
                if (lane == 0) asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            } else {
                const int64_t row = p0 + lane;
                if (row < p.P) {
                    float* dst = p.Y + row * p.K + k0;
#pragma unroll
                    for (int v = 0; v < 32; ++v)
                        if (k0 + v < p.K) dst[v] = p.accumulate ? dst[v] + o[v] : o[v];
                }
            }
        }
        // shared memory stays allocated until the bulk stores have read it and written Y
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTtTmemCols) : "memory");
    }
}

typedef CUresult (*TtEncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

TtEncodeTiledFn tt_encode_fn() {
    static TtEncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (TtEncodeTiledFn)ptr;
    }
    return fn;
}

// a [rows][cols] fp32 matrix with contiguous rows as a tensor of (box_cols x box_rows) boxes, 128-byte swizzle
bool tt_encode(CUtensorMap* map, const float* base, int64_t rows, int64_t cols, uint32_t box_cols, uint32_t box_rows) {
    TtEncodeTiledFn enc = tt_encode_fn();
    if (!enc) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 4};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace
}  // namespace dastac

using namespace dastac;

extern "C" dastac_status dastac_ttm_split_tf32(const dastac_structure* s, const float* X, const float* C, int64_t ldc,
                                               int64_t K, float* Y, int32_t accumulate, int32_t* err_word, void* stream) {
    if (!s || K < 0) return DASTAC_ERR_INVALID_ARG;
    const IndexMap& m = s->map;
    if (m.kind == kEmpty || K == 0) return DASTAC_OK;
    const bool trailing_dense = m.rank == 3 && (m.kind == kUpper || m.kind == kDense || (m.kind == kPlane && m.w != 2) ||
                                                (m.kind == kTetrahedron && m.dims[0] == 1));
    if (!trailing_dense) return DASTAC_ERR_UNSUPPORTED_EXPR;
    const int64_t Q = m.dims[2];
    if (Q <= 0 || m.count == 0) return DASTAC_OK;
    const int64_t P = m.count / Q;
    if (!X || !C || !Y || ldc < Q) return DASTAC_ERR_INVALID_ARG;
    // a row of the packed input must be a row of a tensor map: 16-byte pitch and base
    if ((Q & 3) != 0 || !aligned16(X)) return DASTAC_ERR_ALIGNMENT;
    if (Q > 32 * kTtMaxQBlocks || P >= ((int64_t)1 << 31) || K >= ((int64_t)1 << 31)) return DASTAC_ERR_UNSUPPORTED_EXPR;
    TtParams p;
    p.C = C, p.Y = Y, p.P = P, p.Q = Q, p.K = K, p.ldc = ldc;
    p.q_blocks = (int32_t)((Q + 31) / 32);
    p.row_tiles = (int32_t)((P + kTtRows - 1) / kTtRows);
    p.col_tiles = (int32_t)((K + kTtCols - 1) / kTtCols);
    if (p.col_tiles > 65535) return DASTAC_ERR_OVERFLOW;
    p.tiles = (int64_t)p.row_tiles * p.col_tiles;
    p.accumulate = accumulate;
    p.err_word = err_word;
    const size_t fixed = (size_t)p.q_blocks * kTtCBlock + kTtEpiBytes + 1024 /*alignment*/ + 256 /*barriers*/;
    int stages = (int)((227 * 1024 - fixed) / kTtStageBytes);
    if (stages > kTtMaxStages) stages = kTtMaxStages;
    if (stages < 2) return DASTAC_ERR_UNSUPPORTED_EXPR;
    p.stages = stages;
    const size_t smem = fixed + (size_t)stages * kTtStageBytes;
    CUtensorMap tmap_x, tmap_y;
    std::memset(&tmap_y, 0, sizeof(tmap_y));
    if (!tt_encode(&tmap_x, X, P, Q, 32, kTtRows)) return DASTAC_ERR_CUDA;
    p.tma_y = ((K & 3) == 0) && aligned16(Y);
    p.vec_y = p.tma_y;
    if (p.tma_y && !tt_encode(&tmap_y, Y, P, K, 32, 32)) return DASTAC_ERR_CUDA;
    static bool attr_set[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        if (cudaFuncSetAttribute(ttm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess)
            return DASTAC_ERR_CUDA;
        attr_set[dev] = true;
    }
    int gx = sm_count() / p.col_tiles;
    if (gx < 1) gx = 1;
    if (gx > p.row_tiles) gx = p.row_tiles;
    ttm_tc_kernel<<<dim3((unsigned)gx, (unsigned)p.col_tiles), kTtThreads, smem, (cudaStream_t)stream>>>(tmap_x, tmap_y, p);
    return launch_status();
}
