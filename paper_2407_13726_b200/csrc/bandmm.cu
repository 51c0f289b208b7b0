// C = A B for a banded A (|i - j| <= w), B and C dense row-major, fp32.  A is stored as 2w+1 padded
// diagonals of N slots (described below), or packed exactly, row after row (then the band slice of a
// row tile is gathered by the threads at rowbase(i) + j, everything else is the same).  Slot (d, i) holds A(i, i + d - w): for a fixed diagonal consecutive rows are
// consecutive in memory and the position is the affine map d*N + i.  Padding slots are never read
// into a result: a slot whose column i + d - w falls outside [0, N) is replaced by zero while the
// band is staged, whatever it contains.
//
// A CTA (4 warps) computes 64 rows x 64 columns, walking the diagonals in chunks of at most 72.  Per chunk
//   - its slice of the band (the chunk's diagonals of its 64 rows) is staged in shared memory in the
//     packed layout itself, Ad[d][row]: the [2w+1][N] diagonal array is a 2-D tensor, so the slice
//     is one TMA box (coalesced loads along each diagonal when N*4 is not a multiple of 16 bytes);
//     padding slots only occur in the first and last row tiles and are zeroed there after the copy;
//   - the B rows the chunk touches (rows i0+dc-w .. , 64 columns) arrive in shared memory through
//     one TMA box; rows and columns outside B are zero-filled by the copy, so edge tiles need no
//     special case.  (A B whose base or row pitch is not 16-byte aligned cannot be described by a
//     tensor map; it is read with guarded loads through L1 instead.)
// A lane owns 8 rows x 4 columns.  For diagonal d its eight rows need B rows i+d-w .. i+7+d-w, a
// window that slides down by one row per diagonal: each step loads the eight A values (two
// broadcast 128-bit shared loads) and one new B row segment (one 128-bit shared load) and issues 32
// multiply-adds as 16 packed fp32x2 instructions.  The window lives in registers and rotates with
// period 8; the loop is unrolled by 8 so every register index is static, with a guarded copy of the body for
// the last 1..7 diagonals.  Only the band is visited.
#include <cuda.h>

#include <cstring>

#include "common.cuh"

namespace dastac {
namespace {

constexpr int kRows = 64, kThreads = 128;
constexpr int kPairs = 2;               // column pairs per lane: a lane owns 8 rows x 2*kPairs columns
constexpr int kLaneCols = 2 * kPairs;
constexpr int kCols = 16 * kLaneCols;   // 64 columns per CTA
constexpr int kChunk = 72;              // diagonals per chunk (multiple of 8)
constexpr int kPitchExact = 68;         // words per staged diagonal of the exact layout (68 = 4 mod 32, 16-byte rows)
constexpr int kBRows = kRows + kChunk + 6;  // B rows a chunk touches: 64 + chunk - 1 + 7
constexpr long long kWaitBudget = 4000000000LL;

// Two fp32 multiply-adds per instruction (packed pair in a 64-bit register): d = a * b + d.
typedef unsigned long long pair_t;
__device__ __forceinline__ pair_t pack2(float lo, float hi) {
    pair_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(pair_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ void fma2(pair_t& d, pair_t a, pair_t b) {
    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(a), "l"(b));
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// One new row segment of the window.  TMA_B: from the staged box; otherwise guarded global loads.
template <bool TMA_B>
__device__ __forceinline__ void load_row(pair_t (&dst)[kPairs], const float* __restrict__ Bs, int bs_row,
                                         const float* __restrict__ B, int64_t ldb, int64_t jj, int64_t N,
                                         int64_t c0, int cl, int64_t ncols) {
    if (TMA_B) {
        const ulonglong2 v = *reinterpret_cast<const ulonglong2*>(Bs + bs_row * kCols + cl);
        dst[0] = v.x;
        dst[1] = v.y;
    } else {
        if (jj < 0 || jj >= N) {
            dst[0] = dst[1] = 0ull;
            return;
        }
        const float* src = B + jj * ldb + c0;
#pragma unroll
        for (int e = 0; e < kPairs; ++e)
            dst[e] = pack2((c0 + 2 * e < ncols) ? __ldg(src + 2 * e) : 0.f,
                           (c0 + 2 * e + 1 < ncols) ? __ldg(src + 2 * e + 1) : 0.f);
    }
}

// EXACT: A is packed row after row (no padding); its slice is staged with a row pitch of 68 words so
// that the transposing stores below spread over all banks.
template <bool TMA_B, bool EXACT>
__global__ void __launch_bounds__(kThreads, 4)
bandmm_kernel(const __grid_constant__ CUtensorMap tmap_b, const __grid_constant__ CUtensorMap tmap_a, int tma_a,
              int64_t N, int64_t w, int64_t row_tile0,
              const float* __restrict__ A, const float* __restrict__ B, int64_t ldb, float* __restrict__ C,
              int64_t ldc, int64_t ncols, int accumulate, int vec_c, int32_t* err_word) {
    extern __shared__ __align__(128) uint8_t smem_raw[];
    float* Bs = reinterpret_cast<float*>(smem_raw);                                   // [kBRows][kCols]
    float* Ad = reinterpret_cast<float*>(smem_raw + (TMA_B ? kBRows * kCols * 4 : 0));  // [kChunk][kPitch]
    constexpr int kPitch = EXACT ? kPitchExact : kRows;
    __shared__ __align__(8) uint64_t bar;
    __shared__ int failed;

    const int64_t i0 = (row_tile0 + blockIdx.y) * (int64_t)kRows;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // warp = 16-row pair; lane = (8-row group, 4-column group)
    const int il = 16 * warp + 8 * (lane >> 4);
    const int cl = kLaneCols * (lane & 15);
    const int64_t cb = blockIdx.x * (int64_t)kCols, c0 = cb + cl;
    const int64_t i_f = i0 + il;
    const int64_t diagonals = 2 * w + 1;

    if (TMA_B && tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        failed = 0;
    }

    pair_t acc2[8][kPairs];  // [row][pair of columns]
#pragma unroll
    for (int q = 0; q < 8; ++q)
#pragma unroll
        for (int e = 0; e < kPairs; ++e) acc2[q][e] = 0ull;

    uint32_t phase = 0;
    for (int64_t dc = 0; dc < diagonals; dc += kChunk) {
        __syncthreads();  // previous chunk's readers are done with Ad and Bs
        const int64_t row0 = i0 + dc - w;  // first B row of the chunk (may be negative: zero-filled)
        if (TMA_B && tid == 0) {
            // order the generic-proxy reads of the previous chunk before the async-proxy overwrite
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            const uint32_t bytes = (uint32_t)(kBRows * kCols * 4) + (tma_a ? (uint32_t)(kChunk * kRows * 4) : 0u);
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(&bar)), "r"(bytes)
                         : "memory");
            asm volatile(
                "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                ::"r"(smem_u32(Bs)), "l"(&tmap_b), "r"((int)cb), "r"((int)row0), "r"(smem_u32(&bar))
                : "memory");
            // the band slice is a box of the packed layout itself: diagonals dc.., rows i0..i0+63
            if (tma_a)
                asm volatile(
                    "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                    ::"r"(smem_u32(Ad)), "l"(&tmap_a), "r"((int)i0), "r"((int)dc), "r"(smem_u32(&bar))
                    : "memory");
        }
        const int d_end = (int)((diagonals - dc < kChunk) ? diagonals - dc : kChunk);
        if (EXACT) {
            // A row's band entries are consecutive in memory (rowbase(i) + j, j = i + d - w).  A warp
            // owns 16 rows and copies 4 rows x 8 consecutive diagonals per instruction (32-byte runs)
            // with asynchronous 4-byte copies: all of a thread's copies are in flight at once and none
            // holds a register.  Diagonals past d_end are not staged: the loop below never reads them.
            const bool interior = i0 >= w && i0 + kRows - 1 + w < N;  // every row of the tile has all 2w+1 entries
            const int dq = lane & 7;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const int r = 16 * warp + 4 * b + (lane >> 3);
                const int64_t i = i0 + r;
                const float* src = A + (i < N ? band_row_start(N, w, i) - band_jlo(w, i) + i - w : 0) + dc + dq;
                const uint32_t dst = smem_u32(&Ad[dq * kPitch + r]);
                if (interior) {
#pragma unroll
                    for (int k = 0; k < kChunk / 8; ++k)
                        if (8 * k + dq < d_end)
                            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst + k * 8 * kPitch * 4),
                                         "l"(src + 8 * k)
                                         : "memory");
                } else {
                    // first / last row tiles: entries whose column falls outside [0, N) are zero-filled
                    // (source size 0 reads nothing)
#pragma unroll
                    for (int k = 0; k < kChunk / 8; ++k) {
                        const int64_t jj = i + dc + dq + 8 * k - w;
                        const bool in = 8 * k + dq < d_end && i < N && jj >= 0 && jj < N;
                        asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst + k * 8 * kPitch * 4),
                                     "l"(in ? src + 8 * k : A), "r"(in ? 4 : 0)
                                     : "memory");
                    }
                }
            }
            asm volatile("cp.async.wait_all;" ::: "memory");
        } else if (!(TMA_B && tma_a)) {
            // stage diagonals dc .. dc+kChunk-1 of rows i0 .. i0+63 (slot (d, i) = d N + i); zero
            // outside the band / matrix.  kThreads is a multiple of kRows, so a thread keeps its row.
            static_assert(kThreads % kRows == 0, "a thread must stay on one row of the slice");
            const int r = tid % kRows;
            const int64_t i = i0 + r;
#pragma unroll 12
            for (int dl = tid / kRows; dl < kChunk; dl += kThreads / kRows) {
                const int64_t d = dc + dl, jj = i + d - w;
                Ad[dl * kRows + r] = (d < diagonals && i < N && jj >= 0 && jj < N) ? __ldg(A + d * N + i) : 0.f;
            }
        }
        if (TMA_B) {
            // bounded wait for the box
            if (tid == 0) {
                const long long t0 = clock64();
                uint32_t done = 0;
                while (!done) {
                    asm volatile(
                        "{\n\t.reg .pred p;\n\t"
                        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                        "selp.u32 %0, 1, 0, p;\n\t}"
                        : "=r"(done)
                        : "r"(smem_u32(&bar)), "r"(phase)
                        : "memory");
                    if (!done && clock64() - t0 > kWaitBudget) {
                        failed = 1;
                        if (err_word) atomicCAS(err_word, 0, 16);
                        break;
                    }
                }
            }
            phase ^= 1;
        }
        __syncthreads();
        if (TMA_B && failed) return;
        if (TMA_B && !EXACT && tma_a && (i0 < w || i0 + kRows - 1 + w >= N)) {
            // edge tile: the copied box contains padding slots (column i + d - w outside [0, N)); zero them
            for (int t = tid; t < kChunk * kRows; t += kThreads) {
                const int dl = t / kRows, r = t - dl * kRows;
                const int64_t jj = i0 + r + dc + dl - w;
                if (jj < 0 || jj >= N) Ad[t] = 0.f;
            }
            __syncthreads();
        }
        if (c0 >= ncols || i_f >= N) continue;  // lane has no output; it still helped staging

        // window of B rows: row (i_f + d - w + q) sits in slot (d - dc + q) mod 8
        const int br0 = il;  // Bs row of (i_f + dc - w) is il
        pair_t win[8][kPairs];
#pragma unroll
        for (int q = 0; q < 7; ++q)
            load_row<TMA_B>(win[q], Bs, br0 + q, B, ldb, i_f + dc - w + q, N, c0, cl, ncols);
        // one diagonal: slide the window down by one row of B, then 8 rows x 4 columns of multiply-adds
        auto step = [&](const int db, const int u) {
            load_row<TMA_B>(win[(u + 7) & 7], Bs, br0 + db + u + 7, B, ldb, i_f + dc + db + u - w + 7, N, c0, cl, ncols);
            const float4 a_lo = *reinterpret_cast<const float4*>(&Ad[(db + u) * kPitch + il]);
            const float4 a_hi = *reinterpret_cast<const float4*>(&Ad[(db + u) * kPitch + il + 4]);
            const pair_t a2[8] = {pack2(a_lo.x, a_lo.x), pack2(a_lo.y, a_lo.y), pack2(a_lo.z, a_lo.z),
                                  pack2(a_lo.w, a_lo.w), pack2(a_hi.x, a_hi.x), pack2(a_hi.y, a_hi.y),
                                  pack2(a_hi.z, a_hi.z), pack2(a_hi.w, a_hi.w)};
#pragma unroll
            for (int q = 0; q < 8; ++q)
#pragma unroll
                for (int e = 0; e < kPairs; ++e) fma2(acc2[q][e], a2[q], win[(u + q) & 7][e]);
        };
        int db = 0;
        for (; db + 8 <= d_end; db += 8) {
#pragma unroll
            for (int u = 0; u < 8; ++u) step(db, u);
        }
        if (db < d_end) {  // the last 1..7 diagonals: same rotation, no work on diagonals that do not exist
#pragma unroll
            for (int u = 0; u < 7; ++u)
                if (db + u < d_end) step(db, u);
        }
    }
    if (c0 >= ncols || i_f >= N) return;
    float acc[8][kLaneCols];
#pragma unroll
    for (int q = 0; q < 8; ++q)
#pragma unroll
        for (int e = 0; e < kPairs; ++e) unpack2(acc2[q][e], acc[q][2 * e], acc[q][2 * e + 1]);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const int64_t i = i_f + q;
        if (i >= N) break;
        float* dst = C + i * ldc + c0;
        if (vec_c && c0 + kLaneCols <= ncols) {
            float4 o = make_float4(acc[q][0], acc[q][1], acc[q][2], acc[q][3]);
            if (accumulate) {
                const float4 old = *reinterpret_cast<const float4*>(dst);
                o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
            }
            *reinterpret_cast<float4*>(dst) = o;
        } else {
#pragma unroll
            for (int e = 0; e < kLaneCols; ++e)
                if (c0 + e < ncols) dst[e] = accumulate ? dst[e] + acc[q][e] : acc[q][e];
        }
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)ptr;
    }
    return fn;
}

}  // namespace

dastac_status launch_bandmm(const IndexMap& m, const float* A, const float* B, int64_t ldb, float* C,
                            int64_t ldc, int64_t ncols, int accumulate, int32_t* err_word, cudaStream_t st) {
    const int64_t N = m.N;
    if (N == 0 || ncols == 0) return DASTAC_OK;
    const int64_t gx = (ncols + kCols - 1) / kCols, gy = (N + kRows - 1) / kRows;
    if (gx > 0x7fffffffLL || ncols > 0x7fffffffLL) return DASTAC_ERR_OVERFLOW;
    const int vec_c = ((ldc & 3) == 0) && aligned16(C);
    const bool tma_b = ((ldb & 3) == 0) && aligned16(B);
    CUtensorMap tmap;
    std::memset(&tmap, 0, sizeof(tmap));
    size_t smem = (size_t)kChunk * kRows * sizeof(float);
    if (tma_b) {
        EncodeTiledFn enc = encode_fn();
        if (!enc) return DASTAC_ERR_CUDA;
        const cuuint64_t dims[2] = {(cuuint64_t)ncols, (cuuint64_t)N};
        const cuuint64_t strides[1] = {(cuuint64_t)ldb * 4};
        const cuuint32_t box[2] = {(cuuint32_t)kCols, (cuuint32_t)kBRows};
        const cuuint32_t estr[2] = {1, 1};
        if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(B), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return DASTAC_ERR_CUDA;
        smem += (size_t)kBRows * kCols * sizeof(float);
    }
    // The band itself is a [2w+1][N] array: its slice for a row tile is a TMA box too when the row
    // pitch N*4 is a multiple of 16 bytes.
    CUtensorMap tmap_a;
    std::memset(&tmap_a, 0, sizeof(tmap_a));
    int tma_a = 0;
    const int exact = m.kind == kBandExact;
    if (!exact && tma_b && (N % 4 == 0) && aligned16(A)) {
        const cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)(2 * m.w + 1)};
        const cuuint64_t strides[1] = {(cuuint64_t)N * 4};
        const cuuint32_t box[2] = {(cuuint32_t)kRows, (cuuint32_t)kChunk};
        const cuuint32_t estr[2] = {1, 1};
        if (encode_fn()(&tmap_a, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(A), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return DASTAC_ERR_CUDA;
        tma_a = 1;
    }
    if (exact) smem += (size_t)kChunk * (kPitchExact - kRows) * sizeof(float);
    static bool attr_set[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        const int big = (int)((size_t)kChunk * kRows * 4 + (size_t)kBRows * kCols * 4);
        const int big_exact = (int)((size_t)kChunk * kPitchExact * 4 + (size_t)kBRows * kCols * 4);
        if (cudaFuncSetAttribute(bandmm_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, big) != cudaSuccess ||
            cudaFuncSetAttribute(bandmm_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, big_exact) != cudaSuccess)
            return DASTAC_ERR_CUDA;
        attr_set[dev] = true;
    }
    for (int64_t y0 = 0; y0 < gy; y0 += 65535) {  // gridDim.y is limited to 65535
        const int64_t ny = gy - y0 < 65535 ? gy - y0 : 65535;
        const dim3 grid((unsigned)gx, (unsigned)ny);
#define DASTAC_BANDMM_LAUNCH(TB, EX)                                                                              \
    bandmm_kernel<TB, EX><<<grid, kThreads, smem, st>>>(tmap, tmap_a, tma_a, N, m.w, y0, A, B, ldb, C, ldc, ncols, \
                                                        accumulate, vec_c, err_word)
        if (tma_b && exact) DASTAC_BANDMM_LAUNCH(true, true);
        else if (tma_b) DASTAC_BANDMM_LAUNCH(true, false);
        else if (exact) DASTAC_BANDMM_LAUNCH(false, true);
        else DASTAC_BANDMM_LAUNCH(false, false);
#undef DASTAC_BANDMM_LAUNCH
        dastac_status s = launch_status();
        if (s != DASTAC_OK) return s;
    }
    return DASTAC_OK;
}

}  // namespace dastac
