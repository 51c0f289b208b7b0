// y = S x for a symmetric S stored as its packed upper triangle (unique set x <= y plus the swap
// redundancy map, Section 2, "Redundancy map"), fp32.  Every stored off-diagonal element A(i,j)
// is loaded once and used twice: it adds A(i,j) x[j] to y[i] and A(i,j) x[i] to y[j].
//
// The packed stream is read with aligned 128-bit loads only.  Row i is the contiguous segment
// rowbase(i) + j, and rowbase(i) mod 4 = r changes from row to row, so an aligned quad of memory
// holds columns 4q - r .. 4q - r + 3 of the row, where q counts quads from the row's own origin.
// A thread owns fixed values of q; over the four possible r its quad slides over the seven columns
// 4q-3 .. 4q+3.  It keeps x and a column sum for those seven columns in registers and a uniform
// switch on r picks the four that the current row touches, so every register index is static.
//
// Decomposition: tiles of kTileRows rows by kTileQuads quads (the tiles partition the memory quads
// of each row, so every stored element belongs to exactly one tile).  Tiles entirely above the
// diagonal run without any predicate; tiles that the diagonal or the right edge crosses mask
// columns j < i (they are the tail of the previous row in memory) and j >= N.  rowbase advances by
// N - i - 1 per row and is never re-evaluated.  Row sums: warp shuffle, then shared atomics; each
// tile issues one global atomic per row and per column it covers.
#include "common.cuh"

namespace dastac {
namespace {

constexpr int kThreads = 256;
constexpr int kQ = 2;                       // quads per thread and row
constexpr int kTileQuads = kThreads * kQ;   // 512 quads
constexpr int kTileCols = 4 * kTileQuads;   // 2048 columns
// Rows per tile: 128 for the largest matrices; fewer when 128-row tiles would give the GPU only a
// wave or two of CTAs (the tiles left of the diagonal return at once), chosen by the host.

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// One row's contribution for alignment class R: element e of slot k is column c0 + 4 kThreads k - R + e,
// register 3 - R + e of the slot's seven.
// kSym = false gives the plain upper-triangular product (no mirrored contribution): the same
// streaming pattern serves large triangular matrix-vector products.
template <int R, bool kMasked, bool kSym>
__device__ __forceinline__ void row_fma(const float4 (&a)[kQ], const float (&xw)[kQ][7], float (&cacc)[kQ][7],
                                        const float xi, float& part, const int i, const int N, const int c0) {
#pragma unroll
    for (int k = 0; k < kQ; ++k) {
        const float v[4] = {a[k].x, a[k].y, a[k].z, a[k].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float vr = v[e], vc = v[e];
            if (kMasked) {
                const int j = c0 + k * (4 * kThreads) - R + e;
                const bool in = j >= i && j < N;
                vr = in ? v[e] : 0.f;
                vc = (in && j != i) ? v[e] : 0.f;  // the diagonal element is used once
            }
            part = fmaf(vr, xw[k][3 - R + e], part);
            if (kSym) cacc[k][3 - R + e] = fmaf(vc, xi, cacc[k][3 - R + e]);
        }
    }
}

template <bool kMasked>
__device__ __forceinline__ void load_row(float4 (&a)[kQ], const float4* __restrict__ A4, const int64_t base,
                                         const int64_t q0, const int64_t cap_quads, const int i, const int N,
                                         const int c0) {
    const int64_t m0 = (base >> 2) + q0;
    const int r = (int)(base & 3);
#pragma unroll
    for (int k = 0; k < kQ; ++k) {
        if (kMasked) {
            const int jlo = c0 + k * (4 * kThreads) - r;  // first column of the quad
            const int64_t m = m0 + k * kThreads;
            a[k] = (jlo + 3 >= i && jlo < N && m < cap_quads) ? __ldg(A4 + m) : make_float4(0.f, 0.f, 0.f, 0.f);
        } else {
            a[k] = __ldg(A4 + m0 + k * kThreads);
        }
    }
}

template <bool kMasked, bool kSym>
__device__ __forceinline__ void row_step(const float4 (&a)[kQ], const float (&xw)[kQ][7], float (&cacc)[kQ][7],
                                         const int r, const float xi, const int i, const int N, const int c0,
                                         float* row_sum_slot, const int lane) {
    float part = 0.f;
    switch (r) {
        case 0: row_fma<0, kMasked, kSym>(a, xw, cacc, xi, part, i, N, c0); break;
        case 1: row_fma<1, kMasked, kSym>(a, xw, cacc, xi, part, i, N, c0); break;
        case 2: row_fma<2, kMasked, kSym>(a, xw, cacc, xi, part, i, N, c0); break;
        default: row_fma<3, kMasked, kSym>(a, xw, cacc, xi, part, i, N, c0); break;
    }
    part = warp_sum(part);
    if (lane == 0) atomicAdd(row_sum_slot, part);
}

template <bool kMasked, bool kSym>
__device__ __forceinline__ void tile_rows(const int N, const int64_t cap_quads, const int i0, const int i_end,
                                          const int64_t q0, const int c0, const float4* __restrict__ A4,
                                          const float (&xw)[kQ][7], float (&cacc)[kQ][7], const float* xs,
                                          float* row_sum, const int lane) {
    int64_t base = upper_row_base(N, i0);
    int i = i0;
    for (; i + 1 < i_end; i += 2) {
        const int64_t base1 = base + (N - i - 1);
        float4 a0[kQ], a1[kQ];
        load_row<kMasked>(a0, A4, base, q0, cap_quads, i, N, c0);
        load_row<kMasked>(a1, A4, base1, q0, cap_quads, i + 1, N, c0);
        row_step<kMasked, kSym>(a0, xw, cacc, (int)(base & 3), xs[i - i0], i, N, c0, row_sum + (i - i0), lane);
        row_step<kMasked, kSym>(a1, xw, cacc, (int)(base1 & 3), xs[i + 1 - i0], i + 1, N, c0, row_sum + (i + 1 - i0), lane);
        base = base1 + (N - i - 2);
    }
    if (i < i_end) {
        float4 a0[kQ];
        load_row<kMasked>(a0, A4, base, q0, cap_quads, i, N, c0);
        row_step<kMasked, kSym>(a0, xw, cacc, (int)(base & 3), xs[i - i0], i, N, c0, row_sum + (i - i0), lane);
    }
}

template <int kTileRows, bool kSym>
__global__ void __launch_bounds__(kThreads, 4)
symv_quad_kernel(const int N, const int64_t cap_quads, const int col_tiles, const float* __restrict__ A,
                 const float* __restrict__ x, float* __restrict__ y) {
    __shared__ float col_sum[kTileCols + 8];  // columns J*kTileCols - 4 ..
    __shared__ float row_sum[kTileRows];
    __shared__ float xs[kTileRows];
    const int I = blockIdx.x / col_tiles, J = blockIdx.x - I * col_tiles;
    const int i0 = I * kTileRows;
    const int64_t col_lo = (int64_t)J * kTileCols;  // column of the tile's first quad when r = 0
    if (col_lo + kTileCols - 1 < i0) return;          // every column of the tile lies left of the diagonal
    const int i_end = (i0 + kTileRows < N) ? i0 + kTileRows : N;
    const int tid = threadIdx.x, lane = tid & 31;
    if (kSym)
        for (int t = tid; t < kTileCols + 8; t += kThreads) col_sum[t] = 0.f;
    if (tid < kTileRows) {
        row_sum[tid] = 0.f;
        xs[tid] = (i0 + tid < N) ? x[i0 + tid] : 0.f;
    }
    const int c0 = (int)col_lo + 4 * tid;  // column 4q of the thread's slot 0
    float xw[kQ][7], cacc[kQ][7];
#pragma unroll
    for (int k = 0; k < kQ; ++k)
#pragma unroll
        for (int d = 0; d < 7; ++d) {
            const int j = c0 + k * (4 * kThreads) - 3 + d;
            xw[k][d] = (j >= 0 && j < N) ? __ldg(x + j) : 0.f;
            cacc[k][d] = 0.f;
        }
    __syncthreads();

    const float4* A4 = reinterpret_cast<const float4*>(A);
    const int64_t q0 = (int64_t)J * kTileQuads + tid;
    // strictly above the diagonal for every row and alignment, and inside the matrix
    const bool interior = (col_lo - 3 > (int64_t)i_end - 1) && (col_lo + kTileCols - 1 < N);
    if (interior)
        tile_rows<false, kSym>(N, cap_quads, i0, i_end, q0, c0, A4, xw, cacc, xs, row_sum, lane);
    else
        tile_rows<true, kSym>(N, cap_quads, i0, i_end, q0, c0, A4, xw, cacc, xs, row_sum, lane);

    if (kSym) {
#pragma unroll
        for (int k = 0; k < kQ; ++k)
#pragma unroll
            for (int d = 0; d < 7; ++d) atomicAdd(&col_sum[4 * (k * kThreads + tid) + 1 + d], cacc[k][d]);
    }
    __syncthreads();
    if (tid < kTileRows && i0 + tid < N) atomicAdd(&y[i0 + tid], row_sum[tid]);
    if (kSym) {
        for (int t = tid; t < kTileCols + 8; t += kThreads) {
            const int64_t j = col_lo - 4 + t;
            if (j > i0 && j < N) atomicAdd(&y[j], col_sum[t]);  // column j only receives from rows i < j
        }
    }
}

}  // namespace

size_t symv_workspace_bytes(const IndexMap&) { return 0; }

// symmetric = 0: the plain upper-triangular product y = A x on the same streaming kernel (used for
// matrices too large for the shared-memory copies of x that the small-N kernel keeps).
dastac_status launch_symv(const IndexMap& m, const float* A, const float* x, float* y,
                          int accumulate, void*, cudaStream_t st, int symmetric) {
    const int64_t N = m.N;
    if (N == 0) return DASTAC_OK;
    if (!accumulate && cudaMemsetAsync(y, 0, (size_t)N * sizeof(float), st) != cudaSuccess)
        return DASTAC_ERR_CUDA;
    const int64_t quads_per_row = (N + 2) / 4 + 1;  // quads that can hold a column < N for some alignment
    const int64_t col_tiles = (quads_per_row + kTileQuads - 1) / kTileQuads;
    // about half of the tiles do work; aim at six or more waves of 4 CTAs per SM
    const int64_t want = (int64_t)sm_count() * 4 * 6;
    int rows = 128;
    while (rows > 32 && ((N + rows - 1) / rows) * col_tiles / 2 < want) rows >>= 1;
    const int64_t row_tiles = (N + rows - 1) / rows;
    if (row_tiles * col_tiles > 0x7fffffffLL) return DASTAC_ERR_OVERFLOW;
    const int64_t cap_quads = (m.count + 3) / 4;
    const unsigned grid = (unsigned)(row_tiles * col_tiles);
#define DASTAC_SYMV_LAUNCH(ROWS, SYM) \
    symv_quad_kernel<ROWS, SYM><<<grid, kThreads, 0, st>>>((int)N, cap_quads, (int)col_tiles, A, x, y)
    if (symmetric) {
        if (rows == 128) DASTAC_SYMV_LAUNCH(128, true);
        else if (rows == 64) DASTAC_SYMV_LAUNCH(64, true);
        else DASTAC_SYMV_LAUNCH(32, true);
    } else {
        if (rows == 128) DASTAC_SYMV_LAUNCH(128, false);
        else if (rows == 64) DASTAC_SYMV_LAUNCH(64, false);
        else DASTAC_SYMV_LAUNCH(32, false);
    }
#undef DASTAC_SYMV_LAUNCH
    return launch_status();
}

}  // namespace dastac
