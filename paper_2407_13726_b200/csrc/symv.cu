// y = S x for a symmetric S stored as its packed upper triangle (unique set x <= y plus the swap
// redundancy map, Section 2, "Redundancy map"), fp32.  Every stored off-diagonal element A(i,j)
// is loaded once and used twice: it adds A(i,j) x[j] to y[i] and A(i,j) x[i] to y[j].
//
// Decomposition: the triangle is cut into tiles of kRows rows by kCols columns; only tiles that
// touch the region j >= i exist.  A thread owns kColsPerThread columns of the tile, keeps their
// x[j] and their column sums in registers, and walks the rows; row i of the tile is the
// contiguous packed segment rowbase(i) + j (rowbase advanced by N - i - 1 per row, never
// re-evaluated).  Row sums are reduced with warp shuffles and shared memory, and each tile
// issues one atomic add per row and per column it covers.
#include "common.cuh"

namespace dastac {
namespace {

constexpr int kThreads = 256;
constexpr int kColsPerThread = 4;
constexpr int kCols = kThreads * kColsPerThread;  // 1024
constexpr int kRows = 64;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__global__ void __launch_bounds__(kThreads)
symv_tile_kernel(int64_t N, int64_t col_tiles, const float* __restrict__ A,
                 const float* __restrict__ x, float* __restrict__ y) {
    __shared__ float row_sum[kRows];
    const int64_t I = blockIdx.x / col_tiles, J = blockIdx.x - I * col_tiles;
    const int64_t i0 = I * kRows, j0 = J * kCols;
    if (j0 + kCols - 1 < i0) return;  // tile lies entirely below the diagonal
    const int tid = threadIdx.x, lane = tid & 31;
    if (tid < kRows) row_sum[tid] = 0.f;
    __syncthreads();

    int64_t j[kColsPerThread];
    float xj[kColsPerThread], col_acc[kColsPerThread];
#pragma unroll
    for (int c = 0; c < kColsPerThread; ++c) {
        j[c] = j0 + tid + c * kThreads;
        xj[c] = j[c] < N ? x[j[c]] : 0.f;
        col_acc[c] = 0.f;
    }
    const int64_t i_end = (i0 + kRows < N) ? i0 + kRows : N;
    int64_t base = upper_row_base(N, i0);
#pragma unroll 4
    for (int64_t i = i0; i < i_end; ++i) {
        const float xi = x[i];
        float part = 0.f;
#pragma unroll
        for (int c = 0; c < kColsPerThread; ++c) {
            float a = (j[c] >= i && j[c] < N) ? A[base + j[c]] : 0.f;
            part = fmaf(a, xj[c], part);
            if (j[c] != i) col_acc[c] = fmaf(a, xi, col_acc[c]);
        }
        part = warp_sum(part);
        if (lane == 0) atomicAdd(&row_sum[i - i0], part);
        base += N - i - 1;
    }
    __syncthreads();
    if (tid < kRows && i0 + tid < N) atomicAdd(&y[i0 + tid], row_sum[tid]);
#pragma unroll
    for (int c = 0; c < kColsPerThread; ++c)
        if (j[c] < N && j[c] > i0) atomicAdd(&y[j[c]], col_acc[c]);
}

}  // namespace

size_t symv_workspace_bytes(const IndexMap&) { return 0; }

dastac_status launch_symv(const IndexMap& m, const float* A, const float* x, float* y,
                          int accumulate, void*, cudaStream_t st) {
    const int64_t N = m.N;
    if (N == 0) return DASTAC_OK;
    if (!accumulate && cudaMemsetAsync(y, 0, (size_t)N * sizeof(float), st) != cudaSuccess)
        return DASTAC_ERR_CUDA;
    const int64_t row_tiles = (N + kRows - 1) / kRows, col_tiles = (N + kCols - 1) / kCols;
    if (row_tiles * col_tiles > 0x7fffffffLL) return DASTAC_ERR_OVERFLOW;
    symv_tile_kernel<<<(unsigned)(row_tiles * col_tiles), kThreads, 0, st>>>(N, col_tiles, A, x, y);
    return launch_status();
}

}  // namespace dastac
