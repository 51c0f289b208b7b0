// C = A B for a banded A (|i - j| <= w) stored as 2w+1 padded diagonals of N slots, B and C dense
// row-major, fp32.  Slot (d, i) holds A(i, i + d - w), so for a fixed diagonal consecutive rows
// are consecutive in memory and the position is the affine map d*N + i.  Padding slots are never
// read into a result: the column range is clipped to [0, N) before the slot is touched.
#include "common.cuh"

namespace dastac {
namespace {

constexpr int kRowsPerBlock = 8;

// One thread computes four adjacent columns of one output row.
__global__ void __launch_bounds__(256)
bandmm_kernel(int64_t N, int64_t w, int64_t row0, const float* __restrict__ A,
              const float* __restrict__ B, int64_t ldb, float* __restrict__ C, int64_t ldc,
              int64_t ncols, int accumulate) {
    const int64_t col_groups = (ncols + 3) >> 2;
    const int64_t groups_per_block_row = blockDim.x / kRowsPerBlock;
    const int r = threadIdx.x / groups_per_block_row;
    const int64_t g = blockIdx.x * groups_per_block_row + (threadIdx.x - r * groups_per_block_row);
    const int64_t i = row0 + blockIdx.y * (int64_t)kRowsPerBlock + r;
    if (i >= N || g >= col_groups) return;
    const int64_t c0 = g * 4;
    const bool vec = (c0 + 4 <= ncols) && ((ldb & 3) == 0) && ((ldc & 3) == 0);
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    const int64_t d_lo = (i - w < 0) ? w - i : 0;                     // first diagonal with j >= 0
    const int64_t d_hi = (i + w > N - 1) ? (N - 1 - i + w) : 2 * w;   // last diagonal with j < N
    for (int64_t d = d_lo; d <= d_hi; ++d) {
        const float a = A[d * N + i];
        const float* brow = B + (i + d - w) * ldb + c0;
        if (vec) {
            float4 b = *reinterpret_cast<const float4*>(brow);
            acc[0] = fmaf(a, b.x, acc[0]);
            acc[1] = fmaf(a, b.y, acc[1]);
            acc[2] = fmaf(a, b.z, acc[2]);
            acc[3] = fmaf(a, b.w, acc[3]);
        } else {
            for (int e = 0; e < 4 && c0 + e < ncols; ++e) acc[e] = fmaf(a, brow[e], acc[e]);
        }
    }
    float* crow = C + i * ldc + c0;
    for (int e = 0; e < 4 && c0 + e < ncols; ++e) crow[e] = accumulate ? crow[e] + acc[e] : acc[e];
}

}  // namespace

dastac_status launch_bandmm(const IndexMap& m, const float* A, const float* B, int64_t ldb, float* C,
                            int64_t ldc, int64_t ncols, int accumulate, cudaStream_t st) {
    const int64_t N = m.N;
    if (N == 0 || ncols == 0) return DASTAC_OK;
    const int64_t col_groups = (ncols + 3) >> 2;
    const int64_t groups_per_block_row = 256 / kRowsPerBlock;
    const int64_t gx = (col_groups + groups_per_block_row - 1) / groups_per_block_row;
    const int64_t gy = (N + kRowsPerBlock - 1) / kRowsPerBlock;
    if (gx > 0x7fffffffLL) return DASTAC_ERR_OVERFLOW;
    for (int64_t y0 = 0; y0 < gy; y0 += 65535) {  // gridDim.y is limited to 65535
        const int64_t ny = gy - y0 < 65535 ? gy - y0 : 65535;
        bandmm_kernel<<<dim3((unsigned)gx, (unsigned)ny), 256, 0, st>>>(
            N, m.w, y0 * kRowsPerBlock, A, B, ldb, C, ldc, ncols, accumulate);
        dastac_status s = launch_status();
        if (s != DASTAC_OK) return s;
    }
    return DASTAC_OK;
}

}  // namespace dastac
