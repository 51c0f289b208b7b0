// y = A x for a packed upper-triangular A (the paper's SpMV_UT rule A(i) := B(i,j) * C(j), Table 1),
// fp32, optionally batched over independent instances that share one structure.
//
// Work balance over the uneven rows: row i has N - i stored elements, so rows i and N-1-i together
// always hold N + 1.  One warp owns one such pair; every warp therefore streams the same number
// of packed elements.  Inside a row the position is rowbase(i) + j with rowbase hoisted, the
// loop-invariant part of the ranking polynomial (Section 4, last paragraph; Section 5.3, "Loop
// Invariant Code Motion").
#include "common.cuh"

namespace dastac {
namespace {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Dot product of packed row i (columns i..N-1) with x, distributed over the lanes of a warp.
__device__ __forceinline__ float row_dot(const float* __restrict__ A, const float* __restrict__ x,
                                         int64_t N, int64_t i, int lane) {
    const float* row = A + upper_row_base(N, i);  // row[j] = A(i, j)
    float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
    int64_t j = i + lane;
    for (; j + 96 < N; j += 128) {
        acc0 = fmaf(row[j], x[j], acc0);
        acc1 = fmaf(row[j + 32], x[j + 32], acc1);
        acc2 = fmaf(row[j + 64], x[j + 64], acc2);
        acc3 = fmaf(row[j + 96], x[j + 96], acc3);
    }
    for (; j < N; j += 32) acc0 = fmaf(row[j], x[j], acc0);
    return warp_sum((acc0 + acc1) + (acc2 + acc3));
}

__global__ void __launch_bounds__(256)
trmv_pair_kernel(int64_t N, const float* __restrict__ A, const float* __restrict__ x,
                 float* __restrict__ y, int64_t a_stride, int64_t x_stride, int64_t y_stride,
                 int accumulate) {
    const int lane = threadIdx.x & 31;
    const int64_t pair = blockIdx.x * (int64_t)(blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t pairs = (N + 1) >> 1;
    if (pair >= pairs) return;
    A += blockIdx.y * a_stride;
    x += blockIdx.y * x_stride;
    y += blockIdx.y * y_stride;
    const int64_t i0 = pair, i1 = N - 1 - pair;
    float s0 = row_dot(A, x, N, i0, lane);
    if (lane == 0) y[i0] = accumulate ? y[i0] + s0 : s0;
    if (i1 != i0) {
        float s1 = row_dot(A, x, N, i1, lane);
        if (lane == 0) y[i1] = accumulate ? y[i1] + s1 : s1;
    }
}

}  // namespace

dastac_status launch_trmv(const IndexMap& m, const float* A, const float* x, float* y, int batch,
                          int64_t a_stride, int64_t x_stride, int64_t y_stride, int accumulate,
                          cudaStream_t st) {
    const int64_t N = m.N;
    if (N == 0 || batch == 0) return DASTAC_OK;
    const int64_t pairs = (N + 1) >> 1;
    const int warps = 8;
    dastac_status last = DASTAC_OK;
    for (int b0 = 0; b0 < batch; b0 += 65535) {  // gridDim.y limit
        int nb = batch - b0 < 65535 ? batch - b0 : 65535;
        dim3 grid((unsigned)((pairs + warps - 1) / warps), (unsigned)nb);
        trmv_pair_kernel<<<grid, warps * 32, 0, st>>>(N, A + b0 * a_stride, x + b0 * x_stride,
                                                      y + b0 * y_stride, a_stride, x_stride,
                                                      y_stride, accumulate);
        last = launch_status();
        if (last != DASTAC_OK) return last;
    }
    return last;
}

}  // namespace dastac
