// C = A B for a packed upper-triangular bf16 A and a dense row-major bf16 B, fp32 accumulation and
// fp32 output.  (First version: plain CUDA-core loops; the tensor-core pipeline replaces it.)
#include <cuda_bf16.h>

#include "common.cuh"

namespace dastac {
namespace {

constexpr int kTile = 16;

__global__ void __launch_bounds__(kTile * kTile)
trimm_simt_kernel(int64_t N, const __nv_bfloat16* __restrict__ A,
                  const __nv_bfloat16* __restrict__ B, int64_t ldb, float* __restrict__ C,
                  int64_t ldc, int64_t ncols, int accumulate) {
    __shared__ float As[kTile][kTile + 1];
    __shared__ float Bs[kTile][kTile + 1];
    const int tx = threadIdx.x % kTile, ty = threadIdx.x / kTile;
    const int64_t i = blockIdx.y * (int64_t)kTile + ty, c = blockIdx.x * (int64_t)kTile + tx;
    const int64_t i_first = blockIdx.y * (int64_t)kTile;
    const int64_t base = i < N ? upper_row_base(N, i) : 0;
    float acc = 0.f;
    for (int64_t j0 = i_first; j0 < N; j0 += kTile) {  // columns left of the block's first row are zero
        const int64_t ja = j0 + tx;
        As[ty][tx] = (i < N && ja < N && ja >= i) ? __bfloat162float(A[base + ja]) : 0.f;
        const int64_t jb = j0 + ty;
        Bs[ty][tx] = (jb < N && c < ncols) ? __bfloat162float(B[jb * ldb + c]) : 0.f;
        __syncthreads();
#pragma unroll
        for (int k = 0; k < kTile; ++k) acc = fmaf(As[ty][k], Bs[k][tx], acc);
        __syncthreads();
    }
    if (i < N && c < ncols) C[i * ldc + c] = accumulate ? C[i * ldc + c] + acc : acc;
}

}  // namespace

size_t trimm_workspace_bytes(const IndexMap&, int64_t) { return 0; }

dastac_status launch_trimm_bf16(const IndexMap& m, const void* A, const void* B, int64_t ldb,
                                float* C, int64_t ldc, int64_t ncols, int accumulate, void*,
                                int32_t*, cudaStream_t st) {
    const int64_t N = m.N;
    if (N == 0 || ncols == 0) return DASTAC_OK;
    const int64_t gx = (ncols + kTile - 1) / kTile, gy = (N + kTile - 1) / kTile;
    if (gy > 65535 || gx > 0x7fffffffLL) return DASTAC_ERR_OVERFLOW;
    trimm_simt_kernel<<<dim3((unsigned)gx, (unsigned)gy), kTile * kTile, 0, st>>>(
        N, (const __nv_bfloat16*)A, (const __nv_bfloat16*)B, ldb, C, ldc, ncols, accumulate);
    return launch_status();
}

}  // namespace dastac
