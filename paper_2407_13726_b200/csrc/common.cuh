// Shared host-side helpers of the library: status plumbing, launch accounting, the structure object.
#pragma once
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>

#include "../../include/dastac.h"
#include "generic.cuh"
#include "indexmap.cuh"

struct dastac_structure {
    dastac::IndexMap map;
    dastac::GenericMap* generic = nullptr;  // map.kind == kGeneric: the fitted map (owned)
    ~dastac_structure() { delete generic; }
};

namespace dastac {

extern std::atomic<int64_t> g_launches;

inline void note_launch(int n = 1) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// Status of the launch that was just enqueued (configuration errors only; execution is asynchronous).
inline dastac_status launch_status() {
    note_launch();
    return cudaGetLastError() == cudaSuccess ? DASTAC_OK : DASTAC_ERR_CUDA;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int64_t round_up(int64_t v, int64_t m) { return (v + m - 1) / m * m; }

inline int elt_size(int dtype) { return dtype == DASTAC_BF16 ? 2 : 4; }

// Number of SMs of the current device (cached per device id).
int sm_count();

// ---- kernels' host entry points (one per expression class) ------------------------------------
dastac_status launch_trmv(const IndexMap& m, const float* A, const float* x, float* y, int batch,
                          int64_t a_stride, int64_t x_stride, int64_t y_stride, int accumulate,
                          cudaStream_t st);
bool rowspan_mv_supports(const IndexMap& m);
dastac_status launch_rowspan_mv(const IndexMap& m, const float* A, const float* x, float* y, int batch,
                                int64_t a_stride, int64_t x_stride, int64_t y_stride, int accumulate,
                                cudaStream_t st);
dastac_status launch_rowspan_mm(const IndexMap& m, const float* A, const float* B, int64_t ldb, float* C,
                                int64_t ldc, int64_t ncols, int accumulate, cudaStream_t st);
size_t symv_workspace_bytes(const IndexMap& m);
dastac_status launch_symv(const IndexMap& m, const float* A, const float* x, float* y,
                          int accumulate, void* workspace, cudaStream_t st, int symmetric = 1);
dastac_status launch_bandmm(const IndexMap& m, const float* A, const float* B, int64_t ldb, float* C,
                            int64_t ldc, int64_t ncols, int accumulate, int32_t* err_word, cudaStream_t st);
bool mttkrp_supports(const IndexMap& m);
dastac_status launch_mttkrp(const IndexMap& m, const float* T, const float* B, int64_t ldb,
                            const float* C, int64_t ldc, float* M, int64_t ldm, int64_t R,
                            int accumulate, int32_t* err_word, cudaStream_t st);
dastac_status launch_ttm(int64_t P, int64_t Q, int64_t K, const float* X, const float* C, int64_t ldc, float* Y,
                         int accumulate, cudaStream_t st);
size_t trimm_workspace_bytes(const IndexMap& m, int64_t ncols, int64_t ldb);
dastac_status launch_trimm_bf16(const IndexMap& m, const void* A, const void* B, int64_t ldb,
                                float* C, int64_t ldc, int64_t ncols, int accumulate,
                                void* workspace, int32_t* err_word, cudaStream_t st);
size_t moment2_workspace_bytes(int64_t M, int64_t n, int64_t ldb);
dastac_status launch_moment2_bf16(const IndexMap& mo, const void* B, int64_t ldb, int64_t M, float* out,
                                  int accumulate, void* workspace, int32_t* err_word, cudaStream_t st);
size_t moment3_workspace_bytes(int64_t M, int64_t n, int64_t ldb);
dastac_status launch_moment3_bf16(const IndexMap& mo, const void* B, int64_t ldb, int64_t M, float* out,
                                  int accumulate, void* workspace, int32_t* err_word, cudaStream_t st);
dastac_status launch_hadamard(const IndexMap& m, const float* Bp, const float* C, const int64_t* c_strides,
                              float* out, int accumulate, cudaStream_t stream);

}  // namespace dastac
