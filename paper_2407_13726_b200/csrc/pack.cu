// Index-map batch kernels and compress / decompress (Section 3, "Data Layout Compression":
// iterate over the accessed indices and copy the data in and out of the packed buffer).
//
// pack walks the PACKED stream: a thread owns 16 bytes of consecutive packed positions, unranks
// the first one and steps to the following points with index increments, so the packed side is
// written with one aligned 128-bit store per thread and the dense side is read along rows.
// unpack walks the DENSE box: a thread owns 16 bytes of one dense row, so the zero fill and the
// copy are a single pass with 128-bit stores wherever the dense row allows it.
#include "common.cuh"

namespace dastac {
namespace {

struct Strides {
    int64_t s[3];
};

__global__ void rank_batch_kernel(IndexMap m, const int32_t* __restrict__ idx, int64_t n,
                                  int64_t* __restrict__ off) {
    for (int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; t < n;
         t += (int64_t)gridDim.x * blockDim.x) {
        int32_t p[3] = {0, 0, 0};
        for (int k = 0; k < m.rank; ++k) p[k] = idx[t * m.rank + k];
        off[t] = in_set(m, p) ? rank_of(m, p) : -1;
    }
}

__global__ void unrank_batch_kernel(IndexMap m, const int64_t* __restrict__ off, int64_t n,
                                    int32_t* __restrict__ idx) {
    for (int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; t < n;
         t += (int64_t)gridDim.x * blockDim.x) {
        int32_t p[3] = {-1, -1, -1};
        int64_t o = off[t];
        if (o >= 0 && o < m.slots) unrank_of(m, o, p);
        for (int k = 0; k < m.rank; ++k) idx[t * m.rank + k] = p[k];
    }
}

template <typename T>
struct Vec16 {
    static constexpr int kElems = 16 / sizeof(T);
    T v[kElems];
};

template <typename T>
__global__ void pack_kernel(IndexMap m, const T* __restrict__ dense, Strides st,
                            T* __restrict__ packed) {
    constexpr int E = Vec16<T>::kElems;
    const int64_t groups = (m.slots + E - 1) / E;
    for (int64_t g = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; g < groups;
         g += (int64_t)gridDim.x * blockDim.x) {
        const int64_t p0 = g * E;
        Vec16<T> out;
        if (m.kind == kBandDiagonals) {
            int64_t d = p0 / m.N, i = p0 - d * m.N;
#pragma unroll
            for (int e = 0; e < E; ++e) {
                T val = T(0);
                if (p0 + e < m.slots) {
                    int64_t j = i + d - m.w;
                    if (j >= 0 && j < m.N) val = dense[i * st.s[0] + j * st.s[1]];
                    if (++i == m.N) {
                        i = 0;
                        ++d;
                    }
                }
                out.v[e] = val;
            }
        } else {
            int32_t idx[3] = {0, 0, 0};
            unrank_of(m, p0, idx);
#pragma unroll
            for (int e = 0; e < E; ++e) {
                T val = T(0);
                if (p0 + e < m.count) {
                    val = dense[idx[0] * st.s[0] + idx[1] * st.s[1] + idx[2] * st.s[2]];
                    advance(m, idx);
                }
                out.v[e] = val;
            }
        }
        // The packed buffer's capacity is a multiple of 16 bytes, so the last group may be
        // written whole (positions beyond the count receive zero).
        *reinterpret_cast<uint4*>(packed + p0) = *reinterpret_cast<const uint4*>(out.v);
    }
}

template <typename T>
__global__ void unpack_kernel(IndexMap m, const T* __restrict__ packed, T* __restrict__ dense,
                              Strides st, int vector_ok) {
    constexpr int E = Vec16<T>::kElems;
    const int last = m.rank - 1;
    const int64_t inner = m.dims[last];
    const int64_t groups_per_row = (inner + E - 1) / E;
    int64_t rows = 1;
    for (int k = 0; k < last; ++k) rows *= m.dims[k];
    const int64_t groups = rows * groups_per_row;
    for (int64_t g = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; g < groups;
         g += (int64_t)gridDim.x * blockDim.x) {
        int64_t row = g / groups_per_row;
        const int64_t c0 = (g - row * groups_per_row) * E;
        int32_t idx[3] = {0, 0, 0};
        for (int k = last - 1; k >= 0; --k) {
            int64_t q = row / m.dims[k];
            idx[k] = (int32_t)(row - q * m.dims[k]);
            row = q;
        }
        int64_t base = 0;
        for (int k = 0; k < last; ++k) base += idx[k] * st.s[k];
        Vec16<T> out;
#pragma unroll
        for (int e = 0; e < E; ++e) {
            T val = T(0);
            if (c0 + e < inner) {
                idx[last] = (int32_t)(c0 + e);
                if (in_set(m, idx)) {
                    val = packed[rank_of(m, idx)];
                } else if (m.symmetric) {
                    int32_t sw[3] = {idx[1], idx[0], 0};
                    if (in_set(m, sw)) val = packed[rank_of(m, sw)];
                }
            }
            out.v[e] = val;
        }
        T* dst = dense + base + c0 * st.s[last];
        if (vector_ok && c0 + E <= inner) {
            *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(out.v);
        } else {
            for (int e = 0; e < E && c0 + e < inner; ++e) dst[e * st.s[last]] = out.v[e];
        }
    }
}

int grid_for(int64_t work_items, int threads) {
    int64_t blocks = (work_items + threads - 1) / threads;
    int64_t cap = (int64_t)sm_count() * 16;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

bool strides_ok(const IndexMap& m, const int64_t* s) {
    for (int k = 0; k < m.rank; ++k)
        if (s[k] < 0) return false;
    return true;
}

}  // namespace
}  // namespace dastac

using namespace dastac;

extern "C" dastac_status dastac_rank_batch(const dastac_structure* s, const int32_t* idx, int64_t n,
                                           int64_t* off, void* stream) {
    if (!s || n < 0 || (n > 0 && (!idx || !off))) return DASTAC_ERR_INVALID_ARG;
    if (n == 0) return DASTAC_OK;
    rank_batch_kernel<<<grid_for(n, 256), 256, 0, (cudaStream_t)stream>>>(s->map, idx, n, off);
    return launch_status();
}

extern "C" dastac_status dastac_unrank_batch(const dastac_structure* s, const int64_t* off,
                                             int64_t n, int32_t* idx, void* stream) {
    if (!s || n < 0 || (n > 0 && (!idx || !off))) return DASTAC_ERR_INVALID_ARG;
    if (n == 0) return DASTAC_OK;
    unrank_batch_kernel<<<grid_for(n, 256), 256, 0, (cudaStream_t)stream>>>(s->map, off, n, idx);
    return launch_status();
}

extern "C" dastac_status dastac_pack(const dastac_structure* s, dastac_dtype dtype,
                                     const void* dense, const int64_t* dense_strides, void* packed,
                                     void* stream) {
    if (!s || !dense_strides) return DASTAC_ERR_INVALID_ARG;
    if (dtype != DASTAC_F32 && dtype != DASTAC_BF16) return DASTAC_ERR_INVALID_ARG;
    const IndexMap& m = s->map;
    if (!strides_ok(m, dense_strides)) return DASTAC_ERR_INVALID_ARG;
    if (m.slots == 0) return DASTAC_OK;
    if (!dense || !packed) return DASTAC_ERR_INVALID_ARG;
    if (!aligned16(packed)) return DASTAC_ERR_ALIGNMENT;
    Strides st{{0, 0, 0}};
    for (int k = 0; k < m.rank; ++k) st.s[k] = dense_strides[k];
    const int E = 16 / elt_size(dtype);
    const int grid = grid_for((m.slots + E - 1) / E, 256);
    if (dtype == DASTAC_F32)
        pack_kernel<uint32_t><<<grid, 256, 0, (cudaStream_t)stream>>>(
            m, (const uint32_t*)dense, st, (uint32_t*)packed);
    else
        pack_kernel<uint16_t><<<grid, 256, 0, (cudaStream_t)stream>>>(
            m, (const uint16_t*)dense, st, (uint16_t*)packed);
    return launch_status();
}

extern "C" dastac_status dastac_unpack(const dastac_structure* s, dastac_dtype dtype,
                                       const void* packed, void* dense,
                                       const int64_t* dense_strides, void* stream) {
    if (!s || !dense_strides) return DASTAC_ERR_INVALID_ARG;
    if (dtype != DASTAC_F32 && dtype != DASTAC_BF16) return DASTAC_ERR_INVALID_ARG;
    const IndexMap& m = s->map;
    if (!strides_ok(m, dense_strides)) return DASTAC_ERR_INVALID_ARG;
    int64_t box = 1;
    for (int k = 0; k < m.rank; ++k) box *= m.dims[k];
    if (box == 0) return DASTAC_OK;
    if (!dense || (m.slots > 0 && !packed)) return DASTAC_ERR_INVALID_ARG;
    if (m.slots > 0 && !aligned16(packed)) return DASTAC_ERR_ALIGNMENT;
    Strides st{{0, 0, 0}};
    for (int k = 0; k < m.rank; ++k) st.s[k] = dense_strides[k];
    const int esz = elt_size(dtype);
    const int E = 16 / esz;
    // 128-bit stores need a unit inner stride, a 16-byte aligned base and outer strides that keep
    // every row start on a 16-byte boundary.
    int vector_ok = st.s[m.rank - 1] == 1 && aligned16(dense);
    for (int k = 0; k + 1 < m.rank; ++k) vector_ok = vector_ok && (st.s[k] % E == 0);
    const int last = m.rank - 1;
    int64_t rows = box / m.dims[last];
    const int64_t groups = rows * ((m.dims[last] + E - 1) / E);
    const int grid = grid_for(groups, 256);
    if (dtype == DASTAC_F32)
        unpack_kernel<uint32_t><<<grid, 256, 0, (cudaStream_t)stream>>>(
            m, (const uint32_t*)packed, (uint32_t*)dense, st, vector_ok);
    else
        unpack_kernel<uint16_t><<<grid, 256, 0, (cudaStream_t)stream>>>(
            m, (const uint16_t*)packed, (uint16_t*)dense, st, vector_ok);
    return launch_status();
}
