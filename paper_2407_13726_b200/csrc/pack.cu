// Index-map batch kernels and compress / decompress (Section 3, "Data Layout Compression":
// iterate over the accessed indices and copy the data in and out of the packed buffer).
//
// Row kernels (the fast path, unit inner stride): for fixed outer indices the innermost indices of
// the set are one interval [jlo, jhi) stored contiguously at pbase + j, with pbase the hoisted part
// of the ranking polynomial.  Source and destination of a row differ in their alignment modulo 16
// bytes by a constant, so data moves in aligned 16-byte chunks of the DESTINATION and every chunk
// is cut out of the two aligned source granules that cover it (word select + funnel shift).
//   pack    destination = aligned chunks of the packed span of a row.  Chunks that a row shares
//           with its neighbour (first and last of the row) are written element by element by both.
//   unpack  destination = aligned chunks of a dense row; elements outside [jlo, jhi) become zero,
//           so the zero fill of the rest of the box is the same pass.
// In both, a warp fetches the source of a whole window (256 chunks) with one bulk asynchronous
// copy into its own shared-memory buffer and works on the previous window meanwhile; pack keeps a
// register-only form for dense tensors whose base is not 16-byte aligned.
// Generic kernels (any strides, the padded-diagonal layout, the redundancy swap): pack walks the
// packed stream, a thread unranks the first of its positions and steps with index increments;
// unpack walks the dense box and ranks every point.
#include "common.cuh"
#include "waits.cuh"

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
#pragma unroll
        for (int k = 0; k < 3; ++k)
            if (k < m.rank) p[k] = idx[t * m.rank + k];
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
#pragma unroll
        for (int k = 0; k < 3; ++k)
            if (k < m.rank) idx[t * m.rank + k] = p[k];
    }
}

// ---- structures with a fitted map (generic.cuh): element-wise kernels ---------------------------
__global__ void g_rank_batch_kernel(GenericMap g, const int32_t* __restrict__ idx, int64_t n, int64_t* __restrict__ off) {
    for (int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; t < n; t += (int64_t)gridDim.x * blockDim.x) {
        int64_t p[3] = {0, 0, 0};
        for (int k = 0; k < g.rank; ++k) p[k] = idx[t * g.rank + k];
        off[t] = g_in_domain(g, p) ? g_rank(g, p) : -1;
    }
}

__global__ void g_unrank_batch_kernel(GenericMap g, const int64_t* __restrict__ off, int64_t n, int32_t* __restrict__ idx) {
    for (int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; t < n; t += (int64_t)gridDim.x * blockDim.x) {
        int64_t p[3] = {-1, -1, -1};
        const int64_t o = off[t];
        if (o >= 0 && o < g.count) g_unrank(g, o, p);
        for (int k = 0; k < g.rank; ++k) idx[t * g.rank + k] = (int32_t)p[k];
    }
}

// A warp per fibre of the last index: the position of the fibre's first stored element is evaluated
// once, the lanes then move along the fibre (contiguous in the packed vector, and in the dense tensor
// when its last stride is 1).  UNPACK writes the whole fibre of the box, zeros outside the set.
template <typename T, bool UNPACK>
__global__ void g_fibre_copy_kernel(GenericMap g, T* __restrict__ dense, Strides st, T* __restrict__ packed) {
    const int lane = threadIdx.x & 31;
    const int64_t fibres = g.rank == 2 ? g.dims[0] : g.dims[0] * g.dims[1];
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t last = g.dims[g.rank - 1];
    for (int64_t f = blockIdx.x * (int64_t)(blockDim.x >> 5) + (threadIdx.x >> 5); f < fibres; f += warps) {
        int64_t outer[3] = {f, 0, 0};
        if (g.rank == 3) {
            outer[0] = f / g.dims[1];
            outer[1] = f - outer[0] * g.dims[1];
        }
        int64_t lo, hi;
        const bool live = g_last_bounds(g, outer, lo, hi) && hi >= lo;
        int64_t base = 0;
        if (live) {
            base = g_s1(g, outer[0]);
            if (g.rank == 3) base += g_s2(g, outer[0], outer[1]);
        }
        T* drow = dense + outer[0] * st.s[0] + (g.rank == 3 ? outer[1] * st.s[1] : 0);
        const int64_t ls = st.s[g.rank - 1];
        if (UNPACK) {
            for (int64_t x = lane; x < last; x += 32) drow[x * ls] = (live && x >= lo && x <= hi) ? packed[base + (x - lo)] : T(0);
        } else if (live) {
            for (int64_t x = lo + lane; x <= hi; x += 32) packed[base + (x - lo)] = drow[x * ls];
        }
    }
}

template <typename T>
struct Vec16 {
    static constexpr int kElems = 16 / sizeof(T);
    T v[kElems];
};

// Element of the Hadamard form: the gathered dense value times the packed factor, optionally added
// to what the output holds (values are fp32 carried in the 32-bit copy type).
__device__ __forceinline__ uint32_t mul_acc(uint32_t gathered, uint32_t factor, uint32_t old, bool accumulate) {
    const float v = __uint_as_float(gathered) * __uint_as_float(factor);
    return __float_as_uint(accumulate ? v + __uint_as_float(old) : v);
}
__device__ __forceinline__ uint16_t mul_acc(uint16_t g, uint16_t, uint16_t, bool) { return g; }  // copy type only

// MUL: packed[p] = dense[idx(p)] * factor[p] (+ packed[p]) instead of a plain copy.
template <typename T, bool MUL = false>
__global__ void pack_kernel(IndexMap m, const T* __restrict__ dense, Strides st,
                            T* __restrict__ packed, const T* __restrict__ factor = nullptr, int accumulate = 0) {
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
                    if (j >= 0 && j < m.N) {
                        val = dense[i * st.s[0] + j * st.s[1]];
                        if (MUL) val = mul_acc(val, factor[p0 + e], packed[p0 + e], accumulate != 0);
                    }
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
                    if (MUL) val = mul_acc(val, factor[p0 + e], packed[p0 + e], accumulate != 0);
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

// The 16 bytes that start `sh` bytes into the 32-byte window (lo, hi): word select on sh / 4, then
// a funnel shift by the remaining bytes.  sh is a multiple of the element size.
__device__ __forceinline__ uint4 realign16(const uint4 lo, const uint4 hi, const uint32_t sh) {
    const bool q1 = sh & 4, q2 = sh & 8;
    const uint32_t bits = (sh & 3) * 8;
    const uint32_t X0 = q1 ? lo.y : lo.x, X1 = q1 ? lo.z : lo.y, X2 = q1 ? lo.w : lo.z, X3 = q1 ? hi.x : lo.w,
                   X4 = q1 ? hi.y : hi.x, X5 = q1 ? hi.z : hi.y, X6 = q1 ? hi.w : hi.z;
    const uint32_t T0 = q2 ? X2 : X0, T1 = q2 ? X3 : X1, T2 = q2 ? X4 : X2, T3 = q2 ? X5 : X3, T4 = q2 ? X6 : X4;
    return make_uint4(__funnelshift_r(T0, T1, bits), __funnelshift_r(T1, T2, bits), __funnelshift_r(T2, T3, bits),
                      __funnelshift_r(T3, T4, bits));
}

constexpr int kUnroll = 4;         // 16-byte chunks per lane and pass
constexpr int kWarpsPerBlock = 8;

// Offset of the first dense element of the row that holds idx (outer indices only).
__device__ __forceinline__ int64_t dense_row_offset(const IndexMap& m, const Strides& st, const int32_t* idx) {
    int64_t off = 0;
#pragma unroll
    for (int k = 0; k < 2; ++k)
        if (k + 1 < m.rank) off += idx[k] * st.s[k];
    return off;
}

// pack: a warp item is a run of windows (32 * kUnroll chunks each) of the packed span of one row.
// Items are independent, so short rows (the tip of a triangle) cost one pass each instead of
// serialising a walk, and rows that are shorter than the longest simply have fewer live windows.
template <typename T>
__global__ void __launch_bounds__(32 * kWarpsPerBlock, 4)
pack_stream_kernel(IndexMap m, const T* __restrict__ dense, Strides st, T* __restrict__ packed,
                   int64_t rows, int groups_per_row, int windows_per_group) {
    constexpr int E = 16 / sizeof(T);
    const int lane = threadIdx.x & 31;
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
    const int64_t warps = (int64_t)gridDim.x * kWarpsPerBlock;
    for (int64_t item = blockIdx.x * (int64_t)kWarpsPerBlock + (threadIdx.x >> 5); item < rows * groups_per_row;
         item += warps) {
        int64_t row = item;
        int grp = 0;
        if (groups_per_row > 1) {
            row = item / groups_per_row;
            grp = (int)(item - row * groups_per_row);
        }
        int32_t idx[3] = {0, 0, 0};
        if (m.rank == 2) {
            idx[0] = (int32_t)row;
        } else if (m.rank == 3) {
            const int64_t q = row / m.dims[1];
            idx[1] = (int32_t)(row - q * m.dims[1]);
            idx[0] = (int32_t)q;
        }
        int64_t jlo = 0, jhi = 0, pbase = 0;
        if (!row_span(m, idx, jlo, jhi, pbase)) continue;
        const int64_t ps = pbase + jlo, pe = pbase + jhi;              // the row's span in the packed stream
        const T* drow = dense + dense_row_offset(m, st, idx) - pbase;  // drow[p]: element stored at position p
        const int64_t c_first = ps / E;
        // A packed chunk is 16-byte aligned and every chunk is 16 bytes, so the dense source of all
        // chunks of a row has the same misalignment: one shift and one aligned base per item.
        const uintptr_t d_first = reinterpret_cast<uintptr_t>(drow + c_first * E);
        const uint32_t sh_row = (uint32_t)(d_first & 15);
        const uint4* srcq = reinterpret_cast<const uint4*>(d_first - sh_row);  // srcq[c - c_first]: granule under chunk c
        uint4* dstq = reinterpret_cast<uint4*>(packed) + c_first;
        for (int win = grp * windows_per_group; win < (grp + 1) * windows_per_group; ++win) {
            const int64_t c0 = c_first + (int64_t)win * (32 * kUnroll) + lane;
            if ((c0 - lane) * E >= pe) break;
            if ((c0 - lane) * E >= ps && (c0 - lane + 32 * kUnroll) * E <= pe) {
                // the whole window lies inside the row: no per-chunk tests, addresses are one pointer plus constants
                const uint4* sp = srcq + (int64_t)win * (32 * kUnroll) + lane;
                uint4* dp = dstq + (int64_t)win * (32 * kUnroll) + lane;
                uint4 lo[kUnroll], hi[kUnroll];
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    lo[u] = __ldg(sp + 32 * u);
                    hi[u] = sh_row ? __ldg(sp + 32 * u + 1) : zero4;
                }
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) dp[32 * u] = realign16(lo[u], hi[u], sh_row);
                continue;
            }
            uint4 lo[kUnroll], hi[kUnroll];
            uint32_t sh[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const int64_t p0 = (c0 + 32 * u) * E;
                sh[u] = 0;
                if (p0 >= ps && p0 + E <= pe) {  // whole chunk inside this row: two aligned granules cover it
                    const uintptr_t addr = reinterpret_cast<uintptr_t>(drow + p0);
                    sh[u] = (uint32_t)(addr & 15);
                    const uint4* src = reinterpret_cast<const uint4*>(addr - sh[u]);
                    lo[u] = __ldg(src);
                    hi[u] = sh[u] ? __ldg(src + 1) : zero4;
                }
            }
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const int64_t p0 = (c0 + 32 * u) * E;
                if (p0 >= pe) break;
                if (p0 >= ps && p0 + E <= pe) {
                    *reinterpret_cast<uint4*>(packed + p0) = realign16(lo[u], hi[u], sh[u]);
                } else {  // chunk shared with the neighbouring row, or the tail of the stream
#pragma unroll
                    for (int e = 0; e < E; ++e) {
                        const int64_t p = p0 + e;
                        if (p >= ps && p < pe) packed[p] = drow[p];
                        else if (p >= m.count) packed[p] = T(0);
                    }
                }
            }
        }
    }
}

// pack through shared memory: the source windows arrive by bulk asynchronous copies (one request of
// up to 4 KiB per window instead of 2 x 256 separate 16-byte loads), so a warp always has a whole
// window in flight while it realigns and stores the previous one.  A warp owns two window buffers
// and two mbarriers; nothing is shared between warps.  Per window: the packed chunks that lie
// wholly inside the row are served from the buffer (two aligned 128-bit shared loads around the
// chunk's source bytes, the same word select + funnel shift as above, one 128-bit store); the at
// most two chunks a row shares with its neighbours are written element by element from global
// memory.  The source may be read up to the end of the 16-byte granule that holds a needed element.
constexpr int kBulkWin = 256;                          // chunks (16 bytes each) per window
constexpr int kBulkBufBytes = kBulkWin * 16 + 16;      // + the granule after the last chunk
// Window buffers per warp (depth - 1 windows in flight) and the CTAs per SM their shared memory allows.
// Measured on the bf16 triangle N = 8192: pack 29 us at depth 2 against 33 us at depth 3 and 48 us at
// depth 4; unpack 38 us at depth 3 against 41 us at depth 2 and 63 us at depth 4.
constexpr int kPackDepth = 2, kUnpackDepth = 3;
constexpr int bulk_smem_bytes(int depth) { return kWarpsPerBlock * depth * kBulkBufBytes + kWarpsPerBlock * depth * 8; }
constexpr int bulk_ctas_per_sm(int depth) { return depth <= 2 ? 3 : depth == 3 ? 2 : 1; }
constexpr int kBulkSmemBytesMul = kWarpsPerBlock * 4 * kBulkBufBytes + kWarpsPerBlock * 2 * 8;  // Hadamard form: depth 2, two operands

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

template <typename T, bool MUL = false>
__global__ void __launch_bounds__(32 * kWarpsPerBlock, MUL ? 1 : 3)
pack_bulk_kernel(IndexMap m, const T* __restrict__ dense, Strides st, T* __restrict__ packed, int64_t rows,
                 int windows_per_row, long long wait_budget, int32_t* __restrict__ err_word,
                 const T* __restrict__ factor = nullptr, int accumulate = 0) {
    constexpr int E = 16 / sizeof(T);
    extern __shared__ __align__(128) uint8_t bulk_smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // MUL: two more buffers per warp hold the matching windows of the packed factor
    constexpr int D = MUL ? 2 : kPackDepth;
    constexpr int kBufs = MUL ? 2 * D : D;
    uint8_t* buf0 = bulk_smem + warp * kBufs * kBulkBufBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(bulk_smem + kWarpsPerBlock * kBufs * kBulkBufBytes) + warp * D;
    if (lane == 0) {
        for (int d = 0; d < D; ++d) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(&bars[d])));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();

    // what a window needs, worked out by every lane (uniform in the warp)
    struct Win {
        int64_t ps, pe;          // the row's span in the packed stream
        int64_t c_lo, c_hi;      // chunks of the window that lie wholly inside the row: [c_lo, c_hi)
        int64_t c0;              // first chunk of the window
        const T* drow;           // drow[p] = element stored at position p
        uintptr_t g0;            // aligned source address under chunk c_lo
        uint32_t sh, bytes;      // misalignment of the source (bytes), size of the bulk copy
        bool live;
    };
    const int64_t items = rows * windows_per_row;
    const int64_t warps = (int64_t)gridDim.x * kWarpsPerBlock;
    auto describe = [&](int64_t item, Win& w) {
        w.live = false;
        w.bytes = 0;
        w.sh = 0;
        w.g0 = 0;
        w.c_lo = w.c_hi = 0;
        if (item >= items) return;
        const int64_t row = item / windows_per_row;
        const int win = (int)(item - row * windows_per_row);
        int32_t idx[3] = {0, 0, 0};
        if (m.rank == 2) {
            idx[0] = (int32_t)row;
        } else if (m.rank == 3) {
            const int64_t q = row / m.dims[1];
            idx[1] = (int32_t)(row - q * m.dims[1]);
            idx[0] = (int32_t)q;
        }
        int64_t jlo = 0, jhi = 0, pbase = 0;
        if (!row_span(m, idx, jlo, jhi, pbase)) return;
        w.ps = pbase + jlo;
        w.pe = pbase + jhi;
        w.c0 = w.ps / E + (int64_t)win * kBulkWin;
        if (w.c0 * E >= w.pe) return;
        w.live = true;
        w.drow = dense + dense_row_offset(m, st, idx) - pbase;
        const int64_t first_in = (w.ps + E - 1) / E, last_in = w.pe / E;  // chunks wholly inside: [first_in, last_in)
        w.c_lo = w.c0 > first_in ? w.c0 : first_in;
        w.c_hi = w.c0 + kBulkWin < last_in ? w.c0 + kBulkWin : last_in;
        if (w.c_hi > w.c_lo) {
            const uintptr_t a = reinterpret_cast<uintptr_t>(w.drow + w.c_lo * E);
            w.sh = (uint32_t)(a & 15);
            w.g0 = a - w.sh;
            w.bytes = (uint32_t)(w.c_hi - w.c_lo) * 16 + (w.sh ? 16u : 0u);
        }
    };
    uint32_t pending = 0;  // bit b: a copy into buffer b has been requested and not yet waited for
    auto issue = [&](const Win& w, int b) {
        if (w.bytes == 0) return;
        pending |= 1u << b;
        if (lane != 0) return;
        const uint32_t bar = smem_addr(&bars[b]);
        // the warp's earlier generic-proxy reads of this buffer come before the async-proxy overwrite
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        const uint32_t fbytes = MUL ? (uint32_t)(w.c_hi - w.c_lo) * 16u : 0u;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(w.bytes + fbytes) : "memory");
        if (MUL)  // the packed factor's chunks of the window: aligned and contiguous
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                             smem_addr(buf0 + (D + b) * kBulkBufBytes)),
                         "l"(factor + w.c_lo * E), "r"(fbytes), "r"(bar)
                         : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                         smem_addr(buf0 + b * kBulkBufBytes)),
                     "l"(w.g0), "r"(w.bytes), "r"(bar)
                     : "memory");
    };

    Win ahead[D - 1];  // windows already requested, oldest first (static indices only: stays in registers)
    int64_t item = blockIdx.x * (int64_t)kWarpsPerBlock + warp;
#pragma unroll
    for (int d = 0; d < D - 1; ++d) {
        describe(item + d * warps, ahead[d]);
        issue(ahead[d], d);
    }
    uint32_t phases = 0;  // bit b: parity of the next completion of buffer b
    bool dead = false;    // a wait ran out: stop, report, let the copies in flight land
    int b = 0;
    for (; item < items; item += warps, b = (b + 1 == D ? 0 : b + 1)) {
        const Win cur = ahead[0];
#pragma unroll
        for (int d = 0; d + 1 < D - 1; ++d) ahead[d] = ahead[d + 1];
        // the window D - 1 items ahead goes into the buffer that was consumed one iteration ago (all
        // lanes passed the __syncwarp below)
        describe(item + (D - 1) * warps, ahead[D - 2]);
        issue(ahead[D - 2], b == 0 ? D - 1 : b - 1);
        if (cur.live) {
            if (cur.bytes) {
                // never expected to run out; if it does, nothing of this window is stored
                if (!__all_sync(0xffffffffu, mbar_wait_bounded(smem_addr(&bars[b]), (phases >> b) & 1u, wait_budget))) {
                    dead = true;
                    break;
                }
                pending &= ~(1u << b);
                phases ^= 1u << b;
                const uint8_t* src = buf0 + b * kBulkBufBytes;
                const uint4 zero4 = make_uint4(0, 0, 0, 0);
#pragma unroll 4
                for (int64_t c = cur.c_lo + lane; c < cur.c_hi; c += 32) {
                    const uint4* g = reinterpret_cast<const uint4*>(src + (c - cur.c_lo) * 16);
                    const uint4 lo = g[0];
                    const uint4 hi = cur.sh ? g[1] : zero4;
                    uint4 v = realign16(lo, hi, cur.sh);
                    if (MUL) {  // fp32: four elements per chunk
                        const uint4 f = *reinterpret_cast<const uint4*>(buf0 + (D + b) * kBulkBufBytes + (c - cur.c_lo) * 16);
                        uint4 old = zero4;
                        if (accumulate) old = *reinterpret_cast<const uint4*>(packed + c * E);
                        v.x = mul_acc((T)v.x, (T)f.x, (T)old.x, accumulate != 0);
                        v.y = mul_acc((T)v.y, (T)f.y, (T)old.y, accumulate != 0);
                        v.z = mul_acc((T)v.z, (T)f.z, (T)old.z, accumulate != 0);
                        v.w = mul_acc((T)v.w, (T)f.w, (T)old.w, accumulate != 0);
                    }
                    *reinterpret_cast<uint4*>(packed + c * E) = v;
                }
            }
            // chunks of this window that the row shares with a neighbour (or the tail of the stream)
            for (int side = 0; side < 2; ++side) {
                const int64_t c = side == 0 ? cur.ps / E : cur.pe / E;
                const bool mine = c >= cur.c0 && c < cur.c0 + kBulkWin && (c < cur.c_lo || c >= cur.c_hi) &&
                                  !(side == 1 && c == cur.ps / E) && c * E < cur.pe;
                if (mine && lane < E) {
                    const int64_t p = c * E + lane;
                    if (p >= cur.ps && p < cur.pe)
                        packed[p] = MUL ? mul_acc(cur.drow[p], factor[p], packed[p], accumulate != 0) : cur.drow[p];
                    else if (p >= m.count && !(MUL && accumulate))
                        packed[p] = T(0);
                }
            }
        }
        __syncwarp();
    }
    if (dead) {
        if (lane == 0 && err_word) atomicExch(err_word, kErrWordPack);
        for (int d = 0; d < D; ++d)  // the copies still in flight get one more budget to land
            if (pending & (1u << d)) mbar_wait_bounded(smem_addr(&bars[d]), (phases >> d) & 1u, wait_budget);
    }
}

// unpack through shared memory, the mirror image: a window is 256 aligned chunks of a dense row; the
// packed elements it needs are one contiguous run, fetched by one bulk copy; chunks wholly inside
// the set are realigned from the buffer, chunks wholly outside are zero stores, the at most two
// chunks that straddle an end of the row's interval are assembled element by element.
template <typename T>
__global__ void __launch_bounds__(32 * kWarpsPerBlock, 3)
unpack_bulk_kernel(IndexMap m, const T* __restrict__ packed, T* __restrict__ dense, Strides st, int64_t rows,
                   int windows_per_row, long long wait_budget, int32_t* __restrict__ err_word) {
    constexpr int E = 16 / sizeof(T);
    extern __shared__ __align__(128) uint8_t bulk_smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int D = kUnpackDepth;
    uint8_t* buf0 = bulk_smem + warp * D * kBulkBufBytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(bulk_smem + kWarpsPerBlock * D * kBulkBufBytes) + warp * D;
    if (lane == 0) {
        for (int d = 0; d < D; ++d) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(&bars[d])));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const int inner = (int)(m.rank == 3 ? m.dims[2] : m.rank == 2 ? m.dims[1] : m.dims[0]);

    struct Win {
        int jlo, jhi;        // the row's interval of stored columns
        int wlo, whi;        // columns of the window (whi clipped to the row)
        int c_lo, c_hi;      // columns [c_lo, c_hi): chunks wholly inside the interval, multiples of E
        T* drow;
        const T* prow;       // prow[j] = stored element (row, j)
        uintptr_t g0;        // aligned source address under column c_lo
        uint32_t sh, bytes;
        bool live;
    };
    const int64_t items = rows * windows_per_row;
    const int64_t warps = (int64_t)gridDim.x * kWarpsPerBlock;
    auto describe = [&](int64_t item, Win& w) {
        w.live = false;
        w.bytes = 0;
        w.sh = 0;
        w.g0 = 0;
        w.c_lo = w.c_hi = 0;
        if (item >= items) return;
        const int64_t row = item / windows_per_row;
        const int win = (int)(item - row * windows_per_row);
        w.wlo = win * kBulkWin * E;
        if (w.wlo >= inner) return;
        w.whi = w.wlo + kBulkWin * E < inner ? w.wlo + kBulkWin * E : inner;
        w.live = true;
        int32_t idx[3] = {0, 0, 0};
        if (m.rank == 2) {
            idx[0] = (int32_t)row;
        } else if (m.rank == 3) {
            const int64_t q = row / m.dims[1];
            idx[1] = (int32_t)(row - q * m.dims[1]);
            idx[0] = (int32_t)q;
        }
        int64_t jlo64 = 0, jhi64 = 0, pbase = 0;
        if (!row_span(m, idx, jlo64, jhi64, pbase)) jlo64 = jhi64 = 0;
        w.jlo = (int)jlo64;
        w.jhi = (int)jhi64;
        w.drow = dense + dense_row_offset(m, st, idx);
        w.prow = packed + pbase;
        // whole chunks inside both the interval and the window
        int lo = w.jlo > w.wlo ? w.jlo : w.wlo, hi = w.jhi < w.whi ? w.jhi : w.whi;
        lo = (lo + E - 1) / E * E;
        hi = hi / E * E;
        if (hi > lo) {
            w.c_lo = lo;
            w.c_hi = hi;
            const uintptr_t a = reinterpret_cast<uintptr_t>(w.prow + lo);
            w.sh = (uint32_t)(a & 15);
            w.g0 = a - w.sh;
            w.bytes = (uint32_t)((hi - lo) / E) * 16 + (w.sh ? 16u : 0u);
        }
    };
    uint32_t pending = 0;  // bit b: a copy into buffer b has been requested and not yet waited for
    auto issue = [&](const Win& w, int b) {
        if (w.bytes == 0) return;
        pending |= 1u << b;
        if (lane != 0) return;
        const uint32_t bar = smem_addr(&bars[b]);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(w.bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                         smem_addr(buf0 + b * kBulkBufBytes)),
                     "l"(w.g0), "r"(w.bytes), "r"(bar)
                     : "memory");
    };
    union Chunk {
        uint4 v;
        T e[E];
    };
    const uint4 zero4 = make_uint4(0, 0, 0, 0);

    Win ahead[D - 1];  // windows already requested, oldest first
    int64_t item = blockIdx.x * (int64_t)kWarpsPerBlock + warp;
#pragma unroll
    for (int d = 0; d < D - 1; ++d) {
        describe(item + d * warps, ahead[d]);
        issue(ahead[d], d);
    }
    uint32_t phases = 0;
    bool dead = false;
    int b = 0;
    for (; item < items; item += warps, b = (b + 1 == D ? 0 : b + 1)) {
        const Win cur = ahead[0];
#pragma unroll
        for (int d = 0; d + 1 < D - 1; ++d) ahead[d] = ahead[d + 1];
        describe(item + (D - 1) * warps, ahead[D - 2]);
        issue(ahead[D - 2], b == 0 ? D - 1 : b - 1);
        if (cur.live) {
            if (cur.bytes) {
                // never expected to run out; if it does, nothing of this window is stored
                if (!__all_sync(0xffffffffu, mbar_wait_bounded(smem_addr(&bars[b]), (phases >> b) & 1u, wait_budget))) {
                    dead = true;
                    break;
                }
                pending &= ~(1u << b);
                phases ^= 1u << b;
            }
            const uint8_t* src = buf0 + b * kBulkBufBytes;
            for (int j0 = cur.wlo + lane * E; j0 < cur.whi; j0 += 32 * E) {
                Chunk out;
                out.v = zero4;
                if (j0 >= cur.c_lo && j0 + E <= cur.c_hi) {
                    const uint4* g = reinterpret_cast<const uint4*>(src + (size_t)(j0 - cur.c_lo) / E * 16);
                    out.v = realign16(g[0], cur.sh ? g[1] : zero4, cur.sh);
                } else if (j0 + E > cur.jlo && j0 < cur.jhi) {  // straddles an end of the interval
#pragma unroll
                    for (int e = 0; e < E; ++e)
                        if (j0 + e >= cur.jlo && j0 + e < cur.jhi) out.e[e] = cur.prow[j0 + e];
                }
                if (j0 + E <= inner) {
                    *reinterpret_cast<uint4*>(cur.drow + j0) = out.v;
                } else {
                    for (int e = 0; e < E && j0 + e < inner; ++e) cur.drow[j0 + e] = out.e[e];
                }
            }
        }
        __syncwarp();
    }
    if (dead) {
        if (lane == 0 && err_word) atomicExch(err_word, kErrWordUnpack);
        for (int d = 0; d < D; ++d)  // the copies still in flight get one more budget to land
            if (pending & (1u << d)) mbar_wait_bounded(smem_addr(&bars[d]), (phases >> d) & 1u, wait_budget);
    }
}

// The upper half cube (i <= j, dense l) with compact inner strides is, for copying, a matrix whose
// row i holds the columns j Q + l, j >= i: one long contiguous interval per row instead of N - i short
// ones.  Rewrites the map and the strides in place when that view applies.
void collapse_half_cube(IndexMap& m, Strides& st) {
    if (m.kind == kUpper && m.rank == 3 && m.Q > 1 && st.s[2] == 1 && st.s[1] == m.Q &&
        m.N * m.Q < (int64_t(1) << 30)) {
        m.rank = 2;
        m.dims[1] = m.N * m.Q;
        m.dims[2] = 0;
        st.s[1] = 1;
        st.s[2] = 0;
    }
}

bool row_path(const IndexMap& m) {
    return (m.kind == kDense || (m.kind == kUpper && m.rank == 2) || m.kind == kLower || m.kind == kTetrahedron ||
            m.kind == kBandExact || m.kind == kUpperShifted || m.kind == kBandOffsets) &&
           !m.symmetric;
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

// out[p] = Bp[p] * C[idx(p)] (+ out[p]) over the packed positions of a structure: the tensor Hadamard
// product with a structured first operand (A(i,j,k) := B(i,j,k) * C(i,j,k), Table 1 "THP").  The dense
// factor is gathered exactly as pack gathers it, so this is pack with one multiply per element.
dastac_status launch_hadamard(const IndexMap& m, const float* Bp, const float* C, const int64_t* c_strides,
                              float* out, int accumulate, cudaStream_t stream) {
    if (m.slots == 0) return DASTAC_OK;
    Strides st{{0, 0, 0}};
    for (int k = 0; k < m.rank; ++k) st.s[k] = c_strides[k];
    constexpr int E = 4;
    const uint32_t* Cq = reinterpret_cast<const uint32_t*>(C);
    const uint32_t* Bq = reinterpret_cast<const uint32_t*>(Bp);
    uint32_t* Oq = reinterpret_cast<uint32_t*>(out);
    IndexMap mc = m;
    if (aligned16(C)) collapse_half_cube(mc, st);
    if (mc.rank != m.rank) return launch_hadamard(mc, Bp, C, st.s, out, accumulate, stream);
    if (row_path(m) && st.s[m.rank - 1] == 1 && aligned16(C)) {
        int64_t rows = 1;
        for (int k = 0; k + 1 < m.rank; ++k) rows *= m.dims[k];
        static bool attr_set[64];
        int dev = 0;
        cudaGetDevice(&dev);
        if (dev >= 0 && dev < 64 && !attr_set[dev]) {
            if (cudaFuncSetAttribute(pack_bulk_kernel<uint32_t, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     kBulkSmemBytesMul) != cudaSuccess)
                return DASTAC_ERR_CUDA;
            attr_set[dev] = true;
        }
        const int64_t bwpr = ((m.dims[m.rank - 1] + E - 1) / E + 2 + kBulkWin - 1) / kBulkWin;
        if (bwpr > 0x7fffffffLL) return DASTAC_ERR_OVERFLOW;
        const int64_t items = rows * bwpr;
        int64_t blocks = (items + kWarpsPerBlock - 1) / kWarpsPerBlock;
        if (blocks > (int64_t)sm_count()) blocks = (int64_t)sm_count();  // four buffers per warp: one CTA per SM
        pack_bulk_kernel<uint32_t, true><<<(unsigned)blocks, 32 * kWarpsPerBlock, kBulkSmemBytesMul, stream>>>(
            m, Cq, st, Oq, rows, (int)bwpr, kDefaultWaitBudget, device_error_word(), Bq, accumulate);
        return launch_status();
    }
    const int grid = grid_for((m.slots + E - 1) / E, 256);
    pack_kernel<uint32_t, true><<<grid, 256, 0, stream>>>(m, Cq, st, Oq, Bq, accumulate);
    return launch_status();
}

}  // namespace dastac

using namespace dastac;

extern "C" dastac_status dastac_rank_batch(const dastac_structure* s, const int32_t* idx, int64_t n,
                                           int64_t* off, void* stream) {
    if (!s || n < 0 || (n > 0 && (!idx || !off))) return DASTAC_ERR_INVALID_ARG;
    if (n == 0) return DASTAC_OK;
    if (s->map.kind == kGeneric) {
        g_rank_batch_kernel<<<grid_for(n, 256), 256, 0, (cudaStream_t)stream>>>(*s->generic, idx, n, off);
        return launch_status();
    }
    rank_batch_kernel<<<grid_for(n, 256), 256, 0, (cudaStream_t)stream>>>(s->map, idx, n, off);
    return launch_status();
}

extern "C" dastac_status dastac_unrank_batch(const dastac_structure* s, const int64_t* off,
                                             int64_t n, int32_t* idx, void* stream) {
    if (!s || n < 0 || (n > 0 && (!idx || !off))) return DASTAC_ERR_INVALID_ARG;
    if (n == 0) return DASTAC_OK;
    if (s->map.kind == kGeneric) {
        g_unrank_batch_kernel<<<grid_for(n, 256), 256, 0, (cudaStream_t)stream>>>(*s->generic, off, n, idx);
        return launch_status();
    }
    unrank_batch_kernel<<<grid_for(n, 256), 256, 0, (cudaStream_t)stream>>>(s->map, off, n, idx);
    return launch_status();
}

extern "C" dastac_status dastac_pack(const dastac_structure* s, dastac_dtype dtype,
                                     const void* dense, const int64_t* dense_strides, void* packed,
                                     void* stream) {
    if (!s || !dense_strides) return DASTAC_ERR_INVALID_ARG;
    if (dtype != DASTAC_F32 && dtype != DASTAC_BF16) return DASTAC_ERR_INVALID_ARG;
    IndexMap m = s->map;
    if (!strides_ok(m, dense_strides)) return DASTAC_ERR_INVALID_ARG;
    if (m.slots == 0) return DASTAC_OK;
    if (!dense || !packed) return DASTAC_ERR_INVALID_ARG;
    if (!aligned16(packed)) return DASTAC_ERR_ALIGNMENT;
    Strides st{{0, 0, 0}};
    for (int k = 0; k < m.rank; ++k) st.s[k] = dense_strides[k];
    if (m.kind == kGeneric) {
        const GenericMap& g = *s->generic;
        const int64_t fibres = g.rank == 2 ? g.dims[0] : g.dims[0] * g.dims[1];
        const int grid = grid_for(fibres * 32, 256);
        if (dtype == DASTAC_F32)
            g_fibre_copy_kernel<uint32_t, false><<<grid, 256, 0, (cudaStream_t)stream>>>(g, (uint32_t*)const_cast<void*>(dense), st, (uint32_t*)packed);
        else
            g_fibre_copy_kernel<uint16_t, false><<<grid, 256, 0, (cudaStream_t)stream>>>(g, (uint16_t*)const_cast<void*>(dense), st, (uint16_t*)packed);
        return launch_status();
    }
    const int E = 16 / elt_size(dtype);
    // (the row kernels below only use the row intervals, which the collapsed view provides)
    if ((reinterpret_cast<uintptr_t>(dense) % elt_size(dtype)) == 0) collapse_half_cube(m, st);
    if (row_path(m) && st.s[m.rank - 1] == 1 && (reinterpret_cast<uintptr_t>(dense) % elt_size(dtype)) == 0) {
        int64_t rows = 1;
        for (int k = 0; k + 1 < m.rank; ++k) rows *= m.dims[k];
        const int64_t chunks_per_row = (m.dims[m.rank - 1] + E - 1) / E + 1;  // a span may straddle one more chunk
        const int64_t wpr = (chunks_per_row + 32 * kUnroll - 1) / (32 * kUnroll);
        const int64_t want_items = (int64_t)sm_count() * 3 * kWarpsPerBlock * 4;
        int64_t gpr = rows >= want_items ? 1 : (want_items + rows - 1) / rows;
        if (gpr > wpr) gpr = wpr;
        const int64_t wpg = (wpr + gpr - 1) / gpr;
        gpr = (wpr + wpg - 1) / wpg;
        if (aligned16(dense)) {
            // windows arrive by bulk copies into shared memory
            static bool attr_set[64];
            int dev = 0;
            cudaGetDevice(&dev);
            if (dev >= 0 && dev < 64 && !attr_set[dev]) {
                if (cudaFuncSetAttribute(pack_bulk_kernel<uint32_t>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         bulk_smem_bytes(kPackDepth)) != cudaSuccess ||
                    cudaFuncSetAttribute(pack_bulk_kernel<uint16_t>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         bulk_smem_bytes(kPackDepth)) != cudaSuccess)
                    return DASTAC_ERR_CUDA;
                attr_set[dev] = true;
            }
            const int64_t bwpr = ((m.dims[m.rank - 1] + E - 1) / E + 2 + kBulkWin - 1) / kBulkWin;
            const int64_t items = rows * bwpr;
            int64_t blocks = (items + kWarpsPerBlock - 1) / kWarpsPerBlock;
            if (blocks > (int64_t)sm_count() * bulk_ctas_per_sm(kPackDepth)) blocks = (int64_t)sm_count() * bulk_ctas_per_sm(kPackDepth);
            if (bwpr > 0x7fffffffLL) return DASTAC_ERR_OVERFLOW;
            if (dtype == DASTAC_F32)
                pack_bulk_kernel<uint32_t><<<(unsigned)blocks, 32 * kWarpsPerBlock, bulk_smem_bytes(kPackDepth), (cudaStream_t)stream>>>(
                    m, (const uint32_t*)dense, st, (uint32_t*)packed, rows, (int)bwpr, kDefaultWaitBudget, device_error_word());
            else
                pack_bulk_kernel<uint16_t><<<(unsigned)blocks, 32 * kWarpsPerBlock, bulk_smem_bytes(kPackDepth), (cudaStream_t)stream>>>(
                    m, (const uint16_t*)dense, st, (uint16_t*)packed, rows, (int)bwpr, kDefaultWaitBudget, device_error_word());
            return launch_status();
        }
        const int grid = grid_for(rows * gpr * 32, 32 * kWarpsPerBlock);
        if (dtype == DASTAC_F32)
            pack_stream_kernel<uint32_t><<<grid, 32 * kWarpsPerBlock, 0, (cudaStream_t)stream>>>(
                m, (const uint32_t*)dense, st, (uint32_t*)packed, rows, (int)gpr, (int)wpg);
        else
            pack_stream_kernel<uint16_t><<<grid, 32 * kWarpsPerBlock, 0, (cudaStream_t)stream>>>(
                m, (const uint16_t*)dense, st, (uint16_t*)packed, rows, (int)gpr, (int)wpg);
        return launch_status();
    }
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
    IndexMap m = s->map;
    if (!strides_ok(m, dense_strides)) return DASTAC_ERR_INVALID_ARG;
    int64_t box = 1;
    for (int k = 0; k < m.rank; ++k)
        if (__builtin_mul_overflow(box, m.dims[k], &box)) return DASTAC_ERR_OVERFLOW;  // no such tensor fits in memory
    if (box == 0) return DASTAC_OK;
    if (!dense || (m.slots > 0 && !packed)) return DASTAC_ERR_INVALID_ARG;
    if (m.slots > 0 && !aligned16(packed)) return DASTAC_ERR_ALIGNMENT;
    Strides st{{0, 0, 0}};
    for (int k = 0; k < m.rank; ++k) st.s[k] = dense_strides[k];
    if (m.kind == kGeneric) {
        const GenericMap& g = *s->generic;
        const int64_t fibres = g.rank == 2 ? g.dims[0] : g.dims[0] * g.dims[1];
        const int grid = grid_for(fibres * 32, 256);
        if (dtype == DASTAC_F32)
            g_fibre_copy_kernel<uint32_t, true><<<grid, 256, 0, (cudaStream_t)stream>>>(g, (uint32_t*)dense, st, (uint32_t*)const_cast<void*>(packed));
        else
            g_fibre_copy_kernel<uint16_t, true><<<grid, 256, 0, (cudaStream_t)stream>>>(g, (uint16_t*)dense, st, (uint16_t*)const_cast<void*>(packed));
        return launch_status();
    }
    const int esz = elt_size(dtype);
    const int E = 16 / esz;
    // 128-bit stores need a unit inner stride, a 16-byte aligned base and outer strides that keep
    // every row start on a 16-byte boundary.
    int vector_ok = st.s[m.rank - 1] == 1 && aligned16(dense);
    for (int k = 0; k + 1 < m.rank; ++k) vector_ok = vector_ok && (st.s[k] % E == 0);
    if (vector_ok) collapse_half_cube(m, st);  // the row kernel only uses the row intervals
    if (row_path(m) && vector_ok) {
        const int64_t rows = box / m.dims[m.rank - 1];
        const int64_t chunks_per_row = (m.dims[m.rank - 1] + E - 1) / E;
        {
            static bool attr_set[64];
            int dev = 0;
            cudaGetDevice(&dev);
            if (dev >= 0 && dev < 64 && !attr_set[dev]) {
                if (cudaFuncSetAttribute(unpack_bulk_kernel<uint32_t>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         bulk_smem_bytes(kUnpackDepth)) != cudaSuccess ||
                    cudaFuncSetAttribute(unpack_bulk_kernel<uint16_t>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         bulk_smem_bytes(kUnpackDepth)) != cudaSuccess)
                    return DASTAC_ERR_CUDA;
                attr_set[dev] = true;
            }
            const int64_t bwpr = (chunks_per_row + kBulkWin - 1) / kBulkWin;
            const int64_t items = rows * bwpr;
            int64_t blocks = (items + kWarpsPerBlock - 1) / kWarpsPerBlock;
            if (blocks > (int64_t)sm_count() * bulk_ctas_per_sm(kUnpackDepth)) blocks = (int64_t)sm_count() * bulk_ctas_per_sm(kUnpackDepth);
            if (bwpr > 0x7fffffffLL || m.dims[m.rank - 1] > (int64_t(1) << 30)) return DASTAC_ERR_OVERFLOW;
            if (dtype == DASTAC_F32)
                unpack_bulk_kernel<uint32_t><<<(unsigned)blocks, 32 * kWarpsPerBlock, bulk_smem_bytes(kUnpackDepth), (cudaStream_t)stream>>>(
                    m, (const uint32_t*)packed, (uint32_t*)dense, st, rows, (int)bwpr, kDefaultWaitBudget, device_error_word());
            else
                unpack_bulk_kernel<uint16_t><<<(unsigned)blocks, 32 * kWarpsPerBlock, bulk_smem_bytes(kUnpackDepth), (cudaStream_t)stream>>>(
                    m, (const uint16_t*)packed, (uint16_t*)dense, st, rows, (int)bwpr, kDefaultWaitBudget, device_error_word());
            return launch_status();
        }
    }
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
