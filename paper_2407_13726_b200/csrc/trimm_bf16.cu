// C = A B for a packed upper-triangular bf16 A (row-packed, position rowbase(i) + j) and a dense
// row-major bf16 B, fp32 accumulation in tensor memory, fp32 output.  The paper has no tensor-core
// kernel; this is its SpMV_UT / TTM_UT access pattern (Table 1) widened to a dense right-hand
// side and mapped on tcgen05.
//
// Tiling.  An output tile is 256 rows x 256 columns, computed by a cluster of two CTAs (one SM
// each) with tcgen05.mma.cta_group::2: CTA r holds row block 2P + r (128 rows).  A pair only needs
// K blocks (64 columns of A, 64 rows of B) from its diagonal on: kb = 4P .. ceil(N/64)-1, so the
// executed MMA work is the triangle plus one tile per pair.  Tiles are ordered by decreasing K
// length and dealt to the persistent clusters in boustrophedon order, which gives every cluster
// the same mix of long and short tiles.
//
// Two kernels per call:
//  1. stage_a: the packed row pitch changes with the row and row starts are only 2-byte aligned,
//     so no tensor map can describe A.  Every 128x64 tile of the triangle is therefore re-laid
//     once into the workspace as the exact shared-memory image the K-major, 128-byte-swizzled
//     UMMA descriptor expects (16 KiB per tile): eight lanes cover one row with aligned 128-bit
//     loads, the row's constant misalignment (0..7 elements, a function of rowbase(i) only) is
//     removed in registers with a two-level word select and a funnel shift, and entries left of
//     the diagonal or beyond column N are zeroed.  Doing this once per call instead of once per
//     column tile keeps the realignment off the MMA critical path (each A tile is consumed by
//     every column tile of its row block).  The workspace stays packed: it holds the triangle's
//     tiles only.  The images form a plain [tiles x 128][64] array, which a tensor map without
//     swizzle copies verbatim.
//  2. trimm_pair: warp-specialised pipeline (details at the kernel).
//
// The same CTA-pair pipeline also evaluates the polynomial-regression moments of Table 1 (degree 2:
// B^T B on i1 <= i2 with packed output; degree 3: the packed tetrahedron i1 <= i2 <= i3, with the
// scaled operand in tensor memory); their differences are described at the kernel.
//
// Every wait on an mbarrier is bounded by a clock budget; on expiry the thread records a code in
// the error word and the CTA drains: nothing can spin forever.
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"

namespace dastac {
namespace {

constexpr int kTileM = 128, kTileN = 256, kBlockK = 64;
constexpr int kABytes = kTileM * kBlockK * 2;  // 16 KiB
constexpr int kTmemCols = 512;
constexpr long long kWaitBudget = 4000000000LL;  // clock cycles (~2 s) before a wait gives up

enum ErrCode : int32_t { kErrFull = 1, kErrEmpty = 3, kErrTmemFull = 4, kErrTmemEmpty = 5 };

// ---- PTX wrappers ------------------------------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: returns false (and records `code`) when the clock budget runs out or when another
// thread of the CTA has already given up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int32_t* err_word, int32_t code) {
    if (mbar_test(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        if (mbar_test(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitBudget) {
            *abort_flag = 1;
            if (err_word) atomicCAS(err_word, 0, code);
            return false;
        }
    }
}
// Warp-wide form: lane 0 waits and the verdict is shared, so a warp never splits on a timeout.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                               int32_t* err_word, int32_t code, int lane) {
    int ok = 1;
    if (lane == 0) ok = mbar_wait(bar, parity, abort_flag, err_word, code) ? 1 : 0;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    __syncwarp();
    return ok != 0;
}
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
// 32 consecutive 32-bit columns of this thread's lane, from registers.
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
          "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
          "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() {
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor (sm_100 format): start address, leading / stride byte offsets
// (all in 16-byte units), descriptor version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;  // version
    d |= (uint64_t)2 << 61;  // SWIZZLE_128B
    return d;
}

// Staged tile (I, kb) lives at tile index tile_offset(I) + kb - 4*(I/2): row blocks are stored in
// pairs that start at the same K block, so that two row blocks can later share one K loop; the
// two tiles this adds in front of every odd row block are all zero.
__host__ __device__ __forceinline__ int64_t tile_offset(int64_t I, int64_t k_blocks) {
    const int64_t P = I >> 1;
    return 2 * P * k_blocks - 4 * P * (P - 1) + (I & 1) * (k_blocks - 4 * P);
}

struct Params {
    const __nv_bfloat16* A;      // packed rows (stage_a) / unused (main)
    const uint8_t* tiles;        // staged tile images, 16 KiB each
    float* C;
    int64_t N, ncols, ldc;
    int64_t M;           // moment forms only: number of samples (rows of B)
    // degree-3 moments only: slabs i1 = i1_first .. i1_first + slots - 1 are computed by this launch
    int32_t i1_first, slots;
    int64_t tiles_total;
    int64_t cap_elems;   // capacity of the packed buffer in elements (multiple of 8)
    int32_t row_blocks, col_blocks, k_blocks;
    int32_t accumulate;
    int32_t vector_store;  // C allows 128-bit stores
    int32_t* err_word;
};

// ---- CTA-pair kernel ------------------------------------------------------------------------------
// A 256 x 256 output tile is computed by a cluster of two CTAs with tcgen05.mma.cta_group::2
// (M256 N256 K16).  CTA r of the pair stages the A tile of row block 2P + r and the 128-column half
// r of the B block, so each SM moves 32 KiB per K block and the tensor core of each SM reads half
// of B from its own shared memory and half from its peer's.  Each CTA holds the 128 x 256
// accumulator of its own row block, double buffered in its tensor memory, and its four epilogue
// warps drain one buffer while the MMAs of the next tile fill the other.
//   - Both CTAs' loads of a stage complete on the full barrier of CTA 0 (the MMA issuer); a
//     cta_group::2 tensor copy may name a barrier of the peer CTA.
//   - One commit with a two-CTA mask releases a stage (or publishes an accumulator) in both CTAs.
//   - CTA 1's epilogue warps release an accumulator with an arrive on CTA 0's barrier.
constexpr int kPStages = 6;
constexpr int kPBBytes = kBlockK * (kTileN / 2) * 2;   // 16 KiB: this CTA's half of the B block
constexpr int kPStageBytes = kABytes + kPBBytes;       // 32 KiB
constexpr int kPThreads = 6 * 32;                      // warps 0-3 epilogue, 4 producer, 5 MMA
constexpr int kPWarpTma = 4, kPWarpMma = 5;
constexpr size_t kPSmemBytes = (size_t)kPStages * kPStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
// fp32 accumulator, bf16 A (K-major) and bf16 B (MN-major), M256 N256 across the pair
constexpr uint32_t kPIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (0u << 15) | (1u << 16) |
                             ((uint32_t)(kTileN >> 3) << 17) | ((uint32_t)((2 * kTileM) >> 4) << 24);

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_test_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                  int32_t* err_word, int32_t code) {
    if (mbar_test_cluster(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        if (mbar_test_cluster(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > kWaitBudget) {
            *abort_flag = 1;
            if (err_word) atomicCAS(err_word, 0, code);
            return false;
        }
    }
}
// Tensor copy whose completion bytes go to `bar`, a shared::cluster address that may lie in the peer CTA.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
// Tensor copy into this CTA's shared memory, completing on a barrier of this CTA.
__device__ __forceinline__ void tma_load_2d_local(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t slot_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The same with the A operand in tensor memory (K-major: lane = row, two bf16 per 32-bit column).
__device__ __forceinline__ void umma_bf16_pair_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                                  uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrive on the barrier at this shared-memory offset in both CTAs of the pair once the MMAs issued so far retire.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"((uint16_t)3)
        : "memory");
}

//
// MOMENT2 (the degree-2 moments A2(i1,i2) = sum_x B(x,i1) B(x,i2) of polynomial regression, Table 1,
// kept on i1 <= i2 and stored packed): the same pipeline with both operands read from B.  The "A"
// operand is B transposed, which the tensor core takes directly as an M-major operand: CTA r copies
// the 64 x 128 block of B at columns 128 (2P + r) with the same two swizzled boxes it uses for its
// half of the "B" operand, and the instruction descriptor marks A as M-major.  Tiles are the
// 256 x 256 blocks (P, J) with J >= P, every one with the full K loop over the samples; the
// epilogue writes element (i1, i2) at rowbase(i1) + i2 of the packed triangle and skips i2 < i1.
//
// MODE 2 (degree-3 moments A3(i1,i2,i3) = sum_x B(x,i1) B(x,i2) B(x,i3) on i1 <= i2 <= i3, the
// hyper-triangular domain of Section 1, stored as the packed tetrahedron): for a fixed i1 the slab is
// the degree-2 product of Z_i1(x, i2) = B(x,i1) B(x,i2) with B, kept on i1 <= i2 <= i3.  Z is never
// stored: the "A" operand of the MMAs lives in tensor memory and extra warps write it (six sets of four
// warps, one set per stage, so that the waits inside one K block's work overlap with the others').  The
// host transposes B once (Bt, n x M, a few MB), so that row i2 of a K block is 128 contiguous bytes:
// a second producer copies the 128 x 64 block of Bt (128-byte swizzle) and the 64 values Bt(i1, x) of the
// slab's own column into the stage, completing on a barrier of the CTA itself; thread m of the
// product warps reads row m of the block (eight 128-bit loads), multiplies it by the column with
// packed bf16 multiplies (the product of two bf16 values rounded once, to nearest even) and stores
// the 64 products to lane m of the stage's 32 tensor-memory columns with tcgen05.st.  No generic
// write to shared memory is involved, hence no proxy fence (an earlier form that scaled the block
// in shared memory spent most of its time in fence.proxy.async).  One arrive per warp on the
// leader's full barrier (9 arrivals: 8 warps of the pair plus the producer's expect-tx for the "B"
// operand, which comes from B by TMA as for degree 2) publishes the stage.  Tensor memory holds one
// 256-column accumulator and six 32-column A stages.  Tiles are (slab, P, J) with P from the block
// that holds row i1 and J >= P; the epilogue writes at the tetrahedral position pbase(i1, i2) + i3.
enum PairMode : int { kModeTrimm = 0, kModeMoment2 = 1, kModeMoment3 = 2 };
// product warps 8..31: six sets of four, one set per stage; warp w writes tensor-memory lanes 32 (w mod 4) ..
constexpr int kScaleWarps = 4, kScaleSets = 6, kPWarpScale0 = 8, kPWarpRaw = 6;
constexpr int kPThreadsFused = 32 * (kPWarpScale0 + kScaleWarps * kScaleSets);  // 1024 (warp 6: second producer, warp 7 idle)
constexpr int kCxBytes = kBlockK * 2;                          // the 64 values B(x, i1) of a K block, per stage
constexpr int kTmemAStage0 = kTileN, kTmemAStageCols = kBlockK / 2;  // A stages behind the single accumulator
constexpr size_t kPSmemBytesFused = kPSmemBytes + (size_t)kPStages * kCxBytes;

template <int MODE>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(MODE == kModeMoment3 ? kPThreadsFused : kPThreads, 1)
trimm_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                  const __grid_constant__ CUtensorMap tmap_c, const Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* cxbuf = smem + (size_t)kPStages * kPStageBytes;  // degree 3 only
    uint64_t* bars = (uint64_t*)(cxbuf + (MODE == kModeMoment3 ? kPStages * kCxBytes : 0));
    // barrier slots: full[s], empty[s], tmem_full[2], tmem_empty[2], drain, (tmem slot, abort flag), rawfull[s]
    const uint32_t bar0 = smem_u32(bars);
    auto full = [&](int s) { return bar0 + 8u * s; };
    auto empty = [&](int s) { return bar0 + 8u * (kPStages + s); };
    auto tmem_full = [&](int a) { return bar0 + 8u * (2 * kPStages + a); };
    auto tmem_empty = [&](int a) { return bar0 + 8u * (2 * kPStages + 2 + a); };
    auto drain_bar = [&]() { return bar0 + 8u * (2 * kPStages + 4); };
    auto rawfull = [&](int s) { return bar0 + 8u * (2 * kPStages + 6 + s); };   // degree 3: this CTA's block of Bt has landed
    auto rawempty = [&](int s) { return bar0 + 8u * (3 * kPStages + 6 + s); };  // ... and has been read by the product warps
    uint32_t* tmem_slot = (uint32_t*)(bars + 2 * kPStages + 5);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = smem_u32(smem);
    const uint32_t rank = cluster_ctarank();  // 0: issues the MMAs, owns the full / tmem_empty barriers
    const bool leader = rank == 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kPStages; ++s) {
            mbar_init(full(s), MODE == kModeMoment3 ? 1 + 2 * kScaleWarps : 1);  // degree 3: the product warps of both CTAs as well
            mbar_init(empty(s), 1);
            if (MODE == kModeMoment3) {
                mbar_init(rawfull(s), 1);
                mbar_init(rawempty(s), kScaleWarps);
            }
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tmem_full(a), 1);
            mbar_init(tmem_empty(a), 2 * 4);  // four epilogue warps in each CTA
        }
        mbar_init(drain_bar(), 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == kPWarpMma) {
        tmem_alloc_pair(smem_u32(tmem_slot), kTmemCols);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // the peer's barriers exist before anything is signalled on them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // Tile t = (pair P, column block J), P ascending = K length descending, dealt to the clusters in
    // boustrophedon order.
    const int pair_blocks = (p.row_blocks + 1) >> 1;
    constexpr bool MOMENT2 = MODE != kModeTrimm;  // both moment forms share the operand handling of degree 2
    const int64_t tiles = MODE == kModeMoment3 ? p.tiles_total
                          : MOMENT2            ? (int64_t)pair_blocks * (pair_blocks + 1) / 2
                                               : (int64_t)pair_blocks * p.col_blocks;
    // tile index -> (slab, row-block pair P, column block J); moments: row P of the block triangle holds J = P ..
    auto decode = [&](int64_t t, int& P, int& J, int& slot) {
        slot = 0;
        if (MOMENT2) {
            int r = 0;
            if (MODE == kModeMoment3) {
                // slabs in order; the 256 slabs whose i1 lies in block row r all use block rows r .. and
                // have the same number of tiles
                for (r = 0; r + 1 < pair_blocks; ++r) {
                    const int64_t per_slab = (int64_t)(pair_blocks - r) * (pair_blocks - r + 1) / 2;
                    const int64_t in_block = per_slab * (2 * kTileM);
                    if (t < in_block) break;
                    t -= in_block;
                    slot += 2 * kTileM;
                }
                const int64_t per_slab = (int64_t)(pair_blocks - r) * (pair_blocks - r + 1) / 2;
                slot += (int)(t / per_slab);
                t %= per_slab;
            }
            while (t >= pair_blocks - r) {
                t -= pair_blocks - r;
                ++r;
            }
            P = r;
            J = r + (int)t;
        } else {
            P = (int)(t / p.col_blocks);
            J = (int)(t - (int64_t)P * p.col_blocks);
        }
    };
    auto kb_first = [&](int P) { return MOMENT2 ? 0 : 4 * P; };
    // Degree 3: in the column block that holds i1 itself the columns i3 < i1 belong to no element of
    // the slab; the MMAs of such a tile start at column c0 = i1 rounded down to 16 within the block
    // and are N = 256 - c0 wide (each CTA supplies half of those columns).
    auto col_skip = [&](int P, int J, int slot) {
        if (MODE != kModeMoment3) return 0;
        const int i1 = p.i1_first + slot;
        return (J == P && i1 / kTileN == J) ? ((i1 - J * kTileN) & ~15) : 0;
    };
    constexpr uint32_t kIdesc = MOMENT2 ? (kPIdesc | (1u << 15)) : kPIdesc;  // A operand M-major
    const int64_t G = gridDim.x >> 1, cid = blockIdx.x >> 1;
    auto tile_of = [&](uint32_t n) -> int64_t { return (int64_t)n * G + ((n & 1) ? (G - 1 - cid) : cid); };
    const uint32_t rounds = (uint32_t)((tiles + G - 1) / G);

    if (warp == kPWarpTma) {
        // ---- producer (both CTAs): this CTA's A tile and its half of the B block ---------------------
        if (lane == 0) {
            const uint32_t full0 = map_to_cta(full(0), 0);  // CTA 0's full barriers, 8 bytes apart
            uint32_t it = 0;
            bool ok = true;
            for (uint32_t n = 0; n < rounds && ok; ++n) {
                const int64_t t = tile_of(n);
                if (t >= tiles) continue;
                int P, J, slot;
                decode(t, P, J, slot);
                const int I = 2 * P + (int)rank;
                // staged tile (I, kb) sits at tile index tile_base + kb; a row block past the end of
                // the matrix has no tiles and its loads are out of range of the map: zero fill
                const int64_t tile_base = (I < p.row_blocks) ? tile_offset(I, p.k_blocks) - 4 * P : (int64_t)1 << 22;
                for (int kb = kb_first(P); kb < p.k_blocks; ++kb, ++it) {
                    const int s = it % kPStages;
                    if (it >= kPStages &&
                        !mbar_wait(empty(s), ((it / kPStages) - 1) & 1, abort_flag, p.err_word, kErrEmpty)) {
                        ok = false;
                        break;
                    }
                    const uint32_t dst = smem_base + s * kPStageBytes;
                    // both CTAs' bytes; degree 3: only the "B" operand comes by TMA
                    if (leader) mbar_arrive_expect_tx(full(s), MODE == kModeMoment3 ? 2 * kPBBytes : 2 * kPStageBytes);
                    const uint32_t bar = full0 + 8u * s;
                    if (MODE == kModeMoment3) {
                        // the block of Bt for the product warps has its own producer (below)
                    } else if (MOMENT2) {
#pragma unroll
                        for (int q = 0; q < kTileM / 64; ++q)
                            tma_load_2d_pair(dst + q * (kBlockK * 128), &tmap_b, I * kTileM + q * 64, kb * kBlockK, bar);
                    } else {
                        tma_load_2d_pair(dst, &tmap_a, 0, (int)((tile_base + kb) * kTileM), bar);
                    }
                    const int c0 = col_skip(P, J, slot);
#pragma unroll
                    for (int q = 0; q < kTileN / 128; ++q)
                        tma_load_2d_pair(dst + kABytes + q * (kBlockK * 128), &tmap_b,
                                         J * kTileN + c0 + (int)rank * ((kTileN - c0) / 2) + q * 64, kb * kBlockK, bar);
                }
            }
            if (!ok) {
                // give copies that are still in flight time to land before shared memory is released
                const long long t0 = clock64();
                while (clock64() - t0 < 2000000) {
                }
            }
        }
    } else if (MODE == kModeMoment3 && warp == kPWarpRaw) {
        // ---- second producer, degree 3 (both CTAs): the 128 x 64 block of Bt and the slab's own column for this
        // CTA's product warps.  Its ring is released by the product warps as soon as they have read a
        // block, not by the MMAs, so these copies run ahead of the tensor-memory stages.
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (uint32_t n = 0; n < rounds && ok; ++n) {
                const int64_t t = tile_of(n);
                if (t >= tiles) continue;
                int P, J, slot;
                decode(t, P, J, slot);
                const int I = 2 * P + (int)rank;
                for (int kb = 0; kb < p.k_blocks; ++kb, ++it) {
                    const int s = it % kPStages;
                    if (it >= kPStages &&
                        !mbar_wait(rawempty(s), ((it / kPStages) - 1) & 1, abort_flag, p.err_word, kErrEmpty)) {
                        ok = false;
                        break;
                    }
                    mbar_arrive_expect_tx(rawfull(s), kABytes + kCxBytes);
                    tma_load_2d_local(smem_base + s * kPStageBytes, &tmap_a, kb * kBlockK, I * kTileM, rawfull(s));
                    tma_load_2d_local(smem_u32(cxbuf) + s * kCxBytes, &tmap_c, kb * kBlockK, p.i1_first + slot, rawfull(s));
                }
            }
            if (!ok) {
                const long long t0 = clock64();
                while (clock64() - t0 < 2000000) {
                }
            }
        }
    } else if (MODE == kModeMoment3 && warp >= kPWarpScale0) {
        // ---- product warps (both CTAs): rows of the block times the slab's column, into tensor memory -----
        // A set of four warps handles every kScaleSets-th K block, so that the waits inside one
        // block's work (the copy, the free stage, the tensor-memory store) overlap with the other
        // set's.  A stage is always served by the same set (the stage count is a multiple of the sets).
        static_assert(kPStages % kScaleSets == 0, "a stage must stay with one set of product warps");
        const int set = (warp - kPWarpScale0) / kScaleWarps, quarter = (warp - kPWarpScale0) % kScaleWarps;
        const int m = 32 * quarter + lane;  // row of the block = tensor-memory lane
        const uint32_t full0 = map_to_cta(full(0), 0);
        uint32_t it = 0;
        bool ok = true;
        for (uint32_t n = 0; n < rounds && ok; ++n) {
            const int64_t t = tile_of(n);
            if (t >= tiles) continue;
            for (int kb = 0; kb < p.k_blocks && ok; ++kb, ++it) {
                if ((int)(it % kScaleSets) != set) continue;
                const int s = it % kPStages;
                if (!mbar_wait_warp(rawfull(s), (it / kPStages) & 1, abort_flag, p.err_word, kErrFull, lane)) {
                    ok = false;
                    break;
                }
                const uint8_t* row = smem + s * kPStageBytes + m * 128;  // 128-byte swizzle: chunk j sits at j xor (m mod 8)
                const uint4* cx = reinterpret_cast<const uint4*>(cxbuf + s * kCxBytes);
                uint32_t v[32];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    union {
                        uint4 q;
                        __nv_bfloat162 h[4];
                        uint32_t u[4];
                    } a, c;
                    a.q = *reinterpret_cast<const uint4*>(row + ((j ^ (m & 7)) << 4));
                    c.q = cx[j];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        a.h[e] = __hmul2(a.h[e], c.h[e]);
                        v[4 * j + e] = a.u[e];
                    }
                }
                // the block has been read: its shared-memory slot may be refilled
                __syncwarp();
                if (lane == 0) mbar_arrive(rawempty(s));
                // tensor-memory stage s is free once the MMAs that read it six K blocks ago have retired
                if (it >= kPStages &&
                    !mbar_wait_warp(empty(s), ((it / kPStages) - 1) & 1, abort_flag, p.err_word, kErrEmpty, lane)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                tmem_st32(tmem_base + ((uint32_t)(32 * quarter) << 16) + kTmemAStage0 + s * kTmemAStageCols, v);
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(full0 + 8u * s);
            }
        }
    } else if (warp == kPWarpMma) {
        // ---- MMA issuer (CTA 0 only) -----------------------------------------------------------------
        if (leader && lane == 0) {
            uint32_t it = 0, tile_n = 0;
            bool ok = true;
            for (uint32_t n = 0; n < rounds && ok; ++n) {
                const int64_t t = tile_of(n);
                if (t >= tiles) continue;
                int P, J, slot;
                decode(t, P, J, slot);
                // degree 3 has a single accumulator (the other half of tensor memory holds the A stages)
                const int acc = MODE == kModeMoment3 ? 0 : (tile_n & 1);
                const uint32_t use = MODE == kModeMoment3 ? tile_n : (tile_n >> 1);  // how often this buffer was used before
                if (use >= 1 &&
                    !mbar_wait_cluster(tmem_empty(acc), (use - 1) & 1, abort_flag, p.err_word, kErrTmemEmpty)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * kTileN;
                // degree 3: the instruction's N is the tile's width without the skipped columns
                const uint32_t idesc3 = (kPIdesc & ~(0x3Fu << 17)) | ((uint32_t)((kTileN - col_skip(P, J, slot)) >> 3) << 17);
                for (int kb = kb_first(P); kb < p.k_blocks; ++kb, ++it) {
                    const int s = it % kPStages;
                    if (!mbar_wait_cluster(full(s), (it / kPStages) & 1, abort_flag, p.err_word, kErrFull)) {
                        ok = false;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t a_addr = smem_base + s * kPStageBytes;
                    const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
                    for (int k16 = 0; k16 < kBlockK / 16; ++k16) {
                        const uint64_t da = MOMENT2 ? smem_desc(a_addr + k16 * 2048, kBlockK * 128, 1024)
                                                    : smem_desc(a_addr + k16 * 32, 16, 1024);
                        const uint64_t db = smem_desc(b_addr + k16 * 2048, kBlockK * 128, 1024);
                        if (MODE == kModeMoment3)
                            umma_bf16_pair_ts(d_tmem, tmem_base + kTmemAStage0 + s * kTmemAStageCols + k16 * 8, db, idesc3,
                                              (kb > 0 || k16 > 0) ? 1u : 0u);
                        else
                            umma_bf16_pair(d_tmem, da, db, kIdesc, (kb > kb_first(P) || k16 > 0) ? 1u : 0u);
                    }
                    umma_commit_pair(empty(s));
                }
                if (ok) umma_commit_pair(tmem_full(acc));
                ++tile_n;
            }
            if (!ok) {
                umma_commit_pair(drain_bar());
                const long long t0 = clock64();
                while (!mbar_test(drain_bar(), 0) && clock64() - t0 < kWaitBudget) {
                }
            }
        }
    } else if (warp < 4) {
        // ---- epilogue (both CTAs): this CTA's 128 rows of the tile ------------------------------------
        const uint32_t empty0 = map_to_cta(tmem_empty(0), 0);
        uint32_t tile_n = 0;
        bool ok = true;
        for (uint32_t n = 0; n < rounds && ok; ++n) {
            const int64_t t = tile_of(n);
            if (t >= tiles) continue;
            int P, J, slot;
            decode(t, P, J, slot);
            const int I = 2 * P + (int)rank;
            const int acc = MODE == kModeMoment3 ? 0 : (tile_n & 1);
            const uint32_t use = MODE == kModeMoment3 ? tile_n : (tile_n >> 1);
            if (!mbar_wait_warp(tmem_full(acc), use & 1, abort_flag, p.err_word, kErrTmemFull, lane)) {
                ok = false;
                break;
            }
            tc_fence_after();
            const int64_t i = (int64_t)I * kTileM + warp * 32 + lane;
            const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + acc * kTileN;
            float* crow = MOMENT2 ? p.C : p.C + i * p.ldc + (int64_t)J * kTileN;
            if (MOMENT2) {
                // packed triangle: (i, j) sits at rowbase(i) + j; keep i <= j < n.  A lane's 32 values
                // are consecutive in memory but only 4-byte aligned: scalar stores.
                if (I < p.row_blocks) {
                    // degree 2: row i of the packed triangle.  degree 3: row (i1, i) of the packed
                    // tetrahedron, whose hoisted base is tet(n) - tet(n-i1) + tri(n-i1) - tri(n-i) - i;
                    // rows above i1 are not part of the slab.
                    const int64_t i1 = p.i1_first + slot;
                    const bool row_live = i < p.N && (MODE != kModeMoment3 || i >= i1);
                    int64_t rb = 0;
                    if (row_live)
                        rb = MODE == kModeMoment3
                                 ? tet(p.N) - tet(p.N - i1) + tri(p.N - i1) - tri(p.N - i) - i
                                 : upper_row_base(p.N, i);
                    float* prow = p.C + rb;
#pragma unroll 1
                    const int c0 = col_skip(P, J, slot);  // accumulator column 0 is column c0 of the block
                    const int64_t col_end = (int64_t)(J + 1) * kTileN;
                    for (int cc = 0; cc * 32 < kTileN - c0; ++cc) {
                        const int64_t col0 = (int64_t)J * kTileN + c0 + cc * 32;
                        if (col0 + 32 <= (int64_t)I * kTileM + warp * 32 || col0 >= p.N) continue;  // warp-uniform: nothing kept
                        uint32_t r[32];
                        tmem_ld32(taddr + cc * 32, r);
                        tmem_ld_wait();
                        if (row_live) {
#pragma unroll
                            for (int v = 0; v < 32; ++v) {
                                const int64_t j = col0 + v;
                                if (j >= i && j < p.N && j < col_end) {
                                    float o = __uint_as_float(r[v]);
                                    if (p.accumulate) o += prow[j];
                                    prow[j] = o;
                                }
                            }
                        }
                    }
                }
            } else if (I < p.row_blocks) {
#pragma unroll 1
                for (int cc = 0; cc < kTileN / 32; ++cc) {
                    uint32_t r[32];
                    tmem_ld32(taddr + cc * 32, r);
                    tmem_ld_wait();
                    const int64_t col0 = (int64_t)J * kTileN + cc * 32;
                    if (i < p.N) {
                        if (p.vector_store && col0 + 32 <= p.ncols) {
                            float4* dst = (float4*)(crow + cc * 32);
#pragma unroll
                            for (int v = 0; v < 8; ++v) {
                                float4 o = make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                                       __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
                                if (p.accumulate) {
                                    const float4 old = dst[v];
                                    o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
                                }
                                dst[v] = o;
                            }
                        } else {
#pragma unroll
                            for (int v = 0; v < 32; ++v)
                                if (col0 + v < p.ncols) {
                                    float o = __uint_as_float(r[v]);
                                    if (p.accumulate) o += crow[cc * 32 + v];
                                    crow[cc * 32 + v] = o;
                                }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(empty0 + 8u * acc);
            ++tile_n;
        }
    }

    // Neither CTA may leave, or give back tensor memory, while its peer can still touch it.
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == kPWarpMma) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

// ---- host ------------------------------------------------------------------------------------------

// ---- stage_a: packed rows -> swizzled tile images ----------------------------------------------------
// One CTA builds one 128x64 tile (I, kb): 8 warps x 4 groups of 4 rows, 8 lanes per row.
constexpr int kStageThreads = 256;

__global__ void __launch_bounds__(kStageThreads)
trimm_stage_a_kernel(const Params p, uint8_t* __restrict__ tiles) {
    const int I = blockIdx.y;
    const int kb = blockIdx.x + 4 * (I >> 1);
    if (kb >= p.k_blocks) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int sub = lane >> 3, c = lane & 7;  // row within a 4-row group, 16-byte chunk in the row
    uint8_t* tile = tiles + (tile_offset(I, p.k_blocks) + blockIdx.x) * (int64_t)kABytes;
    const int64_t k0 = (int64_t)kb * kBlockK;
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
    const bool masked = (kb < 2 * I + 2) || (k0 + kBlockK > p.N);
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        const int r = 4 * (warp + 8 * g) + sub;  // 0..127
        const int64_t i = (int64_t)I * kTileM + r;
        const uint32_t soff = (uint32_t)((r >> 3) * 1024 + (r & 7) * 128 + ((c ^ (r & 7)) << 4));
        uint4 out = zero4;
        if (i < p.N && k0 + kBlockK > i) {  // the row has entries in this K block
            const int64_t e0 = upper_row_base(p.N, i) + k0 + 8 * c;  // first element of the lane's chunk
            const int64_t a0 = e0 & ~(int64_t)7;                     // aligned down to 16 bytes
            const uint32_t se = (uint32_t)(e0 & 7);                  // misalignment in elements
            const uint4 lo = (a0 + 8 <= p.cap_elems) ? __ldg((const uint4*)(p.A + a0)) : zero4;
            const uint4 hi = (se != 0 && a0 + 16 <= p.cap_elems) ? __ldg((const uint4*)(p.A + a0 + 8)) : zero4;
            const bool q1 = se & 2, q2 = se & 4;
            const uint32_t sh = (se & 1) * 16;
            const uint32_t W0 = lo.x, W1 = lo.y, W2 = lo.z, W3 = lo.w;
            const uint32_t W4 = hi.x, W5 = hi.y, W6 = hi.z, W7 = hi.w;
            const uint32_t X0 = q1 ? W1 : W0, X1 = q1 ? W2 : W1, X2 = q1 ? W3 : W2, X3 = q1 ? W4 : W3,
                           X4 = q1 ? W5 : W4, X5 = q1 ? W6 : W5, X6 = q1 ? W7 : W6;
            const uint32_t T0 = q2 ? X2 : X0, T1 = q2 ? X3 : X1, T2 = q2 ? X4 : X2, T3 = q2 ? X5 : X3,
                           T4 = q2 ? X6 : X4;
            out.x = __funnelshift_r(T0, T1, sh);
            out.y = __funnelshift_r(T1, T2, sh);
            out.z = __funnelshift_r(T2, T3, sh);
            out.w = __funnelshift_r(T3, T4, sh);
            if (masked) {
                // keep column j only if i <= j < N
                const int64_t j0 = k0 + 8 * c;
                uint32_t* w = &out.x;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int64_t j = j0 + e;
                    if (j < i || j >= p.N) w[e >> 1] &= (e & 1) ? 0x0000FFFFu : 0xFFFF0000u;
                }
            }
        }
        *(uint4*)(tile + soff) = out;
    }
}

__global__ void repitch_bf16_kernel(const uint16_t* __restrict__ src, int64_t lds, uint16_t* __restrict__ dst,
                                    int64_t ldd, int64_t rows, int64_t cols) {
    for (int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; t < rows * ldd;
         t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = t / ldd, c = t - r * ldd;
        dst[t] = c < cols ? src[r * lds + c] : (uint16_t)0;
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

// Workspace: the staged tile images of A, then (only when B's row pitch is not a multiple of
// 16 bytes, which a tensor map cannot describe) a copy of B with the pitch rounded up to 8 elements.
static int64_t staged_tile_count(int64_t N) {
    const int64_t row_blocks = (N + kTileM - 1) / kTileM, k_blocks = (N + kBlockK - 1) / kBlockK;
    return tile_offset(row_blocks, k_blocks);
}
size_t trimm_workspace_bytes(const IndexMap& m, int64_t ncols, int64_t ldb) {
    if (m.N == 0 || ncols == 0) return 0;
    size_t bytes = (size_t)round_up(staged_tile_count(m.N) * kABytes, 256);
    if (ldb % 8 != 0) bytes += (size_t)(m.N * round_up(ncols, 8) * 2);
    return bytes;
}

dastac_status launch_trimm_bf16(const IndexMap& m, const void* A, const void* B, int64_t ldb, float* C,
                                int64_t ldc, int64_t ncols, int accumulate, void* workspace,
                                int32_t* err_word, cudaStream_t st) {
    const int64_t N = m.N;
    if (N == 0 || ncols == 0) return DASTAC_OK;
    // TMA needs a 16-byte aligned base and row pitch for B.
    if (!aligned16(B)) return DASTAC_ERR_ALIGNMENT;
    if (!workspace) return DASTAC_ERR_WORKSPACE;
    uint8_t* tiles = (uint8_t*)workspace;
    if (ldb % 8 != 0) {
        workspace = tiles + round_up(staged_tile_count(N) * kABytes, 256);
        const int64_t ldd = round_up(ncols, 8);
        int64_t blocks = (N * ldd + 255) / 256;
        if (blocks > (int64_t)sm_count() * 32) blocks = (int64_t)sm_count() * 32;
        repitch_bf16_kernel<<<(unsigned)blocks, 256, 0, st>>>((const uint16_t*)B, ldb, (uint16_t*)workspace,
                                                             ldd, N, ncols);
        dastac_status rs = launch_status();
        if (rs != DASTAC_OK) return rs;
        B = workspace;
        ldb = ldd;
    }
    if (ncols > 0x7fffffffLL || N > 0x7fffffffLL) return DASTAC_ERR_OVERFLOW;
    EncodeTiledFn enc = encode_fn();
    if (!enc) return DASTAC_ERR_CUDA;
    CUtensorMap tmap;
    const cuuint64_t dims[2] = {(cuuint64_t)ncols, (cuuint64_t)N};
    const cuuint64_t strides[1] = {(cuuint64_t)ldb * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)kBlockK};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(B), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return DASTAC_ERR_CUDA;

    Params p;
    p.A = (const __nv_bfloat16*)A;
    p.tiles = tiles;
    p.C = C;
    p.N = N;
    p.ncols = ncols;
    p.ldc = ldc;
    p.M = 0;
    p.i1_first = p.slots = 0;
    p.tiles_total = 0;
    p.cap_elems = round_up(m.slots, 8);
    p.row_blocks = (int32_t)((N + kTileM - 1) / kTileM);
    p.col_blocks = (int32_t)((ncols + kTileN - 1) / kTileN);
    p.k_blocks = (int32_t)((N + kBlockK - 1) / kBlockK);
    p.accumulate = accumulate;
    p.vector_store = ((ldc & 3) == 0) && aligned16(C);
    p.err_word = err_word;

    // The staged tile images as a tensor: one 128-byte row per tile row, already in shared-memory order.
    const int64_t staged_tiles = staged_tile_count(N);
    if (staged_tiles * kTileM > 0x7fffffffLL) return DASTAC_ERR_OVERFLOW;
    CUtensorMap tmap_a;
    const cuuint64_t adims[2] = {(cuuint64_t)kBlockK, (cuuint64_t)(staged_tiles * kTileM)};
    const cuuint64_t astrides[1] = {(cuuint64_t)kBlockK * 2};
    const cuuint32_t abox[2] = {(cuuint32_t)kBlockK, (cuuint32_t)kTileM};
    if (enc(&tmap_a, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, tiles, adims, astrides, abox, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return DASTAC_ERR_CUDA;

    static bool attr_set[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        if (cudaFuncSetAttribute(trimm_pair_kernel<kModeTrimm>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kPSmemBytes) != cudaSuccess)
            return DASTAC_ERR_CUDA;
        attr_set[dev] = true;
    }
    if (p.row_blocks > 65535) return DASTAC_ERR_OVERFLOW;  // gridDim.y of the staging kernel
    trimm_stage_a_kernel<<<dim3((unsigned)p.k_blocks, (unsigned)p.row_blocks), kStageThreads, 0, st>>>(p, tiles);
    dastac_status ss = launch_status();
    if (ss != DASTAC_OK) return ss;
    const int64_t n_tiles = (int64_t)((p.row_blocks + 1) / 2) * p.col_blocks;  // pairs of row blocks x column blocks
    const int64_t max_clusters = sm_count() / 2;
    const int clusters = (int)(n_tiles < max_clusters ? n_tiles : max_clusters);
    trimm_pair_kernel<kModeTrimm><<<2 * clusters, kPThreads, kPSmemBytes, st>>>(tmap_a, tmap, tmap, p);  // the third map is not used
    return launch_status();
}

// ---- degree-2 moments: A2 = B^T B on the unique part i1 <= i2, packed output ---------------------------
// Workspace: only when B's row pitch is not a multiple of 16 bytes (a re-pitched copy of B).
size_t moment2_workspace_bytes(int64_t M, int64_t n, int64_t ldb) {
    if (M == 0 || n == 0 || ldb % 8 == 0) return 0;
    return (size_t)(M * round_up(n, 8) * 2);
}

dastac_status launch_moment2_bf16(const IndexMap& mo, const void* B, int64_t ldb, int64_t M, float* out,
                                  int accumulate, void* workspace, int32_t* err_word, cudaStream_t st) {
    const int64_t n = mo.N;
    if (n == 0) return DASTAC_OK;
    if (M == 0) {  // an empty sum: the packed result is zero
        if (!accumulate && cudaMemsetAsync(out, 0, (size_t)mo.count * sizeof(float), st) != cudaSuccess)
            return DASTAC_ERR_CUDA;
        return DASTAC_OK;
    }
    if (!aligned16(B)) return DASTAC_ERR_ALIGNMENT;
    if (M > 0x7fffffffLL - kBlockK || n > 0x7fffffffLL - 2 * kTileN) return DASTAC_ERR_OVERFLOW;
    if (ldb % 8 != 0) {
        if (!workspace) return DASTAC_ERR_WORKSPACE;
        const int64_t ldd = round_up(n, 8);
        int64_t blocks = (M * ldd + 255) / 256;
        if (blocks > (int64_t)sm_count() * 32) blocks = (int64_t)sm_count() * 32;
        repitch_bf16_kernel<<<(unsigned)blocks, 256, 0, st>>>((const uint16_t*)B, ldb, (uint16_t*)workspace, ldd, M, n);
        dastac_status rs = launch_status();
        if (rs != DASTAC_OK) return rs;
        B = workspace;
        ldb = ldd;
    }
    EncodeTiledFn enc = encode_fn();
    if (!enc) return DASTAC_ERR_CUDA;
    CUtensorMap tmap;
    const cuuint64_t dims[2] = {(cuuint64_t)n, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)ldb * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)kBlockK};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(B), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return DASTAC_ERR_CUDA;
    Params p;
    p.A = nullptr;
    p.tiles = nullptr;
    p.C = out;
    p.N = n;
    p.ncols = n;
    p.ldc = 0;
    p.M = M;
    p.i1_first = p.slots = 0;
    p.tiles_total = 0;
    p.cap_elems = 0;
    p.row_blocks = (int32_t)((n + kTileM - 1) / kTileM);
    p.col_blocks = (int32_t)((n + kTileN - 1) / kTileN);
    p.k_blocks = (int32_t)((M + kBlockK - 1) / kBlockK);
    p.accumulate = accumulate;
    p.vector_store = 0;
    p.err_word = err_word;
    static bool attr_set[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        if (cudaFuncSetAttribute(trimm_pair_kernel<kModeMoment2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kPSmemBytes) != cudaSuccess)
            return DASTAC_ERR_CUDA;
        attr_set[dev] = true;
    }
    const int64_t pb = (p.row_blocks + 1) / 2;
    const int64_t n_tiles = pb * (pb + 1) / 2;
    const int64_t max_clusters = sm_count() / 2;
    const int clusters = (int)(n_tiles < max_clusters ? n_tiles : max_clusters);
    trimm_pair_kernel<kModeMoment2><<<2 * clusters, kPThreads, kPSmemBytes, st>>>(tmap, tmap, tmap, p);  // only the second map is used
    return launch_status();
}

// ---- degree-3 moments: A3 on i1 <= i2 <= i3, packed tetrahedron out ------------------------------------
// Bt[i][x] = B[x][i], row pitch ldt elements.
__global__ void transpose_bf16_kernel(const uint16_t* __restrict__ B, int64_t ldb, int64_t M, int64_t n,
                                      uint16_t* __restrict__ Bt, int64_t ldt) {
    __shared__ uint16_t tile[32][33];
    const int64_t x0 = blockIdx.x * 32LL, i0 = blockIdx.y * 32LL;
    for (int r = threadIdx.y; r < 32; r += blockDim.y) {
        const int64_t x = x0 + r, i = i0 + threadIdx.x;
        tile[r][threadIdx.x] = (x < M && i < n) ? B[x * ldb + i] : (uint16_t)0;
    }
    __syncthreads();
    for (int r = threadIdx.y; r < 32; r += blockDim.y) {
        const int64_t i = i0 + r, x = x0 + threadIdx.x;
        if (i < n && x < M) Bt[i * ldt + x] = tile[threadIdx.x][r];
    }
}

// Workspace: the transposed copy of B (n rows of round_up(M, 8) elements), then, only when B's row pitch
// is not a multiple of 16 bytes, a re-pitched copy of B.
size_t moment3_workspace_bytes(int64_t M, int64_t n, int64_t ldb) {
    if (M == 0 || n == 0) return 0;
    return (size_t)round_up(n * round_up(M, 8) * 2, 256) + moment2_workspace_bytes(M, n, ldb);
}

dastac_status launch_moment3_bf16(const IndexMap& mo, const void* B, int64_t ldb, int64_t M, float* out,
                                  int accumulate, void* workspace, int32_t* err_word, cudaStream_t st) {
    const int64_t n = mo.N;
    if (n == 0) return DASTAC_OK;
    if (M == 0) {
        if (!accumulate && cudaMemsetAsync(out, 0, (size_t)mo.count * sizeof(float), st) != cudaSuccess)
            return DASTAC_ERR_CUDA;
        return DASTAC_OK;
    }
    if (!aligned16(B)) return DASTAC_ERR_ALIGNMENT;
    if (!workspace) return DASTAC_ERR_WORKSPACE;
    if (M > 0x7fffffffLL - kBlockK || n > 0x7fffffffLL - 2 * kTileN) return DASTAC_ERR_OVERFLOW;
    const int64_t ldt = round_up(M, 8);
    uint16_t* Bt = (uint16_t*)workspace;
    {
        const int64_t gx = (M + 31) / 32, gy = (n + 31) / 32;
        if (gy > 65535) return DASTAC_ERR_OVERFLOW;
        transpose_bf16_kernel<<<dim3((unsigned)gx, (unsigned)gy), dim3(32, 8), 0, st>>>((const uint16_t*)B, ldb, M, n, Bt, ldt);
        dastac_status rs = launch_status();
        if (rs != DASTAC_OK) return rs;
    }
    if (ldb % 8 != 0) {
        uint16_t* copy = (uint16_t*)((uint8_t*)workspace + round_up(n * ldt * 2, 256));
        const int64_t ldd = round_up(n, 8);
        int64_t blocks = (M * ldd + 255) / 256;
        if (blocks > (int64_t)sm_count() * 32) blocks = (int64_t)sm_count() * 32;
        repitch_bf16_kernel<<<(unsigned)blocks, 256, 0, st>>>((const uint16_t*)B, ldb, copy, ldd, M, n);
        dastac_status rs = launch_status();
        if (rs != DASTAC_OK) return rs;
        B = copy;
        ldb = ldd;
    }
    EncodeTiledFn enc = encode_fn();
    if (!enc) return DASTAC_ERR_CUDA;
    const cuuint32_t estr[2] = {1, 1};
    CUtensorMap tmap_b, tmap_t, tmap_c;
    {
        const cuuint64_t dims[2] = {(cuuint64_t)n, (cuuint64_t)M};
        const cuuint64_t strides[1] = {(cuuint64_t)ldb * 2};
        const cuuint32_t box[2] = {64, (cuuint32_t)kBlockK};
        if (enc(&tmap_b, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(B), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return DASTAC_ERR_CUDA;
    }
    {
        // Bt: 128 rows (features) x 64 samples per box, rows of 128 bytes, swizzled; and one row of 64 samples
        const cuuint64_t dims[2] = {(cuuint64_t)M, (cuuint64_t)n};
        const cuuint64_t strides[1] = {(cuuint64_t)ldt * 2};
        const cuuint32_t box[2] = {(cuuint32_t)kBlockK, (cuuint32_t)kTileM};
        const cuuint32_t cbox[2] = {(cuuint32_t)kBlockK, 1};
        if (enc(&tmap_t, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Bt, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
            enc(&tmap_c, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Bt, dims, strides, cbox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return DASTAC_ERR_CUDA;
    }
    static bool attr_set[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        if (cudaFuncSetAttribute(trimm_pair_kernel<kModeMoment3>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)kPSmemBytesFused) != cudaSuccess)
            return DASTAC_ERR_CUDA;
        attr_set[dev] = true;
    }
    Params p;
    p.A = nullptr;
    p.tiles = nullptr;
    p.C = out;
    p.N = n;
    p.ncols = n;
    p.ldc = 0;
    p.M = M;
    p.cap_elems = 0;
    p.row_blocks = (int32_t)((n + kTileM - 1) / kTileM);
    p.col_blocks = (int32_t)((n + kTileN - 1) / kTileN);
    p.k_blocks = (int32_t)((M + kBlockK - 1) / kBlockK);
    p.accumulate = accumulate;
    p.vector_store = 0;
    p.err_word = err_word;
    p.i1_first = 0;
    p.slots = (int32_t)n;
    const int64_t pb = (p.row_blocks + 1) / 2;
    int64_t n_tiles = 0;
    for (int64_t i1 = 0; i1 < n; ++i1) {
        const int64_t r = i1 / (2 * kTileM);
        n_tiles += (pb - r) * (pb - r + 1) / 2;
    }
    p.tiles_total = n_tiles;
    const int64_t max_clusters = sm_count() / 2;
    const int clusters = (int)(n_tiles < max_clusters ? n_tiles : max_clusters);
    trimm_pair_kernel<kModeMoment3><<<2 * clusters, kPThreadsFused, kPSmemBytesFused, st>>>(tmap_t, tmap_b, tmap_c, p);
    return launch_status();
}

}  // namespace dastac

// ---- entry point that allocates nothing ----------------------------------------------------------
// The staged tile images normally live in the caller's workspace.  Callers that cannot obtain
// device memory at call time get the same contraction with the images in a fixed array that is part
// of the library image.  On the host the array's name is only a handle, so its device address is
// asked for once per device and that pointer is what the kernels receive.
namespace dastac {
namespace {

constexpr int64_t kStaticMaxN = DASTAC_NOALLOC_MAX_N;
constexpr int64_t kStaticRowBlocks = (kStaticMaxN + kTileM - 1) / kTileM;
constexpr int64_t kStaticKBlocks = (kStaticMaxN + kBlockK - 1) / kBlockK;
// tile_offset(row_blocks, k_blocks) written out for an even number of row blocks
constexpr int64_t kStaticTiles = kStaticRowBlocks * kStaticKBlocks - kStaticRowBlocks * (kStaticRowBlocks - 2);
static_assert(kStaticRowBlocks % 2 == 0, "the closed form above assumes whole pairs of row blocks");
constexpr size_t kStaticBytes = (size_t)kStaticTiles * kABytes;
static_assert(kStaticBytes == DASTAC_NOALLOC_SCRATCH_BYTES, "header and array size disagree");

static __device__ __align__(256) uint8_t g_static_tiles[kStaticBytes];

// Device address of g_static_tiles on the current device, looked up on the first call per device.
dastac_status static_tiles_ptr(void** out) {
    static void* ptrs[64];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DASTAC_ERR_CUDA;
    if (!ptrs[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_tiles) != cudaSuccess || !p) return DASTAC_ERR_CUDA;
        ptrs[dev] = p;
    }
    *out = ptrs[dev];
    return DASTAC_OK;
}

}  // namespace
}  // namespace dastac

extern "C" dastac_status dastac_trimm_bf16_noalloc(const dastac_structure* s, const void* A, const void* B,
                                                   int64_t ldb, int64_t ncols, float* C, int64_t ldc,
                                                   int32_t accumulate, int32_t* err_word, void* stream) {
    using namespace dastac;
    if (!s || ncols < 0 || ldb < 0 || ldc < 0) return DASTAC_ERR_INVALID_ARG;
    const IndexMap& m = s->map;
    if (m.kind == kEmpty || ncols == 0) return DASTAC_OK;
    if (!(m.kind == kUpper && m.rank == 2 && m.dims[0] == m.dims[1] && !m.symmetric))
        return DASTAC_ERR_UNSUPPORTED_EXPR;
    if (m.N > kStaticMaxN) return DASTAC_ERR_WORKSPACE;  // the fixed array holds the tiles of N <= DASTAC_NOALLOC_MAX_N
    if (!A || !B || !C) return DASTAC_ERR_INVALID_ARG;
    if (!aligned16(A) || !aligned16(B) || !aligned16(C)) return DASTAC_ERR_ALIGNMENT;
    if (ldb < ncols || ldc < ncols) return DASTAC_ERR_SHAPE;
    // A row pitch of B that is not a multiple of 16 bytes would need a re-pitched copy of B, for
    // which there is no room in the fixed array.
    if (ldb % 8 != 0) return DASTAC_ERR_ALIGNMENT;
    if (trimm_workspace_bytes(m, ncols, ldb) > kStaticBytes) return DASTAC_ERR_WORKSPACE;
    void* tiles = nullptr;
    dastac_status st = static_tiles_ptr(&tiles);
    if (st != DASTAC_OK) return st;
    return launch_trimm_bf16(m, A, B, ldb, C, ldc, ncols, accumulate, tiles, err_word, (cudaStream_t)stream);
}
