// Pieces shared by the split-precision (TF32 hi / lo) tensor-core kernels: barrier and tcgen05
// wrappers, the K-major 128-byte-swizzled operand tile and the fp32 -> (hi, lo) split.
//
// An fp32 value v is split as hi = v with its low 13 mantissa bits cleared (exactly a TF32 number)
// and lo = v - hi (exact in fp32; the tensor core reads its upper 19 bits).  A product a b is then
// taken as ahi bhi + ahi blo + alo bhi in fp32 accumulation; the dropped alo blo is 2^-22 relative.
#pragma once
#include <cstdint>

namespace dastac {

// instruction descriptor, kind::tf32: fp32 accumulator, TF32 A and B, both K-major
constexpr uint32_t tc_idesc_mn(int m_rows, int n_cols) {
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(n_cols >> 3) << 17) | ((uint32_t)(m_rows >> 4) << 24);
}

#ifdef __CUDACC__
__device__ __forceinline__ uint32_t tc_smem(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void tc_mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void tc_mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// K-major operand tile with 128-byte swizzle: rows of 128 bytes (32 fp32 of K), groups of 8 rows
// 1024 bytes apart.  Byte offset of (row r, 16-byte chunk c): (r >> 3) * 1024 + (r & 7) * 128 +
// ((c ^ (r & 7)) << 4).
__device__ __forceinline__ uint64_t tc_desc(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)(16 >> 4) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
__device__ __forceinline__ uint32_t tc_tile_offset(int r, int chunk) {
    return (uint32_t)((r >> 3) * 1024 + (r & 7) * 128 + ((chunk ^ (r & 7)) << 4));
}
__device__ __forceinline__ void tc_mma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
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
// hi / lo parts of an fp32 value as TF32 operands
__device__ __forceinline__ void tc_split(float v, float& hi, float& lo) {
    hi = __uint_as_float(__float_as_uint(v) & 0xffffe000u);
    lo = v - hi;  // exact; the tensor core reads its upper 19 bits
}

// Bounded wait shared by the roles of a CTA: false when the budget ran out here or elsewhere in
// the CTA (abort_flag lives in shared memory); the first expiry records `code` in the error word.
__device__ __forceinline__ bool tc_wait_coded(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* err_word,
                                              int32_t code, long long budget) {
    const long long t0 = clock64();
    for (;;) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(bar), "r"(parity)
            : "memory");
        if (ok) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > budget) {
            *abort_flag = 1;
            if (err_word) atomicCAS(err_word, 0, code);
            return false;
        }
    }
}
#endif

}  // namespace dastac
