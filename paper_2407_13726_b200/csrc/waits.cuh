// Bounded waits on shared-memory barriers, and the library's device error word.
//
// Every wait on an mbarrier in this library has a budget in clock cycles.  A wait that runs out
// does not trap and does not spin on: the kernel records a code in an error word, skips the work
// that depended on the data, gives its copies in flight one more budget to land and returns, so the
// context stays usable and the host can see what happened.
#pragma once
#include <cstdint>

namespace dastac {

constexpr long long kDefaultWaitBudget = 2000000000LL;  // about a second; never expected to run out

// codes stored in an error word (any non-zero value means "a bounded wait expired")
constexpr int32_t kErrWordPack = 0x5041;      // "PA": pack, a window's bulk copy did not land
constexpr int32_t kErrWordUnpack = 0x554e;    // "UN": unpack, likewise
constexpr int32_t kErrWordSelfTest = 0x5354;  // "ST": the self-test kernel's wait ran out, as it must

// The current device's error word: a device int32 owned by the library (one per GPU that loads it),
// written by kernels whose entry points take no error word of the caller's.  nullptr on failure.
int32_t* device_error_word();

#ifdef __CUDACC__
// Waits until the barrier's phase with the given parity completes or `budget` cycles have passed.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, long long budget) {
    const long long t0 = clock64();
    uint32_t done = 0;
    while (!done) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar), "r"(parity)
            : "memory");
        if (!done && clock64() - t0 > budget) break;
    }
    return done != 0;
}
#endif

}  // namespace dastac
