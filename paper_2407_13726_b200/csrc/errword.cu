// The library's device error word, the call that reads it, and a self-test of the bounded waits.
#include <mutex>

#include "common.cuh"
#include "waits.cuh"

namespace dastac {
namespace {

// One word per GPU that loads the library.  Host code must not pass `g_error_word` itself to a
// kernel: in host code the name is a stand-in, the device address comes from
// cudaGetSymbolAddress, looked up once per device with that device current.
__device__ int32_t g_error_word;

// A single warp waits, with a budget, on a barrier that nothing ever arrives on; when the wait has
// run out it records kErrWordSelfTest and returns.  This is the expiry path of every bounded wait
// in the library, exercised without a fault, a trap or an endless loop.
__global__ void wait_expiry_selftest_kernel(long long budget, int32_t* err_word) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"((uint32_t)__cvta_generic_to_shared(&bar)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const bool landed = mbar_wait_bounded((uint32_t)__cvta_generic_to_shared(&bar), 0u, budget);
    if (!__all_sync(0xffffffffu, landed) && threadIdx.x == 0) atomicExch(err_word, kErrWordSelfTest);
}

}  // namespace

int32_t* device_error_word() {
    static std::mutex mu;
    static int32_t* addr[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_error_word) != cudaSuccess) return nullptr;
        addr[dev] = static_cast<int32_t*>(p);
    }
    return addr[dev];
}

}  // namespace dastac

using namespace dastac;

extern "C" dastac_status dastac_device_error(int32_t* word, int32_t clear, void* stream) {
    int32_t* dev_word = device_error_word();
    if (!dev_word) return DASTAC_ERR_CUDA;
    cudaStream_t cs = (cudaStream_t)stream;
    int32_t value = 0;
    if (cudaMemcpyAsync(&value, dev_word, sizeof(value), cudaMemcpyDeviceToHost, cs) != cudaSuccess)
        return DASTAC_ERR_CUDA;
    if (clear && cudaMemsetAsync(dev_word, 0, sizeof(value), cs) != cudaSuccess) return DASTAC_ERR_CUDA;
    if (cudaStreamSynchronize(cs) != cudaSuccess) return DASTAC_ERR_CUDA;
    if (word) *word = value;
    return value == 0 ? DASTAC_OK : DASTAC_ERR_TIMEOUT;
}

extern "C" dastac_status dastac_selftest_wait_expiry(int64_t budget_cycles, void* stream) {
    if (budget_cycles < 0 || budget_cycles > kDefaultWaitBudget) return DASTAC_ERR_INVALID_ARG;
    int32_t* dev_word = device_error_word();
    if (!dev_word) return DASTAC_ERR_CUDA;
    wait_expiry_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((long long)budget_cycles, dev_word);
    return launch_status();
}
