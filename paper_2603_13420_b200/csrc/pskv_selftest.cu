// Self-tests of two pieces of the library that ordinary calls cannot reach:
//   * the bounded device-side wait: a tiny kernel waits, through the same routine every tensor-core
//     kernel waits with, for an mbarrier phase that nothing will ever complete, gives up after a
//     budget of clock cycles, records the time-out in the device status word and returns normally.
//     Nothing asynchronous (no TMA copy, no tcgen05 operation) is in flight in that kernel, so the CTA
//     leaves cleanly; the production kernels are never made to time out.
//   * the per-device bookkeeping of the launch sites (shared-memory opt-in once per DEVICE): pure host
//     logic, exercised with made-up device ordinals.
#include "pskv_common.cuh"
#include "pskv_sm100.cuh"
#include "pskv_tc_common.cuh"

namespace pskv {
namespace {

using namespace sm100;

constexpr unsigned int kErrSelfTestWait = 0x901;

__device__ unsigned int g_selftest_result;  // 1: the wait returned true (wrong), 2: it gave up (right)

__global__ void __launch_bounds__(32, 1)
wait_timeout_kernel(unsigned int *status_word, long long budget_cycles, unsigned int *result)
{
    __shared__ __align__(8) unsigned long long barrier_word;
    __shared__ int abort_word;
    const uint32_t bar = smem_u32(&barrier_word);
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);  // one arrival expected; nobody arrives
        abort_word = 0;
        fence_barrier_init();
    }
    __syncwarp();
    const bool ok = mbar_wait_warp(bar, 0, &abort_word, status_word, kErrSelfTestWait, budget_cycles);
    if (threadIdx.x == 0) *result = ok ? 1u : 2u;  // 2: the wait gave up, as it must
}

}  // namespace
}  // namespace pskv

using namespace pskv;

extern "C" {

pskv_status pskv_selftest_wait_timeout(long long budget_cycles, void *cuda_stream)
{
    if (budget_cycles < 1 || budget_cycles > 1000000000ll) return PSKV_ERR_INVALID_ARG;
    unsigned int *status_word = nullptr;
    const pskv_status st = device_status_word(&status_word);
    if (st != PSKV_OK) return st;
    unsigned int *result = nullptr;  // a word in the library image: nothing is allocated
    if (cudaGetSymbolAddress(reinterpret_cast<void **>(&result), g_selftest_result) != cudaSuccess) return PSKV_ERR_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    wait_timeout_kernel<<<1, 32, 0, stream>>>(status_word, budget_cycles, result);
    count_launches(1);
    return cudaGetLastError() == cudaSuccess ? PSKV_OK : PSKV_ERR_CUDA;
}

int pskv_selftest_per_device_once(void)
{
    // Two made-up devices: each must see "pending" exactly until it is marked, independently of the other;
    // ordinals outside the table are always pending (the set-up is then simply repeated).
    PerDeviceOnce once;
    if (!once.pending(0) || !once.pending(1)) return 1;
    once.mark(0);
    if (once.pending(0)) return 2;
    if (!once.pending(1)) return 3;  // device 1 still has to opt in although device 0 has
    once.mark(1);
    if (once.pending(1) || once.pending(0)) return 4;
    if (!once.pending(63)) return 5;
    once.mark(63);
    if (once.pending(63)) return 6;
    if (!once.pending(-1) || !once.pending(64) || !once.pending(1000)) return 7;
    once.mark(64);  // ignored
    if (!once.pending(64)) return 8;
    PerDeviceOnce other;  // another launch site has its own flags
    if (!other.pending(0)) return 9;
    return 0;
}

}  // extern "C"
