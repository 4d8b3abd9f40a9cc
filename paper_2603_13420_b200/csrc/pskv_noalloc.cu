// pskv_attn_bwd_static: the backward call for callers that cannot hand over scratch memory.
//
// Some users of this library run inside a process whose device memory is entirely owned by
// someone else -- a framework allocator that reserved the whole card at start-up, or a search loop
// with a fixed memory plan -- so they have no pointer to give as `workspace`, and calling
// cudaMalloc themselves would either fail or stall every stream on the device while it
// synchronises.  For them the per-row scratch of the backward pass (D = <dout, out>, one float per
// query row) lives in a fixed array inside the library image instead.
#include <atomic>

#include "pskv_common.cuh"

namespace pskv {
namespace {

constexpr long long kStaticRows = 1ll << 20;  // query rows (B*Hq*S) the built-in scratch can serve: 4 MiB

// Held by every GPU that loads the library, until the process exits.
static __device__ __align__(256) float g_static_row_dot[kStaticRows];

constexpr int kMaxDevices = 64;
std::atomic<float *> g_scratch_ptr[kMaxDevices];  // device address of g_static_row_dot, resolved once per device

}  // namespace
}  // namespace pskv

using namespace pskv;

extern "C" {

long long pskv_attn_bwd_static_max_rows(void) { return kStaticRows; }

pskv_status pskv_attn_bwd_static(const void *dout, const void *q, const void *prefix_k, const void *prefix_v,
                                 const void *suffix_k, const void *suffix_v, const void *out, const float *lse,
                                 float scale, void *dq, void *dk_suffix, void *dv_suffix, int B, int Hq, int Hkv,
                                 int S, int P, int d, void *cuda_stream)
{
    if (B < 1 || Hq < 1 || S < 1) return PSKV_ERR_INVALID_ARG;
    if ((long long)B * Hq * S > kStaticRows) return PSKV_ERR_WORKSPACE;  // beyond the built-in scratch
    if (pskv_attn_bwd_workspace_bytes(B, Hq, Hkv, S, P, d) > sizeof(float) * (size_t)kStaticRows)
        return PSKV_ERR_WORKSPACE;

    // the same device check as every other call, before anything touches the device image
    unsigned int *status_word = nullptr;
    const pskv_status ds = device_status_word(&status_word);
    if (ds != PSKV_OK) return ds;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PSKV_ERR_CUDA;
    float *scratch = g_scratch_ptr[dev].load(std::memory_order_acquire);
    if (scratch == nullptr) {
        // In host code the array's name is only a handle; the address kernels can use comes from
        // the runtime, for the device that is current right now.
        float *ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_static_row_dot);
        if (e != cudaSuccess || ptr == nullptr) return PSKV_ERR_CUDA;
        g_scratch_ptr[dev].store(ptr, std::memory_order_release);  // (two racing first calls store the same address)
        scratch = ptr;
    }
    // Every element the kernels read is written earlier in the same call (the D pre-pass fills one
    // float per row), so nothing has to be cleared between calls.
    return pskv_attn_bwd(dout, q, prefix_k, prefix_v, suffix_k, suffix_v, out, lse, scale, dq, dk_suffix,
                         dv_suffix, B, Hq, Hkv, S, P, d, scratch, sizeof(float) * (size_t)kStaticRows,
                         cuda_stream);
}

}  // extern "C"
