// C ABI of libpskv: host-side validation, kernel-family choice and launch.  No device memory
// is allocated here; everything the kernels touch is passed in by the caller.
#include <stdio.h>
#include <string.h>

#include <atomic>
#include <mutex>
#include <vector>

#include "pskv_common.cuh"

namespace pskv {
namespace {

__device__ unsigned int g_device_status = 0;  // set non-zero by a kernel whose bounded wait expired

thread_local int t_last_cuda_error = 0;

constexpr int kMaxDevices = 64;
struct DeviceInfo {
    int checked;              // 0 = not yet, 1 = sm_100, -1 = other arch
    unsigned int *status_ptr; // device address of g_device_status on that device
};
DeviceInfo g_devices[kMaxDevices];

pskv_status cuda_fail(cudaError_t e)
{
    t_last_cuda_error = (int)e;
    return PSKV_ERR_CUDA;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Pure host checks shared by both calls.  Returns PSKV_OK and fills `dm` when the sizes are usable.
pskv_status check_dims(int B, int Hq, int Hkv, int S, int P, int d, Dims *dm)
{
    if (B < 1 || Hq < 1 || Hkv < 1 || S < 1 || P < 0 || d < 1) return PSKV_ERR_INVALID_ARG;
    if (Hq % Hkv != 0) return PSKV_ERR_INVALID_ARG;
    if (d != 64 && d != 128) return PSKV_ERR_UNSUPPORTED_SHAPE;
    // element counts must stay inside 2^40 so that byte offsets fit comfortably in 64 bits
    const double rows = (double)B * Hq * S;
    if (rows * d > 1.0e12 || (double)Hkv * P * d > 1.0e12) return PSKV_ERR_UNSUPPORTED_SHAPE;
    dm->B = B; dm->Hq = Hq; dm->Hkv = Hkv; dm->S = S; dm->P = P; dm->d = d; dm->n_rep = Hq / Hkv;
    dm->Pstride = P;
    dm->Skv = S;
    dm->ragged = 0;
    return PSKV_OK;
}

// The decode-shaped operator: S query rows per candidate against a suffix cache of Skv >= S rows.
pskv_status check_dims_decode(int B, int Hq, int Hkv, int Sq, int Skv, int P, int d, bool ragged, Dims *dm)
{
    pskv_status st = check_dims(B, Hq, Hkv, Sq, P, d, dm);
    if (st != PSKV_OK) return st;
    if (Skv < Sq) return PSKV_ERR_INVALID_ARG;
    if ((double)B * Hkv * Skv * d > 1.0e12) return PSKV_ERR_UNSUPPORTED_SHAPE;
    dm->Skv = Skv;
    dm->ragged = ragged ? 1 : 0;
    return PSKV_OK;
}

// Device checks: compute capability 10.x, and the address of the status word on this device.
pskv_status check_device(unsigned int **status_ptr)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= kMaxDevices) return PSKV_ERR_UNSUPPORTED_ARCH;
    DeviceInfo &info = g_devices[dev];
    if (info.checked == 0) {
        int major = 0;
        e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) return cuda_fail(e);
        if (major != 10) {
            info.checked = -1;
        } else {
            void *p = nullptr;
            e = cudaGetSymbolAddress(&p, g_device_status);
            if (e != cudaSuccess) return cuda_fail(e);
            info.status_ptr = static_cast<unsigned int *>(p);
            info.checked = 1;
        }
    }
    if (info.checked != 1) return PSKV_ERR_UNSUPPORTED_ARCH;
    *status_ptr = info.status_ptr;
    return PSKV_OK;
}

size_t round256(size_t n) { return (n + 255) & ~(size_t)255; }

size_t simt_bwd_workspace(const Dims &dm) { return round256((size_t)dm.B * dm.Hq * dm.S * sizeof(float)); }

std::atomic<long long> g_launches{0};
std::atomic<int> g_cta_pairs{0};
std::atomic<int> g_multi_form{0};  // see pskv_set_multi_form

// ---- optional per-kernel timing: a bounded list of (kernel id, start event, stop event)
constexpr int kMaxTimed = 8192;
struct TimedLaunch {
    int id;
    cudaEvent_t start, stop;
};
std::mutex g_timing_mutex;
bool g_timing_on = false;
std::vector<TimedLaunch> g_timed;
const char *const kKernelNames[kKernelCount] = {
    "tc_fwd_kernel", "simt_row_dot_kernel", "tc_bwd_dq_kernel", "tc_bwd_dkv_kernel",
    "bwd_dkv_mma_kernel",
    "simt_fwd_kernel", "simt_bwd_dq_kernel", "simt_bwd_dkv_kernel", "ce_fwd_kernel", "ce_finalize_kernel", "tc_bwd_prefix_kernel", "simt_bwd_prefix_kernel"};

}  // namespace

bool cta_pairs_enabled() { return g_cta_pairs.load(std::memory_order_relaxed) != 0; }

pskv_status device_status_word(unsigned int **status_word) { return check_device(status_word); }

void count_launches(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

void *timing_begin(int kernel_id, cudaStream_t stream)
{
    std::lock_guard<std::mutex> lock(g_timing_mutex);
    if (!g_timing_on || (int)g_timed.size() >= kMaxTimed) return nullptr;
    TimedLaunch t;
    t.id = kernel_id;
    if (cudaEventCreate(&t.start) != cudaSuccess) return nullptr;
    if (cudaEventCreate(&t.stop) != cudaSuccess) { cudaEventDestroy(t.start); return nullptr; }
    cudaEventRecord(t.start, stream);
    g_timed.push_back(t);
    return reinterpret_cast<void *>(g_timed.size());  // 1-based index
}

void timing_end(void *token, cudaStream_t stream)
{
    std::lock_guard<std::mutex> lock(g_timing_mutex);
    const size_t idx = reinterpret_cast<size_t>(token);
    if (idx >= 1 && idx <= g_timed.size()) cudaEventRecord(g_timed[idx - 1].stop, stream);
}

}  // namespace pskv

using namespace pskv;

extern "C" {

int pskv_version(void) { return 200; }

long long pskv_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

void pskv_kernel_timing_enable(int on)
{
    std::lock_guard<std::mutex> lock(g_timing_mutex);
    g_timing_on = on != 0;
}

int pskv_kernel_timing_count(void) { return kKernelCount; }

const char *pskv_kernel_timing_name(int kernel_id)
{
    return (kernel_id >= 0 && kernel_id < kKernelCount) ? kKernelNames[kernel_id] : "";
}

pskv_status pskv_kernel_timing_read(int kernel_id, double *total_ms, long long *launches)
{
    if (!total_ms || !launches || kernel_id < 0 || kernel_id >= kKernelCount) return PSKV_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_timing_mutex);
    double ms = 0.0;
    long long n = 0;
    std::vector<TimedLaunch> keep;
    for (const TimedLaunch &t : g_timed) {
        if (t.id != kernel_id) { keep.push_back(t); continue; }
        float one = 0.f;
        cudaError_t e = cudaEventSynchronize(t.stop);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&one, t.start, t.stop);
        cudaEventDestroy(t.start);
        cudaEventDestroy(t.stop);
        if (e != cudaSuccess) { g_timed.swap(keep); return cuda_fail(e); }
        ms += one;
        ++n;
    }
    g_timed.swap(keep);
    *total_ms = ms;
    *launches = n;
    return PSKV_OK;
}

const char *pskv_status_string(pskv_status s)
{
    switch (s) {
    case PSKV_OK: return "PSKV_OK";
    case PSKV_ERR_INVALID_ARG: return "PSKV_ERR_INVALID_ARG";
    case PSKV_ERR_UNSUPPORTED_SHAPE: return "PSKV_ERR_UNSUPPORTED_SHAPE";
    case PSKV_ERR_UNSUPPORTED_ARCH: return "PSKV_ERR_UNSUPPORTED_ARCH";
    case PSKV_ERR_WORKSPACE: return "PSKV_ERR_WORKSPACE";
    case PSKV_ERR_CUDA: return "PSKV_ERR_CUDA";
    case PSKV_ERR_DEVICE_TIMEOUT: return "PSKV_ERR_DEVICE_TIMEOUT";
    }
    return "PSKV_ERR_UNKNOWN";
}

int pskv_last_cuda_error(void) { return t_last_cuda_error; }

int pskv_kernel_family(int backward, int B, int Hq, int Hkv, int S, int P, int d)
{
    Dims dm;
    pskv_status st = check_dims(B, Hq, Hkv, S, P, d, &dm);
    if (st != PSKV_OK) return -(int)st;
    if (!backward && tc_fwd_supported(dm) && cta_pairs_enabled() && tc_fwd_pair_supported(dm)) return 2;
    return (backward ? tc_bwd_supported(dm) : tc_fwd_supported(dm)) ? 1 : 0;
}

pskv_status pskv_set_multi_form(int form)
{
    if (form < 0 || form > 2) return PSKV_ERR_INVALID_ARG;
    g_multi_form.store(form, std::memory_order_relaxed);
    return PSKV_OK;
}

void pskv_enable_cta_pairs(int on) { g_cta_pairs.store(on != 0, std::memory_order_relaxed); }

size_t pskv_attn_fwd_workspace_bytes(int B, int Hq, int Hkv, int S, int P, int d)
{
    Dims dm;
    if (check_dims(B, Hq, Hkv, S, P, d, &dm) != PSKV_OK) return 0;
    return tc_fwd_supported(dm) ? round256(tc_fwd_workspace_bytes(dm)) : 0;
}

size_t pskv_attn_bwd_workspace_bytes(int B, int Hq, int Hkv, int S, int P, int d)
{
    Dims dm;
    if (check_dims(B, Hq, Hkv, S, P, d, &dm) != PSKV_OK) return 0;
    return tc_bwd_supported(dm) ? round256(tc_bwd_workspace_bytes(dm)) : simt_bwd_workspace(dm);
}

namespace {

// Pointer, scale and workspace checks plus the launch, shared by the full-suffix and the
// decode-shaped forward; `dm` has passed check_dims / check_dims_decode.
pskv_status fwd_checked(const Dims &dm, const void *q, const void *prefix_k, const void *prefix_v,
                        const void *suffix_k, const void *suffix_v, const int *suffix_len, float scale, void *out,
                        float *lse, size_t need, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!q || !suffix_k || !suffix_v || !out || !lse) return PSKV_ERR_INVALID_ARG;
    if (dm.P > 0 && (!prefix_k || !prefix_v)) return PSKV_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(prefix_k) || !aligned16(prefix_v) || !aligned16(suffix_k) ||
        !aligned16(suffix_v) || !aligned16(out) || !aligned16(lse))
        return PSKV_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(suffix_len) & 3u) != 0) return PSKV_ERR_INVALID_ARG;
    if (!(scale == scale) || scale <= 0.f || scale > 1.0e6f) return PSKV_ERR_INVALID_ARG;
    if (need > 0 && (!workspace || workspace_bytes < need || !aligned16(workspace)))
        return PSKV_ERR_WORKSPACE;

    unsigned int *status_word = nullptr;
    pskv_status st = check_device(&status_word);
    if (st != PSKV_OK) return st;

    FwdArgs a;
    a.q = static_cast<const __nv_bfloat16 *>(q);
    a.prefix_k = static_cast<const __nv_bfloat16 *>(prefix_k);
    a.prefix_v = static_cast<const __nv_bfloat16 *>(prefix_v);
    a.suffix_k = static_cast<const __nv_bfloat16 *>(suffix_k);
    a.suffix_v = static_cast<const __nv_bfloat16 *>(suffix_v);
    a.out = static_cast<__nv_bfloat16 *>(out);
    a.lse = lse;
    a.suffix_len = suffix_len;
    a.scale = scale;
    a.dims = dm;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = tc_fwd_supported(dm) ? launch_tc_fwd(a, workspace, status_word, stream)
                                         : launch_simt_fwd(a, stream);
    return e == cudaSuccess ? PSKV_OK : cuda_fail(e);
}

pskv_status bwd_checked(const Dims &dm, const void *dout, const float *dlse, const void *q, const void *prefix_k,
                        const void *prefix_v, const void *suffix_k, const void *suffix_v, const int *suffix_len,
                        const void *out, const float *lse, float scale, void *dq, void *dk_suffix, void *dv_suffix, size_t need,
                        void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!dout || !q || !suffix_k || !suffix_v || !out || !lse || !dq || !dk_suffix || !dv_suffix)
        return PSKV_ERR_INVALID_ARG;
    if (dm.P > 0 && (!prefix_k || !prefix_v)) return PSKV_ERR_INVALID_ARG;
    if (!aligned16(dout) || !aligned16(q) || !aligned16(prefix_k) || !aligned16(prefix_v) ||
        !aligned16(suffix_k) || !aligned16(suffix_v) || !aligned16(out) || !aligned16(lse) ||
        !aligned16(dq) || !aligned16(dk_suffix) || !aligned16(dv_suffix))
        return PSKV_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(suffix_len) & 3u) != 0 || !aligned16(dlse)) return PSKV_ERR_INVALID_ARG;
    if (!(scale == scale) || scale <= 0.f || scale > 1.0e6f) return PSKV_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < need || !aligned16(workspace)) return PSKV_ERR_WORKSPACE;

    unsigned int *status_word = nullptr;
    pskv_status st = check_device(&status_word);
    if (st != PSKV_OK) return st;

    BwdArgs a;
    a.dout = static_cast<const __nv_bfloat16 *>(dout);
    a.q = static_cast<const __nv_bfloat16 *>(q);
    a.prefix_k = static_cast<const __nv_bfloat16 *>(prefix_k);
    a.prefix_v = static_cast<const __nv_bfloat16 *>(prefix_v);
    a.suffix_k = static_cast<const __nv_bfloat16 *>(suffix_k);
    a.suffix_v = static_cast<const __nv_bfloat16 *>(suffix_v);
    a.out = static_cast<const __nv_bfloat16 *>(out);
    a.lse = lse;
    a.dq = static_cast<__nv_bfloat16 *>(dq);
    a.dk_suffix = static_cast<__nv_bfloat16 *>(dk_suffix);
    a.dv_suffix = static_cast<__nv_bfloat16 *>(dv_suffix);
    a.row_dot = static_cast<float *>(workspace);
    a.dlse = dlse;
    a.suffix_len = suffix_len;
    a.scale = scale;
    a.dims = dm;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = tc_bwd_supported(dm) ? launch_tc_bwd(a, workspace, status_word, stream)
                                         : launch_simt_bwd(a, stream);
    return e == cudaSuccess ? PSKV_OK : cuda_fail(e);
}

}  // namespace

pskv_status pskv_attn_fwd(const void *q, const void *prefix_k, const void *prefix_v,
                          const void *suffix_k, const void *suffix_v, float scale,
                          void *out, float *lse, int B, int Hq, int Hkv, int S, int P, int d,
                          void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    Dims dm;
    pskv_status st = check_dims(B, Hq, Hkv, S, P, d, &dm);
    if (st != PSKV_OK) return st;
    return fwd_checked(dm, q, prefix_k, prefix_v, suffix_k, suffix_v, nullptr, scale, out, lse,
                       pskv_attn_fwd_workspace_bytes(B, Hq, Hkv, S, P, d), workspace, workspace_bytes, cuda_stream);
}

pskv_status pskv_attn_bwd(const void *dout, const void *q, const void *prefix_k,
                          const void *prefix_v, const void *suffix_k, const void *suffix_v,
                          const void *out, const float *lse, float scale, void *dq,
                          void *dk_suffix, void *dv_suffix, int B, int Hq, int Hkv, int S, int P,
                          int d, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    Dims dm;
    pskv_status st = check_dims(B, Hq, Hkv, S, P, d, &dm);
    if (st != PSKV_OK) return st;
    return bwd_checked(dm, dout, nullptr, q, prefix_k, prefix_v, suffix_k, suffix_v, nullptr, out, lse, scale, dq,
                       dk_suffix, dv_suffix, pskv_attn_bwd_workspace_bytes(B, Hq, Hkv, S, P, d), workspace,
                       workspace_bytes, cuda_stream);
}

pskv_status pskv_attn_bwd_lse(const void *dout, const float *dlse, const void *q, const void *prefix_k,
                              const void *prefix_v, const void *suffix_k, const void *suffix_v, const void *out,
                              const float *lse, float scale, void *dq, void *dk_suffix, void *dv_suffix, int B, int Hq,
                              int Hkv, int S, int P, int d, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    Dims dm;
    pskv_status st = check_dims(B, Hq, Hkv, S, P, d, &dm);
    if (st != PSKV_OK) return st;
    if (!dlse) return PSKV_ERR_INVALID_ARG;
    return bwd_checked(dm, dout, dlse, q, prefix_k, prefix_v, suffix_k, suffix_v, nullptr, out, lse, scale, dq,
                       dk_suffix, dv_suffix, pskv_attn_bwd_workspace_bytes(B, Hq, Hkv, S, P, d), workspace,
                       workspace_bytes, cuda_stream);
}

// ---- decode-shaped variant: the last Sq of each candidate's cached suffix tokens are the queries ------

size_t pskv_attn_fwd_decode_workspace_bytes(int B, int Hq, int Hkv, int Sq, int Skv, int P, int d)
{
    Dims dm;
    if (check_dims_decode(B, Hq, Hkv, Sq, Skv, P, d, true, &dm) != PSKV_OK) return 0;
    return 256;  // the redo counter of the tensor-core forward (whether or not suffix_len is given)
}

size_t pskv_attn_bwd_decode_workspace_bytes(int B, int Hq, int Hkv, int Sq, int Skv, int P, int d)
{
    Dims dm;
    if (check_dims_decode(B, Hq, Hkv, Sq, Skv, P, d, true, &dm) != PSKV_OK) return 0;
    return simt_bwd_workspace(dm);  // one fp32 per query row
}

pskv_status pskv_attn_fwd_decode(const void *q, const void *prefix_k, const void *prefix_v, const void *suffix_k,
                                 const void *suffix_v, const int *suffix_len, float scale, void *out, float *lse,
                                 int B, int Hq, int Hkv, int Sq, int Skv, int P, int d, void *workspace,
                                 size_t workspace_bytes, void *cuda_stream)
{
    Dims dm;
    pskv_status st = check_dims_decode(B, Hq, Hkv, Sq, Skv, P, d, suffix_len != nullptr, &dm);
    if (st != PSKV_OK) return st;
    return fwd_checked(dm, q, prefix_k, prefix_v, suffix_k, suffix_v, suffix_len, scale, out, lse, 256, workspace,
                       workspace_bytes, cuda_stream);
}

pskv_status pskv_attn_bwd_decode(const void *dout, const void *q, const void *prefix_k, const void *prefix_v,
                                 const void *suffix_k, const void *suffix_v, const int *suffix_len, const void *out,
                                 const float *lse, float scale, void *dq, void *dk_suffix, void *dv_suffix, int B,
                                 int Hq, int Hkv, int Sq, int Skv, int P, int d, void *workspace,
                                 size_t workspace_bytes, void *cuda_stream)
{
    Dims dm;
    pskv_status st = check_dims_decode(B, Hq, Hkv, Sq, Skv, P, d, suffix_len != nullptr, &dm);
    if (st != PSKV_OK) return st;
    return bwd_checked(dm, dout, nullptr, q, prefix_k, prefix_v, suffix_k, suffix_v, suffix_len, out, lse, scale, dq,
                       dk_suffix, dv_suffix, simt_bwd_workspace(dm), workspace, workspace_bytes, cuda_stream);
}

// ---- several instructions per call (suffix-centric alignment, Sec. 4.3) --------------------------

size_t pskv_attn_fwd_multi_workspace_bytes(int B, int Bp, int Hq, int Hkv, int S, int Pmax, int d)
{
    Dims dm;
    if (Bp < 1 || B < Bp || B % Bp != 0 || check_dims(B / Bp, Hq, Hkv, S, Pmax, d, &dm) != PSKV_OK) return 0;
    return 256;  // the per-call scratch of the single-prefix forward, reused by every instruction's part
}

size_t pskv_attn_bwd_multi_workspace_bytes(int B, int Bp, int Hq, int Hkv, int S, int Pmax, int d)
{
    Dims dm;
    if (Bp < 1 || B < Bp || B % Bp != 0 || check_dims(B / Bp, Hq, Hkv, S, Pmax, d, &dm) != PSKV_OK) return 0;
    return round256((size_t)B * Hq * S * sizeof(float));  // one fp32 per query row, all instructions in one array
}

namespace {
// The passes of different instructions are independent, and each one fills the GPU with one
// persistent CTA per SM, so back to back on one stream every pass pays its ramp-up, its uneven last
// round and the launch gap in full.  Alternating the passes between the caller's stream and one
// internal stream lets the CTAs of the next pass move onto SMs as the previous pass drains.  The
// internal stream and the two events are created once per device; the mutex keeps the
// fork / enqueue / join sequence of concurrent host threads apart.
struct SideStream {
    cudaStream_t stream;
    cudaEvent_t fork, join;
    int state;  // 0 = not created yet, 1 = usable, -1 = creation failed (passes then stay on the caller's stream)
};
SideStream g_side[kMaxDevices];
std::mutex g_side_mutex;

SideStream *side_stream()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    SideStream &ss = g_side[dev];
    if (ss.state == 0) {
        ss.state = -1;
        if (cudaStreamCreateWithFlags(&ss.stream, cudaStreamNonBlocking) == cudaSuccess &&
            cudaEventCreateWithFlags(&ss.fork, cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreateWithFlags(&ss.join, cudaEventDisableTiming) == cudaSuccess)
            ss.state = 1;
    }
    return ss.state == 1 ? &ss : nullptr;
}

// pskv_set_multi_form: 0 = the library chooses between one launch for all instructions and one pass per
// instruction, 1 = one launch wherever the shapes allow it (the same as 0 today), 2 = always passes.
int multi_form() { return g_multi_form.load(std::memory_order_relaxed); }

// checks shared by the two multi-instruction calls; fills the per-instruction geometry
pskv_status check_multi(int B, int Bp, int Hq, int Hkv, int S, int Pmax, int d, const int *prefix_len)
{
    if (Bp < 1 || B < Bp || B % Bp != 0 || !prefix_len) return PSKV_ERR_INVALID_ARG;
    Dims dm;
    pskv_status st = check_dims(B / Bp, Hq, Hkv, S, Pmax, d, &dm);
    if (st != PSKV_OK) return st;
    for (int i = 0; i < Bp; ++i)
        if (prefix_len[i] < 0 || prefix_len[i] > Pmax) return PSKV_ERR_INVALID_ARG;
    return PSKV_OK;
}
}  // namespace

pskv_status pskv_attn_fwd_multi(const void *q, const void *prefix_k, const void *prefix_v, const int *prefix_len,
                                const void *suffix_k, const void *suffix_v, float scale, void *out, float *lse,
                                int B, int Bp, int Hq, int Hkv, int S, int Pmax, int d, void *workspace,
                                size_t workspace_bytes, void *cuda_stream)
{
    pskv_status st = check_multi(B, Bp, Hq, Hkv, S, Pmax, d, prefix_len);
    if (st != PSKV_OK) return st;
    if (!q || !suffix_k || !suffix_v || !out || !lse) return PSKV_ERR_INVALID_ARG;
    if (Pmax > 0 && (!prefix_k || !prefix_v)) return PSKV_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(prefix_k) || !aligned16(prefix_v) || !aligned16(suffix_k) ||
        !aligned16(suffix_v) || !aligned16(out) || !aligned16(lse))
        return PSKV_ERR_INVALID_ARG;
    if (!(scale == scale) || scale <= 0.f || scale > 1.0e6f) return PSKV_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < 256 || !aligned16(workspace)) return PSKV_ERR_WORKSPACE;

    unsigned int *status_word = nullptr;
    st = check_device(&status_word);
    if (st != PSKV_OK) return st;

    const int Kq = B / Bp;  // candidates per instruction, contiguous in the candidate dimension
    const size_t q_part = (size_t)Kq * Hq * S * d, s_part = (size_t)Kq * Hkv * S * d, l_part = (size_t)Kq * Hq * S;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    for (int i = 0; i < Bp; ++i) {  // all sizes are checked before anything is enqueued
        Dims dm;
        st = check_dims(Kq, Hq, Hkv, S, prefix_len[i], d, &dm);
        if (st != PSKV_OK) return st;
    }
    {
        // One launch over all instructions when every tile lies inside one instruction: the prefix caches
        // are heads of one [Bp*Hkv][Pmax][d] tensor and the left padding is masked like a causal limit.
        Dims dall;
        if (Bp > 1 && multi_form() != 2 && check_dims(B, Hq, Hkv, S, Pmax, d, &dall) == PSKV_OK &&
            tc_fwd_fused_supported(dall, Bp)) {
            FwdArgs a;
            a.q = static_cast<const __nv_bfloat16 *>(q);
            a.prefix_k = static_cast<const __nv_bfloat16 *>(prefix_k);
            a.prefix_v = static_cast<const __nv_bfloat16 *>(prefix_v);
            a.suffix_k = static_cast<const __nv_bfloat16 *>(suffix_k);
            a.suffix_v = static_cast<const __nv_bfloat16 *>(suffix_v);
            a.out = static_cast<__nv_bfloat16 *>(out);
            a.lse = lse;
            a.suffix_len = nullptr;
            a.scale = scale;
            a.dims = dall;
            cudaError_t e = launch_tc_fwd(a, workspace, status_word, stream, Bp, prefix_len);
            return e == cudaSuccess ? PSKV_OK : cuda_fail(e);
        }
    }
    std::lock_guard<std::mutex> lock(g_side_mutex);
    SideStream *side = Bp > 1 ? side_stream() : nullptr;
    if (side) {
        cudaError_t e = cudaEventRecord(side->fork, stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(side->stream, side->fork, 0);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    pskv_status result = PSKV_OK;
    for (int i = 0; i < Bp && result == PSKV_OK; ++i) {
        Dims dm;
        check_dims(Kq, Hq, Hkv, S, prefix_len[i], d, &dm);
        dm.Pstride = Pmax;
        cudaStream_t pass_stream = (side && (i & 1)) ? side->stream : stream;
        // the real tokens of a left-padded prefix are its last prefix_len[i] rows
        const size_t p_off = ((size_t)i * Hkv * Pmax + (size_t)(Pmax - prefix_len[i])) * d;
        FwdArgs a;
        a.q = static_cast<const __nv_bfloat16 *>(q) + i * q_part;
        a.prefix_k = Pmax > 0 ? static_cast<const __nv_bfloat16 *>(prefix_k) + p_off : nullptr;
        a.prefix_v = Pmax > 0 ? static_cast<const __nv_bfloat16 *>(prefix_v) + p_off : nullptr;
        a.suffix_k = static_cast<const __nv_bfloat16 *>(suffix_k) + i * s_part;
        a.suffix_v = static_cast<const __nv_bfloat16 *>(suffix_v) + i * s_part;
        a.out = static_cast<__nv_bfloat16 *>(out) + i * q_part;
        a.lse = lse + i * l_part;
        a.suffix_len = nullptr;
        a.scale = scale;
        a.dims = dm;
        cudaError_t e = tc_fwd_supported(dm) ? launch_tc_fwd(a, workspace, status_word, pass_stream)
                                             : launch_simt_fwd(a, pass_stream);
        if (e != cudaSuccess) result = cuda_fail(e);
    }
    if (side) {  // the caller's stream waits for the passes that ran beside it (also after an error)
        cudaError_t e = cudaEventRecord(side->join, side->stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(stream, side->join, 0);
        if (e != cudaSuccess && result == PSKV_OK) result = cuda_fail(e);
    }
    return result;
}

pskv_status pskv_attn_bwd_multi(const void *dout, const void *q, const void *prefix_k, const void *prefix_v,
                                const int *prefix_len, const void *suffix_k, const void *suffix_v, const void *out,
                                const float *lse, float scale, void *dq, void *dk_suffix, void *dv_suffix, int B,
                                int Bp, int Hq, int Hkv, int S, int Pmax, int d, void *workspace,
                                size_t workspace_bytes, void *cuda_stream)
{
    pskv_status st = check_multi(B, Bp, Hq, Hkv, S, Pmax, d, prefix_len);
    if (st != PSKV_OK) return st;
    if (!dout || !q || !suffix_k || !suffix_v || !out || !lse || !dq || !dk_suffix || !dv_suffix)
        return PSKV_ERR_INVALID_ARG;
    if (Pmax > 0 && (!prefix_k || !prefix_v)) return PSKV_ERR_INVALID_ARG;
    if (!aligned16(dout) || !aligned16(q) || !aligned16(prefix_k) || !aligned16(prefix_v) ||
        !aligned16(suffix_k) || !aligned16(suffix_v) || !aligned16(out) || !aligned16(lse) ||
        !aligned16(dq) || !aligned16(dk_suffix) || !aligned16(dv_suffix))
        return PSKV_ERR_INVALID_ARG;
    if (!(scale == scale) || scale <= 0.f || scale > 1.0e6f) return PSKV_ERR_INVALID_ARG;
    const size_t need = pskv_attn_bwd_multi_workspace_bytes(B, Bp, Hq, Hkv, S, Pmax, d);
    if (!workspace || workspace_bytes < need || !aligned16(workspace)) return PSKV_ERR_WORKSPACE;

    unsigned int *status_word = nullptr;
    st = check_device(&status_word);
    if (st != PSKV_OK) return st;

    const int Kq = B / Bp;
    const size_t q_part = (size_t)Kq * Hq * S * d, s_part = (size_t)Kq * Hkv * S * d, l_part = (size_t)Kq * Hq * S;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    auto fill = [&](BwdArgs &a, int first, const Dims &dm, size_t p_off) {
        // arguments of the candidates [first*Kq, ...) with the prefix cache of one instruction
        a.dout = static_cast<const __nv_bfloat16 *>(dout) + first * q_part;
        a.q = static_cast<const __nv_bfloat16 *>(q) + first * q_part;
        a.prefix_k = Pmax > 0 ? static_cast<const __nv_bfloat16 *>(prefix_k) + p_off : nullptr;
        a.prefix_v = Pmax > 0 ? static_cast<const __nv_bfloat16 *>(prefix_v) + p_off : nullptr;
        a.suffix_k = static_cast<const __nv_bfloat16 *>(suffix_k) + first * s_part;
        a.suffix_v = static_cast<const __nv_bfloat16 *>(suffix_v) + first * s_part;
        a.out = static_cast<const __nv_bfloat16 *>(out) + first * q_part;
        a.lse = lse + first * l_part;
        a.dq = static_cast<__nv_bfloat16 *>(dq) + first * q_part;
        a.dk_suffix = static_cast<__nv_bfloat16 *>(dk_suffix) + first * s_part;
        a.dv_suffix = static_cast<__nv_bfloat16 *>(dv_suffix) + first * s_part;
        a.row_dot = static_cast<float *>(workspace) + first * l_part;  // one contiguous [B*Hq*S] array
        a.dlse = nullptr;
        a.suffix_len = nullptr;
        a.scale = scale;
        a.dims = dm;
    };
    {
        // All instructions in one dQ launch when every tile lies inside one instruction (as in the forward);
        // the row statistic before it and the suffix gradients after it never involved the prefix.
        Dims dall;
        if (Bp > 1 && multi_form() != 2 && check_dims(B, Hq, Hkv, S, Pmax, d, &dall) == PSKV_OK &&
            tc_bwd_fused_supported(dall, Bp)) {
            BwdArgs a;
            fill(a, 0, dall, 0);
            cudaError_t e = launch_tc_bwd(a, workspace, status_word, stream, kBwdPartAll, Bp, prefix_len);
            return e == cudaSuccess ? PSKV_OK : cuda_fail(e);
        }
    }
    // The row statistic D = <dout, out> and the suffix gradients do not involve the prefix: when every
    // instruction's part runs on the tensor-core kernels they are done once over all B candidates, and
    // only the dQ step runs once per instruction.
    bool all_tc = true;
    for (int i = 0; i < Bp && all_tc; ++i) {
        Dims dm;
        st = check_dims(Kq, Hq, Hkv, S, prefix_len[i], d, &dm);
        if (st != PSKV_OK) return st;
        all_tc = tc_bwd_supported(dm);
    }
    Dims whole;
    st = check_dims(B, Hq, Hkv, S, prefix_len[0], d, &whole);
    if (st != PSKV_OK) return st;
    all_tc = all_tc && tc_bwd_supported(whole);
    if (all_tc) {
        BwdArgs a;
        fill(a, 0, whole, 0);
        cudaError_t e = launch_tc_bwd(a, workspace, status_word, stream, kBwdPartRowDot);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    // the dQ passes of different instructions alternate between the caller's stream and the internal one
    std::lock_guard<std::mutex> lock(g_side_mutex);
    SideStream *side = (all_tc && Bp > 1) ? side_stream() : nullptr;
    if (side) {
        cudaError_t e = cudaEventRecord(side->fork, stream);  // behind the D pre-pass
        if (e == cudaSuccess) e = cudaStreamWaitEvent(side->stream, side->fork, 0);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    pskv_status result = PSKV_OK;
    for (int i = 0; i < Bp && result == PSKV_OK; ++i) {
        Dims dm;
        st = check_dims(Kq, Hq, Hkv, S, prefix_len[i], d, &dm);
        if (st != PSKV_OK) { result = st; break; }
        dm.Pstride = Pmax;
        const size_t p_off = ((size_t)i * Hkv * Pmax + (size_t)(Pmax - prefix_len[i])) * d;
        cudaStream_t pass_stream = (side && (i & 1)) ? side->stream : stream;
        BwdArgs a;
        fill(a, i, dm, p_off);
        cudaError_t e = all_tc ? launch_tc_bwd(a, a.row_dot, status_word, pass_stream, kBwdPartDq)
                               : tc_bwd_supported(dm) ? launch_tc_bwd(a, a.row_dot, status_word, stream)
                                                      : launch_simt_bwd(a, stream);
        if (e != cudaSuccess) result = cuda_fail(e);
    }
    if (side) {
        cudaError_t e = cudaEventRecord(side->join, side->stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(stream, side->join, 0);
        if (e != cudaSuccess && result == PSKV_OK) result = cuda_fail(e);
    }
    if (result != PSKV_OK) return result;
    if (all_tc) {
        BwdArgs a;
        fill(a, 0, whole, 0);
        cudaError_t e = launch_tc_bwd(a, workspace, status_word, stream, kBwdPartDkv);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return PSKV_OK;
}

// ---- gradients of the shared prefix cache ---------------------------------------------------------------

size_t pskv_attn_bwd_prefix_workspace_bytes(int B, int Hq, int Hkv, int S, int P, int d)
{
    Dims dm;
    if (check_dims(B, Hq, Hkv, S, P, d, &dm) != PSKV_OK || P < 1) return 0;
    // one fp32 per query row (D), then the fp32 accumulators of both gradients
    return round256((size_t)B * Hq * S * sizeof(float)) + round256(2 * (size_t)Hkv * P * d * sizeof(float));
}

pskv_status pskv_attn_bwd_prefix(const void *dout, const float *dlse, const void *q, const void *prefix_k,
                                 const void *prefix_v, const void *out, const float *lse, float scale,
                                 void *dk_prefix, void *dv_prefix, int B, int Hq, int Hkv, int S, int P, int d,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    Dims dm;
    pskv_status st = check_dims(B, Hq, Hkv, S, P, d, &dm);
    if (st != PSKV_OK) return st;
    if (P < 1) return PSKV_ERR_INVALID_ARG;
    if (!dout || !q || !prefix_k || !prefix_v || !out || !lse || !dk_prefix || !dv_prefix) return PSKV_ERR_INVALID_ARG;
    if (!aligned16(dout) || !aligned16(dlse) || !aligned16(q) || !aligned16(prefix_k) || !aligned16(prefix_v) ||
        !aligned16(out) || !aligned16(lse) || !aligned16(dk_prefix) || !aligned16(dv_prefix))
        return PSKV_ERR_INVALID_ARG;
    if (!(scale == scale) || scale <= 0.f || scale > 1.0e6f) return PSKV_ERR_INVALID_ARG;
    const size_t need = pskv_attn_bwd_prefix_workspace_bytes(B, Hq, Hkv, S, P, d);
    if (!workspace || workspace_bytes < need || !aligned16(workspace)) return PSKV_ERR_WORKSPACE;
    unsigned int *status_word = nullptr;
    st = check_device(&status_word);
    if (st != PSKV_OK) return st;

    BwdArgs a;
    memset(&a, 0, sizeof(a));
    a.dout = static_cast<const __nv_bfloat16 *>(dout);
    a.q = static_cast<const __nv_bfloat16 *>(q);
    a.prefix_k = static_cast<const __nv_bfloat16 *>(prefix_k);
    a.prefix_v = static_cast<const __nv_bfloat16 *>(prefix_v);
    a.out = static_cast<const __nv_bfloat16 *>(out);
    a.lse = lse;
    a.row_dot = static_cast<float *>(workspace);
    a.dlse = dlse;
    a.scale = scale;
    a.dims = dm;
    float *acc32 = reinterpret_cast<float *>(static_cast<char *>(workspace) + round256((size_t)B * Hq * S * sizeof(float)));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = launch_simt_row_dot(a, stream);  // D = <dout, out> - dlse per row
    if (e != cudaSuccess) return cuda_fail(e);
    e = tc_bwd_prefix_supported(dm)
            ? launch_tc_bwd_prefix(a, static_cast<__nv_bfloat16 *>(dk_prefix), static_cast<__nv_bfloat16 *>(dv_prefix),
                                   acc32, status_word, stream)
            : launch_simt_bwd_prefix(a, static_cast<__nv_bfloat16 *>(dk_prefix), static_cast<__nv_bfloat16 *>(dv_prefix),
                                     stream);
    return e == cudaSuccess ? PSKV_OK : cuda_fail(e);
}

// ---- masked target cross-entropy fused with the vocabulary projection ---------------------------------

size_t pskv_target_ce_fwd_workspace_bytes(int N, int Lr, int Dm, int V)
{
    return ce_fwd_supported(N, Lr, Dm, V) ? round256(ce_fwd_workspace_bytes(N, Lr, Dm, V)) : 0;
}

pskv_status pskv_target_ce_fwd(const void *hidden, const void *weight, const int *target, const float *mask,
                               float *nll, float *lse, float *loss, int N, int Lr, int Dm, int V, void *workspace,
                               size_t workspace_bytes, void *cuda_stream)
{
    if (N < 1 || Lr < 1 || Dm < 1 || V < 1) return PSKV_ERR_INVALID_ARG;
    if (!ce_fwd_supported(N, Lr, Dm, V)) return PSKV_ERR_UNSUPPORTED_SHAPE;
    if (!hidden || !weight || !target || !mask || !nll || !lse || !loss) return PSKV_ERR_INVALID_ARG;
    if (!aligned16(hidden) || !aligned16(weight) || !aligned16(target) || !aligned16(mask) || !aligned16(nll) ||
        !aligned16(lse) || !aligned16(loss))
        return PSKV_ERR_INVALID_ARG;
    const size_t need = pskv_target_ce_fwd_workspace_bytes(N, Lr, Dm, V);
    if (!workspace || workspace_bytes < need || !aligned16(workspace)) return PSKV_ERR_WORKSPACE;
    unsigned int *status_word = nullptr;
    pskv_status st = check_device(&status_word);
    if (st != PSKV_OK) return st;
    CeArgs a;
    a.hidden = static_cast<const __nv_bfloat16 *>(hidden);
    a.weight = static_cast<const __nv_bfloat16 *>(weight);
    a.target = target; a.mask = mask; a.nll = nll; a.lse = lse; a.loss = loss;
    a.N = N; a.Lr = Lr; a.Dm = Dm; a.V = V;
    cudaError_t e = launch_ce_fwd(a, workspace, status_word, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? PSKV_OK : cuda_fail(e);
}

pskv_status pskv_poll_device_status(void *cuda_stream)
{
    unsigned int *status_word = nullptr;
    pskv_status st = check_device(&status_word);
    if (st != PSKV_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaStreamSynchronize(stream);
    if (e != cudaSuccess) return cuda_fail(e);
    unsigned int word = 0;
    e = cudaMemcpy(&word, status_word, sizeof(word), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e);
    if (word != 0) {
        e = cudaMemset(status_word, 0, sizeof(word));
        if (e != cudaSuccess) return cuda_fail(e);
        return PSKV_ERR_DEVICE_TIMEOUT;
    }
    return PSKV_OK;
}

}  // extern "C"
