// Shared declarations of the libpskv translation units (host launchers + small device helpers).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "pskv.h"

namespace pskv {

// Dimensions of one call; `n_rep` = Hq / Hkv query heads per KV head.  `Pstride` is the distance, in
// rows, between the prefix blocks of consecutive KV heads (P for a dense prefix cache; the padded
// length when the call works on the real tokens of a left-padded cache).  `S` counts the query rows
// per candidate and `Skv` the rows of its suffix K/V buffer: equal for the full-suffix operator,
// Skv >= S for the decode-shaped one, where the queries are the last S of the candidate's cached
// suffix tokens.  `ragged` is 1 when a per-candidate count of cached tokens (suffix_len) is given.
struct Dims {
    int B, Hq, Hkv, S, P, d, n_rep, Pstride, Skv, ragged;
};

// Cached suffix tokens of candidate b, forced into [S, Skv] so that no value can index outside the
// buffers; query i of the candidate is suffix token suffix_tokens(...) - S + i.
__device__ __forceinline__ int suffix_tokens(const int *suffix_len, int b, int S, int Skv)
{
    if (!suffix_len) return Skv;
    const int L = suffix_len[b];
    return L < S ? S : (L > Skv ? Skv : L);
}

struct FwdArgs {
    const __nv_bfloat16 *q, *prefix_k, *prefix_v, *suffix_k, *suffix_v;
    __nv_bfloat16 *out;
    float *lse;
    const int *suffix_len;  // device, [B], or nullptr: every candidate has Skv cached suffix tokens
    float scale;
    Dims dims;
};

struct BwdArgs {
    const __nv_bfloat16 *dout, *q, *prefix_k, *prefix_v, *suffix_k, *suffix_v, *out;
    const float *lse;
    __nv_bfloat16 *dq, *dk_suffix, *dv_suffix;
    float *row_dot;  // workspace: D[b,h,i] = <dout, out> - dlse[b,h,i], fp32 [B*Hq*S]
    const float *dlse;  // gradient arriving on lse, fp32 [B*Hq*S], or nullptr (none)
    const int *suffix_len;  // as in FwdArgs
    float scale;
    Dims dims;
};

// General CUDA-core kernels (any S, Skv, P; d in {64,128}; ragged or not).
cudaError_t launch_simt_fwd(const FwdArgs &a, cudaStream_t stream);
cudaError_t launch_simt_bwd(const BwdArgs &a, cudaStream_t stream);
// Pieces of the backward the tensor-core path reuses: D = <dout, out> per row into a.row_dot, and
// dk_suffix / dv_suffix (needs row_dot and lse).
cudaError_t launch_simt_row_dot(const BwdArgs &a, cudaStream_t stream);
cudaError_t launch_simt_bwd_dkv(const BwdArgs &a, cudaStream_t stream);
// dk_suffix / dv_suffix on warp-level tensor-core MMAs, one CTA per (candidate, KV head); S <= 64.
bool mma_bwd_dkv_supported(const Dims &d);
cudaError_t launch_mma_bwd_dkv(const BwdArgs &a, cudaStream_t stream);
bool tc_bwd_dkv_supported(const Dims &d);
// Gradients of the shared prefix cache (need row_dot): tensor-core kernel (d = 128; `acc32` holds
// 2 * Hkv * P * d floats of scratch) or the general one.
bool tc_bwd_prefix_supported(const Dims &d);
cudaError_t launch_tc_bwd_prefix(const BwdArgs &a, __nv_bfloat16 *dk_prefix, __nv_bfloat16 *dv_prefix, float *acc32,
                                 unsigned int *status_word, cudaStream_t stream);
cudaError_t launch_simt_bwd_prefix(const BwdArgs &a, __nv_bfloat16 *dk_prefix, __nv_bfloat16 *dv_prefix,
                                   cudaStream_t stream);
// with_d: the kernel also forms D = <dout, out> - dlse per row and writes it to a.row_dot (it then needs
// a.out and no pre-pass); tc_bwd_dkv_row_dot_supported tells whether the shape allows that.
bool tc_bwd_dkv_row_dot_supported(const Dims &d);
cudaError_t launch_tc_bwd_dkv(const BwdArgs &a, unsigned int *status_word, cudaStream_t stream, bool with_d = false);

// tcgen05/TMEM kernels.  `status_word` is the device status flag that bounded waits set.
bool tc_fwd_supported(const Dims &d);
size_t tc_fwd_workspace_bytes(const Dims &d);
// Several instructions in one launch (Sec. 4.3): the B candidates fall into `n_instr` contiguous groups
// of equal size, group i uses prefix cache i of prefix_k / prefix_v [n_instr][Hkv][P][d], whose last
// prefix_len[i] rows (host array) are real tokens and whose first rows are left padding.
constexpr int kMaxFusedInstructions = 64;
bool tc_fwd_fused_supported(const Dims &d, int n_instr);
cudaError_t launch_tc_fwd(const FwdArgs &a, void *workspace, unsigned int *status_word,
                          cudaStream_t stream, int n_instr = 1, const int *prefix_len = nullptr);
// The forward on CTA pairs (cta_group::2), for the shapes it takes; launch_tc_fwd goes there by itself
// unless pairs are switched off (pskv_enable_cta_pairs).
bool tc_fwd_pair_supported(const Dims &d);
cudaError_t launch_tc_fwd_pair(const FwdArgs &a, unsigned int *status_word, cudaStream_t stream);
bool cta_pairs_enabled();
bool tc_bwd_supported(const Dims &d);
size_t tc_bwd_workspace_bytes(const Dims &d);
// `parts` selects which of the three steps run (all by default): the row statistic D and the suffix
// gradients do not involve the prefix, so a caller with several prefixes runs them once over all
// candidates and the dQ step once per prefix.  Where one kernel produces both the row statistic and the
// suffix gradients (tc_bwd_dkv_row_dot_supported) it runs for kBwdPartRowDot and kBwdPartDkv is empty;
// a caller that splits the parts must ask for kBwdPartRowDot before kBwdPartDq either way.
enum { kBwdPartRowDot = 1, kBwdPartDq = 2, kBwdPartDkv = 4, kBwdPartAll = 7 };
bool tc_bwd_fused_supported(const Dims &d, int n_instr);  // several instructions in one dQ launch (as for the forward)
cudaError_t launch_tc_bwd(const BwdArgs &a, void *workspace, unsigned int *status_word,
                          cudaStream_t stream, int parts = kBwdPartAll, int n_instr = 1,
                          const int *prefix_len = nullptr);

// Masked target cross-entropy fused with the vocabulary projection (tcgen05 GEMM whose logits stay on chip).
struct CeArgs {
    const __nv_bfloat16 *hidden, *weight;  // [N*Lr, Dm], [V, Dm]
    const int *target;                     // [N*Lr]
    const float *mask;                     // [N*Lr] loss weights
    float *nll, *lse, *loss;               // [N*Lr], [N*Lr], [N]
    int N, Lr, Dm, V;
};
bool ce_fwd_supported(int N, int Lr, int Dm, int V);
size_t ce_fwd_workspace_bytes(int N, int Lr, int Dm, int V);
cudaError_t launch_ce_fwd(const CeArgs &a, void *workspace, unsigned int *status_word, cudaStream_t stream);

// PSKV_OK and the device address of the status word when the current device is an sm_100 part, else the
// error the public calls return for it (PSKV_ERR_UNSUPPORTED_ARCH, PSKV_ERR_CUDA).
pskv_status device_status_word(unsigned int **status_word);

// Host-side count of kernel launches (read through pskv_kernel_launches()).
void count_launches(int n);

// Optional per-kernel device timing (pskv_kernel_timing_*): when enabled, a launch site brackets
// its kernel with two CUDA events on the launch stream.
enum KernelId {
    kKernelFwdTc = 0, kKernelRowDot, kKernelBwdDqTc, kKernelBwdDkvTc, kKernelBwdDkvMma,
    kKernelFwdSimt, kKernelBwdDqSimt, kKernelBwdDkvSimt, kKernelCeFwd, kKernelCeFinalize, kKernelBwdPrefixTc, kKernelBwdPrefixSimt, kKernelCount
};
void *timing_begin(int kernel_id, cudaStream_t stream);  // returns nullptr when timing is off
void timing_end(void *token, cudaStream_t stream);
struct KernelTiming {
    void *token;
    cudaStream_t stream;
    KernelTiming(int id, cudaStream_t s) : token(timing_begin(id, s)), stream(s) {}
    ~KernelTiming() { if (token) timing_end(token, stream); }
};

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

}  // namespace pskv
