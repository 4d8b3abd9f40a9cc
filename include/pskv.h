/*
 * pskv.h -- C ABI of the shared-prefix attention library (libpskv.so), sm_100a only.
 *
 * The operation is the per-layer attention step of prefix-shared KV caching:
 * B candidate suffixes are scored against ONE compact prefix K/V cache that is
 * stored once and never duplicated along the candidate dimension (paper
 * Sec. 4.2), plus each candidate's own suffix-side K/V.  Mathematically it is
 * scaled-dot-product attention (Eq. 2) over K = prefix (+) suffix, i.e. what
 * the candidate-expanded cache of Eq. 3 would give, without building it.
 *
 * Conventions for every call
 *   - All tensor pointers are DEVICE pointers owned by the caller; the library
 *     never allocates, frees or keeps them.  Tensors are dense, row-major, last
 *     index fastest, and every base address must be 16-byte aligned.
 *   - bf16 tensors are raw 16-bit bfloat16; lse is fp32.
 *   - Query head h reads KV head g = h / (Hq / Hkv) (grouped-query attention,
 *     Appendix E; Table 8 lists the head counts).
 *   - Suffix row i of a candidate sees all P prefix keys and suffix keys 0..i
 *     (causal, diagonal included: the K_{<=t} of Eq. 2).  P = 0 is legal.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*, NULL =
 *     the default stream) and the call returns without synchronising.
 *   - Arguments are validated on the host before anything is launched; a call
 *     that returns non-zero has launched nothing.
 *   - There is no CPU fallback: without an sm_100 device the calls fail.
 */
#ifndef PSKV_H_
#define PSKV_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PSKV_OK = 0,
    PSKV_ERR_INVALID_ARG = 1,       /* null / misaligned pointer, non-positive size, Hq % Hkv != 0 */
    PSKV_ERR_UNSUPPORTED_SHAPE = 2, /* head dim other than 64 or 128, or sizes beyond the kernels' limits */
    PSKV_ERR_UNSUPPORTED_ARCH = 3,  /* current device is not compute capability 10.x */
    PSKV_ERR_WORKSPACE = 4,         /* workspace missing, misaligned or smaller than *_workspace_bytes() */
    PSKV_ERR_CUDA = 5,              /* a CUDA runtime/driver call failed; see pskv_last_cuda_error() */
    PSKV_ERR_DEVICE_TIMEOUT = 6     /* a bounded device-side wait expired (reported by pskv_poll_device_status) */
} pskv_status;

/* Scratch (device global memory) the forward call needs for these sizes; may be 0. */
size_t pskv_attn_fwd_workspace_bytes(int B, int Hq, int Hkv, int S, int P, int d);

/*
 * Forward (Eq. 2 over the shared prefix cache of Sec. 4.2 plus the suffix K/V):
 *   s_j  = scale * <q[b,h,i,:], K_j>,  K = prefix_k[g] (P rows) then suffix_k[b,g] rows 0..i
 *   lse[b,h,i]   = ln sum_j exp(s_j)                      (natural log, scale included)
 *   out[b,h,i,:] = sum_j exp(s_j - lse) V_j                (rounded to bf16)
 * Inputs are read-only; out and lse are fully overwritten.  Accumulation is fp32.
 * Any S is legal.  With B = 1 and P = 0 the call is the causal self-attention of one sequence whose
 * keys and values are passed as suffix_k / suffix_v: the attention step of the prefill that produces a
 * prefix cache in the first place.
 */
pskv_status pskv_attn_fwd(const void *q,        /* bf16 [B,Hq,S,d]  */
                          const void *prefix_k, /* bf16 [Hkv,P,d]   (may be NULL when P == 0) */
                          const void *prefix_v, /* bf16 [Hkv,P,d]   (may be NULL when P == 0) */
                          const void *suffix_k, /* bf16 [B,Hkv,S,d] */
                          const void *suffix_v, /* bf16 [B,Hkv,S,d] */
                          float scale,
                          void *out,            /* bf16 [B,Hq,S,d]  */
                          float *lse,           /* fp32 [B,Hq,S]    */
                          int B, int Hq, int Hkv, int S, int P, int d,
                          void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Scratch the backward call needs for these sizes (holds per-row fp32 statistics). */
size_t pskv_attn_bwd_workspace_bytes(int B, int Hq, int Hkv, int S, int P, int d);

/*
 * Backward of L = sum(out * dout) with the prefix cache frozen (Sec. 4.2: the
 * prefix is computed once; only suffix-side gradients are needed for
 * gradient-guided suffix search).  With p_j = exp(s_j - lse), D = <dout, out>,
 * ds_j = p_j (<dout, V_j> - D):
 *   dq[b,h,i,:]        = scale * sum_j ds_j K_j
 *   dk_suffix[b,g,t,:] = scale * sum over heads h of g and rows i >= t of ds_{P+t} q[b,h,i,:]
 *   dv_suffix[b,g,t,:] =         sum over the same (h, i) of p_{P+t} dout[b,h,i,:]
 * `out` and `lse` are the forward results for the same inputs.  No gradient is
 * produced for prefix_k / prefix_v, and lse carries no incoming gradient here (pskv_attn_bwd_lse
 * takes one).
 * The three outputs are fully overwritten.
 */
pskv_status pskv_attn_bwd(const void *dout,     /* bf16 [B,Hq,S,d]  */
                          const void *q, const void *prefix_k, const void *prefix_v,
                          const void *suffix_k, const void *suffix_v,
                          const void *out,      /* bf16 [B,Hq,S,d], from pskv_attn_fwd */
                          const float *lse,     /* fp32 [B,Hq,S],   from pskv_attn_fwd */
                          float scale,
                          void *dq,             /* bf16 [B,Hq,S,d]  */
                          void *dk_suffix,      /* bf16 [B,Hkv,S,d] */
                          void *dv_suffix,      /* bf16 [B,Hkv,S,d] */
                          int B, int Hq, int Hkv, int S, int P, int d,
                          void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * pskv_attn_bwd with a gradient arriving on the log-sum-exp as well: the backward of
 * L = sum(out * dout) + sum(lse * dlse).  lse is a second output of the forward call; a caller that
 * merges this call's result with another partial attention result by their log-sum-exps, or that uses
 * lse in a loss, sends a gradient back through it.  Since d lse / d s_j = p_j, the formulas of
 * pskv_attn_bwd hold with ds_j = p_j (<dout, V_j> - D + dlse[b,h,i]); dv_suffix is unaffected.
 * dlse is fp32 [B,Hq,S], device, 16-byte aligned, read-only, and must not be NULL (use pskv_attn_bwd).
 * Everything else -- arguments, workspace size, error codes -- is as in pskv_attn_bwd.
 */
pskv_status pskv_attn_bwd_lse(const void *dout,   /* bf16 [B,Hq,S,d] */
                              const float *dlse,  /* fp32 [B,Hq,S]   */
                              const void *q, const void *prefix_k, const void *prefix_v,
                              const void *suffix_k, const void *suffix_v,
                              const void *out, const float *lse, float scale,
                              void *dq, void *dk_suffix, void *dv_suffix,
                              int B, int Hq, int Hkv, int S, int P, int d,
                              void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Gradients of the shared prefix cache: what pskv_attn_bwd leaves out.  The search keeps the prefix
 * frozen (Sec. 4.2) and never needs them; a caller that wants full differentiability (a trainable
 * prefix, a check of the whole backward) gets them here.  With p_j, D and ds_j as in pskv_attn_bwd
 * (dlse may be NULL), for every prefix key j < P of KV head g
 *   dk_prefix[g,j,:] = scale * sum over ALL candidates b, heads h of g and rows i of  ds_j q[b,h,i,:]
 *   dv_prefix[g,j,:] =         sum over the same (b, h, i) of                          p_j dout[b,h,i,:]
 * (every row sees every prefix key).  The suffix K/V are not needed: they enter only through `out`
 * and `lse`, the forward results.  Sums are accumulated in fp32 (atomic adds across candidate chunks on
 * the tensor-core path, so the last bits may differ from run to run) and rounded to bf16 once.
 * P must be at least 1.  dk_prefix, dv_prefix: bf16 [Hkv,P,d], fully overwritten.
 */
size_t pskv_attn_bwd_prefix_workspace_bytes(int B, int Hq, int Hkv, int S, int P, int d);
pskv_status pskv_attn_bwd_prefix(const void *dout,     /* bf16 [B,Hq,S,d] */
                                 const float *dlse,    /* fp32 [B,Hq,S] or NULL */
                                 const void *q, const void *prefix_k, const void *prefix_v,
                                 const void *out, const float *lse, float scale,
                                 void *dk_prefix,      /* bf16 [Hkv,P,d] */
                                 void *dv_prefix,      /* bf16 [Hkv,P,d] */
                                 int B, int Hq, int Hkv, int S, int P, int d,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * pskv_attn_bwd without a workspace argument.  (The paper has no counterpart; this is a
 * convenience of this library.)  It is for callers that cannot allocate device memory: processes
 * in which a framework allocator owns the whole card, or loops with a fixed memory plan in which a
 * cudaMalloc would fail or stall every stream while it synchronises the device.  The per-row
 * scratch of the backward pass lives in a 4 MiB array inside the library image, which every GPU
 * that loads the library holds until the process exits.
 *   - Same arguments, results, layouts and error codes as pskv_attn_bwd; it calls no cudaMalloc,
 *     cudaFree or other allocating routine.
 *   - Sizes with B*Hq*S > pskv_attn_bwd_static_max_rows() (1048576) return PSKV_ERR_WORKSPACE and
 *     launch nothing; use pskv_attn_bwd with your own workspace for those.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call before starting any stream capture.
 *   - All calls share the one array and it keeps the previous call's contents.  Nothing needs
 *     clearing (each call overwrites every element it later reads), but two calls that overlap
 *     on the GPU -- different streams, or different host threads -- race on it and give wrong
 *     gradients; serialise them.
 */
pskv_status pskv_attn_bwd_static(const void *dout, const void *q, const void *prefix_k, const void *prefix_v,
                                 const void *suffix_k, const void *suffix_v, const void *out, const float *lse,
                                 float scale, void *dq, void *dk_suffix, void *dv_suffix,
                                 int B, int Hq, int Hkv, int S, int P, int d, void *cuda_stream);
long long pskv_attn_bwd_static_max_rows(void);

/*
 * Several instructions per call: the batched multi-instruction layout of Sec. 4.3 (suffix-centric
 * alignment) with the position rules of the appendix on position consistency under padding.
 * There are Bp prefix caches, one per instruction, stored left-padded to a common length Pmax:
 *   prefix_k, prefix_v   bf16 [Bp,Hkv,Pmax,d]; the real tokens of instruction i are its LAST
 *                        prefix_len[i] rows (0 <= prefix_len[i] <= Pmax); padding rows may hold any FINITE
 *                        values (they may be read; their scores are masked and their values meet zero
 *                        probabilities)
 *   prefix_len           HOST array of Bp ints (read before the call returns)
 * The B candidates are grouped by instruction: candidate b belongs to instruction b / (B / Bp), so B
 * must be a multiple of Bp and each cache is reused by its B / Bp candidates.  Everything else (q,
 * suffix_k, suffix_v, out, lse, dout, dq, dk_suffix, dv_suffix; scale; causal rule; error codes) is as
 * in pskv_attn_fwd / pskv_attn_bwd, with P replaced per candidate by the true prefix length of its
 * instruction.  When (B / Bp) * (Hq / Hkv) * S is a multiple of the kernels' row tile (128 rows in the
 * usual case), Bp <= 64 and the shape runs on the tensor-core kernels, all instructions are served by one
 * launch per kernel (pskv_set_multi_form(2) turns this off).  Otherwise the work is one pass per instruction; the passes are independent, so every
 * other one is enqueued on a stream of the library's own that forks from `cuda_stream` at the start of the
 * call and joins it again before the call returns (to the caller everything is ordered as if it had run on
 * `cuda_stream`, also under stream capture).
 */
size_t pskv_attn_fwd_multi_workspace_bytes(int B, int Bp, int Hq, int Hkv, int S, int Pmax, int d);

/*
 * How the multi-instruction calls (Sec. 4.3) schedule their work: 0 = the library chooses (one launch for
 * all instructions where the shapes allow it, else one pass per instruction), 1 = the same choice, stated
 * explicitly, 2 = always one pass per instruction.  Both forms compute the same result; the switch exists
 * to compare them.  Process-wide, host side; PSKV_ERR_INVALID_ARG for any other value.
 */
pskv_status pskv_set_multi_form(int form);

pskv_status pskv_attn_fwd_multi(const void *q,        /* bf16 [B,Hq,S,d] */
                                const void *prefix_k, /* bf16 [Bp,Hkv,Pmax,d] (may be NULL when Pmax == 0) */
                                const void *prefix_v, /* bf16 [Bp,Hkv,Pmax,d] */
                                const int *prefix_len, /* host, [Bp] */
                                const void *suffix_k, /* bf16 [B,Hkv,S,d] */
                                const void *suffix_v, /* bf16 [B,Hkv,S,d] */
                                float scale,
                                void *out,            /* bf16 [B,Hq,S,d] */
                                float *lse,           /* fp32 [B,Hq,S] */
                                int B, int Bp, int Hq, int Hkv, int S, int Pmax, int d,
                                void *workspace, size_t workspace_bytes, void *cuda_stream);
size_t pskv_attn_bwd_multi_workspace_bytes(int B, int Bp, int Hq, int Hkv, int S, int Pmax, int d);
pskv_status pskv_attn_bwd_multi(const void *dout, const void *q, const void *prefix_k, const void *prefix_v,
                                const int *prefix_len, const void *suffix_k, const void *suffix_v,
                                const void *out, const float *lse, float scale,
                                void *dq, void *dk_suffix, void *dv_suffix,
                                int B, int Bp, int Hq, int Hkv, int S, int Pmax, int d,
                                void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Decode-shaped variant: the suffix grows token by token (beam-search and sampling-based attacks
 * extend every candidate by a few tokens per step on top of what is already cached), so only the
 * newest tokens of each candidate are queries.  Each candidate b owns a suffix cache buffer of Skv
 * rows, suffix_k / suffix_v [B,Hkv,Skv,d], whose first suffix_len[b] rows are cached suffix tokens
 * (the K/V of the new tokens already appended); the Sq query rows q[b,:,i,:] are the LAST Sq of
 * them: query i is suffix token suffix_len[b] - Sq + i and, by the causal rule of Eq. 2, sees all P
 * prefix keys and suffix keys 0 .. suffix_len[b] - Sq + i.  With Sq == Skv and no suffix_len this is
 * pskv_attn_fwd / pskv_attn_bwd.
 *   suffix_len   DEVICE array of B ints, 4-byte aligned, or NULL (= every candidate has Skv tokens).
 *                Values must lie in [Sq, Skv]; the kernels force them into that range, so a bad
 *                value gives wrong numbers for that candidate but never an out-of-range access.
 *   Rows of suffix_k / suffix_v at or past suffix_len[b] take no part in the result, but they are
 *   loaded and multiplied by a zero probability, so they must hold finite numbers (clear the
 *   buffer once when it is allocated).
 *   Backward: dq [B,Hq,Sq,d]; dk_suffix, dv_suffix [B,Hkv,Skv,d] cover every cached token (also
 *   those older than the queries); rows at or past suffix_len[b] are written as zeros.
 * Everything else (layouts, scale, lse, error codes, stream semantics) is as in the calls above.
 */
size_t pskv_attn_fwd_decode_workspace_bytes(int B, int Hq, int Hkv, int Sq, int Skv, int P, int d);
pskv_status pskv_attn_fwd_decode(const void *q,        /* bf16 [B,Hq,Sq,d] */
                                 const void *prefix_k, /* bf16 [Hkv,P,d] (may be NULL when P == 0) */
                                 const void *prefix_v, /* bf16 [Hkv,P,d] */
                                 const void *suffix_k, /* bf16 [B,Hkv,Skv,d] */
                                 const void *suffix_v, /* bf16 [B,Hkv,Skv,d] */
                                 const int *suffix_len, /* device, [B], or NULL */
                                 float scale,
                                 void *out,            /* bf16 [B,Hq,Sq,d] */
                                 float *lse,           /* fp32 [B,Hq,Sq] */
                                 int B, int Hq, int Hkv, int Sq, int Skv, int P, int d,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream);
size_t pskv_attn_bwd_decode_workspace_bytes(int B, int Hq, int Hkv, int Sq, int Skv, int P, int d);
pskv_status pskv_attn_bwd_decode(const void *dout, const void *q, const void *prefix_k, const void *prefix_v,
                                 const void *suffix_k, const void *suffix_v, const int *suffix_len,
                                 const void *out, const float *lse, float scale,
                                 void *dq, void *dk_suffix, void *dv_suffix,
                                 int B, int Hq, int Hkv, int Sq, int Skv, int P, int d,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Masked target cross-entropy fused with the vocabulary projection (loss appendix: the objective is
 * the masked average of CE(logits, target token) over the target-response span; the logits tensor
 * [candidates x positions x vocabulary] is the memory high-water mark the paper reports for a search
 * step).  For N candidates with Lr scored positions each (rows r = c * Lr + i):
 *   logits[r, v] = <hidden[r, :], weight[v, :]>          (output head without bias; never stored)
 *   lse[r]       = ln sum_v exp(logits[r, v])
 *   nll[r]       = mask[r] * (lse[r] - logits[r, target[r]])      (0 where mask[r] == 0)
 *   loss[c]      = sum_i nll[c*Lr + i] / sum_i mask[c*Lr + i]      (0 for a candidate without weight)
 * The paper's scalar objective is sum_c loss[c] * (weight of c) / (total weight); loss[c] itself is what
 * ranks the candidates of a search step.  Products are exact in fp32 and accumulated in fp32; the
 * logits are never rounded to bf16.
 *   hidden  bf16 [N*Lr, Dm]   final hidden state of every scored position (position r-1 predicts token r)
 *   weight  bf16 [V, Dm]      output-head matrix
 *   target  int32 [N*Lr]      token ids; must lie in [0, V) wherever mask != 0 (else that nll is NaN)
 *   mask    fp32 [N*Lr]       loss weights m^tar (0/1, or any non-negative weight)
 *   nll, lse fp32 [N*Lr], loss fp32 [N]: fully overwritten
 * All pointers are device pointers, 16-byte aligned.  Dm must be a multiple of 8 (else
 * PSKV_ERR_UNSUPPORTED_SHAPE); any N, Lr, V.  Forward only: a search step ranks its candidates by
 * this loss without differentiating through it.
 */
size_t pskv_target_ce_fwd_workspace_bytes(int N, int Lr, int Dm, int V);
pskv_status pskv_target_ce_fwd(const void *hidden, const void *weight, const int *target, const float *mask,
                               float *nll, float *lse, float *loss, int N, int Lr, int Dm, int V,
                               void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * Synchronises `cuda_stream`, then reads and clears the device status word that
 * kernels set when one of their bounded waits gives up.  Returns PSKV_OK,
 * PSKV_ERR_DEVICE_TIMEOUT (results of the affected call are undefined) or
 * PSKV_ERR_CUDA.  Launch calls are asynchronous and cannot report this themselves.
 */
pskv_status pskv_poll_device_status(void *cuda_stream);

/* Static, human-readable name of a status code. */
const char *pskv_status_string(pskv_status status);

/* cudaError_t (as int) recorded by the most recent call that returned PSKV_ERR_CUDA on this thread. */
int pskv_last_cuda_error(void);

/* major * 10000 + minor * 100 + patch */
int pskv_version(void);

/*
 * Which kernel family pskv_attn_fwd / pskv_attn_bwd pick for these sizes:
 * 2 = tcgen05 kernels on CTA pairs (two SMs share every MMA, cta_group::2; only after
 * pskv_enable_cta_pairs(1)), 1 = tcgen05 / TMEM
 * tensor-core kernels, one CTA per tile, 0 = general CUDA-core kernels, negative = sizes rejected.
 * `backward` selects which call is asked about.  Pure host logic; touches no device.
 */
int pskv_kernel_family(int backward, int B, int Hq, int Hkv, int S, int P, int d);

/*
 * The CTA-pair kernels compute the same operator (Eq. 2 over the shared prefix of Sec. 4.2) as the
 * single-CTA tensor-core kernels, for the shapes they take (pskv_kernel_family tells, once they are
 * switched on).  They are OFF by default: at the layer shapes measured so far they are 5-15 % slower
 * than the single-CTA kernels.  on = 1 makes every later call of this process use them where they
 * apply, e.g. to compare the two.  Process-wide, host-side switch; touches no device.
 */
void pskv_enable_cta_pairs(int on);

/*
 * Self-test of the bounded device-side waits (the mechanism behind PSKV_ERR_DEVICE_TIMEOUT): enqueues one
 * tiny kernel on `cuda_stream` in which a single warp waits, through the routine all tensor-core kernels
 * wait with, for a barrier that nothing will ever complete, gives up after `budget_cycles` SM clock cycles
 * (1 .. 1e9), records the time-out in the device status word and returns normally.  The next
 * pskv_poll_device_status on that stream therefore returns PSKV_ERR_DEVICE_TIMEOUT once, and PSKV_OK after
 * that; the device stays fully usable.  Returns PSKV_OK when the kernel was enqueued.  The paper has no
 * counterpart: this checks the library's own failure detection.
 */
pskv_status pskv_selftest_wait_timeout(long long budget_cycles, void *cuda_stream);

/*
 * Self-test of the per-device bookkeeping of the launch sites (per-device opt-in to large dynamic shared
 * memory), run on the host with made-up device ordinals; touches no device.  0 = passed.
 */
int pskv_selftest_per_device_once(void);

/*
 * Number of kernels this library has launched in this process so far (all threads, all devices).
 * A host-side counter for benchmarks that must state how many launches a timed region made.
 */
long long pskv_kernel_launches(void);

/*
 * Optional per-kernel device timing, for benchmarks that must report the duration of one kernel
 * inside a call that launches several.  While enabled, every kernel the library launches is
 * bracketed by two CUDA events on its stream (at most 8192 launches are kept).
 * pskv_kernel_timing_read waits for the recorded launches of one kernel id, returns their summed
 * device time in milliseconds and their count, and forgets them.  Kernel ids run from 0 to
 * pskv_kernel_timing_count() - 1; pskv_kernel_timing_name gives the kernel's name.
 */
void pskv_kernel_timing_enable(int on);
int pskv_kernel_timing_count(void);
const char *pskv_kernel_timing_name(int kernel_id);
pskv_status pskv_kernel_timing_read(int kernel_id, double *total_ms, long long *launches);

#ifdef __cplusplus
}
#endif
#endif /* PSKV_H_ */
