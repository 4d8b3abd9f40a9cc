// Masked target cross-entropy fused with the vocabulary projection, for sm_100a (tcgen05 / TMEM / TMA).
//
// logits = hidden * weight^T is a [rows x V] matrix that is only ever reduced: per row its
// log-sum-exp and the logit of the target token (loss appendix: masked average of CE over the
// target-response span).  Forming it in memory is what the paper names as the memory high-water
// mark of a search step, so here it never leaves the chip: a 128-row x 256-column block of logits is
// accumulated in tensor memory over the hidden dimension, four warps fold it into a running
// (max, sum) per row and pick out the target's logit while the tensor cores already work on the next
// block in the other half of tensor memory.
//
// Work units are (vocabulary panel of 8 blocks, 128-row tile).  Row tiles are taken in groups of a
// quarter of the CTA count; inside a group the units are numbered panel-major, row tile fastest, and
// CTA c takes units c, c + G, c + 2G, ...: the CTAs running at any moment work on about four weight
// panels (16 MB each) against one group of row tiles (1 MB each), a working set that stays in L2, so
// the weight matrix comes from HBM once per row group and the hidden states once.  Each unit
// leaves one partial (max, sum) per row; two small kernels merge the partials of a row into lse
// and nll = mask * (lse - target logit) and form the masked average per candidate.
//
// Roles (256 threads): warp 0 TMA producer (hidden tile and weight block, 64 columns of the hidden
// dimension per stage, 4 stages), warp 1 tcgen05.mma issuer, warp 2 owns the tensor-memory
// allocation, warps 4-7 fold the finished blocks.  Every wait is bounded.
#include <string.h>

#include "pskv_common.cuh"
#include "pskv_sm100.cuh"
#include "pskv_tc_common.cuh"

namespace pskv {
namespace {

using namespace sm100;

constexpr int kCeM = 128;        // rows per tile (tensor-memory lanes)
constexpr int kCeN = 256;        // vocabulary entries per block (one MMA N, half of tensor memory)
constexpr int kCeK = 64;         // hidden columns per stage: one 128-byte swizzle slab
constexpr int kCeStages = 4;
constexpr int kCePanel = 8;      // blocks per panel
constexpr int kCeThreads = 256;
constexpr int kCeABytes = kCeM * 128, kCeBBytes = kCeN * 128, kCeStageBytes = kCeABytes + kCeBBytes;

enum : unsigned int { kErrCeProducer = 0x401, kErrCeMma = 0x402, kErrCeFold = 0x403, kErrCeAlign = 0x404 };

enum { kCeBarFull = 0, kCeBarEmpty = kCeStages, kCeBarAccFull = 2 * kCeStages, kCeBarAccFree = 2 * kCeStages + 2,
       kCeNumBars = 2 * kCeStages + 4 };

struct CeParams {
    const int *target;     // [R]
    float *part_m, *part_l;  // [npanel][Rpad], log2 domain
    float *tlogit;         // [R] logit of the target token (natural units)
    unsigned int *status;
    int R, Rpad, Dm, V;
    int nrt, nvb, npanel, units, ksteps;
    int rg;                // row tiles per group
};

// unit -> (panel, row tile): groups of rg row tiles, panel-major inside a group, the last group smaller
__device__ __forceinline__ void ce_unit(const CeParams &p, int u, int &pn, int &rt)
{
    const int per_group = p.rg * p.npanel;
    const int nfull = p.nrt / p.rg;
    if (u < nfull * per_group) {
        const int gi = u / per_group, rem = u - gi * per_group;
        pn = rem / p.rg;
        rt = gi * p.rg + (rem - pn * p.rg);
    } else {
        const int tail = p.nrt - nfull * p.rg, rem = u - nfull * per_group;
        pn = rem / tail;
        rt = nfull * p.rg + (rem - pn * tail);
    }
}

__global__ void __launch_bounds__(kCeThreads, 1)
ce_fwd_kernel(const __grid_constant__ CUtensorMap tm_h, const __grid_constant__ CUtensorMap tm_w, const CeParams p)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + kCeStages * kCeStageBytes;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + kCeStages * kCeStageBytes + 8 * kCeNumBars + 4);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + kCeStages * kCeStageBytes + 8 * kCeNumBars);

    if ((sbase & 1023u) != 0u) {
        if (tid == 0) atomicCAS(p.status, 0u, (unsigned int)kErrCeAlign);
        return;
    }
    if (tid == 0) {
        for (int i = 0; i < kCeNumBars; ++i) mbar_init(bar(i), i >= kCeBarAccFree ? 4u : 1u);
        *abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();
    if (warp == 2) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    const int n_units = (p.units - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tensormap(&tm_h);
            prefetch_tensormap(&tm_w);
        }
        uint32_t it = 0;
        bool ok = true;
#pragma unroll 1
        for (int tl = 0; tl < n_units && ok; ++tl) {
            const int u = (int)blockIdx.x + tl * (int)gridDim.x;
            int pn, rt;
            ce_unit(p, u, pn, rt);
            const int vb_end = min(p.nvb, (pn + 1) * kCePanel);
#pragma unroll 1
            for (int vb = pn * kCePanel; vb < vb_end && ok; ++vb) {
#pragma unroll 1
                for (int ks = 0; ks < p.ksteps; ++ks, ++it) {
                    const uint32_t s = it % kCeStages;
                    ok = mbar_wait_warp(bar(kCeBarEmpty + s), ((it / kCeStages) & 1) ^ 1, abort_flag, p.status,
                                        kErrCeProducer);
                    if (!ok) break;
                    if (elect_one_sync()) {
                        // boxes that reach past the last row / vocabulary entry / hidden column are
                        // zero-filled and still count their full size
                        mbar_arrive_expect_tx(bar(kCeBarFull + s), (uint32_t)kCeStageBytes);
                        tma_load_2d(sbase + s * kCeStageBytes, &tm_h, bar(kCeBarFull + s), ks * kCeK, rt * kCeM);
                        tma_load_2d(sbase + s * kCeStageBytes + kCeABytes, &tm_w, bar(kCeBarFull + s), ks * kCeK,
                                    vb * kCeN);
                    }
                    __syncwarp();
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        const uint32_t idesc = make_idesc_bf16(kCeM, kCeN, 0);
        uint32_t it = 0, blk = 0;
        bool ok = true;
#pragma unroll 1
        for (int tl = 0; tl < n_units && ok; ++tl) {
            const int u = (int)blockIdx.x + tl * (int)gridDim.x;
            int pn, rt;
            ce_unit(p, u, pn, rt);
            const int vb_end = min(p.nvb, (pn + 1) * kCePanel);
#pragma unroll 1
            for (int vb = pn * kCePanel; vb < vb_end && ok; ++vb, ++blk) {
                const uint32_t a = blk & 1u;
                // the accumulator half is free once the fold warps have read block blk - 2 out of it
                ok = mbar_wait_warp(bar(kCeBarAccFree + a), ((blk >> 1) & 1) ^ 1, abort_flag, p.status, kErrCeMma);
                if (!ok) break;
                tc_fence_after();
#pragma unroll 1
                for (int ks = 0; ks < p.ksteps; ++ks, ++it) {
                    const uint32_t s = it % kCeStages;
                    ok = mbar_wait_warp(bar(kCeBarFull + s), (it / kCeStages) & 1, abort_flag, p.status, kErrCeMma);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t a_desc = make_smem_desc(sbase + s * kCeStageBytes, 0, 1024);
                    const uint64_t b_desc = make_smem_desc(sbase + s * kCeStageBytes + kCeABytes, 0, 1024);
                    if (elect_one_sync()) {
#pragma unroll
                        for (int kk = 0; kk < kCeK / 16; ++kk)
                            mma_ss(tmem + a * kCeN, a_desc + (uint64_t)((kk * 32) >> 4), b_desc + (uint64_t)((kk * 32) >> 4),
                                   idesc, (ks > 0 || kk > 0) ? 1u : 0u);
                        tc_commit(bar(kCeBarEmpty + s));
                        if (ks == p.ksteps - 1) tc_commit(bar(kCeBarAccFull + a));
                    }
                    __syncwarp();
                }
            }
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ fold warps (4..7)
        const int q4 = warp & 3;
        const int row = 32 * q4 + lane;
        const uint32_t lane_addr = (uint32_t)(32 * q4) << 16;
        uint32_t blk = 0;
        bool ok = true;
#pragma unroll 1
        for (int tl = 0; tl < n_units && ok; ++tl) {
            const int u = (int)blockIdx.x + tl * (int)gridDim.x;
            int pn, rt;
            ce_unit(p, u, pn, rt);
            const int vb_end = min(p.nvb, (pn + 1) * kCePanel);
            const int grow = rt * kCeM + row;
            const bool valid = grow < p.R;
            const int z = valid ? p.target[grow] : -1;
            float m = -INFINITY, l = 0.f, zt = 0.f;  // running max and sum in the log2 domain
            bool have_zt = false;
#pragma unroll 1
            for (int vb = pn * kCePanel; vb < vb_end && ok; ++vb, ++blk) {
                const uint32_t a = blk & 1u;
                ok = mbar_wait_warp(bar(kCeBarAccFull + a), (blk >> 1) & 1, abort_flag, p.status, kErrCeFold);
                if (!ok) break;
                tc_fence_after();
                const int col0 = vb * kCeN;
                const int ncol = min(kCeN, p.V - col0);  // real vocabulary entries in this block
#pragma unroll 1
                for (int c = 0; c < kCeN / 32; ++c) {
                    if (c * 32 >= ncol) break;  // warp-uniform: nothing real in the remaining chunks
                    uint32_t rr[32];
                    tmem_ld32(tmem + lane_addr + a * kCeN + c * 32, rr);
                    tmem_wait_ld();
                    const int zrel = z - col0 - c * 32;
                    if (__any_sync(0xffffffffu, (unsigned)zrel < 32u)) {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (zrel == i) { zt = __uint_as_float(rr[i]); have_zt = true; }
                    }
                    float y[32];
                    float cmax = -INFINITY;
                    const int nreal = ncol - c * 32;  // >= 1
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        y[i] = i < nreal ? __uint_as_float(rr[i]) * kLog2e : -INFINITY;
                        cmax = fmaxf(cmax, y[i]);
                    }
                    if (cmax > m) {
                        l *= ex2_approx(m - cmax);  // 2^-inf = 0 on the first chunk
                        m = cmax;
                    }
                    float s0 = 0.f, s1 = 0.f;
#pragma unroll
                    for (int i = 0; i < 32; i += 2) {
                        s0 += ex2_approx(y[i] - m);
                        s1 += ex2_approx(y[i + 1] - m);
                    }
                    l += s0 + s1;
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kCeBarAccFree + a));
            }
            if (ok && valid) {
                p.part_m[(size_t)pn * p.Rpad + grow] = m;
                p.part_l[(size_t)pn * p.Rpad + grow] = l;
                if (have_zt) p.tlogit[grow] = zt;
            }
        }
    }

    if (*abort_flag != 0) __nanosleep(20000);
    tc_fence_before();
    __syncthreads();
    if (warp == 2) tmem_dealloc(tmem, 512);
}

// Merges the partials of every row: one thread per row (consecutive threads read consecutive
// addresses of every panel's partial arrays), lse and nll per row.
__global__ void __launch_bounds__(256)
ce_rows_kernel(const float *part_m, const float *part_l, const float *tlogit, const int *target, const float *mask,
               float *nll, float *lse, long long R, int Rpad, int npanel, int V)
{
    const long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= R) return;
    float M = -INFINITY;
    for (int pn = 0; pn < npanel; ++pn) M = fmaxf(M, part_m[(size_t)pn * Rpad + r]);
    float L = 0.f;
    for (int pn = 0; pn < npanel; ++pn) L += part_l[(size_t)pn * Rpad + r] * exp2f(part_m[(size_t)pn * Rpad + r] - M);
    const float ls = (M + log2f(L)) * kLn2;
    lse[r] = ls;
    const float w = mask[r];
    float v = 0.f;
    if (w != 0.f) {
        const int z = target[r];
        v = (z >= 0 && z < V) ? w * (ls - tlogit[r]) : __int_as_float(0x7fc00000);  // a bad token id shows as NaN
    }
    nll[r] = v;
}

// Masked average per candidate: one warp per candidate.
__global__ void __launch_bounds__(256)
ce_finalize_kernel(const float *nll, const float *mask, float *loss, int N, int Lr)
{
    const int warp = (int)((blockIdx.x * (unsigned)blockDim.x + threadIdx.x) >> 5), lane = threadIdx.x & 31;
    if (warp >= N) return;
    float num = 0.f, den = 0.f;
    for (int i = lane; i < Lr; i += 32) {
        const size_t r = (size_t)warp * Lr + i;
        num += nll[r];
        den += mask[r];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        num += __shfl_xor_sync(0xffffffffu, num, o);
        den += __shfl_xor_sync(0xffffffffu, den, o);
    }
    if (lane == 0) loss[warp] = den != 0.f ? num / den : 0.f;
}

inline bool encode_2d(CUtensorMap *map, const void *base, int cols, long long rows, int box_rows)
{
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t str[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    return encode_map(map, base, 2, dims, str, box);
}

struct CePlan {
    int nrt, nvb, npanel, Rpad, ksteps;
    size_t part_bytes, ws_bytes;
};

CePlan ce_plan(long long R, int Dm, int V)
{
    CePlan pl;
    pl.nrt = (int)((R + kCeM - 1) / kCeM);
    pl.nvb = (V + kCeN - 1) / kCeN;
    pl.npanel = (pl.nvb + kCePanel - 1) / kCePanel;
    pl.Rpad = pl.nrt * kCeM;
    pl.ksteps = (Dm + kCeK - 1) / kCeK;
    pl.part_bytes = (size_t)pl.npanel * pl.Rpad * sizeof(float);
    pl.ws_bytes = 2 * pl.part_bytes + (size_t)pl.Rpad * sizeof(float);
    return pl;
}

}  // namespace

bool ce_fwd_supported(int N, int Lr, int Dm, int V)
{
    if (N < 1 || Lr < 1 || Dm < 8 || V < 1 || Dm % 8 != 0) return false;  // row pitch must be a multiple of 16 bytes
    const long long R = (long long)N * Lr;
    if (R > 16000000ll || (long long)V > 4000000ll) return false;
    const CePlan pl = ce_plan(R, Dm, V);
    return (long long)pl.npanel * pl.nrt < 2000000000ll;
}

size_t ce_fwd_workspace_bytes(int N, int Lr, int Dm, int V)
{
    return ce_plan((long long)N * Lr, Dm, V).ws_bytes;
}

cudaError_t launch_ce_fwd(const CeArgs &a, void *workspace, unsigned int *status_word, cudaStream_t stream)
{
    const long long R = (long long)a.N * a.Lr;
    const CePlan pl = ce_plan(R, a.Dm, a.V);
    CUtensorMap tm_h, tm_w;
    if (!encode_2d(&tm_h, a.hidden, a.Dm, R, kCeM)) return cudaErrorInvalidValue;
    if (!encode_2d(&tm_w, a.weight, a.Dm, a.V, kCeN)) return cudaErrorInvalidValue;
    CeParams p;
    p.target = a.target;
    p.part_m = static_cast<float *>(workspace);
    p.part_l = p.part_m + (size_t)pl.npanel * pl.Rpad;
    p.tlogit = p.part_l + (size_t)pl.npanel * pl.Rpad;
    p.status = status_word;
    p.R = (int)R; p.Rpad = pl.Rpad; p.Dm = a.Dm; p.V = a.V;
    p.nrt = pl.nrt; p.nvb = pl.nvb; p.npanel = pl.npanel; p.units = pl.npanel * pl.nrt; p.ksteps = pl.ksteps;
    p.rg = sm_count() / 4 < 1 ? 1 : sm_count() / 4;
    if (p.rg > pl.nrt) p.rg = pl.nrt;
    const int smem_bytes = kCeStages * kCeStageBytes + 8 * kCeNumBars + 64;
    static PerDeviceOnce attr_set;
    if (cudaError_t e = ensure_max_smem(ce_fwd_kernel, attr_set, smem_bytes); e != cudaSuccess) return e;
    const int grid = p.units < sm_count() ? p.units : sm_count();
    {
        KernelTiming timing(kKernelCeFwd, stream);
        ce_fwd_kernel<<<grid, kCeThreads, smem_bytes, stream>>>(tm_h, tm_w, p);
    }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    {
        KernelTiming timing(kKernelCeFinalize, stream);
        ce_rows_kernel<<<(unsigned)((R + 255) / 256), 256, 0, stream>>>(p.part_m, p.part_l, p.tlogit, a.target, a.mask, a.nll,
                                                                       a.lse, R, pl.Rpad, pl.npanel, a.V);
        const int warps_per_block = 8;
        ce_finalize_kernel<<<(a.N + warps_per_block - 1) / warps_per_block, warps_per_block * 32, 0, stream>>>(
            a.nll, a.mask, a.loss, a.N, a.Lr);
    }
    count_launches(3);
    return cudaGetLastError();
}

}  // namespace pskv
