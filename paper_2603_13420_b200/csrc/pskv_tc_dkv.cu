// Suffix-side gradients dK_suffix, dV_suffix on the tcgen05 tensor cores (head dim 128, S <= 64):
//   dV[b,g,t,:] = sum over heads h of g, rows i >= t of  P[b,h,i,t] dO[b,h,i,:]
//   dK[b,g,t,:] = scale * sum over the same (h, i) of     dS[b,h,i,t] Q[b,h,i,:]
// with P = exp(scale q.k - lse) on the suffix keys only and dS = P (dO.v - D): the block-diagonal
// part of the backward of Eq. 2 (the prefix cache of Sec. 4.2 is frozen and gets no gradient).
//
// A unit of work is one (candidate, KV head) group: its n_rep*S query rows are contiguous and are
// taken 128 at a time.  Per 128-row tile
//   S  = Q  K_s^T  and  dP = dO V_s^T        (M = rows, N = keys, K = d; operands K-major)
//   P, dS element-wise, written to shared memory as bf16 [rows][keys]
//   dV^T += dO^T P  and  dK^T += Q^T dS      (M = d, N = keys, K = rows)
// The second pair reads the very same Q / dO tiles as the first, only as operands whose M index
// (d) is the contiguous one, and P / dS as operands whose N index (keys) is contiguous: no
// transposed copy of anything is made.  The accumulators hold the transposed gradients
// (lane = d, column = key) and stay in tensor memory across the tiles of a group, so the sum over
// the heads of a group needs no atomics and the result is deterministic.
//
// Persistent CTAs, one per SM, each walking over its groups; 20 warps:
//   warp 0      TMA producer (Q and dO tiles, two stages; suffix K / V of a group, two stages)
//   warp 1      tcgen05.mma issuer, score side (owns the tensor-memory allocation)
//   warp 2      tcgen05.mma issuer, gradient side
//   warps 4-19  element-wise stage, four warpgroups taking one 16-key piece each (thread <->
//               query row) and, at the end of a group, the write-back of the two accumulators
// The arithmetic is tiny next to the bytes moved (Q and dO are read once, nothing else is big):
// the kernel is bound by HBM, and everything is arranged to keep two tiles of copies in flight.
//
// Because it streams every dO row anyway and has issue slots to spare, the kernel (instantiated with
// DROW = true) also forms the row statistic of the backward pass, D = <dO, O> (minus the gradient
// arriving on lse, if any), instead of a pre-pass that would read dO a second time: the element-wise
// warps read the O rows of the tile straight from global memory (32 of the 128 columns per warpgroup),
// meet the dO tile in shared memory, exchange their four partial sums through shared memory and write
// D for the query-side kernel, which runs behind this one.
//
// The same kernel, instantiated with PRE = true, produces the gradients of the shared PREFIX cache
// (which the search keeps frozen, Sec. 4.2, but a caller may want: full differentiability).  A unit
// of work is then (KV head, block of 64 prefix keys, chunk of candidates): the block's K/V rows are
// the operands, every key of the block is visible to every row, the row tiles of all candidates of
// the chunk accumulate into the same transposed accumulators, and the write-back adds them into an
// fp32 array in global memory (the chunks of one block meet there), which a small kernel rounds to
// bf16 afterwards.  The key blocks of one (head, chunk) are numbered consecutively, so the CTAs
// that re-read the same Q / dO rows run together and find them in L2.
#include <string.h>

#include "pskv_common.cuh"
#include "pskv_sm100.cuh"
#include "pskv_tc_common.cuh"

namespace pskv {
namespace {

using namespace sm100;

constexpr int kElemGroups = 4;  // element-wise warpgroups: one 16-key piece of every tile each
constexpr int kThreads = 32 * (4 + 4 * kElemGroups);
constexpr int kD = 128;
constexpr int kSlabBytes = kTileM * 128;       // 128 rows x 64 columns of bf16
constexpr int kTileBytes = 2 * kSlabBytes;     // a 128 x 128 tile: two 64-column slabs
// tensor-memory columns: two (S, dP) slots, then the two accumulators
// two sets of accumulators (a group's write-back overlaps the next group's MMAs)
constexpr int kColS = 0, kColDp = 64, kSlotCols = 128, kColAcc = 256, kAccCols = 128, kColDv = 0, kColDk = 64;
constexpr int kTmemCols = 512;

enum : unsigned int {
    kErrDkvProducer = 0x301, kErrDkvMma = 0x302, kErrDkvElem = 0x303, kErrDkvAlign = 0x304
};

enum {
    kBarQFull = 0,       // [2] Q and dO of a tile landed
    kBarStageFree = 2,   // [2] the second MMA pair of the tile that used the stage completed
    kBarKvFull = 4,      // [2] suffix K / V of a group landed
    kBarKvFree = 6,      // [2] every MMA of the group that used them completed
    kBarSFull = 8,       // [2] S and dP of a tile are in tensor memory
    kBarSFree = 10,      // [2] the element-wise warps have read them out (4 arrivals)
    kBarPReady = 12,     // P and dS of a tile are in shared memory (4 arrivals)
    kBarPFree = 13,      // the MMAs that read them completed
    kBarAccFull = 14,    // [2] the accumulators of a group are final
    kBarAccFree = 16,    // [2] the write-back has read them out (one arrival per element-wise warp)
    kBarDFull = 18,      // [2] DROW: the four partial sums of D of a tile are in shared memory (16 arrivals)
    kNumBars = 20
};

struct TcDkvParams {
    const float *lse;      // [B*Hq*S]
    const float *row_dot;  // [B*Hq*S] D per row (read; DROW: written here by this kernel, never read)
    float *row_dot_out;    // DROW: where D goes for the query-side kernel
    const __nv_bfloat16 *out;  // DROW: [B,Hq,S,128] forward output
    const float *dlse;     // DROW: gradient arriving on lse, or nullptr
    __nv_bfloat16 *dk;     // [B,Hkv,S,128]
    __nv_bfloat16 *dv;
    unsigned int *status;
    float sl2, scale;
    int B, Hq, Hkv, S, n_rep, Rg;
    int TP;                // S rounded up to 16: the N of every MMA
    int ntile;             // 128-row tiles per (candidate, KV head)
    int total_groups;      // B * Hkv; prefix mode: Hkv * nbc * nkb
    // prefix mode
    float *dkp32, *dvp32;  // [Hkv][P][128] fp32 accumulators in global memory (zeroed before the launch)
    int P, nkb, nbc, cpc;  // prefix length, key blocks of 64, candidate chunks, candidates per chunk
    FastDiv fd_S, fd_Hkv;
    // shared-memory byte offsets from the 1024-byte aligned base
    int off_q, off_do, off_k, off_v, off_p, off_ds, off_bar, off_misc, off_dpart, kv_bytes;
};

// Warp-level MMA (16 x 8 x 16, bf16 in, fp32 accumulate): used only to form the row statistic D, whose dot
// products over the columns of a row are a diagonal of dO O^T.
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                               uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// unit u of a CTA -> (index of the group within this CTA, tile within the group)
struct Unit {
    int gi, tt, bg, b, g, kb;
    bool first, last;
};
template <bool PRE>
__device__ __forceinline__ Unit unit_of(const TcDkvParams &p, int u)
{
    Unit x;
    if (PRE) {
        // group = (KV head, candidate chunk, key block), key block fastest; cpc * ntile units each
        const int upg = p.cpc * p.ntile;
        x.gi = u / upg;
        const int w = u - x.gi * upg;
        const int cb = w / p.ntile;
        x.tt = w - cb * p.ntile;
        x.bg = blockIdx.x + x.gi * gridDim.x;
        const int rest = x.bg / p.nkb;
        x.kb = x.bg - rest * p.nkb;
        x.g = rest / p.nbc;
        x.b = (rest - x.g * p.nbc) * p.cpc + cb;  // may be >= B in the last chunk: such tiles read as zero
        x.first = w == 0;
        x.last = w == upg - 1;
    } else {
        x.gi = u / p.ntile;
        x.tt = u - x.gi * p.ntile;
        x.bg = blockIdx.x + x.gi * gridDim.x;
        x.b = p.fd_Hkv.div(x.bg);
        x.g = x.bg - x.b * p.Hkv;
        x.kb = 0;
        x.first = x.tt == 0;
        x.last = x.tt == p.ntile - 1;
    }
    return x;
}

// NP = TP / 16: 16-key pieces per row.  PRE: prefix-gradient mode (NP = 4).  DROW: form D = <dO, O>
// here and write it out (never together with PRE).
template <int NP, bool PRE, bool DROW = false>
__global__ void __launch_bounds__(kThreads, 1)
tc_bwd_dkv_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_do,
                  const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                  const __grid_constant__ CUtensorMap tm_o, const TcDkvParams p)
{
    constexpr int TP = NP * 16;
    extern __shared__ __align__(1024) uint8_t smem[];
    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);  // warp-uniform by construction
    PSKV_TRACE_DECL;
    grid_dep_launch();  // the next kernel of the stream may take over SMs as this one's CTAs exit
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + p.off_bar;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + p.off_misc + 4);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + p.off_misc);

    if ((sbase & 1023u) != 0u) {  // the swizzled layouts need a 1024-byte aligned base
        if (tid == 0) atomicCAS(p.status, 0u, (unsigned int)kErrDkvAlign);
        return;
    }
    // rows that no copy ever writes (tile padding, keys past S) must read as zero
    for (int i = tid; i < p.off_bar / 16; i += kThreads) reinterpret_cast<uint4 *>(smem)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
#pragma unroll 1
        for (int i = 0; i < kNumBars; ++i) {
            const bool elem = i == kBarSFree || i == kBarSFree + 1 || i == kBarPReady || i == kBarAccFree ||
                              i == kBarAccFree + 1 || i == kBarDFull || i == kBarDFull + 1;
            mbar_init(bar(i), elem ? (uint32_t)(4 * kElemGroups) : 1u);
        }
        *abort_flag = 0;
        fence_barrier_init();
    }
    fence_proxy_async();
    __syncthreads();
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    // everything above touched shared and tensor memory only: it may run under the tail of the kernel before
    grid_dep_wait();

    const int my_groups = (int)blockIdx.x < p.total_groups ? (p.total_groups - 1 - (int)blockIdx.x) / (int)gridDim.x + 1 : 0;
    const int total_units = my_groups * (PRE ? p.cpc * p.ntile : p.ntile);
    const int box_rows = p.Rg < kTileM ? p.Rg : kTileM;  // rows one Q / dO copy brings (rows past Rg read as zero)
    const uint32_t tile_tx = (uint32_t)(2 * 2 * box_rows * 128);
    const uint32_t kv_tx = PRE ? (uint32_t)(2 * 2 * 64 * 128) : (uint32_t)(2 * 2 * p.S * 128);  // (a full box, zero-filled past P)
    const int kv_slab = TP * 128;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            prefetch_tensormap(&tm_q);
            prefetch_tensormap(&tm_do);
            prefetch_tensormap(&tm_k);
            prefetch_tensormap(&tm_v);
        }
        bool ok = true;
#pragma unroll 1
        for (int u = 0; u < total_units && ok; ++u) {
            const Unit x = unit_of<PRE>(p, u);
            const int st = u & 1;
            if (x.first) {
                const int ks = x.gi & 1;
                ok = mbar_wait_warp(bar(kBarKvFree + ks), ((x.gi >> 1) & 1) ^ 1, abort_flag, p.status, kErrDkvProducer);
                if (!ok) break;
                if (elect_one_sync()) {
                    mbar_arrive_expect_tx(bar(kBarKvFull + ks), kv_tx);
#pragma unroll
                    for (int sl = 0; sl < 2; ++sl) {
                        if (PRE) {
                            tma_load_3d(sbase + p.off_k + ks * p.kv_bytes + sl * kv_slab, &tm_k, bar(kBarKvFull + ks),
                                        sl * 64, x.kb * 64, x.g);
                            tma_load_3d(sbase + p.off_v + ks * p.kv_bytes + sl * kv_slab, &tm_v, bar(kBarKvFull + ks),
                                        sl * 64, x.kb * 64, x.g);
                        } else {
                            tma_load_4d(sbase + p.off_k + ks * p.kv_bytes + sl * kv_slab, &tm_k, bar(kBarKvFull + ks),
                                        sl * 64, 0, x.g, x.b);
                            tma_load_4d(sbase + p.off_v + ks * p.kv_bytes + sl * kv_slab, &tm_v, bar(kBarKvFull + ks),
                                        sl * 64, 0, x.g, x.b);
                        }
                    }
                }
                __syncwarp();
            }
            // the copies of unit u + 2 can only be issued when this stage is free again: ask for
            // its rows in L2 now, so that they are close by then
            if (u + 2 < total_units) {
                const Unit y = unit_of<PRE>(p, u + 2);
                if (elect_one_sync()) {
#pragma unroll
                    for (int sl = 0; sl < 2; ++sl) {
                        tma_prefetch_4d(&tm_q, sl * 64, y.tt * kTileM, y.g, y.b);
                        tma_prefetch_4d(&tm_do, sl * 64, y.tt * kTileM, y.g, y.b);
                        if (DROW) tma_prefetch_4d(&tm_o, sl * 64, y.tt * kTileM, y.g, y.b);  // read by the element-wise warps
                        if (y.first && !PRE) {
                            tma_prefetch_4d(&tm_k, sl * 64, 0, y.g, y.b);
                            tma_prefetch_4d(&tm_v, sl * 64, 0, y.g, y.b);
                        }
                    }
                }
                __syncwarp();
            }
            ok = mbar_wait_warp(bar(kBarStageFree + st), ((u >> 1) & 1) ^ 1, abort_flag, p.status, kErrDkvProducer);
            if (!ok) break;
            PSKV_TRACE_EVENT(1, u);
            if (elect_one_sync()) {
                mbar_arrive_expect_tx(bar(kBarQFull + st), tile_tx);
#pragma unroll
                for (int sl = 0; sl < 2; ++sl) {
                    tma_load_4d(sbase + p.off_q + st * kTileBytes + sl * kSlabBytes, &tm_q, bar(kBarQFull + st), sl * 64,
                                x.tt * kTileM, x.g, x.b);
                    tma_load_4d(sbase + p.off_do + st * kTileBytes + sl * kSlabBytes, &tm_do, bar(kBarQFull + st), sl * 64,
                                x.tt * kTileM, x.g, x.b);
                }
            }
            __syncwarp();
        }
    } else if (warp == 1 || warp == 2) {
        // ------------------------------------------------------------------ MMA issuers
        const uint32_t idesc1 = make_idesc_bf16_ab(kTileM, TP, 0, 0);
        const uint32_t idesc2 = make_idesc_bf16_ab(kD, TP, 1, 1);
        bool ok = true;
        // score side of unit u: S = Q K_s^T, dP = dO V_s^T
        auto score_pair = [&](int u) -> bool {
            const Unit x = unit_of<PRE>(p, u);
            const int st = u & 1, ks = x.gi & 1;
            if (!mbar_wait_warp(bar(kBarQFull + st), (u >> 1) & 1, abort_flag, p.status, kErrDkvMma)) return false;
            if (x.first && !mbar_wait_warp(bar(kBarKvFull + ks), (x.gi >> 1) & 1, abort_flag, p.status, kErrDkvMma))
                return false;
            if (!mbar_wait_warp(bar(kBarSFree + st), ((u >> 1) & 1) ^ 1, abort_flag, p.status, kErrDkvMma)) return false;
            PSKV_TRACE_EVENT(10, u);
            tc_fence_after();
            const uint64_t q_desc = make_smem_desc(sbase + p.off_q + st * kTileBytes, 0, 1024);
            const uint64_t do_desc = make_smem_desc(sbase + p.off_do + st * kTileBytes, 0, 1024);
            const uint64_t k_desc = make_smem_desc(sbase + p.off_k + ks * p.kv_bytes, 0, 1024);
            const uint64_t v_desc = make_smem_desc(sbase + p.off_v + ks * p.kv_bytes, 0, 1024);
            const uint32_t s_tmem = tmem + st * kSlotCols;
            if (elect_one_sync()) {
#pragma unroll
                for (int ks16 = 0; ks16 < kD / 16; ++ks16) {
                    const uint64_t aoff = (uint64_t)(((ks16 >> 2) * kSlabBytes + (ks16 & 3) * 32) >> 4);
                    const uint64_t boff = (uint64_t)(((ks16 >> 2) * kv_slab + (ks16 & 3) * 32) >> 4);
                    mma_ss(s_tmem + kColS, q_desc + aoff, k_desc + boff, idesc1, ks16 > 0 ? 1u : 0u);
                    mma_ss(s_tmem + kColDp, do_desc + aoff, v_desc + boff, idesc1, ks16 > 0 ? 1u : 0u);
                }
                tc_commit(bar(kBarSFull + st));
            }
            __syncwarp();
            return true;
        };
        // gradient side of unit v: dV^T += dO^T P, dK^T += Q^T dS
        auto grad_pair = [&](int v) -> bool {
            const Unit x = unit_of<PRE>(p, v);
            const int st = v & 1, ks = x.gi & 1, as = x.gi & 1;
            if (!mbar_wait_warp(bar(kBarPReady), v & 1, abort_flag, p.status, kErrDkvMma)) return false;
            // the accumulator set must have been written back by the group that used it before
            if (x.first && !mbar_wait_warp(bar(kBarAccFree + as), ((x.gi >> 1) & 1) ^ 1, abort_flag, p.status, kErrDkvMma))
                return false;
            PSKV_TRACE_EVENT(11, v);
            tc_fence_after();
            // operands with the M index (d) / N index (key) contiguous: 64-element groups a slab apart
            const uint64_t qt_desc = make_smem_desc(sbase + p.off_q + st * kTileBytes, kSlabBytes, 1024);
            const uint64_t dot_desc = make_smem_desc(sbase + p.off_do + st * kTileBytes, kSlabBytes, 1024);
            const uint64_t p_desc = make_smem_desc(sbase + p.off_p, kSlabBytes, 1024);
            const uint64_t ds_desc = make_smem_desc(sbase + p.off_ds, kSlabBytes, 1024);
            const int rows = min(kTileM, p.Rg - x.tt * kTileM);
            const int nks = (rows + 15) >> 4;  // rows past `rows` are zero in every operand
            const uint32_t acc0 = x.first ? 0u : 1u;
            const uint32_t acc = tmem + kColAcc + as * kAccCols;
            if (elect_one_sync()) {
#pragma unroll
                for (int ks16 = 0; ks16 < kTileM / 16; ++ks16) {
                    if (ks16 < nks) {
                        const uint64_t off = (uint64_t)((ks16 * 2048) >> 4);
                        mma_ss(acc + kColDv, dot_desc + off, p_desc + off, idesc2, ks16 > 0 ? 1u : acc0);
                        mma_ss(acc + kColDk, qt_desc + off, ds_desc + off, idesc2, ks16 > 0 ? 1u : acc0);
                    }
                }
                tc_commit(bar(kBarPFree));
                tc_commit(bar(kBarStageFree + st));
                if (x.last) {
                    tc_commit(bar(kBarAccFull + as));
                    tc_commit(bar(kBarKvFree + ks));
                }
            }
            __syncwarp();
            return true;
        };
        // warp 1 issues the score side of every unit, warp 2 the gradient side: the two streams
        // only meet through the element-wise warps, and two issuing threads keep the tensor pipe
        // fed where one could not
        if (warp == 1) {
#pragma unroll 1
            for (int u = 0; u < total_units && ok; ++u) ok = score_pair(u);
        } else {
#pragma unroll 1
            for (int u = 0; u < total_units && ok; ++u) ok = grad_pair(u);
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------------ element-wise warps, write-back
        const int row = 32 * (warp & 3) + lane;  // query row of the tile; lane of tensor memory
        const int wg = (warp - 4) >> 2;
        const uint32_t lane_addr = (uint32_t)(32 * (warp & 3)) << 16;
        uint8_t *p_row = smem + p.off_p + row * 128;
        uint8_t *ds_row = smem + p.off_ds + row * 128;
        bool ok = true;
        int pending_gi = -1;  // group whose accumulators are still to be written back
        float *dpart = reinterpret_cast<float *>(smem + p.off_dpart);  // DROW: [stage][warpgroup][row]
        uint4 o_next[4] = {};                                            // DROW: this thread's O slice of the coming unit
        // DROW: the O rows of a unit are read four lanes to a row -- lane 4k+c takes the 16-byte chunk c of this
        // warpgroup's 32 columns of rows 8j+k (j = 0..3) of the warp's 32 rows -- so that a load instruction
        // covers eight 64-byte runs of full sectors instead of 32 half-used ones.
        const int orow_k = lane >> 2, ochunk = lane & 3;
        auto load_o = [&](const Unit &y) {
            const int base = y.tt * kTileM + 32 * (warp & 3);
            const __nv_bfloat16 *o0 = p.out + (((size_t)y.b * p.Hq + (size_t)y.g * p.n_rep) * p.S) * kD + 32 * wg + 8 * ochunk;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int gy = base + 8 * j + orow_k;
                o_next[j] = gy < p.Rg ? __ldg(reinterpret_cast<const uint4 *>(o0 + (size_t)gy * kD)) : make_uint4(0, 0, 0, 0);
            }
        };
        if (DROW && total_units > 0) load_o(unit_of<PRE>(p, 0));
        // write-back of group gi: lane <-> column d, tensor-memory column <-> key
        auto write_back = [&](int gi) -> bool {
            const int as = gi & 1;
            if (!mbar_wait_warp(bar(kBarAccFull + as), (gi >> 1) & 1, abort_flag, p.status, kErrDkvElem)) return false;
            PSKV_TRACE_EVENT(30, gi);
            tc_fence_after();
            const int bg = blockIdx.x + gi * gridDim.x;
            __nv_bfloat16 *dvg = p.dv + (size_t)bg * p.S * kD + row;
            __nv_bfloat16 *dkg = p.dk + (size_t)bg * p.S * kD + row;
            // prefix mode: key block and KV head of the group, keys of the block that exist
            const int rest = PRE ? bg / p.nkb : 0;
            const int kb = bg - rest * p.nkb, gh = PRE ? rest / p.nbc : 0;
            const int nkeys = PRE ? min(64, p.P - kb * 64) : 0;
            if (wg < NP) {
                uint32_t av[16], ak[16];
                const uint32_t acc = tmem + lane_addr + kColAcc + as * kAccCols;
                tmem_ld16(acc + kColDv + wg * 16, av);
                tmem_ld16(acc + kColDk + wg * 16, ak);
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarAccFree + as));
                if (PRE) {
                    // the candidate chunks of a key block meet in global memory: lane <-> d, coalesced adds
                    float *av32 = p.dvp32 + ((size_t)gh * p.P + (size_t)kb * 64) * kD + row;
                    float *ak32 = p.dkp32 + ((size_t)gh * p.P + (size_t)kb * 64) * kD + row;
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        const int t = wg * 16 + c;
                        if (t < nkeys) {
                            atomicAdd(av32 + (size_t)t * kD, __uint_as_float(av[c]));
                            atomicAdd(ak32 + (size_t)t * kD, __uint_as_float(ak[c]) * p.scale);
                        }
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 16; ++c) {
                        const int t = wg * 16 + c;
                        if (t < p.S) {
                            dvg[(size_t)t * kD] = __float2bfloat16_rn(__uint_as_float(av[c]));
                            dkg[(size_t)t * kD] = __float2bfloat16_rn(__uint_as_float(ak[c]) * p.scale);
                        }
                    }
                }
            } else {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarAccFree + as));
            }
            PSKV_TRACE_EVENT(31, gi);
            return true;
        };
        // The next unit is worked out once, and the two per-row statistics of my row in it (lse, D) are asked for
        // a unit ahead, before the write-back, so that their latency lies under it (about 1 % at 192-row groups).
        Unit x_next = unit_of<PRE>(p, 0);
        float lse_next = 0.f, dr_next = 0.f;
        auto load_stats = [&](const Unit &y) {
            const int gy = y.tt * kTileM + row;
            const bool v = gy < p.Rg && (!PRE || y.b < p.B);
            const size_t r0 = ((size_t)y.b * p.Hq + (size_t)y.g * p.n_rep) * p.S;
            lse_next = v ? p.lse[r0 + gy] : 0.f;
            dr_next = (!DROW && v) ? p.row_dot[r0 + gy] : 0.f;
        };
        if (total_units > 0) load_stats(x_next);
#pragma unroll 1
        for (int u = 0; u < total_units && ok; ++u) {
            const Unit x = x_next;
            const int st = u & 1;
            const int gr = x.tt * kTileM + row;  // row inside the group: head-major, then position
            const bool valid = gr < p.Rg && (!PRE || x.b < p.B);
            const size_t row0 = ((size_t)x.b * p.Hq + (size_t)x.g * p.n_rep) * p.S;
            // causal: suffix key t is visible when t <= i; prefix mode: every key of the block that exists
            const int i_pos = !valid ? -1 : PRE ? min(64, p.P - x.kb * 64) - 1 : gr - p.fd_S.div(gr) * p.S;
            const float nl2 = -lse_next * kLog2e;
            float dr = dr_next;
            if (!DROW && u + 1 < total_units) x_next = unit_of<PRE>(p, u + 1);
            if (DROW) {
                // my 32 of the row's 128 columns: O from global memory (requested one unit ahead), dO from the
                // tile in shared memory (64-column slabs of 128-byte rows, 16-byte chunks swizzled by the row)
                ok = mbar_wait_warp(bar(kBarQFull + st), (u >> 1) & 1, abort_flag, p.status, kErrDkvElem);
                if (!ok) break;
                // <dO, O> over my 32 columns for the warp's 32 rows, on the warp-level tensor-core path: for a group
                // of 16 rows, dO (16 x 16 columns) times the transpose of 8 rows of O gives a 16 x 8 block of
                // dO O^T whose diagonal holds 8 of the wanted sums; two such products per 16 rows, two 16-column
                // slices each.  (Conversions and FMAs on the CUDA cores took these warps 1 000 cycles a unit.)
                // The k index is permuted the same way on both sides, which a dot product does not mind: lane
                // 4g+c holds columns 8c..8c+7 of a row, and slice s takes 8c+4s..8c+4s+3 as its k = 2c, 2c+1, 2c+8,
                // 2c+9 -- so a lane's 16-byte chunk of O is its B fragment of both slices as it stands.
                const uint8_t *dotile = smem + p.off_do + st * kTileBytes + (wg >> 1) * kSlabBytes;
                const int g = orow_k, c = ochunk;
#pragma unroll
                for (int G = 0; G < 2; ++G) {
                    const int r_lo = 32 * (warp & 3) + 16 * G + g, r_hi = r_lo + 8;
                    const uint4 alo = *reinterpret_cast<const uint4 *>(dotile + r_lo * 128 + ((((wg & 1) * 4 + c) ^ (r_lo & 7)) << 4));
                    const uint4 ahi = *reinterpret_cast<const uint4 *>(dotile + r_hi * 128 + ((((wg & 1) * 4 + c) ^ (r_hi & 7)) << 4));
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const uint4 b = o_next[2 * G + h];  // O rows 16 G + 8 h + (0..7) of the warp's 32
                        float acc[4] = {0.f, 0.f, 0.f, 0.f};
                        mma_bf16_16816(acc, alo.x, ahi.x, alo.y, ahi.y, b.x, b.y);
                        mma_bf16_16816(acc, alo.z, ahi.z, alo.w, ahi.w, b.z, b.w);
                        // the diagonal: row i of the 16 meets column i (h = 0) or i - 8 (h = 1); lane 4g+c holds
                        // columns 2c, 2c+1 of rows g (acc[0], acc[1]) and g+8 (acc[2], acc[3])
                        if (c == (g >> 1)) {
                            const float v = h == 0 ? ((g & 1) ? acc[1] : acc[0]) : ((g & 1) ? acc[3] : acc[2]);
                            dpart[(st * 4 + wg) * kTileM + 32 * (warp & 3) + 16 * G + 8 * h + g] = v;
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarDFull + st));
                // the O slice of the next unit, in flight while this unit is worked on
                if (u + 1 < total_units) {
                    x_next = unit_of<PRE>(p, u + 1);
                    load_o(x_next);
                }
            }
            ok = mbar_wait_warp(bar(kBarSFull + st), (u >> 1) & 1, abort_flag, p.status, kErrDkvElem);
            if (!ok) break;
            if (DROW) {
                ok = mbar_wait_warp(bar(kBarDFull + st), (u >> 1) & 1, abort_flag, p.status, kErrDkvElem);
                if (!ok) break;
                const float *dp = dpart + st * 4 * kTileM + row;  // the four warpgroups' partial sums, in fixed order
                dr = (dp[0] + dp[kTileM]) + (dp[2 * kTileM] + dp[3 * kTileM]);
                if (valid) {
                    if (p.dlse) dr -= p.dlse[row0 + gr];
                    if (wg == 0) p.row_dot_out[row0 + gr] = dr;
                }
            }
            PSKV_TRACE_EVENT(20, u);
            tc_fence_after();
            // group wg takes the 16-key piece wg of the tile (groups past the last piece only join the barriers)
            uint32_t pkp[8], pkd[8];
            if (wg < NP) {
                uint32_t rs[16], rd[16];
                tmem_ld16(tmem + lane_addr + st * kSlotCols + kColS + wg * 16, rs);
                tmem_ld16(tmem + lane_addr + st * kSlotCols + kColDp + wg * 16, rd);
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const int t0 = wg * 16 + 2 * c;
                    float x0 = __uint_as_float(rs[2 * c]), x1 = __uint_as_float(rs[2 * c + 1]);
                    fma_f32x2(x0, x1, p.sl2, nl2);
                    const float p0 = t0 <= i_pos ? ex2_approx(x0) : 0.f;
                    const float p1 = t0 + 1 <= i_pos ? ex2_approx(x1) : 0.f;
                    float d0 = __uint_as_float(rd[2 * c]), d1 = __uint_as_float(rd[2 * c + 1]);
                    add_f32x2(d0, d1, -dr, -dr);
                    mul_f32x2(d0, d1, p0, p1);
                    pkp[c] = pack_bf16x2(p0, p1);
                    pkd[c] = pack_bf16x2(d0, d1);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarSFree + st));
            // P and dS of the previous unit must have been consumed
            if (u > 0) {
                ok = mbar_wait_warp(bar(kBarPFree), (u - 1) & 1, abort_flag, p.status, kErrDkvElem);
                if (!ok) break;
            }
            // [rows][64 keys] with 128-byte rows, 16-byte chunks swizzled by the row
            if (wg < NP) {
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const int off = ((2 * wg + c) ^ (row & 7)) << 4;
                    *reinterpret_cast<uint4 *>(p_row + off) = make_uint4(pkp[4 * c], pkp[4 * c + 1], pkp[4 * c + 2], pkp[4 * c + 3]);
                    *reinterpret_cast<uint4 *>(ds_row + off) = make_uint4(pkd[4 * c], pkd[4 * c + 1], pkd[4 * c + 2], pkd[4 * c + 3]);
                }
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarPReady));
            PSKV_TRACE_EVENT(24, u);
            if (u + 1 < total_units) load_stats(x_next);
            // the write-back of a group runs one unit late, when its last MMAs have long completed
            if (pending_gi >= 0) {
                ok = write_back(pending_gi);
                pending_gi = -1;
                if (!ok) break;
            }
            if (x.last) pending_gi = x.gi;
        }
        if (ok && pending_gi >= 0) write_back(pending_gi);
    }

    PSKV_TRACE_FLUSH;
    if (*abort_flag != 0) __nanosleep(20000);  // let copies and MMAs still in flight drain
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kTmemCols);
}

// ------------------------------------------------------------------------------ host side

template <int NP, bool PRE, bool DROW = false>
cudaError_t launch_np(const BwdArgs &a, const CUtensorMap &tm_q, const CUtensorMap &tm_do, const CUtensorMap &tm_k,
                      const CUtensorMap &tm_v, const CUtensorMap &tm_o, const TcDkvParams &p, int smem_bytes,
                      cudaStream_t stream)
{
    static PerDeviceOnce attr_set;
    if (cudaError_t e = ensure_max_smem(tc_bwd_dkv_kernel<NP, PRE, DROW>, attr_set); e != cudaSuccess) return e;
    const int grid = p.total_groups < sm_count() ? p.total_groups : sm_count();
    KernelTiming timing(PRE ? kKernelBwdPrefixTc : kKernelBwdDkvTc, stream);
    const cudaError_t e = launch_dependent(tc_bwd_dkv_kernel<NP, PRE, DROW>, grid, kThreads, smem_bytes, stream, tm_q, tm_do,
                                           tm_k, tm_v, tm_o, p);
    count_launches(1);
    return e != cudaSuccess ? e : cudaGetLastError();
}

// fp32 accumulators -> bf16 results
__global__ void __launch_bounds__(256)
prefix_grad_round_kernel(const float *acc_k, const float *acc_v, __nv_bfloat16 *dk, __nv_bfloat16 *dv, size_t n)
{
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        dk[i] = __float2bfloat16_rn(acc_k[i]);
        dv[i] = __float2bfloat16_rn(acc_v[i]);
    }
}

}  // namespace

#ifdef PSKV_TRACE
// Debug builds only: copies this kernel's event trace of CTA 0 to the host.
extern "C" int pskv_debug_read_trace_dkv(long long *host, int max_events)
{
    static long long buf[kTraceWarps * kTraceCap * 2];
    unsigned int cnt[kTraceWarps];
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(cnt, g_trace_n, sizeof(cnt));
    cudaMemcpyFromSymbol(buf, g_trace, sizeof(buf));
    int n = 0;
    for (int w = 0; w < kTraceWarps; ++w)
        for (unsigned int i = 0; i < cnt[w] && i < (unsigned int)kTraceCap && n < max_events; ++i, ++n) {
            host[2 * n] = buf[((size_t)w * kTraceCap + i) * 2];
            host[2 * n + 1] = buf[((size_t)w * kTraceCap + i) * 2 + 1] | ((long long)w << 24);
        }
    return n;
}
#endif

bool tc_bwd_dkv_supported(const Dims &dm)
{
    if (dm.Skv != dm.S || dm.ragged) return false;  // full-suffix operator only
    return dm.d == kD && dm.S >= 1 && dm.S <= 64 && (long long)dm.B * dm.Hkv < 2000000000ll &&
           (long long)dm.n_rep * dm.S < 2000000000ll && get_encode_fn() != nullptr;
}

// Shared-memory bytes of the suffix-gradient launch; with_d adds the partial sums of D.
static int dkv_smem_bytes(int TP, bool with_d)
{
    const int kv_bytes = round_up(2 * TP * 128, 1024);
    return 4 * kTileBytes + 4 * kv_bytes + 2 * kSlabBytes + 256 + 64 + (with_d ? 2 * 4 * kTileM * 4 : 0);
}

// The kernel can form D for any shape it takes whose shared memory has room for the partial sums; it is
// asked to only where a (candidate, KV head) group fills whole 128-row tiles.  With small groups (one
// query head per KV head and a short suffix: 40 rows of 128) the kernel runs at a little over half of
// the HBM bandwidth, and reading O there costs more than the streaming pre-pass that reads dO twice
// (measured at B = 128, 32 heads, S = 40: 151 against 137 us for the whole backward).
bool tc_bwd_dkv_row_dot_supported(const Dims &dm)
{
    return tc_bwd_dkv_supported(dm) && dm.n_rep * dm.S >= kTileM &&
           dkv_smem_bytes((dm.S + 15) / 16 * 16, true) <= kMaxSmem;
}

cudaError_t launch_tc_bwd_dkv(const BwdArgs &a, unsigned int *status_word, cudaStream_t stream, bool with_d)
{
    const Dims &dm = a.dims;
    const int Rg = dm.n_rep * dm.S;
    const int TP = (dm.S + 15) / 16 * 16;
    if (with_d && !tc_bwd_dkv_row_dot_supported(dm)) return cudaErrorInvalidValue;

    TcDkvParams p;
    memset(&p, 0, sizeof(p));
    p.lse = a.lse;
    p.row_dot = a.row_dot;
    p.dk = a.dk_suffix;
    p.dv = a.dv_suffix;
    p.status = status_word;
    p.sl2 = a.scale * kLog2e;
    p.scale = a.scale;
    p.B = dm.B; p.Hq = dm.Hq; p.Hkv = dm.Hkv; p.S = dm.S; p.n_rep = dm.n_rep; p.Rg = Rg;
    p.TP = TP;
    p.ntile = (Rg + kTileM - 1) / kTileM;
    p.total_groups = dm.B * dm.Hkv;
    p.fd_S.init(dm.S);
    p.fd_Hkv.init(dm.Hkv);
    p.kv_bytes = round_up(2 * TP * 128, 1024);
    p.off_q = 0;
    p.off_do = p.off_q + 2 * kTileBytes;
    p.off_k = p.off_do + 2 * kTileBytes;
    p.off_v = p.off_k + 2 * p.kv_bytes;
    p.off_p = p.off_v + 2 * p.kv_bytes;
    p.off_ds = p.off_p + kSlabBytes;
    p.off_bar = p.off_ds + kSlabBytes;
    p.off_misc = p.off_bar + 256;
    p.off_dpart = p.off_misc + 64;
    const int smem_bytes = dkv_smem_bytes(TP, with_d);
    if (smem_bytes > kMaxSmem) return cudaErrorInvalidConfiguration;
    p.row_dot_out = a.row_dot;
    p.out = a.out;
    p.dlse = a.dlse;

    CUtensorMap tm_q, tm_do, tm_k, tm_v, tm_o;
    {
        // q / dout viewed as [B][Hkv][Rg][D]: the n_rep heads of a KV head are contiguous rows
        cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)Rg, (cuuint64_t)dm.Hkv, (cuuint64_t)dm.B};
        cuuint64_t str[3] = {(cuuint64_t)kD * 2, (cuuint64_t)Rg * kD * 2, (cuuint64_t)dm.Hkv * Rg * kD * 2};
        cuuint32_t box[4] = {64, (cuuint32_t)(Rg < kTileM ? Rg : kTileM), 1, 1};
        if (!encode_map(&tm_q, a.q, 4, dims, str, box)) return cudaErrorInvalidValue;
        if (!encode_map(&tm_do, a.dout, 4, dims, str, box)) return cudaErrorInvalidValue;
        if (!encode_map(&tm_o, with_d ? a.out : a.dout, 4, dims, str, box)) return cudaErrorInvalidValue;  // (L2 prefetch only)
    }
    {
        cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)dm.S, (cuuint64_t)dm.Hkv, (cuuint64_t)dm.B};
        cuuint64_t str[3] = {(cuuint64_t)kD * 2, (cuuint64_t)dm.S * kD * 2, (cuuint64_t)dm.Hkv * dm.S * kD * 2};
        cuuint32_t box[4] = {64, (cuuint32_t)dm.S, 1, 1};
        if (!encode_map(&tm_k, a.suffix_k, 4, dims, str, box)) return cudaErrorInvalidValue;
        if (!encode_map(&tm_v, a.suffix_v, 4, dims, str, box)) return cudaErrorInvalidValue;
    }
    if (with_d) {
        switch (TP / 16) {
        case 1: return launch_np<1, false, true>(a, tm_q, tm_do, tm_k, tm_v, tm_o, p, smem_bytes, stream);
        case 2: return launch_np<2, false, true>(a, tm_q, tm_do, tm_k, tm_v, tm_o, p, smem_bytes, stream);
        case 3: return launch_np<3, false, true>(a, tm_q, tm_do, tm_k, tm_v, tm_o, p, smem_bytes, stream);
        default: return launch_np<4, false, true>(a, tm_q, tm_do, tm_k, tm_v, tm_o, p, smem_bytes, stream);
        }
    }
    switch (TP / 16) {
    case 1: return launch_np<1, false>(a, tm_q, tm_do, tm_k, tm_v, tm_o, p, smem_bytes, stream);
    case 2: return launch_np<2, false>(a, tm_q, tm_do, tm_k, tm_v, tm_o, p, smem_bytes, stream);
    case 3: return launch_np<3, false>(a, tm_q, tm_do, tm_k, tm_v, tm_o, p, smem_bytes, stream);
    default: return launch_np<4, false>(a, tm_q, tm_do, tm_k, tm_v, tm_o, p, smem_bytes, stream);
    }
}

bool tc_bwd_prefix_supported(const Dims &dm)
{
    if (dm.Skv != dm.S || dm.ragged) return false;
    return dm.d == kD && dm.P >= 1 && (long long)dm.n_rep * dm.S < 2000000000ll &&
           (long long)dm.Hkv * ((dm.P + 63) / 64) * 4096ll < 2000000000ll;
}

// dk_prefix / dv_prefix [Hkv][P][128] (bf16) from a.row_dot (already computed), through `acc32`
// (2 * Hkv * P * 128 floats of scratch).
cudaError_t launch_tc_bwd_prefix(const BwdArgs &a, __nv_bfloat16 *dk_prefix, __nv_bfloat16 *dv_prefix, float *acc32,
                                 unsigned int *status_word, cudaStream_t stream)
{
    const Dims &dm = a.dims;
    const int Rg = dm.n_rep * dm.S;
    const size_t n_acc = (size_t)dm.Hkv * dm.P * kD;
    TcDkvParams p;
    memset(&p, 0, sizeof(p));
    p.lse = a.lse;
    p.row_dot = a.row_dot;
    p.status = status_word;
    p.sl2 = a.scale * kLog2e;
    p.scale = a.scale;
    p.B = dm.B; p.Hq = dm.Hq; p.Hkv = dm.Hkv; p.S = dm.S; p.n_rep = dm.n_rep; p.Rg = Rg;
    p.TP = 64;
    p.ntile = (Rg + kTileM - 1) / kTileM;
    p.P = dm.P;
    p.nkb = (dm.P + 63) / 64;
    // enough candidate chunks for about two groups per SM, so that the tail of the launch is short
    int nbc = (2 * sm_count() + dm.Hkv * p.nkb - 1) / (dm.Hkv * p.nkb);
    if (nbc > dm.B) nbc = dm.B;
    if (nbc < 1) nbc = 1;
    p.cpc = (dm.B + nbc - 1) / nbc;
    p.nbc = (dm.B + p.cpc - 1) / p.cpc;
    p.total_groups = dm.Hkv * p.nbc * p.nkb;
    p.dkp32 = acc32;
    p.dvp32 = acc32 + n_acc;
    p.fd_S.init(dm.S);
    p.fd_Hkv.init(dm.Hkv);
    p.kv_bytes = round_up(2 * 64 * 128, 1024);
    p.off_q = 0;
    p.off_do = p.off_q + 2 * kTileBytes;
    p.off_k = p.off_do + 2 * kTileBytes;
    p.off_v = p.off_k + 2 * p.kv_bytes;
    p.off_p = p.off_v + 2 * p.kv_bytes;
    p.off_ds = p.off_p + kSlabBytes;
    p.off_bar = p.off_ds + kSlabBytes;
    p.off_misc = p.off_bar + 256;
    const int smem_bytes = p.off_misc + 64;
    if (smem_bytes > kMaxSmem) return cudaErrorInvalidConfiguration;

    CUtensorMap tm_q, tm_do, tm_k, tm_v;
    {
        cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)Rg, (cuuint64_t)dm.Hkv, (cuuint64_t)dm.B};
        cuuint64_t str[3] = {(cuuint64_t)kD * 2, (cuuint64_t)Rg * kD * 2, (cuuint64_t)dm.Hkv * Rg * kD * 2};
        cuuint32_t box[4] = {64, (cuuint32_t)(Rg < kTileM ? Rg : kTileM), 1, 1};
        if (!encode_map(&tm_q, a.q, 4, dims, str, box)) return cudaErrorInvalidValue;
        if (!encode_map(&tm_do, a.dout, 4, dims, str, box)) return cudaErrorInvalidValue;
    }
    {
        cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)dm.P, (cuuint64_t)dm.Hkv};
        cuuint64_t str[2] = {(cuuint64_t)kD * 2, (cuuint64_t)dm.Pstride * kD * 2};
        cuuint32_t box[3] = {64, 64, 1};
        if (!encode_map(&tm_k, a.prefix_k, 3, dims, str, box)) return cudaErrorInvalidValue;
        if (!encode_map(&tm_v, a.prefix_v, 3, dims, str, box)) return cudaErrorInvalidValue;
    }
    cudaError_t e = cudaMemsetAsync(acc32, 0, 2 * n_acc * sizeof(float), stream);
    if (e != cudaSuccess) return e;
    e = launch_np<4, true>(a, tm_q, tm_do, tm_k, tm_v, tm_do, p, smem_bytes, stream);
    if (e != cudaSuccess) return e;
    const int blocks = (int)((n_acc + 255) / 256 < 1184 ? (n_acc + 255) / 256 : 1184);
    prefix_grad_round_kernel<<<blocks, 256, 0, stream>>>(p.dkp32, p.dvp32, dk_prefix, dv_prefix, n_acc);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace pskv
