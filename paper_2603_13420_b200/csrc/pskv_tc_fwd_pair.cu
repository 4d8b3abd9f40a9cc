// Fused shared-prefix attention forward on CTA pairs (sm_100a: tcgen05 cta_group::2 / TMEM / TMA).
//
// Same operator and same pipeline as the single-CTA forward kernel (Eq. 2 over the shared prefix
// cache of Sec. 4.2 followed by the candidates' own suffix keys, one continued softmax, `out` and
// `lse` written once), for the shapes whose prefix stays resident in shared memory.  Two CTAs on
// the two SMs of a TPC work on 256 consecutive rows of a KV head's row list: every MMA instruction
// covers both CTAs' 128 rows, and each CTA holds only HALF of every B operand -- half of the keys of
// a prefix K block, 64 of the 128 value columns of a V block -- so the resident prefix costs half the
// shared memory per CTA.  That pays for what the single-CTA kernel could not afford next to a
// 256-token prefix: two Q buffers (the next tile's queries land while this tile's scores are
// computed), two suffix K / V buffers and an output staging buffer of its own, so that consecutive
// tiles overlap instead of forming one chain; and one issuing thread feeds two tensor cores.
//
// Per CTA, 24 warps (both CTAs run all roles on their own rows; only the MMA issue differs):
//   warp 0      TMA producer, score side: own Q tile, own half of the prefix K blocks and of the suffix keys
//   warp 1      rank 0: issues S = Q K^T for the pair; rank 1: tells rank 0 when its operands have landed
//   warp 2      rank 0: issues O += P V for the pair; rank 1: the same relay for the value side
//               (owns the tensor-memory allocation in both CTAs)
//   warp 3      TMA producer, value side: own 64 columns of the prefix V blocks and of the suffix values
//   warps 4-19  softmax: two groups of eight warps take the items in turn (thread <-> query row, the
//               group's warps split the tile by row quadrant and column half)
//   warps 20-23 epilogue: O / row sum -> bf16 -> staging -> TMA store; lse
// Every copy is a plain single-CTA TMA load into the CTA's own shared memory.  The CTAs meet only at
// mbarriers: commits signal the same barrier in both CTAs, rank 1's warps arrive remotely on rank 0's
// barriers.  Every wait is bounded; a CTA that gives up raises the abort flag of both.
#include <string.h>

#include "pskv_common.cuh"
#include "pskv_rows.cuh"
#include "pskv_sm100.cuh"
#include "pskv_tc_common.cuh"

namespace pskv {
namespace {

using namespace sm100;

constexpr int kD = 128;
constexpr int kSlots = 2;      // score slots (128 fp32 columns) and probability slots (64 columns of bf16 pairs)
constexpr int kPiece = 32;     // score columns a softmax thread handles at a time
constexpr int kGroups = 2;     // softmax groups: they take the items in turn (group = the item's slot)
constexpr int kColSplit = 2;   // warps per row quadrant in a group: each owns 128 / kColSplit score columns
constexpr int kWarpCols = kBlockN / kColSplit;        // score columns of a softmax warp
constexpr int kSub = 16;                              // columns per tensor-memory load of a softmax thread
static_assert(kWarpCols % (2 * kSub) == 0, "pieces come in pairs");
constexpr int kParts = kGroups * kColSplit;            // partial row sums per row and tile
constexpr int kSoftmaxWarps = 4 * kGroups * kColSplit;
constexpr int kThreads = 32 * (4 + kSoftmaxWarps + 4);
constexpr int kPCol = kSlots * kBlockN;            // first tensor-memory column of the probability slots
constexpr int kPSlotCols = kBlockN / 2;
constexpr int kOCol = kPCol + kSlots * kPSlotCols;  // first tensor-memory column of O
static_assert(kOCol + kD <= 512, "tensor memory");
constexpr float kMaxRowSum = 1.2676506002282294e30f;   // 2^100
constexpr float kMinRowSum = 7.8886090522101181e-31f;  // 2^-100
constexpr int kMaxBlocks = 4;            // resident prefix blocks
constexpr int kPairRows = 2 * kTileM;    // rows of a pair tile
constexpr int kSlabBytes = kTileM * 128; // 128 rows x 64 columns of bf16
constexpr int kQBytes = 2 * kSlabBytes;  // a Q tile
constexpr int kKBlockBytes = 2 * 64 * 128;   // this CTA's 64 keys of a prefix K block, two slabs
constexpr int kVBlockBytes = kBlockN * 128;  // 128 keys x this CTA's 64 value columns
constexpr uint16_t kBoth = 3;            // both CTAs of the pair

enum : unsigned int {
    kErrProducerK = 0x401, kErrProducerV = 0x402, kErrMmaQk = 0x403, kErrMmaPv = 0x404,
    kErrSoftmax = 0x405, kErrEpilogue = 0x406, kErrAlign = 0x407, kErrRelay = 0x408
};

struct PairParams {
    float *lse;
    unsigned int *status;
    FwdArgs args;         // the call's raw arguments, for the rows that are redone row by row
    float sl2;            // scale * log2(e)
    int B, Hq, Hkv, S, P, n_rep;
    int Rg;               // rows per candidate in one KV-head group: n_rep * S
    int seg_rows;         // rows per Q / out TMA box: gcd(Rg, 128)
    int pt_per_group;     // pair tiles per KV head
    int total_pt;
    FastDiv fd_ptpg, fd_Rg, fd_S, fd_seg;
    int nblk_p;           // prefix key blocks: ceil(P / 128)
    int tail_rows;        // keys of the last prefix block, rounded up to 32
    int nc;               // candidates a pair tile touches (the same for every pair tile)
    int n_sfx;            // suffix keys of a pair tile: nc * S (a multiple of 16, at least 32)
    int chunk;            // rows per suffix K box: gcd(S, n_sfx / 2)
    FastDiv fd_chunkS;    // division by S for the chunk -> (candidate, row) split
    // shared-memory carve-up (byte offsets from the 1024-byte aligned base)
    int off_pk, off_pv, off_q, off_sk, off_sv, off_stage, off_bar, off_misc, off_ml;
    int sk_bytes, sv_bytes;  // one suffix K / V buffer
};

// barrier indices (the same layout in both CTAs)
enum {
    kBarQFull = 0,                 // [2] Q tile landed (rank 0: in both CTAs)
    kBarQFree = 2,                 // [2] all score MMAs of the tile completed: Q and suffix K buffers free
    kBarSKFull = 4,                // [2]
    kBarSVFull = 6,                // [2]
    kBarSVFree = 8,                // [2] all value MMAs of the tile completed
    kBarOFull = 10,                // O of a tile is complete in tensor memory
    kBarOFree = 11,                // epilogue warps of both CTAs have read O out (rank 0 only)
    kBarStageFull = 12,            // output tile staged (one arrival per epilogue warp)
    kBarStageFree = 13,            // the TMA stores have read it
    kBarSFull = 14,                // [kSlots] scores of an item are in tensor memory
    kBarSFree = kBarSFull + kSlots,    // [kSlots] the group's warps of both CTAs hold the scores in registers (rank 0 only)
    kBarPReady = kBarSFree + kSlots,   // [kSlots] probabilities written, both CTAs (rank 0 only)
    kBarPvDone = kBarPReady + kSlots,  // [kSlots] value MMAs of an item completed: its probability slot is free
    kBarKFull = kBarPvDone + kSlots,   // [kMaxBlocks] resident prefix K block landed
    kBarVFull = kBarKFull + kMaxBlocks,
    kNumBars = kBarVFull + kMaxBlocks
};
constexpr int kBarBytes = 512;
static_assert(kNumBars * 8 <= kBarBytes, "barrier area");

struct PairTile {
    int g, PR0, R0, b_first;
    bool first_of_g;
};

__device__ __forceinline__ PairTile pair_tile(const PairParams &p, int pt, int pt_begin, int rank)
{
    PairTile t;
    t.g = p.fd_ptpg.div(pt);
    const int ptt = pt - t.g * p.pt_per_group;
    t.first_of_g = ptt == 0 || pt == pt_begin;
    t.PR0 = ptt * kPairRows;
    t.R0 = t.PR0 + rank * kTileM;
    t.b_first = p.fd_Rg.div(t.PR0);
    return t;
}

__device__ __forceinline__ int block_keys(const PairParams &p, int k)
{
    return k == p.nblk_p - 1 ? p.tail_rows : kBlockN;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
tc_fwd_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_out,
                   const __grid_constant__ CUtensorMap tm_pk, const __grid_constant__ CUtensorMap tm_pv,
                   const __grid_constant__ CUtensorMap tm_pk_tail, const __grid_constant__ CUtensorMap tm_pv_tail,
                   const __grid_constant__ CUtensorMap tm_sk, const __grid_constant__ CUtensorMap tm_sv,
                   const PairParams p)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);  // warp-uniform by construction
    PSKV_TRACE_DECL;
    const int rank = (int)cluster_cta_rank();  // 0 issues the MMAs of the pair
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + p.off_bar;
    const uint32_t lead_bar0 = map_to_cta(bar0, 0);  // the same barriers in the CTA of rank 0
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    auto lead_bar = [&](int i) { return lead_bar0 + 8u * (uint32_t)i; };
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + p.off_misc + 4);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + p.off_misc);
    int *cta_redo = reinterpret_cast<int *>(smem + p.off_misc + 8);  // rows of this CTA's tiles to redo
    float *ml = reinterpret_cast<float *>(smem + p.off_ml);  // partial row sums [tile % 4][softmax group][128]

    const bool misaligned = (sbase & 1023u) != 0u;  // the swizzled layouts need a 1024-byte aligned base
    // Zero the data area: rows that no TMA box ever writes must hold finite values, because a zero
    // probability times a NaN value row would still poison the accumulator.
    for (int i = tid; i < p.off_bar / 16; i += kThreads) reinterpret_cast<uint4 *>(smem)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
        for (int i = 0; i < kNumBars; ++i) {
            uint32_t count = 1;
            const bool both_land = (i >= kBarQFull && i < kBarQFull + 2) || (i >= kBarSKFull && i < kBarSKFull + 2) ||
                                   (i >= kBarSVFull && i < kBarSVFull + 2) || i >= kBarKFull;
            if (both_land) count = rank == 0 ? 2u : 1u;  // own copies + the other CTA's "landed" arrival
            if (i >= kBarSFree && i < kBarPReady + kSlots) count = 2u * 4u * kColSplit;  // the warps of the item's softmax group, both CTAs
            if (i == kBarOFree) count = 8u;                                             // epilogue warps of both CTAs
            if (i == kBarStageFull) count = 4u;
            mbar_init(bar(i), count);
        }
        *abort_flag = misaligned ? 1 : 0;
        *cta_redo = 0;
        if (misaligned) atomicCAS(p.status, 0u, (unsigned int)kErrAlign);
        fence_barrier_init();
    }
    fence_proxy_async();
    __syncthreads();
    if (warp == 2) {
        tmem_alloc_pair(smem_u32(tmem_slot), 512);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    // the other CTA's barriers must exist before anything arrives on them
    cluster_arrive();
    cluster_wait();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // Pair tiles of this pair of CTAs: a contiguous range (ordered KV head major, so the resident
    // prefix of a head serves a whole run).
    const int pair = (int)blockIdx.x >> 1, npairs = (int)gridDim.x >> 1;
    const int pt_begin = (int)((long long)pair * p.total_pt / npairs);
    const int pt_end = (int)((long long)(pair + 1) * p.total_pt / npairs);
    const int n_tiles = pt_end - pt_begin;
    const int nitems = p.nblk_p + 1;  // prefix blocks + the suffix block
    const int g_first = p.fd_ptpg.div(pt_begin < p.total_pt ? pt_begin : 0);
    const int nseg = p.fd_seg.div(kTileM);
    const int half_sfx = p.n_sfx >> 1;
    const uint32_t seg_bytes = (uint32_t)(p.seg_rows * 128);

    // The roles trade registers: the four control warps need few, a softmax thread holds a whole row
    // of scores, an epilogue thread a whole row of O.
    if (warp < 4) {
    if (misaligned) {
        // nothing runs; fall through to the teardown both CTAs share
    } else if (warp == 0) {
        // ------------------------------------------------------------------ producer, score side
        if (lane == 0) {
            prefetch_tensormap(&tm_q);
            prefetch_tensormap(&tm_sk);
            if (p.P > 0) { prefetch_tensormap(&tm_pk); prefetch_tensormap(&tm_pk_tail); }
        }
        bool ok = true;
#pragma unroll 1
        for (int tl = 0; tl < n_tiles && ok; ++tl) {
            const PairTile t = pair_tile(p, pt_begin + tl, pt_begin, rank);
            const int buf = tl & 1;
            int qb = p.fd_Rg.div(t.R0), qr = t.R0 - qb * p.Rg;
            uint32_t q_dst = sbase + p.off_q + buf * kQBytes;
            // the buffer pair (Q, suffix K) is free once every score MMA of tile tl-2 has completed
            ok = mbar_wait_warp_cl(bar(kBarQFree + buf), ((tl >> 1) & 1) ^ 1, abort_flag, p.status, kErrProducerK);
            if (!ok) break;
            PSKV_TRACE_EVENT(1, tl);
            if (elect_one_sync()) {
                mbar_arrive_expect_tx(bar(kBarQFull + buf), (uint32_t)kQBytes);
#pragma unroll 1
                for (int s = 0; s < nseg; ++s) {
#pragma unroll
                    for (int sl = 0; sl < 2; ++sl)
                        tma_load_4d(q_dst + sl * kSlabBytes, &tm_q, bar(kBarQFull + buf), sl * 64, qr, t.g, qb);
                    q_dst += seg_bytes;
                    qr += p.seg_rows;  // boxes never straddle a candidate: seg_rows divides Rg
                    if (qr >= p.Rg) {
                        qr -= p.Rg;
                        ++qb;
                    }
                }
            }
            __syncwarp();
            if (t.first_of_g && p.nblk_p > 0) {
                // a new KV head: its prefix K replaces the resident blocks once the score MMAs of the
                // previous tile (the last to read them) have completed
                if (tl > 0) {
                    ok = mbar_wait_warp_cl(bar(kBarQFree + ((tl - 1) & 1)), ((tl - 1) >> 1) & 1, abort_flag, p.status,
                                           kErrProducerK);
                    if (!ok) break;
                }
                if (elect_one_sync()) {
#pragma unroll 1
                    for (int k = 0; k < p.nblk_p; ++k) {
                        const bool tail = k == p.nblk_p - 1;
                        const int half = block_keys(p, k) >> 1;  // this CTA's keys of the block
                        mbar_arrive_expect_tx(bar(kBarKFull + k), (uint32_t)(2 * half * 128));
#pragma unroll 1
                        for (int sl = 0; sl < 2; ++sl)
                            tma_load_3d(sbase + p.off_pk + k * kKBlockBytes + sl * half * 128, tail ? &tm_pk_tail : &tm_pk,
                                        bar(kBarKFull + k), sl * 64, k * kBlockN + rank * half, t.g);
                    }
                }
                __syncwarp();
            }
            // this CTA's half of the pair tile's suffix keys: rows [rank * half, rank * half + half) of
            // the candidates' rows laid end to end, in boxes that never straddle a candidate
            if (elect_one_sync()) {
                const uint32_t dst = sbase + p.off_sk + buf * p.sk_bytes;
                mbar_arrive_expect_tx(bar(kBarSKFull + buf), (uint32_t)(2 * half_sfx * 128));
#pragma unroll 1
                for (int flat = 0; flat < half_sfx; flat += p.chunk) {
                    const int row = rank * half_sfx + flat;
                    const int c = p.fd_chunkS.div(row), r = row - c * p.S;
#pragma unroll 1
                    for (int sl = 0; sl < 2; ++sl)
                        tma_load_4d(dst + sl * half_sfx * 128 + flat * 128, &tm_sk, bar(kBarSKFull + buf), sl * 64, r,
                                    t.g, t.b_first + c);
                }
            }
            __syncwarp();
        }
    } else if (warp == 3) {
        // ------------------------------------------------------------------ producer, value side
        if (lane == 0) {
            prefetch_tensormap(&tm_sv);
            if (p.P > 0) { prefetch_tensormap(&tm_pv); prefetch_tensormap(&tm_pv_tail); }
        }
        bool ok = true;
#pragma unroll 1
        for (int tl = 0; tl < n_tiles && ok; ++tl) {
            const PairTile t = pair_tile(p, pt_begin + tl, pt_begin, rank);
            const int buf = tl & 1;
            if (t.first_of_g && p.nblk_p > 0) {
                if (tl > 0) {  // the value MMAs of the previous tile were the last to read the resident V blocks
                    ok = mbar_wait_warp_cl(bar(kBarSVFree + ((tl - 1) & 1)), ((tl - 1) >> 1) & 1, abort_flag, p.status,
                                           kErrProducerV);
                    if (!ok) break;
                }
                if (elect_one_sync()) {
#pragma unroll 1
                    for (int k = 0; k < p.nblk_p; ++k) {
                        const bool tail = k == p.nblk_p - 1;
                        mbar_arrive_expect_tx(bar(kBarVFull + k), (uint32_t)(block_keys(p, k) * 128));
                        // all keys of the block, this CTA's 64 value columns
                        tma_load_3d(sbase + p.off_pv + k * kVBlockBytes, tail ? &tm_pv_tail : &tm_pv, bar(kBarVFull + k),
                                    rank * 64, k * kBlockN, t.g);
                    }
                }
                __syncwarp();
            }
            ok = mbar_wait_warp_cl(bar(kBarSVFree + buf), ((tl >> 1) & 1) ^ 1, abort_flag, p.status, kErrProducerV);
            if (!ok) break;
            if (elect_one_sync()) {
                const uint32_t dst = sbase + p.off_sv + buf * p.sv_bytes;
                mbar_arrive_expect_tx(bar(kBarSVFull + buf), (uint32_t)(p.n_sfx * 128));
#pragma unroll 1
                for (int c = 0; c < p.nc; ++c)
                    tma_load_4d(dst + c * p.S * 128, &tm_sv, bar(kBarSVFull + buf), rank * 64, 0, t.g, t.b_first + c);
            }
            __syncwarp();
            PSKV_TRACE_EVENT(5, tl);
        }
    }
    else if (warp == 1 && rank == 0) {
        // ------------------------------------------------------------------ score MMAs of the pair: S = Q K^T
        bool ok = true;
        int i = 0;
#pragma unroll 1
        for (int tl = 0; tl < n_tiles && ok; ++tl) {
            const PairTile t = pair_tile(p, pt_begin + tl, pt_begin, 0);
            const int buf = tl & 1;
            const uint64_t q_desc = make_smem_desc(sbase + p.off_q + buf * kQBytes, 0, 1024);
#pragma unroll 1
            for (int k = 0; k < nitems && ok; ++k, ++i) {
                const int slot = i % kSlots;
                const bool prefix = k < p.nblk_p;
                const int n = prefix ? block_keys(p, k) : p.n_sfx;
                const uint32_t kaddr = prefix ? sbase + p.off_pk + k * kKBlockBytes : sbase + p.off_sk + buf * p.sk_bytes;
                const uint32_t idesc = make_idesc_bf16(kPairRows, n, 0);
                const uint32_t d_tmem = tmem + slot * kBlockN;
                const uint64_t k_desc = make_smem_desc(kaddr, 0, 1024);
                const uint64_t k_slab = (uint64_t)(((n >> 1) * 128) >> 4);  // this CTA's half of the keys per slab
                // the score slot is free once the softmax warps of item i-2 hold its scores in registers
                PSKV_TRACE_EVENT(16, i);
                ok = mbar_wait_warp_cl(bar(kBarSFree + slot), ((i / kSlots) & 1) ^ 1, abort_flag, p.status, kErrMmaQk);
                if (!ok) break;
                PSKV_TRACE_EVENT(18, i);
                if (k == 0) {  // the Q tiles of both CTAs
                    ok = mbar_wait_warp_cl(bar(kBarQFull + buf), (tl >> 1) & 1, abort_flag, p.status, kErrMmaQk);
                    if (!ok) break;
                }
                PSKV_TRACE_EVENT(19, i);
                if (prefix) {
                    if (t.first_of_g)
                        ok = mbar_wait_warp_cl(bar(kBarKFull + k), (uint32_t)(t.g - g_first) & 1u, abort_flag, p.status,
                                               kErrMmaQk);
                } else {
                    ok = mbar_wait_warp_cl(bar(kBarSKFull + buf), (tl >> 1) & 1, abort_flag, p.status, kErrMmaQk);
                }
                if (!ok) break;
                PSKV_TRACE_EVENT(10, i);
                tc_fence_after();
                if (elect_one_sync()) {
#pragma unroll
                    for (int ks16 = 0; ks16 < kD / 16; ++ks16) {
                        const uint64_t qoff = (uint64_t)(((ks16 >> 2) * kSlabBytes + (ks16 & 3) * 32) >> 4);
                        const uint64_t koff = (uint64_t)(ks16 >> 2) * k_slab + (uint64_t)(((ks16 & 3) * 32) >> 4);
                        mma_ss_pair(d_tmem, q_desc + qoff, k_desc + koff, idesc, ks16 > 0 ? 1u : 0u);
                    }
                    tc_commit_pair(bar(kBarSFull + slot), kBoth);
                    if (k == nitems - 1) tc_commit_pair(bar(kBarQFree + buf), kBoth);  // the suffix block ends the tile's scores
                }
                __syncwarp();
                PSKV_TRACE_EVENT(12, i);
            }
        }
    } else if (warp == 2 && rank == 0) {
        // ------------------------------------------------------------------ value MMAs of the pair: O += P V
        const uint32_t idesc_pv = make_idesc_bf16(kPairRows, kD, 1);
        bool ok = true;
        int i = 0;
#pragma unroll 1
        for (int tl = 0; tl < n_tiles && ok; ++tl) {
            const PairTile t = pair_tile(p, pt_begin + tl, pt_begin, 0);
            const int buf = tl & 1;
#pragma unroll 1
            for (int k = 0; k < nitems && ok; ++k, ++i) {
                const int slot = i % kSlots;
                const bool prefix = k < p.nblk_p;
                const int n = prefix ? block_keys(p, k) : p.n_sfx;
                const uint32_t vaddr = prefix ? sbase + p.off_pv + k * kVBlockBytes : sbase + p.off_sv + buf * p.sv_bytes;
                const uint32_t p_tmem = tmem + kPCol + slot * kPSlotCols;  // bf16 pairs: 8 columns per 16 keys
                // V as [keys][64 columns of this CTA]: the N index is the contiguous one, 8-key groups 1024 bytes apart
                const uint64_t v_desc = make_smem_desc(vaddr, 1024, 1024);
                const int nk = n >> 4;
                const uint32_t acc0 = k > 0 ? 1u : 0u;
                PSKV_TRACE_EVENT(17, i);
                // probabilities of both CTAs written
                ok = mbar_wait_warp_cl(bar(kBarPReady + slot), (i / kSlots) & 1, abort_flag, p.status, kErrMmaPv);
                if (!ok) break;
                if (k == 0 && tl > 0) {
                    // O of the previous tile must have been read out by the epilogue warps of both CTAs
                    PSKV_TRACE_EVENT(15, i);
                    ok = mbar_wait_warp_cl(bar(kBarOFree), (tl - 1) & 1, abort_flag, p.status, kErrMmaPv);
                    if (!ok) break;
                }
                if (prefix) {
                    if (t.first_of_g)
                        ok = mbar_wait_warp_cl(bar(kBarVFull + k), (uint32_t)(t.g - g_first) & 1u, abort_flag, p.status,
                                               kErrMmaPv);
                } else {
                    ok = mbar_wait_warp_cl(bar(kBarSVFull + buf), (tl >> 1) & 1, abort_flag, p.status, kErrMmaPv);
                }
                if (!ok) break;
                PSKV_TRACE_EVENT(11, i);
                tc_fence_after();
                if (elect_one_sync()) {
#pragma unroll
                    for (int ks16 = 0; ks16 < kBlockN / 16; ++ks16) {
                        if (ks16 < nk)
                            mma_ts_pair(tmem + kOCol, p_tmem + ks16 * 8,
                                        v_desc + (uint64_t)(ks16 * (2048 >> 4)), idesc_pv, ks16 > 0 ? 1u : acc0);
                    }
                    tc_commit_pair(bar(kBarPvDone + slot), kBoth);
                    if (k == nitems - 1) {
                        tc_commit_pair(bar(kBarSVFree + buf), kBoth);
                        tc_commit_pair(bar(kBarOFull), kBoth);
                    }
                }
                __syncwarp();
                PSKV_TRACE_EVENT(13, i);
            }
        }
    } else if (warp == 1 || warp == 2) {
        // ------------------------------------------------------------------ rank 1: operands-landed relay
        // Rank 0 may issue an MMA only when the operand halves of BOTH CTAs are in place.  This CTA's
        // copies complete on its own barriers; these two warps wait there (warp 1: Q, prefix K, suffix
        // K; warp 2: prefix V, suffix V) and pass each completion on as one arrival on the same
        // barrier of rank 0.
        const bool score_side = warp == 1;
        bool ok = true;
#pragma unroll 1
        for (int tl = 0; tl < n_tiles && ok; ++tl) {
            const PairTile t = pair_tile(p, pt_begin + tl, pt_begin, 1);
            const int buf = tl & 1;
            const uint32_t par = (tl >> 1) & 1;
            if (score_side) {
                ok = mbar_wait_warp_cl(bar(kBarQFull + buf), par, abort_flag, p.status, kErrRelay);
                if (!ok) break;
                if (lane == 0) mbar_arrive_remote(lead_bar(kBarQFull + buf));
            }
            if (t.first_of_g) {
#pragma unroll 1
                for (int k = 0; k < p.nblk_p && ok; ++k) {
                    const int b = (score_side ? kBarKFull : kBarVFull) + k;
                    ok = mbar_wait_warp_cl(bar(b), (uint32_t)(t.g - g_first) & 1u, abort_flag, p.status, kErrRelay);
                    if (ok && lane == 0) mbar_arrive_remote(lead_bar(b));
                }
                if (!ok) break;
            }
            const int b = (score_side ? kBarSKFull : kBarSVFull) + buf;
            ok = mbar_wait_warp_cl(bar(b), par, abort_flag, p.status, kErrRelay);
            if (!ok) break;
            if (lane == 0) mbar_arrive_remote(lead_bar(b));
            __syncwarp();
        }
    }
    } else if (warp < 4 + kSoftmaxWarps) {
        // ------------------------------------------------------------------ softmax warps
        // Two groups take the items in turn (group = item mod 2 = the item's score and probability
        // slot), so that one group's loads, waits and stores fall under the other one's exponentials.
        // In a group the warps split the tile by row quadrant (tensor memory gives a warp the 32
        // lanes of its quadrant) and by column half; a thread owns one query row and walks its 64
        // columns in 16-column pieces, the load of the next piece in flight while it works on
        // the current one (a tensor-memory load takes 400 to 600 cycles while the MMAs run).  The
        // piece loop is unrolled by two only: with a whole row unrolled the loop body no longer
        // fits the instruction cache (2.4 warps per issue slot stalled for instructions,
        // against 0.5 in this form) and every piece took twice as long.  The score slot goes back
        // to the MMA issuer as soon as the last piece is in registers, the probabilities go to a
        // slot of their own that only the item's value MMAs hold; the first load of the group's
        // next item is issued before this item's bookkeeping.  p = 2^(s * sl2) with no running
        // max (rows whose sum leaves [2^-100, 2^100] are redone at the end); partial row sums go to
        // the epilogue through shared memory.  Both arrivals go to rank 0, whose threads issue
        // the MMAs.
        const int sw = warp - 4;
        const int wg = sw / (4 * kColSplit);
        const int half = (sw >> 2) % kColSplit;
        const int part = wg * kColSplit + half;
        const int row = 32 * (warp & 3) + lane;
        const uint32_t lane_base = tmem + ((uint32_t)(32 * (warp & 3)) << 16);
        const uint32_t s_tmem = lane_base + wg * kBlockN + half * kWarpCols;
        const uint32_t p_tmem = lane_base + kPCol + wg * kPSlotCols + half * (kWarpCols / 2);
        const int col0 = half * kWarpCols;  // first score column of this warp
        bool ok = !misaligned;
        int tl = 0, k = wg;  // item = tl * nitems + k
        while (k >= nitems) { k -= nitems; ++tl; }
        int tl_row = -1, lo_sfx = 0, hi_sfx = 0;
        int n = 0, lo = 0, hi = -1;  // the current item: keys, and this row's valid columns [lo, hi]
        float lsum = 0.f;
        // 0 = beyond the item's keys (never read by the value MMAs), 1 = no valid column for this warp
        // (zeros), 2 = some masked, 3 = all valid
        auto piece_kind = [&](int c0) -> int {
            if (c0 >= n) return 0;
            const bool all_valid = lo <= c0 && hi >= c0 + kSub - 1;
            const bool none_valid = hi < lo || hi < c0 || lo > c0 + kSub - 1;
            return __all_sync(0xffffffffu, all_valid) ? 3 : __all_sync(0xffffffffu, none_valid) ? 1 : 2;
        };
        // this row's limits for item (tl, k); a new tile resets the row sum
        auto begin_item = [&]() {
            if (tl != tl_row) {
                const PairTile t = pair_tile(p, pt_begin + tl, pt_begin, rank);
                const int R = t.R0 + row;
                const int b = p.fd_Rg.div(R), r = R - b * p.Rg;
                lo_sfx = (b - t.b_first) * p.S;              // first suffix column of this row's candidate
                hi_sfx = lo_sfx + (r - p.fd_S.div(r) * p.S); // causal: suffix keys 0..i
                lsum = 0.f;
                tl_row = tl;
            }
            const bool prefix = k < p.nblk_p;
            n = prefix ? block_keys(p, k) : p.n_sfx;
            lo = prefix ? 0 : lo_sfx;
            hi = prefix ? min(kBlockN, p.P - k * kBlockN) - 1 : hi_sfx;
        };
        float ls0 = 0.f, ls1 = 0.f;
        // one 16-column piece: exponentials, row sum, bf16 pairs to the probability slot
        auto piece = [&](const uint32_t (&rr)[kSub], int kind, int c0) {
            uint32_t pk[kSub / 2];
            if (kind == 3) {
#pragma unroll
                for (int j = 0; j < kSub; j += 2) {
                    float x0 = __uint_as_float(rr[j]), x1 = __uint_as_float(rr[j + 1]);
                    mul_f32x2(x0, x1, p.sl2);
                    x0 = ex2_approx(x0);
                    x1 = ex2_approx(x1);
                    add_f32x2(ls0, ls1, x0, x1);
                    pk[j >> 1] = pack_bf16x2(x0, x1);
                }
            } else if (kind == 2) {
                const unsigned span = (unsigned)(hi - lo);
                const int base = c0 - lo;
                const bool any_col = hi >= lo;
#pragma unroll
                for (int j = 0; j < kSub; j += 2) {
                    float x0 = __uint_as_float(rr[j]), x1 = __uint_as_float(rr[j + 1]);
                    mul_f32x2(x0, x1, p.sl2);
                    x0 = ex2_approx(x0);
                    x1 = ex2_approx(x1);
                    x0 = (any_col && (unsigned)(base + j) <= span) ? x0 : 0.f;
                    x1 = (any_col && (unsigned)(base + j + 1) <= span) ? x1 : 0.f;
                    add_f32x2(ls0, ls1, x0, x1);
                    pk[j >> 1] = pack_bf16x2(x0, x1);
                }
            } else {
#pragma unroll
                for (int j = 0; j < kSub / 2; ++j) pk[j] = 0u;
            }
            if (kind != 0) tmem_st8(p_tmem + ((c0 - col0) >> 1), pk);
        };
        uint32_t ra[kSub], rb[kSub];
        int kind_a = 0;
        if (ok && tl < n_tiles) {  // the first item: its scores, and the load of its first piece
            begin_item();
            ok = mbar_wait_warp_cl(bar(kBarSFull + wg), 0, abort_flag, p.status, kErrSoftmax);
            if (ok) {
                tc_fence_after();
                kind_a = piece_kind(col0);
                if (kind_a >= 2) tmem_ld16(s_tmem, ra);
            }
        }
#pragma unroll 1
        for (int use = 0; tl < n_tiles && ok; ++use) {
            PSKV_TRACE_EVENT(20, use * kGroups + wg);
            ls0 = 0.f;
            ls1 = 0.f;
#pragma unroll 1
            for (int it = 0; it < kWarpCols / (2 * kSub); ++it) {
                const int ca = col0 + it * 2 * kSub, cb = ca + kSub;
                const bool last = it == kWarpCols / (2 * kSub) - 1;
                tmem_wait_ld();  // piece A is in registers
                const int kind_b = piece_kind(cb);
                if (kind_b >= 2) tmem_ld16(s_tmem + (cb - col0), rb);
                if (it == 0) {
                    // the probability slot is free once the value MMAs of this group's previous item have
                    // completed (issued a whole item period ago, so this wait rarely spins)
                    ok = mbar_wait_warp_cl(bar(kBarPvDone + wg), (use & 1) ^ 1, abort_flag, p.status, kErrSoftmax);
                    if (!ok) break;
                    tc_fence_after();
                }
                piece(ra, kind_a, ca);
                tmem_wait_ld();  // piece B is in registers
                if (!last) {
                    kind_a = piece_kind(cb + kSub);
                    if (kind_a >= 2) tmem_ld16(s_tmem + (cb + kSub - col0), ra);
                } else {
                    // this warp holds all it needs of the scores: the score MMAs of the group's next item
                    // may overwrite the slot once every warp of the group has said so
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_remote(lead_bar(kBarSFree + wg));
                    PSKV_TRACE_EVENT(21, use * kGroups + wg);
                }
                piece(rb, kind_b, cb);
            }
            if (!ok) break;
            lsum += ls0 + ls1;
            PSKV_TRACE_EVENT(23, use * kGroups + wg);
            // on to the group's next item; a partial row sum is complete when that one lies in another
            // tile, and goes to the epilogue warps through shared memory BEFORE the arrival below (the
            // tile's last value MMAs, which the epilogue waits for, need it)
            const int tl_done = tl;
            k += kGroups;
            while (k >= nitems) { k -= nitems; ++tl; }
            if (tl != tl_done) {
                ml[((tl_done & 3) * kParts + part) * kTileM + row] = lsum;
                __threadfence_block();
            }
            // the probabilities of this item are complete
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(lead_bar(kBarPReady + wg));
            PSKV_TRACE_EVENT(24, use * kGroups + wg);
            // the scores of the next item, and the load of its first piece
            if (tl < n_tiles) {
                begin_item();
                PSKV_TRACE_EVENT(25, (use + 1) * kGroups + wg);
                ok = mbar_wait_warp_cl(bar(kBarSFull + wg), (use + 1) & 1, abort_flag, p.status, kErrSoftmax);
                if (!ok) break;
                tc_fence_after();
                kind_a = piece_kind(col0);
                if (kind_a >= 2) tmem_ld16(s_tmem, ra);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps (20..23)
        // O / l -> bf16 -> staging buffer -> TMA store (issued by the first of these warps); lse; rows
        // to redo.  Thread <-> query row; the row sum is the sum of the four softmax groups' partial sums.
        const int ew = warp & 3;
        const int row = 32 * ew + lane;
        const uint32_t lane_addr = (uint32_t)(32 * ew) << 16;
        const bool issuer = warp == 4 + kSoftmaxWarps;
        const uint32_t stage = sbase + p.off_stage;
        if (issuer && lane == 0) prefetch_tensormap(&tm_out);
        bool ok = !misaligned;
#pragma unroll 1
        for (int te = 0; te < n_tiles && ok; ++te) {
            const PairTile u = pair_tile(p, pt_begin + te, pt_begin, rank);
            ok = mbar_wait_warp_cl(bar(kBarOFull), te & 1, abort_flag, p.status, kErrEpilogue);
            if (!ok) break;
            PSKV_TRACE_EVENT(30, te);
            tc_fence_after();
            // the row sum: partial sums of the softmax groups that had an item of this tile (items go to
            // the groups in turn), added in a fixed order
            const float *mlt = ml + (te & 3) * kParts * kTileM + row;
            float l = 0.f;
            {
                const int first = (te * nitems) % kGroups;  // group of the tile's first item
#pragma unroll
                for (int g = 0; g < kGroups; ++g) {
                    const int dist = g >= first ? g - first : g + kGroups - first;  // items until group g's turn
                    if (dist < nitems) {
#pragma unroll
                        for (int h = 0; h < kColSplit; ++h) l += mlt[(g * kColSplit + h) * kTileM];
                    }
                }
            }
            const bool row_ok = l >= kMinRowSum && l <= kMaxRowSum;  // false for overflow (inf, NaN), underflow
            const float inv = row_ok ? 1.f / l : 0.f;
            // the TMA stores of the previous tile must have read the staging buffer
            ok = mbar_wait_warp_cl(bar(kBarStageFree), (te & 1) ^ 1, abort_flag, p.status, kErrEpilogue);
            if (!ok) break;
            PSKV_TRACE_EVENT(33, te);
            // one 64-column slab per round; O is free for the next tile's first value MMA as soon as the
            // second round's loads have returned
#pragma unroll 1
            for (int sl = 0; sl < 2; ++sl) {
                uint32_t o[2][kPiece];
                tmem_ld32(tmem + lane_addr + kOCol + sl * 64, o[0]);
                tmem_ld32(tmem + lane_addr + kOCol + sl * 64 + kPiece, o[1]);
                tmem_wait_ld();
                if (sl == 1) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_remote(lead_bar(kBarOFree));
                    PSKV_TRACE_EVENT(32, te);
                }
                // 128-byte rows, 16-byte chunks swizzled by the row; rows that failed stage zeros
                uint8_t *srow = smem + p.off_stage + sl * kStagingBytes + row * 128;
#pragma unroll
                for (int c = 0; c < 2; ++c)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint4 v;
                        v.x = pack_bf16x2(__uint_as_float(o[c][8 * j]) * inv, __uint_as_float(o[c][8 * j + 1]) * inv);
                        v.y = pack_bf16x2(__uint_as_float(o[c][8 * j + 2]) * inv, __uint_as_float(o[c][8 * j + 3]) * inv);
                        v.z = pack_bf16x2(__uint_as_float(o[c][8 * j + 4]) * inv, __uint_as_float(o[c][8 * j + 5]) * inv);
                        v.w = pack_bf16x2(__uint_as_float(o[c][8 * j + 6]) * inv, __uint_as_float(o[c][8 * j + 7]) * inv);
                        if (!row_ok) v = make_uint4(0, 0, 0, 0);
                        *reinterpret_cast<uint4 *>(srow + (((c * 4 + j) ^ (row & 7)) << 4)) = v;
                    }
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarStageFull));
            {
                const int R = u.R0 + row;
                const int b = p.fd_Rg.div(R), r = R - b * p.Rg;
                const size_t grow = ((size_t)b * p.Hq + (size_t)u.g * p.n_rep) * p.S + r;
                p.lse[grow] = row_ok ? log2f(l) * kLn2 : __int_as_float(0x7fc00000);
            }
            const unsigned bad = __ballot_sync(0xffffffffu, !row_ok);
            if (bad != 0u && lane == 0) atomicAdd(cta_redo, __popc(bad));
            if (issuer) {
                ok = mbar_wait_warp_cl(bar(kBarStageFull), te & 1, abort_flag, p.status, kErrEpilogue);
                if (!ok) break;
                if (elect_one_sync()) {
#pragma unroll 1
                    for (int sl = 0; sl < 2; ++sl)
#pragma unroll 1
                        for (int s = 0; s < nseg; ++s) {
                            const int R = u.R0 + s * p.seg_rows;
                            const int b = p.fd_Rg.div(R), r = R - b * p.Rg;
                            tma_store_4d(&tm_out, stage + sl * kStagingBytes + s * p.seg_rows * 128, sl * 64, r, u.g, b);
                        }
                    tma_store_commit();
                    tma_store_wait_read();  // the staging buffer may be overwritten after this
                    mbar_arrive(bar(kBarStageFree));
                }
                __syncwarp();
            }
            PSKV_TRACE_EVENT(31, te);
        }
        if (issuer) {
            if (elect_one_sync()) tma_store_wait_all();
            __syncwarp();
        }
    }

    // ---------------------------------------------------------------------- teardown
    PSKV_TRACE_FLUSH;
    if (*abort_flag != 0) {
        // a CTA that gave up takes the other one with it, then lets copies and MMAs in flight drain
        store_remote_u32(map_to_cta(sbase + p.off_misc + 4, (uint32_t)(rank ^ 1)), 1u);
        __nanosleep(20000);
    }
    tc_fence_before();
    __syncthreads();
    // Neither CTA may leave (or free its tensor memory) while the other can still signal its barriers
    // or while MMAs of the pair read its shared memory.
    cluster_arrive();
    cluster_wait();
    if (warp == 2) tmem_dealloc_pair(tmem, 512);
    // Rows whose sum left the safe range carry a NaN lse (and zeros in `out`): all warps of the CTA
    // now walk over its tiles and recompute those rows one warp per row with a running maximum.
    if (*cta_redo > 0 && *abort_flag == 0) {
        float *q_s = reinterpret_cast<float *>(smem) + warp * kD;
#pragma unroll 1
        for (int tl = 0; tl < n_tiles; ++tl) {
            const PairTile t = pair_tile(p, pt_begin + tl, pt_begin, rank);
#pragma unroll 1
            for (int r = warp; r < kTileM; r += kThreads / 32) {
                const int R = t.R0 + r;
                const int b = p.fd_Rg.div(R), rr = R - b * p.Rg;
                const long long grow = ((long long)b * p.Hq + (long long)t.g * p.n_rep) * p.S + rr;
                const float v = p.lse[grow];
                if (v != v) fwd_row<kD>(p.args, grow, q_s, lane);
            }
        }
    }
}

// ------------------------------------------------------------------------------ host side

struct PairPlan {
    bool ok;
    int seg_rows, pt_per_group, nblk_p, tail_rows, nc, n_sfx, chunk;
    int off_pk, off_pv, off_q, off_sk, off_sv, off_stage, off_bar, off_misc, off_ml, sk_bytes, sv_bytes, smem_bytes;
};

// The pair kernel takes the full-suffix operator with head dim 128 when a KV head's row list is a
// whole number of 256-row pair tiles, every pair tile touches the same number of candidates, their
// suffix keys fit one block and split evenly between the two CTAs, and the prefix (at most four
// blocks) fits beside the double buffers.
PairPlan plan_pair(const Dims &dm)
{
    PairPlan pl;
    memset(&pl, 0, sizeof(pl));
    if (dm.d != kD || dm.Skv != dm.S || dm.ragged || dm.Pstride != dm.P || dm.S % 8 != 0) return pl;
    const int Rg = dm.n_rep * dm.S;
    const long long total = (long long)dm.B * Rg;
    if (total % kPairRows != 0 || total / kPairRows > 2000000000ll / dm.Hkv) return pl;
    pl.seg_rows = gcd_int(Rg, kTileM);
    if (pl.seg_rows % 8 != 0) return pl;
    pl.pt_per_group = (int)(total / kPairRows);
    // candidates per pair tile: the pattern repeats every Rg / gcd(Rg, 256) pair tiles
    const long long period = Rg / gcd_int(Rg, kPairRows);
    const long long check = pl.pt_per_group < period ? pl.pt_per_group : period;
    int nc_min = 1 << 30, nc_max = 0;
    for (long long t = 0; t < check; ++t) {
        const int nc = (int)((t * kPairRows + kPairRows - 1) / Rg - (t * kPairRows) / Rg + 1);
        nc_min = nc < nc_min ? nc : nc_min;
        nc_max = nc > nc_max ? nc : nc_max;
    }
    if (nc_min != nc_max) return pl;
    pl.nc = nc_max;
    pl.n_sfx = pl.nc * dm.S;
    if (pl.n_sfx % 16 != 0 || pl.n_sfx < 32 || pl.n_sfx > kBlockN) return pl;
    pl.chunk = gcd_int(dm.S, pl.n_sfx / 2);
    if (pl.chunk % 8 != 0) return pl;
    pl.nblk_p = (dm.P + kBlockN - 1) / kBlockN;
    if (pl.nblk_p > kMaxBlocks) return pl;
    pl.tail_rows = pl.nblk_p ? round_up(dm.P - (pl.nblk_p - 1) * kBlockN, 32) : 0;
    pl.sk_bytes = pl.n_sfx * 128;  // half of the keys x two slabs
    pl.sv_bytes = pl.n_sfx * 128;  // all keys x one slab
    pl.off_pk = 0;
    pl.off_pv = pl.off_pk + pl.nblk_p * kKBlockBytes;
    pl.off_q = pl.off_pv + pl.nblk_p * kVBlockBytes;
    pl.off_sk = pl.off_q + 2 * kQBytes;
    pl.off_sv = pl.off_sk + 2 * pl.sk_bytes;
    pl.off_stage = pl.off_sv + 2 * pl.sv_bytes;
    pl.off_bar = pl.off_stage + 2 * kStagingBytes;
    pl.off_misc = pl.off_bar + kBarBytes;
    pl.off_ml = pl.off_misc + 64;
    pl.smem_bytes = pl.off_ml + 4 * kParts * kTileM * 4;
    pl.ok = pl.smem_bytes <= kMaxSmem;
    return pl;
}

}  // namespace

#ifdef PSKV_TRACE
// Debug builds only: copies this kernel's event trace of CTA 0 to the host.
extern "C" int pskv_debug_read_trace_pair(long long *host, int max_events)
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

bool tc_fwd_pair_supported(const Dims &dm) { return plan_pair(dm).ok; }

cudaError_t launch_tc_fwd_pair(const FwdArgs &a, unsigned int *status_word, cudaStream_t stream)
{
    const Dims &dm = a.dims;
    const PairPlan plan = plan_pair(dm);
    if (!plan.ok) return cudaErrorInvalidValue;
    const int Rg = dm.n_rep * dm.S;
    CUtensorMap tm_q, tm_out, tm_pk, tm_pv, tm_pk_tail, tm_pv_tail, tm_sk, tm_sv;
    memset(&tm_pk, 0, sizeof(tm_pk));
    memset(&tm_pv, 0, sizeof(tm_pv));
    memset(&tm_pk_tail, 0, sizeof(tm_pk_tail));
    memset(&tm_pv_tail, 0, sizeof(tm_pv_tail));
    {
        // q / out viewed as [B][Hkv][Rg][D]: the n_rep heads of a KV head are contiguous rows
        cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)Rg, (cuuint64_t)dm.Hkv, (cuuint64_t)dm.B};
        cuuint64_t str[3] = {(cuuint64_t)kD * 2, (cuuint64_t)Rg * kD * 2, (cuuint64_t)dm.Hkv * Rg * kD * 2};
        cuuint32_t box[4] = {64, (cuuint32_t)plan.seg_rows, 1, 1};
        if (!encode_map(&tm_q, a.q, 4, dims, str, box)) return cudaErrorInvalidValue;
        if (!encode_map(&tm_out, a.out, 4, dims, str, box)) return cudaErrorInvalidValue;
    }
    {
        cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)dm.S, (cuuint64_t)dm.Hkv, (cuuint64_t)dm.B};
        cuuint64_t str[3] = {(cuuint64_t)kD * 2, (cuuint64_t)dm.S * kD * 2, (cuuint64_t)dm.Hkv * dm.S * kD * 2};
        cuuint32_t box_k[4] = {64, (cuuint32_t)plan.chunk, 1, 1};
        cuuint32_t box_v[4] = {64, (cuuint32_t)dm.S, 1, 1};
        if (!encode_map(&tm_sk, a.suffix_k, 4, dims, str, box_k)) return cudaErrorInvalidValue;
        if (!encode_map(&tm_sv, a.suffix_v, 4, dims, str, box_v)) return cudaErrorInvalidValue;
    }
    if (dm.P > 0) {
        cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)dm.P, (cuuint64_t)dm.Hkv};
        cuuint64_t str[2] = {(cuuint64_t)kD * 2, (cuuint64_t)dm.Pstride * kD * 2};
        cuuint32_t box_k[3] = {64, 64, 1}, box_k_tail[3] = {64, (cuuint32_t)(plan.tail_rows / 2), 1};
        cuuint32_t box_v[3] = {64, (cuuint32_t)kBlockN, 1}, box_v_tail[3] = {64, (cuuint32_t)plan.tail_rows, 1};
        if (!encode_map(&tm_pk, a.prefix_k, 3, dims, str, box_k)) return cudaErrorInvalidValue;
        if (!encode_map(&tm_pv, a.prefix_v, 3, dims, str, box_v)) return cudaErrorInvalidValue;
        if (!encode_map(&tm_pk_tail, a.prefix_k, 3, dims, str, box_k_tail)) return cudaErrorInvalidValue;
        if (!encode_map(&tm_pv_tail, a.prefix_v, 3, dims, str, box_v_tail)) return cudaErrorInvalidValue;
    }
    PairParams p;
    memset(&p, 0, sizeof(p));
    p.lse = a.lse;
    p.status = status_word;
    p.args = a;
    p.sl2 = a.scale * kLog2e;
    p.B = dm.B; p.Hq = dm.Hq; p.Hkv = dm.Hkv; p.S = dm.S; p.P = dm.P; p.n_rep = dm.n_rep;
    p.Rg = Rg;
    p.seg_rows = plan.seg_rows;
    p.pt_per_group = plan.pt_per_group;
    p.total_pt = plan.pt_per_group * dm.Hkv;
    p.fd_ptpg.init(plan.pt_per_group);
    p.fd_Rg.init(Rg);
    p.fd_S.init(dm.S);
    p.fd_seg.init(plan.seg_rows);
    p.fd_chunkS.init(dm.S);
    p.nblk_p = plan.nblk_p;
    p.tail_rows = plan.tail_rows;
    p.nc = plan.nc;
    p.n_sfx = plan.n_sfx;
    p.chunk = plan.chunk;
    p.off_pk = plan.off_pk; p.off_pv = plan.off_pv; p.off_q = plan.off_q; p.off_sk = plan.off_sk;
    p.off_sv = plan.off_sv; p.off_stage = plan.off_stage; p.off_bar = plan.off_bar; p.off_misc = plan.off_misc;
    p.off_ml = plan.off_ml;
    p.sk_bytes = plan.sk_bytes;
    p.sv_bytes = plan.sv_bytes;

    static PerDeviceOnce attr_set;
    if (cudaError_t e = ensure_max_smem(tc_fwd_pair_kernel, attr_set); e != cudaSuccess) return e;
    const int pairs = even_grid(p.total_pt, sm_count() / 2);
    {
        KernelTiming timing(kKernelFwdTc, stream);
        tc_fwd_pair_kernel<<<2 * pairs, kThreads, plan.smem_bytes, stream>>>(tm_q, tm_out, tm_pk, tm_pv, tm_pk_tail,
                                                                            tm_pv_tail, tm_sk, tm_sv, p);
    }
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace pskv
