// Shared-prefix attention backward, query side, for sm_100a (tcgen05 / TMEM / TMA):
//   dQ = scale * sum_j dS_j K_j   over the shared prefix keys and the visible suffix keys,
//   dS = P o (dP - D),  P = exp(S - lse),  S = scale Q K^T,  dP = dO V^T,  D = <dO, O>.
// The prefix K/V is frozen (Sec. 4.2): no gradient flows into it, so the prefix part costs three
// contractions per block instead of five.  Tiling, operand staging and roles mirror the forward
// kernel: 128-row tiles of the flat row list of a KV head, prefix blocks resident in shared memory
// when they fit, one suffix block per tile with the block-diagonal causal mask.
//
// Persistent CTA, one per SM, 24 warps:
//   warp 0      TMA producer: Q tile, prefix K blocks, suffix K
//   warp 1      tcgen05.mma issuer: S = Q K^T of every item
//   warp 2      tcgen05.mma issuer: dP = dO V^T of the next item, then dQ += dS K of the current one
//               (owns the TMEM allocation)
//   warp 3      TMA producer: dO tile, prefix V blocks, suffix V
//   warps 4-19  element-wise, four warpgroups sharing each item by 32-column pieces (thread <->
//               query row): dS = exp2(S*sl2 - lse2) * (dP - D) as bf16
//   warps 20-23 epilogue: dQ from tensor memory, * scale, bf16, staging, TMA store
// Tensor memory: two 128-column S slots (dS overwrites the first half of its own slot), one dP
// slot, and the 128 columns of dQ.  D comes from a streaming pre-pass, dK_suffix / dV_suffix from
// a kernel of their own behind this one.  Every wait is bounded.
#include <string.h>

#include "pskv_common.cuh"
#include "pskv_sm100.cuh"
#include "pskv_tc_common.cuh"

namespace pskv {
namespace {

using namespace sm100;

constexpr int kSlots = 2;
constexpr int kGroups = 4;   // element-wise warpgroups: one 32-column piece of every score block each
constexpr int kPiece = 32;
constexpr int kThreads = 32 * (4 + 4 * kGroups + 4);
constexpr int kDpCol = kSlots * kBlockN;
constexpr int kDqCol = kDpCol + kBlockN;
constexpr int kMaxStages = 4;
constexpr int kMaxInstr = kMaxFusedInstructions;  // prefixes one launch can serve

enum : unsigned int {
    kErrProdA = 0x201, kErrProdB = 0x202, kErrMmaS = 0x203, kErrMmaDq = 0x204, kErrElem = 0x205,
    kErrEpi = 0x206, kErrAlign = 0x207
};

struct TcBwdParams {
    const float *lse;      // [B*Hq*S] from the forward pass
    const float *row_dot;  // [B*Hq*S] D = <dout, out>
    unsigned int *status;
    float sl2;             // scale * log2(e)
    float scale;
    int B, Hq, Hkv, S, P, n_rep;
    int Rg, tile_rows, seg_rows, tiles_per_group, total_tiles;
    FastDiv fd_tpg, fd_Rg, fd_S, fd_seg;  // divisions by tiles_per_group, Rg, S, seg_rows
    int nblk_p, tail_rows, resident, stages_k, stages_v, sfx_rows;  // ring stages of prefix K / V (streaming mode)
    int off_pk, off_pv, off_q, off_do, off_sk, off_sv, off_stage, off_bar, off_misc;
    // several instructions in one launch (Sec. 4.3): the candidates of instruction i are contiguous and use
    // prefix cache i of [n_instr][Hkv][P][d], whose first pad[i] rows are left padding
    int n_instr;  // 1: one shared prefix
    int rpi;      // rows of one instruction inside a KV head's row list (a multiple of tile_rows)
    FastDiv fd_rpi;
    int pad[kMaxInstr];
};

template <int D>
struct Cfg {
    static constexpr int kSlabs = D / 64;
    static constexpr int kSlabBytes = kTileM * 128;
    static constexpr int kTileBytes = kSlabs * kSlabBytes;
};

enum {
    kBarQFull = 0,
    kBarQkFree,     // every S MMA of a tile completed: the Q buffer is free
    kBarDoFull,
    kBarDvFree,     // every dP MMA of a tile completed: dO, suffix V (and resident prefix V) are free
    kBarSKFull,
    kBarSVFull,
    kBarDqFull,     // every dQ MMA of a tile completed: dQ is final, suffix K (and resident prefix K) are free
    kBarDqFree,     // the epilogue has read dQ out (4 arrivals)
    kBarStageFull,  // (4 arrivals)
    kBarStageFree,
    kBarDpFull,     // dP of an item is in tensor memory
    kBarDpFree,     // the element-wise warps have read dP (4 arrivals)
    kBarSFull,                        // [kSlots]
    kBarDsReady = kBarSFull + kSlots, // [kSlots] dS written (4 arrivals)
    kBarDqDone = kBarDsReady + kSlots, // [kSlots] the dQ MMAs of an item completed: its S slot is free
    kBarKFull = kBarDqDone + kSlots,
    kBarVFull = kBarKFull + kMaxStages,
    kBarKFree = kBarVFull + kMaxStages,
    kBarVFree = kBarKFree + kMaxStages,
    kNumBars = kBarVFree + kMaxStages
};
constexpr int kBarBytes = 512;
static_assert(kNumBars * 8 <= kBarBytes, "barrier area");

__device__ __forceinline__ int prefix_block_rows(const TcBwdParams &p, int k)
{
    return k == p.nblk_p - 1 ? p.tail_rows : kBlockN;
}

// MODE bit 0: the prefix K blocks of a KV head stay in shared memory; bit 1: the prefix V blocks do
// (else they stream through rings).  A K block is needed through a whole item (the dQ MMA reads it
// after the element-wise stage), a V block only for its dP MMA, so when not both fit it is K that
// stays.  Compile-time, so that each launch carries only the code of its own mode.
template <int D, int MODE, bool MI>
__global__ void __launch_bounds__(kThreads, 1)
tc_bwd_dq_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_do,
                 const __grid_constant__ CUtensorMap tm_dq, const __grid_constant__ CUtensorMap tm_pk,
                 const __grid_constant__ CUtensorMap tm_pv, const __grid_constant__ CUtensorMap tm_pk_tail,
                 const __grid_constant__ CUtensorMap tm_pv_tail, const __grid_constant__ CUtensorMap tm_sk,
                 const __grid_constant__ CUtensorMap tm_sv, const TcBwdParams p)
{
    using C = Cfg<D>;
    constexpr bool RK = (MODE & 1) != 0, RV = (MODE & 2) != 0;
    extern __shared__ __align__(1024) uint8_t smem[];
    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
    PSKV_TRACE_DECL;
    grid_dep_launch();  // the next kernel of the stream may take over SMs as this one's CTAs exit
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + p.off_bar;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + p.off_misc + 4);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + p.off_misc);

    if ((sbase & 1023u) != 0u) {
        if (tid == 0) atomicCAS(p.status, 0u, (unsigned int)kErrAlign);
        return;
    }
    // padding rows of the operand buffers must hold finite values (0 * NaN would poison dQ)
    for (int i = tid; i < p.off_bar / 16; i += kThreads) reinterpret_cast<uint4 *>(smem)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
        for (int i = 0; i < kNumBars; ++i) {
            const bool epi = i == kBarDqFree || i == kBarStageFull;
            const bool elem = i == kBarDpFree || (i >= kBarDsReady && i < kBarDsReady + kSlots);
            mbar_init(bar(i), elem ? (uint32_t)(4 * kGroups) : epi ? 4u : 1u);
        }
        *abort_flag = 0;
        fence_barrier_init();
    }
    fence_proxy_async();
    __syncthreads();
    if (warp == 2) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    // everything above touched shared and tensor memory only: it may run under the tail of the kernel before
    grid_dep_wait();

    const int t_begin = (int)((long long)blockIdx.x * p.total_tiles / gridDim.x);
    const int t_end = (int)((long long)(blockIdx.x + 1) * p.total_tiles / gridDim.x);
    const int n_tiles = t_end - t_begin;
    const int nitems = p.nblk_p + 1;
    // A run of tiles that shares one prefix: a KV head, or (several instructions) one instruction's
    // candidates inside a KV head; resident prefix blocks are reloaded at the start of each run and the
    // barrier parity of those loads follows the run number.
    auto inst_of = [&](const TileInfo &t) { return MI ? p.fd_rpi.div(t.R0) : 0; };
    auto run_of = [&](const TileInfo &t, int inst) { return MI ? t.g * p.n_instr + inst : t.g; };
    auto first_of_run = [&](const TileInfo &t, int inst) { return t.first_of_g || (MI && t.R0 == inst * p.rpi); };
    int run_first;
    {
        const TileInfo t0 = tile_info(p, t_begin < p.total_tiles ? t_begin : 0, t_begin);
        run_first = run_of(t0, inst_of(t0));
    }
    // Several instructions (Sec. 4.3): the prefix of instruction i starts with pad[i] rows of left padding;
    // the key blocks that hold nothing else are left out of its tiles (their probabilities are all zero), so
    // the items of a tile are the blocks from first_block on, then the suffix block.
    auto first_block = [&](const TileInfo &t) { return MI ? p.pad[inst_of(t)] / kBlockN : 0; };
    auto count_items = [&]() {
        if (!MI) return n_tiles * nitems;
        int n = 0;
        for (int tl = 0; tl < n_tiles; ++tl) n += nitems - first_block(tile_info(p, t_begin + tl, t_begin));
        return n;
    };
    const int sfx_slab = p.sfx_rows * 128;
    const int tail_slab = p.tail_rows * 128;
    const uint32_t stages_k = (uint32_t)p.stages_k, stages_v = (uint32_t)p.stages_v;

    if (warp == 0) {
        // ------------------------------------------------------------------ producer: Q, K
        if (lane == 0) {
            prefetch_tensormap(&tm_q);
            prefetch_tensormap(&tm_sk);
            if (p.P > 0) { prefetch_tensormap(&tm_pk); prefetch_tensormap(&tm_pk_tail); }
        }
        uint32_t kload = 0;
        bool ok = true;
#pragma unroll 1
        for (int tl = 0; tl < n_tiles && ok; ++tl) {
            const TileInfo t = tile_info(p, t_begin + tl, t_begin);
            // while idle: ask for the next tile's Q in L2 (its load can only be issued a tile from
            // now, exactly when it is needed)
            if (tl + 1 < n_tiles) {
                const TileInfo tn = tile_info(p, t_begin + tl + 1, t_begin);
                const int nseg_n = p.fd_seg.div(tn.rows);
                int nb = p.fd_Rg.div(tn.R0), nr = tn.R0 - nb * p.Rg;
                if (elect_one_sync()) {
#pragma unroll 1
                    for (int s = 0; s < nseg_n; ++s) {
#pragma unroll
                        for (int sl = 0; sl < C::kSlabs; ++sl) tma_prefetch_4d(&tm_q, sl * 64, nr, tn.g, nb);
                        nr += p.seg_rows;
                        if (nr >= p.Rg) {
                            nr -= p.Rg;
                            ++nb;
                        }
                    }
                }
                __syncwarp();
            }
            // everything the Q loads need is worked out before the wait (the Q buffer is single)
            const int nseg = p.fd_seg.div(t.rows);
            int qb = p.fd_Rg.div(t.R0), qr = t.R0 - qb * p.Rg;
            uint32_t q_dst = sbase + p.off_q;
            ok = mbar_wait_warp(bar(kBarQkFree), (tl & 1) ^ 1, abort_flag, p.status, kErrProdA);
            if (!ok) break;
            if (elect_one_sync()) {
                mbar_arrive_expect_tx(bar(kBarQFull), (uint32_t)(nseg * C::kSlabs * p.seg_rows * 128));
#pragma unroll 1
                for (int s = 0; s < nseg; ++s) {
#pragma unroll
                    for (int sl = 0; sl < C::kSlabs; ++sl)
                        tma_load_4d(q_dst + sl * C::kSlabBytes, &tm_q, bar(kBarQFull), sl * 64, qr, t.g, qb);
                    q_dst += p.seg_rows * 128;
                    qr += p.seg_rows;  // boxes never straddle a candidate: seg_rows divides Rg
                    if (qr >= p.Rg) {
                        qr -= p.Rg;
                        ++qb;
                    }
                }
            }
            __syncwarp();
            if (!RK) {
#pragma unroll 1
                for (int k = first_block(t); k < p.nblk_p; ++k) {
                    const uint32_t ks = kload % stages_k;
                    ok = mbar_wait_warp(bar(kBarKFree + ks), ((kload / stages_k) & 1) ^ 1, abort_flag, p.status, kErrProdA);
                    if (!ok) break;
                    const bool tail = k == p.nblk_p - 1;
                    const int slab = tail ? tail_slab : C::kSlabBytes;
                    if (elect_one_sync()) {
                        mbar_arrive_expect_tx(bar(kBarKFull + ks), (uint32_t)(C::kSlabs * slab));
                        for (int sl = 0; sl < C::kSlabs; ++sl)
                            tma_load_3d(sbase + p.off_pk + ks * C::kTileBytes + sl * slab, tail ? &tm_pk_tail : &tm_pk,
                                        bar(kBarKFull + ks), sl * 64, k * kBlockN, inst_of(t) * p.Hkv + t.g);
                    }
                    __syncwarp();
                    ++kload;
                }
                if (!ok) break;
            }
            // suffix K (and resident prefix K) are read by the dQ MMAs too: free once dQ of the
            // previous tile is final
            if (tl > 0) {
                ok = mbar_wait_warp(bar(kBarDqFull), (tl - 1) & 1, abort_flag, p.status, kErrProdA);
                if (!ok) break;
            }
            if (RK && first_of_run(t, inst_of(t)) && elect_one_sync()) {
                for (int k = 0; k < p.nblk_p; ++k) {
                    const bool tail = k == p.nblk_p - 1;
                    const int slab = tail ? tail_slab : C::kSlabBytes;
                    mbar_arrive_expect_tx(bar(kBarKFull + k), (uint32_t)(C::kSlabs * slab));
                    for (int sl = 0; sl < C::kSlabs; ++sl)
                        tma_load_3d(sbase + p.off_pk + k * C::kTileBytes + sl * slab, tail ? &tm_pk_tail : &tm_pk,
                                    bar(kBarKFull + k), sl * 64, k * kBlockN, inst_of(t) * p.Hkv + t.g);
                }
            }
            __syncwarp();
            if (elect_one_sync()) {
                mbar_arrive_expect_tx(bar(kBarSKFull), (uint32_t)(t.nc * C::kSlabs * p.S * 128));
                for (int c = 0; c < t.nc; ++c)
                    for (int sl = 0; sl < C::kSlabs; ++sl)
                        tma_load_4d(sbase + p.off_sk + sl * sfx_slab + c * p.S * 128, &tm_sk, bar(kBarSKFull),
                                    sl * 64, 0, t.g, t.b_first + c);
            }
            __syncwarp();
        }
    } else if (warp == 3) {
        // ------------------------------------------------------------------ producer: dO, V
        if (lane == 0) {
            prefetch_tensormap(&tm_do);
            prefetch_tensormap(&tm_sv);
            if (p.P > 0) { prefetch_tensormap(&tm_pv); prefetch_tensormap(&tm_pv_tail); }
        }
        uint32_t vload = 0;
        bool ok = true;
#pragma unroll 1
        for (int tl = 0; tl < n_tiles && ok; ++tl) {
            const TileInfo t = tile_info(p, t_begin + tl, t_begin);
            if (tl + 1 < n_tiles) {  // the next tile's dO into L2, a tile ahead
                const TileInfo tn = tile_info(p, t_begin + tl + 1, t_begin);
                const int nseg_n = p.fd_seg.div(tn.rows);
                int nb = p.fd_Rg.div(tn.R0), nr = tn.R0 - nb * p.Rg;
                if (elect_one_sync()) {
#pragma unroll 1
                    for (int s = 0; s < nseg_n; ++s) {
#pragma unroll
                        for (int sl = 0; sl < C::kSlabs; ++sl) tma_prefetch_4d(&tm_do, sl * 64, nr, tn.g, nb);
                        nr += p.seg_rows;
                        if (nr >= p.Rg) {
                            nr -= p.Rg;
                            ++nb;
                        }
                    }
                }
                __syncwarp();
            }
            const int nseg = p.fd_seg.div(t.rows);
            int qb = p.fd_Rg.div(t.R0), qr = t.R0 - qb * p.Rg;
            uint32_t do_dst = sbase + p.off_do;
            ok = mbar_wait_warp(bar(kBarDvFree), (tl & 1) ^ 1, abort_flag, p.status, kErrProdB);
            if (!ok) break;
            if (elect_one_sync()) {
                mbar_arrive_expect_tx(bar(kBarDoFull), (uint32_t)(nseg * C::kSlabs * p.seg_rows * 128));
#pragma unroll 1
                for (int s = 0; s < nseg; ++s) {
#pragma unroll
                    for (int sl = 0; sl < C::kSlabs; ++sl)
                        tma_load_4d(do_dst + sl * C::kSlabBytes, &tm_do, bar(kBarDoFull), sl * 64, qr, t.g, qb);
                    do_dst += p.seg_rows * 128;
                    qr += p.seg_rows;
                    if (qr >= p.Rg) {
                        qr -= p.Rg;
                        ++qb;
                    }
                }
                if (RV && first_of_run(t, inst_of(t))) {
                    for (int k = 0; k < p.nblk_p; ++k) {
                        const bool tail = k == p.nblk_p - 1;
                        const int slab = tail ? tail_slab : C::kSlabBytes;
                        mbar_arrive_expect_tx(bar(kBarVFull + k), (uint32_t)(C::kSlabs * slab));
                        for (int sl = 0; sl < C::kSlabs; ++sl)
                            tma_load_3d(sbase + p.off_pv + k * C::kTileBytes + sl * slab, tail ? &tm_pv_tail : &tm_pv,
                                        bar(kBarVFull + k), sl * 64, k * kBlockN, inst_of(t) * p.Hkv + t.g);
                    }
                }
                mbar_arrive_expect_tx(bar(kBarSVFull), (uint32_t)(t.nc * C::kSlabs * p.S * 128));
                for (int c = 0; c < t.nc; ++c)
                    for (int sl = 0; sl < C::kSlabs; ++sl)
                        tma_load_4d(sbase + p.off_sv + sl * sfx_slab + c * p.S * 128, &tm_sv, bar(kBarSVFull),
                                    sl * 64, 0, t.g, t.b_first + c);
            }
            __syncwarp();
            if (!RV) {
#pragma unroll 1
                for (int k = first_block(t); k < p.nblk_p; ++k) {
                    const uint32_t vs = vload % stages_v;
                    ok = mbar_wait_warp(bar(kBarVFree + vs), ((vload / stages_v) & 1) ^ 1, abort_flag, p.status, kErrProdB);
                    if (!ok) break;
                    const bool tail = k == p.nblk_p - 1;
                    const int slab = tail ? tail_slab : C::kSlabBytes;
                    if (elect_one_sync()) {
                        mbar_arrive_expect_tx(bar(kBarVFull + vs), (uint32_t)(C::kSlabs * slab));
                        for (int sl = 0; sl < C::kSlabs; ++sl)
                            tma_load_3d(sbase + p.off_pv + vs * C::kTileBytes + sl * slab, tail ? &tm_pv_tail : &tm_pv,
                                        bar(kBarVFull + vs), sl * 64, k * kBlockN, inst_of(t) * p.Hkv + t.g);
                    }
                    __syncwarp();
                    ++vload;
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ S = Q K^T
        const int total_items = count_items();
        int tl = 0;
        uint32_t kuse = 0;
        TileInfo t = tile_info(p, t_begin, t_begin);
        int kf = first_block(t), k = kf;
        const uint64_t q_desc = make_smem_desc(sbase + p.off_q, 0, 1024);
        bool ok = true;
#pragma unroll 1
        for (int i = 0; i < total_items && ok; ++i) {
            const int slot = i % kSlots;
            const bool prefix = k < p.nblk_p;
            const int n = prefix ? prefix_block_rows(p, k) : t.n_sfx;
            const int slab = prefix ? n * 128 : sfx_slab;
            const bool last_of_tile = k == nitems - 1;
            const bool ring_k = prefix && !RK;
            const uint32_t idesc = make_idesc_bf16(kTileM, n, 0);
            const uint64_t slab16 = (uint64_t)(slab >> 4);
            // ---- S: the slot is free once the dQ MMAs of item i-2 have completed
            ok = mbar_wait_warp(bar(kBarDqDone + slot), ((i / kSlots) & 1) ^ 1, abort_flag, p.status, kErrMmaS);
            if (!ok) break;
            if (k == kf) ok = mbar_wait_warp(bar(kBarQFull), tl & 1, abort_flag, p.status, kErrMmaS);
            if (!ok) break;
            if (MI && RK && k == kf && first_of_run(t, inst_of(t))) {
                // the resident blocks this run leaves out were fetched with the others: pass their barriers
                // too, so that every block's barrier has completed once per run
                for (int kk = 0; kk < kf && kk < p.nblk_p && ok; ++kk)
                    ok = mbar_wait_warp(bar(kBarKFull + kk), (run_of(t, inst_of(t)) - run_first) & 1, abort_flag, p.status,
                                        kErrMmaS);
                if (!ok) break;
            }
            uint32_t kaddr;
            if (prefix) {
                if (RK) {
                    if (first_of_run(t, inst_of(t)))
                        ok = mbar_wait_warp(bar(kBarKFull + k), (run_of(t, inst_of(t)) - run_first) & 1, abort_flag,
                                            p.status, kErrMmaS);
                    kaddr = sbase + p.off_pk + k * C::kTileBytes;
                } else {
                    const uint32_t ks = kuse % stages_k;
                    ok = mbar_wait_warp(bar(kBarKFull + ks), (kuse / stages_k) & 1, abort_flag, p.status, kErrMmaS);
                    kaddr = sbase + p.off_pk + ks * C::kTileBytes;
                }
            } else {
                ok = mbar_wait_warp(bar(kBarSKFull), tl & 1, abort_flag, p.status, kErrMmaS);
                kaddr = sbase + p.off_sk;
            }
            if (!ok) break;
            PSKV_TRACE_EVENT(10, i);
            tc_fence_after();
            {
                const uint64_t k_desc = make_smem_desc(kaddr, 0, 1024);
                const uint32_t d_tmem = tmem + slot * kBlockN;
                if (elect_one_sync()) {
#pragma unroll
                    for (int ks16 = 0; ks16 < D / 16; ++ks16) {
                        const uint64_t qoff = (uint64_t)(((ks16 >> 2) * C::kSlabBytes + (ks16 & 3) * 32) >> 4);
                        const uint64_t koff = (uint64_t)(ks16 >> 2) * slab16 + (uint64_t)(((ks16 & 3) * 32) >> 4);
                        mma_ss(d_tmem, q_desc + qoff, k_desc + koff, idesc, ks16 > 0 ? 1u : 0u);
                    }
                    tc_commit(bar(kBarSFull + slot));
                    if (last_of_tile) tc_commit(bar(kBarQkFree));
                }
                __syncwarp();
            }
            if (ring_k) ++kuse;
            if (++k == nitems) {
                if (++tl < n_tiles) {
                    t = tile_info(p, t_begin + tl, t_begin);
                    kf = first_block(t);
                }
                k = kf;
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------ dP = dO V^T, dQ += dS K
        // This warp alternates: dP of item i+1 (its buffer comes free early in the element-wise
        // stage of item i), then dQ of item i (whose dS comes at the end of that stage).  The score
        // MMAs of warp 1 run beside both, so two threads keep the tensor pipe fed.
        const int total_items = count_items();
        int tl = 0;
        uint32_t kuse = 0;
        TileInfo t = tile_info(p, t_begin, t_begin);
        int kf = first_block(t), k = kf;
        const uint32_t idesc_dq = make_idesc_bf16(kTileM, D, 1);
        const uint64_t do_desc = make_smem_desc(sbase + p.off_do, 0, 1024);
        bool ok = true;
        // cursor of the dP stream
        int ptl = 0, pkf = kf, pk = kf;
        uint32_t vuse = 0;
        TileInfo pt = t;
        auto issue_dp = [&](int i) -> bool {
            const int tl = ptl, k = pk;
            const TileInfo &t = pt;
            const bool prefix = k < p.nblk_p;
            const int n = prefix ? prefix_block_rows(p, k) : t.n_sfx;
            const int slab = prefix ? n * 128 : sfx_slab;
            const bool last_of_tile = k == nitems - 1;
            const bool ring_v = prefix && !RV;
            const uint32_t idesc = make_idesc_bf16(kTileM, n, 0);
            const uint64_t slab16 = (uint64_t)(slab >> 4);
            bool ok = true;
                // ---- dP: its single slot is free once the element-wise warps have read item i-1
                ok = mbar_wait_warp(bar(kBarDpFree), (i & 1) ^ 1, abort_flag, p.status, kErrMmaDq);
                if (!ok) return false;
                if (k == pkf) ok = mbar_wait_warp(bar(kBarDoFull), tl & 1, abort_flag, p.status, kErrMmaDq);
                if (!ok) return false;
                if (MI && RV && k == pkf && first_of_run(t, inst_of(t))) {  // (as for the K blocks in warp 1)
                    for (int kk = 0; kk < pkf && kk < p.nblk_p && ok; ++kk)
                        ok = mbar_wait_warp(bar(kBarVFull + kk), (run_of(t, inst_of(t)) - run_first) & 1, abort_flag,
                                            p.status, kErrMmaDq);
                    if (!ok) return false;
                }
                uint32_t vaddr;
                if (prefix) {
                    if (RV) {
                        if (first_of_run(t, inst_of(t)))
                            ok = mbar_wait_warp(bar(kBarVFull + k), (run_of(t, inst_of(t)) - run_first) & 1, abort_flag,
                                                p.status, kErrMmaDq);
                        vaddr = sbase + p.off_pv + k * C::kTileBytes;
                    } else {
                        const uint32_t vs = vuse % stages_v;
                        ok = mbar_wait_warp(bar(kBarVFull + vs), (vuse / stages_v) & 1, abort_flag, p.status, kErrMmaDq);
                        vaddr = sbase + p.off_pv + vs * C::kTileBytes;
                    }
                } else {
                    ok = mbar_wait_warp(bar(kBarSVFull), tl & 1, abort_flag, p.status, kErrMmaDq);
                    vaddr = sbase + p.off_sv;
                }
                if (!ok) return false;
                PSKV_TRACE_EVENT(12, i);
                tc_fence_after();
                {
                    const uint64_t v_desc = make_smem_desc(vaddr, 0, 1024);
                    if (elect_one_sync()) {
#pragma unroll
                        for (int ks16 = 0; ks16 < D / 16; ++ks16) {
                            const uint64_t aoff = (uint64_t)(((ks16 >> 2) * C::kSlabBytes + (ks16 & 3) * 32) >> 4);
                            const uint64_t voff = (uint64_t)(ks16 >> 2) * slab16 + (uint64_t)(((ks16 & 3) * 32) >> 4);
                            mma_ss(tmem + kDpCol, do_desc + aoff, v_desc + voff, idesc, ks16 > 0 ? 1u : 0u);
                        }
                        tc_commit(bar(kBarDpFull));
                        if (ring_v) tc_commit(bar(kBarVFree + (vuse % stages_v)));
                        if (last_of_tile) tc_commit(bar(kBarDvFree));
                    }
                    __syncwarp();
                }
            if (!ok) return false;
            if (ring_v) ++vuse;
            if (++pk == nitems) {
                if (++ptl < n_tiles) {
                    pt = tile_info(p, t_begin + ptl, t_begin);
                    pkf = first_block(pt);
                }
                pk = pkf;
            }
            return true;
        };
        if (total_items > 0) ok = issue_dp(0);
#pragma unroll 1
        for (int i = 0; i < total_items && ok; ++i) {
            if (i + 1 < total_items) {
                ok = issue_dp(i + 1);
                if (!ok) break;
            }
            const int slot = i % kSlots;
            const bool prefix = k < p.nblk_p;
            const int n = prefix ? prefix_block_rows(p, k) : t.n_sfx;
            const int slab = prefix ? n * 128 : sfx_slab;
            const bool last_of_tile = k == nitems - 1;
            const bool ring = prefix && !RK;
            ok = mbar_wait_warp(bar(kBarDsReady + slot), (i / kSlots) & 1, abort_flag, p.status, kErrMmaDq);
            if (!ok) break;
            if (k == kf && tl > 0) {
                ok = mbar_wait_warp(bar(kBarDqFree), (tl - 1) & 1, abort_flag, p.status, kErrMmaDq);
                if (!ok) break;
            }
            uint32_t kaddr;
            if (prefix) kaddr = sbase + p.off_pk + (RK ? (uint32_t)k : kuse % stages_k) * C::kTileBytes;
            else kaddr = sbase + p.off_sk;
            PSKV_TRACE_EVENT(11, i);
            tc_fence_after();
            const uint32_t ds_tmem = tmem + slot * kBlockN;  // bf16 pairs: 8 columns per 16 keys
            const uint64_t k_desc = make_smem_desc(kaddr, (uint32_t)slab, 1024);  // K as [keys][d]: d contiguous
            const int nk = n >> 4;
            const uint32_t acc0 = k > kf ? 1u : 0u;
            if (elect_one_sync()) {
#pragma unroll
                for (int ks16 = 0; ks16 < kBlockN / 16; ++ks16) {
                    if (ks16 < nk)
                        mma_ts(tmem + kDqCol, ds_tmem + (ks16 >> 1) * kPiece + (ks16 & 1) * 8, k_desc + (uint64_t)(ks16 * (2048 >> 4)), idesc_dq,
                               ks16 > 0 ? 1u : acc0);
                }
                tc_commit(bar(kBarDqDone + slot));
                if (ring) tc_commit(bar(kBarKFree + (kuse % stages_k)));
                if (last_of_tile) tc_commit(bar(kBarDqFull));
            }
            __syncwarp();
            if (ring) ++kuse;
            if (++k == nitems) {
                if (++tl < n_tiles) {
                    t = tile_info(p, t_begin + tl, t_begin);
                    kf = first_block(t);
                }
                k = kf;
            }
        }
    } else if (warp < 4 + 4 * kGroups) {
        // ------------------------------------------------------------------ element-wise warps (4..19)
        // Four warpgroups share every item: the 128 score columns are four pieces of 32 and group j
        // takes piece j.  Thread <-> query row (tensor-memory lane).  Each thread pulls its piece
        // of S and of dP into registers, hands dP back at once (the next item's dP MMAs are
        // waiting for that buffer), then forms dS = 2^(S sl2 - lse2) (dP - D) and writes it as
        // bf16 pairs over the first half of the S piece it came from.
        const int wg = (warp - 4) >> 2;
        const int row = 32 * (warp & 3) + lane;
        const int c0 = wg * kPiece;  // first column of my piece
        const uint32_t my_tmem = tmem + ((uint32_t)(32 * (warp & 3)) << 16) + c0;
        int item = 0;
        bool ok = true;
#pragma unroll 1
        for (int tl = 0; tl < n_tiles && ok; ++tl) {
            const TileInfo t = tile_info(p, t_begin + tl, t_begin);
            const bool valid = row < t.rows;
            const int R = t.R0 + (valid ? row : 0);
            const int b = p.fd_Rg.div(R), r = R - b * p.Rg;
            const int sfx_lo = (b - t.b_first) * p.S;
            const int sfx_hi = sfx_lo + (r - p.fd_S.div(r) * p.S);
            const size_t grow = ((size_t)b * p.Hq + (size_t)t.g * p.n_rep) * p.S + r;
            // padding rows: lse = +inf makes every probability (and so every dS) zero
            const float neg_lse2 = valid ? -p.lse[grow] * kLog2e : -INFINITY;
            const float drow = valid ? p.row_dot[grow] : 0.f;
            const int pad = MI ? p.pad[inst_of(t)] : 0;
#pragma unroll 1
            for (int k = pad / kBlockN; k < nitems && ok; ++k, ++item) {
                const int slot = item % kSlots;
                int n, lo, hi;
                if (k < p.nblk_p) {
                    n = prefix_block_rows(p, k);
                    lo = max(0, pad - k * kBlockN);  // left padding of this tile's instruction
                    hi = min(kBlockN, p.P - k * kBlockN) - 1;
                } else {
                    n = t.n_sfx;
                    lo = valid ? sfx_lo : 1;
                    hi = valid ? sfx_hi : 0;
                }
                // my piece: 0 = not read by the dQ MMAs, 1 = no valid column for any row of this
                // warp (zeros), 2 = some columns masked, 3 = every column valid for every row
                int kind = 0;
                if (c0 < n) {
                    const bool all_valid = lo <= c0 && hi >= c0 + kPiece - 1;
                    const bool none_valid = hi < lo || hi < c0 || lo > c0 + kPiece - 1;
                    kind = __all_sync(0xffffffffu, all_valid) ? 3 : __all_sync(0xffffffffu, none_valid) ? 1 : 2;
                }
                const uint32_t s_tmem = my_tmem + slot * kBlockN;
                const uint32_t dp_tmem = my_tmem + kDpCol;

                ok = mbar_wait_warp(bar(kBarSFull + slot), (item / kSlots) & 1, abort_flag, p.status, kErrElem);
                if (!ok) break;
                ok = mbar_wait_warp(bar(kBarDpFull), item & 1, abort_flag, p.status, kErrElem);
                if (!ok) break;
                PSKV_TRACE_EVENT(20, item);
                tc_fence_after();
                // two halves of 16 columns; dP goes back as soon as the second half is in registers
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    constexpr int kHalf = kPiece / 2;
                    uint32_t rs[kHalf], rd[kHalf], pk[kHalf / 2];
                    if (kind >= 2) {
                        tmem_ld16(s_tmem + hf * kHalf, rs);
                        tmem_ld16(dp_tmem + hf * kHalf, rd);
                        tmem_wait_ld();
                    }
                    if (hf == 1) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar(kBarDpFree));
                    }
                    if (kind >= 2) {
                        float e[kHalf];
#pragma unroll
                        for (int c = 0; c < kHalf; c += 2) {
                            float x0 = __uint_as_float(rs[c]), x1 = __uint_as_float(rs[c + 1]);
                            fma_f32x2(x0, x1, p.sl2, neg_lse2);
                            e[c] = ex2_approx(x0);
                            e[c + 1] = ex2_approx(x1);
                        }
                        if (kind == 2) {
                            const unsigned span = (unsigned)(hi - lo);
                            const int base = c0 + hf * kHalf - lo;
                            const bool any_col = hi >= lo;
#pragma unroll
                            for (int c = 0; c < kHalf; ++c) e[c] = (any_col && (unsigned)(base + c) <= span) ? e[c] : 0.f;
                        }
#pragma unroll
                        for (int c = 0; c < kHalf / 2; ++c) {
                            float d0 = __uint_as_float(rd[2 * c]), d1 = __uint_as_float(rd[2 * c + 1]);
                            add_f32x2(d0, d1, -drow, -drow);
                            mul_f32x2(d0, d1, e[2 * c], e[2 * c + 1]);
                            pk[c] = pack_bf16x2(d0, d1);
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < kHalf / 2; ++c) pk[c] = 0u;
                    }
                    if (kind != 0) tmem_st8(s_tmem + hf * (kHalf / 2), pk);
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarDsReady + slot));
                PSKV_TRACE_EVENT(24, item);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps (20..23)
        const int ew = warp & 3;
        const int row = 32 * ew + lane;
        const uint32_t lane_addr = (uint32_t)(32 * ew) << 16;
        const uint32_t stage = sbase + p.off_stage;
        const bool issuer = warp == 4 + 4 * kGroups;
        if (issuer && lane == 0) prefetch_tensormap(&tm_dq);
        bool ok = true;
#pragma unroll 1
        for (int tl = 0; tl < n_tiles && ok; ++tl) {
            const TileInfo t = tile_info(p, t_begin + tl, t_begin);
            ok = mbar_wait_warp(bar(kBarDqFull), tl & 1, abort_flag, p.status, kErrEpi);
            if (!ok) break;
            tc_fence_after();
            const int nseg = p.fd_seg.div(t.rows);
            // dQ leaves tensor memory in two load round trips back to back (the first slab is scaled and packed
            // to bf16 in registers while the second one is on its way) and goes back to the MMA issuer right
            // after them: the first dQ MMAs of the next tile wait for exactly that, and with the first slab's
            // staging and stores between the two loads they waited 2 500-4 100 cycles a tile.
            uint32_t pk0[C::kSlabs > 1 ? 32 : 1];
            uint32_t o0[32], o1[32];
            tmem_ld32(tmem + lane_addr + kDqCol, o0);
            tmem_ld32(tmem + lane_addr + kDqCol + 32, o1);
            tmem_wait_ld();
            if (C::kSlabs > 1) {
#pragma unroll
                for (int c = 0; c < 16; ++c) {
                    pk0[c] = pack_bf16x2(__uint_as_float(o0[2 * c]) * p.scale, __uint_as_float(o0[2 * c + 1]) * p.scale);
                    pk0[16 + c] = pack_bf16x2(__uint_as_float(o1[2 * c]) * p.scale, __uint_as_float(o1[2 * c + 1]) * p.scale);
                }
                tmem_ld32(tmem + lane_addr + kDqCol + 64, o0);
                tmem_ld32(tmem + lane_addr + kDqCol + 96, o1);
                tmem_wait_ld();
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarDqFree));
#pragma unroll 1
            for (int sl = 0; sl < C::kSlabs; ++sl) {
                const uint32_t round = (uint32_t)(tl * C::kSlabs + sl);
                ok = mbar_wait_warp(bar(kBarStageFree), (round & 1) ^ 1, abort_flag, p.status, kErrEpi);
                if (!ok) break;
                uint8_t *srow = smem + p.off_stage + row * 128;
                if (C::kSlabs > 1 && sl == 0) {
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        *reinterpret_cast<uint4 *>(srow + ((c ^ (row & 7)) << 4)) =
                            make_uint4(pk0[4 * c], pk0[4 * c + 1], pk0[4 * c + 2], pk0[4 * c + 3]);
                } else {
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint4 v;
                        v.x = pack_bf16x2(__uint_as_float(o0[8 * c]) * p.scale, __uint_as_float(o0[8 * c + 1]) * p.scale);
                        v.y = pack_bf16x2(__uint_as_float(o0[8 * c + 2]) * p.scale, __uint_as_float(o0[8 * c + 3]) * p.scale);
                        v.z = pack_bf16x2(__uint_as_float(o0[8 * c + 4]) * p.scale, __uint_as_float(o0[8 * c + 5]) * p.scale);
                        v.w = pack_bf16x2(__uint_as_float(o0[8 * c + 6]) * p.scale, __uint_as_float(o0[8 * c + 7]) * p.scale);
                        *reinterpret_cast<uint4 *>(srow + ((c ^ (row & 7)) << 4)) = v;
                    }
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint4 v;
                        v.x = pack_bf16x2(__uint_as_float(o1[8 * c]) * p.scale, __uint_as_float(o1[8 * c + 1]) * p.scale);
                        v.y = pack_bf16x2(__uint_as_float(o1[8 * c + 2]) * p.scale, __uint_as_float(o1[8 * c + 3]) * p.scale);
                        v.z = pack_bf16x2(__uint_as_float(o1[8 * c + 4]) * p.scale, __uint_as_float(o1[8 * c + 5]) * p.scale);
                        v.w = pack_bf16x2(__uint_as_float(o1[8 * c + 6]) * p.scale, __uint_as_float(o1[8 * c + 7]) * p.scale);
                        *reinterpret_cast<uint4 *>(srow + (((4 + c) ^ (row & 7)) << 4)) = v;
                    }
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarStageFull));
                if (issuer) {
                    ok = mbar_wait_warp(bar(kBarStageFull), round & 1, abort_flag, p.status, kErrEpi);
                    if (!ok) break;
                    if (elect_one_sync()) {
                        for (int s = 0; s < nseg; ++s) {
                            const int R = t.R0 + s * p.seg_rows;
                            const int b = p.fd_Rg.div(R), r = R - b * p.Rg;
                            tma_store_4d(&tm_dq, stage + s * p.seg_rows * 128, sl * 64, r, t.g, b);
                        }
                        tma_store_commit();
                        tma_store_wait_read();
                        mbar_arrive(bar(kBarStageFree));
                    }
                    __syncwarp();
                }
            }
        }
        if (issuer && elect_one_sync()) tma_store_wait_all();
    }

    PSKV_TRACE_FLUSH;
    if (*abort_flag != 0) __nanosleep(20000);
    tc_fence_before();
    __syncthreads();
    if (warp == 2) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------------------ host side

struct BwdPlan {
    bool ok;
    int tile_rows, seg_rows, tiles_per_group, sfx_rows;
    int nblk_p, tail_rows, resident, stages_k, stages_v;
    int off_pk, off_pv, off_q, off_do, off_sk, off_sv, off_stage, off_bar, off_misc, smem_bytes;
};

BwdPlan plan_bwd(const Dims &dm)
{
    BwdPlan pl;
    memset(&pl, 0, sizeof(pl));
    int nc_best = 0;
    if (!pick_tile_rows(dm, &pl.tile_rows, &pl.seg_rows, &pl.tiles_per_group, &nc_best)) return pl;
    pl.sfx_rows = round_up(nc_best * dm.S, 16);
    pl.nblk_p = (dm.P + kBlockN - 1) / kBlockN;
    pl.tail_rows = pl.nblk_p ? round_up(dm.P - (pl.nblk_p - 1) * kBlockN, 16) : 0;
    const int slabs = dm.d / 64;
    const int tile_bytes = slabs * kTileM * 128;
    const int sfx_bytes = round_up(slabs * pl.sfx_rows * 128, 1024);
    const int tail_bytes = round_up(slabs * pl.tail_rows * 128, 1024);
    const int fixed = 2 * tile_bytes /*Q, dO*/ + 2 * sfx_bytes + kStagingBytes + kBarBytes + 64;
    const int resident_bytes = pl.nblk_p ? (pl.nblk_p - 1) * tile_bytes + tail_bytes : 0;
    int k_bytes = 0, v_bytes = 0;
    if (pl.nblk_p <= kMaxStages && fixed + 2 * resident_bytes <= kMaxSmem) {
        pl.resident = 3;  // K and V resident
        pl.stages_k = pl.stages_v = pl.nblk_p > 0 ? pl.nblk_p : 1;
        k_bytes = v_bytes = resident_bytes;
    } else if (pl.nblk_p <= kMaxStages && fixed + resident_bytes + tile_bytes <= kMaxSmem) {
        // K resident, V through a ring: a K block is needed through a whole item (its dQ MMA comes
        // after the element-wise stage), a V block only for its dP MMA
        pl.resident = 1;
        pl.stages_k = pl.nblk_p;
        int nv = (kMaxSmem - fixed - resident_bytes) / tile_bytes;
        pl.stages_v = nv > kMaxStages ? kMaxStages : nv;
        k_bytes = resident_bytes;
        v_bytes = pl.stages_v * tile_bytes;
    } else {
        // ring mode: K gets the larger share of the stages that fit, for the same reason
        int n = (kMaxSmem - fixed) / tile_bytes;
        if (n > 2 * kMaxStages) n = 2 * kMaxStages;
        if (n < 2) return pl;
        pl.stages_v = n >= 6 ? 2 : 1;
        pl.stages_k = n - pl.stages_v;
        if (pl.stages_k > kMaxStages) pl.stages_k = kMaxStages;
        k_bytes = pl.stages_k * tile_bytes;
        v_bytes = pl.stages_v * tile_bytes;
    }
    pl.off_pk = 0;
    pl.off_pv = k_bytes;
    pl.off_q = k_bytes + v_bytes;
    pl.off_do = pl.off_q + tile_bytes;
    pl.off_sk = pl.off_do + tile_bytes;
    pl.off_sv = pl.off_sk + sfx_bytes;
    pl.off_stage = pl.off_sv + sfx_bytes;
    pl.off_bar = pl.off_stage + kStagingBytes;
    pl.off_misc = pl.off_bar + kBarBytes;
    pl.smem_bytes = pl.off_misc + 64;
    pl.ok = pl.smem_bytes <= kMaxSmem;
    return pl;
}

template <int D>
cudaError_t launch(const BwdArgs &a, const BwdPlan &plan, unsigned int *status_word, cudaStream_t stream, int parts, int n_instr, const int *prefix_len)
{
    const Dims &dm = a.dims;
    const int Rg = dm.n_rep * dm.S;
    CUtensorMap tm_q, tm_do, tm_dq, tm_pk, tm_pv, tm_pk_tail, tm_pv_tail, tm_sk, tm_sv;
    memset(&tm_pk, 0, sizeof(tm_pk));
    memset(&tm_pv, 0, sizeof(tm_pv));
    memset(&tm_pk_tail, 0, sizeof(tm_pk_tail));
    memset(&tm_pv_tail, 0, sizeof(tm_pv_tail));
    {
        cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)Rg, (cuuint64_t)dm.Hkv, (cuuint64_t)dm.B};
        cuuint64_t str[3] = {(cuuint64_t)D * 2, (cuuint64_t)Rg * D * 2, (cuuint64_t)dm.Hkv * Rg * D * 2};
        cuuint32_t box[4] = {64, (cuuint32_t)plan.seg_rows, 1, 1};
        if (!encode_map(&tm_q, a.q, 4, dims, str, box)) return cudaErrorInvalidValue;
        if (!encode_map(&tm_do, a.dout, 4, dims, str, box)) return cudaErrorInvalidValue;
        if (!encode_map(&tm_dq, a.dq, 4, dims, str, box)) return cudaErrorInvalidValue;
    }
    {
        cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)dm.S, (cuuint64_t)dm.Hkv, (cuuint64_t)dm.B};
        cuuint64_t str[3] = {(cuuint64_t)D * 2, (cuuint64_t)dm.S * D * 2, (cuuint64_t)dm.Hkv * dm.S * D * 2};
        cuuint32_t box[4] = {64, (cuuint32_t)dm.S, 1, 1};
        if (!encode_map(&tm_sk, a.suffix_k, 4, dims, str, box)) return cudaErrorInvalidValue;
        if (!encode_map(&tm_sv, a.suffix_v, 4, dims, str, box)) return cudaErrorInvalidValue;
    }
    if (dm.P > 0) {
        cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)dm.P, (cuuint64_t)dm.Hkv * (cuuint64_t)n_instr};
        cuuint64_t str[2] = {(cuuint64_t)D * 2, (cuuint64_t)dm.Pstride * D * 2};
        cuuint32_t box[3] = {64, (cuuint32_t)kBlockN, 1};
        cuuint32_t box_tail[3] = {64, (cuuint32_t)plan.tail_rows, 1};
        if (!encode_map(&tm_pk, a.prefix_k, 3, dims, str, box)) return cudaErrorInvalidValue;
        if (!encode_map(&tm_pv, a.prefix_v, 3, dims, str, box)) return cudaErrorInvalidValue;
        if (!encode_map(&tm_pk_tail, a.prefix_k, 3, dims, str, box_tail)) return cudaErrorInvalidValue;
        if (!encode_map(&tm_pv_tail, a.prefix_v, 3, dims, str, box_tail)) return cudaErrorInvalidValue;
    }
    TcBwdParams p;
    p.lse = a.lse;
    p.row_dot = a.row_dot;
    p.status = status_word;
    p.sl2 = a.scale * kLog2e;
    p.scale = a.scale;
    p.B = dm.B; p.Hq = dm.Hq; p.Hkv = dm.Hkv; p.S = dm.S; p.P = dm.P; p.n_rep = dm.n_rep;
    p.Rg = Rg;
    p.tile_rows = plan.tile_rows;
    p.seg_rows = plan.seg_rows;
    p.tiles_per_group = plan.tiles_per_group;
    p.fd_tpg.init(plan.tiles_per_group);
    p.fd_Rg.init(Rg);
    p.fd_S.init(dm.S);
    p.fd_seg.init(plan.seg_rows);
    p.total_tiles = plan.tiles_per_group * dm.Hkv;
    p.nblk_p = plan.nblk_p;
    p.tail_rows = plan.tail_rows;
    p.stages_k = plan.stages_k > 0 ? plan.stages_k : 1;
    p.stages_v = plan.stages_v > 0 ? plan.stages_v : 1;
    p.sfx_rows = plan.sfx_rows;
    p.off_pk = plan.off_pk; p.off_pv = plan.off_pv; p.off_q = plan.off_q; p.off_do = plan.off_do;
    p.off_sk = plan.off_sk; p.off_sv = plan.off_sv; p.off_stage = plan.off_stage; p.off_bar = plan.off_bar;
    p.off_misc = plan.off_misc;
    p.n_instr = n_instr;
    p.rpi = dm.B / n_instr * Rg;
    p.fd_rpi.init(p.rpi > 0 ? p.rpi : 1);
    for (int i = 0; i < kMaxInstr; ++i) p.pad[i] = (n_instr > 1 && i < n_instr) ? dm.P - prefix_len[i] : 0;

    const bool mi = n_instr > 1;
    auto kernel = plan.resident == 3 ? (mi ? tc_bwd_dq_kernel<D, 3, true> : tc_bwd_dq_kernel<D, 3, false>)
                  : plan.resident == 1 ? (mi ? tc_bwd_dq_kernel<D, 1, true> : tc_bwd_dq_kernel<D, 1, false>)
                                       : (mi ? tc_bwd_dq_kernel<D, 0, true> : tc_bwd_dq_kernel<D, 0, false>);
    static PerDeviceOnce attr_set[8];
    if (cudaError_t e0 = ensure_max_smem(kernel, attr_set[plan.resident + (mi ? 4 : 0)]); e0 != cudaSuccess) return e0;
    // The suffix-gradient kernel streams every dO row anyway, so where the shape allows it forms the row
    // statistic D = <dout, out> itself and runs FIRST (it then stands for both the "row statistic" and the
    // "suffix gradients" part); the query-side kernel behind it reads D.  Otherwise: a streaming pre-pass
    // for D, then dQ, then dK_suffix / dV_suffix.
    const bool d_in_dkv = tc_bwd_dkv_row_dot_supported(dm);
    cudaError_t e = cudaSuccess;
    if (parts & kBwdPartRowDot) {
        e = d_in_dkv ? launch_tc_bwd_dkv(a, status_word, stream, true) : launch_simt_row_dot(a, stream);
        if (e != cudaSuccess) return e;
    }
    if (parts & kBwdPartDq) {
        const int grid = even_grid(p.total_tiles, sm_count());
        {
            KernelTiming timing(kKernelBwdDqTc, stream);
            e = launch_dependent(kernel, grid, kThreads, plan.smem_bytes, stream, tm_q, tm_do, tm_dq, tm_pk, tm_pv,
                                 tm_pk_tail, tm_pv_tail, tm_sk, tm_sv, p);
        }
        count_launches(1);
        if (e == cudaSuccess) e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    if (!(parts & kBwdPartDkv)) return cudaSuccess;
    if (d_in_dkv) return cudaSuccess;  // done together with the row statistic (also for callers that ask part by part)
    if (tc_bwd_dkv_supported(dm)) return launch_tc_bwd_dkv(a, status_word, stream);
    return mma_bwd_dkv_supported(dm) ? launch_mma_bwd_dkv(a, stream) : launch_simt_bwd_dkv(a, stream);
}

}  // namespace

#ifdef PSKV_TRACE
// Debug builds only: copies this kernel's event trace of CTA 0 to the host.
extern "C" int pskv_debug_read_trace_dq(long long *host, int max_events)
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

bool tc_bwd_supported(const Dims &dm)
{
    if (dm.Skv != dm.S || dm.ragged) return false;  // full-suffix operator only
    if (dm.d != 64 && dm.d != 128) return false;
    if ((long long)dm.B * dm.n_rep * dm.S > 2000000000ll) return false;
    const BwdPlan pl = plan_bwd(dm);
    return pl.ok && (long long)pl.tiles_per_group * dm.Hkv <= 2000000000ll;
}

size_t tc_bwd_workspace_bytes(const Dims &dm) { return (size_t)dm.B * dm.Hq * dm.S * sizeof(float); }

// One launch can serve several instructions when an instruction's rows in a KV head's row list are a whole
// number of tiles (every tile then lies inside one instruction).
bool tc_bwd_fused_supported(const Dims &dm, int n_instr)
{
    if (n_instr < 2 || n_instr > kMaxFusedInstructions || dm.B % n_instr != 0 || dm.P < 1 || dm.Pstride != dm.P ||
        !tc_bwd_supported(dm))
        return false;
    const BwdPlan pl = plan_bwd(dm);
    return pl.ok && ((long long)(dm.B / n_instr) * dm.n_rep * dm.S) % pl.tile_rows == 0;
}

cudaError_t launch_tc_bwd(const BwdArgs &a, void *, unsigned int *status_word, cudaStream_t stream, int parts,
                          int n_instr, const int *prefix_len)
{
    const BwdPlan plan = plan_bwd(a.dims);
    if (!plan.ok) return cudaErrorInvalidValue;
    if (n_instr > 1 && (!prefix_len || !tc_bwd_fused_supported(a.dims, n_instr))) return cudaErrorInvalidValue;
    if (n_instr < 1) n_instr = 1;
    return a.dims.d == 128 ? launch<128>(a, plan, status_word, stream, parts, n_instr, prefix_len)
                           : launch<64>(a, plan, status_word, stream, parts, n_instr, prefix_len);
}

}  // namespace pskv
