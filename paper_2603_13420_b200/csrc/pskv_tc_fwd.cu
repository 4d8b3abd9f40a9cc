// Fused shared-prefix attention forward for sm_100a (tcgen05 / TMEM / TMA).
//
// All B*(Hq/Hkv)*S query rows of one KV head form one long row list that is cut into tiles of
// up to 128 rows; each tile is one dense contraction against the single shared prefix K/V of
// that KV head (kept in shared memory across tiles when it fits, never copied per candidate,
// Sec. 4.2), followed by one block holding the suffix keys of the few candidates the tile
// touches (block-diagonal causal mask).  Scores go to tensor memory, one continued online
// softmax runs over prefix blocks and the suffix block (Eq. 2; equivalent to merging the two
// partial results by their log-sum-exp), probabilities go back to tensor memory as bf16 and are
// the A operand of the P*V contraction; `out` and `lse` are written once.
//
// Persistent CTA, one per SM, 24 warps:
//   warp 0      TMA producer, score side (Q tile, prefix K blocks, suffix K of the tile)
//   warp 1      tcgen05.mma issuer for the score blocks  S = Q K^T
//   warp 2      tcgen05.mma issuer for the value blocks  O += P V   (owns the TMEM allocation)
//   warp 3      TMA producer, value side (prefix V blocks, suffix V of the tile); TMA stores of `out`
//   warps 4-19  softmax, four warpgroups sharing each item by 32-column pieces (thread <-> query
//               row = TMEM lane)
//   warps 20-23 epilogue: O / row sum -> bf16 -> staging buffer, lse
// An "item" is one (tile, key block) pair; tensor memory holds three 128-column score slots (the
// bf16 probabilities of an item overwrite parts of its own slot) and the 128 columns of O.  Every
// wait is on an event produced by an earlier item of a role that never waits on the waiter, so
// no wait cycle can form; every wait is bounded.
//
// Three instantiations share this code (see the comment at the kernel): prefix streamed through
// rings, prefix resident in shared memory, and the suffix-ring mode, in which a tile is a run of
// whole candidates (or of rows inside one candidate) and the suffix keys follow the prefix through
// the same rings in as many blocks as it takes -- the mode of the decode-shaped operator, of
// suffixes beyond one key block and of the causal self-attention of a single sequence.
#include <string.h>

#include "pskv_common.cuh"
#include "pskv_rows.cuh"
#include "pskv_sm100.cuh"
#include "pskv_tc_common.cuh"

namespace pskv {
namespace {

using namespace sm100;

constexpr int kSlots = 3;      // score slots of 128 columns; an item's probabilities overwrite its own scores
constexpr int kGroups = 4;     // softmax warpgroups: one 32-column piece of every score block each
constexpr int kThreads = 32 * (4 + 4 * kGroups + 4);
constexpr int kOCol = kSlots * kBlockN;  // first tensor-memory column of O
// Probabilities are 2^(s * sl2) with no max subtracted; rows whose sum leaves
// [kMinRowSum, kMaxRowSum] are redone with max subtraction at the end of the kernel.
constexpr float kMaxRowSum = 1.2676506002282294e30f;   // 2^100
constexpr float kMinRowSum = 7.8886090522101181e-31f;  // 2^-100
constexpr int kMaxStages = 4;
constexpr int kMaxInstr = kMaxFusedInstructions;  // prefixes one launch can serve

enum : unsigned int {
    kErrProducerK = 0x101, kErrProducerV = 0x102, kErrMmaQk = 0x103, kErrMmaPv = 0x104,
    kErrSoftmax = 0x105, kErrEpilogue = 0x106, kErrAlign = 0x107
};

struct TcFwdParams {
    float *lse;
    unsigned int *status;
    FwdArgs args;         // the call's raw arguments, for the rows that are redone row by row
    float sl2;            // scale * log2(e)
    int B, Hq, Hkv, S, P, n_rep;
    int Rg;               // rows per candidate in one KV-head group: n_rep * S
    int tile_rows;        // rows of the flat row list per tile (<= 128, multiple of seg_rows)
    int seg_rows;         // rows per Q / out TMA box: gcd(Rg, tile_rows)
    int tiles_per_group;
    FastDiv fd_tpg, fd_Rg, fd_S, fd_seg;  // divisions by tiles_per_group, Rg, S, seg_rows
    int total_tiles;
    int nblk_p;           // prefix key blocks: ceil(P / 128)
    int tail_rows;        // rows held by the last prefix block (multiple of 16, <= 128)
    int resident;         // 1 when all prefix blocks of a KV head stay in shared memory
    int stages;           // streaming mode: stages of the prefix K and V rings
    int sfx_rows;         // rows of the suffix K / V buffers (multiple of 16, <= 128)
    int alias_stage;      // 1 when the output staging buffer shares its memory with the suffix V buffer
    int slab_stage;       // 1 when the staging buffer holds one 64-column slab: staged and stored a slab at a time
    int ml_mask;          // partial row sums are kept for ml_mask + 1 tiles (3, or 0 behind kBarMlFree)
    // suffix-ring mode (tiles of whole candidates, suffix keys in blocks through the K/V rings)
    const int *suffix_len;  // cached suffix tokens per candidate, or nullptr (= Skv)
    int Skv;              // rows of a candidate's suffix K/V buffer (S counts its query rows)
    int Spad;             // Skv rounded up to 8: rows a candidate takes inside a suffix block
    int cpb;              // candidates per suffix block: 128 / Spad
    FastDiv fd_cpb;
    int deal_by_cost;     // long suffixes: hand tiles to CTAs by cost rank instead of in contiguous ranges
    int long_sfx;         // 1: a tile lies inside ONE candidate and that candidate's suffix keys come in
                          //    128-key blocks (suffix caches or row groups beyond 128); 0: whole-candidate tiles
    // several instructions in one launch (Sec. 4.3): the candidates of instruction i are contiguous and use
    // prefix cache i of [n_instr][Hkv][P][d], whose first pad[i] rows are left padding
    int n_instr;          // 1: one shared prefix
    int rpi;              // rows of one instruction inside a KV head's row list (a multiple of tile_rows)
    FastDiv fd_rpi;
    int pad[kMaxInstr];
    // shared-memory carve-up (byte offsets from the 1024-byte aligned base)
    int off_pk, off_pv, off_q, off_sk, off_sv, off_stage, off_bar, off_misc, off_ml;
};

template <int D>
struct Cfg {
    static constexpr int kSlabs = D / 64;              // 64-column (128-byte) swizzle slabs per row
    static constexpr int kSlabBytes = kTileM * 128;    // a full slab: 128 rows x 128 bytes
    static constexpr int kTileBytes = kSlabs * kSlabBytes;
};

// barrier indices
enum {
    kBarQFull = 0,   // Q tile landed
    kBarQkFree,      // all score MMAs of a tile completed: Q and suffix-K buffers are free
    kBarSKFull,
    kBarSVFull,
    kBarSVFree,      // all value MMAs of a tile completed: suffix-V buffer is free
    kBarOFull,       // O of a tile is complete in tensor memory
    kBarOFree,       // epilogue has read O out (one arrival per softmax warp)
    kBarStageFull,   // the output tile is staged (one arrival per softmax warp)
    kBarStageFree,   // the TMA stores of that slab have read it
    kBarMlFree,      // the epilogue has read a tile's partial row sums (one arrival per epilogue warp)
    kBarSFull,                        // [kSlots] scores of an item are in tensor memory
    kBarPReady = kBarSFull + kSlots,  // [kSlots] probabilities written (one arrival per softmax warp)
    kBarPvDone = kBarPReady + kSlots, // [kSlots] value MMAs of an item completed
    kBarKFull = kBarPvDone + kSlots,  // [stages]
    kBarVFull = kBarKFull + kMaxStages,
    kBarKFree = kBarVFull + kMaxStages,
    kBarVFree = kBarKFree + kMaxStages,
    kNumBars = kBarVFree + kMaxStages
};
constexpr int kBarBytes = 512;
static_assert(kNumBars * 8 <= kBarBytes, "barrier area");

// rows held (and MMA N used) by prefix block k
__device__ __forceinline__ int prefix_block_rows(const TcFwdParams &p, int k)
{
    return k == p.nblk_p - 1 ? p.tail_rows : kBlockN;
}

constexpr int kPiece = 32;  // score columns a softmax thread handles per tensor-memory load
static_assert(kBlockN == 4 * kPiece, "two softmax groups x two pieces cover a score block");

// Suffix-ring mode: candidates [first, first + count) of a tile that suffix block j holds, and the
// MMA N (rows rounded up to 16) of that block.
__device__ __forceinline__ int sfx_block_cands(const TcFwdParams &p, int nc, int j)
{
    return min(p.cpb, nc - j * p.cpb);
}
__device__ __forceinline__ int sfx_block_rows(const TcFwdParams &p, int nc, int j)
{
    return (sfx_block_cands(p, nc, j) * p.Spad + 15) & ~15;
}

// Suffix-ring mode with long suffixes: the tile's rows belong to one candidate; it needs that
// candidate's suffix keys up to the last one any of its rows may see, in blocks of 128.
__device__ __forceinline__ int sfx_blocks_long(const TcFwdParams &p, const TileInfo &t)
{
    const int r0 = t.R0 - t.b_first * p.Rg;
    const int s0 = r0 - p.fd_S.div(r0) * p.S;  // query index of the tile's first row
    const int s_max = (s0 + t.rows > p.S) ? p.S - 1 : s0 + t.rows - 1;  // rows wrap into the next head
    const int pos = suffix_tokens(p.suffix_len, t.b_first, p.S, p.Skv) - p.S + s_max;
    return (pos >> 7) + 1;
}
// MMA N of long-suffix block j (its 128-row box is zero-filled past the end of the cache)
__device__ __forceinline__ int sfx_long_rows(const TcFwdParams &p, int j)
{
    return min(kBlockN, (p.Skv - j * kBlockN + 15) & ~15);
}

// MODE 1: all prefix blocks of a KV head stay in shared memory; MODE 0: they stream through rings,
// and the suffix keys of a tile sit in one block with buffers of its own; MODE 2 (suffix-ring): a
// tile is a run of whole candidates and their suffix keys follow the prefix through the same rings
// in as many blocks as it takes -- the mode of the decode-shaped operator, where a 128-row tile
// spans many candidates, and of full-suffix shapes the other two modes cannot tile.  A compile-time
// switch so that each launch carries only the code of its own mode.
template <int D, int MODE, bool MI>
__global__ void __launch_bounds__(kThreads, 1)
tc_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_out,
              const __grid_constant__ CUtensorMap tm_pk, const __grid_constant__ CUtensorMap tm_pv,
              const __grid_constant__ CUtensorMap tm_pk_tail, const __grid_constant__ CUtensorMap tm_pv_tail,
              const __grid_constant__ CUtensorMap tm_sk, const __grid_constant__ CUtensorMap tm_sv,
              const TcFwdParams p)
{
    using C = Cfg<D>;
    constexpr bool RES = MODE == 1;
    constexpr bool SR = MODE == 2;
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
    int *cta_redo = reinterpret_cast<int *>(smem + p.off_misc + 8);  // rows of this CTA's tiles to redo
    float *ml = reinterpret_cast<float *>(smem + p.off_ml);  // partial row sums [tile % 4][softmax group][128]

    if ((sbase & 1023u) != 0u) {  // the swizzled layouts need a 1024-byte aligned base
        if (tid == 0) atomicCAS(p.status, 0u, (unsigned int)kErrAlign);
        return;
    }

    // Zero the data area: rows that no TMA box ever writes (tile padding) must hold finite values,
    // because a zero probability times a NaN value row would still poison the accumulator.
    for (int i = tid; i < p.off_bar / 16; i += kThreads) reinterpret_cast<uint4 *>(smem)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
        for (int i = 0; i < kNumBars; ++i) {
            const bool all_sm = i >= kBarPReady && i < kBarPReady + kSlots;
            const bool epi = i == kBarOFree || i == kBarStageFull || i == kBarMlFree;
            mbar_init(bar(i), all_sm ? (uint32_t)(4 * kGroups) : epi ? 4u : 1u);
        }
        *abort_flag = 0;
        *cta_redo = 0;
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

    // Tiles of this CTA.  Normally a contiguous range (tiles are ordered KV head major, so the
    // resident prefix of a head serves a whole run).  With long suffixes a tile's cost grows with the
    // position of its rows inside the suffix (causal block skipping), so there -- when tiles do not
    // straddle heads and the suffix K/V of all candidates stays in L2 anyway -- the tiles are dealt out by cost: ranked from the last (longest) suffix
    // position down, round r hands ranks r*G .. r*G+G-1 to the CTAs in alternating direction (the
    // longest-first rule in closed form).
    const int t_begin = (int)((long long)blockIdx.x * p.total_tiles / gridDim.x);
    const int t_end = (int)((long long)(blockIdx.x + 1) * p.total_tiles / gridDim.x);
    const int G = (int)gridDim.x;
    const int n_sp = (SR && p.deal_by_cost) ? p.S / p.tile_rows : 1;  // tiles per head
    const bool dealt = n_sp > 1;
    auto rank_at = [&](int tl) { return tl * G + ((tl & 1) ? G - 1 - (int)blockIdx.x : (int)blockIdx.x); };
    auto tile_at = [&](int tl) {
        if (!dealt) return t_begin + tl;
        // rank -> (suffix position from the end, candidate, KV head, head inside the group)
        const int rank = rank_at(tl), M = p.B * p.Hkv * p.n_rep;
        const int spr = rank / M, m = rank - spr * M;
        const int b = m / (p.Hkv * p.n_rep), gh = m - b * (p.Hkv * p.n_rep);
        const int g = gh / p.n_rep, hr = gh - g * p.n_rep;
        return g * p.tiles_per_group + (b * p.n_rep + hr) * n_sp + (n_sp - 1 - spr);
    };
    const int n_rounds = (p.total_tiles + G - 1) / G;
    const int n_tiles = !dealt ? t_end - t_begin : (n_rounds - 1) + (rank_at(n_rounds - 1) < p.total_tiles ? 1 : 0);
    // items of a tile: prefix blocks + the suffix block(s)
    auto items_of = [&](const TileInfo &t) {
        return p.nblk_p + (!SR ? 1 : p.long_sfx ? sfx_blocks_long(p, t) : p.fd_cpb.div(t.nc + p.cpb - 1));
    };
    // A run of tiles that shares one prefix: a KV head, or (several instructions) one instruction's
    // candidates inside a KV head.  Runs are numbered in tile order; the resident prefix is reloaded at the
    // start of each run and the barrier parity of those loads follows the run number.
    auto inst_of = [&](const TileInfo &t) { return MI ? p.fd_rpi.div(t.R0) : 0; };
    auto run_of = [&](const TileInfo &t, int inst) { return MI ? t.g * p.n_instr + inst : t.g; };
    auto first_of_run = [&](const TileInfo &t, int inst) {
        return t.first_of_g || (MI && t.R0 == inst * p.rpi);
    };
    // First prefix block a tile works on: the blocks that hold nothing but left padding are skipped by
    // every role (the resident copy still holds them, so the block index stays absolute).
    auto first_block = [&](int inst) { return MI ? p.pad[inst] / kBlockN : 0; };
    int run_first;
    {
        const TileInfo t0 = tile_info(p, t_begin < p.total_tiles ? t_begin : 0, t_begin);
        run_first = run_of(t0, inst_of(t0));
    }
    const int sfx_slab = p.sfx_rows * 128;
    const int tail_slab = p.tail_rows * 128;

    // The producer and MMA warps run their loops with all 32 lanes (warp-uniform control flow and
    // addresses, so descriptors can live in uniform registers); one elected lane issues the
    // asynchronous instructions.
    const int role = warp;
    if (role == 0) {
        // ------------------------------------------------------------------ producer, score side
        if (lane == 0) {
            prefetch_tensormap(&tm_q);
            prefetch_tensormap(&tm_sk);
            if (p.P > 0) { prefetch_tensormap(&tm_pk); prefetch_tensormap(&tm_pk_tail); }
        }
        uint32_t kload = 0;  // streaming mode: prefix K blocks loaded so far
        bool ok = true;
#pragma unroll 1
        for (int tl = 0; tl < n_tiles && ok; ++tl) {
            const TileInfo t = tile_info(p, tile_at(tl), t_begin);
            // Everything the Q loads need is worked out before the wait, so that only the copy
            // instructions themselves follow it: the Q buffer is single, and the time from "last
            // score MMA of the previous tile done" to "Q of this tile requested" is exposed.
            // (Suffix-ring mode: one box per slab holds the tile's whole candidates; a box reaching
            // past the last candidate is filled with zeros and still counts its full size.)
            const int nseg = SR ? 1 : p.fd_seg.div(t.rows);  // one box per run of seg_rows rows
            int qb = p.fd_Rg.div(t.R0), qr = t.R0 - qb * p.Rg;
            const uint32_t q_bytes = (uint32_t)(nseg * C::kSlabs * p.seg_rows * 128);
            const uint32_t seg_bytes = (uint32_t)(p.seg_rows * 128);
            uint32_t q_dst = sbase + p.off_q;
            // While there is nothing else to do, ask for the NEXT tile's Q in L2: its load can only
            // be issued a tile from now, right when it is needed, and then finds the data close by.
            if (tl + 1 < n_tiles) {
                const TileInfo tn = tile_info(p, tile_at(tl + 1), t_begin);
                const int nseg_n = SR ? 1 : p.fd_seg.div(tn.rows);
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
            // Q, suffix K and (resident mode) the prefix K blocks are free once every score MMA of
            // the previous tile has completed
            ok = mbar_wait_warp(bar(kBarQkFree), (tl & 1) ^ 1, abort_flag, p.status, kErrProducerK);
            if (!ok) break;
            PSKV_TRACE_EVENT(1, tl);
            if (elect_one_sync()) {
                mbar_arrive_expect_tx(bar(kBarQFull), q_bytes);
#pragma unroll 1
                for (int s = 0; s < nseg; ++s) {
#pragma unroll
                    for (int sl = 0; sl < C::kSlabs; ++sl)
                        tma_load_4d(q_dst + sl * C::kSlabBytes, &tm_q, bar(kBarQFull), sl * 64, qr, t.g, qb);
                    q_dst += seg_bytes;
                    qr += p.seg_rows;  // boxes never straddle a candidate: seg_rows divides Rg
                    if (qr >= p.Rg) {
                        qr -= p.Rg;
                        ++qb;
                    }
                }
            }
            __syncwarp();
            const int inst = inst_of(t);
            const int ph = inst * p.Hkv + t.g;  // head index inside the prefix caches
            if (RES) {
                if (first_of_run(t, inst) && elect_one_sync()) {
#pragma unroll 1
                    for (int k = 0; k < p.nblk_p; ++k) {
                        const bool tail = k == p.nblk_p - 1;
                        const int slab = tail ? tail_slab : C::kSlabBytes;
                        mbar_arrive_expect_tx(bar(kBarKFull + k), (uint32_t)(C::kSlabs * slab));
#pragma unroll 1
                        for (int sl = 0; sl < C::kSlabs; ++sl)
                            tma_load_3d(sbase + p.off_pk + k * C::kTileBytes + sl * slab, tail ? &tm_pk_tail : &tm_pk,
                                        bar(kBarKFull + k), sl * 64, k * kBlockN, ph);
                    }
                }
                __syncwarp();
            } else {
#pragma unroll 1
                for (int k = first_block(inst); k < p.nblk_p; ++k) {
                    const uint32_t ks = kload % (uint32_t)p.stages;
                    ok = mbar_wait_warp(bar(kBarKFree + ks), ((kload / (uint32_t)p.stages) & 1) ^ 1, abort_flag,
                                        p.status, kErrProducerK);
                    if (!ok) break;
                    const bool tail = k == p.nblk_p - 1;
                    const int slab = tail ? tail_slab : C::kSlabBytes;
                    if (elect_one_sync()) {
                        mbar_arrive_expect_tx(bar(kBarKFull + ks), (uint32_t)(C::kSlabs * slab));
#pragma unroll 1
                        for (int sl = 0; sl < C::kSlabs; ++sl)
                            tma_load_3d(sbase + p.off_pk + ks * C::kTileBytes + sl * slab, tail ? &tm_pk_tail : &tm_pk,
                                        bar(kBarKFull + ks), sl * 64, k * kBlockN, ph);
                    }
                    __syncwarp();
                    ++kload;
                }
                if (!ok) break;
            }
            if (SR) {
                // suffix K of the tile's candidates, block by block through the ring: one box of
                // Skv rows per candidate, candidates Spad rows apart inside a block
                const int nbs = items_of(t) - p.nblk_p;
#pragma unroll 1
                for (int j = 0; j < nbs; ++j) {
                    const uint32_t ks = kload % (uint32_t)p.stages;
                    ok = mbar_wait_warp(bar(kBarKFree + ks), ((kload / (uint32_t)p.stages) & 1) ^ 1, abort_flag,
                                        p.status, kErrProducerK);
                    if (!ok) break;
                    if (p.long_sfx) {
                        // keys [128 j, 128 j + 128) of the tile's candidate; rows past the cache are zero-filled
                        if (elect_one_sync()) {
                            mbar_arrive_expect_tx(bar(kBarKFull + ks), (uint32_t)C::kTileBytes);
#pragma unroll 1
                            for (int sl = 0; sl < C::kSlabs; ++sl)
                                tma_load_4d(sbase + p.off_pk + ks * C::kTileBytes + sl * C::kSlabBytes, &tm_sk,
                                            bar(kBarKFull + ks), sl * 64, j * kBlockN, t.g, t.b_first);
                        }
                    } else {
                        const int ncb = sfx_block_cands(p, t.nc, j);
                        const int slab = sfx_block_rows(p, t.nc, j) * 128;
                        if (elect_one_sync()) {
                            mbar_arrive_expect_tx(bar(kBarKFull + ks), (uint32_t)(ncb * C::kSlabs * p.Skv * 128));
#pragma unroll 1
                            for (int c = 0; c < ncb; ++c)
#pragma unroll 1
                                for (int sl = 0; sl < C::kSlabs; ++sl)
                                    tma_load_4d(sbase + p.off_pk + ks * C::kTileBytes + sl * slab + c * p.Spad * 128,
                                                &tm_sk, bar(kBarKFull + ks), sl * 64, 0, t.g, t.b_first + j * p.cpb + c);
                        }
                    }
                    __syncwarp();
                    ++kload;
                }
                if (!ok) break;
            } else {
                // suffix K of the candidates this tile touches: one box per candidate
                if (elect_one_sync()) {
                    mbar_arrive_expect_tx(bar(kBarSKFull), (uint32_t)(t.nc * C::kSlabs * p.S * 128));
#pragma unroll 1
                    for (int c = 0; c < t.nc; ++c)
#pragma unroll 1
                        for (int sl = 0; sl < C::kSlabs; ++sl)
                            tma_load_4d(sbase + p.off_sk + sl * sfx_slab + c * p.S * 128, &tm_sk, bar(kBarSKFull),
                                        sl * 64, 0, t.g, t.b_first + c);
                }
                __syncwarp();
            }
        }
    } else if (role == 3) {
        // ------------------------------------------------------------------ producer, value side
        if (lane == 0) {
            prefetch_tensormap(&tm_sv);
            prefetch_tensormap(&tm_out);
            if (p.P > 0) { prefetch_tensormap(&tm_pv); prefetch_tensormap(&tm_pv_tail); }
        }
        // This warp also issues the TMA stores of each finished output tile.  The staging buffer
        // may share its shared memory with suffix V: tile t's output is staged after that tile's
        // last value MMA has read suffix V, and suffix V of tile t+1 is then fetched only once the
        // stores of tile t have read the staging buffer.
        const uint32_t stage = sbase + p.off_stage;
        uint32_t vload = 0;
        int store_slab = 0;  // slab_stage: slabs of the previous tile's output stored so far
        bool ok = true;
#pragma unroll 1
        for (int tl = 0; tl <= n_tiles && ok; ++tl) {
            const bool have_tile = tl < n_tiles;
            // Two jobs ride along with the prefix loads of tile tl: the stores of tile tl-1 (once it
            // is staged) and the fetch of this tile's suffix V (once its buffer is free: after those
            // stores when it doubles as the staging buffer, else after the previous tile's value MMAs).
            bool pend_store = tl > 0, pend_sv = have_tile && !SR;
            TileInfo t;
            int nk = 0;  // V blocks still to fetch through the ring for this tile
            int ph = 0;  // head index inside the prefix caches
            int kfirst = 0;
            if (have_tile) {
                t = tile_info(p, tile_at(tl), t_begin);
                const int inst = inst_of(t);
                ph = inst * p.Hkv + t.g;
                kfirst = first_block(inst);
                if (RES) {
                    // the resident prefix V blocks are free once every value MMA of the previous tile
                    // has completed
                    ok = mbar_wait_warp(bar(kBarSVFree), (tl & 1) ^ 1, abort_flag, p.status, kErrProducerV);
                    if (!ok) break;
                    if (first_of_run(t, inst) && elect_one_sync()) {
#pragma unroll 1
                        for (int k = 0; k < p.nblk_p; ++k) {
                            const bool tail = k == p.nblk_p - 1;
                            const int slab = tail ? tail_slab : C::kSlabBytes;
                            mbar_arrive_expect_tx(bar(kBarVFull + k), (uint32_t)(C::kSlabs * slab));
#pragma unroll 1
                            for (int sl = 0; sl < C::kSlabs; ++sl)
                                tma_load_3d(sbase + p.off_pv + k * C::kTileBytes + sl * slab,
                                            tail ? &tm_pv_tail : &tm_pv, bar(kBarVFull + k), sl * 64, k * kBlockN, ph);
                        }
                    }
                    __syncwarp();
                } else {
                    nk = SR ? items_of(t) : p.nblk_p;
                }
            }
            int k = nk > 0 ? kfirst : 0;  // (nk stays 0 when the prefix is resident)
#pragma unroll 1
            while (ok && (k < nk || pend_store || pend_sv)) {
                const bool block = k >= nk;  // nothing else left to do for this tile: wait for the jobs
                if (k < nk) {
                    const uint32_t vs = vload % (uint32_t)p.stages;
                    ok = mbar_wait_warp(bar(kBarVFree + vs), ((vload / (uint32_t)p.stages) & 1) ^ 1, abort_flag,
                                        p.status, kErrProducerV);
                    if (!ok) break;
                    if (SR && k >= p.nblk_p) {
                        // a suffix V block: one box of Skv rows per candidate, Spad rows apart
                        const int j = k - p.nblk_p;
                        if (p.long_sfx) {
                            if (elect_one_sync()) {
                                mbar_arrive_expect_tx(bar(kBarVFull + vs), (uint32_t)C::kTileBytes);
#pragma unroll 1
                                for (int sl = 0; sl < C::kSlabs; ++sl)
                                    tma_load_4d(sbase + p.off_pv + vs * C::kTileBytes + sl * C::kSlabBytes, &tm_sv,
                                                bar(kBarVFull + vs), sl * 64, j * kBlockN, t.g, t.b_first);
                            }
                        } else {
                            const int ncb = sfx_block_cands(p, t.nc, j);
                            const int slab = sfx_block_rows(p, t.nc, j) * 128;
                            if (elect_one_sync()) {
                                mbar_arrive_expect_tx(bar(kBarVFull + vs), (uint32_t)(ncb * C::kSlabs * p.Skv * 128));
#pragma unroll 1
                                for (int c = 0; c < ncb; ++c)
#pragma unroll 1
                                    for (int sl = 0; sl < C::kSlabs; ++sl)
                                        tma_load_4d(sbase + p.off_pv + vs * C::kTileBytes + sl * slab + c * p.Spad * 128,
                                                    &tm_sv, bar(kBarVFull + vs), sl * 64, 0, t.g,
                                                    t.b_first + j * p.cpb + c);
                            }
                        }
                    } else {
                        const bool tail = k == p.nblk_p - 1;
                        const int slab = tail ? tail_slab : C::kSlabBytes;
                        if (elect_one_sync()) {
                            mbar_arrive_expect_tx(bar(kBarVFull + vs), (uint32_t)(C::kSlabs * slab));
#pragma unroll 1
                            for (int sl = 0; sl < C::kSlabs; ++sl)
                                tma_load_3d(sbase + p.off_pv + vs * C::kTileBytes + sl * slab,
                                            tail ? &tm_pv_tail : &tm_pv, bar(kBarVFull + vs), sl * 64, k * kBlockN, ph);
                        }
                    }
                    __syncwarp();
                    ++vload;
                    ++k;
                }
                bool sv_ready = false;
                if (pend_sv && !p.alias_stage) {
                    if (tl == 0)
                        sv_ready = true;
                    else if (block)
                        sv_ready = ok = mbar_wait_warp(bar(kBarSVFree), (tl & 1) ^ 1, abort_flag, p.status, kErrProducerV);
                    else
                        sv_ready = __shfl_sync(0xffffffffu, mbar_try_wait(bar(kBarSVFree), (tl & 1) ^ 1) ? 1 : 0, 0) != 0;
                    if (!ok) break;
                }
                if (pend_store && !sv_ready) {
                    // the staging buffer holds the whole tile, or (slab_stage) one 64-column slab per round
                    const uint32_t round = p.slab_stage ? (uint32_t)((tl - 1) * C::kSlabs + store_slab) : (uint32_t)(tl - 1);
                    bool ready;
                    if (block)
                        ready = ok = mbar_wait_warp(bar(kBarStageFull), round & 1, abort_flag, p.status, kErrEpilogue);
                    else
                        ready = __shfl_sync(0xffffffffu, mbar_try_wait(bar(kBarStageFull), round & 1) ? 1 : 0, 0) != 0;
                    if (!ok) break;
                    if (ready) {
                        const TileInfo u = tile_info(p, tile_at(tl - 1), t_begin);
                        const int nseg = SR ? 1 : p.fd_seg.div(u.rows);  // (one box of whole candidates)
                        const int sl_first = p.slab_stage ? store_slab : 0;
                        const int sl_end = p.slab_stage ? store_slab + 1 : C::kSlabs;
                        if (elect_one_sync()) {
#pragma unroll 1
                            for (int sl = sl_first; sl < sl_end; ++sl)
#pragma unroll 1
                                for (int s = 0; s < nseg; ++s) {
                                    const int R = u.R0 + s * p.seg_rows;
                                    const int b = p.fd_Rg.div(R), r = R - b * p.Rg;
                                    tma_store_4d(&tm_out, stage + (p.slab_stage ? 0 : sl) * kStagingBytes + s * p.seg_rows * 128,
                                                 sl * 64, r, u.g, b);
                                }
                            tma_store_commit();
                            tma_store_wait_read();  // the staging buffer may be overwritten after this
                            mbar_arrive(bar(kBarStageFree));
                        }
                        __syncwarp();
                        PSKV_TRACE_EVENT(4, tl - 1);
                        if (p.slab_stage && store_slab + 1 < C::kSlabs) {
                            ++store_slab;
                        } else {
                            store_slab = 0;
                            pend_store = false;
                        }
                    }
                }
                if (pend_sv && p.alias_stage && !pend_store) sv_ready = true;
                if (sv_ready) {
                    if (elect_one_sync()) {
                        mbar_arrive_expect_tx(bar(kBarSVFull), (uint32_t)(t.nc * C::kSlabs * p.S * 128));
#pragma unroll 1
                        for (int c = 0; c < t.nc; ++c)
#pragma unroll 1
                            for (int sl = 0; sl < C::kSlabs; ++sl)
                                tma_load_4d(sbase + p.off_sv + sl * sfx_slab + c * p.S * 128, &tm_sv, bar(kBarSVFull),
                                            sl * 64, 0, t.g, t.b_first + c);
                    }
                    __syncwarp();
                    PSKV_TRACE_EVENT(5, tl);
                    pend_sv = false;
                }
            }
        }
        if (elect_one_sync()) tma_store_wait_all();
        __syncwarp();
    } else if (role == 1) {
        // ------------------------------------------------------------------ score MMAs: S = Q K^T
        int tl = 0;
        uint32_t kuse = 0;  // streaming mode: K blocks consumed from the ring
        TileInfo t = tile_info(p, tile_at(0), t_begin);
        int nitems = items_of(t);
        int kfirst = first_block(inst_of(t)), k = kfirst;
        const uint64_t q_desc = make_smem_desc(sbase + p.off_q, 0, 1024);
        bool ok = true;
        for (int i = 0; tl < n_tiles && ok; ++i) {
            const int slot = i % kSlots;
            // everything that does not depend on a wait comes first, so that it is out of the way
            // when the waits return
            uint32_t kaddr, kbar, kpar;
            int n, slab;
            bool kwait = true;
            if (k < p.nblk_p || SR) {
                n = k < p.nblk_p ? prefix_block_rows(p, k)
                    : p.long_sfx ? sfx_long_rows(p, k - p.nblk_p) : sfx_block_rows(p, t.nc, k - p.nblk_p);
                slab = (SR && p.long_sfx && k >= p.nblk_p) ? C::kSlabBytes : n * 128;  // (full 128-row boxes)
                if (RES) {
                    const int inst = inst_of(t);
                    kwait = first_of_run(t, inst);
                    kbar = bar(kBarKFull + k);
                    kpar = (uint32_t)(run_of(t, inst) - run_first) & 1u;
                    kaddr = sbase + p.off_pk + k * C::kTileBytes;
                } else {
                    const uint32_t ks = kuse % (uint32_t)p.stages;
                    kbar = bar(kBarKFull + ks);
                    kpar = (kuse / (uint32_t)p.stages) & 1u;
                    kaddr = sbase + p.off_pk + ks * C::kTileBytes;
                }
            } else {
                n = t.n_sfx;
                slab = sfx_slab;
                kbar = bar(kBarSKFull);
                kpar = (uint32_t)tl & 1u;
                kaddr = sbase + p.off_sk;
            }
            const uint32_t idesc = make_idesc_bf16(kTileM, n, 0);
            const uint32_t d_tmem = tmem + slot * kBlockN;
            const uint64_t k_desc = make_smem_desc(kaddr, 0, 1024);
            const uint64_t k_slab = (uint64_t)(slab >> 4);
            const bool last_of_tile = k == nitems - 1;
            const bool free_stage = (k < p.nblk_p || SR) && !RES;
            // the slot is free once the value MMAs of item i-3 (which read P from it) have completed
            PSKV_TRACE_EVENT(16, i);
            ok = mbar_wait_warp(bar(kBarPvDone + slot), ((i / kSlots) & 1) ^ 1, abort_flag, p.status, kErrMmaQk);
            if (!ok) break;
            PSKV_TRACE_EVENT(18, i);
            if (k == kfirst) {
                ok = mbar_wait_warp(bar(kBarQFull), tl & 1, abort_flag, p.status, kErrMmaQk);
                if (!ok) break;
            }
            if (kwait) {
                ok = mbar_wait_warp(kbar, kpar, abort_flag, p.status, kErrMmaQk);
                if (!ok) break;
            }
            if (MI && RES && k == kfirst && first_of_run(t, inst_of(t))) {
                // The resident copy of a run always loads every prefix block, also those this run skips as
                // padding.  Nobody multiplies them, so their loads are waited for here: a load must have
                // landed before its buffer and barrier are armed again for the next run, and before the
                // CTA exits.
                const uint32_t par = (uint32_t)(run_of(t, inst_of(t)) - run_first) & 1u;
                for (int kk = 0; kk < kfirst && kk < p.nblk_p && ok; ++kk)
                    ok = mbar_wait_warp(bar(kBarKFull + kk), par, abort_flag, p.status, kErrMmaQk);
                if (!ok) break;
            }
            PSKV_TRACE_EVENT(10, i);
            tc_fence_after();
            if (elect_one_sync()) {
#pragma unroll
                for (int ks16 = 0; ks16 < D / 16; ++ks16) {
                    const uint64_t qoff = (uint64_t)(((ks16 >> 2) * C::kSlabBytes + (ks16 & 3) * 32) >> 4);
                    const uint64_t koff = (uint64_t)(ks16 >> 2) * k_slab + (uint64_t)(((ks16 & 3) * 32) >> 4);
                    mma_ss(d_tmem, q_desc + qoff, k_desc + koff, idesc, ks16 > 0 ? 1u : 0u);
                }
                tc_commit(bar(kBarSFull + slot));
                if (free_stage) tc_commit(bar(kBarKFree + (kuse % (uint32_t)p.stages)));
                if (last_of_tile) tc_commit(bar(kBarQkFree));  // the suffix block ends the tile's scores
            }
            __syncwarp();
            PSKV_TRACE_EVENT(12, i);
            if (free_stage) ++kuse;
            if (++k == nitems) {
                k = 0;
                if (++tl < n_tiles) {
                    t = tile_info(p, tile_at(tl), t_begin);
                    nitems = items_of(t);
                    k = kfirst = first_block(inst_of(t));
                }
            }
        }
    } else if (role == 2) {
        // ------------------------------------------------------------------ value MMAs: O += P V
        int tl = 0;
        uint32_t vuse = 0;
        TileInfo t = tile_info(p, tile_at(0), t_begin);
        int nitems = items_of(t);
        int kfirst = first_block(inst_of(t)), k = kfirst;
        const uint32_t idesc_pv = make_idesc_bf16(kTileM, D, 1);
        bool ok = true;
        for (int i = 0; tl < n_tiles && ok; ++i) {
            const int slot = i % kSlots;
            // everything that does not depend on a wait comes first
            uint32_t vaddr, vbar, vpar;
            int n, slab;
            bool vwait = true;
            if (k < p.nblk_p || SR) {
                n = k < p.nblk_p ? prefix_block_rows(p, k)
                    : p.long_sfx ? sfx_long_rows(p, k - p.nblk_p) : sfx_block_rows(p, t.nc, k - p.nblk_p);
                slab = (SR && p.long_sfx && k >= p.nblk_p) ? C::kSlabBytes : n * 128;  // (full 128-row boxes)
                if (RES) {
                    const int inst = inst_of(t);
                    vwait = first_of_run(t, inst);
                    vbar = bar(kBarVFull + k);
                    vpar = (uint32_t)(run_of(t, inst) - run_first) & 1u;
                    vaddr = sbase + p.off_pv + k * C::kTileBytes;
                } else {
                    const uint32_t vs = vuse % (uint32_t)p.stages;
                    vbar = bar(kBarVFull + vs);
                    vpar = (vuse / (uint32_t)p.stages) & 1u;
                    vaddr = sbase + p.off_pv + vs * C::kTileBytes;
                }
            } else {
                n = t.n_sfx;
                slab = sfx_slab;
                vbar = bar(kBarSVFull);
                vpar = (uint32_t)tl & 1u;
                vaddr = sbase + p.off_sv;
            }
            const uint32_t p_tmem = tmem + slot * kBlockN;  // bf16 pairs: 8 columns per 16 keys
            const uint64_t v_desc = make_smem_desc(vaddr, (uint32_t)slab, 1024);
            const int nk = n >> 4;
            const bool last_of_tile = k == nitems - 1;
            const bool free_stage = (k < p.nblk_p || SR) && !RES;
            const uint32_t acc0 = k > kfirst ? 1u : 0u;
            PSKV_TRACE_EVENT(17, i);
            ok = mbar_wait_warp(bar(kBarPReady + slot), (i / kSlots) & 1, abort_flag, p.status, kErrMmaPv);
            if (!ok) break;
            if (k == kfirst && tl > 0) {
                // O of the previous tile must have been read out by the epilogue warps
                PSKV_TRACE_EVENT(15, i);
                ok = mbar_wait_warp(bar(kBarOFree), (tl - 1) & 1, abort_flag, p.status, kErrMmaPv);
                if (!ok) break;
            }
            if (vwait) {
                PSKV_TRACE_EVENT(14, i);
                ok = mbar_wait_warp(vbar, vpar, abort_flag, p.status, kErrMmaPv);
                if (!ok) break;
            }
            if (MI && RES && k == kfirst && first_of_run(t, inst_of(t))) {  // (as for the K blocks above)
                const uint32_t par = (uint32_t)(run_of(t, inst_of(t)) - run_first) & 1u;
                for (int kk = 0; kk < kfirst && kk < p.nblk_p && ok; ++kk)
                    ok = mbar_wait_warp(bar(kBarVFull + kk), par, abort_flag, p.status, kErrMmaPv);
                if (!ok) break;
            }
            PSKV_TRACE_EVENT(11, i);
            tc_fence_after();
            if (elect_one_sync()) {
#pragma unroll
                for (int ks16 = 0; ks16 < kBlockN / 16; ++ks16) {
                    if (ks16 < nk)
                        mma_ts(tmem + kOCol, p_tmem + (ks16 >> 1) * kPiece + (ks16 & 1) * 8, v_desc + (uint64_t)(ks16 * (2048 >> 4)), idesc_pv,
                               ks16 > 0 ? 1u : acc0);
                }
                tc_commit(bar(kBarPvDone + slot));
                if (free_stage) tc_commit(bar(kBarVFree + (vuse % (uint32_t)p.stages)));
                if (last_of_tile) {
                    tc_commit(bar(kBarSVFree));
                    tc_commit(bar(kBarOFull));
                }
            }
            __syncwarp();
            PSKV_TRACE_EVENT(13, i);
            if (free_stage) ++vuse;
            if (++k == nitems) {
                k = 0;
                if (++tl < n_tiles) {
                    t = tile_info(p, tile_at(tl), t_begin);
                    nitems = items_of(t);
                    k = kfirst = first_block(inst_of(t));
                }
            }
        }
    } else if (warp < 4 + 4 * kGroups) {
        // ------------------------------------------------------------------ softmax warps (4..19)
        // Four warpgroups work on every item: the 128 score columns are four pieces of 32 and
        // group j takes piece j, so that each scheduler always has four independent softmax warps
        // to hide the others' tensor-memory and barrier latencies.  Each thread owns one query
        // row (tensor-memory lane): p = 2^(s * sl2), row sum, bf16 pairs written over the first
        // half of the piece they came from (a group only ever overwrites columns it has read
        // itself).  No running max is subtracted: bf16 and fp32 share an 8-bit exponent, so the
        // quotient O / l is exact to rounding for any row whose sum stays within [2^-100, 2^100];
        // a row outside that range (essentially never, it means logits beyond +-69 nats) is
        // redone with max subtraction by this CTA once its tiles are finished.  The groups share no
        // state; their partial row sums meet in the epilogue, which the same warps run for the
        // previous tile (group j normalises O columns [32j, 32j+32)) right after the first item
        // of the next one, when that tile's last value MMAs have long completed.
        const int wg = (warp - 4) >> 2;
        const int row = 32 * (warp & 3) + lane;
        const uint32_t lane_addr = (uint32_t)(32 * (warp & 3)) << 16;
        bool ok = true;
        float lsum = 0.f;
        int item = 0;  // items handled so far
#pragma unroll 1
        for (int tl = 0; tl < n_tiles && ok; ++tl) {
            const TileInfo t = tile_info(p, tile_at(tl), t_begin);
            const int nitems = items_of(t);
            int lo_sfx = 1, hi_sfx = 0;
            int k_own = p.nblk_p;  // suffix-ring mode: the item that holds this row's candidate
            if (row < t.rows) {
                const int R = t.R0 + row;
                const int b = p.fd_Rg.div(R), r = R - b * p.Rg;
                const int i = r - p.fd_S.div(r) * p.S;  // query index inside the candidate
                if (SR) {
                    // query i is suffix token L - S + i of its candidate: suffix keys 0 .. L - S + i
                    const int pos = suffix_tokens(p.suffix_len, b, p.S, p.Skv) - p.S + i;
                    if (p.long_sfx) {
                        lo_sfx = 0;
                        hi_sfx = pos;  // counted from the candidate's first key; block j starts at 128 j
                    } else {
                        const int c = b - t.b_first, j = p.fd_cpb.div(c);
                        k_own += j;
                        lo_sfx = (c - j * p.cpb) * p.Spad;
                        hi_sfx = lo_sfx + pos;
                    }
                } else {
                    lo_sfx = (b - t.b_first) * p.S;  // first suffix column of this row's candidate
                    hi_sfx = lo_sfx + i;             // causal: suffix keys 0..i
                }
            }
            lsum = 0.f;
            // several instructions: the first `pad` prefix keys of this tile's instruction are left padding
            const int pad = MI ? p.pad[inst_of(t)] : 0;
#pragma unroll 1
            for (int k = pad / kBlockN; k < nitems && ok; ++k, ++item) {
                {
                    const int slot = item % kSlots;
                    const uint32_t s_tmem = tmem + lane_addr + slot * kBlockN + wg * kPiece;
                    // valid columns of this row: [lo, hi].  Padding rows of a tile take part in prefix
                    // blocks like real rows (their scores are finite and never stored) and see no
                    // suffix key.
                    int n, lo, hi;
                    if (k < p.nblk_p) {
                        n = prefix_block_rows(p, k);
                        lo = max(0, pad - k * kBlockN);
                        hi = min(kBlockN, p.P - k * kBlockN) - 1;
                    } else if (SR && p.long_sfx) {
                        n = sfx_long_rows(p, k - p.nblk_p);
                        lo = lo_sfx;  // 0 for a real row, 1 (with hi 0 - ...: nothing visible) for padding
                        hi = lo_sfx == 0 ? hi_sfx - (k - p.nblk_p) * kBlockN : 0;
                    } else if (SR) {
                        n = sfx_block_rows(p, t.nc, k - p.nblk_p);
                        lo = k == k_own ? lo_sfx : 1;  // other candidates' blocks: nothing visible
                        hi = k == k_own ? hi_sfx : 0;
                    } else {
                        n = t.n_sfx;
                        lo = lo_sfx;
                        hi = hi_sfx;
                    }
                    const int c0 = wg * kPiece;  // first column of my piece
                    // my piece: 0 = not read by the value MMAs, 1 = no valid column for this warp
                    // (zeros), 2 = some columns masked, 3 = all columns valid for all rows
                    int kind = 0;
                    if (c0 < n) {
                        const bool all_valid = lo <= c0 && hi >= c0 + kPiece - 1;
                        const bool none_valid = hi < lo || hi < c0 || lo > c0 + kPiece - 1;
                        kind = __all_sync(0xffffffffu, all_valid) ? 3 : __all_sync(0xffffffffu, none_valid) ? 1 : 2;
                    }
                    PSKV_TRACE_EVENT(25, item);
                    ok = mbar_wait_warp(bar(kBarSFull + slot), (item / kSlots) & 1, abort_flag, p.status, kErrSoftmax);
                    if (!ok) break;
                    tc_fence_after();
                    PSKV_TRACE_EVENT(20, item);
                    if (kind != 0) {
                        uint32_t rr[kPiece], pk[kPiece / 2];
                        if (kind >= 2) {
                            tmem_ld32(s_tmem, rr);
                            tmem_wait_ld();
                        }
                        PSKV_TRACE_EVENT(21, item);
                        float ls0 = 0.f, ls1 = 0.f;
                        if (kind >= 2) {
                            // all exponentials first (independent, so they pipeline through the
                            // special-function unit), then sums and bf16 pairs
                            float e[kPiece];
#pragma unroll
                            for (int c = 0; c < kPiece; c += 2) {
                                float x0 = __uint_as_float(rr[c]), x1 = __uint_as_float(rr[c + 1]);
                                mul_f32x2(x0, x1, p.sl2);
                                e[c] = ex2_approx(x0);
                                e[c + 1] = ex2_approx(x1);
                            }
                            if (kind == 2) {
                                const unsigned span = (unsigned)(hi - lo);
                                const int base = c0 - lo;
                                const bool any_col = hi >= lo;
#pragma unroll
                                for (int c = 0; c < kPiece; ++c)
                                    e[c] = (any_col && (unsigned)(base + c) <= span) ? e[c] : 0.f;
                            }
                            float ls2 = 0.f, ls3 = 0.f;
#pragma unroll
                            for (int c = 0; c < kPiece / 4; ++c) {
                                add_f32x2(ls0, ls1, e[4 * c], e[4 * c + 1]);
                                add_f32x2(ls2, ls3, e[4 * c + 2], e[4 * c + 3]);
                                pk[2 * c] = pack_bf16x2(e[4 * c], e[4 * c + 1]);
                                pk[2 * c + 1] = pack_bf16x2(e[4 * c + 2], e[4 * c + 3]);
                            }
                            ls0 += ls2;
                            ls1 += ls3;
                        } else {
#pragma unroll
                            for (int c = 0; c < kPiece / 2; ++c) pk[c] = 0u;
                        }
                        lsum += ls0 + ls1;
                        tmem_st16(s_tmem, pk);
                    }
                    if (k == nitems - 1) {
                        // the tile's partial row sums go to the epilogue warps through shared memory (kept
                        // for four tiles, or for one: then the epilogue must have read the previous tile's)
                        if (p.ml_mask == 0 && tl > 0) {
                            ok = mbar_wait_warp(bar(kBarMlFree), (tl - 1) & 1, abort_flag, p.status, kErrSoftmax);
                            if (!ok) break;
                        }
                        ml[((tl & p.ml_mask) * kGroups + wg) * kTileM + row] = lsum;
                        __threadfence_block();
                    }
                    PSKV_TRACE_EVENT(23, item);
                    tmem_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(kBarPReady + slot));
                    PSKV_TRACE_EVENT(24, item);
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps (20..23)
        // O / l -> bf16 -> staging buffer (TMA-stored by warp 3); lse; rows to redo.  Thread <->
        // query row; the row sum is the sum of the four softmax groups' partial sums.
        const int ew = warp & 3;
        const int row = 32 * ew + lane;
        const uint32_t lane_addr = (uint32_t)(32 * ew) << 16;
        bool ok = true;
#pragma unroll 1
        for (int te = 0; te < n_tiles && ok; ++te) {
            const TileInfo u = tile_info(p, tile_at(te), t_begin);
            ok = mbar_wait_warp(bar(kBarOFull), te & 1, abort_flag, p.status, kErrEpilogue);
            if (!ok) break;
            PSKV_TRACE_EVENT(30, te);
            tc_fence_after();
            const float *mlt = ml + (te & p.ml_mask) * kGroups * kTileM + row;
            const float l = (mlt[0] + mlt[kTileM]) + (mlt[2 * kTileM] + mlt[3 * kTileM]);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarMlFree));
            const bool row_ok = l >= kMinRowSum && l <= kMaxRowSum;  // false for overflow (inf, NaN), underflow
            // staged values must be finite (the buffer may double as suffix V, whose padding rows
            // meet zero probabilities): rows that failed stage zeros, and are redone anyway
            const float inv = row_ok ? 1.f / l : 0.f;
            if (p.slab_stage) {
                // One 64-column slab at a time through a staging buffer of one slab: load, hand O back after
                // the last load, wait for the previous slab's stores to have read the buffer, stage, tell
                // the storing warp.  The buffer is this kernel's own: suffix V of the next tile is fetched
                // as soon as this tile's value MMAs have completed, not behind these stores.
#pragma unroll 1
                for (int sl = 0; sl < C::kSlabs; ++sl) {
                    const uint32_t round = (uint32_t)(te * C::kSlabs + sl);
                    uint32_t o0[kPiece], o1[kPiece];
                    tmem_ld32(tmem + lane_addr + kOCol + sl * 64, o0);
                    tmem_ld32(tmem + lane_addr + kOCol + sl * 64 + kPiece, o1);
                    tmem_wait_ld();
                    PSKV_TRACE_EVENT(34 + sl, te);
                    if (sl == C::kSlabs - 1) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar(kBarOFree));
                        PSKV_TRACE_EVENT(32, te);
                    }
                    ok = mbar_wait_warp(bar(kBarStageFree), (round & 1) ^ 1, abort_flag, p.status, kErrEpilogue);
                    if (!ok) break;
                    uint8_t *srow = smem + p.off_stage + row * 128;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint4 v;
                        v.x = pack_bf16x2(__uint_as_float(o0[8 * c]) * inv, __uint_as_float(o0[8 * c + 1]) * inv);
                        v.y = pack_bf16x2(__uint_as_float(o0[8 * c + 2]) * inv, __uint_as_float(o0[8 * c + 3]) * inv);
                        v.z = pack_bf16x2(__uint_as_float(o0[8 * c + 4]) * inv, __uint_as_float(o0[8 * c + 5]) * inv);
                        v.w = pack_bf16x2(__uint_as_float(o0[8 * c + 6]) * inv, __uint_as_float(o0[8 * c + 7]) * inv);
                        if (!row_ok) v = make_uint4(0, 0, 0, 0);
                        *reinterpret_cast<uint4 *>(srow + ((c ^ (row & 7)) << 4)) = v;
                    }
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint4 v;
                        v.x = pack_bf16x2(__uint_as_float(o1[8 * c]) * inv, __uint_as_float(o1[8 * c + 1]) * inv);
                        v.y = pack_bf16x2(__uint_as_float(o1[8 * c + 2]) * inv, __uint_as_float(o1[8 * c + 3]) * inv);
                        v.z = pack_bf16x2(__uint_as_float(o1[8 * c + 4]) * inv, __uint_as_float(o1[8 * c + 5]) * inv);
                        v.w = pack_bf16x2(__uint_as_float(o1[8 * c + 6]) * inv, __uint_as_float(o1[8 * c + 7]) * inv);
                        if (!row_ok) v = make_uint4(0, 0, 0, 0);
                        *reinterpret_cast<uint4 *>(srow + (((4 + c) ^ (row & 7)) << 4)) = v;
                    }
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(kBarStageFull));
                }
                if (!ok) break;
            } else {
            // the TMA stores of the previous tile must have read the staging buffer
                ok = mbar_wait_warp(bar(kBarStageFree), (te & 1) ^ 1, abort_flag, p.status, kErrEpilogue);
                if (!ok) break;
                PSKV_TRACE_EVENT(33, te);
                // one 64-column slab per round; O is free for the next tile's first value MMA as soon
                // as the last round's loads have returned
    #pragma unroll 1
                for (int sl = 0; sl < C::kSlabs; ++sl) {
                    uint32_t o0[kPiece], o1[kPiece];
                    tmem_ld32(tmem + lane_addr + kOCol + sl * 64, o0);
                    tmem_ld32(tmem + lane_addr + kOCol + sl * 64 + kPiece, o1);
                    tmem_wait_ld();
                    PSKV_TRACE_EVENT(34 + sl, te);
                    if (sl == C::kSlabs - 1) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar(kBarOFree));
                        PSKV_TRACE_EVENT(32, te);
                    }
                    // 128-byte rows, 16-byte chunks swizzled by the row
                    uint8_t *srow = smem + p.off_stage + sl * kStagingBytes + row * 128;
    #pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint4 v;
                        v.x = pack_bf16x2(__uint_as_float(o0[8 * c]) * inv, __uint_as_float(o0[8 * c + 1]) * inv);
                        v.y = pack_bf16x2(__uint_as_float(o0[8 * c + 2]) * inv, __uint_as_float(o0[8 * c + 3]) * inv);
                        v.z = pack_bf16x2(__uint_as_float(o0[8 * c + 4]) * inv, __uint_as_float(o0[8 * c + 5]) * inv);
                        v.w = pack_bf16x2(__uint_as_float(o0[8 * c + 6]) * inv, __uint_as_float(o0[8 * c + 7]) * inv);
                        if (!row_ok) v = make_uint4(0, 0, 0, 0);  // (inf or NaN accumulators times zero are not zero)
                        *reinterpret_cast<uint4 *>(srow + ((c ^ (row & 7)) << 4)) = v;
                    }
    #pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint4 v;
                        v.x = pack_bf16x2(__uint_as_float(o1[8 * c]) * inv, __uint_as_float(o1[8 * c + 1]) * inv);
                        v.y = pack_bf16x2(__uint_as_float(o1[8 * c + 2]) * inv, __uint_as_float(o1[8 * c + 3]) * inv);
                        v.z = pack_bf16x2(__uint_as_float(o1[8 * c + 4]) * inv, __uint_as_float(o1[8 * c + 5]) * inv);
                        v.w = pack_bf16x2(__uint_as_float(o1[8 * c + 6]) * inv, __uint_as_float(o1[8 * c + 7]) * inv);
                        if (!row_ok) v = make_uint4(0, 0, 0, 0);
                        *reinterpret_cast<uint4 *>(srow + (((4 + c) ^ (row & 7)) << 4)) = v;
                    }
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarStageFull));
            }
            const bool stored = row < u.rows;
            if (stored) {
                const int R = u.R0 + row;
                const int b = p.fd_Rg.div(R), r = R - b * p.Rg;
                const size_t grow = ((size_t)b * p.Hq + (size_t)u.g * p.n_rep) * p.S + r;
                p.lse[grow] = row_ok ? log2f(l) * kLn2 : __int_as_float(0x7fc00000);
            }
            const unsigned bad = __ballot_sync(0xffffffffu, stored && !row_ok);
            if (bad != 0u && lane == 0) atomicAdd(cta_redo, __popc(bad));
            PSKV_TRACE_EVENT(31, te);
        }
    }

    // ---------------------------------------------------------------------- teardown
    PSKV_TRACE_FLUSH;
    if (*abort_flag != 0) __nanosleep(20000);  // let copies and MMAs still in flight drain
    tc_fence_before();
    __syncthreads();
    if (warp == 2) tmem_dealloc(tmem, 512);
    // Rows whose sum left the safe range carry a NaN lse (and zeros in `out`): all warps of the CTA
    // now walk over its tiles and recompute those rows one warp per row with a running maximum.
    // Every role has finished, the stores of `out` have completed, so the data area of shared
    // memory is free: each warp stages its query row there.
    if (*cta_redo > 0 && *abort_flag == 0) {
        float *q_s = reinterpret_cast<float *>(smem) + warp * D;
#pragma unroll 1
        for (int tl = 0; tl < n_tiles; ++tl) {
            const TileInfo t = tile_info(p, tile_at(tl), t_begin);
#pragma unroll 1
            for (int r = warp; r < t.rows; r += kThreads / 32) {
                const int R = t.R0 + r;
                const int b = p.fd_Rg.div(R), rr = R - b * p.Rg;
                const long long grow = ((long long)b * p.Hq + (long long)t.g * p.n_rep) * p.S + rr;
                const float v = p.lse[grow];
                if (v != v) {
                    if (MI) {  // the row's own prefix cache, without its left padding
                        const int inst = inst_of(t), pd = p.pad[inst];
                        FwdArgs a2 = p.args;
                        const size_t off = ((size_t)inst * p.Hkv * p.P + (size_t)pd) * D;
                        a2.prefix_k += off;
                        a2.prefix_v += off;
                        a2.dims.P = p.P - pd;
                        fwd_row<D>(a2, grow, q_s, lane);
                    } else {
                        fwd_row<D>(p.args, grow, q_s, lane);
                    }
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------ host side

struct TilePlan {
    bool ok;
    int mode;   // kernel template MODE: 0 rings, 1 resident prefix, 2 suffix-ring
    int cbox, Spad, cpb;  // suffix-ring mode: candidates per tile, rows per candidate in a block, candidates per block
    int long_sfx;         // suffix-ring mode: tiles inside one candidate, its suffix keys in 128-key blocks
    int tile_rows, seg_rows, tiles_per_group, sfx_rows;
    int nblk_p, tail_rows, resident, stages, alias_stage, slab_stage, ml_tiles;
    int off_pk, off_pv, off_q, off_sk, off_sv, off_stage, off_bar, off_misc, off_ml, smem_bytes;
};

// Picks the rows per tile -- the largest multiple of 8 up to 128 such that the suffix keys of all
// candidates a tile can touch fit one 128-key block (candidates x S <= 128) -- and lays out shared
// memory: all prefix blocks of a KV head if they fit beside the other buffers (resident mode), else
// rings of 2..4 block stages.
// Suffix-ring mode: a tile is the largest run of whole candidates with at most 128 rows; the
// suffix keys follow the prefix blocks through K/V rings, 128 / Spad candidates per block.
TilePlan plan_suffix_ring(const Dims &dm)
{
    TilePlan pl;
    memset(&pl, 0, sizeof(pl));
    const int Rg = dm.n_rep * dm.S;
    pl.mode = 2;
    if (Rg > kTileM || dm.Skv > kBlockN) {
        // long suffixes: a tile is a run of rows inside one candidate (the largest divisor of its
        // row count that fits a tile), the candidate's suffix keys come in blocks of 128
        int rows = 0;
        for (int m = kTileM; m >= 16 && !rows; --m)
            if (Rg % m == 0) rows = m;
        if (!rows && Rg <= kTileM) rows = Rg;
        if (!rows) return pl;  // no usable divisor: the general kernels take the shape
        if ((long long)dm.B * (Rg / rows) > 2000000000ll) return pl;
        pl.long_sfx = 1;
        pl.Spad = 8;
        pl.cpb = 1;
        pl.cbox = 1;
        pl.tile_rows = pl.seg_rows = rows;
        pl.tiles_per_group = dm.B * (Rg / rows);
    } else {
        pl.Spad = round_up(dm.Skv, 8);
        pl.cpb = kBlockN / pl.Spad;
        const int cmax = kTileM / Rg < dm.B ? kTileM / Rg : dm.B;
        // Candidates per tile: as many as fit, unless a few less give every SM a tile (or one round of tiles
        // less): a CTA's time is its tiles times the key blocks of a tile.  With 512 candidates of one query row
        // x 4 heads, 32 per tile are 128 tiles of 18 blocks on 148 SMs, 30 per tile are 144 tiles of 17.
        const int sms = sm_count();
        const int nblk = (dm.P + kBlockN - 1) / kBlockN;
        long long best_cost = -1;
        pl.cbox = cmax;
        for (int c = cmax; c >= 1 && c >= cmax - 8; --c) {
            const long long tiles = (long long)dm.Hkv * ((dm.B + c - 1) / c);
            const long long rounds = (tiles + sms - 1) / sms;
            const long long cost = rounds * (nblk + (c + pl.cpb - 1) / pl.cpb);
            if (best_cost < 0 || cost < best_cost) {
                best_cost = cost;
                pl.cbox = c;
            }
        }
        pl.tile_rows = pl.seg_rows = Rg * pl.cbox;
        pl.tiles_per_group = (dm.B + pl.cbox - 1) / pl.cbox;
    }
    pl.nblk_p = (dm.P + kBlockN - 1) / kBlockN;
    pl.tail_rows = pl.nblk_p ? round_up(dm.P - (pl.nblk_p - 1) * kBlockN, 16) : 0;
    const int slabs = dm.d / 64;
    const int tile_bytes = slabs * kTileM * 128;
    const int ml_bytes = 4 * kGroups * kTileM * 4;
    const int stage_bytes = slabs * kStagingBytes;
    const int fixed = tile_bytes /*Q*/ + stage_bytes + ml_bytes + 64 + kBarBytes;
    int st = (kMaxSmem - fixed) / (2 * tile_bytes);
    if (st > kMaxStages) st = kMaxStages;
    if (st < 1) return pl;
    pl.stages = st;
    pl.off_pk = 0;
    pl.off_pv = st * tile_bytes;
    pl.off_q = 2 * st * tile_bytes;
    pl.off_sk = pl.off_sv = pl.off_stage = pl.off_q + tile_bytes;  // no suffix buffers of their own
    pl.off_bar = pl.off_stage + stage_bytes;
    pl.off_misc = pl.off_bar + kBarBytes;
    pl.off_ml = pl.off_misc + 64;
    pl.smem_bytes = pl.off_ml + ml_bytes;
    pl.ok = pl.smem_bytes <= kMaxSmem;
    return pl;
}

TilePlan plan_base(const Dims &dm)
{
    TilePlan pl;
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
    const int ml_bytes = 4 * kGroups * kTileM * 4;  // partial row sums of four tiles in flight
    const int stage_bytes = slabs * kStagingBytes;
    const int tail_area = ml_bytes + 64 /*misc*/ + kBarBytes;
    // The output staging buffer gets memory of its own when that costs neither the residency of
    // the prefix nor a ring stage; otherwise it shares the suffix V buffer (value-side producer).
    const int fixed_own = tile_bytes /*Q*/ + 2 * sfx_bytes + stage_bytes + tail_area;
    const int shared_sv = sfx_bytes > stage_bytes ? sfx_bytes : stage_bytes;
    const int fixed_shared = tile_bytes + sfx_bytes + shared_sv + tail_area;
    const int resident_bytes = pl.nblk_p ? (pl.nblk_p - 1) * tile_bytes + tail_bytes : 0;
    auto ring_stages = [&](int fixed) {
        const int st = (kMaxSmem - fixed) / (2 * tile_bytes);
        return st > kMaxStages ? kMaxStages : st;
    };
    int kv_bytes = 0;  // bytes of the prefix K area (the V area has the same size)
    if (pl.nblk_p <= kMaxStages && fixed_shared + 2 * resident_bytes <= kMaxSmem) {
        pl.resident = 1;
        pl.stages = pl.nblk_p;
        kv_bytes = resident_bytes;
        pl.alias_stage = fixed_own + 2 * resident_bytes <= kMaxSmem ? 0 : 1;
        // Sharing the staging buffer with suffix V chains the next tile's suffix V behind this tile's
        // stores.  A staging buffer of one 64-column slab, with the partial row sums kept for one tile
        // instead of four, may still fit beside everything else: then the output goes a slab at a time.
        const int ml_one = kGroups * kTileM * 4;
        const int fixed_slab = tile_bytes + 2 * sfx_bytes + kStagingBytes + ml_one + 64 + kBarBytes;
        if (pl.alias_stage && slabs == 2 && fixed_slab + 2 * resident_bytes <= kMaxSmem) {
            pl.alias_stage = 0;
            pl.slab_stage = 1;
            pl.ml_tiles = 1;
        }
    } else {
        const int st = ring_stages(fixed_shared);
        if (st < 1) return pl;  // does not fit: the general kernels take the shape
        pl.stages = st;
        kv_bytes = st * tile_bytes;
        pl.alias_stage = ring_stages(fixed_own) == st ? 0 : 1;
    }
    const int sv_bytes = pl.alias_stage ? shared_sv : sfx_bytes;
    pl.off_pk = 0;
    pl.off_pv = pl.off_pk + kv_bytes;
    pl.off_q = pl.off_pv + kv_bytes;
    pl.off_sk = pl.off_q + tile_bytes;
    pl.off_sv = pl.off_sk + sfx_bytes;
    pl.off_stage = pl.alias_stage ? pl.off_sv : pl.off_sv + sv_bytes;
    pl.off_bar = pl.off_stage + (pl.alias_stage ? sv_bytes : pl.slab_stage ? kStagingBytes : stage_bytes);
    pl.off_misc = pl.off_bar + kBarBytes;
    pl.off_ml = pl.off_misc + 64;
    pl.smem_bytes = pl.off_ml + (pl.ml_tiles == 1 ? ml_bytes / 4 : ml_bytes);
    pl.ok = pl.smem_bytes <= kMaxSmem;
    pl.mode = pl.resident ? 1 : 0;
    return pl;
}

// The full-suffix operator takes the tiling with the suffix in one block when it has one; the
// decode-shaped operator, and full-suffix shapes that tiling cannot take, go to suffix-ring mode.
TilePlan plan_tiles(const Dims &dm)
{
    if (dm.Skv == dm.S && !dm.ragged) {
        const TilePlan pl = plan_base(dm);
        if (pl.ok) return pl;
    }
    return plan_suffix_ring(dm);
}

template <int D>
cudaError_t launch(const FwdArgs &a, const TilePlan &plan, void *workspace, unsigned int *status_word,
                   cudaStream_t stream, int n_instr, const int *prefix_len)
{
    const Dims &dm = a.dims;
    const int Rg = dm.n_rep * dm.S;
    CUtensorMap tm_q, tm_out, tm_pk, tm_pv, tm_pk_tail, tm_pv_tail, tm_sk, tm_sv;
    memset(&tm_pk, 0, sizeof(tm_pk));
    memset(&tm_pv, 0, sizeof(tm_pv));
    memset(&tm_pk_tail, 0, sizeof(tm_pk_tail));
    memset(&tm_pv_tail, 0, sizeof(tm_pv_tail));
    {
        // q / out viewed as [B][Hkv][Rg][D]: the n_rep heads of a KV head are contiguous rows
        cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)Rg, (cuuint64_t)dm.Hkv, (cuuint64_t)dm.B};
        cuuint64_t str[3] = {(cuuint64_t)D * 2, (cuuint64_t)Rg * D * 2, (cuuint64_t)dm.Hkv * Rg * D * 2};
        cuuint32_t box[4] = {64, (cuuint32_t)plan.seg_rows, 1, 1};
        if (plan.mode == 2) {  // one box = the whole candidates of a tile, or the tile's rows of one candidate
            box[1] = (cuuint32_t)(plan.long_sfx ? plan.tile_rows : Rg);
            box[3] = (cuuint32_t)plan.cbox;
        }
        if (!encode_map(&tm_q, a.q, 4, dims, str, box)) return cudaErrorInvalidValue;
        if (!encode_map(&tm_out, a.out, 4, dims, str, box)) return cudaErrorInvalidValue;
    }
    {
        cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)dm.Skv, (cuuint64_t)dm.Hkv, (cuuint64_t)dm.B};
        cuuint64_t str[3] = {(cuuint64_t)D * 2, (cuuint64_t)dm.Skv * D * 2, (cuuint64_t)dm.Hkv * dm.Skv * D * 2};
        cuuint32_t box[4] = {64, (cuuint32_t)(plan.long_sfx ? kBlockN : dm.Skv), 1, 1};
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
    TcFwdParams p;
    p.lse = a.lse;
    p.status = status_word;
    p.args = a;
    p.sl2 = a.scale * kLog2e;
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
    p.resident = plan.resident;
    p.stages = plan.stages > 0 ? plan.stages : 1;
    p.sfx_rows = plan.sfx_rows;
    p.alias_stage = plan.alias_stage;
    p.slab_stage = plan.slab_stage;
    p.ml_mask = plan.ml_tiles == 1 ? 0 : 3;
    p.suffix_len = a.suffix_len;
    p.Skv = dm.Skv;
    p.Spad = plan.Spad > 0 ? plan.Spad : 8;
    p.cpb = plan.cpb > 0 ? plan.cpb : 1;
    p.fd_cpb.init(p.cpb);
    p.long_sfx = plan.long_sfx;
    p.n_instr = n_instr;
    p.rpi = dm.B / n_instr * Rg;
    p.fd_rpi.init(p.rpi > 0 ? p.rpi : 1);
    for (int i = 0; i < kMaxInstr; ++i) p.pad[i] = (n_instr > 1 && i < n_instr) ? dm.P - prefix_len[i] : 0;
    // Dealing by cost balances the causal skew but lets every CTA touch every candidate's suffix K/V
    // at several times; it pays when those tensors stay in L2 between the touches.
    p.deal_by_cost = plan.long_sfx && dm.S % plan.tile_rows == 0 && dm.S / plan.tile_rows > 1 &&
                     4.0 * dm.B * dm.Hkv * dm.Skv * D <= 48.0e6;
    p.off_pk = plan.off_pk; p.off_pv = plan.off_pv; p.off_q = plan.off_q; p.off_sk = plan.off_sk;
    p.off_sv = plan.off_sv; p.off_stage = plan.off_stage; p.off_bar = plan.off_bar; p.off_misc = plan.off_misc;
    p.off_ml = plan.off_ml;

    const bool mi = n_instr > 1;  // (never with the suffix-ring tiling)
    auto kernel = plan.mode == 2 ? tc_fwd_kernel<D, 2, false>
                  : plan.mode == 1 ? (mi ? tc_fwd_kernel<D, 1, true> : tc_fwd_kernel<D, 1, false>)
                                   : (mi ? tc_fwd_kernel<D, 0, true> : tc_fwd_kernel<D, 0, false>);
    static PerDeviceOnce attr_set[6];
    if (cudaError_t e = ensure_max_smem(kernel, attr_set[plan.mode + (mi ? 3 : 0)]); e != cudaSuccess) return e;
    const int grid = even_grid(p.total_tiles, sm_count());
    cudaError_t launch_err;
    {
        KernelTiming timing(kKernelFwdTc, stream);
        launch_err = launch_dependent(kernel, grid, kThreads, plan.smem_bytes, stream, tm_q, tm_out, tm_pk, tm_pv, tm_pk_tail,
                                      tm_pv_tail, tm_sk, tm_sv, p);
    }
    count_launches(1);
    return launch_err != cudaSuccess ? launch_err : cudaGetLastError();
}

}  // namespace

#ifdef PSKV_TRACE
// Debug builds only: copies the event trace of CTA 0 to the host (all warps' events concatenated).
extern "C" int pskv_debug_read_trace(long long *host, int max_events)
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

bool tc_fwd_supported(const Dims &dm)
{
    if (dm.d != 64 && dm.d != 128) return false;
    if ((long long)dm.B * dm.n_rep * dm.S > 2000000000ll) return false;  // flat row index fits an int
    const TilePlan pl = plan_tiles(dm);
    return pl.ok && (long long)pl.tiles_per_group * dm.Hkv <= 2000000000ll;  // ... and so does the tile index
}

size_t tc_fwd_workspace_bytes(const Dims &) { return 0; }

// One launch can serve several instructions when every tile lies inside one instruction's candidates (an
// instruction's rows in a KV head's row list are a whole number of tiles) and the tiles are the 128-row
// tiles with one suffix block each (not the suffix-ring tiling).
bool tc_fwd_fused_supported(const Dims &dm, int n_instr)
{
    if (n_instr < 2 || n_instr > kMaxFusedInstructions || dm.B % n_instr != 0 || dm.P < 1 || dm.Pstride != dm.P ||
        dm.ragged || !tc_fwd_supported(dm))
        return false;
    const TilePlan pl = plan_tiles(dm);
    return pl.ok && pl.mode != 2 && ((long long)(dm.B / n_instr) * dm.n_rep * dm.S) % pl.tile_rows == 0;
}

cudaError_t launch_tc_fwd(const FwdArgs &a, void *workspace, unsigned int *status_word, cudaStream_t stream,
                          int n_instr, const int *prefix_len)
{
    const TilePlan plan = plan_tiles(a.dims);
    if (!plan.ok) return cudaErrorInvalidValue;
    if (n_instr > 1 && (!prefix_len || !tc_fwd_fused_supported(a.dims, n_instr))) return cudaErrorInvalidValue;
    if (n_instr < 1) n_instr = 1;
    if (n_instr == 1 && cta_pairs_enabled() && tc_fwd_pair_supported(a.dims))
        return launch_tc_fwd_pair(a, status_word, stream);
    return a.dims.d == 128 ? launch<128>(a, plan, workspace, status_word, stream, n_instr, prefix_len)
                           : launch<64>(a, plan, workspace, status_word, stream, n_instr, prefix_len);
}

}  // namespace pskv
