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
// Persistent CTA, one per SM, 11 warps:
//   warp 0      TMA producer, score side (Q tile, prefix K blocks, suffix K of the tile)
//   warp 1      tcgen05.mma issuer; score blocks run up to three items ahead of P*V
//   warps 2-5   softmax: thread <-> query row (tensor-memory lane)
//   warps 6-9   epilogue: O from tensor memory, normalise, bf16, store; writes lse
//   warp 10     TMA producer, value side (prefix V blocks, suffix V of the tile)
// An "item" is one (tile, key block) pair; score blocks rotate through three 128-column slots of
// tensor memory, O has its own 128 columns.  The two producers wait only on completions of
// score-side resp. value-side MMAs of earlier items, so no wait cycle can form.
#include "pskv_common.cuh"
#include "pskv_sm100.cuh"

namespace pskv {
namespace {

using namespace sm100;

constexpr int kTileM = 128;    // rows of one MMA tile (tensor-memory lanes)
constexpr int kBlockN = 128;   // keys per block
constexpr int kSlots = 3;      // score slots in tensor memory
constexpr int kThreads = 352;
constexpr int kOCol = kSlots * kBlockN;  // first tensor-memory column of O
constexpr float kRescaleGap = 8.0f;      // log2 units the running max may lag before O is rescaled

// Optional event trace of CTA 0 (lane 0 of each warp, a private buffer per warp so that an event
// costs one clock read and two stores): compiled in only with -DPSKV_TRACE=<group mask>.
#ifdef PSKV_TRACE
constexpr int kTraceWarps = 11, kTraceCap = 4096;
__device__ long long g_trace[kTraceWarps * kTraceCap * 2];
__device__ unsigned int g_trace_n[kTraceWarps];
__device__ long long g_trace2[kTraceWarps * kTraceCap * 2];
__device__ unsigned int g_trace_n2[kTraceWarps];
#define PSKV_TRACE_DECL unsigned int trace_i_ = 0
#define PSKV_TRACE_EVENT(tag, val)                                                                     \
    do {                                                                                               \
        if (((PSKV_TRACE >> ((tag) / 10)) & 1) && blockIdx.x == 0 && (threadIdx.x & 31) == 0 &&        \
            trace_i_ < (unsigned int)kTraceCap) {                                                      \
            long long *e_ = g_trace + ((size_t)(threadIdx.x >> 5) * kTraceCap + trace_i_) * 2;         \
            e_[0] = clock64();                                                                         \
            e_[1] = ((long long)(tag) << 32) | (unsigned int)(val);                                    \
            ++trace_i_;                                                                                \
        }                                                                                              \
    } while (0)
#define PSKV_TRACE_EVENT_ONE(tag, val)                                                                 \
    do {                                                                                               \
        if (((PSKV_TRACE >> ((tag) / 10)) & 1) && blockIdx.x == 0) {                                   \
            unsigned int *n_ = &g_trace_n2[threadIdx.x >> 5];                                          \
            if (*n_ < (unsigned int)kTraceCap) {                                                       \
                long long *e_ = g_trace2 + ((size_t)(threadIdx.x >> 5) * kTraceCap + *n_) * 2;         \
                e_[0] = clock64();                                                                     \
                e_[1] = ((long long)(tag) << 32) | (unsigned int)(val);                                \
                *n_ += 1;                                                                              \
            }                                                                                          \
        }                                                                                              \
    } while (0)
#define PSKV_TRACE_FLUSH                                                                               \
    do {                                                                                               \
        if (blockIdx.x == 0 && (threadIdx.x & 31) == 0) g_trace_n[threadIdx.x >> 5] = trace_i_;        \
    } while (0)
#else
#define PSKV_TRACE_DECL do { } while (0)
#define PSKV_TRACE_EVENT_ONE(tag, val) do { } while (0)
#define PSKV_TRACE_FLUSH do { } while (0)
#define PSKV_TRACE_EVENT(tag, val) do { } while (0)
#endif

enum : unsigned int {
    kErrProducerK = 0x101, kErrProducerV = 0x102, kErrMma = 0x103, kErrSoftmax = 0x104,
    kErrEpilogue = 0x105, kErrAlign = 0x106
};

struct TcFwdParams {
    __nv_bfloat16 *out;
    float *lse;
    unsigned int *status;
    float sl2;            // scale * log2(e)
    int B, Hq, Hkv, S, P, n_rep;
    int Rg;               // rows per candidate in one KV-head group: n_rep * S
    int tile_rows;        // rows of the flat row list per tile (<= 128, multiple of seg_rows)
    int seg_rows;         // rows per Q TMA box: gcd(Rg, tile_rows)
    int tiles_per_group;
    int total_tiles;
    int nblk_p;           // prefix key blocks: ceil(P / 128)
    int resident;         // 1 when all prefix blocks of a KV head stay in shared memory
};

template <int D>
struct Cfg {
    static constexpr int kSlabs = D / 64;                 // 64-column (128-byte) swizzle slabs per row
    static constexpr int kSlabBytes = kTileM * 128;       // 128 rows x 128 bytes
    static constexpr int kTileBytes = kSlabs * kSlabBytes;
    static constexpr int kStages = (D == 128) ? 2 : 4;    // prefix K/V block stages
    static constexpr int kOffPK = 0;
    static constexpr int kOffPV = kStages * kTileBytes;
    static constexpr int kOffQ = 2 * kStages * kTileBytes;
    static constexpr int kOffSK = kOffQ + kTileBytes;
    static constexpr int kOffSV = kOffSK + kTileBytes;
    static constexpr int kDataBytes = kOffSV + kTileBytes;
    static constexpr int kOffBar = kDataBytes;            // mbarriers, 8 bytes each
    static constexpr int kOffMisc = kOffBar + 512;        // tmem base, abort flag
    static constexpr int kOffMl = kOffMisc + 64;          // float2 (l, lse2) [2][128]
    static constexpr int kSmemBytes = kOffMl + 2 * kTileM * 8;
};

// barrier indices
enum {
    kBarQFull = 0,   // Q tile landed
    kBarQkFree,      // all score MMAs of a tile completed: Q and suffix-K buffers are free
    kBarSKFull,
    kBarSVFull,
    kBarSVFree,      // all value MMAs of a tile completed: suffix-V buffer is free
    kBarOFull,       // O of a tile is complete in tensor memory
    kBarOFree,       // epilogue has read O out (4 arrivals)
    kBarSFull,                        // [kSlots] scores of an item are in tensor memory
    kBarPReady = kBarSFull + kSlots,  // [kSlots] probabilities written (4 arrivals)
    kBarPvDone = kBarPReady + kSlots, // [kSlots] value MMAs of an item completed
    kBarKFull = kBarPvDone + kSlots,  // [stages]
    kBarVFull = kBarKFull + 4,
    kBarKFree = kBarVFull + 4,
    kBarVFree = kBarKFree + 4,
    kNumBars = kBarVFree + 4
};
static_assert(kNumBars * 8 <= 512, "barrier area");

struct TileInfo {
    int g, R0, rows, b_first, nc, n_sfx;  // n_sfx: suffix columns rounded up to 16
    bool first_of_g;
};

__device__ __forceinline__ TileInfo tile_info(const TcFwdParams &p, int tile, int t_begin)
{
    TileInfo t;
    t.g = tile / p.tiles_per_group;
    const int tt = tile - t.g * p.tiles_per_group;
    t.first_of_g = (tt == 0) || (tile == t_begin);
    t.R0 = tt * p.tile_rows;
    const int total = p.B * p.Rg;
    t.rows = min(p.tile_rows, total - t.R0);
    t.b_first = t.R0 / p.Rg;
    const int b_last = (t.R0 + t.rows - 1) / p.Rg;
    t.nc = b_last - t.b_first + 1;
    t.n_sfx = (t.nc * p.S + 15) & ~15;
    return t;
}

__device__ __forceinline__ int prefix_block_cols(const TcFwdParams &p, int k)
{
    return min(kBlockN, (p.P - k * kBlockN + 15) & ~15);
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
tc_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_pk,
              const __grid_constant__ CUtensorMap tm_pv, const __grid_constant__ CUtensorMap tm_sk,
              const __grid_constant__ CUtensorMap tm_sv, const TcFwdParams p)
{
    using C = Cfg<D>;
    extern __shared__ __align__(1024) uint8_t smem[];
    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);  // warp-uniform by construction
    PSKV_TRACE_DECL;
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bar0 = sbase + C::kOffBar;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + C::kOffMisc + 4);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + C::kOffMisc);
    float2 *ml = reinterpret_cast<float2 *>(smem + C::kOffMl);

    if ((sbase & 1023u) != 0u) {  // the swizzled layouts need a 1024-byte aligned base
        if (tid == 0) atomicCAS(p.status, 0u, (unsigned int)kErrAlign);
        return;
    }

    // Zero the data area: rows that no TMA box ever writes (tile padding) must hold finite values,
    // because a zero probability times a NaN value row would still poison the accumulator.
    for (int i = tid; i < C::kDataBytes / 16; i += kThreads)
        reinterpret_cast<uint4 *>(smem)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) {
        for (int i = 0; i < kNumBars; ++i) {
            const bool four = (i >= kBarPReady && i < kBarPReady + kSlots) || i == kBarOFree;
            mbar_init(bar(i), four ? 4u : 1u);
        }
        *abort_flag = 0;
        fence_barrier_init();
    }
    fence_proxy_async();
    __syncthreads();
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // contiguous range of tiles for this CTA (tiles are ordered KV head major)
    const int t_begin = (int)((long long)blockIdx.x * p.total_tiles / gridDim.x);
    const int t_end = (int)((long long)(blockIdx.x + 1) * p.total_tiles / gridDim.x);
    const int n_tiles = t_end - t_begin;
    const int nitems = p.nblk_p + 1;  // prefix blocks + the suffix block
    const int g_first = t_begin / p.tiles_per_group;

    // The producer and MMA warps run their loops with all 32 lanes (warp-uniform control flow and
    // addresses, so descriptors can live in uniform registers); one elected lane issues the
    // asynchronous instructions.
    if (warp == 0) {
        // ------------------------------------------------------------------ producer, score side
        if (lane == 0) {
            prefetch_tensormap(&tm_q);
            prefetch_tensormap(&tm_sk);
            if (p.P > 0) prefetch_tensormap(&tm_pk);
        }
        uint32_t kload = 0;  // streaming mode: prefix K blocks loaded so far
        bool ok = true;
        for (int tl = 0; tl < n_tiles && ok; ++tl) {
            const TileInfo t = tile_info(p, t_begin + tl, t_begin);
            // Q, suffix K and (resident mode) the prefix K blocks are free once every score MMA of
            // the previous tile has completed
            ok = mbar_wait_warp(bar(kBarQkFree), (tl & 1) ^ 1, abort_flag, p.status, kErrProducerK);
            if (!ok) break;
            PSKV_TRACE_EVENT(1, tl);
            const int nseg = t.rows / p.seg_rows;  // one box per run of seg_rows rows
            if (elect_one_sync()) {
                mbar_arrive_expect_tx(bar(kBarQFull), (uint32_t)(nseg * C::kSlabs * p.seg_rows * 128));
                for (int s = 0; s < nseg; ++s) {
                    const int R = t.R0 + s * p.seg_rows;
                    const int b = R / p.Rg, r = R - b * p.Rg;
                    for (int sl = 0; sl < C::kSlabs; ++sl)
                        tma_load_4d(sbase + C::kOffQ + sl * C::kSlabBytes + s * p.seg_rows * 128, &tm_q,
                                    bar(kBarQFull), sl * 64, r, t.g, b);
                }
            }
            __syncwarp();
            if (p.resident) {
                if (t.first_of_g && elect_one_sync()) {
                    for (int k = 0; k < p.nblk_p; ++k) {
                        mbar_arrive_expect_tx(bar(kBarKFull + k), C::kTileBytes);
                        for (int sl = 0; sl < C::kSlabs; ++sl)
                            tma_load_3d(sbase + C::kOffPK + k * C::kTileBytes + sl * C::kSlabBytes, &tm_pk,
                                        bar(kBarKFull + k), sl * 64, k * kBlockN, t.g);
                    }
                }
                __syncwarp();
            } else {
                for (int k = 0; k < p.nblk_p; ++k) {
                    const uint32_t ks = kload % C::kStages;
                    ok = mbar_wait_warp(bar(kBarKFree + ks), ((kload / C::kStages) & 1) ^ 1, abort_flag, p.status,
                                        kErrProducerK);
                    if (!ok) break;
                    if (elect_one_sync()) {
                        mbar_arrive_expect_tx(bar(kBarKFull + ks), C::kTileBytes);
                        for (int sl = 0; sl < C::kSlabs; ++sl)
                            tma_load_3d(sbase + C::kOffPK + ks * C::kTileBytes + sl * C::kSlabBytes, &tm_pk,
                                        bar(kBarKFull + ks), sl * 64, k * kBlockN, t.g);
                    }
                    __syncwarp();
                    ++kload;
                }
                if (!ok) break;
            }
            // suffix K of the candidates this tile touches: one box per candidate
            if (elect_one_sync()) {
                mbar_arrive_expect_tx(bar(kBarSKFull), (uint32_t)(t.nc * C::kSlabs * p.S * 128));
                for (int c = 0; c < t.nc; ++c)
                    for (int sl = 0; sl < C::kSlabs; ++sl)
                        tma_load_4d(sbase + C::kOffSK + sl * C::kSlabBytes + c * p.S * 128, &tm_sk,
                                    bar(kBarSKFull), sl * 64, 0, t.g, t.b_first + c);
            }
            __syncwarp();
        }
    } else if (warp == 10) {
        // ------------------------------------------------------------------ producer, value side
        if (lane == 0) {
            prefetch_tensormap(&tm_sv);
            if (p.P > 0) prefetch_tensormap(&tm_pv);
        }
        uint32_t vload = 0;
        bool ok = true;
        for (int tl = 0; tl < n_tiles && ok; ++tl) {
            const TileInfo t = tile_info(p, t_begin + tl, t_begin);
            if (p.resident) {
                // suffix V and the resident prefix V blocks are free once every value MMA of the
                // previous tile has completed
                ok = mbar_wait_warp(bar(kBarSVFree), (tl & 1) ^ 1, abort_flag, p.status, kErrProducerV);
                if (!ok) break;
                if (t.first_of_g && elect_one_sync()) {
                    for (int k = 0; k < p.nblk_p; ++k) {
                        mbar_arrive_expect_tx(bar(kBarVFull + k), C::kTileBytes);
                        for (int sl = 0; sl < C::kSlabs; ++sl)
                            tma_load_3d(sbase + C::kOffPV + k * C::kTileBytes + sl * C::kSlabBytes, &tm_pv,
                                        bar(kBarVFull + k), sl * 64, k * kBlockN, t.g);
                    }
                }
                __syncwarp();
            } else {
                for (int k = 0; k < p.nblk_p; ++k) {
                    const uint32_t vs = vload % C::kStages;
                    ok = mbar_wait_warp(bar(kBarVFree + vs), ((vload / C::kStages) & 1) ^ 1, abort_flag, p.status,
                                        kErrProducerV);
                    if (!ok) break;
                    if (elect_one_sync()) {
                        mbar_arrive_expect_tx(bar(kBarVFull + vs), C::kTileBytes);
                        for (int sl = 0; sl < C::kSlabs; ++sl)
                            tma_load_3d(sbase + C::kOffPV + vs * C::kTileBytes + sl * C::kSlabBytes, &tm_pv,
                                        bar(kBarVFull + vs), sl * 64, k * kBlockN, t.g);
                    }
                    __syncwarp();
                    ++vload;
                }
                if (!ok) break;
                ok = mbar_wait_warp(bar(kBarSVFree), (tl & 1) ^ 1, abort_flag, p.status, kErrProducerV);
                if (!ok) break;
            }
            if (elect_one_sync()) {
                mbar_arrive_expect_tx(bar(kBarSVFull), (uint32_t)(t.nc * C::kSlabs * p.S * 128));
                for (int c = 0; c < t.nc; ++c)
                    for (int sl = 0; sl < C::kSlabs; ++sl)
                        tma_load_4d(sbase + C::kOffSV + sl * C::kSlabBytes + c * p.S * 128, &tm_sv,
                                    bar(kBarSVFull), sl * 64, 0, t.g, t.b_first + c);
            }
            __syncwarp();
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        const int total_items = n_tiles * nitems;
        int i_qk = 0, i_pv = 0;
        int tl_qk = 0, k_qk = 0, tl_pv = 0, k_pv = 0;  // (tile, block) of the next score / value item
        uint32_t kuse = 0, vuse = 0;                    // streaming mode: prefix blocks consumed
        TileInfo tq = tile_info(p, t_begin, t_begin), tv = tq;
        // descriptors are built once; per MMA only the 16-byte-granular start address moves
        const uint64_t q_desc = make_smem_desc(sbase + C::kOffQ, 0, 1024);
        const uint32_t idesc_pv = make_idesc_bf16(kTileM, D, 1);
        bool ok = true;
        while (ok && i_pv < total_items) {
            PSKV_TRACE_EVENT(16, i_pv);
            if (i_qk < total_items && i_qk < i_pv + kSlots) {
                // ---- scores of item i_qk:  S[128 x N] = Q[128 x D] * K_blk[N x D]^T
                const int slot = i_qk % kSlots;
                if (k_qk == 0) {
                    ok = mbar_wait_warp(bar(kBarQFull), tl_qk & 1, abort_flag, p.status, kErrMma);
                    if (!ok) break;
                }
                uint32_t kaddr;
                int n;
                if (k_qk < p.nblk_p) {
                    n = prefix_block_cols(p, k_qk);
                    if (p.resident) {
                        if (tq.first_of_g)
                            ok = mbar_wait_warp(bar(kBarKFull + k_qk), (tq.g - g_first) & 1, abort_flag, p.status, kErrMma);
                        kaddr = sbase + C::kOffPK + k_qk * C::kTileBytes;
                    } else {
                        const uint32_t ks = kuse % C::kStages;
                        ok = mbar_wait_warp(bar(kBarKFull + ks), (kuse / C::kStages) & 1, abort_flag, p.status, kErrMma);
                        kaddr = sbase + C::kOffPK + ks * C::kTileBytes;
                    }
                } else {
                    n = tq.n_sfx;
                    ok = mbar_wait_warp(bar(kBarSKFull), tl_qk & 1, abort_flag, p.status, kErrMma);
                    kaddr = sbase + C::kOffSK;
                }
                if (!ok) break;
                PSKV_TRACE_EVENT(10, i_qk);
                tc_fence_after();
#ifdef PSKV_X_QKN
                const uint32_t idesc = make_idesc_bf16(kTileM, PSKV_X_QKN, 0);
#else
                const uint32_t idesc = make_idesc_bf16(kTileM, n, 0);
#endif
                const uint32_t d_tmem = tmem + slot * kBlockN;
                const uint64_t k_desc = make_smem_desc(kaddr, 0, 1024);
                const bool last_of_tile = k_qk == nitems - 1;
                const bool free_stage = k_qk < p.nblk_p && !p.resident;
                if (elect_one_sync()) {
#pragma unroll
                    for (int ks16 = 0; ks16 < D / 16; ++ks16) {
                        const uint64_t off = (uint64_t)(((ks16 >> 2) * C::kSlabBytes + (ks16 & 3) * 32) >> 4);
                        mma_ss(d_tmem, q_desc + off, k_desc + off, idesc, ks16 > 0 ? 1u : 0u);
                        PSKV_TRACE_EVENT_ONE(17, i_qk * 8 + ks16);
                    }
                    tc_commit(bar(kBarSFull + slot));
                    if (free_stage) tc_commit(bar(kBarKFree + (kuse % C::kStages)));
                    if (last_of_tile) tc_commit(bar(kBarQkFree));  // the suffix block ends the tile's scores
                }
                __syncwarp();
                PSKV_TRACE_EVENT(12, i_qk);
                if (free_stage) ++kuse;
                ++i_qk;
                if (++k_qk == nitems) {
                    k_qk = 0;
                    if (++tl_qk < n_tiles) tq = tile_info(p, t_begin + tl_qk, t_begin);
                }
            } else {
                // ---- values of item i_pv:  O[128 x D] (+)= P[128 x N] * V_blk[N x D]
                const int slot = i_pv % kSlots;
                ok = mbar_wait_warp(bar(kBarPReady + slot), (i_pv / kSlots) & 1, abort_flag, p.status, kErrMma);
                if (!ok) break;
                if (k_pv == 0 && tl_pv > 0) {
                    // O of the previous tile must have been read out by the epilogue warps
                    ok = mbar_wait_warp(bar(kBarOFree), (tl_pv - 1) & 1, abort_flag, p.status, kErrMma);
                    if (!ok) break;
                }
                uint32_t vaddr;
                int n;
                if (k_pv < p.nblk_p) {
                    n = prefix_block_cols(p, k_pv);
                    if (p.resident) {
                        if (tv.first_of_g)
                            ok = mbar_wait_warp(bar(kBarVFull + k_pv), (tv.g - g_first) & 1, abort_flag, p.status, kErrMma);
                        vaddr = sbase + C::kOffPV + k_pv * C::kTileBytes;
                    } else {
                        const uint32_t vs = vuse % C::kStages;
                        ok = mbar_wait_warp(bar(kBarVFull + vs), (vuse / C::kStages) & 1, abort_flag, p.status, kErrMma);
                        vaddr = sbase + C::kOffPV + vs * C::kTileBytes;
                    }
                } else {
                    n = tv.n_sfx;
                    ok = mbar_wait_warp(bar(kBarSVFull), tl_pv & 1, abort_flag, p.status, kErrMma);
                    vaddr = sbase + C::kOffSV;
                }
                if (!ok) break;
                PSKV_TRACE_EVENT(11, i_pv);
                tc_fence_after();
                const uint32_t p_tmem = tmem + slot * kBlockN;  // bf16 pairs: 8 columns per 16 keys
                const uint64_t v_desc = make_smem_desc(vaddr, C::kSlabBytes, 1024);
                const int nk = n >> 4;
                const bool last_of_tile = k_pv == nitems - 1;
                const bool free_stage = k_pv < p.nblk_p && !p.resident;
                const uint32_t acc0 = k_pv > 0 ? 1u : 0u;
                if (elect_one_sync()) {
#pragma unroll
                    for (int ks16 = 0; ks16 < kBlockN / 16; ++ks16) {
                        if (ks16 < nk)
                            mma_ts(tmem + kOCol, p_tmem + ks16 * 8, v_desc + (uint64_t)(ks16 * (2048 >> 4)), idesc_pv,
                                   ks16 > 0 ? 1u : acc0);
                    }
                    tc_commit(bar(kBarPvDone + slot));
                    if (free_stage) tc_commit(bar(kBarVFree + (vuse % C::kStages)));
                    if (last_of_tile) {
                        tc_commit(bar(kBarSVFree));
                        tc_commit(bar(kBarOFull));
                    }
                }
                __syncwarp();
                PSKV_TRACE_EVENT(13, i_pv);
                if (free_stage) ++vuse;
                ++i_pv;
                if (++k_pv == nitems) {
                    k_pv = 0;
                    if (++tl_pv < n_tiles) tv = tile_info(p, t_begin + tl_pv, t_begin);
                }
            }
        }
    } else if (warp < 6) {
        // ------------------------------------------------------------------ softmax warps
        // Each thread owns one query row (tensor-memory lane).  Per item: pass 1 reads the score
        // block 32 columns at a time and takes the row max; pass 2 reads it again, exponentiates
        // and writes bf16 probabilities over the first half of the same slot (a probability chunk
        // only ever overwrites score columns that pass 2 has already consumed).
        const int row = 32 * (warp & 3) + lane;
        const uint32_t lane_addr = (uint32_t)(32 * (warp & 3)) << 16;
        int item = 0;
        bool ok = true;
        for (int tl = 0; tl < n_tiles && ok; ++tl) {
            const TileInfo t = tile_info(p, t_begin + tl, t_begin);
            const bool valid = row < t.rows;
            const int R = t.R0 + (valid ? row : 0);
            const int b = R / p.Rg, r = R - b * p.Rg;
            const int sfx_lo = (b - t.b_first) * p.S;   // first suffix column of this row's candidate
            const int sfx_hi = sfx_lo + (r % p.S);      // causal: suffix keys 0..i
            float m_ref = 0.f, l = 0.f;
            for (int k = 0; k < nitems && ok; ++k, ++item) {
                const int slot = item % kSlots;
                int n, lo, hi;                            // valid columns of this row: [lo, hi]
                if (k < p.nblk_p) {
                    n = prefix_block_cols(p, k);
                    lo = 0;
                    hi = valid ? min(kBlockN, p.P - k * kBlockN) - 1 : -1;
                } else {
                    n = t.n_sfx;
                    lo = valid ? sfx_lo : 1;
                    hi = valid ? sfx_hi : 0;
                }
                const int nch = (n + 31) >> 5;
                // chunks [ch_b, ch_e] hold at least one valid column of some row of this warp
                const bool full = __all_sync(0xffffffffu, lo == 0 && hi >= n - 1) && ((n & 31) == 0);
                int ch_b = 0, ch_e = nch - 1;
                if (!full) {
                    const int wlo = __reduce_min_sync(0xffffffffu, hi >= lo ? lo : 0x7fffffff);
                    const int whi = __reduce_max_sync(0xffffffffu, hi >= lo ? hi : -1);
                    ch_b = wlo >> 5;
                    ch_e = min(nch - 1, whi >> 5);
                }
                const unsigned span = (unsigned)(hi - lo);  // hi < lo wraps to a huge span only if hi-lo < 0
                const bool any_col = hi >= lo;
                ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarSFull + slot), (item / kSlots) & 1, abort_flag,
                                                       p.status, kErrSoftmax));
                if (!ok) break;
                if (warp == 2) PSKV_TRACE_EVENT(20, item);
                tc_fence_after();
                const uint32_t s_tmem = tmem + lane_addr + slot * kBlockN;

                // ---- pass 1: row max of the block
                float mb = -INFINITY;
                {
                    float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
                    for (int ch = ch_b; ch <= ch_e; ++ch) {
                        uint32_t rr[32];
                        tmem_ld32(s_tmem + ch * 32, rr);
                        tmem_wait_ld();
                        if (full) {
#pragma unroll
                            for (int c = 0; c < 32; ++c) m4[c & 3] = fmaxf(m4[c & 3], __uint_as_float(rr[c]));
                        } else {
#pragma unroll
                            for (int c = 0; c < 32; ++c) {
                                const bool in = any_col && (unsigned)(ch * 32 + c - lo) <= span;
                                m4[c & 3] = fmaxf(m4[c & 3], in ? __uint_as_float(rr[c]) : -INFINITY);
                            }
                        }
                    }
                    mb = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
                }
                if (warp == 2) PSKV_TRACE_EVENT(22, item);
                const float mx = mb * p.sl2;
                if (k == 0) {
                    m_ref = (mb == -INFINITY) ? 0.f : mx;
                } else {
                    const bool need = mx > m_ref + kRescaleGap;
                    if (__any_sync(0xffffffffu, need)) {
                        // Rare: the running max jumped.  Rescale this row's O in tensor memory after the
                        // previous item's P*V has completed, and before this item's P is handed over.
                        const int prev = item - 1;
                        ok = __all_sync(0xffffffffu, mbar_wait(bar(kBarPvDone + prev % kSlots), (prev / kSlots) & 1,
                                                               abort_flag, p.status, kErrSoftmax));
                        if (!ok) break;
                        tc_fence_after();
                        const float f = need ? exp2f(m_ref - mx) : 1.f;
                        if (need) { l *= f; m_ref = mx; }
#pragma unroll 1
                        for (int ch = 0; ch < D / 32; ++ch) {
                            uint32_t o[32];
                            tmem_ld32(tmem + lane_addr + kOCol + ch * 32, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * f);
                            tmem_st32(tmem + lane_addr + kOCol + ch * 32, o);
                        }
                        tmem_wait_st();
                    }
                }

                // ---- pass 2: p = 2^(s * sl2 - m_ref), row sum, bf16 pairs back to tensor memory
                const float neg_m = -m_ref;
                float ls0 = 0.f, ls1 = 0.f;
                for (int ch = 0; ch < nch; ++ch) {
                    uint32_t pk[16];
                    if (ch >= ch_b && ch <= ch_e) {
                        uint32_t rr[32];
                        tmem_ld32(s_tmem + ch * 32, rr);
                        tmem_wait_ld();
                        if (full) {
#pragma unroll
                            for (int c = 0; c < 16; ++c) {
                                const float p0 = exp2f(fmaf(__uint_as_float(rr[2 * c]), p.sl2, neg_m));
                                const float p1 = exp2f(fmaf(__uint_as_float(rr[2 * c + 1]), p.sl2, neg_m));
                                ls0 += p0;
                                ls1 += p1;
                                pk[c] = pack_bf16x2(p0, p1);
                            }
                        } else {
#pragma unroll
                            for (int c = 0; c < 16; ++c) {
                                const bool in0 = any_col && (unsigned)(ch * 32 + 2 * c - lo) <= span;
                                const bool in1 = any_col && (unsigned)(ch * 32 + 2 * c + 1 - lo) <= span;
                                const float p0 = exp2f(in0 ? fmaf(__uint_as_float(rr[2 * c]), p.sl2, neg_m) : -INFINITY);
                                const float p1 = exp2f(in1 ? fmaf(__uint_as_float(rr[2 * c + 1]), p.sl2, neg_m) : -INFINITY);
                                ls0 += p0;
                                ls1 += p1;
                                pk[c] = pack_bf16x2(p0, p1);
                            }
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < 16; ++c) pk[c] = 0u;
                    }
                    tmem_st16(s_tmem + ch * 16, pk);
                }
                l += ls0 + ls1;
                if (k == nitems - 1) ml[(tl & 1) * kTileM + row] = make_float2(l, m_ref + log2f(l));
                if (warp == 2) PSKV_TRACE_EVENT(23, item);
                tmem_wait_st();
                tc_fence_before();
                __threadfence_block();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarPReady + slot));
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps (6..9)
        const int row = 32 * (warp & 3) + lane;
        const uint32_t lane_addr = (uint32_t)(32 * (warp & 3)) << 16;
        for (int tl = 0; tl < n_tiles; ++tl) {
            const TileInfo t = tile_info(p, t_begin + tl, t_begin);
            if (!__all_sync(0xffffffffu, mbar_wait(bar(kBarOFull), tl & 1, abort_flag, p.status, kErrEpilogue)))
                break;
            if (warp == 6) PSKV_TRACE_EVENT(30, tl);
            tc_fence_after();
            const float2 lm = ml[(tl & 1) * kTileM + row];
            const float inv = 1.f / lm.x;
            uint32_t ob[D / 2];  // normalised row as bf16 pairs
#pragma unroll
            for (int ch = 0; ch < D / 32; ++ch) {
                uint32_t o[32];
                tmem_ld32(tmem + lane_addr + kOCol + ch * 32, o);
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < 16; ++c)
                    ob[ch * 16 + c] = pack_bf16x2(__uint_as_float(o[2 * c]) * inv, __uint_as_float(o[2 * c + 1]) * inv);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarOFree));
            if (row < t.rows) {
                const int R = t.R0 + row;
                const int b = R / p.Rg, r = R - b * p.Rg;
                const size_t grow = ((size_t)b * p.Hq + (size_t)t.g * p.n_rep) * p.S + r;
                uint4 *dst = reinterpret_cast<uint4 *>(p.out + grow * D);
#pragma unroll
#ifdef PSKV_X_NOSTORE
                if (ob[0] == 0x12345678u)
#endif
                for (int v = 0; v < D / 8; ++v) dst[v] = make_uint4(ob[4 * v], ob[4 * v + 1], ob[4 * v + 2], ob[4 * v + 3]);
                p.lse[grow] = lm.y * kLn2;
            }
            if (warp == 6) PSKV_TRACE_EVENT(31, tl);
        }
    }

    // ---------------------------------------------------------------------- teardown
    PSKV_TRACE_FLUSH;
    if (*abort_flag != 0) __nanosleep(20000);  // let copies and MMAs still in flight drain
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------------------ host side

struct TilePlan {
    bool ok;
    int tile_rows, seg_rows, tiles_per_group;
};

int gcd_int(int a, int b) { return b == 0 ? a : gcd_int(b, a % b); }

// Picks the rows per tile: the largest multiple of 8 up to 128 such that the suffix keys of all
// candidates a tile can touch fit one 128-key block (candidates x S <= 128).
TilePlan plan_tiles(const Dims &dm)
{
    TilePlan best{false, 0, 0, 0};
    if (dm.S % 8 != 0 || dm.S > kBlockN) return best;
    const int Rg = dm.n_rep * dm.S;
    const long long total = (long long)dm.B * Rg;
    for (int m = kTileM; m >= 8; m -= 8) {
        const int seg = gcd_int(Rg, m);
        if (seg % 8 != 0) continue;
        // worst number of candidates a window [t*m, t*m + m) overlaps; the pattern repeats every Rg/seg tiles
        const long long ntiles = (total + m - 1) / m;
        const long long period = (long long)Rg / seg;
        const long long check = ntiles < period ? ntiles : period;
        int nc_max = 0;
        for (long long t = 0; t < check; ++t) {
            const long long r0 = t * m;
            long long r1 = r0 + m;
            if (r1 > total) r1 = total;
            const int nc = (int)((r1 - 1) / Rg - r0 / Rg + 1);
            if (nc > nc_max) nc_max = nc;
        }
        if (nc_max * dm.S > kBlockN) continue;
        best.ok = true;
        best.tile_rows = m;
        best.seg_rows = seg;
        best.tiles_per_group = (int)ntiles;
        return best;
    }
    return best;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// bf16 tensor, innermost dimension contiguous, 128-byte swizzle, 64-column boxes.
bool encode_map(CUtensorMap *map, const void *base, int rank, const cuuint64_t *dims,
                const cuuint64_t *strides_bytes, const cuuint32_t *box)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void *>(base), dims,
                    strides_bytes, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

int sm_count()
{
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    }
    return n;
}

template <int D>
cudaError_t launch(const FwdArgs &a, const TilePlan &plan, unsigned int *status_word, cudaStream_t stream)
{
    using C = Cfg<D>;
    const Dims &dm = a.dims;
    const int Rg = dm.n_rep * dm.S;
    CUtensorMap tm_q, tm_pk, tm_pv, tm_sk, tm_sv;
    memset(&tm_pk, 0, sizeof(tm_pk));
    memset(&tm_pv, 0, sizeof(tm_pv));
    {
        // q viewed as [B][Hkv][Rg][D]: the n_rep heads of a KV head are contiguous rows
        cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)Rg, (cuuint64_t)dm.Hkv, (cuuint64_t)dm.B};
        cuuint64_t str[3] = {(cuuint64_t)D * 2, (cuuint64_t)Rg * D * 2, (cuuint64_t)dm.Hkv * Rg * D * 2};
        cuuint32_t box[4] = {64, (cuuint32_t)plan.seg_rows, 1, 1};
        if (!encode_map(&tm_q, a.q, 4, dims, str, box)) return cudaErrorInvalidValue;
    }
    {
        cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)dm.S, (cuuint64_t)dm.Hkv, (cuuint64_t)dm.B};
        cuuint64_t str[3] = {(cuuint64_t)D * 2, (cuuint64_t)dm.S * D * 2, (cuuint64_t)dm.Hkv * dm.S * D * 2};
        cuuint32_t box[4] = {64, (cuuint32_t)dm.S, 1, 1};
        if (!encode_map(&tm_sk, a.suffix_k, 4, dims, str, box)) return cudaErrorInvalidValue;
        if (!encode_map(&tm_sv, a.suffix_v, 4, dims, str, box)) return cudaErrorInvalidValue;
    }
    if (dm.P > 0) {
        cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)dm.P, (cuuint64_t)dm.Hkv};
        cuuint64_t str[2] = {(cuuint64_t)D * 2, (cuuint64_t)dm.P * D * 2};
        cuuint32_t box[3] = {64, (cuuint32_t)kBlockN, 1};
        if (!encode_map(&tm_pk, a.prefix_k, 3, dims, str, box)) return cudaErrorInvalidValue;
        if (!encode_map(&tm_pv, a.prefix_v, 3, dims, str, box)) return cudaErrorInvalidValue;
    }
    TcFwdParams p;
    p.out = a.out;
    p.lse = a.lse;
    p.status = status_word;
    p.sl2 = a.scale * kLog2e;
    p.B = dm.B; p.Hq = dm.Hq; p.Hkv = dm.Hkv; p.S = dm.S; p.P = dm.P; p.n_rep = dm.n_rep;
    p.Rg = Rg;
    p.tile_rows = plan.tile_rows;
    p.seg_rows = plan.seg_rows;
    p.tiles_per_group = plan.tiles_per_group;
    p.total_tiles = plan.tiles_per_group * dm.Hkv;
    p.nblk_p = (dm.P + kBlockN - 1) / kBlockN;
    p.resident = p.nblk_p <= C::kStages ? 1 : 0;

    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(tc_fwd_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             C::kSmemBytes);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    const int grid = p.total_tiles < sm_count() ? p.total_tiles : sm_count();
    tc_fwd_kernel<D><<<grid, kThreads, C::kSmemBytes, stream>>>(tm_q, tm_pk, tm_pv, tm_sk, tm_sv, p);
    count_launches(1);
    return cudaGetLastError();
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
            host[2 * n + 1] = buf[((size_t)w * kTraceCap + i) * 2 + 1];
        }
    cudaMemcpyFromSymbol(cnt, g_trace_n2, sizeof(cnt));
    cudaMemcpyFromSymbol(buf, g_trace2, sizeof(buf));
    for (int w = 0; w < kTraceWarps; ++w)
        for (unsigned int i = 0; i < cnt[w] && i < (unsigned int)kTraceCap && n < max_events; ++i, ++n) {
            host[2 * n] = buf[((size_t)w * kTraceCap + i) * 2];
            host[2 * n + 1] = buf[((size_t)w * kTraceCap + i) * 2 + 1];
        }
    unsigned int zeros[kTraceWarps] = {0};
    cudaMemcpyToSymbol(g_trace_n2, zeros, sizeof(zeros));
    return n;
}
#endif

bool tc_fwd_supported(const Dims &dm)
{
    if (dm.d != 64 && dm.d != 128) return false;
    if ((long long)dm.B * dm.n_rep * dm.S > 2000000000ll) return false;  // flat row index fits an int
    return plan_tiles(dm).ok;
}

size_t tc_fwd_workspace_bytes(const Dims &) { return 0; }

cudaError_t launch_tc_fwd(const FwdArgs &a, void *, unsigned int *status_word, cudaStream_t stream)
{
    const TilePlan plan = plan_tiles(a.dims);
    if (!plan.ok) return cudaErrorInvalidValue;
    return a.dims.d == 128 ? launch<128>(a, plan, status_word, stream) : launch<64>(a, plan, status_word, stream);
}

}  // namespace pskv
