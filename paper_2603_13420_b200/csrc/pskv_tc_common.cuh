// Pieces shared by the tensor-core forward and backward kernels: tile geometry over the flat row
// list of a KV-head group, the optional event trace, and the host-side TMA descriptor helpers.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <atomic>

#include "pskv_common.cuh"

namespace pskv {
namespace {

constexpr int kTileM = 128;    // rows of one MMA tile (tensor-memory lanes)
constexpr int kBlockN = 128;   // keys per block
constexpr int kStagingBytes = kTileM * 128;  // one 64-column slab of an output tile
constexpr int kMaxSmem = 232448;             // dynamic shared memory a CTA may use on sm_100

// Optional event trace of CTA 0 (lane 0 of each warp, a private buffer per warp so that an event
// costs one clock read and two stores): compiled in only with -DPSKV_TRACE=<group mask>.
#ifdef PSKV_TRACE
#ifndef PSKV_TRACE_CTA
#define PSKV_TRACE_CTA 0
#endif
constexpr int kTraceWarps = 28, kTraceCap = 4096;
__device__ long long g_trace[kTraceWarps * kTraceCap * 2];
__device__ unsigned int g_trace_n[kTraceWarps];
#define PSKV_TRACE_DECL unsigned int trace_i_ = 0
#define PSKV_TRACE_EVENT(tag, val)                                                                     \
    do {                                                                                               \
        if (((PSKV_TRACE >> ((tag) / 10)) & 1) && blockIdx.x == PSKV_TRACE_CTA && (threadIdx.x & 31) == 0 &&        \
            trace_i_ < (unsigned int)kTraceCap) {                                                      \
            long long *e_ = g_trace + ((size_t)(threadIdx.x >> 5) * kTraceCap + trace_i_) * 2;         \
            e_[0] = clock64();                                                                         \
            e_[1] = ((long long)(tag) << 32) | (unsigned int)(val);                                    \
            ++trace_i_;                                                                                \
        }                                                                                              \
    } while (0)
#define PSKV_TRACE_FLUSH                                                                               \
    do {                                                                                               \
        if (blockIdx.x == PSKV_TRACE_CTA && (threadIdx.x & 31) == 0) g_trace_n[threadIdx.x >> 5] = trace_i_;        \
    } while (0)
#else
#define PSKV_TRACE_DECL do { } while (0)
#define PSKV_TRACE_FLUSH do { } while (0)
#define PSKV_TRACE_EVENT(tag, val) do { } while (0)
#endif

// Division by a divisor fixed at launch: one 32x32->64 multiply and a shift instead of the long
// instruction sequence of a general integer division.  Exact for 0 <= n < 2^31, 1 <= d < 2^31:
// with L = ceil(log2 d) and M = ceil(2^(31+L) / d), floor(n / d) = (n * M) >> (31 + L).
struct FastDiv {
    unsigned int mul, shift, d;
    __host__ void init(int divisor)
    {
        d = (unsigned int)divisor;
        unsigned int L = 0;
        while ((1ull << L) < (unsigned long long)d) ++L;
        shift = 31u + L;
        mul = (unsigned int)(((1ull << shift) + d - 1) / d);
    }
    __device__ __forceinline__ int div(int n) const
    {
        return (int)(((unsigned long long)(unsigned int)n * mul) >> shift);
    }
};

struct TileInfo {
    int g, R0, rows, b_first, nc, n_sfx;  // n_sfx: suffix columns rounded up to 16
    bool first_of_g;
};

// `Params` is any kernel parameter block with fields B, Rg, S, tile_rows, tiles_per_group, fd_tpg, fd_Rg.
template <class Params>
__device__ __forceinline__ TileInfo tile_info(const Params &p, int tile, int t_begin)
{
    TileInfo t;
    t.g = p.fd_tpg.div(tile);
    const int tt = tile - t.g * p.tiles_per_group;
    t.first_of_g = (tt == 0) || (tile == t_begin);
    t.R0 = tt * p.tile_rows;
    const int total = p.B * p.Rg;
    t.rows = min(p.tile_rows, total - t.R0);
    t.b_first = p.fd_Rg.div(t.R0);
    const int b_last = p.fd_Rg.div(t.R0 + t.rows - 1);
    t.nc = b_last - t.b_first + 1;
    t.n_sfx = (t.nc * p.S + 15) & ~15;
    return t;
}

// ------------------------------------------------------------------------------ host side

// Persistent grid for `units` equal work items on `sms` SMs: every CTA gets the same number of items (the
// longest CTA sets the kernel's duration either way), so that a launch whose items do not fill the last
// round leaves whole SMs free for a kernel running beside it instead of idling them one item early.
inline int even_grid(int units, int sms)
{
    if (units <= sms) return units;
    const int rounds = (units + sms - 1) / sms;
    return (units + rounds - 1) / rounds;
}

inline int gcd_int(int a, int b) { return b == 0 ? a : gcd_int(b, a % b); }
inline int round_up(int x, int m) { return (x + m - 1) / m * m; }


// Picks the rows per tile: the largest multiple of 8 up to 128 such that the suffix keys of all
// candidates a tile can touch fit one 128-key block (candidates x S <= 128).  `nc_max` receives
// that largest number of candidates.
inline bool pick_tile_rows(const Dims &dm, int *tile_rows, int *seg_rows, int *tiles_per_group, int *nc_max_out)
{
    if (dm.S % 8 != 0 || dm.S > kBlockN) return false;
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
        *tile_rows = m;
        *seg_rows = seg;
        *tiles_per_group = (int)ntiles;
        *nc_max_out = nc_max;
        return true;
    }
    return false;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode_fn()
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
// A launch needs eight or nine of these and a search loop calls with the same buffers and shapes step
// after step, so the encoded maps are kept in a small per-thread table keyed by everything that went
// into them (base address, rank, extents, strides, box); a hit costs a compare and a 128-byte copy
// instead of a driver call.  A tensor map holds no reference to the memory: a stale entry for a freed
// and re-used address is still the right map for that address.
struct MapKey {
    const void *base;
    int rank;
    cuuint64_t dims[4], strides[3];
    cuuint32_t box[4];
};
struct MapCacheEntry {
    bool used;
    MapKey key;
    CUtensorMap map;
};
constexpr int kMapCacheSize = 64;  // direct-mapped

inline bool encode_map(CUtensorMap *map, const void *base, int rank, const cuuint64_t *dims,
                const cuuint64_t *strides_bytes, const cuuint32_t *box)
{
    static thread_local MapCacheEntry cache[kMapCacheSize];
    MapKey key;
    memset(&key, 0, sizeof(key));
    key.base = base;
    key.rank = rank;
    for (int i = 0; i < rank && i < 4; ++i) { key.dims[i] = dims[i]; key.box[i] = box[i]; }
    for (int i = 0; i + 1 < rank && i < 3; ++i) key.strides[i] = strides_bytes[i];
    unsigned long long h = (unsigned long long)(uintptr_t)base * 0x9E3779B97F4A7C15ull;
    for (int i = 0; i < 4; ++i) h = (h ^ key.dims[i] ^ ((unsigned long long)key.box[i] << 40)) * 0x100000001B3ull;
    MapCacheEntry &e = cache[(h >> 32) % kMapCacheSize];
#ifndef PSKV_NO_MAP_CACHE  // (defined only to measure what the table saves)
    if (e.used && memcmp(&e.key, &key, sizeof(key)) == 0) {
        memcpy(map, &e.map, sizeof(CUtensorMap));
        return true;
    }
#endif
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void *>(base), dims,
                    strides_bytes, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return false;
    e.used = true;
    e.key = key;
    memcpy(&e.map, map, sizeof(CUtensorMap));
    return true;
}

// Per-device state of the launch sites.  cudaFuncSetAttribute (the opt-in to more than 48 KB of
// dynamic shared memory) and the SM count belong to a DEVICE, not to the process: a process that works
// on several GPUs needs both once per device.
constexpr int kMaxGuardDevices = 64;

// One flag per device ordinal; first_time(dev) is true exactly once per device (ordinals beyond the
// table are always "first", i.e. the caller simply repeats the cheap set-up).
struct PerDeviceOnce {
    std::atomic<unsigned long long> done{0};
    bool pending(int dev) const
    {
        return dev < 0 || dev >= kMaxGuardDevices || ((done.load(std::memory_order_acquire) >> dev) & 1ull) == 0;
    }
    void mark(int dev)
    {
        if (dev >= 0 && dev < kMaxGuardDevices) done.fetch_or(1ull << dev, std::memory_order_release);
    }
};

// Raises a kernel's dynamic shared-memory limit on the current device if that has not been done there yet.
template <class Kernel>
inline cudaError_t ensure_max_smem(Kernel kernel, PerDeviceOnce &once, int bytes = kMaxSmem)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (!once.pending(dev)) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e == cudaSuccess) once.mark(dev);
    return e;
}

// Launch with programmatic stream serialization: the kernel may be scheduled while the kernel before it in the
// stream is still running (that one calls grid_dep_launch() at its start), so that its CTAs take over SMs as
// the other's CTAs exit and run their prologue -- shared-memory zeroing, barrier and tensor-memory set-up, about
// 3 us -- under the other kernel's tail; grid_dep_wait() in the kernel then holds every access to global memory
// back until the kernel before has completed and its writes are visible.  Behind anything that is not such
// a kernel the launch orders as usual.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), int grid, int threads, int smem_bytes, cudaStream_t stream,
                                    Args &&...args)
{
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = (size_t)smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    memset(&attr, 0, sizeof(attr));
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// SM count of the current device (looked up once per device).
inline int sm_count()
{
    static std::atomic<int> count[kMaxGuardDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 1;
    const bool cached = dev >= 0 && dev < kMaxGuardDevices;
    int n = cached ? count[dev].load(std::memory_order_relaxed) : 0;
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 1;
        if (cached) count[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}

}  // namespace
}  // namespace pskv
