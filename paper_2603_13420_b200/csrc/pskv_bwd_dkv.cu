// Suffix-side gradients dK_suffix, dV_suffix (the block-diagonal part of the backward):
//   dV[b,g,t,:] = sum over heads h of g, rows i >= t of  P[b,h,i,t] dO[b,h,i,:]
//   dK[b,g,t,:] = scale * sum over the same (h, i) of     dS[b,h,i,t] Q[b,h,i,:]
// with P = exp(scale q.k - lse) on the suffix keys only and dS = P (dO.v - D).
// One CTA per (candidate, KV head): its n_rep*S query rows and S suffix keys are contiguous in
// memory, so everything is staged with plain coalesced copies.  The four small contractions per
// 64-row chunk (S = Q K^T, dP = dO V^T, then P^T dO and dS^T Q) run on warp-level bf16 MMAs
// (m16n8k16, fp32 accumulation): at 6-7 % of the backward flops and 48x192-sized operands this
// part is bound by its memory traffic, not by tensor throughput.  Sums over the heads of a group
// happen in registers of one CTA, so the result is deterministic and needs no atomics.
#include "pskv_common.cuh"
#include "pskv_tc_common.cuh"

namespace pskv {
namespace {

constexpr int kDkvWarps = 4;
constexpr int kDkvThreads = kDkvWarps * 32;
constexpr int kChunkRows = kDkvWarps * 16;  // 64 query rows per pass

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// 16-byte asynchronous copy global -> shared; `valid` false writes zeros instead
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid)
{
    const int bytes = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_group1() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// Shared memory, all bf16 with 16 bytes of row padding (conflict-free ldmatrix):
//   Qs, Gs  [2][64][D]    query / dout rows of the current chunk and of the next one (two stages)
//   Ks, Vs  [TP][D]       suffix keys / values (TP = S rounded up to 16, padding rows zero)
//   Ps, Ds  [64][TP]      probabilities / dS of the chunk
template <int D, int TP>
struct DkvSmem {
    static constexpr int kRowD = D * 2 + 16;
    static constexpr int kRowT = TP * 2 + 16;
    static constexpr int kStage = 2 * kChunkRows * kRowD;  // one stage: Q rows, then dout rows
    static constexpr int kOffQ = 0;                        // stage 0; stage 1 follows
    static constexpr int kOffG = kOffQ + kChunkRows * kRowD;
    static constexpr int kOffK = kOffQ + 2 * kStage;
    static constexpr int kOffV = kOffK + TP * kRowD;
    static constexpr int kOffP = kOffV + TP * kRowD;
    static constexpr int kOffS = kOffP + kChunkRows * kRowT;
    static constexpr int kBytes = kOffS + kChunkRows * kRowT;
};

template <int D, int TP>
__global__ void __launch_bounds__(kDkvThreads, 2)
bwd_dkv_mma_kernel(BwdArgs a)
{
    using L = DkvSmem<D, TP>;
    extern __shared__ __align__(16) uint8_t smem[];
    const Dims dm = a.dims;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int S = dm.S, Rg = dm.n_rep * S;
    const int nchunk = (Rg + kChunkRows - 1) / kChunkRows;
    const int total_bg = dm.B * dm.Hkv;
    const uint32_t sb = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
    const float sl2 = a.scale * kLog2e;

    // The CTA walks over its (candidate, KV head) groups, a chunk of 64 query rows at a time; the
    // copies of the next chunk (of this group or the next) are in flight while this one is computed.
    // unit u = (group index within this CTA, chunk)
    const int my_groups = blockIdx.x < total_bg ? (total_bg - 1 - blockIdx.x) / gridDim.x + 1 : 0;
    const int total_units = my_groups * nchunk;

    auto issue_qg = [&](int u) {  // asynchronous copies of unit u's query / dout rows into stage u & 1
        const int gi = u / nchunk, c = u - gi * nchunk;
        const int bg = blockIdx.x + gi * gridDim.x;
        const int b = bg / dm.Hkv, g = bg - b * dm.Hkv;
        const size_t row0 = ((size_t)b * dm.Hq + (size_t)g * dm.n_rep) * S + (size_t)c * kChunkRows;
        const __nv_bfloat16 *qg = a.q + row0 * D;
        const __nv_bfloat16 *gg = a.dout + row0 * D;
        const int rows = min(kChunkRows, Rg - c * kChunkRows);
        const uint32_t st = sb + (u & 1) * L::kStage;
        for (int i = tid; i < kChunkRows * (D / 8); i += kDkvThreads) {
            const int r = i / (D / 8), cc = i - r * (D / 8);
            const int rs = r < rows ? r : 0;
            cp_async16(st + L::kOffQ + r * L::kRowD + cc * 16, qg + (size_t)rs * D + cc * 8, r < rows);
            cp_async16(st + L::kOffG + r * L::kRowD + cc * 16, gg + (size_t)rs * D + cc * 8, r < rows);
        }
    };
    auto issue_kv = [&](int gi) {  // suffix K / V of group gi; padding rows zero
        const int bg = blockIdx.x + gi * gridDim.x;
        const __nv_bfloat16 *kg = a.suffix_k + (size_t)bg * S * D;
        const __nv_bfloat16 *vg = a.suffix_v + (size_t)bg * S * D;
        for (int i = tid; i < TP * (D / 8); i += kDkvThreads) {
            const int t = i / (D / 8), c = i - t * (D / 8);
            const int ts = t < S ? t : 0;
            cp_async16(sb + L::kOffK + t * L::kRowD + c * 16, kg + (size_t)ts * D + c * 8, t < S);
            cp_async16(sb + L::kOffV + t * L::kRowD + c * 16, vg + (size_t)ts * D + c * 8, t < S);
        }
    };

    // this warp's output tiles: all m-tiles (keys) x its kNT consecutive n-tiles (8 columns each)
    constexpr int kMT = TP / 16;
    constexpr int kNT = D / 8 / kDkvWarps;
    float accV[kMT][kNT][4], accK[kMT][kNT][4];
#pragma unroll
    for (int m = 0; m < kMT; ++m)
#pragma unroll
        for (int n = 0; n < kNT; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) { accV[m][n][e] = 0.f; accK[m][n][e] = 0.f; }

    if (total_units > 0) {
        issue_kv(0);
        issue_qg(0);
    }
    cp_async_commit();

#pragma unroll 1
    for (int u = 0; u < total_units; ++u) {
        const int gi = u / nchunk, c = u - gi * nchunk;
        const int bg = blockIdx.x + gi * gridDim.x;
        const int b = bg / dm.Hkv, g = bg - b * dm.Hkv;
        const size_t row0 = ((size_t)b * dm.Hq + (size_t)g * dm.n_rep) * S;  // first query row of the group
        const int c0 = c * kChunkRows;
        const int rows = min(kChunkRows, Rg - c0);
        const uint32_t st = sb + (u & 1) * L::kStage;
        const bool last_chunk = c == nchunk - 1;

        // the next unit's rows go into the other stage (free since the barrier that ended unit u-1)
        if (u + 1 < total_units) issue_qg(u + 1);
        cp_async_commit();
        cp_async_wait_group1();  // everything but the copies just issued has landed: unit u (and its K / V)
        __syncthreads();

        // ---- phase 1: this warp's 16 rows: S = Q K^T, dP = dO V^T, then P and dS to shared memory
        {
            const int r_base = warp * 16;
            float sacc[TP / 8][4], pacc[TP / 8][4];
#pragma unroll
            for (int n = 0; n < TP / 8; ++n)
#pragma unroll
                for (int e = 0; e < 4; ++e) { sacc[n][e] = 0.f; pacc[n][e] = 0.f; }
#pragma unroll
            for (int k0 = 0; k0 < D; k0 += 16) {
                uint32_t aq[4], ag[4];
                const uint32_t arow = (uint32_t)(r_base + (lane & 15)) * L::kRowD + (uint32_t)(k0 + (lane >> 4) * 8) * 2;
                ldsm_x4(aq, st + L::kOffQ + arow);
                ldsm_x4(ag, st + L::kOffG + arow);
#pragma unroll
                for (int n = 0; n < TP / 16; ++n) {
                    // two key tiles (16 keys) per ldmatrix.x4: lanes 0-7 keys +0..7 @k0, 8-15 same keys @k0+8,
                    // 16-23 keys +8..15 @k0, 24-31 @k0+8
                    const uint32_t brow = (uint32_t)(n * 16 + (lane & 7) + ((lane >> 4) << 3)) * L::kRowD +
                                          (uint32_t)(k0 + ((lane >> 3) & 1) * 8) * 2;
                    uint32_t bk[4], bv[4];
                    ldsm_x4(bk, sb + L::kOffK + brow);
                    ldsm_x4(bv, sb + L::kOffV + brow);
                    mma_bf16(sacc[2 * n], aq, bk[0], bk[1]);
                    mma_bf16(sacc[2 * n + 1], aq, bk[2], bk[3]);
                    mma_bf16(pacc[2 * n], ag, bv[0], bv[1]);
                    mma_bf16(pacc[2 * n + 1], ag, bv[2], bv[3]);
                }
            }
            // accumulator element e of a tile: row = lane/4 + 8*(e/2), column = 2*(lane%4) + (e%2)
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int r = r_base + (lane >> 2) + 8 * half;  // row inside the chunk
                const int gr = c0 + r;                          // row inside the group: head-major, then position
                const bool rv = r < rows;
                const int i_pos = gr % S;
                const float nl2 = rv ? -a.lse[row0 + gr] * kLog2e : -INFINITY;
                const float dr = rv ? a.row_dot[row0 + gr] : 0.f;
#pragma unroll
                for (int n = 0; n < TP / 8; ++n) {
                    const int t0 = n * 8 + 2 * (lane & 3);
                    float p0 = 0.f, p1 = 0.f, d0 = 0.f, d1 = 0.f;
                    if (rv && t0 <= i_pos) {  // causal: key t visible to suffix position i when t <= i
                        p0 = exp2f(fmaf(sacc[n][2 * half], sl2, nl2));
                        d0 = p0 * (pacc[n][2 * half] - dr);
                    }
                    if (rv && t0 + 1 <= i_pos) {
                        p1 = exp2f(fmaf(sacc[n][2 * half + 1], sl2, nl2));
                        d1 = p1 * (pacc[n][2 * half + 1] - dr);
                    }
                    *reinterpret_cast<uint32_t *>(smem + L::kOffP + r * L::kRowT + t0 * 2) = pack2(p0, p1);
                    *reinterpret_cast<uint32_t *>(smem + L::kOffS + r * L::kRowT + t0 * 2) = pack2(d0, d1);
                }
            }
        }
        __syncthreads();
        // suffix K / V are not read after phase 1: fetch the next group's while phase 2 runs
        if (last_chunk && gi + 1 < my_groups) issue_kv(gi + 1);
        cp_async_commit();  // its own group (possibly empty), so that the wait above covers it next time round

        // ---- phase 2: dV += P^T dO, dK += dS^T Q over the chunk's rows (contraction index = row)
#pragma unroll 1
        for (int k0 = 0; k0 < kChunkRows; k0 += 16) {
            if (k0 >= rows) break;  // rows past `rows` inside a started 16-row step are zero
            uint32_t bg_[kNT][2], bq_[kNT][2];
#pragma unroll
            for (int n = 0; n < kNT; n += 2) {
                // B[k = row][n = column] from row-major [row][column]: transposed 8x8 loads
                const uint32_t off = (uint32_t)(k0 + (lane & 7) + ((lane >> 3) & 1) * 8) * L::kRowD +
                                     (uint32_t)((warp * kNT + n) * 8 + (lane >> 4) * 8) * 2;
                uint32_t t4[4];
                ldsm_x4_trans(t4, st + L::kOffG + off);
                bg_[n][0] = t4[0]; bg_[n][1] = t4[1]; bg_[n + 1][0] = t4[2]; bg_[n + 1][1] = t4[3];
                ldsm_x4_trans(t4, st + L::kOffQ + off);
                bq_[n][0] = t4[0]; bq_[n][1] = t4[1]; bq_[n + 1][0] = t4[2]; bq_[n + 1][1] = t4[3];
            }
#pragma unroll
            for (int m = 0; m < kMT; ++m) {
                // A[m = key][k = row] from [row][key]: transposed loads; matrices: (keys 0-7, rows 0-7),
                // (keys 8-15, rows 0-7), (keys 0-7, rows 8-15), (keys 8-15, rows 8-15)
                const uint32_t off = (uint32_t)(k0 + (lane & 7) + (lane >> 4) * 8) * L::kRowT +
                                     (uint32_t)(m * 16 + ((lane >> 3) & 1) * 8) * 2;
                uint32_t ap[4], as_[4];
                ldsm_x4_trans(ap, sb + L::kOffP + off);
                ldsm_x4_trans(as_, sb + L::kOffS + off);
#pragma unroll
                for (int n = 0; n < kNT; ++n) {
                    mma_bf16(accV[m][n], ap, bg_[n][0], bg_[n][1]);
                    mma_bf16(accK[m][n], as_, bq_[n][0], bq_[n][1]);
                }
            }
        }

        if (last_chunk) {
            // ---- store: accumulator element e: key = m*16 + lane/4 + 8*(e/2), column = n-tile*8 + 2*(lane%4) + (e%2)
            __nv_bfloat16 *dkg = a.dk_suffix + (size_t)bg * S * D;
            __nv_bfloat16 *dvg = a.dv_suffix + (size_t)bg * S * D;
#pragma unroll
            for (int m = 0; m < kMT; ++m)
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int t = m * 16 + (lane >> 2) + 8 * half;
#pragma unroll
                    for (int n = 0; n < kNT; ++n) {
                        if (t < S) {
                            const int col = (warp * kNT + n) * 8 + 2 * (lane & 3);
                            *reinterpret_cast<uint32_t *>(dvg + (size_t)t * D + col) =
                                pack2(accV[m][n][2 * half], accV[m][n][2 * half + 1]);
                            *reinterpret_cast<uint32_t *>(dkg + (size_t)t * D + col) =
                                pack2(accK[m][n][2 * half] * a.scale, accK[m][n][2 * half + 1] * a.scale);
                        }
                        accV[m][n][2 * half] = 0.f; accV[m][n][2 * half + 1] = 0.f;
                        accK[m][n][2 * half] = 0.f; accK[m][n][2 * half + 1] = 0.f;
                    }
                }
        }
        __syncthreads();  // this unit's stage, P and dS are free for the next units
    }
    cp_async_wait_all();
}

template <int D, int TP>
cudaError_t launch_one(const BwdArgs &a, cudaStream_t stream)
{
    using L = DkvSmem<D, TP>;
    static PerDeviceOnce attr_set;
    if (cudaError_t e = ensure_max_smem(bwd_dkv_mma_kernel<D, TP>, attr_set, L::kBytes); e != cudaSuccess) return e;
    KernelTiming timing(kKernelBwdDkvMma, stream);
    const int total_bg = a.dims.B * a.dims.Hkv;
    const int max_ctas = 2 * sm_count();  // two resident CTAs per SM, each walking over its groups
    bwd_dkv_mma_kernel<D, TP><<<total_bg < max_ctas ? total_bg : max_ctas, kDkvThreads, L::kBytes, stream>>>(a);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace

bool mma_bwd_dkv_supported(const Dims &dm)
{
    if (dm.Skv != dm.S || dm.ragged) return false;  // full-suffix operator only
    return (dm.d == 64 || dm.d == 128) && dm.S >= 1 && dm.S <= 64 && (long long)dm.B * dm.Hkv < 2000000000ll;
}

cudaError_t launch_mma_bwd_dkv(const BwdArgs &a, cudaStream_t stream)
{
    const int tp = (a.dims.S + 15) / 16 * 16;
    if (a.dims.d == 128) {
        switch (tp) {
        case 16: return launch_one<128, 16>(a, stream);
        case 32: return launch_one<128, 32>(a, stream);
        case 48: return launch_one<128, 48>(a, stream);
        default: return launch_one<128, 64>(a, stream);
        }
    }
    switch (tp) {
    case 16: return launch_one<64, 16>(a, stream);
    case 32: return launch_one<64, 32>(a, stream);
    case 48: return launch_one<64, 48>(a, stream);
    default: return launch_one<64, 64>(a, stream);
    }
}

}  // namespace pskv
