// General CUDA-core kernels for shared-prefix attention: any P >= 0, any S >= 1, d in {64,128}.
// They serve the shapes the tensor-core kernels do not take.  One warp owns one query row
// (forward, dQ) or one suffix key (dK/dV); the prefix K/V is read in place, shared by all
// candidates (Sec. 4.2), and the softmax is one continued online softmax over prefix keys
// followed by the causally visible suffix keys (Eq. 2).
#include "pskv_common.cuh"
#include "pskv_rows.cuh"

namespace pskv {
namespace {

constexpr int kWarpsPerBlock = 8;

template <int D>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
simt_fwd_kernel(FwdArgs a)
{
    __shared__ float q_s[kWarpsPerBlock][D];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * kWarpsPerBlock + warp;
    if (row >= (long long)a.dims.B * a.dims.Hq * a.dims.S) return;
    fwd_row<D>(a, row, q_s[warp], lane);
}

// Backward, query side: one warp per query row; writes dq and D = <dout, out>.
template <int D>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
simt_bwd_dq_kernel(BwdArgs a)
{
    __shared__ float q_s[kWarpsPerBlock][D];
    __shared__ float do_s[kWarpsPerBlock][D];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const Dims dm = a.dims;
    const long long row = (long long)blockIdx.x * kWarpsPerBlock + warp;
    if (row >= (long long)dm.B * dm.Hq * dm.S) return;
    const int i = (int)(row % dm.S);
    const int h = (int)((row / dm.S) % dm.Hq);
    const int b = (int)(row / ((long long)dm.S * dm.Hq));
    const int g = h / dm.n_rep;
    const __nv_bfloat16 *pk = a.prefix_k + (size_t)g * dm.Pstride * D;
    const __nv_bfloat16 *pv = a.prefix_v + (size_t)g * dm.Pstride * D;
    const __nv_bfloat16 *sk = a.suffix_k + ((size_t)b * dm.Hkv + g) * dm.Skv * D;
    const __nv_bfloat16 *sv = a.suffix_v + ((size_t)b * dm.Hkv + g) * dm.Skv * D;

    stage_row<D>(q_s[warp], a.q + (size_t)row * D, lane);
    stage_row<D>(do_s[warp], a.dout + (size_t)row * D, lane);
    float o[D / 32];
    load_slice<D>(a.out + (size_t)row * D, lane, o);
    __syncwarp();
    float dsum = 0.f;
#pragma unroll
    for (int e = 0; e < D / 32; ++e) dsum = fmaf(o[e], do_s[warp][lane * (D / 32) + e], dsum);
    // d lse / d s_j = p_j, so a gradient on lse enters every ds_j = p_j (dp_j - D) as -D += dlse
    const float Drow = warp_sum(dsum) - (a.dlse ? a.dlse[row] : 0.f);
    if (lane == 0) a.row_dot[row] = Drow;

    const float scale2 = a.scale * kLog2e;
    const float lse2 = a.lse[row] * kLog2e;
    const int n_vis = dm.P + suffix_tokens(a.suffix_len, b, dm.S, dm.Skv) - dm.S + i + 1;
    float acc[D / 32];
#pragma unroll
    for (int e = 0; e < D / 32; ++e) acc[e] = 0.f;
    for (int j0 = 0; j0 < n_vis; j0 += 32) {
        const int j = j0 + lane;
        float ds = 0.f;
        if (j < n_vis) {
            const bool pre = j < dm.P;
            const __nv_bfloat16 *krow = pre ? pk + (size_t)j * D : sk + (size_t)(j - dm.P) * D;
            const __nv_bfloat16 *vrow = pre ? pv + (size_t)j * D : sv + (size_t)(j - dm.P) * D;
            const float p = exp2f(scale2 * dot_row<D>(q_s[warp], krow) - lse2);
            const float dp = dot_row<D>(do_s[warp], vrow);
            ds = p * (dp - Drow);
        }
        const int cnt = min(32, n_vis - j0);
        for (int t = 0; t < cnt; ++t) {
            const float dst = __shfl_sync(0xffffffffu, ds, t);
            const int jj = j0 + t;
            const __nv_bfloat16 *krow = (jj < dm.P) ? pk + (size_t)jj * D : sk + (size_t)(jj - dm.P) * D;
            float k[D / 32];
            load_slice<D>(krow, lane, k);
#pragma unroll
            for (int e = 0; e < D / 32; ++e) acc[e] = fmaf(dst, k[e], acc[e]);
        }
    }
#pragma unroll
    for (int e = 0; e < D / 32; ++e) acc[e] *= a.scale;
    store_slice<D>(a.dq + (size_t)row * D, lane, acc);
}

// D = <dout, out> (minus the gradient arriving on lse, if any) for every query row.  A pure streaming pass over two tensors, so it is laid out
// for bytes in flight: D/8 lanes share a row with one 16-byte load each per tensor, so a warp-wide
// load covers 2 rows (d = 128) or 4 (d = 64), and every thread keeps kRowDotUnroll such loads of
// both tensors outstanding.
constexpr int kRowDotUnroll = 4;
template <int D>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
simt_row_dot_kernel(BwdArgs a)
{
    constexpr int kLanesPerRow = D / 8;             // 16 (d = 128) or 8 (d = 64)
    constexpr int kRowsPerLoad = 32 / kLanesPerRow;  // rows one warp-wide load covers
    constexpr int kRowsPerWarp = kRowsPerLoad * kRowDotUnroll;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long rows = (long long)a.dims.B * a.dims.Hq * a.dims.S;
    const long long first = ((long long)blockIdx.x * kWarpsPerBlock + warp) * kRowsPerWarp;
    if (first >= rows) return;
    const int sub = lane / kLanesPerRow, col = (lane % kLanesPerRow) * 8;
    uint4 o[kRowDotUnroll], g[kRowDotUnroll];
#pragma unroll
    for (int u = 0; u < kRowDotUnroll; ++u) {
        const long long row = first + u * kRowsPerLoad + sub;
        const long long rc = row < rows ? row : rows - 1;  // clamp: the value is dropped below
        o[u] = *reinterpret_cast<const uint4 *>(a.out + (size_t)rc * D + col);
        g[u] = *reinterpret_cast<const uint4 *>(a.dout + (size_t)rc * D + col);
    }
#pragma unroll
    for (int u = 0; u < kRowDotUnroll; ++u) {
        const __nv_bfloat162 *ob = reinterpret_cast<const __nv_bfloat162 *>(&o[u]);
        const __nv_bfloat162 *gb = reinterpret_cast<const __nv_bfloat162 *>(&g[u]);
        float acc = 0.f;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 x = __bfloat1622float2(ob[e]), y = __bfloat1622float2(gb[e]);
            acc = fmaf(x.x, y.x, acc);
            acc = fmaf(x.y, y.y, acc);
        }
#pragma unroll
        for (int off = kLanesPerRow / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        const long long row = first + u * kRowsPerLoad + sub;
        if (lane % kLanesPerRow == 0 && row < rows) a.row_dot[row] = acc - (a.dlse ? a.dlse[row] : 0.f);
    }
}

// Backward, key side: one warp per suffix key (b,g,t); sums over the n_rep heads of the group
// and the query rows that see the key.  Needs row_dot from the query-side kernel.
template <int D>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
simt_bwd_dkv_kernel(BwdArgs a)
{
    __shared__ float k_s[kWarpsPerBlock][D];
    __shared__ float v_s[kWarpsPerBlock][D];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const Dims dm = a.dims;
    const long long key = (long long)blockIdx.x * kWarpsPerBlock + warp;
    if (key >= (long long)dm.B * dm.Hkv * dm.Skv) return;
    const int t = (int)(key % dm.Skv);
    const int g = (int)((key / dm.Skv) % dm.Hkv);
    const int b = (int)(key / ((long long)dm.Skv * dm.Hkv));
    const int L = suffix_tokens(a.suffix_len, b, dm.S, dm.Skv);
    if (t >= L) {  // not a cached token: no query sees it
        float z[D / 32];
#pragma unroll
        for (int e = 0; e < D / 32; ++e) z[e] = 0.f;
        store_slice<D>(a.dk_suffix + (size_t)key * D, lane, z);
        store_slice<D>(a.dv_suffix + (size_t)key * D, lane, z);
        return;
    }

    stage_row<D>(k_s[warp], a.suffix_k + (size_t)key * D, lane);
    stage_row<D>(v_s[warp], a.suffix_v + (size_t)key * D, lane);
    __syncwarp();

    const float scale2 = a.scale * kLog2e;
    // query i is suffix token L - S + i: the key is seen by rows i >= t - (L - S)
    const int i_min = max(0, t - (L - dm.S));
    const int per_head = dm.S - i_min;        // rows i = i_min .. S-1
    const int n_rows = dm.n_rep * per_head;
    float dk[D / 32], dv[D / 32];
#pragma unroll
    for (int e = 0; e < D / 32; ++e) { dk[e] = 0.f; dv[e] = 0.f; }

    for (int r0 = 0; r0 < n_rows; r0 += 32) {
        const int r = r0 + lane;
        float p = 0.f, ds = 0.f;
        if (r < n_rows) {
            const int h = g * dm.n_rep + r / per_head;
            const int i = i_min + r % per_head;
            const size_t row = ((size_t)b * dm.Hq + h) * dm.S + i;
            p = exp2f(scale2 * dot_row<D>(k_s[warp], a.q + row * D) - a.lse[row] * kLog2e);
            const float dp = dot_row<D>(v_s[warp], a.dout + row * D);
            ds = p * (dp - a.row_dot[row]);
        }
        const int cnt = min(32, n_rows - r0);
        for (int u = 0; u < cnt; ++u) {
            const float pu = __shfl_sync(0xffffffffu, p, u);
            const float dsu = __shfl_sync(0xffffffffu, ds, u);
            const int rr = r0 + u;
            const int h = g * dm.n_rep + rr / per_head;
            const int i = i_min + rr % per_head;
            const size_t row = ((size_t)b * dm.Hq + h) * dm.S + i;
            float qv[D / 32], gv[D / 32];
            load_slice<D>(a.q + row * D, lane, qv);
            load_slice<D>(a.dout + row * D, lane, gv);
#pragma unroll
            for (int e = 0; e < D / 32; ++e) {
                dk[e] = fmaf(dsu, qv[e], dk[e]);
                dv[e] = fmaf(pu, gv[e], dv[e]);
            }
        }
    }
#pragma unroll
    for (int e = 0; e < D / 32; ++e) dk[e] *= a.scale;
    store_slice<D>(a.dk_suffix + (size_t)key * D, lane, dk);
    store_slice<D>(a.dv_suffix + (size_t)key * D, lane, dv);
}

// Gradients of the shared prefix cache, general version: one warp per prefix key (g, j); sums over
// every candidate, the n_rep heads of the group and all their rows (every row sees every prefix key).
// Needs row_dot.  Deterministic (no atomics), and slow: it serves the shapes the tensor-core kernel
// does not take.
template <int D>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
simt_bwd_prefix_kernel(BwdArgs a, __nv_bfloat16 *dk_prefix, __nv_bfloat16 *dv_prefix)
{
    __shared__ float k_s[kWarpsPerBlock][D];
    __shared__ float v_s[kWarpsPerBlock][D];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const Dims dm = a.dims;
    const long long key = (long long)blockIdx.x * kWarpsPerBlock + warp;
    if (key >= (long long)dm.Hkv * dm.P) return;
    const int j = (int)(key % dm.P);
    const int g = (int)(key / dm.P);
    stage_row<D>(k_s[warp], a.prefix_k + ((size_t)g * dm.Pstride + j) * D, lane);
    stage_row<D>(v_s[warp], a.prefix_v + ((size_t)g * dm.Pstride + j) * D, lane);
    __syncwarp();
    const float scale2 = a.scale * kLog2e;
    const int per_cand = dm.n_rep * dm.S;
    const long long n_rows = (long long)dm.B * per_cand;
    float dk[D / 32], dv[D / 32];
#pragma unroll
    for (int e = 0; e < D / 32; ++e) { dk[e] = 0.f; dv[e] = 0.f; }
    for (long long r0 = 0; r0 < n_rows; r0 += 32) {
        const long long r = r0 + lane;
        float p = 0.f, ds = 0.f;
        if (r < n_rows) {
            const int b = (int)(r / per_cand), rem = (int)(r - (long long)b * per_cand);
            const size_t row = ((size_t)b * dm.Hq + (size_t)g * dm.n_rep) * dm.S + rem;  // heads of a group are contiguous
            p = exp2f(scale2 * dot_row<D>(k_s[warp], a.q + row * D) - a.lse[row] * kLog2e);
            ds = p * (dot_row<D>(v_s[warp], a.dout + row * D) - a.row_dot[row]);
        }
        const int cnt = (int)(n_rows - r0 < 32 ? n_rows - r0 : 32);
        for (int u = 0; u < cnt; ++u) {
            const float pu = __shfl_sync(0xffffffffu, p, u);
            const float dsu = __shfl_sync(0xffffffffu, ds, u);
            const long long rr = r0 + u;
            const int b = (int)(rr / per_cand), rem = (int)(rr - (long long)b * per_cand);
            const size_t row = ((size_t)b * dm.Hq + (size_t)g * dm.n_rep) * dm.S + rem;
            float qv[D / 32], gv[D / 32];
            load_slice<D>(a.q + row * D, lane, qv);
            load_slice<D>(a.dout + row * D, lane, gv);
#pragma unroll
            for (int e = 0; e < D / 32; ++e) {
                dk[e] = fmaf(dsu, qv[e], dk[e]);
                dv[e] = fmaf(pu, gv[e], dv[e]);
            }
        }
    }
#pragma unroll
    for (int e = 0; e < D / 32; ++e) dk[e] *= a.scale;
    store_slice<D>(dk_prefix + (size_t)key * D, lane, dk);
    store_slice<D>(dv_prefix + (size_t)key * D, lane, dv);
}

inline unsigned int blocks_for(long long items)
{
    return (unsigned int)((items + kWarpsPerBlock - 1) / kWarpsPerBlock);
}

}  // namespace

cudaError_t launch_simt_fwd(const FwdArgs &a, cudaStream_t stream)
{
    const long long rows = (long long)a.dims.B * a.dims.Hq * a.dims.S;
    KernelTiming timing(kKernelFwdSimt, stream);
    if (a.dims.d == 128)
        simt_fwd_kernel<128><<<blocks_for(rows), kWarpsPerBlock * 32, 0, stream>>>(a);
    else
        simt_fwd_kernel<64><<<blocks_for(rows), kWarpsPerBlock * 32, 0, stream>>>(a);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_simt_row_dot(const BwdArgs &a, cudaStream_t stream)
{
    const long long rows = (long long)a.dims.B * a.dims.Hq * a.dims.S;
    KernelTiming timing(kKernelRowDot, stream);
    if (a.dims.d == 128)
        simt_row_dot_kernel<128><<<blocks_for((rows + 2 * kRowDotUnroll - 1) / (2 * kRowDotUnroll)), kWarpsPerBlock * 32, 0,
                                   stream>>>(a);
    else
        simt_row_dot_kernel<64><<<blocks_for((rows + 4 * kRowDotUnroll - 1) / (4 * kRowDotUnroll)), kWarpsPerBlock * 32, 0,
                                  stream>>>(a);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_simt_bwd_dkv(const BwdArgs &a, cudaStream_t stream)
{
    const long long keys = (long long)a.dims.B * a.dims.Hkv * a.dims.Skv;
    KernelTiming timing(kKernelBwdDkvSimt, stream);
    if (a.dims.d == 128)
        simt_bwd_dkv_kernel<128><<<blocks_for(keys), kWarpsPerBlock * 32, 0, stream>>>(a);
    else
        simt_bwd_dkv_kernel<64><<<blocks_for(keys), kWarpsPerBlock * 32, 0, stream>>>(a);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_simt_bwd_prefix(const BwdArgs &a, __nv_bfloat16 *dk_prefix, __nv_bfloat16 *dv_prefix, cudaStream_t stream)
{
    const long long keys = (long long)a.dims.Hkv * a.dims.P;
    KernelTiming timing(kKernelBwdPrefixSimt, stream);
    if (a.dims.d == 128)
        simt_bwd_prefix_kernel<128><<<blocks_for(keys), kWarpsPerBlock * 32, 0, stream>>>(a, dk_prefix, dv_prefix);
    else
        simt_bwd_prefix_kernel<64><<<blocks_for(keys), kWarpsPerBlock * 32, 0, stream>>>(a, dk_prefix, dv_prefix);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_simt_bwd(const BwdArgs &a, cudaStream_t stream)
{
    const long long rows = (long long)a.dims.B * a.dims.Hq * a.dims.S;
    const long long keys = (long long)a.dims.B * a.dims.Hkv * a.dims.Skv;
    {
        KernelTiming timing(kKernelBwdDqSimt, stream);
        if (a.dims.d == 128)
            simt_bwd_dq_kernel<128><<<blocks_for(rows), kWarpsPerBlock * 32, 0, stream>>>(a);
        else
            simt_bwd_dq_kernel<64><<<blocks_for(rows), kWarpsPerBlock * 32, 0, stream>>>(a);
    }
    {
        KernelTiming timing(kKernelBwdDkvSimt, stream);
        if (a.dims.d == 128)
            simt_bwd_dkv_kernel<128><<<blocks_for(keys), kWarpsPerBlock * 32, 0, stream>>>(a);
        else
            simt_bwd_dkv_kernel<64><<<blocks_for(keys), kWarpsPerBlock * 32, 0, stream>>>(a);
    }
    count_launches(2);
    return cudaGetLastError();
}

}  // namespace pskv
