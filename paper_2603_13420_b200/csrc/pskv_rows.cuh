// Warp-per-row building blocks of the general CUDA-core kernels: one warp owns one query row, the
// prefix K/V is read in place (shared by all candidates, Sec. 4.2) and the softmax is one continued
// online softmax over the prefix keys followed by the causally visible suffix keys (Eq. 2).  Shared
// by the general kernels and by the tensor-core forward, which recomputes its rare out-of-range rows
// with the same routine.
#pragma once
#include "pskv_common.cuh"

namespace pskv {
namespace {

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// <x (fp32, shared memory), row (bf16, global)> over D elements, 16-byte loads.
template <int D>
__device__ __forceinline__ float dot_row(const float *x, const __nv_bfloat16 *row)
{
    const uint4 *r4 = reinterpret_cast<const uint4 *>(row);
    float acc = 0.f;
#pragma unroll
    for (int v = 0; v < D / 8; ++v) {
        uint4 u = __ldg(r4 + v);
        const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&u);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float2 f = __bfloat1622float2(h[e]);
            acc = fmaf(x[v * 8 + 2 * e], f.x, acc);
            acc = fmaf(x[v * 8 + 2 * e + 1], f.y, acc);
        }
    }
    return acc;
}

// The lane's D/32 consecutive columns of a bf16 row, widened.
template <int D>
__device__ __forceinline__ void load_slice(const __nv_bfloat16 *row, int lane, float (&v)[D / 32])
{
    if constexpr (D == 128) {
        uint2 u = __ldg(reinterpret_cast<const uint2 *>(row) + lane);
        const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&u);
        float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]);
        v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y;
    } else {
        unsigned int u = __ldg(reinterpret_cast<const unsigned int *>(row) + lane);
        float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&u));
        v[0] = a.x; v[1] = a.y;
    }
}

template <int D>
__device__ __forceinline__ void store_slice(__nv_bfloat16 *row, int lane, const float (&v)[D / 32])
{
    if constexpr (D == 128) {
        __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]);
        __nv_bfloat162 b = __floats2bfloat162_rn(v[2], v[3]);
        uint2 u;
        u.x = *reinterpret_cast<unsigned int *>(&a);
        u.y = *reinterpret_cast<unsigned int *>(&b);
        reinterpret_cast<uint2 *>(row)[lane] = u;
    } else {
        __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]);
        reinterpret_cast<unsigned int *>(row)[lane] = *reinterpret_cast<unsigned int *>(&a);
    }
}

template <int D>
__device__ __forceinline__ void stage_row(float *dst, const __nv_bfloat16 *row, int lane)
{
    float v[D / 32];
    load_slice<D>(row, lane, v);
#pragma unroll
    for (int e = 0; e < D / 32; ++e) dst[lane * (D / 32) + e] = v[e];
}

// Forward for one query row (b,h,i) by one warp; lanes take 32 keys at a time.  `q_s` is this
// warp's D floats of shared memory.
template <int D>
__device__ __forceinline__ void fwd_row(const FwdArgs &a, long long row, float *q_s, int lane)
{
    const Dims dm = a.dims;
    const int i = (int)(row % dm.S);
    const int h = (int)((row / dm.S) % dm.Hq);
    const int b = (int)(row / ((long long)dm.S * dm.Hq));
    const int g = h / dm.n_rep;
    const __nv_bfloat16 *pk = a.prefix_k + (size_t)g * dm.Pstride * D;
    const __nv_bfloat16 *pv = a.prefix_v + (size_t)g * dm.Pstride * D;
    const __nv_bfloat16 *sk = a.suffix_k + ((size_t)b * dm.Hkv + g) * dm.Skv * D;
    const __nv_bfloat16 *sv = a.suffix_v + ((size_t)b * dm.Hkv + g) * dm.Skv * D;

    stage_row<D>(q_s, a.q + (size_t)row * D, lane);
    __syncwarp();

    const float scale2 = a.scale * kLog2e;
    // the query is suffix token L - S + i of its candidate: it sees the prefix and suffix keys up to itself
    const int n_vis = dm.P + suffix_tokens(a.suffix_len, b, dm.S, dm.Skv) - dm.S + i + 1;
    float m = -INFINITY, l = 0.f;
    float acc[D / 32];
#pragma unroll
    for (int e = 0; e < D / 32; ++e) acc[e] = 0.f;

    for (int j0 = 0; j0 < n_vis; j0 += 32) {
        const int j = j0 + lane;
        float s = -INFINITY;
        if (j < n_vis) {
            const __nv_bfloat16 *krow = (j < dm.P) ? pk + (size_t)j * D : sk + (size_t)(j - dm.P) * D;
            s = scale2 * dot_row<D>(q_s, krow);
        }
        const float m_new = fmaxf(m, warp_max(s));  // finite: key j0 is always visible
        const float p = exp2f(s - m_new);           // 0 for lanes past n_vis
        const float corr = exp2f(m - m_new);        // 0 on the first chunk (m = -inf)
        l = l * corr + warp_sum(p);
#pragma unroll
        for (int e = 0; e < D / 32; ++e) acc[e] *= corr;
        const int cnt = min(32, n_vis - j0);
        for (int t = 0; t < cnt; ++t) {
            const float pt = __shfl_sync(0xffffffffu, p, t);
            const int jj = j0 + t;
            const __nv_bfloat16 *vrow = (jj < dm.P) ? pv + (size_t)jj * D : sv + (size_t)(jj - dm.P) * D;
            float v[D / 32];
            load_slice<D>(vrow, lane, v);
#pragma unroll
            for (int e = 0; e < D / 32; ++e) acc[e] = fmaf(pt, v[e], acc[e]);
        }
        m = m_new;
    }
    const float inv = 1.f / l;
#pragma unroll
    for (int e = 0; e < D / 32; ++e) acc[e] *= inv;
    store_slice<D>(a.out + (size_t)row * D, lane, acc);
    if (lane == 0) a.lse[row] = (m + log2f(l)) * kLn2;
    __syncwarp();
}

}  // namespace
}  // namespace pskv
