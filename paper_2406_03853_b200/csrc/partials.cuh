// Device helpers for consumers of projection results: gathering the fp32 partial sums a
// projection left behind (PartView) and the RMSNorm scale of a row (RowScale).
#pragma once
#include "common.cuh"
#include "kernels.cuh"

namespace eesd {

// Sum of the partial results of output elements (m, r .. r + N - 1), N = 1, 2 or 4 (r % N == 0,
// so they share a weight tile), in a fixed order.  All loads of up to four blocks are issued
// before the first add, so a gather costs one round trip to L2, not one per block.
template <int N> struct PartVec;
template <> struct PartVec<1> { typedef float T; };
template <> struct PartVec<2> { typedef float2 T; };
template <> struct PartVec<4> { typedef float4 T; };
__device__ __forceinline__ void vadd(float &a, float b) { a += b; }
__device__ __forceinline__ void vadd(float2 &a, float2 b) { a.x += b.x; a.y += b.y; }
__device__ __forceinline__ void vadd(float4 &a, float4 b) { a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; }

template <int N>
__device__ __forceinline__ typename PartVec<N>::T part_gather_n(const PartView &pv, int m, int r) {
    typedef typename PartVec<N>::T V;
    V v = V();
    if (pv.mode == 0) {
        for (int s = 0; s < pv.S; s++)
            vadd(v, *reinterpret_cast<const V *>(pv.base + (size_t)s * pv.split_stride + (size_t)m * pv.R + r));
    } else {
        const int t = r >> 7;
        const int c0 = pv.sk.owner(t * pv.sk.KB), n = pv.sk.owner((t + 1) * pv.sk.KB - 1) - c0 + 1;
        constexpr size_t BS = (size_t)kMaxRows * 128;   // floats per block
        const V *p = reinterpret_cast<const V *>(pv.base + ((size_t)(c0 + t) * kMaxRows + m) * 128 + (r & 127));
        const V *p1 = reinterpret_cast<const V *>(reinterpret_cast<const float *>(p) + BS);
        const V *p2 = reinterpret_cast<const V *>(reinterpret_cast<const float *>(p) + 2 * BS);
        const V *p3 = reinterpret_cast<const V *>(reinterpret_cast<const float *>(p) + 3 * BS);
        const V a0 = __ldcg(p);
        const V a1 = n > 1 ? __ldcg(p1) : V();
        const V a2 = n > 2 ? __ldcg(p2) : V();
        const V a3 = n > 3 ? __ldcg(p3) : V();
        v = a0;
        vadd(v, a1);
        vadd(v, a2);
        vadd(v, a3);
        for (int i = 4; i < n; i++)
            vadd(v, __ldcg(reinterpret_cast<const V *>(reinterpret_cast<const float *>(p) + (size_t)i * BS)));
    }
    return v;
}
// same for the stream-K layout when the tile's {first block, block count} is already known
template <int N>
__device__ __forceinline__ typename PartVec<N>::T part_gather_blocks(const PartView &pv, int2 tb, int m, int r) {
    typedef typename PartVec<N>::T V;
    constexpr size_t BS = (size_t)kMaxRows * 128;
    const float *p = pv.base + ((size_t)tb.x * kMaxRows + m) * 128 + (r & 127);
    const V a0 = __ldcg(reinterpret_cast<const V *>(p));
    const V a1 = tb.y > 1 ? __ldcg(reinterpret_cast<const V *>(p + BS)) : V();
    const V a2 = tb.y > 2 ? __ldcg(reinterpret_cast<const V *>(p + 2 * BS)) : V();
    const V a3 = tb.y > 3 ? __ldcg(reinterpret_cast<const V *>(p + 3 * BS)) : V();
    V v = a0;
    vadd(v, a1);
    vadd(v, a2);
    vadd(v, a3);
    for (int i = 4; i < tb.y; i++) vadd(v, __ldcg(reinterpret_cast<const V *>(p + (size_t)i * BS)));
    return v;
}
__device__ __forceinline__ int2 tile_blocks(const StreamK &sk, int t) {
    const int c0 = sk.owner(t * sk.KB);
    return make_int2(c0 + t, sk.owner((t + 1) * sk.KB - 1) - c0 + 1);
}
__device__ __forceinline__ float part_gather(const PartView &pv, int m, int r) { return part_gather_n<1>(pv, m, r); }
__device__ __forceinline__ float4 part_gather4(const PartView &pv, int m, int r) { return part_gather_n<4>(pv, m, r); }

__device__ __forceinline__ float row_rstd(const RowScale &rs, int m) {
    if (!rs.ssq) return 1.0f;
    float t = 0.f;
    for (int b = 0; b < rs.nblk; b++) t += rs.ssq[m * kSsqBlocks + b];
    return 1.0f / sqrtf(t * rs.inv_d + rs.eps);
}

}  // namespace eesd
