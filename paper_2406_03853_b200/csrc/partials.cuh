// Device helpers for consumers of projection results: gathering the fp32 partial sums a
// projection left behind (PartView) and the RMSNorm scale of a row (RowScale).
#pragma once
#include "common.cuh"
#include "kernels.cuh"

namespace eesd {

// Sum of the partial results of output elements (m, r .. r + N - 1), N = 1, 2 or 4 (r % N == 0,
// so they share a weight tile), in a fixed order.
template <int N> struct PartVec;
template <> struct PartVec<1> { typedef float T; };
template <> struct PartVec<2> { typedef float2 T; };
template <> struct PartVec<4> { typedef float4 T; };
__device__ __forceinline__ void vadd(float &a, float b) { a += b; }
__device__ __forceinline__ void vadd(float2 &a, float2 b) { a.x += b.x; a.y += b.y; }
__device__ __forceinline__ void vadd(float4 &a, float4 b) { a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; }

// blocks of one tile, first to last (CTA order), with up to kGatherFlight loads in flight: a tile of a
// narrow projection is shared by eight to ten CTAs, and loads issued one after the other would
// each cost a round trip to L2
constexpr int kGatherFlight = 12;
template <int N>
__device__ __forceinline__ typename PartVec<N>::T part_sum_blocks(const float *p, int n) {
    typedef typename PartVec<N>::T V;
    constexpr size_t BS = (size_t)kMaxRows * 128;   // floats per block
    V a[kGatherFlight];
#pragma unroll
    for (int i = 0; i < kGatherFlight; i++) a[i] = i < n ? __ldcg(reinterpret_cast<const V *>(p + (size_t)i * BS)) : V();
    V v = a[0];
#pragma unroll
    for (int i = 1; i < kGatherFlight; i++) vadd(v, a[i]);   // absent blocks add zero
    for (int i = kGatherFlight; i < n; i++) vadd(v, __ldcg(reinterpret_cast<const V *>(p + (size_t)i * BS)));
    return v;
}

template <int N>
__device__ __forceinline__ typename PartVec<N>::T part_gather_n(const PartView &pv, int m, int r) {
    typedef typename PartVec<N>::T V;
    if (pv.mode == 0) {
        V v = V();
        for (int s = 0; s < pv.S; s++)
            vadd(v, *reinterpret_cast<const V *>(pv.base + (size_t)s * pv.split_stride + (size_t)m * pv.R + r));
        return v;
    }
    const int t = r >> 7;
    const int c0 = pv.sk.owner(t * pv.sk.KB), n = pv.sk.owner((t + 1) * pv.sk.KB - 1) - c0 + 1;
    return part_sum_blocks<N>(pv.base + ((size_t)(c0 + t) * kMaxRows + m) * 128 + (r & 127), n);
}
// same for the stream-K layout when the tile's {first block, block count} is already known
template <int N>
__device__ __forceinline__ typename PartVec<N>::T part_gather_blocks(const PartView &pv, int2 tb, int m, int r) {
    return part_sum_blocks<N>(pv.base + ((size_t)tb.x * kMaxRows + m) * 128 + (r & 127), tb.y);
}
__device__ __forceinline__ int2 tile_blocks(const StreamK &sk, int t) {
    const int c0 = sk.owner(t * sk.KB);
    return make_int2(c0 + t, sk.owner((t + 1) * sk.KB - 1) - c0 + 1);
}
__device__ __forceinline__ float part_gather(const PartView &pv, int m, int r) { return part_gather_n<1>(pv, m, r); }
__device__ __forceinline__ float4 part_gather4(const PartView &pv, int m, int r) { return part_gather_n<4>(pv, m, r); }

__device__ __forceinline__ float row_rstd(const RowScale &rs, int m) {
    if (!rs.ssq) return 1.0f;
    float v[kSsqBlocks];
#pragma unroll
    for (int b = 0; b < kSsqBlocks; b++) v[b] = b < rs.nblk ? rs.ssq[m * kSsqBlocks + b] : 0.f;   // all loads in flight
    float t = 0.f;
#pragma unroll
    for (int b = 0; b < kSsqBlocks; b++) t += v[b];
    return 1.0f / sqrtf(t * rs.inv_d + rs.eps);
}

}  // namespace eesd
