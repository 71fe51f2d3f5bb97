// Shared device helpers for the EESD kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace eesd {

constexpr int kMaxRows = 16;  // most token rows per pass

// error bits written to the context's device error word
constexpr int kErrBadToken = 1;
constexpr int kErrWaitTimeout = 2;
constexpr int kErrBadPage = 4;
constexpr int kErrPlan = 8;   // a launcher was asked for more attention slices than can be merged (the configuration check prevents it)

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// 16-byte load of consecutive elements widened to fp32 (8 bf16 or 4 fp32)
template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int N = 4;
    __device__ __forceinline__ static void load(const float *p, float *o) {
        float4 v = __ldg(reinterpret_cast<const float4 *>(p));
        o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
    }
    __device__ __forceinline__ static void load_stream(const float *p, float *o) {
        float4 v = __ldcs(reinterpret_cast<const float4 *>(p));
        o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    __device__ __forceinline__ static void unpack(uint4 v, float *o) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; i++) {
            o[2 * i] = __uint_as_float(w[i] << 16);
            o[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    __device__ __forceinline__ static void load(const __nv_bfloat16 *p, float *o) {
        unpack(__ldg(reinterpret_cast<const uint4 *>(p)), o);
    }
    __device__ __forceinline__ static void load_stream(const __nv_bfloat16 *p, float *o) {
        unpack(__ldcs(reinterpret_cast<const uint4 *>(p)), o);
    }
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// block-wide sum with a fixed combination order (deterministic); all threads get the result
__device__ __forceinline__ float block_sum(float v, float *scratch /* >= 33 floats */) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int i = 0; i < nw; i++) t += scratch[i];
        scratch[32] = t;
    }
    __syncthreads();
    return scratch[32];
}

// the same sum (same order of additions) delivered to thread 0 only: one barrier instead of three
__device__ __forceinline__ float block_sum_thread0(float v, float *scratch /* >= 32 floats */) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    float t = 0.f;
    if (threadIdx.x == 0)
        for (int i = 0; i < nw; i++) t += scratch[i];
    return t;
}

// Programmatic dependent launch.  pdl_trigger lets the next kernel in the stream be scheduled
// early; pdl_wait blocks until every kernel this one depends on has completed and its writes
// are visible.  Both are no-ops for kernels launched without the attribute.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline void launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, bool pdl, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// writes v as two bf16 terms into a [chunk][hi | lo][kMaxRows][K] matrix: token row m belongs to
// chunk m / kMaxRows; its hi term goes to row m % kMaxRows of the chunk's first half, its lo
// term to the same row of the second half (one chunk, [2 * kMaxRows][K], in a decode pass)
__device__ __forceinline__ void store_split(__nv_bfloat16 *xs, int m, size_t K, size_t i, float v) {
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    const size_t row = (size_t)(m / kMaxRows) * (2 * kMaxRows) + (size_t)(m % kMaxRows);
    xs[row * K + i] = hi;
    xs[(row + kMaxRows) * K + i] = __float2bfloat16_rn(v - __bfloat162float(hi));
}

// four consecutive elements at once (i % 4 == 0): one 8-byte store per term
__device__ __forceinline__ void store_split4(__nv_bfloat16 *xs, int m, size_t K, size_t i, float4 v) {
    const __nv_bfloat16 h0 = __float2bfloat16_rn(v.x), h1 = __float2bfloat16_rn(v.y), h2 = __float2bfloat16_rn(v.z), h3 = __float2bfloat16_rn(v.w);
    const __nv_bfloat16 l0 = __float2bfloat16_rn(v.x - __bfloat162float(h0)), l1 = __float2bfloat16_rn(v.y - __bfloat162float(h1));
    const __nv_bfloat16 l2 = __float2bfloat16_rn(v.z - __bfloat162float(h2)), l3 = __float2bfloat16_rn(v.w - __bfloat162float(h3));
    auto pack = [](__nv_bfloat16 a, __nv_bfloat16 b) { return (uint32_t)__bfloat16_as_ushort(a) | ((uint32_t)__bfloat16_as_ushort(b) << 16); };
    const size_t row = (size_t)(m / kMaxRows) * (2 * kMaxRows) + (size_t)(m % kMaxRows);
    *reinterpret_cast<uint2 *>(xs + row * K + i) = make_uint2(pack(h0, h1), pack(h2, h3));
    *reinterpret_cast<uint2 *>(xs + (row + kMaxRows) * K + i) = make_uint2(pack(l0, l1), pack(l2, l3));
}

}  // namespace eesd
