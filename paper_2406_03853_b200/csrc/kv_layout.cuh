// Element order inside one (page, K | V, KV head) block of the paged cache: page_tokens x D elements.
//
// fp32 cache (SIMT attention): keys transposed per page, [D/2][page_tokens][2] (pairs of adjacent
// dimensions, one column per token); values [page_tokens][D] with the 16-byte chunks of token t's
// row permuted (chunk c at c ^ (t & 7)).
//
// bf16 cache (tensor-core attention): both blocks are grids of 8 x 8 core matrices (128 contiguous
// bytes each), [token / 8][D / 8][8][8], which is the un-swizzled operand form of tcgen05.mma, so a
// page block copied to shared memory as it is can be an MMA operand:
//   keys    core matrix = 8 tokens (rows) x 8 dimensions  -> A operand of S^T = K Q^T (contraction over D)
//   values  core matrix = 8 dimensions (rows) x 8 tokens  -> A operand of O^T = V^T P^T (contraction over tokens)
// Page blocks of consecutive pages placed one after the other in shared memory continue the
// token / 8 index, so a slice of several pages is one operand with uniform strides.
#pragma once
#include "common.cuh"

namespace eesd {

// 16-byte chunk permutation of the fp32 value rows
template <typename AT> __device__ __forceinline__ int v_elem(int pos, int e) {
    constexpr int CPV = 16 / (int)sizeof(AT);
    return (((e / CPV) ^ (pos & 7)) * CPV) + (e % CPV);
}

// index of key element (token p of the page, dimension e); pos = absolute position of the token
template <typename AT> __device__ __forceinline__ size_t k_index(int p, int e, int PT, int D);
template <typename AT> __device__ __forceinline__ size_t v_index(int pos, int p, int e, int PT, int D);

template <> __device__ __forceinline__ size_t k_index<float>(int p, int e, int PT, int) {
    return ((size_t)(e >> 1) * PT + p) * 2 + (e & 1);
}
template <> __device__ __forceinline__ size_t v_index<float>(int pos, int p, int e, int, int D) {
    return (size_t)p * D + v_elem<float>(pos, e);
}
template <> __device__ __forceinline__ size_t k_index<__nv_bfloat16>(int p, int e, int, int D) {
    return ((size_t)(p >> 3) * (D >> 3) + (e >> 3)) * 64 + (p & 7) * 8 + (e & 7);
}
template <> __device__ __forceinline__ size_t v_index<__nv_bfloat16>(int, int p, int e, int, int D) {
    return ((size_t)(p >> 3) * (D >> 3) + (e >> 3)) * 64 + (e & 7) * 8 + (p & 7);
}

}  // namespace eesd
