// Model kernels of the EESD decode round (sm_100a): embedding gather, residual + RMSNorm,
// skinny projections (M <= 16 token rows against a streamed weight matrix), RoPE + paged KV
// append, paged decode attention with a causal block of new rows, SwiGLU.
//
// Every reduction has a fixed combination order, so a pass is bit-reproducible.
#include <stdlib.h>

#include "common.cuh"
#include "kernels.cuh"
#include "kv_layout.cuh"
#include "partials.cuh"
#include "tc_ptx.cuh"

namespace eesd {

typedef __nv_bfloat16 bf16;

bool pdl_enabled() {
    static const bool on = getenv("EESD_NO_PDL") == nullptr;   // read once (thread-safe static initialisation)
    return on;
}

// ------------------------------------------------------------------------------------ small utilities
__global__ void set_ints_kernel(int32_t *dst, IntList16 vals, int n) {
    if (threadIdx.x < n) dst[threadIdx.x] = vals.v[threadIdx.x];
}
void launch_set_ints(cudaStream_t s, int32_t *dst, const IntList16 &vals, int n) {
    set_ints_kernel<<<1, 32, 0, s>>>(dst, vals, n);
}

// cos/sin of pos * theta^(-2i/D), evaluated in fp64 and rounded once to fp32
__global__ void rope_table_kernel(float2 *table, int max_ctx, int half, double log_theta, int D) {
    int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= max_ctx * half) return;
    int pos = idx / half, i = idx % half;
    double inv = exp(-2.0 * (double)i / (double)D * log_theta);
    double sn, cs;
    sincos((double)pos * inv, &sn, &cs);
    table[idx] = make_float2((float)cs, (float)sn);
}
void launch_rope_table(cudaStream_t s, float2 *table, int max_ctx, int D, float theta) {
    int n = max_ctx * (D / 2);
    rope_table_kernel<<<(n + 255) / 256, 256, 0, s>>>(table, max_ctx, D / 2, log((double)theta), D);
}

// ------------------------------------------------------------------------------------ residual + RMSNorm
// grid (ceil(d / 1024), M), 256 threads, four elements per thread.
// x[m] += partial sums; y = x[m] * g (fp32 and / or two bf16 terms); ssq[m][block] = sum x^2.
// The RMSNorm scale itself is applied by whoever consumes the projection of y (RowScale).
__global__ void __launch_bounds__(256) resid_kernel(float *x, PartView pv, int has_part, const float *g, float *xn, bf16 *xs,
                                                    float *cap, float *ssq, int d) {
    __shared__ float scratch[33];
    const int m = blockIdx.y, i = blockIdx.x * 1024 + threadIdx.x * 4;
    pdl_trigger();
    pdl_wait();
    float ss = 0.f;
    if (i < d) {
        float *xr = x + (size_t)m * d;
        float4 v = *reinterpret_cast<const float4 *>(xr + i);
        if (has_part) {
            const float4 p = part_gather4(pv, m, i);
            v.x += p.x; v.y += p.y; v.z += p.z; v.w += p.w;
            *reinterpret_cast<float4 *>(xr + i) = v;
        }
        if (cap) *reinterpret_cast<float4 *>(cap + (size_t)m * d + i) = v;
        ss = fmaf(v.w, v.w, fmaf(v.z, v.z, fmaf(v.y, v.y, v.x * v.x)));   // one fixed form wherever these sums are taken
        const float4 g4 = *reinterpret_cast<const float4 *>(g + i);
        const float4 y = make_float4(v.x * g4.x, v.y * g4.y, v.z * g4.z, v.w * g4.w);
        if (xn) *reinterpret_cast<float4 *>(xn + (size_t)m * d + i) = y;
        if (xs) store_split4(xs, m, d, i, y);
    }
    ss = block_sum_thread0(ss, scratch);
    if (threadIdx.x == 0) ssq[m * kSsqBlocks + blockIdx.x] = ss;
}
void launch_resid(cudaStream_t s, float *x, const PartView *pv, const float *g, float *xn, void *xs, float *cap,
                  float *ssq, int M, int d) {
    PartView none = {};
    launch_k(resid_kernel, dim3((d + 1023) / 1024, M), dim3(256), 0, s, pdl_enabled(), x, pv ? *pv : none,
             (int)(pv != nullptr), g, xn, (bf16 *)xs, cap, ssq, d);
}

// Embedding gather and the first layer's rows in one kernel: x[m] = E[token]; then what resid_kernel does with x
// (y = x * g as fp32 and / or two bf16 terms, the sums of squares per 1024 columns, the captured copy).  Same grid
// and the same arithmetic as resid_kernel, so the rows are those of a plain gather followed by resid_kernel.
template <typename WT>
__global__ void __launch_bounds__(256) embed_resid_kernel(const int32_t *tok, int tok_stride, const WT *E, int V, float *x, const float *g,
                                                          float *xn, bf16 *xs, float *cap, float *ssq, int d, int *err) {
    __shared__ float scratch[33];
    const int m = blockIdx.y, i = blockIdx.x * 1024 + threadIdx.x * 4;
    pdl_trigger();
    pdl_wait();
    int t = tok[(size_t)m * tok_stride];
    if (t < 0 || t >= V) {
        if (threadIdx.x == 0 && blockIdx.x == 0) atomicOr(err, kErrBadToken);
        t = 0;
    }
    float ss = 0.f;
    if (i < d) {
        const WT *row = E + (size_t)t * d + i;
        const float4 v = make_float4(to_f(row[0]), to_f(row[1]), to_f(row[2]), to_f(row[3]));
        *reinterpret_cast<float4 *>(x + (size_t)m * d + i) = v;
        if (cap) *reinterpret_cast<float4 *>(cap + (size_t)m * d + i) = v;
        ss = fmaf(v.w, v.w, fmaf(v.z, v.z, fmaf(v.y, v.y, v.x * v.x)));   // one fixed form wherever these sums are taken
        const float4 g4 = *reinterpret_cast<const float4 *>(g + i);
        const float4 y = make_float4(v.x * g4.x, v.y * g4.y, v.z * g4.z, v.w * g4.w);
        if (xn) *reinterpret_cast<float4 *>(xn + (size_t)m * d + i) = y;
        if (xs) store_split4(xs, m, d, i, y);
    }
    ss = block_sum_thread0(ss, scratch);
    if (threadIdx.x == 0) ssq[m * kSsqBlocks + blockIdx.x] = ss;
}
void launch_embed_resid(cudaStream_t s, int dtype, const int32_t *tok, int tok_stride, const void *E, int V, float *x, const float *g,
                        float *xn, void *xs, float *cap, float *ssq, int M, int d, int *err) {
    const dim3 grid((d + 1023) / 1024, M);
    if (dtype == 0) launch_k(embed_resid_kernel<float>, grid, dim3(256), 0, s, pdl_enabled(), tok, tok_stride, (const float *)E, V, x, g, xn, (bf16 *)xs, cap, ssq, d, err);
    else launch_k(embed_resid_kernel<bf16>, grid, dim3(256), 0, s, pdl_enabled(), tok, tok_stride, (const bf16 *)E, V, x, g, xn, (bf16 *)xs, cap, ssq, d, err);
}

// ------------------------------------------------------------------------------------ skinny projection (SIMT)
// out[m][r] = sum_k A[m][k] W[r][k] for m < M <= MT rows.  Each warp owns 4 weight rows and
// streams them with 16-byte loads; the token rows sit in shared memory as fp32.  The k order
// per lane and the lane combination tree do not depend on M.
template <typename WT, typename AT, int MT>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const AT *__restrict__ A, const WT *__restrict__ W,
                                                        float *__restrict__ out, int M, int R, int K) {
    constexpr int VEC = Vec16<WT>::N;
    constexpr int KC = 32 * VEC * 2;  // k elements per staged chunk (two vectors per lane)
    __shared__ __align__(16) float sA[MT][KC];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int r0 = blockIdx.x * 32 + warp * 4;
    pdl_trigger();
    pdl_wait();
    float acc[4][MT];
#pragma unroll
    for (int rr = 0; rr < 4; rr++)
#pragma unroll
        for (int m = 0; m < MT; m++) acc[rr][m] = 0.f;

    for (int k0 = 0; k0 < K; k0 += KC) {
        __syncthreads();
        for (int idx = tid; idx < MT * KC; idx += 256) {
            int m = idx / KC, kk = idx - m * KC;
            sA[m][kk] = (m < M && k0 + kk < K) ? to_f(A[(size_t)m * K + k0 + kk]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < 2; j++) {
            const int kk = j * 32 * VEC + lane * VEC;
            if (k0 + kk < K) {
                float w[4][VEC];
#pragma unroll
                for (int rr = 0; rr < 4; rr++) {
                    if (r0 + rr < R) Vec16<WT>::load_stream(W + (size_t)(r0 + rr) * K + k0 + kk, w[rr]);
                    else {
#pragma unroll
                        for (int v = 0; v < VEC; v++) w[rr][v] = 0.f;
                    }
                }
#pragma unroll
                for (int m = 0; m < MT; m++) {
                    float a[VEC];
#pragma unroll
                    for (int v = 0; v < VEC; v += 4) {
                        float4 t = *reinterpret_cast<const float4 *>(&sA[m][kk + v]);
                        a[v] = t.x; a[v + 1] = t.y; a[v + 2] = t.z; a[v + 3] = t.w;
                    }
#pragma unroll
                    for (int rr = 0; rr < 4; rr++)
#pragma unroll
                        for (int v = 0; v < VEC; v++) acc[rr][m] = fmaf(w[rr][v], a[v], acc[rr][m]);
                }
            }
        }
    }
#pragma unroll
    for (int rr = 0; rr < 4; rr++)
#pragma unroll
        for (int m = 0; m < MT; m++) {
            float v = warp_sum(acc[rr][m]);
            if (lane == 0 && m < M && r0 + rr < R) out[(size_t)m * R + r0 + rr] = v;
        }
}

template <typename WT, typename AT>
static void gemm_simt_dispatch(cudaStream_t s, const void *A, const void *W, float *out, int M, int R, int K) {
    dim3 grid((R + 31) / 32);
    const AT *a = (const AT *)A;
    const WT *w = (const WT *)W;
    const bool pdl = pdl_enabled();
    if (M <= 1) launch_k(gemm_simt_kernel<WT, AT, 1>, grid, dim3(256), 0, s, pdl, a, w, out, M, R, K);
    else if (M <= 2) launch_k(gemm_simt_kernel<WT, AT, 2>, grid, dim3(256), 0, s, pdl, a, w, out, M, R, K);
    else if (M <= 4) launch_k(gemm_simt_kernel<WT, AT, 4>, grid, dim3(256), 0, s, pdl, a, w, out, M, R, K);
    else if (M <= 8) launch_k(gemm_simt_kernel<WT, AT, 8>, grid, dim3(256), 0, s, pdl, a, w, out, M, R, K);
    else launch_k(gemm_simt_kernel<WT, AT, 16>, grid, dim3(256), 0, s, pdl, a, w, out, M, R, K);
}

int launch_gemm(cudaStream_t s, int dtype, const float *A, const void *W, float *out, int M, int R, int K) {
    if (dtype == 0) gemm_simt_dispatch<float, float>(s, A, W, out, M, R, K);
    else gemm_simt_dispatch<bf16, float>(s, A, W, out, M, R, K);
    return 1;
}

// ------------------------------------------------------------------------------------ RoPE + KV append
// grid (heads, M), block D/2: one thread per rotation pair.
template <typename AT>
__global__ void qkv_post_kernel(PartView pv, RowScale rs, int pos0, int H, KvGeom kv, const float2 *rope, float *q,
                                int head_off, int col_off, int *err, TreeRows tr, int tree_on, int row0) {
    const int hh = blockIdx.x + head_off;  // 0..H-1 q, H..H+Hkv-1 k, then v
    const int m = blockIdx.y, i = threadIdx.x, D = kv.D;   // row row0 + m of the pass is position pos0 + m
    const int col = col_off + blockIdx.x * D + 2 * i;
    pdl_trigger();
    pdl_wait();
    const float2 pr = part_gather_n<2>(pv, row0 + m, col);
    const float rstd = row_rstd(rs, row0 + m);
    float a = pr.x * rstd, b = pr.y * rstd;
    const int pos = pos0 + m;   // where the row is stored; a tree row is rotated as its depth's position
    if (hh < H + kv.Hkv) {
        float2 cs = rope[(size_t)(tree_on ? pos0 + tr.depth[m & 15] : pos) * (D / 2) + i];
        float ra = a * cs.x - b * cs.y, rb = a * cs.y + b * cs.x;
        a = ra; b = rb;
    }
    if (hh < H) {
        float *dst = q + (size_t)(row0 + m) * H * D + (size_t)hh * D + 2 * i;
        dst[0] = a; dst[1] = b;
        return;
    }
    const int isV = (hh - H) / kv.Hkv, kh = (hh - H) % kv.Hkv;
    const int page = kv.page_table[pos / kv.page_tokens];
    if (page < 0 || page >= kv.n_pages_total) {
        if (i == 0) atomicOr(err, kErrBadPage);
        return;
    }
    AT *blk = (AT *)kv.slot_base + (((size_t)page * 2 + isV) * kv.Hkv + kh) * (size_t)kv.page_tokens * D;
    const int p = pos % kv.page_tokens;   // element order inside a block: kv_layout.cuh
    if (isV) {
        blk[v_index<AT>(pos, p, 2 * i, kv.page_tokens, D)] = from_f<AT>(a);
        blk[v_index<AT>(pos, p, 2 * i + 1, kv.page_tokens, D)] = from_f<AT>(b);
    } else {
        blk[k_index<AT>(p, 2 * i, kv.page_tokens, D)] = from_f<AT>(a);
        blk[k_index<AT>(p, 2 * i + 1, kv.page_tokens, D)] = from_f<AT>(b);
    }
}
void launch_qkv_post(cudaStream_t s, int dtype, const PartView &pv, const RowScale &rs, int M, int pos0, int H,
                     const KvGeom &kv, const float2 *rope, float *q, bool only_kv, int *err, int kv_col0,
                     const TreeRows *tree, int row0) {
    const int heads = only_kv ? 2 * kv.Hkv : H + 2 * kv.Hkv;
    dim3 grid(heads, M);
    const TreeRows tr = tree ? *tree : chain_rows();
    const int tree_on = tree && M <= 16 ? 1 : 0;
    if (dtype == 0) launch_k(qkv_post_kernel<float>, grid, dim3(kv.D / 2), 0, s, pdl_enabled(), pv, rs, pos0, H, kv, rope, q, only_kv ? H : 0, kv_col0, err, tr, tree_on, row0);
    else launch_k(qkv_post_kernel<bf16>, grid, dim3(kv.D / 2), 0, s, pdl_enabled(), pv, rs, pos0, H, kv, rope, q, only_kv ? H : 0, kv_col0, err, tr, tree_on, row0);
}

// Prompt passes (bf16 cache, plain [split][row][column] projection result): keys / values of many rows into the
// cache, one block per (KV head, group of 8 consecutive positions = one row of core matrices).  Threads
// 0 .. D - 1 take (token, 8 key dimensions): scale, rotate, one 16-byte store; threads 128 .. 128 + D - 1 take one
// value dimension of the 8 tokens: one 16-byte store (the row of a value core matrix), keeping what the
// cache holds for tokens of the group that are not part of this pass.
template <int D>
__global__ void __launch_bounds__(256) kv_append_wide_kernel(PartView pv, RowScale rs, int Mtot, int pos0, KvGeom kv, const float2 *rope,
                                                             int kcol0, int *err) {
    __shared__ float s_rstd[8];
    const int kh = blockIdx.x, grp = (pos0 >> 3) + blockIdx.y, tid = threadIdx.x;
    const int PT = kv.page_tokens;
    pdl_trigger();
    pdl_wait();
    if (tid < 8) {
        const int m = grp * 8 + tid - pos0;
        s_rstd[tid] = (m >= 0 && m < Mtot) ? row_rstd(rs, m) : 0.f;
    }
    __syncthreads();
    const int page = kv.page_table[(grp * 8) / PT], pp = (grp * 8) & (PT - 1);   // the group lies inside one page
    if (page < 0 || page >= kv.n_pages_total) {
        if (tid == 0) atomicOr(err, kErrBadPage);
        return;
    }
    unsigned char *blk_k = (unsigned char *)kv.slot_base + (((size_t)page * 2) * kv.Hkv + kh) * (size_t)PT * D * 2;
    unsigned char *blk_v = blk_k + (size_t)kv.Hkv * PT * D * 2;
    if (tid < D) {   // keys: token tt, dimensions 8 c .. 8 c + 7
        const int tt = tid & 7, c = tid >> 3, m = grp * 8 + tt - pos0;
        if (m >= 0 && m < Mtot) {
            float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
            for (int sp = 0; sp < pv.S; sp++) {
                const float4 *src = reinterpret_cast<const float4 *>(pv.base + (size_t)sp * pv.split_stride + (size_t)m * pv.R + kcol0 + kh * D + 8 * c);
                const float4 la = src[0], lb = src[1];
                a.x += la.x; a.y += la.y; a.z += la.z; a.w += la.w;
                b.x += lb.x; b.y += lb.y; b.z += lb.z; b.w += lb.w;
            }
            const float r = s_rstd[tt];
            const float raw[8] = {a.x * r, a.y * r, a.z * r, a.w * r, b.x * r, b.y * r, b.z * r, b.w * r};
            const float4 *cs = reinterpret_cast<const float4 *>(rope + (size_t)(pos0 + m) * (D / 2) + 4 * c);
            const float4 w0 = cs[0], w1 = cs[1];
            const float cw[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};   // (cos, sin) of four pairs
            uint32_t o[4];
#pragma unroll
            for (int i = 0; i < 4; i++) {
                const float x0 = raw[2 * i], x1 = raw[2 * i + 1];
                const float ra = x0 * cw[2 * i] - x1 * cw[2 * i + 1], rb = x0 * cw[2 * i + 1] + x1 * cw[2 * i];
                o[i] = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(ra)) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(rb)) << 16);
            }
            *reinterpret_cast<uint4 *>(blk_k + ((size_t)(pp >> 3) * (D / 8) + c) * 128 + tt * 16) = make_uint4(o[0], o[1], o[2], o[3]);
        }
    } else if (tid >= 128 && tid < 128 + D) {   // values: dimension d of the group's 8 tokens
        const int d = tid - 128;
        uint4 *dst = reinterpret_cast<uint4 *>(blk_v + ((size_t)(pp >> 3) * (D / 8) + (d >> 3)) * 128 + (d & 7) * 16);
        const int m0 = grp * 8 - pos0;
        const bool whole = m0 >= 0 && m0 + 8 <= Mtot;
        uint4 old = make_uint4(0u, 0u, 0u, 0u);
        if (!whole) old = *dst;
        unsigned short h[8] = {(unsigned short)old.x, (unsigned short)(old.x >> 16), (unsigned short)old.y, (unsigned short)(old.y >> 16),
                               (unsigned short)old.z, (unsigned short)(old.z >> 16), (unsigned short)old.w, (unsigned short)(old.w >> 16)};
        float v[8];
#pragma unroll
        for (int tt = 0; tt < 8; tt++) {
            const int m = m0 + tt;
            v[tt] = 0.f;
            if (m >= 0 && m < Mtot)
                for (int sp = 0; sp < pv.S; sp++)
                    v[tt] += pv.base[(size_t)sp * pv.split_stride + (size_t)m * pv.R + kcol0 + (kv.Hkv + kh) * D + d];
        }
#pragma unroll
        for (int tt = 0; tt < 8; tt++) {
            const int m = m0 + tt;
            if (m >= 0 && m < Mtot) h[tt] = __bfloat16_as_ushort(__float2bfloat16_rn(v[tt] * s_rstd[tt]));
        }
        *dst = make_uint4((uint32_t)h[0] | ((uint32_t)h[1] << 16), (uint32_t)h[2] | ((uint32_t)h[3] << 16),
                          (uint32_t)h[4] | ((uint32_t)h[5] << 16), (uint32_t)h[6] | ((uint32_t)h[7] << 16));
    }
}
void launch_kv_append_wide(cudaStream_t s, const PartView &pv, const RowScale &rs, int Mtot, int pos0, const KvGeom &kv,
                           const float2 *rope, int kcol0, int *err) {
    const dim3 grid(kv.Hkv, ((pos0 + Mtot - 1) >> 3) - (pos0 >> 3) + 1);
    if (kv.D == 64) launch_k(kv_append_wide_kernel<64>, grid, dim3(256), 0, s, pdl_enabled(), pv, rs, Mtot, pos0, kv, rope, kcol0, err);
    else launch_k(kv_append_wide_kernel<128>, grid, dim3(256), 0, s, pdl_enabled(), pv, rs, Mtot, pos0, kv, rope, kcol0, err);
}

// ------------------------------------------------------------------------------------ paged decode attention, fp32 cache
// (models with bf16 weights and cache run the tensor-core kernel of attn_tc.cu instead)
// One kernel per layer: RoPE + KV append + attention over the paged cache + merge.
// grid (H_kv, n_split), 256 threads.  Block (kh, sp) owns `cap` cached positions of KV head kh
// (a whole number of pages) and serves every query head of its group and all M new rows from
// ONE copy of those keys and values: the page blocks are brought into shared memory by bulk
// asynchronous copies on one mbarrier, so the cache is read from HBM once per KV head.
// Keys are cached transposed per page ([D/2][page_tokens] pairs), so that in the score phase
// consecutive lanes read consecutive positions of one pair of dimensions (no bank conflicts)
// while the query values are broadcast; values are cached [page_tokens][D].
// The new rows' q, k, v come straight from the QKV projection's partial sums (times the RMSNorm
// scale, rotated); they are gathered while the cached slice is still arriving.  The block whose
// slice holds a new position places that key/value in its tile and appends it to the cache.
// Row m sees positions <= pos0 + m.  Each block writes, per (query head, row), the
// un-normalised output, maximum and sum of its slice; the block that finishes last for a KV
// head (an arrival counter, no waiting) merges the slices in index order.
constexpr int kAttnPos = 192;     // most positions per block
constexpr int kMaxSlices = 64;    // most slices per head (layout of the per-slice maxima and sums)
constexpr int kRows16 = 24;       // up to this many (head, row) pairs per KV head: batches of 16, beyond: of 32

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// RB: (head, row) pairs per block: 8, 16 or 32; NM: most new rows (M <= NM), which sizes the
// unrolled handling of the new keys / values (a one-row pass runs an eighth of the code); TR: the
// new rows form a tree (per-row depth and visibility mask) instead of a chain.  The chain code is
// kept as its own instantiation: with the mask lookups compiled in, an ordinary 13B pass of 1 / 16
// rows measured 4.90 / 5.49 ms against 4.88 / 5.44 ms.
template <int D, int RB, int NM, bool TR>
__global__ void __launch_bounds__(256) attn_kernel(PartView pv, RowScale rs, const float2 *__restrict__ rope, KvGeom kv,
                                                   float *__restrict__ apart, unsigned int *tickets,
                                                   float *__restrict__ attn_out, bf16 *__restrict__ attn_split,
                                                   int M, int pos0, int H, int pps, int n_split, float scale, int *err,
                                                   int nbat, size_t ml_off, TreeRows tr, uint32_t spin, BatchRows br) {
    typedef float AT;
    typedef float2 KP;   // a pair of adjacent head dimensions of one key
    constexpr int HALF = D / 2;
    constexpr int DPL = D / 32;             // output dimensions per lane in the PV phase
    extern __shared__ __align__(128) unsigned char attn_smem[];
    const int PT = kv.page_tokens, group = H / kv.Hkv;
    const int cap = pps * PT;               // positions this block's tiles hold
    KP *sK = reinterpret_cast<KP *>(attn_smem);                  // [pps][D/2][PT] pairs
    AT *sV = reinterpret_cast<AT *>(sK + (size_t)cap * HALF);   // [cap][D]
    // rotated, scaled queries: fp32 pairs [RB][D/2]
    constexpr int SQ_WORDS = 2 * RB * HALF;
    float2 *sq = reinterpret_cast<float2 *>(sV + (size_t)cap * D);
    const int ss = cap + 12;                                     // row stride of the score matrix
    float *sS = reinterpret_cast<float *>(sq) + SQ_WORDS;        // [RB][ss]
    float *s_m = sS + (size_t)RB * ss;                           // [RB]
    float *s_l = s_m + RB;
    float *s_rstd = s_l + RB;                                    // [kMaxRows]
    uint64_t *bar = reinterpret_cast<uint64_t *>(s_rstd + kMaxRows);
    float *wgt = reinterpret_cast<float *>(bar + 2);             // [RB][n_split] merge weights
    __shared__ int s_last, s_abort;
    // which new rows a row sees and the position it is rotated as (a chain unless the pass verifies a tree)
    __shared__ uint16_t s_vis[kMaxRows];
    __shared__ uint8_t s_dep[kMaxRows];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int kh = blockIdx.x, sp = blockIdx.y;
    int bz = blockIdx.z;   // batch of (head, row) pairs
    // Batch mode: grid z runs over (sequence, batch of pairs); a sequence is an independent problem with its own
    // rows of the pass, positions, page table and slice count (the scratch layouts keep the launch's slice count).
    const int ns_stride = n_split;
    int row_base = 0;
    if (br.n_seq > 0) {
        const int seq = blockIdx.z / nbat;
        bz = blockIdx.z - seq * nbat;
        M = br.rows[seq];
        pos0 = br.pos0[seq];
        row_base = br.row0[seq];
        kv.page_table += br.table_off[seq];
        n_split = ((pos0 + M + PT - 1) / PT + pps - 1) / pps;
        if (sp >= n_split || group * M <= bz * RB) return;   // a shorter sequence fills fewer slices and batches
    }
    // per-slice (maximum, sum) pairs live behind the outputs: [H][16][kMaxSlices]
    float2 *ml = reinterpret_cast<float2 *>(apart + ml_off);
    const int r0 = bz * RB;                  // first (head, row) pair of this block's batch
    const int ctx_len = pos0 + M;
    const int n_pages = (ctx_len + PT - 1) / PT;
    const int page_lo = sp * pps, page_hi = min(n_pages, page_lo + pps);
    const int lo = page_lo * PT;
    const int npos = min(ctx_len, page_hi * PT) - lo;   // valid positions of this block
    const uint32_t blk_bytes = (uint32_t)(PT * D * sizeof(AT));

    pdl_trigger();
    if (TR && tid >= 32 && tid < 32 + kMaxRows) { s_vis[tid - 32] = tr.vis[tid - 32]; s_dep[tid - 32] = tr.depth[tid - 32]; }
    if (tid == 0) {
        s_abort = 0;
        tc::mbar_init(bar, 1);
        tc::mbar_init_fence();
    }
    __syncthreads();
    if (warp == 0) {
        // cached rows were written by earlier passes: no need to wait for this pass's producers.
        // One lane per page, so the page-table reads are in flight together.
        if (lane == 0) {
            const uint32_t total = 2u * blk_bytes * (uint32_t)(page_hi - page_lo);
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(total) : "memory");
        }
        __syncwarp();
        for (int pg = page_lo + lane; pg < page_hi; pg += 32) {
            const int page = kv.page_table[pg];
            const AT *src = (const AT *)kv.slot_base + (((size_t)page * 2) * kv.Hkv + kh) * (size_t)PT * D;
            const size_t v_off = (size_t)kv.Hkv * PT * D;
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_addr(sK + (size_t)(pg - page_lo) * PT * HALF)), "l"(src), "r"(blk_bytes), "r"(smem_addr(bar)) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_addr(sV + (size_t)(pg - page_lo) * PT * D)), "l"(src + v_off), "r"(blk_bytes), "r"(smem_addr(bar)) : "memory");
        }
    }
    // where the partial sums this block needs live (block numbers of the query tiles of its
    // batch and of its key and value tile): integer arithmetic only, done before the wait
    __shared__ int2 s_tb[40];
    const int rows = group * M;   // (head in group, new row) pairs; rho = g * M + m
    const int nb = min(RB, rows - r0);
    const int tq0 = ((kh * group + r0 / M) * D) >> 7, tq1 = ((kh * group + (r0 + nb - 1) / M) * D + D - 1) >> 7;
    const int nq = tq1 - tq0 + 1, tk = ((H + kh) * D) >> 7, tv = ((H + kv.Hkv + kh) * D) >> 7;
    if (pv.mode == 1 && tid < nq + 2 && tid < 40)
        s_tb[tid] = tile_blocks(pv.sk, tid < nq ? tq0 + tid : (tid == nq ? tk : tv));
    __syncthreads();
    auto gather_pair = [&](int m, int col) -> float2 {
        if (pv.mode == 0) return part_gather_n<2>(pv, row_base + m, col);
        const int t = col >> 7;
        return part_gather_blocks<2>(pv, s_tb[t == tk ? nq : (t == tv ? nq + 1 : t - tq0)], row_base + m, col);
    };
    // rotation factors of the new keys and of this block's queries: a constant table, fetched
    // before the wait so that they are not one more round trip behind the partial sums
    constexpr int kNewPerThread = (NM * D + 255) / 256;
    constexpr int kQPerThread = RB * HALF / 256;
    const int p_first = max(lo, pos0), p_last = min(lo + npos, ctx_len);   // [p_first, p_last)
    const int n_new = max(0, p_last - p_first) * D;
    float2 cs_new[kNewPerThread], cs_q[kQPerThread];
#pragma unroll
    for (int it = 0; it < kNewPerThread; it++) {
        const int idx = tid + it * 256;
        const int pn = idx / D, w = idx - pn * D;
        cs_new[it] = (idx < n_new && w < HALF) ? rope[(size_t)(TR ? pos0 + s_dep[p_first + pn - pos0] : p_first + pn) * HALF + w] : make_float2(1.f, 0.f);
    }
#pragma unroll
    for (int it = 0; it < kQPerThread; it++) {
        const int idx = tid + it * 256;
        const int rl = idx / HALF, i = idx - rl * HALF;
        cs_q[it] = idx < nb * HALF ? rope[(size_t)(pos0 + (TR ? (int)s_dep[(r0 + rl) % M] : (r0 + rl) % M)) * HALF + i] : make_float2(1.f, 0.f);
    }
    pdl_wait();   // from here on the QKV projection's partial sums are read
    // One round of global loads: the RMSNorm statistics (threads 0..M-1) and the raw partial
    // sums of this block's queries and of the new keys / values that fall into its slice; they
    // are scaled, rotated and rounded after the barrier, while the cached slice is still arriving.
    if (tid < M) s_rstd[tid] = row_rstd(rs, row_base + tid);
    float raw_a[kNewPerThread], raw_b[kNewPerThread];
    int new_page[kNewPerThread];
#pragma unroll
    for (int it = 0; it < kNewPerThread; it++) {
        const int idx = tid + it * 256;   // -> (position, K pair | V pair)
        if (idx < n_new) {
            const int pn = idx / D, w = idx - pn * D;
            const int m = p_first + pn - pos0;
            new_page[it] = kv.page_table[(p_first + pn) / PT];
            const int isV = w >= HALF, i = isV ? w - HALF : w;
            const int col = (H + (isV ? kv.Hkv : 0) + kh) * D + 2 * i;
            const float2 pr = gather_pair(m, col);
            raw_a[it] = pr.x;
            raw_b[it] = pr.y;
        }
    }
    float qraw_a[kQPerThread], qraw_b[kQPerThread];
#pragma unroll
    for (int it = 0; it < kQPerThread; it++) {
        const int idx = tid + it * 256;
        if (idx < nb * HALF) {
            const int rl = idx / HALF, i = idx - rl * HALF;
            const int g = (r0 + rl) / M, m = (r0 + rl) - g * M;
            const int col = (kh * group + g) * D + 2 * i;
            const float2 pr = gather_pair(m, col);
            qraw_a[it] = pr.x;
            qraw_b[it] = pr.y;
        }
    }
    __syncthreads();
    AT new_a[kNewPerThread], new_b[kNewPerThread];
#pragma unroll
    for (int it = 0; it < kNewPerThread; it++) {
        const int idx = tid + it * 256;
        if (idx < n_new) {
            const int pn = idx / D, w = idx - pn * D;
            const int pos = p_first + pn, m = pos - pos0;
            const int isV = w >= HALF;
            float a = raw_a[it] * s_rstd[m], b = raw_b[it] * s_rstd[m];
            if (!isV) {
                const float2 cs = cs_new[it];
                const float ra = a * cs.x - b * cs.y, rb = a * cs.y + b * cs.x;
                a = ra; b = rb;
            }
            new_a[it] = from_f<AT>(a);
            new_b[it] = from_f<AT>(b);
        }
    }
    {   // rotated, pre-scaled queries of this block's batch
#pragma unroll
        for (int it = 0; it < kQPerThread; it++) {
            const int idx = tid + it * 256;
            if (idx >= nb * HALF) continue;
            const int rl = idx / HALF, i = idx - rl * HALF;
            const int m = (r0 + rl) % M;
            const float a = qraw_a[it] * s_rstd[m], b = qraw_b[it] * s_rstd[m];
            const float2 cs = cs_q[it];
            const float qa = (a * cs.x - b * cs.y) * scale, qb = (a * cs.y + b * cs.x) * scale;
            sq[rl * HALF + i] = make_float2(qa, qb);
        }
    }
    if (warp == 0) {   // wait for the cached slice (bounded); the other warps park at the barrier below
        bool ok = false;
        for (uint32_t i = 0; i < spin && !ok; i++) {
            ok = tc::mbar_try(bar, 0);
            if (!ok) __nanosleep(32);
        }
        if (!ok && tid == 0) { s_abort = 1; atomicOr(err, kErrWaitTimeout); }
    }
    __syncthreads();
    if (s_abort) {   // the wait gave up: nothing of the slice is used; its copies must still land before the block ends
        if (tid == 0) tc::mbar_drain(bar, 0);
        return;
    }
#pragma unroll
    for (int it = 0; it < kNewPerThread; it++) {
        const int idx = tid + it * 256;
        if (idx < n_new) {
            const int pn = idx / D, w = idx - pn * D;
            const int pos = p_first + pn, j = pos - lo;
            const int isV = w >= HALF, i = isV ? w - HALF : w;
            const int page = new_page[it];
            if (page < 0 || page >= kv.n_pages_total) { atomicOr(err, kErrBadPage); continue; }
            AT *blk = (AT *)kv.slot_base + (((size_t)page * 2 + isV) * kv.Hkv + kh) * (size_t)PT * D;
            const bool append = bz == 0;   // every batch needs the row in its tile; one block writes the cache
            if (isV) {
                const int e = v_elem<AT>(pos, 2 * i);
                AT *tile = sV + (size_t)j * D + e;
                tile[0] = new_a[it]; tile[1] = new_b[it];
                if (append) {
                    blk[(size_t)(pos % PT) * D + e] = new_a[it];
                    blk[(size_t)(pos % PT) * D + e + 1] = new_b[it];
                }
            } else {   // keys: pair i of position pos at [i][pos % PT] of the page block
                const KP w2 = make_float2(new_a[it], new_b[it]);
                sK[(size_t)(j / PT) * PT * HALF + (size_t)i * PT + (j % PT)] = w2;
                if (append) reinterpret_cast<KP *>(blk)[(size_t)i * PT + (pos % PT)] = w2;
            }
        }
    }
    __syncthreads();

    {
        {   // scores.  Work item = (16 consecutive positions, 8 rows); lane = position + 16 * (dimension pair parity)
            const int t = lane & 15, eh = lane >> 4;
            const int n_task = (npos + 15) / 16, n_rc = (nb + 7) / 8;
            for (int item = warp; item < n_task * n_rc; item += 8) {
                const int task = item % n_task, rc = item / n_task;
                const int j = task * 16 + t;
                const int jj = min(j, npos - 1);   // lanes past the slice recompute its last position
                const KP *kp = sK + (size_t)(jj / PT) * PT * HALF + (jj % PT);
                const float2 *qp = sq + (size_t)rc * 8 * HALF;
                float acc[8];
#pragma unroll
                for (int i = 0; i < 8; i++) acc[i] = 0.f;
#pragma unroll 4
                for (int e2 = eh; e2 < HALF; e2 += 2) {
                    const KP kk = kp[(size_t)e2 * PT];
                    const float ka = kk.x, kb = kk.y;
#pragma unroll
                    for (int i = 0; i < 8; i++) {
                        const float2 qv = qp[i * HALF + e2];   // rows past nb hold stale values: results dropped
                        acc[i] = fmaf(ka, qv.x, acc[i]);
                        acc[i] = fmaf(kb, qv.y, acc[i]);
                    }
                }
#pragma unroll
                for (int i = 0; i < 8; i++) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], 16);
                if (eh == 0 && j < cap) {
#pragma unroll
                    for (int i = 0; i < 8; i++) {
                        const int rl = rc * 8 + i;
                        if (rl < nb) {
                            const int m = (r0 + rl) % M;
                            const int jn = lo + j - pos0;
                            const bool seen = TR ? (jn < 0 || ((s_vis[m] >> jn) & 1)) : (jn <= m);
                            sS[(size_t)rl * ss + j] = (j < npos && seen) ? acc[i] : -INFINITY;
                        }
                    }
                }
            }
        }
        __syncthreads();
        const int nposw = min(cap, ((npos + 15) / 16) * 16);   // entries the score phase wrote
        const int npos16 = nposw;
        for (int rl = warp; rl < nb; rl += 8) {   // softmax numerators of this slice
            float mx = -INFINITY;
            for (int j = lane; j < nposw; j += 32) mx = fmaxf(mx, sS[(size_t)rl * ss + j]);
            mx = warp_max(mx);
            float sum = 0.f;
            for (int j = lane; j < npos16; j += 32) {
                const float sv = j < nposw ? sS[(size_t)rl * ss + j] : -INFINITY;
                const float p = (sv == -INFINITY) ? 0.f : expf(sv - mx);
                sS[(size_t)rl * ss + j] = p;
                sum += p;
            }
            sum = warp_sum(sum);
            if (lane == 0) { s_m[rl] = mx; s_l[rl] = sum; }
        }
        __syncthreads();
        {   // o = P V.  Warp w owns rows w, w + 8, ... of the batch; lane owns DPL output dimensions
            constexpr int RPW = RB / 8;
            float o[RPW][DPL];
#pragma unroll
            for (int i = 0; i < RPW; i++)
#pragma unroll
                for (int e = 0; e < DPL; e++) o[i][e] = 0.f;
            if (warp < nb) {
                for (int j = 0; j < npos; j++) {
                    float v[DPL];
#pragma unroll
                    for (int e = 0; e < DPL; e++) v[e] = to_f(sV[(size_t)j * D + v_elem<AT>(j, lane * DPL + e)]);
#pragma unroll
                    for (int i = 0; i < RPW; i++) {
                        const int rl = min(warp + 8 * i, RB - 1);
                        const float p = sS[(size_t)rl * ss + j];
#pragma unroll
                        for (int e = 0; e < DPL; e++) o[i][e] = fmaf(p, v[e], o[i][e]);
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < RPW; i++) {
                const int rl = warp + 8 * i;
                if (rl < nb) {
                    const int g = (r0 + rl) / M, m = (r0 + rl) - g * M;
                    const int h = kh * group + g;
                    float *dst = apart + (((size_t)h * ns_stride + sp) * kMaxRows + row_base + m) * D;
#pragma unroll
                    for (int e = 0; e < DPL; e++) dst[lane * DPL + e] = o[i][e];
                    if (lane == 0) ml[((size_t)h * kMaxRows + row_base + m) * kMaxSlices + sp] = make_float2(s_m[rl], s_l[rl]);
                }
            }
        }
        __syncthreads();
    }
    // ---- merge: the block that arrives last for this KV head combines all slices
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        unsigned int *tk = tickets + (size_t)kh * gridDim.z + blockIdx.z;   // one counter per (KV head, sequence, batch)
        const unsigned int prev = atomicAdd(tk, 1u);
        s_last = (prev == (unsigned int)n_split - 1);
        if (s_last) *tk = 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const size_t sstride = (size_t)kMaxRows * D;
    {   // normalised weight of every (pair, slice); a warp's rows are loaded together: one round trip
        constexpr int RPW = RB / 8;
        const float2 none = make_float2(-INFINITY, 0.f);
        float2 v0[RPW], v1[RPW];
#pragma unroll
        for (int i = 0; i < RPW; i++) {
            const int rl = warp + 8 * i, rho = r0 + min(rl, nb - 1);
            const int g = rho / M, m = rho - g * M, h = kh * group + g;
            const float2 *src = ml + ((size_t)h * kMaxRows + row_base + m) * kMaxSlices;
            v0[i] = (rl < nb && lane < n_split) ? __ldcg(src + lane) : none;
            v1[i] = (rl < nb && lane + 32 < n_split) ? __ldcg(src + lane + 32) : none;
        }
#pragma unroll
        for (int i = 0; i < RPW; i++) {
            const int rl = warp + 8 * i;
            const float mx = warp_max(fmaxf(v0[i].x, v1[i].x));
            const float w0 = (v0[i].x == -INFINITY) ? 0.f : expf(v0[i].x - mx), w1 = (v1[i].x == -INFINITY) ? 0.f : expf(v1[i].x - mx);
            const float den = warp_sum(fmaf(w0, v0[i].y, w1 * v1[i].y));   // fixed butterfly over the lanes
            const float inv = den > 0.f ? 1.0f / den : 0.f;
            if (rl < nb) {
                if (lane < n_split) wgt[rl * n_split + lane] = w0 * inv;
                if (lane + 32 < n_split) wgt[rl * n_split + lane + 32] = w1 * inv;
            }
        }
    }
    __syncthreads();
    for (int idx = tid; idx < nb * (D / 4); idx += 256) {   // four output dimensions per item
        const int rl = idx / (D / 4), dd = (idx - rl * (D / 4)) * 4, rho = r0 + rl;
        const int g = rho / M, m = row_base + rho - g * M, h = kh * group + g;   // m: row of the pass
        const float *src = apart + ((size_t)h * ns_stride * kMaxRows + m) * D + dd;
        const float *wr = wgt + rl * n_split;
        float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s2 = 0; s2 < n_split; s2 += 16) {   // sixteen slices in flight, added in slice order
            float4 a[16];
#pragma unroll
            for (int u = 0; u < 16; u++)
                a[u] = __ldcg(reinterpret_cast<const float4 *>(src + (size_t)min(s2 + u, n_split - 1) * sstride));
#pragma unroll
            for (int u = 0; u < 16; u++) {
                const float w = s2 + u < n_split ? wr[s2 + u] : 0.f;
                o.x = fmaf(w, a[u].x, o.x); o.y = fmaf(w, a[u].y, o.y);
                o.z = fmaf(w, a[u].z, o.z); o.w = fmaf(w, a[u].w, o.w);
            }
        }
        const size_t col = (size_t)h * D + dd;
        if (attn_out) *reinterpret_cast<float4 *>(attn_out + (size_t)m * H * D + col) = o;
        if (attn_split) {
            store_split(attn_split, m, (size_t)H * D, col, o.x); store_split(attn_split, m, (size_t)H * D, col + 1, o.y);
            store_split(attn_split, m, (size_t)H * D, col + 2, o.z); store_split(attn_split, m, (size_t)H * D, col + 3, o.w);
        }
    }
}

static size_t attn_smem_bytes(int D, int RB, int cap, int n_split) {
    return (size_t)2 * cap * D * 4 + (size_t)RB * D * 4 + (size_t)RB * (cap + 12) * 4 + 2 * RB * 4 + kMaxRows * 4 + 16 +
           (size_t)RB * n_split * 4 + 16;
}

template <int D, int RB, int NM, bool TR>
static void attn_launch(cudaStream_t s, const PartView &pv, const RowScale &rs, const float2 *rope, const KvGeom &kv,
                        float *apart, unsigned int *tickets, float *attn_out, void *attn_split, int M, int pos0, int H,
                        int pps, int n_split, float scale, bool early, int *err, const TreeRows &tr, uint32_t wait_polls, const BatchRows &br) {
    const int rows = (H / kv.Hkv) * M, nbat = (rows + RB - 1) / RB;
    const size_t ml_off = (size_t)H * kMaxSlices * kMaxRows * D;
    const size_t smem = attn_smem_bytes(D, RB, pps * kv.page_tokens, n_split);
    // once per instantiation (thread-safe static initialisation)
    static const cudaError_t configured =
        cudaFuncSetAttribute(attn_kernel<D, RB, NM, TR>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 1024);
    (void)configured;
    launch_k(attn_kernel<D, RB, NM, TR>, dim3(kv.Hkv, n_split, nbat * (br.n_seq > 0 ? br.n_seq : 1)), dim3(256), smem, s, early && pdl_enabled(),
             pv, rs, rope, kv, apart, tickets, attn_out, (bf16 *)attn_split, M, pos0, H, pps, n_split, scale, err, nbat, ml_off, tr, wait_polls, br);
}

template <int D>
static void attn_dispatch(cudaStream_t s, const PartView &pv, const RowScale &rs, const float2 *rope, const KvGeom &kv,
                          float *apart, unsigned int *tickets, float *attn_out, void *attn_split, int M, int pos0, int H,
                          int pps, int n_split, float scale, bool early, int *err, const TreeRows *tree, uint32_t wait_polls,
                          const BatchRows &br) {
    const int rows = (H / kv.Hkv) * M;
    const TreeRows tr = tree ? *tree : chain_rows();
#define EESD_ATTN(RB, NM) attn_launch<D, RB, NM, false>(s, pv, rs, rope, kv, apart, tickets, attn_out, attn_split, M, pos0, H, pps, n_split, scale, early, err, tr, wait_polls, br)
#define EESD_ATTN_TREE(RB, NM) attn_launch<D, RB, NM, true>(s, pv, rs, rope, kv, apart, tickets, attn_out, attn_split, M, pos0, H, pps, n_split, scale, early, err, tr, wait_polls, br)
    if (tree) {   // tree passes: one instantiation per batch size
        if (rows <= 8) EESD_ATTN_TREE(8, 8);
        else if (rows <= kRows16) EESD_ATTN_TREE(16, 16);
        else EESD_ATTN_TREE(32, 16);
    } else if (rows <= 8) {
        if (M == 1) EESD_ATTN(8, 1);
        else if (M <= 4) EESD_ATTN(8, 4);
        else EESD_ATTN(8, 8);
    } else if (rows <= kRows16) {
        if (M <= 4) EESD_ATTN(16, 4);
        else EESD_ATTN(16, 16);
    } else {
        if (M <= 4) EESD_ATTN(32, 4);
        else EESD_ATTN(32, 16);
    }
#undef EESD_ATTN
#undef EESD_ATTN_TREE
}

// slices of the cached context (fp32 kernel): pages per block and number of blocks per KV head
int attention_splits(int ctx_len, int page_tokens, int Hkv, int n_batches, int n_sm, int max_splits, int *pps_out) {
    const int n_pages = (ctx_len + page_tokens - 1) / page_tokens;
    const int cap = kAttnPos / page_tokens > 0 ? kAttnPos / page_tokens : 1;   // pages one block can hold
    // one wave: about two blocks per SM in flight, so aim for H_kv * n_split <= 2 * n_sm (measured:
    // half and 1.5x as many slices are both slower at 6 to 16 rows)
    int want = 2 * n_sm / (Hkv * n_batches);
    if (want < 1) want = 1;
    if (want > max_splits) want = max_splits;
    int pps = (n_pages + want - 1) / want;
    if (pps > cap) pps = cap;            // longer contexts: more slices than one wave holds
    if (pps < 1) pps = 1;
    if ((pps * page_tokens) % 16) pps++;   // tiles hold a multiple of 16 positions
    *pps_out = pps;
    return (n_pages + pps - 1) / pps;
}

// most context tokens the attention kernels can serve: at most kMaxSlices slices per head, each as
// long as one block can hold (fp32 cache: 192 positions, or one page of 128; bf16 cache: 256)
int attention_max_ctx(int dtype, int page_tokens) {
    if (dtype != 0) return kMaxSlices * 256;
    int pps = kAttnPos / page_tokens > 0 ? kAttnPos / page_tokens : 1;
    if ((pps * page_tokens) % 16) pps++;
    return kMaxSlices * pps * page_tokens;
}

void launch_attention(cudaStream_t s, int dtype, const PartView &pv, const RowScale &rs, const float2 *rope,
                      const KvGeom &kv, float *apart, unsigned int *tickets, float *attn_out, void *attn_split,
                      int M, int pos0, int H, int n_sm, int max_splits, bool early, int *err, const TreeRows *tree,
                      uint32_t wait_polls, const BatchRows *batch) {
    int pps;
    if (batch && batch->n_seq > 0) {   // several sequences: plan for the one with the most rows / the longest context
        M = 0;
        int ctx = 0;
        for (int b = 0; b < batch->n_seq; b++) {
            if (batch->rows[b] > M) M = batch->rows[b];
            if (batch->pos0[b] + batch->rows[b] > ctx) ctx = batch->pos0[b] + batch->rows[b];
        }
        pos0 = ctx - M;
        if (tree) {   // a tree's rows belong to one sequence
            const int e = kErrPlan;
            cudaMemcpyAsync(err, &e, sizeof(e), cudaMemcpyHostToDevice, s);
            return;
        }
    } else {
        batch = nullptr;
    }
    const int rows = (H / kv.Hkv) * M;
    auto refuse = [&](int n_split) {   // more slices than the merge can take: report, launch nothing
        if (n_split <= kMaxSlices && n_split <= max_splits) return false;
        const int e = kErrPlan;
        cudaMemcpyAsync(err, &e, sizeof(e), cudaMemcpyHostToDevice, s);
        return true;
    };
    if (dtype != 0) {   // bf16 cache: tensor-core kernel
        const int nc = attention_tc_columns(rows);
        const int n_split = attention_tc_splits(pos0 + M, kv.page_tokens, kv.Hkv, (rows + nc - 1) / nc * (batch ? batch->n_seq : 1), n_sm,
                                                max_splits, &pps);
        if (refuse(n_split)) return;
        launch_attention_tc(s, pv, rs, rope, kv, apart, tickets, attn_out, attn_split, M, pos0, H, pps, n_split, early, err, tree,
                            wait_polls, batch);
        return;
    }
    const int rb = rows <= 8 ? 8 : rows <= kRows16 ? 16 : 32;
    const int n_split = attention_splits(pos0 + M, kv.page_tokens, kv.Hkv, (rows + rb - 1) / rb * (batch ? batch->n_seq : 1), n_sm, max_splits, &pps);
    if (refuse(n_split)) return;
    BatchRows br = {};
    if (batch) br = *batch;
    const float scale = 1.0f / sqrtf((float)kv.D);
    if (kv.D == 64) attn_dispatch<64>(s, pv, rs, rope, kv, apart, tickets, attn_out, attn_split, M, pos0, H, pps, n_split, scale, early, err, tree, wait_polls, br);
    else attn_dispatch<128>(s, pv, rs, rope, kv, apart, tickets, attn_out, attn_split, M, pos0, H, pps, n_split, scale, early, err, tree, wait_polls, br);
}

// ------------------------------------------------------------------------------------ SwiGLU, partial sums
__global__ void swiglu_kernel(PartView pv, RowScale rs, float *h, bf16 *hs, int F) {
    const int m = blockIdx.y, i = (blockIdx.x * blockDim.x + threadIdx.x) * 4;
    pdl_trigger();
    pdl_wait();
    if (i >= F) return;
    const float4 g = part_gather4(pv, m, i), u = part_gather4(pv, m, F + i);   // requested first: the longest loads
    const float rstd = row_rstd(rs, m);
    const float gg[4] = {g.x * rstd, g.y * rstd, g.z * rstd, g.w * rstd};
    const float uu[4] = {u.x * rstd, u.y * rstd, u.z * rstd, u.w * rstd};
    float v[4];
#pragma unroll
    for (int k = 0; k < 4; k++) v[k] = gg[k] / (1.0f + expf(-gg[k])) * uu[k];
    if (h) *reinterpret_cast<float4 *>(h + (size_t)m * F + i) = make_float4(v[0], v[1], v[2], v[3]);
    if (hs) store_split4(hs, m, F, i, make_float4(v[0], v[1], v[2], v[3]));
}
void launch_swiglu(cudaStream_t s, const PartView &pv, const RowScale &rs, float *h, void *h_split, int M, int F) {
    launch_k(swiglu_kernel, dim3((F / 4 + 255) / 256, M), dim3(256), 0, s, pdl_enabled(), pv, rs, h, (bf16 *)h_split, F);
}

// ------------------------------------------------------------------------------------ tree verification helpers
// Tokens ranked 1..width of one logit row, ranked by logit with the lower id first among equals
// (rank 1, the greedy draft token, goes to *first when given; ranks 2.. to out).  One block; every rank is one pass over the row that keeps
// the best element ranked after the previous pick.  Rows of up to 32768 logits are read once
// into registers (all loads in flight together: the kernel is one block and latency bound).
__global__ void __launch_bounds__(1024) next_best_kernel(const float *__restrict__ logits, int V, int width, int32_t *first,
                                                         int32_t *out) {
    __shared__ float s_v[32];
    __shared__ int s_i[32];
    __shared__ float s_pv;
    __shared__ int s_pi;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    pdl_trigger();
    pdl_wait();
    float pv = INFINITY;
    int pi = -1;
    auto better = [](float v, int i, float bv, int bi) { return v > bv || (v == bv && i < bi); };
    constexpr int kPer = 32;
    const bool in_regs = V <= kPer * (int)blockDim.x;
    float reg[kPer];
    if (in_regs) {
#pragma unroll
        for (int j = 0; j < kPer; j++) {
            const int i = threadIdx.x + j * blockDim.x;
            reg[j] = i < V ? logits[i] : NAN;   // NaN compares false: never picked
        }
    }
    for (int r = 0; r < width; r++) {
        float bv = -INFINITY;
        int bi = 0x7fffffff;
        if (in_regs) {
#pragma unroll
            for (int j = 0; j < kPer; j++) {
                const int i = threadIdx.x + j * blockDim.x;
                const float v = reg[j];
                const bool after = v < pv || (v == pv && i > pi);
                if (after && better(v, i, bv, bi)) { bv = v; bi = i; }
            }
        } else {
            for (int i = threadIdx.x; i < V; i += blockDim.x) {
                const float v = logits[i];
                const bool after = v < pv || (v == pv && i > pi);
                if (after && better(v, i, bv, bi)) { bv = v; bi = i; }
            }
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
        }
        if (lane == 0) { s_v[warp] = bv; s_i[warp] = bi; }
        __syncthreads();
        if (warp == 0) {
            bv = lane < nw ? s_v[lane] : -INFINITY;
            bi = lane < nw ? s_i[lane] : 0x7fffffff;
#pragma unroll
            for (int o = 16; o; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
            }
            if (lane == 0) {
                s_pv = bv;
                s_pi = bi;
                if (r >= 1) out[r - 1] = bi;
                else if (first) *first = bi;
            }
        }
        __syncthreads();
        pv = s_pv;
        pi = s_pi;
        __syncthreads();
    }
}
void launch_next_best(cudaStream_t s, const float *logits, int V, int width, int32_t *first, int32_t *out) {
    launch_k(next_best_kernel, dim3(1), dim3(1024), 0, s, pdl_enabled(), logits, V, width, first, out);
}

__global__ void tree_rows_kernel(const int32_t *chain, const int32_t *leaf, int K, int width, int32_t *rows) {
    const int t = threadIdx.x, M = 1 + K * width;
    if (t < M) rows[t] = t <= K ? chain[t] : leaf[t - K - 1];
}
void launch_tree_rows(cudaStream_t s, const int32_t *src_chain, const int32_t *src_leaf, int K, int width, int32_t *rows) {
    tree_rows_kernel<<<1, 32, 0, s>>>(src_chain, src_leaf, K, width, rows);
}

// Row i (1 <= i <= K) holds chain token x_i, row K + 1 + (i - 1)(width - 1) + j leaf j of depth i.
// top[m] is the target's top-1 token after the path that ends in row m.
__global__ void tree_walk_kernel(const int32_t *top, int32_t *chain, const int32_t *leaf, int K, int width, int32_t *result) {
    if (threadIdx.x != 0) return;
    int a = K, y = top[K], row = -1;
    for (int i = 1; i <= K; i++) {
        const int want = top[i - 1];
        if (want == chain[i]) continue;
        a = i - 1;
        y = want;
        for (int j = 0; j < width - 1; j++) {
            const int li = (i - 1) * (width - 1) + j;
            if (leaf[li] == want) {
                row = K + 1 + li;
                a = i;
                y = top[row];
                chain[i] = want;
                break;
            }
        }
        break;
    }
    result[0] = a;
    result[1] = y;
    result[2] = row;
    chain[0] = y;
}
void launch_tree_walk(cudaStream_t s, const int32_t *top, int32_t *chain, const int32_t *leaf, int K, int width,
                      int32_t *result) {
    tree_walk_kernel<<<1, 32, 0, s>>>(top, chain, leaf, K, width, result);
}

// A kept leaf's keys / values move from the position its row was stored at to the position of
// its depth.  grid (H_kv, slots), D / 2 threads: one rotation pair of the key, two value elements.
template <typename AT>
__global__ void kv_move_kernel(KvGeom kv, size_t slot_bytes, int pos0, const int32_t *result, int *err) {
    const int row = result[2];
    if (row < 0) return;
    const int src = pos0 + row, dst = pos0 + result[0];
    const int kh = blockIdx.x, i = threadIdx.x, D = kv.D, PT = kv.page_tokens;
    const int ps = kv.page_table[src / PT], pd = kv.page_table[dst / PT];
    if (ps < 0 || ps >= kv.n_pages_total || pd < 0 || pd >= kv.n_pages_total) {
        if (i == 0) atomicOr(err, kErrBadPage);
        return;
    }
    AT *base = (AT *)((char *)kv.slot_base + (size_t)blockIdx.y * slot_bytes);
    const size_t blk = (size_t)PT * D;
    const AT *ks = base + (((size_t)ps * 2) * kv.Hkv + kh) * blk, *vs = base + (((size_t)ps * 2 + 1) * kv.Hkv + kh) * blk;
    AT *kd = base + (((size_t)pd * 2) * kv.Hkv + kh) * blk, *vd = base + (((size_t)pd * 2 + 1) * kv.Hkv + kh) * blk;
    const int sj = src % PT, dj = dst % PT;
#pragma unroll
    for (int e = 0; e < 2; e++) {
        kd[k_index<AT>(dj, 2 * i + e, PT, D)] = ks[k_index<AT>(sj, 2 * i + e, PT, D)];
        vd[v_index<AT>(dst, dj, 2 * i + e, PT, D)] = vs[v_index<AT>(src, sj, 2 * i + e, PT, D)];
    }
}
void launch_kv_move(cudaStream_t s, int dtype, const KvGeom &kv0, size_t slot_bytes, int slots, int pos0,
                    const int32_t *result, int *err) {
    if (dtype == 0) kv_move_kernel<float><<<dim3(kv0.Hkv, slots), kv0.D / 2, 0, s>>>(kv0, slot_bytes, pos0, result, err);
    else kv_move_kernel<bf16><<<dim3(kv0.Hkv, slots), kv0.D / 2, 0, s>>>(kv0, slot_bytes, pos0, result, err);
}

// ------------------------------------------------------------------------------------ calibration predictor (Eq. 5)
__global__ void copy_row_kernel(const float *x, int row, const int32_t *row_dev, float *hT, bf16 *xs, int d) {
    pdl_trigger();
    pdl_wait();
    const int r = row_dev ? *row_dev : row;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < d; i += gridDim.x * blockDim.x) {
        const float v = x[(size_t)r * d + i];
        hT[i] = v;
        if (xs) store_split(xs, 0, d, i, v);
    }
}
void launch_copy_row(cudaStream_t s, const float *x, int row, const int32_t *row_dev, float *hT, void *xs, int d) {
    launch_k(copy_row_kernel, dim3((d + 255) / 256), dim3(256), 0, s, pdl_enabled(), x, row, row_dev, hT, (bf16 *)xs, d);
}

// one block: l_c = sum_k Wp[c][k] v[k] + sum_k Wp[c][d + k] hD[k]; theta = 1 / (1 + exp(l_0 - l_1))
__global__ void __launch_bounds__(256) cali_theta_kernel(PartView pv, const float *Wp, const float *hD, int d, float *theta) {
    __shared__ float scratch[33];
    pdl_trigger();
    pdl_wait();
    float l0 = 0.f, l1 = 0.f;
    for (int k = threadIdx.x; k < d; k += blockDim.x) {
        const float v = part_gather(pv, 0, k), h = hD[k];
        l0 = fmaf(Wp[k], v, l0);
        l0 = fmaf(Wp[d + k], h, l0);
        l1 = fmaf(Wp[2 * d + k], v, l1);
        l1 = fmaf(Wp[3 * d + k], h, l1);
    }
    l0 = block_sum(l0, scratch);
    l1 = block_sum(l1, scratch);
    if (threadIdx.x == 0) *theta = 1.0f / (1.0f + expf(l0 - l1));
}
void launch_cali_theta(cudaStream_t s, const PartView &pv, const float *Wp, const float *hD, int d, float *theta) {
    launch_k(cali_theta_kernel, dim3(1), dim3(256), 0, s, pdl_enabled(), pv, Wp, hD, d, theta);
}

// four consecutive outputs per thread (R % 4 == 0: tensor-core shapes are multiples of 128), else one
template <int VEC>
__global__ void reduce_partials_kernel(PartView pv, RowScale rs, float *out, int R, size_t out_stride) {
    const int m = blockIdx.y, r = (blockIdx.x * blockDim.x + threadIdx.x) * VEC;
    pdl_trigger();
    pdl_wait();
    if (r >= R) return;
    if (VEC == 4) {
        const float4 v = part_gather4(pv, m, r);
        const float s = row_rstd(rs, m);
        *reinterpret_cast<float4 *>(out + (size_t)m * out_stride + r) = make_float4(v.x * s, v.y * s, v.z * s, v.w * s);
    } else {
        out[(size_t)m * out_stride + r] = part_gather(pv, m, r) * row_rstd(rs, m);
    }
}
void launch_reduce_partials(cudaStream_t s, const PartView &pv, const RowScale &rs, float *out, int M, int R, size_t out_stride) {
    const size_t stride = out_stride ? out_stride : (size_t)R;
    if (R % 4 == 0 && stride % 4 == 0)
        launch_k(reduce_partials_kernel<4>, dim3((R / 4 + 255) / 256, M), dim3(256), 0, s, pdl_enabled(), pv, rs, out, R, stride);
    else
        launch_k(reduce_partials_kernel<1>, dim3((R + 255) / 256, M), dim3(256), 0, s, pdl_enabled(), pv, rs, out, R, stride);
}

}  // namespace eesd
