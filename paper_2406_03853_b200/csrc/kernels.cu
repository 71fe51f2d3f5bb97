// Model kernels of the EESD decode round (sm_100a): embedding gather, residual + RMSNorm,
// skinny projections (M <= 16 token rows against a streamed weight matrix), RoPE + paged KV
// append, paged decode attention with a causal block of new rows, SwiGLU.
//
// Every reduction has a fixed combination order, so a pass is bit-reproducible.
#include "common.cuh"
#include "kernels.cuh"

namespace eesd {

typedef __nv_bfloat16 bf16;

// sum of the partial results of output element (m, r), in a fixed order
__device__ __forceinline__ float part_gather(const PartView &pv, int m, int r) {
    float v = 0.f;
    if (pv.mode == 0) {
        for (int s = 0; s < pv.S; s++) v += pv.base[(size_t)s * pv.split_stride + (size_t)m * pv.R + r];
    } else {
        const StreamK &sk = pv.sk;
        const int t = r >> 7, rr = r & 127;
        const int c0 = sk.owner(t * sk.KB), c1 = sk.owner((t + 1) * sk.KB - 1);
        for (int c = c0; c <= c1; c++)
            v += pv.base[((size_t)(c * sk.max_seg + (t - sk.first_tile(c))) * kMaxRows + m) * 128 + rr];
    }
    return v;
}

// the same for four consecutive outputs r..r+3 (r % 4 == 0, so they share a weight tile)
__device__ __forceinline__ float4 part_gather4(const PartView &pv, int m, int r) {
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (pv.mode == 0) {
        for (int s = 0; s < pv.S; s++) {
            const float4 t = *reinterpret_cast<const float4 *>(pv.base + (size_t)s * pv.split_stride + (size_t)m * pv.R + r);
            v.x += t.x; v.y += t.y; v.z += t.z; v.w += t.w;
        }
    } else {
        const StreamK &sk = pv.sk;
        const int t = r >> 7, rr = r & 127;
        const int c0 = sk.owner(t * sk.KB), c1 = sk.owner((t + 1) * sk.KB - 1);
        for (int c = c0; c <= c1; c++) {
            const float4 a = __ldcg(reinterpret_cast<const float4 *>(
                pv.base + ((size_t)(c * sk.max_seg + (t - sk.first_tile(c))) * kMaxRows + m) * 128 + rr));
            v.x += a.x; v.y += a.y; v.z += a.z; v.w += a.w;
        }
    }
    return v;
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

// ------------------------------------------------------------------------------------ embedding gather
template <typename WT>
__global__ void embed_kernel(const int32_t *tok, const WT *E, float *x, float *cap, int d, int V, int *err) {
    const int m = blockIdx.x;
    int t = tok[m];
    if (t < 0 || t >= V) {
        if (threadIdx.x == 0) atomicOr(err, kErrBadToken);
        t = 0;
    }
    const WT *row = E + (size_t)t * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        float v = to_f(row[i]);
        x[(size_t)m * d + i] = v;
        if (cap) cap[(size_t)m * d + i] = v;
    }
}
void launch_embed(cudaStream_t s, int dtype, const int32_t *tok, const void *E, float *x, float *cap,
                  int M, int d, int V, int *err) {
    if (dtype == 0) embed_kernel<float><<<M, 256, 0, s>>>(tok, (const float *)E, x, cap, d, V, err);
    else embed_kernel<bf16><<<M, 256, 0, s>>>(tok, (const bf16 *)E, x, cap, d, V, err);
}

// ------------------------------------------------------------------------------------ residual + RMSNorm
// One block of 1024 threads per token row, four elements per thread and step.
// x[m] += partial sums; xn[m] = RMSNorm(x[m]) * g (fp32 and, optionally, as two bf16 terms).
__global__ void __launch_bounds__(1024) resid_norm_kernel(float *x, PartView pv, int has_part, const float *g, float *xn,
                                                          bf16 *xs, float *cap, int d, float eps) {
    extern __shared__ float row[];  // d floats + 33 scratch
    float *scratch = row + d;
    const int m = blockIdx.x;
    float *xr = x + (size_t)m * d;
    float ss = 0.f;
    for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
        float4 v = *reinterpret_cast<const float4 *>(xr + i);
        if (has_part) {
            const float4 p = part_gather4(pv, m, i);
            v.x += p.x; v.y += p.y; v.z += p.z; v.w += p.w;
            *reinterpret_cast<float4 *>(xr + i) = v;
        }
        *reinterpret_cast<float4 *>(row + i) = v;
        if (cap) *reinterpret_cast<float4 *>(cap + (size_t)m * d + i) = v;
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
    if (!g) return;
    ss = block_sum(ss, scratch);
    const float rstd = 1.0f / sqrtf(ss / (float)d + eps);
    for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
        const float4 r4 = *reinterpret_cast<const float4 *>(row + i);
        const float4 g4 = *reinterpret_cast<const float4 *>(g + i);
        const float4 v = make_float4(r4.x * rstd * g4.x, r4.y * rstd * g4.y, r4.z * rstd * g4.z, r4.w * rstd * g4.w);
        *reinterpret_cast<float4 *>(xn + (size_t)m * d + i) = v;
        if (xs) {
            store_split(xs, m, d, i, v.x); store_split(xs, m, d, i + 1, v.y);
            store_split(xs, m, d, i + 2, v.z); store_split(xs, m, d, i + 3, v.w);
        }
    }
}
void launch_resid_norm(cudaStream_t s, float *x, const PartView *pv, const float *g, float *xn, void *xs, float *cap,
                       int M, int d, float eps) {
    size_t smem = (size_t)(d + 33) * sizeof(float);
    PartView none = {};
    resid_norm_kernel<<<M, 1024, smem, s>>>(x, pv ? *pv : none, pv != nullptr, g, xn, (bf16 *)xs, cap, d, eps);
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
    if (M <= 1) gemm_simt_kernel<WT, AT, 1><<<grid, 256, 0, s>>>(a, w, out, M, R, K);
    else if (M <= 2) gemm_simt_kernel<WT, AT, 2><<<grid, 256, 0, s>>>(a, w, out, M, R, K);
    else if (M <= 4) gemm_simt_kernel<WT, AT, 4><<<grid, 256, 0, s>>>(a, w, out, M, R, K);
    else if (M <= 8) gemm_simt_kernel<WT, AT, 8><<<grid, 256, 0, s>>>(a, w, out, M, R, K);
    else gemm_simt_kernel<WT, AT, 16><<<grid, 256, 0, s>>>(a, w, out, M, R, K);
}

int launch_gemm(cudaStream_t s, int dtype, const float *A, const void *W, float *out, int M, int R, int K) {
    if (dtype == 0) gemm_simt_dispatch<float, float>(s, A, W, out, M, R, K);
    else gemm_simt_dispatch<bf16, float>(s, A, W, out, M, R, K);
    return 1;
}

// ------------------------------------------------------------------------------------ RoPE + KV append
// grid (heads, M), block D/2: one thread per rotation pair.
template <typename AT>
__global__ void qkv_post_kernel(PartView pv, int pos0, int H, KvGeom kv, const float2 *rope, float *q, int head_off,
                                int *err) {
    const int hh = blockIdx.x + head_off;  // 0..H-1 q, H..H+Hkv-1 k, then v
    const int m = blockIdx.y, i = threadIdx.x, D = kv.D;
    const int col = blockIdx.x * D + 2 * i;
    float a = part_gather(pv, m, col), b = part_gather(pv, m, col + 1);
    const int pos = pos0 + m;
    if (hh < H + kv.Hkv) {
        float2 cs = rope[(size_t)pos * (D / 2) + i];
        float ra = a * cs.x - b * cs.y, rb = a * cs.y + b * cs.x;
        a = ra; b = rb;
    }
    if (hh < H) {
        float *dst = q + (size_t)m * H * D + (size_t)hh * D + 2 * i;
        dst[0] = a; dst[1] = b;
        return;
    }
    const int isV = (hh - H) / kv.Hkv, kh = (hh - H) % kv.Hkv;
    const int page = kv.page_table[pos / kv.page_tokens];
    if (page < 0 || page >= kv.n_pages_total) {
        if (i == 0) atomicOr(err, kErrBadPage);
        return;
    }
    AT *dst = (AT *)kv.slot_base +
              (((size_t)page * 2 + isV) * kv.Hkv + kh) * (size_t)kv.page_tokens * D +
              (size_t)(pos % kv.page_tokens) * D + 2 * i;
    dst[0] = from_f<AT>(a);
    dst[1] = from_f<AT>(b);
}
void launch_qkv_post(cudaStream_t s, int dtype, const PartView &pv, int M, int pos0, int H,
                     const KvGeom &kv, const float2 *rope, float *q, bool only_kv, int *err) {
    const int heads = only_kv ? 2 * kv.Hkv : H + 2 * kv.Hkv;
    dim3 grid(heads, M);
    if (dtype == 0) qkv_post_kernel<float><<<grid, kv.D / 2, 0, s>>>(pv, pos0, H, kv, rope, q, only_kv ? H : 0, err);
    else qkv_post_kernel<bf16><<<grid, kv.D / 2, 0, s>>>(pv, pos0, H, kv, rope, q, only_kv ? H : 0, err);
}

// ------------------------------------------------------------------------------------ paged decode attention
// grid (H_kv, n_split), 256 threads.  Block (kh, sp) owns up to kAttnPos cached positions of
// KV head kh (a whole number of pages) and serves every query head of its group and all M new
// rows from ONE copy of those keys and values: the page blocks ([page_tokens][D], contiguous)
// are brought into shared memory by bulk asynchronous copies on one mbarrier, so the cache is
// read from HBM once per KV head.  Row m sees positions <= pos0 + m.  The block writes, per
// (query head, row), the un-normalised output, the maximum and the sum of its slice; the
// combine kernel merges the slices in index order.
constexpr int kAttnPos = 128;     // positions per block
constexpr int kAttnRows = 32;     // (head, row) pairs processed per batch

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

template <typename AT, int D>
__global__ void __launch_bounds__(256) attn_kernel(const float *__restrict__ q, KvGeom kv, float *__restrict__ apart,
                                                   int M, int pos0, int H, int pps, int n_split, float scale, int *err) {
    constexpr int VEC = Vec16<AT>::N;       // elements per 16-byte chunk
    constexpr int NCH = D / VEC;            // chunks per row
    extern __shared__ __align__(128) unsigned char attn_smem[];
    AT *sK = reinterpret_cast<AT *>(attn_smem);
    AT *sV = sK + kAttnPos * D;
    float *sq = reinterpret_cast<float *>(sV + kAttnPos * D);   // [kAttnRows][D]
    float *sS = sq + kAttnRows * D;                              // [kAttnRows][kAttnPos]
    float *s_m = sS + kAttnRows * kAttnPos;                      // [kAttnRows]
    float *s_l = s_m + kAttnRows;
    uint64_t *bar = reinterpret_cast<uint64_t *>(s_l + kAttnRows);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int kh = blockIdx.x, sp = blockIdx.y;
    const int PT = kv.page_tokens, group = H / kv.Hkv;
    const int ctx_len = pos0 + M;
    const int n_pages = (ctx_len + PT - 1) / PT;
    const int page_lo = sp * pps, page_hi = min(n_pages, page_lo + pps);
    const int lo = page_lo * PT;
    const int npos = min(ctx_len, page_hi * PT) - lo;   // valid positions of this block
    const uint32_t blk_bytes = (uint32_t)(PT * D * sizeof(AT));

    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_addr(bar)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    if (tid == 0) {
        const uint32_t total = 2u * blk_bytes * (uint32_t)(page_hi - page_lo);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(total) : "memory");
        for (int pg = page_lo; pg < page_hi; pg++) {
            const int page = kv.page_table[pg];
            const AT *src = (const AT *)kv.slot_base + (((size_t)page * 2) * kv.Hkv + kh) * (size_t)PT * D;
            const size_t v_off = (size_t)kv.Hkv * PT * D;
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_addr(sK + (size_t)(pg - page_lo) * PT * D)), "l"(src), "r"(blk_bytes), "r"(smem_addr(bar)) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(smem_addr(sV + (size_t)(pg - page_lo) * PT * D)), "l"(src + v_off), "r"(blk_bytes), "r"(smem_addr(bar)) : "memory");
        }
    }
    const int rows = group * M;   // (head in group, new row) pairs; rho = g * M + m
    bool landed = false;
    for (int r0 = 0; r0 < rows; r0 += kAttnRows) {
        const int nb = min(kAttnRows, rows - r0);
        for (int idx = tid; idx < nb * D; idx += 256) {
            const int rl = idx / D, e = idx - rl * D;
            const int g = (r0 + rl) / M, m = (r0 + rl) - g * M;
            sq[rl * D + e] = q[(size_t)m * H * D + (size_t)(kh * group + g) * D + e] * scale;
        }
        if (!landed) {
            bool ok = false;
            for (uint32_t i = 0; i < (1u << 24) && !ok; i++) {
                uint32_t p;
                asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], 0;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                             : "=r"(p) : "r"(smem_addr(bar)) : "memory");
                ok = p != 0;
                if (!ok) __nanosleep(32);
            }
            if (!ok && tid == 0) atomicOr(err, kErrWaitTimeout);
            landed = true;
        }
        __syncthreads();
        {   // scores: thread -> position j, every second row of the batch
            const int j = tid & (kAttnPos - 1), rsel = tid >> 7;
            float acc[kAttnRows / 2];
#pragma unroll
            for (int i = 0; i < kAttnRows / 2; i++) acc[i] = 0.f;
            if (j < npos) {
#pragma unroll 2
                for (int c = 0; c < NCH; c++) {
                    const int cc = (c + j) % NCH;   // rotate the chunk order: conflict-free shared loads
                    float kvv[VEC];
                    if (sizeof(AT) == 2) Vec16<__nv_bfloat16>::unpack(*reinterpret_cast<const uint4 *>(sK + (size_t)j * D + cc * VEC), kvv);
                    else {
                        const float4 t = *reinterpret_cast<const float4 *>(sK + (size_t)j * D + cc * VEC);
                        kvv[0] = t.x; kvv[1] = t.y; kvv[2] = t.z; kvv[3] = t.w;
                    }
#pragma unroll
                    for (int i = 0; i < kAttnRows / 2; i++) {
                        const int rl = rsel + 2 * i;
                        if (rl < nb) {
                            float qv[VEC];
#pragma unroll
                            for (int v = 0; v < VEC; v += 4) {
                                const float4 t = *reinterpret_cast<const float4 *>(sq + rl * D + cc * VEC + v);
                                qv[v] = t.x; qv[v + 1] = t.y; qv[v + 2] = t.z; qv[v + 3] = t.w;
                            }
#pragma unroll
                            for (int v = 0; v < VEC; v++) acc[i] = fmaf(kvv[v], qv[v], acc[i]);
                        }
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < kAttnRows / 2; i++) {
                const int rl = rsel + 2 * i;
                if (rl < nb) {
                    const int m = (r0 + rl) % M;
                    sS[rl * kAttnPos + j] = (j < npos && lo + j <= pos0 + m) ? acc[i] : -INFINITY;
                }
            }
        }
        __syncthreads();
        for (int rl = warp; rl < nb; rl += 8) {   // softmax numerators of this slice
            float mx = -INFINITY;
            for (int j = lane; j < kAttnPos; j += 32) mx = fmaxf(mx, sS[rl * kAttnPos + j]);
            mx = warp_max(mx);
            float sum = 0.f;
            for (int j = lane; j < kAttnPos; j += 32) {
                const float sv = sS[rl * kAttnPos + j];
                const float p = (sv == -INFINITY) ? 0.f : expf(sv - mx);
                sS[rl * kAttnPos + j] = p;
                sum += p;
            }
            sum = warp_sum(sum);
            if (lane == 0) { s_m[rl] = mx; s_l[rl] = sum; }
        }
        __syncthreads();
        {   // o = P V: thread -> (pair of d, row group)
            constexpr int HALF = D / 2, NG = 256 / HALF, RPT = kAttnRows / NG;
            const int d2 = tid % HALF, rg = tid / HALF;
            float o0[RPT], o1[RPT];
#pragma unroll
            for (int i = 0; i < RPT; i++) { o0[i] = 0.f; o1[i] = 0.f; }
            for (int j = 0; j < npos; j++) {
                float v0, v1;
                if (sizeof(AT) == 2) {
                    const uint32_t w = *reinterpret_cast<const uint32_t *>(sV + (size_t)j * D + 2 * d2);
                    v0 = __uint_as_float(w << 16); v1 = __uint_as_float(w & 0xFFFF0000u);
                } else {
                    const float2 t = *reinterpret_cast<const float2 *>(sV + (size_t)j * D + 2 * d2);
                    v0 = t.x; v1 = t.y;
                }
#pragma unroll
                for (int i = 0; i < RPT; i++) {
                    const int rl = rg + NG * i;
                    if (rl < nb) {
                        const float p = sS[rl * kAttnPos + j];
                        o0[i] = fmaf(p, v0, o0[i]);
                        o1[i] = fmaf(p, v1, o1[i]);
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < RPT; i++) {
                const int rl = rg + NG * i;
                if (rl < nb) {
                    const int g = (r0 + rl) / M, m = (r0 + rl) - g * M;
                    float *dst = apart + (((size_t)(kh * group + g) * n_split + sp) * kMaxRows + m) * (D + 2);
                    dst[2 * d2] = o0[i];
                    dst[2 * d2 + 1] = o1[i];
                    if (d2 == 0) { dst[D] = s_m[rl]; dst[D + 1] = s_l[rl]; }
                }
            }
        }
        __syncthreads();
    }
}

// grid (H, M), block D: merge the splits of one (head, row)
__global__ void attn_combine_kernel(const float *apart, float *out, bf16 *out_split, int H, int D, int n_split) {
    const int h = blockIdx.x, m = blockIdx.y, dd = threadIdx.x;
    const float *src = apart + (size_t)h * n_split * kMaxRows * (D + 2) + (size_t)m * (D + 2);
    const size_t sstride = (size_t)kMaxRows * (D + 2);
    float mx = -INFINITY;
    for (int s = 0; s < n_split; s++) mx = fmaxf(mx, src[s * sstride + D]);
    float num = 0.f, den = 0.f;
    for (int s = 0; s < n_split; s++) {
        const float ms = src[s * sstride + D];
        if (ms == -INFINITY) continue;
        const float w = expf(ms - mx);
        num = fmaf(w, src[s * sstride + dd], num);
        den = fmaf(w, src[s * sstride + D + 1], den);
    }
    const float o = den > 0.f ? num / den : 0.f;
    out[(size_t)m * H * D + (size_t)h * D + dd] = o;
    if (out_split) store_split(out_split, m, (size_t)H * D, (size_t)h * D + dd, o);
}

template <typename AT, int D>
static void attn_launch(cudaStream_t s, const float *q, const KvGeom &kv, float *apart, int M, int pos0, int H, int pps,
                        int n_split, float scale, int *err) {
    const size_t smem = (size_t)2 * kAttnPos * D * sizeof(AT) + (size_t)kAttnRows * D * 4 +
                        (size_t)kAttnRows * kAttnPos * 4 + 2 * kAttnRows * 4 + 16;
    static bool configured = false;
    if (!configured) {
        cudaFuncSetAttribute(attn_kernel<AT, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        configured = true;
    }
    attn_kernel<AT, D><<<dim3(kv.Hkv, n_split), 256, smem, s>>>(q, kv, apart, M, pos0, H, pps, n_split, scale, err);
}

int attention_splits(int ctx_len, int page_tokens, int Hkv, int n_sm, int max_splits, int *pps_out) {
    const int n_pages = (ctx_len + page_tokens - 1) / page_tokens;
    int pps = kAttnPos / page_tokens;                 // most pages one block can hold
    if (pps < 1) pps = 1;
    // enough blocks to fill the machine about twice, while slices stay whole pages
    while (pps > 1 && Hkv * ((n_pages + pps - 1) / pps) < 2 * n_sm) pps--;
    int n_split = (n_pages + pps - 1) / pps;
    while (n_split > max_splits) { pps++; n_split = (n_pages + pps - 1) / pps; }
    *pps_out = pps;
    return n_split;
}

void launch_attention(cudaStream_t s, int dtype, const float *q, const KvGeom &kv, float *apart,
                      float *attn_out, void *attn_split, int M, int pos0, int H, int n_sm, int max_splits, int *err) {
    int pps;
    const int n_split = attention_splits(pos0 + M, kv.page_tokens, kv.Hkv, n_sm, max_splits, &pps);
    const float scale = 1.0f / sqrtf((float)kv.D);
    if (dtype == 0) {
        if (kv.D == 64) attn_launch<float, 64>(s, q, kv, apart, M, pos0, H, pps, n_split, scale, err);
        else attn_launch<float, 128>(s, q, kv, apart, M, pos0, H, pps, n_split, scale, err);
    } else {
        if (kv.D == 64) attn_launch<bf16, 64>(s, q, kv, apart, M, pos0, H, pps, n_split, scale, err);
        else attn_launch<bf16, 128>(s, q, kv, apart, M, pos0, H, pps, n_split, scale, err);
    }
    attn_combine_kernel<<<dim3(H, M), kv.D, 0, s>>>(apart, attn_out, (bf16 *)attn_split, H, kv.D, n_split);
}

// ------------------------------------------------------------------------------------ SwiGLU, partial sums
__global__ void swiglu_kernel(PartView pv, float *h, bf16 *hs, int F) {
    const int m = blockIdx.y, i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= F) return;
    const float g = part_gather(pv, m, i), u = part_gather(pv, m, F + i);
    const float v = g / (1.0f + expf(-g)) * u;
    h[(size_t)m * F + i] = v;
    if (hs) store_split(hs, m, F, i, v);
}
void launch_swiglu(cudaStream_t s, const PartView &pv, float *h, void *h_split, int M, int F) {
    dim3 grid((F + 255) / 256, M);
    swiglu_kernel<<<grid, 256, 0, s>>>(pv, h, (bf16 *)h_split, F);
}

__global__ void reduce_partials_kernel(PartView pv, float *out, int R) {
    const int m = blockIdx.y, r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= R) return;
    out[(size_t)m * R + r] = part_gather(pv, m, r);
}
void launch_reduce_partials(cudaStream_t s, const PartView &pv, float *out, int M, int R) {
    reduce_partials_kernel<<<dim3((R + 255) / 256, M), 256, 0, s>>>(pv, out, R);
}

}  // namespace eesd
