// Model kernels of the EESD decode round (sm_100a): embedding gather, residual + RMSNorm,
// skinny projections (M <= 16 token rows against a streamed weight matrix), RoPE + paged KV
// append, paged decode attention with a causal block of new rows, SwiGLU.
//
// Every reduction has a fixed combination order, so a pass is bit-reproducible.
#include "common.cuh"
#include "kernels.cuh"

namespace eesd {

typedef __nv_bfloat16 bf16;

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
// One block per token row.  x[m] += sum_s part[s][m]; xn[m] = RMSNorm(x[m]) * g.
__global__ void __launch_bounds__(256) resid_norm_kernel(float *x, const float *part, int S, size_t part_stride,
                                                         const float *g, float *xn, float *cap, int d, float eps) {
    extern __shared__ float row[];  // d floats + 33 scratch
    float *scratch = row + d;
    const int m = blockIdx.x;
    float *xr = x + (size_t)m * d;
    float ss = 0.f;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        float v = xr[i];
        for (int s = 0; s < S; s++) v += part[(size_t)s * part_stride + (size_t)m * d + i];
        row[i] = v;
        if (S > 0) xr[i] = v;
        if (cap) cap[(size_t)m * d + i] = v;
        ss += v * v;
    }
    if (!g) return;
    ss = block_sum(ss, scratch);
    const float rstd = 1.0f / sqrtf(ss / (float)d + eps);
    for (int i = threadIdx.x; i < d; i += blockDim.x) xn[(size_t)m * d + i] = row[i] * rstd * g[i];
}
void launch_resid_norm(cudaStream_t s, float *x, const float *part, int S, const float *g, float *xn, float *cap,
                       int M, int d, float eps) {
    size_t smem = (size_t)(d + 33) * sizeof(float);
    size_t stride = (size_t)M * d;
    if (!part) S = 0;
    resid_norm_kernel<<<M, 256, smem, s>>>(x, part, S, stride, g, xn, cap, d, eps);
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
__global__ void qkv_post_kernel(const float *part, int S, size_t part_stride, int Rw, int pos0, int H, KvGeom kv,
                                const float2 *rope, float *q, int head_off, int *err) {
    const int hh = blockIdx.x + head_off;  // 0..H-1 q, H..H+Hkv-1 k, then v
    const int m = blockIdx.y, i = threadIdx.x, D = kv.D;
    const int col = blockIdx.x * D + 2 * i;
    float a = 0.f, b = 0.f;
    for (int s = 0; s < S; s++) {
        const float *p = part + (size_t)s * part_stride + (size_t)m * Rw + col;
        a += p[0];
        b += p[1];
    }
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
void launch_qkv_post(cudaStream_t s, int dtype, const float *part, int S, int M, int pos0, int H,
                     const KvGeom &kv, const float2 *rope, float *q, bool only_kv, int *err) {
    const int heads = only_kv ? 2 * kv.Hkv : H + 2 * kv.Hkv;
    const int Rw = heads * kv.D;
    dim3 grid(heads, M);
    size_t stride = (size_t)M * Rw;
    if (dtype == 0) qkv_post_kernel<float><<<grid, kv.D / 2, 0, s>>>(part, S, stride, Rw, pos0, H, kv, rope, q, only_kv ? H : 0, err);
    else qkv_post_kernel<bf16><<<grid, kv.D / 2, 0, s>>>(part, S, stride, Rw, pos0, H, kv, rope, q, only_kv ? H : 0, err);
}

// ------------------------------------------------------------------------------------ paged decode attention
// grid (H, n_split), 256 threads.  Block (h, sp) handles query head h for all M new rows over
// its share of the cached positions [0, pos0 + M) (split by pages); row m sees positions
// <= pos0 + m.  Writes un-normalised output, running max and sum per row; the combine kernel
// merges the splits in index order.
template <typename AT, int D>
__global__ void __launch_bounds__(256) attn_kernel(const float *__restrict__ q, KvGeom kv, float *__restrict__ apart,
                                                   int M, int pos0, int H, int n_split, float scale) {
    constexpr int CH = 128;        // positions per chunk
    constexpr int G = 256 / D;     // row groups in the PV phase
    constexpr int RPG = kMaxRows / G;
    constexpr int VEC = Vec16<AT>::N;
    __shared__ __align__(16) float sq[kMaxRows][D];
    __shared__ float ssc[kMaxRows][CH];
    __shared__ float s_m[kMaxRows], s_l[kMaxRows], s_c[kMaxRows];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int h = blockIdx.x, sp = blockIdx.y, kh = h / (H / kv.Hkv);
    const int PT = kv.page_tokens;
    const int ctx_len = pos0 + M;
    const int n_pages = (ctx_len + PT - 1) / PT;
    const int pps = (n_pages + n_split - 1) / n_split;
    const int lo = sp * pps * PT;
    const int hi = min(ctx_len, lo + pps * PT);
    const AT *base = (const AT *)kv.slot_base;
    const size_t head_stride = (size_t)PT * D;

    for (int idx = tid; idx < kMaxRows * D; idx += 256) {
        int m = idx / D, e = idx - m * D;
        sq[m][e] = m < M ? q[(size_t)m * H * D + (size_t)h * D + e] * scale : 0.f;
    }
    if (tid < kMaxRows) { s_m[tid] = -INFINITY; s_l[tid] = 0.f; s_c[tid] = 1.f; }
    float o[RPG];
#pragma unroll
    for (int r = 0; r < RPG; r++) o[r] = 0.f;
    __syncthreads();

    for (int c0 = lo; c0 < hi; c0 += CH) {
        {   // phase 1: scores.  thread -> position j, half of the rows
            const int j = tid & (CH - 1), half = tid / CH;
            const int pos = c0 + j;
            const bool valid = pos < hi;
            float acc[8];
#pragma unroll
            for (int r = 0; r < 8; r++) acc[r] = 0.f;
            if (valid && half * 8 < M) {
                const int page = kv.page_table[pos / PT];
                const AT *kp = base + (((size_t)page * 2 + 0) * kv.Hkv + kh) * head_stride + (size_t)(pos % PT) * D;
#pragma unroll 4
                for (int e0 = 0; e0 < D; e0 += VEC) {
                    float kvv[VEC];
                    Vec16<AT>::load(kp + e0, kvv);
#pragma unroll
                    for (int r = 0; r < 8; r++) {
                        const int m = half * 8 + r;
                        if (m < M) {
#pragma unroll
                            for (int v = 0; v < VEC; v++) acc[r] = fmaf(kvv[v], sq[m][e0 + v], acc[r]);
                        }
                    }
                }
            }
#pragma unroll
            for (int r = 0; r < 8; r++) {
                const int m = half * 8 + r;
                ssc[m][j] = (valid && m < M && pos <= pos0 + m) ? acc[r] : -INFINITY;
            }
        }
        __syncthreads();
        // phase 2: online softmax bookkeeping, warp w handles rows w and w + 8
        for (int m = warp; m < M; m += 8) {
            float mx = -INFINITY;
            for (int j = lane; j < CH; j += 32) mx = fmaxf(mx, ssc[m][j]);
            mx = warp_max(mx);
            const float m_old = s_m[m];
            const float m_new = fmaxf(m_old, mx);
            float sum = 0.f;
            for (int j = lane; j < CH; j += 32) {
                float sv = ssc[m][j];
                float p = (sv == -INFINITY) ? 0.f : expf(sv - m_new);
                ssc[m][j] = p;
                sum += p;
            }
            sum = warp_sum(sum);
            if (lane == 0) {
                float c = (m_old == -INFINITY) ? 0.f : expf(m_old - m_new);
                s_c[m] = c;
                s_l[m] = s_l[m] * c + sum;
                s_m[m] = m_new;
            }
        }
        __syncthreads();
        {   // phase 3: o = o * c + P V.  thread -> (d, row group)
            const int dd = tid % D, grp = tid / D;
#pragma unroll
            for (int r = 0; r < RPG; r++) o[r] *= s_c[grp * RPG + r];
            const int nj = min(CH, hi - c0);
            if (grp * RPG < M) {
                for (int j = 0; j < nj; j++) {
                    const int pos = c0 + j;
                    const int page = kv.page_table[pos / PT];
                    const float v = to_f(base[(((size_t)page * 2 + 1) * kv.Hkv + kh) * head_stride +
                                              (size_t)(pos % PT) * D + dd]);
#pragma unroll
                    for (int r = 0; r < RPG; r++) o[r] = fmaf(ssc[grp * RPG + r][j], v, o[r]);
                }
            }
        }
        __syncthreads();
    }
    {
        const int dd = tid % D, grp = tid / D;
        float *dst = apart + ((size_t)h * n_split + sp) * kMaxRows * (D + 2);
#pragma unroll
        for (int r = 0; r < RPG; r++) {
            const int m = grp * RPG + r;
            if (m < M) dst[(size_t)m * (D + 2) + dd] = o[r];
        }
        if (tid < M) {
            dst[(size_t)tid * (D + 2) + D] = s_m[tid];
            dst[(size_t)tid * (D + 2) + D + 1] = s_l[tid];
        }
    }
}

// grid (H, M), block D: merge the splits of one (head, row)
__global__ void attn_combine_kernel(const float *apart, float *out, int H, int D, int n_split) {
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
    out[(size_t)m * H * D + (size_t)h * D + dd] = den > 0.f ? num / den : 0.f;
}

void launch_attention(cudaStream_t s, int dtype, const float *q, const KvGeom &kv, float *apart,
                      float *attn_out, int M, int pos0, int H, int n_split) {
    dim3 grid(H, n_split);
    const float scale = 1.0f / sqrtf((float)kv.D);
    if (dtype == 0) {
        if (kv.D == 64) attn_kernel<float, 64><<<grid, 256, 0, s>>>(q, kv, apart, M, pos0, H, n_split, scale);
        else attn_kernel<float, 128><<<grid, 256, 0, s>>>(q, kv, apart, M, pos0, H, n_split, scale);
    } else {
        if (kv.D == 64) attn_kernel<bf16, 64><<<grid, 256, 0, s>>>(q, kv, apart, M, pos0, H, n_split, scale);
        else attn_kernel<bf16, 128><<<grid, 256, 0, s>>>(q, kv, apart, M, pos0, H, n_split, scale);
    }
    attn_combine_kernel<<<dim3(H, M), kv.D, 0, s>>>(apart, attn_out, H, kv.D, n_split);
}

// ------------------------------------------------------------------------------------ SwiGLU, partial sums
__global__ void swiglu_kernel(const float *part, int S, size_t part_stride, float *h, int F) {
    const int m = blockIdx.y, i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= F) return;
    float g = 0.f, u = 0.f;
    for (int s = 0; s < S; s++) {
        const float *p = part + (size_t)s * part_stride + (size_t)m * 2 * F;
        g += p[i];
        u += p[F + i];
    }
    const float sg = g / (1.0f + expf(-g));
    h[(size_t)m * F + i] = sg * u;
}
void launch_swiglu(cudaStream_t s, const float *part, int S, float *h, int M, int F) {
    dim3 grid((F + 255) / 256, M);
    size_t stride = (size_t)M * 2 * F;
    swiglu_kernel<<<grid, 256, 0, s>>>(part, S, stride, h, F);
}

__global__ void reduce_partials_kernel(const float *part, int S, size_t stride, float *out, size_t n) {
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    float v = 0.f;
    for (int s = 0; s < S; s++) v += part[(size_t)s * stride + i];
    out[i] = v;
}
void launch_reduce_partials(cudaStream_t s, const float *part, int S, float *out, int M, int R) {
    size_t n = (size_t)M * R;
    reduce_partials_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(part, S, n, out, n);
}

}  // namespace eesd
