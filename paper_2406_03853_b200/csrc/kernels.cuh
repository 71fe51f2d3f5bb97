// Host-callable launchers of the EESD model kernels.  `dtype` is EESD_F32 (0) or EESD_BF16 (1)
// and selects the element type of the weights and of the KV cache; the residual stream, the
// token rows fed to projections, partial sums, attention statistics and logits are fp32.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace eesd {

struct IntList16 { int32_t v[16]; };

// geometry of one paged KV cache slot
struct KvGeom {
    void *slot_base;            // first byte of the slot: [page][K|V][H_kv][page_tokens][D]
    const int32_t *page_table;  // logical page -> physical page
    int Hkv, D, page_tokens, n_pages_total;
};

void launch_set_ints(cudaStream_t s, int32_t *dst, const IntList16 &vals, int n);
void launch_rope_table(cudaStream_t s, float2 *table, int max_ctx, int D, float theta);
void launch_embed(cudaStream_t s, int dtype, const int32_t *tok, const void *E, float *x, float *cap,
                  int M, int d, int V, int *err);
// x[m] += sum_s part[s][m] (if part); xn[m] = cast(RMSNorm(x[m]) * g) (if g); cap[m] = x[m] (if cap)
void launch_resid_norm(cudaStream_t s, float *x, const float *part, int S, const float *g, float *xn, float *cap,
                       int M, int d, float eps);
// out[sp][m][r] = sum_{k in split sp} A[m][k] * W[r][k]; returns the number of K splits written
int launch_gemm(cudaStream_t s, int dtype, const float *A, const void *W, float *out, int M, int R, int K);
// RoPE + KV append (+ q store).  part rows are [q heads | k heads | v heads] or, when
// only_kv, [k heads | v heads].
void launch_qkv_post(cudaStream_t s, int dtype, const float *part, int S, int M, int pos0, int H,
                     const KvGeom &kv, const float2 *rope, float *q, bool only_kv, int *err);
void launch_attention(cudaStream_t s, int dtype, const float *q, const KvGeom &kv, float *apart,
                      float *attn_out, int M, int pos0, int H, int n_split);
void launch_swiglu(cudaStream_t s, const float *part, int S, float *h, int M, int F);
void launch_reduce_partials(cudaStream_t s, const float *part, int S, float *out, int M, int R);

// acceptance / sampling (accept.cu)
size_t accept_scratch_bytes(int B, int K);
void launch_accept(cudaStream_t s, const float *p_logits, const float *q_logits, const int32_t *tokens,
                   const float *u_acc, const float *u_res, int B, int K, int V, float T, void *scratch,
                   int32_t *n_acc, int32_t *y, int32_t *pending_out);
void launch_sample_rows(cudaStream_t s, const float *logits, const float *u, int B, int V, float T,
                        int32_t *out);

}  // namespace eesd
