// Host-callable launchers of the EESD model kernels.  `dtype` is EESD_F32 (0) or EESD_BF16 (1)
// and selects the element type of the weights and of the KV cache; the residual stream, partial
// sums, attention statistics and logits are fp32; the token rows fed to the tensor-core
// projections are fp32 values carried as two bf16 terms.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace eesd {

struct IntList16 { int32_t v[16]; };

// geometry of one paged KV cache slot
struct KvGeom {
    void *slot_base;            // first byte of the slot: [page][K|V][H_kv] blocks of page_tokens * D
                                // elements; element order inside a block: kv_layout.cuh
    const int32_t *page_table;  // logical page -> physical page
    int Hkv, D, page_tokens, n_pages_total;
};

// Equal split of U = tiles * KB work units (128-row weight tile x 64-wide k block) over G
// CTAs: CTA c owns units [start(c), start(c+1)); the first `rem` CTAs own one unit more.
// Each (CTA, tile) segment writes one [16][128] fp32 block of partial sums, block number
// cta + tile: unique, because the CTA ranges are disjoint and ordered (if CTA c reaches tile
// t + 1, CTA c + 1 starts no earlier than tile t + 1), and at most G + tiles - 1.  A tile's
// blocks are those of CTAs owner(first unit) .. owner(last unit), consecutive numbers.
struct StreamK {
    int U, KB, G, base, rem, tiles;
    __host__ __device__ int start(int c) const { return c * base + (c < rem ? c : rem); }
    __host__ __device__ int owner(int u) const {
        const int bnd = rem * (base + 1);
        return u < bnd ? u / (base + 1) : rem + (u - bnd) / base;
    }
};

// Where a projection left its fp32 partial sums.
//   mode 0: base[s * split_stride + m * R + r], s < S           (SIMT kernel, S = 1)
//   mode 1: blocks of the stream-K tensor-core kernel (numbered cta + tile, see StreamK)
struct PartView {
    const float *base;
    int mode, S, R;
    size_t split_stride;
    StreamK sk;
};

// RMSNorm statistics of the rows a projection consumed: the projection runs on x * g, and
// whoever reads its result multiplies row m by rstd(m) = 1 / sqrt(sum_b ssq[m][b] / d + eps)
// (the normalisation is a per-row scalar, so it commutes with the projection).
constexpr int kSsqBlocks = 16;   // partial sums of squares per row (1024 elements each)
struct RowScale {
    const float *ssq;   // [16][kSsqBlocks]; null: no scaling
    int nblk;
    float inv_d, eps;
};

// Rows of a verification pass that form a tree instead of a chain (several draft candidates
// per position).  Row m is stored at cache position pos0 + m, is rotated as position
// pos0 + depth[m], and sees every position before pos0 plus the rows whose bit is set in vis[m]
// (its ancestors and itself).  A chain is depth[m] = m, vis[m] = bits 0..m.
struct TreeRows {
    uint16_t vis[16];
    uint8_t depth[16];
};
// Rows of a pass that belong to several sequences decoded together (batch mode; an extension, the
// paper decodes one sequence at a time).  Sequence b owns rows row0[b] .. row0[b] + rows[b] - 1 of
// the pass, at consecutive positions pos0[b] .. of its own context, whose page table starts
// table_off[b] entries into the page-table array.  n_seq == 0: one sequence (the launcher's own
// M, pos0 and page table apply).
constexpr int kMaxSeqs = 8;
struct BatchRows {
    int n_seq;
    int row0[kMaxSeqs], rows[kMaxSeqs], pos0[kMaxSeqs], table_off[kMaxSeqs];
};
inline TreeRows chain_rows() {
    TreeRows t;
    for (int m = 0; m < 16; m++) { t.vis[m] = (uint16_t)((2u << m) - 1u); t.depth[m] = (uint8_t)m; }
    return t;
}

void launch_set_ints(cudaStream_t s, int32_t *dst, const IntList16 &vals, int n);
void launch_rope_table(cudaStream_t s, float2 *table, int max_ctx, int D, float theta);
// x[m] += partial sums (if pv); y = x[m] * g -> xn (fp32, may be null) and xs (two bf16 terms,
// [chunk of 16 rows][hi | lo][16][d], may be null); ssq[m][b] = sum of squares of block b (1024
// columns) of x[m]; cap[m] = x[m] (if cap).  The RMSNorm scale itself is applied by the consumers.
void launch_resid(cudaStream_t s, float *x, const PartView *pv, const float *g, float *xn, void *xs, float *cap,
                  float *ssq, int M, int d);
// Embedding gather (row m takes token tok[m * tok_stride]) and launch_resid(x, no partial sums, g, ...) on the rows, in one
// kernel (d % 4 == 0)
void launch_embed_resid(cudaStream_t s, int dtype, const int32_t *tok, int tok_stride, const void *E, int V, float *x, const float *g,
                        float *xn, void *xs, float *cap, float *ssq, int M, int d, int *err);
// out[sp][m][r] = sum_{k in split sp} A[m][k] * W[r][k]; returns the number of K splits written
int launch_gemm(cudaStream_t s, int dtype, const float *A, const void *W, float *out, int M, int R, int K);
// RoPE + KV append (+ q store).  part rows are [q heads | k heads | v heads] or, when
// only_kv, [k heads | v heads] starting at column kv_col0 of the projection result.
// tree (optional, M <= 16): row m is rotated as position pos0 + depth[m] and stored at pos0 + m.
void launch_qkv_post(cudaStream_t s, int dtype, const PartView &pv, const RowScale &rs, int M, int pos0, int H,
                     const KvGeom &kv, const float2 *rope, float *q, bool only_kv, int *err, int kv_col0 = 0,
                     const TreeRows *tree = nullptr, int row0 = 0);
// The same for the rows of a prompt pass (bf16 cache, D = 64 or 128, pv a plain [split][row][column] result): keys at
// columns kcol0 + kh * D, values H_kv * D columns further; whole 16-byte rows of the cache's core matrices per thread.
void launch_kv_append_wide(cudaStream_t s, const PartView &pv, const RowScale &rs, int Mtot, int pos0, const KvGeom &kv,
                           const float2 *rope, int kcol0, int *err);
// Fused attention step of one layer on M new rows: q/k/v of the new rows are taken from the
// QKV projection's partial sums (scaled by rs, rotated), the new keys/values are appended to
// the paged cache, every KV head's cached slice is read once, and the slices are merged into
// attn_out (fp32 [M][H*D], may be null) and attn_split (two bf16 terms, may be null).
// apart: H * max_splits * 16 * (D + 2) floats; tickets: zero-initialised counters, one per
// (KV head, sequence of a batch, batch of 16 or 32 (head, row) pairs).
// batch (optional, no tree): the rows belong to several sequences; M, pos0 and kv.page_table
// are then taken per sequence from it, and `M` is the largest row count of a sequence.
// early: the kernel may start (and read cached rows) while the kernel before it still runs;
// must be false when that kernel appends rows to the same cache slot.
void launch_attention(cudaStream_t s, int dtype, const PartView &pv, const RowScale &rs, const float2 *rope,
                      const KvGeom &kv, float *apart, unsigned int *tickets, float *attn_out, void *attn_split,
                      int M, int pos0, int H, int n_sm, int max_splits, bool early, int *err,
                      const TreeRows *tree, uint32_t wait_polls, const BatchRows *batch = nullptr);
// most context tokens the attention kernel of `dtype` can serve with pages of page_tokens
int attention_max_ctx(int dtype, int page_tokens);
// tensor-core attention (attn_tc.cu; bf16 cache): columns ((head, row) pairs) per block for `rows` pairs per KV head,
// slices of the context, and the launcher
int attention_tc_columns(int rows);
int attention_tc_splits(int ctx_len, int page_tokens, int Hkv, int n_batches, int n_sm, int max_splits, int *pps_out);
void launch_attention_tc(cudaStream_t s, const PartView &pv, const RowScale &rs, const float2 *rope, const KvGeom &kv, float *apart,
                         unsigned int *tickets, float *attn_out, void *attn_split, int M, int pos0, int H, int pps, int n_split,
                         bool early, int *err, const TreeRows *tree, uint32_t wait_polls, const BatchRows *batch = nullptr);
int attention_splits(int ctx_len, int page_tokens, int Hkv, int n_batches, int n_sm, int max_splits, int *pps_out);
// Causal prompt attention (attn_prompt.cu; bf16 cache, D = 64 or 128): Mtot rows at positions pos0.., 128 rows per
// block; the rows' keys / values must be in the cache already (launch_qkv_post with only_kv on the QKV
// result) and pv must be a plain [Mtot][R] result (mode 0).  attn_split: [chunk][hi | lo][16][H * D] bf16.
void launch_attention_prompt(cudaStream_t s, const PartView &pv, const RowScale &rs, const float2 *rope, const KvGeom &kv,
                             void *attn_split, int Mtot, int pos0, int H, int *err, uint32_t wait_polls);
// H^(T) of the calibration predictor: row `row` (or row *row_dev when row_dev is given) of x[.][d]
// is copied to hT (fp32) and, if xs is given, written as two bf16 terms into a one-chunk [32][d] matrix
void launch_copy_row(cudaStream_t s, const float *x, int row, const int32_t *row_dev, float *hT, void *xs, int d);
// theta_M = softmax(Wp [v ; hD])[1] with v = the d partial results of W^i H^(T) (Eq. 5)
void launch_cali_theta(cudaStream_t s, const PartView &pv, const float *Wp, const float *hD, int d, float *theta);
// Tree verification helpers.  launch_next_best: tokens ranked 1..width of one logit row (by
// logit, lower id first among equals): rank 1 -> *first (optional), ranks 2.. -> out[width - 1].  launch_tree_rows: the pass's token rows
// = chain tokens src_chain[0..K], then the leaves src_leaf[0..K * (width - 1)).
// launch_tree_walk: given the target's top-1 token of every row, walks the tree (chain token
// continues, a leaf ends the round, neither ends it with the target's token); writes
// result[0] = accepted draft tokens, result[1] = the round's last token, result[2] = row of the
// kept leaf or -1; the kept leaf's token replaces the chain token at its depth in chain[],
// and chain[0] becomes the round's last token (the next round's pending token).
// launch_kv_move: when result[2] >= 0, copies the keys / values stored at position
// pos0 + result[2] to position pos0 + result[0] in `slots` cache slots of slot_bytes each.
void launch_next_best(cudaStream_t s, const float *logits, int V, int width, int32_t *first, int32_t *out);
void launch_tree_rows(cudaStream_t s, const int32_t *src_chain, const int32_t *src_leaf, int K, int width, int32_t *rows);
void launch_tree_walk(cudaStream_t s, const int32_t *top, int32_t *chain, const int32_t *leaf, int K, int width,
                      int32_t *result);
void launch_kv_move(cudaStream_t s, int dtype, const KvGeom &kv0, size_t slot_bytes, int slots, int pos0,
                    const int32_t *result, int *err);
void launch_swiglu(cudaStream_t s, const PartView &pv, const RowScale &rs, float *h, void *h_split, int M, int F);
// out_stride: floats between consecutive output rows (0: R)
void launch_reduce_partials(cudaStream_t s, const PartView &pv, const RowScale &rs, float *out, int M, int R, size_t out_stride = 0);
// programmatic dependent launch (kernels start early and wait on-device for their producer):
// on by default, off when the environment variable EESD_NO_PDL is set
bool pdl_enabled();

// tensor-core projection (gemm_tc.cu)
int tc_init();                                   // once per process; 0 on success
bool tc_shape_ok(int R, int K);
// tiled: the matrix is stored tile-major, [rows / 128][cols / 64] tiles of [128][64] (box_rows must be 128)
bool tc_make_map(CUtensorMap *out, const void *base, int rows, int cols, int box_rows, bool tiled = false);
StreamK tc_plan(int R, int K, int n_sm);
// wait_polls: polls after which a wait inside the kernel gives up and raises the error word
void launch_gemm_tc(cudaStream_t s, const CUtensorMap &mW, const CUtensorMap &mX, float *part, const StreamK &sk,
                    int M, bool tiled, int *err, uint32_t wait_polls);
// wide projection for prompt processing: out[m][r] (fp32, row stride R) for m < Mtot rows kept
// as [chunk of 16][hi | lo][16][K] bf16 (mX from tc_make_map_rows); R % 128 == 0, K % 64 == 0
bool tc_make_map_rows(CUtensorMap *out, const void *base, int K, int chunks);
// splits > 1: the k range is cut into `splits` parts whose results land Mtot * R floats apart (PartView
// mode 0 with S = splits); gemm_wide_splits picks the count that fills the SMs best (at most max_splits)
int gemm_wide_splits(int R, int K, int Mtot, int n_sm, int max_splits);
void launch_gemm_wide(cudaStream_t s, const CUtensorMap &mW, const CUtensorMap &mX, float *out, int R, int K, int Mtot,
                      int n_sm, bool tiled, int splits, int *err, uint32_t wait_polls);
void launch_split_rows(cudaStream_t s, const float *x, void *xs, int M, int K);

// acceptance / sampling (accept.cu)
size_t accept_scratch_bytes(int B, int K);
void launch_accept(cudaStream_t s, const float *p_logits, const float *q_logits, const int32_t *tokens,
                   const float *u_acc, const float *u_res, int B, int K, int V, float T, void *scratch,
                   int32_t *n_acc, int32_t *y, int32_t *pending_out, int tok_stride = 0);   // tok_stride: ints between the sequences' token lists (0: K)
// logit_stride: floats between rows (0: V); out_stride: ints between results
void launch_sample_rows(cudaStream_t s, const float *logits, const float *u, int B, int V, float T,
                        int32_t *out, size_t logit_stride = 0, int out_stride = 1);

}  // namespace eesd
