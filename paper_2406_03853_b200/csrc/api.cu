// C ABI of the EESD decode-round library: context, KV page allocator, pass assembly,
// generation loop (Algorithm 1) and the host-side Thompson-sampling controller (Algorithm 2).
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <chrono>
#include <new>
#include <vector>

#include "../../include/eesd.h"
#include "kernels.cuh"

using namespace eesd;

namespace {

struct LayerW {
    const float *g_attn, *g_ffn;
    const char *wqkv, *wo, *wgu, *wd;
    CUtensorMap m_qkv, m_o, m_gu, m_d;  // tensor-core path only
};

// which activation matrix feeds a projection
enum { X_NORM = 0, X_ATTN = 1, X_FFN = 2, X_CALI = 3 };   // X_CALI: H^(T) of the calibration predictor
// the distinct projection shapes of a pass (each has its own stream-K plan and block table)
enum { P_QKV = 0, P_O = 1, P_GU = 2, P_D = 3, P_EXIT_KV = 4, P_HEAD = 5, P_CALI = 6, P_COUNT = 7 };

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

int check_config(const eesd_config *c) {
    if (!c) return EESD_ERR_BADARG;
    if (c->d_model > 1024 * kSsqBlocks || c->n_kv_heads > 1024) return EESD_ERR_UNSUPPORTED;
    if (c->d_model <= 0 || c->n_heads <= 0 || c->n_kv_heads <= 0 || c->ffn_dim <= 0 || c->vocab <= 0 ||
        c->n_layers <= 0 || c->max_ctx <= 1)
        return EESD_ERR_BADARG;
    if (c->n_heads % c->n_kv_heads) return EESD_ERR_BADARG;
    if (c->n_early < 1 || c->n_early > c->n_layers) return EESD_ERR_BADARG;
    if (c->dtype != EESD_F32 && c->dtype != EESD_BF16) return EESD_ERR_BADARG;
    if (c->head_dim != 64 && c->head_dim != 128) return EESD_ERR_UNSUPPORTED;
    if (c->d_model % 8 || c->ffn_dim % 8 || (c->n_heads * c->head_dim) % 8) return EESD_ERR_UNSUPPORTED;
    if (c->page_tokens < 8 || c->page_tokens > 128 || (c->page_tokens & (c->page_tokens - 1))) return EESD_ERR_BADARG;
    // attention: at most 64 slices per head, each as long as one block can hold
    if (c->max_ctx > 12288 || c->max_ctx > attention_max_ctx(c->dtype, c->page_tokens)) return EESD_ERR_UNSUPPORTED;
    if (c->k_cap < 1 || c->k_cap > EESD_MAX_ROWS - 1) return EESD_ERR_BADARG;
    if (c->temperature < 0.f) return EESD_ERR_BADARG;
    if (c->controller != EESD_CTRL_FIXED_K && c->controller != EESD_CTRL_BETA_TS && c->controller != EESD_CTRL_CALI_TS)
        return EESD_ERR_BADARG;
    if (c->controller == EESD_CTRL_CALI_TS && (!(c->cali_sigma_m > 0.f) || !(c->cali_sigma_s > 0.f))) return EESD_ERR_BADARG;
    if (c->controller == EESD_CTRL_FIXED_K && c->fixed_k < 1) return EESD_ERR_BADARG;
    if (c->alpha0 < 1 || c->beta0 < 1) return EESD_ERR_BADARG;
    if (c->rms_eps < 0.f || c->rope_theta <= 1.f) return EESD_ERR_BADARG;
    if (c->n_exit_layers < 0 || c->n_exit_layers > 4) return EESD_ERR_BADARG;
    if (c->tree_width < 0 || c->tree_width > 4) return EESD_ERR_BADARG;
    if (c->tree_width > 1) {   // tree verification: greedy only, 1 + k_cap * width rows in one pass
        if (c->temperature != 0.f || c->controller == EESD_CTRL_CALI_TS) return EESD_ERR_UNSUPPORTED;
        if (1 + c->k_cap * c->tree_width > EESD_MAX_ROWS) return EESD_ERR_BADARG;
    }
    return EESD_OK;
}

struct Workspace {
    size_t x, x_save, xn, attn, h, xs[3], ssq, tickets, part, apart, logits_p, logits_q, rope, page_table, ints, u_dev, u_stage, err,
        accept, wx, wx_save, wout, wout_floats, wxs[3], wssq, wtok, hT, xs_cali, theta, total;
};

constexpr int kPartSplits = 1;   // room for K-split partial sums of one projection
constexpr int kAttnSplits = 64;  // most KV slices per head in attention
constexpr int kIntSlots = 128;   // small device integer area
constexpr int kMaxSm = 256;      // upper bound on the SM count the work splits are planned for
constexpr int kCtasPerSm = 2;    // projection CTAs per SM (gemm_tc.cu: two 4-stage rings fit one SM)
constexpr int kPrefillRows = 512; // most prompt rows per pass of the wide (prompt) path
constexpr uint32_t kDefaultWaitPolls = 1u << 23;   // polls before a wait inside a kernel gives up (a poll parks the thread for up to about 200 ns: under two seconds)

// early-exit layers of the draft model (0 in the configuration reads as 1, the paper's setting)
int n_exit(const eesd_config *c) { return c->n_exit_layers < 1 ? 1 : c->n_exit_layers; }

bool tc_shapes_ok(const eesd_config *c) {
    const int qd = c->n_heads * c->head_dim, kvd = c->n_kv_heads * c->head_dim;
    return c->dtype == EESD_BF16 && qd % 128 == 0 && tc_shape_ok(qd + 2 * kvd, c->d_model) && tc_shape_ok(c->d_model, qd) &&
           tc_shape_ok(2 * c->ffn_dim, c->d_model) && tc_shape_ok(c->d_model, c->ffn_dim) &&
           tc_shape_ok(2 * kvd, c->d_model) && tc_shape_ok(c->vocab, c->d_model);
}

// rows the wide path's buffers hold (a multiple of 128); 0 when the model cannot use it
int prefill_rows(const eesd_config *c) {
    if (!tc_shapes_ok(c)) return 0;
    const int need = (c->max_ctx - 1 + 127) / 128 * 128;
    return need < kPrefillRows ? need : kPrefillRows;
}

// arrival counters of the attention merge: one per (KV head, sequence of a batch, batch of (head, row) pairs); at most
// n_kv_heads * 8 * (pairs of a sequence / 16 + 1) <= n_heads + 8 * n_kv_heads of them are in use
size_t ticket_count(const eesd_config *c) { return 1024 + (size_t)9 * c->n_heads; }

// entries of one sequence's page table
size_t table_len(const eesd_config *c) { return (size_t)c->max_ctx / c->page_tokens + 2; }

Workspace carve(const eesd_config *c) {
    Workspace w;
    const size_t R = EESD_MAX_ROWS;
    const size_t qd = (size_t)c->n_heads * c->head_dim, kvd = (size_t)c->n_kv_heads * c->head_dim;
    size_t maxR = qd + 2 * kvd;
    if ((size_t)2 * c->ffn_dim > maxR) maxR = (size_t)2 * c->ffn_dim;
    if ((size_t)c->vocab > maxR) maxR = c->vocab;
    if ((size_t)c->d_model > maxR) maxR = c->d_model;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    w.x = take(R * c->d_model * 4);
    w.x_save = take(n_exit(c) > 1 ? R * c->d_model * 4 : 0);   // the target's rows while the exit layers before the last run on a copy
    w.xn = take(R * c->d_model * 4);
    w.attn = take(R * qd * 4);
    w.h = take(R * (size_t)c->ffn_dim * 4);
    // the same three activation matrices as two bf16 terms, [32][K] (tensor-core path)
    w.xs[X_NORM] = take(2 * R * (size_t)c->d_model * 2);
    w.xs[X_ATTN] = take(2 * R * qd * 2);
    w.xs[X_FFN] = take(2 * R * (size_t)c->ffn_dim * 2);
    w.ssq = take((size_t)EESD_MAX_ROWS * kSsqBlocks * 4);
    w.tickets = take(ticket_count(c) * 4);
    {   // partial sums: SIMT layout [splits][16][maxR], or stream-K blocks of the widest projection
        size_t part_floats = (size_t)kPartSplits * R * maxR;
        const size_t sk_floats = (maxR / 128 + (size_t)kMaxSm * kCtasPerSm) * R * 128;  // blocks <= tiles + CTAs
        if (sk_floats > part_floats) part_floats = sk_floats;
        w.part = take(part_floats * 4);
    }
    w.apart = take((size_t)c->n_heads * kAttnSplits * R * (c->head_dim + 2) * 4);
    w.logits_p = take(R * (size_t)c->vocab * 4);
    w.logits_q = take(R * (size_t)c->vocab * 4);
    w.rope = take((size_t)c->max_ctx * (c->head_dim / 2) * 8);
    w.page_table = take(table_len(c) * kMaxSeqs * 4);   // one table per sequence of a batch (one sequence: the first)
    w.ints = take(kIntSlots * 4);
    w.u_dev = take((size_t)3 * c->max_ctx * 4);
    w.u_stage = take(64 * 4);
    w.err = take(16);
    w.accept = take(accept_scratch_bytes(kMaxSeqs, EESD_MAX_ROWS));
    w.hT = take((size_t)c->d_model * 4);
    w.xs_cali = take(2 * R * (size_t)c->d_model * 2);
    w.theta = take(16);
    w.wx = w.wx_save = w.wout = w.wout_floats = w.wssq = w.wtok = w.wxs[0] = w.wxs[1] = w.wxs[2] = 0;
    if (const size_t P = (size_t)prefill_rows(c)) {
        // prompt path: residual stream, one projection result, the three activation matrices as
        // two bf16 terms ([chunk of 16][hi | lo][16][K]), RMSNorm statistics, token ids
        size_t wideR = qd + 2 * kvd;
        if ((size_t)2 * c->ffn_dim > wideR) wideR = (size_t)2 * c->ffn_dim;
        if ((size_t)c->d_model > wideR) wideR = c->d_model;
        w.wx = take(P * c->d_model * 4);
        w.wx_save = take(n_exit(c) > 1 ? P * c->d_model * 4 : 0);
        w.wout = take(P * wideR * 4);
        w.wout_floats = P * wideR;
        w.wxs[X_NORM] = take(2 * P * (size_t)c->d_model * 2);
        w.wxs[X_ATTN] = take(2 * P * qd * 2);
        w.wxs[X_FFN] = take(2 * P * (size_t)c->ffn_dim * 2);
        w.wssq = take(P * kSsqBlocks * 4);
        w.wtok = take(P * 4);
    }
    w.total = o;
    return w;
}

// offsets inside the device integer area
constexpr int kRoundTok = 0;   // [17]: pending token, then the round's draft tokens
constexpr int kRowTok = 20;    // [16]: token rows of a prefill chunk / verify_only
constexpr int kResult = 40;    // [3]: n_accept, next token, row of the kept leaf (tree verification) or -1; batch mode: [8] n_accept, [8] next tokens
constexpr int kLeafTok = 64;   // [15]: tree verification: leaves of depth 1, depth 2, ... (width - 1 each)
constexpr int kTreeTop = 80;   // [16]: tree verification: the target's top-1 token of every row

}  // namespace

struct eesd_ctx {
    eesd_config cfg;
    eesd_buffers buf;
    eesd_layout lay;
    cudaStream_t stream;
    size_t es;
    // device pointers
    float *x, *x_save, *xn, *attn, *h, *part, *apart, *logits_p, *logits_q, *u_dev, *u_stage, *capture;
    void *accept_scratch;
    void *xs[4];                 // bf16 hi/lo copies of xn, attn, h, and of H^(T) (calibration predictor)
    float *ssq;                  // RMSNorm partial sums of squares of the rows in xn / xs[X_NORM]
    unsigned int *tickets;       // arrival counters of the attention merge
    CUtensorMap m_x[4];
    // Thompson sampling with calibration
    float *hT, *theta_dev;       // H^(T) (fp32 [d]) and the predictor's output
    const char *cali_w;          // W^1..W^10
    const float *cali_wp;
    CUtensorMap m_cali[10];
    double theta_hat;
    int64_t n_verify, n_trials;
    // prompt (wide) path: up to wide_rows prompt rows per pass
    int wide_rows;
    float *wx, *wx_save, *wout, *wssq;
    size_t wout_floats;          // room in wout
    void *wxs[3];
    int32_t *wtok;
    CUtensorMap m_wx[3];
    CUtensorMap m_exit_kv, m_lm_head, m_exit_head;
    bool use_tc;
    uint32_t wait_polls;         // bound of the waits inside the kernels (eesd_set_wait_limit)
    int n_sm;
    StreamK plan[P_COUNT];       // tensor-core path: work split per shape
    float2 *rope;
    int32_t *page_table, *ints;
    int *err;
    std::vector<LayerW> layers;  // L target layers, then the early-exit layers (indices L .. L + E - 1; cache slots likewise)
    int E;                       // early-exit layers
    const void *embed, *lm_head, *exit_head;
    const float *g_final, *g_exit;
    // KV pool
    int64_t n_pages_total;
    size_t slot_bytes;
    std::vector<int32_t> free_pages, page_of;
    // sequence state
    std::vector<int32_t> tokens;
    bool prefilled;
    // batch mode (several sequences decoded together): the other sequences' state is parked here while one is
    // selected; page_table points at the selected sequence's table inside the array starting at page_table0
    struct Seq { std::vector<int32_t> tokens, page_of; bool prefilled; };
    std::vector<Seq> seqs;       // empty: batch mode off
    int32_t *page_table0;
    const BatchRows *batch_cur;  // geometry of the pass being enqueued (null: one sequence)
    BatchRows batch_rows;
    int round_k;
    int64_t alpha, beta;
    int64_t launches;
    // tree verification: geometry of the pass being enqueued (null: a chain), leaves kept so far
    const TreeRows *tree_cur;
    TreeRows tree_rows;
    int64_t leaves_kept;
    int32_t *h_result;  // pinned: [0] n_accept, [1] next token, [2] error word, [3] row of the kept leaf or -1, [8..23] draft tokens
    cudaEvent_t ev[7];  // prefill start / end, draft start, verify start, round end, start / end of an acceptance or predictor step
    char cuda_err[256];
};

namespace {

#define CU(ctx, call)                                                                       \
    do {                                                                                    \
        cudaError_t e_ = (call);                                                            \
        if (e_ != cudaSuccess) {                                                            \
            snprintf((ctx)->cuda_err, sizeof((ctx)->cuda_err), "%s: %s", #call, cudaGetErrorString(e_)); \
            return EESD_ERR_CUDA;                                                           \
        }                                                                                   \
    } while (0)

int check_launch(eesd_ctx *c) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        snprintf(c->cuda_err, sizeof(c->cuda_err), "kernel launch: %s", cudaGetErrorString(e));
        return EESD_ERR_CUDA;
    }
    return EESD_OK;
}

KvGeom kv_geom(eesd_ctx *c, int slot) {
    KvGeom g;
    g.slot_base = (char *)c->buf.kv_pool + (size_t)slot * c->slot_bytes;
    g.page_table = c->batch_cur ? c->page_table0 : c->page_table;   // a batch pass offsets it per sequence
    g.Hkv = c->cfg.n_kv_heads;
    g.D = c->cfg.head_dim;
    g.page_tokens = c->cfg.page_tokens;
    g.n_pages_total = (int)c->n_pages_total;
    return g;
}

bool tree_on(const eesd_ctx *c) { return c->cfg.tree_width > 1; }

// make sure pages exist for `n_tokens` cache rows; pushes new table entries to the device
int ensure_pages(eesd_ctx *c, int n_tokens) {
    const int PT = c->cfg.page_tokens;
    const int need = (n_tokens + PT - 1) / PT;
    while ((int)c->page_of.size() < need) {
        IntList16 l;
        int first = (int)c->page_of.size(), n = 0;
        while ((int)c->page_of.size() < need && n < 16) {
            if (c->free_pages.empty()) return EESD_ERR_CTX_FULL;
            int32_t p = c->free_pages.back();
            c->free_pages.pop_back();
            c->page_of.push_back(p);
            l.v[n++] = p;
        }
        launch_set_ints(c->stream, c->page_table + first, l, n);
        c->launches++;
    }
    return EESD_OK;
}

// give back pages that hold no valid row when only `n_tokens` rows are valid
void trim_pages(eesd_ctx *c, int n_tokens) {
    const int PT = c->cfg.page_tokens;
    const int need = (n_tokens + PT - 1) / PT;
    while ((int)c->page_of.size() > need) {
        c->free_pages.push_back(c->page_of.back());
        c->page_of.pop_back();
    }
}

// One projection: out = X[which] . W^T.  Tensor-core stream-K kernel when the context uses it
// (bf16, tile-aligned shapes), else the SIMT kernel.  Returns where the partial sums are.
PartView run_proj(eesd_ctx *c, const void *W, const CUtensorMap *mW, int shape, int which, int M, int R, int K) {
    PartView pv = {};
    pv.base = c->part;
    pv.R = R;
    if (c->use_tc) {
        pv.mode = 1;
        pv.sk = c->plan[shape];
        launch_gemm_tc(c->stream, *mW, c->m_x[which], c->part, c->plan[shape], M, true, c->err, c->wait_polls);
    } else {
        const float *A = which == X_NORM ? c->xn : which == X_ATTN ? c->attn : which == X_FFN ? c->h : c->hT;
        pv.mode = 0;
        pv.S = launch_gemm(c->stream, c->cfg.dtype, A, W, c->part, M, R, K);
        pv.split_stride = (size_t)M * R;
    }
    c->launches++;
    return pv;
}

RowScale norm_scale(eesd_ctx *c) {
    RowScale rs;
    rs.ssq = c->ssq;
    rs.nblk = (c->cfg.d_model + 1023) / 1024;
    rs.inv_d = 1.0f / (float)c->cfg.d_model;
    rs.eps = c->cfg.rms_eps;
    return rs;
}

// residual update + the input of the next normalised projection: x += partials; y = x * g
void run_resid(eesd_ctx *c, const PartView *pv, const float *g, float *cap, int M) {
    launch_resid(c->stream, c->x, pv, g, c->use_tc ? nullptr : c->xn, c->xs[X_NORM], cap, c->ssq, M, c->cfg.d_model);
    c->launches++;
}

// embedding rows of M tokens (tok[m * tok_stride]) and, in the same kernel, the first layer's normalised rows
void run_embed(eesd_ctx *c, const int32_t *tok, int tok_stride, int M, float *cap) {
    launch_embed_resid(c->stream, c->cfg.dtype, tok, tok_stride, c->embed, c->cfg.vocab, c->x, c->layers[0].g_attn,
                       c->use_tc ? nullptr : c->xn, c->xs[X_NORM], cap, c->ssq, M, c->cfg.d_model, c->err);
    c->launches++;
}

// one decoder layer on M rows at positions pos0.. ; on entry y = x * g_attn of this layer (and
// its sums of squares) are in place; on exit x holds the layer output and y = x * g_next.
void run_layer(eesd_ctx *c, const LayerW &w, int slot, int M, int pos0, const float *g_next, float *cap) {
    const eesd_config &f = c->cfg;
    const int qd = f.n_heads * f.head_dim, kvd = f.n_kv_heads * f.head_dim, d = f.d_model, F = f.ffn_dim;
    cudaStream_t s = c->stream;
    const RowScale rs = norm_scale(c);
    PartView pv = run_proj(c, w.wqkv, &w.m_qkv, P_QKV, X_NORM, M, qd + 2 * kvd, d);
    launch_attention(s, f.dtype, pv, rs, c->rope, kv_geom(c, slot), c->apart, c->tickets, c->use_tc ? nullptr : c->attn,
                     c->xs[X_ATTN], M, pos0, f.n_heads, c->n_sm, kAttnSplits, true, c->err, c->tree_cur, c->wait_polls, c->batch_cur);
    pv = run_proj(c, w.wo, &w.m_o, P_O, X_ATTN, M, d, qd);
    run_resid(c, &pv, w.g_ffn, nullptr, M);
    pv = run_proj(c, w.wgu, &w.m_gu, P_GU, X_NORM, M, 2 * F, d);
    launch_swiglu(s, pv, rs, c->use_tc ? nullptr : c->h, c->xs[X_FFN], M, F);
    pv = run_proj(c, w.wd, &w.m_d, P_D, X_FFN, M, d, F);
    run_resid(c, &pv, g_next, cap, M);
    c->launches += 2;
}

float *cap_slot(eesd_ctx *c, int index) {
    return c->capture ? c->capture + (size_t)index * EESD_MAX_ROWS * c->cfg.d_model : nullptr;
}

// Target model on M rows (device token ids) at positions pos0.. : all L layers, the exit
// layer's keys/values after layer N, and (optionally) final norm + LM head into logits_p.
int run_target(eesd_ctx *c, const int32_t *d_tok, int M, int pos0, bool want_logits) {
    const eesd_config &f = c->cfg;
    cudaStream_t s = c->stream;
    const int L = f.n_layers, d = f.d_model;
    run_embed(c, d_tok, 1, M, cap_slot(c, 0));
    for (int l = 0; l < L; l++) {
        const bool exit_here = (l == f.n_early - 1);
        const float *g_after = exit_here ? c->layers[L].g_attn : (l + 1 < L ? c->layers[l + 1].g_attn : c->g_final);
        run_layer(c, c->layers[l], l, M, pos0, g_after, cap_slot(c, l + 1));
        if (exit_here) {
            // Keys / values of the early-exit layers for these rows.  Those of the first exit layer depend on H^N
            // only; with several exit layers, layer e sees the output of layer e - 1, so all but the last run in
            // full on these rows (the target's own rows are set aside meanwhile) and the last one contributes
            // its key / value projection.
            const int qd = f.n_heads * f.head_dim, kvd = f.n_kv_heads * f.head_dim, E = c->E;
            if (E > 1) CU(c, cudaMemcpyAsync(c->x_save, c->x, (size_t)M * d * 4, cudaMemcpyDeviceToDevice, s));
            for (int e = 0; e + 1 < E; e++) run_layer(c, c->layers[L + e], L + e, M, pos0, c->layers[L + e + 1].g_attn, nullptr);
            const char *wkv = c->layers[L + E - 1].wqkv + (size_t)qd * d * c->es;
            PartView pv = run_proj(c, wkv, &c->m_exit_kv, P_EXIT_KV, X_NORM, M, 2 * kvd, d);
            if (c->batch_cur) {   // every sequence's rows go to its own positions and pages
                const BatchRows &br = *c->batch_cur;
                for (int b = 0; b < br.n_seq; b++) {
                    KvGeom g = kv_geom(c, L + E - 1);
                    g.page_table += br.table_off[b];
                    launch_qkv_post(s, f.dtype, pv, norm_scale(c), br.rows[b], br.pos0[b], f.n_heads, g, c->rope, nullptr, true, c->err, 0,
                                    nullptr, br.row0[b]);
                }
                c->launches += br.n_seq - 1;
            } else {
                launch_qkv_post(s, f.dtype, pv, norm_scale(c), M, pos0, f.n_heads, kv_geom(c, L + E - 1), c->rope, nullptr, true, c->err, 0,
                                c->tree_cur);
            }
            if (E > 1) CU(c, cudaMemcpyAsync(c->x, c->x_save, (size_t)M * d * 4, cudaMemcpyDeviceToDevice, s));
            const float *g_next = l + 1 < L ? c->layers[l + 1].g_attn : c->g_final;
            run_resid(c, nullptr, g_next, nullptr, M);
            c->launches += 1;
        }
    }
    if (want_logits) {
        PartView pv = run_proj(c, c->lm_head, &c->m_lm_head, P_HEAD, X_NORM, M, f.vocab, d);
        launch_reduce_partials(s, pv, norm_scale(c), c->logits_p, M, f.vocab);
        c->launches += 1;
    }
    return check_launch(c);
}

// Prompt pass (wide path): the target model on Mtot <= wide_rows prompt rows at positions
// p0.., no logits.  Projections run on the wide tensor-core kernel (weights cross HBM once
// per pass); the rows' keys / values are appended first, then the rows attend to the cache 128 at a
// time (causal tensor-core attention); the exit layer's keys / values follow layer N.
int run_prompt_pass(eesd_ctx *c, const int32_t *prompt_host, int p0, int Mtot) {
    const eesd_config &f = c->cfg;
    cudaStream_t s = c->stream;
    const int L = f.n_layers, d = f.d_model, F = f.ffn_dim, H = f.n_heads;
    const int qd = H * f.head_dim, kvd = f.n_kv_heads * f.head_dim;
    CU(c, cudaMemcpyAsync(c->wtok, prompt_host + p0, (size_t)Mtot * 4, cudaMemcpyHostToDevice, s));
    RowScale rs = norm_scale(c);
    rs.ssq = c->wssq;
    auto proj = [&](const CUtensorMap &mW, int which, int R, int K) {
        // narrow results (O, down, exit keys/values) leave SMs idle in the last wave: split their k range
        const int S = gemm_wide_splits(R, K, Mtot, c->n_sm, (int)(c->wout_floats / ((size_t)c->wide_rows * R)));
        launch_gemm_wide(s, mW, c->m_wx[which], c->wout, R, K, Mtot, c->n_sm, true, S, c->err, c->wait_polls);
        c->launches++;
        PartView pv = {};
        pv.base = c->wout; pv.mode = 0; pv.S = S; pv.R = R; pv.split_stride = (size_t)Mtot * R;
        return pv;
    };
    auto resid = [&](const PartView *pv, const float *g) {
        launch_resid(s, c->wx, pv, g, nullptr, c->wxs[X_NORM], nullptr, c->wssq, Mtot, d);
        c->launches++;
    };
    launch_embed_resid(s, f.dtype, c->wtok, 1, c->embed, f.vocab, c->wx, c->layers[0].g_attn, nullptr, c->wxs[X_NORM], nullptr, c->wssq, Mtot, d, c->err);
    c->launches++;
    auto layer = [&](const LayerW &w, int slot, const float *g_after) {
        PartView pv = proj(w.m_qkv, X_NORM, qd + 2 * kvd, d);
        // keys / values of all rows into the cache first, then the causal attention of all rows
        launch_kv_append_wide(s, pv, rs, Mtot, p0, kv_geom(c, slot), c->rope, qd, c->err);
        launch_attention_prompt(s, pv, rs, c->rope, kv_geom(c, slot), c->wxs[X_ATTN], Mtot, p0, H, c->err, c->wait_polls);
        c->launches += 2;
        pv = proj(w.m_o, X_ATTN, d, qd);
        resid(&pv, w.g_ffn);
        pv = proj(w.m_gu, X_NORM, 2 * F, d);
        launch_swiglu(s, pv, rs, nullptr, c->wxs[X_FFN], Mtot, F);
        c->launches++;
        pv = proj(w.m_d, X_FFN, d, F);
        resid(&pv, g_after);
    };
    for (int l = 0; l < L; l++) {
        const bool exit_here = (l == f.n_early - 1);
        layer(c->layers[l], l, exit_here ? c->layers[L].g_attn : (l + 1 < L ? c->layers[l + 1].g_attn : c->g_final));
        if (exit_here) {   // the exit layers' keys / values of the prompt rows (as in a verification pass)
            const int E = c->E;
            if (E > 1) CU(c, cudaMemcpyAsync(c->wx_save, c->wx, (size_t)Mtot * d * 4, cudaMemcpyDeviceToDevice, s));
            for (int e = 0; e + 1 < E; e++) layer(c->layers[L + e], L + e, c->layers[L + e + 1].g_attn);
            PartView pv = proj(c->m_exit_kv, X_NORM, 2 * kvd, d);
            launch_kv_append_wide(s, pv, rs, Mtot, p0, kv_geom(c, L + E - 1), c->rope, 0, c->err);
            c->launches++;
            if (E > 1) CU(c, cudaMemcpyAsync(c->wx, c->wx_save, (size_t)Mtot * d * 4, cudaMemcpyDeviceToDevice, s));
            resid(nullptr, l + 1 < L ? c->layers[l + 1].g_attn : c->g_final);
        }
    }
    return check_launch(c);
}

// Draft model (Eq. 1) on one row: token ints[kRoundTok + i] at position pos, logits into
// logits_q[i], chosen token into ints[kRoundTok + i + 1].
int run_draft_step(eesd_ctx *c, int i, int pos, const float *d_u) {
    const eesd_config &f = c->cfg;
    cudaStream_t s = c->stream;
    const int L = f.n_layers, d = f.d_model, N = f.n_early;
    run_embed(c, c->ints + kRoundTok + i, 1, 1, cap_slot(c, 0));
    for (int l = 0; l < N; l++) {
        const float *g_after = l + 1 < N ? c->layers[l + 1].g_attn : c->layers[L].g_attn;
        run_layer(c, c->layers[l], l, 1, pos, g_after, cap_slot(c, l + 1));
    }
    for (int e = 0; e < c->E; e++)   // the early-exit layer(s), each on its own cache slot
        run_layer(c, c->layers[L + e], L + e, 1, pos, e + 1 < c->E ? c->layers[L + e + 1].g_attn : c->g_exit,
                  e + 1 < c->E ? nullptr : cap_slot(c, L + 1));
    float *lq = c->logits_q + (size_t)i * f.vocab;
    PartView pv = run_proj(c, c->exit_head, &c->m_exit_head, P_HEAD, X_NORM, 1, f.vocab, d);
    launch_reduce_partials(s, pv, norm_scale(c), lq, 1, f.vocab);
    if (tree_on(c))   // greedy token and, in the same kernel, the next-best candidates: leaves of depth i + 1
        launch_next_best(s, lq, f.vocab, f.tree_width, c->ints + kRoundTok + i + 1, c->ints + kLeafTok + i * (f.tree_width - 1));
    else
        launch_sample_rows(s, lq, d_u, 1, f.vocab, f.temperature, c->ints + kRoundTok + i + 1);
    c->launches += 3;
    return check_launch(c);
}

// rows of a tree verification pass after K draft steps: chain rows 0..K, then the leaves by depth
int tree_pass_rows(const eesd_ctx *c, int K) { return 1 + K * c->cfg.tree_width; }

int set_device_ints(eesd_ctx *c, int slot, const int32_t *vals, int n) {
    IntList16 l;
    for (int i = 0; i < n; i++) l.v[i] = vals[i];
    launch_set_ints(c->stream, c->ints + slot, l, n);
    c->launches++;
    return check_launch(c);
}

int read_error_word(eesd_ctx *c) {
    // h_result[2] was copied from the device error word together with the round result
    return c->h_result[2] ? EESD_ERR_DEVICE : EESD_OK;
}

// Controller decisions and posterior updates are pure host functions of the C ABI
// (eesd_ts_decide, eesd_ts_posterior_update, eesd_cali_decide below); the context only keeps the state.
int ts_continue(eesd_ctx *c, const eesd_uniforms *u, int64_t *cursor) {
    if (!u || !u->u_ctrl) return EESD_ERR_RNG;
    return eesd_ts_decide(c->alpha, c->beta, u->u_ctrl, u->n_ctrl, cursor, nullptr);
}

void ts_update(eesd_ctx *c, int q_v, int n_draft) {
    const int64_t a0 = c->alpha, b0 = c->beta;
    eesd_ts_posterior_update(&c->alpha, &c->beta, q_v, n_draft, c->cfg.ts_update_rule);
    const int64_t r = c->alpha - a0, n = r + (c->beta - b0);
    // TS with calibration: observed mean of chi over the verified drafts (theta_hat_0 counts as one)
    c->theta_hat = (c->theta_hat * (double)(c->n_trials + 1) + (double)r) / (double)(c->n_trials + n + 1);
    c->n_trials += n;
    c->n_verify++;
}

bool cali_on(const eesd_ctx *c) { return c->cfg.controller == EESD_CTRL_CALI_TS; }

// H^(T): row `row` (or the row whose index sits in device memory) of a residual-stream matrix
void save_target_state(eesd_ctx *c, const float *x, int row, const int32_t *row_dev) {
    launch_copy_row(c->stream, x, row, row_dev, c->hT, c->use_tc ? c->xs[X_CALI] : nullptr, c->cfg.d_model);
    c->launches++;
}

// theta_M of Eq. 5 for draft step `step` (1-based) of the round; the draft step's residual
// stream after the early-exit layer is row 0 of x
int run_cali_predict(eesd_ctx *c, int step) {
    const int d = c->cfg.d_model, wi = (step < 10 ? step : 10) - 1;
    const char *W = c->cali_w + (size_t)wi * d * d * c->es;
    PartView pv = run_proj(c, W, &c->m_cali[wi], P_CALI, X_CALI, 1, d, d);
    launch_cali_theta(c->stream, pv, c->cali_wp, c->x, d, c->theta_dev);
    c->launches++;
    return check_launch(c);
}

// posterior of Eq. 6-7, then the draw of Algorithm 3
int cali_continue(eesd_ctx *c, float theta_m, const eesd_uniforms *u, int64_t *cursor) {
    if (!u || !u->u_ctrl) return EESD_ERR_RNG;
    double mu, var;
    eesd_cali_posterior(theta_m, c->theta_hat, c->n_verify, c->cfg.cali_sigma_m, c->cfg.cali_sigma_s, &mu, &var);
    return eesd_cali_decide(mu, var, u->u_ctrl, u->n_ctrl, cursor, nullptr);
}

void reset_sequence(eesd_ctx *c) {
    trim_pages(c, 0);
    c->tokens.clear();
    c->prefilled = false;
    c->round_k = 0;
    c->alpha = c->cfg.alpha0;
    c->beta = c->cfg.beta0;
    c->theta_hat = c->cfg.cali_theta0;
    c->n_verify = 0;
    c->n_trials = 0;
}

int prefill_impl(eesd_ctx *c, const int32_t *prompt, int n_prompt) {
    if (!prompt || n_prompt < 1) return EESD_ERR_BADARG;
    if (n_prompt >= c->cfg.max_ctx) return EESD_ERR_CTX_FULL;
    for (int i = 0; i < n_prompt; i++)
        if (prompt[i] < 0 || prompt[i] >= c->cfg.vocab) return EESD_ERR_BADARG;
    reset_sequence(c);
    int st = ensure_pages(c, n_prompt);
    if (st) return st;
    int p = 0;
    // long prompts: wide passes (hidden-state capture holds 16 rows per layer, so it keeps the row-chunk path)
    while (c->wide_rows > 0 && !c->capture && n_prompt - 1 - p > EESD_MAX_ROWS) {
        int M = n_prompt - 1 - p;
        if (M > c->wide_rows) M = c->wide_rows;
        st = run_prompt_pass(c, prompt, p, M);
        if (st) return st;
        p += M;
        if (cali_on(c) && p == n_prompt - 1) save_target_state(c, c->wx, M - 1, nullptr);
    }
    for (; p < n_prompt - 1; p += EESD_MAX_ROWS) {
        int M = n_prompt - 1 - p;
        if (M > EESD_MAX_ROWS) M = EESD_MAX_ROWS;
        st = set_device_ints(c, kRowTok, prompt + p, M);
        if (st) return st;
        st = run_target(c, c->ints + kRowTok, M, p, false);
        if (st) return st;
        if (cali_on(c) && p + M == n_prompt - 1) save_target_state(c, c->x, M - 1, nullptr);
    }
    if (cali_on(c) && n_prompt == 1) {   // the target has processed nothing yet: H^(T) = 0
        CU(c, cudaMemsetAsync(c->hT, 0, (size_t)c->cfg.d_model * 4, c->stream));
        if (c->use_tc) CU(c, cudaMemsetAsync(c->xs[X_CALI], 0, (size_t)2 * EESD_MAX_ROWS * c->cfg.d_model * 2, c->stream));
    }
    st = set_device_ints(c, kRoundTok, prompt + n_prompt - 1, 1);
    if (st) return st;
    c->tokens.assign(prompt, prompt + n_prompt);
    c->prefilled = true;
    return EESD_OK;
}

// draft steps round_k .. round_k + k - 1 of the current round; d_u: device uniforms, one per step
int draft_impl(eesd_ctx *c, int k, const float *d_u, int u_stride) {
    const int T = (int)c->tokens.size();
    if (c->round_k + k > c->cfg.k_cap) return EESD_ERR_CTX_FULL;
    if (T + c->round_k + k > c->cfg.max_ctx - 1) return EESD_ERR_CTX_FULL;
    if (tree_on(c) && T - 1 + tree_pass_rows(c, c->round_k + k) > c->cfg.max_ctx) return EESD_ERR_CTX_FULL;
    int st = ensure_pages(c, T + c->round_k + k);
    if (st) return st;
    for (int j = 0; j < k; j++) {
        const int i = c->round_k;
        st = run_draft_step(c, i, T - 1 + i, d_u ? d_u + (size_t)j * u_stride : nullptr);
        if (st) return st;
        c->round_k++;
    }
    return EESD_OK;
}

// Tree verification (greedy): one pass over the chain x_0..x_K and the width - 1 next-best
// candidates of every depth as leaves; leaf j of depth i is row K + 1 + (i - 1)(width - 1) + j,
// rotated as position T - 1 + i, and sees the cache, chain rows 0..i-1 and itself.  The target's
// top-1 token of every row decides the walk; a kept leaf's keys / values then move from the
// position of its row to the position of its depth in every layer and in the exit layer.
int verify_tree_impl(eesd_ctx *c) {
    const eesd_config &f = c->cfg;
    const int T = (int)c->tokens.size(), K = c->round_k, W = f.tree_width, M = tree_pass_rows(c, K);
    if (T - 1 + M > f.max_ctx) return EESD_ERR_CTX_FULL;
    int st = ensure_pages(c, T - 1 + M);
    if (st) return st;
    TreeRows &tr = c->tree_rows;
    tr = chain_rows();
    for (int i = 1; i <= K; i++)
        for (int j = 0; j < W - 1; j++) {
            const int m = K + 1 + (i - 1) * (W - 1) + j;
            tr.depth[m] = (uint8_t)i;
            tr.vis[m] = (uint16_t)(((1u << i) - 1u) | (1u << m));
        }
    launch_tree_rows(c->stream, c->ints + kRoundTok, c->ints + kLeafTok, K, W, c->ints + kRowTok);
    c->tree_cur = &tr;
    st = run_target(c, c->ints + kRowTok, M, T - 1, true);
    c->tree_cur = nullptr;
    if (st) return st;
    CU(c, cudaEventRecord(c->ev[5], c->stream));
    launch_sample_rows(c->stream, c->logits_p, nullptr, M, f.vocab, 0.f, c->ints + kTreeTop);
    launch_tree_walk(c->stream, c->ints + kTreeTop, c->ints + kRoundTok, c->ints + kLeafTok, K, W, c->ints + kResult);
    launch_kv_move(c->stream, f.dtype, kv_geom(c, 0), c->slot_bytes, f.n_layers + c->E, T - 1, c->ints + kResult, c->err);
    CU(c, cudaEventRecord(c->ev[6], c->stream));
    c->launches += 4;
    st = check_launch(c);
    if (st) return st;
    CU(c, cudaMemcpyAsync(c->h_result, c->ints + kResult, 8, cudaMemcpyDeviceToHost, c->stream));
    CU(c, cudaMemcpyAsync(c->h_result + 2, c->err, 4, cudaMemcpyDeviceToHost, c->stream));
    CU(c, cudaMemcpyAsync(c->h_result + 3, c->ints + kResult + 2, 4, cudaMemcpyDeviceToHost, c->stream));
    return EESD_OK;
}

// verify pass + acceptance; leaves (n_accept, next token, error word) in h_result after a sync
int verify_impl(eesd_ctx *c, const float *d_u_acc, const float *d_u_res) {
    const eesd_config &f = c->cfg;
    const int T = (int)c->tokens.size(), K = c->round_k;
    if (tree_on(c)) return verify_tree_impl(c);
    int st = ensure_pages(c, T + K);
    if (st) return st;
    st = run_target(c, c->ints + kRoundTok, K + 1, T - 1, true);
    if (st) return st;
    CU(c, cudaEventRecord(c->ev[5], c->stream));
    launch_accept(c->stream, c->logits_p, c->logits_q, c->ints + kRoundTok + 1, d_u_acc, d_u_res, 1, K, f.vocab,
                  f.temperature, c->accept_scratch, c->ints + kResult, c->ints + kResult + 1, c->ints + kRoundTok);
    CU(c, cudaEventRecord(c->ev[6], c->stream));
    c->launches++;
    if (cali_on(c)) save_target_state(c, c->x, 0, c->ints + kResult);   // the row that gave the next token
    st = check_launch(c);
    if (st) return st;
    CU(c, cudaMemcpyAsync(c->h_result, c->ints + kResult, 8, cudaMemcpyDeviceToHost, c->stream));
    CU(c, cudaMemcpyAsync(c->h_result + 2, c->err, 4, cudaMemcpyDeviceToHost, c->stream));
    return EESD_OK;
}

// host bookkeeping after the round's result has arrived
int finish_round(eesd_ctx *c, const int32_t *draft_tokens_host, int *n_accept, int32_t *next) {
    const int K = c->round_k;
    const int a = c->h_result[0], y = c->h_result[1];
    if (read_error_word(c) || a < 0 || a > K || y < 0 || y >= c->cfg.vocab) {
        snprintf(c->cuda_err, sizeof(c->cuda_err), "device error word 0x%x, round result n_accept=%d next=%d (K=%d)",
                 c->h_result[2], a, y, K);
        return EESD_ERR_DEVICE;
    }
    for (int i = 0; i < a; i++) c->tokens.push_back(draft_tokens_host[i]);
    c->tokens.push_back(y);
    if (tree_on(c) && c->h_result[3] >= 0) c->leaves_kept++;
    c->round_k = 0;
    trim_pages(c, (int)c->tokens.size() - 1);  // rows of rejected tokens are dropped
    if (n_accept) *n_accept = a;
    if (next) *next = y;
    return EESD_OK;
}


// ------------------------------------------------------------------------------------ batch mode
// Several sequences decoded together (an extension; the paper decodes one at a time): the rows of a
// pass are split among the sequences, every sequence has its own pages, positions and tokens, and
// the weights cross HBM once per pass for all of them.  Host state of the sequences that are not
// selected is parked in c->seqs; select_seq swaps one in, so that the single-sequence code
// (prefill, page bookkeeping) works on it unchanged.
bool batch_on(const eesd_ctx *c) { return !c->seqs.empty(); }

void select_seq(eesd_ctx *c, int b) {
    std::swap(c->tokens, c->seqs[b].tokens);
    std::swap(c->page_of, c->seqs[b].page_of);
    std::swap(c->prefilled, c->seqs[b].prefilled);
    c->page_table = c->page_table0 + (size_t)b * table_len(&c->cfg);
}
void park_seq(eesd_ctx *c, int b) {
    select_seq(c, b);   // the swap is its own inverse
    c->page_table = c->page_table0;
}

// rows of a pass: sequence act[i] gets `rows` rows starting `back` positions before the end of its
// context (its tokens.size() counts the pending token, which takes position size - 1)
void batch_geometry(eesd_ctx *c, const int *act, int n_act, int rows, int step) {
    BatchRows &br = c->batch_rows;
    br.n_seq = n_act;
    for (int i = 0; i < n_act; i++) {
        br.row0[i] = i * rows;
        br.rows[i] = rows;
        br.pos0[i] = (int)c->seqs[act[i]].tokens.size() - 1 + step;
        br.table_off[i] = (int)((size_t)act[i] * table_len(&c->cfg));
    }
}

// pages for `extra` more rows after the pending token of every active sequence
int batch_ensure_pages(eesd_ctx *c, const int *act, int n_act, int extra) {
    for (int i = 0; i < n_act; i++) {
        select_seq(c, act[i]);
        const int st = ensure_pages(c, (int)c->tokens.size() + extra);
        park_seq(c, act[i]);
        if (st) return st;
    }
    return EESD_OK;
}

// Draft step i of a round of draft length K on the active sequences (one row each): token
// chain[a][i] at position T_a - 1 + i; logits into logits_q[a][i], chosen token into chain[a][i + 1]
// (chain = ints + kRowTok, [n_act][K + 1]).  d_u: one uniform per sequence for this step.
int run_batch_draft_step(eesd_ctx *c, const int *act, int n_act, int i, int K, const float *d_u) {
    const eesd_config &f = c->cfg;
    cudaStream_t s = c->stream;
    const int L = f.n_layers, d = f.d_model, N = f.n_early;
    int32_t *chain = c->ints + kRowTok;
    batch_geometry(c, act, n_act, 1, i);
    c->batch_cur = &c->batch_rows;
    run_embed(c, chain + i, K + 1, n_act, nullptr);
    for (int l = 0; l < N; l++)
        run_layer(c, c->layers[l], l, n_act, 0, l + 1 < N ? c->layers[l + 1].g_attn : c->layers[L].g_attn, nullptr);
    for (int e = 0; e < c->E; e++)
        run_layer(c, c->layers[L + e], L + e, n_act, 0, e + 1 < c->E ? c->layers[L + e + 1].g_attn : c->g_exit, nullptr);
    c->batch_cur = nullptr;
    float *lq = c->logits_q + (size_t)i * f.vocab;   // row a of this step is row a * K + i of [n_act][K][V]
    PartView pv = run_proj(c, c->exit_head, &c->m_exit_head, P_HEAD, X_NORM, n_act, f.vocab, d);
    launch_reduce_partials(s, pv, norm_scale(c), lq, n_act, f.vocab, (size_t)K * f.vocab);
    launch_sample_rows(s, lq, d_u, n_act, f.vocab, f.temperature, chain + i + 1, (size_t)K * f.vocab, K + 1);
    c->launches += 3;
    return check_launch(c);
}

// One round of the active sequences: K draft steps, one verification pass of K + 1 rows per
// sequence, the acceptance step for all of them; the result (n_accept and next token per
// sequence, the chains, the error word) is on its way to h_result when this returns.
// h_result: [2] error word, [8..23] the chains, [32..39] n_accept, [40..47] next tokens.
int batch_round(eesd_ctx *c, const int *act, int n_act, int K, const eesd_uniforms *u) {
    const eesd_config &f = c->cfg;
    const bool greedy = f.temperature == 0.f;
    int32_t *chain = c->ints + kRowTok;
    int st = batch_ensure_pages(c, act, n_act, K);
    if (st) return st;
    IntList16 first;   // the pending tokens: chain[a][0]
    for (int i = 0; i < 16; i++) first.v[i] = 0;
    for (int a = 0; a < n_act; a++) first.v[a * (K + 1)] = c->seqs[act[a]].tokens.back();
    launch_set_ints(c->stream, chain, first, n_act * (K + 1));
    c->launches++;
    float *d_ud = c->u_stage, *d_ua = c->u_stage + 16, *d_ur = c->u_stage + 32;
    if (!greedy) {   // this round's uniforms: draft [K][n_act], accept [n_act][K], resample [n_act]
        float h[40];
        for (int a = 0; a < n_act; a++) {
            const int T = (int)c->seqs[act[a]].tokens.size();
            for (int i = 0; i < K; i++) {
                h[i * n_act + a] = u[act[a]].u_draft[T + i];
                h[16 + a * K + i] = u[act[a]].u_accept[T + i];
            }
            h[32 + a] = u[act[a]].u_resample[T];
        }
        CU(c, cudaMemcpyAsync(c->u_stage, h, sizeof(h), cudaMemcpyHostToDevice, c->stream));
    }
    CU(c, cudaEventRecord(c->ev[2], c->stream));
    for (int i = 0; i < K; i++) {
        st = run_batch_draft_step(c, act, n_act, i, K, greedy ? nullptr : d_ud + i * n_act);
        if (st) return st;
    }
    CU(c, cudaEventRecord(c->ev[3], c->stream));
    batch_geometry(c, act, n_act, K + 1, 0);
    c->batch_cur = &c->batch_rows;
    st = run_target(c, chain, n_act * (K + 1), 0, true);
    c->batch_cur = nullptr;
    if (st) return st;
    CU(c, cudaEventRecord(c->ev[5], c->stream));
    launch_accept(c->stream, c->logits_p, c->logits_q, chain + 1, d_ua, d_ur, n_act, K, f.vocab, f.temperature, c->accept_scratch,
                  c->ints + kResult, c->ints + kResult + kMaxSeqs, nullptr, K + 1);
    CU(c, cudaEventRecord(c->ev[6], c->stream));
    c->launches++;
    st = check_launch(c);
    if (st) return st;
    CU(c, cudaMemcpyAsync(c->h_result + 32, c->ints + kResult, 2 * kMaxSeqs * 4, cudaMemcpyDeviceToHost, c->stream));
    CU(c, cudaMemcpyAsync(c->h_result + 8, chain, 16 * 4, cudaMemcpyDeviceToHost, c->stream));
    CU(c, cudaMemcpyAsync(c->h_result + 2, c->err, 4, cudaMemcpyDeviceToHost, c->stream));
    CU(c, cudaEventRecord(c->ev[4], c->stream));
    return EESD_OK;
}

}  // namespace

// =====================================================================================  C ABI
extern "C" {

const char *eesd_strerror(int status) {
    switch (status) {
        case EESD_OK: return "ok";
        case EESD_ERR_BADARG: return "bad argument";
        case EESD_ERR_NOMEM: return "caller-provided buffer too small";
        case EESD_ERR_CUDA: return "CUDA runtime error";
        case EESD_ERR_STATE: return "call not valid in the current state";
        case EESD_ERR_CTX_FULL: return "context, round or KV page pool full";
        case EESD_ERR_RNG: return "uniform stream missing or exhausted";
        case EESD_ERR_DEVICE: return "device-side error word set";
        case EESD_ERR_UNSUPPORTED: return "unsupported shape";
        default: return "unknown status";
    }
}

const char *eesd_last_cuda_error(const eesd_ctx *ctx) { return ctx ? ctx->cuda_err : ""; }

int eesd_weight_layout(const eesd_config *c, eesd_layout *out) {
    int st = check_config(c);
    if (st) return st;
    if (!out) return EESD_ERR_BADARG;
    const size_t es = c->dtype == EESD_F32 ? 4 : 2;
    const size_t d = c->d_model, F = c->ffn_dim, V = c->vocab;
    const size_t qd = (size_t)c->n_heads * c->head_dim, kvd = (size_t)c->n_kv_heads * c->head_dim;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    out->off_g_attn = take(d * 4);
    out->off_wqkv = take((qd + 2 * kvd) * d * es);
    out->off_wo = take(d * qd * es);
    out->off_g_ffn = take(d * 4);
    out->off_wgu = take(2 * F * d * es);
    out->off_wd = take(d * F * es);
    out->layer_stride = o;
    o = 0;
    out->embed = take(V * d * es);
    out->layer0 = o;
    o += out->layer_stride * (size_t)c->n_layers;
    out->final_norm = take(d * 4);
    out->lm_head = take(V * d * es);
    out->exit_layer = o;
    o += out->layer_stride * (size_t)n_exit(c);
    out->exit_norm = take(d * 4);
    out->exit_head = c->tie_exit_head ? out->lm_head : take(V * d * es);
    out->cali_w = out->cali_wp = 0;
    if (c->controller == EESD_CTRL_CALI_TS) {
        out->cali_w = take(10 * d * d * es);
        out->cali_wp = take(4 * d * 4);
    }
    out->total_bytes = o;
    out->tiled = tc_shapes_ok(c) ? 1 : 0;
    return EESD_OK;
}

int eesd_required_bytes(const eesd_config *c, eesd_sizes *out) {
    eesd_layout lay;
    int st = eesd_weight_layout(c, &lay);
    if (st) return st;
    if (!out) return EESD_ERR_BADARG;
    const size_t es = c->dtype == EESD_F32 ? 4 : 2;
    out->weights_bytes = lay.total_bytes;
    out->kv_page_bytes = (size_t)(c->n_layers + n_exit(c)) * 2 * c->n_kv_heads * c->page_tokens * c->head_dim * es;
    out->min_pages = (c->max_ctx + c->page_tokens - 1) / c->page_tokens;
    out->workspace_bytes = carve(c).total;
    return EESD_OK;
}

int eesd_init(const eesd_config *cfg, const eesd_buffers *b, void *cuda_stream, eesd_ctx **out) {
    eesd_layout lay;
    eesd_sizes sz;
    int st = eesd_required_bytes(cfg, &sz);
    if (st) return st;
    eesd_weight_layout(cfg, &lay);
    if (!b || !out || !b->weights || !b->kv_pool || !b->workspace) return EESD_ERR_BADARG;
    if (b->weights_bytes < sz.weights_bytes || b->workspace_bytes < sz.workspace_bytes) return EESD_ERR_NOMEM;
    const int64_t pages = (int64_t)(b->kv_bytes / sz.kv_page_bytes);
    if (pages < sz.min_pages) return EESD_ERR_NOMEM;
    eesd_ctx *c = new (std::nothrow) eesd_ctx();
    if (!c) return EESD_ERR_NOMEM;
    c->cfg = *cfg;
    c->buf = *b;
    c->lay = lay;
    c->stream = (cudaStream_t)cuda_stream;
    c->es = cfg->dtype == EESD_F32 ? 4 : 2;
    c->cuda_err[0] = 0;
    c->capture = nullptr;
    c->launches = 0;
    c->tree_cur = nullptr;
    c->leaves_kept = 0;
    c->wait_polls = kDefaultWaitPolls;
    c->n_pages_total = pages > 0x7fffffff ? 0x7fffffff : pages;
    c->slot_bytes = (size_t)c->n_pages_total * 2 * cfg->n_kv_heads * cfg->page_tokens * cfg->head_dim * c->es;
    Workspace w = carve(cfg);
    char *ws = (char *)b->workspace;
    c->x = (float *)(ws + w.x); c->x_save = (float *)(ws + w.x_save); c->xn = (float *)(ws + w.xn); c->attn = (float *)(ws + w.attn);
    c->h = (float *)(ws + w.h); c->part = (float *)(ws + w.part); c->apart = (float *)(ws + w.apart);
    c->logits_p = (float *)(ws + w.logits_p); c->logits_q = (float *)(ws + w.logits_q);
    c->rope = (float2 *)(ws + w.rope); c->page_table = c->page_table0 = (int32_t *)(ws + w.page_table);
    c->batch_cur = nullptr;
    c->ints = (int32_t *)(ws + w.ints); c->u_dev = (float *)(ws + w.u_dev); c->u_stage = (float *)(ws + w.u_stage);
    c->err = (int *)(ws + w.err); c->accept_scratch = ws + w.accept;
    c->ssq = (float *)(ws + w.ssq); c->tickets = (unsigned int *)(ws + w.tickets);
    for (int i = 0; i < 4; i++) c->xs[i] = nullptr;
    c->hT = (float *)(ws + w.hT); c->theta_dev = (float *)(ws + w.theta);
    c->cali_w = nullptr; c->cali_wp = nullptr;
    c->n_sm = 1;
    {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&c->n_sm, cudaDevAttrMultiProcessorCount, dev);
        if (c->n_sm > kMaxSm) c->n_sm = kMaxSm;
    }
    const int qd_ = cfg->n_heads * cfg->head_dim, kvd_ = cfg->n_kv_heads * cfg->head_dim;
    c->use_tc = tc_shapes_ok(cfg) && tc_init() == 0;
    if (lay.tiled && !c->use_tc) {   // tile-major weights are only read by the tensor-core kernels
        delete c;
        return EESD_ERR_UNSUPPORTED;
    }
    c->wide_rows = c->use_tc ? prefill_rows(cfg) : 0;
    const char *wb = (const char *)b->weights;
    c->E = n_exit(cfg);
    c->layers.resize(cfg->n_layers + c->E);
    for (int l = 0; l < cfg->n_layers + c->E; l++) {
        const char *base = wb + (l < cfg->n_layers ? lay.layer0 + (size_t)l * lay.layer_stride
                                                    : lay.exit_layer + (size_t)(l - cfg->n_layers) * lay.layer_stride);
        LayerW &lw = c->layers[l];
        lw.g_attn = (const float *)(base + lay.off_g_attn); lw.wqkv = base + lay.off_wqkv; lw.wo = base + lay.off_wo;
        lw.g_ffn = (const float *)(base + lay.off_g_ffn); lw.wgu = base + lay.off_wgu; lw.wd = base + lay.off_wd;
    }
    c->embed = wb + lay.embed; c->lm_head = wb + lay.lm_head; c->exit_head = wb + lay.exit_head;
    if (cfg->controller == EESD_CTRL_CALI_TS) { c->cali_w = wb + lay.cali_w; c->cali_wp = (const float *)(wb + lay.cali_wp); }
    if (c->use_tc) {
        const int d = cfg->d_model, F = cfg->ffn_dim, R2 = 2 * EESD_MAX_ROWS;
        bool ok = true;
        for (int i = 0; i < 3; i++) c->xs[i] = ws + w.xs[i];
        c->xs[X_CALI] = ws + w.xs_cali;
        if (c->cali_w && tc_shape_ok(d, d)) {
            ok = ok && tc_make_map(&c->m_x[X_CALI], c->xs[X_CALI], R2, d, R2);
            for (int i = 0; i < 10; i++) ok = ok && tc_make_map(&c->m_cali[i], c->cali_w + (size_t)i * d * d * 2, d, d, 128, true);
        }
        ok = ok && tc_make_map(&c->m_x[X_NORM], c->xs[X_NORM], R2, d, R2);
        ok = ok && tc_make_map(&c->m_x[X_ATTN], c->xs[X_ATTN], R2, qd_, R2);
        ok = ok && tc_make_map(&c->m_x[X_FFN], c->xs[X_FFN], R2, F, R2);
        for (auto &lw : c->layers) {
            ok = ok && tc_make_map(&lw.m_qkv, lw.wqkv, qd_ + 2 * kvd_, d, 128, true);
            ok = ok && tc_make_map(&lw.m_o, lw.wo, d, qd_, 128, true);
            ok = ok && tc_make_map(&lw.m_gu, lw.wgu, 2 * F, d, 128, true);
            ok = ok && tc_make_map(&lw.m_d, lw.wd, d, F, 128, true);
        }
        ok = ok && tc_make_map(&c->m_exit_kv, c->layers[cfg->n_layers + c->E - 1].wqkv + (size_t)qd_ * d * 2, 2 * kvd_, d, 128, true);
        ok = ok && tc_make_map(&c->m_lm_head, c->lm_head, cfg->vocab, d, 128, true);
        ok = ok && tc_make_map(&c->m_exit_head, c->exit_head, cfg->vocab, d, 128, true);
        if (c->wide_rows) {
            c->wx = (float *)(ws + w.wx); c->wx_save = (float *)(ws + w.wx_save); c->wout = (float *)(ws + w.wout); c->wout_floats = w.wout_floats; c->wssq = (float *)(ws + w.wssq);
            c->wtok = (int32_t *)(ws + w.wtok);
            const int ks[3] = {d, qd_, F};
            for (int i = 0; i < 3; i++) {
                c->wxs[i] = ws + w.wxs[i];
                ok = ok && tc_make_map_rows(&c->m_wx[i], c->wxs[i], ks[i], c->wide_rows / EESD_MAX_ROWS);
            }
        }
        // work split of every projection shape
        const int shapes[P_COUNT][2] = {{qd_ + 2 * kvd_, d}, {d, qd_}, {2 * F, d}, {d, F}, {2 * kvd_, d}, {cfg->vocab, d}, {d, d}};
        for (int i = 0; i < P_COUNT; i++) c->plan[i] = tc_plan(shapes[i][0], shapes[i][1], kCtasPerSm * c->n_sm);
        if (!ok) {
            delete c;
            return EESD_ERR_CUDA;
        }
    }
    c->g_final = (const float *)(wb + lay.final_norm); c->g_exit = (const float *)(wb + lay.exit_norm);
    // free list in descending order: the first pages handed out are the highest, so logical
    // and physical page numbers differ and the page table is really exercised
    for (int64_t p = 0; p < c->n_pages_total; p++) c->free_pages.push_back((int32_t)p);
    reset_sequence(c);
    c->h_result = nullptr;
    for (auto &e : c->ev) e = nullptr;
    cudaError_t e = cudaHostAlloc((void **)&c->h_result, 256, cudaHostAllocDefault);
    for (int i = 0; i < 7 && e == cudaSuccess; i++) e = cudaEventCreate(&c->ev[i]);
    if (e != cudaSuccess) {
        eesd_destroy(c);
        return EESD_ERR_CUDA;
    }
    memset(c->h_result, 0, 256);
    cudaMemsetAsync(c->err, 0, 16, c->stream);
    cudaMemsetAsync(c->tickets, 0, ticket_count(cfg) * 4, c->stream);
    cudaMemsetAsync(c->ints, 0, kIntSlots * 4, c->stream);
    cudaMemsetAsync(c->accept_scratch, 0, accept_scratch_bytes(kMaxSeqs, EESD_MAX_ROWS), c->stream);
    // The tensor-core attention multiplies cached values past the end of a slice by weights that are
    // exactly zero; that is only harmless while every value the pool ever holds is finite, so the pool
    // starts as zeros (afterwards only this library writes it).
    cudaMemsetAsync(b->kv_pool, 0, (size_t)(cfg->n_layers + c->E) * c->slot_bytes, c->stream);
    launch_rope_table(c->stream, c->rope, cfg->max_ctx, cfg->head_dim, cfg->rope_theta);
    c->launches++;
    st = check_launch(c);
    if (st) {
        eesd_destroy(c);
        return st;
    }
    *out = c;
    return EESD_OK;
}

int eesd_destroy(eesd_ctx *c) {
    if (!c) return EESD_OK;
    if (c->h_result) cudaFreeHost(c->h_result);
    for (auto &e : c->ev)
        if (e) cudaEventDestroy(e);
    delete c;
    return EESD_OK;
}

int eesd_reset(eesd_ctx *c) {
    if (!c) return EESD_ERR_BADARG;
    reset_sequence(c);
    return EESD_OK;
}

int eesd_prefill(eesd_ctx *c, const int32_t *prompt, int n_prompt) {
    if (!c) return EESD_ERR_BADARG;
    if (batch_on(c)) return EESD_ERR_STATE;   // the sequences of a batch are fed with eesd_batch_prefill
    int st = prefill_impl(c, prompt, n_prompt);
    if (st) return st;
    CU(c, cudaMemcpyAsync(c->h_result + 2, c->err, 4, cudaMemcpyDeviceToHost, c->stream));
    CU(c, cudaStreamSynchronize(c->stream));
    return read_error_word(c);
}

int eesd_draft(eesd_ctx *c, int k, const float *u_draft, int32_t *out_tokens) {
    if (!c || k < 1) return EESD_ERR_BADARG;
    if (!c->prefilled) return EESD_ERR_STATE;
    if (c->round_k + k > c->cfg.k_cap) return EESD_ERR_CTX_FULL;
    const bool greedy = c->cfg.temperature == 0.f;
    if (!greedy && !u_draft) return EESD_ERR_RNG;
    const int first = c->round_k;
    float *d_u = nullptr;
    if (!greedy) {
        d_u = c->u_stage + first;
        CU(c, cudaMemcpyAsync(d_u, u_draft, (size_t)k * 4, cudaMemcpyHostToDevice, c->stream));
    }
    int st = draft_impl(c, k, d_u, 1);
    if (st) return st;
    if (out_tokens) {
        CU(c, cudaMemcpyAsync(out_tokens, c->ints + kRoundTok + 1 + first, (size_t)k * 4, cudaMemcpyDeviceToHost, c->stream));
        CU(c, cudaStreamSynchronize(c->stream));
    }
    return EESD_OK;
}

int eesd_verify_accept(eesd_ctx *c, const float *u_accept, float u_resample, int *n_accept, int32_t *next_token) {
    if (!c) return EESD_ERR_BADARG;
    if (!c->prefilled || c->round_k < 1) return EESD_ERR_STATE;
    const bool greedy = c->cfg.temperature == 0.f;
    if (!greedy && !u_accept) return EESD_ERR_RNG;
    const int K = c->round_k;
    float *d_acc = c->u_stage + 16, *d_res = c->u_stage + 32;
    if (!greedy) {
        CU(c, cudaMemcpyAsync(d_acc, u_accept, (size_t)K * 4, cudaMemcpyHostToDevice, c->stream));
        CU(c, cudaMemcpyAsync(d_res, &u_resample, 4, cudaMemcpyHostToDevice, c->stream));
    }
    int32_t *drafts = c->h_result + 8;
    int st = verify_impl(c, d_acc, d_res);
    if (st) return st;
    CU(c, cudaMemcpyAsync(drafts, c->ints + kRoundTok + 1, (size_t)K * 4, cudaMemcpyDeviceToHost, c->stream));
    CU(c, cudaStreamSynchronize(c->stream));
    int a = 0;
    st = finish_round(c, drafts, &a, next_token);
    if (st) return st;
    if (n_accept) *n_accept = a;
    ts_update(c, a + 1, K);   // the controllers' posteriors follow the observed rounds in the step API too
    return EESD_OK;
}

// rounds of {draft, verify, accept, posterior update} from the current context until max_new
// tokens exist (Algorithm 1, outer loop)
typedef std::chrono::steady_clock host_clock;
static double ms_since(host_clock::time_point t0) { return std::chrono::duration<double, std::milli>(host_clock::now() - t0).count(); }

static int decode_impl(eesd_ctx *c, int max_new, const int32_t *k_schedule, int n_schedule, const eesd_uniforms *u,
                       int32_t *out, eesd_stats *stats, eesd_round *trace, int trace_cap, int *n_rounds,
                       int64_t launches0, float ms_prefill, host_clock::time_point wall0) {
    const eesd_config &f = c->cfg;
    const bool greedy = f.temperature == 0.f;
    if (!greedy && (!u || !u->u_draft || !u->u_accept || !u->u_resample)) return EESD_ERR_RNG;
    if (f.controller != EESD_CTRL_FIXED_K && (!u || !u->u_ctrl)) return EESD_ERR_RNG;
    const int n0 = (int)c->tokens.size();
    if (n0 + max_new + 1 > f.max_ctx) return EESD_ERR_CTX_FULL;
    // tree verification stores its leaves past the chain: leave room for the shortest round (one draft step)
    if (tree_on(c) && n0 + max_new + f.tree_width > f.max_ctx) return EESD_ERR_CTX_FULL;
    float *d_ud = c->u_dev, *d_ua = c->u_dev + f.max_ctx, *d_ur = c->u_dev + 2 * (size_t)f.max_ctx;
    if (!greedy) {
        CU(c, cudaMemcpyAsync(d_ud, u->u_draft, (size_t)f.max_ctx * 4, cudaMemcpyHostToDevice, c->stream));
        CU(c, cudaMemcpyAsync(d_ua, u->u_accept, (size_t)f.max_ctx * 4, cudaMemcpyHostToDevice, c->stream));
        CU(c, cudaMemcpyAsync(d_ur, u->u_resample, (size_t)f.max_ctx * 4, cudaMemcpyHostToDevice, c->stream));
    }
    eesd_stats sacc;
    memset(&sacc, 0, sizeof(sacc));
    int64_t cursor = 0;
    const int64_t leaves0 = c->leaves_kept;
    int t = 0, rounds = 0, st;
    int32_t *drafts = c->h_result + 8;
    while (t < max_new) {
        const int T = (int)c->tokens.size();
        // draft length of this round: the controller's decisions depend on the posterior only,
        // so they are taken before the round is enqueued (Algorithm 2, draft loop)
        int cap = f.k_cap;
        if (f.max_ctx - 1 - T < cap) cap = f.max_ctx - 1 - T;
        if (tree_on(c) && (f.max_ctx - T) / f.tree_width < cap) cap = (f.max_ctx - T) / f.tree_width;
        if (cap < 1) return EESD_ERR_CTX_FULL;
        int K;
        const host_clock::time_point ctrl0 = host_clock::now();
        // TS with calibration needs the predictor's output after every draft step: such rounds
        // are drafted step by step, with a synchronisation per step (Algorithm 3)
        const bool stepwise = f.controller == EESD_CTRL_CALI_TS && !(k_schedule && rounds < n_schedule);
        if (k_schedule && rounds < n_schedule) K = k_schedule[rounds];
        else if (f.controller == EESD_CTRL_FIXED_K) K = f.fixed_k;
        else if (stepwise) K = 1;
        else {
            K = 1;
            while (K < cap) {
                int chi = ts_continue(c, u, &cursor);
                if (chi < 0) return chi;
                if (!chi) break;
                K++;
            }
        }
        if (K < 1) K = 1;
        if (K > cap) K = cap;
        sacc.ms_sampling += ms_since(ctrl0);   // the controller's draws on the host
        float ms_pred = 0.f;                   // device time of this round's predictor steps (calibrated controller)
        CU(c, cudaEventRecord(c->ev[2], c->stream));
        if (!stepwise) {
            st = draft_impl(c, K, greedy ? nullptr : d_ud + T, 1);
            if (st) return st;
        } else {
            for (K = 0;;) {
                st = draft_impl(c, 1, greedy ? nullptr : d_ud + T + K, 1);
                if (st) return st;
                if (++K >= cap) break;
                CU(c, cudaEventRecord(c->ev[5], c->stream));
                st = run_cali_predict(c, K);
                if (st) return st;
                float *h_theta = (float *)(c->h_result + 32);
                CU(c, cudaMemcpyAsync(h_theta, c->theta_dev, 4, cudaMemcpyDeviceToHost, c->stream));
                CU(c, cudaEventRecord(c->ev[6], c->stream));
                CU(c, cudaStreamSynchronize(c->stream));
                float ms_one = 0.f;
                cudaEventElapsedTime(&ms_one, c->ev[5], c->ev[6]);
                ms_pred += ms_one;
                const host_clock::time_point draw0 = host_clock::now();
                const int chi = cali_continue(c, *h_theta, u, &cursor);
                sacc.ms_sampling += ms_since(draw0);
                if (chi < 0) return chi;
                if (!chi) break;
            }
        }
        CU(c, cudaEventRecord(c->ev[3], c->stream));
        st = verify_impl(c, d_ua + T, d_ur + T);
        if (st) return st;
        CU(c, cudaMemcpyAsync(drafts, c->ints + kRoundTok + 1, (size_t)K * 4, cudaMemcpyDeviceToHost, c->stream));
        CU(c, cudaEventRecord(c->ev[4], c->stream));
        CU(c, cudaStreamSynchronize(c->stream));
        int a;
        int32_t y;
        st = finish_round(c, drafts, &a, &y);
        if (st) return st;
        float ms_d = 0.f, ms_v = 0.f, ms_a = 0.f;
        cudaEventElapsedTime(&ms_d, c->ev[2], c->ev[3]);
        cudaEventElapsedTime(&ms_v, c->ev[3], c->ev[4]);
        cudaEventElapsedTime(&ms_a, c->ev[5], c->ev[6]);   // the acceptance step inside the verification
        sacc.ms_draft += ms_d - ms_pred;
        sacc.ms_verify += ms_v - ms_a;
        sacc.ms_sampling += ms_a + ms_pred;
        sacc.drafted += K;
        sacc.accepted += a < max_new - t ? a : max_new - t;
        ts_update(c, a + 1, K);
        if (trace && rounds < trace_cap) { trace[rounds].k = K; trace[rounds].n_accept = a; trace[rounds].next_token = y; }
        t += a + 1;
        rounds++;
    }
    for (int i = 0; i < max_new; i++) out[i] = c->tokens[n0 + i];
    if (n_rounds) *n_rounds = rounds;
    if (stats) {
        sacc.rounds = rounds;
        sacc.emitted = max_new;
        sacc.ms_prefill = ms_prefill;
        sacc.ms_total = ms_since(wall0);
        sacc.ms_other = sacc.ms_total - (sacc.ms_prefill + sacc.ms_draft + sacc.ms_verify + sacc.ms_sampling);
        sacc.kernel_launches = c->launches - launches0;
        sacc.alpha = c->alpha;
        sacc.beta = c->beta;
        sacc.leaves_kept = c->leaves_kept - leaves0;
        *stats = sacc;
    }
    return EESD_OK;
}

// ---- batch mode: several sequences decoded together (an extension; the paper's batch is 1) ----

int eesd_batch_begin(eesd_ctx *c, int n_seq) {
    if (!c || n_seq < 0 || n_seq > kMaxSeqs) return EESD_ERR_BADARG;
    // trees and the per-sequence stopping rules of the controllers have no batch counterpart here
    if (n_seq > 0 && tree_on(c)) return EESD_ERR_UNSUPPORTED;
    if (batch_on(c)) {   // leave batch mode: give every sequence's pages back
        for (size_t b = 0; b < c->seqs.size(); b++) {
            select_seq(c, (int)b);
            trim_pages(c, 0);
            park_seq(c, (int)b);
        }
        c->seqs.clear();
    }
    reset_sequence(c);
    c->page_table = c->page_table0;
    c->seqs.resize((size_t)n_seq);
    for (auto &q : c->seqs) q.prefilled = false;
    return EESD_OK;
}

int eesd_batch_prefill(eesd_ctx *c, int seq, const int32_t *prompt, int n_prompt) {
    if (!c || !batch_on(c) || seq < 0 || seq >= (int)c->seqs.size()) return EESD_ERR_BADARG;
    select_seq(c, seq);
    int st = prefill_impl(c, prompt, n_prompt);   // (resets the selected sequence first)
    if (!st) {
        cudaError_t e = cudaMemcpyAsync(c->h_result + 2, c->err, 4, cudaMemcpyDeviceToHost, c->stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
        st = e != cudaSuccess ? EESD_ERR_CUDA : read_error_word(c);
    }
    park_seq(c, seq);
    return st;
}

int eesd_batch_context_len(const eesd_ctx *c, int seq, int *n_tokens, int *pages_in_use) {
    if (!c || !batch_on(c) || seq < 0 || seq >= (int)c->seqs.size()) return EESD_ERR_BADARG;
    if (n_tokens) *n_tokens = (int)c->seqs[seq].tokens.size();
    if (pages_in_use) *pages_in_use = (int)c->seqs[seq].page_of.size();
    return EESD_OK;
}

int eesd_batch_verify_only(eesd_ctx *c, const int32_t *tokens, int m) {
    if (!c || !batch_on(c) || !tokens || m < 1) return EESD_ERR_BADARG;
    const int B = (int)c->seqs.size();
    if (B * m > EESD_MAX_ROWS) return EESD_ERR_BADARG;
    int act[kMaxSeqs];
    for (int b = 0; b < B; b++) {
        if (!c->seqs[b].prefilled) return EESD_ERR_STATE;
        if ((int)c->seqs[b].tokens.size() - 1 + m > c->cfg.max_ctx) return EESD_ERR_CTX_FULL;
        act[b] = b;
    }
    int st = batch_ensure_pages(c, act, B, m - 1);
    if (st) return st;
    st = set_device_ints(c, kRowTok, tokens, B * m);
    if (st) return st;
    batch_geometry(c, act, B, m, 0);
    c->batch_cur = &c->batch_rows;
    st = run_target(c, c->ints + kRowTok, B * m, 0, true);
    c->batch_cur = nullptr;
    return st;
}

int eesd_batch_decode(eesd_ctx *c, int max_new, const int32_t *k_schedule, int n_schedule, const eesd_uniforms *u,
                      int32_t *out, eesd_stats *stats, eesd_round *trace, int trace_cap, int *n_rounds) {
    if (!c || !batch_on(c) || !out || max_new < 1) return EESD_ERR_BADARG;
    const eesd_config &f = c->cfg;
    const int B = (int)c->seqs.size();
    const bool greedy = f.temperature == 0.f;
    int n0[kMaxSeqs], got[kMaxSeqs], rounds_of[kMaxSeqs];
    for (int b = 0; b < B; b++) {
        if (!c->seqs[b].prefilled) return EESD_ERR_STATE;
        if (!greedy && (!u || !u[b].u_draft || !u[b].u_accept || !u[b].u_resample)) return EESD_ERR_RNG;
        n0[b] = (int)c->seqs[b].tokens.size();
        if (n0[b] + max_new + 1 > f.max_ctx) return EESD_ERR_CTX_FULL;
        got[b] = 0;
        rounds_of[b] = 0;
    }
    const host_clock::time_point wall0 = host_clock::now();
    const int64_t launches0 = c->launches;
    eesd_stats sacc;
    memset(&sacc, 0, sizeof(sacc));
    int rounds = 0;
    for (;;) {
        int act[kMaxSeqs], n_act = 0;   // sequences that still owe tokens
        for (int b = 0; b < B; b++)
            if (got[b] < max_new) act[n_act++] = b;
        if (!n_act) break;
        // one draft length for the whole round: the schedule's or the configured one, as far as the
        // rows of a pass (n_act * (K + 1) <= 16), the round cap and every sequence's context allow
        int K = (k_schedule && rounds < n_schedule) ? k_schedule[rounds] : f.fixed_k;
        if (K > f.k_cap) K = f.k_cap;
        if (K > EESD_MAX_ROWS / n_act - 1) K = EESD_MAX_ROWS / n_act - 1;
        for (int a = 0; a < n_act; a++) {
            const int room = f.max_ctx - 1 - (int)c->seqs[act[a]].tokens.size();
            if (room < K) K = room;
        }
        if (K < 1) return EESD_ERR_CTX_FULL;
        int st = batch_round(c, act, n_act, K, u);
        if (st) return st;
        CU(c, cudaStreamSynchronize(c->stream));
        if (read_error_word(c)) {
            snprintf(c->cuda_err, sizeof(c->cuda_err), "device error word 0x%x in a batch round", c->h_result[2]);
            return EESD_ERR_DEVICE;
        }
        const int32_t *chain = c->h_result + 8, *n_acc = c->h_result + 32, *next = c->h_result + 32 + kMaxSeqs;
        for (int a = 0; a < n_act; a++) {
            const int b = act[a], acc = n_acc[a], y = next[a];
            if (acc < 0 || acc > K || y < 0 || y >= f.vocab) {
                snprintf(c->cuda_err, sizeof(c->cuda_err), "batch round result n_accept=%d next=%d (K=%d, sequence %d)", acc, y, K, b);
                return EESD_ERR_DEVICE;
            }
            select_seq(c, b);
            for (int i = 0; i < acc; i++) c->tokens.push_back(chain[a * (K + 1) + 1 + i]);
            c->tokens.push_back(y);
            trim_pages(c, (int)c->tokens.size() - 1);   // rows of rejected tokens are dropped
            park_seq(c, b);
            if (trace && rounds_of[b] < trace_cap) {
                eesd_round &r = trace[(size_t)b * trace_cap + rounds_of[b]];
                r.k = K; r.n_accept = acc; r.next_token = y;
            }
            rounds_of[b]++;
            sacc.drafted += K;
            sacc.accepted += acc < max_new - got[b] ? acc : max_new - got[b];
            got[b] += acc + 1;
        }
        float ms_d = 0.f, ms_v = 0.f, ms_a = 0.f;
        cudaEventElapsedTime(&ms_d, c->ev[2], c->ev[3]);
        cudaEventElapsedTime(&ms_v, c->ev[3], c->ev[4]);
        cudaEventElapsedTime(&ms_a, c->ev[5], c->ev[6]);
        sacc.ms_draft += ms_d;
        sacc.ms_verify += ms_v - ms_a;
        sacc.ms_sampling += ms_a;
        rounds++;
    }
    for (int b = 0; b < B; b++) {
        for (int i = 0; i < max_new; i++) out[(size_t)b * max_new + i] = c->seqs[b].tokens[(size_t)n0[b] + i];
        if (n_rounds) n_rounds[b] = rounds_of[b];
    }
    if (stats) {
        sacc.rounds = rounds;
        sacc.emitted = (int64_t)B * max_new;
        sacc.ms_total = ms_since(wall0);
        sacc.ms_other = sacc.ms_total - (sacc.ms_draft + sacc.ms_verify + sacc.ms_sampling);
        sacc.kernel_launches = c->launches - launches0;
        sacc.alpha = c->alpha;
        sacc.beta = c->beta;
        *stats = sacc;
    }
    return EESD_OK;
}

int eesd_decode(eesd_ctx *c, int max_new, const int32_t *k_schedule, int n_schedule, const eesd_uniforms *u,
                int32_t *out, eesd_stats *stats, eesd_round *trace, int trace_cap, int *n_rounds) {
    if (!c || !out || max_new < 1) return EESD_ERR_BADARG;
    if (!c->prefilled || c->round_k != 0) return EESD_ERR_STATE;
    return decode_impl(c, max_new, k_schedule, n_schedule, u, out, stats, trace, trace_cap, n_rounds, c->launches, 0.f, host_clock::now());
}

int eesd_generate(eesd_ctx *c, const int32_t *prompt, int n_prompt, int max_new, const int32_t *k_schedule,
                  int n_schedule, const eesd_uniforms *u, int32_t *out, eesd_stats *stats, eesd_round *trace,
                  int trace_cap, int *n_rounds) {
    if (!c || !out || max_new < 1) return EESD_ERR_BADARG;
    if (batch_on(c)) return EESD_ERR_STATE;
    if (n_prompt + max_new + 1 > c->cfg.max_ctx) return EESD_ERR_CTX_FULL;
    const int64_t launches0 = c->launches;
    const host_clock::time_point wall0 = host_clock::now();
    CU(c, cudaEventRecord(c->ev[0], c->stream));
    int st = prefill_impl(c, prompt, n_prompt);
    if (st) return st;
    CU(c, cudaEventRecord(c->ev[1], c->stream));
    CU(c, cudaEventSynchronize(c->ev[1]));
    float ms_p = 0.f;
    cudaEventElapsedTime(&ms_p, c->ev[0], c->ev[1]);
    return decode_impl(c, max_new, k_schedule, n_schedule, u, out, stats, trace, trace_cap, n_rounds, launches0, ms_p, wall0);
}

// -ln u of a controller uniform; a zero uniform counts as half the grid step, 2^-25
static double minus_log_uniform(float u) { return -log(u > 0.0f ? (double)u : 0x1p-25); }

int eesd_ts_decide(int64_t alpha, int64_t beta, const float *u, int64_t n_u, int64_t *cursor, double *theta_out) {
    if (!u || !cursor || alpha < 1 || beta < 1 || *cursor < 0) return EESD_ERR_BADARG;
    if (*cursor + alpha + beta + 1 > n_u) return EESD_ERR_RNG;
    // Beta(alpha, beta) with integer parameters: Gamma(alpha, 1) / (Gamma(alpha, 1) + Gamma(beta, 1)),
    // each Gamma with an integer shape a sum of that many unit exponentials
    const float *p = u + *cursor;
    double ga = 0.0, gb = 0.0;
    for (int64_t i = 0; i < alpha; i++) ga += minus_log_uniform(p[i]);
    for (int64_t i = 0; i < beta; i++) gb += minus_log_uniform(p[alpha + i]);
    const double theta = ga / (ga + gb);
    const int chi = (double)p[alpha + beta] < theta;
    *cursor += alpha + beta + 1;
    if (theta_out) *theta_out = theta;
    return chi;
}

int eesd_ts_posterior_update(int64_t *alpha, int64_t *beta, int q_v, int n_draft, int rule) {
    if (!alpha || !beta || q_v < 1 || n_draft < 1 || q_v > n_draft + 1) return EESD_ERR_BADARG;
    if (rule != EESD_TS_RULE_PAPER && rule != EESD_TS_RULE_SINGLE_FAILURE) return EESD_ERR_BADARG;
    const int64_t r = q_v - 1;                                             // accepted drafts: successes
    const int64_t tried = rule == EESD_TS_RULE_PAPER ? q_v + 1 : q_v;      // |Q_v| + 1 as printed, or |Q_v|
    const int64_t n = tried < n_draft ? tried : n_draft;                   // never below r, because r <= |Q_d|
    *alpha += r;          // Eq. 3
    *beta += n - r;       // Eq. 4
    return EESD_OK;
}

int eesd_cali_decide(double mu, double variance, const float *u, int64_t n_u, int64_t *cursor, double *theta_out) {
    if (!u || !cursor || !(variance >= 0.0) || *cursor < 0) return EESD_ERR_BADARG;
    if (*cursor + 3 > n_u) return EESD_ERR_RNG;
    const float *p = u + *cursor;
    // Box-Muller: a standard normal from two uniforms
    const double z = sqrt(2.0 * minus_log_uniform(p[0])) * cos(6.283185307179586476925286766559 * (double)p[1]);
    const double theta = mu + sqrt(variance) * z;
    *cursor += 3;
    if (theta_out) *theta_out = theta;
    return (double)p[2] < theta ? 1 : 0;
}

int eesd_cali_posterior(double theta_m, double theta_hat, int64_t n, double sigma_m, double sigma_s, double *mu,
                        double *variance) {
    if (!mu || !variance || !(sigma_m > 0.0) || !(sigma_s > 0.0) || n < 0) return EESD_ERR_BADARG;
    const double sm2 = sigma_m * sigma_m, ss2 = sigma_s * sigma_s, den = (double)n * sm2 + ss2;
    *mu = ss2 / den * theta_m + (double)n * sm2 / den * theta_hat;   // Eq. 6
    *variance = sm2 * ss2 / den;                                      // Eq. 7
    return EESD_OK;
}

int eesd_cali_state(const eesd_ctx *c, double *theta_hat, int64_t *n_verify, int64_t *n_trials) {
    if (!c) return EESD_ERR_BADARG;
    if (theta_hat) *theta_hat = c->theta_hat;
    if (n_verify) *n_verify = c->n_verify;
    if (n_trials) *n_trials = c->n_trials;
    return EESD_OK;
}

int eesd_cali_predict(eesd_ctx *c, float *theta_m) {
    if (!c || !theta_m) return EESD_ERR_BADARG;
    if (!cali_on(c) || !c->prefilled || c->round_k < 1) return EESD_ERR_STATE;
    int st = run_cali_predict(c, c->round_k);
    if (st) return st;
    float *h = (float *)(c->h_result + 32);
    CU(c, cudaMemcpyAsync(h, c->theta_dev, 4, cudaMemcpyDeviceToHost, c->stream));
    CU(c, cudaStreamSynchronize(c->stream));
    *theta_m = *h;
    return EESD_OK;
}

int eesd_set_wait_limit(eesd_ctx *c, uint32_t polls) {
    if (!c) return EESD_ERR_BADARG;
    c->wait_polls = polls == 0xffffffffu ? kDefaultWaitPolls : polls;
    return EESD_OK;
}

int eesd_clear_device_error(eesd_ctx *c) {
    if (!c) return EESD_ERR_BADARG;
    // kernels that gave up may have left the merge counters of the attention kernel half counted
    CU(c, cudaMemsetAsync(c->err, 0, 16, c->stream));
    CU(c, cudaMemsetAsync(c->tickets, 0, ticket_count(&c->cfg) * 4, c->stream));
    CU(c, cudaStreamSynchronize(c->stream));
    c->h_result[2] = 0;
    if (batch_on(c)) return eesd_batch_begin(c, 0);   // a round that failed half way leaves the sequences of a batch inconsistent: forget them all
    reset_sequence(c);
    return EESD_OK;
}

int eesd_attention_plan(int dtype, int ctx_len, int page_tokens, int n_kv_heads, int pairs, int n_sm, int *pages_per_block,
                        int *n_slices) {
    if ((dtype != EESD_F32 && dtype != EESD_BF16) || ctx_len < 1 || n_kv_heads < 1 || pairs < 1 || n_sm < 1 || !pages_per_block || !n_slices)
        return EESD_ERR_BADARG;
    if (page_tokens < 8 || page_tokens > 128 || (page_tokens & (page_tokens - 1))) return EESD_ERR_BADARG;
    if (ctx_len > attention_max_ctx(dtype, page_tokens)) return EESD_ERR_UNSUPPORTED;
    if (dtype == EESD_BF16) {
        const int nc = attention_tc_columns(pairs);
        *n_slices = attention_tc_splits(ctx_len, page_tokens, n_kv_heads, (pairs + nc - 1) / nc, n_sm, kAttnSplits, pages_per_block);
    } else {
        const int rb = pairs <= 8 ? 8 : pairs <= 24 ? 16 : 32;
        *n_slices = attention_splits(ctx_len, page_tokens, n_kv_heads, (pairs + rb - 1) / rb, n_sm, kAttnSplits, pages_per_block);
    }
    return EESD_OK;
}

int eesd_context_len(const eesd_ctx *c, int *n_tokens, int *pages_in_use) {
    if (!c) return EESD_ERR_BADARG;
    if (n_tokens) *n_tokens = (int)c->tokens.size();
    if (pages_in_use) *pages_in_use = (int)c->page_of.size();
    return EESD_OK;
}

int eesd_context_tokens(const eesd_ctx *c, int first, int n, int32_t *out) {
    if (!c || !out || first < 0 || n < 0 || (size_t)first + (size_t)n > c->tokens.size()) return EESD_ERR_BADARG;
    for (int i = 0; i < n; i++) out[i] = c->tokens[(size_t)first + i];
    return EESD_OK;
}

int eesd_posterior(const eesd_ctx *c, int64_t *alpha, int64_t *beta) {
    if (!c) return EESD_ERR_BADARG;
    if (alpha) *alpha = c->alpha;
    if (beta) *beta = c->beta;
    return EESD_OK;
}

int eesd_batch_assume_context(eesd_ctx *c, int seq, int n_ctx, int32_t pending) {
    if (!c || !batch_on(c) || seq < 0 || seq >= (int)c->seqs.size()) return EESD_ERR_BADARG;
    if (n_ctx < 1 || pending < 0 || pending >= c->cfg.vocab) return EESD_ERR_BADARG;
    if (n_ctx >= c->cfg.max_ctx) return EESD_ERR_CTX_FULL;
    select_seq(c, seq);
    trim_pages(c, 0);
    int st = ensure_pages(c, n_ctx);
    if (!st) {
        c->tokens.assign(n_ctx, 0);
        c->tokens[n_ctx - 1] = pending;
        c->prefilled = true;
    }
    park_seq(c, seq);
    return st;
}

int eesd_assume_context(eesd_ctx *c, int n_ctx, int32_t pending) {
    if (!c || n_ctx < 1 || pending < 0 || pending >= c->cfg.vocab) return EESD_ERR_BADARG;
    if (batch_on(c)) return EESD_ERR_STATE;
    if (n_ctx >= c->cfg.max_ctx) return EESD_ERR_CTX_FULL;
    reset_sequence(c);
    int st = ensure_pages(c, n_ctx);
    if (st) return st;
    c->tokens.assign(n_ctx, 0);
    c->tokens[n_ctx - 1] = pending;
    st = set_device_ints(c, kRoundTok, &pending, 1);
    if (st) return st;
    c->prefilled = true;
    return EESD_OK;
}

int eesd_verify_only(eesd_ctx *c, const int32_t *tokens, int M) {
    if (!c || !tokens || M < 1 || M > EESD_MAX_ROWS) return EESD_ERR_BADARG;
    if (!c->prefilled) return EESD_ERR_STATE;
    const int T = (int)c->tokens.size();
    if (T - 1 + M > c->cfg.max_ctx) return EESD_ERR_CTX_FULL;
    int st = ensure_pages(c, T - 1 + M);
    if (st) return st;
    st = set_device_ints(c, kRowTok, tokens, M);
    if (st) return st;
    return run_target(c, c->ints + kRowTok, M, T - 1, true);
}

int eesd_logits(const eesd_ctx *c, int which, const float **device_ptr) {
    if (!c || !device_ptr || (which != 0 && which != 1)) return EESD_ERR_BADARG;
    *device_ptr = which == 0 ? c->logits_p : c->logits_q;
    return EESD_OK;
}

int eesd_capture_hidden(eesd_ctx *c, float *device_buf, size_t bytes) {
    if (!c) return EESD_ERR_BADARG;
    if (device_buf && bytes < (size_t)(c->cfg.n_layers + 2) * EESD_MAX_ROWS * c->cfg.d_model * 4) return EESD_ERR_NOMEM;
    c->capture = device_buf;
    return EESD_OK;
}

int eesd_launch_count(const eesd_ctx *c, int64_t *n) {
    if (!c || !n) return EESD_ERR_BADARG;
    *n = c->launches;
    return EESD_OK;
}

size_t eesd_accept_scratch_bytes(int B, int K) {
    if (B < 1 || K < 1) return 0;
    return accept_scratch_bytes(B, K);
}

int eesd_accept_resample(void *cuda_stream, const float *p_logits, const float *q_logits, const int32_t *tokens,
                         const float *u_accept, const float *u_resample, int B, int K, int V, float temperature,
                         void *scratch, size_t scratch_bytes, int32_t *n_accept, int32_t *next_token) {
    if (!p_logits || !q_logits || !tokens || !scratch || !n_accept || !next_token) return EESD_ERR_BADARG;
    if (B < 1 || K < 1 || V < 1 || temperature < 0.f) return EESD_ERR_BADARG;
    if (temperature != 0.f && (!u_accept || !u_resample)) return EESD_ERR_RNG;
    if ((long long)B * (2 * K + 1) > 0x7fffffffLL) return EESD_ERR_UNSUPPORTED;
    if ((uintptr_t)scratch & 15) return EESD_ERR_BADARG;   // the row statistics are read with 16-byte loads
    const size_t need = accept_scratch_bytes(B, K);
    if (scratch_bytes < need) return EESD_ERR_NOMEM;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (cudaMemsetAsync(scratch, 0, (size_t)B * sizeof(unsigned int), s) != cudaSuccess) return EESD_ERR_CUDA;
    launch_accept(s, p_logits, q_logits, tokens, u_accept, u_resample, B, K, V, temperature, scratch, n_accept,
                  next_token, nullptr);
    return cudaGetLastError() == cudaSuccess ? EESD_OK : EESD_ERR_CUDA;
}

static size_t project_scratch_layout(int R, int K, size_t *off_xs, size_t *off_tab, size_t *off_part) {
    size_t o = 256;  // error word
    *off_xs = o;
    o = align_up(o + (size_t)2 * EESD_MAX_ROWS * K * 2, 256);
    *off_tab = o;
    o = align_up(o + ((size_t)R / 128 + 1) * sizeof(int4), 256);
    *off_part = o;
    size_t floats = (size_t)EESD_MAX_ROWS * R;
    const size_t sk = ((size_t)R / 128 + (size_t)kMaxSm * kCtasPerSm) * EESD_MAX_ROWS * 128;
    if (sk > floats) floats = sk;
    return o + floats * 4;
}

size_t eesd_project_scratch_bytes(int R, int K) {
    if (R < 1 || K < 1) return 0;
    size_t a, b, t;
    return project_scratch_layout(R, K, &a, &t, &b);
}

int eesd_project_rows(void *cuda_stream, int dtype, const float *A, const void *W, float *out, int M, int R, int K,
                      void *scratch, size_t scratch_bytes) {
    if (!A || !W || !out || !scratch) return EESD_ERR_BADARG;
    if (M < 1 || M > EESD_MAX_ROWS || R < 1 || K < 8 || (K % 8)) return EESD_ERR_BADARG;
    if (dtype != EESD_F32 && dtype != EESD_BF16) return EESD_ERR_BADARG;
    size_t off_xs, off_tab, off_part;
    if (scratch_bytes < project_scratch_layout(R, K, &off_xs, &off_tab, &off_part)) return EESD_ERR_NOMEM;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    char *sc = (char *)scratch;
    float *part = (float *)(sc + off_part);
    PartView pv = {};
    pv.base = part;
    pv.R = R;
    if (dtype == EESD_BF16 && tc_shape_ok(R, K) && tc_init() == 0) {
        int dev = 0, n_sm = 1;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
        if (n_sm > kMaxSm) n_sm = kMaxSm;
        CUtensorMap mW, mX;
        if (!tc_make_map(&mW, W, R, K, 128) || !tc_make_map(&mX, sc + off_xs, 2 * EESD_MAX_ROWS, K, 2 * EESD_MAX_ROWS))
            return EESD_ERR_CUDA;
        const StreamK sk = tc_plan(R, K, kCtasPerSm * n_sm);
        if (cudaMemsetAsync(sc, 0, 16, s) != cudaSuccess) return EESD_ERR_CUDA;
        launch_split_rows(s, A, sc + off_xs, M, K);
        pv.mode = 1;
        pv.sk = sk;
        launch_gemm_tc(s, mW, mX, part, sk, M, false, (int *)sc, kDefaultWaitPolls);
    } else {
        pv.mode = 0;
        pv.S = launch_gemm(s, dtype, A, W, part, M, R, K);
        pv.split_stride = (size_t)M * R;
    }
    const RowScale none = {nullptr, 0, 0.f, 0.f};
    launch_reduce_partials(s, pv, none, out, M, R);
    return cudaGetLastError() == cudaSuccess ? EESD_OK : EESD_ERR_CUDA;
}

int eesd_time_projection(eesd_ctx *c, int which, int M, float *ms_per_launch, size_t *bytes_per_launch) {
    if (!c || which < 0 || which > 3 || M < 1 || M > EESD_MAX_ROWS || !ms_per_launch || !bytes_per_launch)
        return EESD_ERR_BADARG;
    const eesd_config &f = c->cfg;
    const int qd = f.n_heads * f.head_dim, kvd = f.n_kv_heads * f.head_dim, d = f.d_model, F = f.ffn_dim;
    const int R = which == 0 ? qd + 2 * kvd : which == 2 ? 2 * F : d;
    const int K = which == 1 ? qd : which == 3 ? F : d;
    const int X = which == 1 ? X_ATTN : which == 3 ? X_FFN : X_NORM;
    for (int pass = 0; pass < 2; pass++) {
        if (pass == 1) CU(c, cudaEventRecord(c->ev[0], c->stream));
        for (int l = 0; l < f.n_layers; l++) {
            const LayerW &w = c->layers[l];
            const void *W = which == 0 ? w.wqkv : which == 1 ? w.wo : which == 2 ? w.wgu : w.wd;
            const CUtensorMap *m = which == 0 ? &w.m_qkv : which == 1 ? &w.m_o : which == 2 ? &w.m_gu : &w.m_d;
            run_proj(c, W, m, which, X, M, R, K);
        }
        if (pass == 1) CU(c, cudaEventRecord(c->ev[1], c->stream));
    }
    int st = check_launch(c);
    if (st) return st;
    CU(c, cudaEventSynchronize(c->ev[1]));
    float ms = 0.f;
    cudaEventElapsedTime(&ms, c->ev[0], c->ev[1]);
    *ms_per_launch = ms / f.n_layers;
    *bytes_per_launch = (size_t)R * K * c->es;
    CU(c, cudaMemcpyAsync(c->h_result + 2, c->err, 4, cudaMemcpyDeviceToHost, c->stream));
    CU(c, cudaStreamSynchronize(c->stream));
    return read_error_word(c);
}

int eesd_sample_rows(void *cuda_stream, const float *logits, const float *u, int B, int V, float temperature,
                     int32_t *out) {
    if (!logits || !out || B < 1 || V < 1 || temperature < 0.f) return EESD_ERR_BADARG;
    if (temperature != 0.f && !u) return EESD_ERR_RNG;
    launch_sample_rows((cudaStream_t)cuda_stream, logits, u, B, V, temperature, out);
    return cudaGetLastError() == cudaSuccess ? EESD_OK : EESD_ERR_CUDA;
}

}  // extern "C"
