// Decode attention over the paged bf16 KV cache on the Blackwell tensor cores (sm_100a).
//
// One kernel per layer: RoPE of the new rows' queries and keys, in-place append of the new keys /
// values, attention of all M new rows (and all query heads of a KV group) over one slice of the
// cache, and the merge of the slices.
//
// grid (H_kv, n_split, batches), 256 threads.  Block (kh, sp, bz) owns up to 256 consecutive cached
// positions of KV head kh (whole pages) and up to NC (head, row) pairs ("columns").
//   * The page blocks of the slice are brought into shared memory by bulk asynchronous copies on
//     one mbarrier, issued before the kernel waits for its producer (cached rows do not depend on
//     it).  The cache stores a block as a grid of 8 x 8 core matrices (kv_layout.cuh), so the
//     copied bytes ARE the tensor-core operands, un-swizzled.
//   * scores:  S^T[position][column] = K Q^T, one tcgen05.mma chain per 128-position tile with
//     the key tile as the 128-row A operand and the queries as B.  Queries are fp32 values carried
//     as two bf16 terms (hi and lo columns: exact products, fp32 accumulation in tensor memory).
//   * softmax: thread t of warps 0-3 owns position t of each tile (its tensor-memory lane): it
//     masks, takes column maxima / sums across the warp (redux / shuffles) and across the four
//     warps (shared memory), and writes the numerators back to shared memory as two bf16 terms in
//     operand form.
//   * output:  O^T[dimension][column] = V^T P^T, one chain over the slice's 16-position steps with
//     the value tile as the A operand; thread t then owns output dimension t.
//   * each block writes, per column, its un-normalised output, maximum and sum; the block that
//     arrives last for (KV head, batch) merges the slices in index order (an arrival counter, no
//     waiting).
// Row m sees positions <= pos0 + m (a chain), or the rows its visibility mask names (a tree).
//
// Every wait is bounded.  When one gives up the block raises the error word, skips what is left,
// waits (with the full bound) for its own bulk copies, frees its tensor memory and returns.
#include "common.cuh"
#include "kernels.cuh"
#include "kv_layout.cuh"
#include "partials.cuh"
#include "tc_ptx.cuh"

namespace eesd {

typedef __nv_bfloat16 bf16;

namespace at {

using namespace tc;

constexpr int THREADS = 256;
constexpr int TILE = 128;         // positions per score tile (rows of the A operand)
constexpr int MAX_TILES = 2;      // score tiles per block: at most 256 positions per slice
constexpr int kMaxSlices = 64;    // most slices per head (layout of the per-slice maxima and sums)

// order-preserving map float -> int (for the integer warp reduction)
__device__ __forceinline__ int f2ord(float f) {
    const int i = __float_as_int(f);
    return i ^ ((i >> 31) & 0x7fffffff);
}
__device__ __forceinline__ float ord2f(int i) { return __int_as_float(i ^ ((i >> 31) & 0x7fffffff)); }

// 2^x by the special-function unit (2^-inf = 0)
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Sums of N = 16 or 32 per-lane values v[c] over the 32 lanes of a warp, all columns at once: each
// step halves the columns a lane carries (lanes with the step's bit set keep the upper half and
// hand over the lower one), so the whole reduction takes N shuffles instead of 5 N.  Returns the
// sum of column `lane` (N = 32) or `lane / 2` (N = 16, both lanes of a pair hold it).  The order
// of the additions is fixed.
template <int N>
__device__ __forceinline__ float column_sums(float (&v)[N], int lane) {
    int n = N;
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) {
        if (n == 1) {   // N = 16, last step: the pair's two halves of one column
            v[0] += __shfl_xor_sync(0xffffffffu, v[0], s);
        } else {
            const bool up = (lane & s) != 0;
            n >>= 1;
#pragma unroll
            for (int i = 0; i < N / 2; i++) {
                if (i < n) {
                    const float send = up ? v[i] : v[i + n], keep = up ? v[i + n] : v[i];
                    v[i] = keep + __shfl_xor_sync(0xffffffffu, send, s);
                }
            }
        }
    }
    return v[0];
}

__device__ __forceinline__ uint32_t pack_bf16(bf16 a, bf16 b) {
    return (uint32_t)__bfloat16_as_ushort(a) | ((uint32_t)__bfloat16_as_ushort(b) << 16);
}

// bytes between core matrices adjacent along the contraction index of the query / numerator
// operands: 2 NC columns = 2 NC / 8 core matrices of 128 bytes, plus 16 bytes so that writers of
// neighbouring 16-byte chunks hit different banks
template <int NC> struct Opnd { static constexpr uint32_t LBO = (2 * NC / 8) * 128 + 16; };

struct Smem {
    uint32_t k, v, q, p, wgt, red, misc, total;
};
// shared-memory carve-up for a slice of `cap` positions (a multiple of 16), D, NC, n_split
__host__ __device__ inline Smem carve(int cap, int D, int NC, int n_split) {
    Smem s;
    const uint32_t lbo = (2 * NC / 8) * 128 + 16;
    const int n_tiles = (cap + TILE - 1) / TILE;
    uint32_t o = 0;
    s.k = o; o += (uint32_t)cap * D * 2;
    s.v = o; o += (uint32_t)cap * D * 2;
    s.q = o; o += (uint32_t)(D / 8) * lbo;
    s.p = o; o += (uint32_t)(n_tiles * TILE / 8) * lbo;
    // the score MMAs read 128 key rows per tile whether or not the slice fills them, and the output
    // MMAs read 128 value rows when D = 64: those reads must stay inside the allocation
    const uint32_t reach_k = s.k + (uint32_t)n_tiles * TILE * D * 2, reach_v = s.v + (uint32_t)cap * D * 2 + 2048;
    if (o < reach_k) o = reach_k;
    if (o < reach_v) o = reach_v;
    o = (o + 15u) & ~15u;
    s.wgt = o; o += (uint32_t)NC * n_split * 4;
    s.red = o; o += 2u * 8 * NC * 4;        // per-warp column maxima and sums
    s.misc = o; o += 256;
    s.total = o;
    return s;
}

template <int D, int NC, bool TR>
__global__ void __launch_bounds__(THREADS) attn_tc_kernel(PartView pv, RowScale rs, const float2 *__restrict__ rope, KvGeom kv,
                                                          float *__restrict__ apart, unsigned int *tickets,
                                                          float *__restrict__ attn_out, bf16 *__restrict__ attn_split,
                                                          int M, int pos0, int H, int pps, int n_split, float scale2, int *err,
                                                          TreeRows tr, uint32_t spin, BatchRows br) {
    constexpr int HALF = D / 2;
    constexpr uint32_t LBO_C = Opnd<NC>::LBO;          // query / numerator operands
    constexpr uint32_t GRP = (D / 8) * 128;            // bytes of one 8-position group of a key / value tile
    constexpr uint32_t TCOLS = MAX_TILES * 2 * NC;     // tensor-memory columns: one 2 NC-wide accumulator per score tile
    extern __shared__ __align__(128) unsigned char smem[];
    const int PT = kv.page_tokens, ptl = 31 - __clz(PT), group = H / kv.Hkv;
    const int cap = pps * PT;
    const int ns_stride = n_split;   // slices in the scratch layouts (batch mode: those of the longest sequence)
    const Smem lay = carve(cap, D, NC, ns_stride);
    unsigned char *sK = smem + lay.k, *sV = smem + lay.v, *sQ = smem + lay.q, *sP = smem + lay.p;
    float *wgt = reinterpret_cast<float *>(smem + lay.wgt);       // [NC][n_split] merge weights
    float *s_mx = reinterpret_cast<float *>(smem + lay.red);      // [8][NC] per-warp column maxima
    float *s_sm = s_mx + 8 * NC;                                  // [8][NC] per-warp column sums
    uint64_t *bar_kv = reinterpret_cast<uint64_t *>(smem + lay.misc);   // cached slice has landed
    uint64_t *bar_s = bar_kv + 1, *bar_o = bar_kv + 2;                  // score / output MMAs have completed
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bar_kv + 3);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    int *s_last = const_cast<int *>(abort_flag) + 1;
    float *s_rstd = reinterpret_cast<float *>(s_last + 1);        // [kMaxRows]
    __shared__ uint16_t s_vis[kMaxRows];
    __shared__ uint8_t s_dep[kMaxRows];
    __shared__ int8_t s_colm[NC];                                  // row m of each column
    __shared__ int16_t s_colh[NC];                                 // query head of each column
    __shared__ int2 s_tb[40];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int kh = blockIdx.x, sp = blockIdx.y;
    // Batch mode: grid z runs over (sequence, column batch); a sequence is an independent problem with its
    // own rows of the pass, positions, page table and slice count.
    int bz = blockIdx.z, row_base = 0;
    if (br.n_seq > 0) {
        const int nbat = gridDim.z / br.n_seq, seq = blockIdx.z / nbat;
        bz = blockIdx.z - seq * nbat;
        M = br.rows[seq];
        pos0 = br.pos0[seq];
        row_base = br.row0[seq];
        kv.page_table += br.table_off[seq];
        n_split = (((pos0 + M + PT - 1) >> ptl) + pps - 1) / pps;
        if (sp >= n_split || group * M <= bz * NC) return;   // a shorter sequence fills fewer slices and batches
    }
    // per-slice (maximum, sum) pairs live behind the outputs: [H][16][kMaxSlices]
    float2 *ml = reinterpret_cast<float2 *>(apart + (size_t)H * kMaxSlices * kMaxRows * D);
    const int r0 = bz * NC;                  // first column ((head, row) pair) of this block's batch
    const int nb = min(NC, group * M - r0);  // columns in use; pair rho = r0 + c = g * M + m
    const int ctx_len = pos0 + M;
    const int n_pages = (ctx_len + PT - 1) >> ptl;
    const int page_lo = sp * pps, page_hi = min(n_pages, page_lo + pps);
    const int lo = page_lo << ptl;
    const int npos = min(ctx_len, page_hi << ptl) - lo;   // valid positions of this block
    const int n_tiles = (npos + TILE - 1) / TILE;
    const uint32_t blk_bytes = (uint32_t)(D * 2) << ptl;

    pdl_trigger();
    if (TR && tid >= 32 && tid < 32 + kMaxRows) { s_vis[tid - 32] = tr.vis[tid - 32]; s_dep[tid - 32] = tr.depth[tid - 32]; }
    if (tid >= 64 && tid < 64 + NC) {   // one division per column, here and nowhere else
        const int rho = r0 + tid - 64, g = rho / M;
        s_colm[tid - 64] = (int8_t)(rho - g * M);
        s_colh[tid - 64] = (int16_t)(kh * group + g);
    }
    if (tid == 0) {
        mbar_init(bar_kv, 1);
        mbar_init(bar_s, 1);
        mbar_init(bar_o, 1);
        *abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 5) tmem_alloc(tmem_slot, TCOLS);
    // cached rows were written by earlier passes: no need to wait for this pass's producers.
    // One lane of warp 4 per page (a slice has at most 32), so the page-table reads are in flight together.
    const int pg = page_lo + lane;
    int page = 0;
    if (warp == 4 && pg < page_hi) page = kv.page_table[pg];
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    if (warp == 4) {
        if (lane == 0) mbar_expect_tx(bar_kv, 2u * blk_bytes * (uint32_t)(page_hi - page_lo));
        __syncwarp();
        if (pg < page_hi) {
            const bf16 *src = (const bf16 *)kv.slot_base + ((((size_t)page * 2) * kv.Hkv + kh) << ptl) * D;
            bulk_load(sK + (size_t)lane * blk_bytes, src, blk_bytes, bar_kv);
            bulk_load(sV + (size_t)lane * blk_bytes, src + (((size_t)kv.Hkv) << ptl) * D, blk_bytes, bar_kv);
        }
    }
    // where the partial sums this block needs live (block numbers of the query tiles of its
    // batch and of its key and value tile): integer arithmetic only, done before the wait
    const int tq0 = ((kh * group + r0 / M) * D) >> 7, tq1 = ((kh * group + (r0 + nb - 1) / M) * D + D - 1) >> 7;
    const int nq = tq1 - tq0 + 1, tk = ((H + kh) * D) >> 7, tv = ((H + kv.Hkv + kh) * D) >> 7;
    if (pv.mode == 1 && tid >= 160 && tid - 160 < nq + 2 && tid - 160 < 40)
        s_tb[tid - 160] = tile_blocks(pv.sk, tid - 160 < nq ? tq0 + tid - 160 : (tid - 160 == nq ? tk : tv));
    // new rows that fall into this slice: (position, key pair | value pair) items
    const int p_first = max(lo, pos0), p_last = min(lo + npos, ctx_len);   // [p_first, p_last)
    const int n_new = max(0, p_last - p_first) * D;
    const int n_q = nb * HALF;
    constexpr int kNewMax = (kMaxRows * D + THREADS - 1) / THREADS;
    constexpr int kQMax = (NC * HALF + THREADS - 1) / THREADS;
    // rotation factors: a constant table, fetched before the wait so that they are not one more
    // round trip behind the partial sums
    float2 cs_new[kNewMax], cs_q[kQMax];
#pragma unroll
    for (int it = 0; it < kNewMax; it++) {
        if (it * THREADS >= n_new) break;   // uniform
        const int idx = tid + it * THREADS;
        const int pn = idx / D, w = idx - pn * D;
        cs_new[it] = (idx < n_new && w < HALF) ? rope[(size_t)(TR ? pos0 + s_dep[p_first + pn - pos0] : p_first + pn) * HALF + w] : make_float2(1.f, 0.f);
    }
    __syncthreads();   // column tables, block table
#pragma unroll
    for (int it = 0; it < kQMax; it++) {
        if (it * THREADS >= n_q) break;
        const int idx = tid + it * THREADS;
        const int rl = idx / HALF, i = idx - rl * HALF;
        cs_q[it] = idx < n_q ? rope[(size_t)(pos0 + (TR ? (int)s_dep[s_colm[rl]] : (int)s_colm[rl])) * HALF + i] : make_float2(1.f, 0.f);
    }
    auto gather_pair = [&](int m, int col) -> float2 {
        if (pv.mode != 1) return part_gather_n<2>(pv, m, col);
        const int t = col >> 7;
        return part_gather_blocks<2>(pv, s_tb[t == tk ? nq : (t == tv ? nq + 1 : t - tq0)], m, col);
    };
    pdl_wait();   // from here on the QKV projection's partial sums are read
    // One round of global loads: the RMSNorm statistics (threads 0..M-1) and the raw partial
    // sums of this block's queries and of the new keys / values that fall into its slice.
    if (tid < M) s_rstd[tid] = row_rstd(rs, row_base + tid);
    float raw_a[kNewMax], raw_b[kNewMax];
    int new_page[kNewMax];
#pragma unroll
    for (int it = 0; it < kNewMax; it++) {
        if (it * THREADS >= n_new) break;
        const int idx = tid + it * THREADS;   // -> (position, K pair | V pair)
        if (idx < n_new) {
            const int pn = idx / D, w = idx - pn * D;
            new_page[it] = kv.page_table[(p_first + pn) >> ptl];
            const int isV = w >= HALF, i = isV ? w - HALF : w;
            const float2 pr = gather_pair(row_base + p_first + pn - pos0, (H + (isV ? kv.Hkv : 0) + kh) * D + 2 * i);
            raw_a[it] = pr.x;
            raw_b[it] = pr.y;
        }
    }
    float qraw_a[kQMax], qraw_b[kQMax];
#pragma unroll
    for (int it = 0; it < kQMax; it++) {
        if (it * THREADS >= n_q) break;
        const int idx = tid + it * THREADS;
        if (idx < n_q) {
            const int rl = idx / HALF, i = idx - rl * HALF;
            const float2 pr = gather_pair(row_base + s_colm[rl], s_colh[rl] * D + 2 * i);
            qraw_a[it] = pr.x;
            qraw_b[it] = pr.y;
        }
    }
    __syncthreads();
    // rotated, pre-scaled queries of this block's batch as two bf16 terms, in operand form:
    // column c (hi) and NC + c (lo), dimension e at (e / 8) * LBO_C + (c / 8) * 128 + (c % 8) * 16 + (e % 8) * 2
#pragma unroll
    for (int it = 0; it < kQMax; it++) {
        if (it * THREADS >= n_q) break;
        const int idx = tid + it * THREADS;
        if (idx < n_q) {
            const int rl = idx / HALF, i = idx - rl * HALF;
            const float r = s_rstd[s_colm[rl]];
            const float a = qraw_a[it] * r, b = qraw_b[it] * r;
            const float2 cs = cs_q[it];
            const float qa = (a * cs.x - b * cs.y) * scale2, qb = (a * cs.y + b * cs.x) * scale2;
            const bf16 ha = __float2bfloat16_rn(qa), hb = __float2bfloat16_rn(qb);
            const uint32_t off = (uint32_t)((2 * i) >> 3) * LBO_C + (uint32_t)((2 * i) & 7) * 2;
            *reinterpret_cast<uint32_t *>(sQ + off + (rl >> 3) * 128 + (rl & 7) * 16) = pack_bf16(ha, hb);
            *reinterpret_cast<uint32_t *>(sQ + off + ((NC + rl) >> 3) * 128 + ((NC + rl) & 7) * 16) =
                pack_bf16(__float2bfloat16_rn(qa - __bfloat162float(ha)), __float2bfloat16_rn(qb - __bfloat162float(hb)));
        }
    }
    bf16 new_a[kNewMax], new_b[kNewMax];
#pragma unroll
    for (int it = 0; it < kNewMax; it++) {
        if (it * THREADS >= n_new) break;
        const int idx = tid + it * THREADS;
        if (idx < n_new) {
            const int pn = idx / D, w = idx - pn * D;
            const float r = s_rstd[p_first + pn - pos0];
            float a = raw_a[it] * r, b = raw_b[it] * r;
            if (w < HALF) {
                const float2 cs = cs_new[it];
                const float ra = a * cs.x - b * cs.y, rb = a * cs.y + b * cs.x;
                a = ra; b = rb;
            }
            new_a[it] = __float2bfloat16_rn(a);
            new_b[it] = __float2bfloat16_rn(b);
        }
    }
    if (warp == 0) mbar_wait(bar_kv, 0, abort_flag, spin, 32);   // the cached slice (bounded); the other warps park at the barrier below
    __syncthreads();
    if (!*abort_flag) {
        // the new rows go into the tiles and (by one block of the batches) into the cache
#pragma unroll
        for (int it = 0; it < kNewMax; it++) {
            if (it * THREADS >= n_new) break;
            const int idx = tid + it * THREADS;
            if (idx < n_new) {
                const int pn = idx / D, w = idx - pn * D;
                const int pos = p_first + pn, j = pos - lo;
                const int isV = w >= HALF, e = 2 * (isV ? w - HALF : w);
                const int page = new_page[it];
                if (page < 0 || page >= kv.n_pages_total) { atomicOr(err, kErrBadPage); continue; }
                bf16 *blk = (bf16 *)kv.slot_base + ((((size_t)page * 2 + isV) * kv.Hkv + kh) << ptl) * D;
                const bool append = bz == 0;   // every batch needs the row in its tile; one block writes the cache
                const int pp = pos & (PT - 1);
                // a slice's pages sit one after the other in shared memory: token j of the slice is token j of one long block
                if (isV) {
                    bf16 *tile = reinterpret_cast<bf16 *>(sV);
                    const size_t t0 = v_index<bf16>(pos, j, e, PT, D);     // dimensions e, e + 1: 8 elements apart
                    tile[t0] = new_a[it]; tile[t0 + 8] = new_b[it];
                    if (append) {
                        const size_t g0 = v_index<bf16>(pos, pp, e, PT, D);
                        blk[g0] = new_a[it]; blk[g0 + 8] = new_b[it];
                    }
                } else {
                    const uint32_t w2 = pack_bf16(new_a[it], new_b[it]);   // dimensions e, e + 1 are adjacent in a key core matrix
                    *reinterpret_cast<uint32_t *>(reinterpret_cast<bf16 *>(sK) + k_index<bf16>(j, e, PT, D)) = w2;
                    if (append) *reinterpret_cast<uint32_t *>(blk + k_index<bf16>(pp, e, PT, D)) = w2;
                }
            }
        }
        // The output MMAs take the slice in steps of 16 positions.  With 8-token pages a slice may end on an odd
        // page: the 8 positions after it were never copied, and their weights being zero does not help if the
        // bytes there look like a NaN.  Clear those value rows (one 8-position group, contiguous).
        {
            const int loaded = (page_hi - page_lo) << ptl, need = ((npos + 15) >> 4) << 4;
            if (loaded < need) {
                uint4 *z = reinterpret_cast<uint4 *>(sV + (size_t)(loaded >> 3) * GRP);
                for (int i = tid; i < (int)(((need - loaded) >> 3) * GRP / 16); i += THREADS) z[i] = make_uint4(0u, 0u, 0u, 0u);
            }
        }
        fence_async_smem();   // generic-proxy writes (queries, new rows) before the MMAs read them
    }
    __syncthreads();
    // From here on thread (warp, lane) owns tensor-memory lane 32 (warp % 4) + lane: position
    // 128 t + that lane of score tile t = warp / 4, then output dimension = that lane.
    const int quad = warp & 3, tl = warp >> 2, lane_id = quad * 32 + lane;
    const uint32_t tm_lane = tmem + ((uint32_t)(quad * 32) << 16);
    constexpr uint32_t IDESC = idesc_bf16(2 * NC);
    // operand descriptors of the first step; later steps add their byte offset / 16 to the address field
    const uint64_t dK = smem_desc_plain(smem_u32(sK), 128, GRP), dQ = smem_desc_plain(smem_u32(sQ), LBO_C, 128);
    const uint64_t dV = smem_desc_plain(smem_u32(sV), GRP, 128), dP = smem_desc_plain(smem_u32(sP), LBO_C, 128);
    bool live = !*abort_flag;
    if (live) {
        if (tid == 128) {   // ---- score MMAs: one chain of D / 16 steps per 128-position tile
            tc_fence_after();
#pragma unroll
            for (int t = 0; t < MAX_TILES; t++) {
                if (t < n_tiles) {
#pragma unroll
                    for (int j = 0; j < D / 16; j++)
                        mma_bf16(tmem + (uint32_t)(t * 2 * NC), dK + (uint64_t)((t * (TILE / 8) * GRP + j * 256) >> 4),
                                 dQ + (uint64_t)((j * 2 * LBO_C) >> 4), IDESC, j > 0);
                }
            }
            mma_commit(bar_s);
        }
        __syncwarp();
        mbar_wait(bar_s, 0, abort_flag, spin, 32);
    }
    __syncthreads();   // the eight warps go on together or not at all
    live = !*abort_flag;
    if (live) {
        // ---- softmax numerators (base 2: the queries carry log2 e)
        tc_fence_after();
        float sc[NC];
        const int j = tl * TILE + lane_id;     // position within the slice
        if (tl < n_tiles) {
            uint32_t r[2 * NC];
#pragma unroll
            for (int q = 0; q < 2 * NC / 32; q++) tmem_ld32(tm_lane + (uint32_t)(tl * 2 * NC + q * 32), r + q * 32);
            const int jn = lo + j - pos0;      // >= 0: a new row
#pragma unroll
            for (int c = 0; c < NC; c++) {
                if (c >= nb) break;
                const int m = s_colm[c];
                const bool seen = TR ? (jn < 0 || ((s_vis[m] >> jn) & 1)) : (jn <= m);
                sc[c] = (j < npos && seen) ? __uint_as_float(r[NC + c]) + __uint_as_float(r[c]) : -INFINITY;
            }
        } else {
#pragma unroll
            for (int c = 0; c < NC; c++) sc[c] = -INFINITY;
        }
        tc_fence_before();
        // column maxima: the warp's 32 positions by an integer reduction, the eight warps' through shared memory
#pragma unroll
        for (int c = 0; c < NC; c++) {
            if (c >= nb) break;
            const int o = __reduce_max_sync(0xffffffffu, f2ord(sc[c]));
            if (lane == (c & 31)) s_mx[warp * NC + c] = ord2f(o);
        }
        __syncthreads();
        float mx_lane = -INFINITY;   // lane c: maximum of column c over the slice
        if (lane < nb) {
#pragma unroll
            for (int w = 0; w < 8; w++) mx_lane = fmaxf(mx_lane, s_mx[w * NC + lane]);
        }
        mx_lane = fmaxf(mx_lane, -1e30f);   // a column that sees nothing in this slice: every numerator 2^(-inf) = 0
        float pr[NC];
#pragma unroll
        for (int c = 0; c < NC; c++) {
            if (c >= nb) { pr[c] = 0.f; continue; }
            const float p = ex2(sc[c] - __shfl_sync(0xffffffffu, mx_lane, c));
            pr[c] = p;
            if (tl < n_tiles) {
                // numerators as two bf16 terms in operand form: position j at (j / 8) * LBO_C + (j % 8) * 2
                const bf16 hi = __float2bfloat16_rn(p);
                unsigned char *dst = sP + (uint32_t)(j >> 3) * LBO_C + (j & 7) * 2;
                *reinterpret_cast<bf16 *>(dst + (c >> 3) * 128 + (c & 7) * 16) = hi;
                *reinterpret_cast<bf16 *>(dst + ((NC + c) >> 3) * 128 + ((NC + c) & 7) * 16) = __float2bfloat16_rn(p - __bfloat162float(hi));
            }
        }
        // column sums over the warp's positions (fixed order), one entry per (warp, column)
        if (nb <= 2) {
#pragma unroll
            for (int c = 0; c < 2; c++) {
                if (c >= nb) break;
                const float s = warp_sum(pr[c]);
                if (lane == 0) s_sm[warp * NC + c] = s;
            }
        } else {
            const float s = column_sums<NC>(pr, lane);
            const int c = NC == 32 ? lane : (lane >> 1);
            if ((NC == 32 || !(lane & 1)) && c < nb) s_sm[warp * NC + c] = s;
        }
        fence_async_smem();
        tc_fence_before();
    }
    __syncthreads();
    if (live) {
        if (tid == 128) {   // ---- output MMAs: one chain over the slice's 16-position steps
            tc_fence_after();
            const int steps = (npos + 15) >> 4;
            for (int s = 0; s < steps; s++)
                mma_bf16(tmem, dV + (uint64_t)s * ((2 * GRP) >> 4), dP + (uint64_t)s * ((2 * LBO_C) >> 4), IDESC, s > 0);
            mma_commit(bar_o);
        }
        if (tid < nb) {   // thread c: maximum and sum of column c over this slice
            const int c = tid;
            float l = 0.f, mx = s_mx[c];
#pragma unroll
            for (int w = 0; w < 8; w++) l += s_sm[w * NC + c];
#pragma unroll
            for (int w = 1; w < 8; w++) mx = fmaxf(mx, s_mx[w * NC + c]);
            ml[((size_t)s_colh[c] * kMaxRows + row_base + s_colm[c]) * kMaxSlices + sp] = make_float2(mx, l);
        }
        __syncwarp();
        mbar_wait(bar_o, 0, abort_flag, spin, 32);
    }
    __syncthreads();
    live = !*abort_flag;
    if (live) {
        // ---- un-normalised outputs of the slice: warps 0-3 take the first half of the columns, warps 4-7 the second
        tc_fence_after();
        constexpr int HC = NC / 2;
        const int c0 = tl * HC;
        if (c0 < nb) {
            uint32_t rh[HC], rl[HC];
            tmem_ld<HC>(tm_lane + (uint32_t)c0, rh);
            tmem_ld<HC>(tm_lane + (uint32_t)(NC + c0), rl);
            if (lane_id < D) {
#pragma unroll
                for (int c = 0; c < HC; c++) {
                    if (c0 + c >= nb) break;
                    apart[(((size_t)s_colh[c0 + c] * ns_stride + sp) * kMaxRows + row_base + s_colm[c0 + c]) * D + lane_id] =
                        __uint_as_float(rl[c]) + __uint_as_float(rh[c]);
                }
            }
        }
        tc_fence_before();
    }
    // ---- teardown of the tensor-core part
    __threadfence();
    __syncthreads();
    if (warp == 5) {
        tc_fence_after();
        tmem_dealloc(tmem, TCOLS);
    }
    if (*abort_flag) {
        if (tid == 0) {
            atomicOr(err, kErrWaitTimeout);
            mbar_drain(bar_kv, 0);   // the slice's bulk copies must land before the shared memory is released
        }
        return;
    }
    // ---- merge: the block that arrives last for this (KV head, batch) combines all slices
    if (tid == 0) {
        unsigned int *tkt = tickets + (size_t)kh * gridDim.z + blockIdx.z;   // one counter per (KV head, sequence, batch)
        const unsigned int prev = atomicAdd(tkt, 1u);
        *s_last = (prev == (unsigned int)n_split - 1);
        if (*s_last) *tkt = 0;
    }
    __syncthreads();
    if (!*s_last) return;
    __threadfence();
    const size_t sstride = (size_t)kMaxRows * D;
    // this thread's first item (column, four output dimensions): its first eight slices are requested now,
    // together with the slices' maxima and sums, so that the merge costs one round trip, not two
    float4 pre[8];
    {
        const int rl = min(tid / (D / 4), nb - 1), dd = (tid % (D / 4)) * 4;
        const float *src = apart + ((size_t)s_colh[rl] * ns_stride * kMaxRows + row_base + s_colm[rl]) * D + dd;
#pragma unroll
        for (int u = 0; u < 8; u++)
            pre[u] = (tid < nb * (D / 4) && u < n_split) ? __ldcg(reinterpret_cast<const float4 *>(src + (size_t)u * sstride)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    {   // normalised weight of every (column, slice); a warp's columns are loaded together
        constexpr int CPW = NC / 8;
        const float2 none = make_float2(-INFINITY, 0.f);
        float2 v0[CPW], v1[CPW];
#pragma unroll
        for (int i = 0; i < CPW; i++) {
            const int rl = min(warp + 8 * i, nb - 1);
            const float2 *src = ml + ((size_t)s_colh[rl] * kMaxRows + row_base + s_colm[rl]) * kMaxSlices;
            v0[i] = (warp + 8 * i < nb && lane < n_split) ? __ldcg(src + lane) : none;
            v1[i] = (warp + 8 * i < nb && lane + 32 < n_split) ? __ldcg(src + lane + 32) : none;
        }
#pragma unroll
        for (int i = 0; i < CPW; i++) {
            const int rl = warp + 8 * i;
            if (rl >= nb) break;   // warp-uniform
            const float mx = warp_max(fmaxf(v0[i].x, v1[i].x));
            const float w0 = (v0[i].x == -INFINITY) ? 0.f : exp2f(v0[i].x - mx), w1 = (v1[i].x == -INFINITY) ? 0.f : exp2f(v1[i].x - mx);
            const float den = warp_sum(fmaf(w0, v0[i].y, w1 * v1[i].y));   // fixed butterfly over the lanes
            const float inv = den > 0.f ? 1.0f / den : 0.f;
            if (lane < n_split) wgt[rl * n_split + lane] = w0 * inv;
            if (lane + 32 < n_split) wgt[rl * n_split + lane + 32] = w1 * inv;
        }
    }
    __syncthreads();
    for (int idx = tid; idx < nb * (D / 4); idx += THREADS) {   // four output dimensions per item
        const int rl = idx / (D / 4), dd = (idx - rl * (D / 4)) * 4;
        const int m = row_base + s_colm[rl], h = s_colh[rl];   // row of the pass
        const float *src = apart + ((size_t)h * ns_stride * kMaxRows + m) * D + dd;
        const float *wr = wgt + rl * n_split;
        float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s2 = 0; s2 < n_split; s2 += 8) {   // eight slices in flight, added in slice order
            float4 a[8];
#pragma unroll
            for (int u = 0; u < 8; u++) {
                if (idx == tid && s2 == 0) a[u] = pre[u];
                else a[u] = s2 + u < n_split ? __ldcg(reinterpret_cast<const float4 *>(src + (size_t)(s2 + u) * sstride)) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < 8; u++) {
                const float w = s2 + u < n_split ? wr[s2 + u] : 0.f;
                o.x = fmaf(w, a[u].x, o.x); o.y = fmaf(w, a[u].y, o.y);
                o.z = fmaf(w, a[u].z, o.z); o.w = fmaf(w, a[u].w, o.w);
            }
        }
        const size_t col = (size_t)h * D + dd;
        if (attn_out) *reinterpret_cast<float4 *>(attn_out + (size_t)m * H * D + col) = o;
        if (attn_split) {   // two bf16 terms, four dimensions at a time (store_split's layout)
            const bf16 h0 = __float2bfloat16_rn(o.x), h1 = __float2bfloat16_rn(o.y), h2 = __float2bfloat16_rn(o.z), h3 = __float2bfloat16_rn(o.w);
            bf16 *xh = attn_split + (size_t)m * H * D + col;
            *reinterpret_cast<uint2 *>(xh) = make_uint2(pack_bf16(h0, h1), pack_bf16(h2, h3));
            *reinterpret_cast<uint2 *>(xh + (size_t)kMaxRows * H * D) =
                make_uint2(pack_bf16(__float2bfloat16_rn(o.x - __bfloat162float(h0)), __float2bfloat16_rn(o.y - __bfloat162float(h1))),
                           pack_bf16(__float2bfloat16_rn(o.z - __bfloat162float(h2)), __float2bfloat16_rn(o.w - __bfloat162float(h3))));
        }
    }
}

template <int D, int NC, bool TR>
static void launch(cudaStream_t s, const PartView &pv, const RowScale &rs, const float2 *rope, const KvGeom &kv, float *apart,
                   unsigned int *tickets, float *attn_out, void *attn_split, int M, int pos0, int H, int pps, int n_split,
                   float scale, bool early, int *err, const TreeRows &tr, uint32_t wait_polls, const BatchRows &br) {
    const int rows = (H / kv.Hkv) * M, nbat = (rows + NC - 1) / NC;
    const Smem lay = carve(pps * kv.page_tokens, D, NC, n_split);
    // once per instantiation (thread-safe static initialisation)
    static const cudaError_t configured =
        cudaFuncSetAttribute(attn_tc_kernel<D, NC, TR>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 2048);
    (void)configured;
    launch_k(attn_tc_kernel<D, NC, TR>, dim3(kv.Hkv, n_split, nbat * (br.n_seq > 0 ? br.n_seq : 1)), dim3(THREADS), (size_t)lay.total, s,
             early && pdl_enabled(), pv, rs, rope, kv, apart, tickets, attn_out, (bf16 *)attn_split, M, pos0, H, pps, n_split, scale, err, tr,
             wait_polls, br);
}

}  // namespace at

int attention_tc_columns(int rows) { return rows <= 16 ? 16 : 32; }

// Slices of the cached context for the tensor-core kernel: pages per block (at most 256
// positions, a multiple of 16) and blocks per KV head (at most max_splits <= 64).
int attention_tc_splits(int ctx_len, int page_tokens, int Hkv, int n_batches, int n_sm, int max_splits, int *pps_out) {
    const int n_pages = (ctx_len + page_tokens - 1) / page_tokens;
    const int cap = at::MAX_TILES * at::TILE / page_tokens;   // pages one block can hold (page_tokens <= 128)
    // one wave: about two blocks per SM in flight, so aim for H_kv * batches * n_split <= 2 * n_sm
    int want = 2 * n_sm / (Hkv * n_batches);
    if (want < 1) want = 1;
    if (want > max_splits) want = max_splits;
    int pps = (n_pages + want - 1) / want;
    if (pps > cap) pps = cap;            // longer contexts: more slices than one wave holds
    if (pps < 1) pps = 1;
    if ((pps * page_tokens) % 16) pps++;   // slices hold a multiple of 16 positions (page_tokens 8: an even page count)
    *pps_out = pps;
    return (n_pages + pps - 1) / pps;
}

void launch_attention_tc(cudaStream_t s, const PartView &pv, const RowScale &rs, const float2 *rope, const KvGeom &kv, float *apart,
                         unsigned int *tickets, float *attn_out, void *attn_split, int M, int pos0, int H, int pps, int n_split,
                         bool early, int *err, const TreeRows *tree, uint32_t wait_polls, const BatchRows *batch) {
    // queries are scaled by 1 / sqrt(D) and by log2 e: the softmax numerators are powers of two
    const float scale = 1.4426950408889634f / sqrtf((float)kv.D);
    const int rows = (H / kv.Hkv) * M;
    const TreeRows tr = tree ? *tree : chain_rows();
    BatchRows br = {};
    if (batch) br = *batch;
    const bool wide = attention_tc_columns(rows) == 32;
#define EESD_AT(D, NC, TR) at::launch<D, NC, TR>(s, pv, rs, rope, kv, apart, tickets, attn_out, attn_split, M, pos0, H, pps, n_split, scale, early, err, tr, wait_polls, br)
    if (kv.D == 64) {
        if (tree) { if (wide) EESD_AT(64, 32, true); else EESD_AT(64, 16, true); }
        else { if (wide) EESD_AT(64, 32, false); else EESD_AT(64, 16, false); }
    } else {
        if (tree) { if (wide) EESD_AT(128, 32, true); else EESD_AT(128, 16, true); }
        else { if (wide) EESD_AT(128, 32, false); else EESD_AT(128, 16, false); }
    }
#undef EESD_AT
}

}  // namespace eesd
