// Causal prompt attention over the paged bf16 KV cache on the Blackwell tensor cores (sm_100a).
//
// The prompt pass of the target model (Section 3: the target's cache is built before the first
// decode round) runs hundreds of rows at once.  Their keys / values are in the cache already; this
// kernel is the attention of all those rows, 128 query rows at a time, in the usual streaming
// (online-softmax) form:
//
// grid (H query heads, ceil(Mtot / 128) row tiles), 256 threads, one block per SM.  Block (h, qt)
//   * writes its 128 rotated, pre-scaled query rows to shared memory as two bf16 terms (hi, lo) in
//     operand form (A operand, 128 rows);
//   * walks over the 128-position tiles of KV head h / group up to its last row's position; the
//     page blocks of a tile are brought in by bulk asynchronous copies (keys double-buffered) and
//     are tensor-core operands as they lie in the cache (kv_layout.cuh);
//   * per tile: S = Q K^T (tcgen05.mma, fp32 in tensor memory); row r of the tile is owned by two
//     threads (its tensor-memory lane in warps w and w + 4), one per half of the columns: mask,
//     running maximum, numerators as two bf16 terms written back in operand form; O_t = P V
//     (second MMA chain); the two threads each keep half of the row's output in registers and
//     rescale it when the maximum moves;
//   * divides by the row sums and stores the rows as two bf16 terms, the layout the next
//     projection reads.
// Heavy row tiles (the last ones: most positions) are scheduled first.
//
// Every wait is bounded.  When one gives up the block raises the error word, leaves the loop,
// waits (with the full bound) for its own bulk copies, frees its tensor memory and returns.
#include "common.cuh"
#include "kernels.cuh"
#include "kv_layout.cuh"
#include "partials.cuh"
#include "tc_ptx.cuh"

namespace eesd {

typedef __nv_bfloat16 bf16;

namespace ap {

using namespace tc;

constexpr int THREADS = 256;
constexpr int QT = 128;   // query rows per block (rows of the A operands)
constexpr int KT = 128;   // positions per tile
constexpr uint32_t ROWS_LBO = (QT / 8) * 128;   // bytes between core matrices adjacent along the contraction index of the Q and P operands

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
    return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(a)) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(b)) << 16);
}
// eight fp32 values as two bf16 terms: hi = bf16(v), lo = bf16(v - hi)
__device__ __forceinline__ void split8(const float *v, uint4 &hi, uint4 &lo) {
    uint32_t h[4], l[4];
#pragma unroll
    for (int i = 0; i < 4; i++) {
        const bf16 a = __float2bfloat16_rn(v[2 * i]), b = __float2bfloat16_rn(v[2 * i + 1]);
        h[i] = (uint32_t)__bfloat16_as_ushort(a) | ((uint32_t)__bfloat16_as_ushort(b) << 16);
        l[i] = pack2(v[2 * i] - __bfloat162float(a), v[2 * i + 1] - __bfloat162float(b));
    }
    hi = make_uint4(h[0], h[1], h[2], h[3]);
    lo = make_uint4(l[0], l[1], l[2], l[3]);
}

template <int D> constexpr size_t smem_bytes() {
    return (size_t)2 * QT * D * 2 + (size_t)2 * KT * D * 2 + (size_t)KT * D * 2 + (size_t)2 * QT * KT * 2;
}

template <int D>
__global__ void __launch_bounds__(THREADS, 1) attn_prompt_kernel(PartView pv, RowScale rs, const float2 *__restrict__ rope, KvGeom kv,
                                                                 bf16 *__restrict__ attn_split, int Mtot, int pos0, int H,
                                                                 float scale2, int *err, uint32_t spin) {
    constexpr int HALF = D / 2;
    constexpr uint32_t GRP = (D / 8) * 128;            // bytes of one 8-position group of a key / value tile
    constexpr uint32_t Q_BYTES = QT * D * 2, K_BYTES = KT * D * 2, P_BYTES = QT * KT * 2;
    constexpr uint32_t TCOLS = 256;                    // tensor memory: S in columns 0..127, the tile's output in 128..128 + D
    constexpr int OC = D / 2;                          // output dimensions per thread
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char *sQ = smem, *sK = sQ + 2 * Q_BYTES, *sV = sK + 2 * K_BYTES, *sP = sV + K_BYTES;
    __shared__ uint64_t bars[5];   // keys (two buffers), values, score MMAs, output MMAs
    __shared__ uint32_t tmem_slot;
    __shared__ int s_abort;
    __shared__ float s_rstd[QT];
    __shared__ float s_half[THREADS];
    uint64_t *bar_k = bars, *bar_v = bars + 2, *bar_s = bars + 3, *bar_pv = bars + 4;
    volatile int *abort_flag = &s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int h = blockIdx.x, qt = (int)gridDim.y - 1 - (int)blockIdx.y;   // the longest row tiles first
    const int PT = kv.page_tokens, ptl = 31 - __clz(PT), kh = h / (H / kv.Hkv);
    const int r0 = qt * QT, n_rows = min(QT, Mtot - r0);
    const int T = (pos0 + r0 + n_rows - 1) / KT + 1;          // tiles up to the last row's own position
    const int n_pages = (pos0 + Mtot + PT - 1) >> ptl;        // pages the context holds
    const int ppt = KT >> ptl;                                // pages per tile
    const uint32_t blk_bytes = (uint32_t)(D * 2) << ptl;

    if (tid == 0) {
#pragma unroll
        for (int i = 0; i < 5; i++) mbar_init(&bars[i], 1);
        s_abort = 0;
        mbar_init_fence();
    }
    if (warp == 4) tmem_alloc(&tmem_slot, TCOLS);
    pdl_wait();
    if (tid < QT) s_rstd[tid] = tid < n_rows ? row_rstd(rs, r0 + tid) : 0.f;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;

    // ---- loader (warp 5): one lane per page of a tile
    int n_k[2] = {0, 0}, n_v = 0;   // copies issued per barrier (lane 0's count is the one used)
    auto load_tile = [&](int t, bool keys, unsigned char *dst, uint64_t *bar) {
        if (lane == 0) mbar_expect_tx(bar, blk_bytes * (uint32_t)ppt);
        __syncwarp();
        if (lane < ppt) {
            int page = kv.page_table[min(t * ppt + lane, n_pages - 1)];   // past the context: any finite block (masked)
            if (page < 0 || page >= kv.n_pages_total) { atomicOr(err, kErrBadPage); page = 0; }
            const bf16 *src = (const bf16 *)kv.slot_base + ((((size_t)page * 2 + (keys ? 0 : 1)) * kv.Hkv + kh) << ptl) * D;
            bulk_load(dst + (size_t)lane * blk_bytes, src, blk_bytes, bar);
        }
    };
    if (warp == 5) {
        load_tile(0, true, sK, &bar_k[0]);
        n_k[0]++;
    }

    // ---- queries: item = (row, 8 consecutive dimensions); consecutive lanes take consecutive rows.  Four items at a
    // time, all their loads requested before the first is used (pv is a plain [split][row][column] result here).
    constexpr int QI = QT * (D / 8) / THREADS, QB = 4;
#pragma unroll 1
    for (int g = 0; g < QI; g += QB) {
        float4 a[QB], b[QB], w0[QB], w1[QB];
#pragma unroll
        for (int k = 0; k < QB; k++) {
            const int idx = tid + (g + k) * THREADS, row = idx & (QT - 1), c = idx >> 7;
            a[k] = b[k] = make_float4(0.f, 0.f, 0.f, 0.f);
            w0[k] = w1[k] = make_float4(1.f, 0.f, 1.f, 0.f);
            if (row < n_rows) {
                const float4 *cs = reinterpret_cast<const float4 *>(rope + (size_t)(pos0 + r0 + row) * HALF + 4 * c);
                w0[k] = cs[0];
                w1[k] = cs[1];
            }
        }
        for (int sp = 0; sp < pv.S; sp++) {   // the k-range splits of the projection, added in order
            float4 la[QB], lb[QB];
#pragma unroll
            for (int k = 0; k < QB; k++) {
                const int idx = tid + (g + k) * THREADS, row = idx & (QT - 1), c = idx >> 7;
                la[k] = lb[k] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (row < n_rows) {
                    const float4 *src = reinterpret_cast<const float4 *>(pv.base + (size_t)sp * pv.split_stride + (size_t)(r0 + row) * pv.R + h * D + 8 * c);
                    la[k] = src[0];
                    lb[k] = src[1];
                }
            }
#pragma unroll
            for (int k = 0; k < QB; k++) {
                a[k].x += la[k].x; a[k].y += la[k].y; a[k].z += la[k].z; a[k].w += la[k].w;
                b[k].x += lb[k].x; b[k].y += lb[k].y; b[k].z += lb[k].z; b[k].w += lb[k].w;
            }
        }
#pragma unroll
        for (int k = 0; k < QB; k++) {
            const int idx = tid + (g + k) * THREADS, row = idx & (QT - 1), c = idx >> 7;
            uint4 hi = make_uint4(0, 0, 0, 0), lo = hi;
            if (row < n_rows) {
                const float r = s_rstd[row];
                const float raw[8] = {a[k].x * r, a[k].y * r, a[k].z * r, a[k].w * r, b[k].x * r, b[k].y * r, b[k].z * r, b[k].w * r};
                const float cw[8] = {w0[k].x, w0[k].y, w0[k].z, w0[k].w, w1[k].x, w1[k].y, w1[k].z, w1[k].w};   // (cos, sin) of four pairs
                float q[8];
#pragma unroll
                for (int i = 0; i < 4; i++) {
                    q[2 * i] = (raw[2 * i] * cw[2 * i] - raw[2 * i + 1] * cw[2 * i + 1]) * scale2;
                    q[2 * i + 1] = (raw[2 * i] * cw[2 * i + 1] + raw[2 * i + 1] * cw[2 * i]) * scale2;
                }
                split8(q, hi, lo);
            }
            unsigned char *dst = sQ + (uint32_t)c * ROWS_LBO + (uint32_t)row * 16;   // (row / 8) * 128 + (row % 8) * 16
            *reinterpret_cast<uint4 *>(dst) = hi;
            *reinterpret_cast<uint4 *>(dst + Q_BYTES) = lo;
        }
    }
    fence_async_smem();
    __syncthreads();

    const int quad = warp & 3, hf = warp >> 2, lane_id = quad * 32 + lane;    // this thread's row and column half
    const uint32_t tm_lane = tmem + ((uint32_t)(quad * 32) << 16);
    const int p_row = pos0 + r0 + lane_id;                                    // last position the row sees
    constexpr uint32_t IDESC_S = idesc_bf16(KT), IDESC_O = idesc_bf16(D);
    const uint64_t dQ = smem_desc_plain(smem_u32(sQ), ROWS_LBO, 128), dP = smem_desc_plain(smem_u32(sP), ROWS_LBO, 128);
    const uint64_t dK = smem_desc_plain(smem_u32(sK), 128, GRP), dV = smem_desc_plain(smem_u32(sV), GRP, 128);
    auto issue_scores = [&](int t) {   // S = (Q_hi + Q_lo) K_t^T
        const uint64_t dKt = dK + (uint64_t)(((t & 1) * K_BYTES) >> 4);
#pragma unroll
        for (int half = 0; half < 2; half++)
#pragma unroll
            for (int j = 0; j < D / 16; j++)
                mma_bf16(tmem, dQ + (uint64_t)((half * Q_BYTES + j * 2 * ROWS_LBO) >> 4), dKt + (uint64_t)((j * 256) >> 4), IDESC_S,
                         (half | j) != 0);
        mma_commit(bar_s);
    };
    if (tid == 128) {
        if (mbar_wait(&bar_k[0], 0, abort_flag, spin, 32)) {
            tc_fence_after();
            issue_scores(0);
        }
    }

    float o_acc[OC];
#pragma unroll
    for (int i = 0; i < OC; i++) o_acc[i] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;
    bool live = true;
    for (int t = 0; t < T; t++) {
        if (warp == 5) {   // keys of the next tile, values of this one (their buffers are free: see the waits below)
            if (t + 1 < T) {
                load_tile(t + 1, true, sK + ((t + 1) & 1) * K_BYTES, &bar_k[(t + 1) & 1]);
                n_k[(t + 1) & 1]++;
            }
            load_tile(t, false, sV, bar_v);
            n_v++;
        }
        // ---- scores of this tile: mask, running maximum
        mbar_wait(bar_s, t & 1, abort_flag, spin, 32);
        tc_fence_after();
        float sc[64];
        {
            uint32_t r[64];
            tmem_ld32(tm_lane + (uint32_t)(hf * 64), r);
            tmem_ld32(tm_lane + (uint32_t)(hf * 64 + 32), r + 32);
            const int p_first = t * KT + hf * 64;   // position of column 0 of this half
            const int n_seen = p_row - p_first;      // columns 0..n_seen are visible
#pragma unroll
            for (int c = 0; c < 64; c++) sc[c] = c <= n_seen ? __uint_as_float(r[c]) : -INFINITY;
        }
        tc_fence_before();
        float mx = sc[0];
#pragma unroll
        for (int c = 1; c < 64; c++) mx = fmaxf(mx, sc[c]);
        s_half[tid] = mx;
        __syncthreads();
        // no wait sits between this barrier and the next one, so the flag reads the same for every thread
        if (*abort_flag) { live = false; break; }
        const float m_new = fmaxf(fmaxf(m_run, fmaxf(mx, s_half[tid ^ 128])), -1e30f);
        const float alpha = ex2(m_run - m_new);
        m_run = m_new;
        float l_tile = 0.f;
#pragma unroll
        for (int j = 0; j < 8; j++) {   // numerators of 8 positions as two bf16 terms, one 16-byte store each
            float p[8];
#pragma unroll
            for (int i = 0; i < 8; i++) {
                p[i] = ex2(sc[8 * j + i] - m_new);
                l_tile += p[i];
            }
            uint4 hi, lo;
            split8(p, hi, lo);
            unsigned char *dst = sP + (uint32_t)(hf * 8 + j) * ROWS_LBO + (uint32_t)lane_id * 16;
            *reinterpret_cast<uint4 *>(dst) = hi;
            *reinterpret_cast<uint4 *>(dst + P_BYTES) = lo;
        }
        l_run = l_run * alpha + l_tile;
        fence_async_smem();
        tc_fence_before();
        __syncthreads();
        if (tid == 128) {   // O_t = (P_hi + P_lo) V_t, then the next tile's scores behind it
            if (mbar_wait(bar_v, t & 1, abort_flag, spin, 32)) {
                tc_fence_after();
#pragma unroll
                for (int half = 0; half < 2; half++)
#pragma unroll
                    for (int s = 0; s < KT / 16; s++)
                        mma_bf16(tmem + 128, dP + (uint64_t)((half * P_BYTES + s * 2 * ROWS_LBO) >> 4), dV + (uint64_t)((s * 2 * GRP) >> 4),
                                 IDESC_O, (half | s) != 0);
                mma_commit(bar_pv);
                if (t + 1 < T && mbar_wait(&bar_k[(t + 1) & 1], ((t + 1) >> 1) & 1, abort_flag, spin, 32)) {
                    tc_fence_after();
                    issue_scores(t + 1);
                }
            }
        }
        __syncwarp();
        // ---- this tile's output into the running one.  Once this wait has passed the output MMAs have
        // read the numerators and the values, and (earlier) the score MMAs the keys: their buffers are free.
        mbar_wait(bar_pv, t & 1, abort_flag, spin, 32);
        tc_fence_after();
#pragma unroll
        for (int q = 0; q < OC / 32; q++) {
            uint32_t r[32];
            tmem_ld32(tm_lane + (uint32_t)(128 + hf * OC + q * 32), r);
#pragma unroll
            for (int i = 0; i < 32; i++) o_acc[q * 32 + i] = fmaf(o_acc[q * 32 + i], alpha, __uint_as_float(r[i]));
        }
        tc_fence_before();
    }
    // ---- row sums of the two halves, then the rows as two bf16 terms
    __syncthreads();
    if (live && *abort_flag) live = false;   // uniform: the last waits are behind the barrier above
    if (live) {
        s_half[tid] = l_run;
        __syncthreads();
        const float other = s_half[tid ^ 128];
        const float inv = 1.0f / (hf ? other + l_run : l_run + other);   // the same sum in both threads
        if (lane_id < n_rows) {
            const int m = r0 + lane_id;
            bf16 *dst = attn_split + ((size_t)(m / kMaxRows) * 2 * kMaxRows + (m % kMaxRows)) * H * D + (size_t)h * D + hf * OC;
#pragma unroll
            for (int j = 0; j < OC / 8; j++) {
                float v[8];
#pragma unroll
                for (int i = 0; i < 8; i++) v[i] = o_acc[8 * j + i] * inv;
                uint4 hi, lo;
                split8(v, hi, lo);
                *reinterpret_cast<uint4 *>(dst + 8 * j) = hi;
                *reinterpret_cast<uint4 *>(dst + (size_t)kMaxRows * H * D + 8 * j) = lo;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) {
        tc_fence_after();
        tmem_dealloc(tmem, TCOLS);
    }
    if (!live) {
        if (tid == 0) atomicOr(err, kErrWaitTimeout);
        if (warp == 5 && lane == 0) {   // copies already issued must land before the shared memory is released
            if (n_k[0]) mbar_drain(&bar_k[0], (n_k[0] - 1) & 1);
            if (n_k[1]) mbar_drain(&bar_k[1], (n_k[1] - 1) & 1);
            if (n_v) mbar_drain(bar_v, (n_v - 1) & 1);
        }
    }
}

template <int D>
static void launch(cudaStream_t s, const PartView &pv, const RowScale &rs, const float2 *rope, const KvGeom &kv, void *attn_split,
                   int Mtot, int pos0, int H, float scale, int *err, uint32_t wait_polls) {
    static const cudaError_t configured =
        cudaFuncSetAttribute(attn_prompt_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes<D>());
    (void)configured;
    launch_k(attn_prompt_kernel<D>, dim3(H, (Mtot + QT - 1) / QT), dim3(THREADS), smem_bytes<D>(), s, false, pv, rs, rope, kv,
             (bf16 *)attn_split, Mtot, pos0, H, scale, err, wait_polls);
}

}  // namespace ap

void launch_attention_prompt(cudaStream_t s, const PartView &pv, const RowScale &rs, const float2 *rope, const KvGeom &kv,
                             void *attn_split, int Mtot, int pos0, int H, int *err, uint32_t wait_polls) {
    // queries are scaled by 1 / sqrt(D) and by log2 e: the softmax numerators are powers of two
    const float scale = 1.4426950408889634f / sqrtf((float)kv.D);
    if (kv.D == 64) ap::launch<64>(s, pv, rs, rope, kv, attn_split, Mtot, pos0, H, scale, err, wait_polls);
    else ap::launch<128>(s, pv, rs, rope, kv, attn_split, Mtot, pos0, H, scale, err, wait_polls);
}

}  // namespace eesd
