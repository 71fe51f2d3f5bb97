// Weight-streaming skinny projection on the Blackwell tensor cores (sm_100a).
//
//   out[m][r] = sum_k X[m][k] * W[r][k],   m < M <= 16 token rows,  W bf16 [R][K] row-major
//
// HBM-bound: every weight byte is read exactly once per pass, the token rows are tiny.  The
// kernel therefore exists to keep the memory system full:
//   * persistent grid (two CTAs per SM), work = (128-row weight tile, 64-wide k block) units
//     dealt out as one contiguous, equal range per CTA ("stream-K"), so every SM streams the
//     same number of bytes whatever R and K are;
//   * a 4-stage TMA ring per CTA (16 KB weight tile + 4 KB token tile per stage, 128-byte swizzle)
//     fed by one producer thread; nothing but mbarriers between HBM and the tensor core;
//   * tcgen05.mma with the weight tile as the 128-row A operand and the token rows as the
//     32-column B operand; fp32 accumulators in tensor memory, two buffers so the epilogue of
//     one segment overlaps the MMAs of the next;
//   * token rows are fp32 values split into two bf16 terms (hi + lo, rows 0..15 and 16..31 of
//     the B operand): products are exact, accumulation is fp32, and the result equals an fp32
//     activation times a bf16 weight to about 2^-17 relative.  The extra columns cost tensor
//     time only, which this kernel has to spare.
// Each segment (part of one tile's k range done by one CTA) is written as an fp32 partial
// block (numbered cta + tile); consumers add the blocks of a tile in CTA order, so results are bit-reproducible and do
// not depend on M.
//
// Every wait is bounded: on expiry the thread raises the error word, the CTA drains its
// outstanding TMA copies (bounded as well), frees its tensor memory and returns.
#include <cuda.h>

#include "common.cuh"
#include "kernels.cuh"
#include "tc_ptx.cuh"

namespace eesd {

namespace tc {

constexpr int BM = 128, BK = 64, BN = 32;
constexpr int STAGES = 4;   // per CTA; two CTAs share an SM (measured: 2 x 4 stages beat 1 x 8 by 1.8 % of a 13B pass, 3 x 3 and 2 x 3 do not)
constexpr int STAGE_W = BM * BK * 2, STAGE_X = BN * BK * 2;
constexpr int STAGE_BYTES = STAGE_W + STAGE_X;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;
constexpr int THREADS = 192;  // warps 0-3 epilogue, warp 4 TMA producer, warp 5 MMA issuer
constexpr uint32_t TMEM_COLS = 64;   // two 128 x 32 fp32 accumulators
// The tensor core adds into its fp32 accumulator with truncation, so a long chain of MMAs
// drifts towards zero.  Chains are therefore cut after KSEG k blocks (4 * KSEG MMAs): the
// epilogue warps drain the accumulator and carry the sum in registers with IEEE fp32 adds.
constexpr int KSEG = 16;

// instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = 32
constexpr uint32_t IDESC = idesc_bf16(BN);

__global__ void __launch_bounds__(THREADS, 2)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
               float *__restrict__ part, StreamK sk, int M, int tiled, int *err, uint32_t spin) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *sbase = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *sW = sbase;
    uint8_t *sX = sbase + STAGES * STAGE_W;
    uint64_t *full = (uint64_t *)(sbase + STAGES * STAGE_BYTES);
    uint64_t *empty = full + STAGES;
    uint64_t *acc_full = empty + STAGES;   // [2]
    uint64_t *acc_empty = acc_full + 2;    // [2]
    uint32_t *tmem_slot = (uint32_t *)(acc_empty + 2);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x;
    const int u0 = sk.start(cta), u1 = sk.start(cta + 1);
    int issued = 0;   // producer thread: stages requested so far
    pdl_trigger();

    if (tid == 0) {
        for (int i = 0; i < STAGES; i++) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
        for (int i = 0; i < 2; i++) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], 4); }
        *abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 5) {
        tmem_alloc(tmem_slot, TMEM_COLS);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 4) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            // The weights do not depend on the kernel before this one: fill the ring with weight
            // tiles at once, and only then wait for the producer of the token rows.
            const uint64_t stream_once = policy_evict_first();
            const int pre = min(u1 - u0, STAGES);
            for (int i = 0; i < pre; i++) {
                const int u = u0 + i, tile = u / sk.KB, kb = u - tile * sk.KB;
                mbar_expect_tx(&full[i], STAGE_BYTES);
                tma_load_2d_hint(sW + i * STAGE_W, &tmW, &full[i], tiled ? 0 : kb * BK, tiled ? (tile * sk.KB + kb) * BM : tile * BM, stream_once);
            }
            pdl_wait();
            for (int i = 0; i < pre; i++) {
                const int u = u0 + i, kb = u % sk.KB;
                tma_load_2d(sX + i * STAGE_X, &tmX, &full[i], kb * BK, 0);
            }
            issued = pre;
            bool ok = true;
            for (int u = u0 + pre; u < u1 && ok; u++, issued++) {
                const int s = issued % STAGES, round = issued / STAGES;
                ok = mbar_wait(&empty[s], (round & 1) ^ 1, abort_flag, spin);
                if (!ok) break;
                const int tile = u / sk.KB, kb = u - tile * sk.KB;
                mbar_expect_tx(&full[s], STAGE_BYTES);
                tma_load_2d_hint(sW + s * STAGE_W, &tmW, &full[s], tiled ? 0 : kb * BK, tiled ? (tile * sk.KB + kb) * BM : tile * BM, stream_once);
                tma_load_2d(sX + s * STAGE_X, &tmX, &full[s], kb * BK, 0);
            }
        }
    } else if (warp == 5) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            int it = 0, sub = 0;   // sub: accumulator chains started so far (buffer = sub & 1)
            bool ok = true;
            for (int u = u0; u < u1 && ok;) {
                const int tile = u / sk.KB;
                const int u_end = min(u1, (tile + 1) * sk.KB);
                for (int c0 = u; c0 < u_end && ok; c0 += KSEG, sub++) {
                    const int c1 = min(u_end, c0 + KSEG);
                    const int b = sub & 1, use = sub >> 1;
                    ok = mbar_wait(&acc_empty[b], (use & 1) ^ 1, abort_flag, spin);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t d_addr = tmem_base + (uint32_t)(b * BN);
                    for (int uu = c0; uu < c1; uu++, it++) {
                        const int s = it % STAGES, round = it / STAGES;
                        ok = mbar_wait(&full[s], round & 1, abort_flag, spin);
                        if (!ok) break;
                        tc_fence_after();
                        const uint64_t da = smem_desc_sw128(smem_u32(sW + s * STAGE_W));
                        const uint64_t db = smem_desc_sw128(smem_u32(sX + s * STAGE_X));
#pragma unroll
                        for (int j = 0; j < BK / 16; j++)
                            mma_bf16(d_addr, da + (uint64_t)(j * 2), db + (uint64_t)(j * 2), IDESC, (uu > c0 || j > 0) ? 1u : 0u);
                        mma_commit(&empty[s]);   // the stage may be refilled once these MMAs have read it
                    }
                    if (!ok) break;
                    mma_commit(&acc_full[b]);    // chain complete
                }
                u = u_end;
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue (warps 0-3)
        pdl_wait();   // the partial-sum buffer may still be read by the kernel before this one
        int sub = 0;
        bool ok = true;
        for (int u = u0; u < u1 && ok;) {
            const int tile = u / sk.KB;
            const int u_end = min(u1, (tile + 1) * sk.KB);
            float acc[kMaxRows];
#pragma unroll
            for (int m = 0; m < kMaxRows; m++) acc[m] = 0.f;
            for (int c0 = u; c0 < u_end; c0 += KSEG, sub++) {
                const int b = sub & 1, use = sub >> 1;
                ok = mbar_wait(&acc_full[b], use & 1, abort_flag, spin, 64);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                uint32_t r[32];
                tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(b * BN), r);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&acc_empty[b]);
#pragma unroll
                for (int m = 0; m < kMaxRows; m++) acc[m] += __uint_as_float(r[m]) + __uint_as_float(r[16 + m]);
            }
            if (!ok) break;
            float *dst = part + ((size_t)(cta + tile) * kMaxRows) * BM + warp * 32 + lane;
#pragma unroll
            for (int m = 0; m < kMaxRows; m++)
                if (m < M) dst[(size_t)m * BM] = acc[m];
            u = u_end;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {   // some wait gave up (every role has stopped by now)
        if (tid == 0) atomicOr(err, kErrWaitTimeout);
        // let every copy still in flight land before the CTA's shared memory is released
        if (warp == 4 && lane == 0)
            for (int i = issued > STAGES ? issued - STAGES : 0; i < issued; i++) mbar_drain(&full[i % STAGES], (uint32_t)((i / STAGES) & 1));
    }
    if (warp == 5) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}


// ------------------------------------------------------------------------------------------------
// Wide variant for prompt processing: up to 128 token rows per tile (256 operand columns: hi
// and lo terms), the whole k range per tile, result written directly as out[m][r] (fp32).
//
//   * tile = (128-row weight tile, 128-row token panel); tiles are dealt round-robin with the
//     panels of one weight tile adjacent, so CTAs running side by side share it through L2 and
//     the weights cross HBM once per pass over all panels;
//   * 4-stage ring of (16 KB weight tile + 32 KB token tile); the token tile is two boxes of a
//     4-D map over the [chunk][hi|lo][16][K] activation layout (8 chunks of 16 rows each);
//   * tcgen05.mma M = 128, N = 256, K = 16; two accumulators of 256 columns fill the tensor memory.
constexpr int WN = 256, WROWS = 128;               // operand columns / token rows per panel
constexpr int WSTAGES = 4;
constexpr int WSTAGE_X = WN * BK * 2, WSTAGE_BYTES = STAGE_W + WSTAGE_X;
constexpr int WSMEM_BYTES = WSTAGES * WSTAGE_BYTES + 1024 + 256;
constexpr uint32_t WTMEM_COLS = 512;
constexpr uint32_t IDESC_W = idesc_bf16(WN);

__global__ void __launch_bounds__(THREADS, 1)
gemm_wide_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
                 float *__restrict__ out, int R, int KB, int Mtot, int panels, int tiled, int S, size_t split_stride, int *err, uint32_t spin) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *sbase = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *sW = sbase;
    uint8_t *sX = sbase + WSTAGES * STAGE_W;
    uint64_t *full = (uint64_t *)(sbase + WSTAGES * WSTAGE_BYTES);
    uint64_t *empty = full + WSTAGES;
    uint64_t *acc_full = empty + WSTAGES;   // [2]
    uint64_t *acc_empty = acc_full + 2;     // [2]
    uint32_t *tmem_slot = (uint32_t *)(acc_empty + 2);
    volatile int *abort_flag = (volatile int *)(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // work item = (tile, k split): item t covers k blocks [ks * KBs, (ks + 1) * KBs) of tile t / S and
    // writes its sums to out + ks * split_stride (the consumers add the S results)
    const int KBs = KB / S;
    const int n_tiles = (R / BM) * panels * S;
    const int my_tiles = (n_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;   // items cta, cta + G, ...
    const int n_units = my_tiles * KBs;
    int issued = 0;   // producer thread: stages requested so far
    pdl_trigger();

    if (tid == 0) {
        for (int i = 0; i < WSTAGES; i++) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
        for (int i = 0; i < 2; i++) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], 4); }
        *abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 5) {
        tmem_alloc(tmem_slot, WTMEM_COLS);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 4) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            // unit i of this CTA -> (tile, k block)
            auto w_load = [&](int i, int s) {
                const int it = (int)blockIdx.x + (i / KBs) * (int)gridDim.x, t = it / S, kb = (it % S) * KBs + i % KBs;
                mbar_expect_tx(&full[s], WSTAGE_BYTES);
                tma_load_2d(sW + s * STAGE_W, &tmW, &full[s], tiled ? 0 : kb * BK, tiled ? ((t / panels) * KB + kb) * BM : (t / panels) * BM);
            };
            auto x_load = [&](int i, int s) {
                const int it = (int)blockIdx.x + (i / KBs) * (int)gridDim.x, t = it / S, kb = (it % S) * KBs + i % KBs;
                const int chunk0 = (t % panels) * (WROWS / 16);
                tma_load_4d(sX + s * WSTAGE_X, &tmX, &full[s], kb * BK, 0, 0, chunk0);
                tma_load_4d(sX + s * WSTAGE_X + WSTAGE_X / 2, &tmX, &full[s], kb * BK, 0, 1, chunk0);
            };
            const int pre = min(n_units, WSTAGES);
            for (int i = 0; i < pre; i++) w_load(i, i);   // weights do not depend on the previous kernel
            pdl_wait();
            for (int i = 0; i < pre; i++) x_load(i, i);
            issued = pre;
            for (; issued < n_units; issued++) {
                const int s = issued % WSTAGES, round = issued / WSTAGES;
                if (!mbar_wait(&empty[s], (round & 1) ^ 1, abort_flag, spin)) break;
                w_load(issued, s);
                x_load(issued, s);
            }
        }
    } else if (warp == 5) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            int it = 0, sub = 0;
            bool ok = true;
            for (int seg = 0; seg < my_tiles && ok; seg++) {
                for (int c0 = 0; c0 < KBs && ok; c0 += KSEG, sub++) {
                    const int c1 = min(KBs, c0 + KSEG);
                    const int b = sub & 1, use = sub >> 1;
                    ok = mbar_wait(&acc_empty[b], (use & 1) ^ 1, abort_flag, spin);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t d_addr = tmem_base + (uint32_t)(b * WN);
                    for (int kb = c0; kb < c1; kb++, it++) {
                        const int s = it % WSTAGES, round = it / WSTAGES;
                        ok = mbar_wait(&full[s], round & 1, abort_flag, spin);
                        if (!ok) break;
                        tc_fence_after();
                        const uint64_t da = smem_desc_sw128(smem_u32(sW + s * STAGE_W));
                        const uint64_t db = smem_desc_sw128(smem_u32(sX + s * WSTAGE_X));
#pragma unroll
                        for (int j = 0; j < BK / 16; j++)
                            mma_bf16(d_addr, da + (uint64_t)(j * 2), db + (uint64_t)(j * 2), IDESC_W, (kb > c0 || j > 0) ? 1u : 0u);
                        mma_commit(&empty[s]);
                    }
                    if (!ok) break;
                    mma_commit(&acc_full[b]);
                }
            }
        }
    } else {
        // ---------------------------------------------------------------- epilogue (warps 0-3)
        pdl_wait();   // the output buffer may still be read by the kernel before this one
        bool ok = true;
        int sub = 0;
        for (int seg = 0; seg < my_tiles && ok; seg++) {
            const int it = (int)blockIdx.x + seg * (int)gridDim.x, t = it / S, ks = it % S, wt = t / panels, pn = t % panels;
            float acc[WROWS];   // this thread's weight row against the panel's 128 token rows
#pragma unroll
            for (int i = 0; i < WROWS; i++) acc[i] = 0.f;
            for (int c0 = 0; c0 < KBs; c0 += KSEG, sub++) {
                const int b = sub & 1, use = sub >> 1;
                ok = mbar_wait(&acc_full[b], use & 1, abort_flag, spin, 64);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(b * WN);
#pragma unroll
                for (int j = 0; j < WROWS / 32; j++) {
                    uint32_t v[32];
                    tmem_ld32(taddr + (uint32_t)(WROWS + j * 32), v);   // lo terms first: the smaller addend
#pragma unroll
                    for (int i = 0; i < 32; i++) acc[j * 32 + i] += __uint_as_float(v[i]);
                    tmem_ld32(taddr + (uint32_t)(j * 32), v);
#pragma unroll
                    for (int i = 0; i < 32; i++) acc[j * 32 + i] += __uint_as_float(v[i]);
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&acc_empty[b]);
            }
            if (!ok) break;
            float *dst = out + (size_t)ks * split_stride + (size_t)(pn * WROWS) * R + (size_t)wt * BM + warp * 32 + lane;
            const int rows_left = Mtot - pn * WROWS;
#pragma unroll
            for (int i = 0; i < WROWS; i++)
                if (i < rows_left) dst[(size_t)i * R] = acc[i];
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        if (tid == 0) atomicOr(err, kErrWaitTimeout);
        if (warp == 4 && lane == 0)
            for (int i = issued > WSTAGES ? issued - WSTAGES : 0; i < issued; i++) mbar_drain(&full[i % WSTAGES], (uint32_t)((i / WSTAGES) & 1));
    }
    if (warp == 5) {
        tc_fence_after();
        tmem_dealloc(tmem_base, WTMEM_COLS);
    }
}

}  // namespace tc

// ---------------------------------------------------------------------------------------- host side
typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                             const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeFn encode_fn() {
    // looked up once; the initialisation of a function-local static is thread-safe
    static const EncodeFn fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            return (EncodeFn)p;
        return (EncodeFn) nullptr;
    }();
    return fn;
}

bool tc_make_map(CUtensorMap *out, const void *base, int rows, int cols, int box_rows, bool tiled) {
    EncodeFn fn = encode_fn();
    if (!fn) return false;
    if (((uintptr_t)base & 15) || (cols % 8)) return false;
    // tile-major storage: [rows / 128][cols / 64] tiles of [128][64], each 16 KB contiguous; seen
    // by the copy engine as rows * cols / 64 rows of 64 elements, one box = one tile
    if (tiled && (box_rows != tc::BM || rows % tc::BM || cols % tc::BK)) return false;
    cuuint64_t dims[2] = {(cuuint64_t)(tiled ? tc::BK : cols), (cuuint64_t)(tiled ? (size_t)rows * cols / tc::BK : rows)};
    cuuint64_t strides[1] = {(cuuint64_t)(tiled ? tc::BK : cols) * 2};
    cuuint32_t box[2] = {(cuuint32_t)tc::BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides,
                    box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// 4-D map over token rows kept as [chunk][hi | lo][16][K] bf16; box = 64 k x 16 rows x 1 x 8 chunks
bool tc_make_map_rows(CUtensorMap *out, const void *base, int K, int chunks) {
    EncodeFn fn = encode_fn();
    if (!fn) return false;
    if (((uintptr_t)base & 15) || (K % 8)) return false;
    cuuint64_t dims[4] = {(cuuint64_t)K, 16, 2, (cuuint64_t)chunks};
    cuuint64_t strides[3] = {(cuuint64_t)K * 2, (cuuint64_t)K * 2 * 16, (cuuint64_t)K * 2 * 32};
    cuuint32_t box[4] = {(cuuint32_t)tc::BK, 16, 1, (cuuint32_t)(tc::WROWS / 16)};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides,
                    box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool tc_shape_ok(int R, int K) { return R > 0 && K > 0 && R % tc::BM == 0 && K % tc::BK == 0; }

StreamK tc_plan(int R, int K, int n_sm) {
    StreamK sk;
    sk.KB = K / tc::BK;
    sk.tiles = R / tc::BM;
    sk.U = sk.tiles * sk.KB;
    sk.G = sk.U < n_sm ? sk.U : n_sm;
    sk.base = sk.U / sk.G;
    sk.rem = sk.U % sk.G;
    return sk;
}

int tc_init() {
    // once per process, whichever host thread comes first (thread-safe static initialisation)
    static const int rc = [] {
        if (cudaFuncSetAttribute(tc::gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_BYTES) != cudaSuccess)
            return -1;
        if (cudaFuncSetAttribute(tc::gemm_wide_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::WSMEM_BYTES) != cudaSuccess)
            return -1;
        return encode_fn() ? 0 : -1;
    }();
    return rc;
}

void launch_gemm_tc(cudaStream_t s, const CUtensorMap &mW, const CUtensorMap &mX, float *part, const StreamK &sk,
                    int M, bool tiled, int *err, uint32_t wait_polls) {
    launch_k(tc::gemm_tc_kernel, dim3(sk.G), dim3(tc::THREADS), (size_t)tc::SMEM_BYTES, s, pdl_enabled(), mW, mX, part, sk, M,
             (int)tiled, err, wait_polls);
}

int gemm_wide_splits(int R, int K, int Mtot, int n_sm, int max_splits) {
    const int panels = (Mtot + tc::WROWS - 1) / tc::WROWS, tiles = (R / tc::BM) * panels, KB = K / tc::BK;
    int best = 1;
    double cost = 1e30;
    for (int S = 1; S <= max_splits && S <= 4; S++) {
        if (KB % S) continue;
        const int G = tiles * S < n_sm ? tiles * S : n_sm;
        const double c = (double)((tiles * S + G - 1) / G) / S + 0.02 * (S - 1);   // waves of 1/S of a tile, a little for each extra result
        if (c < cost - 1e-9) { cost = c; best = S; }
    }
    return best;
}

void launch_gemm_wide(cudaStream_t s, const CUtensorMap &mW, const CUtensorMap &mX, float *out, int R, int K, int Mtot,
                      int n_sm, bool tiled, int splits, int *err, uint32_t wait_polls) {
    const int panels = (Mtot + tc::WROWS - 1) / tc::WROWS;
    const int tiles = (R / tc::BM) * panels * splits;
    launch_k(tc::gemm_wide_kernel, dim3(tiles < n_sm ? tiles : n_sm), dim3(tc::THREADS), (size_t)tc::WSMEM_BYTES, s, pdl_enabled(),
             mW, mX, out, R, K / tc::BK, Mtot, panels, (int)tiled, splits, (size_t)Mtot * R, err, wait_polls);
}

// fp32 rows -> two bf16 terms: rows 0..15 hold hi = bf16(x), rows 16..31 hold lo = bf16(x - hi)
__global__ void split_rows_kernel(const float *x, __nv_bfloat16 *xs, int K) {
    const int m = blockIdx.y;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= K) return;
    const float v = x[(size_t)m * K + i];   // launched without early start: x is complete
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    xs[(size_t)m * K + i] = hi;
    xs[(size_t)(kMaxRows + m) * K + i] = __float2bfloat16_rn(v - __bfloat162float(hi));
}
void launch_split_rows(cudaStream_t s, const float *x, void *xs, int M, int K) {
    split_rows_kernel<<<dim3((K + 255) / 256, M), 256, 0, s>>>(x, (__nv_bfloat16 *)xs, K);
}

}  // namespace eesd
