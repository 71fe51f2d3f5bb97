// Fused vocabulary-wide softmax / speculative acceptance / residual resampling, and the
// draft-token sampler (sm_100a).
//
// The paper's verification keeps the output distribution of the target model ("lossless");
// the rule is the standard one: accept x_i iff u_i q_i(x_i) < p_i(x_i); at the first rejection
// j draw y ~ normalize(max(0, p_j - q_j)); otherwise y ~ p_{K+1}.  Greedy decoding (the
// paper's experiments): accept while x_i equals the target's top-1.
//
// Arithmetic contract (every fp32 operation rounds to nearest even; no contraction, no fast
// math).  It makes each decision a pure function of (logits, uniforms), whatever the
// reduction order, so any implementation of the contract yields the same bits:
//   m = max_v l_v;  t_v = (l_v - m) / T;  e_v = exp_c(t_v)
//   Z = sum_v trunc(e_v * 2^40) as a 64-bit integer;  Zf = float(Z) * 2^-40;  P_v = e_v / Zf
//   exp_c(t) = 0 for t < -64, else with n = rint(t * log2e): r = fma(-n, ln2_hi, t),
//   r = fma(-n, ln2_lo, r), degree-6 Horner polynomial 1 + r + r^2/2 + ... + r^6/720 in fma
//   form, times 2^n.  Constants are given as fp32 bit patterns below.
//   draw from weights w_v <= 1 with u = m_u 2^-24: W = sum_v trunc(w_v * 2^32) (64-bit),
//   tau = (m_u * W) >> 24, result = smallest v whose inclusive integer prefix sum exceeds tau.
#include <atomic>

#include "../../include/eesd.h"
#include "common.cuh"
#include "kernels.cuh"

namespace eesd {

constexpr int kAccThreads = 1024;

__device__ __forceinline__ float exp_c(float t) {
    if (!(t >= -64.0f)) return 0.0f;
    const float log2e = __uint_as_float(0x3FB8AA3Bu);
    const float ln2_hi = __uint_as_float(0x3F317200u);
    const float ln2_lo = __uint_as_float(0x35BFBE8Eu);
    const float n = rintf(__fmul_rn(t, log2e));
    float r = __fmaf_rn(-n, ln2_hi, t);
    r = __fmaf_rn(-n, ln2_lo, r);
    float p = __uint_as_float(0x3AB60B61u);               // 1/720
    p = __fmaf_rn(p, r, __uint_as_float(0x3C088889u));    // 1/120
    p = __fmaf_rn(p, r, __uint_as_float(0x3D2AAAABu));    // 1/24
    p = __fmaf_rn(p, r, __uint_as_float(0x3E2AAAABu));    // 1/6
    p = __fmaf_rn(p, r, 0.5f);
    p = __fmaf_rn(p, r, 1.0f);
    p = __fmaf_rn(p, r, 1.0f);
    return __fmul_rn(p, __int_as_float(((int)n + 127) << 23));
}

// (x / 1 is x exactly, so the division is skipped at T = 1 without changing a bit)
__device__ __forceinline__ float expo(float l, float m, float T) {
    const float d = __fsub_rn(l, m);
    return exp_c(T == 1.0f ? d : __fdiv_rn(d, T));
}
__device__ __forceinline__ unsigned long long fix40(float e) { return __float2ull_rz(__fmul_rn(e, 1099511627776.0f)); }
__device__ __forceinline__ unsigned long long fix32(float w) { return __float2ull_rz(__fmul_rn(w, 4294967296.0f)); }
__device__ __forceinline__ float z_to_float(unsigned long long Z) {
    return __fmul_rn(__ull2float_rn(Z), 1.0f / 1099511627776.0f);
}

struct __align__(16) RowStat {
    float m;                 // max logit
    int arg;                 // lowest index attaining it
    unsigned long long Z;    // integer normaliser
};

// read a RowStat written by another block (bypasses L1)
__device__ __forceinline__ RowStat ld_stat(const RowStat *p) {
    int4 raw = __ldcg(reinterpret_cast<const int4 *>(p));
    RowStat r;
    r.m = __int_as_float(raw.x);
    r.arg = raw.y;
    r.Z = ((unsigned long long)(unsigned int)raw.w << 32) | (unsigned int)raw.z;
    return r;
}

// ---- block-wide helpers (blockDim.x == kAccThreads) -----------------------------------------------
__device__ __forceinline__ void block_argmax(float &v, int &idx, float *sv, int *si) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        float ov = __shfl_xor_sync(0xffffffffu, v, o);
        int oi = __shfl_xor_sync(0xffffffffu, idx, o);
        if (ov > v || (ov == v && oi < idx)) { v = ov; idx = oi; }
    }
    __syncthreads();
    if (lane == 0) { sv[warp] = v; si[warp] = idx; }
    __syncthreads();
    if (warp == 0) {
        v = sv[lane]; idx = si[lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            float ov = __shfl_xor_sync(0xffffffffu, v, o);
            int oi = __shfl_xor_sync(0xffffffffu, idx, o);
            if (ov > v || (ov == v && oi < idx)) { v = ov; idx = oi; }
        }
        if (lane == 0) { sv[0] = v; si[0] = idx; }
    }
    __syncthreads();
    v = sv[0]; idx = si[0];
    __syncthreads();
}

__device__ __forceinline__ unsigned long long block_sum_u64(unsigned long long v, unsigned long long *s64) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if (lane == 0) s64[warp] = v;
    __syncthreads();
    if (warp == 0) {
        v = s64[lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) s64[32] = v;
    }
    __syncthreads();
    v = s64[32];
    __syncthreads();
    return v;
}

// exclusive prefix of one value per thread; *total receives the block sum
__device__ __forceinline__ unsigned long long block_excl_scan_u64(unsigned long long v, unsigned long long *s64,
                                                                  unsigned long long *total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        unsigned long long t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    __syncthreads();
    if (lane == 31) s64[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        unsigned long long w = s64[lane], winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            unsigned long long t = __shfl_up_sync(0xffffffffu, winc, o);
            if (lane >= o) winc += t;
        }
        s64[lane] = winc - w;  // exclusive prefix of the warp sums
        if (lane == 31) s64[32] = winc;
    }
    __syncthreads();
    const unsigned long long res = s64[warp] + inc - v;
    *total = s64[32];
    __syncthreads();
    return res;
}

struct AccSmem {
    float sv[32];
    int si[32];
    unsigned long long s64[33];
    int found;
};

// max / argmax / integer normaliser of one row.  Rows of up to kRegRow logits (16-byte aligned,
// V % 4 == 0) are read from memory ONCE, eight 16-byte loads per thread all in flight, and both
// passes (maximum, then the integer normaliser) run from registers; other rows take two passes
// over memory.  Every sum is an exact integer sum, so the result does not depend on the path.
constexpr int kRegVec = 8;                              // float4 per thread held in registers
constexpr int kRegRow = kAccThreads * kRegVec * 4;      // 32768 logits
__device__ RowStat row_stat(const float *l, int V, float T, bool need_z, AccSmem &sm) {
    RowStat st;
    if (V <= kRegRow && (V & 3) == 0 && ((uintptr_t)l & 15) == 0) {
        const int nv = V >> 2;
        float4 x[kRegVec];
#pragma unroll
        for (int k = 0; k < kRegVec; k++) {
            const int i = threadIdx.x + k * kAccThreads;
            x[k] = i < nv ? __ldcs(reinterpret_cast<const float4 *>(l) + i) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        }
        float v = -INFINITY;
        int idx = 0x7fffffff;
#pragma unroll
        for (int k = 0; k < kRegVec; k++) {   // ascending index within the thread: strict > keeps the lowest
            const int i4 = (threadIdx.x + k * kAccThreads) * 4;
            if (x[k].x > v) { v = x[k].x; idx = i4; }
            if (x[k].y > v) { v = x[k].y; idx = i4 + 1; }
            if (x[k].z > v) { v = x[k].z; idx = i4 + 2; }
            if (x[k].w > v) { v = x[k].w; idx = i4 + 3; }
        }
        block_argmax(v, idx, sm.sv, sm.si);
        st.m = v; st.arg = idx; st.Z = 0;
        if (need_z) {
            unsigned long long z = 0;
#pragma unroll
            for (int k = 0; k < kRegVec; k++) {
                if (threadIdx.x + k * kAccThreads < nv)
                    z += fix40(expo(x[k].x, v, T)) + fix40(expo(x[k].y, v, T)) + fix40(expo(x[k].z, v, T)) + fix40(expo(x[k].w, v, T));
            }
            st.Z = block_sum_u64(z, sm.s64);
        }
        return st;
    }
    float v = -INFINITY;
    int idx = 0x7fffffff;
    for (int i = threadIdx.x; i < V; i += blockDim.x) {
        float x = l[i];
        if (x > v) { v = x; idx = i; }
    }
    block_argmax(v, idx, sm.sv, sm.si);
    st.m = v; st.arg = idx; st.Z = 0;
    if (need_z) {
        unsigned long long z = 0;
        for (int i = threadIdx.x; i < V; i += blockDim.x) z += fix40(expo(l[i], v, T));
        st.Z = block_sum_u64(z, sm.s64);
    }
    return st;
}

__device__ __forceinline__ float prob_of(float l, const RowStat &st, float T) {
    return __fdiv_rn(expo(l, st.m, T), z_to_float(st.Z));
}

// weight of vocabulary entry v: the target probability (lq == nullptr) or the positive part of
// the difference of target and draft probabilities
__device__ __forceinline__ float weight_of(int v, const float *lp, const RowStat &sp, const float *lq,
                                           const RowStat &sq, float T) {
    float p = prob_of(lp[v], sp, T);
    if (!lq) return p;
    float r = __fsub_rn(p, prob_of(lq[v], sq, T));
    return r > 0.0f ? r : 0.0f;
}

// inverse-CDF draw over the whole block; returns -1 when every weight truncates to zero.
// Warp w owns the contiguous entries [w * chunk, (w + 1) * chunk) and walks them 32 at a time
// (lane = entry within the group: coalesced reads); the warp that holds tau walks its chunk
// once more with an inclusive scan per group to find the entry.
__device__ int block_draw(const float *lp, const RowStat &sp, const float *lq, const RowStat &sq, float T,
                          int V, float u, AccSmem &sm) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
    const int chunk = ((V + nwarp - 1) / nwarp + 31) & ~31;   // a multiple of 32 entries per warp
    const int lo = min(V, warp * chunk), hi = min(V, lo + chunk);
    unsigned long long mine = 0;
    for (int v = lo + lane; v < hi; v += 32) mine += fix32(weight_of(v, lp, sp, lq, sq, T));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);   // the warp's total, in every lane
    __syncthreads();
    if (lane == 0) sm.s64[warp] = mine;
    if (threadIdx.x == 0) sm.found = -1;
    __syncthreads();
    unsigned long long off = 0, W = 0;
    for (int w = 0; w < nwarp; w++) {   // 32 values from shared memory: exclusive prefix and total
        const unsigned long long t = sm.s64[w];
        if (w < warp) off += t;
        W += t;
    }
    if (W != 0) {
        const unsigned long long mu = __float2ull_rz(__fmul_rn(u, 16777216.0f));
        const unsigned long long tau = (mu * W) >> 24;
        if (off <= tau && tau < off + mine) {   // warp-uniform
            unsigned long long acc = off;
            for (int base = lo; base < hi; base += 32) {
                const int v = base + lane;
                const unsigned long long w = v < hi ? fix32(weight_of(v, lp, sp, lq, sq, T)) : 0ull;
                unsigned long long inc = w;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const unsigned long long t = __shfl_up_sync(0xffffffffu, inc, o);
                    if (lane >= o) inc += t;
                }
                const unsigned int hit = __ballot_sync(0xffffffffu, acc + inc > tau);
                if (hit) {
                    if (lane == 0) sm.found = base + __ffs(hit) - 1;   // smallest entry whose inclusive prefix exceeds tau
                    break;
                }
                acc += __shfl_sync(0xffffffffu, inc, 31);
            }
        }
    }
    __syncthreads();
    const int res = sm.found;
    __syncthreads();
    return res;
}

// ---- accept kernel -------------------------------------------------------------------------------
// scratch: one 32-bit arrival counter per sequence (zero on entry, reset to zero by the
// finishing block; at the start so its place does not move with K), then per sequence
// RowStat[2K+1] (p rows 0..K, then q rows 0..K-1).
// grid = B * (2K+1) blocks.  Each block computes the statistics of one row; the block that
// arrives last for its sequence runs the acceptance tests and the draw.
__global__ void __launch_bounds__(kAccThreads) accept_kernel(const float *p_logits, const float *q_logits,
                                                             const int32_t *tokens, const float *u_acc,
                                                             const float *u_res, int K, int V, float T,
                                                             RowStat *stats, unsigned int *counters,
                                                             int32_t *n_acc, int32_t *y, int32_t *pending_out, int tok_stride) {
    __shared__ AccSmem sm;
    __shared__ int s_last, s_j;
    const int rows = 2 * K + 1;
    const int b = blockIdx.x / rows, row = blockIdx.x % rows;
    const bool greedy = (T == 0.0f);
    const float *pl = p_logits + (size_t)b * (K + 1) * V;
    const float *ql = q_logits + (size_t)b * K * V;
    RowStat *st = stats + (size_t)b * rows;

    if (!(greedy && row > K)) {
        const float *l = row <= K ? pl + (size_t)row * V : ql + (size_t)(row - K - 1) * V;
        RowStat r = row_stat(l, V, greedy ? 1.0f : T, !greedy, sm);
        if (threadIdx.x == 0) st[row] = r;
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned int prev = atomicAdd(&counters[b], 1u);
        s_last = (prev == (unsigned int)rows - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    const int32_t *x = tokens + (size_t)b * tok_stride;   // the sequence's K drafted tokens
    __shared__ int s_ok[EESD_MAX_ROWS];
    if ((int)threadIdx.x < K && K <= EESD_MAX_ROWS) {   // one test per thread: their loads are in flight together
        const int j = threadIdx.x, t = x[j];
        bool ok;
        if (t < 0 || t >= V) {   // not a token of this vocabulary: rejected where it stands, no address is formed
            ok = false;
        } else if (greedy) {
            ok = t == ld_stat(&st[j]).arg;
        } else {
            const float p = prob_of(pl[(size_t)j * V + t], ld_stat(&st[j]), T);
            const float q = prob_of(ql[(size_t)j * V + t], ld_stat(&st[K + 1 + j]), T);
            ok = __fmul_rn(u_acc[(size_t)b * K + j], q) < p;
        }
        s_ok[j] = ok;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int j = 0;
        if (K <= EESD_MAX_ROWS) {
            while (j < K && s_ok[j]) j++;
        } else if (greedy) {
            while (j < K && x[j] == ld_stat(&st[j]).arg) j++;
        } else {
            for (; j < K; j++) {
                const int t = x[j];
                if (t < 0 || t >= V) break;
                const float p = prob_of(pl[(size_t)j * V + t], ld_stat(&st[j]), T);
                const float q = prob_of(ql[(size_t)j * V + t], ld_stat(&st[K + 1 + j]), T);
                if (!(__fmul_rn(u_acc[(size_t)b * K + j], q) < p)) break;
            }
        }
        s_j = j;
        counters[b] = 0;
    }
    __syncthreads();
    const int j = s_j;
    int tok;
    if (greedy) {
        tok = ld_stat(&st[j]).arg;
    } else {
        const RowStat sp = ld_stat(&st[j]);
        const float *lp = pl + (size_t)j * V;
        const float u = u_res[b];
        if (j == K) {
            tok = block_draw(lp, sp, nullptr, sp, T, V, u, sm);
        } else {
            tok = block_draw(lp, sp, ql + (size_t)j * V, ld_stat(&st[K + 1 + j]), T, V, u, sm);
            if (tok < 0) tok = block_draw(lp, sp, nullptr, sp, T, V, u, sm);  // p == q to the last bit
        }
    }
    if (threadIdx.x == 0) {
        n_acc[b] = j;
        y[b] = tok;
        if (pending_out) pending_out[b] = tok;
    }
}

size_t accept_scratch_bytes(int B, int K) {
    size_t counters = ((size_t)B * sizeof(unsigned int) + 15) / 16 * 16;
    return counters + (size_t)B * (2 * K + 1) * sizeof(RowStat);
}

void launch_accept(cudaStream_t s, const float *p_logits, const float *q_logits, const int32_t *tokens,
                   const float *u_acc, const float *u_res, int B, int K, int V, float T, void *scratch,
                   int32_t *n_acc, int32_t *y, int32_t *pending_out, int tok_stride) {
    unsigned int *counters = (unsigned int *)scratch;
    RowStat *stats = (RowStat *)((char *)scratch + ((size_t)B * sizeof(unsigned int) + 15) / 16 * 16);
    accept_kernel<<<B * (2 * K + 1), kAccThreads, 0, s>>>(p_logits, q_logits, tokens, u_acc, u_res, K, V, T,
                                                         stats, counters, n_acc, y, pending_out, tok_stride ? tok_stride : K);
}

// ---- draft-token sampler -------------------------------------------------------------------------
__global__ void __launch_bounds__(kAccThreads) sample_rows_kernel(const float *logits, const float *u, int V, float T,
                                                                  int32_t *out, size_t logit_stride, int out_stride) {
    __shared__ AccSmem sm;
    const int b = blockIdx.x;
    const float *l = logits + (size_t)b * logit_stride;
    const bool greedy = (T == 0.0f);
    pdl_trigger();   // (programmatic dependent launch: resident early, reads the logits only once their producer is done)
    pdl_wait();
    RowStat st = row_stat(l, V, greedy ? 1.0f : T, !greedy, sm);
    int tok = st.arg;
    if (!greedy) tok = block_draw(l, st, nullptr, st, T, V, u[b], sm);
    if (threadIdx.x == 0) out[(size_t)b * out_stride] = tok;
}

void launch_sample_rows(cudaStream_t s, const float *logits, const float *u, int B, int V, float T, int32_t *out,
                        size_t logit_stride, int out_stride) {
    launch_k(sample_rows_kernel, dim3(B), dim3(kAccThreads), 0, s, pdl_enabled(), logits, u, V, T, out, logit_stride ? logit_stride : (size_t)V,
             out_stride);
}

}  // namespace eesd

// ---- acceptance without any caller-provided or allocated scratch ------------------------------------
// Library-owned scratch for eesd_accept_resample_static: lives in every GPU context that loads
// this library, from load to exit.  Sized for EESD_STATIC_ACCEPT_MAX_ROWS logit rows
// (B * (2K + 1)) and EESD_STATIC_ACCEPT_MAX_BATCH sequences.
static __device__ __align__(256) unsigned char g_static_accept_scratch
    [((EESD_STATIC_ACCEPT_MAX_BATCH * sizeof(unsigned int) + 15) / 16) * 16 + EESD_STATIC_ACCEPT_MAX_ROWS * sizeof(eesd::RowStat)];

extern "C" int eesd_accept_resample_static(void *cuda_stream, const float *p_logits, const float *q_logits,
                                           const int32_t *tokens, const float *u_accept, const float *u_resample,
                                           int B, int K, int V, float temperature, int32_t *n_accept,
                                           int32_t *next_token) {
    if (!p_logits || !q_logits || !tokens || !n_accept || !next_token) return EESD_ERR_BADARG;
    if (B < 1 || K < 1 || V < 1 || temperature < 0.f) return EESD_ERR_BADARG;
    if (temperature != 0.f && (!u_accept || !u_resample)) return EESD_ERR_RNG;
    if (B > EESD_STATIC_ACCEPT_MAX_BATCH || (long long)B * (2 * K + 1) > EESD_STATIC_ACCEPT_MAX_ROWS)
        return EESD_ERR_NOMEM;   // beyond the built-in scratch: use eesd_accept_resample with caller scratch
    // The array's name is only a host-side handle; the device address is looked up once per
    // device (with that device current) and remembered.
    // Threads may race to fill a slot: they store the same address (atomically), so any order is
    // fine.  The address belongs to the device's primary context and holds for its lifetime.
    constexpr int kMaxDevices = 64;
    static std::atomic<void *> dev_ptr[kMaxDevices];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return EESD_ERR_CUDA;
    void *scratch = dev_ptr[dev].load(std::memory_order_acquire);
    if (!scratch) {
        if (cudaGetSymbolAddress(&scratch, g_static_accept_scratch) != cudaSuccess || !scratch) return EESD_ERR_CUDA;
        dev_ptr[dev].store(scratch, std::memory_order_release);
    }
    cudaStream_t s = (cudaStream_t)cuda_stream;
    // the arrival counters must start at zero; the row statistics are overwritten before use
    if (cudaMemsetAsync(scratch, 0, (size_t)B * sizeof(unsigned int), s) != cudaSuccess) return EESD_ERR_CUDA;
    eesd::launch_accept(s, p_logits, q_logits, tokens, u_accept, u_resample, B, K, V, temperature, scratch,
                        n_accept, next_token, nullptr);
    return cudaGetLastError() == cudaSuccess ? EESD_OK : EESD_ERR_CUDA;
}

