// disc_topm: the M most probable tokens of every row (Algorithm 2, line 3), i.e. the M largest
// logits, by an exact radix selection; and, as a by-product of the same passes, the row's sum over
// the whole vocabulary as a pair (m, s) with sum_v 2^(z_v log2e / T) = 2^m * s.
//
// One block of 256 threads per row.  A logit is mapped to a 32-bit key whose unsigned order is the
// order of the values (NaN lowest); the key of the M-th largest logit is found eleven bits at a
// time (a 2048-bin histogram in shared memory of the next bits among the keys that match the bits
// found so far - wide enough that logits of one row seldom meet in a bin; bf16 keys take two such
// passes, fp32 keys three).  A last pass writes out, in ascending token id, every
// token whose key is larger, and of the tokens whose key is equal the lowest ids until M are
// filled: equal logits are common in bf16, and the rule "the lower id first" makes the selection
// unique.  Every pass streams the row again; after the first it comes from L2.

#include <math_constants.h>

#include "disc_internal.cuh"

namespace {

constexpr int TOPM_THREADS = 256;
constexpr int TOPM_WARPS = TOPM_THREADS / 32;
constexpr unsigned FULL = 0xffffffffu;
constexpr float LOG2E_F = 1.4426950408889634f;

struct TopmParams {
    const void* logits;
    int64_t ld;
    int32_t V, M;
    float c2;
    const uint8_t* done;     // nullable: rows with done != 0 are skipped
    int32_t* cand;           // [n][M]
    float2* lse;             // [n] (nullable)
};

__device__ __forceinline__ uint32_t order_key(float x) {
    if (x != x) return 0u;
    const uint32_t b = __float_as_uint(x);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int DT>
struct Row {
    static constexpr int EPV = DT == DISC_BF16 ? 8 : 4;
    // element e of the row as fp32
    __device__ static __forceinline__ float at(const void* base, int e) {
        if (DT == DISC_BF16) return __uint_as_float(uint32_t(__ldg(static_cast<const unsigned short*>(base) + e)) << 16);
        return __ldg(static_cast<const float*>(base) + e);
    }
    // EPV consecutive elements starting at e (e a multiple of EPV, row 16-byte aligned)
    __device__ static __forceinline__ void vec(const void* base, int e, float* x) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(static_cast<const char*>(base) + size_t(e) * (DT == DISC_BF16 ? 2 : 4)));
        if (DT == DISC_BF16) {
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) { x[2 * j] = __uint_as_float(w[j] << 16); x[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u); }
        } else {
            x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y); x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
        }
    }
};

// Calls f(element index, value) for the elements of the row this thread owns: thread t takes the
// EPV consecutive elements t*EPV.. of every chunk of 256*EPV, so that (chunk, thread, element) is
// the order of the token ids.
template <int DT, bool VEC, class F>
__device__ __forceinline__ void for_row(const void* rowp, int V, F f) {
    constexpr int EPV = Row<DT>::EPV;
    constexpr int CHUNK = TOPM_THREADS * EPV;
    for (int c0 = 0; c0 < V; c0 += CHUNK) {
        const int e0 = c0 + threadIdx.x * EPV;
        float x[EPV];
        if (VEC && e0 + EPV <= V) Row<DT>::vec(rowp, e0, x);
        else {
#pragma unroll
            for (int j = 0; j < EPV; ++j) x[j] = (e0 + j < V) ? Row<DT>::at(rowp, e0 + j) : 0.f;
        }
        f(c0, e0, x);
    }
}

constexpr int RADIX_BITS = 11;
constexpr int BINS = 1 << RADIX_BITS;
constexpr int BINS_PER_THREAD = BINS / TOPM_THREADS;

template <int DT, bool VEC>
__global__ void __launch_bounds__(TOPM_THREADS) disc_topm_kernel(const TopmParams p) {
    constexpr int EPV = Row<DT>::EPV;
    constexpr int PASSES = DT == DISC_BF16 ? 2 : 3;
    __shared__ unsigned int hist[BINS];
    __shared__ unsigned int s_prefix, s_remaining;
    __shared__ float s_red[TOPM_WARPS];
    __shared__ unsigned int s_wsum[TOPM_WARPS];
    __shared__ int s_scan[TOPM_WARPS][2];
    __shared__ int s_flag;
    const int64_t row = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int32_t* out = p.cand + size_t(row) * p.M;
    if (p.done && p.done[row]) {
        for (int m = tid; m < p.M; m += TOPM_THREADS) out[m] = -1;
        if (p.lse && tid == 0) p.lse[row] = make_float2(-CUDART_INF_F, 0.f);
        return;
    }
    const char* rowp = static_cast<const char*>(p.logits) + size_t(row) * size_t(p.ld) * (DT == DISC_BF16 ? 2 : 4);
    const int want = min(p.M, p.V);
    if (tid == 0) { s_prefix = 0u; s_remaining = unsigned(want); s_flag = 0; }

    float row_max = -CUDART_INF_F;     // over the values that are not NaN
    float sum = 0.f;
    for (int pass = 0; pass < PASSES; ++pass) {
        for (int b = tid; b < BINS; b += TOPM_THREADS) hist[b] = 0u;
        __syncthreads();
        // the window of key bits this pass looks at: [shift, shift + width)
        const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
        const int width = pass == 2 ? 10 : 11;
        const uint32_t prefix = s_prefix;
        const float ref = (fabsf(row_max) < CUDART_INF_F) ? row_max * p.c2 : 0.f;
        float mx = -CUDART_INF_F;
        int nan_seen = 0;
        for_row<DT, VEC>(rowp, p.V, [&](int, int e0, const float* x) {
#pragma unroll
            for (int j = 0; j < EPV; ++j) {
                if (e0 + j < p.V) {
                    const uint32_t key = order_key(x[j]);
                    // the bits above the window must match what earlier passes found
                    if (pass == 0 || (key >> (shift + width)) == (prefix >> (shift + width)))
                        atomicAdd(&hist[(key >> shift) & ((1u << width) - 1u)], 1u);
                    if (pass == 0) { if (x[j] != x[j]) nan_seen = 1; else mx = fmaxf(mx, x[j]); }
                    else if (pass == 1) sum += ex2_approx(fmaf(x[j], p.c2, -ref));
                }
            }
        });
        if (pass == 0) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, o));
            if (lane == 0) s_red[warp] = mx;
            if (nan_seen) s_flag = 1;
        }
        __syncthreads();
        if (pass == 0) {
            row_max = s_red[0];
#pragma unroll
            for (int w2 = 1; w2 < TOPM_WARPS; ++w2) row_max = fmaxf(row_max, s_red[w2]);
        }
        // From the largest bin down: the bin that holds the `remaining`-th largest key.  Thread t
        // owns the bins [t*8, t*8+8); `above` = keys in the bins of higher threads.
        {
            const unsigned int rem = s_remaining;
            unsigned int mine = 0;
#pragma unroll
            for (int b = 0; b < BINS_PER_THREAD; ++b) mine += hist[tid * BINS_PER_THREAD + b];
            unsigned int incl = mine;                           // suffix sum over the lanes of the warp
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned int v = __shfl_down_sync(FULL, incl, o);
                if (lane + o < 32) incl += v;
            }
            if (lane == 0) s_wsum[warp] = incl;
            __syncthreads();
            unsigned int above = incl - mine;
            for (int w2 = warp + 1; w2 < TOPM_WARPS; ++w2) above += s_wsum[w2];
            __syncthreads();
            if (above < rem && above + mine >= rem) {           // exactly one thread
                unsigned int left = rem - above;
                int b = BINS_PER_THREAD - 1;
                for (; b > 0; --b) {
                    const unsigned int cnt = hist[tid * BINS_PER_THREAD + b];
                    if (cnt >= left) break;
                    left -= cnt;
                }
                s_prefix = prefix | (uint32_t(tid * BINS_PER_THREAD + b) << shift);
                s_remaining = left;
            }
        }
        __syncthreads();
    }
    if (p.lse) {
        // the row's sum over the whole vocabulary, 2^m * s (NaN or +Inf among the logits poison s)
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(FULL, sum, o);
        __syncthreads();
        if (lane == 0) s_red[warp] = sum;
        __syncthreads();
        if (tid == 0) {
            float s = 0.f;
            for (int w2 = 0; w2 < TOPM_WARPS; ++w2) s += s_red[w2];
            const bool fin = fabsf(row_max) < CUDART_INF_F;
            if (s_flag || row_max == CUDART_INF_F) s = CUDART_NAN_F;
            p.lse[row] = make_float2(row_max == -CUDART_INF_F ? -CUDART_INF_F : (fin ? row_max * p.c2 : 0.f),
                                     row_max == -CUDART_INF_F ? 0.f : s);
        }
    }

    // ---- write-out in ascending token id: keys above the threshold, then the lowest ids among the
    // keys equal to it until `want` are filled
    const uint32_t thr = s_prefix;
    const int take_eq = int(s_remaining);
    int gt_total = 0, eq_total = 0;
    for_row<DT, VEC>(rowp, p.V, [&](int, int e0, const float* x) {
        int gt = 0, eq = 0;
        uint32_t fl_gt = 0u, fl_eq = 0u;
#pragma unroll
        for (int j = 0; j < EPV; ++j) {
            if (e0 + j < p.V) {
                uint32_t key = order_key(x[j]);
                if (DT == DISC_BF16) key &= 0xfffffc00u;      // the passes looked at bits 31..10; the rest is constant for bf16
                if (key > thr) { ++gt; fl_gt |= 1u << j; }
                else if (key == thr) { ++eq; fl_eq |= 1u << j; }
            }
        }
        // exclusive counts over the threads of the block (ids ascend with the thread index)
        int sg = gt, se = eq;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int a = __shfl_up_sync(FULL, sg, o), b = __shfl_up_sync(FULL, se, o);
            if (lane >= o) { sg += a; se += b; }
        }
        __syncthreads();
        if (lane == 31) { s_scan[warp][0] = sg; s_scan[warp][1] = se; }
        __syncthreads();
        int bg = gt_total, be = eq_total, tot_g = 0, tot_e = 0;
#pragma unroll
        for (int w2 = 0; w2 < TOPM_WARPS; ++w2) {
            if (w2 < warp) { bg += s_scan[w2][0]; be += s_scan[w2][1]; }
            tot_g += s_scan[w2][0]; tot_e += s_scan[w2][1];
        }
        int g_before = bg + sg - gt, e_before = be + se - eq;
#pragma unroll
        for (int j = 0; j < EPV; ++j) {
            if ((fl_gt >> j) & 1u) { out[g_before + min(e_before, take_eq)] = e0 + j; ++g_before; }
            else if ((fl_eq >> j) & 1u) {
                if (e_before < take_eq) out[g_before + e_before] = e0 + j;
                ++e_before;
            }
        }
        gt_total += tot_g;
        eq_total += tot_e;
    });
    for (int m = want + tid; m < p.M; m += TOPM_THREADS) out[m] = -1;
}

}  // namespace

extern "C" int disc_topm(const void* logits, disc_dtype_t dtype, int64_t ld, int64_t n, int32_t vocab_size, int32_t M,
                         float inv_temperature, const uint8_t* done, int32_t* cand_out, float* lse_out, void* stream) {
    if (n < 0 || vocab_size <= 0 || M <= 0 || ld < vocab_size) return DISC_ERR_ARG;
    if (n == 0) return DISC_OK;
    if (!logits || !cand_out) return DISC_ERR_ARG;
    if (dtype != DISC_F32 && dtype != DISC_BF16) return DISC_ERR_UNSUPPORTED;
    if (n >= (int64_t(1) << 31) || vocab_size > (1 << 30)) return DISC_ERR_UNSUPPORTED;
    if (lse_out && (!(inv_temperature > 0.f) || !(inv_temperature <= 3.0e38f))) return DISC_ERR_ARG;
    TopmParams p;
    p.logits = logits; p.ld = ld; p.V = vocab_size; p.M = M; p.c2 = inv_temperature * LOG2E_F;
    p.done = done; p.cand = cand_out; p.lse = reinterpret_cast<float2*>(lse_out);
    const size_t esize = dtype == DISC_F32 ? 4 : 2;
    const bool vec = (reinterpret_cast<uintptr_t>(logits) % 16 == 0) && ((size_t(ld) * esize) % 16 == 0);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const unsigned grid = unsigned(n);
    if (dtype == DISC_F32) {
        if (vec) disc_topm_kernel<DISC_F32, true><<<grid, TOPM_THREADS, 0, st>>>(p);
        else disc_topm_kernel<DISC_F32, false><<<grid, TOPM_THREADS, 0, st>>>(p);
    } else {
        if (vec) disc_topm_kernel<DISC_BF16, true><<<grid, TOPM_THREADS, 0, st>>>(p);
        else disc_topm_kernel<DISC_BF16, false><<<grid, TOPM_THREADS, 0, st>>>(p);
    }
    DISC_CUDA(cudaGetLastError());
    return DISC_OK;
}

extern "C" int64_t disc_step_topm_scratch_bytes(int64_t n, int32_t M) {
    if (n < 0 || M <= 0) return DISC_ERR_ARG;
    return n * 8 /* (m, s) */ + n * 8 /* lo, hi */ + n * int64_t(M) /* validity */ + 64;
}

extern "C" int disc_step_topm(const disc_set_t* s, const void* logits, disc_dtype_t dtype, int64_t ld, int64_t n, int32_t M,
                              float inv_temperature, uint64_t seed, uint32_t step, int64_t row_base, int32_t* node,
                              int32_t* lo, int32_t* hi, int32_t* depth, float* logw, uint8_t* done, int32_t* token_out,
                              int32_t* seq_tokens, int32_t seq_ld, float* logq_out, float* logp_out, uint32_t* mask_out,
                              uint8_t* status_out, int32_t* cand_out, void* scratch, int64_t scratch_bytes,
                              void* stream) {
    if (!s || n < 0 || n >= (int64_t(1) << 31)) return DISC_ERR_ARG;
    if (const int rc = disc::check_device(s)) return rc;
    if (n == 0) return DISC_OK;
    if (!logits || !node || !lo || !hi || !depth || !logw || !done || !token_out || !status_out || !cand_out || !scratch ||
        !seq_tokens)
        return DISC_ERR_ARG;
    if (ld < s->V || row_base < 0 || seq_ld < s->l_max) return DISC_ERR_ARG;
    if (!(inv_temperature > 0.f) || !(inv_temperature <= 3.0e38f)) return DISC_ERR_ARG;
    if (dtype != DISC_F32 && dtype != DISC_BF16) return DISC_ERR_UNSUPPORTED;
    if (M <= 0 || M > 1024) return DISC_ERR_UNSUPPORTED;
    if (row_base + n > (int64_t(1) << 32)) return DISC_ERR_UNSUPPORTED;
    if (scratch_bytes < disc_step_topm_scratch_bytes(n, M) || (reinterpret_cast<uintptr_t>(scratch) & 7u)) return DISC_ERR_ARG;
    unsigned char* sc = static_cast<unsigned char*>(scratch);
    float* lse = reinterpret_cast<float*>(sc);
    int32_t* lo_v = reinterpret_cast<int32_t*>(sc + size_t(n) * 8);
    int32_t* hi_v = lo_v + n;
    uint8_t* valid = sc + size_t(n) * 16;
    // Algorithm 2, line 3: candidates; lines 4-5: verification against the sorted array; then
    // Algorithm 1, lines 7-8 over the verified candidates
    if (const int rc = disc_topm(logits, dtype, ld, n, s->V, M, inv_temperature, done, cand_out, lse, stream)) return rc;
    if (const int rc = disc_verify(s, seq_tokens, seq_ld, depth, n, cand_out, M, valid, nullptr, nullptr, lo_v, hi_v, stream))
        return rc;
    return disc::step_with_candidates(s, logits, dtype, ld, n, inv_temperature, seed, step, row_base, node, lo, hi, depth,
                                      logw, done, token_out, seq_tokens, seq_ld, logq_out, logp_out, mask_out, status_out,
                                      cand_out, valid, M, reinterpret_cast<const float2*>(lse),
                                      static_cast<cudaStream_t>(stream));
}
