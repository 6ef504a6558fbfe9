// disc_step: one decoding step of Algorithm 1 (lines 5-8) for a batch of candidates, fused:
// valid-set lookup, masked and unmasked log-sum-exp over the V logits, Gumbel-max sampling,
// importance log-weight update and the move of the row's cursor to the extended prefix.
//
// One thread block per row.  The row's V logits are streamed once with 16-byte loads; each
// thread accumulates sum 2^(z*log2e/T - ref) against its own reference (the maximum of the first
// vector it sees), which keeps the inner loop at one FMA, one ex2 and one add per logit.  The
// valid set comes from the prefix index as a contiguous child list.  Rows with few children gather
// their logits directly ("gather path"); rows with many children turn the list into a bitmask in
// shared memory that the streaming loop consults ("dense path").  A row whose fast sums are not
// finite, or whose valid mass underflowed, is redone by a plain two-pass routine ("careful path").

#include <math_constants.h>

#include "disc_internal.cuh"

namespace {

using namespace disc;

constexpr int STEP_THREADS = 256;
constexpr int STEP_WARPS = STEP_THREADS / 32;
constexpr int GATHER_MAX = 1024;   // rows with at most this many children skip the bitmask
constexpr int UNROLL = 4;
constexpr float LOG2E_F = 1.4426950408889634f;
constexpr float LN2_F = 0.6931471805599453f;

struct StepParams {
    const void* logits;
    int64_t ld;
    float inv_t;
    float c2;            // inv_t * log2(e)
    PhiloxKey key;
    uint32_t step;
    uint32_t row_base;
    // state
    int32_t *node, *lo, *hi, *depth;
    float* logw;
    uint8_t* done;
    // outputs
    int32_t* token_out;
    int32_t* seq_tokens;
    int32_t seq_ld;
    float *logq_out, *logp_out;
    uint32_t* mask_out;
    uint8_t* status_out;
    // set
    const int32_t *node_tok, *node_lo, *child_begin, *root_child;
    const uint32_t* root_mask;
    int32_t V, W;
    int64_t M;
};

// value 2^m * s; the empty sum is (m = -inf, s = 0)
struct MS {
    float m, s;
};

__device__ __forceinline__ MS ms_merge(MS a, MS b) {
    float M = fmaxf(a.m, b.m);
    if (M == -CUDART_INF_F) return MS{M, 0.f};
    return MS{M, a.s * exp2f(a.m - M) + b.s * exp2f(b.m - M)};
}

struct Best {
    float score;
    int32_t tok;     // -1: none yet
    int32_t child;   // node id of the child when known, else -1
};

__device__ __forceinline__ Best best_merge(Best a, Best b) {
    if (b.tok < 0) return a;
    if (a.tok < 0) return b;
    if (b.score > a.score || (b.score == a.score && b.tok < a.tok)) return b;
    return a;
}

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint4 ld_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

template <int DT>
struct Elem;
template <>
struct Elem<DISC_F32> {
    static constexpr int SIZE = 4;
    static constexpr int EPV = 4;
    __device__ static __forceinline__ float load(const void* base, int64_t i) {
        return __ldg(static_cast<const float*>(base) + i);
    }
    __device__ static __forceinline__ void unpack(const uint4& v, float (&x)[4]) {
        x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y);
        x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
    }
};
template <>
struct Elem<DISC_BF16> {
    static constexpr int SIZE = 2;
    static constexpr int EPV = 8;
    __device__ static __forceinline__ float load(const void* base, int64_t i) {
        return __uint_as_float(uint32_t(__ldg(static_cast<const unsigned short*>(base) + i)) << 16);
    }
    __device__ static __forceinline__ void unpack(const uint4& v, float (&x)[8]) {
        x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xffff0000u);
        x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xffff0000u);
        x[4] = __uint_as_float(v.z << 16); x[5] = __uint_as_float(v.z & 0xffff0000u);
        x[6] = __uint_as_float(v.w << 16); x[7] = __uint_as_float(v.w & 0xffff0000u);
    }
};

struct RowRng {
    PhiloxKey key;
    uint32_t step, row;
};

// Gumbel-perturbed score of a token with raw logit x, relative to the row's reference logit xref.
// The argmax does not depend on the common shift, and subtracting before scaling keeps the score
// accurate to a few ulp of (x - xref) whatever offset the logits carry.
__device__ __forceinline__ float gumbel_score(float x, float xref, float inv_t, uint32_t word) {
    return (x - xref) * inv_t + gumbel_from_uniform(uniform_from_bits(word));
}

__device__ __forceinline__ void consider(Best& b, float score, int32_t tok, int32_t child) {
    // Tokens arrive in ascending order inside a thread, so strict '>' keeps the lowest id on a
    // tie.  NaN and -inf scores never win; a row without any finite score falls back to its
    // lowest valid token at the end.
    if (score > b.score) { b.score = score; b.tok = tok; b.child = child; }
}

// ---- block-wide helpers -----------------------------------------------------------------------
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ float block_max(float v, float* scratch) {
    v = warp_max(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = scratch[0];
#pragma unroll
    for (int w = 1; w < STEP_WARPS; ++w) r = fmaxf(r, scratch[w]);
    return r;
}
__device__ float block_sum(float v, float* scratch) {
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = scratch[0];
#pragma unroll
    for (int w = 1; w < STEP_WARPS; ++w) r += scratch[w];
    return r;
}

// Valid set of `node` as a bitmask in shared memory (all threads of the block).
__device__ void build_mask(uint32_t* smask, const StepParams& p, int32_t node, int32_t cb, int32_t ce) {
    if (node == 0) {
        for (int w = threadIdx.x; w < p.W; w += STEP_THREADS) smask[w] = __ldg(p.root_mask + w);
    } else {
        for (int w = threadIdx.x; w < p.W; w += STEP_THREADS) smask[w] = 0u;
        __syncthreads();
        for (int i = cb + threadIdx.x; i < ce; i += STEP_THREADS) {
            int32_t t = __ldg(p.node_tok + i);
            atomicOr(&smask[t >> 5], 1u << (t & 31));
        }
    }
    __syncthreads();
}

// position of token t among the sorted children [cb, ce) of a node, found by one warp: each round
// 32 lanes probe evenly spaced keys and keep the sub-range that can still hold t.  -1 if absent.
__device__ int32_t warp_find_child(const int32_t* __restrict__ node_tok, int32_t cb, int32_t ce, int32_t t) {
    const int lane = threadIdx.x & 31;
    int32_t a = cb, b = ce;
    while (b - a > 32) {
        int32_t stride = (b - a + 31) / 32;
        int32_t i = a + lane * stride;
        bool le = (i < b) && (__ldg(node_tok + i) <= t);
        uint32_t bal = __ballot_sync(0xffffffffu, le);
        if (bal == 0) return -1;
        int32_t k = 31 - __clz(bal);
        a = a + k * stride;
        b = min(a + stride, b);
    }
    int32_t i = a + lane;
    bool eq = (i < b) && (__ldg(node_tok + i) == t);
    uint32_t bal = __ballot_sync(0xffffffffu, eq);
    return bal ? a + (__ffs(bal) - 1) : -1;
}

// ---- the kernel ---------------------------------------------------------------------------------
template <int DT, bool VEC>
__global__ void __launch_bounds__(STEP_THREADS, 4) disc_step_kernel(const StepParams p) {
    using E = Elem<DT>;
    constexpr int EPV = VEC ? E::EPV : 1;
    extern __shared__ __align__(16) uint32_t smask[];
    __shared__ float red_f[6][STEP_WARPS];
    __shared__ int32_t red_i[2][STEP_WARPS];
    __shared__ float scratch[STEP_WARPS];
    __shared__ float fin[4];        // (m, s) of the full row and of the valid set
    __shared__ int32_t s_flag;

    const int64_t row = blockIdx.x;
    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;

    if (p.done[row]) {
        if (tid == 0) { p.token_out[row] = -1; p.status_out[row] = DISC_ROW_DONE; }
        return;
    }
    const int32_t node = p.node[row];
    int32_t cb = 0, ce = 0;
    if (node >= 0 && int64_t(node) < p.M) { cb = __ldg(p.child_begin + node); ce = __ldg(p.child_begin + node + 1); }
    const int32_t c = ce - cb;
    if (c <= 0) {   // not a prefix of any member, or already a complete member
        if (tid == 0) {
            p.token_out[row] = -1;
            bool leaf = node > 0 && int64_t(node) < p.M;
            p.status_out[row] = leaf ? DISC_ROW_DONE : DISC_ROW_DEAD;
            if (leaf) p.done[row] = 1;
        }
        return;
    }

    const char* rowp = static_cast<const char*>(p.logits) + size_t(row) * size_t(p.ld) * E::SIZE;
    const RowRng rng{p.key, p.step, uint32_t(p.row_base + uint32_t(row))};
    const bool dense = (c > GATHER_MAX) || (p.mask_out != nullptr);
    float xref = E::load(rowp, 0);
    if (!(fabsf(xref) < CUDART_INF_F)) xref = 0.f;

    MS ok{-CUDART_INF_F, 0.f};
    Best best{-CUDART_INF_F, -1, -1};
    bool poisoned = false;

    if (dense) {
        build_mask(smask, p, node, cb, ce);
        if (p.mask_out) {
            uint32_t* mo = p.mask_out + size_t(row) * p.W;
            for (int w = tid; w < p.W; w += STEP_THREADS) mo[w] = smask[w];
        }
    } else {
        // gather path: the few allowed logits are read directly
        for (int i = tid; i < c; i += STEP_THREADS) {
            int32_t v = __ldg(p.node_tok + cb + i);
            float x = E::load(rowp, v);
            // sum of 2^(x*c2) kept as 2^m * s; fma(x, c2, -m) is the exact product minus the
            // reference, so a large common offset of the logits costs no accuracy
            const float y = x * p.c2;
            if (!(y < CUDART_INF_F)) poisoned = true;                 // NaN or +inf: careful path
            else if (y > ok.m) { ok.s = ok.s * exp2f(ok.m - y) + exp2f(fmaf(x, p.c2, -y)); ok.m = y; }
            else if (y != -CUDART_INF_F) ok.s += exp2f(fmaf(x, p.c2, -ok.m));
            uint4 r = philox4x32_10(uint32_t(v) >> 2, rng.step, rng.row, 0u, rng.key);
            consider(best, gumbel_score(x, xref, p.inv_t, pick_word(r, v & 3)), v, cb + i);
        }
    }

    // ---- stream the row
    const int nvec = p.V / EPV;
    float mref = 0.f;
    float s_all[2] = {0.f, 0.f};
    float s_ok = 0.f;
    bool touched = false;
    bool lost = false;   // an allowed finite logit underflowed against this thread's reference

    auto process = [&](const uint4& raw, float xs, int idx) {
        float x[EPV];
        if constexpr (VEC) E::unpack(raw, x); else x[0] = xs;
        float e[EPV];
#pragma unroll
        for (int j = 0; j < EPV; ++j) {
            e[j] = ex2_approx(fmaf(x[j], p.c2, -mref));
            s_all[j & 1] += e[j];
        }
        if (dense) {
            const int v0 = idx * EPV;
            uint32_t bits = (smask[v0 >> 5] >> (v0 & 31)) & ((1u << EPV) - 1u);
            if (bits) {
#pragma unroll
                for (int q = 0; q < (EPV + 3) / 4; ++q) {
                    uint32_t nib = (bits >> (4 * q)) & 0xFu;
                    if (nib) {
                        uint4 r = philox4x32_10(uint32_t(v0 >> 2) + q, rng.step, rng.row, 0u, rng.key);
#pragma unroll
                        for (int l = 0; l < (EPV < 4 ? EPV : 4); ++l) {
                            if ((nib >> l) & 1u) {
                                const int j = 4 * q + l;
                                const int v = v0 + j;
                                s_ok += e[j];
                                lost |= (e[j] == 0.f) && (x[j] > -CUDART_INF_F);
                                consider(best, gumbel_score(x[j], xref, p.inv_t, pick_word(r, v & 3)), v, -1);
                            }
                        }
                    }
                }
            }
        }
    };

    if constexpr (VEC) {
        const uint4* vp = reinterpret_cast<const uint4*>(rowp);
        constexpr int STRIDE = STEP_THREADS * UNROLL;
        for (int base = 0; base < nvec; base += STRIDE) {
            uint4 raw[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                int idx = base + u * STEP_THREADS + tid;
                if (idx < nvec) raw[u] = ld_stream16(vp + idx);
            }
            if (base == 0 && tid < nvec) {
                float x[EPV];
                E::unpack(raw[0], x);
                float mx = x[0];
#pragma unroll
                for (int j = 1; j < EPV; ++j) mx = fmaxf(mx, x[j]);
                float r = mx * p.c2;
                mref = (fabsf(r) < CUDART_INF_F) ? r : 0.f;
                touched = true;
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                int idx = base + u * STEP_THREADS + tid;
                if (idx < nvec) process(raw[u], 0.f, idx);
            }
        }
        // ragged tail: V not a multiple of the vector width
        const int v = nvec * EPV + tid;
        if (v < p.V) {
            float x = E::load(rowp, v);
            if (!touched) { float r = x * p.c2; mref = (fabsf(r) < CUDART_INF_F) ? r : 0.f; touched = true; }
            float e = ex2_approx(fmaf(x, p.c2, -mref));
            s_all[0] += e;
            if (dense && ((smask[v >> 5] >> (v & 31)) & 1u)) {
                s_ok += e;
                lost |= (e == 0.f) && (x > -CUDART_INF_F);
                uint4 r = philox4x32_10(uint32_t(v) >> 2, rng.step, rng.row, 0u, rng.key);
                consider(best, gumbel_score(x, xref, p.inv_t, pick_word(r, v & 3)), v, -1);
            }
        }
    } else {
        for (int idx = tid; idx < p.V; idx += STEP_THREADS) {
            float x = E::load(rowp, idx);
            if (!touched) { float r = x * p.c2; mref = (fabsf(r) < CUDART_INF_F) ? r : 0.f; touched = true; }
            process(uint4{}, x, idx);
        }
    }

    MS all = touched ? MS{mref, s_all[0] + s_all[1]} : MS{-CUDART_INF_F, 0.f};
    if (dense) ok = touched ? MS{mref, s_ok} : MS{-CUDART_INF_F, 0.f};
    if (poisoned) ok.s = CUDART_NAN_F;

    const int any_lost = __syncthreads_or(lost ? 1 : 0);

    // ---- block reduction of (all, ok, best)
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        MS a2{__shfl_xor_sync(0xffffffffu, all.m, o), __shfl_xor_sync(0xffffffffu, all.s, o)};
        MS k2{__shfl_xor_sync(0xffffffffu, ok.m, o), __shfl_xor_sync(0xffffffffu, ok.s, o)};
        Best b2{__shfl_xor_sync(0xffffffffu, best.score, o), __shfl_xor_sync(0xffffffffu, best.tok, o),
                __shfl_xor_sync(0xffffffffu, best.child, o)};
        all = ms_merge(all, a2);
        ok = ms_merge(ok, k2);
        best = best_merge(best, b2);
    }
    if (lane == 0) {
        red_f[0][warp] = all.m; red_f[1][warp] = all.s; red_f[2][warp] = ok.m; red_f[3][warp] = ok.s;
        red_f[4][warp] = best.score; red_i[0][warp] = best.tok; red_i[1][warp] = best.child;
    }
    __syncthreads();
    if (warp == 0) {
        if (lane < STEP_WARPS) {
            all = MS{red_f[0][lane], red_f[1][lane]};
            ok = MS{red_f[2][lane], red_f[3][lane]};
            best = Best{red_f[4][lane], red_i[0][lane], red_i[1][lane]};
        } else {
            all = MS{-CUDART_INF_F, 0.f};
            ok = MS{-CUDART_INF_F, 0.f};
            best = Best{-CUDART_INF_F, -1, -1};
        }
#pragma unroll
        for (int o = STEP_WARPS / 2; o > 0; o >>= 1) {
            MS a2{__shfl_xor_sync(0xffffffffu, all.m, o), __shfl_xor_sync(0xffffffffu, all.s, o)};
            MS k2{__shfl_xor_sync(0xffffffffu, ok.m, o), __shfl_xor_sync(0xffffffffu, ok.s, o)};
            Best b2{__shfl_xor_sync(0xffffffffu, best.score, o), __shfl_xor_sync(0xffffffffu, best.tok, o),
                    __shfl_xor_sync(0xffffffffu, best.child, o)};
            all = ms_merge(all, a2);
            ok = ms_merge(ok, k2);
            best = best_merge(best, b2);
        }
        if (lane == 0) {
            fin[0] = all.m; fin[1] = all.s; fin[2] = ok.m; fin[3] = ok.s;
            const float l2_all = all.m + log2f(all.s);
            const float l2_ok = ok.m + log2f(ok.s);
            // the fast sums are trusted only when both are finite and no allowed term was lost
            s_flag = (fabsf(l2_all) < CUDART_INF_F && fabsf(l2_ok) < CUDART_INF_F && !any_lost) ? 0 : 1;
        }
    }
    __syncthreads();

    if (s_flag) {
        // ---- careful path: plain two-pass log-sum-exp over the row with an explicit mask and
        // separate maxima for the full row and for the valid set
        if (!dense) build_mask(smask, p, node, cb, ce);
        float mx_all = -CUDART_INF_F, mx_ok = -CUDART_INF_F;
        int nan_all = 0, nan_ok = 0;
        for (int v = tid; v < p.V; v += STEP_THREADS) {
            const float x = E::load(rowp, v);
            const bool allowed = (smask[v >> 5] >> (v & 31)) & 1u;
            if (x != x) { nan_all = 1; nan_ok |= allowed; }
            else { mx_all = fmaxf(mx_all, x); if (allowed) mx_ok = fmaxf(mx_ok, x); }
        }
        mx_all = block_max(mx_all, scratch);
        mx_ok = block_max(mx_ok, scratch);
        nan_all = __syncthreads_or(nan_all);
        nan_ok = __syncthreads_or(nan_ok);
        const bool fin_all = fabsf(mx_all) < CUDART_INF_F, fin_ok = fabsf(mx_ok) < CUDART_INF_F;
        const float r_all = mx_all * p.c2, r_ok = mx_ok * p.c2;
        float sum_all = 0.f, sum_ok = 0.f;
        for (int v = tid; v < p.V; v += STEP_THREADS) {
            const float x = E::load(rowp, v);
            const bool allowed = (smask[v >> 5] >> (v & 31)) & 1u;
            if (fin_all) sum_all += exp2f(fmaf(x, p.c2, -r_all));
            if (fin_ok && allowed) sum_ok += exp2f(fmaf(x, p.c2, -r_ok));
        }
        sum_all = block_sum(sum_all, scratch);
        sum_ok = block_sum(sum_ok, scratch);
        if (tid == 0) {
            // (m, s) with value 2^m * s; +inf maximum -> (+inf, 1), empty or all -inf -> (-inf, 0)
            fin[0] = nan_all ? CUDART_NAN_F : (fin_all ? r_all : mx_all);
            fin[1] = nan_all ? CUDART_NAN_F : (fin_all ? sum_all : (mx_all > 0.f ? 1.f : 0.f));
            fin[2] = nan_ok ? CUDART_NAN_F : (fin_ok ? r_ok : mx_ok);
            fin[3] = nan_ok ? CUDART_NAN_F : (fin_ok ? sum_ok : (mx_ok > 0.f ? 1.f : 0.f));
        }
        __syncthreads();
    }

    // ---- finalise: one warp moves the row's cursor to the chosen child
    if (warp == 0) {
        best.score = __shfl_sync(0xffffffffu, best.score, 0);
        best.tok = __shfl_sync(0xffffffffu, best.tok, 0);
        best.child = __shfl_sync(0xffffffffu, best.child, 0);
        int32_t tok = best.tok, child = best.child;
        if (tok < 0) { tok = __ldg(p.node_tok + cb); child = cb; }     // no finite score: lowest id
        if (child < 0) {
            child = (node == 0) ? __ldg(p.root_child + tok) : warp_find_child(p.node_tok, cb, ce, tok);
        }
        if (child < 0) {   // cannot happen for a consistent index; never index with it
            if (lane == 0) { p.token_out[row] = -1; p.status_out[row] = DISC_ROW_DEAD; p.done[row] = 1; }
        } else if (lane == 0) {
            const MS A{fin[0], fin[1]}, K{fin[2], fin[3]};
            const float lg_all = log2f(A.s), lg_ok = log2f(K.s);
            const float l2_all = A.m + lg_all, l2_ok = K.m + lg_ok;
            const bool f_all = fabsf(l2_all) < CUDART_INF_F, f_ok = fabsf(l2_ok) < CUDART_INF_F;
            // Differences are formed between references first, so that a large common offset of
            // the logits does not eat the low bits: log_mass = log2(sum_ok / sum_all) * ln 2.
            const float log_mass = (f_all && f_ok) ? ((K.m - A.m) + (lg_ok - lg_all)) * LN2_F
                                                   : (l2_ok - l2_all) * LN2_F;
            uint8_t st = 0;
            if (!f_all) st |= DISC_ROW_NONFINITE;
            if (!f_ok) st |= DISC_ROW_NOMASS;
            const float xt = E::load(rowp, tok);
            const float logq = f_ok ? (fmaf(xt, p.c2, -K.m) - lg_ok) * LN2_F : (xt * p.c2 - l2_ok) * LN2_F;
            const float logp = f_all ? (fmaf(xt, p.c2, -A.m) - lg_all) * LN2_F : (xt * p.c2 - l2_all) * LN2_F;
            const int32_t d = p.depth[row];
            const int32_t hi_old = p.hi[row];
            p.token_out[row] = tok;
            if (p.seq_tokens && d < p.seq_ld) p.seq_tokens[size_t(row) * p.seq_ld + d] = tok;
            if (p.logq_out) p.logq_out[row] = logq;
            if (p.logp_out) p.logp_out[row] = logp;
            p.logw[row] += log_mass;
            p.node[row] = child;
            p.lo[row] = __ldg(p.node_lo + child);
            p.hi[row] = (child + 1 < ce) ? __ldg(p.node_lo + child + 1) : hi_old;
            p.depth[row] = d + 1;
            p.done[row] = (__ldg(p.child_begin + child) == __ldg(p.child_begin + child + 1)) ? 1 : 0;
            p.status_out[row] = st;
        }
    }
}

__global__ void k_state_init(int64_t n, int32_t N, int32_t* node, int32_t* lo, int32_t* hi, int32_t* depth,
                             float* logw, uint8_t* done) {
    int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n) return;
    node[i] = 0; lo[i] = 0; hi[i] = N; depth[i] = 0; logw[i] = 0.f; done[i] = 0;
}

__global__ void k_sampling_uniforms(PhiloxKey key, uint32_t step, uint32_t row, int32_t v0, int32_t n, float* out) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    uint32_t v = uint32_t(v0 + i);
    uint4 r = philox4x32_10(v >> 2, step, row, 0u, key);
    out[i] = uniform_from_bits(pick_word(r, v & 3));
}

template <int DT, bool VEC>
int launch_step(const StepParams& p, int64_t n, size_t smem, cudaStream_t st) {
    if (smem > 48 * 1024) {
        DISC_CUDA(cudaFuncSetAttribute(disc_step_kernel<DT, VEC>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       int(smem)));
    }
    disc_step_kernel<DT, VEC><<<unsigned(n), STEP_THREADS, smem, st>>>(p);
    DISC_CUDA(cudaGetLastError());
    return DISC_OK;
}

}  // namespace

extern "C" {

int disc_state_init(const disc_set_t* s, int64_t n, int32_t* node, int32_t* lo, int32_t* hi, int32_t* depth,
                    float* logw, uint8_t* done, void* stream) {
    if (!s || n < 0) return DISC_ERR_ARG;
    if (n == 0) return DISC_OK;
    if (!node || !lo || !hi || !depth || !logw || !done) return DISC_ERR_ARG;
    k_state_init<<<unsigned((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        n, int32_t(s->N), node, lo, hi, depth, logw, done);
    DISC_CUDA(cudaGetLastError());
    return DISC_OK;
}

int disc_step(const disc_set_t* s, const void* logits, disc_dtype_t dtype, int64_t ld, int64_t n,
              float inv_temperature, uint64_t seed, uint32_t step, int64_t row_base, int32_t* node, int32_t* lo,
              int32_t* hi, int32_t* depth, float* logw, uint8_t* done, int32_t* token_out, int32_t* seq_tokens,
              int32_t seq_ld, float* logq_out, float* logp_out, uint32_t* mask_out, uint8_t* status_out,
              void* stream) {
    if (!s || n < 0 || n >= (int64_t(1) << 31)) return DISC_ERR_ARG;
    if (n == 0) return DISC_OK;
    if (!logits || !node || !lo || !hi || !depth || !logw || !done || !token_out || !status_out) return DISC_ERR_ARG;
    if (ld < s->V || row_base < 0 || (seq_tokens && seq_ld <= 0)) return DISC_ERR_ARG;
    if (!(inv_temperature > 0.f) || !(inv_temperature <= 3.0e38f)) return DISC_ERR_ARG;
    if (dtype != DISC_F32 && dtype != DISC_BF16) return DISC_ERR_UNSUPPORTED;
    const size_t smem = (size_t(s->W) * 4 + 15) & ~size_t(15);
    if (smem > 200 * 1024) return DISC_ERR_UNSUPPORTED;

    StepParams p;
    p.logits = logits; p.ld = ld; p.inv_t = inv_temperature; p.c2 = inv_temperature * LOG2E_F;
    p.key = philox_key(seed); p.step = step; p.row_base = uint32_t(row_base);
    p.node = node; p.lo = lo; p.hi = hi; p.depth = depth; p.logw = logw; p.done = done;
    p.token_out = token_out; p.seq_tokens = seq_tokens; p.seq_ld = seq_ld;
    p.logq_out = logq_out; p.logp_out = logp_out; p.mask_out = mask_out; p.status_out = status_out;
    p.node_tok = s->node_tok; p.node_lo = s->node_lo; p.child_begin = s->child_begin;
    p.root_child = s->root_child; p.root_mask = s->root_mask; p.V = s->V; p.W = s->W; p.M = s->M;

    const size_t esize = dtype == DISC_F32 ? 4 : 2;
    const bool vec = (reinterpret_cast<uintptr_t>(logits) % 16 == 0) && ((size_t(ld) * esize) % 16 == 0);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (dtype == DISC_F32) return vec ? launch_step<DISC_F32, true>(p, n, smem, st) : launch_step<DISC_F32, false>(p, n, smem, st);
    return vec ? launch_step<DISC_BF16, true>(p, n, smem, st) : launch_step<DISC_BF16, false>(p, n, smem, st);
}

int disc_sampling_uniforms(uint64_t seed, uint32_t step, uint32_t row, int32_t v0, int32_t n, float* out,
                           void* stream) {
    if (n < 0 || v0 < 0 || (n > 0 && !out)) return DISC_ERR_ARG;
    if (n == 0) return DISC_OK;
    k_sampling_uniforms<<<(n + 255) / 256, 256, 0, static_cast<cudaStream_t>(stream)>>>(philox_key(seed), step, row,
                                                                                       v0, n, out);
    DISC_CUDA(cudaGetLastError());
    return DISC_OK;
}

}  // extern "C"
