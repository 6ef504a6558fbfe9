// disc_step: one decoding step of Algorithm 1 (lines 5-8) for a batch of candidates, fused:
// valid-set lookup, masked and unmasked log-sum-exp over the V logits, Gumbel-max sampling,
// importance log-weight update and the move of the row's cursor to the extended prefix.
//
// One thread block per row.
//   * Streaming.  The row's logits are pulled into a shared-memory ring by bulk asynchronous
//     copies (cp.async.bulk + mbarrier, one elected thread issues them), so several chunks are in
//     flight per block whatever the register budget; rows that are not 16-byte aligned take a
//     plain scalar-load path.
//   * Sums.  Each thread accumulates sum 2^(x*c - ref) against its own reference (the maximum of
//     the first vector it sees), c = log2(e)/T: one FMA, one ex2 and one add per logit.  Partial
//     sums are kept as (m, s) pairs meaning 2^m * s and merged exactly.  All differences are formed
//     between references before any large value is added, so a common offset of the logits does
//     not cost accuracy.
//   * Valid set.  The prefix index gives the row's children as a contiguous list.  Rows with at
//     most DISC_HEAVY_MIN children gather their few logits directly ("gather path").  Rows with
//     more use a bitmask in shared memory (prebuilt at set-build time) that the streaming loop
//     consults ("dense path").
//   * Sampling.  token = argmax over allowed v of (x_v - xref)/T + g_v with g_v = -log(-log u_v),
//     u_v from Philox4x32-10 keyed by (token, step, row).  In the dense path a token is evaluated
//     exactly only if it can still win: with w = 1 - u, g > t implies w < e^-t, so a token whose
//     w is at least e^(z - best) (times a safety factor) is skipped without taking a logarithm;
//     e^(z - best) is the already computed 2^(x*c - ref) times a per-thread constant.
//   * A row whose fast sums are not finite, or that lost an allowed term to underflow, is redone
//     by a plain two-pass routine with exact scores ("careful path").

#include <math_constants.h>

#include "disc_internal.cuh"

namespace {

using namespace disc;

constexpr int STEP_THREADS = 256;
constexpr int STEP_WARPS = STEP_THREADS / 32;
constexpr int CHUNK_BYTES = 8192;                       // one ring stage
constexpr int STAGES = 4;
constexpr int VPT = CHUNK_BYTES / 16 / STEP_THREADS;    // 16-byte vectors per thread and stage
constexpr int RING_BYTES = CHUNK_BYTES * STAGES;
constexpr uint64_t WAIT_LIMIT_NS = 250ull * 1000 * 1000;  // an mbarrier wait gives up after 0.25 s
constexpr float LOG2E_F = 1.4426950408889634f;
constexpr float LN2_F = 0.6931471805599453f;
constexpr float SAFETY = 1.0009765625f;                 // 1 + 2^-10 on the skip bound
constexpr float TWO_M24 = 5.9604644775390625e-08f;      // 2^-24: smallest possible w

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
    const int32_t *node_tok, *node_lo, *child_begin, *root_child, *heavy_nodes;
    const uint32_t *root_mask, *heavy_masks;
    int32_t V, W, n_heavy;
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

// ---- mbarrier / bulk-copy wrappers -------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return uint32_t(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: gives up (returns false) after WAIT_LIMIT_NS without the phase completing.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity) {
    const uint64_t t0 = global_ns();
    while (!mbar_try_wait(bar, parity)) {
        if (global_ns() - t0 > WAIT_LIMIT_NS) return false;
    }
    return true;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    return mbar_try_wait(bar, parity) ? true : mbar_wait_slow(bar, parity);
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
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

// Gumbel-perturbed score of a token with raw logit x, relative to the row's reference logit xref.
// The argmax does not depend on the common shift, and subtracting before scaling keeps the score
// accurate to a few ulp of (x - xref) whatever offset the logits carry.
__device__ __forceinline__ float gumbel_score(float x, float xref, float inv_t, uint32_t word) {
    return (x - xref) * inv_t + gumbel_from_uniform(uniform_from_bits(word));
}

// w = 1 - u of a random word, exact: with k' the complement of the word's top 23 bits,
// w = (2k'+1) * 2^-24.  No integer-to-float conversion is needed: 1.k' - (1 - 2^-24).
__device__ __forceinline__ float complement_uniform(uint32_t word) {
    return __uint_as_float(0x3f800000u | ((~word) >> 9)) - 0.99999994039535522f;
}

// Per-thread accumulators of the streaming loop.
struct Acc {
    float mref = 0.f;        // reference exponent (log2 domain) of this thread's sums
    float s_all0 = 0.f, s_all1 = 0.f;
    float s_ok = 0.f;
    bool touched = false;
    bool lost = false;       // an allowed term underflowed to zero against mref
    // sampling
    Best best{-__builtin_huge_valf(), -1, -1};
    float cbound = __builtin_huge_valf();   // SAFETY * 2^(mref - xref*c - best*log2e): e * cbound bounds e^(z - best)
};

struct RowCtx {
    float c2, inv_t, xref;
    PhiloxKey key;
    uint32_t step, row;
};

__device__ __forceinline__ void set_reference(Acc& a, const RowCtx& r, float xmax) {
    const float m = xmax * r.c2;
    a.mref = (fabsf(m) < CUDART_INF_F) ? m : 0.f;
    a.touched = true;
}

__device__ __forceinline__ void update_bound(Acc& a, const RowCtx& r) {
    // exponent of e^(z - best) / 2^(x*c - mref); fma keeps (mref - xref*c) exact to one rounding
    a.cbound = SAFETY * exp2f(fmaf(-r.xref, r.c2, a.mref) - a.best.score * LOG2E_F);
}

__device__ __forceinline__ void exact_candidate(Acc& a, const RowCtx& r, float x, uint32_t word, int32_t v) {
    // Tokens arrive in ascending order inside a thread, so strict '>' keeps the lowest id on a
    // tie.  NaN and -inf scores never win; a row without any finite score falls back to its
    // lowest valid token at the end.
    const float score = gumbel_score(x, r.xref, r.inv_t, word);
    if (score > a.best.score) {
        a.best.score = score; a.best.tok = v; a.best.child = -1;
        update_bound(a, r);
    }
}

// one vector of EPV logits starting at token v0
template <int EPV, bool DENSE>
__device__ __forceinline__ void consume(Acc& a, const RowCtx& r, const float (&x)[EPV], int v0,
                                        const uint32_t* __restrict__ smask) {
    float e[EPV];
#pragma unroll
    for (int j = 0; j < EPV; ++j) e[j] = ex2_approx(fmaf(x[j], r.c2, -a.mref));
#pragma unroll
    for (int j = 0; j < EPV; j += 2) {
        a.s_all0 += e[j];
        if (j + 1 < EPV) a.s_all1 += e[j + 1];
    }
    if constexpr (DENSE) {
        const uint32_t bits = (smask[v0 >> 5] >> (v0 & 31)) & ((1u << EPV) - 1u);
        if (bits) {
#pragma unroll
            for (int j = 0; j < EPV; ++j) {
                const bool on = (bits >> j) & 1u;
                a.s_ok += on ? e[j] : 0.f;
                a.lost |= on && !(e[j] > 0.f);
            }
#pragma unroll
            for (int q = 0; q < (EPV + 3) / 4; ++q) {
                const uint32_t nib = (bits >> (4 * q)) & 0xFu;
                if (nib) {
                    // no token of this group can win if even the largest noise is not enough:
                    // w >= 2^-24 always, so e*cbound < 2^-24 for all four means "skip" without
                    // drawing the random numbers
                    float emax = e[4 * q];
#pragma unroll
                    for (int l = 1; l < (EPV < 4 ? EPV : 4); ++l) emax = fmaxf(emax, e[4 * q + l]);
                    if (!(emax * a.cbound < TWO_M24)) {
                        const uint4 w4 = philox4x32_10(uint32_t(v0 >> 2) + q, r.step, r.row, 0u, r.key);
#pragma unroll
                        for (int l = 0; l < (EPV < 4 ? EPV : 4); ++l) {
                            if ((nib >> l) & 1u) {
                                const int j = 4 * q + l;
                                const int v = v0 + j;
                                const uint32_t word = pick_word(w4, v & 3);
                                if (!(complement_uniform(word) >= e[j] * a.cbound))
                                    exact_candidate(a, r, x[j], word, v);
                            }
                        }
                    }
                }
            }
        }
    }
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

// Valid set of `node` as a bitmask in shared memory (all threads of the block): a copy of the
// prebuilt row for the root and for heavy nodes, else built from the child list.
__device__ void build_mask(uint32_t* smask, const StepParams& p, int32_t node, int32_t cb, int32_t ce,
                           int32_t* s_tmp) {
    const uint32_t* src = nullptr;
    if (node == 0) {
        src = p.root_mask;
    } else if (ce - cb > DISC_HEAVY_MIN) {
        if (threadIdx.x == 0) *s_tmp = heavy_index(p.heavy_nodes, p.n_heavy, node);
        __syncthreads();
        const int32_t h = *s_tmp;
        if (h >= 0) src = p.heavy_masks + size_t(h) * p.W;
    }
    if (src) {
        for (int w = threadIdx.x; w < p.W; w += STEP_THREADS) smask[w] = __ldg(src + w);
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

// ---- streaming loops ---------------------------------------------------------------------------
// Bulk-copy ring: returns false if an mbarrier wait gave up.
template <int DT, bool DENSE>
__device__ bool stream_ring(Acc& a, const RowCtx& r, const char* rowp, int V, unsigned char* ring,
                            uint64_t* full_bar, uint64_t* empty_bar, const uint32_t* smask) {
    using E = Elem<DT>;
    constexpr int EPV = E::EPV;
    const int tid = threadIdx.x, lane = tid & 31;
    const int nvec = V / EPV;
    const uint32_t vec_bytes = uint32_t(nvec) * 16u;
    const int n_chunks = int((vec_bytes + CHUNK_BYTES - 1) / CHUNK_BYTES);
    const uint32_t ring_s = smem_u32(ring);
    bool ok = true;

    auto issue = [&](int c) {
        const int s = c % STAGES;
        const uint32_t off = uint32_t(c) * CHUNK_BYTES;
        const uint32_t bytes = min(uint32_t(CHUNK_BYTES), vec_bytes - off);
        const uint32_t bar = smem_u32(&full_bar[s]);
        mbar_expect_tx(bar, bytes);
        bulk_g2s(ring_s + uint32_t(s) * CHUNK_BYTES, rowp + off, bytes, bar);
    };
    if (tid == 0) {
        for (int c = 0; c < STAGES && c < n_chunks; ++c) issue(c);
    }
    for (int c = 0; c < n_chunks; ++c) {
        const int s = c % STAGES;
        const uint32_t use = uint32_t(c / STAGES);     // how often stage s was used before
        // the give-up decision is taken per warp, so that all lanes leave the loop together
        if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&full_bar[s]), use & 1u))) { ok = false; break; }
        uint4 raw[VPT];
#pragma unroll
        for (int j = 0; j < VPT; ++j) {
            const int in_chunk = j * STEP_THREADS + tid;
            const int g = c * (CHUNK_BYTES / 16) + in_chunk;
            if (g < nvec) raw[j] = *reinterpret_cast<const uint4*>(ring + s * CHUNK_BYTES + in_chunk * 16);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&empty_bar[s]));
        // refill the stage released one iteration ago (every warp has long passed it)
        if (tid == 0 && c >= 1 && c - 1 + STAGES < n_chunks) {
            const int sp = (c - 1) % STAGES;
            const uint32_t usep = uint32_t((c - 1) / STAGES);
            if (!mbar_wait(smem_u32(&empty_bar[sp]), usep & 1u)) ok = false;
            else issue(c - 1 + STAGES);
        }
        if (c == 0 && tid < nvec) {
            float x[EPV];
            E::unpack(raw[0], x);
            float mx = x[0];
#pragma unroll
            for (int j = 1; j < EPV; ++j) mx = fmaxf(mx, x[j]);
            set_reference(a, r, mx);
            if constexpr (DENSE) update_bound(a, r);
        }
#pragma unroll
        for (int j = 0; j < VPT; ++j) {
            const int g = c * (CHUNK_BYTES / 16) + j * STEP_THREADS + tid;
            if (g < nvec) {
                float x[EPV];
                E::unpack(raw[j], x);
                consume<EPV, DENSE>(a, r, x, g * EPV, smask);
            }
        }
    }
    // ragged tail: V not a multiple of the vector width
    const int v = nvec * EPV + tid;
    if (v < V) {
        float x[1] = {E::load(rowp, v)};
        if (!a.touched) { set_reference(a, r, x[0]); if constexpr (DENSE) update_bound(a, r); }
        consume<1, DENSE>(a, r, x, v, smask);
    }
    return ok;
}

template <int DT, bool DENSE>
__device__ void stream_scalar(Acc& a, const RowCtx& r, const char* rowp, int V, const uint32_t* smask) {
    using E = Elem<DT>;
    for (int v = threadIdx.x; v < V; v += STEP_THREADS) {
        float x[1] = {E::load(rowp, v)};
        if (!a.touched) { set_reference(a, r, x[0]); if constexpr (DENSE) update_bound(a, r); }
        consume<1, DENSE>(a, r, x, v, smask);
    }
}

// ---- the kernel ---------------------------------------------------------------------------------
template <int DT, bool RING>
__global__ void __launch_bounds__(STEP_THREADS, 3) disc_step_kernel(const StepParams p) {
    using E = Elem<DT>;
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    unsigned char* ring = dyn_smem;                                             // RING_BYTES (RING only)
    uint32_t* smask = reinterpret_cast<uint32_t*>(dyn_smem + (RING ? RING_BYTES : 0));
    __shared__ __align__(8) uint64_t full_bar[STAGES];
    __shared__ __align__(8) uint64_t empty_bar[STAGES];
    __shared__ float red_f[6][STEP_WARPS];
    __shared__ int32_t red_i[2][STEP_WARPS];
    __shared__ float scratch[STEP_WARPS];
    __shared__ float fin[4];        // (m, s) of the full row and of the valid set
    __shared__ int32_t s_flag, s_tmp, s_fault;

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

    if (RING) {
        if (tid == 0) {
            for (int s = 0; s < STAGES; ++s) {
                mbar_init(smem_u32(&full_bar[s]), 1);
                mbar_init(smem_u32(&empty_bar[s]), STEP_WARPS);
            }
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
    }
    if (tid == 0) s_fault = 0;
    __syncthreads();

    const char* rowp = static_cast<const char*>(p.logits) + size_t(row) * size_t(p.ld) * E::SIZE;
    RowCtx r;
    r.c2 = p.c2; r.inv_t = p.inv_t; r.key = p.key; r.step = p.step; r.row = uint32_t(p.row_base + uint32_t(row));
    r.xref = E::load(rowp, 0);
    if (!(fabsf(r.xref) < CUDART_INF_F)) r.xref = 0.f;
    const bool dense = (c > DISC_HEAVY_MIN) || (p.mask_out != nullptr);

    Acc a;
    MS ok{-CUDART_INF_F, 0.f};
    bool poisoned = false;

    if (dense) {
        build_mask(smask, p, node, cb, ce, &s_tmp);
        if (p.mask_out) {
            uint32_t* mo = p.mask_out + size_t(row) * p.W;
            for (int w = tid; w < p.W; w += STEP_THREADS) mo[w] = smask[w];
        }
    } else {
        // gather path: the few allowed logits are read directly
        for (int i = tid; i < c; i += STEP_THREADS) {
            const int32_t v = __ldg(p.node_tok + cb + i);
            const float x = E::load(rowp, v);
            // sum of 2^(x*c2) kept as 2^m * s; fma(x, c2, -m) is the exact product minus the
            // reference, so a large common offset of the logits costs no accuracy
            const float y = x * p.c2;
            if (!(y < CUDART_INF_F)) poisoned = true;                 // NaN or +inf: careful path
            else if (y > ok.m) { ok.s = ok.s * exp2f(ok.m - y) + exp2f(fmaf(x, p.c2, -y)); ok.m = y; }
            else if (y != -CUDART_INF_F) ok.s += exp2f(fmaf(x, p.c2, -ok.m));
            const uint4 w4 = philox4x32_10(uint32_t(v) >> 2, r.step, r.row, 0u, r.key);
            const float score = gumbel_score(x, r.xref, r.inv_t, pick_word(w4, v & 3));
            if (score > a.best.score) { a.best.score = score; a.best.tok = v; a.best.child = cb + i; }
        }
    }

    // ---- stream the row
    bool waits_ok = true;
    if (RING) {
        waits_ok = dense ? stream_ring<DT, true>(a, r, rowp, p.V, ring, full_bar, empty_bar, smask)
                         : stream_ring<DT, false>(a, r, rowp, p.V, ring, full_bar, empty_bar, smask);
    } else {
        if (dense) stream_scalar<DT, true>(a, r, rowp, p.V, smask);
        else stream_scalar<DT, false>(a, r, rowp, p.V, smask);
    }
    if (!waits_ok) s_fault = 1;

    MS all = a.touched ? MS{a.mref, a.s_all0 + a.s_all1} : MS{-CUDART_INF_F, 0.f};
    if (dense) ok = a.touched ? MS{a.mref, a.s_ok} : MS{-CUDART_INF_F, 0.f};
    if (poisoned) ok.s = CUDART_NAN_F;
    Best best = a.best;

    const int any_lost = __syncthreads_or(a.lost ? 1 : 0);
    if (s_fault) {
        // A bulk copy never signalled completion.  Report it and leave the row untouched; give
        // outstanding copies a bounded time to land before the block's shared memory is released.
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
        if (tid == 0) { p.token_out[row] = -1; p.status_out[row] = DISC_ROW_FAULT; }
        return;
    }

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
    }
    __syncthreads();       // every warp has read its red_* partials; lane 0 may now overwrite slot 0
    if (warp == 0 && lane == 0) {
        fin[0] = all.m; fin[1] = all.s; fin[2] = ok.m; fin[3] = ok.s;
        const float l2_all = all.m + log2f(all.s);
        const float l2_ok = ok.m + log2f(ok.s);
        // the fast sums are trusted only when both are finite and no allowed term was lost
        s_flag = (fabsf(l2_all) < CUDART_INF_F && fabsf(l2_ok) < CUDART_INF_F && !any_lost) ? 0 : 1;
        red_f[4][0] = best.score; red_i[0][0] = best.tok; red_i[1][0] = best.child;
    }
    __syncthreads();

    if (s_flag) {
        // ---- careful path: plain two-pass log-sum-exp over the row with an explicit mask and
        // separate maxima for the full row and for the valid set; in the dense path the scores of
        // all allowed tokens are evaluated exactly again (its skip bound relies on terms that did
        // not underflow)
        if (!dense) build_mask(smask, p, node, cb, ce, &s_tmp);
        float mx_all = -CUDART_INF_F, mx_ok = -CUDART_INF_F;
        int nan_all = 0, nan_ok = 0;
        Best cbest{-CUDART_INF_F, -1, -1};
        for (int v = tid; v < p.V; v += STEP_THREADS) {
            const float x = E::load(rowp, v);
            const bool allowed = (smask[v >> 5] >> (v & 31)) & 1u;
            if (x != x) { nan_all = 1; nan_ok |= allowed; }
            else { mx_all = fmaxf(mx_all, x); if (allowed) mx_ok = fmaxf(mx_ok, x); }
            if (allowed && dense) {
                const uint4 w4 = philox4x32_10(uint32_t(v) >> 2, r.step, r.row, 0u, r.key);
                const float score = gumbel_score(x, r.xref, r.inv_t, pick_word(w4, v & 3));
                if (score > cbest.score) { cbest.score = score; cbest.tok = v; }
            }
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
        if (dense) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                Best b2{__shfl_xor_sync(0xffffffffu, cbest.score, o), __shfl_xor_sync(0xffffffffu, cbest.tok, o), -1};
                cbest = best_merge(cbest, b2);
            }
            __syncthreads();
            if (lane == 0) { red_f[5][warp] = cbest.score; red_i[0][warp] = cbest.tok; }
            __syncthreads();
            if (tid == 0) {
                Best b{red_f[5][0], red_i[0][0], -1};
                for (int w = 1; w < STEP_WARPS; ++w) b = best_merge(b, Best{red_f[5][w], red_i[0][w], -1});
                red_f[4][0] = b.score; red_i[0][0] = b.tok; red_i[1][0] = -1;
            }
        }
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
        int32_t tok = red_i[0][0], child = red_i[1][0];
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

template <int DT, bool RING>
int launch_step(const StepParams& p, int64_t n, size_t smem, cudaStream_t st) {
    DISC_CUDA(cudaFuncSetAttribute(disc_step_kernel<DT, RING>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   int(smem)));
    disc_step_kernel<DT, RING><<<unsigned(n), STEP_THREADS, smem, st>>>(p);
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
    const size_t mask_bytes = (size_t(s->W) * 4 + 15) & ~size_t(15);
    if (mask_bytes > 160 * 1024) return DISC_ERR_UNSUPPORTED;

    StepParams p;
    p.logits = logits; p.ld = ld; p.inv_t = inv_temperature; p.c2 = inv_temperature * LOG2E_F;
    p.key = philox_key(seed); p.step = step; p.row_base = uint32_t(row_base);
    p.node = node; p.lo = lo; p.hi = hi; p.depth = depth; p.logw = logw; p.done = done;
    p.token_out = token_out; p.seq_tokens = seq_tokens; p.seq_ld = seq_ld;
    p.logq_out = logq_out; p.logp_out = logp_out; p.mask_out = mask_out; p.status_out = status_out;
    p.node_tok = s->node_tok; p.node_lo = s->node_lo; p.child_begin = s->child_begin;
    p.root_child = s->root_child; p.root_mask = s->root_mask;
    p.heavy_nodes = s->heavy_nodes; p.heavy_masks = s->heavy_masks; p.n_heavy = s->n_heavy;
    p.V = s->V; p.W = s->W; p.M = s->M;

    const size_t esize = dtype == DISC_F32 ? 4 : 2;
    // the bulk-copy ring needs 16-byte aligned rows; other layouts take the scalar path
    const bool ring = (reinterpret_cast<uintptr_t>(logits) % 16 == 0) && ((size_t(ld) * esize) % 16 == 0);
    const size_t smem = mask_bytes + (ring ? RING_BYTES : 0);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (dtype == DISC_F32) return ring ? launch_step<DISC_F32, true>(p, n, smem, st) : launch_step<DISC_F32, false>(p, n, smem, st);
    return ring ? launch_step<DISC_BF16, true>(p, n, smem, st) : launch_step<DISC_BF16, false>(p, n, smem, st);
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
