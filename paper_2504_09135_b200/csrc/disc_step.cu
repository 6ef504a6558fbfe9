// disc_step: one decoding step of Algorithm 1 (lines 5-8) for a batch of candidates, fused:
// valid-set lookup, masked and unmasked log-sum-exp over the V logits, sampling from the masked
// distribution, importance log-weight update and the move of the row's cursor to the extended
// prefix.
//
// One thread block per row.
//   * Streaming.  The row is read with plain read-only 16-byte loads.  Sparse rows: thread t takes
//     vectors t, t+128, ... with seven independent loads in flight; dense rows: a 16 KB chunk has
//     256 slots, slot s owns vectors s, s+256, s+512, s+768 (four loads in flight), and the block
//     passes over the slots 128 at a time.  Seven blocks per SM keep some 100 KB per SM in
//     flight.  (A shared-memory ring filled by bulk asynchronous copies was measured slower than
//     this on the same data, and needed waits that this version does not have.)  Rows that are
//     not 16-byte aligned take a scalar-load path.
//   * Latency.  Outside its streaming loop a block follows a chain of dependent loads (state,
//     child range, child tokens, their logits; at the end the winner's index entries).  Loads
//     that depend on nothing are issued first and together; each thread's first child token is
//     fetched before the streaming loop and its logit during it; the gather work runs after the
//     loop; a row with a single valid token draws nothing and has its next cursor prefetched.
//   * Sums.  Each thread accumulates sum 2^(x*c - ref) against its own reference (the maximum of
//     the first logits it sees), c = log2(e)/T.  Per pair of logits: two unpack operations, one
//     packed fp32x2 FMA, two ex2 and one packed add.  Partial sums are kept as (m, s) pairs meaning
//     2^m * s and brought to a common reference before they are added.  All differences are
//     formed between references before any large value is added, so a common offset of the logits
//     does not cost accuracy.
//   * Valid set.  The prefix index gives the row's children as a contiguous list.  Rows with at
//     most DISC_HEAVY_MIN children gather their few logits directly ("gather path").  Rows with
//     more have a prebuilt bitmask row in global memory (a few MB in total, L2 resident), read
//     one byte per group of 8 tokens next to the logits it covers ("dense path").
//   * Sampling (exact draw from P.mask/|P.mask|_1, Algorithm 1 line 7) in two stages.  Stage 1 is
//     Gumbel-max over groups of 8 consecutive token ids: score_G = log(allowed mass of G) + g_G,
//     g_G = -log(-log u_G), u_G from Philox4x32-10 keyed by (group, step, row); the best group
//     wins, the lowest on a tie.  Stage 2 is an inverse-CDF draw among the winner's allowed tokens
//     with one more uniform.  In the dense path a group is evaluated exactly only if it can still
//     win: with w = 1 - u, g > t implies w < e^-t, so a group whose w is at least
//     mass_G / e^best (times a safety factor) is skipped without taking a logarithm; mass_G is
//     the already accumulated sum of 2^(x*c - ref) times a per-thread constant.  `best` is the
//     best score any lane of the warp has seen (shared when a lane improves it).  The four
//     groups a slot owns in one chunk share one Philox call, issued right after the slot's loads
//     so that its integer chain overlaps with the load latency and the exponentials.
//   * A row whose fast sums are not finite, or whose valid mass is so small that terms may have
//     underflowed against a thread's reference, is redone by a plain two-pass routine with exact
//     scores ("careful path").

#include <math_constants.h>

#include <type_traits>

#include "disc_internal.cuh"

// 128 threads per row and 7 blocks per SM (72 registers per thread) measured best on B200 for a
// whole decode: small blocks keep the share of time a block spends outside its streaming loop low,
// and seven loads in flight per thread (sparse rows) keep a lone row fast when few rows are left
// (seven measured 1.5 % faster over a whole decode than eight, six 1.3 %, five 0.4 %).
#ifndef DISC_MIN_BLOCKS
#define DISC_MIN_BLOCKS 7
#endif

namespace {

using namespace disc;

#ifndef DISC_STEP_THREADS
#define DISC_STEP_THREADS 128
#endif
constexpr int STEP_THREADS = DISC_STEP_THREADS;
constexpr int STEP_WARPS = STEP_THREADS / 32;
constexpr int VPT = 4;                                   // 16-byte vectors in flight per thread
constexpr int SLOTS = 256;                               // a chunk is SLOTS x VPT vectors = 16 KB of the row;
constexpr int CHUNK_VECS = VPT * SLOTS;                  // slot s owns vectors s, s+256, s+512, s+768 of it
static_assert(SLOTS % STEP_THREADS == 0 && STEP_THREADS % 32 == 0, "a block covers a chunk in whole passes");
constexpr int GROUP = 8;                                 // tokens per sampling group
constexpr float LOG2E_F = 1.4426950408889634f;
constexpr float LN2_F = 0.6931471805599453f;
constexpr float SAFETY = 1.0009765625f;                 // 1 + 2^-10 on the skip bound
constexpr float TWO_M24 = 5.9604644775390625e-08f;      // 2^-24: smallest possible w
constexpr float MASS_FLOOR_LOG2 = 60.f;   // dense sums are trusted while log2(mass) >= -60 (see below)

struct StepParams {
    const void* logits;
    int64_t ld;
    float inv_t;
    float c2;            // inv_t * log2(e)
    PhiloxRoundKeys rk;
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
    int32_t V, W, Wp, n_heavy;
    int64_t M;
    // the sums over the whole vocabulary given from outside (the fused projection): per row n_parts
    // pairs (m, s), sum over the part = 2^m * s; used by rows that take the gather path
    const float2* parts;
    int32_t n_parts;
    // top-M mode: the row's candidate tokens (ascending id) and which of them were verified; the
    // valid set of the row is the verified candidates instead of the node's children
    const int32_t* cand;
    const uint8_t* cand_valid;
    int32_t cand_M;
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

// sum of 2^(x*c2) kept as 2^m * s; fma(x, c2, -m) is the exact product minus the reference, so a
// large common offset of the logits costs no accuracy.  NaN and +inf poison the sum (s = NaN).
__device__ __forceinline__ void ms_add(MS& a, float x, float c2) {
    const float y = x * c2;
    if (!(y < CUDART_INF_F)) a.s = CUDART_NAN_F;
    else if (y > a.m) { a.s = a.s * exp2f(a.m - y) + exp2f(fmaf(x, c2, -y)); a.m = y; }
    else if (y != -CUDART_INF_F) a.s += exp2f(fmaf(x, c2, -a.m));
}

struct Best {
    float score;
    int32_t key;     // -1: none yet; dense rows: winning group (token id >> 3); gather rows: the token
                     // already drawn inside the winning group
    int32_t child;   // gather rows: index node of that token, else -1
};

__device__ __forceinline__ Best best_merge(Best a, Best b) {
    if (b.key < 0) return a;
    if (a.key < 0) return b;
    if (b.score > a.score || (b.score == a.score && b.key < a.key)) return b;
    return a;
}

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// ---- element types ------------------------------------------------------------------------------
template <int DT>
struct Elem;
template <>
struct Elem<DISC_F32> {
    static constexpr int SIZE = 4;
    static constexpr int EPV = 4;       // elements per 16-byte vector
    __device__ static __forceinline__ float load(const void* base, int64_t i) {
        return __ldg(static_cast<const float*>(base) + i);
    }
    __device__ static __forceinline__ void unpack(const uint4& v, float2* x) {
        x[0] = make_float2(__uint_as_float(v.x), __uint_as_float(v.y));
        x[1] = make_float2(__uint_as_float(v.z), __uint_as_float(v.w));
    }
};
template <>
struct Elem<DISC_BF16> {
    static constexpr int SIZE = 2;
    static constexpr int EPV = 8;
    __device__ static __forceinline__ float load(const void* base, int64_t i) {
        return __uint_as_float(uint32_t(__ldg(static_cast<const unsigned short*>(base) + i)) << 16);
    }
    __device__ static __forceinline__ float2 pair(uint32_t w) {
        return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
    }
    __device__ static __forceinline__ void unpack(const uint4& v, float2* x) {
        x[0] = pair(v.x); x[1] = pair(v.y); x[2] = pair(v.z); x[3] = pair(v.w);
    }
};

// ---- sampling helpers ---------------------------------------------------------------------------
// Philox counter word 0 and output word of group G.  The four groups a thread owns in one
// chunk (256 apart) share a counter.
__device__ __forceinline__ uint32_t group_slot(uint32_t G) { return ((G >> 10) << 8) | (G & 255u); }
__device__ __forceinline__ uint32_t group_word(uint32_t G) { return (G >> 8) & 3u; }

// Exact score of a group whose allowed mass is 2^mlog2 (relative to the row's reference logit):
// ln(mass) + Gumbel noise.  Kept out of line: it runs for a handful of groups per warp and row.
__device__ __noinline__ float group_score(float mlog2, uint32_t word) {
    return mlog2 * LN2_F + gumbel_from_uniform(uniform_from_bits(word));
}

// w = 1 - u of a random word, exact: with k' the complement of the word's top 23 bits,
// w = (2k'+1) * 2^-24.  No integer-to-float conversion is needed: 1.k' - (1 - 2^-24).
__device__ __forceinline__ float complement_uniform(uint32_t word) {
    return __uint_as_float(0x3f800000u | ((~word) >> 9)) - 0.99999994039535522f;
}

__device__ __forceinline__ uint32_t mask_byte(const uint32_t* __restrict__ gmask, uint32_t G) {
    return (__ldg(gmask + (G >> 2)) >> ((G & 3u) * 8u)) & 0xFFu;
}

// Per-thread accumulators of the streaming loop.
struct Acc {
    float mref = 0.f;        // reference exponent (log2 domain) of this thread's sums
    float2 sa = {0.f, 0.f}, sb = {0.f, 0.f};      // four partial sums over all logits
    float2 ok2 = {0.f, 0.f};                      // two partial sums over the allowed logits
    bool touched = false;
    bool improved = false;   // bound_best rose since the warp last shared its bounds
    // sampling
    Best best{-__builtin_huge_valf(), -1, -1};
    float bound_best = -__builtin_huge_valf();   // best score known to this warp (>= best.score)
    float cbase = 0.f;                            // mref - xref*c: log2 of (thread sums -> row-relative mass)
    float cbound = __builtin_huge_valf();   // SAFETY * 2^(cbase - bound_best*log2e): t*cbound >= mass/e^best
};

struct RowCtx {
    float c2, inv_t, xref;
    uint32_t step, row;
};

__device__ __forceinline__ void update_bound(Acc& a) {
    a.cbound = SAFETY * exp2f(a.cbase - a.bound_best * LOG2E_F);
}

__device__ __forceinline__ void set_reference(Acc& a, const RowCtx& r, float xmax) {
    const float m = xmax * r.c2;
    a.mref = (fabsf(m) < CUDART_INF_F) ? m : 0.f;
    a.cbase = fmaf(-r.xref, r.c2, a.mref);      // one rounding of the exact difference
    a.touched = true;
    update_bound(a);
}

// exact evaluation of group G whose allowed terms sum to t (against this thread's reference)
__device__ __forceinline__ void exact_group(Acc& a, float t, uint32_t word, int32_t G) {
    // Groups arrive in ascending order inside a thread, so strict '>' keeps the lowest group on a
    // tie.  NaN and -inf scores never win; a row without any finite score falls back to its
    // lowest valid token at the end.
    const float score = group_score(a.cbase + log2f(t), word);
    if (score > a.best.score) { a.best.score = score; a.best.key = G; a.best.child = -1; }
    if (score > a.bound_best) { a.bound_best = score; a.improved = true; update_bound(a); }
}

// skip test + exact evaluation of one group
__device__ __forceinline__ void sample_group(Acc& a, float t, uint32_t word, int32_t G) {
    if (!(complement_uniform(word) >= t * a.cbound)) exact_group(a, t, word, G);
}

// share the best score of the warp's lanes (called at warp-uniform points)
__device__ __forceinline__ void share_bound(Acc& a) {
    float b = a.bound_best;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) b = fmaxf(b, __shfl_xor_sync(0xffffffffu, b, o));
    a.bound_best = b;
    update_bound(a);
}

// exponentials of one 16-byte vector; returns their pairwise sum in t
template <int DT>
__device__ __forceinline__ float2 vec_exp(const Acc& a, const RowCtx& r, const uint4& raw, float2* e) {
    using E = Elem<DT>;
    constexpr int NP = E::EPV / 2;
    float2 x[NP];
    E::unpack(raw, x);
    const float2 cc = make_float2(r.c2, r.c2), nm = make_float2(-a.mref, -a.mref);
#pragma unroll
    for (int i = 0; i < NP; ++i) {
        const float2 y = __ffma2_rn(x[i], cc, nm);
        e[i] = make_float2(ex2_approx(y.x), ex2_approx(y.y));
    }
    float2 t = __fadd2_rn(e[0], e[1]);
    if constexpr (NP == 4) t = __fadd2_rn(t, __fadd2_rn(e[2], e[3]));
    return t;
}

// sparse rows: one 16-byte vector of logits
template <int DT>
__device__ __forceinline__ void consume_vec_sparse(Acc& a, const RowCtx& r, const uint4& raw) {
    using E = Elem<DT>;
    constexpr int NP = E::EPV / 2;
    float2 x[NP];
    E::unpack(raw, x);
    const float2 cc = make_float2(r.c2, r.c2), nm = make_float2(-a.mref, -a.mref);
#pragma unroll
    for (int i = 0; i < NP; i += 2) {
        const float2 y0 = __ffma2_rn(x[i], cc, nm), y1 = __ffma2_rn(x[i + 1], cc, nm);
        a.sa = __fadd2_rn(a.sa, make_float2(ex2_approx(y0.x), ex2_approx(y0.y)));
        a.sb = __fadd2_rn(a.sb, make_float2(ex2_approx(y1.x), ex2_approx(y1.y)));
    }
}

// dense rows: the allowed part of one vector's exponentials; nb = allowed flags of its tokens.
// tab[f] holds the four flags of nibble f as floats (1 or 0), so that masking is a multiply-add on
// the packed pipe and costs the same whatever the mask looks like.  (A non-finite exponential times
// a zero flag gives NaN; such rows have a non-finite full sum as well and are redone by the careful
// path.)
template <int NP>
__device__ __forceinline__ float masked_sum(const float2* e, const float4* __restrict__ tab, uint32_t nb) {
    const float4 m0 = tab[nb & 15u];
    float2 acc = __fmul2_rn(e[0], make_float2(m0.x, m0.y));
    acc = __ffma2_rn(e[1], make_float2(m0.z, m0.w), acc);
    if constexpr (NP == 4) {
        const float4 m1 = tab[(nb >> 4) & 15u];
        acc = __ffma2_rn(e[2], make_float2(m1.x, m1.y), acc);
        acc = __ffma2_rn(e[3], make_float2(m1.z, m1.w), acc);
    }
    return acc.x + acc.y;
}

// one group given as up to 8 scalars (scalar path, ragged tails, careful use): x[j] for j < nvalid
template <bool DENSE>
__device__ __forceinline__ void consume_group_scalar(Acc& a, const RowCtx& r, const PhiloxRoundKeys& rk,
                                                     const float* x, int nvalid, uint32_t G, uint32_t bits) {
    if (!a.touched) {
        float mx = x[0];
        for (int j = 1; j < nvalid; ++j) mx = fmaxf(mx, x[j]);
        set_reference(a, r, mx);
    }
    float t = 0.f;
    for (int j = 0; j < nvalid; ++j) {
        const float e = ex2_approx(fmaf(x[j], r.c2, -a.mref));
        a.sa.x += e;
        if (DENSE && ((bits >> j) & 1u)) t += e;
    }
    if (DENSE && bits) {
        a.ok2.x += t;
        if (!(t * a.cbound < TWO_M24)) {
            const uint4 w4 = philox4x32_10(group_slot(G), r.step, r.row, 0u, rk);
            sample_group(a, t, pick_word(w4, group_word(G)), int32_t(G));
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
// 16-byte read-only load of streamed data (not worth keeping in L1)
__device__ __forceinline__ uint4 ld_stream16(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Dense rows: the first n_groups whole groups of the row, read with 16-byte loads.
// A chunk of CHUNK_VECS vectors has 256 slots and the block passes over them STEP_THREADS at a
// time.  A slot works on groups of 8 tokens: bf16 - vectors s, s+256, s+512, s+768 of the chunk
// (one group each); f32 - groups s and s+256 of the chunk's 512 (two adjacent vectors each).
// Either way the groups of one slot are 256 apart and share a Philox counter.
template <int DT>
__device__ __forceinline__ void stream_dense(Acc& a, const RowCtx& r, const PhiloxRoundKeys& rk, const char* rowp,
                                             const uint32_t* gmask, int n_groups, const float4* tab) {
    using E = Elem<DT>;
    constexpr int EPV = E::EPV;
    constexpr int NP = EPV / 2;
    constexpr int VPG = GROUP / EPV;                          // vectors per group: 1 (bf16) or 2 (f32)
    constexpr int GPT = VPT / VPG;                            // groups per thread and chunk
    constexpr int GPC = GPT * SLOTS;                          // groups per chunk
    const uint4* row4 = reinterpret_cast<const uint4*>(rowp);
    const unsigned char* gbytes = reinterpret_cast<const unsigned char*>(gmask);
    const int nvec = n_groups * VPG;
    const int n_chunks = (nvec + CHUNK_VECS - 1) / CHUNK_VECS;
    const int n_full = nvec / CHUNK_VECS;

    for (int c = 0; c < n_chunks; ++c) {
        auto body = [&](auto full_tag, int slot) {
            constexpr bool FULL = decltype(full_tag)::value;
            uint4 raw[VPT];
            uint32_t bits[GPT];
            bool have[VPT];
            // vector index inside the chunk of this thread's k-th vector
            auto vidx = [&](int k) { return ((k / VPG) * SLOTS + slot) * VPG + (k % VPG); };
#pragma unroll
            for (int k = 0; k < VPT; ++k) {
                have[k] = FULL || (c * CHUNK_VECS + vidx(k) < nvec);
                if (have[k]) raw[k] = ld_stream16(row4 + c * CHUNK_VECS + vidx(k));
            }
#pragma unroll
            for (int j = 0; j < GPT; ++j) {
                const int G = c * GPC + j * SLOTS + slot;
                bits[j] = (FULL || G < n_groups) ? uint32_t(__ldg(gbytes + G)) : 0u;
            }
            // The random words of the slot's groups, computed here and not where they are used: the
            // integer work then overlaps with the exponentials below.  (Skipping the call when every
            // group of the slot is hopeless even with the luckiest noise was measured: it almost
            // never applies, even for very peaked logits, and costs the overlap.)
            const uint32_t G0 = uint32_t(c * GPC + slot);
            const uint4 w4 = philox4x32_10(group_slot(G0), r.step, r.row, 0u, rk);
            if (!a.touched && have[0]) {
                float2 x[NP];
                E::unpack(raw[0], x);
                float mx = fmaxf(x[0].x, x[0].y);
#pragma unroll
                for (int i = 1; i < NP; ++i) mx = fmaxf(mx, fmaxf(x[i].x, x[i].y));
                set_reference(a, r, mx);
            }
            {
                float tg[GPT];
#pragma unroll
                for (int j = 0; j < GPT; ++j) {
                    tg[j] = 0.f;
#pragma unroll
                    for (int h = 0; h < VPG; ++h) {
                        const int k = j * VPG + h;
                        if (have[k]) {
                            float2 e[NP];
                            const float2 t = vec_exp<DT>(a, r, raw[k], e);
                            a.sa = __fadd2_rn(a.sa, t);
                            tg[j] += masked_sum<NP>(e, tab, bits[j] >> (h * EPV));
                        }
                    }
                    a.ok2.x += tg[j];
                }
                // stage 1 of the sampling for this slot's groups of the chunk.  One test for all of
                // them first: the largest of the four words gives the smallest w, the largest group
                // mass the largest right-hand side.
                float tmax = tg[0];
#pragma unroll
                for (int j = 1; j < GPT; ++j) tmax = fmaxf(tmax, tg[j]);
                const uint32_t wmax = max(max(w4.x, w4.y), max(w4.z, w4.w));
                if (!(complement_uniform(wmax) >= tmax * a.cbound)) {
#pragma unroll
                    for (int j = 0; j < GPT; ++j) {
                        const uint32_t G = G0 + uint32_t(j * SLOTS);
                        sample_group(a, tg[j], pick_word(w4, group_word(G)), int32_t(G));
                    }
                }
                // a better score found by any lane tightens the whole warp's bound
                if (__any_sync(0xffffffffu, a.improved)) {
                    share_bound(a);
                    a.improved = false;
                }
            }
        };
        for (int slot = threadIdx.x; slot < SLOTS; slot += STEP_THREADS) {
            if (c < n_full) body(std::true_type{}, slot); else body(std::false_type{}, slot);
        }
    }
}

#ifndef DISC_SPARSE_UNROLL
#define DISC_SPARSE_UNROLL 7
#endif
// Sparse rows need only the sum over all logits, so any split of the vectors will do: thread t
// takes vectors t, t+T, t+2T, ... and keeps DISC_SPARSE_UNROLL loads in flight.
// `after_first` runs once, right after the first batch of loads has been consumed (or at once if
// the row is shorter than a batch): the kernel uses it to issue loads whose addresses have arrived
// in the meantime.
template <int DT, class Hook>
__device__ __forceinline__ void stream_sparse(Acc& a, const RowCtx& r, const char* rowp, int n_groups,
                                              Hook after_first) {
    using E = Elem<DT>;
    constexpr int NP = E::EPV / 2;
    constexpr int U = DISC_SPARSE_UNROLL;
    const uint4* row4 = reinterpret_cast<const uint4*>(rowp);
    const int nvec = n_groups * (GROUP / E::EPV);
    int i = threadIdx.x;
    if (i < nvec) {
        float2 x[NP];
        E::unpack(__ldg(row4 + i), x);
        float mx = fmaxf(x[0].x, x[0].y);
#pragma unroll
        for (int k = 1; k < NP; ++k) mx = fmaxf(mx, fmaxf(x[k].x, x[k].y));
        set_reference(a, r, mx);
    }
    bool first = true;
    for (; i + (U - 1) * STEP_THREADS < nvec; i += U * STEP_THREADS) {
        uint4 raw[U];
#pragma unroll
        for (int u = 0; u < U; ++u) raw[u] = ld_stream16(row4 + i + u * STEP_THREADS);
        if (first) { after_first(); first = false; }
#pragma unroll
        for (int u = 0; u < U; ++u) consume_vec_sparse<DT>(a, r, raw[u]);
    }
    if (first) after_first();
    for (; i < nvec; i += STEP_THREADS) consume_vec_sparse<DT>(a, r, ld_stream16(row4 + i));
}

// groups [g_begin, g_end) of the row read with scalar loads (whole row on the scalar path; the
// ragged last group on the vector path)
template <int DT, bool DENSE>
__device__ void stream_groups_scalar(Acc& a, const RowCtx& r, const PhiloxRoundKeys& rk, const char* rowp, int V,
                                     const uint32_t* gmask, int g_begin, int g_end) {
    using E = Elem<DT>;
    for (int G = g_begin + threadIdx.x; G < g_end; G += STEP_THREADS) {
        float x[GROUP];
        const int v0 = G * GROUP;
        const int nvalid = min(GROUP, V - v0);
        for (int j = 0; j < nvalid; ++j) x[j] = E::load(rowp, v0 + j);
        const uint32_t bits = DENSE ? mask_byte(gmask, uint32_t(G)) : 0u;
        consume_group_scalar<DENSE>(a, r, rk, x, nvalid, uint32_t(G), bits);
    }
}

// ---- the kernel ---------------------------------------------------------------------------------
// MODE 1 (sums given): rows that take the gather path do not stream their logits; their sum over
// the whole vocabulary comes from p.parts, and only the logits of their valid tokens are read (the
// rest of the row need not have been written).
// MODE 2 (top-M): as mode 1, and the valid set of a row is its verified candidates (p.cand,
// p.cand_valid; at most TOPM_MAX of them) instead of the children of its node; every row takes the
// gather path; a row without a verified candidate has run into a dead end.
constexpr int TOPM_MAX = 1024;
template <int DT, bool VEC, int MODE = 0>
__global__ void __launch_bounds__(STEP_THREADS, DISC_MIN_BLOCKS)
disc_step_kernel(const __grid_constant__ StepParams p) {
    constexpr bool PARTS = MODE >= 1;
    constexpr bool LIST = MODE == 2;
    __shared__ int32_t s_list[LIST ? TOPM_MAX : 1];
    __shared__ int32_t s_count;
    using E = Elem<DT>;
    __shared__ float red_f[6][STEP_WARPS];
    __shared__ int32_t red_i[2][STEP_WARPS];
    __shared__ float scratch[STEP_WARPS];
    __shared__ float fin[4];        // (m, s) of the full row and of the valid set
    __shared__ int32_t s_flag, s_tmp;
    __shared__ __align__(16) float4 flag_tab[16];   // the four bits of a nibble as floats (dense rows)

    const int64_t row = blockIdx.x;
    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;

    // The block's time outside its streaming loop is a chain of dependent loads; everything that
    // does not depend on anything is fetched here, side by side.
    const char* rowp = static_cast<const char*>(p.logits) + size_t(row) * size_t(p.ld) * E::SIZE;
    const uint8_t was_done = p.done[row];
    const int32_t node = p.node[row];
    const int32_t depth_old = tid == 0 ? p.depth[row] : 0, hi_old = tid == 0 ? p.hi[row] : 0;
    if (was_done) {
        if (tid == 0) { p.token_out[row] = -1; p.status_out[row] = DISC_ROW_DONE; }
        return;
    }
    const float x_first_logit = PARTS ? 0.f : E::load(rowp, 0);     // with PARTS element 0 may not have been written
    const int n_groups = (p.V + GROUP - 1) / GROUP;       // the last one may be ragged
    const int n_vec_groups = VEC ? p.V / GROUP : 0;       // whole groups are read with 16-byte loads

    int32_t cb = 0, ce = 0;
    if (node >= 0 && int64_t(node) < p.M) { cb = __ldg(p.child_begin + node); ce = __ldg(p.child_begin + node + 1); }
    int32_t c = ce - cb;
    if (c <= 0) {   // not a prefix of any member, or already a complete member
        if (tid == 0) {
            p.token_out[row] = -1;
            bool leaf = node > 0 && int64_t(node) < p.M;
            p.status_out[row] = leaf ? DISC_ROW_DONE : DISC_ROW_DEAD;
            if (leaf) p.done[row] = 1;
        }
        return;
    }

    if (LIST) {
        // the verified candidates, in ascending id, become the row's valid set
        if (warp == 0) {
            const int32_t* cd = p.cand + size_t(row) * p.cand_M;
            const uint8_t* ok = p.cand_valid + size_t(row) * p.cand_M;
            int32_t cnt = 0;
            for (int j0 = 0; j0 < p.cand_M; j0 += 32) {
                const int j = j0 + lane;
                const int32_t v = j < p.cand_M ? cd[j] : -1;
                const bool keep = j < p.cand_M && v >= 0 && v < p.V && ok[j] != 0;
                const uint32_t bal = __ballot_sync(0xffffffffu, keep);
                if (keep) s_list[cnt + __popc(bal & ((1u << lane) - 1u))] = v;
                cnt += __popc(bal);
            }
            if (lane == 0) s_count = cnt;
        }
        __syncthreads();
        c = s_count;
        if (c == 0) {   // none of the candidates extends the prefix: Algorithm 1's "a in S" will fail for this row
            if (tid == 0) {
                p.token_out[row] = -1;
                p.status_out[row] = DISC_ROW_DEAD;
                p.done[row] = 1;
                p.logw[row] = -CUDART_INF_F;
            }
            return;
        }
    }
    auto kid = [&](int32_t i) -> int32_t { return LIST ? s_list[i] : __ldg(p.node_tok + cb + i); };

    // dense rows: locate the prebuilt mask row (root, or a heavy node)
    if (VEC && tid >= 32 && tid < 48) {
        const int f = tid - 32;
        flag_tab[f] = make_float4(float(f & 1), float((f >> 1) & 1), float((f >> 2) & 1), float((f >> 3) & 1));
    }
    int32_t hsel = -2;                                    // -2: not dense
    if (!LIST && (node == 0 || c > DISC_HEAVY_MIN)) {     // the same for every thread of the block
        if (tid == 0) {
            int32_t h = -2;
            if (node == 0) h = -1;                        // -1: the root's row
            else { h = heavy_index(p.heavy_nodes, p.n_heavy, node); if (h < 0) h = -2; }
            s_tmp = h;
        }
        __syncthreads();
        hsel = s_tmp;
    }
    const bool dense = hsel != -2;
    const uint32_t* gmask = !dense ? nullptr : (hsel == -1 ? p.root_mask : p.heavy_masks + size_t(hsel) * p.Wp);

    RowCtx r;
    r.c2 = p.c2; r.inv_t = p.inv_t; r.step = p.step; r.row = uint32_t(p.row_base + uint32_t(row));
    r.xref = x_first_logit;
    if (!(fabsf(r.xref) < CUDART_INF_F)) r.xref = 0.f;

    Acc a;
    MS ok{-CUDART_INF_F, 0.f};

    if (p.mask_out) {
        // optional output of the valid-set mask
        uint32_t* mo = p.mask_out + size_t(row) * p.W;
        if (dense) {
            for (int w = tid; w < p.W; w += STEP_THREADS) mo[w] = __ldg(gmask + w);
        } else {
            for (int w = tid; w < p.W; w += STEP_THREADS) mo[w] = 0u;
            __syncthreads();
            for (int i = tid; i < c; i += STEP_THREADS) {
                const int32_t t = kid(i);
                atomicOr(&mo[t >> 5], 1u << (t & 31));
            }
        }
    }
    // Loads of the gather path and of the final cursor update that can be issued now and used
    // after the row has been streamed: this thread's first child; for a row with a single child
    // (a forced step, the common case deep in the tree) the child's index entries as well.
    const int32_t v_mine = (!dense && tid < c) ? kid(tid) : -1;
    float x_mine = 0.f;
    int32_t only_lo = 0, only_cb = 0, only_ce = 0;
    if (!LIST && c == 1 && tid == 0) {
        only_lo = __ldg(p.node_lo + cb);
        only_cb = __ldg(p.child_begin + cb);
        only_ce = __ldg(p.child_begin + cb + 1);
    }

    // ---- stream the row
    const bool use_parts = PARTS && !dense;
    MS all_parts{-CUDART_INF_F, 0.f};
    if (use_parts) {
        const float2* pr = p.parts + size_t(row) * p.n_parts;
        for (int j = tid; j < p.n_parts; j += STEP_THREADS) {
            const float2 v = __ldg(pr + j);
            all_parts = ms_merge(all_parts, MS{v.x, v.y});
        }
        if (v_mine >= 0) x_mine = E::load(rowp, v_mine);
    } else if (VEC) {
        if (dense) stream_dense<DT>(a, r, p.rk, rowp, gmask, n_vec_groups, flag_tab);
        else stream_sparse<DT>(a, r, rowp, n_vec_groups, [&] { if (v_mine >= 0) x_mine = E::load(rowp, v_mine); });
    } else if (v_mine >= 0) {
        x_mine = E::load(rowp, v_mine);
    }
    if (dense) stream_groups_scalar<DT, true>(a, r, p.rk, rowp, p.V, gmask, n_vec_groups, n_groups);
    else if (!use_parts) stream_groups_scalar<DT, false>(a, r, p.rk, rowp, p.V, gmask, n_vec_groups, n_groups);

    if (!dense) {
        // ---- gather path: the few allowed logits are read directly.  Every thread adds its child to
        // the valid-set sum; the thread holding the first child of a group also collects the
        // group's members (at most 8 children), forms the group's exact score and, if that score
        // is the best it has seen, draws the token inside the group right away (stage 2), so that
        // nothing of this is left for the end of the block.
        // The first child of every thread was fetched before the row was streamed and its logit
        // while the row was streamed (see above).
        for (int i = tid; i < c; i += STEP_THREADS) {
            const int32_t v = i == tid ? v_mine : kid(i);
            const float x = i == tid ? x_mine : E::load(rowp, v);
            ms_add(ok, x, p.c2);
            const int32_t G = v >> 3;
            if (c == 1) {           // a forced step: nothing to draw
                a.best.score = 0.f; a.best.key = v; a.best.child = LIST ? -1 : cb;
                break;
            }
            const bool leader = (i == 0) || ((kid(i - 1) >> 3) != G);
            if (leader) {
                float xs[GROUP];
                xs[0] = x;
                int n = 1;
#pragma unroll
                for (int k = 1; k < GROUP; ++k) {
                    if (n == k && i + k < c) {
                        const int32_t v2 = kid(i + k);
                        if ((v2 >> 3) == G) { xs[k] = E::load(rowp, v2); n = k + 1; }
                    }
                }
                MS gm{-CUDART_INF_F, 0.f};
#pragma unroll
                for (int k = 0; k < GROUP; ++k)
                    if (k < n) ms_add(gm, xs[k], p.c2);
                const uint4 w4 = philox4x32_10(group_slot(uint32_t(G)), r.step, r.row, 0u, p.rk);
                const float score = group_score(fmaf(-r.xref, p.c2, gm.m) + log2f(gm.s),
                                                pick_word(w4, group_word(uint32_t(G))));
                if (score > a.best.score) {
                    int pick = 0;
                    if (n > 1) {
                        // inverse CDF over the members' weights 2^(x*c2 - gm.m), ascending token id
                        float cum[GROUP];
                        float total = 0.f;
#pragma unroll
                        for (int k = 0; k < GROUP; ++k) {
                            if (k < n) total += exp2f(fmaf(xs[k], p.c2, -gm.m));
                            cum[k] = total;
                        }
                        if (total > 0.f && total < CUDART_INF_F) {
                            const uint4 u4 = philox4x32_10(uint32_t(G), r.step, r.row, 3u, p.rk);
                            const float target = uniform_from_bits(u4.x) * total;
                            pick = n - 1;
#pragma unroll
                            for (int k = GROUP - 2; k >= 0; --k)
                                if (k < n && cum[k] > target) pick = k;
                        }
                    }
                    a.best.score = score;
                    a.best.key = kid(i + pick);
                    a.best.child = LIST ? -1 : cb + i + pick;
                }
            }
        }
    }

    MS all = a.touched ? MS{a.mref, (a.sa.x + a.sa.y) + (a.sb.x + a.sb.y)} : MS{-CUDART_INF_F, 0.f};
    if (use_parts) all = all_parts;
    if (dense) ok = a.touched ? MS{a.mref, a.ok2.x + a.ok2.y} : MS{-CUDART_INF_F, 0.f};
    Best best = a.best;

    // ---- block reduction of (all, ok, best).  Inside a warp the (m, s) pairs are brought to the
    // warp's largest reference first (one exponential per lane), then summed; a lane without
    // terms (m = -inf) adds zero, a poisoned sum (s = NaN) stays poisoned.
    {
        const float M_all = warp_max(all.m), M_ok = warp_max(ok.m);
        float s_all = (M_all == -CUDART_INF_F) ? 0.f : all.s * exp2f(all.m - M_all);
        float s_ok = (M_ok == -CUDART_INF_F) ? 0.f : ok.s * exp2f(ok.m - M_ok);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            s_all += __shfl_xor_sync(0xffffffffu, s_all, o);
            s_ok += __shfl_xor_sync(0xffffffffu, s_ok, o);
            Best b2{__shfl_xor_sync(0xffffffffu, best.score, o), __shfl_xor_sync(0xffffffffu, best.key, o),
                    __shfl_xor_sync(0xffffffffu, best.child, o)};
            best = best_merge(best, b2);
        }
        all = MS{M_all, s_all};
        ok = MS{M_ok, s_ok};
    }
    if (lane == 0) {
        red_f[0][warp] = all.m; red_f[1][warp] = all.s; red_f[2][warp] = ok.m; red_f[3][warp] = ok.s;
        red_f[4][warp] = best.score; red_i[0][warp] = best.key; red_i[1][warp] = best.child;
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
            Best b2{__shfl_xor_sync(0xffffffffu, best.score, o), __shfl_xor_sync(0xffffffffu, best.key, o),
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
        // The fast sums are trusted when both are finite.  In the dense path the valid-set sum
        // shares each thread's reference with the full sum, so an allowed term 2^-126 below a
        // thread's reference is flushed to zero (and its group may be skipped by the bound).
        // all.m is the largest reference; while log2(valid mass) >= all.m - 60 every flushed term
        // is below 2^-49 of the valid sum even if all 2^17 of them were flushed, and no group made
        // of flushed terms can win (its score trails the best group by more than the largest noise).
        bool trust = fabsf(l2_all) < CUDART_INF_F && fabsf(l2_ok) < CUDART_INF_F;
        if (dense && !(l2_ok >= all.m - MASS_FLOOR_LOG2)) trust = false;
        // sums given from outside were formed against exact maxima; the row's logits cannot be
        // re-read in full, so what the sums say stands (a row with NaN or +Inf gets its status bits)
        if (use_parts) trust = true;
        s_flag = trust ? 0 : 1;
        red_f[4][0] = best.score; red_i[0][0] = best.key; red_i[1][0] = best.child;
    }
    __syncthreads();

    if (s_flag) {
        // ---- careful path: plain two-pass log-sum-exp with separate maxima for the full row and
        // for the valid set, group by group.  Dense rows test the prebuilt mask and evaluate the
        // score of every group exactly again; gather rows walk their child list (their group
        // scores were exact already).
        float mx_all = -CUDART_INF_F, mx_ok = -CUDART_INF_F;
        int nan_all = 0, nan_ok = 0;
        for (int G = tid; G < n_groups; G += STEP_THREADS) {
            const uint32_t bits = dense ? mask_byte(gmask, uint32_t(G)) : 0u;
            for (int j = 0; j < GROUP && G * GROUP + j < p.V; ++j) {
                const float x = E::load(rowp, G * GROUP + j);
                const bool allowed = (bits >> j) & 1u;
                if (x != x) { nan_all = 1; nan_ok |= allowed; }
                else { mx_all = fmaxf(mx_all, x); if (allowed) mx_ok = fmaxf(mx_ok, x); }
            }
        }
        if (!dense) {
            for (int i = tid; i < c; i += STEP_THREADS) {
                const float x = E::load(rowp, kid(i));
                if (x != x) nan_ok = 1; else mx_ok = fmaxf(mx_ok, x);
            }
        }
        mx_all = block_max(mx_all, scratch);
        mx_ok = block_max(mx_ok, scratch);
        nan_all = __syncthreads_or(nan_all);
        nan_ok = __syncthreads_or(nan_ok);
        const bool fin_all = fabsf(mx_all) < CUDART_INF_F, fin_ok = fabsf(mx_ok) < CUDART_INF_F;
        const float r_all = mx_all * p.c2, r_ok = mx_ok * p.c2;
        float sum_all = 0.f, sum_ok = 0.f;
        Best cbest{-CUDART_INF_F, -1, -1};
        for (int G = tid; G < n_groups; G += STEP_THREADS) {
            const uint32_t bits = dense ? mask_byte(gmask, uint32_t(G)) : 0u;
            float tg = 0.f;
            for (int j = 0; j < GROUP && G * GROUP + j < p.V; ++j) {
                const float x = E::load(rowp, G * GROUP + j);
                if (fin_all) sum_all += exp2f(fmaf(x, p.c2, -r_all));
                if (fin_ok && ((bits >> j) & 1u)) tg += exp2f(fmaf(x, p.c2, -r_ok));
            }
            if (bits && fin_ok) {
                sum_ok += tg;
                const uint4 w4 = philox4x32_10(group_slot(uint32_t(G)), r.step, r.row, 0u, p.rk);
                const float score = group_score(fmaf(-r.xref, p.c2, r_ok) + log2f(tg),
                                                pick_word(w4, group_word(uint32_t(G))));
                if (score > cbest.score) { cbest.score = score; cbest.key = G; }
            }
        }
        if (!dense && fin_ok) {
            for (int i = tid; i < c; i += STEP_THREADS)
                sum_ok += exp2f(fmaf(E::load(rowp, kid(i)), p.c2, -r_ok));
        }
        sum_all = block_sum(sum_all, scratch);
        sum_ok = block_sum(sum_ok, scratch);
        if (dense) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                Best b2{__shfl_xor_sync(0xffffffffu, cbest.score, o), __shfl_xor_sync(0xffffffffu, cbest.key, o), -1};
                cbest = best_merge(cbest, b2);
            }
            __syncthreads();
            if (lane == 0) { red_f[5][warp] = cbest.score; red_i[0][warp] = cbest.key; }
            __syncthreads();
            if (tid == 0) {
                Best b{red_f[5][0], red_i[0][0], -1};
                for (int w = 1; w < STEP_WARPS; ++w) b = best_merge(b, Best{red_f[5][w], red_i[0][w], -1});
                red_f[4][0] = b.score; red_i[0][0] = b.key; red_i[1][0] = -1;
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

    // ---- finalise: stage 2 of the sampling, then one warp moves the row's cursor to the child
    if (warp == 0) {
        const int32_t key = red_i[0][0];
        int32_t tok = -1, child = -1;
        if (key < 0) {
            tok = kid(0); child = LIST ? -1 : cb;                     // no group with a finite score: lowest id
        } else if (!dense) {
            tok = key; child = red_i[1][0];                           // drawn in the gather loop already
        } else {
            // stage 2 for a dense row: the winning group's allowed tokens (ascending) and their
            // weights against the group's largest logit
            const int32_t Gw = key;
            const uint32_t bits = mask_byte(gmask, uint32_t(Gw));
            float xs[GROUP];
            float xm = -CUDART_INF_F;
#pragma unroll
            for (int j = 0; j < GROUP; ++j) {
                const bool on = ((bits >> j) & 1u) && Gw * GROUP + j < p.V;
                xs[j] = on ? E::load(rowp, Gw * GROUP + j) : -CUDART_INF_F;
                xm = fmaxf(xm, xs[j]);
            }
            const float ref = xm * p.c2;
            float cum[GROUP];
            float total = 0.f;
            int last = -1, first = -1;
#pragma unroll
            for (int j = 0; j < GROUP; ++j) {
                const bool on = (bits >> j) & 1u;
                if (on) { total += exp2f(fmaf(xs[j], p.c2, -ref)); last = j; if (first < 0) first = j; }
                cum[j] = total;
            }
            int pick = first;
            if (total > 0.f && total < CUDART_INF_F) {
                const uint4 u4 = philox4x32_10(uint32_t(Gw), r.step, r.row, 3u, p.rk);
                const float target = uniform_from_bits(u4.x) * total;
                pick = last;
#pragma unroll
                for (int j = GROUP - 1; j >= 0; --j)
                    if (((bits >> j) & 1u) && cum[j] > target) pick = j;
            }
            if (pick >= 0) tok = Gw * GROUP + pick;
            else { tok = kid(0); child = LIST ? -1 : cb; }
        }
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
            const float xt = (c == 1 && !dense) ? x_mine : E::load(rowp, tok);
            const float logq = f_ok ? (fmaf(xt, p.c2, -K.m) - lg_ok) * LN2_F : (xt * p.c2 - l2_ok) * LN2_F;
            const float logp = f_all ? (fmaf(xt, p.c2, -A.m) - lg_all) * LN2_F : (xt * p.c2 - l2_all) * LN2_F;
            const int32_t d = depth_old;
            p.token_out[row] = tok;
            if (p.seq_tokens && d < p.seq_ld) p.seq_tokens[size_t(row) * p.seq_ld + d] = tok;
            if (p.logq_out) p.logq_out[row] = logq;
            if (p.logp_out) p.logp_out[row] = logp;
            p.logw[row] += log_mass;
            p.node[row] = child;
            if (c == 1 && !LIST) {       // fetched before the row was streamed
                p.lo[row] = only_lo;
                p.hi[row] = hi_old;
                p.done[row] = only_cb == only_ce ? 1 : 0;
            } else {
                p.lo[row] = __ldg(p.node_lo + child);
                p.hi[row] = (child + 1 < ce) ? __ldg(p.node_lo + child + 1) : hi_old;
                p.done[row] = (__ldg(p.child_begin + child) == __ldg(p.child_begin + child + 1)) ? 1 : 0;
            }
            p.depth[row] = d + 1;
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

__global__ void k_sampling_uniforms(PhiloxRoundKeys rk, uint32_t step, uint32_t row, int32_t g0, int32_t n,
                                    float* out) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const uint32_t G = uint32_t(g0 + i);
    const uint4 r = philox4x32_10(group_slot(G), step, row, 0u, rk);
    out[i] = uniform_from_bits(pick_word(r, group_word(G)));
}

template <int DT, bool VEC, int MODE = 0>
int launch_step(const StepParams& p, int64_t n, cudaStream_t st) {
    disc_step_kernel<DT, VEC, MODE><<<unsigned(n), STEP_THREADS, 0, st>>>(p);
    DISC_CUDA(cudaGetLastError());
    return DISC_OK;
}

int fill_step_params(StepParams& p, const disc_set_t* s, const void* logits, int64_t ld, float inv_temperature,
                     uint64_t seed, uint32_t step, int64_t row_base, int32_t* node, int32_t* lo, int32_t* hi,
                     int32_t* depth, float* logw, uint8_t* done, int32_t* token_out, int32_t* seq_tokens, int32_t seq_ld,
                     float* logq_out, float* logp_out, uint32_t* mask_out, uint8_t* status_out) {
    p.logits = logits; p.ld = ld; p.inv_t = inv_temperature; p.c2 = inv_temperature * LOG2E_F;
    p.rk = philox_round_keys(seed); p.step = step; p.row_base = uint32_t(row_base);
    p.node = node; p.lo = lo; p.hi = hi; p.depth = depth; p.logw = logw; p.done = done;
    p.token_out = token_out; p.seq_tokens = seq_tokens; p.seq_ld = seq_ld;
    p.logq_out = logq_out; p.logp_out = logp_out; p.mask_out = mask_out; p.status_out = status_out;
    p.node_tok = s->node_tok; p.node_lo = s->node_lo; p.child_begin = s->child_begin;
    p.root_child = s->root_child; p.root_mask = s->root_mask;
    p.heavy_nodes = s->heavy_nodes; p.heavy_masks = s->heavy_masks; p.n_heavy = s->n_heavy;
    p.V = s->V; p.W = s->W; p.Wp = s->Wp; p.M = s->M;
    p.parts = nullptr; p.n_parts = 0;
    p.cand = nullptr; p.cand_valid = nullptr; p.cand_M = 0;
    return DISC_OK;
}

}  // namespace

// disc_step for the fused projection (disc_project.cu): bf16 logits with 16-byte aligned rows of
// which only the pieces holding valid tokens need to have been written, and the sums over the whole
// vocabulary as per-part (m, s) pairs.  Arguments are checked by the caller.
int disc::step_with_parts(const disc_set_t* s, const void* logits, disc_dtype_t dtype, int64_t ld, int64_t n,
                          float inv_temperature, uint64_t seed, uint32_t step, int64_t row_base, int32_t* node,
                          int32_t* lo, int32_t* hi, int32_t* depth, float* logw, uint8_t* done, int32_t* token_out,
                          int32_t* seq_tokens, int32_t seq_ld, float* logq_out, float* logp_out, uint8_t* status_out,
                          const float2* parts, int32_t n_parts, cudaStream_t st) {
    if (dtype != DISC_BF16 || !parts || n_parts <= 0) return DISC_ERR_ARG;
    StepParams p;
    fill_step_params(p, s, logits, ld, inv_temperature, seed, step, row_base, node, lo, hi, depth, logw, done, token_out,
                     seq_tokens, seq_ld, logq_out, logp_out, nullptr, status_out);
    p.parts = parts; p.n_parts = n_parts;
    return launch_step<DISC_BF16, true, 1>(p, n, st);
}

// disc_step in top-M mode: the valid set of row i is the verified candidates among cand[i][0..M)
// (ascending id), its sum over the whole vocabulary is lse[i] = (m, s).  Arguments are checked by
// the caller.
int disc::step_with_candidates(const disc_set_t* s, const void* logits, disc_dtype_t dtype, int64_t ld, int64_t n,
                               float inv_temperature, uint64_t seed, uint32_t step, int64_t row_base, int32_t* node,
                               int32_t* lo, int32_t* hi, int32_t* depth, float* logw, uint8_t* done,
                               int32_t* token_out, int32_t* seq_tokens, int32_t seq_ld, float* logq_out,
                               float* logp_out, uint32_t* mask_out, uint8_t* status_out, const int32_t* cand,
                               const uint8_t* valid, int32_t M, const float2* lse, cudaStream_t st) {
    if (!cand || !valid || !lse || M <= 0 || M > TOPM_MAX) return DISC_ERR_ARG;
    StepParams p;
    fill_step_params(p, s, logits, ld, inv_temperature, seed, step, row_base, node, lo, hi, depth, logw, done, token_out,
                     seq_tokens, seq_ld, logq_out, logp_out, mask_out, status_out);
    p.parts = lse; p.n_parts = 1;
    p.cand = cand; p.cand_valid = valid; p.cand_M = M;
    const size_t esize = dtype == DISC_F32 ? 4 : 2;
    const bool vec = (reinterpret_cast<uintptr_t>(logits) % 16 == 0) && ((size_t(ld) * esize) % 16 == 0);
    if (dtype == DISC_F32) return vec ? launch_step<DISC_F32, true, 2>(p, n, st) : launch_step<DISC_F32, false, 2>(p, n, st);
    return vec ? launch_step<DISC_BF16, true, 2>(p, n, st) : launch_step<DISC_BF16, false, 2>(p, n, st);
}

extern "C" {

int disc_state_init(const disc_set_t* s, int64_t n, int32_t* node, int32_t* lo, int32_t* hi, int32_t* depth,
                    float* logw, uint8_t* done, void* stream) {
    if (!s || n < 0) return DISC_ERR_ARG;
    if (const int rc = check_device(s)) return rc;
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
    if (const int rc = check_device(s)) return rc;
    if (n == 0) return DISC_OK;
    if (!logits || !node || !lo || !hi || !depth || !logw || !done || !token_out || !status_out) return DISC_ERR_ARG;
    if (ld < s->V || row_base < 0 || (seq_tokens && seq_ld <= 0)) return DISC_ERR_ARG;
    if (!(inv_temperature > 0.f) || !(inv_temperature <= 3.0e38f)) return DISC_ERR_ARG;
    if (dtype != DISC_F32 && dtype != DISC_BF16) return DISC_ERR_UNSUPPORTED;
    // the row coordinate of the random numbers is one 32-bit counter word
    if (row_base + n > (int64_t(1) << 32)) return DISC_ERR_UNSUPPORTED;

    StepParams p;
    fill_step_params(p, s, logits, ld, inv_temperature, seed, step, row_base, node, lo, hi, depth, logw, done,
                     token_out, seq_tokens, seq_ld, logq_out, logp_out, mask_out, status_out);

    const size_t esize = dtype == DISC_F32 ? 4 : 2;
    // 16-byte loads need 16-byte aligned rows; other layouts take the scalar path
    const bool vec = (reinterpret_cast<uintptr_t>(logits) % 16 == 0) && ((size_t(ld) * esize) % 16 == 0);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (dtype == DISC_F32) return vec ? launch_step<DISC_F32, true>(p, n, st) : launch_step<DISC_F32, false>(p, n, st);
    return vec ? launch_step<DISC_BF16, true>(p, n, st) : launch_step<DISC_BF16, false>(p, n, st);
}

int disc_sampling_uniforms(uint64_t seed, uint32_t step, uint32_t row, int32_t g0, int32_t n, float* out,
                           void* stream) {
    if (n < 0 || g0 < 0 || (n > 0 && !out)) return DISC_ERR_ARG;
    if (n == 0) return DISC_OK;
    k_sampling_uniforms<<<(n + 255) / 256, 256, 0, static_cast<cudaStream_t>(stream)>>>(philox_round_keys(seed),
                                                                                       step, row, g0, n, out);
    DISC_CUDA(cudaGetLastError());
    return DISC_OK;
}

}  // extern "C"
