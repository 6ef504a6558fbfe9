// disc_topm: the M most probable tokens of every row (Algorithm 2, line 3), i.e. the M largest
// logits, exactly; and, as a by-product of the same pass, the row's sum over the whole vocabulary
// as a pair (m, s) with sum_v 2^(z_v log2e / T) = 2^m * s.
//
// Order of the values: larger first, -0 = +0, NaN below everything; among equal values the lower
// token id first, which makes the selection unique (equal logits are common in bf16).
//
// Two kernels, one block of 256 threads per row in both.
//
// M <= 1024 (the sizes the paper uses): ONE pass over the row, in three steps.
//   A. A threshold from a sample.  8,192 logits spread evenly over the row (runs of 256 bytes) are
//      read, 32 per thread; the r-th largest of the 256 threads' maxima (256-bin histograms in
//      shared memory over the key bits, eight at a time) is at most the r-th largest of the
//      sample, and r is chosen so that this is below the M-th largest of the whole row except
//      once in about a thousand rows: with f the sampled share, the sample holds about Mf of the
//      row's M best, and r = Mf + 3 sqrt(Mf) + 1.  (A row no longer than the sample is its own
//      sample, and the M-th largest is found exactly.)
//   B. The row is streamed once with eight 16-byte loads in flight per thread and no barrier.  The
//      sum for the log-sum-exp is accumulated, and a vector is tested as a whole against the
//      threshold (one packed maximum); the few vectors that reach it (about r/f logits do:
//      some 150 for M = 50, 1,400 for M = 1000) are noted in a list in shared memory.
//   C. The noted vectors are read again, their logits that reach the threshold become the
//      candidates (order key, token id), the M best of them are selected exactly (the same
//      histograms, then over the token ids among the keys equal to the M-th), and the M ids are
//      sorted and written out.
//   Whether the threshold was low enough is known in C: at least M logits reached it.  If not, or
//   if the lists overflowed (a row of equal logits, a row without numbers), the row is done again
//   by the kernel for larger M below, so the result is exact in every case.  The order in which the
//   row is read plays no part in it.
//
// Larger M: the key of the M-th largest logit is found by histogram passes over the whole row
// (bf16 keys take two, fp32 keys three), and a last pass writes the selection out in ascending id.
// Every pass streams the row again; after the first it comes from L2.

#include <cuda_bf16.h>
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

// unsigned order of the keys = order of the values; -0 and +0 share a key, NaN has the lowest
__device__ __forceinline__ uint32_t order_key(float x) {
    if (x != x) return 0u;
    uint32_t b = __float_as_uint(x);
    if (b == 0x80000000u) b = 0u;
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

// shared memory of the histogram passes
struct RadixSmem {
    unsigned int hist[BINS];
    unsigned int prefix, remaining;
    float red[TOPM_WARPS];
    unsigned int wsum[TOPM_WARPS];
    int scan[TOPM_WARPS][2];
    int flag;
};

// The selection of one row by histogram passes over the whole row (any M); called by the whole block.
template <int DT, bool VEC>
__device__ void radix_row(const TopmParams& p, int64_t row, RadixSmem& sm, bool write_lse) {
    constexpr int EPV = Row<DT>::EPV;
    constexpr int PASSES = DT == DISC_BF16 ? 2 : 3;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int32_t* out = p.cand + size_t(row) * p.M;
    const char* rowp = static_cast<const char*>(p.logits) + size_t(row) * size_t(p.ld) * (DT == DISC_BF16 ? 2 : 4);
    const int want = min(p.M, p.V);
    if (tid == 0) { sm.prefix = 0u; sm.remaining = unsigned(want); sm.flag = 0; }

    float row_max = -CUDART_INF_F;     // over the values that are not NaN
    float sum = 0.f;
    for (int pass = 0; pass < PASSES; ++pass) {
        for (int b = tid; b < BINS; b += TOPM_THREADS) sm.hist[b] = 0u;
        __syncthreads();
        // the window of key bits this pass looks at: [shift, shift + width)
        const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
        const int width = pass == 2 ? 10 : 11;
        const uint32_t prefix = sm.prefix;
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
                        atomicAdd(&sm.hist[(key >> shift) & ((1u << width) - 1u)], 1u);
                    if (pass == 0) { if (x[j] != x[j]) nan_seen = 1; else mx = fmaxf(mx, x[j]); }
                    else if (pass == 1) sum += ex2_approx(fmaf(x[j], p.c2, -ref));
                }
            }
        });
        if (pass == 0) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, o));
            if (lane == 0) sm.red[warp] = mx;
            if (nan_seen) sm.flag = 1;
        }
        __syncthreads();
        if (pass == 0) {
            row_max = sm.red[0];
#pragma unroll
            for (int w2 = 1; w2 < TOPM_WARPS; ++w2) row_max = fmaxf(row_max, sm.red[w2]);
        }
        // From the largest bin down: the bin that holds the `remaining`-th largest key.  Thread t
        // owns the bins [t*8, t*8+8); `above` = keys in the bins of higher threads.
        {
            const unsigned int rem = sm.remaining;
            unsigned int mine = 0;
#pragma unroll
            for (int b = 0; b < BINS_PER_THREAD; ++b) mine += sm.hist[tid * BINS_PER_THREAD + b];
            unsigned int incl = mine;                           // suffix sum over the lanes of the warp
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned int v = __shfl_down_sync(FULL, incl, o);
                if (lane + o < 32) incl += v;
            }
            if (lane == 0) sm.wsum[warp] = incl;
            __syncthreads();
            unsigned int above = incl - mine;
            for (int w2 = warp + 1; w2 < TOPM_WARPS; ++w2) above += sm.wsum[w2];
            __syncthreads();
            if (above < rem && above + mine >= rem) {           // exactly one thread
                unsigned int left = rem - above;
                int b = BINS_PER_THREAD - 1;
                for (; b > 0; --b) {
                    const unsigned int cnt = sm.hist[tid * BINS_PER_THREAD + b];
                    if (cnt >= left) break;
                    left -= cnt;
                }
                sm.prefix = prefix | (uint32_t(tid * BINS_PER_THREAD + b) << shift);
                sm.remaining = left;
            }
        }
        __syncthreads();
    }
    if (p.lse && write_lse) {
        // the row's sum over the whole vocabulary, 2^m * s (NaN or +Inf among the logits poison s)
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(FULL, sum, o);
        __syncthreads();
        if (lane == 0) sm.red[warp] = sum;
        __syncthreads();
        if (tid == 0) {
            float s = 0.f;
            for (int w2 = 0; w2 < TOPM_WARPS; ++w2) s += sm.red[w2];
            const bool fin = fabsf(row_max) < CUDART_INF_F;
            if (sm.flag || row_max == CUDART_INF_F) s = CUDART_NAN_F;
            p.lse[row] = make_float2(row_max == -CUDART_INF_F ? -CUDART_INF_F : (fin ? row_max * p.c2 : 0.f),
                                     row_max == -CUDART_INF_F ? 0.f : s);
        }
    }

    // ---- write-out in ascending token id: keys above the threshold, then the lowest ids among the
    // keys equal to it until `want` are filled
    const uint32_t thr = sm.prefix;
    const int take_eq = int(sm.remaining);
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
        if (lane == 31) { sm.scan[warp][0] = sg; sm.scan[warp][1] = se; }
        __syncthreads();
        int bg = gt_total, be = eq_total, tot_g = 0, tot_e = 0;
#pragma unroll
        for (int w2 = 0; w2 < TOPM_WARPS; ++w2) {
            if (w2 < warp) { bg += sm.scan[w2][0]; be += sm.scan[w2][1]; }
            tot_g += sm.scan[w2][0]; tot_e += sm.scan[w2][1];
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

template <int DT, bool VEC>
__global__ void __launch_bounds__(TOPM_THREADS) disc_topm_kernel(const TopmParams p) {
    __shared__ RadixSmem sm;
    const int64_t row = blockIdx.x;
    if (p.done && p.done[row]) {
        int32_t* out = p.cand + size_t(row) * p.M;
        for (int m = threadIdx.x; m < p.M; m += TOPM_THREADS) out[m] = -1;
        if (p.lse && threadIdx.x == 0) p.lse[row] = make_float2(-CUDART_INF_F, 0.f);
        return;
    }
    radix_row<DT, VEC>(p, row, sm, true);
}

// ---- one pass over the row (M <= 1024) ----------------------------------------------------------------
#ifndef DISC_TOPM_U
#define DISC_TOPM_U 8
#endif
#ifndef DISC_TOPM_BLOCKS
#define DISC_TOPM_BLOCKS 4
#endif
#ifndef DISC_TOPM_CAP
#define DISC_TOPM_CAP 3072
#endif
constexpr int SEL_U = DISC_TOPM_U;       // 16-byte loads a thread keeps in flight
constexpr int SEL_KEEP = 1024;           // largest M this kernel takes
constexpr int SEL_CAP = DISC_TOPM_CAP;   // candidates shared memory has room for
constexpr int SEL_HITS = 3 * SEL_KEEP;   // vectors holding a candidate

// the value of a key other than NaN's
__device__ __forceinline__ float key_value(uint32_t k) {
    return (k & 0x80000000u) ? __uint_as_float(k & 0x7fffffffu) : __uint_as_float(~k);
}

__device__ __forceinline__ uint4 ld_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// A 16-byte vector of the row held in registers.
template <int DT>
struct Lane;
template <>
struct Lane<DISC_BF16> {
    static constexpr int EPV = 8;
    __device__ static __forceinline__ void unpack(const uint4& v, float* x) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) { x[2 * j] = __uint_as_float(w[j] << 16); x[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u); }
    }
    // the largest element (NaN only if all eight are)
    __device__ static __forceinline__ float vmax(const uint4& v) {
        const __nv_bfloat162 a = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&v.x), *reinterpret_cast<const __nv_bfloat162*>(&v.y));
        const __nv_bfloat162 b = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&v.z), *reinterpret_cast<const __nv_bfloat162*>(&v.w));
        const __nv_bfloat162 c = __hmax2(a, b);
        const uint32_t w = *reinterpret_cast<const uint32_t*>(&c);
        return fmaxf(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
    }
    // does any element reach thr (a value of the row's own type)?  Packed: three maxima and one
    // comparison of both halves; a vector of NaNs counts as reaching it, which costs a look at it
    // later and nothing else.
    __device__ static __forceinline__ bool reaches(const uint4& v, float thr) {
        const __nv_bfloat162 a = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&v.x), *reinterpret_cast<const __nv_bfloat162*>(&v.y));
        const __nv_bfloat162 b = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&v.z), *reinterpret_cast<const __nv_bfloat162*>(&v.w));
        return !__hblt2(__hmax2(a, b), __float2bfloat162_rn(thr));
    }
    // elements id0 .. id0+7 read one by one; -inf where the row has ended
    __device__ static __forceinline__ uint4 gather(const void* rowp, int id0, int V) {
        uint32_t w[4];
        const unsigned short* r = static_cast<const unsigned short*>(rowp);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t lo = (id0 + 2 * j < V) ? uint32_t(__ldg(r + id0 + 2 * j)) : 0xFF80u;
            const uint32_t hi = (id0 + 2 * j + 1 < V) ? uint32_t(__ldg(r + id0 + 2 * j + 1)) : 0xFF80u;
            w[j] = lo | (hi << 16);
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
};
template <>
struct Lane<DISC_F32> {
    static constexpr int EPV = 4;
    __device__ static __forceinline__ void unpack(const uint4& v, float* x) {
        x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y); x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
    }
    __device__ static __forceinline__ float vmax(const uint4& v) {
        return fmaxf(fmaxf(__uint_as_float(v.x), __uint_as_float(v.y)), fmaxf(__uint_as_float(v.z), __uint_as_float(v.w)));
    }
    __device__ static __forceinline__ bool reaches(const uint4& v, float thr) { return vmax(v) >= thr; }
    __device__ static __forceinline__ uint4 gather(const void* rowp, int id0, int V) {
        uint32_t w[4];
        const uint32_t* r = static_cast<const uint32_t*>(rowp);
#pragma unroll
        for (int j = 0; j < 4; ++j) w[j] = (id0 + j < V) ? __ldg(r + id0 + j) : 0xFF800000u;
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
};

// The selections inside a block use 256-bin histograms, one bin per thread, over eight key bits at a
// time: the candidates are a few hundred, and finding the bin then costs one block-wide suffix sum.
// Of the keys counted in hist (bins of the key bits [shift, shift+8) among the keys that agree with
// `prefix` above them), the bin that holds the *rem_io-th largest: *prefix_out gets the bin's bits
// added, *rem_io its rank inside the bin, *ties_out the bin's count.  Called by the whole block;
// ends with a barrier.
__device__ __forceinline__ void pick_bin256(const unsigned int* hist, uint32_t prefix, int shift, unsigned int* s_wsum,
                                            unsigned int* prefix_out, unsigned int* rem_io, unsigned int* ties_out) {
    static_assert(TOPM_THREADS == 256, "one bin per thread");
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned int rem = *rem_io;
    const unsigned int mine = hist[tid];
    unsigned int incl = mine;                           // suffix sum over the lanes of the warp
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned int v = __shfl_down_sync(FULL, incl, o);
        if (lane + o < 32) incl += v;
    }
    if (lane == 0) s_wsum[warp] = incl;
    __syncthreads();
    unsigned int above = incl - mine;
#pragma unroll
    for (int w2 = 1; w2 < TOPM_WARPS; ++w2) above += w2 > warp ? s_wsum[w2] : 0u;
    __syncthreads();
    if (above < rem && above + mine >= rem) {           // exactly one thread
        *prefix_out = prefix | (uint32_t(tid) << shift);
        *rem_io = rem - above;
        *ties_out = mine;
    }
    __syncthreads();
}

// Control words of a block's selection, in shared memory.
struct SelCtl {
    unsigned int count;        // an allocator: vectors that hold a candidate, then candidates
    unsigned int prefix, remaining, ties, kept;
    unsigned int n_sample;
};

// Of the cnt candidates (keys, ids) in shared memory exactly the `want` best stay, stored in front
// (c.count = want).  `hist` (2048 words) is scratch: histograms first, then the place the kept
// candidates are collected in.  Called by the whole block with cnt > want; begins and ends with a
// barrier.  Out of line: it runs once per row.
__device__ __noinline__ void select_best(uint32_t* keys, int32_t* ids, unsigned int cnt, unsigned int want, int V,
                                         bool bf16, unsigned int* hist, unsigned int* s_wsum, SelCtl& c) {
    const int tid = threadIdx.x;
    // bf16: the keys differ in their upper 16 bits only
    const uint32_t key_mask = bf16 ? 0xffff0000u : 0xffffffffu;
    const int low = bf16 ? 16 : 0;
    __syncthreads();
    if (tid == 0) { c.prefix = 0u; c.remaining = want; c.kept = 0u; }
    for (int shift = 24; shift >= low; shift -= 8) {
        hist[tid] = 0u;
        __syncthreads();
        const uint32_t prefix = c.prefix;
        for (unsigned int i = tid; i < cnt; i += TOPM_THREADS) {
            const uint32_t k = keys[i];
            if (shift == 24 || (k >> (shift + 8)) == (prefix >> (shift + 8))) atomicAdd(&hist[(k >> shift) & 255u], 1u);
        }
        __syncthreads();
        pick_bin256(hist, prefix, shift, s_wsum, &c.prefix, &c.remaining, &c.ties);
    }
    const uint32_t thr_key = c.prefix;            // key (its bits under key_mask) of the want-th best
    const unsigned int left = c.remaining;        // how many of the candidates with that key stay
    const unsigned int ties = c.ties;             // how many there are
    int32_t id_thr = 0x7fffffff;                  // those with an id up to this one
    if (ties > left) {
        // the left-th lowest id among the tied candidates: the same search over idmask - id
        const int nb = 32 - __clz(V - 1);         // V >= 2 here; ids fit nb <= 30 bits
        const uint32_t idmask = (1u << nb) - 1u;
        __syncthreads();                          // everyone has read the key search's results
        if (tid == 0) { c.prefix = 0u; c.remaining = left; }
        for (int top = nb; top > 0;) {
            const int shift = max(top - 8, 0);    // the window [shift, top), at most eight bits
            hist[tid] = 0u;
            __syncthreads();
            const uint32_t prefix = c.prefix;
            for (unsigned int i = tid; i < cnt; i += TOPM_THREADS) {
                if ((keys[i] & key_mask) == thr_key) {
                    const uint32_t k2 = idmask - uint32_t(ids[i]);
                    if (top == nb || (k2 >> top) == (prefix >> top)) atomicAdd(&hist[(k2 >> shift) & ((1u << (top - shift)) - 1u)], 1u);
                }
            }
            __syncthreads();
            pick_bin256(hist, prefix, shift, s_wsum, &c.prefix, &c.remaining, &c.ties);
            top = shift;
        }
        id_thr = int32_t(idmask - c.prefix);
    }
    // the kept candidates are collected in the histogram's place (the last barrier of the search has
    // passed, nobody reads the histogram any more), then moved to the front
    uint32_t* tk = hist;
    int32_t* ti = reinterpret_cast<int32_t*>(hist + SEL_KEEP);
    for (unsigned int i0 = 0; i0 < cnt; i0 += TOPM_THREADS) {             // the lanes of a warp stay together
        const unsigned int i = i0 + tid;
        const uint32_t k = i < cnt ? keys[i] : 0u, km = k & key_mask;
        const int32_t id = i < cnt ? ids[i] : 0;
        const bool keep = i < cnt && (km > thr_key || (km == thr_key && id <= id_thr));
        const uint32_t ballot = __ballot_sync(FULL, keep);                // one reservation per warp
        const int lane = tid & 31;
        unsigned int base = 0u;
        if (lane == 0 && ballot) base = atomicAdd(&c.kept, unsigned(__popc(ballot)));
        const unsigned int pos = __shfl_sync(FULL, base, 0) + unsigned(__popc(ballot & ((1u << lane) - 1u)));
        if (keep && pos < unsigned(SEL_KEEP)) { tk[pos] = k; ti[pos] = id; }
    }
    __syncthreads();
    const unsigned int n_kept = min(c.kept, unsigned(SEL_KEEP));      // = want
    for (unsigned int i = tid; i < n_kept; i += TOPM_THREADS) { keys[i] = tk[i]; ids[i] = ti[i]; }
    if (tid == 0) c.count = n_kept;
    __syncthreads();
}

template <int DT, bool VEC>
__global__ void __launch_bounds__(TOPM_THREADS, DISC_TOPM_BLOCKS) disc_topm_stream_kernel(const TopmParams p) {
    using L = Lane<DT>;
    constexpr int EPV = L::EPV;
    constexpr int ESIZE = DT == DISC_BF16 ? 2 : 4;
    constexpr int SEL_SAMPLE = DT == DISC_BF16 ? 4 : 8;         // vectors per thread in the sample: 8192 logits
    constexpr int SAMPLE_VECS = SEL_SAMPLE * TOPM_THREADS;      // vectors of the sample
    __shared__ uint32_t keys[SEL_CAP];
    __shared__ int32_t ids[SEL_CAP];
    __shared__ int32_t hits[SEL_HITS];
    __shared__ RadixSmem rs;
    __shared__ SelCtl ctl;
    __shared__ float s_red[2][TOPM_WARPS];
    __shared__ int s_flag;
    static_assert(BINS >= 2 * SEL_KEEP, "the histogram's place holds the kept candidates");

    const int64_t row = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int32_t* out = p.cand + size_t(row) * p.M;
    if (p.done && p.done[row]) {
        for (int m = tid; m < p.M; m += TOPM_THREADS) out[m] = -1;
        if (p.lse && tid == 0) p.lse[row] = make_float2(-CUDART_INF_F, 0.f);
        return;
    }
    const char* rowp = static_cast<const char*>(p.logits) + size_t(row) * size_t(p.ld) * ESIZE;
    const int V = p.V;
    const unsigned int want = unsigned(min(p.M, V));
    const int nvec = (V + EPV - 1) / EPV;
    auto load_vec = [&](int vi) -> uint4 {
        const int id0 = vi * EPV;
        if (VEC && id0 + EPV <= V) return ld_stream16(rowp + size_t(id0) * ESIZE);
        return L::gather(rowp, id0, V);
    };

    // this thread's share of sum_v 2^(x_v c2 - mref), taken in the first attempt
    float mref = 0.f;
    float2 acc0 = {0.f, 0.f}, acc1 = {0.f, 0.f};
    bool touched = false;
    // Two attempts.  The second, with a threshold far lower in the sample, runs if the first one's
    // threshold turned out too high; it costs one more pass over the row (which then comes from L2
    // in part), a fraction of what the histogram passes cost, so that the odd unlucky row does not
    // hold up its launch.
    bool finished = false;
    for (int attempt = 0; attempt < 2 && !finished; ++attempt) {
    __syncthreads();
    // ---- A. a threshold from a sample.  SAMPLE_VECS vectors spread evenly over the row (the whole
    // row if it has no more) are read; with f the sampled share of the row, about want*f of the
    // row's `want` best are among them, and the r-th best of the sample, r = want*f + 3 sqrt(want*f)
    // + 1, is below the want-th best of the row except once in about a thousand rows.  Whether it
    // was is known at the end (at least `want` logits reached it).
    // the k-th vector of the sample: runs of 16 vectors (256 bytes), the runs spread evenly
    auto sample_vec = [&](int k) -> int {
        if (nvec <= SAMPLE_VECS) return k;
        return int((int64_t(k >> 4) * nvec) / (SAMPLE_VECS >> 4)) + (k & 15);
    };
    uint4 sv[SEL_SAMPLE];
    unsigned int n_mine = 0u;
#pragma unroll
    for (int i = 0; i < SEL_SAMPLE; ++i) {
        const int k = i * TOPM_THREADS + tid;
        const int vi = sample_vec(k);
        sv[i] = load_vec(vi < nvec ? vi : nvec);          // past the end: a vector of -inf that is not counted
        n_mine += vi < nvec ? unsigned(min(EPV, V - vi * EPV)) : 0u;
    }
    if (tid == 0) { ctl.count = 0u; ctl.kept = 0u; ctl.n_sample = 0u; ctl.prefix = 0u; }
    __syncthreads();
    {
        const unsigned int wn = __reduce_add_sync(FULL, n_mine);
        if (lane == 0) atomicAdd(&ctl.n_sample, wn);
    }
    __syncthreads();
    const unsigned int n_sample = ctl.n_sample;
    unsigned int r = want;
    if (unsigned(V) > n_sample) {
        const float mean = float(want) * float(n_sample) / float(V);
        r = unsigned(ceilf(mean + 3.f * sqrtf(mean) + 1.f));
        if (attempt) r = 2u * r + 8u;
        r = min(n_sample, r);
    }
    const bool can_lower = attempt == 0 && r < n_sample;
    if (tid == 0) ctl.remaining = r;
    if (nvec > SAMPLE_VECS) {
        // A row much longer than the sample: every thread takes the largest of its 32 sampled
        // logits, and the r-th largest of these 256 maxima stands in for the r-th largest of the
        // sample.  It is never above it (the maxima are r different sampled logits), so the
        // threshold only gets safer, and a little lower when two of the sample's best share a
        // thread; one key per thread makes the passes cheap.
        float mx = L::vmax(sv[0]);
#pragma unroll
        for (int i = 1; i < SEL_SAMPLE; ++i) mx = fmaxf(mx, L::vmax(sv[i]));
        const uint32_t key = order_key(mx);
        if (tid == 0) ctl.remaining = min(r, unsigned(TOPM_THREADS));
#pragma unroll 1
        for (int shift = 24; shift >= (DT == DISC_BF16 ? 16 : 0); shift -= 8) {
            rs.hist[tid] = 0u;
            __syncthreads();
            const uint32_t prefix = ctl.prefix;
            if (shift == 24 || (key >> (shift + 8)) == (prefix >> (shift + 8))) atomicAdd(&rs.hist[(key >> shift) & 255u], 1u);
            __syncthreads();
            pick_bin256(rs.hist, prefix, shift, rs.wsum, &ctl.prefix, &ctl.remaining, &ctl.ties);
        }
    } else {
        // The r-th largest key of the sample, eight bits at a time.  The -inf that stands for "past the
        // end of the row" has the lowest key of all numbers and r counts real logits only, so the
        // fill never matters.  bf16: the two 16-bit keys of a word are formed together, and a NaN
        // counts as a large value here (the threshold is then too high and the row is done again).
#pragma unroll 1
        for (int shift = 24; shift >= (DT == DISC_BF16 ? 16 : 0); shift -= 8) {
            rs.hist[tid] = 0u;
            __syncthreads();
            const uint32_t prefix = ctl.prefix;
#pragma unroll
            for (int i = 0; i < SEL_SAMPLE; ++i) {
                if (DT == DISC_BF16) {
                    const uint32_t w[4] = {sv[i].x, sv[i].y, sv[i].z, sv[i].w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t neg = (w[j] & 0x80008000u) >> 15;             // 1 in the halves that are negative
                        const uint32_t k2 = w[j] ^ ((neg * 0xFFFFu) | 0x80008000u);  // ~h there, h ^ 0x8000 elsewhere
                        const uint32_t ka = k2 & 0xFFFFu, kb = k2 >> 16;
                        if (shift == 24) {
                            atomicAdd(&rs.hist[ka >> 8], 1u);
                            atomicAdd(&rs.hist[kb >> 8], 1u);
                        } else {
                            if ((ka >> 8) == (prefix >> 24)) atomicAdd(&rs.hist[ka & 255u], 1u);
                            if ((kb >> 8) == (prefix >> 24)) atomicAdd(&rs.hist[kb & 255u], 1u);
                        }
                    }
                } else {
                    float x[EPV];
                    L::unpack(sv[i], x);
#pragma unroll
                    for (int j = 0; j < EPV; ++j) {
                        const uint32_t key = order_key(x[j]);
                        if (shift == 24 || (key >> (shift + 8)) == (prefix >> (shift + 8))) atomicAdd(&rs.hist[(key >> shift) & 255u], 1u);
                    }
                }
            }
            __syncthreads();
            pick_bin256(rs.hist, prefix, shift, rs.wsum, &ctl.prefix, &ctl.remaining, &ctl.ties);
        }
    }
    // a logit is a candidate if it is at least this (a NaN key: no threshold, every logit is one)
    float thr = -CUDART_INF_F;
    {
        uint32_t full = ctl.prefix;
        if (DT == DISC_BF16 && !(full & 0x80000000u)) full |= 0xffffu;
        if (ctl.prefix != 0u) thr = key_value(full);
    }

    // ---- B. one pass over the row: the sum for the log-sum-exp, and the vectors that hold a candidate
    // (a vector is tested as a whole; what it holds is looked at in C).  No barriers: thread t
    // takes the vectors t, t+256, ... with SEL_U loads in flight.  Which of its vectors reach the
    // threshold a thread keeps as bits in a register and writes to the list every 64 vectors: inside
    // the loop a hit then costs a predicated OR, not a branch that most warps would take at large M.
    auto add_to_sum = [&](const uint4& raw) {
        if (attempt != 0) return;
        float x[EPV];
        L::unpack(raw, x);
        if (!touched) {
            float mx = x[0];
#pragma unroll
            for (int j = 1; j < EPV; ++j) mx = fmaxf(mx, x[j]);
            const float m = mx * p.c2;
            mref = (fabsf(m) < CUDART_INF_F) ? m : 0.f;
            touched = true;
        }
        const float2 cc = make_float2(p.c2, p.c2), nm = make_float2(-mref, -mref);
#pragma unroll
        for (int j = 0; j < EPV; j += 4) {
            const float2 y0 = __ffma2_rn(make_float2(x[j], x[j + 1]), cc, nm);
            const float2 y1 = __ffma2_rn(make_float2(x[j + 2], x[j + 3]), cc, nm);
            acc0 = __fadd2_rn(acc0, make_float2(ex2_approx(y0.x), ex2_approx(y0.y)));
            acc1 = __fadd2_rn(acc1, make_float2(ex2_approx(y1.x), ex2_approx(y1.y)));
        }
    };
    auto note = [&](int vi) {
        const unsigned int pos = atomicAdd(&ctl.count, 1u);
        if (pos < unsigned(SEL_HITS)) hits[pos] = vi;
    };
    {
        static_assert(64 % SEL_U == 0, "whole batches per 64-bit word");
        constexpr int BATCHES = 64 / SEL_U;          // batches of SEL_U vectors per word of hit bits
        // whole batches (the same number for every thread of the block), then the few vectors left
        const int n_batches = nvec / (SEL_U * TOPM_THREADS);
        for (int b0 = 0; b0 < n_batches; b0 += BATCHES) {
            const int vi0 = tid + b0 * SEL_U * TOPM_THREADS;
            const int nb = min(BATCHES, n_batches - b0);
            unsigned long long bits = 0ull;
#pragma unroll 1
            for (int it = 0; it < nb; ++it) {
                const int vi = vi0 + it * SEL_U * TOPM_THREADS;
                uint4 raw[SEL_U];
#pragma unroll
                for (int u = 0; u < SEL_U; ++u) raw[u] = load_vec(vi + u * TOPM_THREADS);
                unsigned int m = 0u;
#pragma unroll
                for (int u = 0; u < SEL_U; ++u) {
                    add_to_sum(raw[u]);
                    m |= L::reaches(raw[u], thr) ? (1u << u) : 0u;
                }
                bits |= static_cast<unsigned long long>(m) << (it * SEL_U);
            }
            // the warp's hits go to the list with one reservation (the lanes are together here: the
            // loop above runs the same number of times in every thread)
            const unsigned int mine = unsigned(__popcll(bits));
            unsigned int incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned int v = __shfl_up_sync(FULL, incl, o);
                if (lane >= o) incl += v;
            }
            unsigned int base = 0u;
            if (lane == 31 && incl) base = atomicAdd(&ctl.count, incl);
            unsigned int pos = __shfl_sync(FULL, base, 31) + incl - mine;
            while (bits) {                            // bit it*SEL_U + u: vector vi0 + (it*SEL_U + u) * 256
                const int bpos = __ffsll(static_cast<long long>(bits)) - 1;
                bits &= bits - 1ull;
                if (pos < unsigned(SEL_HITS)) hits[pos] = vi0 + bpos * TOPM_THREADS;
                ++pos;
            }
        }
        for (int vi = tid + n_batches * SEL_U * TOPM_THREADS; vi < nvec; vi += TOPM_THREADS) {
            const uint4 raw = load_vec(vi);
            add_to_sum(raw);
            if (L::reaches(raw, thr)) note(vi);
        }
    }

    // ---- the row's sum over the whole vocabulary
    if (p.lse && attempt == 0) {
        float m = touched ? mref : -CUDART_INF_F;
        float s = (acc0.x + acc0.y) + (acc1.x + acc1.y);
        float mw = m;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mw = fmaxf(mw, __shfl_xor_sync(FULL, mw, o));
        s = (m == -CUDART_INF_F) ? 0.f : s * exp2f(m - mw);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(FULL, s, o);
        if (lane == 0) { s_red[0][warp] = mw; s_red[1][warp] = s; }
        __syncthreads();
        float mb = s_red[0][0];
#pragma unroll
        for (int w2 = 1; w2 < TOPM_WARPS; ++w2) mb = fmaxf(mb, s_red[0][w2]);
        float sb = 0.f;
#pragma unroll
        for (int w2 = 0; w2 < TOPM_WARPS; ++w2)
            sb += (s_red[0][w2] == -CUDART_INF_F) ? 0.f : s_red[1][w2] * exp2f(s_red[0][w2] - mb);
        if (sb > 0.f && sb < CUDART_INF_F) {
            if (tid == 0) p.lse[row] = make_float2(mb, sb);
        } else {
            // Nothing finite, NaN or +Inf among the logits, or a sum that overflowed against the
            // references of the first logits: the plain way, maximum first, then the sum.
            float mx = -CUDART_INF_F;
            int nan_seen = 0;
            for_row<DT, VEC>(rowp, V, [&](int, int e0, const float* x) {
#pragma unroll
                for (int j = 0; j < EPV; ++j)
                    if (e0 + j < V) { if (x[j] != x[j]) nan_seen = 1; else mx = fmaxf(mx, x[j]); }
            });
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, o));
            if (tid == 0) s_flag = 0;
            __syncthreads();
            if (lane == 0) s_red[0][warp] = mx;
            if (nan_seen) s_flag = 1;
            __syncthreads();
            float row_max = s_red[0][0];
#pragma unroll
            for (int w2 = 1; w2 < TOPM_WARPS; ++w2) row_max = fmaxf(row_max, s_red[0][w2]);
            const bool fin = fabsf(row_max) < CUDART_INF_F;
            const float ref = fin ? row_max * p.c2 : 0.f;
            float sum = 0.f;
            for_row<DT, VEC>(rowp, V, [&](int, int e0, const float* x) {
#pragma unroll
                for (int j = 0; j < EPV; ++j)
                    if (e0 + j < V) sum += ex2_approx(fmaf(x[j], p.c2, -ref));
            });
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(FULL, sum, o);
            if (lane == 0) s_red[1][warp] = sum;
            __syncthreads();
            if (tid == 0) {
                float t = 0.f;
                for (int w2 = 0; w2 < TOPM_WARPS; ++w2) t += s_red[1][w2];
                if (s_flag || row_max == CUDART_INF_F) t = CUDART_NAN_F;
                p.lse[row] = make_float2(row_max == -CUDART_INF_F ? -CUDART_INF_F : ref, row_max == -CUDART_INF_F ? 0.f : t);
            }
        }
    }

    // ---- C. the candidates themselves, the `want` best of them, in ascending id
    __syncthreads();
    const unsigned int n_hits = ctl.count;
    __syncthreads();
    if (tid == 0) ctl.count = 0u;
    __syncthreads();
    bool redo = n_hits > unsigned(SEL_HITS), too_few = false;
    if (!redo) {
        for (unsigned int h0 = 0; h0 < n_hits; h0 += TOPM_THREADS) {      // the lanes of a warp stay together
            const unsigned int h = h0 + tid;
            const int vi = h < n_hits ? hits[h] : 0;
            float x[EPV];
            L::unpack(load_vec(vi), x);
            unsigned int take = 0u;                       // which of the vector's logits are candidates
#pragma unroll
            for (int j = 0; j < EPV; ++j) take |= (h < n_hits && vi * EPV + j < V && x[j] >= thr) ? (1u << j) : 0u;
            // one reservation per warp
            const unsigned int mine = unsigned(__popc(take));
            unsigned int incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned int v = __shfl_up_sync(FULL, incl, o);
                if (lane >= o) incl += v;
            }
            unsigned int base = 0u;
            if (lane == 31 && incl) base = atomicAdd(&ctl.count, incl);
            unsigned int pos = __shfl_sync(FULL, base, 31) + incl - mine;
#pragma unroll
            for (int j = 0; j < EPV; ++j) {
                if ((take >> j) & 1u) {
                    if (pos < unsigned(SEL_CAP)) { keys[pos] = order_key(x[j]); ids[pos] = vi * EPV + j; }
                    ++pos;
                }
            }
        }
        __syncthreads();
        const unsigned int cnt = ctl.count;
        redo = cnt > unsigned(SEL_CAP) || cnt < want;
        too_few = cnt < want;
        if (!redo) {
            unsigned int n = cnt;
            if (cnt > want) {
                select_best(keys, ids, cnt, want, V, DT == DISC_BF16, rs.hist, rs.wsum, ctl);
                n = ctl.count;
            }
            // the ids in ascending order: few - every thread counts the ids below its own; many - a
            // counting sort over the ids' upper eleven bits, then order inside the (tiny) buckets
            __syncthreads();
            const int32_t* tids;
            if (n <= unsigned(TOPM_THREADS)) {
                int32_t* dst = reinterpret_cast<int32_t*>(rs.hist);
                if (unsigned(tid) < n) {
                    const int32_t mine = ids[tid];
                    unsigned int below = 0u;
                    for (unsigned int j = 0; j < n; ++j) below += ids[j] < mine ? 1u : 0u;
                    dst[below] = mine;
                }
                tids = dst;
                __syncthreads();
            } else {
                const int shift = max(32 - __clz(V - 1) - RADIX_BITS, 0);      // id >> shift < BINS
                unsigned int* cnt = rs.hist;
                int32_t* dst = reinterpret_cast<int32_t*>(keys);               // the keys have done their work
                for (int i = tid; i < BINS; i += TOPM_THREADS) cnt[i] = 0u;
                __syncthreads();
                for (unsigned int i = tid; i < n; i += TOPM_THREADS) atomicAdd(&cnt[ids[i] >> shift], 1u);
                __syncthreads();
                // exclusive prefix sums over the buckets: thread t owns the buckets [8t, 8t+8)
                unsigned int len[BINS_PER_THREAD], mine = 0u;
#pragma unroll
                for (int k = 0; k < BINS_PER_THREAD; ++k) { len[k] = cnt[tid * BINS_PER_THREAD + k]; mine += len[k]; }
                unsigned int incl = mine;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const unsigned int v = __shfl_up_sync(FULL, incl, o);
                    if (lane >= o) incl += v;
                }
                if (lane == 31) rs.wsum[warp] = incl;
                __syncthreads();
                unsigned int start = incl - mine;
                for (int w2 = 0; w2 < warp; ++w2) start += rs.wsum[w2];
                unsigned int first[BINS_PER_THREAD];
#pragma unroll
                for (int k = 0; k < BINS_PER_THREAD; ++k) { first[k] = start; cnt[tid * BINS_PER_THREAD + k] = start; start += len[k]; }
                __syncthreads();
                for (unsigned int i = tid; i < n; i += TOPM_THREADS) {
                    const int32_t id = ids[i];
                    dst[atomicAdd(&cnt[id >> shift], 1u)] = id;
                }
                __syncthreads();
#pragma unroll
                for (int k = 0; k < BINS_PER_THREAD; ++k) {
                    for (unsigned int i = first[k] + 1u; i < first[k] + len[k]; ++i) {      // insertion sort of a bucket
                        const int32_t v = dst[i];
                        unsigned int j = i;
                        for (; j > first[k] && dst[j - 1] > v; --j) dst[j] = dst[j - 1];
                        dst[j] = v;
                    }
                }
                tids = dst;
                __syncthreads();
            }
            for (int m = tid; m < p.M; m += TOPM_THREADS) out[m] = unsigned(m) < n ? tids[m] : -1;
        }
    }
    finished = !redo;
    if (redo && !(too_few && can_lower)) break;      // a lower threshold would not help
    }
    if (!finished) {
        // Both thresholds too high, or too low for the room there is (rows of equal logits, rows
        // without numbers): the histogram passes.
        __syncthreads();
        radix_row<DT, VEC>(p, row, rs, false);
    }
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
    if (min(M, vocab_size) <= SEL_KEEP) {
        if (dtype == DISC_F32) {
            if (vec) disc_topm_stream_kernel<DISC_F32, true><<<grid, TOPM_THREADS, 0, st>>>(p);
            else disc_topm_stream_kernel<DISC_F32, false><<<grid, TOPM_THREADS, 0, st>>>(p);
        } else {
            if (vec) disc_topm_stream_kernel<DISC_BF16, true><<<grid, TOPM_THREADS, 0, st>>>(p);
            else disc_topm_stream_kernel<DISC_BF16, false><<<grid, TOPM_THREADS, 0, st>>>(p);
        }
    } else if (dtype == DISC_F32) {
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
