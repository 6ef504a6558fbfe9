// disc_verify: Algorithm 2 as the paper states it - the validity of M candidate tokens per partial
// sequence, decided by binary searches in the lexicographically sorted member array alone (the
// prefix index that disc_mask and disc_step walk is not touched, so this is also an independent
// check of it on the device).
//
// For candidate t_m of prefix a the paper searches the smallest row of X that is not smaller than
// V_m = a + [t_m]; t_m is valid iff V_m is a prefix of that row (Section 3.2, "Parallel
// Verification").  All M rows V_m share a, so the work is split in two kernels:
//   1. verify_range_kernel, one warp per prefix: the rows having a as a prefix form a contiguous
//      range [lo, hi) of X; both ends come from one binary search each, with the lanes comparing
//      the positions of a row against a in parallel (first difference decides; a row that ends
//      inside a is smaller).
//   2. inside [lo, hi) all rows agree with a, so V_m is located by a binary search on the single
//      column |a|; the search lands on the same row index as a search over all of X would.  One
//      thread per candidate when a prefix has few (verify_candidates_kernel); with 128 or more, one
//      block per prefix that first narrows every search between two of 256 pivot rows held in
//      shared memory (verify_candidates_pivot_kernel).
// Rows are ragged (no padding token): a row shorter than the compared position counts as smaller.

#include "disc_internal.cuh"

namespace {

constexpr int VR_THREADS = 128;
constexpr int VR_WARPS = VR_THREADS / 32;

struct VerifyParams {
    const int32_t* tok;          // [E] sorted table
    const uint32_t* row_off;     // [N+1]
    int32_t N, V;
    const int32_t* prefix;
    int32_t prefix_ld;
    const int32_t* prefix_len;
    int64_t n;
    const int32_t* cand;
    int32_t M;
    uint8_t* valid_out;
    int32_t* row_out;
    uint32_t* mask_out;
    int32_t W;
    int32_t *lo_out, *hi_out;
};

// Is row j of the table "before" the key a[0..len)?  upper = false: row < a (lower bound of a);
// upper = true: row < a or row has a as a prefix (lower bound of the first row beyond a's range).
// One warp; len <= DISC_MAX_DEPTH, two positions per lane.
__device__ __forceinline__ bool row_before(const VerifyParams& p, int32_t j, int32_t a0, int32_t a1, int32_t len,
                                           bool upper, int lane) {
    const uint32_t b = __ldg(p.row_off + j), e = __ldg(p.row_off + j + 1);
    const int32_t rl = int32_t(e - b);
    // state of position q: 0 equal, 1 row smaller here (or row ended), 2 row larger here
    auto state = [&](int q, int32_t aq) -> int {
        if (q >= len) return 0;
        if (q >= rl) return 1;
        const int32_t t = __ldg(p.tok + b + q);
        return t < aq ? 1 : (t > aq ? 2 : 0);
    };
    const int s0 = state(lane, a0), s1 = state(lane + 32, a1);
    const uint32_t d0 = __ballot_sync(0xffffffffu, s0 != 0), d1 = __ballot_sync(0xffffffffu, s1 != 0);
    if (d0) return __shfl_sync(0xffffffffu, s0, __ffs(d0) - 1) == 1;
    if (d1) return __shfl_sync(0xffffffffu, s1, __ffs(d1) - 1) == 1;
    return upper;            // the row has a as a prefix (rl >= len): inside the range
}

__global__ void __launch_bounds__(VR_THREADS) verify_range_kernel(const VerifyParams p) {
    const int lane = threadIdx.x & 31;
    const int64_t i = int64_t(blockIdx.x) * VR_WARPS + (threadIdx.x >> 5);
    if (i >= p.n) return;
    int32_t len = p.prefix_len[i];
    const bool bad = len < 0 || len > p.prefix_ld || len > DISC_MAX_DEPTH;
    if (bad) len = 0;
    const int32_t* a = p.prefix + i * p.prefix_ld;
    const int32_t a0 = lane < len ? a[lane] : 0, a1 = lane + 32 < len ? a[lane + 32] : 0;
    int32_t bound[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
        int32_t x = 0, y = p.N;                     // the first row not "before" the key is in [x, y]
        while (x < y) {
            const int32_t mid = x + ((y - x) >> 1);
            if (row_before(p, mid, a0, a1, len, u == 1, lane)) x = mid + 1; else y = mid;
        }
        bound[u] = x;
    }
    if (lane == 0) {
        p.lo_out[i] = bad ? 0 : bound[0];
        p.hi_out[i] = bad ? 0 : bound[1];
    }
}

// What the searches of one prefix share: its range, the column, and where the search starts.
// Inside [lo, hi) every row has the prefix, so it has at least d tokens; only a row that IS the
// prefix has exactly d, and it sorts first.  It is smaller than every a + [t], so the searches skip
// it and a row's key is simply its token at column d (two dependent loads per probe, not three).
struct RowRange {
    int32_t lo, hi, d, first;     // first: the first row the searches look at (lo or lo + 1)
};
__device__ __forceinline__ RowRange row_range(const VerifyParams& p, int64_t i) {
    RowRange r;
    r.lo = p.lo_out[i];
    r.hi = p.hi_out[i];
    r.d = p.prefix_len[i];
    if (r.d < 0 || r.d > p.prefix_ld || r.d > DISC_MAX_DEPTH) r.d = 0;      // such a prefix got the empty range
    r.first = r.lo;
    if (r.lo < r.hi && int32_t(__ldg(p.row_off + r.lo + 1) - __ldg(p.row_off + r.lo)) <= r.d) r.first = r.lo + 1;
    return r;
}
__device__ __forceinline__ int32_t key_at(const VerifyParams& p, int32_t j, int32_t d) {
    return __ldg(p.tok + __ldg(p.row_off + j) + d);
}
// the first row of [x, y) whose key is not below t (y if there is none), then what the search says
__device__ __forceinline__ void finish_candidate(const VerifyParams& p, const RowRange& r, int64_t i, int64_t g, int32_t t,
                                                 int32_t x, int32_t y) {
    while (x < y) {
        const int32_t mid = x + ((y - x) >> 1);
        if (key_at(p, mid, r.d) < t) x = mid + 1; else y = mid;
    }
    const bool ok = t >= 0 && t < p.V && x < r.hi && key_at(p, x, r.d) == t;
    p.valid_out[g] = ok ? 1 : 0;
    if (p.row_out) p.row_out[g] = x;
    if (ok && p.mask_out) atomicOr(p.mask_out + i * p.W + (t >> 5), 1u << (t & 31));
}

// Few candidates per prefix: one thread per candidate.
__global__ void __launch_bounds__(256) verify_candidates_kernel(const VerifyParams p) {
    const int64_t g = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (g >= p.n * p.M) return;
    const int64_t i = g / p.M;
    const RowRange r = row_range(p, i);
    finish_candidate(p, r, i, g, p.cand[g], r.first, r.hi);
}

// Many candidates per prefix: one block per prefix.  The block first reads the keys of VP evenly
// spaced rows of the range into shared memory; a candidate finds its place among these pivots
// there (8 steps that touch no global memory) and searches only between two neighbouring pivots.
// The searches of a prefix all run over the same rows, so the pivots' 2 x VP loads replace eight
// probes of every candidate.
constexpr int VP = 256;
__global__ void __launch_bounds__(VP) verify_candidates_pivot_kernel(const VerifyParams p) {
    __shared__ int32_t piv[VP];
    const int64_t i = blockIdx.x;
    const RowRange r = row_range(p, i);
    const int64_t span = int64_t(r.hi) - r.first;
    const bool use_piv = span > 4 * VP;
    auto pos = [&](int k) -> int32_t { return r.first + int32_t((int64_t(k + 1) * span) / (VP + 1)); };   // k = 0 .. VP-1
    if (use_piv) piv[threadIdx.x] = key_at(p, pos(threadIdx.x), r.d);
    __syncthreads();
    for (int m = threadIdx.x; m < p.M; m += VP) {
        const int64_t g = i * p.M + m;
        const int32_t t = p.cand[g];
        int32_t x = r.first, y = r.hi;
        if (use_piv) {
            int a = 0, b = VP;                      // the first pivot whose key is not below t
            while (a < b) {
                const int mid = (a + b) >> 1;
                if (piv[mid] < t) a = mid + 1; else b = mid;
            }
            if (a > 0) x = pos(a - 1) + 1;
            if (a < VP) y = pos(a);
        }
        finish_candidate(p, r, i, g, t, x, y);
    }
}

}  // namespace

extern "C" int disc_verify(const disc_set_t* s, const int32_t* prefix, int32_t prefix_ld, const int32_t* prefix_len,
                           int64_t n, const int32_t* cand, int32_t M, uint8_t* valid_out, int32_t* row_out,
                           uint32_t* mask_out, int32_t* lo_out, int32_t* hi_out, void* stream) {
    if (!s || n < 0 || prefix_ld < 0 || M < 0) return DISC_ERR_ARG;
    if (const int rc = disc::check_device(s)) return rc;
    if (n == 0) return DISC_OK;
    if (!prefix_len || !lo_out || !hi_out || (prefix_ld > 0 && !prefix)) return DISC_ERR_ARG;
    if (M > 0 && (!cand || !valid_out)) return DISC_ERR_ARG;
    if (n * int64_t(M > 0 ? M : 1) >= (int64_t(1) << 38)) return DISC_ERR_UNSUPPORTED;
    VerifyParams p;
    p.tok = s->tok; p.row_off = s->row_off; p.N = int32_t(s->N); p.V = s->V;
    p.prefix = prefix; p.prefix_ld = prefix_ld; p.prefix_len = prefix_len; p.n = n;
    p.cand = cand; p.M = M; p.valid_out = valid_out; p.row_out = row_out; p.mask_out = mask_out; p.W = s->W;
    p.lo_out = lo_out; p.hi_out = hi_out;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (mask_out) DISC_CUDA(cudaMemsetAsync(mask_out, 0, size_t(n) * size_t(s->W) * sizeof(uint32_t), st));
    verify_range_kernel<<<unsigned((n + VR_WARPS - 1) / VR_WARPS), VR_THREADS, 0, st>>>(p);
    DISC_CUDA(cudaGetLastError());
    if (M > 0) {
        if (M >= 128) {
            verify_candidates_pivot_kernel<<<unsigned(n), VP, 0, st>>>(p);
        } else {
            const int64_t total = n * M;
            verify_candidates_kernel<<<unsigned((total + 255) / 256), 256, 0, st>>>(p);
        }
        DISC_CUDA(cudaGetLastError());
    }
    return DISC_OK;
}
