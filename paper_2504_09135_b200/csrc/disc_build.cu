// disc_build_set and friends: device-side preparation of the constraint array
// (Algorithm 2, line 1; Section 3.2 "Array Preparation").
//
// The members are sorted on the GPU by a least-significant-position-first sequence of stable radix
// sorts (one pass per token position, key = token+1, 0 past the end of a member so that a shorter
// member sorts before its extensions), then de-duplicated, checked for prefix-freeness, and indexed
// level by level: a member row creates one index node for every prefix length in
// (lcp with the previous row, its own length], so node counts and positions come from prefix sums.
// Sorting and scans use CUB; this code is off the per-step path.

#include <chrono>
#include <new>
#include <vector>
#include <cstring>
#include <new>

#include <cub/cub.cuh>

#include "disc_internal.cuh"

namespace disc {
thread_local int g_last_cuda_error = 0;
}

namespace {

using disc::cuda_fail;

struct DevBuf {
    void* p = nullptr;
    size_t bytes = 0;
    DevBuf() = default;
    DevBuf(const DevBuf&) = delete;
    DevBuf& operator=(const DevBuf&) = delete;
    ~DevBuf() { release(); }
    void release() {
        if (p) cudaFree(p);
        p = nullptr;
        bytes = 0;
    }
    cudaError_t alloc(size_t n) {
        release();
        bytes = n ? n : 16;
        return cudaMalloc(&p, bytes);
    }
    template <class T>
    T* as() const { return static_cast<T*>(p); }
    void* take() {
        void* q = p;
        p = nullptr;
        return q;
    }
};

enum : uint32_t { ERRBIT_TOKEN = 1, ERRBIT_EMPTY = 2, ERRBIT_ARG = 4, ERRBIT_PREFIX = 8 };

constexpr int TPB = 256;
inline unsigned blocks_for(int64_t n) { return unsigned((n + TPB - 1) / TPB); }

__global__ void k_validate_tokens(const int32_t* __restrict__ tok, int64_t E, int32_t V, uint32_t* err) {
    int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < E) {
        int32_t t = tok[i];
        if (t < 0 || t >= V) atomicOr(err, ERRBIT_TOKEN);
    }
}

__global__ void k_row_len(const int64_t* __restrict__ off64, int64_t n, int64_t base, int32_t* len,
                          uint32_t* off32, uint32_t* err, int32_t* lmax) {
    int64_t r = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (r >= n) return;
    int64_t a = off64[r], b = off64[r + 1];
    int64_t l = b - a;
    if (l < 0) { atomicOr(err, ERRBIT_ARG); l = 0; }
    if (l == 0) atomicOr(err, ERRBIT_EMPTY);
    if (l > DISC_MAX_DEPTH) { atomicMax(lmax, DISC_MAX_DEPTH + 1); l = DISC_MAX_DEPTH + 1; }
    len[r] = int32_t(l);
    off32[r] = uint32_t(a - base);
    atomicMax(lmax, int32_t(l));
}

__global__ void k_iota(uint32_t* p, int64_t n) {
    int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < n) p[i] = uint32_t(i);
}

// key of row perm[i] at token position d: token+1, or 0 when the row is shorter
__global__ void k_position_keys(const uint32_t* __restrict__ perm, const int32_t* __restrict__ len,
                                const uint32_t* __restrict__ off, const int32_t* __restrict__ tok,
                                int32_t d, uint32_t* __restrict__ keys, int64_t n) {
    int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n) return;
    uint32_t r = perm[i];
    keys[i] = d < len[r] ? uint32_t(tok[off[r] + d]) + 1u : 0u;
}

// compare each sorted row with its predecessor: common prefix length, duplicate flag, prefix check
__global__ void k_adjacent(const uint32_t* __restrict__ perm, const int32_t* __restrict__ len,
                           const uint32_t* __restrict__ off, const int32_t* __restrict__ tok, int64_t n,
                           int32_t* __restrict__ lcp, uint32_t* __restrict__ keep, uint32_t* err) {
    int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n) return;
    if (i == 0) { lcp[0] = 0; keep[0] = 1; return; }
    uint32_t a = perm[i - 1], b = perm[i];
    int32_t la = len[a], lb = len[b];
    const int32_t* pa = tok + off[a];
    const int32_t* pb = tok + off[b];
    int32_t m = la < lb ? la : lb, c = 0;
    while (c < m && pa[c] == pb[c]) ++c;
    bool dup = (c == la) && (c == lb);
    if (!dup && c == la) atomicOr(err, ERRBIT_PREFIX);   // predecessor is a proper prefix of this row
    lcp[i] = c;
    keep[i] = dup ? 0u : 1u;
}

__global__ void k_compact(const uint32_t* __restrict__ perm, const int32_t* __restrict__ len,
                          const int32_t* __restrict__ lcp, const uint32_t* __restrict__ keep,
                          const uint32_t* __restrict__ pos, int64_t n, uint32_t* __restrict__ s_src,
                          uint32_t* __restrict__ s_len, int32_t* __restrict__ s_lcp) {
    int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= n || !keep[i]) return;
    uint32_t j = pos[i];
    s_src[j] = perm[i];
    s_len[j] = uint32_t(len[perm[i]]);
    s_lcp[j] = lcp[i];
}

__global__ void k_copy_rows(const uint32_t* __restrict__ s_src, const uint32_t* __restrict__ s_len,
                            const uint32_t* __restrict__ in_off, const int32_t* __restrict__ in_tok,
                            const uint32_t* __restrict__ row_off, int32_t* __restrict__ out_tok, int64_t N) {
    int64_t j = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (j >= N) return;
    const int32_t* src = in_tok + in_off[s_src[j]];
    int32_t* dst = out_tok + row_off[j];
    uint32_t l = s_len[j];
    for (uint32_t k = 0; k < l; ++k) dst[k] = src[k];
}

// flag[j] = 1 iff sorted row j creates a node at level d (prefix length d+1)
__global__ void k_level_flags(const int32_t* __restrict__ s_lcp, const uint32_t* __restrict__ s_len,
                              int32_t d, uint32_t* __restrict__ flag, int64_t N) {
    int64_t j = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (j < N) flag[j] = (s_lcp[j] <= d && uint32_t(d) < s_len[j]) ? 1u : 0u;
}

// write the nodes of level d.  scan_d / scan_d1: exclusive prefix sums of the level-d / level-(d+1)
// flags; the first child of the node created by row j at level d is the level-(d+1) node at
// position scan_d1[j].
__global__ void k_scatter_level(const int32_t* __restrict__ s_lcp, const uint32_t* __restrict__ s_len,
                                const uint32_t* __restrict__ scan_d, const uint32_t* __restrict__ scan_d1,
                                int32_t d, int64_t N, int64_t off_d, int64_t off_d1,
                                const int32_t* __restrict__ tok, const uint32_t* __restrict__ row_off,
                                int32_t* __restrict__ node_tok, int32_t* __restrict__ node_lo,
                                int32_t* __restrict__ child_begin) {
    int64_t j = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (j >= N) return;
    if (!(s_lcp[j] <= d && uint32_t(d) < s_len[j])) return;
    int64_t g = off_d + scan_d[j];
    node_tok[g] = tok[row_off[j] + d];
    node_lo[g] = int32_t(j);
    child_begin[g] = int32_t(off_d1 + (scan_d1 ? scan_d1[j] : 0u));
}

__global__ void k_root_tables(const int32_t* __restrict__ node_tok, int64_t first, int64_t count,
                              int32_t* __restrict__ root_child, uint32_t* __restrict__ root_mask) {
    int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= count) return;
    int32_t t = node_tok[first + i];
    root_child[t] = int32_t(first + i);
    atomicOr(&root_mask[t >> 5], 1u << (t & 31));
}

struct HeavyPred {
    const int32_t* child_begin;
    __device__ bool operator()(int32_t j) const {
        return j > 0 && (child_begin[j + 1] - child_begin[j]) > DISC_HEAVY_MIN;
    }
};

// one block per heavy node: set the bits of its children in its prebuilt mask row
__global__ void k_heavy_masks(const int32_t* __restrict__ heavy_nodes, const int32_t* __restrict__ child_begin,
                              const int32_t* __restrict__ node_tok, int32_t W, uint32_t* __restrict__ masks) {
    const int32_t j = heavy_nodes[blockIdx.x];
    uint32_t* row = masks + size_t(blockIdx.x) * W;
    for (int32_t i = child_begin[j] + threadIdx.x; i < child_begin[j + 1]; i += blockDim.x) {
        int32_t t = node_tok[i];
        atomicOr(&row[t >> 5], 1u << (t & 31));
    }
}

__global__ void k_fill_i32(int32_t* p, int32_t v, int64_t n) {
    int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < n) p[i] = v;
}

__global__ void k_off_to_i64(const uint32_t* __restrict__ in, int64_t* __restrict__ out, int64_t n) {
    int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < n) out[i] = int64_t(in[i]);
}

int exclusive_sum(const uint32_t* in, uint32_t* out, int64_t n, DevBuf& temp, cudaStream_t st) {
    size_t need = 0;
    DISC_CUDA(cub::DeviceScan::ExclusiveSum(nullptr, need, in, out, int(n), st));
    if (need > temp.bytes) DISC_CUDA(temp.alloc(need));
    DISC_CUDA(cub::DeviceScan::ExclusiveSum(temp.p, need, in, out, int(n), st));
    return DISC_OK;
}

// last element of an exclusive scan + last input element = total
int scan_total(const uint32_t* in, const uint32_t* scan, int64_t n, cudaStream_t st, uint64_t* total) {
    uint32_t a = 0, b = 0;
    DISC_CUDA(cudaMemcpyAsync(&a, in + (n - 1), 4, cudaMemcpyDeviceToHost, st));
    DISC_CUDA(cudaMemcpyAsync(&b, scan + (n - 1), 4, cudaMemcpyDeviceToHost, st));
    DISC_CUDA(cudaStreamSynchronize(st));
    *total = uint64_t(a) + uint64_t(b);
    return DISC_OK;
}

int build_impl(const int32_t* tokens, const int64_t* row_offsets, int64_t n, int32_t V, cudaStream_t st,
               disc_set* S) {
    const int64_t base = row_offsets[0];
    const int64_t E_in = row_offsets[n] - base;
    if (base < 0 || E_in < 0) return DISC_ERR_ARG;
    if (E_in == 0) return DISC_ERR_EMPTY;
    if (n >= (int64_t(1) << 31) - 1 || E_in >= (int64_t(1) << 32) - 1) return DISC_ERR_UNSUPPORTED;

    DISC_CUDA(cudaGetDevice(&S->device));
    S->V = V;
    S->W = (V + 31) / 32;
    S->Wp = (S->W + 3) & ~3;

    DevBuf in_tok, in_off64, in_off, len, err, lmax_d;
    DISC_CUDA(in_tok.alloc(size_t(E_in) * 4));
    DISC_CUDA(in_off64.alloc(size_t(n + 1) * 8));
    DISC_CUDA(in_off.alloc(size_t(n) * 4));
    DISC_CUDA(len.alloc(size_t(n) * 4));
    DISC_CUDA(err.alloc(8));
    DISC_CUDA(lmax_d.alloc(8));
    DISC_CUDA(cudaMemcpyAsync(in_tok.p, tokens + base, size_t(E_in) * 4, cudaMemcpyHostToDevice, st));
    DISC_CUDA(cudaMemcpyAsync(in_off64.p, row_offsets, size_t(n + 1) * 8, cudaMemcpyHostToDevice, st));
    DISC_CUDA(cudaMemsetAsync(err.p, 0, 8, st));
    DISC_CUDA(cudaMemsetAsync(lmax_d.p, 0, 8, st));

    k_validate_tokens<<<blocks_for(E_in), TPB, 0, st>>>(in_tok.as<int32_t>(), E_in, V, err.as<uint32_t>());
    k_row_len<<<blocks_for(n), TPB, 0, st>>>(in_off64.as<int64_t>(), n, base, len.as<int32_t>(),
                                             in_off.as<uint32_t>(), err.as<uint32_t>(), lmax_d.as<int32_t>());
    DISC_CUDA(cudaGetLastError());
    uint32_t h_err = 0;
    int32_t l_max = 0;
    DISC_CUDA(cudaMemcpyAsync(&h_err, err.p, 4, cudaMemcpyDeviceToHost, st));
    DISC_CUDA(cudaMemcpyAsync(&l_max, lmax_d.p, 4, cudaMemcpyDeviceToHost, st));
    DISC_CUDA(cudaStreamSynchronize(st));
    in_off64.release();
    if (h_err & ERRBIT_ARG) return DISC_ERR_ARG;
    if (h_err & ERRBIT_EMPTY) return DISC_ERR_EMPTY;
    if (h_err & ERRBIT_TOKEN) return DISC_ERR_TOKEN;
    if (l_max > DISC_MAX_DEPTH) return DISC_ERR_UNSUPPORTED;
    S->l_max = l_max;

    // ---- lexicographic sort of the rows: one stable radix pass per token position, last first
    DevBuf perm_a, perm_b, key_a, key_b, temp;
    DISC_CUDA(perm_a.alloc(size_t(n) * 4));
    DISC_CUDA(perm_b.alloc(size_t(n) * 4));
    DISC_CUDA(key_a.alloc(size_t(n) * 4));
    DISC_CUDA(key_b.alloc(size_t(n) * 4));
    k_iota<<<blocks_for(n), TPB, 0, st>>>(perm_a.as<uint32_t>(), n);
    int end_bit = 1;
    while ((uint64_t(1) << end_bit) <= uint64_t(V)) ++end_bit;   // keys lie in [0, V]
    cub::DoubleBuffer<uint32_t> keys(key_a.as<uint32_t>(), key_b.as<uint32_t>());
    cub::DoubleBuffer<uint32_t> perm(perm_a.as<uint32_t>(), perm_b.as<uint32_t>());
    size_t sort_bytes = 0;
    DISC_CUDA(cub::DeviceRadixSort::SortPairs(nullptr, sort_bytes, keys, perm, int(n), 0, end_bit, st));
    DISC_CUDA(temp.alloc(sort_bytes));
    for (int32_t d = l_max - 1; d >= 0; --d) {
        k_position_keys<<<blocks_for(n), TPB, 0, st>>>(perm.Current(), len.as<int32_t>(), in_off.as<uint32_t>(),
                                                      in_tok.as<int32_t>(), d, keys.Current(), n);
        size_t bytes = temp.bytes;
        DISC_CUDA(cub::DeviceRadixSort::SortPairs(temp.p, bytes, keys, perm, int(n), 0, end_bit, st));
    }
    DISC_CUDA(cudaGetLastError());

    // ---- duplicates, prefix-freeness, common prefix lengths
    DevBuf lcp, keep, pos;
    DISC_CUDA(lcp.alloc(size_t(n) * 4));
    DISC_CUDA(keep.alloc(size_t(n) * 4));
    DISC_CUDA(pos.alloc(size_t(n) * 4));
    k_adjacent<<<blocks_for(n), TPB, 0, st>>>(perm.Current(), len.as<int32_t>(), in_off.as<uint32_t>(),
                                             in_tok.as<int32_t>(), n, lcp.as<int32_t>(), keep.as<uint32_t>(),
                                             err.as<uint32_t>());
    int rc = exclusive_sum(keep.as<uint32_t>(), pos.as<uint32_t>(), n, temp, st);
    if (rc) return rc;
    uint64_t N64 = 0;
    rc = scan_total(keep.as<uint32_t>(), pos.as<uint32_t>(), n, st, &N64);
    if (rc) return rc;
    DISC_CUDA(cudaMemcpy(&h_err, err.p, 4, cudaMemcpyDeviceToHost));
    if (h_err & ERRBIT_PREFIX) return DISC_ERR_PREFIX;
    const int64_t N = int64_t(N64);
    S->N = N;

    DevBuf s_src, s_len, s_lcp;
    DISC_CUDA(s_src.alloc(size_t(N) * 4));
    DISC_CUDA(s_len.alloc(size_t(N) * 4));
    DISC_CUDA(s_lcp.alloc(size_t(N) * 4));
    k_compact<<<blocks_for(n), TPB, 0, st>>>(perm.Current(), len.as<int32_t>(), lcp.as<int32_t>(),
                                            keep.as<uint32_t>(), pos.as<uint32_t>(), n, s_src.as<uint32_t>(),
                                            s_len.as<uint32_t>(), s_lcp.as<int32_t>());
    DISC_CUDA(cudaGetLastError());
    DISC_CUDA(cudaStreamSynchronize(st));
    perm_a.release(); perm_b.release(); key_a.release(); key_b.release();
    lcp.release(); keep.release(); pos.release(); len.release();

    // ---- sorted table
    DevBuf row_off;
    DISC_CUDA(row_off.alloc(size_t(N + 1) * 4));
    rc = exclusive_sum(s_len.as<uint32_t>(), row_off.as<uint32_t>(), N, temp, st);
    if (rc) return rc;
    uint64_t E64 = 0;
    rc = scan_total(s_len.as<uint32_t>(), row_off.as<uint32_t>(), N, st, &E64);
    if (rc) return rc;
    const int64_t E = int64_t(E64);
    S->E = E;
    uint32_t E32 = uint32_t(E);
    DISC_CUDA(cudaMemcpyAsync(row_off.as<uint32_t>() + N, &E32, 4, cudaMemcpyHostToDevice, st));
    DevBuf tok;
    DISC_CUDA(tok.alloc(size_t(E) * 4));
    k_copy_rows<<<blocks_for(N), TPB, 0, st>>>(s_src.as<uint32_t>(), s_len.as<uint32_t>(), in_off.as<uint32_t>(),
                                              in_tok.as<int32_t>(), row_off.as<uint32_t>(), tok.as<int32_t>(), N);
    DISC_CUDA(cudaGetLastError());
    DISC_CUDA(cudaStreamSynchronize(st));
    in_tok.release(); in_off.release(); s_src.release();

    // ---- level sizes
    DevBuf flag, scan_cur, scan_next;
    DISC_CUDA(flag.alloc(size_t(N) * 4));
    DISC_CUDA(scan_cur.alloc(size_t(N) * 4));
    DISC_CUDA(scan_next.alloc(size_t(N) * 4));
    int64_t level_n[DISC_MAX_DEPTH + 1] = {0};
    for (int32_t d = 0; d < l_max; ++d) {
        k_level_flags<<<blocks_for(N), TPB, 0, st>>>(s_lcp.as<int32_t>(), s_len.as<uint32_t>(), d,
                                                    flag.as<uint32_t>(), N);
        rc = exclusive_sum(flag.as<uint32_t>(), scan_cur.as<uint32_t>(), N, temp, st);
        if (rc) return rc;
        uint64_t c = 0;
        rc = scan_total(flag.as<uint32_t>(), scan_cur.as<uint32_t>(), N, st, &c);
        if (rc) return rc;
        level_n[d] = int64_t(c);
    }
    S->level_off[0] = 1;
    for (int32_t d = 0; d < l_max; ++d) S->level_off[d + 1] = S->level_off[d] + level_n[d];
    const int64_t M = S->level_off[l_max];
    if (M >= (int64_t(1) << 31) - 2) return DISC_ERR_UNSUPPORTED;
    S->M = M;

    // ---- index nodes, deepest level first so that the next level's scan is at hand
    DevBuf node_tok, node_lo, child_begin, root_mask, root_child;
    DISC_CUDA(node_tok.alloc(size_t(M) * 4));
    DISC_CUDA(node_lo.alloc(size_t(M) * 4));
    DISC_CUDA(child_begin.alloc(size_t(M + 1) * 4));
    DISC_CUDA(root_mask.alloc(size_t(S->Wp) * 4));
    DISC_CUDA(root_child.alloc(size_t(V) * 4));
    bool have_next = false;
    for (int32_t d = l_max - 1; d >= 0; --d) {
        k_level_flags<<<blocks_for(N), TPB, 0, st>>>(s_lcp.as<int32_t>(), s_len.as<uint32_t>(), d,
                                                    flag.as<uint32_t>(), N);
        rc = exclusive_sum(flag.as<uint32_t>(), scan_cur.as<uint32_t>(), N, temp, st);
        if (rc) return rc;
        k_scatter_level<<<blocks_for(N), TPB, 0, st>>>(
            s_lcp.as<int32_t>(), s_len.as<uint32_t>(), scan_cur.as<uint32_t>(),
            have_next ? scan_next.as<uint32_t>() : nullptr, d, N, S->level_off[d], S->level_off[d + 1],
            tok.as<int32_t>(), row_off.as<uint32_t>(), node_tok.as<int32_t>(), node_lo.as<int32_t>(),
            child_begin.as<int32_t>());
        void* t = scan_cur.p; scan_cur.p = scan_next.p; scan_next.p = t;
        have_next = true;
    }
    // root node and sentinel
    {
        int32_t root_vals[3] = {-1, 0, 1};
        int32_t sentinel = int32_t(M);
        DISC_CUDA(cudaMemcpyAsync(node_tok.p, &root_vals[0], 4, cudaMemcpyHostToDevice, st));
        DISC_CUDA(cudaMemcpyAsync(node_lo.p, &root_vals[1], 4, cudaMemcpyHostToDevice, st));
        DISC_CUDA(cudaMemcpyAsync(child_begin.p, &root_vals[2], 4, cudaMemcpyHostToDevice, st));
        DISC_CUDA(cudaMemcpyAsync(child_begin.as<int32_t>() + M, &sentinel, 4, cudaMemcpyHostToDevice, st));
        DISC_CUDA(cudaStreamSynchronize(st));
    }
    DISC_CUDA(cudaMemsetAsync(root_mask.p, 0, size_t(S->Wp) * 4, st));
    k_fill_i32<<<blocks_for(V), TPB, 0, st>>>(root_child.as<int32_t>(), -1, V);
    k_root_tables<<<blocks_for(level_n[0]), TPB, 0, st>>>(node_tok.as<int32_t>(), 1, level_n[0],
                                                         root_child.as<int32_t>(), root_mask.as<uint32_t>());
    DISC_CUDA(cudaGetLastError());
    DISC_CUDA(cudaStreamSynchronize(st));

    // ---- prebuilt masks of heavy nodes (each has more than DISC_HEAVY_MIN children, so there are
    // fewer than M / DISC_HEAVY_MIN of them)
    DevBuf heavy_nodes, heavy_masks, n_sel;
    {
        const int64_t cap = M / DISC_HEAVY_MIN + 1;
        DISC_CUDA(heavy_nodes.alloc(size_t(cap) * 4));
        DISC_CUDA(n_sel.alloc(8));
        cub::CountingInputIterator<int32_t> ids(0);
        HeavyPred pred{child_begin.as<int32_t>()};
        size_t need = 0;
        DISC_CUDA(cub::DeviceSelect::If(nullptr, need, ids, heavy_nodes.as<int32_t>(), n_sel.as<int32_t>(), int(M),
                                        pred, st));
        if (need > temp.bytes) DISC_CUDA(temp.alloc(need));
        DISC_CUDA(cub::DeviceSelect::If(temp.p, need, ids, heavy_nodes.as<int32_t>(), n_sel.as<int32_t>(), int(M),
                                        pred, st));
        int32_t H = 0;
        DISC_CUDA(cudaMemcpyAsync(&H, n_sel.p, 4, cudaMemcpyDeviceToHost, st));
        DISC_CUDA(cudaStreamSynchronize(st));
        S->n_heavy = H;
        DISC_CUDA(heavy_masks.alloc(size_t(H > 0 ? H : 1) * size_t(S->Wp) * 4));
        if (H > 0) {
            DISC_CUDA(cudaMemsetAsync(heavy_masks.p, 0, size_t(H) * size_t(S->Wp) * 4, st));
            k_heavy_masks<<<unsigned(H), 256, 0, st>>>(heavy_nodes.as<int32_t>(), child_begin.as<int32_t>(),
                                                     node_tok.as<int32_t>(), S->Wp, heavy_masks.as<uint32_t>());
            DISC_CUDA(cudaGetLastError());
            DISC_CUDA(cudaStreamSynchronize(st));
        }
    }

    // scratch of disc_mask: a row counter its writer kernel draws work from (see disc_mask.cu)
    DevBuf work_counter;
    DISC_CUDA(work_counter.alloc(256));
    DISC_CUDA(cudaMemsetAsync(work_counter.p, 0, 256, st));
    DISC_CUDA(cudaStreamSynchronize(st));
    S->work_counter = static_cast<unsigned int*>(work_counter.take());

    S->device_bytes = int64_t(tok.bytes + row_off.bytes + node_tok.bytes + node_lo.bytes + child_begin.bytes +
                              root_mask.bytes + root_child.bytes + heavy_nodes.bytes + heavy_masks.bytes + 256);
    S->heavy_nodes = static_cast<int32_t*>(heavy_nodes.take());
    S->heavy_masks = static_cast<uint32_t*>(heavy_masks.take());
    S->tok = static_cast<int32_t*>(tok.take());
    S->row_off = static_cast<uint32_t*>(row_off.take());
    S->node_tok = static_cast<int32_t*>(node_tok.take());
    S->node_lo = static_cast<int32_t*>(node_lo.take());
    S->child_begin = static_cast<int32_t*>(child_begin.take());
    S->root_mask = static_cast<uint32_t*>(root_mask.take());
    S->root_child = static_cast<int32_t*>(root_child.take());
    return DISC_OK;
}

}  // namespace

extern "C" {

int disc_build_set(const int32_t* tokens, const int64_t* row_offsets, int64_t n_rows, int32_t vocab_size,
                   uint32_t flags, void* stream, disc_set_t** out) {
    if (!out) return DISC_ERR_ARG;
    *out = nullptr;
    if (!tokens || !row_offsets || n_rows < 0 || vocab_size <= 0 || flags != 0) return DISC_ERR_ARG;
    if (n_rows == 0) return DISC_ERR_EMPTY;
    if (vocab_size > 4000000) return DISC_ERR_UNSUPPORTED;
    auto t0 = std::chrono::steady_clock::now();
    disc_set* S = new (std::nothrow) disc_set();
    if (!S) return DISC_ERR_OOM;
    int rc = build_impl(tokens, row_offsets, n_rows, vocab_size, static_cast<cudaStream_t>(stream), S);
    if (rc != DISC_OK) {
        cudaGetLastError();   // clear a sticky launch error, if any
        disc_free_set(S);
        return rc;
    }
    S->build_seconds = std::chrono::duration<double>(std::chrono::steady_clock::now() - t0).count();
    *out = S;
    return DISC_OK;
}

// Sets in which a member may be a proper prefix of another (Section 2.1: when the text generated
// so far is itself a member, the end-of-keyword token is valid next to the tokens that extend
// it).  Every member is closed by eok_token on a host copy, which makes the set prefix-free, and
// the ordinary build follows: the valid set of a prefix that is a member then contains eok_token,
// and a candidate is complete once it has produced it.
int disc_build_set_eok(const int32_t* tokens, const int64_t* row_offsets, int64_t n_rows, int32_t vocab_size,
                       int32_t eok_token, void* stream, disc_set_t** out) {
    if (!out) return DISC_ERR_ARG;
    *out = nullptr;
    if (!tokens || !row_offsets || n_rows < 0 || vocab_size <= 0) return DISC_ERR_ARG;
    if (eok_token < 0 || eok_token >= vocab_size) return DISC_ERR_TOKEN;
    if (n_rows == 0) return DISC_ERR_EMPTY;
    const int64_t E = row_offsets[n_rows] - row_offsets[0];
    if (E < 0) return DISC_ERR_ARG;
    std::vector<int32_t> tok;
    std::vector<int64_t> off;
    try {
        tok.reserve(size_t(E + n_rows));
        off.reserve(size_t(n_rows + 1));
    } catch (const std::bad_alloc&) {
        return DISC_ERR_OOM;
    }
    off.push_back(0);
    for (int64_t r = 0; r < n_rows; ++r) {
        const int64_t a = row_offsets[r], b = row_offsets[r + 1];
        if (b < a) return DISC_ERR_ARG;
        if (b == a) return DISC_ERR_EMPTY;
        for (int64_t i = a; i < b; ++i) {
            if (tokens[i] == eok_token) return DISC_ERR_TOKEN;     // the closing token must not occur inside a member
            tok.push_back(tokens[i]);
        }
        tok.push_back(eok_token);
        off.push_back(int64_t(tok.size()));
    }
    return disc_build_set(tok.data(), off.data(), n_rows, vocab_size, 0u, stream, out);
}

void disc_free_set(disc_set_t* s) {
    if (!s) return;
    cudaFree(s->tok);
    cudaFree(s->row_off);
    cudaFree(s->node_tok);
    cudaFree(s->node_lo);
    cudaFree(s->child_begin);
    cudaFree(s->root_mask);
    cudaFree(s->root_child);
    cudaFree(s->heavy_nodes);
    cudaFree(s->heavy_masks);
    cudaFree(s->work_counter);
    delete s;
}

int disc_set_info(const disc_set_t* s, disc_set_info_t* info) {
    if (!s || !info) return DISC_ERR_ARG;
    std::memset(info, 0, sizeof(*info));
    info->n_members = s->N;
    info->n_entries = s->E;
    info->n_nodes = s->M - 1;
    info->vocab_size = s->V;
    info->mask_words = s->W;
    info->l_max = s->l_max;
    info->n_heavy = s->n_heavy;
    info->device_bytes = s->device_bytes;
    info->build_seconds = s->build_seconds;
    for (int d = 0; d < s->l_max; ++d) info->level_nodes[d] = s->level_off[d + 1] - s->level_off[d];
    return DISC_OK;
}

int disc_set_rows(const disc_set_t* s, int32_t* tokens_out, int64_t* row_offsets_out) {
    if (!s || !tokens_out || !row_offsets_out) return DISC_ERR_ARG;
    DISC_CUDA(cudaMemcpy(tokens_out, s->tok, size_t(s->E) * 4, cudaMemcpyDeviceToHost));
    DevBuf tmp;
    DISC_CUDA(tmp.alloc(size_t(s->N + 1) * 8));
    k_off_to_i64<<<blocks_for(s->N + 1), TPB>>>(s->row_off, tmp.as<int64_t>(), s->N + 1);
    DISC_CUDA(cudaGetLastError());
    DISC_CUDA(cudaMemcpy(row_offsets_out, tmp.p, size_t(s->N + 1) * 8, cudaMemcpyDeviceToHost));
    return DISC_OK;
}

const char* disc_error_string(int code) {
    switch (code) {
        case DISC_OK: return "ok";
        case DISC_ERR_ARG: return "invalid argument";
        case DISC_ERR_EMPTY: return "empty set or empty member";
        case DISC_ERR_TOKEN: return "token id outside the vocabulary";
        case DISC_ERR_PREFIX: return "a member is a proper prefix of another member";
        case DISC_ERR_OOM: return "out of memory";
        case DISC_ERR_CUDA: return "CUDA error";
        case DISC_ERR_UNSUPPORTED: return "unsupported size or dtype";
        default: return "unknown error";
    }
}

int disc_last_cuda_error(void) { return disc::g_last_cuda_error; }

}  // extern "C"
