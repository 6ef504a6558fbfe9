// disc_mask: valid-set masks of a batch of prefixes (Algorithm 2 in the M = |V| limit).
//
// The work has two halves that want opposite shapes.  Walking a prefix down the index (the first
// token through a direct table, every further token by a search among the current node's sorted
// children) is a chain of a dozen dependent loads of scattered 32-byte sectors: it is fast only
// when thousands of walks are in flight, and it is cheapest for DRAM when nothing else is going on
// (scattered reads mixed into a write stream were measured to cost their full time on top of the
// writes, however they were overlapped).  Writing the packed mask row (Section 2.1's valid set of
// the node reached: a copy of a prebuilt row for the empty prefix and for nodes with many
// children, otherwise zeros with the children's bits merged in) is 16 KB of stores that need no
// answer, and HBM takes them fastest when the rows in flight are few and neighbours (see the
// second half of this file).
//
// Rows of at least 128 bytes that are 16-byte aligned and a multiple of 16 bytes long (the large
// vocabularies): two kernels, disc_mask_walk_kernel (every walk, one thread per prefix) and disc_mask_team_kernel
// (the rows, by teams of warps that draw row indices from one counter); they are described where
// they stand.
//
// Other rows: one kernel, one block per SM, in rounds of two phases:
//   1. every warp draws up to 32 rows from a global counter and walks their prefixes, one THREAD
//      per prefix, all walks of the GPU in flight at once.  Range, cursor and status go out; a
//      128-byte descriptor (row, node, child range, which prebuilt row to copy, the first
//      children) goes into shared memory.
//   2. after a block barrier, twelve warps write the block's rows from the descriptors with
//      16-byte streaming stores, every byte of a row exactly once and in full 16-byte pieces, so
//      that DRAM never sees a partial write.  The root's mask row sits in shared memory; a child
//      list too long for the descriptor is staged there by asynchronous copies while the previous
//      row is written; a heavy node's prebuilt row is copied from L2 (or staged likewise when the
//      staging buffer is built large enough to hold a row).
// There are no waits other than block barriers.
//
// Calls that ask for no mask (ranges, cursor and status only) run the walks alone.
//
// The global counter (two words: rows handed out, blocks finished) lives in the set handle, or for
// disc_mask_static in a word block of the module image.  The last block to finish puts both words
// back to zero, so that every call finds and leaves them zero; two calls that share a counter must
// not run at the same time on the device (calls on one stream never do).

#include <mutex>

#include "disc_internal.cuh"

namespace {

constexpr int MASK_THREADS = 128;
constexpr unsigned FULL = 0xffffffffu;

struct MaskParams {
    const int32_t* prefix;
    int32_t prefix_ld;
    const int32_t* prefix_len;
    int64_t n;
    uint32_t* mask_out;
    int32_t *lo_out, *hi_out, *node_out;
    uint8_t* status_out;
    const int32_t *node_tok, *node_lo, *child_begin, *root_child, *heavy_nodes;
    const uint32_t *root_mask, *heavy_masks;
    int32_t V, W, Wp, N, n_heavy, l_max;
    int32_t draw;                 // rows a warp draws per round (1..32)
    int32_t single_round;         // the first round hands out every row
    unsigned int* work_counter;   // [0] rows handed out so far, [1] blocks that have finished
};

// ---- one thread per prefix (calls without a mask output) ------------------------------------------
// The child with token t among the sorted children [cb, ce) of a node (one thread).  A walk is a
// chain of dependent loads, so each round probes eight evenly spaced keys at once (independent
// loads, one latency) and keeps the ninth of the range that can still hold t: a node with 80,000
// children takes 5 rounds instead of the 17 of a binary search.  The walk next needs the child's
// first member row, its next sibling's, and its own child range: those are fetched for every
// candidate of the last round together with the candidates' tokens, so that a level of the walk
// costs one memory latency instead of two.  k = -1 if t is not among the children.
struct ChildInfo {
    int32_t k, lo, lo_next, cb, ce;
};
__device__ __forceinline__ ChildInfo find_child_info(const int32_t* __restrict__ node_tok,
                                                     const int32_t* __restrict__ node_lo,
                                                     const int32_t* __restrict__ child_begin, int32_t cb, int32_t ce,
                                                     int32_t t) {
    constexpr int P = 8;
    int32_t a = cb, b = ce;                 // the first key >= t, if any, is in [a, b]
    while (b - a > P) {
        const int32_t s = (b - a + P) / (P + 1);
        int32_t key[P];
#pragma unroll
        for (int j = 0; j < P; ++j) {
            const int32_t q = a + (j + 1) * s - 1;
            key[j] = q < b ? __ldg(node_tok + q) : 0x7fffffff;
        }
        int cnt = 0;
#pragma unroll
        for (int j = 0; j < P; ++j) cnt += key[j] < t ? 1 : 0;
        const int32_t na = a + cnt * s;
        const int32_t nb = cnt < P ? min(b, a + (cnt + 1) * s - 1) : b;
        a = na;
        b = nb;
    }
    int32_t key[P + 1], nlo[P + 2], cbg[P + 2];
#pragma unroll
    for (int j = 0; j <= P; ++j) key[j] = (a + j < ce) ? __ldg(node_tok + a + j) : 0x7fffffff;
#pragma unroll
    for (int j = 0; j <= P + 1; ++j) {
        nlo[j] = (a + j < ce) ? __ldg(node_lo + a + j) : 0;
        cbg[j] = (a + j <= ce) ? __ldg(child_begin + a + j) : 0;
    }
    ChildInfo r{-1, 0, 0, 0, 0};
#pragma unroll
    for (int j = P; j >= 0; --j)
        if (a + j <= b && key[j] == t) r = ChildInfo{a + j, nlo[j], nlo[j + 1], cbg[j], cbg[j + 1]};
    return r;
}

__global__ void __launch_bounds__(MASK_THREADS) disc_mask_search_kernel(const MaskParams p) {
    const int64_t i = int64_t(blockIdx.x) * MASK_THREADS + threadIdx.x;
    if (i >= p.n) return;
    const int32_t len = p.prefix_len[i];
    const int32_t* pre = p.prefix + i * p.prefix_ld;
    bool ok = (len >= 0 && len <= p.prefix_ld);
    int32_t node = 0, lo = 0, hi = p.N, cb = 0, ce = 0;
    if (ok) { cb = __ldg(p.child_begin); ce = __ldg(p.child_begin + 1); }
    int32_t t_next = (ok && len > 0) ? pre[0] : 0;
    for (int32_t d = 0; ok && d < len; ++d) {
        const int32_t t = t_next;
        if (d + 1 < len) t_next = pre[d + 1];        // fetched while this level is searched
        if (t < 0 || t >= p.V) { ok = false; break; }
        if (node == 0) {
            const int32_t k = __ldg(p.root_child + t);
            if (k < 0) { ok = false; break; }
            lo = __ldg(p.node_lo + k);
            if (k + 1 < ce) hi = __ldg(p.node_lo + k + 1);
            node = k;
            cb = __ldg(p.child_begin + k);
            ce = __ldg(p.child_begin + k + 1);
        } else {
            const ChildInfo c = find_child_info(p.node_tok, p.node_lo, p.child_begin, cb, ce, t);
            if (c.k < 0) { ok = false; break; }
            lo = c.lo;
            if (c.k + 1 < ce) hi = c.lo_next;
            node = c.k;
            cb = c.cb;
            ce = c.ce;
        }
    }
    if (p.lo_out) p.lo_out[i] = ok ? lo : -1;
    if (p.hi_out) p.hi_out[i] = ok ? hi : -1;
    if (p.node_out) p.node_out[i] = ok ? node : -1;
    p.status_out[i] = ok ? 0 : DISC_ROW_DEAD;
}

// ---- one warp per row (calls with a mask output) ------------------------------------------------------
__device__ __forceinline__ void st_stream16(uint4* p, const uint4& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

// The prebuilt rows (a few MB) are read again and again while a gigabyte of masks streams out:
// loads of them ask L2 to keep the lines, the streaming stores above ask it to drop theirs first.
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint4 ld_keep16(const uint4* p, uint64_t pol) {
    uint4 v;
    asm volatile("ld.global.nc.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p), "l"(pol));
    return v;
}

// index of `node` among the ascending heavy nodes, by one warp in two rounds; -1 if absent
__device__ __forceinline__ int32_t warp_heavy_index(const int32_t* __restrict__ heavy, int32_t n, int32_t node, int lane) {
    int32_t a = 0, b = n;
    while (b - a > 32) {
        const int32_t stride = (b - a + 31) / 32;
        const int32_t i = a + lane * stride;
        const uint32_t bal = __ballot_sync(FULL, (i < b) && (__ldg(heavy + i) <= node));
        if (bal == 0) return -1;
        const int32_t j = 31 - __clz(bal);
        a = a + j * stride;
        b = min(a + stride, b);
    }
    const uint32_t hit = __ballot_sync(FULL, (a + lane < b) && (__ldg(heavy + a + lane) == node));
    return hit ? a + (__ffs(hit) - 1) : -1;
}

// store the finished words of a 32-child chunk; the chunk's last word is carried to the next chunk
__device__ __forceinline__ void put_chunk(uint32_t* row, int lane, int nvalid, int32_t t, uint32_t& carry_word,
                                          uint32_t& carry_val) {
    const bool have = lane < nvalid;
    const uint32_t word = have ? uint32_t(t >> 5) : 0xfffffffeu;
    const uint32_t bit = have ? (1u << (t & 31)) : 0u;
    // the children are sorted, so the tokens of one mask word sit in neighbouring lanes
    const uint32_t peers = __match_any_sync(FULL, word);
    uint32_t val = __reduce_or_sync(peers, bit);
    const uint32_t first_word = __shfl_sync(FULL, word, 0);
    if (carry_word != 0xffffffffu) {
        if (carry_word == first_word) { if (word == first_word) val |= carry_val; }
        else if (lane == 0) row[carry_word] = carry_val;
    }
    const uint32_t last_word = __shfl_sync(FULL, word, nvalid - 1);
    const uint32_t last_val = __shfl_sync(FULL, val, nvalid - 1);
    if (have && lane == (__ffs(peers) - 1) && word != last_word) row[word] = val;
    carry_word = last_word;
    carry_val = last_val;
}

// ---- the fused kernel ---------------------------------------------------------------------------------
#ifndef DISC_MASK_WRITERS
#define DISC_MASK_WRITERS 12
#endif
#ifndef DISC_MASK_WARPS
#define DISC_MASK_WARPS 16
#endif
constexpr int WRITER_WARPS = DISC_MASK_WRITERS;  // warps that write rows in phase 2
constexpr int FUSED_WARPS = DISC_MASK_WARPS;     // warps of a block; all of them walk in phase 1
constexpr int FUSED_THREADS = 32 * FUSED_WARPS;
constexpr int ROUND_ROWS = FUSED_THREADS;        // rows of a round: one per thread
constexpr int DESC_WORDS = 32;                   // one descriptor = 128 bytes, read by a writer warp in one go:
constexpr int DESC_TOKENS = DESC_WORDS - 5;      //   row (-1: none), node (-1: dead), child begin, child end,
                                                 //   prebuilt row (-2 none, -1 the root's, >= 0 a heavy node's), first children
constexpr int ROOT_SMEM_WORDS = 4096;            // the root's mask row is kept in shared memory when it fits

// One mask row written by one warp.  t0: the row's first 32 children, one per lane (0x7fffffff
// beyond the last child), valid when have_t0; otherwise the children are read from `staged` (the
// writer's buffer in shared memory, filled ahead of time) or, when that is null, from the index.
// sel: -2 no prebuilt row, -1 the root's, >= 0 a heavy node's; a heavy node's row comes from
// `staged` as well when it was put there.  s_root: the root's row in shared memory, or null.
template <bool VEC>
__device__ __forceinline__ void write_row(const MaskParams& p, int64_t i, int32_t node, int32_t cb, int32_t ce,
                                          int32_t sel, int32_t t0, bool have_t0, const uint32_t* s_root,
                                          const uint32_t* staged, uint32_t* patch, uint64_t keep, int lane) {
    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
    const int nc = ce - cb;
    const uint32_t* src = sel == -2 ? nullptr : (sel == -1 ? p.root_mask : p.heavy_masks + size_t(sel) * p.Wp);
    uint32_t* row = p.mask_out + size_t(i) * p.W;
    int merged = 0;                     // leading children already contained in the fill stores
    if (VEC) {
        uint4* row4 = reinterpret_cast<uint4*>(row);
        const int n4 = p.W >> 2;
        const int n_it = (n4 + 31) >> 5;        // 512-byte spans (4096 tokens) of the row
        if ((sel == -1 && s_root) || (sel >= 0 && staged)) {
            const uint4* src4 = reinterpret_cast<const uint4*>(sel == -1 ? s_root : staged);
            for (int w = lane; w < n4; w += 32) st_stream16(row4 + w, src4[w]);
        } else if (src) {
            // eight 16-byte loads in flight per lane before the first store
            const uint4* src4 = reinterpret_cast<const uint4*>(src);
            int w = lane;
            for (; w + 7 * 32 < n4; w += 8 * 32) {
                uint4 v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) v[u] = ld_keep16(src4 + w + u * 32, keep);
#pragma unroll
                for (int u = 0; u < 8; ++u) st_stream16(row4 + w + u * 32, v[u]);
            }
            for (; w < n4; w += 32) st_stream16(row4 + w, ld_keep16(src4 + w, keep));
        } else if (have_t0 && n_it <= 32) {
            // Zero fill with the children's bits merged into the 16-byte stores (a word stored
            // separately afterwards would be a partial write to a line that may have left L2
            // already, i.e. a read-modify-write in DRAM in the middle of the write stream).
            // The children sit one per lane; `spans` has a bit for every span that holds one.
            const bool have = lane < nc;
            const uint32_t spans = __reduce_or_sync(FULL, have ? (1u << (t0 >> 12)) : 0u);
            for (int it = 0; it < n_it; ++it) {
                uint4 v = z;
                if ((spans >> it) & 1u) {
                    uint32_t todo = __ballot_sync(FULL, have && (t0 >> 12) == it);
                    while (todo) {
                        const int cl = __ffs(todo) - 1;
                        todo &= todo - 1;
                        const int32_t tc = __shfl_sync(FULL, t0, cl);
                        if (((tc >> 7) & 31) == lane) {
                            const uint32_t bit = 1u << (tc & 31);
                            const int wsel = (tc >> 5) & 3;
                            v.x |= wsel == 0 ? bit : 0u; v.y |= wsel == 1 ? bit : 0u;
                            v.z |= wsel == 2 ? bit : 0u; v.w |= wsel == 3 ? bit : 0u;
                        }
                    }
                }
                if (it * 32 + lane < n4) st_stream16(row4 + it * 32 + lane, v);
            }
            merged = nc;
        } else {
            // More children than lanes (or a very long row): the children are sorted by token,
            // so the ones of a span are consecutive in the list; the warp walks the list once,
            // 32 children at a time, and spans that hold a child go through a per-warp patch
            // buffer in shared memory.
            auto chunk_token = [&](int ch) -> int32_t {
                const int j = ch * 32 + lane;
                if (j >= nc) return 0x7fffffff;
                return staged ? int32_t(staged[j]) : __ldg(p.node_tok + cb + j);
            };
            int ch = 0;
            int32_t t = chunk_token(0), tn = chunk_token(1);
                        for (int it = 0; it < n_it; ++it) {
                bool dirty = false;
                for (;;) {
                    const bool in = (t >> 12) == it;
                    if (__ballot_sync(FULL, in)) {
                        if (!dirty) {
                            reinterpret_cast<uint4*>(patch)[lane] = z;
                            __syncwarp();
                            dirty = true;
                        }
                        if (in) atomicOr(&patch[(t >> 5) & 127], 1u << (t & 31));
                    }
                    // the chunk is used up once its last child lies in this span or before it
                    if ((__shfl_sync(FULL, t, 31) >> 12) > it) break;
                    ++ch;
                    t = tn;
                    tn = chunk_token(ch + 1);
                }
                uint4 v = z;
                if (dirty) {
                    __syncwarp();
                    v = reinterpret_cast<const uint4*>(patch)[lane];
                    __syncwarp();
                }
                if (it * 32 + lane < n4) st_stream16(row4 + it * 32 + lane, v);
            }
            merged = nc;
        }
    } else {
        for (int w = lane; w < p.W; w += 32) row[w] = src ? __ldg(src + w) : 0u;
    }
    if (!src && nc > merged) {
        __syncwarp();   // the fill is ordered before this warp's word stores
        uint32_t carry_word = 0xffffffffu, carry_val = 0u;     // pending word of the store loop (warp-uniform)
        for (int32_t k0 = merged; k0 < nc; k0 += 32) {
            const int32_t t = (k0 + lane < nc) ? __ldg(p.node_tok + cb + k0 + lane) : 0;
            put_chunk(row, lane, min(32, nc - k0), t, carry_word, carry_val);
        }
        if (carry_word != 0xffffffffu && lane == 0) row[carry_word] = carry_val;
    }
}

// 16-byte and 4-byte asynchronous copies from global to shared memory (the writer stages the next
// row's children, or its prebuilt mask row, while it writes the current row)
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(uint32_t(__cvta_generic_to_shared(smem))), "l"(gmem)
                 : "memory");
}
__device__ __forceinline__ void cp_async4(void* smem, const void* gmem) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(uint32_t(__cvta_generic_to_shared(smem))), "l"(gmem)
                 : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;" ::: "memory");
}

#ifndef DISC_MASK_STAGE_WORDS
#define DISC_MASK_STAGE_WORDS 1024               // per writer warp: the child list of any node that has no prebuilt row
#endif
constexpr int STAGE_WORDS = DISC_MASK_STAGE_WORDS;

struct RowDesc {
    int64_t row;
    int32_t node, cb, ce, sel, t0;
    bool have_t0, staged;
};

template <bool VEC>
__global__ void __launch_bounds__(FUSED_THREADS, 1) disc_mask_kernel(const MaskParams p) {
    // dynamic shared memory: the round's descriptors, the root's mask row (when it fits), one
    // staging buffer per writer warp
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint32_t (*s_desc)[DESC_WORDS] = reinterpret_cast<uint32_t (*)[DESC_WORDS]>(smem_raw);
    uint32_t* s_root_buf = reinterpret_cast<uint32_t*>(smem_raw) + ROUND_ROWS * DESC_WORDS;
    uint32_t* s_stage = s_root_buf + ROOT_SMEM_WORDS;
    __shared__ __align__(16) uint32_t s_patch[WRITER_WARPS][128];
    __shared__ unsigned int s_next;       // next descriptor a writer warp takes
    __shared__ int s_more;                // some warp of the block drew rows this round
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t* s_root = (VEC && p.W <= ROOT_SMEM_WORDS) ? s_root_buf : nullptr;
    if (s_root) for (int w = threadIdx.x; w < p.W; w += FUSED_THREADS) s_root_buf[w] = __ldg(p.root_mask + w);
    const uint64_t keep = l2_policy_evict_last();

    for (;;) {
        if (threadIdx.x == 0) { s_next = 0u; s_more = 0; }
        __syncthreads();
        // ---- phase 1: one prefix per thread
        {
            unsigned int first = 0;
            if (lane == 0) first = atomicAdd(p.work_counter, unsigned(p.draw));
            const int64_t base = int64_t(__shfl_sync(FULL, first, 0));
            const int64_t i = base + lane;
            const bool mine = lane < p.draw && i < p.n;
            uint32_t* dsc = s_desc[threadIdx.x];
            if (!mine) dsc[0] = 0xffffffffu;
            else {
                if (lane == 0) s_more = 1;
                const int32_t len = __ldg(p.prefix_len + i);
                const int32_t* pre = p.prefix + i * p.prefix_ld;
                bool ok = (len >= 0 && len <= p.prefix_ld && len <= p.l_max);     // no member is longer than l_max
                int32_t node = 0, lo = 0, hi = p.N, cb = 0, ce = 0;
                if (ok) { cb = __ldg(p.child_begin); ce = __ldg(p.child_begin + 1); }
                int32_t t_next = (ok && len > 0) ? __ldg(pre) : 0;
                for (int32_t d = 0; ok && d < len; ++d) {
                    const int32_t t = t_next;
                    if (d + 1 < len) t_next = __ldg(pre + d + 1);        // fetched while this level is searched
                    if (t < 0 || t >= p.V) { ok = false; break; }
                    if (node == 0) {
                        const int32_t k = __ldg(p.root_child + t);
                        if (k < 0) { ok = false; break; }
                        lo = __ldg(p.node_lo + k);
                        if (k + 1 < ce) hi = __ldg(p.node_lo + k + 1);
                        node = k;
                        cb = __ldg(p.child_begin + k);
                        ce = __ldg(p.child_begin + k + 1);
                    } else {
                        const ChildInfo c = find_child_info(p.node_tok, p.node_lo, p.child_begin, cb, ce, t);
                        if (c.k < 0) { ok = false; break; }
                        lo = c.lo;
                        if (c.k + 1 < ce) hi = c.lo_next;
                        node = c.k;
                        cb = c.cb;
                        ce = c.ce;
                    }
                }
                if (p.lo_out) p.lo_out[i] = ok ? lo : -1;
                if (p.hi_out) p.hi_out[i] = ok ? hi : -1;
                if (p.node_out) p.node_out[i] = ok ? node : -1;
                p.status_out[i] = ok ? 0 : DISC_ROW_DEAD;
                // which prebuilt row to copy: -2 none (zero fill), -1 the root's, >= 0 a heavy node's
                int32_t sel = -2;
                if (!ok) { cb = 0; ce = 0; }
                else if (node == 0) sel = -1;
                else if (ce - cb > DISC_HEAVY_MIN) sel = -3;      // a heavy node: the writer looks up which
                dsc[0] = uint32_t(i); dsc[1] = uint32_t(ok ? node : -1); dsc[2] = uint32_t(cb); dsc[3] = uint32_t(ce);
                dsc[4] = uint32_t(sel);
                // the first children, nine loads in flight at a time (most nodes have one or two)
                const int32_t m = sel == -2 ? min(ce - cb, DESC_TOKENS) : 0;
                for (int32_t j0 = 0; j0 < m; j0 += 9) {
                    int32_t v[9];
#pragma unroll
                    for (int u = 0; u < 9; ++u) v[u] = (j0 + u < m) ? __ldg(p.node_tok + cb + j0 + u) : 0;
#pragma unroll
                    for (int u = 0; u < 9; ++u)
                        if (j0 + u < m) dsc[5 + j0 + u] = uint32_t(v[u]);
                }
            }
        }
        __syncthreads();
        if (!s_more) break;              // the counter is used up

        // ---- phase 2: a few warps write the block's rows
        if (warp < WRITER_WARPS) {
            uint32_t* patch = s_patch[warp];
            uint32_t* stage = s_stage + size_t(warp) * STAGE_WORDS;
            auto write = [&](const RowDesc& r) {
                if (r.staged) { cp_async_wait_all(); __syncwarp(); }
                write_row<VEC>(p, r.row, r.node, r.cb, r.ce, r.sel, r.t0, r.have_t0, s_root, r.staged ? stage : nullptr,
                               patch, keep, lane);
                if (r.staged) __syncwarp();          // every lane is done with the buffer
            };
            RowDesc cur;
            bool have_cur = false;
            for (;;) {
                unsigned int h = 0;
                if (lane == 0) h = atomicAdd(&s_next, 1u);
                const unsigned int slot = __shfl_sync(FULL, h, 0);
                if (slot >= unsigned(ROUND_ROWS)) break;
                const uint32_t word = s_desc[slot][lane];
                RowDesc nx;
                nx.row = int64_t(int32_t(__shfl_sync(FULL, word, 0)));
                if (nx.row < 0) continue;            // a thread without a row
                nx.node = int32_t(__shfl_sync(FULL, word, 1));
                nx.cb = int32_t(__shfl_sync(FULL, word, 2));
                nx.ce = int32_t(__shfl_sync(FULL, word, 3));
                nx.sel = int32_t(__shfl_sync(FULL, word, 4));
                if (nx.sel == -3) {
                    const int32_t h = warp_heavy_index(p.heavy_nodes, p.n_heavy, nx.node, lane);
                    nx.sel = h >= 0 ? h : -2;
                }
                // children 0..26 sit in words 5..31: lane l takes child l
                const int32_t tk = int32_t(__shfl_sync(FULL, word, (lane + 5) & 31));
                const int nc = nx.ce - nx.cb;
                nx.have_t0 = nc <= DESC_TOKENS;
                nx.t0 = (nx.have_t0 && lane < nc) ? tk : 0x7fffffff;
                // rows with more children, and heavy nodes' prebuilt rows, are staged in shared
                // memory while the row in hand is written
                const bool stage_children = VEC && nx.sel == -2 && !nx.have_t0 && nc <= STAGE_WORDS;
                const bool stage_mask = VEC && nx.sel >= 0 && p.W <= STAGE_WORDS;
                nx.staged = stage_children || stage_mask;
                if (nx.staged && have_cur && cur.staged) { write(cur); have_cur = false; }     // the buffer is taken
                if (stage_children) {
                    for (int j = lane; j < nc; j += 32) cp_async4(stage + j, p.node_tok + nx.cb + j);
                } else if (stage_mask) {
                    const uint4* src4 = reinterpret_cast<const uint4*>(p.heavy_masks + size_t(nx.sel) * p.Wp);
                    for (int w = lane; w < (p.W >> 2); w += 32) cp_async16(reinterpret_cast<uint4*>(stage) + w, src4 + w);
                }
                if (have_cur) write(cur);
                cur = nx;
                have_cur = true;
            }
            if (have_cur) write(cur);
        }
        if (p.single_round) break;
        __syncthreads();                 // the descriptors are free for the next round
    }

    // The last block to get here has seen every other block stop drawing: it puts the counter back
    // to zero for the next call.
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(p.work_counter + 1, 1u) == gridDim.x - 1) {
            p.work_counter[0] = 0u;
            p.work_counter[1] = 0u;
            __threadfence();
        }
    }
}


// ---- two kernels: every walk first, then the rows in the order of their indices ------------------------
// HBM takes a stream of 16 KB rows fastest when the rows being written at any moment are neighbours
// and few: on B200, rows of zeros drawn one by one from a global counter reach 7.2-7.3 TB/s with four
// to six rows in flight per SM (600-900 on the GPU), 4.5 TB/s with eight or more, and 6.1 TB/s when
// every SM works through a share of its own, whatever the order inside it.  So the rows are written
// by TEAMS of warps (a row's 512-byte spans dealt out among the team's warps: enough warps to
// generate the rows, few rows in flight), every team drawing the next row index from one counter.
// That needs every prefix's walk done before the first row is written, so the walks are a kernel
// of their own (one thread per prefix, all of them in flight at once while DRAM has nothing else to
// do), which parks what the writer needs - node, child range, which prebuilt row to copy, the
// first 27 children - in the first 128 bytes of the prefix's own mask row, to be read back by the
// team (from L2) before it overwrites them.  Rows shorter than that, and rows that are not 16-byte
// aligned, take the one-kernel path above.
#ifndef DISC_MASK_TEAM
#define DISC_MASK_TEAM 4
#endif
#ifndef DISC_MASK_TEAMS
#define DISC_MASK_TEAMS 6
#endif
constexpr int TEAM = DISC_MASK_TEAM;             // warps that write one row together
constexpr int TEAMS = DISC_MASK_TEAMS;           // rows in flight per SM
constexpr int TEAM_THREADS = 32 * TEAM * TEAMS;
static_assert(TEAMS <= 15, "one named barrier per team");
constexpr int WALK_THREADS = 256;

__global__ void __launch_bounds__(WALK_THREADS) disc_mask_walk_kernel(const MaskParams p) {
    // The team kernel is launched with programmatic stream serialisation: its blocks may be placed
    // (and load the root's row, and draw their first rows) on SMs that this kernel's blocks have
    // left; it reads no descriptor before this kernel has completed.
    asm volatile("griddepcontrol.launch_dependents;");
    const int64_t i = int64_t(blockIdx.x) * WALK_THREADS + threadIdx.x;
    if (i >= p.n) return;
    const int32_t len = __ldg(p.prefix_len + i);
    const int32_t* pre = p.prefix + i * p.prefix_ld;
    bool ok = (len >= 0 && len <= p.prefix_ld && len <= p.l_max);     // no member is longer than l_max
    int32_t node = 0, lo = 0, hi = p.N, cb = 0, ce = 0;
    if (ok) { cb = __ldg(p.child_begin); ce = __ldg(p.child_begin + 1); }
    int32_t t_next = (ok && len > 0) ? __ldg(pre) : 0;
    for (int32_t d = 0; ok && d < len; ++d) {
        const int32_t t = t_next;
        if (d + 1 < len) t_next = __ldg(pre + d + 1);        // fetched while this level is searched
        if (t < 0 || t >= p.V) { ok = false; break; }
        if (node == 0) {
            const int32_t k = __ldg(p.root_child + t);
            if (k < 0) { ok = false; break; }
            lo = __ldg(p.node_lo + k);
            if (k + 1 < ce) hi = __ldg(p.node_lo + k + 1);
            node = k;
            cb = __ldg(p.child_begin + k);
            ce = __ldg(p.child_begin + k + 1);
        } else {
            const ChildInfo c = find_child_info(p.node_tok, p.node_lo, p.child_begin, cb, ce, t);
            if (c.k < 0) { ok = false; break; }
            lo = c.lo;
            if (c.k + 1 < ce) hi = c.lo_next;
            node = c.k;
            cb = c.cb;
            ce = c.ce;
        }
    }
    if (p.lo_out) p.lo_out[i] = ok ? lo : -1;
    if (p.hi_out) p.hi_out[i] = ok ? hi : -1;
    if (p.node_out) p.node_out[i] = ok ? node : -1;
    p.status_out[i] = ok ? 0 : DISC_ROW_DEAD;
    // the descriptor: node (-1: dead), child range, prebuilt row (-2 none, -1 the root's, -3 a heavy
    // node's: the writer looks up which), a spare word, the first DESC_TOKENS children
    uint32_t dsc[DESC_WORDS];
    int32_t sel = -2;
    if (!ok) { cb = 0; ce = 0; }
    else if (node == 0) sel = -1;
    else if (ce - cb > DISC_HEAVY_MIN) sel = -3;
    dsc[0] = uint32_t(ok ? node : -1); dsc[1] = uint32_t(cb); dsc[2] = uint32_t(ce); dsc[3] = uint32_t(sel); dsc[4] = 0u;
    const int32_t m = sel == -2 ? min(ce - cb, DESC_TOKENS) : 0;
#pragma unroll
    for (int j0 = 0; j0 < DESC_TOKENS; j0 += 9) {
#pragma unroll
        for (int u = 0; u < 9; ++u) dsc[5 + j0 + u] = (j0 + u < m) ? uint32_t(__ldg(p.node_tok + cb + j0 + u)) : 0u;
    }
    // parked with the request that L2 keep the lines: they are read back while a gigabyte of mask
    // rows streams through L2 (stored "evict first"), and a descriptor that had to come back from
    // DRAM would be a read in the middle of the write stream
    uint4* head = reinterpret_cast<uint4*>(p.mask_out + size_t(i) * p.W);
    const uint64_t keep = l2_policy_evict_last();
#pragma unroll
    for (int q = 0; q < DESC_WORDS / 4; ++q) {
        asm volatile("st.global.L2::cache_hint.v4.u32 [%0], {%1,%2,%3,%4}, %5;" ::"l"(head + q), "r"(dsc[4 * q]), "r"(dsc[4 * q + 1]),
                     "r"(dsc[4 * q + 2]), "r"(dsc[4 * q + 3]), "l"(keep)
                     : "memory");
    }
}

__device__ __forceinline__ void team_barrier(int team) {
    asm volatile("bar.sync %0, %1;" ::"r"(team + 1), "r"(TEAM * 32) : "memory");
}

// What a team knows of a row from its parked descriptor (the same in every lane of every warp).
struct TeamRow {
    int32_t node, cb, ce, sel;     // sel: -2 no prebuilt row, -1 the root's, -3 a heavy node's
    int32_t tk;                    // lane l: child l of the row (l < DESC_TOKENS)
    int kind;                      // 0: written straight from the descriptor (or the root's row), 1: a heavy
                                   // node's prebuilt row, 2: more children than the descriptor holds
};
__device__ __forceinline__ TeamRow team_row(uint32_t word, int lane) {
    TeamRow r;
    r.node = int32_t(__shfl_sync(FULL, word, 0));
    r.cb = int32_t(__shfl_sync(FULL, word, 1));
    r.ce = int32_t(__shfl_sync(FULL, word, 2));
    r.sel = int32_t(__shfl_sync(FULL, word, 3));
    r.tk = int32_t(__shfl_sync(FULL, word, (lane + 5) & 31));
    r.kind = r.sel == -3 ? 1 : ((r.sel == -2 && r.node >= 0 && r.ce - r.cb > DESC_TOKENS) ? 2 : 0);
    return r;
}

// Rows of kind 1 and 2 are put together in the team's buffer in shared memory (bm: a whole mask
// row; ts: up to DISC_HEAVY_MIN child tokens) and streamed out from there.  prepare_row starts that
// a row ahead: asynchronous copies of the prebuilt row, or of the child list (and the buffer is
// zeroed for the bits to come).  Warp h of the team, thread tt of its TEAM*32.
__device__ __forceinline__ void prepare_row(const MaskParams& p, const TeamRow& r, uint32_t* bm, uint32_t* ts, int h, int lane) {
    const int n4 = p.W >> 2;
    const int tt = h * 32 + lane;
    if (r.kind == 1) {
        const int32_t hv = warp_heavy_index(p.heavy_nodes, p.n_heavy, r.node, lane);
        if (hv >= 0) {
            const uint4* src4 = reinterpret_cast<const uint4*>(p.heavy_masks + size_t(hv) * p.Wp);
            for (int w = tt; w < n4; w += TEAM * 32) cp_async16(reinterpret_cast<uint4*>(bm) + w, src4 + w);
        } else {                         // cannot happen for a consistent set: an empty row
            for (int w = tt; w < n4; w += TEAM * 32) reinterpret_cast<uint4*>(bm)[w] = make_uint4(0u, 0u, 0u, 0u);
        }
    } else {
        const int nc = r.ce - r.cb;
        for (int j = tt; j < nc; j += TEAM * 32) cp_async4(ts + j, p.node_tok + r.cb + j);
        for (int w = tt; w < n4; w += TEAM * 32) reinterpret_cast<uint4*>(bm)[w] = make_uint4(0u, 0u, 0u, 0u);
    }
}

// The share of warp h of a team in one mask row: the spans it with it % TEAM == h (a span = 32
// 16-byte vectors = 4,096 tokens).  bm/ts: the team's buffers (null when a row does not fit them:
// rows of kind 1 and 2 are then generated span by span from global memory); prepared: prepare_row
// has run for this row.  Every warp of the team takes the same path (it contains team barriers).
__device__ __forceinline__ void write_row_team(const MaskParams& p, int64_t i, const TeamRow& r, int team, int h,
                                               const uint32_t* s_root, uint32_t* bm, uint32_t* ts, bool prepared,
                                               uint32_t* patch, uint64_t keep, int lane) {
    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
    const int nc = r.ce - r.cb;
    uint4* row4 = reinterpret_cast<uint4*>(p.mask_out + size_t(i) * p.W);
    const int n4 = p.W >> 2;
    const int n_it = (n4 + 31) >> 5;
    if (r.kind != 0 && bm) {
        if (!prepared) prepare_row(p, r, bm, ts, h, lane);
        cp_async_wait_all();
        team_barrier(team);                          // the copies and the zeros of all four warps are in place
        if (r.kind == 2) {
            for (int j = h * 32 + lane; j < nc; j += TEAM * 32) {
                const uint32_t t = ts[j];
                atomicOr(&bm[t >> 5], 1u << (t & 31));
            }
            team_barrier(team);
        }
        const uint4* src4 = reinterpret_cast<const uint4*>(bm);
        for (int w = h * 32 + lane; w < n4; w += TEAM * 32) st_stream16(row4 + w, src4[w]);
        return;
    }
    int32_t sel = r.sel;
    if (sel == -3) {
        const int32_t hv = warp_heavy_index(p.heavy_nodes, p.n_heavy, r.node, lane);
        sel = hv >= 0 ? hv : -2;
    }
    if (sel == -1 && s_root) {
        const uint4* src4 = reinterpret_cast<const uint4*>(s_root);
        for (int w = h * 32 + lane; w < n4; w += TEAM * 32) st_stream16(row4 + w, src4[w]);
    } else if (sel != -2) {
        // a prebuilt row from L2, up to eight 16-byte loads in flight per lane before the first store
        const uint4* src4 = reinterpret_cast<const uint4*>(sel == -1 ? p.root_mask : p.heavy_masks + size_t(sel) * p.Wp);
        int w = h * 32 + lane;
        for (; w + 7 * TEAM * 32 < n4; w += 8 * TEAM * 32) {
            uint4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = ld_keep16(src4 + w + u * TEAM * 32, keep);
#pragma unroll
            for (int u = 0; u < 8; ++u) st_stream16(row4 + w + u * TEAM * 32, v[u]);
        }
        for (; w < n4; w += TEAM * 32) st_stream16(row4 + w, ld_keep16(src4 + w, keep));
    } else if (r.node < 0 || nc <= DESC_TOKENS) {
        // zeros with the children's bits merged into the 16-byte stores; the children sit one per
        // lane (a dead row has none)
        const bool have = r.node >= 0 && lane < nc;
        const int32_t t0 = have ? r.tk : 0;
        // `spans` has a bit for every span that holds a child (rows of up to 32 spans; longer rows
        // look at every span)
        const uint32_t spans = n_it <= 32 ? __reduce_or_sync(FULL, have ? (1u << (t0 >> 12)) : 0u) : 0xffffffffu;
        for (int it = h; it < n_it; it += TEAM) {
            uint4 v = z;
            if (n_it > 32 || ((spans >> it) & 1u)) {
                uint32_t todo = __ballot_sync(FULL, have && (t0 >> 12) == it);
                while (todo) {
                    const int cl = __ffs(todo) - 1;
                    todo &= todo - 1;
                    const int32_t tc = __shfl_sync(FULL, t0, cl);
                    if (((tc >> 7) & 31) == lane) {
                        const uint32_t bit = 1u << (tc & 31);
                        const int wsel = (tc >> 5) & 3;
                        v.x |= wsel == 0 ? bit : 0u; v.y |= wsel == 1 ? bit : 0u;
                        v.z |= wsel == 2 ? bit : 0u; v.w |= wsel == 3 ? bit : 0u;
                    }
                }
            }
            if (it * 32 + lane < n4) st_stream16(row4 + it * 32 + lane, v);
        }
    } else {
        // More children than the descriptor holds and no buffer: the children are sorted by token,
        // so the ones of a span are consecutive in the list; the warp walks the list once, 32
        // children at a time, and its own spans that hold a child go through its patch buffer.
        auto chunk_token = [&](int ch) -> int32_t {
            const int j = ch * 32 + lane;
            return j < nc ? __ldg(p.node_tok + r.cb + j) : 0x7fffffff;
        };
        int ch = 0;
        int32_t t = chunk_token(0), tn = chunk_token(1);
        for (int it = 0; it < n_it; ++it) {
            const bool mine = (it % TEAM) == h;
            bool dirty = false;
            for (;;) {
                const bool in = (t >> 12) == it;
                if (mine && __ballot_sync(FULL, in)) {
                    if (!dirty) {
                        reinterpret_cast<uint4*>(patch)[lane] = z;
                        __syncwarp();
                        dirty = true;
                    }
                    if (in) atomicOr(&patch[(t >> 5) & 127], 1u << (t & 31));
                }
                // the chunk is used up once its last child lies in this span or before it
                if ((__shfl_sync(FULL, t, 31) >> 12) > it) break;
                ++ch;
                t = tn;
                tn = chunk_token(ch + 1);
            }
            if (mine) {
                uint4 v = z;
                if (dirty) {
                    __syncwarp();
                    v = reinterpret_cast<const uint4*>(patch)[lane];
                    __syncwarp();
                }
                if (it * 32 + lane < n4) st_stream16(row4 + it * 32 + lane, v);
            }
        }
    }
}

// dynamic shared memory of the team kernel: the root's mask row, then per team a buffer for a whole
// mask row and one for a child list, then a patch buffer per warp
constexpr size_t TEAM_SMEM = size_t(ROOT_SMEM_WORDS + TEAMS * (ROOT_SMEM_WORDS + DISC_HEAVY_MIN) + TEAM * TEAMS * 128) * 4;

__global__ void __launch_bounds__(TEAM_THREADS, 1) disc_mask_team_kernel(const MaskParams p) {
    extern __shared__ __align__(16) unsigned char team_smem[];
    uint32_t* s_root_buf = reinterpret_cast<uint32_t*>(team_smem);
    __shared__ unsigned int s_slot[TEAMS][2];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int team = warp / TEAM, h = warp % TEAM;
    const bool fits = p.W <= ROOT_SMEM_WORDS;           // a mask row fits the buffers
    const uint32_t* s_root = fits ? s_root_buf : nullptr;
    uint32_t* bm = fits ? s_root_buf + ROOT_SMEM_WORDS + size_t(team) * (ROOT_SMEM_WORDS + DISC_HEAVY_MIN) : nullptr;
    uint32_t* ts = fits ? bm + ROOT_SMEM_WORDS : nullptr;
    uint32_t* patch = s_root_buf + ROOT_SMEM_WORDS + size_t(TEAMS) * (ROOT_SMEM_WORDS + DISC_HEAVY_MIN) + size_t(warp) * 128;
    if (s_root) for (int w = threadIdx.x; w < p.W; w += TEAM_THREADS) s_root_buf[w] = __ldg(p.root_mask + w);
    __syncthreads();
    const uint64_t keep = l2_policy_evict_last();
    const bool leader = h == 0 && lane == 0;
    const unsigned int n = unsigned(p.n);               // n < 2^31 - 2^20, so draws past the end do not wrap

    // The lane's word of a row's descriptor (read through L2: the walk kernel wrote it).
    auto load_desc = [&](unsigned int i) -> uint32_t {
        return i < n ? __ldcg(p.mask_out + size_t(i) * p.W + lane) : 0u;
    };
    // A team works three rows deep: the row in hand, the next one (its descriptor on the way), and
    // the one after it (its index on the way back from the counter), so that neither the counter's
    // nor L2's latency is waited for.
    unsigned int pend = 0u;
    if (leader) {
        s_slot[team][0] = atomicAdd(p.work_counter, 1u);
        s_slot[team][1] = atomicAdd(p.work_counter, 1u);
        pend = atomicAdd(p.work_counter, 1u);
    }
    team_barrier(team);
    unsigned int i_cur = s_slot[team][0], i_next = s_slot[team][1];
    team_barrier(team);                                  // the slots are free again
    asm volatile("griddepcontrol.wait;" ::: "memory");   // the walks are done: their descriptors can be read
    uint32_t d_cur = load_desc(i_cur), d_next = load_desc(i_next);
    int par = 0;
    bool cur_prepared = false;
    while (i_cur < n) {
        if (leader) {
            s_slot[team][par] = pend;
            pend = atomicAdd(p.work_counter, 1u);
        }
        // After this barrier every warp of the team holds the descriptor of the row in hand (its
        // load was issued two barriers ago), so the warp that owns the row's first span may
        // overwrite the place it was parked in; and every warp is done with the row before, so
        // the team's buffers are free.
        team_barrier(team);
        const unsigned int i_nn = s_slot[team][par];
        par ^= 1;
        const uint32_t d_nn = load_desc(i_nn);
        const TeamRow rc = team_row(d_cur, lane);
        // the next row's prebuilt mask or child list starts its way into the buffers now, if the
        // row in hand does not need them
        bool next_prepared = false;
        if (bm && rc.kind == 0 && i_next < n) {
            const TeamRow rn = team_row(d_next, lane);
            if (rn.kind != 0) {
                prepare_row(p, rn, bm, ts, h, lane);
                next_prepared = true;
            }
        }
        write_row_team(p, int64_t(i_cur), rc, team, h, s_root, bm, ts, cur_prepared, patch, keep, lane);
        i_cur = i_next; d_cur = d_next; cur_prepared = next_prepared;
        i_next = i_nn; d_next = d_nn;
    }
    // The last block to get here has seen every other block stop drawing: it puts the counter back
    // to zero for the next call.
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(p.work_counter + 1, 1u) == gridDim.x - 1) {
            p.work_counter[0] = 0u;
            p.work_counter[1] = 0u;
            __threadfence();
        }
    }
}

// ---- host side ------------------------------------------------------------------------------------
constexpr int MAX_DEVICES = 64;
std::mutex g_mutex;

static_assert((ROOT_SMEM_WORDS * 4) % 16 == 0 && (STAGE_WORDS * 4) % 16 == 0,
              "the pieces of the dynamic shared memory stay 16-byte aligned");
constexpr size_t FUSED_SMEM = size_t(ROUND_ROWS * DESC_WORDS + ROOT_SMEM_WORDS + WRITER_WARPS * STAGE_WORDS) * 4;

// blocks of the fused kernel that are resident at once, per device (SM count x blocks per SM), looked up once
int g_resident[MAX_DEVICES] = {0};

int resident_blocks(int* out) {
    int dev = 0;
    DISC_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return DISC_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_resident[dev]) {
        int sms = 0, per_sm = 0;
        DISC_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        DISC_CUDA(cudaFuncSetAttribute(disc_mask_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(FUSED_SMEM)));
        DISC_CUDA(cudaFuncSetAttribute(disc_mask_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(FUSED_SMEM)));
        DISC_CUDA(cudaFuncSetAttribute(disc_mask_team_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(TEAM_SMEM)));
        DISC_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, disc_mask_kernel<true>, FUSED_THREADS, FUSED_SMEM));
        if (per_sm > 1) per_sm = 1;          // one block per SM on purpose: few writing warps, phases aligned
        g_resident[dev] = sms * (per_sm < 1 ? 1 : per_sm);
    }
    *out = g_resident[dev];
    return DISC_OK;
}

// Argument checks and launches shared by disc_mask and disc_mask_static; `counter` is the two-word
// row counter the mask kernel draws from (zero before and after every call).
int launch_mask(const disc_set_t* s, const int32_t* prefix, int32_t prefix_ld, const int32_t* prefix_len, int64_t n,
                uint32_t* mask_out, int32_t* lo_out, int32_t* hi_out, int32_t* node_out, uint8_t* status_out,
                unsigned int* counter, cudaStream_t st) {
    MaskParams p;
    p.prefix = prefix; p.prefix_ld = prefix_ld; p.prefix_len = prefix_len; p.n = n;
    p.mask_out = mask_out; p.lo_out = lo_out; p.hi_out = hi_out; p.node_out = node_out; p.status_out = status_out;
    p.node_tok = s->node_tok; p.node_lo = s->node_lo; p.child_begin = s->child_begin;
    p.root_child = s->root_child; p.root_mask = s->root_mask;
    p.heavy_nodes = s->heavy_nodes; p.heavy_masks = s->heavy_masks; p.n_heavy = s->n_heavy;
    p.V = s->V; p.W = s->W; p.Wp = s->Wp; p.N = int32_t(s->N); p.l_max = s->l_max;
    p.work_counter = counter;
    p.draw = 1;
    p.single_round = 0;

    if (!mask_out) {
        disc_mask_search_kernel<<<unsigned((n + MASK_THREADS - 1) / MASK_THREADS), MASK_THREADS, 0, st>>>(p);
        DISC_CUDA(cudaGetLastError());
        return DISC_OK;
    }
    const bool vec = (reinterpret_cast<uintptr_t>(mask_out) % 16 == 0) && (s->W % 4 == 0);
    int resident = 0;
    if (const int rc = resident_blocks(&resident)) return rc;
    if (vec && s->W >= DESC_WORDS) {
        // walks, then the rows by teams of warps, one persistent block per SM
        disc_mask_walk_kernel<<<unsigned((n + WALK_THREADS - 1) / WALK_THREADS), WALK_THREADS, 0, st>>>(p);
        DISC_CUDA(cudaGetLastError());
        const int64_t want_blocks = (n + TEAMS - 1) / TEAMS;
        const unsigned tgrid = unsigned(want_blocks < resident ? want_blocks : resident);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(tgrid); cfg.blockDim = dim3(TEAM_THREADS); cfg.dynamicSmemBytes = TEAM_SMEM; cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        DISC_CUDA(cudaLaunchKernelEx(&cfg, disc_mask_team_kernel, p));
        return DISC_OK;
    }
    // One wave of blocks.  Every warp draws `draw` rows per round: as many as it takes to hand out
    // all rows in one round when they fit (then every block gets the same share), else 32.
    const int64_t warps = int64_t(resident) * FUSED_WARPS;
    int64_t draw = (n + warps - 1) / warps;
    draw = draw < 1 ? 1 : (draw > 32 ? 32 : draw);
    p.draw = int32_t(draw);
    p.single_round = (warps * draw >= n) ? 1 : 0;
    const int64_t want = ((n + draw - 1) / draw + FUSED_WARPS - 1) / FUSED_WARPS;
    const unsigned grid = unsigned(want < resident ? want : resident);
    if (vec) disc_mask_kernel<true><<<grid, FUSED_THREADS, FUSED_SMEM, st>>>(p);
    else disc_mask_kernel<false><<<grid, FUSED_THREADS, FUSED_SMEM, st>>>(p);
    DISC_CUDA(cudaGetLastError());
    return DISC_OK;
}

// scratch of disc_mask_static, one copy per device: words 0 and 1 are the row counter, the rest is unused
static __device__ __align__(256) unsigned int g_mask_static_scratch[64];

unsigned int* g_static_ptr[MAX_DEVICES] = {nullptr};

// address of the scratch block on the current device; looked up once per device and kept for the
// life of the process (it does not survive a cudaDeviceReset)
int static_counter(unsigned int** out) {
    int dev = 0;
    DISC_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return DISC_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_static_ptr[dev]) {
        unsigned int* ptr = nullptr;
        DISC_CUDA(cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_mask_static_scratch));
        if (!ptr) return DISC_ERR_CUDA;
        g_static_ptr[dev] = ptr;
    }
    *out = g_static_ptr[dev];
    return DISC_OK;
}

int check_mask_args(const disc_set_t* s, const int32_t* prefix, int32_t prefix_ld, const int32_t* prefix_len,
                    int64_t n, const uint8_t* status_out) {
    if (!s || n < 0 || prefix_ld < 0) return DISC_ERR_ARG;
    if (const int rc = disc::check_device(s)) return rc;
    if (n == 0) return DISC_OK;
    if (!prefix_len || !status_out || (prefix_ld > 0 && !prefix)) return DISC_ERR_ARG;
    return DISC_OK;
}

}  // namespace

extern "C" int disc_mask(const disc_set_t* s, const int32_t* prefix, int32_t prefix_ld, const int32_t* prefix_len,
                         int64_t n, uint32_t* mask_out, int32_t* lo_out, int32_t* hi_out, int32_t* node_out,
                         uint8_t* status_out, void* stream) {
    if (const int rc = check_mask_args(s, prefix, prefix_ld, prefix_len, n, status_out)) return rc;
    if (n == 0) return DISC_OK;
    if (n >= (int64_t(1) << 31) - (1 << 20)) return DISC_ERR_UNSUPPORTED;   // the row counter is 32 bits wide
    return launch_mask(s, prefix, prefix_ld, prefix_len, n, mask_out, lo_out, hi_out, node_out, status_out,
                       s->work_counter, static_cast<cudaStream_t>(stream));
}

// disc_mask_static: the same kernels with the row counter in a word block that is part of this
// module's image instead of the allocation disc_build_set makes for the handle.
extern "C" int disc_mask_static(const disc_set_t* s, const int32_t* prefix, int32_t prefix_ld, const int32_t* prefix_len,
                                int64_t n, uint32_t* mask_out, int32_t* lo_out, int32_t* hi_out,
                                int32_t* node_out, uint8_t* status_out, void* stream) {
    if (const int rc = check_mask_args(s, prefix, prefix_ld, prefix_len, n, status_out)) return rc;
    if (n == 0) return DISC_OK;
    if (n > DISC_MASK_STATIC_MAX_ROWS) return DISC_ERR_UNSUPPORTED;   // beyond what the static counter can hand out
    unsigned int* counter = nullptr;
    if (const int rc = static_counter(&counter)) return rc;
    return launch_mask(s, prefix, prefix_ld, prefix_len, n, mask_out, lo_out, hi_out, node_out, status_out, counter,
                       static_cast<cudaStream_t>(stream));
}
