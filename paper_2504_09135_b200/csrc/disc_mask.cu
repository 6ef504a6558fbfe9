// disc_mask: valid-set masks of a batch of prefixes (Algorithm 2 in the M = |V| limit).
//
// Two kernels, because the two halves of the work want opposite shapes.
//   1. disc_mask_search_kernel, one THREAD per prefix.  The thread walks its prefix down the
//      index - the first token through a direct table, every further token by a binary search
//      (lower bound) among the current node's children, which are sorted by token id.  A walk is a
//      chain of a few dozen dependent loads and moves almost no bytes, so the only way to make it
//      fast is to have all of them in flight at once.  The node reached gives the member range
//      and, through its child list, the valid set (Section 2.1).  What the writer needs is parked
//      in the head of the prefix's own mask row (it is overwritten afterwards): the node, its child
//      range, which prebuilt row to copy if any, and the first child tokens themselves.
//   2. disc_mask_write_kernel, one WARP per row.  The warp reads the row head with one coalesced
//      load and writes the packed mask row with 16-byte streaming stores: a copy of the prebuilt
//      row for the empty prefix and for nodes with many children, otherwise zeros with the
//      children's bits merged in before the store (every byte of the row is written exactly once,
//      in full 16-byte pieces, so that DRAM never sees a partial write).  Rows cost different
//      amounts, so the warps draw small batches of rows from a counter.  This half is bound by
//      HBM write bandwidth.
// The counter lives in the set handle: two disc_mask calls on the same handle must not run at the
// same time on the device (calls on one stream never do).

#include <mutex>

#include "disc_internal.cuh"

namespace {

constexpr int MASK_THREADS = 128;
constexpr int MASK_WARPS = MASK_THREADS / 32;
constexpr int HEAD_WORDS = 64;                   // row head used as scratch between the kernels
constexpr int HEAD_TOKENS = HEAD_WORDS - 4;      // child tokens that fit behind the 4 control words
#ifndef DISC_MASK_BATCH
#define DISC_MASK_BATCH 2
#endif
constexpr int WRITE_BATCH = DISC_MASK_BATCH;     // rows whose heads a writer warp loads before it writes

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
    int32_t V, W, Wp, N, n_heavy;
    unsigned int* work_counter;   // rows handed out so far by the writer kernel
};

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

// HEAD: rows are at least HEAD_WORDS long, so the full head (control words + tokens) is parked;
// otherwise only the node id goes into word 0.
template <bool HEAD>
__global__ void __launch_bounds__(MASK_THREADS) disc_mask_search_kernel(const MaskParams p) {
    const int64_t i = int64_t(blockIdx.x) * MASK_THREADS + threadIdx.x;
    if (i >= p.n) return;
    if (i == 0 && p.mask_out) *p.work_counter = 0u;     // the writer kernel follows in stream order
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
    if (!p.mask_out) return;
    uint32_t* row = p.mask_out + size_t(i) * p.W;
    if (!HEAD) { row[0] = uint32_t(ok ? node : -1); return; }
    // which prebuilt row to copy: -2 none (zero fill), -1 the root's, >= 0 a heavy node's
    int32_t sel = -2;
    if (ok && node == 0) sel = -1;
    else if (ok && ce - cb > DISC_HEAVY_MIN) {
        const int32_t h = disc::heavy_index(p.heavy_nodes, p.n_heavy, node);
        if (h >= 0) sel = h;
    }
    if (!ok) { cb = 0; ce = 0; }
    row[0] = uint32_t(ok ? node : -1); row[1] = uint32_t(cb); row[2] = uint32_t(ce); row[3] = uint32_t(sel);
    if (sel == -2) {
        // child tokens into the head, twelve loads in flight at a time (a store has to wait for its
        // load, so one load per store would make this a chain as well)
        const int32_t m = min(ce - cb, HEAD_TOKENS);
        for (int32_t j0 = 0; j0 < m; j0 += 12) {
            int32_t v[12];
#pragma unroll
            for (int u = 0; u < 12; ++u) v[u] = (j0 + u < m) ? __ldg(p.node_tok + cb + j0 + u) : 0;
#pragma unroll
            for (int u = 0; u < 12; ++u)
                if (j0 + u < m) row[4 + j0 + u] = uint32_t(v[u]);
        }
    }
}

// store the finished words of a 32-child chunk; the chunk's last word is carried to the next chunk
__device__ __forceinline__ void put_chunk(uint32_t* row, int lane, int nvalid, int32_t t, uint32_t& carry_word,
                                          uint32_t& carry_val) {
    const bool have = lane < nvalid;
    const uint32_t word = have ? uint32_t(t >> 5) : 0xfffffffeu;
    const uint32_t bit = have ? (1u << (t & 31)) : 0u;
    // the children are sorted, so the tokens of one mask word sit in neighbouring lanes
    const uint32_t peers = __match_any_sync(0xffffffffu, word);
    uint32_t val = __reduce_or_sync(peers, bit);
    const uint32_t first_word = __shfl_sync(0xffffffffu, word, 0);
    if (carry_word != 0xffffffffu) {
        if (carry_word == first_word) { if (word == first_word) val |= carry_val; }
        else if (lane == 0) row[carry_word] = carry_val;
    }
    const uint32_t last_word = __shfl_sync(0xffffffffu, word, nvalid - 1);
    const uint32_t last_val = __shfl_sync(0xffffffffu, val, nvalid - 1);
    if (have && lane == (__ffs(peers) - 1) && word != last_word) row[word] = val;
    carry_word = last_word;
    carry_val = last_val;
}

template <bool VEC, bool HEAD>
__global__ void __launch_bounds__(MASK_THREADS) disc_mask_write_kernel(const MaskParams p) {
    __shared__ __align__(16) uint32_t s_patch[MASK_WARPS][128];
    const int lane = threadIdx.x & 31;

    auto load_head = [&](int64_t i, uint32_t& h0, uint32_t& h1) {
        const volatile uint32_t* row = p.mask_out + size_t(i) * p.W;
        if (HEAD) { h0 = row[lane]; h1 = row[32 + lane]; }
        else { h0 = row[0]; h1 = 0u; }
    };

    // Rows cost very different amounts (a copied row reads 16 KB, a zero-filled one reads nothing),
    // so warps draw batches of WRITE_BATCH consecutive rows from a counter instead of owning a
    // fixed share.  The heads of a batch are loaded together before its first row is written.
    const uint64_t keep = l2_policy_evict_last();
    for (;;) {
    unsigned int first = 0;
    if (lane == 0) first = atomicAdd(p.work_counter, unsigned(WRITE_BATCH));
    const int64_t base = int64_t(__shfl_sync(0xffffffffu, first, 0));
    if (base >= p.n) break;
    uint32_t hh0[WRITE_BATCH], hh1[WRITE_BATCH];
#pragma unroll
    for (int b = 0; b < WRITE_BATCH; ++b) {
        hh0[b] = 0xffffffffu; hh1[b] = 0u;
        if (base + b < p.n) load_head(base + b, hh0[b], hh1[b]);
    }
#pragma unroll
    for (int b = 0; b < WRITE_BATCH; ++b) {
        const int64_t i = base + b;
        if (i >= p.n) break;
        const uint32_t h0 = hh0[b], h1 = hh1[b];
        uint32_t* row = p.mask_out + size_t(i) * p.W;
        const int32_t node = int32_t(__shfl_sync(0xffffffffu, h0, 0));
        const bool ok = node >= 0;
        int32_t cb = 0, ce = 0, sel = -2;
        if (HEAD) {
            cb = int32_t(__shfl_sync(0xffffffffu, h0, 1));
            ce = int32_t(__shfl_sync(0xffffffffu, h0, 2));
            sel = int32_t(__shfl_sync(0xffffffffu, h0, 3));
        } else if (ok) {
            cb = __ldg(p.child_begin + node);
            ce = __ldg(p.child_begin + node + 1);
            if (node == 0) sel = -1;
            else if (ce - cb > DISC_HEAVY_MIN) {
                const int32_t h = disc::heavy_index(p.heavy_nodes, p.n_heavy, node);
                if (h >= 0) sel = h;
            }
        }
        // child tokens 0..31 and 32..63 of the row, from the head as far as it holds them
        int32_t tk0 = 0, tk1 = 0;
        if (HEAD) {
            const uint32_t a0 = __shfl_sync(0xffffffffu, h0, (lane + 4) & 31);
            const uint32_t a1 = __shfl_sync(0xffffffffu, h1, (lane + 4) & 31);
            tk0 = int32_t(lane < 28 ? a0 : a1);          // children 28..31 sit in words 32..35
            tk1 = int32_t(a1);                           // children 32..59 sit in words 36..63 (lanes 0..27)
        }
        __syncwarp();                       // every lane has what it needs from the row head

        const uint32_t* src = sel == -2 ? nullptr : (sel == -1 ? p.root_mask : p.heavy_masks + size_t(sel) * p.Wp);
        int merged = 0;                     // leading children already contained in the fill stores
        uint32_t carry_word = 0xffffffffu, carry_val = 0u;     // pending word of the store loop (warp-uniform)
        if (VEC) {
            uint4* row4 = reinterpret_cast<uint4*>(row);
            const uint4* src4 = reinterpret_cast<const uint4*>(src);
            const int n4 = p.W >> 2;
            if (src) {
                // eight 16-byte loads in flight per lane before the first store
                int w = lane;
                for (; w + 7 * 32 < n4; w += 8 * 32) {
                    uint4 v[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) v[u] = ld_keep16(src4 + w + u * 32, keep);
#pragma unroll
                    for (int u = 0; u < 8; ++u) st_stream16(row4 + w + u * 32, v[u]);
                }
                for (; w < n4; w += 32) st_stream16(row4 + w, ld_keep16(src4 + w, keep));
                for (int w2 = (n4 << 2) + lane; w2 < p.W; w2 += 32) row[w2] = __ldg(src + w2);
            } else {
                // Zero fill with the row's children merged into the 16-byte stores: a word stored
                // separately afterwards would be a partial write to a line that has already left
                // L2, i.e. a read-modify-write in DRAM in the middle of the write stream.  The
                // children are sorted by token, so the ones of a 512-byte span (4096 tokens) are
                // consecutive in the list: the warp walks the list once, 32 children at a time,
                // and spans that hold a child go through a per-warp patch buffer in shared memory.
                const uint4 z = make_uint4(0u, 0u, 0u, 0u);
                const int nc = ok ? ce - cb : 0;
                auto chunk_token = [&](int c) -> int32_t {
                    const int j = c * 32 + lane;
                    if (j >= nc) return 0x7fffffff;
                    if (HEAD && j < 32) return tk0;
                    if (HEAD && j < HEAD_TOKENS) return tk1;
                    return __ldg(p.node_tok + cb + j);
                };
                int c = 0;
                int32_t t = chunk_token(0), tn = chunk_token(1);
                uint32_t* patch = s_patch[threadIdx.x >> 5];
                for (int it = 0; it * 32 < n4; ++it) {
                    bool dirty = false;
                    for (;;) {
                        const bool in = (t >> 12) == it;
                        if (__ballot_sync(0xffffffffu, in)) {
                            if (!dirty) {
                                reinterpret_cast<uint4*>(patch)[lane] = z;
                                __syncwarp();
                                dirty = true;
                            }
                            if (in) atomicOr(&patch[(t >> 5) & 127], 1u << (t & 31));
                        }
                        // the chunk is used up once its last child lies in this span or before it
                        if ((__shfl_sync(0xffffffffu, t, 31) >> 12) > it) break;
                        ++c;
                        t = tn;
                        tn = chunk_token(c + 1);
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
        if (ok && !src && ce > cb + merged) {
            __syncwarp();   // the fill is ordered before this warp's word stores
            for (int32_t k0 = cb + merged; k0 < ce; k0 += 32) {
                const int32_t j = k0 - cb + lane;                        // child number
                int32_t t;
                if (HEAD && j < 32) t = tk0;
                else if (HEAD && j < 64 && j < HEAD_TOKENS) t = tk1;
                else t = (k0 + lane < ce) ? __ldg(p.node_tok + k0 + lane) : 0;
                put_chunk(row, lane, min(32, ce - k0), t, carry_word, carry_val);
            }
            if (carry_word != 0xffffffffu && lane == 0) row[carry_word] = carry_val;
        }
    }
    }
}

}  // namespace

extern "C" int disc_mask(const disc_set_t* s, const int32_t* prefix, int32_t prefix_ld, const int32_t* prefix_len,
                         int64_t n, uint32_t* mask_out, int32_t* lo_out, int32_t* hi_out, int32_t* node_out,
                         uint8_t* status_out, void* stream) {
    if (!s || n < 0 || prefix_ld < 0) return DISC_ERR_ARG;
    if (const int rc = disc::check_device(s)) return rc;
    if (n == 0) return DISC_OK;
    if (!prefix_len || !status_out || (prefix_ld > 0 && !prefix)) return DISC_ERR_ARG;
    if (n >= (int64_t(1) << 31) - 65536) return DISC_ERR_UNSUPPORTED;   // the row counter is 32 bits wide
    MaskParams p;
    p.prefix = prefix; p.prefix_ld = prefix_ld; p.prefix_len = prefix_len; p.n = n;
    p.mask_out = mask_out; p.lo_out = lo_out; p.hi_out = hi_out; p.node_out = node_out; p.status_out = status_out;
    p.node_tok = s->node_tok; p.node_lo = s->node_lo; p.child_begin = s->child_begin;
    p.root_child = s->root_child; p.root_mask = s->root_mask;
    p.heavy_nodes = s->heavy_nodes; p.heavy_masks = s->heavy_masks; p.n_heavy = s->n_heavy;
    p.V = s->V; p.W = s->W; p.Wp = s->Wp; p.N = int32_t(s->N);
    p.work_counter = s->work_counter;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool head = s->W >= HEAD_WORDS;
    const unsigned sgrid = unsigned((n + MASK_THREADS - 1) / MASK_THREADS);
    if (head) disc_mask_search_kernel<true><<<sgrid, MASK_THREADS, 0, st>>>(p);
    else disc_mask_search_kernel<false><<<sgrid, MASK_THREADS, 0, st>>>(p);
    DISC_CUDA(cudaGetLastError());
    if (!mask_out) return DISC_OK;

    int dev = 0, sms = 0;
    DISC_CUDA(cudaGetDevice(&dev));
    DISC_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const bool vec = (reinterpret_cast<uintptr_t>(mask_out) % 16 == 0) && (s->W % 4 == 0);
    void (*kern)(const MaskParams) = vec ? (head ? disc_mask_write_kernel<true, true> : disc_mask_write_kernel<true, false>)
                                         : (head ? disc_mask_write_kernel<false, true> : disc_mask_write_kernel<false, false>);
    // one wave of blocks: they share the rows through the counter
    int per_sm = 0;
    DISC_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, MASK_THREADS, 0));
    if (per_sm < 1) per_sm = 1;
    const int64_t want = (n + MASK_WARPS * WRITE_BATCH - 1) / (MASK_WARPS * WRITE_BATCH);
    const int64_t resident = int64_t(sms) * per_sm;
    const unsigned grid = unsigned(want < resident ? want : resident);
    kern<<<grid, MASK_THREADS, 0, st>>>(p);
    DISC_CUDA(cudaGetLastError());
    return DISC_OK;
}

// ---- disc_mask_static: the same two kernels with the writer's row counter in a word block that is
// part of this module's image instead of the allocation disc_build_set makes for the handle.
namespace {

// scratch of disc_mask_static, one copy per device: word 0 is the row counter, the rest is unused
static __device__ __align__(256) unsigned int g_mask_static_scratch[64];

constexpr int MAX_DEVICES = 64;
unsigned int* g_static_ptr[MAX_DEVICES] = {nullptr};
std::mutex g_static_mutex;

// address of the scratch block on the current device; looked up once per device
int static_counter(unsigned int** out) {
    int dev = 0;
    DISC_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return DISC_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        unsigned int* ptr = nullptr;
        DISC_CUDA(cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_mask_static_scratch));
        if (!ptr) return DISC_ERR_CUDA;
        g_static_ptr[dev] = ptr;
    }
    *out = g_static_ptr[dev];
    return DISC_OK;
}

}  // namespace

extern "C" int disc_mask_static(const disc_set_t* s, const int32_t* prefix, int32_t prefix_ld, const int32_t* prefix_len,
                                int64_t n, uint32_t* mask_out, int32_t* lo_out, int32_t* hi_out,
                                int32_t* node_out, uint8_t* status_out, void* stream) {
    if (!s || n < 0 || prefix_ld < 0) return DISC_ERR_ARG;
    if (const int rc = disc::check_device(s)) return rc;
    if (n == 0) return DISC_OK;
    if (!prefix_len || !status_out || (prefix_ld > 0 && !prefix)) return DISC_ERR_ARG;
    if (n > DISC_MASK_STATIC_MAX_ROWS) return DISC_ERR_UNSUPPORTED;   // beyond what the static counter can hand out
    unsigned int* counter = nullptr;
    if (const int rc = static_counter(&counter)) return rc;
    MaskParams p;
    p.prefix = prefix; p.prefix_ld = prefix_ld; p.prefix_len = prefix_len; p.n = n;
    p.mask_out = mask_out; p.lo_out = lo_out; p.hi_out = hi_out; p.node_out = node_out; p.status_out = status_out;
    p.node_tok = s->node_tok; p.node_lo = s->node_lo; p.child_begin = s->child_begin;
    p.root_child = s->root_child; p.root_mask = s->root_mask;
    p.heavy_nodes = s->heavy_nodes; p.heavy_masks = s->heavy_masks; p.n_heavy = s->n_heavy;
    p.V = s->V; p.W = s->W; p.Wp = s->Wp; p.N = int32_t(s->N);
    p.work_counter = counter;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool head = s->W >= HEAD_WORDS;
    const unsigned sgrid = unsigned((n + MASK_THREADS - 1) / MASK_THREADS);
    if (head) disc_mask_search_kernel<true><<<sgrid, MASK_THREADS, 0, st>>>(p);
    else disc_mask_search_kernel<false><<<sgrid, MASK_THREADS, 0, st>>>(p);
    DISC_CUDA(cudaGetLastError());
    if (!mask_out) return DISC_OK;

    int dev = 0, sms = 0;
    DISC_CUDA(cudaGetDevice(&dev));
    DISC_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const bool vec = (reinterpret_cast<uintptr_t>(mask_out) % 16 == 0) && (s->W % 4 == 0);
    void (*kern)(const MaskParams) = vec ? (head ? disc_mask_write_kernel<true, true> : disc_mask_write_kernel<true, false>)
                                         : (head ? disc_mask_write_kernel<false, true> : disc_mask_write_kernel<false, false>);
    // one wave of blocks: they share the rows through the counter
    int per_sm = 0;
    DISC_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, MASK_THREADS, 0));
    if (per_sm < 1) per_sm = 1;
    const int64_t want = (n + MASK_WARPS * WRITE_BATCH - 1) / (MASK_WARPS * WRITE_BATCH);
    const int64_t resident = int64_t(sms) * per_sm;
    const unsigned grid = unsigned(want < resident ? want : resident);
    kern<<<grid, MASK_THREADS, 0, st>>>(p);
    DISC_CUDA(cudaGetLastError());
    return DISC_OK;
}
