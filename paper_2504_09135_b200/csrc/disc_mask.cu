// disc_mask: valid-set masks of a batch of prefixes (Algorithm 2 in the M = |V| limit).
//
// One warp per prefix.  The warp walks the prefix down the index: the first token goes through a
// direct table, every further token is located among the current node's sorted children by
// warp-cooperative range narrowing (32 probes per round).  The node's children are the valid set
// (Section 2.1).  The warp then writes the packed mask row with 16-byte stores: a copy of the
// prebuilt row for the empty prefix and for nodes with many children, otherwise a zero fill
// followed by the few set words.

#include "disc_internal.cuh"

namespace {

constexpr int MASK_THREADS = 128;
constexpr int MASK_WARPS = MASK_THREADS / 32;

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
};

__device__ __forceinline__ int32_t find_child(const int32_t* __restrict__ node_tok, int32_t cb, int32_t ce, int32_t t,
                                              int lane) {
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

__device__ __forceinline__ void st_stream16(uint4* p, const uint4& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

template <bool VEC>
__global__ void __launch_bounds__(MASK_THREADS) disc_mask_kernel(const MaskParams p) {
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = int64_t(blockIdx.x) * MASK_WARPS + (threadIdx.x >> 5);
    const int64_t nwarps = int64_t(gridDim.x) * MASK_WARPS;

    for (int64_t i = warp0; i < p.n; i += nwarps) {
        const int32_t len = p.prefix_len[i];
        const int32_t* pre = p.prefix + i * p.prefix_ld;
        int32_t node = 0, lo = 0, hi = p.N;
        bool ok = (len >= 0 && len <= p.prefix_ld);
        int32_t cb = 0, ce = 0;
        if (ok) { cb = __ldg(p.child_begin); ce = __ldg(p.child_begin + 1); }
        for (int32_t d = 0; ok && d < len; ++d) {
            const int32_t t = pre[d];
            int32_t k = -1;
            if (t >= 0 && t < p.V) {
                k = (node == 0) ? __ldg(p.root_child + t) : find_child(p.node_tok, cb, ce, t, lane);
            }
            if (k < 0) { ok = false; break; }
            lo = __ldg(p.node_lo + k);
            if (k + 1 < ce) hi = __ldg(p.node_lo + k + 1);
            node = k;
            cb = __ldg(p.child_begin + k);
            ce = __ldg(p.child_begin + k + 1);
        }
        if (lane == 0) {
            if (p.lo_out) p.lo_out[i] = ok ? lo : -1;
            if (p.hi_out) p.hi_out[i] = ok ? hi : -1;
            if (p.node_out) p.node_out[i] = ok ? node : -1;
            p.status_out[i] = ok ? 0 : DISC_ROW_DEAD;
        }
        if (!p.mask_out) continue;

        // source row: prebuilt (root or heavy node) or zeros
        const uint32_t* src = nullptr;
        if (ok && node == 0) src = p.root_mask;
        else if (ok && ce - cb > DISC_HEAVY_MIN) {
            const int32_t h = disc::heavy_index(p.heavy_nodes, p.n_heavy, node);
            if (h >= 0) src = p.heavy_masks + size_t(h) * p.Wp;
        }
        uint32_t* row = p.mask_out + size_t(i) * p.W;
        if (VEC) {
            uint4* row4 = reinterpret_cast<uint4*>(row);
            const uint4* src4 = reinterpret_cast<const uint4*>(src);
            const int n4 = p.W >> 2;
            if (src) {
                for (int w = lane; w < n4; w += 32) st_stream16(row4 + w, __ldg(src4 + w));
                for (int w = (n4 << 2) + lane; w < p.W; w += 32) row[w] = __ldg(src + w);
            } else {
                const uint4 z = make_uint4(0u, 0u, 0u, 0u);
                for (int w = lane; w < n4; w += 32) row4[w] = z;
                for (int w = (n4 << 2) + lane; w < p.W; w += 32) row[w] = 0u;
            }
        } else {
            for (int w = lane; w < p.W; w += 32) row[w] = src ? __ldg(src + w) : 0u;
        }
        if (!ok || src) continue;
        __syncwarp();   // the zero fill is ordered before this warp's bit updates
        for (int32_t j = cb + lane; j < ((ce - cb + 31) / 32) * 32 + cb; j += 32) {
            const bool have = j < ce;
            const int32_t t = have ? __ldg(p.node_tok + j) : -1;
            const uint32_t word = have ? uint32_t(t >> 5) : 0xffffffffu;
            const uint32_t bit = have ? (1u << (t & 31)) : 0u;
            // children are sorted, so equal words sit in neighbouring lanes: combine them
            const uint32_t peers = __match_any_sync(0xffffffffu, word);
            const uint32_t val = __reduce_or_sync(peers, bit);
            if (have && lane == (__ffs(peers) - 1)) atomicOr(row + word, val);
        }
    }
}

}  // namespace

extern "C" int disc_mask(const disc_set_t* s, const int32_t* prefix, int32_t prefix_ld, const int32_t* prefix_len,
                         int64_t n, uint32_t* mask_out, int32_t* lo_out, int32_t* hi_out, int32_t* node_out,
                         uint8_t* status_out, void* stream) {
    if (!s || n < 0 || prefix_ld < 0) return DISC_ERR_ARG;
    if (n == 0) return DISC_OK;
    if (!prefix_len || !status_out || (prefix_ld > 0 && !prefix)) return DISC_ERR_ARG;
    MaskParams p;
    p.prefix = prefix; p.prefix_ld = prefix_ld; p.prefix_len = prefix_len; p.n = n;
    p.mask_out = mask_out; p.lo_out = lo_out; p.hi_out = hi_out; p.node_out = node_out; p.status_out = status_out;
    p.node_tok = s->node_tok; p.node_lo = s->node_lo; p.child_begin = s->child_begin;
    p.root_child = s->root_child; p.root_mask = s->root_mask;
    p.heavy_nodes = s->heavy_nodes; p.heavy_masks = s->heavy_masks; p.n_heavy = s->n_heavy;
    p.V = s->V; p.W = s->W; p.Wp = s->Wp; p.N = int32_t(s->N);

    int dev = 0, sms = 0;
    DISC_CUDA(cudaGetDevice(&dev));
    DISC_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const int64_t want = (n + MASK_WARPS - 1) / MASK_WARPS;
    const int64_t resident = int64_t(sms) * (2048 / MASK_THREADS);
    const unsigned grid = unsigned(want < resident ? want : resident);
    const bool vec = mask_out && (reinterpret_cast<uintptr_t>(mask_out) % 16 == 0) && (s->W % 4 == 0);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (vec) disc_mask_kernel<true><<<grid, MASK_THREADS, 0, st>>>(p);
    else disc_mask_kernel<false><<<grid, MASK_THREADS, 0, st>>>(p);
    DISC_CUDA(cudaGetLastError());
    return DISC_OK;
}
