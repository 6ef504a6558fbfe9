// Internal declarations shared by the library's translation units.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "disc.h"

struct disc_set {
    int32_t V = 0;            // vocabulary size
    int32_t W = 0;            // mask words per row
    int32_t Wp = 0;           // row stride of the prebuilt masks in words (W rounded up to 4: 16-byte rows)
    int32_t l_max = 0;
    int64_t N = 0;            // members
    int64_t E = 0;            // table entries
    int64_t M = 0;            // index nodes including the root (node 0)
    int device = 0;
    // sorted table (the array X of Algorithm 2, ragged instead of padded)
    int32_t* tok = nullptr;        // [E]
    uint32_t* row_off = nullptr;   // [N+1]
    // prefix index, breadth-first: node 0 = empty prefix, then all prefixes of length 1, 2, ...
    // in sorted order.  The children of node j are nodes child_begin[j] .. child_begin[j+1]-1,
    // ascending in token id.
    int32_t* node_tok = nullptr;     // [M]   last token of the prefix
    int32_t* node_lo = nullptr;      // [M]   first table row having the prefix
    int32_t* child_begin = nullptr;  // [M+1]
    // first level shortcuts
    uint32_t* root_mask = nullptr;   // [W]   valid set of the empty prefix
    int32_t* root_child = nullptr;   // [V]   node of the one-token prefix [v], or -1
    // prebuilt masks of the nodes with more than DISC_HEAVY_MIN children ("heavy" nodes)
    int32_t n_heavy = 0;
    int32_t* heavy_nodes = nullptr;  // [n_heavy] ascending node ids
    uint32_t* heavy_masks = nullptr; // [n_heavy][Wp]
    // scratch of disc_mask: rows handed out so far by its writer kernel (reset by its search
    // kernel).  Calls of disc_mask on one handle must therefore not overlap on the GPU.
    unsigned int* work_counter = nullptr;
    int64_t level_off[DISC_MAX_DEPTH + 2] = {0};  // node id where level d starts (level_off[0] = 1)
    int64_t device_bytes = 0;
    double build_seconds = 0.0;
};

// a node with more children than this has its valid-set mask prebuilt at set-build time
#define DISC_HEAVY_MIN 1024

namespace disc {

extern thread_local int g_last_cuda_error;

// index of `node` in the ascending list of heavy nodes, or -1 (one thread; the list is small)
__device__ __forceinline__ int32_t heavy_index(const int32_t* __restrict__ heavy_nodes, int32_t n_heavy,
                                               int32_t node) {
    int32_t a = 0, b = n_heavy;
    while (a < b) {
        int32_t m = (a + b) >> 1;
        int32_t v = __ldg(heavy_nodes + m);
        if (v == node) return m;
        if (v < node) a = m + 1; else b = m;
    }
    return -1;
}

inline int cuda_fail(cudaError_t e) {
    g_last_cuda_error = int(e);
    return e == cudaErrorMemoryAllocation ? DISC_ERR_OOM : DISC_ERR_CUDA;
}

// the handle's memory lives on the device it was built on: calls with another device current are refused
inline int check_device(const disc_set* s) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return DISC_ERR_CUDA;
    return dev == s->device ? DISC_OK : DISC_ERR_ARG;
}

#define DISC_CUDA(call)                                         \
    do {                                                        \
        cudaError_t e__ = (call);                               \
        if (e__ != cudaSuccess) return ::disc::cuda_fail(e__);  \
    } while (0)

// ------------------------------------------------------------------ Philox4x32-10
// Counter-based generator of Salmon et al. (SC'11).  Round keys depend only on the seed.
struct PhiloxKey {
    uint32_t k0, k1;
};

__host__ __device__ __forceinline__ PhiloxKey philox_key(uint64_t seed) {
    return PhiloxKey{uint32_t(seed), uint32_t(seed >> 32)};
}

__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               PhiloxKey key) {
    uint32_t k0 = key.k0, k1 = key.k1;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = uint64_t(0xD2511F53u) * c0;
        uint64_t p1 = uint64_t(0xCD9E8D57u) * c2;
        uint32_t n0 = uint32_t(p1 >> 32) ^ c1 ^ k0;
        uint32_t n2 = uint32_t(p0 >> 32) ^ c3 ^ k1;
        c1 = uint32_t(p1);
        c3 = uint32_t(p0);
        c0 = n0;
        c2 = n2;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return make_uint4(c0, c1, c2, c3);
}

// The ten round keys (k0 + r*W0, k1 + r*W1), computed once on the host and passed as kernel
// parameters, so that a round is two wide multiplies and two three-input XORs.
struct PhiloxRoundKeys {
    uint32_t k[20];
};

inline PhiloxRoundKeys philox_round_keys(uint64_t seed) {
    PhiloxRoundKeys rk;
    uint32_t k0 = uint32_t(seed), k1 = uint32_t(seed >> 32);
    for (int r = 0; r < 10; ++r) {
        rk.k[2 * r] = k0;
        rk.k[2 * r + 1] = k1;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return rk;
}

__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               const PhiloxRoundKeys& rk) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = uint64_t(0xD2511F53u) * c0;
        uint64_t p1 = uint64_t(0xCD9E8D57u) * c2;
        uint32_t n0 = uint32_t(p1 >> 32) ^ c1 ^ rk.k[2 * r];
        uint32_t n2 = uint32_t(p0 >> 32) ^ c3 ^ rk.k[2 * r + 1];
        c1 = uint32_t(p1);
        c3 = uint32_t(p0);
        c0 = n0;
        c2 = n2;
    }
    return make_uint4(c0, c1, c2, c3);
}

// disc_step with the sums over the whole vocabulary given as per-part (m, s) pairs (disc_step.cu)
int step_with_parts(const disc_set* s, const void* logits, disc_dtype_t dtype, int64_t ld, int64_t n,
                    float inv_temperature, uint64_t seed, uint32_t step, int64_t row_base, int32_t* node, int32_t* lo,
                    int32_t* hi, int32_t* depth, float* logw, uint8_t* done, int32_t* token_out, int32_t* seq_tokens,
                    int32_t seq_ld, float* logq_out, float* logp_out, uint8_t* status_out, const float2* parts,
                    int32_t n_parts, cudaStream_t st);

// disc_step in top-M mode (disc_step.cu): the valid set is the verified candidates, the sums come from disc_topm
int step_with_candidates(const disc_set* s, const void* logits, disc_dtype_t dtype, int64_t ld, int64_t n,
                         float inv_temperature, uint64_t seed, uint32_t step, int64_t row_base, int32_t* node, int32_t* lo,
                         int32_t* hi, int32_t* depth, float* logw, uint8_t* done, int32_t* token_out, int32_t* seq_tokens,
                         int32_t seq_ld, float* logq_out, float* logp_out, uint32_t* mask_out, uint8_t* status_out,
                         const int32_t* cand, const uint8_t* valid, int32_t M, const float2* lse, cudaStream_t st);

// top 23 bits k of a word -> u = (2k+1) * 2^-24, exact in fp32, as is 1-u
__device__ __forceinline__ float uniform_from_bits(uint32_t r) {
    return float((r >> 9) * 2u + 1u) * 5.9604644775390625e-08f;
}

__device__ __forceinline__ uint32_t pick_word(const uint4& w, uint32_t lane) {
    return lane == 0 ? w.x : lane == 1 ? w.y : lane == 2 ? w.z : w.w;
}

// Gumbel noise -log(-log u) with accurate logarithms
__device__ __forceinline__ float gumbel_from_uniform(float u) { return -logf(-logf(u)); }

}  // namespace disc
