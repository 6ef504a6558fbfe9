// disc_resample: K-way importance draw (Algorithm 1, line 22); disc_accept: the accept test
// (Algorithm 1, line 16); disc_accept_resample: both in the order of Algorithm 1, lines 11-22.
//
// One warp per query.  The K log-weights are read three times from L1/L2 (maximum, total, scan
// and search); the inclusive prefix sums come from a shuffle scan over tiles of 32 candidates with
// a running carry, computed identically in the last two passes so that the threshold u * total is
// compared with the very sums it was derived from.

#include <math_constants.h>

#include "disc_internal.cuh"

namespace {

using namespace disc;

constexpr int RS_THREADS = 128;
constexpr int RS_WARPS = RS_THREADS / 32;

__device__ __forceinline__ float warp_inclusive_scan(float x, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        float y = __shfl_up_sync(0xffffffffu, x, o);
        if (lane >= o) x += y;
    }
    return x;
}

// K-way draw of one query by one warp: pick with probability e^{w_k} / sum_j e^{w_j} at the uniform u.
__device__ __forceinline__ void resample_query(const float* __restrict__ w, int32_t K, float u, int lane,
                                               int32_t& pick, float& logz, uint8_t& st) {
    float m = -CUDART_INF_F;
    int has_nan = 0;
    for (int k = lane; k < K; k += 32) {
        float x = w[k];
        if (x != x) has_nan = 1; else m = fmaxf(m, x);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    has_nan = __any_sync(0xffffffffu, has_nan);
    st = has_nan ? DISC_ROW_NONFINITE : 0;

    if (!(fabsf(m) < CUDART_INF_F)) {
        // no candidate with a finite weight: uniform pick
        st |= DISC_ROW_NOMASS;
        pick = min(K - 1, int32_t(floorf(u * float(K))));
        logz = (m > 0.f) ? m : -CUDART_INF_F;
        return;
    }
    const int tiles = (K + 31) / 32;
    float carry = 0.f;
    for (int t = 0; t < tiles; ++t) {
        int k = t * 32 + lane;
        float x = (k < K) ? w[k] : CUDART_NAN_F;
        float e = (x == x) ? expf(x - m) : 0.f;
        float c = warp_inclusive_scan(e, lane) + carry;
        carry = __shfl_sync(0xffffffffu, c, 31);
    }
    const float total = carry;
    const float target = u * total;
    pick = K - 1;
    carry = 0.f;
    for (int t = 0; t < tiles; ++t) {
        int k = t * 32 + lane;
        float x = (k < K) ? w[k] : CUDART_NAN_F;
        float e = (x == x) ? expf(x - m) : 0.f;
        float c = warp_inclusive_scan(e, lane) + carry;
        carry = __shfl_sync(0xffffffffu, c, 31);
        uint32_t hit = __ballot_sync(0xffffffffu, (k < K) && (c > target));
        if (hit) { pick = t * 32 + (__ffs(hit) - 1); break; }
    }
    logz = m + logf(total / float(K));
}

__global__ void __launch_bounds__(RS_THREADS) disc_resample_kernel(
    const float* __restrict__ logw, int32_t B, int32_t K, PhiloxKey key, uint32_t query_base,
    int32_t* __restrict__ idx_out, float* __restrict__ logz_out, const int32_t* __restrict__ seq_tokens,
    int32_t seq_ld, int32_t* __restrict__ tokens_out, uint8_t* __restrict__ status_out) {
    const int lane = threadIdx.x & 31;
    const int b = blockIdx.x * RS_WARPS + (threadIdx.x >> 5);
    if (b >= B) return;
    const uint4 r = philox4x32_10(query_base + uint32_t(b), 0u, 0u, 1u, key);
    int32_t pick;
    float logz;
    uint8_t st;
    resample_query(logw + size_t(b) * K, K, uniform_from_bits(r.x), lane, pick, logz, st);
    if (lane == 0) {
        idx_out[b] = pick;
        if (logz_out) logz_out[b] = logz;
        status_out[b] = st;
    }
    if (seq_tokens && tokens_out) {
        const int32_t* src = seq_tokens + (size_t(b) * K + pick) * seq_ld;
        for (int t = lane; t < seq_ld; t += 32) tokens_out[size_t(b) * seq_ld + t] = src[t];
    }
}

// Algorithm 1, lines 11-22 on 2K finished candidates per query: the accept test over candidates
// 0..K-1 in order (32 at a time, one per lane), then, if all were rejected, the K-way draw over
// candidates K..2K-1.  One warp per query.
__global__ void __launch_bounds__(RS_THREADS) disc_accept_resample_kernel(
    const float* __restrict__ logw, int32_t B, int32_t K, PhiloxKey key, uint32_t query_base,
    int32_t* __restrict__ choice_out, int32_t* __restrict__ first_out, float* __restrict__ logz_out,
    const int32_t* __restrict__ seq_tokens, int32_t seq_ld, int32_t* __restrict__ tokens_out,
    uint8_t* __restrict__ status_out) {
    const int lane = threadIdx.x & 31;
    const int b = blockIdx.x * RS_WARPS + (threadIdx.x >> 5);
    if (b >= B) return;
    const float* w = logw + size_t(b) * 2 * K;
    const uint32_t q = query_base + uint32_t(b);
    int32_t first = -1;
    for (int t = 0; t * 32 < K && first < 0; ++t) {
        const int k = t * 32 + lane;
        bool ok = false;
        if (k < K) {
            const uint4 r = philox4x32_10(q, uint32_t(k), 0u, 2u, key);
            ok = w[k] > logf(uniform_from_bits(r.x));
        }
        const uint32_t hit = __ballot_sync(0xffffffffu, ok);
        if (hit) first = t * 32 + (__ffs(hit) - 1);
    }
    const uint4 r = philox4x32_10(q, 0u, 0u, 1u, key);
    int32_t pick;
    float logz;
    uint8_t st;
    resample_query(w + K, K, uniform_from_bits(r.x), lane, pick, logz, st);
    const int32_t choice = first >= 0 ? first : K + pick;
    if (lane == 0) {
        choice_out[b] = choice;
        if (first_out) first_out[b] = first;
        if (logz_out) logz_out[b] = logz;
        status_out[b] = st;
    }
    if (seq_tokens && tokens_out) {
        const int32_t* src = seq_tokens + (size_t(b) * 2 * K + choice) * seq_ld;
        for (int t = lane; t < seq_ld; t += 32) tokens_out[size_t(b) * seq_ld + t] = src[t];
    }
}

__global__ void disc_accept_kernel(const float* __restrict__ logw, int32_t B, int32_t K, PhiloxKey key,
                                   uint32_t query_base, int32_t* __restrict__ first_out) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    int32_t first = -1;
    for (int k = 0; k < K; ++k) {
        const uint4 r = philox4x32_10(query_base + uint32_t(b), uint32_t(k), 0u, 2u, key);
        const float eps = uniform_from_bits(r.x);
        if (logw[size_t(b) * K + k] > logf(eps)) { first = k; break; }
    }
    first_out[b] = first;
}

}  // namespace

extern "C" {

int disc_resample(const float* logw, int32_t B, int32_t K, uint64_t seed, int64_t query_base, int32_t* idx_out,
                  float* logz_out, const int32_t* seq_tokens, int32_t seq_ld, int32_t* tokens_out,
                  uint8_t* status_out, void* stream) {
    if (B < 0 || K <= 0 || query_base < 0) return DISC_ERR_ARG;
    if (query_base + B > (int64_t(1) << 32)) return DISC_ERR_UNSUPPORTED;   // the query coordinate is one 32-bit word
    if (B == 0) return DISC_OK;
    if (!logw || !idx_out || !status_out) return DISC_ERR_ARG;
    if ((seq_tokens || tokens_out) && seq_ld <= 0) return DISC_ERR_ARG;
    disc_resample_kernel<<<(B + RS_WARPS - 1) / RS_WARPS, RS_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
        logw, B, K, philox_key(seed), uint32_t(query_base), idx_out, logz_out, seq_tokens, seq_ld, tokens_out,
        status_out);
    DISC_CUDA(cudaGetLastError());
    return DISC_OK;
}

int disc_accept_resample(const float* logw, int32_t B, int32_t K, uint64_t seed, int64_t query_base,
                         int32_t* choice_out, int32_t* first_out, float* logz_out, const int32_t* seq_tokens,
                         int32_t seq_ld, int32_t* tokens_out, uint8_t* status_out, void* stream) {
    if (B < 0 || K <= 0 || K > (1 << 29) || query_base < 0) return DISC_ERR_ARG;
    if (query_base + B > (int64_t(1) << 32)) return DISC_ERR_UNSUPPORTED;   // the query coordinate is one 32-bit word
    if (B == 0) return DISC_OK;
    if (!logw || !choice_out || !status_out) return DISC_ERR_ARG;
    if ((seq_tokens || tokens_out) && seq_ld <= 0) return DISC_ERR_ARG;
    disc_accept_resample_kernel<<<(B + RS_WARPS - 1) / RS_WARPS, RS_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(
        logw, B, K, philox_key(seed), uint32_t(query_base), choice_out, first_out, logz_out, seq_tokens, seq_ld,
        tokens_out, status_out);
    DISC_CUDA(cudaGetLastError());
    return DISC_OK;
}

int disc_accept(const float* logw, int32_t B, int32_t K, uint64_t seed, int64_t query_base, int32_t* first_out,
                void* stream) {
    if (B < 0 || K <= 0 || query_base < 0) return DISC_ERR_ARG;
    if (query_base + B > (int64_t(1) << 32)) return DISC_ERR_UNSUPPORTED;   // the query coordinate is one 32-bit word
    if (B == 0) return DISC_OK;
    if (!logw || !first_out) return DISC_ERR_ARG;
    disc_accept_kernel<<<(B + 127) / 128, 128, 0, static_cast<cudaStream_t>(stream)>>>(
        logw, B, K, philox_key(seed), uint32_t(query_base), first_out);
    DISC_CUDA(cudaGetLastError());
    return DISC_OK;
}

}  // extern "C"
