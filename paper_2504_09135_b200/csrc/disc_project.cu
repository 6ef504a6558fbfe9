// disc_project_step: the language model's last projection fused with the decoding step
// (Algorithm 1, lines 5-8 with P = L(a, T) of line 5 computed in place).
//
// logits[r][v] = bf16( sum_k h[r][k] * Wt[v][k] ), h = the R hidden vectors (bf16, d wide), Wt = the
// vocabulary projection stored one vocabulary entry per row (bf16, [V][d]), fp32 accumulation.
// The unfused path writes these R x V logits to HBM (1.05 GB per position at V = 128,256 and
// R = 4,096) and disc_step reads them back.  Here the projection runs on the tensor cores
// (tcgen05.mma, accumulators in tensor memory) and its epilogue keeps, per row and per 256-wide
// vocabulary tile, only the pair (m, s) with  sum_v 2^(z_v log2e / T) = 2^m * s  over the tile,
// i.e. what the step needs for the log-sum-exp over the whole vocabulary.  The logits themselves
// are stored only where the step will look at them: the tiles that hold a valid next token of the
// row (a 512-byte piece of the row for the typical row deep in the prefix tree; the whole row for
// a row at the root or at a node with a prebuilt mask).  disc_step then runs with the (m, s) pairs
// in place of its streaming pass.
//
// The GEMM: persistent, one CTA per SM, the CTAs of neighbouring SMs paired into clusters of two
// (cta_group::2).  A pair works on one 256 x 256 output tile at a time, tiles taken
// vocabulary-tile-major (the pairs that run at the same time share a tile of Wt through L2, so Wt
// crosses HBM once per call), K in blocks of 64.  Each CTA holds 128 rows of h and 128 of the 256
// vocabulary rows of Wt in its shared memory; the MMA, issued by the first CTA of the pair for both,
// reads the halves of Wt from both, and each CTA's tensor memory receives the 128 x 256
// accumulators of its own rows.
//   warp 0      one lane issues the TMA loads (cp.async.bulk.tensor, 128-byte swizzle) of this
//               CTA's h block and Wt half-block into a six-stage ring in shared memory; the loads
//               carry the cta_group::2 qualifier, which makes their byte counts arrive at the
//               first CTA's "full" barrier; none of them is multicast;
//   warp 1      allocates the tensor memory (both CTAs); in the first CTA one lane issues the MMAs
//               (four of M 256, N 256, K 16 per block) and commits them, multicast to both CTAs,
//               to the ring's "empty" barriers and, at the end of a tile, to the "accumulator
//               full" barriers;
//   warps 2-5   the epilogue: each thread owns one row of the tile, reads its 256 accumulators
//               from tensor memory in pieces of 32 columns (tcgen05.ld), rounds them to bf16 as
//               the unfused path would have stored them, and forms (m, s) in two passes (exact
//               maximum first).  Two accumulator buffers (2 x 256 columns) let the MMAs of the
//               next tile run under the epilogue of the current one; the epilogue warps of both
//               CTAs report to the first CTA's "accumulator empty" barrier.
// Every wait on an mbarrier is bounded by a clock; a wait that runs out sets the error word, makes
// every role of the CTA leave its loop (the other CTA of the pair follows when its own waits run
// out), and the kernel frees its tensor memory and returns.
// The tensor maps cover memory of this GPU only and no load is multicast.

#include <cuda.h>
#include <cuda_bf16.h>
#include <math_constants.h>

#include <mutex>

#include "disc_internal.cuh"

namespace {

using namespace disc;

constexpr int TILE_M = 128;                  // rows per CTA and tile (TMEM lanes); a pair of CTAs covers 256
constexpr int TILE_N = 256;                  // vocabulary entries per tile (TMEM columns, fp32)
constexpr int BLOCK_K = 64;                  // bf16 per row and K block = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int A_BYTES = TILE_M * BLOCK_K * 2;                 // 16 KB
constexpr int PROJ_THREADS = 192;
constexpr int TMEM_COLS = 512;               // two accumulators of 256 columns
constexpr long long WAIT_CYCLES = 1ll << 32;  // a wait gives up after this many SM clocks (about two seconds)
constexpr float LOG2E_F = 1.4426950408889634f;

struct ProjParams {
    int32_t R, V, d;
    int32_t m_tiles, n_tiles;
    float c2;                       // log2(e) / T
    float2* parts;                  // [R][n_tiles]: (m, s), sum over the tile = 2^m * s
    __nv_bfloat16* logits;          // [R][ld]
    int64_t ld;
    const uint32_t* tile_bits;      // [R][bits_ld]: bit n set = store row r's logits of tile n; null = store all
    int32_t bits_ld;
    unsigned int* error;            // set to 1 when a wait ran out
};

// ---- PTX wrappers ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return uint32_t(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// bounded wait; false when it gave up or another role of the CTA already had (then *abort is set)
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t i = 0;; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 63u) == 63u) {
            if (*abort) return false;
            if (clock64() - t0 > WAIT_CYCLES) break;
        }
    }
    *abort = 1;
    return false;
}
// the same for a whole warp that must stay converged: lane 0 waits, the others take over its result
// and then observe the completed phase themselves
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, volatile int* abort, int lane) {
    int ok = 1;
    if (lane == 0) ok = mbar_wait(bar, parity, abort) ? 1 : 0;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    if (!ok) return false;
    for (int i = 0; i < 1024 && !mbar_try_wait(bar, parity); ++i) {}
    return true;
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 32 consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* v) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major operand tile laid out by TMA with the 128-byte
// swizzle: rows of 64 bf16 (128 bytes), groups of eight rows 1024 bytes apart.
//   bits [0,14) start address >> 4; [16,30) leading byte offset >> 4 (not used by swizzled K-major
//   layouts, 1); [32,46) stride byte offset >> 4 (1024 >> 4); [46,48) version 1; [61,64) layout 2.
__device__ __forceinline__ uint64_t smem_desc_sw128(const void* tile) {
    const uint64_t addr = uint64_t(smem_u32(tile) >> 4) & 0x3FFFu;
    return addr | (uint64_t(1) << 16) | (uint64_t(1024 >> 4) << 32) | (uint64_t(1) << 46) | (uint64_t(2) << 61);
}

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float bf16_round(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

// The epilogue of one row of one tile: the 256 accumulators at `taddr` (this thread's lane of tensor
// memory) are read twice in pieces of 32 columns - exact maximum, then bf16 rounding and the sum
// of 2^(x*c2 - m) - and the rounded logits are stored where the step will read them.  Returns
// (m, s) with the tile's sum = 2^m * s.  Every lane of the warp must call it (tcgen05.ld is a
// warp-wide instruction); lanes whose row lies beyond R compute on zeros and store nothing.
__device__ __forceinline__ float2 epilogue_row(const ProjParams& p, const uint32_t taddr, const int row, const int n_idx) {
    const int col0 = n_idx * TILE_N;
    const bool row_ok = row < p.R;
    bool store = row_ok;
    if (row_ok && p.tile_bits)
        store = (__ldg(p.tile_bits + size_t(row) * p.bits_ld + (n_idx >> 5)) >> (n_idx & 31)) & 1u;
    // pass 1: the row's maximum over the tile
    float mx = -CUDART_INF_F;
    bool has_nan = false;
#pragma unroll 1
    for (int c = 0; c < TILE_N / 32; ++c) {
        uint32_t v[32];
        tmem_ld32(taddr + c * 32, v);
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            const float x = __uint_as_float(v[j]);
            if (col0 + c * 32 + j < p.V) { mx = fmaxf(mx, x); has_nan |= (x != x); }
        }
    }
    const float xm = bf16_round(mx);
    const float ref = (fabsf(xm) < CUDART_INF_F) ? xm * p.c2 : 0.f;
    // pass 2: bf16 rounding, sum of 2^(x*c2 - ref), logits out where the step will read them
    float s0 = 0.f, s1 = 0.f;
#pragma unroll 1
    for (int c = 0; c < TILE_N / 32; ++c) {
        uint32_t v[32];
        tmem_ld32(taddr + c * 32, v);
        uint32_t packed[16];
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
            const __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(v[j]), __uint_as_float(v[j + 1]));
            packed[j >> 1] = *reinterpret_cast<const uint32_t*>(&b2);
            const float x0 = __uint_as_float(packed[j >> 1] << 16);
            const float x1 = __uint_as_float(packed[j >> 1] & 0xffff0000u);
            const int col = col0 + c * 32 + j;
            if (col < p.V) s0 += ex2_approx(fmaf(x0, p.c2, -ref));
            if (col + 1 < p.V) s1 += ex2_approx(fmaf(x1, p.c2, -ref));
        }
        if (store) {
            __nv_bfloat16* dst = p.logits + size_t(row) * p.ld + col0 + c * 32;
            if (col0 + c * 32 + 32 <= p.V && (reinterpret_cast<uintptr_t>(dst) & 15u) == 0) {
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    reinterpret_cast<uint4*>(dst)[q] = make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
            } else {
                for (int j = 0; j < 32; ++j)
                    if (col0 + c * 32 + j < p.V)
                        reinterpret_cast<unsigned short*>(dst)[j] =
                            (unsigned short)((packed[j >> 1] >> ((j & 1) * 16)) & 0xffffu);
            }
        }
    }
    float s = s0 + s1;
    if (has_nan || !(fabsf(xm) < CUDART_INF_F)) s = (mx == -CUDART_INF_F) ? 0.f : CUDART_NAN_F;
    return make_float2((mx == -CUDART_INF_F) ? -CUDART_INF_F : ref, s);
}

// ---- the kernel: pairs of CTAs (cta_group::2) -------------------------------------------------------
constexpr int STAGES2 = 6;
constexpr int B2_BYTES = (TILE_N / 2) * BLOCK_K * 2;           // this CTA's half of the Wt block: 16 KB
constexpr int STAGE2_BYTES = A_BYTES + B2_BYTES;               // 32 KB
constexpr size_t PROJ2_SMEM = size_t(STAGES2) * STAGE2_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;
// Instruction descriptor: D fp32 (bits 4-5 = 1), A and B bf16 (bits 7-9, 10-12 = 1), both K-major
// (bits 15, 16 = 0), N >> 3 at bit 17, M >> 4 at bit 24 (M = 256: the two CTAs' rows together).
constexpr uint32_t IDESC2 = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(TILE_N >> 3) << 17) | (uint32_t((2 * TILE_M) >> 4) << 24);
constexpr uint32_t PEER_MASK = 0xFEFFFFFFu;                    // clears the bit that tells the two CTAs of a pair apart

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar) & PEER_MASK)
        : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// arrives, once every MMA issued so far has completed, on the barrier at this offset in BOTH CTAs
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"((unsigned short)3)
                 : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* slot, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t addr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
// arrive on the barrier at the same offset in the first CTA of the pair
__device__ __forceinline__ void mbar_arrive_leader(uint64_t* bar) {
    asm volatile(
        "{\n\t.reg .b32 ra;\n\t"
        "mapa.shared::cluster.u32 ra, %0, 0;\n\t"
        "mbarrier.arrive.release.cluster.shared::cluster.b64 _, [ra];\n\t}"
        ::"r"(smem_u32(bar))
        : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(PROJ_THREADS, 1)
disc_project_pair_kernel(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_w,
                         const ProjParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* tiles = reinterpret_cast<unsigned char*>((uintptr_t(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + size_t(STAGES2) * STAGE2_BYTES);
    uint64_t* full_bar = bars;                     // [STAGES2] loads of both CTAs -> MMA; used in the first CTA
    uint64_t* empty_bar = bars + STAGES2;          // [STAGES2] MMA -> loads, in each CTA
    uint64_t* acc_full = bars + 2 * STAGES2;       // [2] MMA -> epilogue, in each CTA
    uint64_t* acc_empty = bars + 2 * STAGES2 + 2;  // [2] epilogues of both CTAs -> MMA; used in the first CTA
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES2 + 4);
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();
    const bool leader = rank == 0;
    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s = 0; s < STAGES2; ++s) { mbar_init(full_bar + s, 1); mbar_init(empty_bar + s, 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(acc_full + a, 1); mbar_init(acc_empty + a, 8); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    cluster_sync_all();                            // the peer's barriers exist before anything signals them
    if (warp == 1) tmem_alloc_pair(tmem_slot, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(tmem_slot);
    volatile int* abort = &s_abort;

    const int k_blocks = (p.d + BLOCK_K - 1) / BLOCK_K;
    const int m_pairs = (p.m_tiles + 1) / 2;
    const int total_tiles = m_pairs * p.n_tiles;
    const int first = int(blockIdx.x >> 1), stride = int(gridDim.x >> 1);

    if (warp == 0) {
        // ---- loads: each CTA fetches its own 128 rows of h and its half of the Wt block
        if (lane == 0) {
            uint32_t it = 0;
            for (int tile = first; tile < total_tiles && !*abort; tile += stride) {
                const int n_idx = tile / m_pairs, m_idx = tile % m_pairs;
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    const int s = it % STAGES2;
                    const uint32_t round = it / STAGES2;
                    if (round > 0 && !mbar_wait(empty_bar + s, (round - 1) & 1u, abort)) break;
                    unsigned char* a_dst = tiles + size_t(s) * STAGE2_BYTES;
                    if (leader) mbar_expect_tx(full_bar + s, 2 * STAGE2_BYTES);
                    tma_load_2d_pair(a_dst, &map_h, kb * BLOCK_K, m_idx * 2 * TILE_M + int(rank) * TILE_M, full_bar + s);
                    tma_load_2d_pair(a_dst + A_BYTES, &map_w, kb * BLOCK_K, n_idx * TILE_N + int(rank) * (TILE_N / 2),
                                     full_bar + s);
                }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer: one lane of the first CTA, for both
        if (leader && lane == 0) {
            uint32_t it = 0, local = 0;
            for (int tile = first; tile < total_tiles && !*abort; tile += stride, ++local) {
                const uint32_t acc = local & 1u, use = local >> 1;
                if (use > 0 && !mbar_wait(acc_empty + acc, (use - 1) & 1u, abort)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * TILE_N;
                bool ok = true;
                for (int kb = 0; kb < k_blocks; ++kb, ++it) {
                    const int s = it % STAGES2;
                    if (!mbar_wait(full_bar + s, (it / STAGES2) & 1u, abort)) { ok = false; break; }
                    tc_fence_after();
                    const unsigned char* a_src = tiles + size_t(s) * STAGE2_BYTES;
                    const uint64_t a_desc = smem_desc_sw128(a_src), b_desc = smem_desc_sw128(a_src + A_BYTES);
#pragma unroll
                    for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
                        umma_bf16_pair(d_tmem, a_desc + uint64_t(2 * k), b_desc + uint64_t(2 * k), IDESC2, (kb | k) ? 1u : 0u);
                    umma_commit_pair(empty_bar + s);
                }
                if (!ok) break;
                umma_commit_pair(acc_full + acc);
            }
        }
    } else {
        // ---- epilogue of this CTA's 128 rows
        const int quarter = warp & 3;
        uint32_t local = 0;
        for (int tile = first; tile < total_tiles; tile += stride, ++local) {
            const int n_idx = tile / m_pairs, m_idx = tile % m_pairs;
            const uint32_t acc = local & 1u, use = local >> 1;
            if (!mbar_wait_warp(acc_full + acc, use & 1u, abort, lane)) break;
            tc_fence_after();
            const int row = m_idx * 2 * TILE_M + int(rank) * TILE_M + quarter * 32 + lane;
            const float2 ms = epilogue_row(p, tmem_base + acc * TILE_N + (uint32_t(quarter * 32) << 16), row, n_idx);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (leader) mbar_arrive(acc_empty + acc); else mbar_arrive_leader(acc_empty + acc);
            }
            if (row < p.R) p.parts[size_t(row) * p.n_tiles + n_idx] = ms;
        }
    }

    // ---- teardown: both CTAs are done with each other's shared and tensor memory before either leaves
    tc_fence_before();
    __syncthreads();
    if (s_abort && threadIdx.x == 0) {
        atomicExch(p.error, 1u);
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
    }
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

// Which 256-wide vocabulary tiles hold a valid next token of each row (one warp per row): every
// tile for a row at the root or at a heavy node (the step reads its whole row), the tiles of the
// children otherwise, none for a row that is complete.
__global__ void disc_tile_bits_kernel(int64_t n, const int32_t* __restrict__ node, const uint8_t* __restrict__ done,
                                      const int32_t* __restrict__ child_begin, const int32_t* __restrict__ node_tok,
                                      int64_t M, int32_t n_tiles, int32_t bits_ld, uint32_t* __restrict__ bits) {
    const int64_t row = (int64_t(blockIdx.x) * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (row >= n) return;
    uint32_t* out = bits + size_t(row) * bits_ld;
    const int32_t nd = node[row];
    int32_t cb = 0, ce = 0;
    if (!done[row] && nd >= 0 && int64_t(nd) < M) { cb = __ldg(child_begin + nd); ce = __ldg(child_begin + nd + 1); }
    const int32_t c = ce - cb;
    const bool all = c > 0 && (nd == 0 || c > DISC_HEAVY_MIN);
    for (int w = lane; w < bits_ld; w += 32) {
        uint32_t word = 0u;
        if (all) {
            const int lo_tile = w * 32;
            const int cnt = min(32, n_tiles - lo_tile);
            word = cnt >= 32 ? 0xffffffffu : (cnt > 0 ? ((1u << cnt) - 1u) : 0u);
        }
        out[w] = word;
    }
    if (all || c <= 0) return;
    __syncwarp();
    for (int32_t i = cb + lane; i < ce; i += 32) {
        const int32_t tile = __ldg(node_tok + i) / TILE_N;
        atomicOr(out + (tile >> 5), 1u << (tile & 31));
    }
}

// ---- host side ------------------------------------------------------------------------------------
using EncodeTiled = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                 const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
std::mutex g_proj_mutex;
EncodeTiled g_encode = nullptr;
bool g_attr_set = false;

int get_encode(EncodeTiled* out) {
    std::lock_guard<std::mutex> lock(g_proj_mutex);
    if (!g_encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        DISC_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
        if (!fn || q != cudaDriverEntryPointSuccess) return DISC_ERR_CUDA;
        g_encode = reinterpret_cast<EncodeTiled>(fn);
    }
    if (!g_attr_set) {
        DISC_CUDA(cudaFuncSetAttribute(disc_project_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(PROJ2_SMEM)));
        g_attr_set = true;
    }
    *out = g_encode;
    return DISC_OK;
}

// a [rows][d] bf16 row-major matrix as a 2-D tensor map with boxes of 64 x box_rows and the 128-byte swizzle
int make_map(EncodeTiled enc, CUtensorMap* map, const void* base, int64_t rows, int64_t d, int64_t ld, int box_rows) {
    const cuuint64_t dims[2] = {cuuint64_t(d), cuuint64_t(rows)};
    const cuuint64_t strides[1] = {cuuint64_t(ld) * 2};
    const cuuint32_t box[2] = {cuuint32_t(BLOCK_K), cuuint32_t(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { g_last_cuda_error = int(cudaErrorInvalidValue); return DISC_ERR_CUDA; }
    return DISC_OK;
}

}  // namespace

extern "C" {

int64_t disc_project_scratch_bytes(const disc_set_t* s, int64_t n) {
    if (!s || n < 0) return DISC_ERR_ARG;
    const int64_t n_tiles = (s->V + TILE_N - 1) / TILE_N;
    const int64_t bits_ld = (n_tiles + 31) / 32;
    return 256 + n * n_tiles * 8 + n * bits_ld * 4;
}

int disc_project_step(const disc_set_t* s, const void* hidden, int64_t hidden_ld, const void* wt, int64_t wt_ld,
                      int32_t d, int64_t n, float inv_temperature, uint64_t seed, uint32_t step, int64_t row_base,
                      int32_t* node, int32_t* lo, int32_t* hi, int32_t* depth, float* logw, uint8_t* done,
                      int32_t* token_out, int32_t* seq_tokens, int32_t seq_ld, float* logq_out, float* logp_out,
                      uint8_t* status_out, void* logits_buf, int64_t logits_ld, int32_t store_all, void* scratch,
                      int64_t scratch_bytes, void* stream) {
    if (!s || n < 0 || n >= (int64_t(1) << 31) || d <= 0) return DISC_ERR_ARG;
    if (const int rc = check_device(s)) return rc;
    if (n == 0) return DISC_OK;
    if (!hidden || !wt || !node || !lo || !hi || !depth || !logw || !done || !token_out || !status_out || !logits_buf ||
        !scratch)
        return DISC_ERR_ARG;
    if (hidden_ld < d || wt_ld < d || logits_ld < s->V || row_base < 0 || (seq_tokens && seq_ld <= 0)) return DISC_ERR_ARG;
    if (!(inv_temperature > 0.f) || !(inv_temperature <= 3.0e38f)) return DISC_ERR_ARG;
    // TMA: 16-byte aligned bases and row pitches; the step's vector loads: 16-byte aligned logits rows
    if ((reinterpret_cast<uintptr_t>(hidden) | reinterpret_cast<uintptr_t>(wt) | reinterpret_cast<uintptr_t>(logits_buf) |
         reinterpret_cast<uintptr_t>(scratch)) & 15u)
        return DISC_ERR_ARG;
    if ((hidden_ld * 2) % 16 || (wt_ld * 2) % 16 || (logits_ld * 2) % 16 || d % 8) return DISC_ERR_UNSUPPORTED;
    if (row_base + n > (int64_t(1) << 32)) return DISC_ERR_UNSUPPORTED;
    if (scratch_bytes < disc_project_scratch_bytes(s, n)) return DISC_ERR_ARG;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    EncodeTiled enc = nullptr;
    if (const int rc = get_encode(&enc)) return rc;

    ProjParams p;
    p.R = int32_t(n); p.V = s->V; p.d = d;
    p.m_tiles = int32_t((n + TILE_M - 1) / TILE_M);
    p.n_tiles = (s->V + TILE_N - 1) / TILE_N;
    p.c2 = inv_temperature * LOG2E_F;
    p.bits_ld = (p.n_tiles + 31) / 32;
    unsigned char* sc = static_cast<unsigned char*>(scratch);
    p.error = reinterpret_cast<unsigned int*>(sc);
    p.parts = reinterpret_cast<float2*>(sc + 256);
    uint32_t* bits = reinterpret_cast<uint32_t*>(sc + 256 + size_t(n) * p.n_tiles * 8);
    p.tile_bits = store_all ? nullptr : bits;
    p.logits = static_cast<__nv_bfloat16*>(logits_buf);
    p.ld = logits_ld;

    alignas(64) CUtensorMap map_h, map_w;
    if (const int rc = make_map(enc, &map_h, hidden, n, d, hidden_ld, TILE_M)) return rc;
    if (const int rc = make_map(enc, &map_w, wt, s->V, d, wt_ld, TILE_N / 2)) return rc;      // each CTA of a pair loads half

    DISC_CUDA(cudaMemsetAsync(p.error, 0, 4, st));
    if (!store_all) {
        disc_tile_bits_kernel<<<unsigned((n * 32 + 255) / 256), 256, 0, st>>>(n, node, done, s->child_begin, s->node_tok,
                                                                             s->M, p.n_tiles, p.bits_ld, bits);
        DISC_CUDA(cudaGetLastError());
    }
    int dev = 0, sms = 0;
    DISC_CUDA(cudaGetDevice(&dev));
    DISC_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const int pairs_total = ((p.m_tiles + 1) / 2) * p.n_tiles, pairs_max = sms / 2;
    const int pairs = pairs_total < pairs_max ? pairs_total : pairs_max;
    disc_project_pair_kernel<<<unsigned(2 * pairs), PROJ_THREADS, PROJ2_SMEM, st>>>(map_h, map_w, p);
    DISC_CUDA(cudaGetLastError());
    return step_with_parts(s, logits_buf, DISC_BF16, logits_ld, n, inv_temperature, seed, step, row_base, node, lo, hi,
                           depth, logw, done, token_out, seq_tokens, seq_ld, logq_out, logp_out, status_out, p.parts,
                           p.n_tiles, st);
}

int disc_project_error(const void* scratch, void* stream) {
    if (!scratch) return DISC_ERR_ARG;
    unsigned int e = 0;
    DISC_CUDA(cudaMemcpyAsync(&e, scratch, 4, cudaMemcpyDeviceToHost, static_cast<cudaStream_t>(stream)));
    DISC_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    return e ? DISC_ERR_CUDA : DISC_OK;
}

}  // extern "C"
