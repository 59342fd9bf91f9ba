// Prefill GEMM on the 5th-generation tensor cores (sm_100a): C[M, n] (=|+=) A[M, K] * W[n, K]^T,
// bf16 operands, fp32 accumulation in tensor memory.  Three kernels, chosen by problem size in tgpk_gemm_tc(): one
// tile per CTA (below), a persistent kernel with 128 x 256 tiles and double-buffered accumulators, and - for the large
// products of a prefill - a kernel in which the two CTAs of a cluster share 256 x 256 tiles through the two-SM MMA.
//
// One CTA computes a 128 x BN tile.  Warp 0 (one lane) feeds a shared-memory ring of ST stages with TMA
// (128-byte swizzle, 64 bf16 of K per stage); warp 1 (one lane) issues tcgen05.mma (M=128, N=BN, K=16,
// four per stage) into a TMEM accumulator and releases stages with tcgen05.commit; warps 2-5 wait for the
// last commit, read the accumulator with tcgen05.ld (each warp its own 32-lane quarter) and store fp32 rows.
// Out-of-range rows / columns / K are zero-filled by TMA and masked in the epilogue, so any M, n and
// any K % 8 == 0 work.  Every mbarrier wait is bounded in time: a wait that runs out records an error code
// and the CTA drains and returns instead of hanging the GPU.
#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cudaTypedefs.h>
#include <cstdint>
#include "tgp.h"
#include "tgp_kernels.h"
#include "tgp_sm100.cuh"

namespace {

using namespace tgp_sm100;
constexpr int BK = 64, GROUP_M = 16;

__device__ int g_gemm_tc_error = 0;                    // 0 ok; else (role << 8) | stage of the first wait that ran out

// Optional epilogue: the accumulator is the up projection u of a SwiGLU FFN and the gate projection g of the same
// elements is already in memory (fp32, same geometry as C).  Instead of storing u, the epilogue stores
// a = bf16(g / (1 + exp(-g)) * u) - the arithmetic of the stand-alone SwiGLU kernel, on the very values it would have
// read - so u never goes to memory, g is read once instead of twice and the SwiGLU launch disappears.
struct Epi { const float *gate; __nv_bfloat16 *aout; };

// 32 consecutive elements of one output row, element offset `off` in C's geometry, `cnt` of them inside the matrix
__device__ __forceinline__ void swiglu_store32(const Epi &ep, size_t off, const float *v, uint32_t cnt) {
    const float *g = ep.gate + off;
    __nv_bfloat16 *a = ep.aout + off;
    if (cnt == 32 && (off & 7) == 0 && ((reinterpret_cast<uintptr_t>(ep.gate) | reinterpret_cast<uintptr_t>(ep.aout)) & 15u) == 0) {
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
            const float4 g0 = *reinterpret_cast<const float4 *>(g + j), g1 = *reinterpret_cast<const float4 *>(g + j + 4);
            const float gv[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
            uint32_t w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                __nv_bfloat162 pk = __floats2bfloat162_rn(gv[2 * i] / (1.0f + expf(-gv[2 * i])) * v[j + 2 * i],
                                                          gv[2 * i + 1] / (1.0f + expf(-gv[2 * i + 1])) * v[j + 2 * i + 1]);
                w[i] = *reinterpret_cast<uint32_t *>(&pk);
            }
            *reinterpret_cast<uint4 *>(a + j) = make_uint4(w[0], w[1], w[2], w[3]);
        }
    } else {
        for (uint32_t j = 0; j < cnt; ++j) a[j] = __float2bfloat16_rn(g[j] / (1.0f + expf(-g[j])) * v[j]);
    }
}

template <int BN, int ST, int KH>
struct Smem {
    static constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, HALF_BYTES = A_BYTES + B_BYTES, STAGE_BYTES = KH * HALF_BYTES;
    static constexpr int BAR_OFF = ST * STAGE_BYTES;
    static constexpr int TOTAL = BAR_OFF + 256 + 1024;        // barriers (2 * ST + 1, TMEM slot, flag) + slack to align the base to 1024 bytes
};

// (ST stages of KH 64-wide K blocks each: with KH = 2 the producer and the MMA thread meet half as often)
// SWAP: the operands trade places - the tile's 128 rows are weight rows (M counts them), its BN columns activation rows
// (n counts them) - and the tile is stored transposed, C[activation row][col0 + weight row].  For products of up to 128
// activation rows a CTA then streams 128 weight rows through its TMA ring instead of BN, which is what such a product
// is bound by.
template <int BN, int ST, int KH, bool SWAP>
__global__ void __launch_bounds__(192) tgp_matmul_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                                                      float *__restrict__ C, uint32_t M, uint32_t n, uint32_t K, uint32_t ldc, uint32_t col0, int accumulate, const Epi ep) {
    extern __shared__ uint8_t smem_raw[];
    using S = Smem<BN, ST, KH>;
    constexpr int STAGES = ST;                      // depth of this instantiation's TMA ring
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + S::BAR_OFF);
    uint64_t *empty = full + STAGES;
    uint64_t *acc_full = empty + STAGES;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_full + 1);
    volatile uint32_t *failed = tmem_slot + 1;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Tile order: groups of GROUP_M row tiles are swept across all column tiles before the next group starts, so the
    // CTAs in flight together share a few A panels and a few W panels that fit in L2 (instead of re-streaming A from
    // HBM once per column tile when M is large).
    const uint32_t tiles_m = (M + BM - 1) / BM, tiles_n = (n + BN - 1) / BN;
    const uint32_t group = blockIdx.x / (GROUP_M * tiles_n), first_m = group * GROUP_M;
    const uint32_t rows_in_group = min((uint32_t)GROUP_M, tiles_m - first_m);
    const uint32_t in_group = blockIdx.x - group * GROUP_M * tiles_n;
    const uint32_t m0 = (first_m + in_group % rows_in_group) * BM, n0 = (in_group / rows_in_group) * BN;
    const uint32_t num_k = (K + KH * BK - 1) / (KH * BK);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(acc_full, 1);
        *failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"((uint32_t)BN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t armed = 0;
            const uint32_t withhold = blockIdx.x == 0 ? (uint32_t)g_withhold_step : 0xffffffffu;     // test hook: this stage is never loaded
            for (uint32_t kb = 0; kb < num_k; ++kb) {
                const uint32_t s = kb % STAGES, ph = (kb / STAGES) & 1;
                if (kb == withhold) break;
                if (*failed || !mbar_wait(&empty[s], ph ^ 1, failed)) { if (!*failed) { *failed = 1; atomicCAS(&g_gemm_tc_error, 0, (1 << 8) | (int)s); } break; }
                mbar_expect_tx(&full[s], S::STAGE_BYTES);
#pragma unroll
                for (int h = 0; h < KH; ++h) {
                    tma_load_2d(smem + s * S::STAGE_BYTES + h * S::HALF_BYTES, &tmA, (int)((kb * KH + h) * BK), (int)m0, &full[s]);
                    tma_load_2d(smem + s * S::STAGE_BYTES + h * S::HALF_BYTES + S::A_BYTES, &tmB, (int)((kb * KH + h) * BK), (int)n0, &full[s]);
                }
                armed = kb + 1;
            }
            if (*failed) {
                // let the copies this thread started land before the CTA's shared memory is given up
                volatile uint32_t never = 0;
                for (uint32_t kb = armed > STAGES ? armed - STAGES : 0; kb < armed; ++kb) mbar_wait(&full[kb % STAGES], (kb / STAGES) & 1, &never);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc(BN);
            bool ok = true;
            for (uint32_t kb = 0; kb < num_k && ok; ++kb) {
                const uint32_t s = kb % STAGES, ph = (kb / STAGES) & 1;
                if (*failed || !mbar_wait(&full[s], ph, failed)) { if (!*failed) { *failed = 1; atomicCAS(&g_gemm_tc_error, 0, (2 << 8) | (int)s); } ok = false; break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                for (uint32_t h = 0; h < KH; ++h) {
                    const uint64_t da = umma_desc(smem_u32(smem + s * S::STAGE_BYTES + h * S::HALF_BYTES));
                    const uint64_t db = umma_desc(smem_u32(smem + s * S::STAGE_BYTES + h * S::HALF_BYTES + S::A_BYTES));
#pragma unroll
                    for (uint32_t k = 0; k < BK / 16; ++k) umma(tmem_base, da + 2 * k, db + 2 * k, idesc, (kb | h | k) != 0);   // +32 bytes of K per step
                }
                umma_commit(&empty[s]);
            }
            if (ok) umma_commit(acc_full);
        }
    } else {
        bool ready = !*failed && mbar_wait(acc_full, 0, failed);
        if (!ready && !*failed) { *failed = 1; atomicCAS(&g_gemm_tc_error, 0, 3 << 8); }
        ready = __all_sync(0xffffffffu, ready && !*failed);      // tcgen05.ld is warp-collective: decide per warp
        if (ready) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t quarter = warp & 3;                    // TMEM lanes this warp may read
            const uint32_t row = m0 + quarter * 32 + lane;
            const bool vec = ((ldc | col0) & 3u) == 0 && (reinterpret_cast<uintptr_t>(C) & 15u) == 0;
#pragma unroll 1
            for (uint32_t c = 0; c < BN / 32; ++c) {
                float v[32];
                tmem_ld32(tmem_base + ((quarter * 32) << 16) + c * 32, v);
                if (SWAP) {
                    // a warp's 32 lanes hold 32 consecutive weight rows: for each activation row they write 128 contiguous bytes
                    if (row < M) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (n0 + c * 32 + j < n) {
                                float *d = C + (size_t)(n0 + c * 32 + j) * ldc + col0 + row;
                                *d = accumulate ? *d + v[j] : v[j];
                            }
                    }
                } else if (row < M) {
                    float *dst = C + (size_t)row * ldc + col0 + n0 + c * 32;
                    const uint32_t col = n0 + c * 32;
                    if (ep.aout) { if (col < n) swiglu_store32(ep, (size_t)row * ldc + col0 + col, v, min(32u, n - col)); }
                    else if (vec && col + 32 <= n) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            float4 o = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                            if (accumulate) { const float4 old = *reinterpret_cast<const float4 *>(dst + j); o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w; }
                            *reinterpret_cast<float4 *>(dst + j) = o;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (col + j < n) dst[j] = accumulate ? dst[j] + v[j] : v[j];
                    }
                }
            }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    __syncthreads();
    if (warp == 2) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)BN) : "memory");
    }
}

// ---- persistent variant for large problems ------------------------------------------------------------------
// One CTA per SM walks 128 x 256 tiles (grouped order as above).  Four TMA stages of 48 KB; the TMEM holds two
// 256-column accumulators, so the MMA warp starts the next tile while the four epilogue warps drain the previous
// one (acc_full / acc_empty barriers per buffer).  Same bounded waits and error word as the kernel above.
constexpr int P_BN = 256, P_STAGES = 4;

__global__ void __launch_bounds__(192, 1) tgp_matmul_tc_persistent_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                                                                    float *__restrict__ C, uint32_t M, uint32_t n, uint32_t K, uint32_t ldc, uint32_t col0, int accumulate, const Epi ep) {
    extern __shared__ uint8_t smem_raw[];
    constexpr int A_BYTES = BM * BK * 2, B_BYTES = P_BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + P_STAGES * STAGE_BYTES);
    uint64_t *empty = full + P_STAGES;
    uint64_t *acc_full = empty + P_STAGES;           // [2]
    uint64_t *acc_empty = acc_full + 2;              // [2]
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);
    volatile uint32_t *failed = tmem_slot + 1;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t num_k = (K + BK - 1) / BK;
    const uint32_t tiles_m = (M + BM - 1) / BM, tiles_n = (n + P_BN - 1) / P_BN, tiles = tiles_m * tiles_n;

    if (threadIdx.x == 0) {
        for (int s = 0; s < P_STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 4); }
        *failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    auto tile_origin = [&](uint32_t tile, uint32_t &m0, uint32_t &n0) {
        const uint32_t group = tile / (GROUP_M * tiles_n), first_m = group * GROUP_M;
        const uint32_t rows_in_group = min((uint32_t)GROUP_M, tiles_m - first_m);
        const uint32_t in_group = tile - group * GROUP_M * tiles_n;
        m0 = (first_m + in_group % rows_in_group) * BM;
        n0 = (in_group / rows_in_group) * P_BN;
    };

    if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0, armed = 0;
            bool ok = true;
            const uint32_t withhold = blockIdx.x == 0 ? (uint32_t)g_withhold_step : 0xffffffffu;     // test hook: this stage is never loaded
            for (uint32_t tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
                uint32_t m0, n0;
                tile_origin(tile, m0, n0);
                for (uint32_t kb = 0; kb < num_k; ++kb, ++it) {
                    const uint32_t s = it % P_STAGES, ph = (it / P_STAGES) & 1;
                    if (it == withhold) { ok = false; break; }
                    if (*failed || !mbar_wait(&empty[s], ph ^ 1, failed)) { if (!*failed) { *failed = 1; atomicCAS(&g_gemm_tc_error, 0, (1 << 8) | (int)s); } ok = false; break; }
                    mbar_expect_tx(&full[s], STAGE_BYTES);
                    tma_load_2d(smem + s * STAGE_BYTES, &tmA, (int)(kb * BK), (int)m0, &full[s]);
                    tma_load_2d(smem + s * STAGE_BYTES + A_BYTES, &tmB, (int)(kb * BK), (int)n0, &full[s]);
                    armed = it + 1;
                }
            }
            if (*failed) {
                volatile uint32_t never = 0;
                for (uint32_t k = armed > P_STAGES ? armed - P_STAGES : 0; k < armed; ++k) mbar_wait(&full[k % P_STAGES], (k / P_STAGES) & 1, &never);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc(P_BN);
            uint32_t it = 0, lt = 0;
            bool ok = true;
            for (uint32_t tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++lt) {
                const uint32_t buf = lt & 1, use = lt >> 1;
                if (*failed || !mbar_wait(&acc_empty[buf], (use & 1) ^ 1, failed)) { if (!*failed) { *failed = 1; atomicCAS(&g_gemm_tc_error, 0, (2 << 8) | 0x80 | (int)buf); } break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t tacc = tmem_base + buf * P_BN;
                for (uint32_t kb = 0; kb < num_k; ++kb, ++it) {
                    const uint32_t s = it % P_STAGES, ph = (it / P_STAGES) & 1;
                    if (*failed || !mbar_wait(&full[s], ph, failed)) { if (!*failed) { *failed = 1; atomicCAS(&g_gemm_tc_error, 0, (2 << 8) | (int)s); } ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint64_t da = umma_desc(smem_u32(smem + s * STAGE_BYTES));
                    const uint64_t db = umma_desc(smem_u32(smem + s * STAGE_BYTES + A_BYTES));
#pragma unroll
                    for (uint32_t k = 0; k < BK / 16; ++k) umma(tacc, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
                    umma_commit(&empty[s]);
                }
                if (ok) umma_commit(&acc_full[buf]);
            }
        }
    } else {
        const uint32_t quarter = warp & 3;
        const bool vec = ((ldc | col0) & 3u) == 0 && (reinterpret_cast<uintptr_t>(C) & 15u) == 0;
        uint32_t lt = 0;
        for (uint32_t tile = blockIdx.x; tile < tiles; tile += gridDim.x, ++lt) {
            const uint32_t buf = lt & 1, use = lt >> 1;
            bool ready = !*failed && mbar_wait(&acc_full[buf], use & 1, failed);
            if (!ready && !*failed) { *failed = 1; atomicCAS(&g_gemm_tc_error, 0, 3 << 8); }
            ready = __all_sync(0xffffffffu, ready && !*failed);
            if (!ready) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            uint32_t m0, n0;
            tile_origin(tile, m0, n0);
            const uint32_t row = m0 + quarter * 32 + lane;
#pragma unroll 1
            for (uint32_t c = 0; c < P_BN / 32; ++c) {
                float v[32];
                tmem_ld32(tmem_base + ((quarter * 32) << 16) + buf * P_BN + c * 32, v);
                const uint32_t col = n0 + c * 32;
                if (row < M && col < n) {
                    float *dst = C + (size_t)row * ldc + col0 + col;
                    if (ep.aout) swiglu_store32(ep, (size_t)row * ldc + col0 + col, v, min(32u, n - col));
                    else if (vec && col + 32 <= n) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            float4 o = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                            if (accumulate) { const float4 old = *reinterpret_cast<const float4 *>(dst + j); o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w; }
                            *reinterpret_cast<float4 *>(dst + j) = o;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (col + j < n) dst[j] = accumulate ? dst[j] + v[j] : v[j];
                    }
                }
            }
            // this warp has read its quarter of the buffer: hand it back to the MMA warp
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&acc_empty[buf])) : "memory");
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    __syncthreads();
    if (warp == 2) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// ---- paired variant: one 256 x 256 tile per CTA pair (cta_group::2) -------------------------------------------------
// What limits the kernel above is not the tensor pipe but what an SM can pull from L2: 48 KB per 64-wide K block is
// 54 B per clock, and the MMA thread waits for data a third of the time.  Here the two CTAs of a cluster sit on the two
// SMs of a TPC and share one MMA of M = 256: each loads its own 128 rows of A and HALF of the 256 rows of W (B), 32 KB
// per K block for the same arithmetic per SM; a stage holds two K blocks (128 wide: half the barrier hand-overs of 64-wide
// stages, 4 % faster), three stages deep.  Only the even CTA (the leader) issues MMAs; the TMA loads
// of both CTAs count on the leader's `full` barrier; an MMA commit arrives on the `empty` / `acc_full` barriers of both
// CTAs; both CTAs drain their own 128 rows of the accumulator from their own TMEM and arrive (the odd one remotely) on
// the leader's `acc_empty`.  No multicast load anywhere.  Same bounded waits and error word; a cluster barrier before
// TMEM is freed keeps either CTA from leaving while its partner still works on its memory.
constexpr int Q_HALVES = 2, Q_STAGES = 6 / Q_HALVES;   // a stage holds Q_HALVES 64-wide K blocks

__global__ void __launch_bounds__(192, 1) tgp_matmul_tc_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                                                              float *__restrict__ C, uint32_t M, uint32_t n, uint32_t K, uint32_t ldc, uint32_t col0, int accumulate, const Epi ep) {
    extern __shared__ uint8_t smem_raw[];
    constexpr int A_BYTES = BM * BK * 2, B_BYTES = (P_BN / 2) * BK * 2, STAGE_BYTES = Q_HALVES * (A_BYTES + B_BYTES);
    constexpr int QK = Q_HALVES * BK;
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + Q_STAGES * STAGE_BYTES);      // used in the leader only
    uint64_t *empty = full + Q_STAGES;
    uint64_t *acc_full = empty + Q_STAGES;           // [2]
    uint64_t *acc_empty = acc_full + 2;              // [2], used in the leader only: 4 warps of each CTA
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(acc_empty + 2);
    volatile uint32_t *failed = tmem_slot + 1;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank(), pair = blockIdx.x >> 1, pairs = gridDim.x >> 1;
    const uint32_t num_k = (K + QK - 1) / QK;
    const uint32_t tiles_m = (M + 2 * BM - 1) / (2 * BM), tiles_n = (n + P_BN - 1) / P_BN, tiles = tiles_m * tiles_n;

    if (threadIdx.x == 0) {
        for (int s = 0; s < Q_STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 8); }
        *failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {                                  // the same warp in both CTAs of the pair
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    cluster_sync_all();                               // barriers of both CTAs initialised, TMEM allocated
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    auto tile_origin = [&](uint32_t tile, uint32_t &m0, uint32_t &n0) {       // of the pair's 256 x 256 tile
        const uint32_t group = tile / (GROUP_M * tiles_n), first_m = group * GROUP_M;
        const uint32_t rows_in_group = min((uint32_t)GROUP_M, tiles_m - first_m);
        const uint32_t in_group = tile - group * GROUP_M * tiles_n;
        m0 = (first_m + in_group % rows_in_group) * (2 * BM);
        n0 = (in_group / rows_in_group) * P_BN;
    };

    if (warp == 0) {
        if (lane == 0) {                              // TMA thread of this CTA: its rows of A, its half of B
            uint32_t it = 0, armed = 0;
            const uint32_t withhold = pair == 0 ? (uint32_t)g_withhold_step : 0xffffffffu;     // test hook: both CTAs of the first pair never load this stage
            for (uint32_t tile = pair; tile < tiles; tile += pairs) {
                uint32_t m0, n0;
                tile_origin(tile, m0, n0);
                bool ok = true;
                for (uint32_t kb = 0; kb < num_k; ++kb, ++it) {
                    const uint32_t s = it % Q_STAGES, ph = (it / Q_STAGES) & 1;
                    if (it == withhold) { ok = false; break; }
                    if (*failed || !mbar_wait(&empty[s], ph ^ 1, failed)) { if (!*failed) { *failed = 1; atomicCAS(&g_gemm_tc_error, 0, (1 << 8) | (int)s); } ok = false; break; }
                    if (rank == 0) mbar_expect_tx(&full[s], 2 * STAGE_BYTES);
#pragma unroll
                    for (int h = 0; h < Q_HALVES; ++h) {
                        tma_load_2d_pair(smem + s * STAGE_BYTES + h * (A_BYTES + B_BYTES), &tmA, (int)(kb * QK + h * BK), (int)(m0 + rank * BM), &full[s]);
                        tma_load_2d_pair(smem + s * STAGE_BYTES + h * (A_BYTES + B_BYTES) + A_BYTES, &tmB, (int)(kb * QK + h * BK), (int)(n0 + rank * (P_BN / 2)), &full[s]);
                    }
                    armed = it + 1;
                }
                if (!ok) break;
            }
            if (*failed && rank == 0) {               // loads of both CTAs still in flight land on these barriers (bounded wait)
                volatile uint32_t never = 0;
                for (uint32_t q = armed > Q_STAGES ? armed - Q_STAGES : 0; q < armed; ++q) mbar_wait(&full[q % Q_STAGES], (q / Q_STAGES) & 1, &never);
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {                 // MMA thread of the pair
            constexpr uint32_t idesc = umma_idesc_pair(P_BN);
            uint32_t it = 0, lt = 0;
            bool ok = true;
            for (uint32_t tile = pair; tile < tiles && ok; tile += pairs, ++lt) {
                const uint32_t buf = lt & 1, use = lt >> 1;
                if (*failed || !mbar_wait(&acc_empty[buf], (use & 1) ^ 1, failed)) { if (!*failed) { *failed = 1; atomicCAS(&g_gemm_tc_error, 0, (2 << 8) | 0x80 | (int)buf); } break; }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t tacc = tmem_base + buf * P_BN;
                for (uint32_t kb = 0; kb < num_k; ++kb, ++it) {
                    const uint32_t s = it % Q_STAGES, ph = (it / Q_STAGES) & 1;
                    if (*failed || !mbar_wait(&full[s], ph, failed)) { if (!*failed) { *failed = 1; atomicCAS(&g_gemm_tc_error, 0, (2 << 8) | (int)s); } ok = false; break; }
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                    for (uint32_t h = 0; h < Q_HALVES; ++h) {
                        const uint64_t da = umma_desc(smem_u32(smem + s * STAGE_BYTES + h * (A_BYTES + B_BYTES)));
                        const uint64_t db = umma_desc(smem_u32(smem + s * STAGE_BYTES + h * (A_BYTES + B_BYTES) + A_BYTES));
#pragma unroll
                        for (uint32_t k = 0; k < BK / 16; ++k) umma_pair(tacc, da + 2 * k, db + 2 * k, idesc, (kb | h | k) != 0);
                    }
                    umma_commit_pair(&empty[s]);
                }
                if (ok) umma_commit_pair(&acc_full[buf]);
            }
        }
    } else {
        const uint32_t quarter = warp & 3;
        const bool vec = ((ldc | col0) & 3u) == 0 && (reinterpret_cast<uintptr_t>(C) & 15u) == 0;
        uint32_t lt = 0;
        for (uint32_t tile = pair; tile < tiles; tile += pairs, ++lt) {
            const uint32_t buf = lt & 1, use = lt >> 1;
            bool ready = !*failed && mbar_wait(&acc_full[buf], use & 1, failed);
            if (!ready && !*failed) { *failed = 1; atomicCAS(&g_gemm_tc_error, 0, 3 << 8); }
            ready = __all_sync(0xffffffffu, ready && !*failed);
            if (!ready) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            uint32_t m0, n0;
            tile_origin(tile, m0, n0);
            const uint32_t row = m0 + rank * BM + quarter * 32 + lane;
#pragma unroll 1
            for (uint32_t c = 0; c < P_BN / 32; ++c) {
                float v[32];
                tmem_ld32(tmem_base + ((quarter * 32) << 16) + buf * P_BN + c * 32, v);
                const uint32_t col = n0 + c * 32;
                if (row < M && col < n) {
                    float *dst = C + (size_t)row * ldc + col0 + col;
                    if (ep.aout) swiglu_store32(ep, (size_t)row * ldc + col0 + col, v, min(32u, n - col));
                    else if (vec && col + 32 <= n) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            float4 o = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                            if (accumulate) { const float4 old = *reinterpret_cast<const float4 *>(dst + j); o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w; }
                            *reinterpret_cast<float4 *>(dst + j) = o;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (col + j < n) dst[j] = accumulate ? dst[j] + v[j] : v[j];
                    }
                }
            }
            // this warp has read its quarter of this CTA's half of the buffer: tell the pair's MMA thread
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(&acc_empty[buf], 0);
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    cluster_sync_all();                               // neither CTA frees TMEM or leaves while its partner may still touch it
    if (warp == 2) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// 2-D bf16 row-major [rows, K] map with a [box_rows, 64] box, 128-byte swizzle, zero fill outside.
bool make_map(CUtensorMap *map, const void *base, uint64_t rows, uint64_t K, uint32_t box_rows) {
    static_assert(BK == 64, "the shared tensor-map helper encodes 64-element boxes");
    return tensor_map_bf16_2d(map, base, rows, K, K * 2, box_rows);
}

}  // namespace

extern thread_local uint64_t tgpk_launches;

template <int BN, int ST, int KH, bool SWAP = false>
static bool launch_tile(const CUtensorMap &ma, const CUtensorMap &mb, float *C, uint32_t M, uint32_t n, uint32_t K, uint32_t ldc, uint32_t col0, int accumulate, cudaStream_t st, const Epi ep = Epi{nullptr, nullptr}) {
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(tgp_matmul_tc_kernel<BN, ST, KH, SWAP>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem<BN, ST, KH>::TOTAL) != cudaSuccess) return false;
        attr_set = true;
    }
    dim3 grid(((M + BM - 1) / BM) * ((n + BN - 1) / BN));
    tgp_matmul_tc_kernel<BN, ST, KH, SWAP><<<grid, 192, Smem<BN, ST, KH>::TOTAL, st>>>(ma, mb, C, M, n, K, ldc, col0, accumulate, ep);
    return true;
}

static int g_tc_variant = 0;     // 0 auto, 1 force the 128x128 per-tile kernel, 2 the persistent 128x256 kernel, 3 the paired 256x256 kernel,
                                 // 4 the per-tile kernel with the weights as the 128-row operand (M <= 128 only; else as 0)

int tgpk_gemm_tc(const void *A, const void *W, float *C, uint32_t M, uint32_t n, uint32_t K, uint32_t ldc, uint32_t col0, int accumulate, cudaStream_t st,
                 const float *gate, void *aout) {
    constexpr int BN = 128;
    const Epi ep{aout ? gate : nullptr, gate ? (__nv_bfloat16 *)aout : nullptr};
    if (ep.aout && accumulate) return TGP_E_INVAL;
    if ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(W)) & 15u) return TGP_E_INVAL;     // TMA needs 16-byte aligned bases
    if (K % 8) return TGP_E_INVAL;                                                                       // and 16-byte row strides
    static int sms = 0;
    if (!sms) { int dev = 0; cudaGetDevice(&dev); if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) sms = 148; }
    // Up to 64 activation rows on a block with 128-row tiles for a good part of the SMs: the weights become the 128-row
    // operand (see tgp_matmul_tc_kernel), the activations the narrow one.  A CTA takes in about 100 GB/s through its TMA ring
    // whatever the tile, so the form pays from 64 weight tiles on (n=8192, K=8192, M=64: 34 us against 47 us), for more
    // than 32 rows from 32 tiles on (n=4096, K=14336, M=64: 48 us against 70 us); with fewer tiles the weight-streaming
    // kernels and the narrow tiles below have more CTAs at work
    const uint32_t w_tiles = (n + BM - 1) / BM;
    if (!ep.aout && M <= 128 && (g_tc_variant == 4 || (g_tc_variant == 0 && M <= 64 && (w_tiles >= 64 || (M > 32 && w_tiles >= 32))))) {
        CUtensorMap mw, mx;
        const uint32_t bx = M <= 32 ? 32 : M <= 64 ? 64 : 128;
        if (!make_map(&mw, W, n, K, BM) || !make_map(&mx, A, M, K, bx)) return TGP_E_CUDA;
        const bool ok = bx == 32 ? launch_tile<32, 3, 3, true>(mw, mx, C, n, M, K, ldc, col0, accumulate, st)
                      : bx == 64 ? launch_tile<64, 3, 3, true>(mw, mx, C, n, M, K, ldc, col0, accumulate, st)
                                 : launch_tile<128, 2, 3, true>(mw, mx, C, n, M, K, ldc, col0, accumulate, st);
        if (!ok || cudaGetLastError() != cudaSuccess) return TGP_E_CUDA;
        tgpk_launches += 1;
        tgpk_last_gemm_kernel = "tgp_matmul_tc_kernel (weights as the 128-row operand)";
        return TGP_OK;
    }
    const uint32_t tiles_p = ((M + BM - 1) / BM) * ((n + P_BN - 1) / P_BN);
    const uint32_t tiles_q = ((M + 2 * BM - 1) / (2 * BM)) * ((n + P_BN - 1) / P_BN);
    // measured on 8192 x {640 .. 4096} x {4096, 14336}, {1024 .. 4096} x 4096 x 4096 and {512, 1024} x 8192 x 2048: the paired
    // kernel is ahead as soon as every pair of SMs has a 256 x 256 tile, the persistent one from about 64 tiles of 128 x 256
    const bool paired = g_tc_variant == 3 || (g_tc_variant == 0 && 2 * tiles_q >= (uint32_t)sms);
    const bool persistent = !paired && (g_tc_variant == 2 || (g_tc_variant == 0 && tiles_p >= 64u));
    // small problems, one tile per CTA: an MMA into one accumulator costs the same 75 cycles for N = 32 as for N = 128, so
    // a CTA's time is set by its K loop, and narrower tiles simply put more CTAs to work: the widest tile that still
    // gives every SM one
    const uint32_t tm = (M + BM - 1) / BM;
    uint32_t bn = BN;
    // ... as long as the A panel is not re-read by more than 32 column tiles (L2 bandwidth then takes over)
    if (g_tc_variant == 0) while (bn > 32 && tm * ((n + bn - 1) / bn) < (uint32_t)sms && (n + bn / 2 - 1) / (bn / 2) <= 32) bn /= 2;
    CUtensorMap ma, mb;
    if (!make_map(&ma, A, M, K, BM) || !make_map(&mb, W, n, K, paired ? P_BN / 2 : persistent ? P_BN : bn)) return TGP_E_CUDA;
    if (paired) {
        constexpr int SMEM = Q_STAGES * Q_HALVES * (BM * BK * 2 + (P_BN / 2) * BK * 2) + 160 + 1024;
        static bool attr_q = false;
        if (!attr_q) {
            if (cudaFuncSetAttribute(tgp_matmul_tc_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM) != cudaSuccess) return TGP_E_CUDA;
            attr_q = true;
        }
        const uint32_t pairs_max = (uint32_t)sms / 2, npairs = tiles_q < pairs_max ? tiles_q : pairs_max;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * npairs);
        cfg.blockDim = dim3(192);
        cfg.dynamicSmemBytes = SMEM;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, tgp_matmul_tc_pair_kernel, ma, mb, C, M, n, K, ldc, col0, accumulate, ep) != cudaSuccess) return TGP_E_CUDA;
    } else if (persistent) {
        constexpr int SMEM = P_STAGES * (BM * BK * 2 + P_BN * BK * 2) + 128 + 1024;
        static bool attr_p = false;
        if (!attr_p) {
            if (cudaFuncSetAttribute(tgp_matmul_tc_persistent_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM) != cudaSuccess) return TGP_E_CUDA;
            attr_p = true;
        }
        tgp_matmul_tc_persistent_kernel<<<tiles_p < (uint32_t)sms ? tiles_p : (uint32_t)sms, 192, SMEM, st>>>(ma, mb, C, M, n, K, ldc, col0, accumulate, ep);
    } else if (bn == 128) {
        // fewer tiles than SMs: one CTA per SM, so the ring may take all of shared memory (a 3-stage ring leaves a lone
        // CTA waiting on L2 latency); otherwise two CTAs per SM with three stages each
        const bool lone = tm * ((n + 127) / 128) <= (uint32_t)sms;
        if (!(lone ? launch_tile<128, 2, 3>(ma, mb, C, M, n, K, ldc, col0, accumulate, st, ep) : launch_tile<128, 3, 1>(ma, mb, C, M, n, K, ldc, col0, accumulate, st, ep))) return TGP_E_CUDA;
    } else if (bn == 64) {
        if (!launch_tile<64, 3, 3>(ma, mb, C, M, n, K, ldc, col0, accumulate, st, ep)) return TGP_E_CUDA;
    } else {
        if (!launch_tile<32, 3, 3>(ma, mb, C, M, n, K, ldc, col0, accumulate, st, ep)) return TGP_E_CUDA;
    }
    if (cudaGetLastError() != cudaSuccess) return TGP_E_CUDA;
    tgpk_launches += 1;
    tgpk_last_gemm_kernel = paired ? "tgp_matmul_tc_pair_kernel" : persistent ? "tgp_matmul_tc_persistent_kernel" : "tgp_matmul_tc_kernel";
    return TGP_OK;
}

extern "C" int tgp_k_gemm_tc_variant(int v) {
    if (v < 0 || v > 4) return TGP_E_INVAL;
    g_tc_variant = v;
    return TGP_OK;
}

int tgpk_gemm_wait_test(unsigned long long limit_ns, int withhold_step) {
    if (cudaMemcpyToSymbol(g_wait_limit_ns, &limit_ns, sizeof(limit_ns)) != cudaSuccess) return TGP_E_CUDA;
    return cudaMemcpyToSymbol(g_withhold_step, &withhold_step, sizeof(withhold_step)) == cudaSuccess ? TGP_OK : TGP_E_CUDA;
}

int tgpk_gemm_status_clear() { const int z = 0; return cudaMemcpyToSymbol(g_gemm_tc_error, &z, sizeof(z)) == cudaSuccess ? TGP_OK : TGP_E_CUDA; }

extern "C" int tgp_k_gemm_status(int *error_code) {
    if (!error_code) return TGP_E_INVAL;
    if (cudaMemcpyFromSymbol(error_code, g_gemm_tc_error, sizeof(int)) != cudaSuccess) return TGP_E_CUDA;
    return TGP_OK;
}
