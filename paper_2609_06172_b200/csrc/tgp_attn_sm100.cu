// Causal GQA attention for prefill on the 5th-generation tensor cores (sm_100a).
//
// One CTA of 128 threads owns 128 consecutive queries of one (sequence, query head); thread t is query row t and
// TMEM lane t.  K and V blocks of 64 keys are staged by cp.async (16-byte chunks, two stages each) as 64-wide
// head-dimension blocks of [64 keys x 128 B] with the 128-byte swizzle; K is then a K-major operand (head dimension
// contiguous) and V, in the very same layout, an MN-major operand (its contiguous dimension is the output dimension
// of P V).  TMEM holds S (64 columns) and the output accumulator O (Dh columns), which the tensor core accumulates
// over all key blocks.  Per block j:
//   1. wait for S_j; read this thread's row of it into registers;
//   2. K_{j+1} has landed (requested a whole block earlier): one thread issues S_{j+1} = Q K_{j+1}^T, which the
//      tensor core computes while the CUDA cores do steps 3-4;
//   3. row max of the scaled, masked scores.  The exponent reference m only moves when some row of the warp exceeds
//      it by more than 8 (in log2 units): then, once P V of block j-1 has completed, the warp multiplies its 32 rows
//      of O in TMEM and its running sums by 2^(m_old - m_new).  Otherwise P may reach 2^8, which fp32 sums and bf16 P
//      hold without loss, and O is not touched by the CUDA cores at all;
//   4. P = exp2(S - m) as bf16 into a K-major shared tile (free once P V of block j-1 has completed);
//   5. one thread issues O += P V_j.
// At the end every thread reads its row of O once, divides by its sum and stores bf16.
// Two CTAs fit on an SM (112 KB of shared memory, 256 TMEM columns each) and fill each other's barrier waits.
// P is rounded to bf16 for the second product (the one rounding of this path the CPU oracle does not mirror).
// Every mbarrier wait is bounded; a wait that runs out sets an error word and the CTA leaves without storing.
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cstdint>
#include "tgp.h"
#include "tgp_kernels.h"
#include "tgp_sm100.cuh"

namespace {

using namespace tgp_sm100;
typedef __nv_bfloat16 bf16;
constexpr int BQ = 128, BKV = 64;

__device__ int g_attn_tc_error = 0;                     // 0 ok; 1 / 2: the wait for S / for P V ran out; 3: shared memory base not 1024-byte aligned

struct TArgs {
    const bf16 *qb; bf16 *ob;
    uint32_t Hq, Hkv, TK, q_len, pos0;
    float scale_log2;
    TgpTilePtrs tiles;
};

__device__ __forceinline__ void cp_async16z(uint32_t dst, const void *src, bool valid) {
    const uint32_t n = valid ? 16u : 0u;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}

// MN-major operand in the same swizzled storage: 64 contiguous elements (128 B) of the MN dimension per row, rows are
// K; the next 64 MN elements start `lbo` bytes further (leading byte offset), the next 8 K rows 1024 bytes further.
__device__ __forceinline__ uint64_t umma_desc_mn(uint32_t smem_addr, uint32_t lbo) {
    return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}

// byte offset of 16-byte chunk c (0..7) of row r inside a [rows x 128 B] K-major tile with 128-byte swizzle
__device__ __forceinline__ uint32_t sw128(uint32_t r, uint32_t c) { return r * 128u + ((c ^ (r & 7u)) << 4); }

__device__ __forceinline__ float ex2(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// at most two of this thread's copy groups still in flight; what landed is made visible to the tensor core
__device__ __forceinline__ void cp_wait2() {
    asm volatile("cp.async.wait_group 2;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

template <int DH>
__global__ void __launch_bounds__(128, 2) attn_prefill_tc_kernel(TArgs a) {
    extern __shared__ __align__(1024) uint8_t smem[];
    constexpr int KB = DH / 64;                          // 64-wide blocks of the head dimension
    constexpr int Q_BYTES = KB * BQ * 128, KV_BYTES = KB * BKV * 128, P_BYTES = BQ * 128;
    uint8_t *Qs = smem, *Ks = Qs + Q_BYTES, *Vs = Ks + 2 * KV_BYTES, *Ps = Vs + 2 * KV_BYTES;      // K and V: two stages each
    uint64_t *bar_s = reinterpret_cast<uint64_t *>(Ps + P_BYTES);
    uint64_t *bar_o = bar_s + 1;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bar_o + 1);
    volatile uint32_t *failed = tmem_slot + 1;

    const uint32_t tid = threadIdx.x, warp = tid >> 5;
    if (smem_u32(smem) & 1023u) {                            // the swizzle below assumes 1024-byte aligned tiles
        if (tid == 0) atomicCAS(&g_attn_tc_error, 0, 3);
        return;
    }
    const uint32_t qblk = blockIdx.x, hq = blockIdx.y, b = blockIdx.z, hk = hq / (a.Hq / a.Hkv);
    const uint32_t q0 = qblk * BQ, kvlen = a.pos0 + a.q_len;
    const uint32_t last_q = min(a.q_len, q0 + BQ) - 1;
    const uint32_t nblk = (a.pos0 + last_q + 1 + BKV - 1) / BKV;
    const bool row_ok = q0 + tid < a.q_len;
    const uint32_t qpos = a.pos0 + min(q0 + tid, a.q_len - 1);      // padding rows take the last query's mask

    if (tid == 0) {
        mbar_init(bar_s, 1);
        mbar_init(bar_o, 1);
        *failed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(256u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    auto stage = [&](uint8_t *dst, void *const *tiles, uint32_t jb) {      // one [64 keys x DH] block, 64-wide dh blocks
        const uint32_t j0 = jb * BKV;
        if (a.TK % BKV == 0) {                                               // the block lies inside one KV tile
            const bf16 *base = reinterpret_cast<const bf16 *>(tiles[j0 / a.TK]) + ((size_t)(b * a.Hkv + hk) * a.TK + j0 % a.TK) * DH;
            for (uint32_t i = tid; i < BKV * (DH / 8); i += 128) {
                const uint32_t r = i / (DH / 8), c = i % (DH / 8);
                const bool ok = j0 + r < kvlen;
                cp_async16z(smem_u32(dst + (c / 8) * (BKV * 128) + sw128(r, c % 8)), base + (ok ? r * DH + c * 8 : 0), ok);
            }
        } else {
            for (uint32_t i = tid; i < BKV * (DH / 8); i += 128) {
                const uint32_t r = i / (DH / 8), c = i % (DH / 8), j = j0 + r;
                const bool ok = j < kvlen;
                const uint32_t jj = ok ? j : 0;
                const bf16 *src = reinterpret_cast<const bf16 *>(tiles[jj / a.TK]) + ((size_t)(b * a.Hkv + hk) * a.TK + jj % a.TK) * DH + c * 8;
                cp_async16z(smem_u32(dst + (c / 8) * (BKV * 128) + sw128(r, c % 8)), src, ok);
            }
        }
    };
    // ---- copy groups, in the order the loop below retires them: {Q, K_0}, {K_1}, {V_0} ----
    for (uint32_t i = tid; i < BQ * (DH / 8); i += 128) {                   // Q tile: [128 rows x DH], rows past q_len zero
        const uint32_t r = i / (DH / 8), c = i % (DH / 8), p = q0 + r;
        const bool ok = p < a.q_len;
        const bf16 *src = a.qb + ((size_t)(b * a.q_len + (ok ? p : 0)) * a.Hq + hq) * DH + c * 8;
        cp_async16z(smem_u32(Qs + (c / 8) * (BQ * 128) + sw128(r, c % 8)), src, ok);
    }
    stage(Ks, a.tiles.k, 0);
    cp_commit();
    if (1 < nblk) stage(Ks + KV_BYTES, a.tiles.k, 1);
    cp_commit();
    stage(Vs, a.tiles.v, 0);
    cp_commit();
    cp_wait2();                                                             // Q and K_0 have landed
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_S = tmem_base, tmem_O = tmem_base + 64;
    const uint32_t lane_addr = (warp * 32u) << 16;          // this warp's quarter of the TMEM lanes
    constexpr uint32_t idesc_s = umma_idesc(BKV), idesc_o = umma_idesc(DH) | (1u << 16);     // bit 16: B operand is MN-major

    auto issue_s = [&](uint32_t jb) {                        // S = Q K_jb^T
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint8_t *Kj = Ks + (jb & 1) * KV_BYTES;
#pragma unroll
        for (uint32_t kb = 0; kb < KB; ++kb) {
            const uint64_t dq = umma_desc(smem_u32(Qs + kb * (BQ * 128))), dk = umma_desc(smem_u32(Kj + kb * (BKV * 128)));
#pragma unroll
            for (uint32_t k = 0; k < 4; ++k) umma(tmem_S, dq + 2 * k, dk + 2 * k, idesc_s, (kb | k) != 0);
        }
        umma_commit(bar_s);
    };
    if (tid == 0) issue_s(0);
    float m_ref = -INFINITY, lrow = 0.f;                     // exponent reference and running sum of this row

    for (uint32_t jb = 0; jb < nblk; ++jb) {
        // ---- 1. S_jb (issued during the previous block, or in the prologue) ----
        bool ok = mbar_wait(bar_s, jb & 1, failed);
        if (!ok && !*failed) { *failed = 1; atomicCAS(&g_attn_tc_error, 0, 1); }
        ok = __all_sync(0xffffffffu, ok);
        if (ok && jb + 2 < nblk) stage(Ks + (jb & 1) * KV_BYTES, a.tiles.k, jb + 2);     // the tensor core is done with K_jb
        cp_commit();
        float s[BKV];
        if (ok) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            tmem_ld32(tmem_S + lane_addr, s);
            tmem_ld32(tmem_S + lane_addr + 32, s + 32);
        }
        // ---- 2. K_jb+1 has landed, S is free again: the next S runs behind this block's softmax ----
        cp_wait2();
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        if (warp == 0) {
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (tid == 0 && jb + 1 < nblk && !*failed) issue_s(jb + 1);
        } else {
            asm volatile("bar.arrive 1, 128;" ::: "memory");
        }
        // ---- 3. row max; the exponent reference moves only when it has to ----
        if (jb * BKV + BKV - 1 > a.pos0 + q0) {                              // this block crosses the diagonal of some row
#pragma unroll
            for (uint32_t i = 0; i < BKV; ++i)
                if (jb * BKV + i > qpos) s[i] = -INFINITY;
        }
        float mblk = s[0];
#pragma unroll
        for (uint32_t i = 1; i < BKV; ++i) mblk = fmaxf(mblk, s[i]);
        mblk *= a.scale_log2;                                                // scale > 0: max commutes with it
        if (jb > 0) {
            bool ok2 = mbar_wait(bar_o, (jb - 1) & 1, failed);               // P V of the previous block: O, P and its V stage are free
            if (!ok2 && !*failed) { *failed = 1; atomicCAS(&g_attn_tc_error, 0, 2); }
            ok = __all_sync(0xffffffffu, ok && ok2);
        }
        if (ok && jb + 1 < nblk) stage(Vs + ((jb + 1) & 1) * KV_BYTES, a.tiles.v, jb + 1);
        cp_commit();
        if (jb == 0) {
            m_ref = mblk;                                                    // block 0 holds key 0 <= qpos: finite
        } else if (__any_sync(0xffffffffu, mblk > m_ref + 8.f) && ok) {
            const float m_new = fmaxf(m_ref, mblk), alpha = ex2(m_ref - m_new);
            m_ref = m_new;
            lrow *= alpha;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
            for (uint32_t h = 0; h < DH / 32; ++h) {
                float v[32];
                tmem_ld32(tmem_O + lane_addr + h * 32, v);
#pragma unroll
                for (uint32_t i = 0; i < 32; ++i) v[i] *= alpha;
                tmem_st32(tmem_O + lane_addr + h * 32, v);
            }
            tmem_wait_st();
        }
        // ---- 4. P = exp2(S * scale - m) as bf16, this thread's row of the K-major tile ----
        if (ok) {
            const float nm = -m_ref;
            float lsum = 0.f;
#pragma unroll
            for (uint32_t c = 0; c < BKV / 8; ++c) {
                uint32_t w[4];
#pragma unroll
                for (uint32_t i = 0; i < 4; ++i) {
                    const float p0 = ex2(fmaf(s[c * 8 + 2 * i], a.scale_log2, nm));      // a masked score is -inf: p = 0
                    const float p1 = ex2(fmaf(s[c * 8 + 2 * i + 1], a.scale_log2, nm));
                    lsum += p0 + p1;
                    __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
                    w[i] = *reinterpret_cast<uint32_t *>(&pk);
                }
                *reinterpret_cast<uint4 *>(Ps + sw128(tid, c)) = make_uint4(w[0], w[1], w[2], w[3]);
            }
            lrow += lsum;
        }
        cp_wait2();                                                          // V_jb has landed
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();                                                     // P complete, O rescaled where needed
        if (*failed) break;
        // ---- 5. O += P V_jb ----
        if (tid == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint64_t dp = umma_desc(smem_u32(Ps)), dv = umma_desc_mn(smem_u32(Vs + (jb & 1) * KV_BYTES), BKV * 128);
#pragma unroll
            for (uint32_t k = 0; k < 4; ++k) umma(tmem_O, dp + 2 * k, dv + 128 * k, idesc_o, (jb | k) != 0);   // 16 keys = 2048 B of V rows per step
            umma_commit(bar_o);
        }
    }
    // ---- the last P V; normalise and store this thread's row ----
    bool ok = !*failed && mbar_wait(bar_o, (nblk - 1) & 1, failed);
    if (!ok && !*failed) { *failed = 1; atomicCAS(&g_attn_tc_error, 0, 2); }
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const float inv = 1.0f / lrow;
        bf16 *dst = a.ob + ((size_t)(b * a.q_len + q0 + tid) * a.Hq + hq) * DH;
#pragma unroll
        for (uint32_t h = 0; h < DH / 32; ++h) {
            float v[32];
            tmem_ld32(tmem_O + lane_addr + h * 32, v);
            if (row_ok) {
#pragma unroll
                for (uint32_t c = 0; c < 4; ++c) {
                    uint32_t w[4];
#pragma unroll
                    for (uint32_t i = 0; i < 4; ++i) {
                        __nv_bfloat162 pk = __floats2bfloat162_rn(v[c * 8 + 2 * i] * inv, v[c * 8 + 2 * i + 1] * inv);
                        w[i] = *reinterpret_cast<uint32_t *>(&pk);
                    }
                    *reinterpret_cast<uint4 *>(dst + h * 32 + c * 8) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
        }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u) : "memory");
    }
}

template <int DH> constexpr int smem_bytes() { return (DH / 64) * (BQ + 4 * BKV) * 128 + BQ * 128 + 64; }

}  // namespace

extern thread_local uint64_t tgpk_launches;

int tgpk_attn_prefill_tc5(const void *qb, const TgpTilePtrs &tiles, void *ob, const tgp_model_cfg *c, uint32_t B, uint32_t q_len, uint32_t pos0, cudaStream_t st) {
    TArgs a{(const bf16 *)qb, (bf16 *)ob, c->Hq, c->Hkv, c->TK, q_len, pos0, 1.4426950408889634f / sqrtf((float)c->Dh), tiles};
    dim3 grid((q_len + BQ - 1) / BQ, c->Hq, B);
    static bool attr64 = false, attr128 = false;
    if (c->Dh == 64) {
        if (!attr64) { if (cudaFuncSetAttribute(attn_prefill_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<64>()) != cudaSuccess) return TGP_E_CUDA; cudaFuncSetAttribute(attn_prefill_tc_kernel<64>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared); attr64 = true; }
        attn_prefill_tc_kernel<64><<<grid, 128, smem_bytes<64>(), st>>>(a);
    } else if (c->Dh == 128) {
        if (!attr128) { if (cudaFuncSetAttribute(attn_prefill_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<128>()) != cudaSuccess) return TGP_E_CUDA; cudaFuncSetAttribute(attn_prefill_tc_kernel<128>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared); attr128 = true; }
        attn_prefill_tc_kernel<128><<<grid, 128, smem_bytes<128>(), st>>>(a);
    } else {
        return TGP_E_INVAL;
    }
    if (cudaGetLastError() != cudaSuccess) return TGP_E_CUDA;
    tgpk_launches += 1;
    return TGP_OK;
}

extern "C" int tgp_k_attn_status(int *error_code) {
    if (!error_code) return TGP_E_INVAL;
    if (cudaMemcpyFromSymbol(error_code, g_attn_tc_error, sizeof(int)) != cudaSuccess) return TGP_E_CUDA;
    return TGP_OK;
}
