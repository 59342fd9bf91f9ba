// Causal GQA attention for prefill on the 5th-generation tensor cores (sm_100a).
//
// One CTA of 128 threads owns 128 consecutive queries of one (sequence, query head); thread t is query row t and
// TMEM lane t.  For every block of 64 keys:
//   1. all threads stage K and V (cp.async, 16-byte chunks) into shared memory as 64-wide head-dimension blocks of
//      [64 keys x 128 B] with the 128-byte swizzle; K is then a K-major operand (head dimension contiguous) and V,
//      in the very same layout, an MN-major operand (its contiguous dimension is the output dimension of P V);
//      the next block's K is requested as soon as S has been computed, the next V as soon as O_j has;
//   2. one thread issues S = Q K^T (M=128, N=64) into TMEM and commits to an mbarrier (for block j+1 this happens
//      right behind step 4 of block j, so that its latency hides behind step 5);
//   3. every thread reads its row of S from TMEM, applies scale and causal mask, updates its running max / sum and
//      writes P = exp2(S - max) as bf16 into a K-major shared tile;
//   4. one thread issues O_j = P V_j (M=128, N=Dh) into a second TMEM accumulator;
//   5. every thread reads its row of O_j and folds it into its register accumulator: o = o * alpha + O_j.
// The accumulator over key blocks stays in registers, so TMEM is only ever written by the tensor core.  Two CTAs fit
// on an SM (80 KB of shared memory, 256 TMEM columns each) and overlap one's softmax with the other's MMAs.
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

__device__ int g_attn_tc_error = 0;                     // 0 ok; else the phase (1 S wait, 2 O wait) of the first wait that ran out

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

template <int DH>
__global__ void __launch_bounds__(128, 2) attn_prefill_tc_kernel(TArgs a) {
    extern __shared__ uint8_t smem_raw[];
    constexpr int KB = DH / 64;                          // 64-wide blocks of the head dimension
    constexpr int Q_BYTES = KB * BQ * 128, K_BYTES = KB * BKV * 128, V_BYTES = KB * BKV * 128, P_BYTES = BQ * 128;
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t *Qs = smem, *Ks = Qs + Q_BYTES, *Vs = Ks + K_BYTES, *Ps = Vs + V_BYTES;
    uint64_t *bar_s = reinterpret_cast<uint64_t *>(Ps + P_BYTES);
    uint64_t *bar_o = bar_s + 1;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bar_o + 1);
    volatile uint32_t *failed = tmem_slot + 1;

    const uint32_t tid = threadIdx.x, warp = tid >> 5;
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
    // ---- Q tile: [128 rows x DH], rows past q_len zero ----
    for (uint32_t i = tid; i < BQ * (DH / 8); i += 128) {
        const uint32_t r = i / (DH / 8), c = i % (DH / 8), p = q0 + r;
        const bool ok = p < a.q_len;
        const bf16 *src = a.qb + ((size_t)(b * a.q_len + (ok ? p : 0)) * a.Hq + hq) * DH + c * 8;
        cp_async16z(smem_u32(Qs + (c / 8) * (BQ * 128) + sw128(r, c % 8)), src, ok);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_S = tmem_base, tmem_O = tmem_base + 64;
    const uint32_t lane_addr = (warp * 32u) << 16;          // this warp's quarter of the TMEM lanes

    float o[DH];
#pragma unroll
    for (int i = 0; i < DH; ++i) o[i] = 0.f;
    float mrow = -INFINITY, lrow = 0.f;
    constexpr uint32_t idesc_s = umma_idesc(BKV), idesc_o = umma_idesc(DH) | (1u << 16);     // bit 16: B operand is MN-major

    auto stage = [&](uint8_t *dst, void *const *tiles, uint32_t jb) {      // one [64 keys x DH] block, 64-wide dh blocks
        for (uint32_t i = tid; i < BKV * (DH / 8); i += 128) {
            const uint32_t r = i / (DH / 8), c = i % (DH / 8), j = jb * BKV + r;
            const bool ok = j < kvlen;
            const uint32_t jj = ok ? j : 0;
            const bf16 *src = reinterpret_cast<const bf16 *>(tiles[jj / a.TK]) + ((size_t)(b * a.Hkv + hk) * a.TK + jj % a.TK) * DH + c * 8;
            cp_async16z(smem_u32(dst + (c / 8) * (BKV * 128) + sw128(r, c % 8)), src, ok);
        }
    };
    stage(Ks, a.tiles.k, 0);
    stage(Vs, a.tiles.v, 0);

    auto issue_s = [&]() {                                   // S = Q K^T for the K block now in shared memory
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
        for (uint32_t kb = 0; kb < KB; ++kb) {
            const uint64_t dq = umma_desc(smem_u32(Qs + kb * (BQ * 128))), dk = umma_desc(smem_u32(Ks + kb * (BKV * 128)));
#pragma unroll
            for (uint32_t k = 0; k < 4; ++k) umma(tmem_S, dq + 2 * k, dk + 2 * k, idesc_s, (kb | k) != 0);
        }
        umma_commit(bar_s);
    };
    // ---- prologue: Q, K_0, V_0 have landed; S_0 is issued ----
    asm volatile("cp.async.wait_all;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");            // generic-proxy writes -> visible to the tensor core
    __syncthreads();
    if (tid == 0) issue_s();

    for (uint32_t jb = 0; jb < nblk; ++jb) {
        // (S_jb was issued one step ahead: behind P V of the previous block, or in the prologue)
        // ---- 3. softmax on this thread's row ----
        bool ok = mbar_wait(bar_s, jb & 1, failed);
        if (!ok && !*failed) { *failed = 1; atomicCAS(&g_attn_tc_error, 0, 1); }
        ok = __all_sync(0xffffffffu, ok);
        if (ok && jb + 1 < nblk) stage(Ks, a.tiles.k, jb + 1);            // the tensor core is done with K_j
        float alpha = 1.f;
        if (ok) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            float s[32];
            float mnew = mrow;
#pragma unroll
            for (uint32_t h = 0; h < 2; ++h) {
                tmem_ld32(tmem_S + lane_addr + h * 32, s);
#pragma unroll
                for (uint32_t i = 0; i < 32; ++i) {
                    const uint32_t key = jb * BKV + h * 32 + i;
                    if (key <= qpos) mnew = fmaxf(mnew, s[i] * a.scale_log2);
                }
            }
            alpha = exp2f(mrow - mnew);                    // block 0 always holds key 0 <= qpos, so mnew is finite
            mrow = mnew;
            float lsum = 0.f;
#pragma unroll
            for (uint32_t h = 0; h < 2; ++h) {
                tmem_ld32(tmem_S + lane_addr + h * 32, s);
#pragma unroll
                for (uint32_t c = 0; c < 4; ++c) {
                    uint32_t w[4];
#pragma unroll
                    for (uint32_t i = 0; i < 4; ++i) {
                        const uint32_t k0 = h * 32 + c * 8 + 2 * i, key = jb * BKV + k0;
                        const float p0 = key <= qpos ? exp2f(s[c * 8 + 2 * i] * a.scale_log2 - mnew) : 0.f;
                        const float p1 = key + 1 <= qpos ? exp2f(s[c * 8 + 2 * i + 1] * a.scale_log2 - mnew) : 0.f;
                        lsum += p0 + p1;
                        __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
                        w[i] = *reinterpret_cast<uint32_t *>(&pk);
                    }
                    *reinterpret_cast<uint4 *>(Ps + sw128(tid, h * 4 + c)) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
            lrow = lrow * alpha + lsum;
        }
        asm volatile("cp.async.wait_all;" ::: "memory");                     // V_jb and the prefetched K_jb+1 have landed
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();                                                     // every thread has read S_jb and written its row of P
        if (*failed) break;
        // ---- 4. O_j = P V_j, and right behind it S of the next block (its accumulator is free again) ----
        if (tid == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint64_t dp = umma_desc(smem_u32(Ps)), dv = umma_desc_mn(smem_u32(Vs), BKV * 128);
#pragma unroll
            for (uint32_t k = 0; k < 4; ++k) umma(tmem_O, dp + 2 * k, dv + 128 * k, idesc_o, k != 0);   // 16 keys = 2048 B of V rows per step
            umma_commit(bar_o);
            if (jb + 1 < nblk) issue_s();
        }
        // ---- 5. fold O_j into the register accumulator ----
        ok = mbar_wait(bar_o, jb & 1, failed);
        if (!ok && !*failed) { *failed = 1; atomicCAS(&g_attn_tc_error, 0, 2); }
        ok = __all_sync(0xffffffffu, ok);
        if (ok && jb + 1 < nblk) stage(Vs, a.tiles.v, jb + 1);            // the tensor core is done with V_j
        if (ok) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
            for (uint32_t h = 0; h < DH / 32; ++h) {
                float v[32];
                tmem_ld32(tmem_O + lane_addr + h * 32, v);
#pragma unroll
                for (uint32_t i = 0; i < 32; ++i) o[h * 32 + i] = o[h * 32 + i] * alpha + v[i];
            }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncthreads();
        if (*failed) break;
    }
    // ---- normalise and store this thread's row ----
    if (row_ok && !*failed) {
        const float inv = 1.0f / lrow;
        bf16 *dst = a.ob + ((size_t)(b * a.q_len + q0 + tid) * a.Hq + hq) * DH;
#pragma unroll
        for (uint32_t c = 0; c < DH / 8; ++c) {
            uint32_t w[4];
#pragma unroll
            for (uint32_t i = 0; i < 4; ++i) {
                __nv_bfloat162 pk = __floats2bfloat162_rn(o[c * 8 + 2 * i] * inv, o[c * 8 + 2 * i + 1] * inv);
                w[i] = *reinterpret_cast<uint32_t *>(&pk);
            }
            *reinterpret_cast<uint4 *>(dst + c * 8) = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u) : "memory");
    }
}

template <int DH> constexpr int smem_bytes() { return (DH / 64) * (BQ + 2 * BKV) * 128 + BQ * 128 + 64 + 1024; }

}  // namespace

extern thread_local uint64_t tgpk_launches;

int tgpk_attn_prefill_tc5(const void *qb, const TgpTilePtrs &tiles, void *ob, const tgp_model_cfg *c, uint32_t B, uint32_t q_len, uint32_t pos0, cudaStream_t st) {
    TArgs a{(const bf16 *)qb, (bf16 *)ob, c->Hq, c->Hkv, c->TK, q_len, pos0, 1.4426950408889634f / sqrtf((float)c->Dh), tiles};
    dim3 grid((q_len + BQ - 1) / BQ, c->Hq, B);
    static bool attr64 = false, attr128 = false;
    if (c->Dh == 64) {
        if (!attr64) { if (cudaFuncSetAttribute(attn_prefill_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<64>()) != cudaSuccess) return TGP_E_CUDA; attr64 = true; }
        attn_prefill_tc_kernel<64><<<grid, 128, smem_bytes<64>(), st>>>(a);
    } else if (c->Dh == 128) {
        if (!attr128) { if (cudaFuncSetAttribute(attn_prefill_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<128>()) != cudaSuccess) return TGP_E_CUDA; attr128 = true; }
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
