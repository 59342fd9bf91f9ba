// Causal GQA attention for prefill on the 5th-generation tensor cores (sm_100a).
//
// One CTA of eight warps owns 128 consecutive queries of one (sequence, query head); the longest query blocks are
// launched first.  Roles:
//   warps 0-3  softmax: thread t is query row t and TMEM lane t;
//   warp 4     lane 0 issues S_j = Q K_j^T;          warp 6  lane 0 issues O += P_j V_j;
//   warp 5     lane 0 issues every TMA load;         warp 7  idle (completes the second warpgroup for setmaxnreg).
// Shared memory holds Q and two stages each of K and V blocks of 64 keys as 64-wide blocks of [rows x 128 B] with the
// 128-byte swizzle (what a TMA box of 64 elements writes); K is then a K-major operand (head dimension contiguous) and
// V, in the very same layout, an MN-major operand (its contiguous dimension is the output dimension of P V).  One tensor
// map covers the address span of all KV tiles of the layer (tile bases differ by whole rows, a key block never crosses
// a tile), one the query activations, one the output.
// TMEM (256 columns): S (64, fp32), the output accumulator O (Dh, fp32, accumulated over all key blocks by the tensor
// core) and two buffers of P (32 each: bf16 pairs, read by the second product as its A operand straight from TMEM).
// Nothing in the key loop is a CTA-wide barrier; the roles hand over through mbarriers:
//   K_j landed, S_{j-1} in registers  -> S warp issues S_j; its completion releases S to the softmax warps and the K
//                                        stage to the TMA warp, which refills it with K_{j+2};
//   P_j written, V_j landed           -> P V warp issues O += P_j V_j; its completion releases the P buffer and the V
//                                        stage (refilled with V_{j+2}).
// An MMA accumulating into the same TMEM tile costs 75-90 cycles whatever its N <= 128, so S (8 MMAs) and P V (4) are
// issued by different warps and overlap with each other and with the other CTA of the SM.
// Softmax: the exponent reference m of a row is its max over block 0.  Later blocks use it as it is - P = exp2(S - m)
// may then exceed 1, which fp32 sums and bf16 P hold without loss of precision - and never compute a row max; only
// when a block's sum of exponentials exceeds 2^40 (or overflowed) does the warp wait for the P V in flight, move m to
// the new max and multiply its 32 rows of O in TMEM and its sums by 2^(m_old - m_new).  Scale-and-subtract and the sums
// use packed fp32 pairs.  At the end every thread reads its row of O once, divides by its sum, and the tile leaves
// through the (now free) Q buffer by TMA store (partial tiles: plain stores).
// Two CTAs fit on an SM (96 KB of shared memory, 256 TMEM columns, 128 registers per thread each, of which setmaxnreg
// moves the single-thread warps' share to the softmax warps).  KV tiles must hold a multiple of 64 keys; other
// geometries go to the mma.sync kernel.  Rows of the last V block past the sequence are zeroed in shared memory
// (0 * stale NaN would poison O); stale K rows only produce masked scores.
// P is rounded to bf16 for the second product (the one rounding of this path the CPU oracle does not mirror).
// Every mbarrier wait is bounded; a wait that runs out sets an error word, every role leaves its loop, the TMA warp
// waits (bounded) for the loads it still has in flight, TMEM is freed and nothing is stored.
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cstdint>
#include "tgp.h"
#include "tgp_kernels.h"
#include "tgp_sm100.cuh"

namespace {

using namespace tgp_sm100;
typedef __nv_bfloat16 bf16;
constexpr int BQ = 128, BKV = 64, THREADS = 256;   // warps 0-3 softmax, 4 S, 5 TMA, 6 P V, 7 idle (fills the second warpgroup)

__device__ int g_attn_tc_error = 0;   // 0 ok; 1 S, 2 P V, 3 K/V load, 4 softmax hand-over: the wait that ran out; 5 shared memory misaligned

struct TArgs {
    bf16 *ob;
    uint32_t Hq, Hkv, TK, q_len, pos0;
    float scale_log2;
    int32_t krow[TGP_MAX_TILES], vrow[TGP_MAX_TILES];       // first row of each KV tile in the map over all tiles
};

// MN-major operand in the same swizzled storage: 64 contiguous elements (128 B) of the MN dimension per row, rows are
// K; the next 64 MN elements start `lbo` bytes further (leading byte offset), the next 8 K rows 1024 bytes further.
__device__ __forceinline__ uint64_t umma_desc_mn(uint32_t smem_addr, uint32_t lbo) {
    return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}

// byte offset of 16-byte chunk c (0..7) of row r inside a [rows x 128 B] tile with the 128-byte swizzle
__device__ __forceinline__ uint32_t sw128(uint32_t r, uint32_t c) { return r * 128u + ((c ^ (r & 7u)) << 4); }

__device__ __forceinline__ float ex2(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
// two fp32 values per instruction (sm_100 packed arithmetic) and the three-input maximum
__device__ __forceinline__ uint64_t pack2(float lo, float hi) { uint64_t r; asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi)); return r; }
__device__ __forceinline__ void unpack2(uint64_t r, float &lo, float &hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(r)); }
__device__ __forceinline__ uint64_t fma2(uint64_t x, uint64_t y, uint64_t z) { uint64_t d; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(x), "l"(y), "l"(z)); return d; }
__device__ __forceinline__ uint64_t add2(uint64_t x, uint64_t y) { uint64_t d; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(x), "l"(y)); return d; }
__device__ __forceinline__ float max3(float x, float y, float z) { float d; asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(x), "f"(y), "f"(z)); return d; }

template <int DH>
__global__ void __launch_bounds__(THREADS, 2) tgp_attn_prefill_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKV, const __grid_constant__ CUtensorMap tmO, const TArgs a) {
    extern __shared__ __align__(1024) uint8_t smem[];
    constexpr int KB = DH / 64;                          // 64-wide blocks of the head dimension
    constexpr uint32_t Q_BYTES = KB * BQ * 128, KV_BYTES = KB * BKV * 128;
    uint8_t *Qs = smem, *Ks = Qs + Q_BYTES, *Vs = Ks + 2 * KV_BYTES;                            // K and V: two stages each
    uint64_t *bar_k = reinterpret_cast<uint64_t *>(Vs + 2 * KV_BYTES);      // [2] K stage landed (stage 0's first use also carries Q)
    uint64_t *bar_v = bar_k + 2;                                       // [2] V stage landed
    uint64_t *bar_s = bar_v + 2;                                       // S complete in TMEM (tensor core)
    uint64_t *bar_sfree = bar_s + 1;                                   // all 128 rows of S are in registers
    uint64_t *bar_p = bar_sfree + 1;                                   // [2] all 128 rows of P_j (buffer j & 1) written, O rescaled where needed
    uint64_t *bar_o = bar_p + 2;                                       // [2] P V_j complete (tensor core): P buffer j & 1 and the V stage are free
    uint64_t *bar_kfree = bar_o + 2;                                   // [2] S_j complete: K stage j & 1 is free
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bar_kfree + 2);
    volatile uint32_t *failed = tmem_slot + 1;

    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (smem_u32(smem) & 1023u) {                            // the swizzle assumes 1024-byte aligned tiles
        if (tid == 0) atomicCAS(&g_attn_tc_error, 0, 5);
        return;
    }
    const uint32_t qblk = gridDim.x - 1 - blockIdx.x, hq = blockIdx.y, b = blockIdx.z, hk = hq / (a.Hq / a.Hkv);      // longest (latest) query blocks are launched first
    const uint32_t q0 = qblk * BQ, kvlen = a.pos0 + a.q_len;
    const uint32_t last_q = min(a.q_len, q0 + BQ) - 1;
    const uint32_t nblk = (a.pos0 + last_q + 1 + BKV - 1) / BKV;

    // The TMA thread (warp 5, lane 0) initialises the barriers and requests Q and the first K and V blocks at once, before
    // the TMEM allocation and the CTA-wide barrier below.  Its state: blocks requested so far (block i uses stage i & 1)
    // and, for the next K and V block, the KV tile and the key offset inside it.
    uint32_t nk = 0, nv = 0, k_tile = 0, k_off = 0, v_tile = 0, v_off = 0;
    const uint32_t head_row = (b * a.Hkv + hk) * a.TK;
    auto load_kv = [&](uint8_t *dst, int y, uint64_t *bar, uint32_t more_bytes) {
        mbar_expect_tx(bar, KV_BYTES + more_bytes);
#pragma unroll
        for (uint32_t kb = 0; kb < KB; ++kb) tma_load_2d(dst + kb * (BKV * 128), &tmKV, kb * 64, y, bar);
    };
    auto next_k = [&](uint32_t more_bytes) {
        load_kv(Ks + (nk & 1) * KV_BYTES, a.krow[k_tile] + (int)(head_row + k_off), bar_k + (nk & 1), more_bytes);
        nk += 1;
        if ((k_off += BKV) == a.TK) { k_off = 0; k_tile += 1; }
    };
    auto next_v = [&]() {
        load_kv(Vs + (nv & 1) * KV_BYTES, a.vrow[v_tile] + (int)(head_row + v_off), bar_v + (nv & 1), 0);
        nv += 1;
        if ((v_off += BKV) == a.TK) { v_off = 0; v_tile += 1; }
    };
    if (warp == 5 && lane == 0) {
        mbar_init(bar_k, 1); mbar_init(bar_k + 1, 1); mbar_init(bar_v, 1); mbar_init(bar_v + 1, 1);
        mbar_init(bar_s, 1); mbar_init(bar_sfree, 128); mbar_init(bar_p, 128); mbar_init(bar_p + 1, 128); mbar_init(bar_o, 1); mbar_init(bar_o + 1, 1); mbar_init(bar_kfree, 1); mbar_init(bar_kfree + 1, 1);
        failed[0] = 0;
        failed[1] = 0;                                       // a flag nothing ever sets, for waits that must not be cut short
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmQ) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmKV) : "memory");
        next_k(Q_BYTES);                                     // K_0 and, on the same barrier, Q
#pragma unroll
        for (uint32_t kb = 0; kb < KB; ++kb) tma_load_2d(Qs + kb * (BQ * 128), &tmQ, hq * DH + kb * 64, b * a.q_len + q0, bar_k);
        if (1 < nblk) next_k(0);
        next_v();
    }
    if (warp == 4) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(256u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_S = tmem_base, tmem_O = tmem_base + 64, tmem_P = tmem_base + 192;     // P: two buffers of 32 columns (bf16 pairs)
    auto give_up = [&](int code) { if (!*failed) { *failed = 1; atomicCAS(&g_attn_tc_error, 0, code); } };
    // Registers move from the second warpgroup (three single-thread roles and an idle warp) to the softmax warpgroup:
    // 128 * 64 + 128 * 192 is the 128 per thread the CTA is launched with.
    if (warp >= 4) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 64;" ::: "memory");
        if (warp == 5) {
            // ======================= TMA warp: lane 0 requests the remaining K and V blocks =======================
            if (lane == 0) {
                // test hook: the first CTA of the grid never loads this V block, so the wait for it runs out
                const uint32_t withhold = (blockIdx.x | blockIdx.y | blockIdx.z) == 0 ? (uint32_t)g_withhold_step : 0xffffffffu;
                for (uint32_t jb = 0; jb + 1 < nblk; ++jb) {
                    const uint32_t st = jb & 1;
                    if (jb + 1 == withhold) break;
                    if (jb + 2 < nblk) {                                         // K_jb+2 goes where K_jb is, once S_jb is complete
                        if (!mbar_wait(bar_kfree + st, (jb >> 1) & 1, failed)) { give_up(1); break; }
                        next_k(0);
                    }
                    if (jb >= 1 && !mbar_wait(bar_o + (st ^ 1), ((jb - 1) >> 1) & 1, failed)) { give_up(2); break; }   // V_jb+1 goes where V_jb-1 is
                    next_v();
                }
                // every load requested must have landed before the CTA may exit (bounded; `never` is never set)
                volatile uint32_t *never = failed + 1;
                for (uint32_t st = 0; st < 2; ++st) {
                    const uint32_t ck = (nk + 1 - st) >> 1, cv = (nv + 1 - st) >> 1;     // loads requested into this stage
                    if (ck) mbar_wait(bar_k + st, (ck - 1) & 1, never);
                    if (cv) mbar_wait(bar_v + st, (cv - 1) & 1, never);
                }
            }
        } else if (warp == 4) {
            // ======================= S warp: lane 0 issues S_j = Q K_j^T =======================
            constexpr uint32_t idesc_s = umma_idesc(BKV);
            auto wait = [&](uint64_t *bar, uint32_t parity, int code) {
                bool ok = mbar_wait(bar, parity, failed);
                if (!ok) give_up(code);
                return __all_sync(0xffffffffu, ok);
            };
            for (uint32_t jb = 0; jb < nblk; ++jb) {
                if (jb >= 1 && !wait(bar_sfree, (jb - 1) & 1, 4)) break;         // S_jb-1 is in registers
                if (!wait(bar_k + (jb & 1), (jb >> 1) & 1, 3)) break;            // K_jb (and Q with K_0) has landed
                if (lane == 0) {
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint8_t *Kj = Ks + (jb & 1) * KV_BYTES;
#pragma unroll
                    for (uint32_t kb = 0; kb < KB; ++kb) {
                        const uint64_t dq = umma_desc(smem_u32(Qs + kb * (BQ * 128))), dk = umma_desc(smem_u32(Kj + kb * (BKV * 128)));
#pragma unroll
                        for (uint32_t k = 0; k < 4; ++k) umma(tmem_S, dq + 2 * k, dk + 2 * k, idesc_s, (kb | k) != 0);
                    }
                    umma_commit(bar_s);
                    umma_commit(bar_kfree + (jb & 1));                           // its completion also frees the K stage
                }
                __syncwarp();
            }
        } else if (warp == 6) {
            // ======================= P V warp: lane 0 issues O += P_j V_j =======================
            constexpr uint32_t idesc_o = umma_idesc(DH) | (1u << 16);           // bit 16: B operand is MN-major
            auto wait = [&](uint64_t *bar, uint32_t parity, int code) {
                bool ok = mbar_wait(bar, parity, failed);
                if (!ok) give_up(code);
                return __all_sync(0xffffffffu, ok);
            };
            for (uint32_t jb = 0; jb < nblk; ++jb) {
                const uint32_t st = jb & 1;
                if (!wait(bar_p + st, (jb >> 1) & 1, 4)) break;
                if (!wait(bar_v + st, (jb >> 1) & 1, 3)) break;
                if (jb * BKV + BKV > kvlen) {                                    // rows past the sequence: whatever the tile holds there
                    const uint32_t valid = kvlen - jb * BKV;
                    for (uint32_t i = lane; i < (BKV - valid) * KB * 8; i += 32) {
                        const uint32_t r = valid + i / (KB * 8), kb = (i / 8) % KB, c = i % 8;
                        *reinterpret_cast<uint4 *>(Vs + st * KV_BYTES + kb * (BKV * 128) + r * 128 + c * 16) = make_uint4(0, 0, 0, 0);
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                }
                if (lane == 0) {
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint64_t dv = umma_desc_mn(smem_u32(Vs + st * KV_BYTES), BKV * 128);
#pragma unroll
                    for (uint32_t k = 0; k < 4; ++k)                             // 16 keys per step: 8 columns of P, 2048 B of V rows
                        umma_ts(tmem_O, tmem_P + st * 32 + 8 * k, dv + 128 * k, idesc_o, (jb | k) != 0);
                    umma_commit(bar_o + st);
                }
                __syncwarp();
            }
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 192;" ::: "memory");
        // ======================= softmax warps: thread = query row = TMEM lane =======================
        const bool row_ok = q0 + tid < a.q_len;
        const uint32_t qpos = a.pos0 + min(q0 + tid, a.q_len - 1);          // padding rows take the last query's mask
        const uint32_t lane_addr = (warp * 32u) << 16;                       // this warp's quarter of the TMEM lanes
        float m_ref = -INFINITY, lrow = 0.f;                                 // exponent reference and running sum of this row
        auto wait = [&](uint64_t *bar, uint32_t parity, int code) {
            bool ok = mbar_wait(bar, parity, failed);
            if (!ok) give_up(code);
            return __all_sync(0xffffffffu, ok);
        };
        bool ok = true;
        for (uint32_t jb = 0; jb < nblk; ++jb) {
            if (!(ok = wait(bar_s, jb & 1, 1))) break;
            float s[BKV];
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            tmem_ld64(tmem_S + lane_addr, s);
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            mbar_arrive(bar_sfree);
            if (jb * BKV + BKV - 1 > a.pos0 + q0) {                          // this block crosses the diagonal of some row
#pragma unroll
                for (uint32_t i = 0; i < BKV; ++i)
                    if (jb * BKV + i > qpos) s[i] = -INFINITY;
            }
            auto row_max = [&]() {                                           // of the scaled scores (scale > 0: max commutes with it)
                float m0 = max3(s[0], s[1], s[2]), m1 = max3(s[3], s[4], s[5]);
#pragma unroll
                for (uint32_t i = 6; i + 3 < BKV; i += 4) { m0 = max3(m0, s[i], s[i + 1]); m1 = max3(m1, s[i + 2], s[i + 3]); }
                return max3(m0, m1, fmaxf(s[BKV - 2], s[BKV - 1])) * a.scale_log2;
            };
            uint32_t w[BKV / 2];
            auto exps = [&](float m) {                                       // w = exp2(S * scale - m) as bf16 pairs; returns their fp32 sum
                const uint64_t sc2 = pack2(a.scale_log2, a.scale_log2), nm2 = pack2(-m, -m);
                uint64_t acc0 = pack2(0.f, 0.f), acc1 = acc0;
#pragma unroll
                for (uint32_t i = 0; i < BKV / 2; ++i) {
                    float x0, x1;
                    unpack2(fma2(pack2(s[2 * i], s[2 * i + 1]), sc2, nm2), x0, x1);
                    const float p0 = ex2(x0), p1 = ex2(x1);                  // a masked score is -inf: p = 0
                    if (i & 1) acc1 = add2(acc1, pack2(p0, p1)); else acc0 = add2(acc0, pack2(p0, p1));
                    __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);       // .x = p0 in the lower half
                    w[i] = *reinterpret_cast<uint32_t *>(&pk);
                }
                float l0, l1;
                unpack2(add2(acc0, acc1), l0, l1);
                return l0 + l1;
            };
            // The exponent reference m is the row max of block 0 (which holds key 0 <= qpos: finite).  Later blocks use it
            // as it is and never look for their own max: only when a block's sum says that a score of one of the warp's
            // rows lies more than about 2^40 above m (or overflowed) does the warp take the slow path.
            if (jb == 0) m_ref = row_max();
            float lblk = exps(m_ref);
            if (jb > 0 && __any_sync(0xffffffffu, !(lblk <= 0x1p40f))) {
                if (!(ok = wait(bar_o + ((jb - 1) & 1), ((jb - 1) >> 1) & 1, 2))) break;           // P V_{j-1}: nothing is accumulating into O
                const float m_new = fmaxf(m_ref, row_max()), alpha = ex2(m_ref - m_new);
                m_ref = m_new;
                lrow *= alpha;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
                for (uint32_t h = 0; h < DH / 32; ++h) {
                    float v[32];
                    uint32_t u[32];
                    tmem_ld32(tmem_O + lane_addr + h * 32, v);
#pragma unroll
                    for (uint32_t i = 0; i < 32; ++i) u[i] = __float_as_uint(v[i] * alpha);
                    tmem_st32(tmem_O + lane_addr + h * 32, u);
                }
                lblk = exps(m_ref);
            }
            lrow += lblk;
            if (jb >= 2 && !(ok = wait(bar_o + (jb & 1), ((jb - 2) >> 1) & 1, 2))) break;      // P V_{j-2}: this P buffer is free
            tmem_st32(tmem_P + (jb & 1) * 32 + lane_addr, w);
            tmem_wait_st();
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            mbar_arrive(bar_p + (jb & 1));
        }
        // ---- the last P V; normalise and store this thread's row ----
        if (ok) ok = wait(bar_o + ((nblk - 1) & 1), ((nblk - 1) >> 1) & 1, 2);
        if (ok) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const float inv = 1.0f / lrow;
            const bool full_tile = q0 + BQ <= a.q_len;                       // a TMA store would spill padding rows into the next sequence
            bf16 *dst = a.ob + ((size_t)(b * a.q_len + q0 + tid) * a.Hq + hq) * DH;
#pragma unroll
            for (uint32_t h = 0; h < DH / 32; ++h) {
                float v[32];
                tmem_ld32(tmem_O + lane_addr + h * 32, v);
#pragma unroll
                for (uint32_t c = 0; c < 4; ++c) {
                    uint32_t w[4];
#pragma unroll
                    for (uint32_t i = 0; i < 4; ++i) {
                        __nv_bfloat162 pk = __floats2bfloat162_rn(v[c * 8 + 2 * i] * inv, v[c * 8 + 2 * i + 1] * inv);
                        w[i] = *reinterpret_cast<uint32_t *>(&pk);
                    }
                    // the Q tile is no longer read (every S is complete): it stages the output tile in the same layout
                    if (full_tile) *reinterpret_cast<uint4 *>(Qs + (h / 2) * (BQ * 128) + sw128(tid, (h % 2) * 4 + c)) = make_uint4(w[0], w[1], w[2], w[3]);
                    else if (row_ok) *reinterpret_cast<uint4 *>(dst + h * 32 + c * 8) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
            if (full_tile) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                mbar_arrive(bar_sfree);                                      // one more phase of this barrier: the four softmax warps meet
                if (wait(bar_sfree, nblk & 1, 4) && tid == 0) {
#pragma unroll
                    for (uint32_t kb = 0; kb < KB; ++kb)
                        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                                     ::"l"(&tmO), "r"((int)(hq * DH + kb * 64)), "r"((int)(b * a.q_len + q0)), "r"(smem_u32(Qs + kb * (BQ * 128))) : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");     // shared memory must outlive the read
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 4) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256u) : "memory");
    }
}

template <int DH> constexpr int smem_bytes() { return (DH / 64) * (BQ + 4 * BKV) * 128 + 128; }

}  // namespace

extern thread_local uint64_t tgpk_launches;

int tgpk_attn_prefill_tc5(const void *qb, const TgpTilePtrs &tiles, void *ob, const tgp_model_cfg *c, uint32_t B, uint32_t q_len, uint32_t pos0, cudaStream_t st) {
    if (c->Dh != 64 && c->Dh != 128) return TGP_E_INVAL;
    const uint32_t n_tiles = (pos0 + q_len + c->TK - 1) / c->TK;
    const uint64_t row_bytes = (uint64_t)c->Dh * 2, tile_rows = (uint64_t)B * c->Hkv * c->TK;
    if (n_tiles > TGP_MAX_TILES) return TGP_E_INVAL;
    // one map over the span of all KV tiles: possible when tile bases differ by whole rows and a key block stays in a tile
    uintptr_t lo = ~(uintptr_t)0, hi = 0;
    for (uint32_t t = 0; t < n_tiles; ++t)
        for (int kv = 0; kv < 2; ++kv) {
            const uintptr_t p = (uintptr_t)(kv ? tiles.v[t] : tiles.k[t]);
            lo = lo < p ? lo : p;
            hi = hi > p ? hi : p;
        }
    bool fits = c->TK % BKV == 0 && lo % 16 == 0 && (uintptr_t)qb % 16 == 0 && (uintptr_t)ob % 16 == 0 && ((hi - lo) / row_bytes + tile_rows) < (1ull << 31);
    for (uint32_t t = 0; fits && t < n_tiles; ++t)
        fits = ((uintptr_t)tiles.k[t] - lo) % row_bytes == 0 && ((uintptr_t)tiles.v[t] - lo) % row_bytes == 0;
    if (!fits) return tgpk_attn_prefill_tc(qb, tiles, ob, c, B, q_len, pos0, st);
    TArgs a{(bf16 *)ob, c->Hq, c->Hkv, c->TK, q_len, pos0, 1.4426950408889634f / sqrtf((float)c->Dh), {}, {}};
    for (uint32_t t = 0; t < n_tiles; ++t) {
        a.krow[t] = (int32_t)(((uintptr_t)tiles.k[t] - lo) / row_bytes);
        a.vrow[t] = (int32_t)(((uintptr_t)tiles.v[t] - lo) / row_bytes);
    }
    CUtensorMap mq, mkv, mo;
    if (!tensor_map_bf16_2d(&mq, qb, (uint64_t)B * q_len, (uint64_t)c->Hq * c->Dh, (uint64_t)c->Hq * c->Dh * 2, BQ) ||
        !tensor_map_bf16_2d(&mkv, (const void *)lo, (hi - lo) / row_bytes + tile_rows, c->Dh, row_bytes, BKV) ||
        !tensor_map_bf16_2d(&mo, ob, (uint64_t)B * q_len, (uint64_t)c->Hq * c->Dh, (uint64_t)c->Hq * c->Dh * 2, BQ))
        return TGP_E_CUDA;
    dim3 grid((q_len + BQ - 1) / BQ, c->Hq, B);
    static bool attr64 = false, attr128 = false;
    if (c->Dh == 64) {
        if (!attr64) {
            if (cudaFuncSetAttribute(tgp_attn_prefill_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<64>()) != cudaSuccess) return TGP_E_CUDA;
            cudaFuncSetAttribute(tgp_attn_prefill_tc_kernel<64>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
            attr64 = true;
        }
        tgp_attn_prefill_tc_kernel<64><<<grid, THREADS, smem_bytes<64>(), st>>>(mq, mkv, mo, a);
    } else {
        if (!attr128) {
            if (cudaFuncSetAttribute(tgp_attn_prefill_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<128>()) != cudaSuccess) return TGP_E_CUDA;
            cudaFuncSetAttribute(tgp_attn_prefill_tc_kernel<128>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
            attr128 = true;
        }
        tgp_attn_prefill_tc_kernel<128><<<grid, THREADS, smem_bytes<128>(), st>>>(mq, mkv, mo, a);
    }
    if (cudaGetLastError() != cudaSuccess) return TGP_E_CUDA;
    tgpk_launches += 1;
    return TGP_OK;
}

int tgpk_attn_wait_test(unsigned long long limit_ns, int withhold_step) {
    if (cudaMemcpyToSymbol(g_wait_limit_ns, &limit_ns, sizeof(limit_ns)) != cudaSuccess) return TGP_E_CUDA;
    return cudaMemcpyToSymbol(g_withhold_step, &withhold_step, sizeof(withhold_step)) == cudaSuccess ? TGP_OK : TGP_E_CUDA;
}

int tgpk_attn_status_clear() { const int z = 0; return cudaMemcpyToSymbol(g_attn_tc_error, &z, sizeof(z)) == cudaSuccess ? TGP_OK : TGP_E_CUDA; }

extern "C" int tgp_k_attn_status(int *error_code) {
    if (!error_code) return TGP_E_INVAL;
    if (cudaMemcpyFromSymbol(error_code, g_attn_tc_error, sizeof(int)) != cudaSuccess) return TGP_E_CUDA;
    return TGP_OK;
}
