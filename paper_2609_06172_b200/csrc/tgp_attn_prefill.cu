// Causal GQA attention for prefill on tensor cores: o = softmax(q K^T / sqrt(Dh)) V, one CTA per
// (64 queries, query head, sequence).  Flash-style: K/V blocks of 64 keys are gathered through the KV tile
// pointer table with cp.async (double-buffered), S = Q K^T and O += P V run on mma.sync m16n8k16 (bf16 in,
// fp32 accumulate), the softmax is online (running max / sum per row) in registers.  P is rounded to bf16
// for the second product; that is the one rounding of this path the CPU oracle does not mirror.
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cstdint>
#include "tgp.h"
#include "tgp_kernels.h"

namespace {

typedef __nv_bfloat16 bf16;
constexpr int BM = 64, BN = 64;

struct PArgs {
    const bf16 *qb; bf16 *ob;
    uint32_t Hq, Hkv, TK, q_len, pos0;
    float scale_log2;
    TgpTilePtrs tiles;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid) {
    const uint32_t n = valid ? 16u : 0u;                   // 0 source bytes: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm4t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float *d, const uint32_t *a, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// byte offset of 16-byte chunk c of row r in a [rows][DH] bf16 tile; chunks are XOR-swizzled by the row so that
// the 8 rows an ldmatrix phase reads fall into different banks
template <int DH> __device__ __forceinline__ uint32_t tile_off(uint32_t r, uint32_t c) { return r * (DH * 2) + ((c ^ (r & 7u)) << 4); }

template <int DH>
__global__ void __launch_bounds__(128) tgp_attn_prefill_mma_kernel(PArgs a) {
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int CH = DH / 8;                              // 16-byte chunks per row
    constexpr int TILE = BN * DH * 2;
    uint8_t *Qs = smem, *Ks = smem + BM * DH * 2, *Vs = Ks + 2 * TILE;
    const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t qblk = blockIdx.x, hq = blockIdx.y, b = blockIdx.z, hk = hq / (a.Hq / a.Hkv);
    const uint32_t q0 = qblk * BM;
    const uint32_t kvlen = a.pos0 + a.q_len;
    const uint32_t last_q = min(a.q_len, q0 + BM) - 1;      // last valid query of this block
    const uint32_t nkeys = a.pos0 + last_q + 1;             // keys any query of the block may see
    const uint32_t nblk = (nkeys + BN - 1) / BN;

    // ---- Q tile -> shared (rows past q_len are zero) ----
    for (uint32_t i = tid; i < BM * CH; i += 128) {
        const uint32_t r = i / CH, c = i % CH, p = q0 + r;
        const bool ok = p < a.q_len;
        const bf16 *src = a.qb + ((size_t)(b * a.q_len + (ok ? p : 0)) * a.Hq + hq) * DH + c * 8;
        cp_async16(smem_u32(Qs + tile_off<DH>(r, c)), src, ok);
    }
    auto load_kv = [&](uint32_t jb, uint32_t stage) {
        for (uint32_t i = tid; i < BN * CH; i += 128) {
            const uint32_t r = i / CH, c = i % CH, j = jb * BN + r;
            const bool ok = j < kvlen;
            const uint32_t jj = ok ? j : 0;
            const size_t off = ((size_t)(b * a.Hkv + hk) * a.TK + jj % a.TK) * DH + c * 8;
            cp_async16(smem_u32(Ks + stage * TILE + tile_off<DH>(r, c)), reinterpret_cast<const bf16 *>(a.tiles.k[jj / a.TK]) + off, ok);
            cp_async16(smem_u32(Vs + stage * TILE + tile_off<DH>(r, c)), reinterpret_cast<const bf16 *>(a.tiles.v[jj / a.TK]) + off, ok);
        }
    };
    load_kv(0, 0);
    cp_async_commit();

    float o[DH / 8][4];
#pragma unroll
    for (int t = 0; t < DH / 8; ++t) { o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f; }
    float mrow[2] = {-INFINITY, -INFINITY}, lrow[2] = {0.f, 0.f};
    uint32_t qf[DH / 16][4];
    const uint32_t row_in_warp = lane >> 2;                 // accumulator rows: row_in_warp and row_in_warp + 8
    uint32_t qpos[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) qpos[h] = a.pos0 + min(q0 + warp * 16 + row_in_warp + 8 * h, a.q_len - 1);   // clamp padding rows

    for (uint32_t jb = 0; jb < nblk; ++jb) {
        const uint32_t stage = jb & 1;
        if (jb + 1 < nblk) { load_kv(jb + 1, stage ^ 1); cp_async_commit(); cp_async_wait<1>(); }
        else cp_async_wait<0>();
        __syncthreads();
        if (jb == 0) {
#pragma unroll
            for (int ks = 0; ks < DH / 16; ++ks)
                ldsm4(smem_u32(Qs + tile_off<DH>(warp * 16 + (lane & 7) + 8 * ((lane >> 3) & 1), ks * 2 + (lane >> 4))), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
        }
        // ---- S = Q K^T (16 x 64 per warp) ----
        float s[BN / 8][4];
#pragma unroll
        for (int t = 0; t < BN / 8; ++t) { s[t][0] = s[t][1] = s[t][2] = s[t][3] = 0.f; }
        const uint8_t *Kst = Ks + stage * TILE, *Vst = Vs + stage * TILE;
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks)
#pragma unroll
            for (int nt = 0; nt < BN / 8; nt += 2) {
                uint32_t b0, b1, b2, b3;
                ldsm4(smem_u32(Kst + tile_off<DH>(nt * 8 + (lane & 7) + 8 * (lane >> 4), ks * 2 + ((lane >> 3) & 1))), b0, b1, b2, b3);
                mma16816(s[nt], qf[ks], b0, b1);
                mma16816(s[nt + 1], qf[ks], b2, b3);
            }
        // ---- scale, causal mask, online softmax ----
        float mnew[2] = {mrow[0], mrow[1]};
#pragma unroll
        for (int t = 0; t < BN / 8; ++t)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t key = jb * BN + t * 8 + 2 * (lane & 3) + (i & 1);
                const float v = (key <= qpos[i >> 1]) ? s[t][i] * a.scale_log2 : -INFINITY;
                s[t][i] = v;
                mnew[i >> 1] = fmaxf(mnew[i >> 1], v);
            }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            mnew[h] = fmaxf(mnew[h], __shfl_xor_sync(0xffffffffu, mnew[h], 1));
            mnew[h] = fmaxf(mnew[h], __shfl_xor_sync(0xffffffffu, mnew[h], 2));
        }
        float alpha[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) { alpha[h] = exp2f(mrow[h] - mnew[h]); mrow[h] = mnew[h]; lrow[h] *= alpha[h]; }
#pragma unroll
        for (int t = 0; t < BN / 8; ++t)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float p = exp2f(s[t][i] - mnew[i >> 1]);
                s[t][i] = p;
                lrow[i >> 1] += p;
            }
#pragma unroll
        for (int t = 0; t < DH / 8; ++t) { o[t][0] *= alpha[0]; o[t][1] *= alpha[0]; o[t][2] *= alpha[1]; o[t][3] *= alpha[1]; }
        // ---- O += P V ----
#pragma unroll
        for (int kk = 0; kk < BN / 16; ++kk) {
            uint32_t pf[4] = {pack2(s[2 * kk][0], s[2 * kk][1]), pack2(s[2 * kk][2], s[2 * kk][3]),
                              pack2(s[2 * kk + 1][0], s[2 * kk + 1][1]), pack2(s[2 * kk + 1][2], s[2 * kk + 1][3])};
#pragma unroll
            for (int nt = 0; nt < DH / 8; nt += 2) {
                uint32_t b0, b1, b2, b3;
                ldsm4t(smem_u32(Vst + tile_off<DH>(kk * 16 + (lane & 7) + 8 * ((lane >> 3) & 1), nt + (lane >> 4))), b0, b1, b2, b3);
                mma16816(o[nt], pf, b0, b1);
                mma16816(o[nt + 1], pf, b2, b3);
            }
        }
        __syncthreads();                                    // everyone is done with this stage before it is refilled
    }
    // ---- normalise and store ----
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        lrow[h] += __shfl_xor_sync(0xffffffffu, lrow[h], 1);
        lrow[h] += __shfl_xor_sync(0xffffffffu, lrow[h], 2);
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint32_t p = q0 + warp * 16 + row_in_warp + 8 * h;
        if (p >= a.q_len) continue;
        const float inv = 1.0f / lrow[h];
        bf16 *dst = a.ob + ((size_t)(b * a.q_len + p) * a.Hq + hq) * DH + 2 * (lane & 3);
#pragma unroll
        for (int t = 0; t < DH / 8; ++t)
            *reinterpret_cast<__nv_bfloat162 *>(dst + t * 8) = __floats2bfloat162_rn(o[t][2 * h] * inv, o[t][2 * h + 1] * inv);
    }
}

}  // namespace

extern thread_local uint64_t tgpk_launches;

int tgpk_attn_prefill_tc(const void *qb, const TgpTilePtrs &tiles, void *ob, const tgp_model_cfg *c, uint32_t B, uint32_t q_len, uint32_t pos0, cudaStream_t st) {
    PArgs a{(const bf16 *)qb, (bf16 *)ob, c->Hq, c->Hkv, c->TK, q_len, pos0, 1.4426950408889634f / sqrtf((float)c->Dh), tiles};
    dim3 grid((q_len + BM - 1) / BM, c->Hq, B);
    static bool attr64 = false, attr128 = false;
    if (c->Dh == 64) {
        constexpr int SM = (BM + 4 * BN) * 64 * 2;
        if (!attr64) { if (cudaFuncSetAttribute(tgp_attn_prefill_mma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM) != cudaSuccess) return TGP_E_CUDA; attr64 = true; }
        tgp_attn_prefill_mma_kernel<64><<<grid, 128, SM, st>>>(a);
    } else if (c->Dh == 128) {
        constexpr int SM = (BM + 4 * BN) * 128 * 2;
        if (!attr128) { if (cudaFuncSetAttribute(tgp_attn_prefill_mma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM) != cudaSuccess) return TGP_E_CUDA; attr128 = true; }
        tgp_attn_prefill_mma_kernel<128><<<grid, 128, SM, st>>>(a);
    } else {
        return TGP_E_INVAL;
    }
    if (cudaGetLastError() != cudaSuccess) return TGP_E_CUDA;
    tgpk_launches += 1;
    return TGP_OK;
}
