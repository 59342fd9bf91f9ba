// Internal launch interface between the step engine and the kernels.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>
#include "tgp.h"

#define TGP_MAX_TILES 64      // KV tiles per layer a kernel can address (pointer table passed by value)

struct TgpTilePtrs { void *k[TGP_MAX_TILES]; void *v[TGP_MAX_TILES]; };

// rows of token ids outside [0, V) are written as zeros and recorded (tgp_k_embed_status)
int tgpk_embed(const void *table, const int32_t *tok, float *x, uint32_t M, uint32_t d, uint32_t V, cudaStream_t st);
int tgpk_rmsnorm(const float *x, uint32_t ldx, const void *g, void *h, uint32_t M, uint32_t d, float eps, cudaStream_t st);
int tgpk_gemm(const void *A, const void *W, float *C, uint32_t M, uint32_t n, uint32_t K, uint32_t ldc, uint32_t col0, int accumulate, cudaStream_t st);
// products over the same activations A [M, K]: C[s][m, j] (=|+=) sum_k A[m, k] * W[s][j, k].  Blocks with the same non-zero
// tgpk_gemm_group_key() are served by one launch (up to TGP_GEMM_GROUP_MAX of them), anything else by one launch per part;
// the bits are the same either way
uint32_t tgpk_gemm_group_key(uint32_t M, uint32_t n, uint32_t K);
int tgpk_gemm_group(const void *A, uint32_t count, const void *const *W, float *const *C, const uint32_t *n, const uint32_t *ldc, uint32_t M, uint32_t K,
                    int accumulate, cudaStream_t st);
// tcgen05 path (tgp_gemm_sm100.cu): any M, n; K % 8 == 0; A and W 16-byte aligned
// gate / aout (both or neither): the accumulator is the up projection of a SwiGLU FFN; instead of storing it to C the epilogue
// stores aout[m, col0 + j] = bf16(silu(gate[m, col0 + j]) * acc) (gate fp32 and aout bf16 in C's geometry); not with accumulate
int tgpk_gemm_tc(const void *A, const void *W, float *C, uint32_t M, uint32_t n, uint32_t K, uint32_t ldc, uint32_t col0, int accumulate, cudaStream_t st,
                 const float *gate = nullptr, void *aout = nullptr);
// true if a product of M activation rows takes the tensor-core GEMM, whose epilogue can apply SwiGLU (M > 128, tensor cores selected)
bool tgpk_swiglu_fusable(uint32_t M);
int tgpk_rope_kv(const float *q32, const float *k32, const float *v32, void *qb, const TgpTilePtrs &tiles, const float *cos_t, const float *sin_t,
                 const tgp_model_cfg *c, uint32_t B, uint32_t q_len, uint32_t pos0, cudaStream_t st);
int tgpk_attn(const void *qb, const TgpTilePtrs &tiles, uint32_t n_tiles, void *ob, const tgp_model_cfg *c, uint32_t B, uint32_t q_len, uint32_t pos0,
              float *scratch, cudaStream_t st);
// tcgen05 causal attention for q_len > 1 (tgp_attn_sm100.cu); Dh 64 or 128
int tgpk_attn_prefill_tc5(const void *qb, const TgpTilePtrs &tiles, void *ob, const tgp_model_cfg *c, uint32_t B, uint32_t q_len, uint32_t pos0, cudaStream_t st);
// mma.sync flash-style causal attention for q_len > 1 (tgp_attn_prefill.cu); Dh 64 or 128
int tgpk_attn_prefill_tc(const void *qb, const TgpTilePtrs &tiles, void *ob, const tgp_model_cfg *c, uint32_t B, uint32_t q_len, uint32_t pos0, cudaStream_t st);
int tgpk_swiglu(const float *g, const float *u, void *ab, uint64_t n, cudaStream_t st);
// MoE: router logits + top-k (1 or 2) + gates, then per-expert token lists rows[e*stride + i], gates[e*stride + i], counts[e]
int tgpk_router(const void *h, const void *Wr, const float *bias, int32_t *idx, float *gate, int32_t *rows, float *gates, int32_t *counts,
                uint32_t M, uint32_t stride, uint32_t d, uint32_t E, uint32_t topk, cudaStream_t st);
int tgpk_gather_rows(const void *src, const int32_t *rows, void *dst, uint32_t m, uint32_t d, cudaStream_t st);
int tgpk_scatter_add(float *x, const float *y, const int32_t *rows, const float *gates, uint32_t m, uint32_t d, cudaStream_t st);
int tgpk_argmax(const float *logits, int32_t *out, uint32_t B, uint32_t V, cudaStream_t st);
// cos/sin tables [max_len, Dh/2] fp32 (angle = pos * base^(-2i/Dh), evaluated in double) written to device memory
int tgp_rope_tables_upload(uint32_t Dh, uint32_t max_len, float base, float *cos_dev, float *sin_dev);
// reset of the tensor-core kernels' error words (tgp_gemm_sm100.cu, tgp_attn_sm100.cu)
int tgpk_gemm_status_clear();
int tgpk_attn_status_clear();
// name of the kernel the last tgpk_gemm / tgpk_gemm_group / tgpk_gemm_tc call of this thread launched
extern thread_local const char *tgpk_last_gemm_kernel;
// set while the caller vouches that this thread's kernel launches are all that is enqueued on their streams (see tgp_k_gemm_chain)
extern thread_local bool tgpk_chain_ok;
// test hooks of the tensor-core kernels' bounded waits (see tgp_k_wait_test)
int tgpk_gemm_wait_test(unsigned long long limit_ns, int withhold_step);
int tgpk_attn_wait_test(unsigned long long limit_ns, int withhold_step);
// products of M <= 2 rows with the activations computed on the fly: mode 1 the RMSNorm of x (row stride ldx, gain, eps),
// mode 2 SwiGLU of (g32, u32); bit-identical to the separate kernels followed by tgpk_gemm_group()
int tgpk_gemm_group_fused(int mode, const float *x, uint32_t ldx, const void *gain, float eps, const float *g32, const float *u32, uint32_t count,
                          const void *const *W, float *const *C, const uint32_t *n, const uint32_t *ldc, uint32_t M, uint32_t K, int accumulate, cudaStream_t st);
