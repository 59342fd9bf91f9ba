// Hand-written sm_100a kernels of the forward pass and their C entry points.
// Precision contract: bf16 weights / KV / GEMM inputs, fp32 accumulation and residual stream.
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cstdint>
#include <type_traits>
#include <algorithm>
#include "tgp.h"
#include "tgp_kernels.h"

thread_local uint64_t tgpk_launches = 0;     // kernels launched by this thread (reported in the step statistics)
// true while the caller vouches that this thread's launches are all that is enqueued on their streams (tgp_step does; direct
// callers say so through tgp_k_gemm_chain): consecutive weight products over the same activations may then read them early
thread_local bool tgpk_chain_ok = false;
namespace { struct ProductChain { const void *A; cudaStream_t st; uint64_t launches_before; }; thread_local ProductChain g_chain = {nullptr, nullptr, 0}; }
thread_local const char *tgpk_last_gemm_kernel = "";   // name of the kernel the last weight-block product of this thread launched
#define LAUNCH_CHECK(n) do { cudaError_t e_ = cudaGetLastError(); if (e_ != cudaSuccess) return TGP_E_CUDA; tgpk_launches += (n); } while (0)

typedef __nv_bfloat16 bf16;

__device__ __forceinline__ void unpack8(const uint4 &v, float *f) {
    const __nv_bfloat162 *p = reinterpret_cast<const __nv_bfloat162 *>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) { float2 t = __bfloat1622float2(p[i]); f[2 * i] = t.x; f[2 * i + 1] = t.y; }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Activations are produced by the grid under which this one may already have been launched (programmatic dependent
// launch), so they are read with an ordinary load after griddepcontrol.wait - never through the read-only path
// (ld.global.nc, what __ldg and const __restrict__ pointers compile to), whose cached lines may predate the wait and
// were seen to serve the previous layer's values.  The activation pointers of these kernels are therefore not
// __restrict__, and the load is a plain one (an asm volatile load costs the M <= 2 kernel a tenth of its speed, an
// L2-only load a third).
__device__ __forceinline__ uint4 ld_act(const uint4 *p) { return *p; }

// Programmatic dependent launch for the small kernels of a decode step: the grid lets its successor be scheduled at
// once and then waits for its predecessor to complete and flush, before it reads anything - the dependency is the full
// one, but the successor's launch latency (a microsecond or two, as long as these kernels run) overlaps this grid's
// execution.  Every thread of every kernel launched through launch_pdl() executes this first.
__device__ __forceinline__ void pdl_enter() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

static int g_small_pdl = 1;      // small kernels are launched as programmatic dependents of their predecessor (0: plain launches)

template <typename... KArgs, typename... Args>
static void launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = g_small_pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- embedding gather ------------------------------------------------------------------------
// A token id outside [0, V) would index past the table (which may be mapped host memory): such a row is written as
// zeros and the first offending (row, id) is recorded in g_embed_error for tgp_k_embed_status().
__device__ unsigned long long g_embed_error = 0;      // 0, or 1 << 63 | row << 32 | (uint32_t)id of the first bad token

__global__ void tgp_embed_kernel(const bf16 *__restrict__ table, const int32_t *tok, float *x, uint32_t d, uint32_t V) {
    pdl_enter();
    const uint32_t m = blockIdx.x;
    const int32_t id = tok[m];
    float4 *out = reinterpret_cast<float4 *>(x + (size_t)m * d);
    if (id < 0 || (uint32_t)id >= V) {
        for (uint32_t i = threadIdx.x; i < d / 4; i += blockDim.x) out[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (threadIdx.x == 0) atomicCAS(&g_embed_error, 0ull, (1ull << 63) | ((unsigned long long)m << 32) | (uint32_t)id);
        return;
    }
    const uint4 *row = reinterpret_cast<const uint4 *>(table + (size_t)id * d);
    for (uint32_t i = threadIdx.x; i < d / 8; i += blockDim.x) {
        float f[8];
        unpack8(row[i], f);
        out[2 * i] = make_float4(f[0], f[1], f[2], f[3]);
        out[2 * i + 1] = make_float4(f[4], f[5], f[6], f[7]);
    }
}

// ---- RMSNorm -> bf16 -------------------------------------------------------------------------
// One step of a thread's sum of squares, written with explicit roundings so that the fused form below (a consumer that
// normalises its activations itself) reproduces the kernel's statistics bit for bit.
__device__ __forceinline__ float sumsq4(float ss, const float4 &v) {
    return __fadd_rn(ss, __fmaf_rn(v.w, v.w, __fmaf_rn(v.z, v.z, __fmaf_rn(v.y, v.y, __fmul_rn(v.x, v.x)))));
}

__global__ void tgp_rmsnorm_kernel(const float *x, uint32_t ldx, const bf16 *__restrict__ g, bf16 *h, uint32_t d, float eps) {
    pdl_enter();
    __shared__ float red[32];
    const float4 *row = reinterpret_cast<const float4 *>(x + (size_t)blockIdx.x * ldx);
    float ss = 0.f;
    for (uint32_t i = threadIdx.x; i < d / 4; i += blockDim.x) ss = sumsq4(ss, row[i]);
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x < 32) {
        float t = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0.f;
        t = warp_sum(t);
        if (threadIdx.x == 0) red[0] = 1.0f / sqrtf(t / (float)d + eps);
    }
    __syncthreads();
    const float r = red[0];
    __nv_bfloat162 *out = reinterpret_cast<__nv_bfloat162 *>(h + (size_t)blockIdx.x * d);
    const __nv_bfloat162 *gg = reinterpret_cast<const __nv_bfloat162 *>(g);
    for (uint32_t i = threadIdx.x; i < d / 4; i += blockDim.x) {
        float4 v = row[i];
        float2 g0 = __bfloat1622float2(gg[2 * i]), g1 = __bfloat1622float2(gg[2 * i + 1]);
        out[2 * i] = __floats2bfloat162_rn(v.x * r * g0.x, v.y * r * g0.y);
        out[2 * i + 1] = __floats2bfloat162_rn(v.z * r * g1.x, v.w * r * g1.y);
    }
}

// ---- GEMV / skinny GEMM (M <= 8 activation rows): pure weight streaming --------------------------------
// Persistent warps: the grid fills every SM once; each warp walks row groups of R output rows with a
// grid stride and keeps R x U independent 16-byte loads in flight per lane (U chunks of 256 K-elements).
// No block barrier and no shared memory, so no SM idles while another warp reduces; the summation order
// is fixed (lane-strided partials, butterfly), hence results are deterministic run to run.
template <int MT, int R, int U>
__global__ void __launch_bounds__(256) tgp_wstream_kernel(const bf16 *A, const bf16 *__restrict__ W, float *__restrict__ C,
                                                   uint32_t Mrows, uint32_t n, uint32_t K, uint32_t ldc, uint32_t col0, int accumulate) {
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t gwarp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarp = (gridDim.x * blockDim.x) >> 5;
    // Programmatic dependent launch: the weights are not produced by the previous kernel in the stream, so this grid
    // may start streaming them while that kernel drains.  Everything it does produce (the activations A, the output C)
    // is touched only after griddepcontrol.wait, which returns once the previous grid has completed and flushed.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool synced = false;
    for (uint32_t row0 = gwarp * R; row0 < n; row0 += nwarp * R) {
        float acc[R][MT];
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int m = 0; m < MT; ++m) acc[r][m] = 0.f;
        const bf16 *wrow[R];
#pragma unroll
        for (int r = 0; r < R; ++r) wrow[r] = W + (size_t)min(row0 + r, n - 1) * K;   // tail rows re-read the last row, never stored
        for (uint32_t k0 = lane * 8; k0 < K; k0 += 256 * U) {
            uint4 wv[U][R];
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int r = 0; r < R; ++r)
                    wv[u][r] = (k0 + 256 * u < K) ? __ldcs(reinterpret_cast<const uint4 *>(wrow[r] + k0 + 256 * u)) : make_uint4(0, 0, 0, 0);
            if (!synced) { asm volatile("griddepcontrol.wait;" ::: "memory"); synced = true; }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t k = k0 + 256 * u;
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    float xf[8];
                    unpack8((k < K && m < (int)Mrows) ? ld_act(reinterpret_cast<const uint4 *>(A + (size_t)m * K + k)) : make_uint4(0, 0, 0, 0), xf);
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        float wf[8];
                        unpack8(wv[u][r], wf);
#pragma unroll
                        for (int i = 0; i < 8; ++i) acc[r][m] = fmaf(wf[i], xf[i], acc[r][m]);
                    }
                }
            }
        }
        if (!synced) { asm volatile("griddepcontrol.wait;" ::: "memory"); synced = true; }      // K == 0 never happens; belt and braces
        // a product added to the residual stream goes out as a reduction (one add per element, by one thread: the same
        // rounded sum as load, add, store, and deterministic) that nothing waits for: the launch ends a memory round trip sooner
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                const float s = warp_sum(acc[r][m]);
                if ((int)lane == r * MT + m && row0 + r < n && m < (int)Mrows) {
                    if (accumulate) atomicAdd(&C[(size_t)m * ldc + col0 + row0 + r], s);
                    else C[(size_t)m * ldc + col0 + row0 + r] = s;
                }
            }
    }
}

// Several products that read the same activations (the q, k and v projections of a layer) in one launch: the output
// rows of the parts are walked as one list, one warp per row, with exactly the arithmetic of tgp_wstream_kernel<MT, 1, U>, so
// the result is bit-identical to separate launches; what is saved is two launch floors of about a microsecond each.
// (groups[s]: CTAs' worth of rows in part s, for the kernels that walk row groups instead of rows)
struct GemvParts { const bf16 *W[TGP_GEMM_GROUP_MAX]; float *C[TGP_GEMM_GROUP_MAX]; uint32_t n[TGP_GEMM_GROUP_MAX], ldc[TGP_GEMM_GROUP_MAX], groups[TGP_GEMM_GROUP_MAX], count; };

// Where the activations of a product come from.  mode 0: bf16 rows A[m, K].  mode 1: the RMSNorm of the fp32 rows x[m, :K]
// (row stride ldx) with gain g - the warp computes the row statistics itself, exactly as tgp_rmsnorm_kernel's 256 threads
// do (lane l plays threads l, 32 + l, ... of that kernel), and rounds each normalised value to bf16 as that kernel
// stores it.  mode 2: SwiGLU of the fp32 rows g32, u32 [m, K], rounded to bf16 as tgp_swiglu_kernel stores it.  The fused
// modes give bit for bit what the separate kernels followed by mode 0 give; they save a launch and a round trip for
// the decode steps of small models, where every warp recomputing a row of a few hundred elements costs nothing.
struct ASrc { int mode; const float *x; uint32_t ldx; const bf16 *gain; float eps; const float *g32, *u32; };

__device__ __forceinline__ float rms_scale_as_kernel(const float *xrow, uint32_t d, float eps, uint32_t lane) {
    const float4 *row = reinterpret_cast<const float4 *>(xrow);
    float red[8];
#pragma unroll
    for (uint32_t w = 0; w < 8; ++w) {
        float ss = 0.f;
        for (uint32_t i = 32 * w + lane; i < d / 4; i += 256) ss = sumsq4(ss, row[i]);
        red[w] = warp_sum(ss);
    }
    float t = 0.f;
#pragma unroll
    for (uint32_t w = 0; w < 8; ++w) if (lane == w) t = red[w];
    t = warp_sum(t);
    return 1.0f / sqrtf(t / (float)d + eps);
}

__device__ __forceinline__ void act8(const ASrc &s, const bf16 *A, uint32_t m, uint32_t K, uint32_t k, float r, float *xf) {
    if (s.mode == 0) { unpack8(ld_act(reinterpret_cast<const uint4 *>(A + (size_t)m * K + k)), xf); return; }
    if (s.mode == 1) {
        const float4 *xr = reinterpret_cast<const float4 *>(s.x + (size_t)m * s.ldx + k);
        const float4 v0 = xr[0], v1 = xr[1];
        float g[8];
        unpack8(*reinterpret_cast<const uint4 *>(s.gain + k), g);
        const float v[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) xf[i] = __bfloat162float(__float2bfloat16_rn(v[i] * r * g[i]));
        return;
    }
    const float4 *gr = reinterpret_cast<const float4 *>(s.g32 + (size_t)m * K + k), *ur = reinterpret_cast<const float4 *>(s.u32 + (size_t)m * K + k);
    const float4 g0 = gr[0], g1 = gr[1], u0 = ur[0], u1 = ur[1];
    const float gv[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w}, uv[8] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) xf[i] = __bfloat162float(__float2bfloat16_rn(gv[i] / (1.0f + expf(-gv[i])) * uv[i]));
}

template <int MT, int U>
__global__ void __launch_bounds__(256) tgp_wstream_group_kernel(const bf16 *A, const GemvParts p, uint32_t Mrows, uint32_t n_total, uint32_t K, int accumulate, const ASrc src) {
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t gwarp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarp = (gridDim.x * blockDim.x) >> 5;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool synced = false;
    float rs[MT];
#pragma unroll
    for (int m = 0; m < MT; ++m) rs[m] = 0.f;
    for (uint32_t row = gwarp; row < n_total; row += nwarp) {
        const bf16 *W = p.W[0];
        float *C = p.C[0];
        uint32_t ldc = p.ldc[0], r = row, start = p.n[0];
#pragma unroll
        for (int s = 1; s < (int)TGP_GEMM_GROUP_MAX; ++s)
            if (s < (int)p.count) {
                if (row >= start) { W = p.W[s]; C = p.C[s]; ldc = p.ldc[s]; r = row - start; }
                start += p.n[s];
            }
        const bf16 *wrow = W + (size_t)r * K;
        float acc[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) acc[m] = 0.f;
        for (uint32_t k0 = lane * 8; k0 < K; k0 += 256 * U) {
            uint4 wv[U];
#pragma unroll
            for (int u = 0; u < U; ++u)
                wv[u] = (k0 + 256 * u < K) ? __ldcs(reinterpret_cast<const uint4 *>(wrow + k0 + 256 * u)) : make_uint4(0, 0, 0, 0);
            if (!synced) {
                asm volatile("griddepcontrol.wait;" ::: "memory");
                synced = true;
                if (src.mode == 1) {
#pragma unroll
                    for (int m = 0; m < MT; ++m) if (m < (int)Mrows) rs[m] = rms_scale_as_kernel(src.x + (size_t)m * src.ldx, K, src.eps, lane);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t k = k0 + 256 * u;
                float wf[8];
                unpack8(wv[u], wf);
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    float xf[8];
                    if (k < K && m < (int)Mrows) act8(src, A, m, K, k, rs[m], xf);
                    else {
#pragma unroll
                        for (int i = 0; i < 8; ++i) xf[i] = 0.f;
                    }
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[m] = fmaf(wf[i], xf[i], acc[m]);
                }
            }
        }
        if (!synced) { asm volatile("griddepcontrol.wait;" ::: "memory"); synced = true; }
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            const float s = warp_sum(acc[m]);
            if ((int)lane == m && m < (int)Mrows) {
                if (accumulate) atomicAdd(&C[(size_t)m * ldc + r], s);
                else C[(size_t)m * ldc + r] = s;
            }
        }
    }
}

// Same product for blocks with few rows (n below two waves of warps): one CTA of 8 warps owns RB rows and its warps
// split K in interleaved chunks of 256 elements, so n / RB CTAs spread over the SMs almost evenly where n warps of whole
// rows leave a quarter of them with half the work.  The 8 partial sums of a row meet in shared memory and are added in
// warp order: deterministic.  Same dependent-launch protocol.
template <int MT, int RB, int U>
__global__ void __launch_bounds__(256) tgp_wstream_splitk_kernel(const bf16 *A, const bf16 *__restrict__ W, float *__restrict__ C,
                                                          uint32_t Mrows, uint32_t n, uint32_t K, uint32_t ldc, uint32_t col0, int accumulate) {
    __shared__ float part[8][RB * MT];
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool synced = false;
    for (uint32_t row0 = blockIdx.x * RB; row0 < n; row0 += gridDim.x * RB) {
        float acc[RB][MT];
#pragma unroll
        for (int r = 0; r < RB; ++r)
#pragma unroll
            for (int m = 0; m < MT; ++m) acc[r][m] = 0.f;
        const bf16 *wrow[RB];
#pragma unroll
        for (int r = 0; r < RB; ++r) wrow[r] = W + (size_t)min(row0 + r, n - 1) * K;
        const bool mine = threadIdx.x < RB * MT && row0 + threadIdx.x / MT < n && threadIdx.x % MT < Mrows;
        for (uint32_t k0 = warp * 256 + lane * 8; k0 < K; k0 += 2048 * U) {
            uint4 wv[U][RB];
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int r = 0; r < RB; ++r)
                    wv[u][r] = (k0 + 2048 * u < K) ? __ldcs(reinterpret_cast<const uint4 *>(wrow[r] + k0 + 2048 * u)) : make_uint4(0, 0, 0, 0);
            if (!synced) { asm volatile("griddepcontrol.wait;" ::: "memory"); synced = true; }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t k = k0 + 2048 * u;
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    float xf[8];
                    unpack8((k < K && m < (int)Mrows) ? ld_act(reinterpret_cast<const uint4 *>(A + (size_t)m * K + k)) : make_uint4(0, 0, 0, 0), xf);
#pragma unroll
                    for (int r = 0; r < RB; ++r) {
                        float wf[8];
                        unpack8(wv[u][r], wf);
#pragma unroll
                        for (int i = 0; i < 8; ++i) acc[r][m] = fmaf(wf[i], xf[i], acc[r][m]);
                    }
                }
            }
        }
        if (!synced) { asm volatile("griddepcontrol.wait;" ::: "memory"); synced = true; }     // a warp whose K slice is empty
#pragma unroll
        for (int r = 0; r < RB; ++r)
#pragma unroll
            for (int m = 0; m < MT; ++m) {
                const float sacc = warp_sum(acc[r][m]);
                if (lane == 0) part[warp][r * MT + m] = sacc;
            }
        __syncthreads();
        if (mine) {
            float t = 0.f;
#pragma unroll
            for (int w = 0; w < 8; ++w) t += part[w][threadIdx.x];
            float *cptr = C + (size_t)(threadIdx.x % MT) * ldc + col0 + row0 + threadIdx.x / MT;
            if (accumulate) atomicAdd(cptr, t);                 // one add per element by one thread, not waited for
            else *cptr = t;
        }
        __syncthreads();
    }
}

// ---- skinny GEMM for 3 <= M <= 32 activation rows: weight streaming through mma.sync ---------------------------
// out^T[16 rows of W, 8 activation rows] += W[16 x 16] * x^T[16 x 8] per instruction.  Each lane loads 16 contiguous
// bytes (8 values of K) of W rows g and g+8 and of activation row g straight from global memory; the 8 values feed two
// instructions.  Which physical k lands in which logical k-slot of the instruction does not matter for a dot product
// as long as both operands use the same assignment, and they do (same lane, same byte offsets), so no shuffle or
// shared-memory staging is needed and every weight byte is loaded exactly once.  Persistent warps, 16 rows each,
// NB groups of 8 activation rows re-use the weight registers.  Same dependent-launch protocol as tgp_wstream_kernel.
__device__ __forceinline__ void mma_bf16_16816(float *d, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int NB, int U>
__global__ void __launch_bounds__(256) tgp_wstream_mma_kernel(const bf16 *A, const bf16 *__restrict__ W, float *__restrict__ C,
                                                       uint32_t Mrows, uint32_t n, uint32_t K, uint32_t ldc, uint32_t col0, int accumulate) {
    const uint32_t lane = threadIdx.x & 31, g = lane >> 2, c = lane & 3;
    const uint32_t gwarp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarp = (gridDim.x * blockDim.x) >> 5;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool synced = false;
    for (uint32_t row0 = gwarp * 16; row0 < n; row0 += nwarp * 16) {
        const bf16 *wlo = W + (size_t)min(row0 + g, n - 1) * K + c * 8;        // tail rows re-read the last row, never stored
        const bf16 *whi = W + (size_t)min(row0 + g + 8, n - 1) * K + c * 8;
        float acc[NB][4];
#pragma unroll
        for (int b = 0; b < NB; ++b) { acc[b][0] = acc[b][1] = acc[b][2] = acc[b][3] = 0.f; }
        for (uint32_t k0 = 0; k0 < K; k0 += 32 * U) {
            uint4 lo[U], hi[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const bool in = k0 + 32 * u < K;
                lo[u] = in ? __ldcs(reinterpret_cast<const uint4 *>(wlo + k0 + 32 * u)) : make_uint4(0, 0, 0, 0);
                hi[u] = in ? __ldcs(reinterpret_cast<const uint4 *>(whi + k0 + 32 * u)) : make_uint4(0, 0, 0, 0);
            }
            if (!synced) { asm volatile("griddepcontrol.wait;" ::: "memory"); synced = true; }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t k = k0 + 32 * u;
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    const uint32_t m = b * 8 + g;
                    const uint4 xv = (k < K && m < Mrows) ? ld_act(reinterpret_cast<const uint4 *>(A + (size_t)m * K + k + c * 8)) : make_uint4(0, 0, 0, 0);
                    mma_bf16_16816(acc[b], lo[u].x, hi[u].x, lo[u].y, hi[u].y, xv.x, xv.y);
                    mma_bf16_16816(acc[b], lo[u].z, hi[u].z, lo[u].w, hi[u].w, xv.z, xv.w);
                }
            }
        }
        if (!synced) { asm volatile("griddepcontrol.wait;" ::: "memory"); synced = true; }
#pragma unroll
        for (int b = 0; b < NB; ++b)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t m = b * 8 + 2 * c + (i & 1), row = row0 + g + 8 * (i >> 1);
                if (m < Mrows && row < n) {
                    float *p = C + (size_t)m * ldc + col0 + row;
                    if (accumulate) atomicAdd(p, acc[b][i]);      // one add per element by one thread, not waited for
                    else *p = acc[b][i];
                }
            }
    }
}

// ---- generic tiled GEMM on CUDA cores (any M, n; K % 8 == 0): 64x64 tile, 4x4 per thread ---------
__global__ void __launch_bounds__(256) tgp_matmul_simt_kernel(const bf16 *A, const bf16 *__restrict__ W, float *__restrict__ C,
                                                        uint32_t M, uint32_t n, uint32_t K, uint32_t ldc, uint32_t col0, int accumulate) {
    __shared__ float As[32][64 + 4];
    __shared__ float Ws[32][64 + 4];
    const uint32_t m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
    const uint32_t tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    float acc[4][4] = {};
    const uint32_t lr = threadIdx.x >> 2, lk = (threadIdx.x & 3) * 8;     // 64 rows x 4 vectors of 8
    for (uint32_t k0 = 0; k0 < K; k0 += 32) {
        float fa[8], fw[8];
        uint4 va = make_uint4(0, 0, 0, 0), vw = va;
        if (m0 + lr < M && k0 + lk < K) va = *reinterpret_cast<const uint4 *>(A + (size_t)(m0 + lr) * K + k0 + lk);
        if (n0 + lr < n && k0 + lk < K) vw = *reinterpret_cast<const uint4 *>(W + (size_t)(n0 + lr) * K + k0 + lk);
        unpack8(va, fa); unpack8(vw, fw);
#pragma unroll
        for (int i = 0; i < 8; ++i) { As[lk + i][lr] = fa[i]; Ws[lk + i][lr] = fw[i]; }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 32; ++kk) {
            float a[4], w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = As[kk][ty * 4 + i]; w[i] = Ws[kk][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t m = m0 + ty * 4 + i, c = n0 + tx * 4 + j;
            if (m < M && c < n) { float *p = C + (size_t)m * ldc + col0 + c; *p = accumulate ? *p + acc[i][j] : acc[i][j]; }
        }
}

// ---- RoPE + bf16 rounding + KV append -----------------------------------------------------------
struct RopeArgs {
    const float *q32, *k32, *v32; bf16 *qb; const float *cos_t, *sin_t;
    uint32_t Hq, Hkv, Dh, TK, q_len, pos0;
    TgpTilePtrs tiles;
};

__global__ void tgp_rope_kv_kernel(RopeArgs a) {
    pdl_enter();
    const uint32_t m = blockIdx.x, b = m / a.q_len, pos = a.pos0 + m % a.q_len;
    const uint32_t half = a.Dh / 2, qd = a.Hq * a.Dh, kd = a.Hkv * a.Dh;
    const float *cs = a.cos_t + (size_t)pos * half, *sn = a.sin_t + (size_t)pos * half;
    const uint32_t j = pos / a.TK, slot = pos % a.TK;
    for (uint32_t idx = threadIdx.x; idx < (a.Hq + 2 * a.Hkv) * half; idx += blockDim.x) {
        const uint32_t h = idx / half, i = idx % half;
        if (h < a.Hq) {
            const float *s = a.q32 + (size_t)m * qd + h * a.Dh;
            float x0 = s[i], x1 = s[i + half], c = cs[i], sv = sn[i];
            bf16 *o = a.qb + (size_t)m * qd + h * a.Dh;
            o[i] = __float2bfloat16_rn(x0 * c - x1 * sv);
            o[i + half] = __float2bfloat16_rn(x1 * c + x0 * sv);
        } else if (h < a.Hq + a.Hkv) {
            const uint32_t hk = h - a.Hq;
            const float *s = a.k32 + (size_t)m * kd + hk * a.Dh;
            float x0 = s[i], x1 = s[i + half], c = cs[i], sv = sn[i];
            bf16 *o = reinterpret_cast<bf16 *>(a.tiles.k[j]) + ((size_t)(b * a.Hkv + hk) * a.TK + slot) * a.Dh;
            o[i] = __float2bfloat16_rn(x0 * c - x1 * sv);
            o[i + half] = __float2bfloat16_rn(x1 * c + x0 * sv);
        } else {
            const uint32_t hk = h - a.Hq - a.Hkv;
            const float *s = a.v32 + (size_t)m * kd + hk * a.Dh;
            bf16 *o = reinterpret_cast<bf16 *>(a.tiles.v[j]) + ((size_t)(b * a.Hkv + hk) * a.TK + slot) * a.Dh;
            o[i] = __float2bfloat16_rn(s[i]);
            o[i + half] = __float2bfloat16_rn(s[i + half]);
        }
    }
}

// ---- attention -------------------------------------------------------------------------------------
struct AttnArgs {
    const bf16 *qb; bf16 *ob; float *scratch;
    uint32_t Hq, Hkv, Dh, TK, q_len, pos0, n_tiles;
    float scale;
    TgpTilePtrs tiles;
    uint32_t n_parts;                 // partials per head the merge kernel reads; 0: one per KV tile with valid keys
};

// One warp per query row, 32 keys per pass: lane = key for the scores, lane = output dims for P.V.
template <int DH>
__global__ void __launch_bounds__(128) tgp_attn_rows_kernel(AttnArgs a) {
    __shared__ float qs[4][DH];
    const uint32_t w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t p = blockIdx.x * 4 + w, hq = blockIdx.y, b = blockIdx.z;
    const bool live = p < a.q_len;
    const uint32_t m = b * a.q_len + (live ? p : 0), hk = hq / (a.Hq / a.Hkv);
    const bf16 *q = a.qb + (size_t)m * a.Hq * DH + hq * DH;
    for (int i = lane; i < DH; i += 32) qs[w][i] = __bfloat162float(q[i]);
    __syncwarp();
    if (!live) return;
    const uint32_t nkeys = a.pos0 + p + 1;
    constexpr int DPL = DH / 32;
    float o[DPL];
#pragma unroll
    for (int i = 0; i < DPL; ++i) o[i] = 0.f;
    float mx = -INFINITY, l = 0.f;
    for (uint32_t j0 = 0; j0 < nkeys; j0 += 32) {
        const uint32_t j = j0 + lane;
        float s = -INFINITY;
        if (j < nkeys) {
            const uint4 *kr = reinterpret_cast<const uint4 *>(reinterpret_cast<const bf16 *>(a.tiles.k[j / a.TK]) + ((size_t)(b * a.Hkv + hk) * a.TK + j % a.TK) * DH);
            float acc = 0.f;
#pragma unroll
            for (int v = 0; v < DH / 8; ++v) {
                float f[8];
                unpack8(kr[v], f);
#pragma unroll
                for (int i = 0; i < 8; ++i) acc = fmaf(qs[w][v * 8 + i], f[i], acc);
            }
            s = acc * a.scale;
        }
        const float mnew = fmaxf(mx, warp_max(s));
        const float alpha = expf(mx - mnew);
        const float pj = (j < nkeys) ? expf(s - mnew) : 0.f;
        l = l * alpha + warp_sum(pj);
#pragma unroll
        for (int i = 0; i < DPL; ++i) o[i] *= alpha;
        const uint32_t cnt = min(32u, nkeys - j0);
        for (uint32_t t = 0; t < cnt; ++t) {
            const float pt = __shfl_sync(0xffffffffu, pj, t);
            const uint32_t jj = j0 + t;
            const bf16 *vr = reinterpret_cast<const bf16 *>(a.tiles.v[jj / a.TK]) + ((size_t)(b * a.Hkv + hk) * a.TK + jj % a.TK) * DH;
#pragma unroll
            for (int i = 0; i < DPL; ++i) o[i] = fmaf(pt, __bfloat162float(vr[lane + 32 * i]), o[i]);
        }
        mx = mnew;
    }
    bf16 *out = a.ob + (size_t)m * a.Hq * DH + hq * DH;
#pragma unroll
    for (int i = 0; i < DPL; ++i) out[lane + 32 * i] = __float2bfloat16_rn(o[i] / l);
}

// Decode (one query per sequence): grid (tile, kv head, batch).  The block has G x SPLIT warps: SPLIT warps share
// one query head of the group and take the tile's keys in strided 32-key passes (lane = key for the scores, lane =
// output dims for P.V, fully unrolled so a pass's V loads are in flight together); their partial (max, sum, o[Dh])
// meet in shared memory and one unnormalised partial per (query head, tile) goes to scratch.
template <int DH>
__global__ void tgp_attn_decode_partial_kernel(AttnArgs a, uint32_t SPLIT) {
    pdl_enter();
    extern __shared__ float dsm[];
    const uint32_t G = a.Hq / a.Hkv;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t g = warp / SPLIT, sp = warp % SPLIT;
    const uint32_t tile = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
    const uint32_t hq = hk * G + g;
    const uint32_t kvlen = a.pos0 + 1;
    const uint32_t nk = min(a.TK, kvlen - tile * a.TK);
    float *qs = dsm + g * DH;                               // [G][DH] query rows as fp32
    float *parts = dsm + G * DH;                            // [G][SPLIT][DH + 2]
    if (sp == 0) {
        const bf16 *q = a.qb + (size_t)b * a.Hq * DH + hq * DH;
        for (int i = lane; i < DH; i += 32) qs[i] = __bfloat162float(q[i]);
    }
    __syncthreads();
    constexpr int DPL = DH / 32;
    float o[DPL];
#pragma unroll
    for (int i = 0; i < DPL; ++i) o[i] = 0.f;
    float mx = -INFINITY, l = 0.f;
    const bf16 *kt = reinterpret_cast<const bf16 *>(a.tiles.k[tile]) + (size_t)(b * a.Hkv + hk) * a.TK * DH;
    const bf16 *vt = reinterpret_cast<const bf16 *>(a.tiles.v[tile]) + (size_t)(b * a.Hkv + hk) * a.TK * DH;
    for (uint32_t j0 = sp * 32; j0 < nk; j0 += SPLIT * 32) {
        const uint32_t j = j0 + lane;
        float s = -INFINITY;
        if (j < nk) {
            const uint4 *kr = reinterpret_cast<const uint4 *>(kt + (size_t)j * DH);
            float acc = 0.f;
#pragma unroll
            for (int v = 0; v < DH / 8; ++v) {
                float f[8];
                unpack8(kr[v], f);
#pragma unroll
                for (int i = 0; i < 8; ++i) acc = fmaf(qs[v * 8 + i], f[i], acc);
            }
            s = acc * a.scale;
        }
        const float mnew = fmaxf(mx, warp_max(s));
        const float alpha = expf(mx - mnew);
        const float pj = (j < nk) ? expf(s - mnew) : 0.f;
        l = l * alpha + warp_sum(pj);
#pragma unroll
        for (int i = 0; i < DPL; ++i) o[i] *= alpha;
        const uint32_t cnt = min(32u, nk - j0);
#pragma unroll
        for (uint32_t t = 0; t < 32; ++t) {                 // rows past the end re-read the last valid row with weight 0
            const float pt = __shfl_sync(0xffffffffu, pj, t);
            const bf16 *vr = vt + (size_t)(j0 + min(t, cnt - 1)) * DH;
#pragma unroll
            for (int i = 0; i < DPL; ++i) o[i] = fmaf(pt, __bfloat162float(vr[lane + 32 * i]), o[i]);
        }
        mx = mnew;
    }
    float *mine = parts + (size_t)(g * SPLIT + sp) * (DH + 2);
    if (lane == 0) { mine[0] = mx; mine[1] = l; }
#pragma unroll
    for (int i = 0; i < DPL; ++i) mine[2 + lane + 32 * i] = o[i];
    __syncthreads();
    if (sp == 0) {                                          // fixed-order merge of the SPLIT partials of this head
        const float *p0 = parts + (size_t)g * SPLIT * (DH + 2);
        float m = -INFINITY;
        for (uint32_t k = 0; k < SPLIT; ++k) m = fmaxf(m, p0[k * (DH + 2)]);
        float lsum = 0.f, acc[DPL];
#pragma unroll
        for (int i = 0; i < DPL; ++i) acc[i] = 0.f;
        for (uint32_t k = 0; k < SPLIT; ++k) {
            const float w = expf(p0[k * (DH + 2)] - m);     // a warp that saw no key has max -inf and weight 0
            lsum += w * p0[k * (DH + 2) + 1];
#pragma unroll
            for (int i = 0; i < DPL; ++i) acc[i] += w * p0[k * (DH + 2) + 2 + lane + 32 * i];
        }
        float *part = a.scratch + ((size_t)(b * a.Hq + hq) * a.n_tiles + tile) * (DH + 2);
        if (lane == 0) { part[0] = m; part[1] = lsum; }
#pragma unroll
        for (int i = 0; i < DPL; ++i) part[2 + lane + 32 * i] = acc[i];
    }
}

// Merge the per-tile partials of one (batch, query head): grid (Hq, B), DH threads.
// Decode attention over one KV tile for all G query heads of a KV head at once (G = Hq / Hkv in {1, 2, 4, 8}): the tile's
// K and V rows are read once, not once per query head.  One CTA per (tile, KV head, sequence); warp w walks the keys
// w*32, (w + SPLIT)*32, ... of the tile in chunks of 32: lane = key for the scores (the lane reads its whole K row with
// 16-byte loads, all in flight at once, and dots it with the G queries held in shared memory), then lane = DH/32
// consecutive output dimensions for P V (each V row is one coalesced warp load; the G weights of a key come by
// shuffle).  Per-warp online softmax; the SPLIT partials of a head are merged in warp order; output as in the
// per-head kernel: (max, sum, unnormalised o[DH]) per (sequence, head, tile) for tgp_attn_decode_merge_kernel.
template <int DH, int G>
__global__ void __launch_bounds__(256, 2) tgp_attn_decode_group_kernel(AttnArgs a, uint32_t SPLIT) {
    pdl_enter();
    extern __shared__ float dsm[];
    constexpr int DPL = DH / 32;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t tile = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
    const uint32_t kvlen = a.pos0 + 1;
    const uint32_t nk = min(a.TK, kvlen - tile * a.TK);
    float *qs = dsm;                                        // [G][DH] query rows as fp32
    float *parts = dsm + G * DH;                            // [G][SPLIT][DH + 2]
    {
        const bf16 *q = a.qb + ((size_t)b * a.Hq + hk * G) * DH;          // the G heads of this group are contiguous
        for (uint32_t i = threadIdx.x; i < G * DH; i += blockDim.x) qs[i] = __bfloat162float(q[i]);
    }
    __syncthreads();
    float o[G][DPL], mx[G], l[G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        mx[g] = -INFINITY; l[g] = 0.f;
#pragma unroll
        for (int i = 0; i < DPL; ++i) o[g][i] = 0.f;
    }
    const bf16 *kt = reinterpret_cast<const bf16 *>(a.tiles.k[tile]) + (size_t)(b * a.Hkv + hk) * a.TK * DH;
    const bf16 *vt = reinterpret_cast<const bf16 *>(a.tiles.v[tile]) + (size_t)(b * a.Hkv + hk) * a.TK * DH;
    for (uint32_t j0 = warp * 32; j0 < nk; j0 += SPLIT * 32) {
        const uint32_t j = j0 + lane, cnt = min(32u, nk - j0);
        const bool valid = j < nk;
        // the first 16 value rows are requested before the scores are computed: they depend on nothing computed here, and
        // the chunk is one serial chain per warp (key rows, scores, softmax, value rows), so every load moved off it counts
        typedef typename std::conditional<DPL == 4, uint2, uint32_t>::type vraw_t;
        constexpr uint32_t PRE = (G * DPL >= 32) ? 4 : 16;          // eight heads of 128 dimensions leave few registers for it
        vraw_t vpre[PRE];
#pragma unroll
        for (uint32_t t = 0; t < PRE; ++t)
            vpre[t] = *reinterpret_cast<const vraw_t *>(vt + (size_t)(j0 + min(t, cnt - 1)) * DH + lane * DPL);
        // ---- scores: this lane's key against the G queries ----
        float acc[G];
#pragma unroll
        for (int g = 0; g < G; ++g) acc[g] = 0.f;
        {
            const uint4 *kr = reinterpret_cast<const uint4 *>(kt + (size_t)min(j, nk - 1) * DH);
            uint4 kv[4], nx[4];                                      // 64 bytes of the row at a time, the next 64 already requested
#pragma unroll
            for (int v = 0; v < 4; ++v) kv[v] = kr[v];
#pragma unroll 1
            for (int v0 = 0; v0 < DH / 8; v0 += 4) {
                if (v0 + 4 < DH / 8) {
#pragma unroll
                    for (int v = 0; v < 4; ++v) nx[v] = kr[v0 + 4 + v];
                }
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    float f[8];
                    unpack8(kv[v], f);
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        const float4 q0 = *reinterpret_cast<const float4 *>(qs + g * DH + (v0 + v) * 8), q1 = *reinterpret_cast<const float4 *>(qs + g * DH + (v0 + v) * 8 + 4);
                        acc[g] = fmaf(q0.x, f[0], acc[g]); acc[g] = fmaf(q0.y, f[1], acc[g]); acc[g] = fmaf(q0.z, f[2], acc[g]); acc[g] = fmaf(q0.w, f[3], acc[g]);
                        acc[g] = fmaf(q1.x, f[4], acc[g]); acc[g] = fmaf(q1.y, f[5], acc[g]); acc[g] = fmaf(q1.z, f[6], acc[g]); acc[g] = fmaf(q1.w, f[7], acc[g]);
                    }
                }
#pragma unroll
                for (int v = 0; v < 4; ++v) kv[v] = nx[v];
            }
        }
        float p[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const float sc = valid ? acc[g] * a.scale : -INFINITY;
            const float mnew = fmaxf(mx[g], warp_max(sc));
            const float alpha = expf(mx[g] - mnew);
            p[g] = valid ? expf(sc - mnew) : 0.f;
            l[g] = l[g] * alpha + warp_sum(p[g]);
#pragma unroll
            for (int i = 0; i < DPL; ++i) o[g][i] *= alpha;
            mx[g] = mnew;
        }
        // ---- P V: this lane's DPL output dimensions; rows past the end re-read the last valid row with weight 0 ----
        vraw_t vlate[16];
#pragma unroll
        for (uint32_t t = 0; t < 16; ++t)
            vlate[t] = *reinterpret_cast<const vraw_t *>(vt + (size_t)(j0 + min(t + PRE, cnt - 1)) * DH + lane * DPL);
#pragma unroll
        for (uint32_t t = 0; t < 32; ++t) {
            if constexpr (PRE < 16) {                                // fewer than 16 rows were requested early: a third batch
                if (t == PRE + 16) {
#pragma unroll
                    for (uint32_t u = 0; u + PRE < 16; ++u)
                        vlate[u] = *reinterpret_cast<const vraw_t *>(vt + (size_t)(j0 + min(u + PRE + 16, cnt - 1)) * DH + lane * DPL);
                }
            }
            const vraw_t raw = t < PRE ? vpre[t % PRE] : vlate[(t - PRE) % 16];
            float f[DPL];
            if constexpr (DPL == 4) {
                const __nv_bfloat162 a0 = *reinterpret_cast<const __nv_bfloat162 *>(&raw.x), a1 = *reinterpret_cast<const __nv_bfloat162 *>(&raw.y);
                f[0] = __low2float(a0); f[1] = __high2float(a0); f[2] = __low2float(a1); f[3] = __high2float(a1);
            } else {
                const __nv_bfloat162 a0 = *reinterpret_cast<const __nv_bfloat162 *>(&raw);
                f[0] = __low2float(a0); f[1 % DPL] = __high2float(a0);
            }
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const float pt = __shfl_sync(0xffffffffu, p[g], t);
#pragma unroll
                for (int i = 0; i < DPL; ++i) o[g][i] = fmaf(pt, f[i], o[g][i]);
            }
        }
    }
#pragma unroll
    for (int g = 0; g < G; ++g) {
        float *mine = parts + (size_t)(g * SPLIT + warp) * (DH + 2);
        if (lane == 0) { mine[0] = mx[g]; mine[1] = l[g]; }
#pragma unroll
        for (int i = 0; i < DPL; ++i) mine[2 + lane * DPL + i] = o[g][i];
    }
    __syncthreads();
    for (uint32_t g = warp; g < G; g += SPLIT) {            // fixed-order merge of the SPLIT partials of head g
        const float *p0 = parts + (size_t)g * SPLIT * (DH + 2);
        float m = -INFINITY;
        for (uint32_t k = 0; k < SPLIT; ++k) m = fmaxf(m, p0[k * (DH + 2)]);
        float lsum = 0.f, accm[DPL];
#pragma unroll
        for (int i = 0; i < DPL; ++i) accm[i] = 0.f;
        for (uint32_t k = 0; k < SPLIT; ++k) {
            const float w = expf(p0[k * (DH + 2)] - m);     // a warp that saw no key has max -inf and weight 0
            lsum += w * p0[k * (DH + 2) + 1];
#pragma unroll
            for (int i = 0; i < DPL; ++i) accm[i] += w * p0[k * (DH + 2) + 2 + lane * DPL + i];
        }
        float *part = a.scratch + ((size_t)(b * a.Hq + hk * G + g) * a.n_tiles + tile) * (DH + 2);
        if (lane == 0) { part[0] = m; part[1] = lsum; }
#pragma unroll
        for (int i = 0; i < DPL; ++i) part[2 + lane * DPL + i] = accm[i];
    }
}

template <int DH>
__global__ void tgp_attn_decode_merge_kernel(AttnArgs a) {
    pdl_enter();
    const uint32_t hq = blockIdx.x, b = blockIdx.y, i = threadIdx.x;
    const uint32_t nt = a.n_parts ? a.n_parts : (a.pos0 + 1 + a.TK - 1) / a.TK;
    const float *part = a.scratch + (size_t)(b * a.Hq + hq) * a.n_tiles * (DH + 2);
    float mx = -INFINITY;
    for (uint32_t t = 0; t < nt; ++t) mx = fmaxf(mx, part[t * (DH + 2)]);
    float l = 0.f, o = 0.f;
    for (uint32_t t = 0; t < nt; ++t) {
        const float w = expf(part[t * (DH + 2)] - mx);
        l += w * part[t * (DH + 2) + 1];
        o += w * part[t * (DH + 2) + 2 + i];
    }
    a.ob[(size_t)b * a.Hq * DH + hq * DH + i] = __float2bfloat16_rn(o / l);
}

// ---- decode attention on the tensor cores (mma.sync), K and V staged through shared memory ---------------------------------
// The group kernel above is a latency chain: a warp's 32-key chunk is loads, 4*G*Dh FMAs per lane and shuffles, one after
// the other, and a B200 needs ~35 KB in flight per SM to keep HBM busy.  Here the G query heads of a KV head are the rows
// of a 16-row MMA tile (rows >= G are zero), a warp works on chunks of 16 keys, and the K and V rows of the next chunks are
// already on their way: every warp owns DEC_STAGES private stages that it fills with cp.async (16 bytes per lane and
// instruction, rows past the sequence zero-filled) - no block-wide barrier in the key loop.  Per chunk:
//   S[16 x 16 keys] = Q K^T      2 x Dh/16 MMAs (m16n8k16, bf16 -> fp32), K fragments by ldmatrix from the swizzled stage;
//   online softmax per row       (the running maximum moves rarely: O is rescaled only when a row's maximum grew);
//   O[16 x Dh] += P V            Dh/8 MMAs, P straight from the S accumulators as the A fragment, V fragments by
//                                ldmatrix.trans (V rows are keys: the transposed load makes keys the contraction index).
// P is rounded to bf16 for the second product, as in the prefill kernels.  A CTA of four warps owns a contiguous range of
// chunks of one (sequence, KV head); its warps take every fourth chunk, merge their four partials through shared memory
// and write one (max, sum, unnormalised O) per query head and CTA to the scratch array tgp_attn_decode_merge_kernel reads.
// Stage layout: row = key, 2*DH bytes, 16-byte chunk j of row r at chunk position j ^ (r & 7): conflict-free for the
// ldmatrix reads (eight rows, same j) and for the cp.async writes.
constexpr int DEC_STAGES = 3, DEC_WARPS = 4, DEC_KEYS = 16;

__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float fast_ex2(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }

template <int DH, int G>
__global__ void __launch_bounds__(DEC_WARPS * 32) tgp_attn_decode_mma_kernel(AttnArgs a, uint32_t chunks_per_cta) {
    pdl_enter();
    extern __shared__ __align__(128) uint8_t dec_sm[];
    constexpr uint32_t ROW = DH * 2, CPR = ROW / 16;                  // bytes and 16-byte chunks per key row
    constexpr uint32_t KV_BYTES = DEC_KEYS * ROW, STAGE = 2 * KV_BYTES;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31, r = lane >> 2, c = lane & 3;
    const uint32_t part = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
    const uint32_t kvlen = a.pos0 + 1, nchunks = (kvlen + DEC_KEYS - 1) / DEC_KEYS;
    const uint32_t q_lo = part * chunks_per_cta, q_hi = min(nchunks, q_lo + chunks_per_cta);
    uint8_t *mine = dec_sm + (size_t)warp * DEC_STAGES * STAGE;
    const uint32_t mine_u = (uint32_t)__cvta_generic_to_shared(mine);
    const float sl2 = a.scale * 1.4426950408889634f;                  // scores are kept in units of log2

    // Q fragments of this group: rows 0..G-1 real, the rest zero; held in registers for the whole kernel
    uint32_t qf[DH / 16][2];
    {
        const bf16 *q = a.qb + ((size_t)b * a.Hq + hk * G) * DH + (size_t)r * DH;
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks) {
            qf[ks][0] = r < G ? *reinterpret_cast<const uint32_t *>(q + ks * 16 + 2 * c) : 0u;
            qf[ks][1] = r < G ? *reinterpret_cast<const uint32_t *>(q + ks * 16 + 2 * c + 8) : 0u;
        }
    }
    // chunk q: its KV tile and offset; lane l copies 16-byte pieces idx = i * 32 + l of the chunk's K and V rows
    auto issue = [&](uint32_t q, uint32_t stage) {
        const uint32_t key0 = q * DEC_KEYS, tile = key0 / a.TK, off = key0 - tile * a.TK;
        const uint8_t *kg = reinterpret_cast<const uint8_t *>(a.tiles.k[tile]) + ((size_t)(b * a.Hkv + hk) * a.TK + off) * ROW;
        const uint8_t *vg = reinterpret_cast<const uint8_t *>(a.tiles.v[tile]) + ((size_t)(b * a.Hkv + hk) * a.TK + off) * ROW;
        const uint32_t base = mine_u + stage * STAGE;
#pragma unroll
        for (uint32_t i = 0; i < DEC_KEYS * CPR / 32; ++i) {
            const uint32_t idx = i * 32 + lane, row = idx / CPR, j = idx % CPR;
            const uint32_t dst = row * ROW + ((j ^ (row & 7)) << 4);
            const uint32_t nbytes = key0 + row < kvlen ? 16u : 0u;  // rows past the sequence are written as zeros, not read
            cp_async16(base + dst, kg + (size_t)row * ROW + j * 16, nbytes);
            cp_async16(base + KV_BYTES + dst, vg + (size_t)row * ROW + j * 16, nbytes);
        }
    };
    // this warp's chunks: q_lo + warp, q_lo + warp + 4, ...
    uint32_t issued = 0, total = 0;
    for (uint32_t q = q_lo + warp; q < q_hi; q += DEC_WARPS) ++total;
#pragma unroll
    for (int s = 0; s < DEC_STAGES - 1; ++s) {
        if (issued < total) { issue(q_lo + warp + issued * DEC_WARPS, issued % DEC_STAGES); ++issued; }
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    float o[DH / 8][4];
#pragma unroll
    for (int j = 0; j < DH / 8; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
    float m_run = -INFINITY, l_run = 0.f;                             // of row r (replicated over the four lanes of the row)
    for (uint32_t it = 0; it < total; ++it) {
        if (issued < total) { issue(q_lo + warp + issued * DEC_WARPS, issued % DEC_STAGES); ++issued; }
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group %0;" ::"n"(DEC_STAGES - 1) : "memory");
        __syncwarp();
        const uint32_t q = q_lo + warp + it * DEC_WARPS, key0 = q * DEC_KEYS;
        const uint32_t kb = mine_u + (it % DEC_STAGES) * STAGE, vb = kb + KV_BYTES;
        // ---- S = Q K^T: two n-tiles of 8 keys ----
        float sacc[2][4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.f;
#pragma unroll
            for (int kp = 0; kp < DH / 32; ++kp) {
                const uint32_t row = nt * 8 + (lane & 7), j = kp * 4 + (lane >> 3);
                uint32_t b0, b1, b2, b3;
                ldsm_x4(kb + row * ROW + ((j ^ (row & 7)) << 4), b0, b1, b2, b3);
                mma_bf16(sacc[nt], qf[2 * kp][0], 0u, qf[2 * kp][1], 0u, b0, b1);
                mma_bf16(sacc[nt], qf[2 * kp + 1][0], 0u, qf[2 * kp + 1][1], 0u, b2, b3);
            }
        }
        // ---- online softmax of row r over the chunk's 16 keys (this lane: keys 2c, 2c+1, 8+2c, 9+2c) ----
        float sv[4] = {sacc[0][0] * sl2, sacc[0][1] * sl2, sacc[1][0] * sl2, sacc[1][1] * sl2};
        if (key0 + DEC_KEYS > kvlen) {
            const uint32_t kk[4] = {2 * c, 2 * c + 1, 8 + 2 * c, 9 + 2 * c};
#pragma unroll
            for (int i = 0; i < 4; ++i) if (key0 + kk[i] >= kvlen) sv[i] = -INFINITY;
        }
        float mx = fmaxf(fmaxf(sv[0], sv[1]), fmaxf(sv[2], sv[3]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_run, mx);                          // finite: every chunk holds a valid key
        if (__any_sync(0xffffffffu, m_new > m_run)) {
            const float alpha = fast_ex2(m_run - m_new);              // first chunk: ex2(-inf) = 0 on zeros
            l_run *= alpha;
#pragma unroll
            for (int j = 0; j < DH / 8; ++j) { o[j][0] *= alpha; o[j][1] *= alpha; }
            m_run = m_new;
        }
        float p[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) p[i] = fast_ex2(sv[i] - m_run);
        float ls = (p[0] + p[1]) + (p[2] + p[3]);
        ls += __shfl_xor_sync(0xffffffffu, ls, 1);
        ls += __shfl_xor_sync(0xffffffffu, ls, 2);
        l_run += ls;
        __nv_bfloat162 plo = __floats2bfloat162_rn(p[0], p[1]), phi = __floats2bfloat162_rn(p[2], p[3]);
        const uint32_t pa0 = *reinterpret_cast<uint32_t *>(&plo), pa2 = *reinterpret_cast<uint32_t *>(&phi);
        // ---- O += P V: Dh/8 n-tiles, two per ldmatrix ----
#pragma unroll
        for (int jp = 0; jp < DH / 16; ++jp) {
            const uint32_t row = ((lane >> 3) & 1) * 8 + (lane & 7), j = 2 * jp + (lane >> 4);
            uint32_t v0, v1, v2, v3;
            ldsm_x4_t(vb + row * ROW + ((j ^ (row & 7)) << 4), v0, v1, v2, v3);
            mma_bf16(o[2 * jp], pa0, 0u, pa2, 0u, v0, v1);
            mma_bf16(o[2 * jp + 1], pa0, 0u, pa2, 0u, v2, v3);
        }
        __syncwarp();                                                 // the stage may be refilled two iterations from now
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    // ---- merge the four warps' partials (rows < G), write one partial per head for this CTA ----
    // (each warp's partial goes to the start of its own stages, which it no longer needs: [G][DH + 2] floats)
    __syncwarp();
    constexpr size_t WSTRIDE = (size_t)DEC_STAGES * STAGE / sizeof(float);
    float *wp = reinterpret_cast<float *>(dec_sm);
    if (r < G) {
        float *dst = wp + (size_t)warp * WSTRIDE + (size_t)r * (DH + 2);
        if (c == 0) { dst[0] = m_run; dst[1] = l_run; }
#pragma unroll
        for (int j = 0; j < DH / 8; ++j) { dst[2 + j * 8 + 2 * c] = o[j][0]; dst[2 + j * 8 + 2 * c + 1] = o[j][1]; }
    }
    __syncthreads();
    for (uint32_t e = threadIdx.x; e < G * DH; e += blockDim.x) {
        const uint32_t g = e / DH, d = e % DH;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < DEC_WARPS; ++w) M = fmaxf(M, wp[(size_t)w * WSTRIDE + (size_t)g * (DH + 2)]);
        float l = 0.f, acc = 0.f;
#pragma unroll
        for (int w = 0; w < DEC_WARPS; ++w) {
            const float *src = wp + (size_t)w * WSTRIDE + (size_t)g * (DH + 2);
            const float wgt = src[0] == -INFINITY ? 0.f : fast_ex2(src[0] - M);       // a warp without a chunk: weight 0
            l += wgt * src[1];
            acc += wgt * src[2 + d];
        }
        if (a.n_parts == 1) {                                              // the CTA saw the whole context: this is the result
            a.ob[((size_t)b * a.Hq + hk * G + g) * DH + d] = __float2bfloat16_rn(acc / l);
            continue;
        }
        float *out = a.scratch + ((size_t)(b * a.Hq + hk * G + g) * a.n_tiles + part) * (DH + 2);
        if (d == 0) { out[0] = M * 0.6931471805599453f; out[1] = l; }      // the merge kernel works in natural-log units
        out[2 + d] = acc;
    }
}

// ---- SwiGLU -----------------------------------------------------------------------------------------
__global__ void tgp_swiglu_kernel(const float4 *g, const float4 *u, __nv_bfloat162 *out, uint64_t n4) {
    pdl_enter();
    for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n4; i += (uint64_t)gridDim.x * blockDim.x) {
        float4 a = g[i], b = u[i];
        float r0 = a.x / (1.0f + expf(-a.x)) * b.x, r1 = a.y / (1.0f + expf(-a.y)) * b.y;
        float r2 = a.z / (1.0f + expf(-a.z)) * b.z, r3 = a.w / (1.0f + expf(-a.w)) * b.w;
        out[2 * i] = __floats2bfloat162_rn(r0, r1);
        out[2 * i + 1] = __floats2bfloat162_rn(r2, r3);
    }
}

// ---- argmax, lowest index on ties -----------------------------------------------------------------
__global__ void __launch_bounds__(1024) tgp_argmax_kernel(const float *logits, int32_t *out, uint32_t V) {
    pdl_enter();
    __shared__ float bv[32];
    __shared__ uint32_t bi[32];
    const float *row = logits + (size_t)blockIdx.x * V;
    // the index starts at 0, not at a sentinel: a row of NaNs (no comparison holds) must still give a legal token id
    float best = -INFINITY; uint32_t idx = 0u;
    for (uint32_t j = threadIdx.x; j < V; j += blockDim.x) { float v = row[j]; if (v > best || (v == best && j < idx)) { best = v; idx = j; } }
    auto merge = [](float &v, uint32_t &i, float ov, uint32_t oi) { if (ov > v || (ov == v && oi < i)) { v = ov; i = oi; } };
#pragma unroll
    for (int o = 16; o; o >>= 1) merge(best, idx, __shfl_xor_sync(0xffffffffu, best, o), __shfl_xor_sync(0xffffffffu, idx, o));
    if ((threadIdx.x & 31) == 0) { bv[threadIdx.x >> 5] = best; bi[threadIdx.x >> 5] = idx; }
    __syncthreads();
    if (threadIdx.x < 32) {
        best = threadIdx.x < (blockDim.x >> 5) ? bv[threadIdx.x] : -INFINITY;
        idx = threadIdx.x < (blockDim.x >> 5) ? bi[threadIdx.x] : 0u;
#pragma unroll
        for (int o = 16; o; o >>= 1) merge(best, idx, __shfl_xor_sync(0xffffffffu, best, o), __shfl_xor_sync(0xffffffffu, idx, o));
        if (threadIdx.x == 0) out[blockIdx.x] = (int32_t)idx;
    }
}

// ---- MoE: router, top-2, gates (one warp per token) ------------------------------------------------------
// logits[e] = sum_k h[m,k] * Wr[e,k] + bias[e] in fp32; the two largest (ties: lower expert id); gates = softmax
// over those two logits.
template <int E>
__global__ void __launch_bounds__(256) tgp_router_kernel(const bf16 *__restrict__ h, const bf16 *__restrict__ Wr, const float *__restrict__ bias,
                                                     int32_t *__restrict__ idx, float *__restrict__ gate, uint32_t M, uint32_t d, uint32_t topk) {
    const uint32_t m = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (m >= M) return;
    float acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;
    for (uint32_t k = lane * 8; k < d; k += 256) {
        float xf[8];
        unpack8(*reinterpret_cast<const uint4 *>(h + (size_t)m * d + k), xf);
#pragma unroll
        for (int e = 0; e < E; ++e) {
            float wf[8];
            unpack8(__ldg(reinterpret_cast<const uint4 *>(Wr + (size_t)e * d + k)), wf);
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[e] = fmaf(xf[i], wf[i], acc[e]);
        }
    }
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = warp_sum(acc[e]) + bias[e];
    if (lane == 0) {
        int i0 = 0;                                    // strict > while visiting ascending ids keeps the lower id on ties
#pragma unroll
        for (int e = 1; e < E; ++e) if (acc[e] > acc[i0]) i0 = e;
        if (E == 1 || topk == 1) {
            idx[2 * m] = i0; idx[2 * m + 1] = -1;
            gate[2 * m] = 1.0f; gate[2 * m + 1] = 0.0f;
        } else {
            int i1 = i0 == 0 ? 1 : 0;
#pragma unroll
            for (int e = 0; e < E; ++e) if (e != i0 && acc[e] > acc[i1]) i1 = e;
            const float e1 = expf(acc[i1] - acc[i0]);
            idx[2 * m] = i0; idx[2 * m + 1] = i1;
            gate[2 * m] = 1.0f / (1.0f + e1); gate[2 * m + 1] = e1 / (1.0f + e1);
        }
    }
}

// Tokens of expert e in ascending token order: rows[e*stride + pos] = m, gates[e*stride + pos] = that token's gate for e.
// One block per expert walks the tokens in chunks; positions come from a block-wide exclusive scan, so the
// grouping is deterministic.  topk = number of routed slots per token (1 or 2).
__global__ void __launch_bounds__(1024) tgp_route_fill_kernel(const int32_t *__restrict__ idx, const float *__restrict__ gate, int32_t *__restrict__ rows,
                                                          float *__restrict__ gates, int32_t *__restrict__ counts, uint32_t M, uint32_t stride, uint32_t topk) {
    __shared__ uint32_t warp_tot[32];
    __shared__ uint32_t base;
    const uint32_t e = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) base = 0;
    __syncthreads();
    for (uint32_t m0 = 0; m0 < M; m0 += blockDim.x) {
        const uint32_t m = m0 + threadIdx.x;
        int slot = -1;
        if (m < M) {
            if (idx[2 * m] == (int)e) slot = 0;
            else if (topk > 1 && idx[2 * m + 1] == (int)e) slot = 1;
        }
        const uint32_t bal = __ballot_sync(0xffffffffu, slot >= 0);
        const uint32_t before = __popc(bal & ((1u << lane) - 1));
        if (lane == 0) warp_tot[warp] = __popc(bal);
        __syncthreads();
        uint32_t woff = 0;
        for (uint32_t w = 0; w < warp; ++w) woff += warp_tot[w];
        const uint32_t b0 = base;
        if (slot >= 0) { rows[(size_t)e * stride + b0 + woff + before] = (int32_t)m; gates[(size_t)e * stride + b0 + woff + before] = gate[2 * m + slot]; }
        __syncthreads();
        if (threadIdx.x == 0) { uint32_t t = 0; for (uint32_t w = 0; w < (blockDim.x >> 5); ++w) t += warp_tot[w]; base = b0 + t; }
        __syncthreads();
    }
    if (threadIdx.x == 0) counts[e] = (int32_t)base;
}

__global__ void tgp_gather_rows_kernel(const bf16 *__restrict__ src, const int32_t *__restrict__ rows, bf16 *__restrict__ dst, uint32_t d) {
    const uint4 *s = reinterpret_cast<const uint4 *>(src + (size_t)rows[blockIdx.x] * d);
    uint4 *o = reinterpret_cast<uint4 *>(dst + (size_t)blockIdx.x * d);
    for (uint32_t i = threadIdx.x; i < d / 8; i += blockDim.x) o[i] = s[i];
}

// x[rows[i], :] += gates[i] * y[i, :]   (each token appears at most once per expert: no write conflicts)
__global__ void tgp_scatter_add_kernel(float *__restrict__ x, const float *__restrict__ y, const int32_t *__restrict__ rows, const float *__restrict__ gates, uint32_t d) {
    const float g = gates[blockIdx.x];
    float4 *o = reinterpret_cast<float4 *>(x + (size_t)rows[blockIdx.x] * d);
    const float4 *s = reinterpret_cast<const float4 *>(y + (size_t)blockIdx.x * d);
    for (uint32_t i = threadIdx.x; i < d / 4; i += blockDim.x) {
        float4 a = o[i];
        const float4 b = s[i];
        a.x += g * b.x; a.y += g * b.y; a.z += g * b.z; a.w += g * b.w;
        o[i] = a;
    }
}

// ============================ launchers (internal) ===================================================
int tgpk_router(const void *h, const void *Wr, const float *bias, int32_t *idx, float *gate, int32_t *rows, float *gates, int32_t *counts,
                uint32_t M, uint32_t stride, uint32_t d, uint32_t E, uint32_t topk, cudaStream_t st) {
    if (!M) return TGP_OK;
    if (d % 8 || topk < 1 || topk > 2) return TGP_E_INVAL;
    const uint32_t blocks = (M + 7) / 8;
    switch (E) {
    case 1: tgp_router_kernel<1><<<blocks, 256, 0, st>>>((const bf16 *)h, (const bf16 *)Wr, bias, idx, gate, M, d, topk); break;
    case 2: tgp_router_kernel<2><<<blocks, 256, 0, st>>>((const bf16 *)h, (const bf16 *)Wr, bias, idx, gate, M, d, topk); break;
    case 4: tgp_router_kernel<4><<<blocks, 256, 0, st>>>((const bf16 *)h, (const bf16 *)Wr, bias, idx, gate, M, d, topk); break;
    case 8: tgp_router_kernel<8><<<blocks, 256, 0, st>>>((const bf16 *)h, (const bf16 *)Wr, bias, idx, gate, M, d, topk); break;
    case 16: tgp_router_kernel<16><<<blocks, 256, 0, st>>>((const bf16 *)h, (const bf16 *)Wr, bias, idx, gate, M, d, topk); break;
    default: return TGP_E_INVAL;
    }
    tgp_route_fill_kernel<<<E, 1024, 0, st>>>(idx, gate, rows, gates, counts, M, stride, topk);
    LAUNCH_CHECK(2);
    return TGP_OK;
}

int tgpk_gather_rows(const void *src, const int32_t *rows, void *dst, uint32_t m, uint32_t d, cudaStream_t st) {
    if (!m) return TGP_OK;
    tgp_gather_rows_kernel<<<m, 128, 0, st>>>((const bf16 *)src, rows, (bf16 *)dst, d);
    LAUNCH_CHECK(1);
    return TGP_OK;
}

int tgpk_scatter_add(float *x, const float *y, const int32_t *rows, const float *gates, uint32_t m, uint32_t d, cudaStream_t st) {
    if (!m) return TGP_OK;
    tgp_scatter_add_kernel<<<m, 256, 0, st>>>(x, y, rows, gates, d);
    LAUNCH_CHECK(1);
    return TGP_OK;
}

int tgpk_embed(const void *table, const int32_t *tok, float *x, uint32_t M, uint32_t d, uint32_t V, cudaStream_t st) {
    if (!M) return TGP_OK;
    if (d % 8 || !V) return TGP_E_INVAL;
    launch_pdl(tgp_embed_kernel, dim3(M), dim3(128), 0, st, (const bf16 *)table, tok, x, d, V);
    LAUNCH_CHECK(1);
    return TGP_OK;
}

int tgpk_rmsnorm(const float *x, uint32_t ldx, const void *g, void *h, uint32_t M, uint32_t d, float eps, cudaStream_t st) {
    if (!M) return TGP_OK;
    if (d % 4 || ldx % 4) return TGP_E_INVAL;
    launch_pdl(tgp_rmsnorm_kernel, dim3(M), dim3(256), 0, st, x, ldx, (const bf16 *)g, (bf16 *)h, d, eps);
    LAUNCH_CHECK(1);
    return TGP_OK;
}

static int g_skinny_impl = 0;    // 0: tensor-core skinny kernel for 3 <= M <= 32; 1: CUDA-core GEMV (an on-device cross-check)
static int g_gemm_impl = 0;      // 0: tensor cores for M > 16; 1: CUDA-core tiles (kept as an on-device cross-check)
static int g_gemv_splitk = 1;    // small-n blocks at M <= 2: CTA per RB rows with K split over its warps (0: one warp per row)
static int g_gemm_group = 1;     // products over the same activations: one launch where the parts allow it (0: always one launch each)
static int g_gemv_balance = 1;   // grouped skinny launches: rows per group chosen so that every persistent CTA gets the same number of groups
static int g_gemv_pdl = 1;       // consecutive weight-streaming launches may overlap (programmatic dependent launch)

template <int MT, int R, int U>
static void launch_gemv(const bf16 *A, const bf16 *W, float *C, uint32_t Mrows, uint32_t n, uint32_t K, uint32_t ldc, uint32_t col0, int acc, cudaStream_t st) {
    static int blocks_per_sm = 0, sms = 0;
    if (!blocks_per_sm) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks_per_sm, tgp_wstream_kernel<MT, R, U>, 256, 0) != cudaSuccess || blocks_per_sm < 1) blocks_per_sm = 1;
        if (sms < 1) sms = 148;
    }
    uint32_t need = (n + R * 8 - 1) / (R * 8), full = (uint32_t)(sms * blocks_per_sm);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(need < full ? need : full);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = g_gemv_pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, tgp_wstream_kernel<MT, R, U>, A, W, C, Mrows, n, K, ldc, col0, acc);
    tgpk_last_gemm_kernel = "tgp_wstream_kernel";
}

// Same product for blocks with two to eight 16-row groups per SM: one CTA owns ROWS rows of W and its NW warps split K
// (interleaved chunks of 32*U), so n/ROWS CTAs of NW warps fill the machine where n/16 warps would not.  The partial
// tiles meet in shared memory and are summed in warp order: deterministic.  RPC <= ROWS: rows a CTA owns (the tile's
// remaining rows re-read its last row and are not stored; a row's sum does not depend on its place in the tile).
// (Blocks of fewer rows take tgp_wstream_mma_group_kernel.)
template <int NB, int U, int NW, int ROWS, int RPC = ROWS>
__global__ void __launch_bounds__(NW * 32) tgp_wstream_mma_splitk_kernel(const bf16 *A, const bf16 *__restrict__ W, float *__restrict__ C,
                                                              uint32_t Mrows, uint32_t n, uint32_t K, uint32_t ldc, uint32_t col0, int accumulate) {
    constexpr int UL = ROWS == 8 ? 2 * U : U;             // half a tile per load step: twice the steps in flight
    __shared__ float part[NW][NB * 4][32];
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, c = lane & 3;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool synced = false;
    for (uint32_t row0 = blockIdx.x * RPC; row0 < n; row0 += gridDim.x * RPC) {
        const uint32_t rlast = min(row0 + RPC, n) - 1;
        const bf16 *wlo = W + (size_t)min(row0 + g, rlast) * K + c * 8;
        const bf16 *whi = W + (size_t)min(row0 + g + 8, rlast) * K + c * 8;
        float acc[NB][4];
#pragma unroll
        for (int b = 0; b < NB; ++b) { acc[b][0] = acc[b][1] = acc[b][2] = acc[b][3] = 0.f; }
        for (uint32_t k0 = warp * 32 * UL; k0 < K; k0 += NW * 32 * UL) {
            uint4 lo[UL], hi[UL];
#pragma unroll
            for (int u = 0; u < UL; ++u) {
                const bool in = k0 + 32 * u < K;
                lo[u] = in ? __ldcs(reinterpret_cast<const uint4 *>(wlo + k0 + 32 * u)) : make_uint4(0, 0, 0, 0);
                hi[u] = (in && ROWS == 16) ? __ldcs(reinterpret_cast<const uint4 *>(whi + k0 + 32 * u)) : make_uint4(0, 0, 0, 0);   // ROWS == 8: the upper half of the tile stays empty
            }
            if (!synced) { asm volatile("griddepcontrol.wait;" ::: "memory"); synced = true; }
#pragma unroll
            for (int u = 0; u < UL; ++u) {
                const uint32_t k = k0 + 32 * u;
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    const uint32_t m = b * 8 + g;
                    const uint4 xv = (k < K && m < Mrows) ? ld_act(reinterpret_cast<const uint4 *>(A + (size_t)m * K + k + c * 8)) : make_uint4(0, 0, 0, 0);
                    mma_bf16_16816(acc[b], lo[u].x, hi[u].x, lo[u].y, hi[u].y, xv.x, xv.y);
                    mma_bf16_16816(acc[b], lo[u].z, hi[u].z, lo[u].w, hi[u].w, xv.z, xv.w);
                }
            }
        }
        if (!synced) { asm volatile("griddepcontrol.wait;" ::: "memory"); synced = true; }
#pragma unroll
        for (int b = 0; b < NB; ++b)
#pragma unroll
            for (int i = 0; i < 4; ++i) part[warp][b * 4 + i][lane] = acc[b][i];
        __syncthreads();
        for (uint32_t v = threadIdx.x; v < NB * 4 * 32; v += NW * 32) {
            const uint32_t slot = v >> 5, ln = v & 31, b = slot >> 2, i = slot & 3;
            float sum = 0.f;
#pragma unroll
            for (int w = 0; w < NW; ++w) sum += part[w][slot][ln];
            const uint32_t m = b * 8 + 2 * (ln & 3) + (i & 1), row = row0 + (ln >> 2) + 8 * (i >> 1);
            if (m < Mrows && row < n && (RPC == ROWS || row < row0 + RPC) && (ROWS == 16 || (i >> 1) == 0)) {
                float *p = C + (size_t)m * ldc + col0 + row;
                if (accumulate) atomicAdd(p, sum);               // one add per element by one thread, not waited for
                else *p = sum;
            }
        }
        __syncthreads();
    }
}

// The product for blocks of fewer than two 16-row groups per SM, one block or a list of blocks that read the same
// activations (the pieces of one matrix; the q, k and v projections): one persistent CTA per SM walks the row groups
// as one list, RG consecutive groups at a time, whose MMAs share each activation fragment - every CTA reads its K
// slices of all activation rows from L2, so at 16 rows per CTA that traffic equals the weights'; RG row groups divide
// it by RG.  K is split over the CTA's NW warps in interleaved chunks of 32*U columns and the partial tiles are summed
// in warp order.  A group's arithmetic (which warp adds which k, in which order) depends on NB, U, NW and K alone -
// not on RG, the rows per group or the list: a block gives the same bits alone or in any list.
template <int NB, int U, int NW, int ROWS, int RG>
__global__ void __launch_bounds__(NW * 32) tgp_wstream_mma_group_kernel(const bf16 *A, const GemvParts p, uint32_t Mrows, uint32_t groups_total,
                                                              uint32_t K, int accumulate, uint32_t rpc, int acts_early) {
    constexpr int UL = ROWS == 8 ? 2 * U : U;             // half a tile per load step: twice the steps in flight
    constexpr int G = RG, SK = UL / (2 * G);              // a register set holds SK load steps of G groups: two sets are as many loads as UL steps of one group
    static_assert(UL % (2 * G) == 0 && SK >= 1, "row groups per CTA must divide half the load steps");
    // the warps' partial tiles: static where they fit the 48 KB a kernel may declare, else the launch's dynamic shared memory
    constexpr bool PART_DYNAMIC = (size_t)NW * G * NB * 4 * 32 * 4 > 48 * 1024;
    __shared__ float part_static[PART_DYNAMIC ? 1 : NW * G * NB * 4 * 32];
    extern __shared__ float part_dynamic[];
    float (*part)[G * NB * 4][32] = reinterpret_cast<float (*)[G * NB * 4][32]>(PART_DYNAMIC ? part_dynamic : part_static);
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, c = lane & 3;
    uint32_t grp0 = blockIdx.x * G;
    if (grp0 >= groups_total) return;
    const bf16 *wlo[G], *whi[G];
    uint4 lo[2][G][SK], hi[2][G][SK];                     // two register sets of SK load steps of every group
    // the activation fragments of a set are loaded with its weights (they come from L2 more often than from L1 -
    // a long K does not fit there - and would otherwise be waited for inside the MMA sequence)
    constexpr bool XPRE = !(NB >= 2 && G == 1);           // (those instances have no registers left for them)
    uint4 xs[2][XPRE ? SK : 1][XPRE ? NB : 1];
    float acc[G][NB][4];
    // which block a group belongs to: looked up here for the weights and again after the K loop for the output, so
    // that the output's pointer and stride do not occupy registers while the loads are in flight
    auto locate = [&](uint32_t first) {
#pragma unroll
        for (int r = 0; r < G; ++r) {
            const uint32_t grp = min(first + r, groups_total - 1);         // a group past the end re-reads the last one, never stored
            const bf16 *W = p.W[0];
            uint32_t n = p.n[0], local = grp;
            {
                uint32_t start = p.groups[0];
#pragma unroll
                for (int s = 1; s < (int)TGP_GEMM_GROUP_MAX; ++s)
                    if (s < (int)p.count) {
                        if (grp >= start) { W = p.W[s]; n = p.n[s]; local = grp - start; }
                        start += p.groups[s];
                    }
            }
            // rpc <= ROWS rows per group, chosen by the launcher so that the persistent CTAs all get the same number of
            // groups; the tile's rows beyond rpc re-read the group's last row and are not stored (a row's sum does not
            // depend on its place in the tile)
            const uint32_t rlast = min(local * rpc + rpc, n) - 1;
            wlo[r] = W + (size_t)min(local * rpc + g, rlast) * K + c * 8;
            whi[r] = W + (size_t)min(local * rpc + g + 8, rlast) * K + c * 8;
        }
    };
    auto issue = [&](auto set, uint32_t kb) {              // SK load steps of every group, from column kb on, into one register set
        constexpr int S = decltype(set)::value;
#pragma unroll
        for (int u = 0; u < SK; ++u) {
            const uint32_t k = kb + 32 * u;
#pragma unroll
            for (int r = 0; r < G; ++r) {
                lo[S][r][u] = k < K ? __ldcs(reinterpret_cast<const uint4 *>(wlo[r] + k)) : make_uint4(0, 0, 0, 0);
                hi[S][r][u] = (k < K && ROWS == 16) ? __ldcs(reinterpret_cast<const uint4 *>(whi[r] + k)) : make_uint4(0, 0, 0, 0);   // ROWS == 8: the upper half of the tile stays empty
            }
        }
    };
    auto issue_act = [&](auto set, uint32_t kb) {          // the activation fragments that go with a set; only after griddepcontrol.wait
        constexpr int S = decltype(set)::value;
        if constexpr (XPRE) {
#pragma unroll
            for (int u = 0; u < SK; ++u) {
                const uint32_t k = kb + 32 * u;
#pragma unroll
                for (int b = 0; b < NB; ++b)
                    xs[S][u][b] = (k < K && b * 8 + g < Mrows) ? ld_act(reinterpret_cast<const uint4 *>(A + (size_t)(b * 8 + g) * K + k + c * 8)) : make_uint4(0, 0, 0, 0);
            }
        }
    };
    auto consume = [&](auto set, uint32_t kb) {
        constexpr int S = decltype(set)::value;
#pragma unroll
        for (int u = 0; u < SK; ++u) {
            const uint32_t k = kb + 32 * u;
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                const uint32_t m = b * 8 + g;
                uint4 xv;
                if constexpr (XPRE) xv = xs[S][u][b];
                else xv = (k < K && m < Mrows) ? ld_act(reinterpret_cast<const uint4 *>(A + (size_t)m * K + k + c * 8)) : make_uint4(0, 0, 0, 0);
#pragma unroll
                for (int r = 0; r < G; ++r) {
                    mma_bf16_16816(acc[r][b], lo[S][r][u].x, hi[S][r][u].x, lo[S][r][u].y, hi[S][r][u].y, xv.x, xv.y);
                    mma_bf16_16816(acc[r][b], lo[S][r][u].z, hi[S][r][u].z, lo[S][r][u].w, hi[S][r][u].w, xv.z, xv.w);
                }
            }
        }
    };
    auto clear = [&]() {
#pragma unroll
        for (int r = 0; r < G; ++r)
#pragma unroll
            for (int b = 0; b < NB; ++b) { acc[r][b][0] = acc[r][b][1] = acc[r][b][2] = acc[r][b][3] = 0.f; }
    };
    const std::integral_constant<int, 0> set0;
    const std::integral_constant<int, 1> set1;
    // One stream of loads over all the groups this CTA takes.  A warp's chunk of 32 * UL columns is G pairs of load steps;
    // the two register sets alternate, a set is loaded again as soon as its MMAs are issued, so a warp always has one
    // or two sets in flight - also across the end of a group: the next group's first pair is on its way while the CTA
    // meets in shared memory to sum and store the group it has finished, and the memory pipe never drains.  Per group
    // the k order of a warp's additions is that of its chunks, ascending: the bits do not depend on the pairing.  A warp
    // whose first chunk lies beyond K runs one pair of zeros (the sums do not change).
    uint32_t grp = grp0, k0 = warp * 32 * UL, pr = 0;       // the pair that is loaded next: group, chunk, pair within the chunk
    auto advance = [&]() -> bool {                         // moves on by one pair; true: the pair just passed ended its group
        if (++pr == (uint32_t)G) { pr = 0; k0 += NW * 32 * UL; }
        if (k0 < K) return false;
        grp += gridDim.x * G;
        k0 = warp * 32 * UL;
        pr = 0;
        if (grp < groups_total) locate(grp);
        return true;
    };
    locate(grp);
    uint32_t kb_cur = k0;
    issue(set0, kb_cur);
    issue(set1, kb_cur + 32 * SK);
    bool cur_last = advance();
    // Weights are never written by a kernel, so they are requested before the previous launch of the stream has finished.
    // The activations are read after it has - unless the launcher knows that they are older than that launch (it read the
    // same activations): then they are requested with the weights.  The next launch is released only here, after the wait:
    // when it starts, everything before this launch is complete, which is what lets it read its activations early in turn.
    if (acts_early) { issue_act(set0, kb_cur); issue_act(set1, kb_cur + 32 * SK); }
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (!acts_early) { issue_act(set0, kb_cur); issue_act(set1, kb_cur + 32 * SK); }
    clear();
    for (;;) {
        const bool have_next = grp < groups_total;
        const uint32_t kb_next = k0 + pr * 64 * SK;
        consume(set0, kb_cur);
        if (have_next) { issue(set0, kb_next); issue_act(set0, kb_next); }
        consume(set1, kb_cur + 32 * SK);
        if (have_next) { issue(set1, kb_next + 32 * SK); issue_act(set1, kb_next + 32 * SK); }
        const bool next_last = have_next ? advance() : false;
        kb_cur = kb_next;
        if (!cur_last) { cur_last = next_last; continue; }
        cur_last = next_last;
        // this warp has finished the group(s) at grp0
#pragma unroll
        for (int r = 0; r < G; ++r)
#pragma unroll
            for (int b = 0; b < NB; ++b)
#pragma unroll
                for (int i = 0; i < 4; ++i) part[warp][(r * NB + b) * 4 + i][lane] = acc[r][b][i];
        __syncthreads();
        for (uint32_t v = threadIdx.x; v < G * NB * 4 * 32; v += NW * 32) {
            const uint32_t slot = v >> 5, ln = v & 31, r = slot / (NB * 4), b = (slot >> 2) % NB, i = slot & 3;
            const uint32_t gi = grp0 + r;
            if (gi >= groups_total) continue;
            float sum = 0.f;
#pragma unroll
            for (int w = 0; w < NW; ++w) sum += part[w][slot][ln];
            float *C = p.C[0];
            uint32_t ldc = p.ldc[0], n = p.n[0], row0 = gi * rpc;
            {
                uint32_t start = p.groups[0];
#pragma unroll
                for (int s = 1; s < (int)TGP_GEMM_GROUP_MAX; ++s)
                    if (s < (int)p.count) {
                        if (gi >= start) { C = p.C[s]; ldc = p.ldc[s]; n = p.n[s]; row0 = (gi - start) * rpc; }
                        start += p.groups[s];
                    }
            }
            const uint32_t m = b * 8 + 2 * (ln & 3) + (i & 1), row = row0 + (ln >> 2) + 8 * (i >> 1);
            if (m < Mrows && row < min(row0 + rpc, n) && (ROWS == 16 || (i >> 1) == 0)) {
                float *out = C + (size_t)m * ldc + row;
                if (accumulate) atomicAdd(out, sum);             // one add per element by one thread, not waited for
                else *out = sum;
            }
        }
        grp0 += gridDim.x * G;
        if (grp0 >= groups_total) break;
        __syncthreads();
        clear();
    }
}

// Which skinny kernel serves a block of n rows at M activation rows: NB groups of 8 activation rows, U load steps in
// flight, and for blocks too small to give every SM eight 16-row warps the split-K kernel with NW warps per CTA over
// ROWS rows.  The choice depends on the block alone, so a block computes the same bits alone or as part of a group.
struct SkinnyPick { int nb, u, nw, rows; bool split, persistent; };

static int device_sms() {
    static int sms = 0;
    if (!sms) { int dev = 0; cudaGetDevice(&dev); if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) sms = 148; }
    return sms;
}

static SkinnyPick pick_skinny(uint32_t M, uint32_t n, uint32_t K) {
    const uint32_t sms = (uint32_t)device_sms(), groups16 = (n + 15) / 16;
    SkinnyPick k;
    k.nb = M <= 8 ? 1 : M <= 16 ? 2 : 4;
    k.split = n < 16u * 8u * sms;                         // too few 16-row groups to give every SM eight warps
    // fewer than two 16-row groups per SM: one persistent CTA per SM walks the row groups of the block, or of a list of such
    // blocks (tgp_wstream_mma_group_kernel).  One choice per class of M for all of them, so that the pieces of a matrix share
    // a launch whatever the rows of its last piece:
    //   M <= 8   16 warps, 8 load steps per warp and chunk
    //   M <= 16  8 warps of twice the registers, 16 load steps: room for the activation fragments of a register set
    //   M <= 32  the same with 8 load steps (four groups of activation rows take the registers)
    k.persistent = k.split && groups16 < 2u * sms;
    if (k.persistent) {
        k.nw = k.nb == 1 ? 16 : 8;
        k.u = k.nb == 1 ? 8 : k.nb == 2 ? 16 : 8;
        k.rows = 16;
    } else {
        k.nw = 8;
        k.u = M <= 16 ? 4 : 2;
        k.rows = 16;
    }
    return k;
}

template <int NB, int U>
static void launch_skinny(const bf16 *A, GemvParts p, const SkinnyPick &k, uint32_t Mrows, uint32_t K, int acc, cudaStream_t st) {
    static int blocks_per_sm = 0, blocks_per_sm_split = 0;
    constexpr bool STREAMS = U <= 4;                         // the load depths of the kernels that are not persistent
    if constexpr (STREAMS) {
        if (!blocks_per_sm && (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks_per_sm, tgp_wstream_mma_kernel<NB, U>, 256, 0) != cudaSuccess || blocks_per_sm < 1)) blocks_per_sm = 1;
        if (!blocks_per_sm_split && (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks_per_sm_split, tgp_wstream_mma_splitk_kernel<NB, U, 8, 16>, 256, 0) != cudaSuccess || blocks_per_sm_split < 1))
            blocks_per_sm_split = 1;
    }
    const uint32_t sms = (uint32_t)device_sms();
    uint32_t need = 0, rows_total = 0, rpc = (uint32_t)k.rows;
    if (k.split) for (uint32_t s = 0; s < p.count; ++s) { p.groups[s] = (p.n[s] + k.rows - 1) / k.rows; need += p.groups[s]; rows_total += p.n[s]; }
    else need = (p.n[0] + 16 * 8 - 1) / (16 * 8);           // whole blocks of many rows are launched alone
    const bool persistent = k.persistent;                   // one block or several: the kernel that walks a list of row groups
    // (the persistent kernels use the whole register file: one CTA per SM)
    const uint32_t full = persistent ? sms : sms * (uint32_t)(k.split ? blocks_per_sm_split : blocks_per_sm);
    uint32_t per_cta = 1;
    if (persistent) {
        // The grid is one persistent CTA per SM, each walking its share of the row groups, G groups at a time whose MMAs share
        // each activation fragment (every CTA reads its K slices of all activation rows per round, so at one group per round
        // that traffic equals the weights').  Rows per group r <= the tile's rows: fewer rows make more groups, so that a
        // block of few rows reaches every SM and no CTA waits for the others' last round (4096 rows: 256 groups of 16 leave
        // 40 SMs one round short, 293 of 14 do not) - but the rows a tile lacks still occupy its load slots (their lanes
        // re-read the group's last row; fewer than 9 rows per group measured no faster for blocks of few rows).  G and r are the
        // pair with the least estimated time of the busiest CTA: rounds x (G x (r + tile rows) / 2 + 4 NB), in rows read.
        const uint32_t tile = (uint32_t)k.rows, gmax = NB == 1 ? 2 : 4;
        uint32_t best = 0xffffffffu, best_r = tile;
        for (uint32_t G = gmax; G >= 1; G >>= 1)
            for (uint32_t r = g_gemv_balance ? tile / 2 + 1 : tile; r <= tile; ++r) {
                uint32_t groups = 0;
                for (uint32_t s = 0; s < p.count; ++s) groups += (p.n[s] + r - 1) / r;
                const uint32_t ctas = (groups + G - 1) / G, rounds = (ctas + full - 1) / full;
                const uint32_t cost = rounds * (G * (r + tile) + 8 * NB);           // twice the estimate
                if (cost < best) { best = cost; best_r = r; per_cta = G; }
            }
        rpc = best_r;
        need = 0;
        for (uint32_t s = 0; s < p.count; ++s) { p.groups[s] = (p.n[s] + rpc - 1) / rpc; need += p.groups[s]; }
        need = (need + per_cta - 1) / per_cta;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(need < full ? need : full);
    cfg.blockDim = dim3(k.split ? k.nw * 32 : 256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = g_gemv_pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    uint32_t total = 0;
    for (uint32_t s = 0; k.split && s < p.count; ++s) total += p.groups[s];
    // the previous launch of this thread was a product of this family over the same activations on the same stream, and the
    // caller vouches that nothing else was enqueued there in between: the activations are older than that launch
    const int early = persistent && tgpk_chain_ok && g_gemv_pdl && g_chain.A == (const void *)A && g_chain.st == st && g_chain.launches_before + 1 == tgpk_launches;
    if (persistent) { g_chain.A = A; g_chain.st = st; g_chain.launches_before = tgpk_launches; }
    else g_chain.A = nullptr;
    tgpk_last_gemm_kernel = !k.split ? "tgp_wstream_mma_kernel" : persistent ? "tgp_wstream_mma_group_kernel" : "tgp_wstream_mma_splitk_kernel";
    if (persistent) {
        if constexpr (NB == 1 && U == 8) {
            if (per_cta == 2) cudaLaunchKernelEx(&cfg, tgp_wstream_mma_group_kernel<NB, U, 16, 16, 2>, A, p, Mrows, total, K, acc, rpc, early);
            else cudaLaunchKernelEx(&cfg, tgp_wstream_mma_group_kernel<NB, U, 16, 16, 1>, A, p, Mrows, total, K, acc, rpc, early);
        } else if constexpr (NB == 2 && U == 16) {
            if (per_cta == 4) cudaLaunchKernelEx(&cfg, tgp_wstream_mma_group_kernel<NB, U, 8, 16, 4>, A, p, Mrows, total, K, acc, rpc, early);
            else if (per_cta == 2) cudaLaunchKernelEx(&cfg, tgp_wstream_mma_group_kernel<NB, U, 8, 16, 2>, A, p, Mrows, total, K, acc, rpc, early);
            else cudaLaunchKernelEx(&cfg, tgp_wstream_mma_group_kernel<NB, U, 8, 16, 1>, A, p, Mrows, total, K, acc, rpc, early);
        } else if constexpr (NB == 4 && U == 8) {
            if (per_cta == 4) {
                // four groups of 32 activation rows: the warps' partial tiles take 64 KB of dynamic shared memory
                constexpr size_t smem = (size_t)8 * 4 * NB * 4 * 32 * 4;
                static bool attr_set = false;
                if (!attr_set) { cudaFuncSetAttribute(tgp_wstream_mma_group_kernel<NB, U, 8, 16, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); attr_set = true; }
                cfg.dynamicSmemBytes = smem;
                cudaLaunchKernelEx(&cfg, tgp_wstream_mma_group_kernel<NB, U, 8, 16, 4>, A, p, Mrows, total, K, acc, rpc, early);
            } else if (per_cta == 2) cudaLaunchKernelEx(&cfg, tgp_wstream_mma_group_kernel<NB, U, 8, 16, 2>, A, p, Mrows, total, K, acc, rpc, early);
            else cudaLaunchKernelEx(&cfg, tgp_wstream_mma_group_kernel<NB, U, 8, 16, 1>, A, p, Mrows, total, K, acc, rpc, early);
        }
    } else if constexpr (STREAMS) {
        if (!k.split) cudaLaunchKernelEx(&cfg, tgp_wstream_mma_kernel<NB, U>, A, p.W[0], p.C[0], Mrows, p.n[0], K, p.ldc[0], 0u, acc);
        else cudaLaunchKernelEx(&cfg, tgp_wstream_mma_splitk_kernel<NB, U, 8, 16>, A, p.W[0], p.C[0], Mrows, p.n[0], K, p.ldc[0], 0u, acc);
    }
}

static void launch_skinny_pick(const bf16 *A, const GemvParts &p, const SkinnyPick &k, uint32_t Mrows, uint32_t K, int acc, cudaStream_t st) {
    if (k.nb == 1) { if (k.u == 8) launch_skinny<1, 8>(A, p, k, Mrows, K, acc, st); else launch_skinny<1, 4>(A, p, k, Mrows, K, acc, st); }
    else if (k.nb == 2) { if (k.u == 16) launch_skinny<2, 16>(A, p, k, Mrows, K, acc, st); else launch_skinny<2, 4>(A, p, k, Mrows, K, acc, st); }
    else { if (k.u == 8) launch_skinny<4, 8>(A, p, k, Mrows, K, acc, st); else launch_skinny<4, 2>(A, p, k, Mrows, K, acc, st); }
}

template <int MT, int RB, int U>
static void launch_gemv_splitk(const bf16 *A, const bf16 *W, float *C, uint32_t Mrows, uint32_t n, uint32_t K, uint32_t ldc, uint32_t col0, int acc, cudaStream_t st) {
    static int blocks_per_sm = 0, sms = 0;
    if (!blocks_per_sm) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks_per_sm, tgp_wstream_splitk_kernel<MT, RB, U>, 256, 0) != cudaSuccess || blocks_per_sm < 1) blocks_per_sm = 1;
        if (sms < 1) sms = 148;
    }
    uint32_t need = (n + RB - 1) / RB, full = (uint32_t)(sms * blocks_per_sm);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(need < full ? need : full);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = g_gemv_pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, tgp_wstream_splitk_kernel<MT, RB, U>, A, W, C, Mrows, n, K, ldc, col0, acc);
    tgpk_last_gemm_kernel = "tgp_wstream_splitk_kernel";
}

// rows per warp: fewer when the block has few rows, so that every SM still gets warps
template <int MT>
static void launch_gemv_rows(const bf16 *A, const bf16 *W, float *C, uint32_t Mrows, uint32_t n, uint32_t K, uint32_t ldc, uint32_t col0, int acc, cudaStream_t st) {
    if constexpr (MT <= 2) {
        if (n >= 2 * 148 * 16) return launch_gemv<MT, 2, 4>(A, W, C, Mrows, n, K, ldc, col0, acc, st);
        if (g_gemv_splitk && K >= 8192) {                    // at least four 256-element chunks per warp and row
            if (n <= 1024) return launch_gemv_splitk<MT, 1, 4>(A, W, C, Mrows, n, K, ldc, col0, acc, st);
            return launch_gemv_splitk<MT, 2, 4>(A, W, C, Mrows, n, K, ldc, col0, acc, st);
        }
        return launch_gemv<MT, 1, 8>(A, W, C, Mrows, n, K, ldc, col0, acc, st);
    } else {
        if (n >= 2 * 148 * 16) return launch_gemv<MT, 2, 2>(A, W, C, Mrows, n, K, ldc, col0, acc, st);
        return launch_gemv<MT, 1, 4>(A, W, C, Mrows, n, K, ldc, col0, acc, st);
    }
}

template <int MT>
static void launch_gemv_group(const bf16 *A, const GemvParts &p, uint32_t Mrows, uint32_t n_total, uint32_t K, int acc, cudaStream_t st, const ASrc &src = ASrc{}) {
    static int blocks_per_sm = 0, sms = 0;
    if (!blocks_per_sm) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks_per_sm, tgp_wstream_group_kernel<MT, 8>, 256, 0) != cudaSuccess || blocks_per_sm < 1) blocks_per_sm = 1;
        if (sms < 1) sms = 148;
    }
    uint32_t need = (n_total + 7) / 8, full = (uint32_t)(sms * blocks_per_sm);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(need < full ? need : full);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = g_gemv_pdl ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, tgp_wstream_group_kernel<MT, 8>, A, p, Mrows, n_total, K, acc, src);
    tgpk_last_gemm_kernel = "tgp_wstream_group_kernel";
}

// Which products may share a launch: those with the same non-zero key.  A key names the kernel a block takes on its own
// (M <= 2: tgp_wstream_kernel<MT, 1, 8>; 3 <= M <= 32: one instance of the split-K skinny kernel); blocks of so many rows that
// they fill the machine alone, and the shapes served by other kernels, have key 0 and are launched alone.
uint32_t tgpk_gemm_group_key(uint32_t M, uint32_t n, uint32_t K) {
    if (!g_gemm_group || !M || !n || !K || K % 8) return 0;
    if (M >= 3 && M <= 32 && K % 32 == 0 && g_skinny_impl == 0) {
        const SkinnyPick k = pick_skinny(M, n, K);
        // the blocks served by the persistent 16-warp kernel, which walks the row groups of any number of blocks
        return k.persistent ? (0x1000000u | (uint32_t)k.nb | (uint32_t)k.u << 4 | (uint32_t)k.nw << 8 | (uint32_t)k.rows << 16) : 0;
    }
    if (M <= 2) return (n < 2 * 148 * 16 && !(g_gemv_splitk && K >= 8192)) ? M : 0;
    return 0;
}

int tgpk_gemm_group(const void *A, uint32_t count, const void *const *W, float *const *C, const uint32_t *n, const uint32_t *ldc, uint32_t M, uint32_t K,
                    int accumulate, cudaStream_t st) {
    if (!count || !M) return TGP_OK;
    const uint32_t key = tgpk_gemm_group_key(M, n[0], K);
    bool same = key != 0 && count >= 2 && count <= TGP_GEMM_GROUP_MAX;
    for (uint32_t s = 1; s < count && same; ++s) same = tgpk_gemm_group_key(M, n[s], K) == key;
    if (!same) {
        for (uint32_t s = 0; s < count; ++s) {
            const int rc = tgpk_gemm(A, W[s], C[s], M, n[s], K, ldc[s], 0, accumulate, st);
            if (rc) return rc;
        }
        return TGP_OK;
    }
    GemvParts p;
    memset(&p, 0, sizeof(p));
    uint32_t total = 0;
    for (uint32_t s = 0; s < count; ++s) { p.W[s] = (const bf16 *)W[s]; p.C[s] = C[s]; p.n[s] = n[s]; p.ldc[s] = ldc[s]; total += n[s]; }
    p.count = count;
    if (M == 1) launch_gemv_group<1>((const bf16 *)A, p, M, total, K, accumulate, st);
    else if (M == 2) launch_gemv_group<2>((const bf16 *)A, p, M, total, K, accumulate, st);
    else launch_skinny_pick((const bf16 *)A, p, pick_skinny(M, n[0], K), M, K, accumulate, st);
    LAUNCH_CHECK(1);
    return TGP_OK;
}


// Products of M <= 2 activation rows whose activations are computed on the fly (see ASrc): the RMSNorm of x, or SwiGLU of
// (g32, u32).  Every block must carry the M <= 2 group key (tgpk_gemm_group_key(M, n, K) == M); K % 8 == 0.
int tgpk_gemm_group_fused(int mode, const float *x, uint32_t ldx, const void *gain, float eps, const float *g32, const float *u32, uint32_t count,
                          const void *const *W, float *const *C, const uint32_t *n, const uint32_t *ldc, uint32_t M, uint32_t K, int accumulate, cudaStream_t st) {
    if (!count || count > TGP_GEMM_GROUP_MAX || !M || M > 2 || K % 8 || (mode != 1 && mode != 2)) return TGP_E_INVAL;
    for (uint32_t s = 0; s < count; ++s) if (tgpk_gemm_group_key(M, n[s], K) != M) return TGP_E_INVAL;
    GemvParts p;
    memset(&p, 0, sizeof(p));
    uint32_t total = 0;
    for (uint32_t s = 0; s < count; ++s) { p.W[s] = (const bf16 *)W[s]; p.C[s] = C[s]; p.n[s] = n[s]; p.ldc[s] = ldc[s]; total += n[s]; }
    p.count = count;
    const ASrc src{mode, x, ldx, (const bf16 *)gain, eps, g32, u32};
    if (M == 1) launch_gemv_group<1>(nullptr, p, M, total, K, accumulate, st, src);
    else launch_gemv_group<2>(nullptr, p, M, total, K, accumulate, st, src);
    LAUNCH_CHECK(1);
    return TGP_OK;
}

int tgpk_gemm(const void *A, const void *W, float *C, uint32_t M, uint32_t n, uint32_t K, uint32_t ldc, uint32_t col0, int accumulate, cudaStream_t st) {
    if (!M || !n) return TGP_OK;
    if (K % 8 || !K) return TGP_E_INVAL;
    const bf16 *a = (const bf16 *)A, *w = (const bf16 *)W;
    // 17 - 32 activation rows on a block of 64 or more 128-row tiles: the tiled GEMM with the weights as its 128-row operand
    // is ahead of the weight-streaming kernel (n=8192, K=8192, M=32: 33 us against 41 us)
    const bool tiles_win = M > 16 && (n + 127) / 128 >= 64 && g_gemm_impl == 0;
    if (M >= 3 && M <= 32 && K % 32 == 0 && g_skinny_impl == 0 && !tiles_win) {
        GemvParts p;
        memset(&p, 0, sizeof(p));
        p.W[0] = w; p.C[0] = C + col0; p.n[0] = n; p.ldc[0] = ldc; p.count = 1;
        launch_skinny_pick(a, p, pick_skinny(M, n, K), M, K, accumulate, st);
    } else if (M > 32 && M <= 64 && K % 32 == 0 && g_skinny_impl == 0 && g_gemm_impl == 0 && n < 4096) {
        // 33 - 64 activation rows on a block of few rows: the tiled GEMM would run a handful of CTAs with a serial K loop
        // (n=1024, K=4096: 15.8 us); two weight-streaming launches of half the rows each read the block twice, the
        // second time from L2, and are faster (9.9 us); from 32 tiles of 128 rows on the tiled GEMM takes the weights as its
        // 128-row operand instead
        const uint32_t m1 = (M + 1) / 2;
        for (uint32_t m0 = 0; m0 < M; m0 += m1) {
            const uint32_t mr = M - m0 < m1 ? M - m0 : m1;
            GemvParts p;
            memset(&p, 0, sizeof(p));
            p.W[0] = w; p.C[0] = C + (size_t)m0 * ldc + col0; p.n[0] = n; p.ldc[0] = ldc; p.count = 1;
            launch_skinny_pick(a + (size_t)m0 * K, p, pick_skinny(mr, n, K), mr, K, accumulate, st);
            if (m0) tgpk_launches += 1;
        }
    } else if (M <= 16) {
        for (uint32_t m0 = 0; m0 < M; m0 += 8) {
            uint32_t mr = M - m0 < 8 ? M - m0 : 8;
            const bf16 *am = a + (size_t)m0 * K;
            float *cm = C + (size_t)m0 * ldc;
            if (mr == 1) launch_gemv_rows<1>(am, w, cm, mr, n, K, ldc, col0, accumulate, st);
            else if (mr == 2) launch_gemv_rows<2>(am, w, cm, mr, n, K, ldc, col0, accumulate, st);
            else if (mr <= 4) launch_gemv_rows<4>(am, w, cm, mr, n, K, ldc, col0, accumulate, st);
            else launch_gemv_rows<8>(am, w, cm, mr, n, K, ldc, col0, accumulate, st);
            if (m0) tgpk_launches += 1;
        }
    } else if (g_gemm_impl == 0) {
        return tgpk_gemm_tc(A, W, C, M, n, K, ldc, col0, accumulate, st);
    } else {
        dim3 grid((n + 63) / 64, (M + 63) / 64);
        tgp_matmul_simt_kernel<<<grid, 256, 0, st>>>(a, w, C, M, n, K, ldc, col0, accumulate);
        tgpk_last_gemm_kernel = "tgp_matmul_simt_kernel";
    }
    LAUNCH_CHECK(1);
    return TGP_OK;
}

bool tgpk_swiglu_fusable(uint32_t M) { return M > 128 && g_gemm_impl == 0; }

int tgpk_rope_kv(const float *q32, const float *k32, const float *v32, void *qb, const TgpTilePtrs &tiles, const float *cos_t, const float *sin_t,
                 const tgp_model_cfg *c, uint32_t B, uint32_t q_len, uint32_t pos0, cudaStream_t st) {
    if (!B || !q_len) return TGP_OK;
    RopeArgs a{q32, k32, v32, (bf16 *)qb, cos_t, sin_t, c->Hq, c->Hkv, c->Dh, c->TK, q_len, pos0, tiles};
    launch_pdl(tgp_rope_kv_kernel, dim3(B * q_len), dim3(256), 0, st, a);
    LAUNCH_CHECK(1);
    return TGP_OK;
}

static int g_attn_decode_grouped = 1;   // decode: one pass over a KV tile serves all query heads of the group (0: one pass per head)
static int g_attn_decode_impl = 0;      // decode: 0 by size, 1 the CUDA-core per-tile kernels only, 2 the tensor-core kernel wherever its geometry allows
static int g_attn_impl = 0;      // q_len >= 16: 0 by problem size, 3 tcgen05 kernel, 2 mma.sync flash kernel, 1 warp-per-row CUDA-core kernel

int tgpk_attn(const void *qb, const TgpTilePtrs &tiles, uint32_t n_tiles, void *ob, const tgp_model_cfg *c, uint32_t B, uint32_t q_len, uint32_t pos0,
              float *scratch, cudaStream_t st) {
    if (!B || !q_len) return TGP_OK;
    if (c->Dh != 64 && c->Dh != 128) return TGP_E_INVAL;
    AttnArgs a{(const bf16 *)qb, (bf16 *)ob, scratch, c->Hq, c->Hkv, c->Dh, c->TK, q_len, pos0, n_tiles, 1.0f / sqrtf((float)c->Dh), tiles};
    if (q_len == 1 && scratch) {
        const uint32_t nt = (pos0 + 1 + c->TK - 1) / c->TK, G = c->Hq / c->Hkv;
        if (G > 32) return TGP_E_TOO_LARGE;
        uint32_t split = (c->TK + 31) / 32;
        if (split > 32 / G) split = 32 / G;
        if (split < 1) split = 1;
        dim3 grid(nt, c->Hkv, B);
        const bool grouped = g_attn_decode_grouped && (G == 1 || G == 2 || G == 4 || G == 8) && c->Hq % c->Hkv == 0;
        // tensor-core decode kernel: whole 16-key chunks inside a tile, 16-byte aligned rows; the context must be long enough
        // to give its warps a few chunks each (below that the per-tile kernel's single pass is as fast)
        const uint32_t nchunks = (pos0 + 1 + DEC_KEYS - 1) / DEC_KEYS;
        bool aligned16 = (reinterpret_cast<uintptr_t>(qb) & 3u) == 0;
        for (uint32_t t = 0; t < nt && aligned16; ++t) aligned16 = ((reinterpret_cast<uintptr_t>(tiles.k[t]) | reinterpret_cast<uintptr_t>(tiles.v[t])) & 15u) == 0;
        if (grouped && g_attn_decode_impl != 1 && c->TK % DEC_KEYS == 0 && aligned16 && (g_attn_decode_impl == 2 || nchunks * B * c->Hkv >= 256)) {
            static int sms = 0;
            if (!sms) { int dev = 0; cudaGetDevice(&dev); if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) sms = 148; }
            const uint32_t units = B * c->Hkv, per_sm = c->Dh == 64 ? 4 : 2;             // CTAs that fit an SM (96 / 48 KB of shared memory each)
            uint32_t parts = (uint32_t)sms * per_sm / units;                              // CTAs per (sequence, KV head): one wave at most
            parts = std::max(1u, std::min(parts, std::min(n_tiles, (nchunks + DEC_WARPS - 1) / DEC_WARPS)));
            const uint32_t per_cta = (nchunks + parts - 1) / parts;
            parts = (nchunks + per_cta - 1) / per_cta;                                    // no CTA without a chunk
            a.n_parts = parts;
            const size_t smem = (size_t)DEC_WARPS * DEC_STAGES * 2 * DEC_KEYS * c->Dh * 2;        // 96 KB at Dh = 128, 48 KB at 64
            dim3 g2(parts, c->Hkv, B);
#define TGP_DECODE_MMA(DH_, G_) do { \
                static bool attr_set = false; \
                if (!attr_set) { if (cudaFuncSetAttribute(tgp_attn_decode_mma_kernel<DH_, G_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return TGP_E_CUDA; attr_set = true; } \
                launch_pdl(tgp_attn_decode_mma_kernel<DH_, G_>, g2, dim3(DEC_WARPS * 32), smem, st, a, per_cta); } while (0)
#define TGP_DECODE_MMA_G(DH_) do { if (G == 1) TGP_DECODE_MMA(DH_, 1); else if (G == 2) TGP_DECODE_MMA(DH_, 2); else if (G == 4) TGP_DECODE_MMA(DH_, 4); else TGP_DECODE_MMA(DH_, 8); } while (0)
            if (c->Dh == 64) { TGP_DECODE_MMA_G(64); if (parts > 1) launch_pdl(tgp_attn_decode_merge_kernel<64>, dim3(c->Hq, B), dim3(64), 0, st, a); }
            else { TGP_DECODE_MMA_G(128); if (parts > 1) launch_pdl(tgp_attn_decode_merge_kernel<128>, dim3(c->Hq, B), dim3(128), 0, st, a); }
#undef TGP_DECODE_MMA_G
#undef TGP_DECODE_MMA
            LAUNCH_CHECK(parts > 1 ? 2 : 1);
            return TGP_OK;
        }
        if (grouped) {                                      // K and V read once for the whole group of query heads
            split = (c->TK + 31) / 32;
            if (split > 8) split = 8;
        }
        const size_t sm = (size_t)(G * c->Dh + G * split * (c->Dh + 2)) * sizeof(float);
#define TGP_DECODE_GROUP(DH_) do { \
            if (G == 1) launch_pdl(tgp_attn_decode_group_kernel<DH_, 1>, grid, dim3(32 * split), sm, st, a, split); \
            else if (G == 2) launch_pdl(tgp_attn_decode_group_kernel<DH_, 2>, grid, dim3(32 * split), sm, st, a, split); \
            else if (G == 4) launch_pdl(tgp_attn_decode_group_kernel<DH_, 4>, grid, dim3(32 * split), sm, st, a, split); \
            else launch_pdl(tgp_attn_decode_group_kernel<DH_, 8>, grid, dim3(32 * split), sm, st, a, split); } while (0)
        if (c->Dh == 64) {
            if (grouped) TGP_DECODE_GROUP(64); else launch_pdl(tgp_attn_decode_partial_kernel<64>, grid, dim3(32 * G * split), sm, st, a, split);
            launch_pdl(tgp_attn_decode_merge_kernel<64>, dim3(c->Hq, B), dim3(64), 0, st, a);
        } else {
            if (grouped) TGP_DECODE_GROUP(128); else launch_pdl(tgp_attn_decode_partial_kernel<128>, grid, dim3(32 * G * split), sm, st, a, split);
            launch_pdl(tgp_attn_decode_merge_kernel<128>, dim3(c->Hq, B), dim3(128), 0, st, a);
        }
#undef TGP_DECODE_GROUP
        tgpk_launches += 1;
    } else if (q_len >= 16 && (g_attn_impl == 0 || g_attn_impl == 2 || g_attn_impl == 3)) {
        // the tcgen05 kernel works on 128 queries per CTA (it hands geometries it cannot map with TMA to the mma.sync
        // kernel itself); below that the mma.sync kernel's 64-query CTAs waste less
        if (g_attn_impl == 3 || (g_attn_impl == 0 && q_len >= 128)) return tgpk_attn_prefill_tc5(qb, tiles, ob, c, B, q_len, pos0, st);
        return tgpk_attn_prefill_tc(qb, tiles, ob, c, B, q_len, pos0, st);
    } else {
        dim3 grid((q_len + 3) / 4, c->Hq, B);
        if (c->Dh == 64) tgp_attn_rows_kernel<64><<<grid, 128, 0, st>>>(a);
        else tgp_attn_rows_kernel<128><<<grid, 128, 0, st>>>(a);
    }
    LAUNCH_CHECK(1);
    return TGP_OK;
}

int tgpk_swiglu(const float *g, const float *u, void *ab, uint64_t n, cudaStream_t st) {
    if (!n) return TGP_OK;
    if (n % 4) return TGP_E_INVAL;
    uint64_t n4 = n / 4;
    uint32_t blocks = (uint32_t)((n4 + 255) / 256 < 148 * 16 ? (n4 + 255) / 256 : 148 * 16);
    launch_pdl(tgp_swiglu_kernel, dim3(blocks), dim3(256), 0, st, (const float4 *)g, (const float4 *)u, (__nv_bfloat162 *)ab, n4);
    LAUNCH_CHECK(1);
    return TGP_OK;
}

int tgpk_argmax(const float *logits, int32_t *out, uint32_t B, uint32_t V, cudaStream_t st) {
    if (!B) return TGP_OK;
    launch_pdl(tgp_argmax_kernel, dim3(B), dim3(1024), 0, st, logits, out, V);
    LAUNCH_CHECK(1);
    return TGP_OK;
}

// ============================ C entry points ===========================================================
static int fill_tiles(TgpTilePtrs &t, void *const *k, void *const *v, uint32_t n) {
    if (n > TGP_MAX_TILES) return TGP_E_TOO_LARGE;
    if (!k || !v) return TGP_E_INVAL;
    for (uint32_t i = 0; i < n; ++i) { t.k[i] = k[i]; t.v[i] = v[i]; }
    return TGP_OK;
}

extern "C" {

int tgp_k_embed(const void *table, const int32_t *tok_dev, float *x_dev, uint32_t M, uint32_t d, uint32_t V, void *stream) {
    if (!table || !tok_dev || !x_dev) return TGP_E_INVAL;
    return tgpk_embed(table, tok_dev, x_dev, M, d, V, (cudaStream_t)stream);
}

int tgp_k_embed_status(int *bad, uint32_t *row, int32_t *token) {
    if (!bad) return TGP_E_INVAL;
    unsigned long long w = 0;
    if (cudaMemcpyFromSymbol(&w, g_embed_error, sizeof(w)) != cudaSuccess) return TGP_E_CUDA;
    *bad = (w >> 63) ? 1 : 0;
    if (row) *row = (uint32_t)((w >> 32) & 0x7fffffffu);
    if (token) *token = (int32_t)(uint32_t)w;
    return TGP_OK;
}

int tgp_k_wait_test(uint64_t limit_ns, int withhold_step) {
    if (cudaDeviceSynchronize() != cudaSuccess) return TGP_E_CUDA;
    if (!limit_ns) { limit_ns = 2000000000ull; withhold_step = -1; }
    if (limit_ns < 100000ull || withhold_step < -1) return TGP_E_INVAL;
    int rc = tgpk_gemm_wait_test(limit_ns, withhold_step);
    return rc ? rc : tgpk_attn_wait_test(limit_ns, withhold_step);
}

int tgp_k_status_clear(void) {
    if (cudaDeviceSynchronize() != cudaSuccess) return TGP_E_CUDA;
    const unsigned long long z = 0;
    if (cudaMemcpyToSymbol(g_embed_error, &z, sizeof(z)) != cudaSuccess) return TGP_E_CUDA;
    int rc = tgpk_gemm_status_clear();
    return rc ? rc : tgpk_attn_status_clear();
}

int tgp_k_rmsnorm(const float *x_dev, uint32_t ldx, const void *g_dev, void *h_dev, uint32_t M, uint32_t d, float eps, void *stream) {
    if (!x_dev || !g_dev || !h_dev) return TGP_E_INVAL;
    return tgpk_rmsnorm(x_dev, ldx, g_dev, h_dev, M, d, eps, (cudaStream_t)stream);
}

int tgp_k_skinny_select(int impl) {
    if (impl != 0 && impl != 1) return TGP_E_INVAL;
    g_skinny_impl = impl;
    return TGP_OK;
}

int tgp_k_gemm_group(const void *A_dev, uint32_t count, const void *const *W_dev, float *const *C_dev, const uint32_t *n, const uint32_t *ldc,
                     uint32_t M, uint32_t K, int accumulate, void *stream) {
    if (!A_dev || !W_dev || !C_dev || !n || !ldc || !count || count > TGP_GEMM_GROUP_MAX || !K || K % 8) return TGP_E_INVAL;
    for (uint32_t s = 0; s < count; ++s) if (!W_dev[s] || !C_dev[s] || n[s] > ldc[s]) return TGP_E_INVAL;
    return tgpk_gemm_group(A_dev, count, W_dev, C_dev, n, ldc, M, K, accumulate, (cudaStream_t)stream);
}

int tgp_k_gemm_group_key(uint32_t M, uint32_t n, uint32_t K, uint32_t *key) {
    if (!key) return TGP_E_INVAL;
    *key = tgpk_gemm_group_key(M, n, K);
    return TGP_OK;
}

int tgp_k_gemm_last_kernel(char *name, uint32_t capacity) {
    if (!name || !capacity) return TGP_E_INVAL;
    const char *k = tgpk_last_gemm_kernel;
    uint32_t i = 0;
    for (; k[i] && i + 1 < capacity; ++i) name[i] = k[i];
    name[i] = 0;
    return TGP_OK;
}

int tgp_k_gemm_group_select(int enable) {
    g_gemm_group = enable ? 1 : 0;
    return TGP_OK;
}

int tgp_k_gemm_chain(int enable) {
    tgpk_chain_ok = enable != 0;
    g_chain.A = nullptr;
    return TGP_OK;
}

int tgp_k_gemv_overlap(int enable) {
    g_gemv_pdl = enable ? 1 : 0;
    g_small_pdl = enable ? 1 : 0;
    return TGP_OK;
}

int tgp_k_attn_decode_select(int impl) {
    if (impl < 0 || impl > 2) return TGP_E_INVAL;
    g_attn_decode_impl = impl;
    return TGP_OK;
}

int tgp_k_attn_select(int impl) {
    if (impl < 0 || impl > 3) return TGP_E_INVAL;
    g_attn_impl = impl;
    return TGP_OK;
}

int tgp_k_gemm_select(int impl) {
    if (impl != 0 && impl != 1) return TGP_E_INVAL;
    g_gemm_impl = impl;
    return TGP_OK;
}

int tgp_k_gemm(const void *A_dev, const void *W_dev, float *C_dev, uint32_t M, uint32_t n, uint32_t K, uint32_t ldc, uint32_t col0, int accumulate, void *stream) {
    if (!A_dev || !W_dev || !C_dev || col0 + (uint64_t)n > ldc) return TGP_E_INVAL;
    return tgpk_gemm(A_dev, W_dev, C_dev, M, n, K, ldc, col0, accumulate, (cudaStream_t)stream);
}

int tgp_k_rope_kv(const float *q32, const float *k32, const float *v32, void *qb, void *const *k_tiles, void *const *v_tiles, uint32_t n_tiles,
                  const float *cos_dev, const float *sin_dev, const tgp_model_cfg *cfg, uint32_t B, uint32_t q_len, uint32_t pos0, void *stream) {
    if (!q32 || !k32 || !v32 || !qb || !cfg || !cos_dev || !sin_dev) return TGP_E_INVAL;
    if (pos0 + q_len > cfg->max_len || (uint64_t)n_tiles * cfg->TK < pos0 + q_len || cfg->Dh % 2) return TGP_E_INVAL;
    TgpTilePtrs t;
    int rc = fill_tiles(t, k_tiles, v_tiles, n_tiles);
    if (rc) return rc;
    return tgpk_rope_kv(q32, k32, v32, qb, t, cos_dev, sin_dev, cfg, B, q_len, pos0, (cudaStream_t)stream);
}

int tgp_k_attn(const void *qb, void *const *k_tiles, void *const *v_tiles, uint32_t n_tiles, void *ob, const tgp_model_cfg *cfg, uint32_t B, uint32_t q_len,
               uint32_t pos0, float *scratch_dev, void *stream) {
    if (!qb || !ob || !cfg || !cfg->Hkv || cfg->Hq % cfg->Hkv) return TGP_E_INVAL;
    if ((uint64_t)n_tiles * cfg->TK < pos0 + q_len) return TGP_E_INVAL;
    TgpTilePtrs t;
    int rc = fill_tiles(t, k_tiles, v_tiles, n_tiles);
    if (rc) return rc;
    return tgpk_attn(qb, t, n_tiles, ob, cfg, B, q_len, pos0, scratch_dev, (cudaStream_t)stream);
}

// ---- decode attention for callers that cannot allocate ------------------------------------------------
// The per-tile partials live in a fixed array inside the library image instead of caller memory.  In host
// code the array's name is only a handle; its device address is looked up once per device.
static __device__ __align__(256) float g_static_attn_scratch[TGP_STATIC_SCRATCH_BYTES / sizeof(float)];
static float *g_static_attn_scratch_addr[TGP_STATIC_MAX_DEVICES] = {};

int tgp_k_attn_decode_static(const void *qb, void *const *k_tiles, void *const *v_tiles, uint32_t n_tiles, void *ob,
                             const tgp_model_cfg *cfg, uint32_t B, uint32_t pos0, void *stream) {
    if (!qb || !ob || !cfg || !cfg->Hkv || cfg->Hq % cfg->Hkv || !cfg->TK || !B) return TGP_E_INVAL;
    if ((uint64_t)n_tiles * cfg->TK < (uint64_t)pos0 + 1) return TGP_E_INVAL;
    const uint64_t need = (uint64_t)B * cfg->Hq * n_tiles * (cfg->Dh + 2) * sizeof(float);
    if (need > TGP_STATIC_SCRATCH_BYTES) return TGP_E_TOO_LARGE;
    TgpTilePtrs t;
    int rc = fill_tiles(t, k_tiles, v_tiles, n_tiles);
    if (rc) return rc;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return TGP_E_CUDA;
    if (dev < 0 || dev >= TGP_STATIC_MAX_DEVICES) return TGP_E_TOO_LARGE;
    if (!g_static_attn_scratch_addr[dev]) {                       // first call on this device, with it current
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_attn_scratch) != cudaSuccess || !p) return TGP_E_CUDA;
        g_static_attn_scratch_addr[dev] = (float *)p;
    }
    return tgpk_attn(qb, t, n_tiles, ob, cfg, B, 1, pos0, g_static_attn_scratch_addr[dev], (cudaStream_t)stream);
}

int tgp_k_attn_scratch_bytes(const tgp_model_cfg *cfg, uint64_t *bytes) {
    if (!cfg || !bytes || !cfg->TK) return TGP_E_INVAL;
    uint64_t nt = (cfg->max_len + cfg->TK - 1) / cfg->TK;
    *bytes = (uint64_t)cfg->B * cfg->Hq * nt * (cfg->Dh + 2) * sizeof(float);
    return TGP_OK;
}

int tgp_k_swiglu(const float *g32, const float *u32, void *ab, uint64_t n_elems, void *stream) {
    if (!g32 || !u32 || !ab) return TGP_E_INVAL;
    return tgpk_swiglu(g32, u32, ab, n_elems, (cudaStream_t)stream);
}

int tgp_k_argmax(const float *logits, int32_t *out, uint32_t B, uint32_t V, void *stream) {
    if (!logits || !out || !V) return TGP_E_INVAL;
    return tgpk_argmax(logits, out, B, V, (cudaStream_t)stream);
}

}  // extern "C"
