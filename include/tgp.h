/*
 * tgp - tensor-granular prefetch for oversubscribed transformer inference (sm_100a).
 *
 * C ABI of the library.  The calls follow the paper's statement of the problem:
 * a framework allocator carves one big pool into tensors that are invisible below it
 * (Section II-B), so the caller REGISTERS the pool and its sub-ranges (Section IV-B,
 * stable two-level tensor identity); one pass RECORDS which tensors each op touches
 * (Section IV-D, kernel-tensor access tracing); device capacity is CONSTRAINED to a
 * budget (Section V-A); a roofline policy picks the transfers that matter (Section III-C,
 * IV-D "UVM Analyzer") and an engine stages exactly those tensors ahead of use
 * (Section IV-E "Prefetch Engine") while the model step RUNS.
 *
 * Conventions
 *  - Every function returns TGP_OK (0) or a negative TGP_E_* code; nothing throws, aborts
 *    or prints across this boundary.  tgp_strerror() names a code; tgp_last_error() adds
 *    the detail of the last failure on that context.
 *  - "host" pointers are CPU addresses, "dev" pointers are addresses valid on the current
 *    CUDA device.  Streams are cudaStream_t passed as void*.
 *  - Ownership: the caller owns the host pool, the device arena, the workspace, the logits
 *    and token buffers and the streams, and keeps them alive while the context uses them.
 *    The library owns the context, the plan and its CUDA events.  It allocates no device
 *    memory except a few bytes of bookkeeping at tgp_model_bind().
 *  - A context is used by one thread at a time.
 *  - Export calls use the two-call form: pass buf == NULL to get the size in *bytes.
 *  - All multi-byte fields of exported blobs are little-endian and packed.
 */
#ifndef TGP_H
#define TGP_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TGP_OK                  0
#define TGP_E_INVAL            -1   /* bad argument or call order                                  */
#define TGP_E_OVERLAP          -2   /* sub-range overlaps a registered one                         */
#define TGP_E_RANGE            -3   /* sub-range or address outside its pool                       */
#define TGP_E_UNKNOWN_TENSOR   -4   /* trace names a tensor id that was never registered           */
#define TGP_E_BUDGET_TOO_SMALL -5   /* budget below the ring minimum, or a stay would wait on itself */
#define TGP_E_NO_PLAN          -6   /* tgp_plan() has not succeeded yet                            */
#define TGP_E_CUDA             -7   /* a CUDA call failed; tgp_last_error() has its text           */
#define TGP_E_MISMATCH         -8   /* run-time access differs from the recorded trace             */
#define TGP_E_STATE            -9   /* object not in the state this call needs                     */
#define TGP_E_TOO_LARGE       -10   /* size beyond a documented fixed maximum                      */

/* pool flags */
#define TGP_POOL_PINNED   1u   /* page-locked host memory (cudaHostAlloc / cudaHostRegister'ed by the caller) */
#define TGP_POOL_MANAGED  2u   /* cudaMallocManaged memory                                                    */
#define TGP_POOL_PLAIN    4u   /* ordinary host memory: enough for planning; tgp_model_bind() page-locks it   */
/* tensor flags */
#define TGP_T_READONLY 1u
#define TGP_T_MUTABLE  2u
/* access modes */
#define TGP_R 1u
#define TGP_W 2u
/* step kinds */
#define TGP_PREFILL 0u
#define TGP_DECODE  1u
/* op kinds of the trace */
#define TGP_OP_EMBED 0u
#define TGP_OP_RMSNORM 1u
#define TGP_OP_GEMM 2u
#define TGP_OP_ROPE_KV 3u
#define TGP_OP_ATTN 4u
#define TGP_OP_SWIGLU 5u
#define TGP_OP_ROUTER 6u
#define TGP_OP_ARGMAX 7u
/* tensor kinds (role of a sub-range in the model) */
#define TGP_K_EMBED 0u
#define TGP_K_G1 1u
#define TGP_K_WQ 2u
#define TGP_K_WK 3u
#define TGP_K_WV 4u
#define TGP_K_WO 5u
#define TGP_K_G2 6u
#define TGP_K_WG 7u
#define TGP_K_WU 8u
#define TGP_K_WD 9u
#define TGP_K_GF 10u
#define TGP_K_LM 11u
#define TGP_K_ROUTER 12u
#define TGP_K_KTILE 13u
#define TGP_K_VTILE 14u
/* execution variants */
#define TGP_VAR_EXPLICIT_RING   0u  /* staged copies into the arena on a copy stream, events, no demand faults */
#define TGP_VAR_MANAGED_HINTS   1u  /* managed pool + cudaMemPrefetchAsync on critical tensors + cudaMemAdvise on pins */
#define TGP_VAR_MANAGED_DEMAND  2u  /* managed pool, no hints: the demand-paged baseline                        */
#define TGP_VAR_MANAGED_OBJECT  3u  /* managed pool; ahead of each op, a prefetch of every whole allocator segment its tensors overlap */
/* policy bits (ablation switches of the paper's Section V-E: T is always on) */
#define TGP_BIT_A  1u   /* look-ahead affinity: residency (pin) set              */
#define TGP_BIT_P  2u   /* roofline selectivity; off = every op with pool traffic is link-bound */
#define TGP_BIT_ZC 4u   /* sparse read-only accesses are served in place over the link          */
#define TGP_BIT_W  8u   /* windowed pin reservation: the slot of a pinned tensor that is born on the device in a later
                           step (a KV tile of positions not reached yet) houses unpinned read-only tensors until then */
/* plan export selectors */
#define TGP_X_CLASSES  0u   /* u8 per op: 0 LINK, 1 HBM, 2 COMPUTE                                   */
#define TGP_X_TENSORS  1u   /* per tensor: u8 critical, u8 zero-copy, u64 score (link bytes residency saves) */
#define TGP_X_PINS     2u   /* (u32 tensor, u64 arena offset) ascending tensor id, then u64 ring base, u64 ring size */
#define TGP_X_COMMANDS 3u   /* per command: u32 seq, u8 kind(0 H2D,1 ALLOC,2 D2H), u32 tensor, u64 bytes, u64 pool offset,
                               u64 arena offset, i32 wait_op, i32 first_use, i32 release_after      */
#define TGP_X_TOTALS   4u   /* per step: u64 h2d bytes, u64 d2h bytes, u64 zero-copy bytes, u64 commands */
#define TGP_X_TAIL 0x100u   /* or-ed into a selector: the tail plan that waits for tgp_replan_commit() (after tgp_replan_wait()) */

typedef struct tgp_ctx tgp_ctx;

/* Roofline constants, integers per second: bf16 tensor peak, HBM bandwidth, host->device and
 * device->host link bandwidth (Section III-C: compute roof, memory roof, interconnect roof). */
typedef struct { uint64_t peak_flops, hbm_Bps, h2d_Bps, d2h_Bps; } tgp_machine;

typedef struct { uint32_t tensor; uint32_t mode; uint64_t touched_bytes; } tgp_access;

/* Decoder shape.  E == 0: dense SwiGLU FFN.  max_len = prompt + decode tokens; TK = tokens per KV tile. */
typedef struct {
    uint32_t L, d, Hq, Hkv, Dh, F, V, E, topk, B, max_len, TK;
    float rope_base, eps;
} tgp_model_cfg;

/* One registered sub-range in its model role: rows [row0, row0+rows) of the [out, in] matrix
 * `kind` of `layer` (expert -1 unless an expert weight); for KV tiles `block` is the tile index. */
typedef struct { uint32_t kind; int32_t layer; int32_t expert; uint32_t block, row0, rows, tensor; } tgp_role_entry;

typedef struct {
    uint64_t h2d_bytes, d2h_bytes, zc_bytes;   /* bytes this step moved (plan figures for this step)   */
    uint32_t n_cmds, n_launches, n_mismatch;   /* copy commands issued, kernels launched, fallbacks    */
    float    step_ms;                          /* device time of the step, CUDA events on the compute stream */
} tgp_step_stats;

/* ---- context ------------------------------------------------------------------------------- */
int  tgp_create(tgp_ctx **out, const tgp_machine *m);
void tgp_destroy(tgp_ctx *ctx);
const char *tgp_strerror(int code);
const char *tgp_last_error(const tgp_ctx *ctx);

/* ---- registry (Section II-B, IV-B): what the allocator hides -------------------------------- */
/* Registers one pool [host_base, host_base+bytes).  host_base must be 512-byte aligned. */
int  tgp_pool_register(tgp_ctx *ctx, void *host_base, uint64_t bytes, uint32_t flags, uint32_t *pool_id);
/* Registers sub-range [offset, offset+bytes) of a pool.  offset must be 512-byte aligned.  site_hash stands
 * for the creation-site call-stack hash; the library appends its own per-site allocation counter, so
 * (site_hash, counter) is the stable identity that survives a move of the pool (Section IV-B). */
int  tgp_tensor_register(tgp_ctx *ctx, uint32_t pool, uint64_t offset, uint64_t bytes, uint64_t site_hash,
                         int32_t layer, uint32_t kind, uint32_t flags, uint32_t *tensor_id);
/* Address -> (tensor, offset inside it); TGP_E_RANGE if no registered sub-range holds host_addr. */
int  tgp_tensor_lookup(const tgp_ctx *ctx, const void *host_addr, uint32_t *tensor_id, uint64_t *inner_offset);
/* Stable identity of a tensor: its site hash and per-site counter. */
int  tgp_tensor_identity(const tgp_ctx *ctx, uint32_t tensor_id, uint64_t *site_hash, uint64_t *counter);

/* ---- trace (Section IV-D): ordered ops, each with the tensors it touches --------------------- */
int  tgp_trace_begin(tgp_ctx *ctx);                         /* discards any earlier trace and plan        */
int  tgp_trace_step(tgp_ctx *ctx, uint32_t step_kind);      /* opens the next step                        */
int  tgp_trace_op(tgp_ctx *ctx, uint64_t op_site, int32_t layer, uint32_t op_kind, uint64_t flops,
                  uint64_t hbm_bytes, uint32_t n_acc, const tgp_access *acc);
int  tgp_trace_end(tgp_ctx *ctx);
/* Records the analytic trace of the bound model itself: prefill of S tokens then T decode steps.
 * expert_counts (MoE only, else NULL): [(1+T) * L * E] tokens routed to each expert per step. */
int  tgp_model_trace(tgp_ctx *ctx, uint32_t S, uint32_t T, const uint32_t *expert_counts);
/* Canonical blob of the trace: per op u32 step, u64 site, i32 layer, u32 kind, u64 flops, u64 hbm bytes,
 * u32 n_acc, then n_acc x (u32 tensor, u32 mode, u64 touched). */
int  tgp_trace_export(const tgp_ctx *ctx, void *buf, uint64_t *bytes);

/* ---- policy (Section III-C, IV-D, IV-E) ------------------------------------------------------ */
int  tgp_set_budget(tgp_ctx *ctx, uint64_t bytes);          /* device bytes for resident pool tensors     */
int  tgp_set_variant(tgp_ctx *ctx, uint32_t variant, uint32_t policy_bits);
/* Segment size of TGP_VAR_MANAGED_OBJECT: the prefetcher of the paper's motivation (Section III-B) sees the
 * allocator's objects, not the tensors inside them, so it asks for every `bytes`-sized, `bytes`-aligned piece of the
 * pool that a tensor of the coming op overlaps, whole (default 20 MiB, the large-block size of PyTorch's caching
 * allocator; at least 64 KiB).  tgp_step_stats.h2d_bytes then counts the bytes it asked for, whether they were
 * already resident or not; nothing is advised and nothing is evicted explicitly. */
int  tgp_set_object_bytes(tgp_ctx *ctx, uint64_t bytes);
/* Runtime monitor (Section IV-E): measured kernel times, one per op of the finished trace, in integer nanoseconds
 * (0 = not measured: that op keeps its analytic class).  With a time t the link test becomes mig / Bl > t, i.e. an
 * op is link-bound iff moving its pool bytes takes longer than the kernel ran; the next tgp_plan() uses it.
 * n_ops == 0 clears the log; a new trace clears it too.  Integers make the re-plan reproducible: the same log fed
 * to another planner gives the same schedule. */
int  tgp_set_measured_times(tgp_ctx *ctx, const uint64_t *op_ns, uint64_t n_ops);
/* Runtime monitor, while the run is under way (Section IV-E: classes are re-evaluated from measured kernel times and the
 * engine adapts, in parallel with the kernels that follow).  tgp_replan_begin() takes the timing log so far - one entry
 * per op of the whole trace in integer nanoseconds, 0 = not measured (n_ops == 0 keeps the stored log) - and plans the
 * steps from first_step on as a trace of their own on a helper thread, while tgp_step() goes on executing the current
 * plan.  The tail plan assumes an empty arena at the boundary and that tensors written in earlier steps hold data in
 * the pool.  tgp_replan_wait() waits for the planner and reports its result.  tgp_replan_commit() must be called when
 * the run stands exactly at the boundary (first_step steps done): it waits for the device, copies the pinned tensors
 * that were written back to the pool, and switches; tgp_plan_export() then exports the tail plan (op indices of the whole
 * trace; classes and totals cover the tail only).  tgp_run_reset() brings the whole-run plan back.  Explicit engine only. */
int  tgp_replan_begin(tgp_ctx *ctx, uint32_t first_step, const uint64_t *op_ns, uint64_t n_ops);
int  tgp_replan_wait(tgp_ctx *ctx);
int  tgp_replan_commit(tgp_ctx *ctx);
/* keep != 0: tail plans made from now on keep the pinned tensors of the plan in use that are on the device at the
 * boundary.  A tensor the tail plan pins again stays where it is - with the newest data, so the commit writes back only
 * the written pins that are given up - and is not loaded again; newly pinned tensors go into the first gap between the
 * kept ones that holds them; the windowed reservation (TGP_BIT_W) is not applied to such a plan.  The switch then costs
 * the link only what the new plan pins anew.  Default 0 (the tail plan starts from an empty arena). */
int  tgp_set_replan_keep(tgp_ctx *ctx, int keep);
/* Classifies ops, selects critical / zero-copy / pinned tensors, sizes the ring and builds the ordered
 * command list.  Host only; no CUDA call. */
int  tgp_plan(tgp_ctx *ctx);
int  tgp_plan_export(const tgp_ctx *ctx, uint32_t what, void *buf, uint64_t *bytes);

/* ---- execution ------------------------------------------------------------------------------- */
/* Device arena of at least the budget, 512-byte aligned, caller-owned. */
int  tgp_set_arena(tgp_ctx *ctx, void *arena_dev, uint64_t bytes);
/* Activation workspace the model needs for steps of up to max_tokens tokens (B * q_len). */
int  tgp_model_workspace_bytes(const tgp_model_cfg *cfg, uint32_t max_tokens, uint64_t *bytes);
/* Binds the model shape, the role of every registered tensor and the workspace.  router_bias_host: fp32
 * [L, E] (MoE) or NULL.  May be called before tracing (tgp_model_trace needs it) with workspace NULL and
 * again later with the workspace; page-locks a TGP_POOL_PLAIN pool when a workspace is given. */
int  tgp_model_bind(tgp_ctx *ctx, const tgp_model_cfg *cfg, const tgp_role_entry *roles, uint32_t n_roles,
                    const float *router_bias_host, void *workspace_dev, uint64_t ws_bytes, uint32_t max_tokens);
/* Rewinds execution to step 0 with a cold arena (waits for work in flight first). */
int  tgp_run_reset(tgp_ctx *ctx);
/* Runs the next step of the plan: enqueues its copies on copy_stream and its kernels on compute_stream and
 * returns without waiting unless stats != NULL.  tokens_host [B, q_len] int32, or NULL in a decode step to
 * feed the previous step's argmax, which stays on the device.  A host token outside [0, V) is refused with TGP_E_INVAL
 * before anything is enqueued.  logits_dev [B, V] fp32 of the last position;
 * argmax_dev [B] int32 or NULL.  With stats the step is waited for, and TGP_E_CUDA is returned if a tensor-core kernel
 * of this process has recorded a bounded wait that ran out (tgp_k_gemm_status / tgp_k_attn_status). */
int  tgp_step(tgp_ctx *ctx, uint32_t step_kind, const int32_t *tokens_host, uint32_t B, uint32_t q_len,
              float *logits_dev, int32_t *argmax_dev, void *compute_stream, void *copy_stream,
              tgp_step_stats *stats);

/* Copy coalescing: consecutive host-to-device commands of the plan whose pool ranges and arena slots continue one another
 * (sub-ranges that were registered next to each other and placed next to each other), that need no further wait and
 * together stay under 1 MiB, are carried by one cudaMemcpyAsync (a pinned copy of a few hundred KiB is mostly latency).
 * The schedule itself does not change.  tgp_k_merge_copies(0) switches it off (process-wide; default on);
 * tgp_copies_issued() returns the host-to-device copies issued since the last tgp_run_reset(). */
int  tgp_k_merge_copies(int enable);
int  tgp_copies_issued(tgp_ctx *ctx, uint64_t *n);
/* MoE profile (Section IV-D: one profiling pass recovers which tensors the kernels really touch): the tokens
 * routed to each expert, per step and layer, in the run since the last tgp_run_reset(): uint32 [steps, L, E].
 * Two-call form: out == NULL returns the element count in *n.  Feed it to tgp_model_trace() to trace exactly the
 * experts in use.  At run time an expert the router picks but the trace does not list is fetched synchronously
 * into a spill buffer and counted in tgp_step_stats.n_mismatch. */
int  tgp_expert_counts(tgp_ctx *ctx, uint32_t *out, uint64_t *n);

/* Managed-memory helpers for the two managed variants (Section II-A: cudaMallocManaged pools that migrate on
 * demand).  tgp_managed_alloc() returns cudaMallocManaged memory the caller fills and registers with
 * TGP_POOL_MANAGED and later frees with tgp_managed_free(); tgp_managed_evict() moves a managed range back to
 * host memory and waits (a cold start for a managed run). */
int  tgp_managed_alloc(void **out, uint64_t bytes);
int  tgp_managed_free(void *ptr);
int  tgp_managed_evict(void *ptr, uint64_t bytes);

/* Activation tap, for parity checks at every rounding point.  While a tap buffer is set, tgp_step() copies each
 * bf16-rounded activation it produces into it (on the compute stream, 256-byte aligned, in op order): normed
 * hidden states, rotated q, the KV tiles an append touched, attention output, the SwiGLU output (dense FFN: all tokens,
 * sub-index 0; mixture of experts: per expert the rows routed to it in ascending token order, sub-index = expert),
 * the final normed state.  tgp_tap_index() returns 5 uint64 per record: op index, tag, sub-index (tile), offset,
 * bytes (two-call form: out == NULL gives the word count).  tgp_set_tap() also rewinds the buffer; NULL disables. */
#define TGP_TAP_H 0u
#define TGP_TAP_HF 1u
#define TGP_TAP_Q 2u
#define TGP_TAP_KTILE 3u
#define TGP_TAP_VTILE 4u
#define TGP_TAP_O 5u
#define TGP_TAP_A 6u
int  tgp_set_tap(tgp_ctx *ctx, void *tap_dev, uint64_t bytes);
int  tgp_tap_index(tgp_ctx *ctx, uint64_t *out, uint64_t *n_words);

/* Per-op timestamps (Section IV-E "Runtime Monitor": lightweight timestamping).  While enabled, tgp_step()
 * brackets every op with CUDA events on the compute stream (after the op's copies have been waited for, so
 * the figure is kernel time, not stall time).  tgp_op_times() waits for the last timed step and returns one
 * duration in ms per op of that step, ops [*first_op, *first_op + *n_ops) of the trace; ms == NULL asks
 * for the count only. */
int  tgp_set_op_timing(tgp_ctx *ctx, int enable);
int  tgp_op_times(tgp_ctx *ctx, float *ms, uint32_t capacity, uint32_t *first_op, uint32_t *n_ops);

/* Whole-run CUDA graph (dense models, explicit engine).  Between tgp_run_capture_begin() and tgp_run_capture_end()
 * the caller issues the run's tgp_step() calls as usual (same two streams, stats == NULL, decode steps with
 * tokens_host == NULL so the device's own argmax is fed back); nothing executes, the copies, kernels and their
 * cross-stream ordering are recorded instead.  tgp_run_graph_launch() then replays the whole run - cold arena to
 * last logits - with a single launch; logits_dev / argmax_dev given to the captured steps receive each step's result.
 * The prompt buffer given to the captured prefill step is read again at every replay and must stay valid.
 * Call tgp_run_reset() before capturing, run the plan once un-captured first (one-time kernel attribute set-up is not
 * capturable), and call tgp_run_reset() again before going back to plain tgp_step() calls. */
int  tgp_run_capture_begin(tgp_ctx *ctx, void *compute_stream, void *copy_stream);
int  tgp_run_capture_end(tgp_ctx *ctx);
int  tgp_run_graph_launch(tgp_ctx *ctx, void *stream);

/* ---- single kernels (device pointers; used by the model step, exported for parity tests and timing) ---- */
/* x[m, :] = fp32(table[tok[m], :]);  table bf16 [V, d] (device or mapped host), tok int32 [M].  A token id outside
 * [0, V) never indexes the table: its row of x is written as zeros and the first such (row, id) is kept in an error
 * word that tgp_k_embed_status() reads and that tgp_step() reports (TGP_E_CUDA) when called with statistics. */
int  tgp_k_embed(const void *table, const int32_t *tok_dev, float *x_dev, uint32_t M, uint32_t d, uint32_t V, void *stream);
/* *bad = 1 if an embedding gather of this process met a token id outside its vocabulary since the last
 * tgp_k_status_clear(), with the row and the id of the first one (row, token may be NULL).  Synchronous. */
int  tgp_k_embed_status(int *bad, uint32_t *row, int32_t *token);
/* Clears the three device-side error words (tgp_k_gemm_status, tgp_k_attn_status, tgp_k_embed_status) of the
 * current device after waiting for it to go idle. */
int  tgp_k_status_clear(void);
/* h = bf16(x * rsqrt(mean(x^2) + eps) * g);  x fp32 [M, d] with row stride ldx elements, g bf16 [d], h bf16 [M, d]. */
int  tgp_k_rmsnorm(const float *x_dev, uint32_t ldx, const void *g_dev, void *h_dev, uint32_t M, uint32_t d,
                   float eps, void *stream);
/* C[m, col0 + j] (=|+=) sum_k A[m, k] * W[j, k]: A bf16 [M, K] row-major, W bf16 [n, K] row-major (one out-row
 * block), C fp32 with row stride ldc.  accumulate != 0 adds to C (fused residual).  K % 8 == 0. */
int  tgp_k_gemm(const void *A_dev, const void *W_dev, float *C_dev, uint32_t M, uint32_t n, uint32_t K,
                uint32_t ldc, uint32_t col0, int accumulate, void *stream);
/* Several products over the same activations in one call (Section II-B's kernel sequence: the q, k and v projections of a
 * layer, or the pieces a large matrix was registered as): C_dev[s][m, j] (=|+=) sum_k A[m, k] * W_dev[s][j, k] for
 * s < count <= TGP_GEMM_GROUP_MAX, W_dev[s] bf16 [n[s], K], C_dev[s] fp32 with row stride ldc[s] >= n[s]; accumulate != 0
 * adds to C (fused residual).  The pointer and size arrays are host arrays (of device pointers), read before the call
 * returns.  Blocks whose tgp_k_gemm_group_key() is the same non-zero value are served by one launch - a block of few
 * rows alone leaves most SMs without work - anything else by one launch per part; the results are bit-identical to
 * tgp_k_gemm() per part either way, because the key names the kernel the block takes on its own (M <= 2: fewer than
 * 4736 rows and K < 8192; 3 <= M <= 32 with K % 32 == 0: blocks of fewer 16-row groups than the GPU has SMs, which pick
 * the same split-K kernel instance).
 * tgp_k_gemm_group_select(0) makes every key 0 (process-wide; default 1), also inside tgp_step(), which groups
 * consecutive weight-block products of a decode step that read the same activations this way when their copies have
 * all been enqueued and no tap is set, except blocks under 2 MiB whose arena slot a later copy waits for (with op timing
 * the launch's time is reported for the first product of the group and an empty bracket for the others). */
#define TGP_GEMM_GROUP_MAX 8u
int  tgp_k_gemm_group(const void *A_dev, uint32_t count, const void *const *W_dev, float *const *C_dev, const uint32_t *n,
                      const uint32_t *ldc, uint32_t M, uint32_t K, int accumulate, void *stream);
/* *key = 0 if a block [n, K] at M activation rows is always launched alone, else a value such that blocks of equal
 * key may share a launch.  Needs a current device (the rule depends on its SM count). */
int  tgp_k_gemm_group_key(uint32_t M, uint32_t n, uint32_t K, uint32_t *key);
int  tgp_k_gemm_group_select(int enable);
/* Name of the kernel that the calling thread's last tgp_k_gemm() / tgp_k_gemm_group() launched (the choice depends on
 * M, n, K and the GPU's SM count), as a NUL-terminated string of at most capacity - 1 characters; "" before the first. */
int  tgp_k_gemm_last_kernel(char *name, uint32_t capacity);
/* Prefill (more than 128 activation rows, dense FFN): the tensor-core GEMM that computes the up projection applies SwiGLU in
 * its epilogue - a = bf16(silu(g) * u) from the gate projection already in memory and the accumulator - so the up
 * projection is never stored, the gate is read once and the step's SwiGLU op launches nothing (at the 70B shape that is
 * 7.5 GB of HBM traffic per layer).  Bit-identical to the separate kernel; 0 switches it off.  Process-wide; default on. */
int  tgp_k_swiglu_epilogue(int enable);
/* Decode steps of at most two sequences on models whose rows hold at most 1024 elements (d for the norms, F for SwiGLU):
 * tgp_step() lets the products that consume a normalised state or a SwiGLU output compute it themselves (each warp of
 * the weight-streaming kernel redoes the row, bit for bit as the separate kernel would), so those ops launch nothing.
 * Results are identical either way.  Process-wide; default off: on the tiny configuration it takes a decode step from 50
 * launches to 32, but a fused span waits for the copies of all its blocks, and the step got no faster (measured). */
int  tgp_k_decode_fuse(int enable);
/* Which kernel serves M > 16: 0 (default) the tcgen05 tensor-core GEMM, 1 the CUDA-core tile kernel (an on-device
 * cross-check).  M <= 16 always takes the weight-streaming GEMV.  Process-wide. */
int  tgp_k_gemm_select(int impl);
/* Which kernel serves 3 <= M <= 32 (K % 32 == 0; and, as two launches of half the rows, 33 <= M <= 64 on blocks of fewer
 * than 4096 rows): 0 (default) the weight-streaming tensor-core kernel, 1 the
 * CUDA-core GEMV (M <= 16) / GEMM paths (an on-device cross-check).  Process-wide. */
int  tgp_k_skinny_select(int impl);
/* Weight-streaming launches (M <= 32) and the small kernels of a step (embedding gather, RMSNorm, RoPE + KV append, decode
 * attention and its merge, SwiGLU, argmax) use programmatic dependent launch: a launch lets its successor be scheduled
 * at once; a weight-streaming kernel starts reading its weights while the previous kernel of the stream drains and
 * waits for it only before it touches activations or output, a small kernel waits first thing, so that only its launch
 * latency overlaps.  0 switches that off (each launch then starts after the previous one has completed).  Results are
 * identical either way.  Process-wide; default on. */
int  tgp_k_gemv_overlap(int enable);
/* A promise by a caller of the kernel entry points, for the calling thread: between consecutive tgp_k_gemm() /
 * tgp_k_gemm_group() calls on one stream nothing but this library's kernels (launched by this thread) is enqueued on that
 * stream.  A product of 3 - 32 activation rows that directly follows another one over the same activation pointer then
 * requests its activations together with its weights, before the previous launch has finished (they are older than that
 * launch); results are identical.  tgp_step() works this way by itself.  Default off: a caller that rewrites the
 * activations between two calls by other means must leave it off. */
int  tgp_k_gemm_chain(int enable);
/* Tensor-core GEMM variant: 0 (default) picks by problem size, 1 forces the 128x128 one-tile-per-CTA kernel,
 * 2 the persistent 128x256 kernel with double-buffered accumulators, 3 the paired kernel (256x256 tiles on the two SMs
 * of a CTA pair, each loading half of the weight tile), 4 the one-tile-per-CTA kernel with the operands swapped (the
 * weights are the 128-row operand, the tile is stored transposed; for M <= 128, else as 0; picked by size for M <= 64 on
 * blocks of many rows).  Process-wide; for tests and timing. */
int  tgp_k_gemm_tc_variant(int variant);
/* Which kernel serves attention with q_len >= 16: 0 (default) by problem size - the tcgen05 kernel (S and O in TMEM,
 * K/V fed by TMA) for q_len >= 128, else the mma.sync flash-style kernel;
 * 3 / 2 force one or the other; 1 the warp-per-query-row CUDA-core kernel (an on-device cross-check).  The tcgen05
 * kernel needs KV tiles of a multiple of 64 keys whose base addresses differ by whole rows of Dh elements (and
 * 16-byte aligned q); any other geometry is served by the mma.sync kernel even when 3 is forced.  Process-wide. */
int  tgp_k_attn_select(int impl);
/* Which kernel serves decode attention (q_len == 1 with scratch): 0 (default) by size - the tensor-core kernel (the G query
 * heads of a KV head as rows of an mma.sync tile, K and V staged through shared memory with cp.async three chunks of 16
 * keys deep, P rounded to bf16 for the second product) when KV tiles hold a multiple of 16 keys, G is 1, 2, 4 or 8 and
 * the batch's context adds up to 256 chunks or more, else the CUDA-core kernels (one pass per KV tile and group of query
 * heads); 1 forces the CUDA-core kernels, 2 the tensor-core kernel wherever its geometry allows.  Process-wide. */
int  tgp_k_attn_decode_select(int impl);
/* Error word of the tcgen05 attention kernel: 0, or which bounded wait ran out first (1 for S, 2 for P V, 3 for a K/V
 * load, 4 for the hand-over between the softmax warps and the MMA warp), or 5 if shared memory was not 1024-byte
 * aligned.  A CTA that gives up stores nothing.  Synchronous. */
int  tgp_k_attn_status(int *error_code);
/* Error word of the tensor-core GEMM: 0, or (role << 8 | stage) of the first bounded wait that ran out
 * (role 1 TMA producer, 2 MMA issuer, 3 epilogue).  Synchronous. */
int  tgp_k_gemm_status(int *error_code);
/* For tests of the give-up path of the tensor-core kernels (every wait on an mbarrier in them is bounded in time; a wait
 * that runs out records an error word, the CTA drains its copies in flight, frees its tensor memory, stores nothing and
 * returns).  Sets, for the current device and until changed back, the time limit of those waits (default 2 s; at least
 * 100 us) and the index of one load step - a K block of the GEMM kernels, a V block of the attention kernel - that the
 * TMA thread of the grid's first CTA (CTA pair) leaves out (-1: none), so that the wait for it runs out; nothing traps or
 * faults, the other CTAs of the launch complete normally.  limit_ns == 0 restores the defaults.  Waits for the device to
 * go idle first.  Process-wide. */
int  tgp_k_wait_test(uint64_t limit_ns, int withhold_step);
/* Fills caller-owned device tables cos/sin fp32 [max_len, Dh/2]: angle = pos * base^(-2i/Dh), evaluated in
 * double on the host.  Synchronous. */
int  tgp_k_rope_tables(uint32_t Dh, uint32_t max_len, float base, float *cos_dev, float *sin_dev);
/* Rotary embedding (rotate-half pairs (i, i+Dh/2)) on q and k, bf16 rounding, and append of k, v to the KV
 * tiles.  q32/k32/v32 fp32 [B*q_len, H*Dh]; qb bf16 out; k_tiles/v_tiles: HOST arrays of n_tiles (<= 64)
 * device pointers, tile layout [B, Hkv, TK, Dh] bf16; token (b, p) sits at position pos0 + p. */
int  tgp_k_rope_kv(const float *q32, const float *k32, const float *v32, void *qb, void *const *k_tiles,
                   void *const *v_tiles, uint32_t n_tiles, const float *cos_dev, const float *sin_dev,
                   const tgp_model_cfg *cfg, uint32_t B, uint32_t q_len, uint32_t pos0, void *stream);
/* Causal GQA attention of q_len new queries per sequence against the tiles (kvlen = pos0 + q_len valid
 * tokens): o = softmax(q K^T / sqrt(Dh)) V, bf16 out [B*q_len, Hq*Dh].  k_tiles/v_tiles as above (host arrays
 * of device pointers).  Dh must be 64 or 128.  scratch_dev: fp32 workspace of
 * tgp_k_attn_scratch_bytes() used when q_len == 1 (split over KV tiles), else may be NULL. */
int  tgp_k_attn(const void *qb, void *const *k_tiles, void *const *v_tiles, uint32_t n_tiles, void *ob,
                const tgp_model_cfg *cfg, uint32_t B, uint32_t q_len, uint32_t pos0, float *scratch_dev,
                void *stream);
int  tgp_k_attn_scratch_bytes(const tgp_model_cfg *cfg, uint64_t *bytes);
/* (No counterpart in the paper: a convenience of this library.)
 * Decode attention (q_len == 1) for callers that must not allocate device memory: code running where the
 * whole device budget is already handed out to the arena and workspace, inside a serving loop that cannot
 * afford the device-wide synchronisation an allocation or free may cause, or under a framework whose memory
 * pool they are not allowed to touch.  Same computation and arguments as tgp_k_attn() with q_len = 1, but the
 * per-tile partial results go to a fixed array of TGP_STATIC_SCRATCH_BYTES that is part of the library image
 * (every GPU that loads the library holds those 4 MiB until the process exits).  The call allocates and frees
 * nothing.  It returns TGP_E_TOO_LARGE, and launches nothing, when B * Hq * n_tiles * (Dh + 2) * 4 exceeds
 * TGP_STATIC_SCRATCH_BYTES or the device ordinal is >= TGP_STATIC_MAX_DEVICES.
 * The first call on each device looks up the array's device address (that device must be current); make that
 * first call before starting any stream capture.  All calls on a device share the one array: it keeps whatever
 * the previous call left (nothing in it needs to start at zero - every partial that is read is written first by
 * the same call), and two calls whose kernels overlap on the GPU (different streams) race on it. */
#define TGP_STATIC_SCRATCH_BYTES (4u << 20)
#define TGP_STATIC_MAX_DEVICES   64
int  tgp_k_attn_decode_static(const void *qb, void *const *k_tiles, void *const *v_tiles, uint32_t n_tiles, void *ob,
                              const tgp_model_cfg *cfg, uint32_t B, uint32_t pos0, void *stream);
/* a = bf16(silu(g) * u), g/u fp32 [M, F]. */
int  tgp_k_swiglu(const float *g32, const float *u32, void *ab, uint64_t n_elems, void *stream);
/* out[b] = argmax_j logits[b, j], lowest index on ties. */
int  tgp_k_argmax(const float *logits, int32_t *out, uint32_t B, uint32_t V, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* TGP_H */
