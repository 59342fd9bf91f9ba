// Step engine: executes the plan.  Copies run on the caller's copy stream (host -> arena) and on a
// library-owned write-back stream (arena -> host); kernels run on the caller's compute stream; CUDA
// events order the two.  No kernel ever touches a non-resident byte, so there are no demand faults.
//
// Ordering rules (per command c of the plan, per op i of the trace):
//   H2D/ALLOC c : copy stream waits done[c.wait_op] (the last op that used the bytes being overwritten)
//                 and the newest write-back, copies, then records copied[c.first_use] if c is the last
//                 placement of that op.
//   op i        : compute stream waits copied[i] (if the op has placements), runs, records done[i]
//                 if some command waits on i.
//   D2H c       : write-back stream waits done[c.wait_op], copies the tensor back, records wb.
// A command is enqueued as soon as the op it waits on has been enqueued, so the copy stream runs as far
// ahead of compute as ring space allows, across step boundaries too.
#include <cuda_runtime.h>
#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <map>
#include <vector>
#include "tgp_internal.h"
#include "tgp_kernels.h"

extern thread_local uint64_t tgpk_launches;

#define CU(ctx, call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return tgp_fail(ctx, TGP_E_CUDA, std::string(#call) + ": " + cudaGetErrorString(e_)); } while (0)

static int g_small_copy_streams = 1;     // plans of small copies use three copy streams (0: always one)
static int g_merge_copies = 1;           // adjacent small loads that need no further wait share one cudaMemcpyAsync
static int g_fuse_swiglu_epilogue = 1;   // prefill: the up projection's tensor-core epilogue applies SwiGLU (0: separate kernel)
static int g_fuse_small = 0;             // decode steps of small models: RMSNorm and SwiGLU are computed by the products that consume them (off:
                                         // 32 instead of 50 launches per step of the tiny configuration, but a span waits for all its copies, and
                                         // with a ring of two blocks copies and kernels already alternate more than they overlap: 0.56 against 0.58)

struct TgpEngine {
    // workspace carve-up
    int32_t *tok = nullptr, *amax = nullptr;
    float *x = nullptr, *q32 = nullptr, *k32 = nullptr, *v32 = nullptr, *g32 = nullptr, *u32 = nullptr, *cos_t = nullptr, *sin_t = nullptr, *scratch = nullptr;
    char *h = nullptr, *qb = nullptr, *ob = nullptr, *ab = nullptr, *hf = nullptr;
    // MoE
    int32_t *topk_idx = nullptr, *erow = nullptr, *ecount = nullptr;
    float *topk_gate = nullptr, *egate = nullptr, *y32 = nullptr, *bias_dev = nullptr;
    char *hg = nullptr, *spill = nullptr;
    int32_t *ecount_host = nullptr;                      // pinned mirror of the per-expert counts
    std::vector<uint32_t> cnt;                           // counts of the layer being executed
    int32_t cur_expert = -1;
    uint32_t max_tokens = 0;
    // run state
    std::vector<cudaEvent_t> done_ev, copied_ev;         // per op, created on first use
    cudaEvent_t wb_ev = nullptr, t0 = nullptr, t1 = nullptr;
    cudaStream_t wb_stream = nullptr;
    bool wb_pending = false;                             // a write-back was recorded since the copy stream last waited
    int32_t copy_waited_op = -1;
    // A plan made of small copies only (a pinned copy of 128 KiB moves at a third of the link rate: latency) spreads
    // its H2D commands round-robin over the caller's copy stream and two library-owned ones, so that their latencies
    // overlap; the streams meet at every op's last placement.  Large copies, and a run being captured into a graph,
    // keep the one FIFO stream.
    static constexpr int NCOPY = 3;
    cudaStream_t xcopy[NCOPY - 1] = {nullptr, nullptr};
    cudaEvent_t xmark[NCOPY] = {nullptr, nullptr, nullptr};
    uint32_t n_copy = 1, rr = 0;
    int32_t waited[NCOPY] = {-1, -1, -1};
    bool wb_pend[NCOPY] = {false, false, false};
    size_t next_cmd = 0;
    uint64_t n_dma = 0;                                   // host-to-device copies issued since the last reset (merged commands count once)
    uint32_t next_step = 0, pos = 0;
    const int32_t *tok_src = nullptr;
    int device = -1;
    // optional per-op timestamps (Section IV-E "Runtime Monitor": lightweight timestamping of kernels)
    bool op_timing = false;
    std::vector<cudaEvent_t> ta, tb_;
    uint32_t timed_op0 = 0, timed_nops = 0;
    // whole-run CUDA graph (dense models): capture state and the instantiated graph
    bool capturing = false;
    cudaStream_t cap_cs = nullptr, cap_cp = nullptr;
    cudaEvent_t fork_ev = nullptr, join_cp = nullptr, join_wb = nullptr;
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t graph_exec = nullptr;
    // activation tap (parity testing): device buffer the rounded activations are copied to, and what went where
    char *tap = nullptr; uint64_t tap_bytes = 0, tap_used = 0;
    std::vector<uint64_t> tap_index;                     // 5 words per record: op, tag, sub-index, offset, bytes
    // managed-hints variant
    bool advised = false, evict_explicit = true;
    uint64_t recent_objects[8] = {~0ull, ~0ull, ~0ull, ~0ull, ~0ull, ~0ull, ~0ull, ~0ull};      // object-level variant: last segments requested
    uint32_t recent_pos = 0;
    std::map<int32_t, std::vector<uint32_t>> evict_at;   // op -> read-only ring tensors whose planned stay ends there
};

static inline uint64_t up256(uint64_t x) { return (x + 255) / 256 * 256; }

struct WsLayout { uint64_t tok, amax, x, h, q32, k32, v32, qb, ob, g32, u32, ab, hf, cos_t, sin_t, scratch, topk_idx, topk_gate, erow, egate, ecount, hg, y32, bias, spill, total; };

static WsLayout ws_layout(const tgp_model_cfg &c, uint64_t Mx) {
    WsLayout w{};
    uint64_t o = 0;
    auto take = [&](uint64_t bytes) { uint64_t at = o; o = up256(o + bytes); return at; };
    const uint64_t qd = (uint64_t)c.Hq * c.Dh, kd = (uint64_t)c.Hkv * c.Dh;
    w.tok = take(Mx * 4); w.amax = take((uint64_t)c.B * 4);
    w.x = take(Mx * c.d * 4); w.h = take(Mx * c.d * 2);
    w.q32 = take(Mx * qd * 4); w.k32 = take(Mx * kd * 4); w.v32 = take(Mx * kd * 4);
    w.qb = take(Mx * qd * 2); w.ob = take(Mx * qd * 2);
    w.g32 = take(Mx * c.F * 4); w.u32 = take(Mx * c.F * 4); w.ab = take(Mx * c.F * 2);
    w.hf = take((uint64_t)c.B * c.d * 2);
    w.cos_t = take((uint64_t)c.max_len * (c.Dh / 2) * 4); w.sin_t = take((uint64_t)c.max_len * (c.Dh / 2) * 4);
    uint64_t sb = 0; tgp_k_attn_scratch_bytes(&c, &sb);
    w.scratch = take(sb);
    if (c.E) {
        w.topk_idx = take(Mx * 2 * 4); w.topk_gate = take(Mx * 2 * 4);
        w.erow = take((uint64_t)c.E * Mx * 4); w.egate = take((uint64_t)c.E * Mx * 4); w.ecount = take((uint64_t)c.E * 4);
        w.hg = take(Mx * c.d * 2); w.y32 = take(Mx * c.d * 4); w.bias = take((uint64_t)c.L * c.E * 4);
        w.spill = take(std::max<uint64_t>((uint64_t)c.F * c.d * 2, 512));        // one whole expert matrix: the largest block a fallback fetches
    }
    w.total = o;
    return w;
}

int tgp_rope_tables_upload(uint32_t Dh, uint32_t max_len, float base, float *cos_dev, float *sin_dev) {
    const uint32_t half = Dh / 2;
    std::vector<float> c((size_t)max_len * half), s((size_t)max_len * half);
    for (uint32_t i = 0; i < half; ++i) {
        const double inv = std::pow((double)base, -2.0 * (double)i / (double)Dh);
        for (uint32_t p = 0; p < max_len; ++p) { const double a = (double)p * inv; c[(size_t)p * half + i] = (float)std::cos(a); s[(size_t)p * half + i] = (float)std::sin(a); }
    }
    if (cudaMemcpy(cos_dev, c.data(), c.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess) return TGP_E_CUDA;
    if (cudaMemcpy(sin_dev, s.data(), s.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess) return TGP_E_CUDA;
    return TGP_OK;
}

void tgp_engine_free(tgp_ctx *ctx) {
    if (!ctx) return;
    for (TgpPool &p : ctx->pools)
        if (p.locked_by_us) { cudaHostUnregister(p.host_base); p.locked_by_us = false; }
    TgpEngine *e = ctx->eng;
    if (!e) return;
    cudaDeviceSynchronize();
    for (cudaEvent_t ev : e->done_ev) if (ev) cudaEventDestroy(ev);
    for (cudaEvent_t ev : e->copied_ev) if (ev) cudaEventDestroy(ev);
    for (cudaEvent_t ev : e->ta) if (ev) cudaEventDestroy(ev);
    for (cudaEvent_t ev : e->tb_) if (ev) cudaEventDestroy(ev);
    if (e->wb_ev) cudaEventDestroy(e->wb_ev);
    if (e->t0) cudaEventDestroy(e->t0);
    if (e->t1) cudaEventDestroy(e->t1);
    if (e->graph_exec) cudaGraphExecDestroy(e->graph_exec);
    if (e->graph) cudaGraphDestroy(e->graph);
    for (cudaEvent_t ev : {e->fork_ev, e->join_cp, e->join_wb}) if (ev) cudaEventDestroy(ev);
    for (cudaEvent_t ev : e->xmark) if (ev) cudaEventDestroy(ev);
    for (cudaStream_t xs : e->xcopy) if (xs) cudaStreamDestroy(xs);
    if (e->wb_stream) cudaStreamDestroy(e->wb_stream);
    if (e->ecount_host) cudaFreeHost(e->ecount_host);
    delete e;
    ctx->eng = nullptr;
}

extern "C" {

int tgp_k_rope_tables(uint32_t Dh, uint32_t max_len, float base, float *cos_dev, float *sin_dev) {
    if (!cos_dev || !sin_dev || Dh % 2 || !max_len) return TGP_E_INVAL;
    return tgp_rope_tables_upload(Dh, max_len, base, cos_dev, sin_dev);
}

int tgp_set_arena(tgp_ctx *ctx, void *arena_dev, uint64_t bytes) {
    if (!ctx || !arena_dev || !bytes) return TGP_E_INVAL;
    if ((uintptr_t)arena_dev % 512) return tgp_fail(ctx, TGP_E_INVAL, "arena not 512-byte aligned");
    ctx->arena = arena_dev; ctx->arena_bytes = bytes;
    return TGP_OK;
}

int tgp_model_workspace_bytes(const tgp_model_cfg *cfg, uint32_t max_tokens, uint64_t *bytes) {
    if (!cfg || !bytes || !max_tokens || !cfg->TK || !cfg->Dh) return TGP_E_INVAL;
    *bytes = ws_layout(*cfg, max_tokens).total;
    return TGP_OK;
}

int tgp_model_bind(tgp_ctx *ctx, const tgp_model_cfg *cfg, const tgp_role_entry *roles, uint32_t n_roles,
                   const float *router_bias_host, void *workspace_dev, uint64_t ws_bytes, uint32_t max_tokens) {
    if (!ctx || !cfg || !roles || !n_roles) return TGP_E_INVAL;
    const tgp_model_cfg &c = *cfg;
    if (!c.L || !c.d || !c.Hq || !c.Hkv || c.Hq % c.Hkv || !c.Dh || c.Dh % 2 || !c.V || !c.B || !c.TK || !c.max_len || c.d % 8 || c.F % 8)
        return tgp_fail(ctx, TGP_E_INVAL, "model shape");
    if ((c.max_len + c.TK - 1) / c.TK > TGP_MAX_TILES) return tgp_fail(ctx, TGP_E_TOO_LARGE, "more KV tiles per layer than a kernel can address (64)");
    if (c.E && !router_bias_host) return tgp_fail(ctx, TGP_E_INVAL, "MoE needs the router bias");
    std::vector<TgpRole> rs(n_roles);
    std::vector<int32_t> rot(ctx->tensors.size(), -1);
    for (uint32_t i = 0; i < n_roles; ++i) {
        const tgp_role_entry &r = roles[i];
        if (r.tensor >= ctx->tensors.size()) return tgp_fail(ctx, TGP_E_UNKNOWN_TENSOR, "role names an unregistered tensor");
        if (r.kind > TGP_K_VTILE || !r.rows) return tgp_fail(ctx, TGP_E_INVAL, "role entry");
        if (rot[r.tensor] >= 0) return tgp_fail(ctx, TGP_E_INVAL, "tensor bound to two roles");
        const TgpTensor &t = ctx->tensors[r.tensor];
        if (t.size % (2ull * r.rows)) return tgp_fail(ctx, TGP_E_INVAL, "tensor size is not rows x cols bf16");
        rs[i] = {r.kind, r.layer, r.expert, r.block, r.row0, r.rows, r.tensor};
        rot[r.tensor] = (int32_t)i;
    }
    ctx->cfg = c; ctx->roles.swap(rs); ctx->role_of_tensor.swap(rot);
    ctx->router_bias.assign(router_bias_host ? router_bias_host : nullptr, router_bias_host ? router_bias_host + (size_t)c.L * c.E : nullptr);
    ctx->bound = true;
    ctx->role_index.clear();
    for (uint32_t i = 0; i < n_roles; ++i) ctx->role_index[std::make_tuple(ctx->roles[i].kind, ctx->roles[i].layer, ctx->roles[i].expert)].push_back(i);
    for (auto &kv : ctx->role_index)
        std::sort(kv.second.begin(), kv.second.end(), [&](uint32_t a, uint32_t b) { return ctx->roles[a].block < ctx->roles[b].block; });
    if (!workspace_dev) return TGP_OK;
    if (!max_tokens) return TGP_E_INVAL;
    const WsLayout w = ws_layout(c, max_tokens);
    if (ws_bytes < w.total) return tgp_fail(ctx, TGP_E_INVAL, "workspace smaller than tgp_model_workspace_bytes()");
    if ((uintptr_t)workspace_dev % 256) return tgp_fail(ctx, TGP_E_INVAL, "workspace not 256-byte aligned");
    tgp_engine_free(ctx);
    TgpEngine *e = new TgpEngine();
    ctx->eng = e;
    char *b = (char *)workspace_dev;
    e->tok = (int32_t *)(b + w.tok); e->amax = (int32_t *)(b + w.amax);
    e->x = (float *)(b + w.x); e->h = b + w.h; e->q32 = (float *)(b + w.q32); e->k32 = (float *)(b + w.k32); e->v32 = (float *)(b + w.v32);
    e->qb = b + w.qb; e->ob = b + w.ob; e->g32 = (float *)(b + w.g32); e->u32 = (float *)(b + w.u32); e->ab = b + w.ab; e->hf = b + w.hf;
    e->cos_t = (float *)(b + w.cos_t); e->sin_t = (float *)(b + w.sin_t); e->scratch = (float *)(b + w.scratch);
    e->max_tokens = max_tokens;
    if (c.E) {
        e->topk_idx = (int32_t *)(b + w.topk_idx); e->topk_gate = (float *)(b + w.topk_gate); e->erow = (int32_t *)(b + w.erow);
        e->egate = (float *)(b + w.egate); e->ecount = (int32_t *)(b + w.ecount); e->hg = b + w.hg; e->y32 = (float *)(b + w.y32);
        e->bias_dev = (float *)(b + w.bias); e->spill = b + w.spill;
        CU(ctx, cudaMemcpy(e->bias_dev, ctx->router_bias.data(), (size_t)c.L * c.E * 4, cudaMemcpyHostToDevice));
        CU(ctx, cudaHostAlloc((void **)&e->ecount_host, (size_t)c.E * 4, cudaHostAllocDefault));
        e->cnt.assign(c.E, 0);
    }
    CU(ctx, cudaGetDevice(&e->device));
    for (TgpPool &p : ctx->pools) {
        if (p.flags == TGP_POOL_PLAIN && !p.locked_by_us) {
            CU(ctx, cudaHostRegister(p.host_base, p.bytes, cudaHostRegisterPortable | cudaHostRegisterMapped));
            p.locked_by_us = true;
        }
        if (p.flags == TGP_POOL_MANAGED) p.dev_alias = p.host_base;
        else { void *dp = nullptr; CU(ctx, cudaHostGetDevicePointer(&dp, p.host_base, 0)); p.dev_alias = (char *)dp; }
    }
    if (tgp_rope_tables_upload(c.Dh, c.max_len, c.rope_base, e->cos_t, e->sin_t)) return tgp_fail(ctx, TGP_E_CUDA, "rope table upload");
    CU(ctx, cudaEventCreateWithFlags(&e->wb_ev, cudaEventDisableTiming));
    CU(ctx, cudaEventCreate(&e->t0));
    CU(ctx, cudaEventCreate(&e->t1));
    CU(ctx, cudaStreamCreateWithFlags(&e->wb_stream, cudaStreamNonBlocking));
    for (cudaStream_t &xs : e->xcopy) CU(ctx, cudaStreamCreateWithFlags(&xs, cudaStreamNonBlocking));
    for (cudaEvent_t &ev : e->xmark) CU(ctx, cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
    return TGP_OK;
}

int tgp_run_reset(tgp_ctx *ctx) {
    if (!ctx || !ctx->eng) return TGP_E_STATE;
    CU(ctx, cudaDeviceSynchronize());
    TgpEngine *e = ctx->eng;
    if (ctx->base_plan.valid) {                          // the run ended on a tail plan: the whole-run plan comes back
        ctx->plan = std::move(ctx->base_plan);
        ctx->base_plan = TgpPlan();
    }
    e->next_cmd = 0; e->next_step = 0; e->pos = 0; e->wb_pending = false; e->copy_waited_op = -1; e->tok_src = nullptr;
    e->n_dma = 0;
    e->rr = 0;
    for (int i = 0; i < TgpEngine::NCOPY; ++i) { e->waited[i] = -1; e->wb_pend[i] = false; }
    {   // small-copy plans use all copy streams (decided per run: the plan may have changed)
        uint64_t biggest = 0;
        for (const TgpCmd &c : ctx->plan.cmds) if (c.kind == CMD_H2D && c.bytes > biggest) biggest = c.bytes;
        e->n_copy = (ctx->plan.valid && biggest && biggest <= (512u << 10) && g_small_copy_streams) ? TgpEngine::NCOPY : 1;
    }
    e->evict_at.clear();
    e->advised = false;                                  // the plan may have changed since the last run
    for (uint64_t &r : e->recent_objects) r = ~0ull;
    ctx->run_counts.clear();
    return TGP_OK;
}

}  // extern "C"

static int get_event(tgp_ctx *ctx, std::vector<cudaEvent_t> &v, size_t i, cudaEvent_t *out) {
    if (v.size() < ctx->ops.size()) v.resize(ctx->ops.size(), nullptr);
    if (!v[i]) CU(ctx, cudaEventCreateWithFlags(&v[i], cudaEventDisableTiming));
    *out = v[i];
    return TGP_OK;
}

// Enqueue, in plan order, every command whose wait_op has been enqueued (wait_op <= limit).
static int pump(tgp_ctx *ctx, int32_t limit, cudaStream_t copy, uint32_t *n_cmds) {
    TgpEngine *e = ctx->eng;
    const TgpPlan &pl = ctx->plan;
    while (e->next_cmd < pl.cmds.size() && pl.cmds[e->next_cmd].wait_op <= limit) {
        const TgpCmd &c = pl.cmds[e->next_cmd];
        const TgpPool &pool = ctx->pools[ctx->tensors[c.tensor].pool];
        char *dev = (char *)ctx->arena + c.arena_off;
        char *host = pool.host_base + c.pool_off;
        cudaEvent_t ev;
        if (c.kind == CMD_D2H) {
            int rc = get_event(ctx, e->done_ev, (size_t)c.wait_op, &ev);
            if (rc) return rc;
            CU(ctx, cudaStreamWaitEvent(e->wb_stream, ev, 0));
            CU(ctx, cudaMemcpyAsync(host, dev, c.bytes, cudaMemcpyDeviceToHost, e->wb_stream));
            CU(ctx, cudaEventRecord(e->wb_ev, e->wb_stream));
            e->wb_pending = true;
            for (bool &b : e->wb_pend) b = true;
        } else {
            // Placement (H2D or ALLOC).  With several copy streams (plans of small copies) this command goes to the next
            // of them, each stream keeping its own record of what it has already waited for.
            const uint32_t si = e->n_copy > 1 ? e->rr++ % e->n_copy : 0;
            cudaStream_t mine = si ? e->xcopy[si - 1] : copy;
            int32_t &waited = e->n_copy > 1 ? e->waited[si] : e->copy_waited_op;
            bool &wbp = e->n_copy > 1 ? e->wb_pend[si] : e->wb_pending;
            if (c.wait_op > waited) {
                int rc = get_event(ctx, e->done_ev, (size_t)c.wait_op, &ev);
                if (rc) return rc;
                CU(ctx, cudaStreamWaitEvent(mine, ev, 0));
                waited = c.wait_op;
            }
            if (wbp) { CU(ctx, cudaStreamWaitEvent(mine, e->wb_ev, 0)); wbp = false; }
            // Coalescing: the commands that follow are carried by the same copy when they are loads that need no further
            // wait, their pool ranges and arena slots continue this one's at the same distance (the alignment padding
            // between two sub-ranges travels along: it lies inside the earlier tensor's slot), and the whole stays small -
            // a copy of a few hundred KiB is mostly latency, while merging megabytes would only delay the first tensor.
            size_t last = e->next_cmd;
            uint64_t span_bytes = c.bytes;
            if (c.kind == CMD_H2D && g_merge_copies)
                while (last + 1 < pl.cmds.size()) {
                    const TgpCmd &d = pl.cmds[last + 1], &p = pl.cmds[last];
                    if (d.kind != CMD_H2D || d.wait_op > waited || d.wait_op > limit || ctx->tensors[d.tensor].pool != ctx->tensors[c.tensor].pool) break;
                    if (d.pool_off < p.pool_off + p.bytes || d.pool_off - p.pool_off != d.arena_off - p.arena_off || d.pool_off - (p.pool_off + p.bytes) >= 512) break;
                    if (d.pool_off + d.bytes - c.pool_off > (1u << 20)) break;
                    span_bytes = d.pool_off + d.bytes - c.pool_off;
                    ++last;
                }
            if (c.kind == CMD_H2D) CU(ctx, cudaMemcpyAsync(dev, host, span_bytes, cudaMemcpyHostToDevice, mine));
            for (size_t k = e->next_cmd; k <= last; ++k) {
                const TgpCmd &m = pl.cmds[k];
                if (pl.op_last_place[m.first_use] != (int32_t)k) continue;
                if (e->n_copy > 1) {
                    // commands are in first-use order, so everything the other streams hold is wanted by this op or an
                    // earlier one: this stream waits for what they hold now, and its event covers all of it
                    for (uint32_t sj = 0; sj < e->n_copy; ++sj) {
                        if (sj == si) continue;
                        cudaStream_t other = sj ? e->xcopy[sj - 1] : copy;
                        CU(ctx, cudaEventRecord(e->xmark[sj], other));
                        CU(ctx, cudaStreamWaitEvent(mine, e->xmark[sj], 0));
                    }
                }
                int rc = get_event(ctx, e->copied_ev, (size_t)m.first_use, &ev);
                if (rc) return rc;
                CU(ctx, cudaEventRecord(ev, mine));
            }
            if (n_cmds) *n_cmds += (uint32_t)(last - e->next_cmd);
            if (c.kind == CMD_H2D) e->n_dma += 1;
            e->next_cmd = last;
        }
        if (n_cmds) ++*n_cmds;
        ++e->next_cmd;
    }
    return TGP_OK;
}

// address of access k of op o on the device
static inline char *where(const tgp_ctx *ctx, const TgpOp &o, uint32_t k) {
    const tgp_access &a = ctx->acc[o.acc0 + k];
    const TgpTensor &t = ctx->tensors[a.tensor];
    if (ctx->variant != TGP_VAR_EXPLICIT_RING) return ctx->pools[t.pool].dev_alias + t.off;
    const uint64_t w = ctx->plan.acc_where[o.acc0 + k];
    return w == UINT64_MAX ? ctx->pools[t.pool].dev_alias + t.off : (char *)ctx->arena + w;
}

// ---- managed-hints variant (the paper's mechanism, Section IV-E: cudaMemPrefetchAsync at tensor granularity and
// cudaMemAdvise for resident tensors) driven by the same plan as the ring --------------------------------------------
// advice, once per run: pins prefer the device; in-place (zero-copy) tensors stay on the host, mapped into the GPU.
// (Read-mostly duplication of the weights was measured slower here than plain migration with explicit eviction.)
static int advise_once(tgp_ctx *ctx) {
    TgpEngine *e = ctx->eng;
    if (e->advised) return TGP_OK;
    const TgpPlan &pl = ctx->plan;
    for (size_t t = 0; t < ctx->tensors.size(); ++t) {
        const TgpTensor &tt = ctx->tensors[t];
        char *p = ctx->pools[tt.pool].host_base + tt.off;
        if (pl.zc[t]) {
            CU(ctx, cudaMemAdvise(p, tt.size, cudaMemAdviseSetPreferredLocation, cudaCpuDeviceId));
            CU(ctx, cudaMemAdvise(p, tt.size, cudaMemAdviseSetAccessedBy, e->device));
        } else {
            CU(ctx, cudaMemAdvise(p, tt.size, cudaMemAdviseUnsetPreferredLocation, e->device));   // advice of an earlier plan
        }
    }
    for (auto &pin : pl.pins) {
        const TgpTensor &tt = ctx->tensors[pin.first];
        CU(ctx, cudaMemAdvise(ctx->pools[tt.pool].host_base + tt.off, tt.size, cudaMemAdviseSetPreferredLocation, e->device));
    }
    e->advised = true;
    return TGP_OK;
}

// Same walk as pump(): a planned H2D becomes a prefetch to the device on the copy stream (after the op that frees its
// room), a planned write-back becomes a prefetch home; the stay's tensor is queued for eviction at its release op.
static int pump_managed(tgp_ctx *ctx, int32_t limit, cudaStream_t copy, uint32_t *n_cmds) {
    TgpEngine *e = ctx->eng;
    const TgpPlan &pl = ctx->plan;
    while (e->next_cmd < pl.cmds.size() && pl.cmds[e->next_cmd].wait_op <= limit) {
        const TgpCmd &c = pl.cmds[e->next_cmd];
        const TgpTensor &tt = ctx->tensors[c.tensor];
        char *p = ctx->pools[tt.pool].host_base + tt.off;
        cudaEvent_t ev;
        if (c.kind == CMD_D2H) {
            int rc = get_event(ctx, e->done_ev, (size_t)c.wait_op, &ev);
            if (rc) return rc;
            CU(ctx, cudaStreamWaitEvent(e->wb_stream, ev, 0));
            CU(ctx, cudaMemPrefetchAsync(p, c.bytes, cudaCpuDeviceId, e->wb_stream));
            CU(ctx, cudaEventRecord(e->wb_ev, e->wb_stream));
            e->wb_pending = true;
        } else {
            if (c.wait_op > e->copy_waited_op) {
                int rc = get_event(ctx, e->done_ev, (size_t)c.wait_op, &ev);
                if (rc) return rc;
                CU(ctx, cudaStreamWaitEvent(copy, ev, 0));
                e->copy_waited_op = c.wait_op;
            }
            if (e->wb_pending) { CU(ctx, cudaStreamWaitEvent(copy, e->wb_ev, 0)); e->wb_pending = false; }
            if (c.kind == CMD_H2D) CU(ctx, cudaMemPrefetchAsync(p, c.bytes, e->device, copy));
            if (pl.op_last_place[c.first_use] == (int32_t)e->next_cmd) {
                int rc = get_event(ctx, e->copied_ev, (size_t)c.first_use, &ev);
                if (rc) return rc;
                CU(ctx, cudaEventRecord(ev, copy));
            }
            if (c.arena_off >= pl.ring_base && tt.flags == TGP_T_READONLY && e->evict_explicit) e->evict_at[c.release_after].push_back(c.tensor);
        }
        if (n_cmds) ++*n_cmds;
        ++e->next_cmd;
    }
    return TGP_OK;
}

// Object-level prefetch (the strawman of Section III-B): before op i runs, every whole segment of the pool that one of
// its tensors overlaps is requested on the copy stream.  No events: a kernel that gets there first faults the pages
// in itself, as under any managed-memory prefetcher.  A segment requested among the last eight is not requested again.
static int prefetch_objects(tgp_ctx *ctx, uint32_t i, cudaStream_t copy, uint64_t *bytes) {
    TgpEngine *e = ctx->eng;
    const TgpOp &o = ctx->ops[i];
    const uint64_t seg = ctx->object_bytes;
    for (uint32_t k = 0; k < o.nacc; ++k) {
        const TgpTensor &tt = ctx->tensors[ctx->acc[o.acc0 + k].tensor];
        const TgpPool &p = ctx->pools[tt.pool];
        for (uint64_t sgm = tt.off / seg; sgm <= (tt.off + tt.size - 1) / seg; ++sgm) {
            const uint64_t key = ((uint64_t)tt.pool << 48) | sgm;
            bool recent = false;
            for (uint64_t r : e->recent_objects) recent |= r == key;
            if (recent) continue;
            const uint64_t lo = sgm * seg, len = std::min(seg, p.bytes - lo);
            CU(ctx, cudaMemPrefetchAsync(p.host_base + lo, len, e->device, copy));
            e->recent_objects[e->recent_pos++ % 8] = key;
            *bytes += len;
        }
    }
    return TGP_OK;
}

// after op i: record its completion if anything waits on it, and send home the read-only tensors released there
static int after_op_managed(tgp_ctx *ctx, uint32_t i, cudaStream_t cs) {
    TgpEngine *e = ctx->eng;
    auto it = e->evict_at.find((int32_t)i);
    const bool evict = it != e->evict_at.end();
    if (!ctx->plan.op_is_wait_target[i] && !evict) return TGP_OK;
    cudaEvent_t ev;
    int rc = get_event(ctx, e->done_ev, i, &ev);
    if (rc) return rc;
    CU(ctx, cudaEventRecord(ev, cs));
    if (evict) {
        CU(ctx, cudaStreamWaitEvent(e->wb_stream, ev, 0));
        for (uint32_t t : it->second) {
            const TgpTensor &tt = ctx->tensors[t];
            CU(ctx, cudaMemPrefetchAsync(ctx->pools[tt.pool].host_base + tt.off, tt.size, cudaCpuDeviceId, e->wb_stream));
        }
        CU(ctx, cudaEventRecord(e->wb_ev, e->wb_stream));
        e->wb_pending = true;
        e->evict_at.erase(it);
    }
    return TGP_OK;
}

// One weight block of expert r.expert applied to the rows routed to it.  Gate/up read the gathered rows of h,
// down writes y32 and, with its last block, the gate-scaled rows are added into the residual stream.
static int run_expert_block(tgp_ctx *ctx, const TgpRole &r, const void *W, uint32_t K, cudaStream_t cs) {
    TgpEngine *e = ctx->eng;
    const tgp_model_cfg &c = ctx->cfg;
    const uint32_t me = e->cnt[r.expert];
    if (!me) return TGP_OK;                                // traced but not routed to in this run: nothing to compute
    const int32_t *rows = e->erow + (size_t)r.expert * e->max_tokens;
    const float *gates = e->egate + (size_t)r.expert * e->max_tokens;
    int rc = TGP_OK;
    switch (r.kind) {
    case TGP_K_WG:
        if (r.row0 == 0 && (rc = tgpk_gather_rows(e->h, rows, e->hg, me, c.d, cs))) return rc;
        return tgpk_gemm(e->hg, W, e->g32, me, r.rows, K, c.F, r.row0, 0, cs);
    case TGP_K_WU:
        return tgpk_gemm(e->hg, W, e->u32, me, r.rows, K, c.F, r.row0, 0, cs);
    case TGP_K_WD:
        if ((rc = tgpk_gemm(e->ab, W, e->y32, me, r.rows, K, c.d, r.row0, 0, cs))) return rc;
        if (r.row0 + r.rows == c.d) rc = tgpk_scatter_add(e->x, e->y32, rows, gates, me, c.d, cs);
        return rc;
    default:
        return TGP_E_MISMATCH;
    }
}

// An expert the router chose but the trace does not list (Section IV-D: identity mismatch -> no prefetch for it):
// its blocks are fetched one at a time into the spill buffer on the compute stream and used at once.
static int run_expert_fallback(tgp_ctx *ctx, int32_t layer, int32_t expert, cudaStream_t cs) {
    TgpEngine *e = ctx->eng;
    const tgp_model_cfg &c = ctx->cfg;
    const uint32_t kinds[3] = {TGP_K_WG, TGP_K_WU, TGP_K_WD};
    for (uint32_t kind : kinds) {
        auto it = ctx->role_index.find(std::make_tuple(kind, layer, expert));
        if (it == ctx->role_index.end()) return TGP_E_MISMATCH;
        if (kind == TGP_K_WD) { int rc = tgpk_swiglu(e->g32, e->u32, e->ab, (uint64_t)e->cnt[expert] * c.F, cs); if (rc) return rc; }
        for (uint32_t ri : it->second) {
            const TgpRole &r = ctx->roles[ri];
            const TgpTensor &t = ctx->tensors[r.tensor];
            if (t.size > std::max<uint64_t>((uint64_t)c.F * c.d * 2, 512)) return TGP_E_TOO_LARGE;
            const char *src = ctx->pools[t.pool].host_base + t.off;
            if (cudaMemcpyAsync(e->spill, src, t.size, ctx->pools[t.pool].flags == TGP_POOL_MANAGED ? cudaMemcpyDefault : cudaMemcpyHostToDevice, cs) != cudaSuccess) return TGP_E_CUDA;
            int rc = run_expert_block(ctx, r, e->spill, (uint32_t)(t.size / (2ull * r.rows)), cs);
            if (rc) return rc;
        }
    }
    return TGP_OK;
}

// Model role of access k of op o, or nullptr when the op has no such access or its tensor was never bound to a role
// (a trace recorded by hand through tgp_trace_op(), a tensor registered after tgp_model_bind()).
static inline const TgpRole *role_of(const tgp_ctx *ctx, const TgpOp &o, uint32_t k) {
    if (k >= o.nacc) return nullptr;
    const uint32_t t = ctx->acc[o.acc0 + k].tensor;
    if (t >= ctx->role_of_tensor.size()) return nullptr;
    const int32_t ri = ctx->role_of_tensor[t];
    return ri < 0 ? nullptr : &ctx->roles[ri];
}

// What a dense weight block is multiplied with and where its product goes: activations, output (row stride ldc, the
// block writes columns [row0, row0 + rows)), whether it is added to the residual stream, and the activation rows.
struct GemmTarget { const void *A; float *C; uint32_t ldc, Mrows; int acc; };

static bool gemm_target(const TgpEngine *e, const tgp_model_cfg &c, const TgpRole &r, uint32_t M, uint32_t B, float *logits_dev, GemmTarget *t) {
    const uint32_t qd = c.Hq * c.Dh, kd = c.Hkv * c.Dh;
    if (r.expert >= 0) {                                  // expert block: the gathered rows of the tokens routed to it (see run_expert_block)
        if ((uint32_t)r.expert >= c.E) return false;
        const uint32_t me = e->cnt[r.expert];
        switch (r.kind) {
        case TGP_K_WG: *t = {e->hg, e->g32, c.F, me, 0}; return true;
        case TGP_K_WU: *t = {e->hg, e->u32, c.F, me, 0}; return true;
        case TGP_K_WD: *t = {e->ab, e->y32, c.d, me, 0}; return true;
        default: return false;
        }
    }
    switch (r.kind) {
    case TGP_K_WQ: *t = {e->h, e->q32, qd, M, 0}; return true;
    case TGP_K_WK: *t = {e->h, e->k32, kd, M, 0}; return true;
    case TGP_K_WV: *t = {e->h, e->v32, kd, M, 0}; return true;
    case TGP_K_WO: *t = {e->ob, e->x, c.d, M, 1}; return true;
    case TGP_K_WG: *t = {e->h, e->g32, c.F, M, 0}; return true;
    case TGP_K_WU: *t = {e->h, e->u32, c.F, M, 0}; return true;
    case TGP_K_WD: *t = {e->ab, e->x, c.d, M, 1}; return true;
    case TGP_K_LM: *t = {e->hf, logits_dev, c.V, B, 0}; return true;
    default: return false;
    }
}

extern "C" int tgp_step(tgp_ctx *ctx, uint32_t step_kind, const int32_t *tokens_host, uint32_t B, uint32_t q_len,
                        float *logits_dev, int32_t *argmax_dev, void *compute_stream, void *copy_stream, tgp_step_stats *stats) {
    if (!ctx || !logits_dev) return TGP_E_INVAL;
    if (!ctx->plan.valid) return TGP_E_NO_PLAN;
    // host tokens are checked before anything is enqueued: an id outside the vocabulary would make the embedding gather
    // read past its table (the device kernel zeroes such a row and records it, but a caller's mistake is reported here)
    if (tokens_host && ctx->bound)
        for (uint64_t i = 0, n = (uint64_t)B * q_len; i < n; ++i)
            if (tokens_host[i] < 0 || (uint32_t)tokens_host[i] >= ctx->cfg.V)
                return tgp_fail(ctx, TGP_E_INVAL, "token id outside the vocabulary at index " + std::to_string(i));
    TgpEngine *e = ctx->eng;
    if (!e || !ctx->bound) return tgp_fail(ctx, TGP_E_STATE, "no model bound with a workspace");
    const bool ring = ctx->variant == TGP_VAR_EXPLICIT_RING;
    if (ring && (!ctx->arena || ctx->arena_bytes < ctx->budget)) return tgp_fail(ctx, TGP_E_STATE, "arena missing or smaller than the budget");
    if (!ring)
        for (const TgpPool &p : ctx->pools) if (p.flags != TGP_POOL_MANAGED) return tgp_fail(ctx, TGP_E_STATE, "managed variants need a managed pool");
    if (e->next_step >= ctx->steps.size()) return tgp_fail(ctx, TGP_E_STATE, "the plan has no further step; call tgp_run_reset()");
    const TgpStep &st = ctx->steps[e->next_step];
    const tgp_model_cfg &c = ctx->cfg;
    if (st.kind != step_kind || B != c.B || !q_len || (step_kind == TGP_DECODE && q_len != 1)) return tgp_fail(ctx, TGP_E_INVAL, "step kind, batch or q_len differ from the plan");
    if ((uint64_t)B * q_len > e->max_tokens || e->pos + q_len > c.max_len) return tgp_fail(ctx, TGP_E_INVAL, "more tokens than the workspace or max_len allow");
    if (!tokens_host && (step_kind != TGP_DECODE || e->next_step == 0)) return tgp_fail(ctx, TGP_E_INVAL, "tokens are required for this step");
    if (e->capturing && (stats || e->op_timing || e->tap || compute_stream != (void *)e->cap_cs || copy_stream != (void *)e->cap_cp))
        return tgp_fail(ctx, TGP_E_STATE, "while a run is being captured: no statistics, timing or tap, and the streams given to tgp_run_capture_begin()");
    cudaStream_t cs = (cudaStream_t)compute_stream, cp = (cudaStream_t)copy_stream;
    const uint32_t M = B * q_len, pos0 = e->pos;
    const uint64_t launches0 = tgpk_launches;
    // every kernel of the step is launched from here on the compute stream: consecutive products over the same activations
    // may read them before their predecessor has finished
    struct ChainScope { bool was; ChainScope() : was(tgpk_chain_ok) { tgpk_chain_ok = true; } ~ChainScope() { tgpk_chain_ok = was; } } chain_scope;
    uint32_t n_cmds = 0, n_mismatch = 0;
    e->cur_expert = -1;
    if (stats) CU(ctx, cudaEventRecord(e->t0, cs));
    const int32_t *tok = e->amax;
    if (tokens_host) { CU(ctx, cudaMemcpyAsync(e->tok, tokens_host, (size_t)M * 4, cudaMemcpyHostToDevice, cs)); tok = e->tok; }
    int rc;
    const bool hints = ctx->variant == TGP_VAR_MANAGED_HINTS, objects = ctx->variant == TGP_VAR_MANAGED_OBJECT;
    uint64_t object_bytes_asked = 0;
    if (hints && (rc = advise_once(ctx))) return rc;
    if (objects && (rc = prefetch_objects(ctx, st.op0, cp, &object_bytes_asked))) return rc;
    if (ring && (rc = pump(ctx, (int32_t)st.op0 - 1, cp, &n_cmds))) return rc;
    if (hints && (rc = pump_managed(ctx, (int32_t)st.op0 - 1, cp, &n_cmds))) return rc;
    const uint32_t qd = c.Hq * c.Dh;
    int32_t glu_fused_layer = -1;                            // layer whose SwiGLU was applied by its up projection's epilogue
    for (uint32_t i = st.op0; i < st.op0 + st.nops; ++i) {
        const TgpOp &o = ctx->ops[i];
        // Consecutive weight-block products of a decode step that read the same activations (the q, k and v projections, gate
        // and up, the pieces one large matrix is registered as) run as one launch when the kernels say they may share one
        // and their copies have all been enqueued already: a block of few rows alone leaves most SMs without work.
        uint32_t span = 1, gK = 0, gn[TGP_GEMM_GROUP_MAX], gld[TGP_GEMM_GROUP_MAX];
        float *gC[TGP_GEMM_GROUP_MAX];
        GemmTarget g0 = {};
        int32_t g_expert = -1;
        bool g_gather = false, g_scatter = false;
        uint32_t gbase = i;                                  // first product of the span (after a fused norm / SwiGLU op: i + 1)
        int fuse = 0;                                        // 1: op i is an RMSNorm computed by its consumers; 2: a SwiGLU computed by its consumers
        // products from op `base` on that may share a launch: same layer, activations, accumulation, K and group key
        auto form_group = [&](uint32_t base, uint32_t *key_out) -> uint32_t {
            uint32_t cnt = 0, key0 = 0;
            for (uint32_t j = 0; j < TGP_GEMM_GROUP_MAX && base + j < st.op0 + st.nops; ++j) {
                const TgpOp &f = ctx->ops[base + j];
                if (f.kind != TGP_OP_GEMM || f.layer != ctx->ops[base].layer || !f.nacc) break;
                const TgpRole *rp = role_of(ctx, f, 0);
                if (!rp) break;
                const TgpRole &r = *rp;
                GemmTarget t;
                if (!r.rows || !gemm_target(e, c, r, M, B, logits_dev, &t) || !t.Mrows || t.Mrows > 32) break;
                const uint32_t Kj = (uint32_t)(ctx->tensors[ctx->acc[f.acc0].tensor].size / (2ull * r.rows));
                const uint32_t key = tgpk_gemm_group_key(t.Mrows, r.rows, Kj);
                if (!key) break;
                if (j == 0) { g0 = t; gK = Kj; key0 = key; g_expert = r.expert; }
                else if (t.A != g0.A || t.acc != g0.acc || t.Mrows != g0.Mrows || Kj != gK || key != key0 || r.expert != g_expert) break;
                if (ctx->plan.op_last_place[base + j] >= 0 && (size_t)ctx->plan.op_last_place[base + j] >= e->next_cmd) break;   // its copy is not enqueued yet
                gC[j] = t.C + r.row0; gn[j] = r.rows; gld[j] = t.ldc;
                cnt = j + 1;
            }
            if (key_out) *key_out = key0;
            return cnt;
        };
        if (ring && o.kind == TGP_OP_GEMM && !e->tap) {
            uint32_t cnt = form_group(i, nullptr);
            // A grouped launch keeps the ring slots of its first blocks until its last block has arrived and the launch has
            // run, and the copies that wait for those slots start that much later: the link idles.  So a block whose slot a
            // later copy waits for ends its group (pinned blocks, which nothing waits for, group freely).
            for (uint32_t j = 0; j + 1 < cnt; ++j)
                if (ctx->plan.op_is_wait_target[i + j]) { cnt = j + 1; break; }
            if (cnt >= 2) span = cnt;
            for (uint32_t j = 0; j < span && span > 1 && g_expert >= 0; ++j) {       // what run_expert_block does around an expert's products
                const TgpRole &r = *role_of(ctx, ctx->ops[i + j], 0);
                g_gather |= r.kind == TGP_K_WG && r.row0 == 0;
                g_scatter |= r.kind == TGP_K_WD && r.row0 + r.rows == c.d;
            }
        } else if (ring && g_fuse_small && !e->tap && !c.E && q_len == 1 && M <= 2 && (o.kind == TGP_OP_RMSNORM || o.kind == TGP_OP_SWIGLU) &&
                   i + 1 < st.op0 + st.nops && (ctx->plan.op_last_place[i] < 0 || (size_t)ctx->plan.op_last_place[i] < e->next_cmd)) {
            // Launch-bound decode steps of small models (one or two sequences, rows of at most 1024 elements): the products
            // that consume a normalised state or a SwiGLU output compute it themselves, bit for bit as the separate kernel
            // would have (every warp redoes a row of a few hundred elements), and the op's own launch disappears.  The span
            // is the op and the products after it that may share a launch; all wait for all placements, as a group does.
            const TgpRole *np = o.kind == TGP_OP_RMSNORM ? role_of(ctx, o, 0) : nullptr;
            uint32_t key = 0;
            const uint32_t cnt = form_group(i + 1, &key);
            const void *want_A = o.kind == TGP_OP_SWIGLU ? (const void *)e->ab : (np && np->kind == TGP_K_GF) ? (const void *)e->hf : (const void *)e->h;
            const bool norm_ok = o.kind == TGP_OP_RMSNORM && np && gK == c.d && c.d <= 1024;
            const bool glu_ok = o.kind == TGP_OP_SWIGLU && gK == c.F && c.F <= 1024;
            if (cnt >= 1 && g0.A == want_A && g0.Mrows <= 2 && key == g0.Mrows && g_expert < 0 && (norm_ok || glu_ok)) {
                // ... and nothing else reads the state the op would have written: the products after the span are another op's
                bool later_reader = false;
                for (uint32_t j = i + 1 + cnt; j < st.op0 + st.nops && !later_reader; ++j) {
                    const TgpOp &f = ctx->ops[j];
                    if (f.kind == o.kind) break;                                   // the state is rewritten here
                    if (f.kind != TGP_OP_GEMM) continue;
                    const TgpRole *rp = role_of(ctx, f, 0);
                    GemmTarget t;
                    if (rp && gemm_target(e, c, *rp, M, B, logits_dev, &t) && t.A == want_A) later_reader = true;
                }
                if (!later_reader) { fuse = o.kind == TGP_OP_RMSNORM ? 1 : 2; span = 1 + cnt; gbase = i + 1; }
            }
        }
        for (uint32_t j = i; j < i + span; ++j)
            if ((ring || hints) && ctx->plan.op_last_place[j] >= 0) {
                if ((size_t)ctx->plan.op_last_place[j] >= e->next_cmd) return tgp_fail(ctx, TGP_E_STATE, "a placement was not enqueued before its op");
                cudaEvent_t ev;
                if ((rc = get_event(ctx, e->copied_ev, j, &ev))) return rc;
                CU(ctx, cudaStreamWaitEvent(cs, ev, 0));
            }
        const uint32_t ti = i - st.op0;
        if (e->op_timing) {
            if (e->ta.size() < ti + span) { e->ta.resize(ti + span, nullptr); e->tb_.resize(ti + span, nullptr); }
            for (uint32_t j = ti; j < ti + span; ++j)
                if (!e->ta[j]) { CU(ctx, cudaEventCreate(&e->ta[j])); CU(ctx, cudaEventCreate(&e->tb_[j])); }
            CU(ctx, cudaEventRecord(e->ta[ti], cs));
        }
        rc = TGP_OK;
        switch (o.kind) {
        case TGP_OP_EMBED:
            if (!o.nacc) return tgp_fail(ctx, TGP_E_MISMATCH, "embedding op without a table");
            rc = tgpk_embed(where(ctx, o, 0), tok, e->x, M, c.d, c.V, cs);
            break;
        case TGP_OP_RMSNORM: {
            const TgpRole *rp = role_of(ctx, o, 0);
            if (!rp || (rp->kind != TGP_K_G1 && rp->kind != TGP_K_G2 && rp->kind != TGP_K_GF)) return tgp_fail(ctx, TGP_E_MISMATCH, "norm op on a tensor that is not a bound gain");
            const TgpRole &r = *rp;
            if (fuse == 1) {
                const void *gW[TGP_GEMM_GROUP_MAX];
                for (uint32_t j = 0; j + 1 < span; ++j) gW[j] = where(ctx, ctx->ops[gbase + j], 0);
                const bool fin = r.kind == TGP_K_GF;
                rc = tgpk_gemm_group_fused(1, fin ? e->x + (size_t)(q_len - 1) * c.d : e->x, fin ? q_len * c.d : c.d, where(ctx, o, 0), c.eps, nullptr, nullptr,
                                           span - 1, gW, gC, gn, gld, g0.Mrows, gK, g0.acc, cs);
                break;
            }
            if (r.kind == TGP_K_GF) rc = tgpk_rmsnorm(e->x + (size_t)(q_len - 1) * c.d, q_len * c.d, where(ctx, o, 0), e->hf, B, c.d, c.eps, cs);
            else rc = tgpk_rmsnorm(e->x, c.d, where(ctx, o, 0), e->h, M, c.d, c.eps, cs);
            break;
        }
        case TGP_OP_GEMM: {
            const TgpRole *rp = role_of(ctx, o, 0);
            if (!rp || !rp->rows) return tgp_fail(ctx, TGP_E_MISMATCH, "GEMM op on a tensor with no model role");
            const tgp_access &a = ctx->acc[o.acc0];
            const TgpRole &r = *rp;
            const uint32_t K = (uint32_t)(ctx->tensors[a.tensor].size / (2ull * r.rows));
            const void *W = where(ctx, o, 0);
            if (span > 1) {
                const void *gW[TGP_GEMM_GROUP_MAX];
                for (uint32_t j = 0; j < span; ++j) gW[j] = where(ctx, ctx->ops[i + j], 0);
                if (g_expert >= 0) {
                    e->cur_expert = g_expert;
                    const int32_t *rows = e->erow + (size_t)g_expert * e->max_tokens;
                    if (g_gather && (rc = tgpk_gather_rows(e->h, rows, e->hg, g0.Mrows, c.d, cs))) break;
                    if ((rc = tgpk_gemm_group(g0.A, span, gW, gC, gn, gld, g0.Mrows, gK, 0, cs))) break;
                    if (g_scatter) rc = tgpk_scatter_add(e->x, e->y32, rows, e->egate + (size_t)g_expert * e->max_tokens, g0.Mrows, c.d, cs);
                    break;
                }
                rc = tgpk_gemm_group(g0.A, span, gW, gC, gn, gld, g0.Mrows, gK, g0.acc, cs);
                break;
            }
            if (r.expert >= 0) {                          // expert weight block: rows of the tokens routed to that expert
                if ((uint32_t)r.expert >= c.E || !c.E) return tgp_fail(ctx, TGP_E_MISMATCH, "expert weight in a dense model");
                e->cur_expert = r.expert;
                rc = run_expert_block(ctx, r, W, K, cs);
                break;
            }
            GemmTarget t;
            if (!gemm_target(e, c, r, M, B, logits_dev, &t)) return tgp_fail(ctx, TGP_E_MISMATCH, "GEMM op on a tensor that is not a weight");
            if (r.kind == TGP_K_WU && g_fuse_swiglu_epilogue && tgpk_swiglu_fusable(t.Mrows)) {
                // prefill: the gate projection of these rows is complete (its blocks come first), so the up projection's
                // epilogue applies SwiGLU itself and stores bf16 a; the step's SwiGLU op then has nothing left to do
                rc = tgpk_gemm_tc(t.A, W, t.C, t.Mrows, r.rows, K, t.ldc, r.row0, 0, cs, e->g32, e->ab);
                glu_fused_layer = o.layer;
                break;
            }
            rc = tgpk_gemm(t.A, W, t.C, t.Mrows, r.rows, K, t.ldc, r.row0, t.acc, cs);
            break;
        }
        case TGP_OP_ROUTER: {
            if (!c.E || !o.nacc) return tgp_fail(ctx, TGP_E_MISMATCH, "router op in a dense model or without its weight");
            rc = tgpk_router(e->h, where(ctx, o, 0), e->bias_dev + (size_t)o.layer * c.E, e->topk_idx, e->topk_gate, e->erow, e->egate, e->ecount,
                             M, e->max_tokens, c.d, c.E, c.topk, cs);
            if (rc) break;
            // the host needs the counts to size the expert launches (and to detect experts the trace does not list)
            CU(ctx, cudaMemcpyAsync(e->ecount_host, e->ecount, (size_t)c.E * 4, cudaMemcpyDeviceToHost, cs));
            CU(ctx, cudaStreamSynchronize(cs));
            std::vector<uint8_t> traced(c.E, 0);
            for (uint32_t j = i + 1; j < st.op0 + st.nops && ctx->ops[j].layer == o.layer; ++j) {
                const TgpOp &f = ctx->ops[j];
                if (f.kind != TGP_OP_GEMM) { if (f.kind == TGP_OP_SWIGLU) continue; break; }
                const TgpRole *fr = role_of(ctx, f, 0);
                if (fr && fr->expert >= 0 && (uint32_t)fr->expert < c.E) traced[fr->expert] = 1;
            }
            const size_t slot = ((size_t)e->next_step * c.L + o.layer) * c.E;
            if (ctx->run_counts.size() < slot + c.E) ctx->run_counts.resize(slot + c.E, 0);
            for (uint32_t x = 0; x < c.E; ++x) {
                e->cnt[x] = (uint32_t)e->ecount_host[x];
                ctx->run_counts[slot + x] = e->cnt[x];
                if (e->cnt[x] && !traced[x]) {            // run-time access the trace does not have: fetch synchronously, count it
                    if ((rc = run_expert_fallback(ctx, o.layer, (int32_t)x, cs))) return tgp_fail(ctx, rc, "expert fallback failed");
                    ++n_mismatch;
                }
            }
            break;
        }
        case TGP_OP_ROPE_KV:
        case TGP_OP_ATTN: {
            TgpTilePtrs tp;
            memset(&tp, 0, sizeof(tp));
            uint32_t nt = 0;
            for (uint32_t k = 0; k < o.nacc; ++k) {
                const TgpRole *rp = role_of(ctx, o, k);
                if (!rp || (rp->kind != TGP_K_KTILE && rp->kind != TGP_K_VTILE)) return tgp_fail(ctx, TGP_E_MISMATCH, "attention op on a tensor that is not a bound KV tile");
                const TgpRole &r = *rp;
                if (r.block >= TGP_MAX_TILES) return tgp_fail(ctx, TGP_E_TOO_LARGE, "KV tile index");
                (r.kind == TGP_K_KTILE ? tp.k : tp.v)[r.block] = where(ctx, o, k);
                nt = std::max(nt, r.block + 1);
            }
            {   // every tile the kernel will address must have been listed by the op (an append touches the tiles of the new
                // positions, attention every tile below the cached length)
                const uint32_t t_lo = o.kind == TGP_OP_ROPE_KV ? pos0 / c.TK : 0, t_hi = (pos0 + q_len - 1) / c.TK;
                for (uint32_t j = t_lo; j <= t_hi; ++j)
                    if (j >= TGP_MAX_TILES || !tp.k[j] || !tp.v[j]) return tgp_fail(ctx, TGP_E_MISMATCH, "the trace does not list a KV tile this step addresses");
            }
            if (o.kind == TGP_OP_ROPE_KV) rc = tgpk_rope_kv(e->q32, e->k32, e->v32, e->qb, tp, e->cos_t, e->sin_t, &c, B, q_len, pos0, cs);
            else rc = tgpk_attn(e->qb, tp, (c.max_len + c.TK - 1) / c.TK, e->ob, &c, B, q_len, pos0, e->scratch, cs);
            break;
        }
        case TGP_OP_SWIGLU:
            if (fuse == 2) {
                const void *gW[TGP_GEMM_GROUP_MAX];
                for (uint32_t j = 0; j + 1 < span; ++j) gW[j] = where(ctx, ctx->ops[gbase + j], 0);
                rc = tgpk_gemm_group_fused(2, nullptr, 0, nullptr, 0.f, e->g32, e->u32, span - 1, gW, gC, gn, gld, g0.Mrows, gK, g0.acc, cs);
                break;
            }
            if (!c.E && glu_fused_layer == o.layer) break;                  // done in the up projection's epilogue
            if (c.E) { if (e->cur_expert >= 0 && e->cnt[e->cur_expert]) rc = tgpk_swiglu(e->g32, e->u32, e->ab, (uint64_t)e->cnt[e->cur_expert] * c.F, cs); }
            else rc = tgpk_swiglu(e->g32, e->u32, e->ab, (uint64_t)M * c.F, cs);
            break;
        case TGP_OP_ARGMAX:
            rc = tgpk_argmax(logits_dev, e->amax, B, c.V, cs);
            if (!rc && argmax_dev) CU(ctx, cudaMemcpyAsync(argmax_dev, e->amax, (size_t)B * 4, cudaMemcpyDeviceToDevice, cs));
            break;
        default:
            return tgp_fail(ctx, TGP_E_MISMATCH, "op kind the bound model cannot run");
        }
        if (rc) return tgp_fail(ctx, rc, "kernel launch failed");
        if (e->tap) {
            auto tap_copy = [&](uint64_t tag, uint64_t sub, const void *src, uint64_t bytes) -> int {
                const uint64_t at = (e->tap_used + 255) / 256 * 256;
                if (at + bytes > e->tap_bytes) return tgp_fail(ctx, TGP_E_TOO_LARGE, "activation tap buffer is full");
                CU(ctx, cudaMemcpyAsync(e->tap + at, src, bytes, cudaMemcpyDeviceToDevice, cs));
                const uint64_t rec[5] = {i, tag, sub, at, bytes};
                e->tap_index.insert(e->tap_index.end(), rec, rec + 5);
                e->tap_used = at + bytes;
                return TGP_OK;
            };
            int trc = TGP_OK;
            if (o.kind == TGP_OP_RMSNORM) {
                const bool fin = role_of(ctx, o, 0)->kind == TGP_K_GF;
                trc = fin ? tap_copy(TGP_TAP_HF, 0, e->hf, (uint64_t)B * c.d * 2) : tap_copy(TGP_TAP_H, 0, e->h, (uint64_t)M * c.d * 2);
            } else if (o.kind == TGP_OP_ROPE_KV) {
                trc = tap_copy(TGP_TAP_Q, 0, e->qb, (uint64_t)M * qd * 2);
                for (uint32_t k = 0; k < o.nacc && !trc; ++k) {
                    const TgpRole &r = *role_of(ctx, o, k);
                    trc = tap_copy(r.kind == TGP_K_KTILE ? TGP_TAP_KTILE : TGP_TAP_VTILE, r.block, where(ctx, o, k), ctx->tensors[ctx->acc[o.acc0 + k].tensor].size);
                }
            } else if (o.kind == TGP_OP_ATTN) {
                trc = tap_copy(TGP_TAP_O, 0, e->ob, (uint64_t)M * qd * 2);
            } else if (o.kind == TGP_OP_SWIGLU && !c.E) {
                trc = tap_copy(TGP_TAP_A, 0, e->ab, (uint64_t)M * c.F * 2);
            } else if (o.kind == TGP_OP_SWIGLU && e->cur_expert >= 0 && e->cnt[e->cur_expert]) {
                // mixture of experts: the rows routed to this expert, in ascending token order; the sub-index is the expert
                trc = tap_copy(TGP_TAP_A, (uint64_t)e->cur_expert, e->ab, (uint64_t)e->cnt[e->cur_expert] * c.F * 2);
            }
            if (trc) return trc;
        }
        if (e->op_timing) {                              // ops that shared a launch: its time goes to the first, the others get an empty bracket
            CU(ctx, cudaEventRecord(e->tb_[ti], cs));
            for (uint32_t j = ti + 1; j < ti + span; ++j) { CU(ctx, cudaEventRecord(e->ta[j], cs)); CU(ctx, cudaEventRecord(e->tb_[j], cs)); }
        }
        if (ring) {
            for (uint32_t j = i; j < i + span; ++j) {
                if (ctx->plan.op_is_wait_target[j]) {
                    cudaEvent_t ev;
                    if ((rc = get_event(ctx, e->done_ev, j, &ev))) return rc;
                    CU(ctx, cudaEventRecord(ev, cs));
                }
                if ((rc = pump(ctx, (int32_t)j, cp, &n_cmds))) return rc;
            }
            i += span - 1;
        } else if (hints) {
            if ((rc = after_op_managed(ctx, i, cs))) return rc;
            if ((rc = pump_managed(ctx, (int32_t)i, cp, &n_cmds))) return rc;
        } else if (objects && i + 1 < st.op0 + st.nops) {
            if ((rc = prefetch_objects(ctx, i + 1, cp, &object_bytes_asked))) return rc;
        }
    }
    e->pos += q_len;
    e->next_step++;
    if (e->op_timing) { e->timed_op0 = st.op0; e->timed_nops = st.nops; } else e->timed_nops = 0;
    if (stats) {
        CU(ctx, cudaEventRecord(e->t1, cs));
        CU(ctx, cudaEventSynchronize(e->t1));
        if (ring) CU(ctx, cudaStreamSynchronize(e->wb_stream));
        const uint64_t *tot = &ctx->plan.totals[(size_t)(e->next_step - 1) * 4];
        stats->h2d_bytes = ring ? tot[0] : objects ? object_bytes_asked : 0; stats->d2h_bytes = ring ? tot[1] : 0; stats->zc_bytes = objects ? 0 : tot[2];
        stats->n_cmds = n_cmds; stats->n_launches = (uint32_t)(tgpk_launches - launches0); stats->n_mismatch = n_mismatch;
        CU(ctx, cudaEventElapsedTime(&stats->step_ms, e->t0, e->t1));
        // the step has been waited for: a tensor-core kernel whose bounded wait ran out has left its mark
        int gemm_err = 0, attn_err = 0, bad_tok = 0;
        uint32_t bad_row = 0; int32_t bad_id = 0;
        if (tgp_k_gemm_status(&gemm_err) == TGP_OK && tgp_k_attn_status(&attn_err) == TGP_OK && (gemm_err || attn_err))
            return tgp_fail(ctx, TGP_E_CUDA, "a tensor-core kernel gave up on a bounded wait (GEMM code " + std::to_string(gemm_err) + ", attention code " + std::to_string(attn_err) + "): results of this step are incomplete");
        if (tgp_k_embed_status(&bad_tok, &bad_row, &bad_id) == TGP_OK && bad_tok)
            return tgp_fail(ctx, TGP_E_CUDA, "the embedding gather met token id " + std::to_string(bad_id) + " (row " + std::to_string(bad_row) + "), outside the vocabulary: that row was computed from zeros");
    }
    return TGP_OK;
}

// Switches to the tail plan built by tgp_replan_begin() at its step boundary.  Stays never cross a step, so after the
// device has drained the only data the arena alone holds are pinned tensors that were written: those go home, then the
// tail plan starts from an empty arena.
extern "C" int tgp_replan_commit(tgp_ctx *ctx) {
    if (!ctx || !ctx->eng) return TGP_E_STATE;
    TgpEngine *e = ctx->eng;
    if (e->capturing) return tgp_fail(ctx, TGP_E_STATE, "a run being captured cannot switch plans");
    int rc = tgp_replan_wait(ctx);
    if (rc) return rc;
    if (!ctx->tail_ready || !ctx->tail_plan.valid) return tgp_fail(ctx, TGP_E_STATE, "no re-plan to commit");
    if (e->next_step != ctx->tail_plan.first_step) return tgp_fail(ctx, TGP_E_STATE, "the run is not at the boundary the re-plan was made for");
    CU(ctx, cudaDeviceSynchronize());
    std::vector<uint8_t> written(ctx->tensors.size(), 0);
    for (uint32_t i = 0; i < ctx->tail_plan.first_op; ++i)
        for (uint32_t k = 0; k < ctx->ops[i].nacc; ++k)
            if (ctx->acc[ctx->ops[i].acc0 + k].mode & TGP_W) written[ctx->acc[ctx->ops[i].acc0 + k].tensor] = 1;
    // written pinned tensors go back to the pool - except those the tail plan keeps where they are (they hold the newest data)
    std::vector<uint8_t> kept(ctx->tensors.size(), 0);
    for (uint32_t t : ctx->tail_plan.kept) kept[t] = 1;
    for (auto &pin : ctx->plan.pins) {
        const TgpTensor &t = ctx->tensors[pin.first];
        if (t.flags == TGP_T_MUTABLE && written[pin.first] && !kept[pin.first])
            CU(ctx, cudaMemcpy(ctx->pools[t.pool].host_base + t.off, (char *)ctx->arena + pin.second, t.size, cudaMemcpyDeviceToHost));
    }
    if (!ctx->base_plan.valid) ctx->base_plan = std::move(ctx->plan);       // kept for the next tgp_run_reset()
    ctx->plan = std::move(ctx->tail_plan);
    ctx->tail_plan = TgpPlan();
    ctx->tail_ready = false;
    e->next_cmd = 0; e->wb_pending = false; e->copy_waited_op = -1; e->rr = 0;
    for (int i = 0; i < TgpEngine::NCOPY; ++i) { e->waited[i] = -1; e->wb_pend[i] = false; }
    uint64_t biggest = 0;
    for (const TgpCmd &c : ctx->plan.cmds) if (c.kind == CMD_H2D && c.bytes > biggest) biggest = c.bytes;
    e->n_copy = (biggest && biggest <= (512u << 10) && g_small_copy_streams) ? TgpEngine::NCOPY : 1;
    return TGP_OK;
}

extern "C" int tgp_k_merge_copies(int enable) {
    g_merge_copies = enable ? 1 : 0;
    return TGP_OK;
}

extern "C" int tgp_copies_issued(tgp_ctx *ctx, uint64_t *n) {
    if (!ctx || !ctx->eng || !n) return TGP_E_STATE;
    *n = ctx->eng->n_dma;
    return TGP_OK;
}

extern "C" int tgp_k_swiglu_epilogue(int enable) {
    g_fuse_swiglu_epilogue = enable ? 1 : 0;
    return TGP_OK;
}

extern "C" int tgp_k_decode_fuse(int enable) {
    g_fuse_small = enable ? 1 : 0;
    return TGP_OK;
}

extern "C" int tgp_set_op_timing(tgp_ctx *ctx, int enable) {
    if (!ctx || !ctx->eng) return TGP_E_STATE;
    ctx->eng->op_timing = enable != 0;
    return TGP_OK;
}

extern "C" int tgp_op_times(tgp_ctx *ctx, float *ms, uint32_t capacity, uint32_t *first_op, uint32_t *n_ops) {
    if (!ctx || !ctx->eng || !n_ops) return TGP_E_STATE;
    TgpEngine *e = ctx->eng;
    *n_ops = e->timed_nops;
    if (first_op) *first_op = e->timed_op0;
    if (!ms) return TGP_OK;
    if (capacity < e->timed_nops) return TGP_E_INVAL;
    for (uint32_t i = 0; i < e->timed_nops; ++i) {
        CU(ctx, cudaEventSynchronize(e->tb_[i]));
        CU(ctx, cudaEventElapsedTime(&ms[i], e->ta[i], e->tb_[i]));
    }
    return TGP_OK;
}

// ---- managed-memory helpers for the managed variants (the pool itself stays caller-owned) ----------------
extern "C" int tgp_managed_alloc(void **out, uint64_t bytes) {
    if (!out || !bytes) return TGP_E_INVAL;
    void *p = nullptr;
    if (cudaMallocManaged(&p, bytes, cudaMemAttachGlobal) != cudaSuccess) { cudaGetLastError(); return TGP_E_CUDA; }
    *out = p;
    return TGP_OK;
}

extern "C" int tgp_managed_free(void *ptr) {
    if (!ptr) return TGP_OK;
    return cudaFree(ptr) == cudaSuccess ? TGP_OK : TGP_E_CUDA;
}

// Moves a managed range back to host memory (cold start for a managed run) and waits for it.
extern "C" int tgp_managed_evict(void *ptr, uint64_t bytes) {
    if (!ptr || !bytes) return TGP_E_INVAL;
    if (cudaMemPrefetchAsync(ptr, bytes, cudaCpuDeviceId, 0) != cudaSuccess) { cudaGetLastError(); return TGP_E_CUDA; }
    return cudaDeviceSynchronize() == cudaSuccess ? TGP_OK : TGP_E_CUDA;
}

// Tokens routed to each expert in the run since the last tgp_run_reset(): [steps run, L, E] (MoE only).  This is
// the profile a first pass records so that the next trace lists exactly the experts that are used.
extern "C" int tgp_expert_counts(tgp_ctx *ctx, uint32_t *out, uint64_t *n) {
    if (!ctx || !n) return TGP_E_INVAL;
    if (out) { if (*n < ctx->run_counts.size()) return TGP_E_INVAL; memcpy(out, ctx->run_counts.data(), ctx->run_counts.size() * 4); }
    *n = ctx->run_counts.size();
    return TGP_OK;
}

extern "C" int tgp_set_tap(tgp_ctx *ctx, void *tap_dev, uint64_t bytes) {
    if (!ctx || !ctx->eng) return TGP_E_STATE;
    ctx->eng->tap = (char *)tap_dev; ctx->eng->tap_bytes = tap_dev ? bytes : 0; ctx->eng->tap_used = 0;
    ctx->eng->tap_index.clear();
    return TGP_OK;
}

extern "C" int tgp_tap_index(tgp_ctx *ctx, uint64_t *out, uint64_t *n_words) {
    if (!ctx || !ctx->eng || !n_words) return TGP_E_STATE;
    const std::vector<uint64_t> &v = ctx->eng->tap_index;
    if (out) { if (*n_words < v.size()) return TGP_E_INVAL; memcpy(out, v.data(), v.size() * 8); }
    *n_words = v.size();
    return TGP_OK;
}

// ---- whole-run CUDA graph ----------------------------------------------------------------------------------------
// A planned run of a dense model is a fixed DAG of copies and kernels over three streams (tokens come from the prompt
// and then from the device-side argmax), so it can be captured once and replayed: the host then issues one graph
// launch per pass instead of a few hundred API calls per step, which is what bounds steps of ~0.1 ms.
extern "C" int tgp_run_capture_begin(tgp_ctx *ctx, void *compute_stream, void *copy_stream) {
    if (!ctx || !ctx->eng) return TGP_E_STATE;
    TgpEngine *e = ctx->eng;
    if (!ctx->plan.valid) return TGP_E_NO_PLAN;
    if (ctx->variant != TGP_VAR_EXPLICIT_RING) return tgp_fail(ctx, TGP_E_STATE, "only the explicit engine can be captured");
    if (ctx->cfg.E) return tgp_fail(ctx, TGP_E_STATE, "an MoE step reads routing counts on the host and cannot be captured");
    if (e->capturing || e->next_step != 0 || e->next_cmd != 0) return tgp_fail(ctx, TGP_E_STATE, "call tgp_run_reset() first");
    if (e->op_timing || e->tap) return tgp_fail(ctx, TGP_E_STATE, "switch timing and tap off before capturing");
    if (!compute_stream || !copy_stream || compute_stream == copy_stream) return tgp_fail(ctx, TGP_E_INVAL, "two distinct non-default streams are required");
    if (e->graph_exec) { cudaGraphExecDestroy(e->graph_exec); e->graph_exec = nullptr; }
    if (e->graph) { cudaGraphDestroy(e->graph); e->graph = nullptr; }
    for (cudaEvent_t *ev : {&e->fork_ev, &e->join_cp, &e->join_wb})
        if (!*ev) CU(ctx, cudaEventCreateWithFlags(ev, cudaEventDisableTiming));
    // every event the run will use exists before capture starts (creation is not a stream operation)
    for (size_t i = 0; i < ctx->ops.size(); ++i) {
        cudaEvent_t ev;
        int rc;
        if (ctx->plan.op_is_wait_target[i] && (rc = get_event(ctx, e->done_ev, i, &ev))) return rc;
        if (ctx->plan.op_last_place[i] >= 0 && (rc = get_event(ctx, e->copied_ev, i, &ev))) return rc;
    }
    e->cap_cs = (cudaStream_t)compute_stream; e->cap_cp = (cudaStream_t)copy_stream;
    e->n_copy = 1;                                       // in a graph the joins of several copy branches cost more than they hide (measured: the tiny
                                                         // configuration at 512 KiB blocks replays at 0.56 / 0.52 / 0.51 of its roofline with 1 / 2 / 3 copy streams)
    CU(ctx, cudaStreamBeginCapture(e->cap_cs, cudaStreamCaptureModeRelaxed));
    // fork: the copy and write-back streams join the capture
    cudaError_t er = cudaEventRecord(e->fork_ev, e->cap_cs);
    if (er == cudaSuccess) er = cudaStreamWaitEvent(e->cap_cp, e->fork_ev, 0);
    if (er == cudaSuccess) er = cudaStreamWaitEvent(e->wb_stream, e->fork_ev, 0);
    for (uint32_t k = 1; k < e->n_copy && er == cudaSuccess; ++k) er = cudaStreamWaitEvent(e->xcopy[k - 1], e->fork_ev, 0);
    if (er != cudaSuccess) {
        cudaGraph_t g = nullptr;
        cudaStreamEndCapture(e->cap_cs, &g);
        if (g) cudaGraphDestroy(g);
        return tgp_fail(ctx, TGP_E_CUDA, std::string("capture fork: ") + cudaGetErrorString(er));
    }
    e->capturing = true;
    return TGP_OK;
}

extern "C" int tgp_run_capture_end(tgp_ctx *ctx) {
    if (!ctx || !ctx->eng || !ctx->eng->capturing) return TGP_E_STATE;
    TgpEngine *e = ctx->eng;
    e->capturing = false;
    // join: the capturing stream waits for everything the other two streams were given
    cudaError_t er = cudaEventRecord(e->join_cp, e->cap_cp);
    if (er == cudaSuccess) er = cudaEventRecord(e->join_wb, e->wb_stream);
    if (er == cudaSuccess) er = cudaStreamWaitEvent(e->cap_cs, e->join_cp, 0);
    if (er == cudaSuccess) er = cudaStreamWaitEvent(e->cap_cs, e->join_wb, 0);
    for (uint32_t k = 1; k < e->n_copy && er == cudaSuccess; ++k) {      // the library's extra copy streams, when the captured run used them
        er = cudaEventRecord(e->xmark[k], e->xcopy[k - 1]);
        if (er == cudaSuccess) er = cudaStreamWaitEvent(e->cap_cs, e->xmark[k], 0);
    }
    cudaGraph_t g = nullptr;
    cudaError_t ee = cudaStreamEndCapture(e->cap_cs, &g);
    if (er != cudaSuccess || ee != cudaSuccess || !g) {
        if (g) cudaGraphDestroy(g);
        cudaGetLastError();
        return tgp_fail(ctx, TGP_E_CUDA, std::string("capture end: ") + cudaGetErrorString(er != cudaSuccess ? er : ee));
    }
    e->graph = g;
    CU(ctx, cudaGraphInstantiate(&e->graph_exec, e->graph, 0));
    return TGP_OK;
}

extern "C" int tgp_run_graph_launch(tgp_ctx *ctx, void *stream) {
    if (!ctx || !ctx->eng || !ctx->eng->graph_exec) return TGP_E_STATE;
    CU(ctx, cudaGraphLaunch(ctx->eng->graph_exec, (cudaStream_t)stream));
    return TGP_OK;
}
